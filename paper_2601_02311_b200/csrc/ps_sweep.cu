// Fused sweep: enumerate -> evaluate -> filter -> reduce, nothing materialised.
//
// grid = (n_chunks, n_models).  A block owns one model and a contiguous range
// of its factorisations ("units"); its warps take units round-robin.  For a
// unit the warp computes the shard quantities once (all divisions), writes
// small per-mode tables to its shared-memory slice, and then walks the
// placement codes: a lane owns up to four (Theta, Omega, G) triples for the
// whole kernel (their modes and the activation digits their flags allow never
// change), keeps each triple's own bytes, communication and host bytes in
// registers and visits the activation variants and activation digits.  Because
// the activation bytes of a (variant, digit) are the same for every triple, the
// capacity test of a point is one 64-bit compare of the triple's bytes against a
// per-(variant, digit) bound; the sum is formed only for candidates.
//
// Reductions.  Every warp keeps a private sorted list in shared memory
// (Pareto staircase or top-k), tests its candidates against it lane-parallel
// and inserts the few that pass warp-cooperatively.  A warp that has run out of
// units writes its list to global scratch and is done -- the warps of a block
// never wait for one another; k_sweep_merge combines the partial lists of a
// model (one block per model: rank merge, prune) and emits entries,
// re-evaluating each emitted point from its index as a self-check.  A frontier
// that outgrows a list is handed to a slow exact path in the merge kernel.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

constexpr int LIST_CAP = SWEEP_LIST_CAP;       // entries per warp list / per partial list
constexpr u32 LIST_OVERFLOWED = 0xffffffffu;   // length of a partial list whose staircase outgrew LIST_CAP
constexpr u64 U64MAX = ~0ull;

// per-warp tables, rebuilt for every unit: what depends on the activation
// variant and digit.  (What depends on the (Theta, Omega, G) triple needs no
// table: see the per-lane coefficients in k_sweep.)
struct WarpTables {
  // per activation variant vt = (v, tau) and activation digit d
  // a triple whose own bytes are below bound[d][vt] fits the capacity with digit d
  // under variant vt (0 for variants the space does not have)
  __align__(16) u64 bound[5][4];
  // the same bounds as doubles, exact while they are below 2^53 (see the evaluation pass)
  __align__(16) double bound_f64[5][4];
  u64 act[4][5];           // activation bytes of digit d
  u64 host_bound[4];       // a triple whose own host bytes are below this may offload activations
  __align__(16) double host_bound_f64[4];   // the same as doubles (the fast case compares there)
  u64 c_axis[4];           // tensor + pipeline traffic of the variant (0 if not in the objective)
  // Pareto: for every set of digits the one with the least activation bytes
  // (lowest digit on ties), NM for the empty set
  unsigned char least[4][32];
};

struct Key {
  u64 a, b;   // Pareto: (mem, comm); top-k: (comm, mem)
  u32 i;      // index within the model
};
__device__ __forceinline__ bool key_less(const Key& x, const Key& y) {
  if (x.a != y.a) return x.a < y.a;
  if (x.b != y.b) return x.b < y.b;
  return x.i < y.i;
}

// ------------------------------------------------------------------ warp lists
struct WarpList {
  u64* a;
  u64* b;
  u32* i;
  int n;
  int over;   // Pareto: the staircase outgrew the list (the merge kernel then takes the slow exact path)
};

// Pareto staircase: a = mem ascending, b = comm strictly descending.
// A coarse staircase shared by the warps of a block: stair[j] is the least
// communication of any survivor inserted so far whose bytes fall in bucket j or
// a lower one (buckets: leading bit and the two bits after it, so a lower bucket
// means strictly fewer bytes).  A candidate in bucket B with at least
// stair[B-1] communication is strictly dominated.
constexpr int STAIR = 256;
__device__ __forceinline__ int stair_bucket(u64 m) {
  if (m < 4) return (int)m;
  const int top = 63 - __clzll((long long)m);
  return 4 * (top - 1) + (int)((m >> (top - 2)) & 3);
}
__device__ __forceinline__ void stair_publish(unsigned long long* stair, u64 m, u64 c, int lane) {
  for (int j = stair_bucket(m) + lane; j < STAIR; j += 32)
    if (stair[j] > c) atomicMin(&stair[j], (unsigned long long)c);
}

// warp-cooperative insertion; all lanes hold the same (m, c, idx).  Entries are
// handled 32 at a time, so a short staircase (the usual case) takes one round.
__device__ __noinline__ void pareto_insert(WarpList& w, u64 m, u64 c, u32 idx, int lane,
                                           unsigned long long* stair) {
  constexpr int PER = LIST_CAP / 32;
  const int rounds = (w.n + 31) >> 5;
  u64 ea[PER], eb[PER];
  u32 ei[PER];
  int below = 0, killed = 0;
  bool dominated = false;
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    if (k < rounds) {
      const int e = lane + 32 * k;
      const bool valid = e < w.n;
      ea[k] = valid ? w.a[e] : U64MAX;
      eb[k] = valid ? w.b[e] : 0;
      ei[k] = valid ? w.i[e] : 0;
      if (valid && ea[k] == m && eb[k] == c) {          // same pair: smallest index stays
        if (idx < ei[k]) w.i[e] = idx;
        dominated = true;
      } else if (valid && ea[k] <= m && eb[k] <= c) {
        dominated = true;
      }
      below += __popc(__ballot_sync(0xffffffffu, valid && ea[k] < m));
      killed += __popc(__ballot_sync(0xffffffffu, valid && ea[k] >= m && eb[k] >= c));
    }
  }
  if (__any_sync(0xffffffffu, dominated)) { __syncwarp(); return; }
  const int n_new = w.n - killed + 1;
  if (n_new > LIST_CAP) {
    w.over = 1;
    return;
  }
  __syncwarp();
  const int shift = 1 - killed;                        // entries after the killed run move by this
  if (shift != 0) {
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int e = lane + 32 * k;
      if (k < rounds && e < w.n && e >= below + killed) {
        w.a[e + shift] = ea[k];
        w.b[e + shift] = eb[k];
        w.i[e + shift] = ei[k];
      }
    }
  }
  if (lane == 0) { w.a[below] = m; w.b[below] = c; w.i[below] = idx; }
  w.n = n_new;
  stair_publish(stair, m, c, lane);
  __syncwarp();
}

// Top-k list of a warp: entries [0, n) are unordered candidates that were below
// the threshold when they arrived.  When the list is full the warp sorts it,
// keeps the k smallest and tightens the threshold to the k-th; until the first
// such compaction the threshold is "everything".  A stale threshold only lets
// extra candidates in, never keeps a wanted one out.
//
// The sort runs in registers: lane l holds entries 4l .. 4l+3, a bitonic network
// exchanges within a lane for distances below four and by shuffles above.
__device__ __forceinline__ Key key_shfl_xor(const Key& x, int lanes) {
  Key o;
  o.a = __shfl_xor_sync(0xffffffffu, x.a, lanes);
  o.b = __shfl_xor_sync(0xffffffffu, x.b, lanes);
  o.i = __shfl_xor_sync(0xffffffffu, x.i, lanes);
  return o;
}

__device__ __noinline__ void topk_compact(WarpList& w, int k_keep, int lane, Key& threshold,
                                          unsigned long long* block_comm_limit) {
  constexpr int PER = LIST_CAP / 32;
  Key e[PER];
#pragma unroll
  for (int r = 0; r < PER; ++r) {
    const int p = PER * lane + r;
    if (p < w.n) { e[r].a = w.a[p]; e[r].b = w.b[p]; e[r].i = w.i[p]; }
    else { e[r].a = U64MAX; e[r].b = U64MAX; e[r].i = 0xffffffffu; }
  }
  // the network's steps as rolled loops: this code runs rarely, so it is kept
  // small (a long unrolled sequence that is not in the instruction cache costs
  // more to fetch than to execute)
  static_assert(PER == 4, "the exchanges inside a lane are written out for four entries");
#pragma unroll 1
  for (int k = 2; k <= LIST_CAP; k <<= 1) {
#pragma unroll 1
    for (int j = k >> 1; j > 0; j >>= 1) {
      if (j >= PER) {
        const int lanes = j / PER;
        const bool lower = (lane & lanes) == 0;            // this lane holds the lower index of each pair
#pragma unroll
        for (int r = 0; r < PER; ++r) {
          const Key o = key_shfl_xor(e[r], lanes);
          const bool up = ((PER * lane + r) & k) == 0;     // ascending run
          const bool o_less = key_less(o, e[r]);
          if ((lower == up) ? o_less : !o_less) e[r] = o;   // keep the smaller / the larger of the pair
        }
      } else if (j == 2) {
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const bool up = ((PER * lane + r) & k) == 0;
          if (key_less(e[r + 2], e[r]) == up) { const Key t = e[r]; e[r] = e[r + 2]; e[r + 2] = t; }
        }
      } else {
#pragma unroll
        for (int r = 0; r < PER; r += 2) {
          const bool up = ((PER * lane + r) & k) == 0;
          if (key_less(e[r + 1], e[r]) == up) { const Key t = e[r]; e[r] = e[r + 1]; e[r + 1] = t; }
        }
      }
    }
  }
  const int n_new = min(w.n, k_keep);
  __syncwarp();
#pragma unroll
  for (int r = 0; r < PER; ++r) {
    const int p = PER * lane + r;
    if (p < n_new) { w.a[p] = e[r].a; w.b[p] = e[r].b; w.i[p] = e[r].i; }
  }
  w.n = n_new;
  __syncwarp();
  if (w.n == k_keep) {
    threshold.a = w.a[k_keep - 1]; threshold.b = w.b[k_keep - 1]; threshold.i = w.i[k_keep - 1];
    // k points with at most this much communication exist: tell the other warps
    if (lane == 0) atomicMin(block_comm_limit, (unsigned long long)threshold.a);
  }
  __syncwarp();
}

// every lane may bring one candidate
__device__ __forceinline__ void topk_append(WarpList& w, bool cand, const Key& key, int k_keep,
                                            int lane, Key& threshold,
                                            unsigned long long* block_comm_limit) {
  u32 votes = __ballot_sync(0xffffffffu, cand);
  if (votes == 0) return;
  if (w.n + __popc(votes) > LIST_CAP) {
    topk_compact(w, k_keep, lane, threshold, block_comm_limit);
    cand = cand && key_less(key, threshold);
    votes = __ballot_sync(0xffffffffu, cand);
  }
  if (cand) {
    const int p = w.n + __popc(votes & ((1u << lane) - 1u));
    w.a[p] = key.a; w.b[p] = key.b; w.i[p] = key.i;
  }
  w.n += __popc(votes);
  __syncwarp();
}

// Fast case (every degree a power of two): what depends on the model and on the
// tensor degree alone, or on the pipeline degree alone, for every possible
// degree 2^s -- built once per block, so that a unit's prologue is a few loads
// and the shifts by the remaining degrees.
constexpr int MAX_LOG2_DEGREE = 25;        // device counts are at most 2^24
struct __align__(16) TensorDegree {
  u64 E1;        // ceil(P / T): elements of a state on one tensor rank
  u64 u;         // ceil(unit / T)
  u64 EA[2];     // ceil(A[v] / T): activations under sequence parallelism
  u64 UA[2];     // ceil(UA[v] / T)
  u64 tp_x;      // ring volume of a boundary tensor over T devices
  u64 sbh_t;     // ceil(Sbh / T)
  u32 t_heads;   // T divides the head count
  u32 pad[3];
};
struct PipelineDegree {
  u32 lps;       // ceil(L / K)
  u32 k_layers;  // K divides the layer count
};

template <int WARPS>
struct SweepShared {
  WarpTables tables[WARPS];
  TensorDegree by_t[MAX_LOG2_DEGREE];
  PipelineDegree by_k[MAX_LOG2_DEGREE];
  u64 list_a[WARPS * LIST_CAP];
  u64 list_b[WARPS * LIST_CAP];
  u32 list_i[WARPS * LIST_CAP];
  u32 next_unit;
  unsigned long long block_comm_limit;   // top-k: no point with more communication can matter
  unsigned long long stair[STAIR];       // Pareto: coarse staircase of the block
  ModelRec rec;
};

// ------------------------------------------------------------------ the sweep
// a * k + acc for a 64-bit a and a small 32-bit k: two multiply-adds
__device__ __forceinline__ u64 mad_small(u64 a, u32 k, u64 acc) {
  u64 r = (u64)(u32)a * (u64)k + acc;
  r += (u64)((u32)(a >> 32) * k) << 32;
  return r;
}

// n += (m >= bound): a 64-bit subtraction whose borrow is folded into the
// counter by one more subtract-with-borrow (n - (0xffffffff + borrow) = n + 1 - borrow)
__device__ __forceinline__ void count_not_below(u32& n, u64 m, u64 bound) {
  asm("{\n\t"
      ".reg .u32 diff;\n\t"
      "sub.cc.u32 diff, %1, %3;\n\t"
      "subc.cc.u32 diff, %2, %4;\n\t"
      "subc.u32 %0, %0, 0xffffffff;\n\t"
      "}"
      : "+r"(n)
      : "r"((u32)m), "r"((u32)(m >> 32)), "r"((u32)bound), "r"((u32)(bound >> 32)));
}

// digits whose capacity compares run on the fp64 pipe when the unit's numbers are
// exact there; the other digits use the carry chain, so both pipes work
constexpr u32 F64_DIGITS = 0x1f;

// With several copies of every shard (k-way replication) a triple's communication is
// kx * x plus what reducing gradients to shards and all-reducing them cost beyond
// that: x2 per reduce-to-shards, x3 per all-reduce over all devices (both zero with
// one copy).  Needed only where the exact volume is (the reduction pass).
__device__ __forceinline__ u64 copies_traffic(u32 om, u32 gr, u32 w_grad, bool ext_in_objective, u64 x2, u64 x3) {
  const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
  u32 n2 = gr == PS_MODE_S ? 1u : 0u, n3 = gr == PS_MODE_R ? 1u : 0u;
  if (ext_in_objective) {
    if (gr == PS_MODE_SG || gr == PS_MODE_O || (gr == PS_MODE_M && on_shard)) n2 += 1;
    if (gr == PS_MODE_M && !on_shard) n3 += 1;
  }
  return (u64)w_grad * (n2 * x2 + n3 * x3);
}

// On request only (ps_filter.skip_rejected): a factorisation whose composition bits
// already miss a required flag has no survivor, so a warp need not take it.  By
// default every factorisation is taken and every point's capacity compare executed
// and then masked, so that the throughput of a sweep says how fast points are
// evaluated, not how many the filter lets the kernel jump over.
__device__ __noinline__ bool unit_rejected(const SpaceDev& sp, const ModelRec& rec, u32 unit, u32 req_cv) {
  const Fact f = sp.facts[unit];
  const bool t_heads = rec.heads % f.T == 0, k_layers = rec.L % f.K == 0, tp_le = f.T <= sp.tp_max_valid;
  const bool whole = (u64)f.T * f.K * f.D == (u64)f.N;
  u32 cv = (t_heads ? PS_F_T_DIV_HEADS : 0) | (k_layers ? PS_F_K_DIV_LAYERS : 0) | (tp_le ? PS_F_TP_LE_MAX : 0) |
           PS_F_AXIS_FORM;
  if (t_heads && k_layers && tp_le && whole) cv |= PS_F_CV;
  return (cv & req_cv) != req_cv;
}

// KIND: the reduction; NM: allowed modes; WARPS x 32 threads per block, compiled
// for MIN_BLOCKS resident blocks per SM; HOST_LIMITED: the filter has a host
// budget (without one the host bytes are never formed); FAST: every degree of
// the space is a power of two and every byte count is below 2^53 (no division
// and no 64-bit integer compare is compiled into the evaluation)
// SKIP: the kernel honours ps_filter.skip_rejected (the fast case is also compiled
// without, so that the default sweep carries no trace of it)
template <int KIND, int NM, int WARPS, int MIN_BLOCKS, bool HOST_LIMITED, bool FAST, bool SKIP>
__global__ void __launch_bounds__(WARPS * 32, MIN_BLOCKS) k_sweep(SpaceDev sp, SweepArgs args) {
  constexpr int THREADS = WARPS * 32;
  constexpr int N2 = NM * NM, N3 = NM * NM * NM, NC = N3 * NM;
  constexpr int R = (N3 + 31) / 32;                 // triples per lane
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SweepShared<WARPS>& sh = *reinterpret_cast<SweepShared<WARPS>*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // blocks are handed out in grid order: the models with the most expected work first
  const u32 model = sp.order[blockIdx.y], chunk = blockIdx.x, n_chunks = gridDim.x;

  // stage the model record with 16-byte loads (6 x 16 B)
  if (tid < (int)(sizeof(ModelRec) / 16))
    reinterpret_cast<uint4*>(&sh.rec)[tid] = reinterpret_cast<const uint4*>(&sp.recs[model])[tid];
  const u32 u_begin = (u32)(((u64)blockIdx.x * sp.n_facts) / gridDim.x);
  const u32 u_end = (u32)(((u64)(blockIdx.x + 1) * sp.n_facts) / gridDim.x);
  if (tid == 0) { sh.next_unit = u_begin + WARPS; sh.block_comm_limit = U64MAX; }
  if (KIND == PS_REDUCE_PARETO)
    for (int j = tid; j < STAIR; j += THREADS) sh.stair[j] = U64MAX;
  __syncthreads();
  const ModelRec& rec = sh.rec;
  if (FAST) {
    for (int sft = tid; sft < MAX_LOG2_DEGREE; sft += THREADS) {
      TensorDegree t;
      t.E1 = ceil_shift(rec.P, sft);
      t.u = ceil_shift(rec.unit, sft);
      t.EA[0] = ceil_shift(rec.A[0], sft); t.EA[1] = ceil_shift(rec.A[1], sft);
      t.UA[0] = ceil_shift(rec.UA[0], sft); t.UA[1] = ceil_shift(rec.UA[1], sft);
      t.tp_x = rec.Sbh - (rec.Sbh >> sft);
      t.sbh_t = ceil_shift(rec.Sbh, sft);
      t.t_heads = (rec.heads & ((1u << sft) - 1u)) == 0 ? 1u : 0u;
      t.pad[0] = t.pad[1] = t.pad[2] = 0;
      sh.by_t[sft] = t;
      PipelineDegree k;
      k.lps = (rec.L + ((1u << sft) - 1u)) >> sft;
      k.k_layers = (rec.L & ((1u << sft) - 1u)) == 0 ? 1u : 0u;
      sh.by_k[sft] = k;
    }
    __syncthreads();
  }

  WarpTables& tb = sh.tables[warp];
  WarpList list{sh.list_a + warp * LIST_CAP, sh.list_b + warp * LIST_CAP,
                sh.list_i + warp * LIST_CAP, 0, 0};
  const int k_keep = (int)args.k_keep;
  Key threshold{U64MAX, U64MAX, 0xffffffffu};
  u32 survivors = 0;
  u64 dom_m = U64MAX, dom_c = U64MAX;               // Pareto: a point known to be a survivor

  // the fast case is compiled for spaces with one copy of every shard
  const u32 repl = FAST ? 1u : sp.repl;
  const u32 req = args.require_flags;
  const bool ext_in_objective = args.comm_kind == PS_COMM_PAPER_PLUS_EXT;
  const u32 nvt = sp.nvt;
  const u32 per_unit = nvt * NC;
  // capacities as exclusive bounds (memory and host bytes stay below 2^63)
  const u64 cap_x = min(args.cap_max, (u64)1 << 62) + 1;
  const u64 host_x = min(args.host_cap, (u64)1 << 62) + 1;
  constexpr bool host_limited = HOST_LIMITED;      // the launcher tests args.host_cap < 2^62
  constexpr u32 CV_BITS = PS_F_CV | PS_F_T_DIV_HEADS | PS_F_K_DIV_LAYERS | PS_F_TP_LE_MAX | PS_F_AXIS_FORM;
  const u32 req_cv = req & CV_BITS;

  // with all five modes allowed digit d is mode d: the compiler then knows every
  // per-digit property below (which digit offloads, which keep a replica's own
  // activations) and drops the tests
  const u32 modemap = (NM == 5) ? 0x43210u : sp.modemap;
  // activation-digit classes (Theorem 3: a replica needs its own activations)
  u32 all = (1u << NM) - 1u, own = 0, is_o = 0, not_mo = 0;
#pragma unroll
  for (int d = 0; d < NM; ++d) {
    const u32 ac = digit_mode(modemap, d);
    if (in_set(SET_ACT_OWN, ac)) own |= 1u << d;
    if (ac == PS_MODE_O) is_o |= 1u << d;
    if (!in_set(SET_M_OR_O, ac)) not_mo |= 1u << d;
  }

  // This lane's triples.  With E = elements of a state on one (t, k) position,
  // s = its largest data-axis shard, u = the reconstruction unit and x = the ring
  // volume in elements (all four the same for Theta, Omega and G), a triple's
  //   bytes          = ka * E + kb * s + kc * u     (Theorem 1, widths of Remark 1)
  //   communication  = kx * x                       (Theorem 2 [+ unpriced traffic])
  //   host bytes     = kh * s                       (mode O)
  // with small integer coefficients that depend only on the triple's modes and
  // the model's byte widths -- fixed for the whole kernel.
  u32 t_local[R];      // triple number (0 if the lane has none in this round)
  u32 t_allowed[R];    // allowed activation digits: bits 0..4, 8..12, 16..20 for the three CLS_* of a unit
  u32 ka[R], kb[R], kc[R], kx[R], kh[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const u32 t = lane + 32 * r;
    const bool live = t < (u32)N3;
    const u32 tt = live ? t : 0;
    const u32 modes[3] = {digit_mode(modemap, tt % NM), digit_mode(modemap, (tt / NM) % NM),
                          digit_mode(modemap, tt / N2)};
    const u32 width[3] = {rec.wT, rec.wO, rec.wG};
    const u32 th = modes[0], om = modes[1], gr = modes[2];
    const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
    u32 a = 0, b = 0, c = 0, h = 0;
#pragma unroll
    for (int st = 0; st < 3; ++st) {
      if (modes[st] == PS_MODE_R) a += width[st];
      if (in_set(SET_SHARDLIKE, modes[st])) b += width[st];
      if (modes[st] == PS_MODE_SG) c += width[st] * sp.sstar_units;   // one or two unit buffers
      if (modes[st] == PS_MODE_M) c += width[st];
    }
    // Theorem 2: all-reduce of replicated gradients, reduce-scatter of sharded
    // ones, two all-gathers of gathered parameters for each micro-batch
    u32 ct = (th == PS_MODE_SG) ? 2 * sp.accum : 0, co = 0;
    u32 cg = (gr == PS_MODE_R) ? 2 : (gr == PS_MODE_S ? 1 : 0);
    if (ext_in_objective) {                  // traffic the theorem does not price
      if (th == PS_MODE_O) ct += 2 * sp.accum;
      if (th == PS_MODE_R && on_shard) ct += 1;
      if (om == PS_MODE_SG) co = 1;
      if (gr == PS_MODE_SG) cg += 2;
      if (gr == PS_MODE_M) cg += on_shard ? 1 : 2;
      if (gr == PS_MODE_O) cg += 1;
    }
    if (th == PS_MODE_O) h += (2 * sp.accum + 1) * rec.wT;
    if (om == PS_MODE_O) h += 2 * rec.wO;
    if (gr == PS_MODE_O) h += 2 * rec.wG;
    t_local[r] = tt;
    ka[r] = a; kb[r] = b; kc[r] = c; kh[r] = h;
    kx[r] = ct * rec.wT + co * rec.wO + cg * rec.wG;
    const u32 a_many = allowed_act_digits(triple_bits(th, om, gr, CLS_SHARDED), req, all, own, is_o, not_mo);
    const u32 a_one = allowed_act_digits(triple_bits(th, om, gr, CLS_ONE_DEVICE), req, all, all, is_o, not_mo);
    const u32 a_copies = allowed_act_digits(triple_bits(th, om, gr, CLS_ALL_COPIES), req, all, all, is_o, not_mo);
    t_allowed[r] = live ? (a_many | (a_one << 8) | (a_copies << 16)) : 0;
    // keep the coefficients in registers instead of recomputing them for every unit
    asm volatile("" : "+r"(ka[r]), "+r"(kb[r]), "+r"(kc[r]), "+r"(kx[r]), "+r"(kh[r]), "+r"(t_allowed[r]));
  }

  // this lane's table entry (variant, digit), also fixed for the whole kernel
  const u32 tl_vt = lane / NM, tl_d = lane - tl_vt * NM;
  const bool tl_mine = tl_vt < nvt;
  const u32 tl_v = tl_mine ? tl_vt / sp.nt : 0;
  const u32 tl_tau = tl_mine ? tl_vt - tl_v * sp.nt : 0;
  const u32 tl_mode = digit_mode(modemap, tl_d);
  const u64 tl_A = rec.A[tl_v], tl_UA = rec.UA[tl_v];

  // warps take the block's units in turn: the first one by warp number, then
  // whichever is next when they finish (their work differs with the candidates)
  u32 unit = u_begin + warp;
  while (SKIP && args.skip_rejected && unit < u_end && unit_rejected(sp, rec, unit, req_cv)) {
    u32 nxt = 0;
    if (lane == 0) nxt = atomicAdd(&sh.next_unit, 1u);
    unit = __shfl_sync(0xffffffffu, nxt, 0);
  }
  while (unit < u_end) {
    const Fact f = sp.facts[unit];
    const Pow2 p2 = FAST ? pow2_of(f) : pow2_of(f, repl);
    UnitBase ub;
    if (FAST) {
      // the tensor and pipeline parts come from the block's tables
      const TensorDegree& td = sh.by_t[p2.sT];
      const PipelineDegree kd = sh.by_k[p2.sK];
      ub.E2 = ceil_shift(td.E1, p2.sK);
      // (one copy of every shard here: the shard positions are the D devices)
      ub.G = f.D;
      ub.sh = ceil_shift(ub.E2, p2.sD);
      ub.x = ub.E2 - (ub.E2 >> p2.sD);
      ub.x2 = 0;
      ub.x3 = 0;
      ub.cls = f.D == 1 ? CLS_ONE_DEVICE : CLS_SHARDED;
      ub.u = td.u;
      ub.tp_x = td.tp_x;
      ub.sbh_t = td.sbh_t;
      ub.lps = kd.lps;
      const bool tp_le = f.T <= sp.tp_max_valid;
      const bool whole = ((u64)f.T * f.K * f.D == (u64)f.N);
      u32 cv = (td.t_heads ? PS_F_T_DIV_HEADS : 0) | (kd.k_layers ? PS_F_K_DIV_LAYERS : 0) |
               (tp_le ? PS_F_TP_LE_MAX : 0) | PS_F_AXIS_FORM;
      if (td.t_heads && kd.k_layers && tp_le && whole) cv |= PS_F_CV;
      ub.cv = cv;
      ub.d1 = (f.D == 1);
    } else {
      ub = p2.all ? unit_base_pow2(rec, f, p2, sp.tp_max_valid, true)
                  : unit_base(rec, f, sp.tp_max_valid, true, repl);
    }
    __syncwarp();
    {
      // lane (vt, d): activation bytes of digit d under variant vt, and the bound
      // a triple's own bytes must stay below for the sum to fit the capacity
      ActBase ab;
      if (FAST) {
        const TensorDegree& td = sh.by_t[tl_tau == 0 ? p2.sT : 0];     // degree 1 = not sharded
        ab.EA = td.EA[tl_v];
        ab.uA = td.UA[tl_v];
        ab.shA = ceil_shift(ab.EA, p2.sD);
      } else if (p2.all) {
        const u32 s = tl_tau == 0 ? p2.sT : 0;
        ab.EA = ceil_shift(tl_A, s);
        ab.uA = ceil_shift(tl_UA, s);
        ab.shA = ceil_shift(ab.EA, p2.sG);
      } else {
        ab.EA = tl_tau == 0 ? div_ceil(tl_A, f.T) : tl_A;
        ab.uA = tl_tau == 0 ? div_ceil(tl_UA, f.T) : tl_UA;
        ab.shA = div_ceil(ab.EA, ub.G);
      }
      const u64 am = mu_elems(tl_mode, ab.EA, ab.shA, ab.uA, sp.sstar_units);
      if (tl_mine) {
        const u64 bound = am < cap_x ? cap_x - am : 0;
        tb.bound[tl_d][tl_vt] = bound;
        tb.bound_f64[tl_d][tl_vt] = (double)bound;
        tb.act[tl_vt][tl_d] = am;
        if (tl_d == 0) {
          const u64 ah = 2 * ab.EA * sp.accum;                 // offload after fwd, reload for bwd, per micro-batch
          const u64 hb = ah < host_x ? host_x - ah : 0;
          tb.host_bound[tl_vt] = hb;
          tb.host_bound_f64[tl_vt] = (double)hb;      // rounded only above 2^53, where no host figure of the fast case reaches
          tb.c_axis[tl_vt] = ext_in_objective ? model_axis_traffic(rec, f, ub, tl_tau, sp.tp_coll, sp.accum) : 0;
        }
      } else if (tl_vt < 4) {
        tb.bound[tl_d][tl_vt] = 0;
        tb.bound_f64[tl_d][tl_vt] = 0.0;
        if (tl_d == 0) { tb.host_bound[tl_vt] = 0; tb.host_bound_f64[tl_vt] = 0.0; }
      }
    }
    __syncwarp();
    // the lane's triples for this unit: own bytes, own communication, allowed digits
    const bool unit_ok = (ub.cv & req_cv) == req_cv;
    const u32 a_shift = FAST ? (ub.d1 ? 8u : 0u) : 8 * ub.cls;
    u64 mem3[R], comm3[R], host3[R];
    double mem3_f64[R], host3_f64[R];
    const double e2_f64 = (double)ub.E2, sh_f64 = (double)ub.sh, u_f64 = (double)ub.u;
    u32 allowed[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      // the fast case forms the bytes as a double right away (three exact fused
      // multiply-adds) and the integer only if the reduction pass needs it
      if (FAST) mem3_f64[r] = fma((double)ka[r], e2_f64, fma((double)kb[r], sh_f64, (double)kc[r] * u_f64));
      else mem3[r] = mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0)));
      if (!FAST) {                                      // the fast case forms it where it is needed
        comm3[r] = mad_small(ub.x, kx[r], 0);
        if (repl > 1)
          comm3[r] += copies_traffic(digit_mode(modemap, (t_local[r] / NM) % NM), digit_mode(modemap, t_local[r] / N2),
                                     rec.wG, ext_in_objective, ub.x2, ub.x3);
      }
      bool host_fits = true;                    // the triple's own host bytes against the budget
      if (host_limited) {
        if (FAST) { host3_f64[r] = (double)kh[r] * sh_f64; host_fits = host3_f64[r] < (double)host_x; }
        else { host3[r] = mad_small(ub.sh, kh[r], 0); host_fits = host3[r] < host_x; }
      } else {
        host3[r] = 0;
      }
      allowed[r] = (unit_ok && host_fits) ? ((t_allowed[r] >> a_shift) & all) : 0;
    }
    const u32 unit_first = unit * per_unit;      // index of the unit's first point in the model

    // ---- evaluation pass: every point of the unit.  Point (triple r, variant vt,
    // digit d) is a survivor if the flags allow the digit, the triple's bytes are
    // below the (variant, digit) bound and, for the offload digit, the host bytes
    // fit.  Survivors are counted per triple.
    u32 n_pass[R];
#pragma unroll
    for (int r = 0; r < R; ++r) n_pass[r] = 0;
    // Integers below 2^53 are exact in fp64, so when every quantity of the unit is
    // that small (uniform test) the compares run on the fp64 pipe, which is idle
    // otherwise, and only the counting stays on the integer pipe.
    const bool small = FAST || (cap_x < ((u64)1 << 53) &&
                                (u64)(rec.wT + rec.wO + rec.wG) * (ub.E2 + 2 * ub.u) < ((u64)1 << 53));
    if (small) {
      double mem_f64[R];
      float pass_f32[R];
#pragma unroll
      for (int r = 0; r < R; ++r) { mem_f64[r] = FAST ? mem3_f64[r] : (double)mem3[r]; pass_f32[r] = 0.0f; }
#pragma unroll
      for (int d = 0; d < NM; ++d) {
        const bool host_check = host_limited && ((is_o >> d) & 1u);
        if (((F64_DIGITS >> d) & 1u) || host_check) {
          double bound[4];
          {
            const double2 b01 = *reinterpret_cast<const double2*>(&tb.bound_f64[d][0]);
            const double2 b23 = *reinterpret_cast<const double2*>(&tb.bound_f64[d][2]);
            bound[0] = b01.x; bound[1] = b01.y; bound[2] = b23.x; bound[3] = b23.y;
          }
#pragma unroll
          for (int r = 0; r < R; ++r) {
            // compare on the fp64 pipe, count with predicated fp32 adds (small
            // integers are exact): nothing here uses the integer ALU pipe
            float c = 0.0f;
            if (host_check) {
              // offloading activations also has to fit the host budget of the variant
#pragma unroll
              for (int vt = 0; vt < 4; ++vt)
                if (mem_f64[r] < bound[vt] &&
                    (FAST ? host3_f64[r] < tb.host_bound_f64[vt] : host3[r] < tb.host_bound[vt]))
                  c += 1.0f;
            } else {
#pragma unroll
              for (int vt = 0; vt < 4; ++vt)
                if (mem_f64[r] < bound[vt]) c += 1.0f;
            }
            if ((allowed[r] >> d) & 1u) pass_f32[r] += c;
          }
        } else {
          u64 bound[4];
          {
            const ulonglong2 b01 = *reinterpret_cast<const ulonglong2*>(&tb.bound[d][0]);
            const ulonglong2 b23 = *reinterpret_cast<const ulonglong2*>(&tb.bound[d][2]);
            bound[0] = b01.x; bound[1] = b01.y; bound[2] = b23.x; bound[3] = b23.y;
          }
#pragma unroll
          for (int r = 0; r < R; ++r) {
            u32 not_below = 0;
#pragma unroll
            for (int vt = 0; vt < 4; ++vt) count_not_below(not_below, mem3[r], bound[vt]);
            n_pass[r] += ((allowed[r] >> d) & 1u) ? 4u - not_below : 0u;
          }
        }
      }
#pragma unroll
      for (int r = 0; r < R; ++r) n_pass[r] += (u32)pass_f32[r];
    } else {
#pragma unroll
    for (int d = 0; d < NM; ++d) {
      u64 bound[4];
      {
        const ulonglong2 b01 = *reinterpret_cast<const ulonglong2*>(&tb.bound[d][0]);
        const ulonglong2 b23 = *reinterpret_cast<const ulonglong2*>(&tb.bound[d][2]);
        bound[0] = b01.x; bound[1] = b01.y; bound[2] = b23.x; bound[3] = b23.y;
      }
      if (host_limited && ((is_o >> d) & 1u)) {
        // offloading activations also has to fit the host budget of the variant
#pragma unroll
        for (int r = 0; r < R; ++r) {
          u32 c = 0;
#pragma unroll
          for (int vt = 0; vt < 4; ++vt)
            c += (mem3[r] < bound[vt] && host3[r] < tb.host_bound[vt]) ? 1u : 0u;
          n_pass[r] += ((allowed[r] >> d) & 1u) ? c : 0u;
        }
      } else {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          u32 not_below = 0;               // variants whose bound the triple's bytes reach
#pragma unroll
          for (int vt = 0; vt < 4; ++vt) count_not_below(not_below, mem3[r], bound[vt]);
          n_pass[r] += ((allowed[r] >> d) & 1u) ? 4u - not_below : 0u;
        }
      }
    }

    }
    // ---- reduction pass, only if some survivor of this warp can matter
    bool matters = false;
    u32 alive = 0;                         // Pareto: the lane's triples that may still add to the frontier
    if (KIND == PS_REDUCE_PARETO) {
      // A triple with survivors matters unless every point of it is beaten already: its own
      // bytes and its volume plus the least axis traffic bound its points from below, and a
      // point known to survive (the cached one, or the block's coarse staircase) that beats
      // the bounds strictly beats them all.
      bool some = false;
#pragma unroll
      for (int r = 0; r < R; ++r) some = some || n_pass[r] != 0;
      if (some) {
        const u64 least_axis = tb.c_axis[0];   // tau = 0 sends the smaller boundary tensor; v does not matter
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const u64 m_lb = FAST ? mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0))) : mem3[r];
          const u64 c_lb = (FAST ? mad_small(ub.x, kx[r], 0) : comm3[r]) + least_axis;
          const int bucket = stair_bucket(m_lb);
          const bool beaten = (dom_m <= m_lb && dom_c <= c_lb && (dom_m != m_lb || dom_c != c_lb)) ||
                              (bucket > 0 && sh.stair[bucket - 1] <= c_lb);
          if (n_pass[r] != 0 && !beaten) alive |= 1u << r;
        }
      }
      matters = alive != 0;
    } else {
      const u64 comm_limit = min(threshold.a, (u64)sh.block_comm_limit);
      const u64 least_axis = tb.c_axis[0];   // tau = 0 sends the smaller boundary tensor; v does not matter
      if (FAST) {
        // a triple's volume is below 2^53 here, so it is compared as a double against
        // what the limit leaves after the axis traffic (exact below 2^53, and above
        // it every volume passes anyway)
        const double room = comm_limit >= least_axis ? (double)(comm_limit - least_axis) : -1.0;
        const double x_f64 = (double)ub.x;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          survivors += n_pass[r];
          matters = matters || (n_pass[r] != 0 && (double)kx[r] * x_f64 <= room);
        }
      } else {
#pragma unroll
        for (int r = 0; r < R; ++r) {
          survivors += n_pass[r];
          matters = matters || (n_pass[r] != 0 && comm3[r] + least_axis <= comm_limit);
        }
      }
    }
    if (KIND == PS_REDUCE_PARETO && __any_sync(0xffffffffu, matters)) {
      // About one unit in ten comes here (every unit with a survivor).  Written as
      // rolled loops over the lane's triples, whose values it first copies to arrays
      // that can be indexed at run time, so that this part's registers do not weigh on
      // the evaluation pass; only the digits of a point are tested side by side.
      u64 l_mem[R], l_comm[R], l_host[R];
      u32 l_allowed[R], l_triple[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        l_mem[r] = FAST ? mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0))) : mem3[r];
        l_comm[r] = FAST ? mad_small(ub.x, kx[r], 0) : comm3[r];
        l_host[r] = (FAST && host_limited) ? mad_small(ub.sh, kh[r], 0) : host3[r];
        l_allowed[r] = allowed[r]; l_triple[r] = t_local[r];
      }
      {
        // lane = a set of activation digits; which of them costs the least bytes
        // (the variants side by side: four independent chains)
        u64 least[4];
        u32 which[4];
#pragma unroll
        for (int vt = 0; vt < 4; ++vt) { least[vt] = U64MAX; which[vt] = NM; }
#pragma unroll
        for (int d = NM - 1; d >= 0; --d) {
#pragma unroll
          for (int vt = 0; vt < 4; ++vt) {
            const u64 am = tb.act[vt < (int)nvt ? vt : 0][d];
            if (((lane >> d) & 1) && am <= least[vt]) { least[vt] = am; which[vt] = d; }
          }
        }
#pragma unroll
        for (int vt = 0; vt < 4; ++vt) tb.least[vt][lane] = (unsigned char)which[vt];
      }
      __syncwarp();
      // rounds of triples in which some lane's triple is still alive
      u32 rounds = 0;
#pragma unroll
      for (int r = 0; r < R; ++r) rounds |= __any_sync(0xffffffffu, (alive >> r) & 1u) ? (1u << r) : 0u;

      // Variants in an order in which later ones seldom beat earlier ones (the result
      // does not depend on the order, the work does): the tensor axis that shards
      // activations first, and full checkpointing before stored activations -- fewer
      // bytes at the same communication.
#pragma unroll 1
      for (u32 vt_step = 0; vt_step < nvt; ++vt_step) {
        const u32 vt = (sp.nv - 1 - vt_step % sp.nv) * sp.nt + vt_step / sp.nv;
        const u64 c_axis = tb.c_axis[vt], host_bound = tb.host_bound[vt];
        const u32 vt_first = unit_first + vt * NC;
        u64 bound[NM];
#pragma unroll
        for (int d = 0; d < NM; ++d) bound[d] = tb.bound[d][vt];
#pragma unroll 1
        for (int r = 0; r < R; ++r) {
          if (!((rounds >> r) & 1u)) continue;
          // digit d of (triple, variant) is a survivor if the triple's bytes are below the
          // digit's bound and the flags allow the digit
          const u64 lm = l_mem[r];
          u32 fit = 0;
#pragma unroll
          for (int d = 0; d < NM; ++d) fit |= (lm < bound[d]) ? (1u << d) : 0u;
          // offloading activations adds host bytes: drop that digit if they do not fit
          const u32 allow_vt = (l_host[r] < host_bound) ? l_allowed[r] : (l_allowed[r] & ~is_o);
          const u32 pass = fit & allow_vt;
          // For a triple and variant the communication is the same for all NM activation
          // digits, so of the surviving digits only the one with the least bytes (lowest
          // digit on ties) can be on the frontier.
          const bool has = pass != 0;
          const u32 d = has ? tb.least[vt][pass] : 0;
          const u64 m = lm + tb.act[vt][d];
          const u64 c = l_comm[r] + c_axis;
          const u32 idx = vt_first + l_triple[r] + d * N3;
          // cheap tests first: strictly dominated by a point already known to survive,
          // or by the block's coarse staircase
          bool cand = has && !(dom_m <= m && dom_c <= c && (dom_m != m || dom_c != c));
          if (cand) {
            const int bucket = stair_bucket(m);
            if (bucket > 0 && sh.stair[bucket - 1] <= c) cand = false;
          }
          if (!__any_sync(0xffffffffu, cand)) continue;
          if (cand) {
            int lo = 0, hi = list.n;
            while (lo < hi) {               // entries with mem <= m
              const int mid = (lo + hi) >> 1;
              if (list.a[mid] <= m) lo = mid + 1; else hi = mid;
            }
            if (lo > 0) {
              const u64 em = list.a[lo - 1], ec = list.b[lo - 1];
              if (ec < c || (ec == c && (em < m || list.i[lo - 1] < idx))) {
                cand = false;
                dom_m = em; dom_c = ec;
              }
            }
          }
          u32 pending = __ballot_sync(0xffffffffu, cand);
          while (pending) {
            const int src = __ffs(pending) - 1;
            const u64 pm = __shfl_sync(0xffffffffu, m, src);
            const u64 pc = __shfl_sync(0xffffffffu, c, src);
            const u32 pi = __shfl_sync(0xffffffffu, idx, src);
            pareto_insert(list, pm, pc, pi, lane, sh.stair);
            pending &= pending - 1;
          }
        }
      }
    }
    if (KIND == PS_REDUCE_TOPK && __any_sync(0xffffffffu, matters)) {
      // This part runs for a few units in a hundred, so it is written as rolled
      // loops over the lane's triples, whose values it first copies to arrays that
      // can be indexed at run time: code that is rarely executed is not in the
      // instruction cache, and fetching a long unrolled sequence costs far more
      // than executing it.
      u64 l_mem[R], l_comm[R], l_host[R];
      u32 l_allowed[R], l_triple[R], l_pass[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        l_mem[r] = FAST ? mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0))) : mem3[r];
        l_comm[r] = FAST ? mad_small(ub.x, kx[r], 0) : comm3[r];
        l_host[r] = (FAST && host_limited) ? mad_small(ub.sh, kh[r], 0) : host3[r];
        l_allowed[r] = allowed[r]; l_triple[r] = t_local[r];
      }
#pragma unroll 1
      for (u32 vt_step = 0; vt_step < nvt; ++vt_step) {
        const u32 vt = (sp.nv - 1 - vt_step % sp.nv) * sp.nt + vt_step / sp.nv;
        const u64 c_axis = tb.c_axis[vt], host_bound = tb.host_bound[vt];
        const u32 vt_first = unit_first + vt * NC;
        // every point of (triple, variant): digit d is a survivor if the triple's
        // bytes are below the digit's bound and the flags allow the digit
        u64 bound[NM];
#pragma unroll
        for (int d = 0; d < NM; ++d) bound[d] = tb.bound[d][vt];
        {
          // the k-th smallest communication known to this warp or to any warp of the block
          const u64 comm_limit = min(threshold.a, (u64)sh.block_comm_limit);
          // every point of (triple, variant): digit d is a survivor if the triple's bytes
          // are below the digit's bound and the flags allow the digit; the survivors below
          // the threshold key are candidates, per triple as digit bits
          u32 mine = 0;
#pragma unroll 1
          for (int r = 0; r < R; ++r) {
            const u64 lm = l_mem[r];
            u32 fit = 0;
#pragma unroll
            for (int d = 0; d < NM; ++d) fit |= (lm < bound[d]) ? (1u << d) : 0u;
            // offloading activations adds host bytes: drop that digit if they do not fit
            const u32 allow_vt = (l_host[r] < host_bound) ? l_allowed[r] : (l_allowed[r] & ~is_o);
            const u32 pass = fit & allow_vt;
            const u64 c = l_comm[r] + c_axis;
            u32 cand = (c < threshold.a && c <= comm_limit) ? pass : 0u;
            if (c == threshold.a && pass != 0) {
#pragma unroll 1
              for (int d = 0; d < NM; ++d) {
                const Key key{c, lm + tb.act[vt][d], vt_first + l_triple[r] + d * N3};
                if (((pass >> d) & 1u) && key_less(key, threshold)) cand |= 1u << d;
              }
            }
            l_pass[r] = cand;
            mine += __popc(cand);
          }
          u32 incl = mine;                               // inclusive prefix sum over the lanes
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const u32 up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
          }
          const u32 total = __shfl_sync(0xffffffffu, incl, 31);
          if (total == 0) continue;
          if (list.n + total <= (u32)LIST_CAP) {
            int p = list.n + (int)(incl - mine);
#pragma unroll 1
            for (int r = 0; r < R; ++r) {
              u32 bits = l_pass[r];
              while (bits) {
                const u32 d = __ffs(bits) - 1;
                bits &= bits - 1;
                list.a[p] = l_comm[r] + c_axis;
                list.b[p] = l_mem[r] + tb.act[vt][d];
                list.i[p] = vt_first + l_triple[r] + d * N3;
                ++p;
              }
            }
            list.n += (int)total;
            __syncwarp();
          } else {
            // does not fit in one go: one (triple round, digit) at a time, compacting as
            // needed; digits downwards, because the higher modes (offloaded, recomputed,
            // sharded) keep fewer activation bytes, so that what comes later seldom gets in
#pragma unroll 1
            for (int d = NM - 1; d >= 0; --d) {
              const u64 am = tb.act[vt][d];
#pragma unroll 1
              for (int r = 0; r < R; ++r) {
                const Key key{l_comm[r] + c_axis, l_mem[r] + am, vt_first + l_triple[r] + d * N3};
                topk_append(list, ((l_pass[r] >> d) & 1u) && key_less(key, threshold), key, k_keep, lane,
                            threshold, &sh.block_comm_limit);
              }
            }
          }
          // the first k candidates give the first threshold
          if (threshold.i == 0xffffffffu && threshold.a == U64MAX && list.n >= k_keep)
            topk_compact(list, k_keep, lane, threshold, &sh.block_comm_limit);
        }
      }
    }
    // next unit
    do {
      u32 nxt = 0;
      if (lane == 0) nxt = atomicAdd(&sh.next_unit, 1u);
      unit = __shfl_sync(0xffffffffu, nxt, 0);
    } while (SKIP && args.skip_rejected && unit < u_end && unit_rejected(sp, rec, unit, req_cv));
  }

  // ---- the warp's list goes to global scratch, sorted (top-k: its k smallest
  // by key; Pareto: the staircase, ascending bytes); nothing waits for the other warps
  for (int o = 16; o > 0; o >>= 1) survivors += __shfl_xor_sync(0xffffffffu, survivors, o);
  if (KIND == PS_REDUCE_TOPK && list.n > 0) topk_compact(list, k_keep, lane, threshold, &sh.block_comm_limit);
  __syncwarp();
  const u64 slot = ((u64)model * n_chunks + chunk) * WARPS + warp;
  PartialEntry* dst = args.partial + slot * LIST_CAP;
  for (int p = lane; p < list.n; p += 32) {
    PartialEntry e;
    e.a = list.a[p]; e.b = list.b[p]; e.i = list.i[p]; e.pad = 0;
    dst[p] = e;
  }
  if (lane == 0) args.partial_n[slot] = make_uint2(list.over ? LIST_OVERFLOWED : (u32)list.n, survivors);
}

// ------------------------------------------------------------------ merge + emit
// One block per model: combine the partial lists of the model's warps (n_lists
// = blocks per model x warps per block), then write the entries of every
// capacity.  Every list arrives sorted by key -- (mem, comm, idx) for Pareto,
// where a staircase has distinct ascending bytes, (comm, mem, idx) for top-k --
// and no point is in two lists, so an entry's place in the sorted union is its
// place at home plus, for every other list, the number of entries below it
// there: binary searches, no sort.  The union is then cut back (top-k: the k
// smallest; Pareto: entries whose communication is below that of everything
// before them).  Lists are taken in rounds -- as many as fit beside what has been
// kept so far, so any number can be combined.  Each emitted point is evaluated
// again from its index (host bytes and flags come from there; mem and comm must
// agree).
//
// A frontier with more than LIST_CAP entries -- in one warp's share of a model
// or after merging -- does not fit these lists.  The block then computes the
// model's frontier by the definition instead, one entry per pass over the
// model's points: the next entry is the survivor with the fewest bytes among
// those with more bytes and less communication than the last entry (fewest
// communication, then smallest index, on ties).  Slow (passes = frontier
// length), bounded memory, any length.
#ifndef SWEEP_MERGE_THREADS
#define SWEEP_MERGE_THREADS 128
#endif
constexpr int MERGE_THREADS = SWEEP_MERGE_THREADS;
constexpr int MERGE_LISTS = 16;             // most lists a round takes (they are usually far from full)
constexpr int MERGE_MAX_LISTS = SWEEP_MAX_CHUNKS * (SWEEP_WARPS_PARETO > SWEEP_WARPS_TOPK ? SWEEP_WARPS_PARETO : SWEEP_WARPS_TOPK);

struct MergeShared {
  u64 in_a[MERGE_CAP], in_b[MERGE_CAP];     // the kept entries, then the round's lists
  u32 in_i[MERGE_CAP];
  u64 a[MERGE_CAP], b[MERGE_CAP];           // the sorted union; after the cut, the kept entries
  u32 i[MERGE_CAP];
  int off[MERGE_LISTS + 2];                 // start of each list in in_*
  int from[MERGE_LISTS + 1];                // which of the model's lists sits there
  int taken;                                // lists of this round
  int next;                                 // first list the next round looks at
  unsigned short len[MERGE_MAX_LISTS];      // entries of every list of the model
  u64 warp_min[MERGE_THREADS / 32];
  int warp_sum[MERGE_THREADS / 32];
  u32 survivors;
};

// exclusive prefix minimum / prefix sum over the threads of a block
__device__ __forceinline__ u64 block_excl_min(u64 mine, u64* warp_min, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  u64 incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const u64 up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl = min(incl, up);
  }
  u64 excl = __shfl_up_sync(0xffffffffu, incl, 1);
  if (lane == 0) excl = U64MAX;
  if (lane == 31) warp_min[warp] = incl;
  __syncthreads();
  for (int w = 0; w < warp; ++w) excl = min(excl, warp_min[w]);
  __syncthreads();
  return excl;
}
__device__ __forceinline__ int block_excl_sum(int mine, int* warp_sum, int tid, int* total) {
  const int lane = tid & 31, warp = tid >> 5;
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  int before = 0, all = 0;
  for (int w = 0; w < MERGE_THREADS / 32; ++w) {
    if (w < warp) before += warp_sum[w];
    all += warp_sum[w];
  }
  __syncthreads();
  *total = all;
  return before + incl - mine;
}

// one point of a model from its index, as an output entry; the objective is returned through *comm
__device__ __forceinline__ PointOut eval_local(const SpaceDev& sp, const ModelRec& rec, u32 lidx) {
  const LocalPoint lp = decode_local(sp, lidx);
  const Fact f = sp.facts[lp.unit];
  return eval_point(rec, f, lp.v, lp.tau, digit_mode(sp.modemap, lp.dth), digit_mode(sp.modemap, lp.dom),
                    digit_mode(sp.modemap, lp.dgr), digit_mode(sp.modemap, lp.dac), sp.tp_max_valid,
                    sp.tp_coll, true, sp.sstar_units, sp.accum, sp.repl);
}

// The slow exact path for a model whose frontier outgrew the lists: see above.
// A kernel of its own, launched after every Pareto merge, so that the merge kernel does not
// carry its registers; a block whose model needs no slow path returns at once.
__global__ void __launch_bounds__(MERGE_THREADS) k_frontier_by_definition(SpaceDev sp, MergeArgs args) {
  __shared__ Key pass_best[MERGE_THREADS / 32];    // the warps' best candidates of a pass
  const u32 model = blockIdx.x;
  if (args.slow_path[model] == 0) return;
  const ModelRec rec = sp.recs[model];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  u32 found[PS_MAX_CAPS];
  for (u32 ci = 0; ci < PS_MAX_CAPS; ++ci) found[ci] = 0;
  u64 last_mem = 0, last_comm = U64MAX;
  bool have_last = false;
  const u32 ppm = (u32)sp.ppm;
  for (u32 pass = 0; pass <= ppm; ++pass) {             // a frontier has at most ppm entries
    Key best{U64MAX, U64MAX, 0xffffffffu};
    for (u32 lidx = tid; lidx < ppm; lidx += MERGE_THREADS) {
      const PointOut po = eval_local(sp, rec, lidx);
      const u64 comm = args.comm_kind == PS_COMM_PAPER ? po.comm_paper : po.comm_paper + po.comm_ext;
      const bool survivor = po.mem <= args.cap_max && po.host <= args.host_cap &&
                            (po.flags & args.require_flags) == args.require_flags;
      const bool beyond = !have_last || (po.mem > last_mem && comm < last_comm);
      const Key key{po.mem, comm, lidx};
      if (survivor && beyond && key_less(key, best)) best = key;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const Key other = key_shfl_xor(best, o);
      if (key_less(other, best)) best = other;
    }
    if (lane == 0) pass_best[warp] = best;
    __syncthreads();
    best = pass_best[0];
    for (int w = 1; w < MERGE_THREADS / 32; ++w)
      if (key_less(pass_best[w], best)) best = pass_best[w];
    __syncthreads();
    if (best.i == 0xffffffffu) break;                   // nothing beyond the last entry: done
    for (u32 ci = 0; ci < args.n_caps; ++ci) {
      if (best.a > args.caps[ci]) continue;
      const u32 slot = found[ci]++;
      if (slot < args.max_entries && tid == 0) {
        const PointOut po = eval_local(sp, rec, best.i);
        ps_front_entry e;
        e.mem = po.mem; e.comm = best.b; e.host = po.host;
        e.idx = (u64)model * sp.ppm + best.i;
        e.flags = po.flags | PS_F_FEASIBLE; e.pad = 0;
        args.out[((u64)model * args.n_caps_total + ci) * args.max_entries + slot] = e;
      }
    }
    last_mem = best.a; last_comm = best.b; have_last = true;
  }
  for (u32 ci = 0; ci < args.n_caps; ++ci) {
    ps_front_entry* out = args.out + ((u64)model * args.n_caps_total + ci) * args.max_entries;
    ps_front_entry zero;
    zero.mem = 0; zero.comm = 0; zero.host = 0; zero.idx = 0; zero.flags = 0; zero.pad = 0;
    for (u32 p = found[ci] + tid; p < args.max_entries; p += MERGE_THREADS) out[p] = zero;
    if (tid == 0) {
      args.counts[(u64)model * args.n_caps_total + ci] = found[ci];
      if (found[ci] > args.max_entries) atomicOr(args.status, ST_TRUNCATED);
    }
  }
}

// compiled for eight resident blocks per SM (64 registers): the kernel is a chain of
// short steps between barriers, so it lives on many blocks in flight
#ifndef SWEEP_MERGE_MIN_BLOCKS
#define SWEEP_MERGE_MIN_BLOCKS 8
#endif
template <int KIND>
__global__ void __launch_bounds__(MERGE_THREADS, SWEEP_MERGE_MIN_BLOCKS) k_sweep_merge(SpaceDev sp, MergeArgs args) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  MergeShared& sh = *reinterpret_cast<MergeShared*>(smem_raw);
  const int tid = threadIdx.x;
  const u32 model = blockIdx.x;
  const u32 n_lists = args.n_lists;
  const uint2* list_n = args.partial_n + (u64)model * n_lists;
  const PartialEntry* lists = args.partial + (u64)model * n_lists * LIST_CAP;
  if (tid == 0) sh.survivors = 0;
  __syncthreads();
  bool overflowed = false;
  {
    u32 surv = 0;
    for (u32 l = tid; l < n_lists; l += MERGE_THREADS) {
      const uint2 ln = list_n[l];
      surv += ln.y;
      overflowed = overflowed || ln.x == LIST_OVERFLOWED;
      sh.len[l] = (unsigned short)min(ln.x, (u32)LIST_CAP);
    }
    if (surv) atomicAdd(&sh.survivors, surv);
  }
  overflowed = __syncthreads_or(overflowed) != 0;
  int n_list = 0;                                  // entries kept so far: sh.a/b/i[0, n_list), sorted
  for (u32 next = 0; next < n_lists && !overflowed;) {
    // list 0 = the kept entries, lists 1..taken = as many of the next non-empty lists as
    // fit (at least one does: kept entries and a list are at most LIST_CAP each)
    if (tid == 0) {
      int off = n_list, c = 0;
      u32 l = next;
      sh.off[0] = 0;
      for (; c < MERGE_LISTS && l < n_lists; ++l) {
        const int n = sh.len[l];
        if (n == 0) continue;
        if (off + n > MERGE_CAP) break;
        sh.off[c + 1] = off;
        sh.from[c + 1] = (int)l;
        off += n;
        ++c;
      }
      sh.off[c + 1] = off;
      sh.taken = c;
      sh.next = (int)l;
    }
    for (int p = tid; p < n_list; p += MERGE_THREADS) { sh.in_a[p] = sh.a[p]; sh.in_b[p] = sh.b[p]; sh.in_i[p] = sh.i[p]; }
    __syncthreads();
    const int taken = sh.taken;
    const int total = sh.off[taken + 1];
    for (int c = 1; c <= taken; ++c) {
      const PartialEntry* src = lists + (u64)sh.from[c] * LIST_CAP;
      const int base = sh.off[c], n = sh.off[c + 1] - base;
      for (int p = tid; p < n; p += MERGE_THREADS) {
        const PartialEntry e = src[p];
        sh.in_a[base + p] = e.a; sh.in_b[base + p] = e.b; sh.in_i[base + p] = e.i;
      }
    }
    __syncthreads();
    // place every entry in the sorted union
    for (int e = tid; e < total; e += MERGE_THREADS) {
      int home = 0;
      while (sh.off[home + 1] <= e) ++home;
      const Key key{sh.in_a[e], sh.in_b[e], sh.in_i[e]};
      int rank = e - sh.off[home];
      for (int c = 0; c <= taken; ++c) {
        if (c == home) continue;
        int lo = sh.off[c], hi = sh.off[c + 1];
        const int base = lo;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          const Key other{sh.in_a[mid], sh.in_b[mid], sh.in_i[mid]};
          if (key_less(other, key)) lo = mid + 1; else hi = mid;
        }
        rank += lo - base;
      }
      sh.a[rank] = key.a; sh.b[rank] = key.b; sh.i[rank] = key.i;
    }
    __syncthreads();
    if (KIND == PS_REDUCE_TOPK) {
      n_list = min(total, (int)args.k_keep);
    } else {
      // an entry stays iff its communication is below that of every entry before it
      constexpr int PER = (MERGE_CAP + MERGE_THREADS - 1) / MERGE_THREADS;
      const int lo = min(tid * PER, total), hi = min(lo + PER, total);
      u64 local = U64MAX;
      for (int p = lo; p < hi; ++p) local = min(local, sh.b[p]);
      const u64 before = block_excl_min(local, sh.warp_min, tid);
      Key keep[PER];
      int nk = 0;
      u64 run = before;
#pragma unroll
      for (int k = 0; k < PER; ++k) {
        const int p = lo + k;
        if (p < hi && sh.b[p] < run) { run = sh.b[p]; keep[nk].a = sh.a[p]; keep[nk].b = sh.b[p]; keep[nk].i = sh.i[p]; ++nk; }
      }
      int kept_total;
      const int offset = block_excl_sum(nk, sh.warp_sum, tid, &kept_total);   // barriers inside: all reads above are done
      for (int k = 0; k < nk; ++k)
        if (offset + k < MERGE_CAP) { sh.a[offset + k] = keep[k].a; sh.b[offset + k] = keep[k].b; sh.i[offset + k] = keep[k].i; }
      n_list = kept_total;
      if (n_list > LIST_CAP) overflowed = true;      // the same for every thread
    }
    next = (u32)sh.next;
    __syncthreads();
  }
  const u32 s_survivors = sh.survivors;

  const ModelRec rec = sp.recs[model];
  if (KIND == PS_REDUCE_PARETO) {
    // a frontier that outgrew the lists is left to the slow exact kernel that follows
    if (tid == 0) args.slow_path[model] = overflowed ? 1u : 0u;
    if (overflowed) return;
  }
  for (u32 ci = 0; ci < args.n_caps; ++ci) {
    const u64 cap = args.caps[ci];
    // Pareto: a tighter capacity keeps the head of the staircase (dominance only
    // ever looks at entries with smaller-or-equal memory).  Top-k runs once per
    // capacity, so everything in the list already fits.
    int n_cap = n_list;
    if (KIND == PS_REDUCE_PARETO) {
      int lo = 0, hi = n_list;
      while (lo < hi) { int mid = (lo + hi) >> 1; if (sh.a[mid] <= cap) lo = mid + 1; else hi = mid; }
      n_cap = lo;
    }
    const u32 cap_slot = (KIND == PS_REDUCE_PARETO) ? ci : args.cap_index;
    ps_front_entry* out = args.out + ((u64)model * args.n_caps_total + cap_slot) * args.max_entries;
    if (tid == 0) {
      args.counts[(u64)model * args.n_caps_total + cap_slot] =
          (KIND == PS_REDUCE_PARETO) ? (u32)n_cap : s_survivors;
      // a frontier that does not fit the caller's rows: its head is written, the count is the true one
      if (KIND == PS_REDUCE_PARETO && n_cap > (int)args.max_entries) atomicOr(args.status, ST_TRUNCATED);
    }
    const int n_emit = min(min(n_cap, (int)args.max_entries), KIND == PS_REDUCE_PARETO ? n_cap : (int)args.k_keep);
    for (int p = tid; p < (int)args.max_entries; p += MERGE_THREADS) {
      ps_front_entry e;
      e.mem = 0; e.comm = 0; e.host = 0; e.idx = 0; e.flags = 0; e.pad = 0;
      if (p < n_emit) {
        const u32 lidx = sh.i[p];
        const PointOut po = eval_local(sp, rec, lidx);
        const u64 comm = args.comm_kind == PS_COMM_PAPER ? po.comm_paper : po.comm_paper + po.comm_ext;
        const u64 list_mem = (KIND == PS_REDUCE_PARETO) ? sh.a[p] : sh.b[p];
        const u64 list_comm = (KIND == PS_REDUCE_PARETO) ? sh.b[p] : sh.a[p];
        if (po.mem != list_mem || comm != list_comm) atomicOr(args.status, ST_SELF_CHECK);
        e.mem = po.mem; e.comm = comm; e.host = po.host;
        e.idx = (u64)model * sp.ppm + lidx;
        e.flags = po.flags | PS_F_FEASIBLE;
      }
      out[p] = e;
    }
  }
}

}  // namespace

// ------------------------------------------------------------------ launchers
template <int KIND, int NM, bool HOST_LIMITED, bool FAST, bool SKIP, bool MANY = false>
static cudaError_t launch_sweep_p(const SpaceDev& sp, const SweepArgs& a, u32 n_chunks, cudaStream_t stream) {
  constexpr int WARPS = KIND == PS_REDUCE_PARETO ? SWEEP_WARPS_PARETO : (MANY ? SWEEP_WARPS_TOPK_MANY : SWEEP_WARPS_TOPK);
  constexpr int MIN_BLOCKS = KIND == PS_REDUCE_PARETO ? SWEEP_BLOCKS_PARETO
                                                      : (MANY ? SWEEP_BLOCKS_TOPK_MANY : SWEEP_BLOCKS_TOPK);
  dim3 grid(n_chunks, sp.n_models);
  const size_t smem = sizeof(SweepShared<WARPS>);
  cudaError_t e = cudaFuncSetAttribute(k_sweep<KIND, NM, WARPS, MIN_BLOCKS, HOST_LIMITED, FAST, SKIP>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  k_sweep<KIND, NM, WARPS, MIN_BLOCKS, HOST_LIMITED, FAST, SKIP><<<grid, WARPS * 32, smem, stream>>>(sp, a);
  return cudaGetLastError();
}

template <int KIND, int NM>
static cudaError_t launch_sweep_t(const SpaceDev& sp, const SweepArgs& a, u32 n_chunks, cudaStream_t stream) {
  const bool host_limited = a.host_cap < ((u64)1 << 62);
  // the fast case: powers of two everywhere, every byte count exact in a double
  if (sp.all_pow2 && sp.all_small && sp.repl == 1 && a.cap_max < ((u64)1 << 53) - 1) {
    if (a.skip_rejected)
      return host_limited ? launch_sweep_p<KIND, NM, true, true, true>(sp, a, n_chunks, stream)
                          : launch_sweep_p<KIND, NM, false, true, true>(sp, a, n_chunks, stream);
    if (KIND == PS_REDUCE_TOPK && a.many_models)
      return host_limited ? launch_sweep_p<KIND, NM, true, true, false, KIND == PS_REDUCE_TOPK>(sp, a, n_chunks, stream)
                          : launch_sweep_p<KIND, NM, false, true, false, KIND == PS_REDUCE_TOPK>(sp, a, n_chunks, stream);
    return host_limited ? launch_sweep_p<KIND, NM, true, true, false>(sp, a, n_chunks, stream)
                        : launch_sweep_p<KIND, NM, false, true, false>(sp, a, n_chunks, stream);
  }
  return host_limited ? launch_sweep_p<KIND, NM, true, false, true>(sp, a, n_chunks, stream)
                      : launch_sweep_p<KIND, NM, false, false, true>(sp, a, n_chunks, stream);
}

template <int KIND>
static cudaError_t launch_sweep_k(const SpaceDev& sp, const SweepArgs& a, u32 n_chunks, cudaStream_t stream) {
  switch (sp.nm) {
    case 1: return launch_sweep_t<KIND, 1>(sp, a, n_chunks, stream);
    case 2: return launch_sweep_t<KIND, 2>(sp, a, n_chunks, stream);
    case 3: return launch_sweep_t<KIND, 3>(sp, a, n_chunks, stream);
    case 4: return launch_sweep_t<KIND, 4>(sp, a, n_chunks, stream);
    default: return launch_sweep_t<KIND, 5>(sp, a, n_chunks, stream);
  }
}

cudaError_t launch_sweep(int kind, const SpaceDev& sp, const SweepArgs& a, u32 n_chunks,
                         cudaStream_t stream) {
  return kind == PS_REDUCE_PARETO ? launch_sweep_k<PS_REDUCE_PARETO>(sp, a, n_chunks, stream)
                                  : launch_sweep_k<PS_REDUCE_TOPK>(sp, a, n_chunks, stream);
}

cudaError_t launch_sweep_merge(int kind, const SpaceDev& sp, const MergeArgs& a, cudaStream_t stream) {
  size_t smem = sizeof(MergeShared);
  cudaError_t e;
  if (kind == PS_REDUCE_PARETO) {
    e = cudaFuncSetAttribute(k_sweep_merge<PS_REDUCE_PARETO>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep_merge<PS_REDUCE_PARETO><<<sp.n_models, MERGE_THREADS, smem, stream>>>(sp, a);
    k_frontier_by_definition<<<sp.n_models, MERGE_THREADS, 0, stream>>>(sp, a);
  } else {
    e = cudaFuncSetAttribute(k_sweep_merge<PS_REDUCE_TOPK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep_merge<PS_REDUCE_TOPK><<<sp.n_models, MERGE_THREADS, smem, stream>>>(sp, a);
  }
  return cudaGetLastError();
}

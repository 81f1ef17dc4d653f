// Small kernels: model-table derivation, single-point evaluation, integer-pipe
// microbenchmark.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

// Section 2.1: P = 12 L H^2 + V H; Definition 3: unit = 12 H^2 elements;
// Remark 1: byte widths.  Activations of one replica (the paper gives no
// formula; this is the per-layer count of the selective-recomputation analysis
// it cites for sequence parallelism): 34 S b H + 5 a S^2 b bytes stored,
// 2 S b H with full checkpointing.
__global__ void k_model_derive(const ps_model_shape* __restrict__ shapes, ModelRec* __restrict__ recs,
                               u32 n, u32* status) {
  const u32 i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  // 48-byte shape as three 16-byte loads
  ps_model_shape s;
  {
    const uint4* src = reinterpret_cast<const uint4*>(shapes + i);
    uint4* dst = reinterpret_cast<uint4*>(&s);
    dst[0] = __ldg(src); dst[1] = __ldg(src + 1); dst[2] = __ldg(src + 2);
  }
  bool ok = s.layers >= 1 && s.layers <= (1u << 10) && s.hidden >= 1 && s.hidden <= (1u << 16) &&
            s.heads >= 1 && s.heads <= (1u << 16) && s.vocab >= 1 && s.vocab <= (1u << 24) &&
            s.seq >= 1 && s.seq <= (1u << 17) && s.micro_batch >= 1 && s.micro_batch <= (1u << 10) &&
            s.w_param >= 1 && s.w_param <= 16 && s.w_grad >= 1 && s.w_grad <= 16 &&
            s.w_opt >= 1 && s.w_opt <= 16 && s.w_act >= 1 && s.w_act <= 16;
  ModelRec r;
  const u64 L = s.layers, H = s.hidden, V = s.vocab, S = s.seq, b = s.micro_batch, a = s.heads;
  r.P = s.param_elems_override ? s.param_elems_override : 12 * L * H * H + V * H;
  r.unit = s.unit_from_shape ? 12 * H * H : 0;
  r.Sbh = S * b * H;                              // <= 2^43 here; supported up to 2^40
  ok = ok && r.Sbh <= ((u64)1 << 40);
  // per-layer activation bytes; 5 a S^2 b can reach 2^63, so bound it first
  const u64 attn_unit = a * S;                    // <= 2^33
  const u64 attn_rest = S * b;                    // <= 2^27
  ok = ok && attn_unit <= (((u64)1 << 58) / 5) / attn_rest;
  u64 per_layer = 0, per_layer_ckpt = 0;
  if (ok && s.act_enabled) {
    per_layer = 34 * r.Sbh + 5 * attn_unit * attn_rest;
    per_layer_ckpt = 2 * r.Sbh;
    ok = ok && per_layer <= ((u64)1 << 58) / L;
  }
  ok = ok && r.P >= 1 && r.P <= ((u64)1 << 46);
  r.A[0] = ok ? L * per_layer : 0;
  r.A[1] = ok ? L * per_layer_ckpt : 0;
  r.UA[0] = ok ? per_layer : 0;
  r.UA[1] = ok ? per_layer_ckpt : 0;
  r.L = s.layers;
  r.heads = s.heads;
  r.wT = s.w_param; r.wO = s.w_opt; r.wG = s.w_grad; r.wA = s.w_act;
  r.ok = ok ? 1 : 0;
  r.pad[0] = r.pad[1] = r.pad[2] = 0;
  if (!ok) {
    // keep every later division and product harmless
    r.P = 1; r.unit = 0; r.Sbh = 1; r.L = 1; r.heads = 1;
    r.wT = r.wO = r.wG = r.wA = 1;
    atomicOr(status, ST_BAD_SHAPE);
  }
  recs[i] = r;
}

__global__ void k_check_point(const ModelRec* rec, Fact f, u32 v, u32 tau, u32 code_dp,
                              u32 tp_max_valid, u32 tp_coll, u32 axis_form, u32 comm_kind,
                              u64 cap_bytes, ps_front_entry* out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const u32 th = code_dp % 5, om = (code_dp / 5) % 5, gr = (code_dp / 25) % 5, ac = (code_dp / 125) % 5;
  const PointOut p = eval_point(*rec, f, v, tau, th, om, gr, ac, tp_max_valid, tp_coll, axis_form != 0);
  ps_front_entry e;
  e.mem = p.mem;
  e.comm = comm_kind == PS_COMM_PAPER ? p.comm_paper : p.comm_paper + p.comm_ext;
  e.host = p.host;
  e.idx = 0;
  e.flags = p.flags | (p.mem <= cap_bytes ? PS_F_FEASIBLE : 0);
  e.pad = 0;
  *out = e;
}

// Division of a device count by a small tensor degree t without dividing: with
// magic[t] = ceil(2^32 / t) the high word of n * magic[t] is floor(n / t) whenever
// n * t < 2^32 (the error of the magic, below t / 2^32 per unit of n, then stays
// below 1 / t).  Filled on the host for t <= SELECT_MAGIC_MAX; device counts up to
// 2^24 qualify.
constexpr u32 SELECT_MAGIC_MAX = 64;
struct SelectMagic {
  u32 m[SELECT_MAGIC_MAX + 1];
  double inv[SELECT_MAGIC_MAX + 1];   // 1 / t, correctly rounded
};

// floor(a / d) from a reciprocal of d that is correct to the last bit: for a < 2^52
// the product is off by less than one, so its integer part is the quotient or a
// neighbour of it, and the remainder says which.  One code path for every lane.
__device__ __forceinline__ u64 div_by_reciprocal(u64 a, u32 d, double recip) {
  if (a >= ((u64)1 << 52)) return a / d;
  u64 q = (u64)__double2ll_rz((double)(long long)a * recip);
  const long long rem = (long long)(a - q * d);
  if (rem < 0) --q;
  else if (rem >= (long long)d) ++q;
  return q;
}

// the largest t <= tp_degree that divides n
__device__ __forceinline__ u32 largest_tensor_degree(u32 n, u32 tp_degree, const SelectMagic& magic) {
  const u32 top = min(tp_degree, n);
  if (tp_degree <= SELECT_MAGIC_MAX && n <= (1u << 24)) {
    u32 best = 1;
    for (u32 t = 2; t <= tp_degree; ++t) {               // the same trip count for every lane
      const u32 q = __umulhi(n, magic.m[t]);
      if (q * t == n && t <= top) best = t;
    }
    return best;
  }
  for (u32 t = top; t > 1; --t)
    if (n % t == 0) return t;
  return 1;
}

// 128-bit unsigned integers as four 32-bit limbs, for products of a 64-bit count
// with one or two factors of at most 32 bits (a generic 128 x 128 multiplication
// costs several times more).
struct Wide {
  u32 w[4];
};
__device__ __forceinline__ Wide wide_mul(u64 a, u32 k) {
  const u64 p0 = (u64)(u32)a * k;
  const u64 p1 = (u64)(u32)(a >> 32) * k + (p0 >> 32);
  return Wide{{(u32)p0, (u32)p1, (u32)(p1 >> 32), 0u}};
}
__device__ __forceinline__ Wide wide_mul(const Wide& a, u32 k) {      // a below 2^96
  const u64 q0 = (u64)a.w[0] * k;
  const u64 q1 = (u64)a.w[1] * k + (q0 >> 32);
  const u64 q2 = (u64)a.w[2] * k + (q1 >> 32);
  return Wide{{(u32)q0, (u32)q1, (u32)q2, (u32)(q2 >> 32)}};
}
__device__ __forceinline__ bool wide_less(const Wide& a, const Wide& b) {
  const u64 ah = ((u64)a.w[3] << 32) | a.w[2], al = ((u64)a.w[1] << 32) | a.w[0];
  const u64 bh = ((u64)b.w[3] << 32) | b.w[2], bl = ((u64)b.w[1] << 32) | b.w[0];
  return ah < bh || (ah == bh && al < bl);
}

// Algorithm 1 for one query.  Thresholds are rationals; the comparisons are
// carried out exactly in 128-bit integers.
__device__ __forceinline__ ps_select_result select_one(const ps_select_query& s, u32 head_num,
                                                       u32 head_den, u32 layer_num, u32 layer_den,
                                                       u32 tp_degree, const SelectMagic& magic) {
  const u32 wsum = (u32)s.w_param + s.w_grad + s.w_opt;
  const Wide m_model = wide_mul(wide_mul(s.param_elems, wsum), head_den);     // M_model * head_den
  const Wide budget = wide_mul(s.device_bytes, head_num);                      // headroom * M_d, times head_den
  u32 branch, T = 1, code = 32;                                // ZeRO-3 unless data parallel fits
  if (wide_less(m_model, budget)) {
    branch = 0; code = 0;
  } else if (wide_less(m_model, wide_mul(budget, s.n_devices))) {
    branch = 1;
  } else {
    const Wide layer = wide_mul(wide_mul(s.layer_elems, wsum), layer_den);
    if (s.fast_interconnect && wide_less(wide_mul(s.device_bytes, layer_num), layer)) {
      branch = 2;
      T = largest_tensor_degree(s.n_devices, tp_degree, magic);
    } else {
      branch = 3;
    }
  }
  // Theorem 1 and Theorem 2 for the choice, written out for the two specifications
  // the algorithm can return (no activations, no pipeline axis): with E = ceil(P / T)
  // elements per tensor rank over D = N / T replicas,
  //   data parallel (R,R,R,R), T = 1:  bytes (w_T + w_O + w_G) P,  volume 2 x w_G
  //   ZeRO-3 (S*,S,S,R):               bytes (w_T + w_O + w_G) ceil(E / D) + w_T ceil(unit / T),
  //                                    volume x w_G + 2 x w_T
  // where x = E - floor(E / D) is the ring volume in elements (Section 2.3).
  // T is 1 or a small divisor of the device count: the divisions by it use the
  // host's tables where they reach (one path for all lanes of a warp)
  u32 D = s.n_devices;
  u64 E = s.param_elems, unit_t = s.layer_elems;
  if (T > 1) {
    if (T <= SELECT_MAGIC_MAX && s.n_devices <= (1u << 24)) {
      D = __umulhi(s.n_devices, magic.m[T]);
      E = div_by_reciprocal(s.param_elems + (T - 1), T, magic.inv[T]);
      unit_t = div_by_reciprocal(s.layer_elems + (T - 1), T, magic.inv[T]);
    } else {
      D = s.n_devices / T;
      E = div_ceil(s.param_elems, T);
      unit_t = div_ceil(s.layer_elems, T);
    }
  }
  const u64 quot = div_by_reciprocal(E, D, __drcp_rn((double)D));
  const u64 x = E - quot;
  u64 mem, comm;
  if (code == 0) {
    mem = (u64)wsum * E;
    comm = 2 * x * s.w_grad;
  } else {
    const u64 shard = quot + ((quot * D != E) ? 1 : 0);
    mem = (u64)wsum * shard + (u64)s.w_param * unit_t;
    comm = x * s.w_grad + 2 * x * s.w_param;
  }
  ps_select_result o;
  o.mem = mem; o.comm = comm; o.branch = branch; o.T = T; o.code_dp = code;
  o.flags = mem <= s.device_bytes ? PS_F_FEASIBLE : 0;
  return o;
}

// SELECT_PER_THREAD queries per thread, SELECT_THREADS apart, all of their 16-byte
// loads in flight before any arithmetic: the kernel streams 64 bytes per query, read
// once and written once (streaming loads and stores, nothing is reused).
#ifndef SELECT_THREADS_PER_BLOCK
#define SELECT_THREADS_PER_BLOCK 128
#endif
#ifndef SELECT_QUERIES_PER_THREAD
#define SELECT_QUERIES_PER_THREAD 2
#endif
// resident blocks per SM the kernel is compiled for: 12 x 128 threads caps it at 40
// registers, and a kernel that streams needs the warps more than the registers
#ifndef SELECT_MIN_BLOCKS
#define SELECT_MIN_BLOCKS 12
#endif
constexpr int SELECT_THREADS = SELECT_THREADS_PER_BLOCK;
constexpr int SELECT_PER_THREAD = SELECT_QUERIES_PER_THREAD;
__global__ void __launch_bounds__(SELECT_THREADS, SELECT_MIN_BLOCKS) k_select(const ps_select_query* __restrict__ q, u64 n,
                                                           u32 head_num, u32 head_den, u32 layer_num,
                                                           u32 layer_den, u32 tp_degree, SelectMagic magic,
                                                           ps_select_result* __restrict__ out) {
  const u64 first = (u64)blockIdx.x * (SELECT_PER_THREAD * SELECT_THREADS) + threadIdx.x;
  ps_select_query s[SELECT_PER_THREAD];
#pragma unroll
  for (int j = 0; j < SELECT_PER_THREAD; ++j) {
    const u64 i = first + (u64)j * SELECT_THREADS;
    if (i < n) {
      const uint4* src = reinterpret_cast<const uint4*>(q + i);
      uint4* dst = reinterpret_cast<uint4*>(&s[j]);
      dst[0] = __ldcs(src); dst[1] = __ldcs(src + 1);
    }
  }
#pragma unroll
  for (int j = 0; j < SELECT_PER_THREAD; ++j) {
    const u64 i = first + (u64)j * SELECT_THREADS;
    if (i < n) {
      const ps_select_result o = select_one(s[j], head_num, head_den, layer_num, layer_den, tp_degree, magic);
      uint4* dst = reinterpret_cast<uint4*>(out + i);
      const uint4* src = reinterpret_cast<const uint4*>(&o);
      __stcs(dst, src[0]); __stcs(dst + 1, src[1]);
    }
  }
}

// Algorithm 1's choice for every model of a space, as a point of the space, against
// the model's frontier (one thread per model).
__global__ void __launch_bounds__(128) k_select_compare(SpaceDev sp, u32 unit_begin, u32 unit_end, u32 N,
                                                        u64 device_bytes, u32 fast, u32 head_num, u32 head_den,
                                                        u32 layer_num, u32 layer_den, u32 tp_degree,
                                                        SelectMagic magic, u64 host_cap,
                                                        u32 require_flags, u32 comm_kind,
                                                        const ps_front_entry* __restrict__ frontier,
                                                        const u32* __restrict__ counts, u32 n_caps, u32 cap_index,
                                                        u32 max_entries, ps_select_compare_result* __restrict__ out) {
  const u32 model = blockIdx.x * blockDim.x + threadIdx.x;
  if (model >= sp.n_models) return;
  const ModelRec rec = sp.recs[model];
  ps_select_query q;
  q.param_elems = rec.P; q.layer_elems = rec.unit; q.device_bytes = device_bytes; q.n_devices = N;
  q.w_param = (uint8_t)rec.wT; q.w_grad = (uint8_t)rec.wG; q.w_opt = (uint8_t)rec.wO;
  q.fast_interconnect = (uint8_t)(fast ? 1 : 0);
  const ps_select_result pick = select_one(q, head_num, head_den, layer_num, layer_den, tp_degree, magic);
  ps_select_compare_result r;
  r.branch = pick.branch; r.T = pick.T; r.code_dp = pick.code_dp; r.pad = 0;
  u32 status = 0;
  // the choice as a point of the space: (N, T, K = 1), first variants, the code's modes as digits
  const u32 modes[4] = {pick.code_dp % 5, (pick.code_dp / 5) % 5, (pick.code_dp / 25) % 5, pick.code_dp / 125};
  u32 digits[4];
  bool in_space = true;
  for (int st = 0; st < 4; ++st) {
    digits[st] = 0xffffffffu;
    for (u32 d = 0; d < sp.nm; ++d)
      if (digit_mode(sp.modemap, d) == modes[st]) digits[st] = d;
    in_space = in_space && digits[st] != 0xffffffffu;
  }
  u32 unit = 0xffffffffu;
  for (u32 u = unit_begin; u < unit_end; ++u) {
    const Fact f = sp.facts[u];
    if (f.N == N && f.T == pick.T && f.K == 1) { unit = u; break; }
  }
  in_space = in_space && unit != 0xffffffffu;
  const Fact f = in_space ? sp.facts[unit] : Fact{N, pick.T, 1, N / pick.T};
  const PointOut po = eval_point(rec, f, 0, 0, modes[0], modes[1], modes[2], modes[3], sp.tp_max_valid, sp.tp_coll,
                                 true, sp.sstar_units, sp.accum, sp.repl);
  const u64 comm = comm_kind == PS_COMM_PAPER ? po.comm_paper : po.comm_paper + po.comm_ext;
  r.alg_mem = po.mem; r.alg_comm = comm;
  r.alg_idx = 0;
  if (in_space) {
    const u32 code = digits[0] + sp.nm * (digits[1] + sp.nm * (digits[2] + sp.nm * digits[3]));
    r.alg_idx = (u64)model * sp.ppm + (u64)unit * sp.nvt * sp.n_codes + code;
    status |= PS_SEL_IN_SPACE;
  }
  const bool fits = po.mem <= device_bytes;
  r.alg_flags = po.flags | (fits ? PS_F_FEASIBLE : 0);
  if (fits && po.host <= host_cap && (po.flags & require_flags) == require_flags) status |= PS_SEL_SURVIVOR;
  // the frontier of this model under this capacity
  const u32 count = counts[(u64)model * n_caps + cap_index];
  const ps_front_entry* fr = frontier + ((u64)model * n_caps + cap_index) * max_entries;
  const u32 written = count < max_entries ? count : max_entries;
  if (count == 0) status |= PS_SEL_FRONTIER_EMPTY;
  if (count > max_entries) status |= PS_SEL_FRONTIER_TRUNCATED;
  r.best_mem = 0; r.best_comm = 0; r.best_idx = 0;
  for (u32 e = 0; e < written; ++e) {
    const u64 m = fr[e].mem, c = fr[e].comm;
    if (m == po.mem && c == comm) status |= PS_SEL_ON_FRONTIER;
    else if (m <= po.mem && c <= comm) status |= PS_SEL_DOMINATED;
  }
  if (written) { r.best_mem = fr[written - 1].mem; r.best_comm = fr[written - 1].comm; r.best_idx = fr[written - 1].idx; }
  r.status = status;
  out[model] = r;
}

// 8 independent chains per thread; each round applies to every chain an add
// and an xor with loop-carried values the compiler cannot fold, so a round is
// 16 independent-across-chains 32-bit operations and a chain's operations are
// dependent (8 chains hide the pipe latency).
__global__ void __launch_bounds__(256) k_int_peak(u32 iters, u32* sink) {
  u32 c0 = threadIdx.x, c1 = c0 + 1, c2 = c0 + 2, c3 = c0 + 3, c4 = c0 + 4, c5 = c0 + 5,
      c6 = c0 + 6, c7 = c0 + 7;
  u32 k = blockIdx.x | 1u, m = (blockIdx.x << 7) | 5u;
  for (u32 it = 0; it < iters; ++it) {
#pragma unroll
    for (int r = 0; r < 8; ++r) {
      c0 += k; c1 += k; c2 += k; c3 += k; c4 += k; c5 += k; c6 += k; c7 += k;
      c0 ^= m; c1 ^= m; c2 ^= m; c3 ^= m; c4 ^= m; c5 ^= m; c6 ^= m; c7 ^= m;
    }
    k += it;
    m ^= k;
  }
  const u32 r = c0 ^ c1 ^ c2 ^ c3 ^ c4 ^ c5 ^ c6 ^ c7;
  if (r == 0x9e3779b9u) atomicAdd(sink, r);   // practically never; keeps the chains alive
  if (threadIdx.x == 0 && blockIdx.x == 0) atomicAdd(sink, r & 1u);
}

}  // namespace

cudaError_t launch_model_derive(const ps_model_shape* d_shapes, ModelRec* d_recs, u32 n, u32* status,
                                cudaStream_t stream) {
  k_model_derive<<<(n + 127) / 128, 128, 0, stream>>>(d_shapes, d_recs, n, status);
  return cudaGetLastError();
}

cudaError_t launch_check_point(const ModelRec* d_rec, Fact f, u32 v, u32 tau, u32 code_dp,
                               u32 tp_max_valid, u32 tp_coll, u32 axis_form, u32 comm_kind,
                               u64 cap_bytes, ps_front_entry* d_out, cudaStream_t stream) {
  k_check_point<<<1, 32, 0, stream>>>(d_rec, f, v, tau, code_dp, tp_max_valid, tp_coll, axis_form,
                                      comm_kind, cap_bytes, d_out);
  return cudaGetLastError();
}

static SelectMagic select_magic() {
  SelectMagic g;
  g.m[0] = g.m[1] = 0;
  g.inv[0] = g.inv[1] = 1.0;
  for (u32 t = 2; t <= SELECT_MAGIC_MAX; ++t) {
    g.m[t] = (u32)((((u64)1 << 32) + t - 1) / t);
    g.inv[t] = 1.0 / (double)t;
  }
  return g;
}

cudaError_t launch_select(const ps_select_query* d_q, u64 n, u32 head_num, u32 head_den, u32 layer_num,
                          u32 layer_den, u32 tp_degree, ps_select_result* d_out, cudaStream_t stream) {
  const u64 per_block = (u64)SELECT_PER_THREAD * SELECT_THREADS;
  k_select<<<(unsigned)((n + per_block - 1) / per_block), SELECT_THREADS, 0, stream>>>(
      d_q, n, head_num, head_den, layer_num, layer_den, tp_degree, select_magic(), d_out);
  return cudaGetLastError();
}

cudaError_t launch_int_peak(u32 blocks, u32 iters, u32* d_sink, cudaStream_t stream) {
  k_int_peak<<<blocks, 256, 0, stream>>>(iters, d_sink);
  return cudaGetLastError();
}

cudaError_t launch_select_compare(const SpaceDev& sp, u32 unit_begin, u32 unit_end, u32 N, u64 device_bytes, u32 fast,
                                  u32 head_num, u32 head_den, u32 layer_num, u32 layer_den, u32 tp_degree,
                                  u64 host_cap, u32 require_flags, u32 comm_kind, const ps_front_entry* d_frontier,
                                  const u32* d_counts, u32 n_caps, u32 cap_index, u32 max_entries,
                                  ps_select_compare_result* d_out, cudaStream_t stream) {
  k_select_compare<<<(sp.n_models + 127) / 128, 128, 0, stream>>>(
      sp, unit_begin, unit_end, N, device_bytes, fast, head_num, head_den, layer_num, layer_den, tp_degree,
      select_magic(), host_cap,
      require_flags, comm_kind, d_frontier, d_counts, n_caps, cap_index, max_entries, d_out);
  return cudaGetLastError();
}

// Fused sweep: enumerate -> evaluate -> filter -> reduce, nothing materialised.
//
// grid = (n_chunks, n_models).  A block owns one model and a contiguous range
// of its factorisations ("units"); its warps take units round-robin.  For a
// unit the warp computes the shard quantities once (all divisions), writes
// small per-mode tables to its shared-memory slice, and then walks the
// placement codes: a lane owns a (Theta, Omega, G) triple, keeps that triple's
// partial sums in registers and visits the activation variants and activation
// modes with adds, compares and selects only.
//
// Reductions.  Every warp keeps a private sorted list in shared memory
// (Pareto staircase or top-k), tests its candidates against it lane-parallel
// and inserts the few that pass warp-cooperatively.  At the end the block sorts
// the union of its warps' lists, prunes it and writes one partial list per
// block to global scratch; k_sweep_merge combines the partial lists of a model
// and emits entries, re-evaluating each emitted point from its index as a
// self-check.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

constexpr int WARPS = SWEEP_WARPS;
constexpr int THREADS = WARPS * 32;
constexpr int LIST_CAP = SWEEP_LIST_CAP;       // entries per warp list / per partial list
constexpr int BLOCK_CAP = WARPS * LIST_CAP;    // union of the warps' lists
constexpr u64 U64MAX = ~0ull;

// per-warp tables, rebuilt for every unit (all u64)
struct WarpTables {
  u64 mem[3][5];       // state (Theta, Omega, G) x mode: bytes of Theorem 1
  u64 c_theta[2][5];   // [update on shard][mode]: objective communication terms
  u64 c_omega[5];
  u64 c_grad[2][5];
  u64 act[4][5];       // variant (v, tau) x activation mode: bytes
  u64 act_host[4];     // host bytes when activations are offloaded
  u64 c_axis[4];       // tensor + pipeline traffic of the variant (0 if not in the objective)
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
};

// Pareto staircase: a = mem ascending, b = comm strictly descending.
// Is (m, c, idx) dominated by, or a later duplicate of, an entry?  Per lane.
__device__ __forceinline__ bool pareto_rejects(const WarpList& w, u64 m, u64 c, u32 idx) {
  int lo = 0, hi = w.n;
  while (lo < hi) {               // number of entries with mem <= m
    int mid = (lo + hi) >> 1;
    if (w.a[mid] <= m) lo = mid + 1; else hi = mid;
  }
  if (lo == 0) return false;
  u64 ec = w.b[lo - 1];           // smallest comm among entries with mem <= m
  if (ec < c) return true;
  if (ec > c) return false;
  return w.a[lo - 1] < m || w.i[lo - 1] < idx;
}

// warp-cooperative insertion; all lanes hold the same (m, c, idx)
__device__ __forceinline__ void pareto_insert(WarpList& w, u64 m, u64 c, u32 idx, int lane,
                                              u32* status) {
  constexpr int PER = LIST_CAP / 32;
  u64 ea[PER], eb[PER];
  u32 ei[PER];
  int below = 0, killed = 0;
  bool dominated = false;
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    int e = lane + 32 * k;
    bool valid = e < w.n;
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
  if (__any_sync(0xffffffffu, dominated)) { __syncwarp(); return; }
  int n_new = w.n - killed + 1;
  if (n_new > LIST_CAP) {
    if (lane == 0) atomicOr(status, ST_LIST_OVERFLOW);
    return;
  }
  __syncwarp();
  int shift = 1 - killed;                              // entries after the killed run move by this
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    int e = lane + 32 * k;
    if (e < w.n && e >= below + killed && shift != 0) {
      w.a[e + shift] = ea[k];
      w.b[e + shift] = eb[k];
      w.i[e + shift] = ei[k];
    }
  }
  if (lane == 0) { w.a[below] = m; w.b[below] = c; w.i[below] = idx; }
  w.n = n_new;
  __syncwarp();
}

// top-k list: keys ascending, at most k entries
__device__ __forceinline__ void topk_insert(WarpList& w, const Key& key, int k_keep, int lane,
                                            Key& threshold) {
  constexpr int PER = LIST_CAP / 32;
  Key e[PER];
  int below = 0;
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    int p = lane + 32 * k;
    bool valid = p < w.n;
    e[k].a = valid ? w.a[p] : U64MAX;
    e[k].b = valid ? w.b[p] : U64MAX;
    e[k].i = valid ? w.i[p] : 0xffffffffu;
    below += __popc(__ballot_sync(0xffffffffu, valid && key_less(e[k], key)));
  }
  if (below >= k_keep) return;                         // (cannot happen after the threshold test)
  __syncwarp();
  int n_new = min(w.n + 1, k_keep);
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    int p = lane + 32 * k;
    if (p < w.n && p >= below && p + 1 < k_keep) {
      w.a[p + 1] = e[k].a; w.b[p + 1] = e[k].b; w.i[p + 1] = e[k].i;
    }
  }
  if (lane == 0) { w.a[below] = key.a; w.b[below] = key.b; w.i[below] = key.i; }
  w.n = n_new;
  __syncwarp();
  if (w.n == k_keep) {
    threshold.a = w.a[k_keep - 1]; threshold.b = w.b[k_keep - 1]; threshold.i = w.i[k_keep - 1];
  }
}

// ------------------------------------------------------------------ block sort / prune
// Bitonic sort of n_pad (power of two) keys in shared memory by key_less.
__device__ void block_sort(u64* a, u64* b, u32* i, int n_pad, int tid, int n_threads) {
  for (int k = 2; k <= n_pad; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int p = tid; p < n_pad; p += n_threads) {
        int q = p ^ j;
        if (q > p) {
          Key x{a[p], b[p], i[p]}, y{a[q], b[q], i[q]};
          bool up = (p & k) == 0;
          if (key_less(y, x) == up) {
            a[p] = y.a; b[p] = y.b; i[p] = y.i;
            a[q] = x.a; b[q] = x.b; i[q] = x.i;
          }
        }
      }
      __syncthreads();
    }
  }
}

// After sorting by (mem, comm, idx): an entry is on the frontier iff its comm
// is below the comm of every earlier entry.  Keeps the frontier at the front,
// returns its length.  `scratch` holds >= n_threads u64 and n_threads int.
__device__ int block_pareto_prune(u64* a, u64* b, u32* i, int n, int tid, int n_threads,
                                  u64* smin, int* scount) {
  int per = (n + n_threads - 1) / n_threads;
  int lo = min(tid * per, n), hi = min(lo + per, n);
  u64 local = U64MAX;
  for (int p = lo; p < hi; ++p) local = min(local, b[p]);
  smin[tid] = local;
  __syncthreads();
  u64 before = U64MAX;                               // min comm of all entries before lo
  for (int t = 0; t < tid; ++t) before = min(before, smin[t]);
  int kept = 0;
  u64 run = before;
  for (int p = lo; p < hi; ++p) {
    if (b[p] < run) { ++kept; run = b[p]; }
  }
  scount[tid] = kept;
  __syncthreads();
  int offset = 0, total = 0;
  for (int t = 0; t < n_threads; ++t) {
    if (t < tid) offset += scount[t];
    total += scount[t];
  }
  // gather survivors into registers (at most `per`), then write after a barrier
  Key keep[SWEEP_MAX_PER_THREAD];
  int nk = 0;
  run = before;
  for (int p = lo; p < hi; ++p) {
    if (b[p] < run) { run = b[p]; keep[nk].a = a[p]; keep[nk].b = b[p]; keep[nk].i = i[p]; ++nk; }
  }
  __syncthreads();
  for (int k = 0; k < nk; ++k) { a[offset + k] = keep[k].a; b[offset + k] = keep[k].b; i[offset + k] = keep[k].i; }
  __syncthreads();
  return total;
}

__device__ __forceinline__ int next_pow2(int n) {
  int p = 1;
  while (p < n) p <<= 1;
  return p;
}

struct SweepShared {
  WarpTables tables[WARPS];
  u64 list_a[BLOCK_CAP];
  u64 list_b[BLOCK_CAP];
  u32 list_i[BLOCK_CAP];
  u64 merge_a[BLOCK_CAP];
  u64 merge_b[BLOCK_CAP];
  u32 merge_i[BLOCK_CAP];
  u64 smin[THREADS];
  int scount[THREADS];
  int warp_n[WARPS];
  u32 warp_survivors[WARPS];
  ModelRec rec;
};

// ------------------------------------------------------------------ the sweep
template <int KIND>
__global__ void __launch_bounds__(THREADS) k_sweep(SpaceDev sp, SweepArgs args) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  SweepShared& sh = *reinterpret_cast<SweepShared*>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const u32 model = blockIdx.y, chunk = blockIdx.x, n_chunks = gridDim.x;

  // stage the model record with 16-byte loads (6 x 16 B)
  if (tid < (int)(sizeof(ModelRec) / 16))
    reinterpret_cast<uint4*>(&sh.rec)[tid] = reinterpret_cast<const uint4*>(&sp.recs[model])[tid];
  __syncthreads();
  const ModelRec rec = sh.rec;

  WarpTables& tb = sh.tables[warp];
  WarpList list{sh.list_a + warp * LIST_CAP, sh.list_b + warp * LIST_CAP,
                sh.list_i + warp * LIST_CAP, 0};
  const int k_keep = (int)args.k_keep;
  Key threshold{U64MAX, U64MAX, 0xffffffffu};
  u32 survivors = 0;

  const u32 req = args.require_flags;
  const bool ext_in_objective = args.comm_kind == PS_COMM_PAPER_PLUS_EXT;
  const u32 per_unit = sp.nvt * sp.n_codes;
  const u32 u_begin = (u32)(((u64)chunk * sp.n_facts) / n_chunks);
  const u32 u_end = (u32)(((u64)(chunk + 1) * sp.n_facts) / n_chunks);

  for (u32 unit = u_begin + warp; unit < u_end; unit += WARPS) {
    const Fact f = sp.facts[unit];
    const UnitBase ub = unit_base(rec, f, sp.tp_max_valid, true);
    const u64 hostT = 3 * ub.sh * rec.wT, hostO = 2 * ub.sh * rec.wO, hostG = 2 * ub.sh * rec.wG;
    __syncwarp();
    if (lane < 5) {
      const u32 pi = lane;
      const u64 pe = mu_elems(pi, ub.E2, ub.sh, ub.u);
      tb.mem[0][pi] = rec.wT * pe;
      tb.mem[1][pi] = rec.wO * pe;
      tb.mem[2][pi] = rec.wG * pe;
      const u64 xT = ub.x * rec.wT, xO = ub.x * rec.wO, xG = ub.x * rec.wG;
      // Theorem 2's terms, plus (if asked for) the traffic it does not price
      u64 ct0 = (pi == PS_MODE_SG) ? 2 * xT : 0, ct1 = ct0, co = 0;
      u64 cg0 = (pi == PS_MODE_R) ? 2 * xG : (pi == PS_MODE_S ? xG : 0), cg1 = cg0;
      if (ext_in_objective) {
        if (pi == PS_MODE_O) { ct0 += 2 * xT; ct1 += 2 * xT; }
        if (pi == PS_MODE_R) ct1 += xT;                       // re-replicate updated shards
        if (pi == PS_MODE_SG) { cg0 += 2 * xG; cg1 += 2 * xG; co = xO; }
        if (pi == PS_MODE_M) { cg0 += 2 * xG; cg1 += xG; }
        if (pi == PS_MODE_O) { cg0 += xG; cg1 += xG; }
      }
      tb.c_theta[0][pi] = ct0; tb.c_theta[1][pi] = ct1;
      tb.c_omega[pi] = co;
      tb.c_grad[0][pi] = cg0; tb.c_grad[1][pi] = cg1;
      for (u32 v = 0; v < sp.nv; ++v)
        for (u32 tau = 0; tau < sp.nt; ++tau) {
          const ActBase ab = act_base(rec, f, v, tau);
          tb.act[v * sp.nt + tau][pi] = mu_elems(pi, ab.EA, ab.shA, ab.uA);
          if (pi == 0) {
            tb.act_host[v * sp.nt + tau] = 2 * ab.EA;
            tb.c_axis[v * sp.nt + tau] =
                ext_in_objective ? model_axis_traffic(rec, f, ub, tau, sp.tp_coll) : 0;
          }
        }
    }
    __syncwarp();

    const u32 unit_first = unit * per_unit;      // index of the unit's first point in the model
    for (u32 t0 = 0; t0 < sp.n3; t0 += 32) {
      const u32 t = t0 + lane;
      const bool live = t < sp.n3;
      const u32 tt = live ? t : 0;
      const u32 dth = tt % sp.nm, dom = (tt / sp.nm) % sp.nm, dgr = tt / (sp.nm * sp.nm);
      const u32 th = digit_mode(sp.modemap, dth), om = digit_mode(sp.modemap, dom),
                gr = digit_mode(sp.modemap, dgr);
      const u32 on_shard = in_set(SET_UPDATE_ON_SHARD, om) ? 1 : 0;
      const u64 mem3 = tb.mem[0][th] + tb.mem[1][om] + tb.mem[2][gr];
      const u64 comm3 = tb.c_theta[on_shard][th] + tb.c_omega[om] + tb.c_grad[on_shard][gr];
      const u64 host3 = (th == PS_MODE_O ? hostT : 0) + (om == PS_MODE_O ? hostO : 0) +
                        (gr == PS_MODE_O ? hostG : 0);
      // which activation modes give a point that has every required flag
      u32 ok_modes = 0;
      if (live) {
        // data-axis traffic beyond Theorem 2 (needed for the paper-priced flag only)
        const bool ext0 = ub.d1 || !((th == PS_MODE_O) || (th == PS_MODE_R && on_shard) ||
                                     in_set((1u << PS_MODE_SG) | SET_M_OR_O, gr) || om == PS_MODE_SG);
        for (u32 da = 0; da < sp.nm; ++da) {
          const u32 ac = digit_mode(sp.modemap, da);
          const u32 fl = point_flags(th, om, gr, ac, ub.d1, ub.cv, ext0);
          if ((fl & req) == req) ok_modes |= 1u << da;
        }
      }
      const bool host3_ok = host3 <= args.host_cap;

      for (u32 vt = 0; vt < sp.nvt; ++vt) {
        const u64 comm = comm3 + tb.c_axis[vt];
        const u32 vt_first = unit_first + vt * sp.n_codes + tt;   // + da * n3
        if (KIND == PS_REDUCE_PARETO) {
          // same communication for the nm activation modes: the smallest memory
          // (first on ties) is the only one that can be on the frontier
          u64 best = U64MAX;
          u32 best_da = 0;
          for (u32 da = 0; da < sp.nm; ++da) {
            const u32 ac = digit_mode(sp.modemap, da);
            const u64 mem = mem3 + tb.act[vt][ac];
            const bool host_ok = (ac == PS_MODE_O) ? (host3 + tb.act_host[vt] <= args.host_cap) : host3_ok;
            if (((ok_modes >> da) & 1u) && host_ok && mem < best) { best = mem; best_da = da; }
          }
          const u32 idx = vt_first + best_da * sp.n3;
          bool cand = best <= args.cap_max;
          if (cand) cand = !pareto_rejects(list, best, comm, idx);
          u32 pending = __ballot_sync(0xffffffffu, cand);
          while (pending) {
            const int src = __ffs(pending) - 1;
            pending &= pending - 1;
            const u64 m = __shfl_sync(0xffffffffu, best, src);
            const u64 c = __shfl_sync(0xffffffffu, comm, src);
            const u32 ix = __shfl_sync(0xffffffffu, idx, src);
            pareto_insert(list, m, c, ix, lane, args.status);
          }
        } else {
          for (u32 da = 0; da < sp.nm; ++da) {
            const u32 ac = digit_mode(sp.modemap, da);
            const u64 mem = mem3 + tb.act[vt][ac];
            const bool host_ok = (ac == PS_MODE_O) ? (host3 + tb.act_host[vt] <= args.host_cap) : host3_ok;
            const bool pass = ((ok_modes >> da) & 1u) && host_ok && mem <= args.cap_max;
            survivors += pass ? 1 : 0;
            const Key key{comm, mem, vt_first + da * sp.n3};
            u32 pending = __ballot_sync(0xffffffffu, pass && key_less(key, threshold));
            while (pending) {
              const int src = __ffs(pending) - 1;
              pending &= pending - 1;
              Key k;
              k.a = __shfl_sync(0xffffffffu, key.a, src);
              k.b = __shfl_sync(0xffffffffu, key.b, src);
              k.i = __shfl_sync(0xffffffffu, key.i, src);
              if (key_less(k, threshold)) topk_insert(list, k, k_keep, lane, threshold);
            }
          }
        }
      }
    }
  }

  // ---- block-level merge of the warps' lists
  for (int o = 16; o > 0; o >>= 1) survivors += __shfl_xor_sync(0xffffffffu, survivors, o);
  if (lane == 0) { sh.warp_n[warp] = list.n; sh.warp_survivors[warp] = survivors; }
  __syncthreads();
  int total = 0, my_off = 0;
  for (int w = 0; w < WARPS; ++w) {
    if (w < warp) my_off += sh.warp_n[w];
    total += sh.warp_n[w];
  }
  const int n_pad = next_pow2(max(total, 1));
  for (int p = lane; p < list.n; p += 32) {
    sh.merge_a[my_off + p] = list.a[p]; sh.merge_b[my_off + p] = list.b[p]; sh.merge_i[my_off + p] = list.i[p];
  }
  for (int p = total + tid; p < n_pad; p += THREADS) {
    sh.merge_a[p] = U64MAX; sh.merge_b[p] = U64MAX; sh.merge_i[p] = 0xffffffffu;
  }
  __syncthreads();
  block_sort(sh.merge_a, sh.merge_b, sh.merge_i, n_pad, tid, THREADS);
  int n_out;
  if (KIND == PS_REDUCE_PARETO) {
    n_out = block_pareto_prune(sh.merge_a, sh.merge_b, sh.merge_i, total, tid, THREADS, sh.smin, sh.scount);
    if (n_out > LIST_CAP) {
      if (tid == 0) atomicOr(args.status, ST_LIST_OVERFLOW);
      n_out = LIST_CAP;
    }
  } else {
    n_out = min(total, k_keep);
  }
  const u64 slot = (u64)model * n_chunks + chunk;
  PartialEntry* dst = args.partial + slot * LIST_CAP;
  for (int p = tid; p < n_out; p += THREADS) {
    PartialEntry e;
    e.a = sh.merge_a[p]; e.b = sh.merge_b[p]; e.i = sh.merge_i[p]; e.pad = 0;
    dst[p] = e;
  }
  if (tid == 0) {
    u32 s = 0;
    for (int w = 0; w < WARPS; ++w) s += sh.warp_survivors[w];
    args.partial_n[slot] = make_uint2((u32)n_out, s);
  }
}

// ------------------------------------------------------------------ merge + emit
// One block per model: combine the n_chunks partial lists, then write the
// entries of every capacity.  Each emitted point is evaluated again from its
// index (host bytes and flags come from there; mem and comm must agree).
struct MergeShared {
  u64 a[MERGE_CAP];
  u64 b[MERGE_CAP];
  u32 i[MERGE_CAP];
  u64 smin[THREADS];
  int scount[THREADS];
};

template <int KIND>
__global__ void __launch_bounds__(THREADS) k_sweep_merge(SpaceDev sp, MergeArgs args) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  MergeShared& sh = *reinterpret_cast<MergeShared*>(smem_raw);
  const int tid = threadIdx.x;
  const u32 model = blockIdx.x;
  const u32 n_chunks = args.n_chunks;
  __shared__ int s_off[SWEEP_MAX_CHUNKS + 1];
  __shared__ u32 s_survivors;
  if (tid == 0) {
    int off = 0;
    u32 surv = 0;
    for (u32 c = 0; c < n_chunks; ++c) {
      s_off[c] = off;
      uint2 pn = args.partial_n[(u64)model * n_chunks + c];
      off += (int)pn.x;
      surv += pn.y;
    }
    s_off[n_chunks] = off;
    s_survivors = surv;
  }
  __syncthreads();
  const int total = s_off[n_chunks];
  for (u32 c = 0; c < n_chunks; ++c) {
    const PartialEntry* src = args.partial + ((u64)model * n_chunks + c) * LIST_CAP;
    const int n = s_off[c + 1] - s_off[c];
    for (int p = tid; p < n; p += THREADS) {
      PartialEntry e = src[p];
      sh.a[s_off[c] + p] = e.a; sh.b[s_off[c] + p] = e.b; sh.i[s_off[c] + p] = e.i;
    }
  }
  const int n_pad = next_pow2(max(total, 1));
  for (int p = total + tid; p < n_pad; p += THREADS) { sh.a[p] = U64MAX; sh.b[p] = U64MAX; sh.i[p] = 0xffffffffu; }
  __syncthreads();
  block_sort(sh.a, sh.b, sh.i, n_pad, tid, THREADS);
  int n_list = total;
  if (KIND == PS_REDUCE_PARETO)
    n_list = block_pareto_prune(sh.a, sh.b, sh.i, total, tid, THREADS, sh.smin, sh.scount);

  const ModelRec rec = sp.recs[model];
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
    if (tid == 0)
      args.counts[(u64)model * args.n_caps_total + cap_slot] =
          (KIND == PS_REDUCE_PARETO) ? (u32)n_cap : s_survivors;
    const int n_emit = min(min(n_cap, (int)args.max_entries), KIND == PS_REDUCE_PARETO ? n_cap : (int)args.k_keep);
    for (int p = tid; p < (int)args.max_entries; p += THREADS) {
      ps_front_entry e;
      e.mem = 0; e.comm = 0; e.host = 0; e.idx = 0; e.flags = 0; e.pad = 0;
      if (p < n_emit) {
        const u32 lidx = sh.i[p];
        const LocalPoint lp = decode_local(sp, lidx);
        const Fact f = sp.facts[lp.unit];
        const PointOut po = eval_point(rec, f, lp.v, lp.tau, digit_mode(sp.modemap, lp.dth),
                                       digit_mode(sp.modemap, lp.dom), digit_mode(sp.modemap, lp.dgr),
                                       digit_mode(sp.modemap, lp.dac), sp.tp_max_valid, sp.tp_coll, true);
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
size_t sweep_shared_bytes() { return sizeof(SweepShared); }
size_t merge_shared_bytes() { return sizeof(MergeShared); }

cudaError_t launch_sweep(int kind, const SpaceDev& sp, const SweepArgs& a, u32 n_chunks,
                         cudaStream_t stream) {
  dim3 grid(n_chunks, sp.n_models);
  size_t smem = sizeof(SweepShared);
  cudaError_t e;
  if (kind == PS_REDUCE_PARETO) {
    e = cudaFuncSetAttribute(k_sweep<PS_REDUCE_PARETO>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep<PS_REDUCE_PARETO><<<grid, THREADS, smem, stream>>>(sp, a);
  } else {
    e = cudaFuncSetAttribute(k_sweep<PS_REDUCE_TOPK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep<PS_REDUCE_TOPK><<<grid, THREADS, smem, stream>>>(sp, a);
  }
  return cudaGetLastError();
}

cudaError_t launch_sweep_merge(int kind, const SpaceDev& sp, const MergeArgs& a, cudaStream_t stream) {
  size_t smem = sizeof(MergeShared);
  cudaError_t e;
  if (kind == PS_REDUCE_PARETO) {
    e = cudaFuncSetAttribute(k_sweep_merge<PS_REDUCE_PARETO>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep_merge<PS_REDUCE_PARETO><<<sp.n_models, THREADS, smem, stream>>>(sp, a);
  } else {
    e = cudaFuncSetAttribute(k_sweep_merge<PS_REDUCE_TOPK>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    k_sweep_merge<PS_REDUCE_TOPK><<<sp.n_models, THREADS, smem, stream>>>(sp, a);
  }
  return cudaGetLastError();
}

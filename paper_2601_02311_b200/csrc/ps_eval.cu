// Batch evaluation of a window of the space: materialise every output, or
// filter and compact the survivors in index order.
//
// A "group" is the n_codes consecutive points that share (model, factorisation,
// activation variant, tensor-axis variant).  One warp owns one group: it
// computes the group's shard quantities once, builds two pair tables in its
// shared-memory slice -- (Theta, Omega) digits and (G, A) digits, each entry
// holding the pair's mem / comm_paper / comm_ext / host contributions and flag
// bits -- and then every point is two table reads, a few adds and the flag
// logic.  Lanes take consecutive codes, so all output stores are coalesced.
//
// Compaction is count -> scan -> write: the count pass stores the survivors of
// each warp's group, a single-block scan turns them into offsets, the write
// pass evaluates again and places survivors with ballot/popc prefix sums.
// Output order is the index order, so the result is unique.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

constexpr int THREADS = EVAL_THREADS;
constexpr int WARPS = THREADS / 32;

// internal flag bits of the pair tables (above the public 13 bits)
enum : u32 {
  X_ON_SHARD = 1u << 16,   // update committed on a shard (Omega in S, S*, O)
  X_M_OR_O = 1u << 17,     // some state materialised or offloaded
  X_G_FULL = 1u << 18,     // gradients delivered in full (G in R, S*, M)
  X_G_IS_M = 1u << 19,
  X_D1 = 1u << 20,
  X_PUBLIC = 0x1FFFu
};

struct __align__(16) PairEntry {
  u64 mem, comm_paper, comm_ext, host;
};

struct WarpGroupTables {
  PairEntry p1[25];   // index dth + nm*dom
  PairEntry p2[25];   // index dgr + nm*dac
  u32 f1[25];
  u32 f2[25];
};

struct GroupConst {
  u64 xG;        // ring bytes of G: added once more when G is materialised and the update is on the full range
  u64 c_axis;    // tensor + pipeline traffic
  u32 fbase;     // composition bits, X_D1
  u64 lo, hi;    // window of this group's points, as offsets into the space
  u64 group_first;
};

// build the tables of global group `g`; returns false if the group lies outside the window
__device__ __forceinline__ bool build_group(const SpaceDev& sp, const EvalArgs& a, u64 g, int lane,
                                            WarpGroupTables& tb, GroupConst& gc) {
  const u64 gfirst = g * sp.n_codes;
  gc.group_first = gfirst;
  gc.lo = max(gfirst, a.first);
  gc.hi = min(gfirst + sp.n_codes, a.first + a.count);
  if (gc.lo >= gc.hi) return false;
  const u64 groups_per_model = (u64)sp.n_facts * sp.nvt;
  const u32 model = (u32)(g / groups_per_model);
  const u32 gl = (u32)(g - (u64)model * groups_per_model);
  const u32 unit = gl / sp.nvt, vt = gl - unit * sp.nvt;
  const u32 v = vt / sp.nt, tau = vt - v * sp.nt;
  // the model record: 96 bytes as six 16-byte loads through the read-only path
  ModelRec rec;
  {
    const uint4* src = reinterpret_cast<const uint4*>(&sp.recs[model]);
    uint4* dst = reinterpret_cast<uint4*>(&rec);
#pragma unroll
    for (int k = 0; k < 6; ++k) dst[k] = __ldg(src + k);
  }
  const Fact f = sp.facts[unit];
  const UnitBase ub = unit_base(rec, f, sp.tp_max_valid, true);
  const ActBase ab = act_base(rec, f, v, tau);
  const u64 xT = ub.x * rec.wT, xO = ub.x * rec.wO, xG = ub.x * rec.wG;
  gc.xG = xG;
  gc.c_axis = model_axis_traffic(rec, f, ub, tau, sp.tp_coll);
  gc.fbase = ub.cv | (ub.d1 ? X_D1 : 0);
  const u32 nm2 = sp.nm * sp.nm;
  __syncwarp();
  if (lane < (int)nm2) {
    const u32 d0 = lane % sp.nm, d1 = lane / sp.nm;
    {  // (Theta, Omega)
      const u32 th = digit_mode(sp.modemap, d0), om = digit_mode(sp.modemap, d1);
      const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
      PairEntry e;
      e.mem = rec.wT * mu_elems(th, ub.E2, ub.sh, ub.u) + rec.wO * mu_elems(om, ub.E2, ub.sh, ub.u);
      e.comm_paper = (th == PS_MODE_SG) ? 2 * xT : 0;
      e.comm_ext = (th == PS_MODE_O ? 2 * xT : 0) + ((th == PS_MODE_R && on_shard) ? xT : 0) +
                   (om == PS_MODE_SG ? xO : 0);
      e.host = (th == PS_MODE_O ? 3 * ub.sh * rec.wT : 0) + (om == PS_MODE_O ? 2 * ub.sh * rec.wO : 0);
      const bool omega_full = (om == PS_MODE_R) || (ub.d1 && in_set(SET_SHARDLIKE, om));
      const bool theta_avail = in_set(SET_THETA_ALWAYS, th) || (th == PS_MODE_S && ub.d1) ||
                               (th == PS_MODE_M && omega_full);
      u32 fl = (theta_avail ? PS_F_THETA_AVAIL : 0) | (om != PS_MODE_M ? PS_F_SC : 0) |
               (on_shard ? X_ON_SHARD : 0);
      if (th == PS_MODE_O || om == PS_MODE_O) fl |= PS_F_USES_HOST;
      if (in_set(SET_M_OR_O, th) || in_set(SET_M_OR_O, om)) fl |= X_M_OR_O;
      tb.p1[lane] = e;
      tb.f1[lane] = fl;
    }
    {  // (G, A); comm_ext as if the update is committed on a shard
      const u32 gr = digit_mode(sp.modemap, d0), ac = digit_mode(sp.modemap, d1);
      PairEntry e;
      e.mem = rec.wG * mu_elems(gr, ub.E2, ub.sh, ub.u) + mu_elems(ac, ab.EA, ab.shA, ab.uA);
      e.comm_paper = (gr == PS_MODE_R) ? 2 * xG : (gr == PS_MODE_S ? xG : 0);
      e.comm_ext = (gr == PS_MODE_SG ? 2 * xG : 0) + ((gr == PS_MODE_M || gr == PS_MODE_O) ? xG : 0);
      e.host = (gr == PS_MODE_O ? 2 * ub.sh * rec.wG : 0) + (ac == PS_MODE_O ? 2 * ab.EA : 0);
      u32 fl = (in_set(SET_GRAD_FULL, gr) ? X_G_FULL : 0) | (gr == PS_MODE_M ? X_G_IS_M : 0) |
               ((ub.d1 || in_set(SET_ACT_OWN, ac)) ? PS_F_ACT_AVAIL : 0);
      if (gr == PS_MODE_O || ac == PS_MODE_O) fl |= PS_F_USES_HOST;
      if (in_set(SET_M_OR_O, gr) || in_set(SET_M_OR_O, ac)) fl |= X_M_OR_O;
      tb.p2[lane] = e;
      tb.f2[lane] = fl;
    }
  }
  __syncwarp();
  return true;
}

struct PointVals {
  u64 mem, comm_paper, comm_ext, host;
  u32 flags;
};

__device__ __forceinline__ PointVals eval_from_tables(const WarpGroupTables& tb, const GroupConst& gc,
                                                      u32 i1, u32 i2) {
  const PairEntry a = tb.p1[i1], b = tb.p2[i2];
  const u32 x = tb.f1[i1] | tb.f2[i2] | gc.fbase;
  PointVals o;
  o.mem = a.mem + b.mem;
  o.comm_paper = a.comm_paper + b.comm_paper;
  o.host = a.host + b.host;
  u64 ext = a.comm_ext + b.comm_ext;
  if ((x & (X_G_IS_M | X_ON_SHARD)) == X_G_IS_M) ext += gc.xG;   // reduced per unit by all-reduce
  u32 fl = x & X_PUBLIC;
  if (x & (X_ON_SHARD | X_G_FULL | X_D1)) fl |= PS_F_GRAD_COVER;
  constexpr u32 gi_needs = PS_F_THETA_AVAIL | PS_F_ACT_AVAIL | PS_F_GRAD_COVER;
  if ((fl & gi_needs) == gi_needs) fl |= PS_F_GI;
  if (ext == 0 && !(x & X_M_OR_O)) fl |= PS_F_PAPER_PRICED;
  o.comm_ext = ext + gc.c_axis;
  o.flags = fl;
  return o;
}

// walks the codes lane, lane+32, ... of a group's window, keeping the two
// table indices incrementally
struct CodeWalk {
  u32 i1, i2, step_q, step_r, nm2;
  __device__ __forceinline__ void init(u32 code, u32 nm2_) {
    nm2 = nm2_;
    i2 = code / nm2;
    i1 = code - i2 * nm2;
    step_q = 32 / nm2;
    step_r = 32 - step_q * nm2;
  }
  __device__ __forceinline__ void next() {
    i1 += step_r;
    i2 += step_q;
    if (i1 >= nm2) { i1 -= nm2; ++i2; }
  }
};

enum { MODE_MATERIALISE = 0, MODE_COUNT = 1, MODE_WRITE = 2 };

template <int MODE>
__global__ void __launch_bounds__(THREADS) k_eval(SpaceDev sp, EvalArgs a) {
  __shared__ WarpGroupTables tables[WARPS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const u64 seg = (u64)blockIdx.x * WARPS + warp;      // which group of the window
  const u64 g = a.first_group + seg;
  WarpGroupTables& tb = tables[warp];
  GroupConst gc;
  const bool any = build_group(sp, a, g, lane, tb, gc);
  if (!any) {
    if (MODE == MODE_COUNT && lane == 0 && seg < a.n_tiles) a.tile_count[seg] = 0;
    return;
  }
  const u32 n_pts = (u32)(gc.hi - gc.lo);
  const u32 code0 = (u32)(gc.lo - gc.group_first);
  CodeWalk walk;
  walk.init(code0 + lane, sp.nm * sp.nm);
  const u64 out_base = gc.lo - a.first;                // output position of the group's first point

  u32 n_kept = 0;                                      // survivors so far (warp-uniform)
  u64 write_base = 0;
  if (MODE == MODE_WRITE) write_base = a.tile_offset[seg];

  for (u32 k = 0; k < n_pts; k += 32, walk.next()) {
    const bool live = k + lane < n_pts;
    PointVals p;
    if (live) p = eval_from_tables(tb, gc, walk.i1, walk.i2);
    if (MODE == MODE_MATERIALISE) {
      if (live) {
        const u64 o = out_base + k + lane;
        if (a.out.mem) a.out.mem[o] = p.mem;
        if (a.out.comm_paper) a.out.comm_paper[o] = p.comm_paper;
        if (a.out.comm_ext) a.out.comm_ext[o] = p.comm_ext;
        if (a.out.host) a.out.host[o] = p.host;
        if (a.out.flags) a.out.flags[o] = p.flags;
      }
    } else {
      const bool pass = live && p.mem <= a.cap_bytes && p.host <= a.host_cap &&
                        (p.flags & a.require_flags) == a.require_flags;
      const u32 votes = __ballot_sync(0xffffffffu, pass);
      if (MODE == MODE_WRITE && pass) {
        const u64 o = write_base + n_kept + __popc(votes & ((1u << lane) - 1u));
        if (a.idx_out) a.idx_out[o] = gc.lo + k + lane;
        if (a.out.mem) a.out.mem[o] = p.mem;
        if (a.out.comm_paper) a.out.comm_paper[o] = p.comm_paper;
        if (a.out.comm_ext) a.out.comm_ext[o] = p.comm_ext;
        if (a.out.host) a.out.host[o] = p.host;
        if (a.out.flags) a.out.flags[o] = p.flags | PS_F_FEASIBLE;
      }
      n_kept += __popc(votes);
    }
  }
  if (MODE == MODE_COUNT && lane == 0) a.tile_count[seg] = n_kept;
}

// exclusive prefix sum of the per-group survivor counts; one block
__global__ void __launch_bounds__(1024) k_tile_scan(EvalArgs a) {
  __shared__ u64 part[1024];
  const int tid = threadIdx.x;
  const u32 n = a.n_tiles;
  const u32 per = (n + 1023) / 1024;
  const u32 lo = min((u32)tid * per, n), hi = min(lo + per, n);
  u64 s = 0;
  for (u32 i = lo; i < hi; ++i) s += a.tile_count[i];
  part[tid] = s;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {     // inclusive scan of the partial sums
    u64 add = (tid >= off) ? part[tid - off] : 0;
    __syncthreads();
    part[tid] += add;
    __syncthreads();
  }
  u64 run = part[tid] - s;
  for (u32 i = lo; i < hi; ++i) {
    a.tile_offset[i] = run;
    run += a.tile_count[i];
  }
  if (tid == 1023) *a.n_out = part[1023];
}

}  // namespace

static unsigned eval_blocks(const EvalArgs& a) { return (a.n_tiles + WARPS - 1) / WARPS; }

cudaError_t launch_eval_materialise(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  k_eval<MODE_MATERIALISE><<<eval_blocks(a), THREADS, 0, stream>>>(sp, a);
  return cudaGetLastError();
}
cudaError_t launch_eval_count(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  k_eval<MODE_COUNT><<<eval_blocks(a), THREADS, 0, stream>>>(sp, a);
  return cudaGetLastError();
}
cudaError_t launch_tile_scan(const EvalArgs& a, cudaStream_t stream) {
  k_tile_scan<<<1, 1024, 0, stream>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_eval_write(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  k_eval<MODE_WRITE><<<eval_blocks(a), THREADS, 0, stream>>>(sp, a);
  return cudaGetLastError();
}

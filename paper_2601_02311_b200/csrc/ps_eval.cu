// Batch evaluation of a window of the space: materialise every output, or
// filter and compact the survivors in index order.
//
// A "group" is the n_codes consecutive points that share (model, factorisation,
// activation variant, tensor-axis variant).  A warp owns a contiguous run of the
// window's groups.  Within a group a lane owns up to four (Theta, Omega, G)
// triples.  A triple's bytes, priced communication, unpriced communication and
// host bytes are small-integer multiples of four per-group scalars (elements per
// position E, largest shard s, reconstruction unit u, ring volume x), and the
// integer coefficients depend only on the triple's modes and the model's byte
// widths -- so they are computed once per model and a group costs a few
// multiply-adds per triple.  The activation digit then adds one of NM
// per-group values.  Codes of a group run digit-major, triple-minor, so for a
// fixed digit the lanes write consecutive elements.  Materialise stages one
// output array of a group in shared memory and stores it with one bulk copy
// (shared -> global, asynchronous), so the warp computes the next array while
// the previous one drains.
//
// Compaction is count -> scan -> write.  The count pass (k_compact_count, one
// warp per run of up to 32 consecutive groups) never forms a point's bytes or
// flags: like the sweeps it compares a triple's own bytes with a per-(variant,
// digit) bound and masks the result with the digits the required flags allow.
// It stores the survivors of each group and of each run and appends the groups
// that have survivors to a list.  A single-block scan turns the runs' totals
// into offsets.  The write pass takes the listed groups one per warp, evaluates
// them and places their survivors with ballot/popc prefix sums; a group's offset
// is its run's plus the counts of the run's earlier groups.  Output order is the
// index order, so the result is unique.
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

// Launch shapes (blocks of four warps per SM; four are resident at a time).  Materialise is
// fastest with about one group per warp: short-lived blocks keep the warps of an
// SM at different stages (set-up, staging, draining stores) and the running
// warps write neighbouring stretches of every output array.  The count pass
// prefers long runs of groups per warp (what a model and a factorisation fix is
// then computed once).  The write pass takes the listed groups round-robin; with
// many short blocks the stores of neighbouring groups are in flight together
// (every point surviving: 0.56 of the copy bandwidth with 32 warps in the grid per
// SM, 0.62 with 256).
#ifndef EVAL_BULK_EVICT_FIRST
#define EVAL_BULK_EVICT_FIRST 1
#endif
#ifndef EVAL_GRID_PER_SM_MATERIALISE
#define EVAL_GRID_PER_SM_MATERIALISE 128
#endif
#ifndef EVAL_GRID_PER_SM_COMPACT
#define EVAL_GRID_PER_SM_COMPACT 2
#endif
#ifndef EVAL_GRID_PER_SM_WRITE
#define EVAL_GRID_PER_SM_WRITE 64
#endif
constexpr int THREADS = EVAL_THREADS;
constexpr int WARPS = THREADS / 32;

// internal bits of a triple's static description (above the public flag bits)
enum : u32 {
  X_HOST3 = 1u << 16,     // one of Theta, Omega, G is offloaded
  X_MO3 = 1u << 17,       // one of them is materialised or offloaded
  X_EXT0 = 1u << 18       // the data axis moves nothing beyond Theorem 2's terms
};

__device__ __forceinline__ u64 mad_small(u64 a, u32 k, u64 acc) {
  u64 r = (u64)(u32)a * (u64)k + acc;
  r += (u64)((u32)(a >> 32) * k) << 32;
  return r;
}

// static description of a triple when the data axis has several shard positions (d1 = false)
// or a single device (d1 = true)
__device__ __forceinline__ u32 triple_static(u32 th, u32 om, u32 gr, bool d1) {
  const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
  const bool omega_full = (om == PS_MODE_R) || (d1 && in_set(SET_SHARDLIKE, om));
  const bool theta_avail = in_set(SET_THETA_ALWAYS, th) || (th == PS_MODE_S && d1) ||
                           (th == PS_MODE_M && omega_full);
  const bool grad_cover = d1 || on_shard || in_set(SET_GRAD_FULL, gr);
  const u32 seen = (1u << th) | (1u << om) | (1u << gr);
  // with one replica nothing moves; otherwise the unpriced data-axis terms are
  // non-zero exactly when their mode conditions hold (ring volume >= 1 element)
  const bool ext0 = d1 || !((th == PS_MODE_O) || (th == PS_MODE_R && on_shard) ||
                            in_set((1u << PS_MODE_SG) | SET_M_OR_O, gr) || om == PS_MODE_SG);
  return (theta_avail ? PS_F_THETA_AVAIL : 0) | (grad_cover ? PS_F_GRAD_COVER : 0) |
         (om != PS_MODE_M ? PS_F_SC : 0) | (((seen >> PS_MODE_O) & 1u) ? X_HOST3 : 0) |
         ((seen & SET_M_OR_O) ? X_MO3 : 0) | (ext0 ? X_EXT0 : 0);
}

// the same for a factorisation whose shards are all held by every device (several copies,
// one shard position): a shard is the whole tensor as on a single device, the gathers move
// nothing, but the gradient modes Theorem 2 does not price still move data
__device__ __forceinline__ u32 triple_static_all_copies(u32 th, u32 om, u32 gr) {
  const u32 st = triple_static(th, om, gr, true) & ~X_EXT0;
  return st | (in_set((1u << PS_MODE_SG) | SET_M_OR_O, gr) ? 0u : X_EXT0);
}

enum { MODE_MATERIALISE = 0, MODE_WRITE = 2 };

// Staging for the materialise path.  A warp builds one output array of one
// group (NC elements) in shared memory and hands it to the copy engine as a
// single bulk store (cp.async.bulk, shared -> global), then goes on computing the
// next array while the store drains; two staging buffers per warp alternate.
// A bulk store needs both addresses 16-byte aligned and a size that is a
// multiple of 16 bytes, while an output array is only aligned to its element and
// a group starts anywhere in it.  So element c of the group is staged at slot
// c + skew, where skew = (destination address / element size) mod (16 / element
// size): the shared and global addresses of every element then agree modulo 16,
// the elements before the first 16-byte boundary and after the last one (at
// most 16 / element size - 1 each) are written with plain stores, and everything
// between goes out as one bulk store.
template <int NC>
struct Stage {
  static constexpr int SLOTS = NC + 4;                                   // u64 slots, room for the skew
  static constexpr int BYTES = ((SLOTS * 8 + 127) / 128) * 128;          // one buffer
};

__device__ __forceinline__ u32 smem_addr(const void* p) { return (u32)__cvta_generic_to_shared(p); }

// lane 0 owns the warp's bulk stores: wait until at most `pending` of them still read shared memory
template <int PENDING>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(PENDING) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// All lanes have written `n` elements of type T to buf[skew ...]; store them to dst[0 .. n).
template <typename T>
__device__ __forceinline__ void warp_bulk_store(T* __restrict__ dst, const T* buf, int skew, int n, int lane) {
  constexpr int PER16 = 16 / (int)sizeof(T);
  // make the lanes' shared-memory writes visible to the copy engine
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  const int head = min((PER16 - skew) & (PER16 - 1), n);                 // elements before the first boundary
  const int body = ((n - head) / PER16) * PER16;
  if (lane < head) dst[lane] = buf[skew + lane];
  const int tail = n - head - body;
  if (lane < tail) dst[head + body + lane] = buf[skew + head + body + lane];
  if (lane == 0 && body > 0) {
#if EVAL_BULK_EVICT_FIRST
    // The output is written once and not read back by this kernel: with the evict-first
    // policy the lines leave the L2 as whole lines.  (Without a policy the same stores
    // cost 12 % more DRAM write traffic than the bytes stored.)
    unsigned long long policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                 ::"l"(dst + head), "r"(smem_addr(buf + skew + head)), "r"(body * (int)sizeof(T)), "l"(policy)
                 : "memory");
#else
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst + head), "r"(smem_addr(buf + skew + head)), "r"(body * (int)sizeof(T))
                 : "memory");
#endif
  }
  if (lane == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// POW2: every degree of the space is a power of two (no division is compiled in)
template <int MODE, int NM, bool POW2>
__global__ void __launch_bounds__(THREADS, EVAL_MIN_BLOCKS) k_eval(SpaceDev sp, EvalArgs a) {
  constexpr int N2 = NM * NM, N3 = NM * NM * NM, NC = N3 * NM;
  constexpr int R = (N3 + 31) / 32;
  // materialise: two staging buffers per warp (dynamic shared memory, none in the other modes)
  extern __shared__ __align__(128) unsigned char stage_all[];
  unsigned char* const stage_warp = stage_all + (threadIdx.x >> 5) * 2 * Stage<NC>::BYTES;
  u32 stage_turn = 0;                                                     // which buffer is next
  const int lane = threadIdx.x & 31;
  const u32 warp_global = blockIdx.x * WARPS + (threadIdx.x >> 5);
  const u32 n_warps = gridDim.x * WARPS;
  // materialise: the window's groups are dealt evenly, a contiguous stretch per warp;
  // write: the groups that have survivors, from the count pass's list, dealt round-robin
  const u32 per_warp = (a.n_tiles + n_warps - 1) / n_warps;
  const u32 it_begin = MODE == MODE_WRITE ? warp_global : (u32)min((u64)warp_global * per_warp, (u64)a.n_tiles);
  const u32 it_end = MODE == MODE_WRITE ? *a.n_nonempty : min(it_begin + per_warp, a.n_tiles);
  const u32 it_step = MODE == MODE_WRITE ? n_warps : 1u;
  const u32 groups_per_model = sp.n_facts * sp.nvt;

  // with all five modes allowed digit d is mode d, and the compiler knows every
  // per-digit property below
  const u32 modemap = (NM == 5) ? 0x43210u : sp.modemap;
  // the lane's triples: modes never change
  u32 th[R], om[R], gr[R];
  bool live[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const u32 t = lane + 32 * r;
    live[r] = t < (u32)N3;
    const u32 tt = live[r] ? t : 0;
    th[r] = digit_mode(modemap, tt % NM);
    om[r] = digit_mode(modemap, (tt / NM) % NM);
    gr[r] = digit_mode(modemap, tt / N2);
  }
  // classes of the activation digit (Theorem 3: a replica needs its own activations)
  u32 own = 0, is_o = 0, not_mo = 0;
#pragma unroll
  for (int d = 0; d < NM; ++d) {
    const u32 ac = digit_mode(modemap, d);
    if (in_set(SET_ACT_OWN, ac)) own |= 1u << d;
    if (ac == PS_MODE_O) is_o |= 1u << d;
    if (!in_set(SET_M_OR_O, ac)) not_mo |= 1u << d;
  }

  // per model: widths and the coefficients that follow from them
  u32 model_cur = 0xffffffffu;
  ModelRec rec;
  u32 ka[R], kb[R], kc[R], kp[R], ke[R], kh[R];   // bytes (E, s, u), priced / unpriced comm (x), host (s)
  u32 st_many[R], st_one[R];                      // static description of a triple by the class of the factorisation
  u32 st_copies[POW2 ? 1 : R];                    // (the third class needs several copies of a shard)

  for (u32 it = it_begin; it < it_end; it += it_step) {
    const u32 seg = MODE == MODE_WRITE ? a.nonempty[it] : it;
    const u64 g = a.first_group + seg;
    // (a 32-bit division where the group number allows it: it is done once per group by every lane)
    const u32 model = (g >> 32) == 0 ? (u32)g / groups_per_model : (u32)(g / groups_per_model);
    const u32 gl = (u32)(g - (u64)model * groups_per_model);
    const u32 unit = gl / sp.nvt, vt = gl - unit * sp.nvt;
    const u32 v = vt / sp.nt, tau = vt - v * sp.nt;
    if (model != model_cur) {
      model_cur = model;
      const uint4* src = reinterpret_cast<const uint4*>(&sp.recs[model]);
      uint4* dst = reinterpret_cast<uint4*>(&rec);
#pragma unroll
      for (int k = 0; k < 6; ++k) dst[k] = __ldg(src + k);   // the 96-byte record, 16 bytes at a time
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const u32 modes[3] = {th[r], om[r], gr[r]};
        const u32 width[3] = {rec.wT, rec.wO, rec.wG};
        const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om[r]);
        u32 ca = 0, cb = 0, cc = 0;
#pragma unroll
        for (int s = 0; s < 3; ++s) {        // Theorem 1: R holds E, S and S* a shard, S* and M a unit
          if (modes[s] == PS_MODE_R) ca += width[s];
          if (in_set(SET_SHARDLIKE, modes[s])) cb += width[s];
          if (modes[s] == PS_MODE_SG) cc += width[s] * sp.sstar_units;   // one or two unit buffers
          if (modes[s] == PS_MODE_M) cc += width[s];
        }
        ka[r] = ca; kb[r] = cb; kc[r] = cc;
        // Theorem 2: all-reduce (2x) or reduce-scatter (1x) of G, two all-gathers of gathered
        // Theta for every micro-batch
        kp[r] = (th[r] == PS_MODE_SG ? 2 * sp.accum * rec.wT : 0) +
                (gr[r] == PS_MODE_R ? 2 * rec.wG : (gr[r] == PS_MODE_S ? rec.wG : 0));
        // what the execution model moves beyond that
        u32 e = 0;
        if (th[r] == PS_MODE_O) e += 2 * sp.accum * rec.wT;
        if (th[r] == PS_MODE_R && on_shard) e += rec.wT;
        if (om[r] == PS_MODE_SG) e += rec.wO;
        if (gr[r] == PS_MODE_SG) e += 2 * rec.wG;
        if (gr[r] == PS_MODE_M) e += (on_shard ? 1 : 2) * rec.wG;
        if (gr[r] == PS_MODE_O) e += rec.wG;
        ke[r] = e;
        kh[r] = (th[r] == PS_MODE_O ? (2 * sp.accum + 1) * rec.wT : 0) + (om[r] == PS_MODE_O ? 2 * rec.wO : 0) +
                (gr[r] == PS_MODE_O ? 2 * rec.wG : 0);
        st_many[r] = triple_static(th[r], om[r], gr[r], false);
        st_one[r] = triple_static(th[r], om[r], gr[r], true);
        if (!POW2) st_copies[r] = triple_static_all_copies(th[r], om[r], gr[r]);
      }
    }

    // ---- per group: shard quantities (all divisions), activation bytes per digit
    const Fact f = sp.facts[unit];
    const u32 repl = POW2 ? 1u : sp.repl;        // the power-of-two case is compiled for one copy of every shard
    const Pow2 p2 = POW2 ? pow2_of(f) : pow2_of(f, repl);
    const UnitBase ub = POW2 ? unit_base_pow2_one_copy(rec, f, p2, sp.tp_max_valid, true)
                        : p2.all ? unit_base_pow2(rec, f, p2, sp.tp_max_valid, true)
                                 : unit_base(rec, f, sp.tp_max_valid, true, repl);
    const ActBase ab = POW2 ? act_base_pow2_one_copy(rec, p2, v, tau)
                       : p2.all ? act_base_pow2(rec, p2, v, tau) : act_base(rec, f, v, tau, ub.G);
    const u64 c_axis = model_axis_traffic(rec, f, ub, tau, sp.tp_coll, sp.accum);
    u64 act[NM];
#pragma unroll
    for (int d = 0; d < NM; ++d) act[d] = mu_elems(digit_mode(modemap, d), ab.EA, ab.shA, ab.uA, sp.sstar_units);
    const u64 act_host = 2 * ab.EA * sp.accum;
    const u32 avail = ub.d1 ? ((1u << NM) - 1u) : own;     // digits with PS_F_ACT_AVAIL

    u64 mem3[R], paper3[R], ext3[R], host3[R];
    u32 st[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      mem3[r] = mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0)));
      paper3[r] = mad_small(ub.x, kp[r], 0);
      ext3[r] = mad_small(ub.x, ke[r], 0);
      if (repl > 1) {
        // several copies of every shard: reducing gradients to shards costs x2 more, an
        // all-reduce over all devices x3 more (both zero with one copy)
        const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om[r]);
        paper3[r] += (u64)rec.wG * ((gr[r] == PS_MODE_S ? ub.x2 : 0) + (gr[r] == PS_MODE_R ? ub.x3 : 0));
        ext3[r] += (u64)rec.wG * (((gr[r] == PS_MODE_SG || gr[r] == PS_MODE_O || (gr[r] == PS_MODE_M && on_shard)) ? ub.x2 : 0) +
                                  ((gr[r] == PS_MODE_M && !on_shard) ? ub.x3 : 0));
      }
      host3[r] = mad_small(ub.sh, kh[r], 0);
      // (with one copy of every shard a factorisation is sharded or a single device)
      if (POW2) st[r] = ub.d1 ? st_one[r] : st_many[r];
      else st[r] = ub.cls == CLS_SHARDED ? st_many[r] : (ub.cls == CLS_ONE_DEVICE ? st_one[r] : st_copies[POW2 ? 0 : r]);
    }

    // ---- the group's points inside the window
    const u64 group_first = g * NC;
    const u32 code_lo = a.first > group_first ? (u32)(a.first - group_first) : 0u;
    const u64 window_end = a.first + a.count;
    const u32 code_hi = window_end < group_first + NC ? (u32)(window_end - group_first) : (u32)NC;
    const u64 out_base = group_first - a.first;          // (wraps when the group starts before the window; only used with code >= code_lo)

    u32 n_kept = 0;
    u64 write_base = 0;
    if (MODE == MODE_WRITE) {
      // survivors before this group = those of the runs before its run (scanned) plus
      // those of the run's earlier groups
      const u32 run = seg / a.run_len;
      u64 part = 0;
      for (u32 j = run * a.run_len + lane; j < seg; j += 32) part += a.tile_count[j];
      for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
      write_base = a.tile_offset[run] + part;
    }

    // flags of a point = what the triple fixes | what the digit fixes | what needs both:
    //   gradient integrity needs the triple's two availability bits and the digit's,
    //   "paper priced" needs a triple without M/O and unpriced traffic and a digit without M/O
    u32 fl_base[R], fl_gi[R], fl_priced[R];
    constexpr u32 both = PS_F_THETA_AVAIL | PS_F_GRAD_COVER;
#pragma unroll
    for (int r = 0; r < R; ++r) {
      fl_base[r] = ub.cv | (st[r] & (both | PS_F_SC)) | ((st[r] & X_HOST3) ? PS_F_USES_HOST : 0);
      fl_gi[r] = ((st[r] & both) == both) ? PS_F_GI : 0;
      fl_priced[r] = ((st[r] & (X_EXT0 | X_MO3)) == X_EXT0) ? PS_F_PAPER_PRICED : 0;
    }
    const bool whole = code_lo == 0 && code_hi == (u32)NC;      // the window covers the group
    const bool all_out = a.out.mem && a.out.comm_paper && a.out.comm_ext && a.out.host && a.out.flags;

    if (MODE == MODE_MATERIALISE && whole && all_out) {
      // one output array at a time: stage the group's NC values, hand them to the copy engine
#pragma unroll
      for (int which = 0; which < 5; ++which) {
        u64* const stage = reinterpret_cast<u64*>(stage_warp + (stage_turn & 1u) * Stage<NC>::BYTES);
        u32* const stage32 = reinterpret_cast<u32*>(stage);
        ++stage_turn;
        u64* const dst64 = (which == 0 ? a.out.mem : which == 1 ? a.out.comm_paper
                            : which == 2 ? a.out.comm_ext : a.out.host) + out_base;
        u32* const dst32 = a.out.flags + out_base;
        const int skew = which < 4 ? (int)((reinterpret_cast<uintptr_t>(dst64) >> 3) & 1)
                                   : (int)((reinterpret_cast<uintptr_t>(dst32) >> 2) & 3);
        // the store that used this buffer two arrays ago must have read it completely
        if (lane == 0) bulk_wait_read<1>();
        __syncwarp();
#pragma unroll
        for (int d = 0; d < NM; ++d) {
          const bool d_avail = (avail >> d) & 1u, d_off = (is_o >> d) & 1u, d_notmo = (not_mo >> d) & 1u;
          const u32 fl_digit = (d_avail ? PS_F_ACT_AVAIL : 0) | (d_off ? PS_F_USES_HOST : 0);
          const u32 gi_mask = d_avail ? ~0u : 0u, priced_mask = d_notmo ? ~0u : 0u;
          const u64 host_add = d_off ? act_host : 0;
#pragma unroll
          for (int r = 0; r < R; ++r) {
            if (!live[r]) continue;
            const u32 slot = lane + 32 * r + d * N3 + skew;
            if (which == 0) stage[slot] = mem3[r] + act[d];
            else if (which == 1) stage[slot] = paper3[r];
            else if (which == 2) stage[slot] = ext3[r] + c_axis;
            else if (which == 3) stage[slot] = host3[r] + host_add;
            else stage32[slot] = fl_base[r] | fl_digit | (fl_gi[r] & gi_mask) | (fl_priced[r] & priced_mask);
          }
        }
        if (which < 4) warp_bulk_store(dst64, stage, skew, NC, lane);
        else warp_bulk_store(dst32, stage32, skew, NC, lane);
      }
      continue;
    }

#pragma unroll
    for (int d = 0; d < NM; ++d) {
      const bool d_avail = (avail >> d) & 1u, d_off = (is_o >> d) & 1u, d_notmo = (not_mo >> d) & 1u;
      const u32 fl_digit = (d_avail ? PS_F_ACT_AVAIL : 0) | (d_off ? PS_F_USES_HOST : 0);
      const u32 gi_mask = d_avail ? ~0u : 0u, priced_mask = d_notmo ? ~0u : 0u;
      const u64 host_add = d_off ? act_host : 0;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const u32 code = lane + 32 * r + d * N3;
        const bool inside = live[r] && (whole || (code >= code_lo && code < code_hi));
        const u64 mem = mem3[r] + act[d];
        const u64 host = host3[r] + host_add;
        const u32 fl = fl_base[r] | fl_digit | (fl_gi[r] & gi_mask) | (fl_priced[r] & priced_mask);
        if (MODE == MODE_MATERIALISE) {
          if (inside) {
            const u64 o = out_base + code;
            if (all_out) {
              a.out.mem[o] = mem;
              a.out.comm_paper[o] = paper3[r];
              a.out.comm_ext[o] = ext3[r] + c_axis;
              a.out.host[o] = host;
              a.out.flags[o] = fl;
            } else {
              if (a.out.mem) a.out.mem[o] = mem;
              if (a.out.comm_paper) a.out.comm_paper[o] = paper3[r];
              if (a.out.comm_ext) a.out.comm_ext[o] = ext3[r] + c_axis;
              if (a.out.host) a.out.host[o] = host;
              if (a.out.flags) a.out.flags[o] = fl;
            }
          }
        } else {
          const bool pass = inside && mem <= a.cap_bytes && host <= a.host_cap &&
                            (fl & a.require_flags) == a.require_flags;
          const u32 votes = __ballot_sync(0xffffffffu, pass);
          if (MODE == MODE_WRITE && pass) {
            const u64 o = write_base + n_kept + __popc(votes & ((1u << lane) - 1u));
            if (a.idx_out) a.idx_out[o] = group_first + code;
            if (a.out.mem) a.out.mem[o] = mem;
            if (a.out.comm_paper) a.out.comm_paper[o] = paper3[r];
            if (a.out.comm_ext) a.out.comm_ext[o] = ext3[r] + c_axis;
            if (a.out.host) a.out.host[o] = host;
            if (a.out.flags) a.out.flags[o] = fl | PS_F_FEASIBLE;
          }
          n_kept += __popc(votes);
        }
      }
    }
  }
  // the staging buffers must outlive the bulk stores that read them
  if (MODE == MODE_MATERIALISE && lane == 0) bulk_wait_all();
}

// The count pass of the compaction.  One warp per run of consecutive groups.  What
// a factorisation fixes is computed once for its (up to four) groups: the lanes'
// triples' own bytes and host bytes, and for every (variant, digit) the bound the
// own bytes must stay below for the point to fit the capacity (cap + 1 - activation
// bytes) and the host budget.  A point then costs one compare, masked by the
// digits the required flags allow for its triple (fixed for the whole kernel).
struct CountTables {
  u64 bound[5][4];       // [digit][variant]
  __align__(16) double bound_f64[5][4];   // the same as doubles (exact below 2^53), 0 for variants the space lacks
  u64 host_bound[4];     // the triple's own host bytes must stay below this to offload activations
};

template <int NM, bool POW2>
__global__ void __launch_bounds__(THREADS, EVAL_MIN_BLOCKS) k_compact_count(SpaceDev sp, EvalArgs a) {
  constexpr int N2 = NM * NM, N3 = NM * NM * NM, NC = N3 * NM;
  constexpr int R = (N3 + 31) / 32;
  __shared__ CountTables tables[WARPS];
  const int lane = threadIdx.x & 31;
  const u32 run = blockIdx.x * WARPS + (threadIdx.x >> 5);
  if (run >= a.n_runs) return;
  CountTables& tb = tables[threadIdx.x >> 5];
  const u32 seg_begin = run * a.run_len;
  const u32 seg_end = min(seg_begin + a.run_len, a.n_tiles);
  const u32 groups_per_model = sp.n_facts * sp.nvt;
  const u32 modemap = (NM == 5) ? 0x43210u : sp.modemap;
  const u32 req = a.require_flags;
  constexpr u32 CV_BITS = PS_F_CV | PS_F_T_DIV_HEADS | PS_F_K_DIV_LAYERS | PS_F_TP_LE_MAX | PS_F_AXIS_FORM;
  const u32 req_cv = req & CV_BITS;
  // capacities as exclusive bounds (memory and host bytes stay below 2^62)
  const u64 cap_x = min(a.cap_bytes, (u64)1 << 62) + 1;
  const u64 host_x = min(a.host_cap, (u64)1 << 62) + 1;
  u32 all = (1u << NM) - 1u, own = 0, is_o = 0, not_mo = 0;
#pragma unroll
  for (int d = 0; d < NM; ++d) {
    const u32 ac = digit_mode(modemap, d);
    if (in_set(SET_ACT_OWN, ac)) own |= 1u << d;
    if (ac == PS_MODE_O) is_o |= 1u << d;
    if (!in_set(SET_M_OR_O, ac)) not_mo |= 1u << d;
  }
  // the lane's triples: modes and the activation digits the required flags allow
  // (bits 0..4, 8..12, 16..20 for the three classes of a factorisation), fixed for the kernel
  u32 th[R], om[R], gr[R], t_allowed[R];
#pragma unroll
  for (int r = 0; r < R; ++r) {
    const u32 t = lane + 32 * r;
    const bool live = t < (u32)N3;
    const u32 tt = live ? t : 0;
    th[r] = digit_mode(modemap, tt % NM);
    om[r] = digit_mode(modemap, (tt / NM) % NM);
    gr[r] = digit_mode(modemap, tt / N2);
    const u32 a_many = allowed_act_digits(triple_bits(th[r], om[r], gr[r], CLS_SHARDED), req, all, own, is_o, not_mo);
    const u32 a_one = allowed_act_digits(triple_bits(th[r], om[r], gr[r], CLS_ONE_DEVICE), req, all, all, is_o, not_mo);
    const u32 a_copies = allowed_act_digits(triple_bits(th[r], om[r], gr[r], CLS_ALL_COPIES), req, all, all, is_o, not_mo);
    t_allowed[r] = live ? (a_many | (a_one << 8) | (a_copies << 16)) : 0;
  }
  // this lane's table entry (variant, digit)
  const u32 tl_vt = lane / NM, tl_d = lane - tl_vt * NM;
  const bool tl_mine = tl_vt < sp.nvt;
  const u32 tl_v = tl_mine ? tl_vt / sp.nt : 0;
  const u32 tl_tau = tl_mine ? tl_vt - tl_v * sp.nt : 0;
  const u32 tl_mode = digit_mode(modemap, tl_d);

  u32 model_cur = 0xffffffffu, unit_cur = 0xffffffffu;
  ModelRec rec;
  u32 ka[R], kb[R], kc[R], kh[R];
  u64 mem3[R], host3[R];
  bool small = false;                      // the factorisation's byte counts are exact as doubles
  u32 allowed[R];
  u64 run_total = 0;
  u32 with_survivors = 0;                  // bit j: group seg_begin + j has survivors
  const u64 window_end = a.first + a.count;

  // the run's first group by division, the following ones by counting up
  u32 model, unit, vt;
  {
    const u64 g0 = a.first_group + seg_begin;
    model = (u32)(g0 / groups_per_model);
    const u32 gl = (u32)(g0 - (u64)model * groups_per_model);
    unit = gl / sp.nvt;
    vt = gl - unit * sp.nvt;
  }
  for (u32 seg = seg_begin; seg < seg_end;) {
    const u64 g0 = a.first_group + seg;
    if (model != model_cur) {
      model_cur = model;
      unit_cur = 0xffffffffu;
      const uint4* src = reinterpret_cast<const uint4*>(&sp.recs[model]);
      uint4* dst = reinterpret_cast<uint4*>(&rec);
#pragma unroll
      for (int k = 0; k < 6; ++k) dst[k] = __ldg(src + k);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const u32 modes[3] = {th[r], om[r], gr[r]};
        const u32 width[3] = {rec.wT, rec.wO, rec.wG};
        u32 ca = 0, cb = 0, cc = 0;
#pragma unroll
        for (int s = 0; s < 3; ++s) {        // Theorem 1: R holds E, S and S* a shard, S* and M a unit
          if (modes[s] == PS_MODE_R) ca += width[s];
          if (in_set(SET_SHARDLIKE, modes[s])) cb += width[s];
          if (modes[s] == PS_MODE_SG) cc += width[s] * sp.sstar_units;
          if (modes[s] == PS_MODE_M) cc += width[s];
        }
        ka[r] = ca; kb[r] = cb; kc[r] = cc;
        kh[r] = (th[r] == PS_MODE_O ? (2 * sp.accum + 1) * rec.wT : 0) + (om[r] == PS_MODE_O ? 2 * rec.wO : 0) +
                (gr[r] == PS_MODE_O ? 2 * rec.wG : 0);
      }
    }
    if (unit != unit_cur) {
      unit_cur = unit;
      const Fact f = sp.facts[unit];
      const u32 repl = POW2 ? 1u : sp.repl;
      const Pow2 p2 = POW2 ? pow2_of(f) : pow2_of(f, repl);
      const UnitBase ub = POW2 ? unit_base_pow2_one_copy(rec, f, p2, sp.tp_max_valid, true)
                          : p2.all ? unit_base_pow2(rec, f, p2, sp.tp_max_valid, true)
                                   : unit_base(rec, f, sp.tp_max_valid, true, repl);
      __syncwarp();                            // the previous factorisation's bounds have been read
      if (tl_mine) {
        const ActBase ab = POW2 ? act_base_pow2_one_copy(rec, p2, tl_v, tl_tau)
                           : p2.all ? act_base_pow2(rec, p2, tl_v, tl_tau) : act_base(rec, f, tl_v, tl_tau, ub.G);
        const u64 am = mu_elems(tl_mode, ab.EA, ab.shA, ab.uA, sp.sstar_units);
        const u64 bound = am < cap_x ? cap_x - am : 0;
        tb.bound[tl_d][tl_vt] = bound;
        tb.bound_f64[tl_d][tl_vt] = (double)bound;
        if (tl_d == 0) {
          const u64 ah = 2 * ab.EA * sp.accum;  // offloaded after forward, reloaded for backward, per micro-batch
          tb.host_bound[tl_vt] = ah < host_x ? host_x - ah : 0;
        }
      } else if (tl_vt < 4) {
        tb.bound_f64[tl_d][tl_vt] = 0.0;
        if (tl_d == 0) tb.host_bound[tl_vt] = 0;
      }
      __syncwarp();
      const bool unit_ok = (ub.cv & req_cv) == req_cv;
      const u32 shift = POW2 ? (ub.d1 ? 8u : 0u) : 8 * ub.cls;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        mem3[r] = mad_small(ub.E2, ka[r], mad_small(ub.sh, kb[r], mad_small(ub.u, kc[r], 0)));
        host3[r] = mad_small(ub.sh, kh[r], 0);
        allowed[r] = (unit_ok && host3[r] < host_x) ? ((t_allowed[r] >> shift) & all) : 0;
      }
      // Integers below 2^53 are exact as doubles: when the capacity and every triple's bytes
      // are that small (one test for the warp), whole factorisations are counted with
      // compares on the fp64 pipe and predicated fp32 adds (see below).
      small = cap_x < ((u64)1 << 53) && (u64)(rec.wT + rec.wO + rec.wG) * (ub.E2 + 2 * ub.u) < ((u64)1 << 53);
    }
    // the factorisation's groups inside this run: variants vt .. vt + n_here - 1
    const u32 n_here = min(sp.nvt - vt, seg_end - seg);
    u32 cnt[4] = {0, 0, 0, 0};             // this lane's survivors per variant
    if (small && g0 * NC >= a.first && (g0 + n_here) * NC <= window_end) {
      // The usual case, every group whole inside the window: all variants at once.  A
      // triple's digit is tested for the four variants with one mask bit; a point costs a
      // compare on the fp64 pipe and a predicated fp32 add.
      float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
      for (int d = 0; d < NM; ++d) {
        double bound[4];
        {
          const double2 b01 = *reinterpret_cast<const double2*>(&tb.bound_f64[d][0]);
          const double2 b23 = *reinterpret_cast<const double2*>(&tb.bound_f64[d][2]);
          bound[0] = b01.x; bound[1] = b01.y; bound[2] = b23.x; bound[3] = b23.y;
        }
        const bool offload = (is_o >> d) & 1u;
#pragma unroll
        for (int r = 0; r < R; ++r) {
          const bool on = (allowed[r] >> d) & 1u;
          const double m = (double)mem3[r];
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (on && m < bound[j] && (!offload || host3[r] < tb.host_bound[j])) c[j] += 1.0f;
        }
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) cnt[j] = (u32)c[j];
    } else {
#pragma unroll 1
      for (u32 k = 0; k < n_here; ++k) {
        // a group at the window's edge (or byte counts beyond 2^53): only the codes inside the window
        const u64 group_first = (g0 + k) * NC;
        const u32 code_lo = a.first > group_first ? (u32)(a.first - group_first) : 0u;
        const u32 code_hi = window_end < group_first + NC ? (u32)(window_end - group_first) : (u32)NC;
        const u64 host_bound = tb.host_bound[vt + k];
        u32 n = 0;
#pragma unroll 1
        for (int d = 0; d < NM; ++d) {
          const u64 bound = tb.bound[d][vt + k];
          const bool offload = (is_o >> d) & 1u;
#pragma unroll
          for (int r = 0; r < R; ++r) {
            const u32 code = lane + 32 * r + d * N3;
            const bool pass = ((allowed[r] >> d) & 1u) && mem3[r] < bound && (!offload || host3[r] < host_bound) &&
                              code >= code_lo && code < code_hi;
            n += pass ? 1u : 0u;
          }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j)
          if ((u32)j == vt + k) cnt[j] = n;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if ((u32)j >= vt && (u32)j < vt + n_here) {              // (the same for every lane)
        const u32 n = __reduce_add_sync(0xffffffffu, cnt[j]);
        const u32 at = seg + ((u32)j - vt);
        if (lane == 0) a.tile_count[at] = n;
        run_total += n;
        if (n) with_survivors |= 1u << (at - seg_begin);
      }
    }
    // the next factorisation, else the next model
    seg += n_here;
    vt = 0;
    if (++unit == sp.n_facts) { unit = 0; ++model; }
  }
  if (lane == 0) a.tile_offset[run] = run_total;
  // the groups with survivors join the write pass's list (in any order: a group's place
  // in the output comes from the scan, not from the list)
  const u32 n_listed = __popc(with_survivors);
  if (n_listed) {
    u32 base = 0;
    if (lane == 0) base = atomicAdd(a.n_nonempty, n_listed);
    base = __shfl_sync(0xffffffffu, base, 0);
    if ((with_survivors >> lane) & 1u)
      a.nonempty[base + __popc(with_survivors & ((1u << lane) - 1u))] = seg_begin + lane;
  }
}

// exclusive prefix sum, in place, of the survivors of the count pass's runs
// (a.tile_offset[0 .. n_runs)); the total goes to *a.n_out.  One block: there are
// a few thousand runs, four per thread and tile.
constexpr int SCAN_THREADS = 1024, SCAN_ITEMS = 4;
__global__ void __launch_bounds__(SCAN_THREADS) k_tile_scan(EvalArgs a) {
  __shared__ u64 warp_sum[32];
  __shared__ u64 carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const u32 n = a.n_runs;
  if (tid == 0) carry = 0;
  __syncthreads();
  for (u32 tile = 0; tile < n; tile += SCAN_THREADS * SCAN_ITEMS) {
    const u32 i0 = tile + SCAN_ITEMS * tid;
    u64 c[SCAN_ITEMS];
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) c[k] = (i0 + k < n) ? a.tile_offset[i0 + k] : 0;
    u64 mine = 0;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) mine += c[k];
    u64 incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const u64 up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    u64 before = carry;                          // everything before this warp
    for (int w = 0; w < warp; ++w) before += warp_sum[w];
    u64 run = before + incl - mine;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
      if (i0 + k < n) a.tile_offset[i0 + k] = run;
      run += c[k];
    }
    __syncthreads();
    if (tid == SCAN_THREADS - 1) carry = before + incl;
    __syncthreads();
  }
  if (tid == 0) {
    *a.n_out = carry;
    *a.n_nonempty_other = 0;      // the next compaction's list starts empty
  }
}

template <int MODE, int NM, bool POW2>
cudaError_t launch_eval_p(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  // one warp per run of groups; enough blocks to fill the GPU, no more than groups
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned needed = (a.n_tiles + WARPS - 1) / WARPS;
  const unsigned most = (unsigned)sms * (MODE == MODE_MATERIALISE ? EVAL_GRID_PER_SM_MATERIALISE
                                                                  : EVAL_GRID_PER_SM_WRITE);
  const unsigned blocks = needed < most ? needed : most;
  constexpr int NC = NM * NM * NM * NM;
  const size_t smem = MODE == MODE_MATERIALISE ? (size_t)WARPS * 2 * Stage<NC>::BYTES : 0;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_eval<MODE, NM, POW2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  k_eval<MODE, NM, POW2><<<blocks, THREADS, smem, stream>>>(sp, a);
  return cudaGetLastError();
}

template <int MODE, int NM>
cudaError_t launch_eval_t(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  return (sp.all_pow2 && sp.repl == 1) ? launch_eval_p<MODE, NM, true>(sp, a, stream)
                                       : launch_eval_p<MODE, NM, false>(sp, a, stream);
}

template <int MODE>
cudaError_t launch_eval_m(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  switch (sp.nm) {
    case 1: return launch_eval_t<MODE, 1>(sp, a, stream);
    case 2: return launch_eval_t<MODE, 2>(sp, a, stream);
    case 3: return launch_eval_t<MODE, 3>(sp, a, stream);
    case 4: return launch_eval_t<MODE, 4>(sp, a, stream);
    default: return launch_eval_t<MODE, 5>(sp, a, stream);
  }
}

}  // namespace

// The count pass's runs: as many as fill the GPU with long-lived warps, but no
// run longer than 32 groups (the write pass adds up the counts of a run's
// earlier groups with one load per lane).
void eval_plan_runs(EvalArgs& a) {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const u32 target = (u32)sms * EVAL_GRID_PER_SM_COMPACT * WARPS;
  u32 len = (a.n_tiles + target - 1) / target;
  if (len < 1) len = 1;
  if (len > 32) len = 32;
  a.run_len = len;
  a.n_runs = (a.n_tiles + len - 1) / len;
}

cudaError_t launch_eval_materialise(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  return launch_eval_m<MODE_MATERIALISE>(sp, a, stream);
}
template <int NM>
static cudaError_t launch_count_t(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  const unsigned blocks = (a.n_runs + WARPS - 1) / WARPS;       // a warp per run
  if (sp.all_pow2 && sp.repl == 1) k_compact_count<NM, true><<<blocks, THREADS, 0, stream>>>(sp, a);
  else k_compact_count<NM, false><<<blocks, THREADS, 0, stream>>>(sp, a);
  return cudaGetLastError();
}
cudaError_t launch_eval_count(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  switch (sp.nm) {
    case 1: return launch_count_t<1>(sp, a, stream);
    case 2: return launch_count_t<2>(sp, a, stream);
    case 3: return launch_count_t<3>(sp, a, stream);
    case 4: return launch_count_t<4>(sp, a, stream);
    default: return launch_count_t<5>(sp, a, stream);
  }
}
cudaError_t launch_tile_scan(const EvalArgs& a, cudaStream_t stream) {
  k_tile_scan<<<1, SCAN_THREADS, 0, stream>>>(a);
  return cudaGetLastError();
}
cudaError_t launch_eval_write(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream) {
  return launch_eval_m<MODE_WRITE>(sp, a, stream);
}

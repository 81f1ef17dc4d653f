// Device-side data structures and arithmetic shared by the kernels of the
// placement-semantics sweep.  Everything is unsigned integer arithmetic.
#pragma once
#include <stdint.h>
#include "ps.h"

typedef uint64_t u64;
typedef uint32_t u32;

// ---------------------------------------------------------------- records
// What one model contributes to the formulas; derived on the device from a
// ps_model_shape (Section 2.1, Remark 1, Definition 3).  96 bytes, 16-aligned.
struct __align__(16) ModelRec {
  u64 P;        // parameter elements
  u64 unit;     // reconstruction unit in elements (Definition 3), 0 = none
  u64 A[2];     // activation bytes of one replica: stored / full checkpointing
  u64 UA[2];    // one layer of them
  u64 Sbh;      // elements of one layer-boundary tensor, S*b*H
  u32 L, heads;
  u32 wT, wO, wG, wA;  // bytes per element of Theta, Omega, G, activation elements
  u32 ok;       // 1 if the shape was within the supported ranges
  u32 pad[3];
};
static_assert(sizeof(ModelRec) == 96, "model record is 96 bytes");

// One factorisation N = T*K*D.  The list of all factorisations of all N of a
// space (model independent, at most a few thousand entries) is the only
// enumeration table that exists.
struct __align__(16) Fact {
  u32 N, T, K, D;
};

// The space as the kernels see it (passed by value).
struct SpaceDev {
  const ModelRec* recs;
  const Fact* facts;
  const u32* order;   // the models in the order in which the sweeps' blocks take them (most work first)
  u64 ppm;            // points per model = n_facts * nvt * n_codes
  u32 n_models;
  u32 n_facts;        // factorisations of all N together ("units" per model)
  u32 nv, nt, nvt;    // activation variants, tensor-axis variants, product
  u32 nm;             // allowed modes on the data axis
  u32 modemap;        // digit d -> mode, 4 bits each, ascending modes
  u32 n_codes;        // nm^4
  u32 n3;             // nm^3
  u32 tp_max_valid, tp_coll;
  u32 sstar_units;    // unit buffers a gathered (S*) state holds at a time: 1, or 2 when gathers overlap computation
  u32 accum;          // micro-batches per step (gradient accumulation), >= 1
  u32 repl;           // copies of every shard (k-way replication of the sharded modes), >= 1
  u32 all_pow2;       // 1 if every device count of the space is a power of two (then every T, K, D is)
  u32 all_small;      // 1 if for every model (4 accum + 1) (w_T + w_O + w_G) (P + 2 unit) < 2^53: the device
                      // bytes, host bytes and data-axis volume of a (Theta, Omega, G) triple are then
                      // exact in a double
};

enum : u32 {
  SET_SHARDLIKE = (1u << PS_MODE_S) | (1u << PS_MODE_SG),
  SET_TRANSIENT = (1u << PS_MODE_SG) | (1u << PS_MODE_M),
  SET_UPDATE_ON_SHARD = (1u << PS_MODE_S) | (1u << PS_MODE_SG) | (1u << PS_MODE_O),
  SET_THETA_ALWAYS = (1u << PS_MODE_R) | (1u << PS_MODE_SG) | (1u << PS_MODE_O),
  SET_GRAD_FULL = (1u << PS_MODE_R) | (1u << PS_MODE_SG) | (1u << PS_MODE_M),
  SET_ACT_OWN = (1u << PS_MODE_R) | (1u << PS_MODE_M) | (1u << PS_MODE_O),
  SET_M_OR_O = (1u << PS_MODE_M) | (1u << PS_MODE_O)
};

__device__ __forceinline__ bool in_set(u32 set, u32 mode) { return (set >> mode) & 1u; }
__device__ __forceinline__ u32 digit_mode(u32 modemap, u32 digit) { return (modemap >> (4 * digit)) & 7u; }

// ---------------------------------------------------------------- division
// Divisors are degrees (< 2^24).  Powers of two, the common case, are shifts;
// the branch is uniform wherever a warp works on one factorisation.
__device__ __forceinline__ u64 div_floor(u64 a, u32 d) {
  if ((d & (d - 1)) == 0) return a >> (31 - __clz(d));
  if (a < ((u64)1 << 52)) {
    // The correctly rounded double quotient is off by less than a half, and never
    // below an integer the true quotient reaches, so its integer part is the
    // quotient or one more; the remainder tells which.
    u64 q = (u64)__double2ll_rz((double)(long long)a / (double)d);
    if ((long long)(a - q * d) < 0) --q;
    return q;
  }
  return a / d;
}
__device__ __forceinline__ u64 div_ceil(u64 a, u32 d) { return div_floor(a + (d - 1), d); }

// ---------------------------------------------------------------- per factorisation
// Quantities that depend on (model, T, K, D) only.  Remark 4: the tensor split
// is innermost, the pipeline split next, the data axis outermost.  Both model
// axes shard Theta, Omega and G (Table 2).
// k-way replication: the D devices of the data axis form k = gcd(repl, D) shard
// groups of G = D / k devices; a sharded state is cut into G shards, each held by
// the k devices at the same position of their groups.  Gathers run inside a
// group; a gradient is reduced to shards by a reduce-scatter inside every group
// and an all-reduce of each shard across its copies.
enum : u32 {
  CLS_SHARDED = 0,    // several shard positions (G > 1)
  CLS_ONE_DEVICE = 1, // D = 1: nothing moves, a shard is the tensor
  CLS_ALL_COPIES = 2  // G = 1 < D: a "shard" is the tensor, held by every device
};
struct UnitBase {
  u64 E2;     // elements of Theta (= Omega = G) left on one (t, k) position
  u64 sh;     // largest data-axis shard of them, ceil(E2 / G)   (eq. (2))
  u64 x;      // ring volume inside a shard group, E2 - floor(E2 / G)  (Section 2.3)
  u64 x2;     // all-reduce of the largest shard across its k copies, 2 (sh - floor(sh / k)); 0 if k = 1
  u64 x3;     // what an all-reduce over all D devices moves beyond 2 x; 0 if k = 1
  u32 G;      // shard positions
  u32 cls;    // CLS_*
  u64 u;      // reconstruction unit after the tensor split
  u64 tp_x;   // ring volume of a boundary tensor over the tensor axis
  u64 sbh_t;  // ceil(Sbh / T)
  u32 lps;    // layers per pipeline stage, ceil(L / K)
  u32 cv;     // PS_F_CV and its reason bits (axis form assumed)
  bool d1;    // one shard position (G == 1): a shard is the whole tensor
};

__device__ __forceinline__ u32 gcd_u32(u32 a, u32 b) {
  while (b) { const u32 t = a % b; a = b; b = t; }
  return a;
}

__device__ __forceinline__ UnitBase unit_base(const ModelRec& r, const Fact& f, u32 tp_max_valid,
                                              bool axis_form, u32 repl = 1) {
  UnitBase b;
  u64 E1 = div_ceil(r.P, f.T);
  b.E2 = div_ceil(E1, f.K);
  const u32 k = repl > 1 ? gcd_u32(repl, f.D) : 1u;
  b.G = f.D / k;
  u64 q = div_floor(b.E2, b.G);
  b.sh = q + ((q * b.G != b.E2) ? 1 : 0);
  b.x = b.E2 - q;
  b.x2 = 0;
  b.x3 = 0;
  if (k > 1) {
    b.x2 = 2 * (b.sh - div_floor(b.sh, k));
    b.x3 = 2 * ((b.E2 - div_floor(b.E2, f.D)) - b.x);
  }
  b.cls = f.D == 1 ? CLS_ONE_DEVICE : (b.G == 1 ? CLS_ALL_COPIES : CLS_SHARDED);
  b.u = div_ceil(r.unit, f.T);
  u64 qs = div_floor(r.Sbh, f.T);
  b.tp_x = r.Sbh - qs;
  b.sbh_t = qs + ((qs * f.T != r.Sbh) ? 1 : 0);
  u32 ql = (u32)div_floor((u64)r.L, f.K);
  bool k_layers = (ql * f.K == r.L);
  b.lps = ql + (k_layers ? 0 : 1);
  u32 qh = (u32)div_floor((u64)r.heads, f.T);
  bool t_heads = (qh * f.T == r.heads);
  bool tp_le = f.T <= tp_max_valid;
  bool whole = ((u64)f.T * f.K * f.D == (u64)f.N);
  u32 cv = (t_heads ? PS_F_T_DIV_HEADS : 0) | (k_layers ? PS_F_K_DIV_LAYERS : 0) |
           (tp_le ? PS_F_TP_LE_MAX : 0) | (axis_form ? PS_F_AXIS_FORM : 0);
  if (t_heads && k_layers && tp_le && axis_form && whole) cv |= PS_F_CV;
  b.cv = cv;
  b.d1 = (b.G == 1);
  return b;
}

// Degrees that are all powers of two (every benchmark configuration): the
// divisions become shifts.  Same values as unit_base / act_base.
struct Pow2 {
  u32 sT, sK, sD;
  u32 sC;     // log2 of the copies of a shard: gcd(repl, D) = the lowest set bit of repl, at most D
  u32 sG;     // log2 of the shard positions, sD - sC
  bool all;
};
__device__ __forceinline__ Pow2 pow2_of(const Fact& f) {          // one copy of every shard
  Pow2 p;
  p.all = (((f.T & (f.T - 1)) | (f.K & (f.K - 1)) | (f.D & (f.D - 1))) == 0);
  p.sT = 31 - __clz(f.T);
  p.sK = 31 - __clz(f.K);
  p.sD = 31 - __clz(f.D);
  p.sC = 0;
  p.sG = p.sD;
  return p;
}
__device__ __forceinline__ Pow2 pow2_of(const Fact& f, u32 repl) {
  Pow2 p = pow2_of(f);
  p.sC = min((u32)(__ffs(repl) - 1), p.sD);      // repl >= 1
  p.sG = p.sD - p.sC;
  return p;
}
__device__ __forceinline__ u64 ceil_shift(u64 a, u32 s) { return (a + (((u64)1 << s) - 1)) >> s; }

__device__ __forceinline__ UnitBase unit_base_pow2(const ModelRec& r, const Fact& f, const Pow2& p,
                                                   u32 tp_max_valid, bool axis_form) {
  UnitBase b;
  b.E2 = ceil_shift(ceil_shift(r.P, p.sT), p.sK);
  b.G = 1u << p.sG;
  b.sh = ceil_shift(b.E2, p.sG);
  b.x = b.E2 - (b.E2 >> p.sG);
  b.x2 = 2 * (b.sh - (b.sh >> p.sC));             // 0 when there is one copy
  b.x3 = 2 * ((b.E2 - (b.E2 >> p.sD)) - b.x);
  b.cls = f.D == 1 ? CLS_ONE_DEVICE : (p.sG == 0 ? CLS_ALL_COPIES : CLS_SHARDED);
  b.u = ceil_shift(r.unit, p.sT);
  b.tp_x = r.Sbh - (r.Sbh >> p.sT);
  b.sbh_t = ceil_shift(r.Sbh, p.sT);
  b.lps = (r.L + (f.K - 1)) >> p.sK;
  const bool k_layers = (r.L & (f.K - 1)) == 0;
  const bool t_heads = (r.heads & (f.T - 1)) == 0;
  const bool tp_le = f.T <= tp_max_valid;
  const bool whole = ((u64)f.T * f.K * f.D == (u64)f.N);
  u32 cv = (t_heads ? PS_F_T_DIV_HEADS : 0) | (k_layers ? PS_F_K_DIV_LAYERS : 0) |
           (tp_le ? PS_F_TP_LE_MAX : 0) | (axis_form ? PS_F_AXIS_FORM : 0);
  if (t_heads && k_layers && tp_le && axis_form && whole) cv |= PS_F_CV;
  b.cv = cv;
  b.d1 = (p.sG == 0);
  return b;
}

// the same with one copy of every shard (the shard positions are the D devices)
__device__ __forceinline__ UnitBase unit_base_pow2_one_copy(const ModelRec& r, const Fact& f, const Pow2& p,
                                                   u32 tp_max_valid, bool axis_form) {
  UnitBase b;
  b.E2 = ceil_shift(ceil_shift(r.P, p.sT), p.sK);
  b.G = f.D;
  b.sh = ceil_shift(b.E2, p.sD);
  b.x = b.E2 - (b.E2 >> p.sD);
  b.x2 = 0;
  b.x3 = 0;
  b.cls = f.D == 1 ? CLS_ONE_DEVICE : CLS_SHARDED;
  b.u = ceil_shift(r.unit, p.sT);
  b.tp_x = r.Sbh - (r.Sbh >> p.sT);
  b.sbh_t = ceil_shift(r.Sbh, p.sT);
  b.lps = (r.L + (f.K - 1)) >> p.sK;
  const bool k_layers = (r.L & (f.K - 1)) == 0;
  const bool t_heads = (r.heads & (f.T - 1)) == 0;
  const bool tp_le = f.T <= tp_max_valid;
  const bool whole = ((u64)f.T * f.K * f.D == (u64)f.N);
  u32 cv = (t_heads ? PS_F_T_DIV_HEADS : 0) | (k_layers ? PS_F_K_DIV_LAYERS : 0) |
           (tp_le ? PS_F_TP_LE_MAX : 0) | (axis_form ? PS_F_AXIS_FORM : 0);
  if (t_heads && k_layers && tp_le && axis_form && whole) cv |= PS_F_CV;
  b.cv = cv;
  b.d1 = (f.D == 1);
  return b;
}

// Activations of one replica for variant v (stored / checkpointed) when the
// tensor axis shards them (tau = 0, sequence parallel) or not (tau = 1); the
// pipeline axis leaves them whole (Table 2).  Bytes.
struct ActBase {
  u64 EA, shA, uA;
};
__device__ __forceinline__ ActBase act_base(const ModelRec& r, const Fact& f, u32 v, u32 tau, u32 G) {
  ActBase a;
  a.EA = tau == 0 ? div_ceil(r.A[v], f.T) : r.A[v];
  a.uA = tau == 0 ? div_ceil(r.UA[v], f.T) : r.UA[v];
  a.shA = div_ceil(a.EA, G);                      // G = shard positions of the data axis
  return a;
}

__device__ __forceinline__ ActBase act_base_pow2(const ModelRec& r, const Pow2& p, u32 v, u32 tau) {
  ActBase a;
  const u32 s = tau == 0 ? p.sT : 0;
  a.EA = ceil_shift(r.A[v], s);
  a.uA = ceil_shift(r.UA[v], s);
  a.shA = ceil_shift(a.EA, p.sG);
  return a;
}
__device__ __forceinline__ ActBase act_base_pow2_one_copy(const ModelRec& r, const Pow2& p, u32 v, u32 tau) {
  ActBase a;
  const u32 s = tau == 0 ? p.sT : 0;
  a.EA = ceil_shift(r.A[v], s);
  a.uA = ceil_shift(r.UA[v], s);
  a.shA = ceil_shift(a.EA, p.sD);
  return a;
}

// tensor-axis and pipeline-axis traffic per step (not priced by Theorem 2):
// per layer of a stage, tp_coll all-reduces of a boundary tensor over T
// devices; between stages the boundary tensor goes forward and its gradient
// comes back, so the busiest device sends two of them when it has a neighbour on
// either side (K >= 3) and one when there are two stages; all of it once per
// micro-batch (accum micro-batches per step)
__device__ __forceinline__ u64 model_axis_traffic(const ModelRec& r, const Fact& f,
                                                  const UnitBase& b, u32 tau, u32 tp_coll,
                                                  u32 accum = 1) {
  const u32 per_elem = 2 * tp_coll * r.wA;                 // <= 2 * 64 * 16
  const u64 tp = b.tp_x * (u64)(b.lps * per_elem);         // lps <= 2^10
  const u32 sends = f.K >= 3 ? 2u : f.K - 1;                // K >= 1
  const u64 pp = (tau == 0 ? b.sbh_t : r.Sbh) * (u64)(sends * r.wA);
  return (tp + pp) * accum;
}

// Theorem 1: persistent plus transient elements of a state under mode pi.  A
// gathered state (S*) holds sstar_units unit buffers: one, or two when the next
// unit is gathered while the current one is in use (the theorem's proof, case S*).
__device__ __forceinline__ u64 mu_elems(u32 pi, u64 full, u64 shard, u64 unit, u32 sstar_units = 1) {
  u64 p = (pi == PS_MODE_R) ? full : (in_set(SET_SHARDLIKE, pi) ? shard : 0);
  u64 t = (pi == PS_MODE_SG) ? unit * sstar_units : (pi == PS_MODE_M ? unit : 0);
  return p + t;
}

// ---------------------------------------------------------------- one point
struct PointOut {
  u64 mem, comm_paper, comm_ext, host;
  u32 flags;  // without PS_F_FEASIBLE
};

// flags of a point from its four modes; ext_data_zero says whether the data
// axis moves nothing beyond Theorem 2's terms
__device__ __forceinline__ u32 point_flags(u32 th, u32 om, u32 gr, u32 ac, bool d1, u32 cv,
                                           bool ext_data_zero) {
  bool omega_full = (om == PS_MODE_R) || (d1 && in_set(SET_SHARDLIKE, om));
  bool theta_avail = in_set(SET_THETA_ALWAYS, th) || (th == PS_MODE_S && d1) ||
                     (th == PS_MODE_M && omega_full);
  bool act_avail = d1 || in_set(SET_ACT_OWN, ac);
  bool grad_cover = d1 || in_set(SET_UPDATE_ON_SHARD, om) || in_set(SET_GRAD_FULL, gr);
  bool sc = (om != PS_MODE_M);
  u32 modes_seen = (1u << th) | (1u << om) | (1u << gr) | (1u << ac);
  bool uses_host = (modes_seen >> PS_MODE_O) & 1u;
  bool priced = ext_data_zero && !(modes_seen & SET_M_OR_O);
  u32 fl = cv;
  if (theta_avail && act_avail && grad_cover) fl |= PS_F_GI;
  if (sc) fl |= PS_F_SC;
  if (theta_avail) fl |= PS_F_THETA_AVAIL;
  if (act_avail) fl |= PS_F_ACT_AVAIL;
  if (grad_cover) fl |= PS_F_GRAD_COVER;
  if (uses_host) fl |= PS_F_USES_HOST;
  if (priced) fl |= PS_F_PAPER_PRICED;
  return fl;
}

// The whole evaluation of one point, with nothing hoisted.  Used where single
// points are needed (ps_check_composition, re-deriving host bytes and flags of
// the few entries a sweep emits).
// sstar_units: unit buffers of a gathered state; accum: micro-batches per step --
// what happens once per micro-batch (gathering Theta for forward and backward,
// loading offloaded Theta, moving activations to the host and back, tensor- and
// pipeline-axis traffic) is counted accum times, what happens once per step
// (synchronising gradients, the update and what it moves) once.
__device__ __forceinline__ PointOut eval_point(const ModelRec& r, const Fact& f, u32 v, u32 tau,
                                               u32 th, u32 om, u32 gr, u32 ac, u32 tp_max_valid,
                                               u32 tp_coll, bool axis_form, u32 sstar_units = 1,
                                               u32 accum = 1, u32 repl = 1) {
  UnitBase b = unit_base(r, f, tp_max_valid, axis_form, repl);
  ActBase a = act_base(r, f, v, tau, b.G);
  PointOut o;
  o.mem = r.wT * mu_elems(th, b.E2, b.sh, b.u, sstar_units) + r.wO * mu_elems(om, b.E2, b.sh, b.u, sstar_units) +
          r.wG * mu_elems(gr, b.E2, b.sh, b.u, sstar_units) + mu_elems(ac, a.EA, a.shA, a.uA, sstar_units);
  u64 xT = b.x * r.wT, xO = b.x * r.wO, xG = b.x * r.wG;
  // a gradient reduced to shards (inside the group, then across the copies of a shard), and
  // all-reduced over all devices; with one copy of every shard these are xG and 2 xG
  const u64 to_shards = xG + b.x2 * r.wG, all_reduce = 2 * xG + b.x3 * r.wG;
  // Theorem 2
  o.comm_paper = (gr == PS_MODE_R ? all_reduce : 0) + (gr == PS_MODE_S ? to_shards : 0) +
                 (th == PS_MODE_SG ? 2 * xT * accum : 0);
  bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
  u64 ext = 0;
  if (th == PS_MODE_O) ext += 2 * xT * accum;
  if (th == PS_MODE_R && on_shard) ext += xT;
  if (gr == PS_MODE_SG) ext += to_shards + xG;
  if (gr == PS_MODE_M) ext += on_shard ? to_shards : all_reduce;
  if (gr == PS_MODE_O) ext += to_shards;
  if (om == PS_MODE_SG) ext += xO;
  o.comm_ext = ext + model_axis_traffic(r, f, b, tau, tp_coll, accum);
  o.host = (th == PS_MODE_O ? (2 * accum + 1) * b.sh * r.wT : 0) + (om == PS_MODE_O ? 2 * b.sh * r.wO : 0) +
           (gr == PS_MODE_O ? 2 * b.sh * r.wG : 0) + (ac == PS_MODE_O ? 2 * a.EA * accum : 0);
  o.flags = point_flags(th, om, gr, ac, b.d1, b.cv, ext == 0);
  return o;
}

// ---------------------------------------------------------------- filters on (Theta, Omega, G) triples
// bits of a triple's static description
enum : u32 {
  T_THETA_AVAIL = 1u << 0, T_GRAD_COVER = 1u << 1, T_SC = 1u << 2, T_HOST = 1u << 3,
  T_M_OR_O = 1u << 4, T_EXT0 = 1u << 5
};

// cls: CLS_* of the factorisation (a shard is the whole tensor unless CLS_SHARDED)
__device__ __forceinline__ u32 triple_bits(u32 th, u32 om, u32 gr, u32 cls) {
  const bool d1 = cls != CLS_SHARDED;
  const bool on_shard = in_set(SET_UPDATE_ON_SHARD, om);
  const bool omega_full = (om == PS_MODE_R) || (d1 && in_set(SET_SHARDLIKE, om));
  const bool theta_avail = in_set(SET_THETA_ALWAYS, th) || (th == PS_MODE_S && d1) ||
                           (th == PS_MODE_M && omega_full);
  const bool grad_cover = d1 || on_shard || in_set(SET_GRAD_FULL, gr);
  const u32 seen = (1u << th) | (1u << om) | (1u << gr);
  // data-axis traffic beyond Theorem 2: none with a single device (nothing moves); with
  // every device holding every "shard" the gathers move nothing, the gradient modes that
  // Theorem 2 does not price still do
  const bool grad_unpriced = in_set((1u << PS_MODE_SG) | SET_M_OR_O, gr);
  const bool ext0 = cls == CLS_ONE_DEVICE ||
                    (cls == CLS_ALL_COPIES ? !grad_unpriced
                                           : !((th == PS_MODE_O) || (th == PS_MODE_R && on_shard) ||
                                               grad_unpriced || om == PS_MODE_SG));
  return (theta_avail ? T_THETA_AVAIL : 0) | (grad_cover ? T_GRAD_COVER : 0) |
         (om != PS_MODE_M ? T_SC : 0) | ((seen >> PS_MODE_O) & 1u ? T_HOST : 0) |
         ((seen & SET_M_OR_O) ? T_M_OR_O : 0) | (ext0 ? T_EXT0 : 0);
}

// which activation digits give a point with every required flag, for a triple
// with static bits `tb` (the composition bits are checked per unit)
__device__ __forceinline__ u32 allowed_act_digits(u32 tb, u32 req, u32 all, u32 own, u32 is_o, u32 not_mo) {
  u32 ok = all;
  if ((req & PS_F_SC) && !(tb & T_SC)) ok = 0;
  if ((req & PS_F_THETA_AVAIL) && !(tb & T_THETA_AVAIL)) ok = 0;
  if ((req & PS_F_GRAD_COVER) && !(tb & T_GRAD_COVER)) ok = 0;
  if (req & PS_F_GI) ok &= ((tb & T_THETA_AVAIL) && (tb & T_GRAD_COVER)) ? own : 0;
  if (req & PS_F_ACT_AVAIL) ok &= own;
  if (req & PS_F_USES_HOST) ok &= (tb & T_HOST) ? all : is_o;
  if (req & PS_F_PAPER_PRICED) ok &= ((tb & T_EXT0) && !(tb & T_M_OR_O)) ? not_mo : 0;
  return ok;
}

// linear index within a model -> unit, variant, digits of the data-axis code
struct LocalPoint {
  u32 unit, v, tau, dth, dom, dgr, dac;
};
__device__ __forceinline__ LocalPoint decode_local(const SpaceDev& sp, u32 lidx) {
  LocalPoint p;
  u32 per_unit = sp.nvt * sp.n_codes;
  p.unit = lidx / per_unit;
  u32 r = lidx - p.unit * per_unit;
  u32 vt = r / sp.n_codes;
  u32 code = r - vt * sp.n_codes;
  p.v = vt / sp.nt;
  p.tau = vt - p.v * sp.nt;
  p.dth = code % sp.nm; code /= sp.nm;
  p.dom = code % sp.nm; code /= sp.nm;
  p.dgr = code % sp.nm;
  p.dac = code / sp.nm;
  return p;
}

// status word bits set by kernels
enum : u32 {
  ST_BAD_SHAPE = 1u << 0,      // a model shape outside the supported ranges
  ST_SELF_CHECK = 1u << 2,     // an emitted entry did not re-evaluate to itself
  ST_TRUNCATED = 1u << 3,      // a frontier was longer than the caller's max_entries (a notice, not a fault)
  ST_BAD_CASE = 1u << 4        // a verifier case outside the supported ranges or the given data
};

// TEST INFRASTRUCTURE -- the CPU oracle of the placement-semantics sweep.
//
// A plain, slow, one-point-at-a-time evaluation of the paper's rules, written
// from the paper and used only to check the CUDA library (tests, the smoke
// check and the benchmark's CPU-baseline leg).  It shares no code with the
// CUDA path: own structs, own helpers, fresh divisions for every point, no
// tables, no hoisting.  Nothing in the product may call it.
//
// What follows which passage of the paper
//   sizes |Theta| |Omega| |G| in bytes        Remark 1, Table 1
//   P = 12 L H^2 (+ V H embeddings)            Section 2.1 and its footnote
//   reconstruction unit 12 H^2 elements        Definition 3
//   ring collective volumes                    Section 2.3
//   shard boundaries floor(i |X| / N)          Definition 1, eq. (2)
//   per-state memory mu(pi, s)                 Theorem 1
//   priced communication                       Theorem 2, Corollary 1
//   gradient integrity / state consistency     Theorems 3 and 4
//   composition, nesting order, validity       Definition 5, Theorems 6-7,
//                                              Proposition 1, Remark 4, Table 2
//
// Readings taken where the paper is silent (each also listed in the design
// notes): element-granular shards, per-device figure = largest shard; ring
// volume = E - floor(E/n) elements sent by the busiest device; activations
// from the selective-recomputation analysis the paper cites for sequence
// parallelism (34 S b H + 5 a S^2 b bytes per layer; 2 S b H with full
// checkpointing); offloaded state lives as shards on the hosts.
//
// Pins: tests/test_oracle_pins.py (the paper's printed numbers, closed forms,
// invariants, Table 2), tests/test_oracle_vs_sim.py (a brute-force fp64
// training simulator with explicit shard bookkeeping) and
// tests/test_oracle_vs_composition_sim.py (a tensor x pipeline x data grid run
// of a small network whose rings and stage-to-stage transfers count the bytes
// they send: pins the tensor- and pipeline-axis traffic, with the number of
// all-reduces per layer left a parameter).  The paper prints no activation
// size, no host-link figure and no model-axis volume, so against the paper
// these three stay readings.  "parity unpinned": the coefficients of the
// activation formula (34 S b H + 5 a S^2 b; 2 S b H) -- only their wiring into
// the rules (times L, checkpoint variant, unit = one layer, tensor-axis split)
// is pinned.

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>

typedef uint64_t u64;
typedef uint32_t u32;

namespace {

// ---------------------------------------------------------------- inputs
struct OShape {  // one model, 48 bytes (layout of the input table)
  u64 param_elems_override;
  u32 layers, hidden, heads, vocab, seq, micro_batch;
  uint8_t w_param, w_grad, w_opt, w_act;
  uint8_t unit_from_shape, act_enabled;
  uint8_t pad[10];
};
static_assert(sizeof(OShape) == 48, "input record is 48 bytes");

struct ODesc {  // the design space
  const OShape* models;
  u32 n_models;
  const u32* n_values;
  u32 n_n;
  u32 t_enum_max, k_enum_max, tp_max_valid;
  u32 n_act_variants, n_tpa_variants, mode_mask, tp_coll_per_layer;
  u32 sstar_units;       // 0 or 1: Theorem 1 as stated; 2: overlapped gathers (the proof's note)
  u32 grad_accum_steps;  // 0 or 1: none; g: micro-batches per step ("Limitations")
  u32 replication_k;     // 0 or 1: plain sharding; k: every shard is held k times (Section 1's
                         // "k-way replication for 1 < k < N")
};

struct OFilter {
  u64 host_cap;
  u32 require_flags;
  u32 comm_kind;  // 0: Theorem-2 volume only, 1: plus the unpriced traffic
  u64 cap_bytes;
};

struct OEntry {  // 40 bytes
  u64 mem, comm, host, idx;
  u32 flags, pad;
};
static_assert(sizeof(OEntry) == 40, "entry is 40 bytes");

struct OPoint {
  u32 model, N, T, K, D, act_variant, tpa_variant;
  uint16_t code_dp, code_tp, code_pp, pad;
};

// what one model contributes to the formulas
struct ORecord {
  u64 P;        // parameter elements
  u64 unit;     // reconstruction unit, elements (Definition 3), 0 if unknown
  u64 A[2];     // activation bytes of one replica: [0] stored, [1] full checkpointing
  u64 UA[2];    // one layer's activations
  u64 Sbh;      // elements of one boundary tensor S*b*H
  u32 L, heads;
  u32 w_theta, w_omega, w_grad, w_act;
};

enum Mode { R = 0, S = 1, SG = 2, M = 3, O = 4 };  // SG is the paper's S*

enum : u32 {
  F_GI = 1u << 0, F_SC = 1u << 1, F_CV = 1u << 2, F_FEASIBLE = 1u << 3,
  F_T_HEADS = 1u << 4, F_K_LAYERS = 1u << 5, F_TP_LE_MAX = 1u << 6, F_AXIS_FORM = 1u << 7,
  F_THETA_AVAIL = 1u << 8, F_ACT_AVAIL = 1u << 9, F_GRAD_COVER = 1u << 10,
  F_USES_HOST = 1u << 11, F_PAPER_PRICED = 1u << 12
};

struct OResult {
  u64 mem, comm_paper, comm_ext, host;
  u32 flags;
};

u64 ceil_div(u64 a, u64 b) { return (a + b - 1) / b; }

// Section 2.3: a ring reduce-scatter or all-gather over n devices moves
// (n-1)/n of the tensor; with element shards of eq. (2) the busiest device
// sends every element except its smallest possible shard.
u64 ring_elems(u64 E, u64 n) { return E - E / n; }

// ---------------------------------------------------------------- model record
ORecord derive_record(const OShape& s) {
  ORecord r;
  u64 L = s.layers, H = s.hidden, V = s.vocab, Sq = s.seq, b = s.micro_batch, a = s.heads;
  // Section 2.1: P ~ 12 L H^2, embeddings add V H (footnote)
  r.P = s.param_elems_override ? s.param_elems_override : 12 * L * H * H + V * H;
  // Definition 3: one transformer layer, 12 H^2 elements
  r.unit = s.unit_from_shape ? 12 * H * H : 0;
  if (s.act_enabled) {
    u64 per_layer_stored = 34 * Sq * b * H + 5 * a * Sq * Sq * b;
    u64 per_layer_ckpt = 2 * Sq * b * H;
    r.A[0] = L * per_layer_stored;
    r.A[1] = L * per_layer_ckpt;
    r.UA[0] = per_layer_stored;
    r.UA[1] = per_layer_ckpt;
  } else {
    r.A[0] = r.A[1] = r.UA[0] = r.UA[1] = 0;
  }
  r.Sbh = Sq * b * H;
  r.L = s.layers;
  r.heads = s.heads;
  // Remark 1: 2 B parameters, 2 B gradients, 12 B optimizer incl. master copy
  r.w_theta = s.w_param;
  r.w_omega = s.w_opt;
  r.w_grad = s.w_grad;
  r.w_act = s.w_act;
  return r;
}

// ---------------------------------------------------------------- one point
// Theorem 1 on the data axis: persistent and transient elements of a state of
// E elements whose reconstruction unit is u, under mode pi over D devices.
// The proof of case S* notes that an implementation which overlaps the gather
// of the next unit with computation holds two unit buffers: gather_buffers.
void mu_elems(int pi, u64 E, u64 u, u64 D, u64 gather_buffers, u64* persistent, u64* transient) {
  switch (pi) {
    case R:  *persistent = E;              *transient = 0; break;
    case S:  *persistent = ceil_div(E, D); *transient = 0; break;
    case SG: *persistent = ceil_div(E, D); *transient = gather_buffers * u; break;
    case M:  *persistent = 0;              *transient = u; break;
    default: *persistent = 0;              *transient = 0; break;  // O
  }
}

u64 gcd_u64(u64 a, u64 b) { while (b) { u64 t = a % b; a = b; b = t; } return a; }

OResult eval_point(const ORecord& m, u64 N, u64 T, u64 K, u64 D, int v, int tau,
                   int pi_theta, int pi_omega, int pi_grad, int pi_act,
                   u32 tp_max_valid, u32 tp_coll_per_layer, bool axis_form_ok,
                   u32 sstar_units = 1, u32 grad_accum_steps = 1, u32 replication_k = 1) {
  OResult out;
  // the extensions: unit buffers of a gathered state, micro-batches per step
  const u64 nbuf = sstar_units ? sstar_units : 1;
  const u64 g = grad_accum_steps ? grad_accum_steps : 1;
  // k-way replication of the sharded modes: the D devices of the data axis form
  // k shard groups of Gp = D / k devices; a sharded state is cut into Gp shards,
  // each held by the k devices at the same position of their groups.  Where the
  // requested k does not divide D the largest common divisor is used.
  const u64 k = gcd_u64(replication_k ? replication_k : 1, D);
  const u64 Gp = D / k;
  // Remark 4: tensor parallelism innermost, pipeline in the middle, data
  // outermost.  Table 2: both model axes shard Theta, Omega and G.
  u64 E1 = ceil_div(m.P, T);        // intra-layer split
  u64 u1 = ceil_div(m.unit, T);     // ... which also splits every layer
  u64 E2 = ceil_div(E1, K);         // inter-layer split
  u64 u2 = u1;                      // ... which leaves a layer whole
  // activations: the tensor axis shards them (tau = 0, sequence parallel) or
  // replicates them (tau = 1); the pipeline axis replicates them (Table 2)
  u64 EA = (tau == 0) ? ceil_div(m.A[v], T) : m.A[v];
  u64 uA = (tau == 0) ? ceil_div(m.UA[v], T) : m.UA[v];

  u64 p, t;
  out.mem = 0;
  mu_elems(pi_theta, E2, u2, Gp, nbuf, &p, &t); out.mem += (u64)m.w_theta * (p + t);
  mu_elems(pi_omega, E2, u2, Gp, nbuf, &p, &t); out.mem += (u64)m.w_omega * (p + t);
  mu_elems(pi_grad,  E2, u2, Gp, nbuf, &p, &t); out.mem += (u64)m.w_grad  * (p + t);
  mu_elems(pi_act,   EA, uA, Gp, nbuf, &p, &t); out.mem += p + t;   // already bytes

  u64 sh = ceil_div(E2, Gp);      // largest shard of Theta / Omega / G
  u64 x = ring_elems(E2, Gp);     // ring volume in elements of a gather or scatter inside a shard group
  u64 xT = x * m.w_theta, xO = x * m.w_omega;
  // a gradient reduced to shards: reduce-scatter inside the shard group, then an
  // all-reduce of every shard across its k copies (the busiest device holds the
  // largest shard); an all-reduce over all D devices
  u64 to_shards = (x + 2 * ring_elems(sh, k)) * m.w_grad;
  u64 all_reduce = 2 * ring_elems(E2, D) * m.w_grad;
  u64 gatherG = x * m.w_grad;

  // Theorem 2: the three priced transitions, nothing else.  With gradient
  // accumulation ("Limitations") a step runs g micro-batches and synchronises
  // gradients once: the gradient terms stay, and whatever every micro-batch's
  // forward and backward need is paid g times.  Per micro-batch the gradient
  // terms are thus divided by g, as the paper says.
  out.comm_paper = 0;
  if (pi_grad == R) out.comm_paper += all_reduce;      // all-reduce, once per step
  if (pi_grad == S) out.comm_paper += to_shards;       // reduce-scatter (to shards), once per step
  if (pi_theta == SG) out.comm_paper += g * 2 * xT;    // gather for forward and backward of every micro-batch

  // the update is committed on a shard when Omega's home is a shard
  bool update_on_shard = (pi_omega == S || pi_omega == SG || pi_omega == O);

  // traffic of the execution model that Theorem 2 does not price
  u64 ext_data = 0;
  if (pi_theta == O) ext_data += g * 2 * xT;                 // gather after each host load, every micro-batch
  if (pi_theta == R && update_on_shard) ext_data += xT;      // re-replicate updated shards
  if (pi_grad == SG) ext_data += to_shards + gatherG;        // reduce-scatter, then gather
  if (pi_grad == M) ext_data += update_on_shard ? to_shards : all_reduce;
  if (pi_grad == O) ext_data += to_shards;                   // reduce-scatter before offload
  if (pi_omega == SG) ext_data += xO;                        // gather Omega for the update
  u64 layers_per_stage = ceil_div(m.L, K);
  u64 ext_tp = layers_per_stage * tp_coll_per_layer * 2 * ring_elems(m.Sbh, T) * m.w_act;
  // between pipeline stages a device passes on what it holds of the boundary tensor
  // (all of it, or its 1/T shard under sequence parallelism): an interior stage sends
  // one forward and one gradient backward, the first and the last stage only one of
  // the two -- bytes sent by the busiest device, as for the rings (Section 2.3)
  u64 boundary_sends = (K >= 3) ? 2 : (K == 2 ? 1 : 0);
  u64 ext_pp = boundary_sends * ceil_div(m.Sbh, tau == 0 ? T : 1) * m.w_act;
  out.comm_ext = ext_data + g * (ext_tp + ext_pp);           // model-axis traffic of every micro-batch

  // host-link bytes (mode O): shards live on the hosts
  out.host = 0;
  if (pi_theta == O) out.host += (2 * g + 1) * sh * m.w_theta;   // load for fwd and bwd of every micro-batch, one store
  if (pi_omega == O) out.host += 2 * sh * m.w_omega;   // load, store
  if (pi_grad == O)  out.host += 2 * sh * m.w_grad;    // store, load at the update
  if (pi_act == O)   out.host += g * 2 * EA;           // store after fwd, load for bwd, every micro-batch

  // Theorems 3 and 4 as static predicates over the placement
  // (a "shard" is the whole tensor when there is one shard position: one device, or
  // as many copies as devices)
  bool whole = (Gp == 1);
  bool omega_full = (pi_omega == R) || (whole && (pi_omega == S || pi_omega == SG));
  bool theta_avail = (pi_theta == R || pi_theta == SG || pi_theta == O) ||
                     (pi_theta == S && whole) || (pi_theta == M && omega_full);
  bool act_avail = (pi_act == R || pi_act == M || pi_act == O) || whole;
  bool grad_cover = update_on_shard || (pi_grad == R || pi_grad == SG || pi_grad == M) || whole;
  bool gi = theta_avail && act_avail && grad_cover;
  bool sc = (pi_omega != M);

  // Theorems 6-7, Proposition 1, Remark 4
  bool t_heads = (m.heads % T) == 0;
  bool k_layers = (m.L % K) == 0;
  bool tp_le = T <= tp_max_valid;
  bool cv = (T * K * D == N) && t_heads && k_layers && tp_le && axis_form_ok;

  bool uses_host = pi_theta == O || pi_omega == O || pi_grad == O || pi_act == O;
  bool any_m_or_o = uses_host || pi_theta == M || pi_omega == M || pi_grad == M || pi_act == M;
  bool paper_priced = (ext_data == 0) && !any_m_or_o;

  out.flags = (gi ? F_GI : 0) | (sc ? F_SC : 0) | (cv ? F_CV : 0) |
              (t_heads ? F_T_HEADS : 0) | (k_layers ? F_K_LAYERS : 0) |
              (tp_le ? F_TP_LE_MAX : 0) | (axis_form_ok ? F_AXIS_FORM : 0) |
              (theta_avail ? F_THETA_AVAIL : 0) | (act_avail ? F_ACT_AVAIL : 0) |
              (grad_cover ? F_GRAD_COVER : 0) | (uses_host ? F_USES_HOST : 0) |
              (paper_priced ? F_PAPER_PRICED : 0);
  return out;
}

// ---------------------------------------------------------------- enumeration
struct Fact { u32 T, K, D; };

// all (T, K) with T | N, T <= t_max, K | N/T, K <= k_max; T ascending, then K
std::vector<Fact> factorisations(u32 N, u32 t_max, u32 k_max) {
  std::vector<Fact> out;
  for (u32 T = 1; T <= N && T <= t_max; ++T) {
    if (N % T) continue;
    u32 rest = N / T;
    for (u32 K = 1; K <= rest && K <= k_max; ++K) {
      if (rest % K) continue;
      out.push_back({T, K, rest / K});
    }
  }
  return out;
}

std::vector<int> allowed_modes(u32 mask) {
  std::vector<int> out;
  for (int m = 0; m < 5; ++m)
    if (mask & (1u << m)) out.push_back(m);
  return out;
}

struct Space {
  const ODesc* d;
  std::vector<std::vector<Fact>> facts;  // per entry of n_values
  std::vector<int> modes;
  u64 n_codes, pts_per_model;
  explicit Space(const ODesc* desc) : d(desc) {
    modes = allowed_modes(desc->mode_mask);
    u64 nm = modes.size();
    n_codes = nm * nm * nm * nm;
    pts_per_model = 0;
    for (u32 i = 0; i < desc->n_n; ++i) {
      facts.push_back(factorisations(desc->n_values[i], desc->t_enum_max, desc->k_enum_max));
      pts_per_model += (u64)facts.back().size() * desc->n_act_variants * desc->n_tpa_variants * n_codes;
    }
  }
  u64 size() const { return pts_per_model * d->n_models; }

  struct Decoded {
    u32 model, N, T, K, D, v, tau;
    int pi[4];   // theta, omega, grad, act
    u32 code;    // pi[0] + 5 pi[1] + 25 pi[2] + 125 pi[3]
  };

  // model-major; device counts in the given order; factorisations; activation
  // variant; tensor-axis activation variant; data-axis code fastest, its
  // Theta digit fastest of all
  Decoded decode(u64 idx) const {
    Decoded p;
    p.model = (u32)(idx / pts_per_model);
    u64 r = idx % pts_per_model;
    u64 per_fact = (u64)d->n_act_variants * d->n_tpa_variants * n_codes;
    u32 i = 0;
    while (r >= facts[i].size() * per_fact) { r -= facts[i].size() * per_fact; ++i; }
    p.N = d->n_values[i];
    const Fact& f = facts[i][r / per_fact];
    r %= per_fact;
    p.T = f.T; p.K = f.K; p.D = f.D;
    p.v = (u32)(r / (d->n_tpa_variants * n_codes));
    r %= d->n_tpa_variants * n_codes;
    p.tau = (u32)(r / n_codes);
    r %= n_codes;
    u64 nm = modes.size();
    p.code = 0;
    u32 weight = 1;
    for (int s = 0; s < 4; ++s) {
      p.pi[s] = modes[r % nm];
      r /= nm;
      p.code += weight * p.pi[s];
      weight *= 5;
    }
    return p;
  }

  OResult eval(u64 idx) const {
    Decoded p = decode(idx);
    ORecord rec = derive_record(d->models[p.model]);
    return eval_point(rec, p.N, p.T, p.K, p.D, p.v, p.tau, p.pi[0], p.pi[1], p.pi[2], p.pi[3],
                      d->tp_max_valid, d->tp_coll_per_layer, true, d->sstar_units, d->grad_accum_steps,
                      d->replication_k);
  }
};

// a point under a filter and one capacity: flags gain the FEASIBLE bit; the
// point survives if it fits, its host traffic fits and it has every required bit
bool passes(const OResult& r, const OFilter& f, u64 cap, u32* flags_out) {
  u32 fl = r.flags | (r.mem <= cap ? F_FEASIBLE : 0);
  *flags_out = fl;
  return r.mem <= cap && r.host <= f.host_cap && (fl & f.require_flags) == f.require_flags;
}

u64 objective_comm(const OResult& r, const OFilter& f) {
  return f.comm_kind == 0 ? r.comm_paper : r.comm_paper + r.comm_ext;
}

// Pareto frontier by the plain definition: keep p unless some kept q has
// q.mem <= p.mem and q.comm <= p.comm; on arrival p evicts everything it
// dominates.  Points arrive in index order, so of several points with equal
// (mem, comm) the smallest index stays.  Kept sorted by mem ascending.
void frontier_insert(std::vector<OEntry>& fr, const OEntry& p) {
  for (const OEntry& q : fr)
    if (q.mem <= p.mem && q.comm <= p.comm) return;
  std::vector<OEntry> keep;
  for (const OEntry& q : fr)
    if (!(p.mem <= q.mem && p.comm <= q.comm)) keep.push_back(q);
  keep.push_back(p);
  std::sort(keep.begin(), keep.end(), [](const OEntry& a, const OEntry& b) { return a.mem < b.mem; });
  fr.swap(keep);
}

void reduce_model(const Space& sp, u32 model, const OFilter& f, const u64* caps, u32 n_caps,
                  u32 kind, u32 max_entries, OEntry* out, u32* counts) {
  for (u32 c = 0; c < n_caps; ++c) {
    std::vector<OEntry> acc;
    u64 first = (u64)model * sp.pts_per_model;
    for (u64 idx = first; idx < first + sp.pts_per_model; ++idx) {
      OResult r = sp.eval(idx);
      u32 fl;
      if (!passes(r, f, caps[c], &fl)) continue;
      OEntry e{r.mem, objective_comm(r, f), r.host, idx, fl, 0};
      if (kind == 0) frontier_insert(acc, e);
      else acc.push_back(e);
    }
    if (kind != 0) {
      // top-k: smallest by (comm, mem, idx)
      std::sort(acc.begin(), acc.end(), [](const OEntry& a, const OEntry& b) {
        if (a.comm != b.comm) return a.comm < b.comm;
        if (a.mem != b.mem) return a.mem < b.mem;
        return a.idx < b.idx;
      });
    }
    OEntry* dst = out + ((u64)model * n_caps + c) * max_entries;
    counts[(u64)model * n_caps + c] = (u32)acc.size();
    for (u32 i = 0; i < max_entries; ++i) {
      if (i < acc.size()) dst[i] = acc[i];
      else std::memset(&dst[i], 0, sizeof(OEntry));
    }
  }
}

}  // namespace

// ---------------------------------------------------------------- C interface
extern "C" {

u64 orc_space_size(const ODesc* d) { return Space(d).size(); }

u64 orc_points_per_model(const ODesc* d) { return Space(d).pts_per_model; }

u32 orc_num_factorisations(u32 N, u32 t_max, u32 k_max) {
  return (u32)factorisations(N, t_max, k_max).size();
}

void orc_decode(const ODesc* d, u64 idx, OPoint* out) {
  Space sp(d);
  Space::Decoded p = sp.decode(idx);
  out->model = p.model; out->N = p.N; out->T = p.T; out->K = p.K; out->D = p.D;
  out->act_variant = p.v; out->tpa_variant = p.tau;
  out->code_dp = (uint16_t)p.code;
  out->code_tp = p.tau == 0 ? 156 : 31;   // Table 2: (S,S,S,S) or (S,S,S,R)
  out->code_pp = 31;                      // Table 2: (S,S,S,R)
  out->pad = 0;
}

// every point of [first, first+count); any output may be null.  With a filter
// the flags carry the FEASIBLE bit for filter->cap_bytes.
void orc_eval_range(const ODesc* d, u64 first, u64 count, const OFilter* filter,
                    u64* mem, u64* comm_paper, u64* comm_ext, u64* host, u32* flags) {
  Space sp(d);
  for (u64 i = 0; i < count; ++i) {
    OResult r = sp.eval(first + i);
    u32 fl = r.flags;
    if (filter) passes(r, *filter, filter->cap_bytes, &fl);
    if (mem) mem[i] = r.mem;
    if (comm_paper) comm_paper[i] = r.comm_paper;
    if (comm_ext) comm_ext[i] = r.comm_ext;
    if (host) host[i] = r.host;
    if (flags) flags[i] = fl;
  }
}

// survivors of the filter, densely, in index order; returns how many
u64 orc_compact_range(const ODesc* d, u64 first, u64 count, const OFilter* filter, u64* idx_out,
                      u64* mem, u64* comm_paper, u64* comm_ext, u64* host, u32* flags) {
  Space sp(d);
  u64 n = 0;
  for (u64 i = 0; i < count; ++i) {
    OResult r = sp.eval(first + i);
    u32 fl;
    if (!passes(r, *filter, filter->cap_bytes, &fl)) continue;
    if (idx_out) idx_out[n] = first + i;
    if (mem) mem[n] = r.mem;
    if (comm_paper) comm_paper[n] = r.comm_paper;
    if (comm_ext) comm_ext[n] = r.comm_ext;
    if (host) host[n] = r.host;
    if (flags) flags[n] = fl;
    ++n;
  }
  return n;
}

// kind 0: Pareto frontier of (mem, comm), both minimised, sorted by mem;
// kind 1: the max_entries smallest by (comm, mem, idx).  counts holds the
// frontier size (kind 0) or the number of survivors (kind 1), which may exceed
// max_entries.  Models [model_first, model_first+model_count) only, split over
// n_threads threads; out and counts are indexed by absolute model number.
void orc_sweep(const ODesc* d, const OFilter* f, const u64* caps, u32 n_caps, u32 kind,
               u32 max_entries, OEntry* out, u32* counts, u32 model_first, u32 model_count,
               u32 n_threads) {
  Space sp(d);
  if (n_threads <= 1) {
    for (u32 m = model_first; m < model_first + model_count; ++m)
      reduce_model(sp, m, *f, caps, n_caps, kind, max_entries, out, counts);
    return;
  }
  std::vector<std::thread> pool;
  for (u32 t = 0; t < n_threads; ++t)
    pool.emplace_back([&, t]() {
      for (u32 m = model_first + t; m < model_first + model_count; m += n_threads)
        reduce_model(sp, m, *f, caps, n_caps, kind, max_entries, out, counts);
    });
  for (auto& th : pool) th.join();
}

// one composition with arbitrary per-axis codes (0..624 each)
void orc_check_composition(const OShape* shape, u32 N, u32 T, u32 K, u32 D, u32 code_tp,
                           u32 code_pp, u32 code_dp, u32 act_variant, u64 cap_bytes,
                           u32 tp_max_valid, u32 tp_coll_per_layer, u32 comm_kind, OEntry* out) {
  ORecord rec = derive_record(*shape);
  int pi[4];
  u32 c = code_dp;
  for (int s = 0; s < 4; ++s) { pi[s] = c % 5; c /= 5; }
  // Table 2: the tensor axis is (S,S,S,S) or (S,S,S,R), the pipeline axis (S,S,S,R);
  // an axis of degree 1 is absent and its code is not looked at
  bool tp_form = (T == 1) || code_tp == 156 || code_tp == 31;
  bool pp_form = (K == 1) || code_pp == 31;
  int tau = ((code_tp / 125) % 5 == S) ? 0 : 1;
  OResult r = eval_point(rec, N, T, K, D, (int)act_variant, tau, pi[0], pi[1], pi[2], pi[3],
                         tp_max_valid, tp_coll_per_layer, tp_form && pp_form);
  out->mem = r.mem;
  out->comm = comm_kind == 0 ? r.comm_paper : r.comm_paper + r.comm_ext;
  out->host = r.host;
  out->idx = 0;
  out->flags = r.flags | (r.mem <= cap_bytes ? F_FEASIBLE : 0);
  out->pad = 0;
}

// the formulas on an explicit record (used by the brute-force simulator tests,
// whose toy models have no transformer shape).  rec: P, unit, A0, A1, UA0,
// UA1, Sbh, L, heads, w_theta, w_omega, w_grad, w_act as 13 u64.
void orc_eval_record(const u64* rec, u32 N, u32 T, u32 K, u32 D, u32 v, u32 tau, u32 code,
                     u32 tp_max_valid, u32 tp_coll_per_layer, u32 sstar_units, u32 grad_accum_steps,
                     u32 replication_k, u64* out5) {
  ORecord m;
  m.P = rec[0]; m.unit = rec[1]; m.A[0] = rec[2]; m.A[1] = rec[3]; m.UA[0] = rec[4]; m.UA[1] = rec[5];
  m.Sbh = rec[6]; m.L = (u32)rec[7]; m.heads = (u32)rec[8];
  m.w_theta = (u32)rec[9]; m.w_omega = (u32)rec[10]; m.w_grad = (u32)rec[11]; m.w_act = (u32)rec[12];
  int pi[4];
  for (int s = 0; s < 4; ++s) { pi[s] = code % 5; code /= 5; }
  OResult r = eval_point(m, N, T, K, D, (int)v, (int)tau, pi[0], pi[1], pi[2], pi[3],
                         tp_max_valid, tp_coll_per_layer, true, sstar_units, grad_accum_steps, replication_k);
  out5[0] = r.mem; out5[1] = r.comm_paper; out5[2] = r.comm_ext; out5[3] = r.host; out5[4] = r.flags;
}

// the derived record of a shape, same 13 u64
void orc_model_record(const OShape* shape, u64* rec) {
  ORecord m = derive_record(*shape);
  rec[0] = m.P; rec[1] = m.unit; rec[2] = m.A[0]; rec[3] = m.A[1]; rec[4] = m.UA[0]; rec[5] = m.UA[1];
  rec[6] = m.Sbh; rec[7] = m.L; rec[8] = m.heads;
  rec[9] = m.w_theta; rec[10] = m.w_omega; rec[11] = m.w_grad; rec[12] = m.w_act;
}

// Algorithm 1 of the paper, one query at a time.  query: P, layer elements,
// device bytes, N, w_param, w_grad, w_opt, fast (8 u64).  out: mem, comm,
// branch, T, code, flags (6 u64).  Thresholds are the rationals hn/hd (0.7) and
// ln/ld (0.3); comparisons are exact.
void orc_select(const u64* query, u64 n, u32 hn, u32 hd, u32 ln, u32 ld, u32 tp_degree, u64* out) {
  typedef unsigned __int128 u128;
  for (u64 i = 0; i < n; ++i) {
    const u64* q = query + 8 * i;
    u64 P = q[0], layer = q[1], Md = q[2], N = q[3];
    u64 wsum = q[4] + q[5] + q[6];
    bool fast = q[7] != 0;
    u128 m_model = (u128)wsum * P;                    // line 1: params + optimizer + gradients
    u32 branch, T = 1, code;
    if (m_model * hd < (u128)hn * Md) {               // fits one device with headroom: data parallel
      branch = 0; code = 0;
    } else if (m_model * hd < (u128)hn * Md * N) {    // fits when sharded N ways: ZeRO-3 / FSDP
      branch = 1; code = 32;
    } else if (fast && (u128)wsum * layer * ld > (u128)ln * Md) {   // a layer is too big: add TP
      branch = 2; code = 32;
      for (u64 t = std::min<u64>(tp_degree, N); t >= 1; --t)
        if (N % t == 0) { T = (u32)t; break; }
    } else {
      branch = 3; code = 32;
    }
    ORecord m;
    m.P = P; m.unit = layer; m.A[0] = m.A[1] = m.UA[0] = m.UA[1] = 0; m.Sbh = 1; m.L = 1; m.heads = T;
    m.w_theta = (u32)q[4]; m.w_grad = (u32)q[5]; m.w_omega = (u32)q[6]; m.w_act = 1;
    int pi[4]; u32 c = code;
    for (int s = 0; s < 4; ++s) { pi[s] = c % 5; c /= 5; }
    OResult r = eval_point(m, N, T, 1, N / T, 0, 0, pi[0], pi[1], pi[2], pi[3], 0xffffffffu, 0, true);
    u64* o = out + 6 * i;
    o[0] = r.mem; o[1] = r.comm_paper; o[2] = branch; o[3] = T; o[4] = code;
    o[5] = r.mem <= Md ? F_FEASIBLE : 0;
  }
}

// Algorithm 1 beside the frontier: for every model, Algorithm 1's choice at device
// count n_values[n_index] and M_d = device_bytes, taken as a point of the space
// (K = 1, first variants), evaluated like any other point, and held against the
// model's frontier under that capacity (frontier[n_models][n_caps][max_entries],
// counts[n_models][n_caps]).  out: 12 u64 per model -- alg mem, comm, idx; best
// mem, comm, idx (the frontier's last written entry); branch, T, code, point
// flags, status (1 in space, 2 survivor, 4 on frontier, 8 dominated, 16 frontier
// empty, 32 frontier truncated), 0.
void orc_select_compare(const ODesc* d, u32 n_index, u64 Md, u32 fast, u32 hn, u32 hd, u32 ln, u32 ld,
                        u32 tp_degree, const OFilter* f, const OEntry* frontier, const u32* counts,
                        u32 n_caps, u32 cap_index, u32 max_entries, u64* out) {
  Space sp(d);
  const u64 N = d->n_values[n_index];
  for (u32 model = 0; model < d->n_models; ++model) {
    ORecord rec = derive_record(d->models[model]);
    u64 query[8] = {rec.P, rec.unit, Md, N, rec.w_theta, rec.w_grad, rec.w_omega, fast ? 1ull : 0ull};
    u64 pick[6];
    orc_select(query, 1, hn, hd, ln, ld, tp_degree, pick);
    const u32 branch = (u32)pick[2], T = (u32)pick[3], code = (u32)pick[4];
    // is the choice a point of the space?  Walk the space's own order to find it.
    bool in_space = false;
    u64 idx = 0;
    {
      u64 at = (u64)model * sp.pts_per_model;
      const u64 per_fact = (u64)d->n_act_variants * d->n_tpa_variants * sp.n_codes;
      for (u32 i = 0; i < d->n_n && !in_space; ++i) {
        for (size_t k = 0; k < sp.facts[i].size() && !in_space; ++k) {
          const Fact& fa = sp.facts[i][k];
          if (i == n_index && fa.T == T && fa.K == 1) {
            // the code's modes as digits of the allowed-mode numbering
            u64 digits = 0, weight = 1;
            bool ok = true;
            u32 c = code;
            for (int st = 0; st < 4; ++st) {
              int mode = c % 5; c /= 5;
              int pos = -1;
              for (size_t q = 0; q < sp.modes.size(); ++q) if (sp.modes[q] == mode) pos = (int)q;
              if (pos < 0) ok = false;
              digits += weight * (u64)(pos < 0 ? 0 : pos);
              weight *= sp.modes.size();
            }
            if (ok) { in_space = true; idx = at + digits; }
          }
          at += per_fact;
        }
      }
    }
    int pi[4]; u32 c = code;
    for (int st = 0; st < 4; ++st) { pi[st] = c % 5; c /= 5; }
    OResult r = eval_point(rec, N, T, 1, N / T, 0, 0, pi[0], pi[1], pi[2], pi[3], d->tp_max_valid,
                           d->tp_coll_per_layer, true, d->sstar_units, d->grad_accum_steps, d->replication_k);
    const u64 comm = objective_comm(r, *f);
    u32 fl;
    const bool survivor = passes(r, *f, Md, &fl);
    u32 status = (in_space ? 1u : 0u) | (survivor ? 2u : 0u);
    const u32 count = counts[(u64)model * n_caps + cap_index];
    const OEntry* fr = frontier + ((u64)model * n_caps + cap_index) * max_entries;
    const u32 written = std::min(count, max_entries);
    if (count == 0) status |= 16u;
    if (count > max_entries) status |= 32u;
    for (u32 e = 0; e < written; ++e) {
      if (fr[e].mem == r.mem && fr[e].comm == comm) status |= 4u;
      else if (fr[e].mem <= r.mem && fr[e].comm <= comm) status |= 8u;
    }
    u64* o = out + 12 * (u64)model;
    o[0] = r.mem; o[1] = comm; o[2] = in_space ? idx : 0;
    o[3] = written ? fr[written - 1].mem : 0; o[4] = written ? fr[written - 1].comm : 0;
    o[5] = written ? fr[written - 1].idx : 0;
    o[6] = branch; o[7] = T; o[8] = code; o[9] = fl; o[10] = status; o[11] = 0;
  }
}

u32 orc_hardware_threads() { return std::thread::hardware_concurrency(); }

}  // extern "C"

/* ps.h -- C interface of the placement-semantics sweep library (CUDA, sm_100a).
 *
 * The library evaluates, on one GPU, the derivation rules of "Placement
 * Semantics for Distributed Deep Learning" over a design space that is
 * enumerated on the device, never stored:
 *
 *   a point = (model shape, device count N, factorisation N = T*K*D into tensor,
 *              pipeline and data degrees, activation variant, tensor-axis
 *              activation variant, one of the five modes R,S,S*,M,O for each of
 *              Theta, Omega, G, A on the data axis)
 *
 * and for every point yields, as exact unsigned 64-bit integers,
 *
 *   mem         per-device GPU bytes                      (Theorem 1)
 *   comm_paper  per-step bytes priced by the paper         (Theorem 2, Corollary 1)
 *   comm_ext    per-step bytes the execution model moves that Theorem 2 does
 *               not price (re-replication, offload gathers, tensor/pipeline
 *               traffic; Proposition 1 names the per-layer collectives)
 *   host        per-step bytes over the host link (mode O, Definition 1 eq. (5))
 *   flags       gradient integrity (Theorem 3), state consistency (Theorem 4),
 *               composition validity (Theorems 6-7, Proposition 1, Remark 4)
 *               and their reasons.
 *
 * No result is ever rounded: every figure is an exact integer (a sweep compares
 * on the fp64 pipe only where all numbers of a factorisation are below 2^53,
 * which doubles hold exactly).  Shards are element-granular with the
 * boundaries of Definition 1 eq. (2); the per-device figure is the largest
 * shard, ceil(E/n); a ring reduce-scatter or all-gather (Section 2.3) moves
 * E - floor(E/n) elements on its busiest device; an all-reduce twice that.
 *
 * Conventions.  Every function returns 0 (PS_OK) or a negative PS_E_* code and
 * never aborts.  "device pointer" = memory of the context's GPU, owned by the
 * caller; "host pointer" = ordinary host memory.  All device work is enqueued
 * on the stream the context borrows; outputs are valid once the caller has
 * synchronised that stream (or called ps_status).  Kernels never trap: a
 * kernel that detects an inconsistency sets a status word that ps_status and
 * every later call report as PS_E_DEVICE.
 */
#ifndef PS_H_
#define PS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ------------------------------------------------------------------ codes */
enum {
  PS_OK = 0,
  PS_E_NULLPTR = -1,       /* a required pointer is null                         */
  PS_E_ALIGN = -2,         /* a device pointer is not aligned to its element     */
  PS_E_RANGE = -3,         /* a size, shape or count is outside the stated range */
  PS_E_BADINDEX = -4,      /* [first, first+count) leaves the space              */
  PS_E_TRUNCATED = -5,     /* a notice from ps_status: some Pareto frontier was longer than
                              max_entries (its head was written, d_counts is true)    */
  PS_E_CUDA = -6,          /* a CUDA runtime call failed                          */
  PS_E_UNIMPLEMENTED = -7,
  PS_E_DEVICE = -8,        /* a kernel reported an inconsistency (status word)   */
  PS_E_NOALLOC_LIMIT = -10 /* the window is too large for ps_eval_compact_noalloc's
                              fixed scratch array (PS_NOALLOC_MAX_GROUPS groups)  */
};

/* placement modes of Definition 1 */
enum { PS_MODE_R = 0, PS_MODE_S = 1, PS_MODE_SG = 2 /* S* */, PS_MODE_M = 3, PS_MODE_O = 4 };

/* A placement specification (Definition 2) as a code:
 *   code = pi_Theta + 5*pi_Omega + 25*pi_G + 125*pi_A        (0..624)
 * Table 2's rows: DP 0, ZeRO-1 5, ZeRO-2 30, ZeRO-3/FSDP 32, ZeRO-Offload 49,
 * tensor parallel (S,S,S,S) 156, pipeline parallel (S,S,S,R) 31. */
#define PS_CODE_TP_SEQPAR 156
#define PS_CODE_TP 31
#define PS_CODE_PP 31

/* flags */
enum {
  PS_F_GI = 1u << 0,          /* gradient integrity (Theorem 3)                      */
  PS_F_SC = 1u << 1,          /* state consistency (Theorem 4)                       */
  PS_F_CV = 1u << 2,          /* composition valid = bits 4..7 all set and T*K*D = N */
  PS_F_FEASIBLE = 1u << 3,    /* mem <= capacity (only where a capacity is given)    */
  PS_F_T_DIV_HEADS = 1u << 4, /* T divides the head count                            */
  PS_F_K_DIV_LAYERS = 1u << 5,/* K divides the layer count                           */
  PS_F_TP_LE_MAX = 1u << 6,   /* T <= tp_max_valid (Proposition 1: TP stays in-node) */
  PS_F_AXIS_FORM = 1u << 7,   /* model axes have Table 2's forms                     */
  PS_F_THETA_AVAIL = 1u << 8, /* every replica can obtain all parameters             */
  PS_F_ACT_AVAIL = 1u << 9,   /* every replica has its own activations for backward  */
  PS_F_GRAD_COVER = 1u << 10, /* reduced gradients reach every element that is updated */
  PS_F_USES_HOST = 1u << 11,  /* some state is offloaded                             */
  PS_F_PAPER_PRICED = 1u << 12/* Theorem 2 prices all data-axis traffic of this point */
};

enum { PS_COMM_PAPER = 0, PS_COMM_PAPER_PLUS_EXT = 1 };
enum { PS_REDUCE_PARETO = 0, PS_REDUCE_TOPK = 1 };

#define PS_NO_LIMIT UINT64_MAX
#define PS_TOPK_MAX 64           /* largest max_entries of a top-k sweep            */
#define PS_FRONTIER_FAST 128     /* a model whose frontier (or the part of it one warp of the
                                    sweep finds) is longer is reduced by a slow exact path */

/* ------------------------------------------------------------------ types */
typedef struct ps_ctx ps_ctx;     /* opaque: device, borrowed stream, scratch memory      */
typedef struct ps_space ps_space; /* opaque: device copy of the model table + enumeration */

/* One model, 48 bytes (Section 2.1, Remark 1, Definition 3).
 * Ranges: layers <= 2^10, hidden <= 2^16, heads <= 2^16, vocab <= 2^24,
 * seq <= 2^17, micro_batch <= 2^10, widths 1..16, parameter count <= 2^46,
 * stored activations <= 2^58 bytes; all >= 1.  Outside: PS_E_RANGE. */
typedef struct {
  uint64_t param_elems_override; /* 0: P = 12*L*H^2 + V*H (Section 2.1); else P    */
  uint32_t layers, hidden, heads, vocab, seq, micro_batch;
  uint8_t w_param, w_grad, w_opt, w_act; /* bytes per element; Remark 1: 2, 2, 12, 2 */
  uint8_t unit_from_shape;       /* 1: reconstruction unit = 12*H^2 elements (Def. 3); 0: none */
  uint8_t act_enabled;           /* 0: |A| = 0 ("excluding activations", Example 3)  */
  uint8_t pad[10];
} ps_model_shape;

/* The design space.  Linear index order: model-major; then N in the order
 * given; then factorisations (T ascending, then K ascending) over all T | N,
 * T <= t_enum_max, K | N/T, K <= k_enum_max, D = N/(T*K), independent of the
 * model; then the activation variant; then the tensor-axis variant; then the
 * data-axis code, fastest, written in base |mode_mask| over the allowed modes
 * in ascending order with the Theta digit fastest. */
typedef struct {
  const ps_model_shape* models; /* host pointer, copied by ps_space_create            */
  uint32_t n_models;            /* 1 .. 2^20                                           */
  const uint32_t* n_values;     /* host pointer, copied; each 1 .. 2^24                */
  uint32_t n_n;                 /* 1 .. 64                                             */
  uint32_t t_enum_max;          /* >= 1                                                */
  uint32_t k_enum_max;          /* >= 1                                                */
  uint32_t tp_max_valid;        /* T above this clears PS_F_TP_LE_MAX                  */
  uint32_t n_act_variants;      /* 1: activations stored; 2: {stored, full checkpointing} */
  uint32_t n_tpa_variants;      /* 1: tensor axis shards activations (pi_A = S);
                                   2: {S, R}                                            */
  uint32_t mode_mask;           /* bit m set: mode m allowed on the data axis; != 0    */
  uint32_t tp_coll_per_layer;   /* all-reduces per layer per step on the tensor axis, <= 64 */
  /* Three extensions the paper names without working them out.  Each applies to
   * the whole space (sweep once per value to compare values); 0 means 1. */
  uint32_t sstar_units;         /* 1 or 2: unit buffers a gathered (S*) state holds.  Theorem 1
                                   charges one; its proof notes that an implementation which
                                   gathers the next unit while the current one is in use needs
                                   2 * s_unit.  Applies to all four states. */
  uint32_t grad_accum_steps;    /* 1 .. 64: micro-batches per step (Section "Limitations":
                                   gradient accumulation).  All figures stay per step.  Once
                                   per step: every gradient synchronisation term, the update
                                   and what it moves (gathered optimizer state, re-replicated
                                   parameters, offloaded Omega and G, storing offloaded Theta).
                                   Once per micro-batch: the two all-gathers of gathered
                                   parameters (Theorem 2's third term), loading and gathering
                                   offloaded parameters, moving offloaded activations, tensor-
                                   and pipeline-axis traffic.  A placement whose only traffic
                                   is gradient synchronisation therefore moves the same bytes
                                   per step for g times the samples: the paper's "reduced by a
                                   factor equal to the number of accumulation steps".  Memory
                                   and the predicates do not change. */
  uint32_t replication_k;       /* 1 .. 2^24: copies of every shard ("k-way replication for
                                   1 < k < N", Section 1).  The sharded modes S, S*, O of a data
                                   axis of D devices cut a state into G = D / k shards, each held
                                   by the k devices at the same position of k groups of G devices
                                   (k = gcd(replication_k, D) where it does not divide D).  A shard
                                   is ceil(E / G) elements; gathers run inside a group and move
                                   E - floor(E / G); a gradient is reduced to shards inside every
                                   group and then all-reduced across the copies of each shard.  With
                                   G = 1 a shard is the whole tensor and the predicates treat the
                                   sharded modes as they do on a single device.  Modes R and M and
                                   the model axes are not affected. */
} ps_space_desc;

/* survivors of a filter: mem <= cap_bytes, host <= host_cap and every bit of
 * require_flags set (PS_F_FEASIBLE in require_flags is implied by the cap). */
typedef struct {
  uint64_t host_cap;      /* PS_NO_LIMIT for none                                  */
  uint32_t require_flags;
  uint32_t comm_kind;     /* objective of the sweeps: PS_COMM_PAPER or ..._PLUS_EXT */
  uint64_t cap_bytes;     /* ps_eval_batch only; the sweeps take their own list     */
  uint32_t skip_rejected; /* sweeps only.  0: every point is evaluated (its capacity compare is
                             executed, then masked by the flags) -- what the throughput figures
                             are quoted on.  1: a factorisation whose composition bits (T | heads,
                             K | layers, T <= tp_max_valid) already miss a required flag is not
                             evaluated at all; same results, less work when the filter requires
                             PS_F_CV or one of its reasons */
  uint32_t pad;
} ps_filter;

/* structure-of-arrays outputs of ps_eval_batch: device pointers, any may be
 * null (skipped); u64 arrays 8-byte aligned (16 preferred), flags 4-byte. */
typedef struct {
  uint64_t *mem, *comm_paper, *comm_ext, *host;
  uint32_t* flags;
} ps_out_soa;

/* one entry of a frontier or top-k list, 40 bytes */
typedef struct {
  uint64_t mem, comm, host, idx;
  uint32_t flags, pad;
} ps_front_entry;

/* a decoded point; device rank layout is rank = (d*K + k)*T + t (Remark 4:
 * tensor innermost, pipeline in the middle, data outermost; Theorem 6(1)) */
typedef struct {
  uint32_t model, N, T, K, D, act_variant, tpa_variant;
  uint16_t code_dp, code_tp, code_pp, pad;
} ps_point;

/* ------------------------------------------------------------------ context */
/* Create a context on `device` that enqueues on `cuda_stream` (a cudaStream_t
 * passed as void*, borrowed, may be null = default stream).  Allocates a small
 * scratch area that later calls grow on demand. */
int ps_create(ps_ctx** out, int device, void* cuda_stream);
void ps_destroy(ps_ctx* ctx);
/* Synchronise the stream and return PS_OK or the first error a kernel
 * recorded since the last call of ps_status (which also clears it). */
int ps_status(ps_ctx* ctx);
const char* ps_strerror(int code);

/* ------------------------------------------------------------------ space */
/* Validate the description, enumerate the factorisations of every N on the
 * host, copy the shape table to the device and derive the per-model records
 * there (Section 2.1, Remark 1, Definition 3).  The space keeps no table of
 * points.  Points per model must stay below 2^32. */
int ps_space_create(ps_ctx* ctx, const ps_space_desc* desc, ps_space** out);
void ps_space_destroy(ps_space* space);
/* Replace the shape table (same n_models) from host memory: one asynchronous
 * copy plus the derivation kernel on the context's stream.  `models` must stay
 * valid until the stream has passed the copy (pinned memory makes it truly
 * asynchronous). */
int ps_space_set_models(ps_space* space, const ps_model_shape* models, uint32_t n_models);
/* Run the derivation kernel again on the shape table already resident on the
 * device (Section 2.1, Remark 1, Definition 3); no host memory is touched. */
int ps_space_rederive(ps_space* space);
uint64_t ps_space_size(const ps_space* space);
uint64_t ps_space_points_per_model(const ps_space* space);
/* host-side decoding of a linear index (for reports) */
int ps_space_decode(const ps_space* space, uint64_t idx, ps_point* out);

/* ------------------------------------------------------------------ hot path */
/* Evaluate points [first, first+count) (Theorems 1-4, 6-7).
 *  filter == NULL: materialise -- out.X[i] belongs to point first+i.
 *  filter != NULL: stream compaction -- the survivors are written densely in
 *    index order; d_idx_out (device, may be null) receives their indices,
 *    *d_n_out (device scalar, required) their number; flags carry
 *    PS_F_FEASIBLE.  Outputs need room for `count` elements in the worst case.
 * count may be 0. */
int ps_eval_batch(ps_ctx* ctx, const ps_space* space, uint64_t first, uint64_t count,
                  const ps_filter* filter, ps_out_soa out, uint64_t* d_idx_out,
                  uint64_t* d_n_out);

/* Sweep the whole space and reduce it per (model, capacity).
 *  PS_REDUCE_PARETO: the distinct non-dominated (mem, comm) pairs among the
 *    survivors, both minimised (the trade-off of Corollary 1), each represented
 *    by its smallest linear index, sorted by mem ascending.
 *  PS_REDUCE_TOPK: the max_entries (<= PS_TOPK_MAX) smallest survivors by
 *    (comm, mem, idx).
 * d_out is [n_models][n_caps][max_entries] (device, 8-byte aligned); unused
 * slots are zeroed.  d_counts[n_models][n_caps] (device) receives the true
 * frontier length, or for top-k the number of survivors, even when that
 * exceeds max_entries; a Pareto frontier longer than max_entries also makes the
 * next ps_status return PS_E_TRUNCATED once (a notice: the head of the frontier
 * was written and later calls are not affected).  Frontiers of any length are
 * exact; one longer than PS_FRONTIER_FAST is computed by a slow path (one pass
 * over the model's points per entry).  n_caps <= 8.  The call may grow the
 * context's scratch (one partial list per warp of the sweep). */
int ps_sweep_pareto(ps_ctx* ctx, const ps_space* space, const ps_filter* filter,
                    const uint64_t* caps_bytes /* host */, uint32_t n_caps, uint32_t reduce_kind,
                    uint32_t max_entries, ps_front_entry* d_out, uint32_t* d_counts);

/* One composition with arbitrary per-axis codes (Definition 5): N devices as
 * T x K x D, code_tp on the tensor axis, code_pp on the pipeline axis, code_dp
 * on the data axis (each 0..624).  Evaluated on the device; h_out (host) is
 * filled before the call returns (this call synchronises).  The numbers assume
 * Table 2's forms on the model axes, the tensor-axis activation mode taken from
 * code_tp; PS_F_AXIS_FORM says whether the given codes have those forms (an
 * axis of degree 1 is not looked at).  idx of the entry is 0. */
int ps_check_composition(ps_ctx* ctx, const ps_model_shape* shape /* host */, uint32_t N,
                         uint32_t T, uint32_t K, uint32_t D, uint16_t code_tp, uint16_t code_pp,
                         uint16_t code_dp, uint32_t act_variant, uint64_t cap_bytes,
                         uint32_t tp_max_valid, uint32_t tp_coll_per_layer, uint32_t comm_kind,
                         ps_front_entry* h_out);

/* ------------------------------------------------------------------ Algorithm 1 */
/* Batched form of the paper's illustrative strategy selection (Algorithm 1).
 * For every query, with M_model = (w_param + w_grad + w_opt) * P bytes (line 1:
 * "16P") and headroom = headroom_num / headroom_den (the paper's 0.7):
 *   branch 0  M_model < headroom * M_d            -> (R,R,R,R), data parallel
 *   branch 1  M_model / N < headroom * M_d        -> (S*,S,S,R), ZeRO-3 / FSDP
 *   branch 2  otherwise, if one layer's model state (w sum * layer_elems) exceeds
 *             layer_num / layer_den (0.3) of M_d and the interconnect is fast
 *                                                  -> ZeRO-3 composed with tensor
 *             parallelism of degree T = the largest divisor of N not above tp_degree
 *   branch 3  otherwise                            -> ZeRO-3 alone (nothing of the
 *             algorithm fits; the caller must look further)
 * All comparisons are exact (integers, no rounding of the thresholds).  The
 * result also carries Theorem 1's bytes and Theorem 2's volume of the chosen
 * specification (activations excluded, as in the algorithm) and PS_F_FEASIBLE
 * if those bytes fit M_d.  d_queries and d_out are device pointers (16-byte
 * aligned), n may be 0.  Ranges as commented in the query; values outside give
 * unspecified numbers but no fault. */
typedef struct {
  uint64_t param_elems;     /* P, 1 .. 2^46                                   */
  uint64_t layer_elems;     /* elements of one layer (12 H^2, Def. 3), may be 0 */
  uint64_t device_bytes;    /* M_d, <= 2^50                                    */
  uint32_t n_devices;       /* N, 1 .. 2^24                                    */
  uint8_t w_param, w_grad, w_opt; /* bytes per element, 1..16 (Remark 1: 2, 2, 12) */
  uint8_t fast_interconnect;
} ps_select_query;          /* 32 bytes */
typedef struct {
  uint64_t mem, comm;       /* Theorem 1, Theorem 2 for the chosen specification */
  uint32_t branch;          /* 0..3 as above                                    */
  uint32_t T;               /* tensor-parallel degree (1 unless branch 2)       */
  uint32_t code_dp;         /* data-axis code: 0 (DP) or 32 (ZeRO-3)            */
  uint32_t flags;           /* PS_F_FEASIBLE or 0                               */
} ps_select_result;         /* 32 bytes */
int ps_select(ps_ctx* ctx, const ps_select_query* d_queries, uint64_t n, uint32_t headroom_num,
              uint32_t headroom_den, uint32_t layer_num, uint32_t layer_den, uint32_t tp_degree,
              ps_select_result* d_out);

/* Algorithm 1 beside the exhaustive answer.  For every model of a space, run
 * Algorithm 1 with the model's own parameter count, layer size and byte widths,
 * the device count n_values[n_index] and M_d = device_bytes, take its choice as
 * a point of the space (tensor degree T of branch 2 or 1, no pipeline axis,
 * D = N / T, the space's first activation and tensor-axis variants, data-axis
 * code 0 or 32), evaluate that point as the space does (Theorems 1-4, with
 * activations and the traffic Theorem 2 does not price, per filter->comm_kind),
 * and hold it against the model's Pareto frontier under the same capacity, as
 * ps_sweep_pareto wrote it (d_frontier[n_models][n_caps][max_entries],
 * d_counts[n_models][n_caps]; the capacity at cap_index must be device_bytes and
 * the filter the sweep's).  Sweep a space whose only device count is that N to
 * compare like with like.  status bits:
 *   PS_SEL_IN_SPACE     the choice is a point of the space (alg_idx is its index)
 *   PS_SEL_SURVIVOR     it fits device_bytes, the host budget and the required flags
 *   PS_SEL_ON_FRONTIER  the frontier has an entry with its (mem, comm)
 *   PS_SEL_DOMINATED    some entry is no worse in both and better in one
 *   PS_SEL_FRONTIER_EMPTY / PS_SEL_FRONTIER_TRUNCATED (count > max_entries: only
 *                       the written head was looked at)
 * best_* is the frontier's last written entry: the least communication that fits.
 * All pointers but filter are device pointers; d_out has n_models records. */
enum {
  PS_SEL_IN_SPACE = 1u << 0, PS_SEL_SURVIVOR = 1u << 1, PS_SEL_ON_FRONTIER = 1u << 2,
  PS_SEL_DOMINATED = 1u << 3, PS_SEL_FRONTIER_EMPTY = 1u << 4, PS_SEL_FRONTIER_TRUNCATED = 1u << 5
};
typedef struct {
  uint64_t alg_mem, alg_comm, alg_idx;     /* Algorithm 1's choice as the space evaluates it   */
  uint64_t best_mem, best_comm, best_idx;  /* the frontier's least-communication entry          */
  uint32_t branch, T, code_dp;             /* as in ps_select_result                            */
  uint32_t alg_flags;                      /* PS_F_* of the choice (PS_F_FEASIBLE vs device_bytes) */
  uint32_t status, pad;
} ps_select_compare_result;                /* 72 bytes */
int ps_select_compare(ps_ctx* ctx, const ps_space* space, uint32_t n_index, uint64_t device_bytes,
                      uint32_t fast_interconnect, uint32_t headroom_num, uint32_t headroom_den,
                      uint32_t layer_num, uint32_t layer_den, uint32_t tp_degree,
                      const ps_filter* filter /* host */, const ps_front_entry* d_frontier,
                      const uint32_t* d_counts, uint32_t n_caps, uint32_t cap_index,
                      uint32_t max_entries, ps_select_compare_result* d_out);

/* The filter-and-compact form of ps_eval_batch for callers that cannot
 * allocate device memory.  (The paper has no counterpart: this is a property of
 * the library, not of the method.)
 *
 * Who needs it: a program whose GPU memory is wholly owned by another
 * allocator -- a training framework's caching pool, or a serving process that
 * has handed every byte to its cache -- where a raw cudaMalloc from a library
 * can fail or fragment that pool; and a loop that cannot afford the implicit
 * device-wide synchronisation of cudaFree/cudaMalloc.  ps_eval_batch may do
 * both when its scratch has to grow.  This function never calls cudaMalloc,
 * cudaFree or any allocating routine: its scratch tables (a survivor count per
 * group of |mode_mask|^4 consecutive points, the list of groups that have
 * survivors, and a prefix sum per run of up to 32 groups) sit in a fixed 2 MiB
 * array inside the library image, which every GPU that loads the library holds
 * until the process ends.
 *
 * Arguments, outputs, order of the survivors and error behaviour are those of
 * ps_eval_batch with a non-null filter (which is required here).  Limits and
 * rules of its own:
 *  - the window may touch at most PS_NOALLOC_MAX_GROUPS groups, else
 *    PS_E_NOALLOC_LIMIT is returned and nothing is enqueued;
 *  - the first call on each device looks up the array's device address (with
 *    that device made current); make that first call before any stream
 *    capture is begun;
 *  - all calls on a device share the one array, and it keeps the previous
 *    call's contents (the function clears what it is about to use): two calls
 *    whose kernels overlap on the GPU -- different streams, or different
 *    contexts on the same device -- race on it.  Serialise them. */
#define PS_NOALLOC_MAX_GROUPS 131072
int ps_eval_compact_noalloc(ps_ctx* ctx, const ps_space* space, uint64_t first, uint64_t count,
                            const ps_filter* filter, ps_out_soa out, uint64_t* d_idx_out,
                            uint64_t* d_n_out);

/* ------------------------------------------------------------------ verification protocol */
/* The paper's verification protocol (Section 7.1: gradient-integrity check,
 * state-consistency check, trajectory check) as a batched brute-force run.
 * Every case trains a tiny layered network -- `units` layers of `h` parameters,
 * layer l maps a to tanh(theta_l * a) elementwise, loss 0.5 |out - y|^2 -- with
 * Adam in fp64 on D logical devices that hold Theta, Omega (master copy, first
 * and second moment), G and A exactly as the placement code says (Definition 1:
 * full copies, element shards with eq. (2)'s boundaries, nothing, or shards in a
 * host arena), moving data through explicit rings that count the bytes each
 * device sends (Section 2.3), and beside it the single-device run on the global
 * batch (Definition 4).  What a placement leaves unavailable when it is needed
 * reads as zeros.  A result says whether the reassembled Theta and Omega of
 * every step equal the single-device state (Theorem 5: exactly the placements
 * with gradient integrity and state consistency), and gives the last step's
 * per-device bytes held (persistent high-water mark plus unit buffers, largest
 * device), bytes sent (each collective charged to its busiest device) and bytes
 * over the host link.  The kernel evaluates none of Theorems 1-4: it executes
 * the mechanism, so its figures check the rules (ps_eval_batch,
 * ps_check_composition) from outside.
 *
 * d_cases, d_data, d_out, d_theta_out are device pointers (8-byte aligned);
 * d_theta_out (may be null) receives units * h doubles per case: the parameters
 * the job holds after the last step.  A case's data sits at d_data +
 * data_offset: theta0[units*h], then the inputs x[accum][D][b][h], then the
 * targets y[accum][D][b][h].  A case with D outside 1..4, a code above 624 or
 * data outside [0, data_len) gets a zero result and makes ps_status return
 * PS_E_DEVICE; nothing is read or written out of bounds.  The call may grow the
 * context's scratch (a workspace per case).  Ranges of the shape: see its
 * comments; outside them PS_E_RANGE. */
typedef struct {
  uint32_t units, h, b;          /* layers 1..8, parameters per layer 1..32, samples per device and micro-batch 1..4 */
  uint32_t accum, steps;         /* micro-batches per step 1..4, optimizer steps 1..16                              */
  uint32_t gather_buffers;       /* unit buffers of a gathered state: 1, or 2 (Theorem 1's proof, case S*)           */
  uint32_t w_theta, w_omega, w_grad; /* bytes per element, 1..16; w_omega a multiple of 3 (three rows)               */
  uint32_t pad;
  double lr, beta1, beta2, eps;  /* Adam                                                                             */
  double rtol, atol;             /* equal means |got - want| <= atol + rtol * |want|                                 */
} ps_verify_shape;
typedef struct {
  uint32_t code;                 /* data-axis placement code, 0..624                                                 */
  uint32_t D;                    /* logical devices, 1..4                                                            */
  uint64_t data_offset;          /* in doubles                                                                       */
} ps_verify_case;                /* 16 bytes */
typedef struct {
  uint64_t mem, comm, host;      /* bytes, last step                                                                 */
  uint32_t match;                /* 1: every step's state equals the single-device run                               */
  uint32_t pad;
  double max_rel_err;            /* largest relative deviation beyond atol that was seen                             */
} ps_verify_result;              /* 40 bytes */
int ps_verify_batch(ps_ctx* ctx, const ps_verify_shape* shape /* host */, const ps_verify_case* d_cases,
                    uint64_t n, const double* d_data, uint64_t data_len, ps_verify_result* d_out,
                    double* d_theta_out);

/* ------------------------------------------------------------------ measurement */
/* Integer-pipe microbenchmark: `blocks` x 256 threads each run `iters` rounds
 * of 8 independent 32-bit add/logic chains of 16 operations.  Returns through
 * *thread_ops the number of 32-bit thread operations issued; the caller times
 * the stream.  d_sink (device, >= 4 bytes) receives a value that depends on
 * every chain. */
int ps_int_peak(ps_ctx* ctx, uint32_t blocks, uint32_t iters, uint32_t* d_sink,
                uint64_t* thread_ops);

#ifdef __cplusplus
}
#endif
#endif /* PS_H_ */

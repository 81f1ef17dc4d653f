// The C interface: argument validation, host-side enumeration of the
// factorisations, scratch management and kernel launches.  No arithmetic of the
// method happens on the host; every evaluation runs in the kernels.
#include <cuda_runtime.h>
#include <stdlib.h>
#include <string.h>
#include <algorithm>
#include <new>
#include <vector>

#include "ps.h"
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

#define CUDA_OK(call)                         \
  do {                                        \
    if ((call) != cudaSuccess) return PS_E_CUDA; \
  } while (0)

struct DeviceGuard {
  int prev;
  bool ok;
  explicit DeviceGuard(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// the supported ranges of a shape (the same limits the derivation kernel checks)
bool shape_in_range(const ps_model_shape& s, u32 tp_coll, u32 accum = 1) {
  if (s.layers < 1 || s.layers > (1u << 10)) return false;
  if (s.hidden < 1 || s.hidden > (1u << 16)) return false;
  if (s.heads < 1 || s.heads > (1u << 16)) return false;
  if (s.vocab < 1 || s.vocab > (1u << 24)) return false;
  if (s.seq < 1 || s.seq > (1u << 17)) return false;
  if (s.micro_batch < 1 || s.micro_batch > (1u << 10)) return false;
  const uint8_t w[4] = {s.w_param, s.w_grad, s.w_opt, s.w_act};
  for (int i = 0; i < 4; ++i)
    if (w[i] < 1 || w[i] > 16) return false;
  if (tp_coll > 64) return false;
  typedef unsigned __int128 u128;
  const u128 L = s.layers, H = s.hidden, V = s.vocab, S = s.seq, b = s.micro_batch, a = s.heads;
  const u128 P = s.param_elems_override ? (u128)s.param_elems_override : 12 * L * H * H + V * H;
  if (P < 1 || P > ((u128)1 << 46)) return false;
  if (S * b * H > ((u128)1 << 40)) return false;
  if (s.act_enabled) {
    const u128 A0 = L * (34 * S * b * H + 5 * a * S * S * b);
    if (A0 > ((u128)1 << 58)) return false;
    if (2 * A0 * accum > ((u128)1 << 62)) return false;        // host bytes of offloaded activations
  } else if (5 * a * S * S * b > ((u128)1 << 58)) {
    return false;
  }
  // tensor- and pipeline-axis bytes per step
  if ((L * 2 * tp_coll * s.w_act + 2 * s.w_act) * S * b * H * accum > ((u128)1 << 62)) return false;
  return true;
}

// whether every byte count of a (Theta, Omega, G) triple of this model -- device
// bytes (at most wsum * (P + 2 unit)), host bytes (at most (2 accum + 1) * wsum * P)
// and data-axis volume (at most (4 accum + 1) * wsum * P) -- stays below 2^53
bool shape_is_small(const ps_model_shape& s, u32 accum) {
  typedef unsigned __int128 u128;
  const u128 H = s.hidden;
  const u128 P = s.param_elems_override ? (u128)s.param_elems_override
                                        : 12 * (u128)s.layers * H * H + (u128)s.vocab * H;
  const u128 unit = s.unit_from_shape ? 12 * H * H : 0;
  const u128 wsum = (u128)s.w_param + s.w_grad + s.w_opt;
  return (4 * (u128)accum + 1) * wsum * (P + 2 * unit) < ((u128)1 << 53);
}

int ensure_scratch(ps_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->scratch_bytes) return PS_OK;
  CUDA_OK(cudaStreamSynchronize(ctx->stream));
  if (ctx->scratch) CUDA_OK(cudaFree(ctx->scratch));
  ctx->scratch = nullptr;
  ctx->scratch_bytes = 0;
  size_t want = (bytes + (size_t(1) << 20) - 1) & ~((size_t(1) << 20) - 1);
  CUDA_OK(cudaMalloc(&ctx->scratch, want));
  ctx->scratch_bytes = want;
  return PS_OK;
}

// a kernel-reported problem seen by an earlier status copy
int pending_device_error(ps_ctx* ctx) {
  const u32 st = *ctx->h_status & ~(u32)ST_TRUNCATED;     // a truncated frontier blocks nothing
  if (st) return PS_E_DEVICE;
  return PS_OK;
}

// flag bits a filter may require
constexpr u32 KNOWN_FLAGS = (PS_F_PAPER_PRICED << 1) - 1u;

int enqueue_status_copy(ps_ctx* ctx) {
  CUDA_OK(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(u32), cudaMemcpyDeviceToHost, ctx->stream));
  return PS_OK;
}

u32 pick_chunks(const ps_ctx* ctx, const ps_space* sp, int kind, bool many) {
  // Blocks per model.  Every extra block of a model builds its lists from
  // scratch -- a top-k block takes every survivor as a candidate until it has
  // found its own first k -- so only as many as fill the GPU once (top-k) or
  // twice (Pareto, whose blocks are fewer and longer).
  const u64 waves = kind == PS_REDUCE_PARETO ? 2 : 1;
  const u64 target = (u64)ctx->sm_count * sweep_blocks_per_sm(kind, many) * waves;
  u64 c = (target + sp->dev.n_models / 2) / sp->dev.n_models;       // to the nearest: one block too few is cheaper than a second list
  if (c < 1) c = 1;
  if (c > SWEEP_MAX_CHUNKS) c = SWEEP_MAX_CHUNKS;
  const u64 by_units = (sp->dev.n_facts + sweep_warps(kind, many) - 1) / sweep_warps(kind, many);   // a unit per warp at least
  if (c > by_units) c = by_units;
  if (c < 1) c = 1;
  return (u32)c;
}

}  // namespace

extern "C" {

const char* ps_strerror(int code) {
  switch (code) {
    case PS_OK: return "ok";
    case PS_E_NULLPTR: return "a required pointer is null";
    case PS_E_ALIGN: return "a device pointer is misaligned";
    case PS_E_RANGE: return "a size, shape or count is outside the supported range";
    case PS_E_BADINDEX: return "the index window leaves the space";
    case PS_E_TRUNCATED: return "an output was too short";
    case PS_E_CUDA: return "a CUDA runtime call failed";
    case PS_E_UNIMPLEMENTED: return "not implemented";
    case PS_E_DEVICE: return "a kernel reported an inconsistency";
    case PS_E_NOALLOC_LIMIT:
      return "the window needs more scratch than the no-allocation entry point's fixed array holds";
    default: return "unknown error";
  }
}

int ps_create(ps_ctx** out, int device, void* cuda_stream) {
  if (!out) return PS_E_NULLPTR;
  *out = nullptr;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) return PS_E_CUDA;
  if (device < 0 || device >= n_dev) return PS_E_RANGE;
  DeviceGuard guard(device);
  if (!guard.ok) return PS_E_CUDA;
  ps_ctx* ctx = new (std::nothrow) ps_ctx();
  if (!ctx) return PS_E_CUDA;
  ctx->device = device;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  ctx->scratch = nullptr;
  ctx->scratch_bytes = 0;
  ctx->d_status = nullptr;
  ctx->h_status = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return PS_E_CUDA; }
  ctx->sm_count = prop.multiProcessorCount;
  ctx->compact_calls = 0;
  if (cudaMalloc(&ctx->d_status, 4 * sizeof(u32)) != cudaSuccess ||
      cudaMallocHost(&ctx->h_status, sizeof(u32)) != cudaSuccess ||
      cudaMemsetAsync(ctx->d_status, 0, 4 * sizeof(u32), ctx->stream) != cudaSuccess) {
    ps_destroy(ctx);
    return PS_E_CUDA;
  }
  *ctx->h_status = 0;
  if (ensure_scratch(ctx, size_t(8) << 20) != PS_OK) { ps_destroy(ctx); return PS_E_CUDA; }
  *out = ctx;
  return PS_OK;
}

void ps_destroy(ps_ctx* ctx) {
  if (!ctx) return;
  DeviceGuard guard(ctx->device);
  cudaStreamSynchronize(ctx->stream);
  if (ctx->scratch) cudaFree(ctx->scratch);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->h_status) cudaFreeHost(ctx->h_status);
  delete ctx;
}

int ps_status(ps_ctx* ctx) {
  if (!ctx) return PS_E_NULLPTR;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(u32), cudaMemcpyDeviceToHost, ctx->stream));
  CUDA_OK(cudaStreamSynchronize(ctx->stream));
  int rc = pending_device_error(ctx);
  if (rc == PS_OK && (*ctx->h_status & ST_TRUNCATED)) rc = PS_E_TRUNCATED;
  if (rc != PS_OK) {
    *ctx->h_status = 0;
    CUDA_OK(cudaMemsetAsync(ctx->d_status, 0, sizeof(u32), ctx->stream));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
  }
  return rc;
}

// ------------------------------------------------------------------ space
int ps_space_create(ps_ctx* ctx, const ps_space_desc* desc, ps_space** out) {
  if (!ctx || !desc || !out || !desc->models || !desc->n_values) return PS_E_NULLPTR;
  *out = nullptr;
  if (desc->n_models < 1 || desc->n_models > (1u << 20)) return PS_E_RANGE;
  if (desc->n_n < 1 || desc->n_n > 64) return PS_E_RANGE;
  if (desc->t_enum_max < 1 || desc->k_enum_max < 1) return PS_E_RANGE;
  if (desc->n_act_variants < 1 || desc->n_act_variants > 2) return PS_E_RANGE;
  if (desc->n_tpa_variants < 1 || desc->n_tpa_variants > 2) return PS_E_RANGE;
  if ((desc->mode_mask & 0x1Fu) == 0 || (desc->mode_mask & ~0x1Fu)) return PS_E_RANGE;
  if (desc->tp_coll_per_layer > 64) return PS_E_RANGE;
  for (u32 i = 0; i < desc->n_n; ++i)
    if (desc->n_values[i] < 1 || desc->n_values[i] > (1u << 24)) return PS_E_RANGE;
  if (desc->sstar_units > 2 || desc->grad_accum_steps > 64 || desc->replication_k > (1u << 24)) return PS_E_RANGE;
  const u32 accum = desc->grad_accum_steps ? desc->grad_accum_steps : 1;
  for (u32 i = 0; i < desc->n_models; ++i)
    if (!shape_in_range(desc->models[i], desc->tp_coll_per_layer, accum)) return PS_E_RANGE;

  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  ps_space* sp = new (std::nothrow) ps_space();
  if (!sp) return PS_E_CUDA;
  sp->ctx = ctx;
  sp->desc = *desc;
  sp->desc.models = nullptr;
  sp->desc.n_values = nullptr;
  sp->d_shapes = nullptr;
  sp->d_recs = nullptr;
  sp->d_facts = nullptr;
  sp->d_order = nullptr;
  sp->n_values.assign(desc->n_values, desc->n_values + desc->n_n);
  // all (T, K) with T | N, K | N/T inside the enumeration limits: T ascending, then K
  for (u32 i = 0; i < desc->n_n; ++i) {
    sp->fact_begin.push_back((u32)sp->facts.size());
    const u32 N = desc->n_values[i];
    std::vector<u32> sorted;                      // divisors of N, ascending
    for (u32 d = 1; (u64)d * d <= N; ++d)
      if (N % d == 0) { sorted.push_back(d); if (d != N / d) sorted.push_back(N / d); }
    std::sort(sorted.begin(), sorted.end());
    for (u32 T : sorted) {
      if (T > desc->t_enum_max) break;
      const u32 rest = N / T;
      for (u32 K : sorted) {
        if (K > desc->k_enum_max || K > rest) break;
        if (rest % K) continue;
        sp->facts.push_back(Fact{N, T, K, rest / K});
      }
    }
    if (sp->facts.size() > (size_t(1) << 20)) { delete sp; return PS_E_RANGE; }
  }
  sp->fact_begin.push_back((u32)sp->facts.size());
  if (sp->facts.empty()) { delete sp; return PS_E_RANGE; }
  u32 modemap = 0, nm = 0;
  for (u32 m = 0; m < 5; ++m)
    if (desc->mode_mask & (1u << m)) { modemap |= m << (4 * nm); sp->modes.push_back(m); ++nm; }
  SpaceDev& d = sp->dev;
  d.n_models = desc->n_models;
  d.n_facts = (u32)sp->facts.size();
  d.nv = desc->n_act_variants;
  d.nt = desc->n_tpa_variants;
  d.nvt = d.nv * d.nt;
  d.nm = nm;
  d.modemap = modemap;
  d.n3 = nm * nm * nm;
  d.n_codes = d.n3 * nm;
  d.tp_max_valid = desc->tp_max_valid;
  d.tp_coll = desc->tp_coll_per_layer;
  d.sstar_units = desc->sstar_units ? desc->sstar_units : 1;
  d.accum = accum;
  d.repl = desc->replication_k ? desc->replication_k : 1;
  d.all_pow2 = 1;
  for (u32 i = 0; i < desc->n_n; ++i)
    if (desc->n_values[i] & (desc->n_values[i] - 1)) d.all_pow2 = 0;
  const u64 ppm = (u64)d.n_facts * d.nvt * d.n_codes;
  if (ppm >= ((u64)1 << 32)) { delete sp; return PS_E_RANGE; }
  d.ppm = ppm;

  bool ok = cudaMalloc(&sp->d_shapes, sizeof(ps_model_shape) * (size_t)desc->n_models) == cudaSuccess &&
            cudaMalloc(&sp->d_recs, sizeof(ModelRec) * (size_t)desc->n_models) == cudaSuccess &&
            cudaMalloc(&sp->d_facts, sizeof(Fact) * sp->facts.size()) == cudaSuccess &&
            cudaMalloc(&sp->d_order, sizeof(u32) * (size_t)desc->n_models) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(sp->d_facts, sp->facts.data(), sizeof(Fact) * sp->facts.size(),
                             cudaMemcpyHostToDevice, ctx->stream) == cudaSuccess;
  if (!ok) { ps_space_destroy(sp); return PS_E_CUDA; }
  d.recs = sp->d_recs;
  d.facts = sp->d_facts;
  d.order = sp->d_order;
  int rc = ps_space_set_models(sp, desc->models, desc->n_models);
  if (rc == PS_OK && cudaStreamSynchronize(ctx->stream) != cudaSuccess) rc = PS_E_CUDA;
  if (rc != PS_OK) { ps_space_destroy(sp); return rc; }
  *out = sp;
  return PS_OK;
}

// The order in which the sweeps' blocks take the models: most expected work first, so
// that the blocks still running when the grid runs out are short ones.  A sweep block's
// duration grows with the number of factorisations that pass the composition tests for
// its model (T divides the heads, K divides the layers, T within the valid tensor
// degree): only those have survivors under a filter that requires a valid composition,
// and a unit with survivors costs several times one without.  The count is a sum over
// the distinct (T, K) pairs of the space, weighted by how many device counts have them.
static void sweep_order(ps_space* sp, const ps_model_shape* models, u32 n_models) {
  std::vector<std::pair<u32, std::vector<std::pair<u32, u32>>>> by_t;   // T -> (K, number of factorisations)
  for (const Fact& f : sp->facts) {
    if (f.T > sp->dev.tp_max_valid) continue;
    auto t = std::find_if(by_t.begin(), by_t.end(), [&](const auto& e) { return e.first == f.T; });
    if (t == by_t.end()) { by_t.push_back({f.T, {}}); t = by_t.end() - 1; }
    auto k = std::find_if(t->second.begin(), t->second.end(), [&](const auto& e) { return e.first == f.K; });
    if (k == t->second.end()) t->second.push_back({f.K, 1u}); else ++k->second;
  }
  std::vector<u32> work(n_models, 0);
  for (u32 i = 0; i < n_models; ++i)
    for (const auto& t : by_t) {
      if (models[i].heads % t.first) continue;
      for (const auto& k : t.second)
        if (models[i].layers % k.first == 0) work[i] += k.second;
    }
  sp->order.resize(n_models);
  for (u32 i = 0; i < n_models; ++i) sp->order[i] = i;
  // (among models with the same count the smaller first: more of its points fit a capacity)
  std::stable_sort(sp->order.begin(), sp->order.end(), [&](u32 a, u32 b) {
    if (work[a] != work[b]) return work[a] > work[b];
    const u64 pa = (u64)models[a].layers * models[a].hidden * models[a].hidden;
    const u64 pb = (u64)models[b].layers * models[b].hidden * models[b].hidden;
    return pa < pb;
  });
}

int ps_space_set_models(ps_space* sp, const ps_model_shape* models, uint32_t n_models) {
  if (!sp || !models) return PS_E_NULLPTR;
  if (n_models != sp->dev.n_models) return PS_E_RANGE;
  u32 all_small = 1;
  for (u32 i = 0; i < n_models; ++i) {
    if (!shape_in_range(models[i], sp->dev.tp_coll, sp->dev.accum)) return PS_E_RANGE;
    if (!shape_is_small(models[i], sp->dev.accum)) all_small = 0;
  }
  sp->dev.all_small = all_small;
  sweep_order(sp, models, n_models);
  ps_ctx* ctx = sp->ctx;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(cudaMemcpyAsync(sp->d_order, sp->order.data(), sizeof(u32) * (size_t)n_models, cudaMemcpyHostToDevice,
                          ctx->stream));
  CUDA_OK(cudaMemcpyAsync(sp->d_shapes, models, sizeof(ps_model_shape) * (size_t)n_models,
                          cudaMemcpyHostToDevice, ctx->stream));
  CUDA_OK(launch_model_derive(sp->d_shapes, sp->d_recs, n_models, ctx->d_status, ctx->stream));
  return PS_OK;
}

int ps_space_rederive(ps_space* sp) {
  if (!sp) return PS_E_NULLPTR;
  ps_ctx* ctx = sp->ctx;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(launch_model_derive(sp->d_shapes, sp->d_recs, sp->dev.n_models, ctx->d_status, ctx->stream));
  return PS_OK;
}

void ps_space_destroy(ps_space* sp) {
  if (!sp) return;
  DeviceGuard guard(sp->ctx->device);
  cudaStreamSynchronize(sp->ctx->stream);
  if (sp->d_shapes) cudaFree(sp->d_shapes);
  if (sp->d_recs) cudaFree(sp->d_recs);
  if (sp->d_facts) cudaFree(sp->d_facts);
  if (sp->d_order) cudaFree(sp->d_order);
  delete sp;
}

uint64_t ps_space_size(const ps_space* sp) { return sp ? sp->dev.ppm * sp->dev.n_models : 0; }
uint64_t ps_space_points_per_model(const ps_space* sp) { return sp ? sp->dev.ppm : 0; }

int ps_space_decode(const ps_space* sp, uint64_t idx, ps_point* out) {
  if (!sp || !out) return PS_E_NULLPTR;
  if (idx >= ps_space_size(sp)) return PS_E_BADINDEX;
  const SpaceDev& d = sp->dev;
  out->model = (u32)(idx / d.ppm);
  u64 r = idx % d.ppm;
  const u64 per_unit = (u64)d.nvt * d.n_codes;
  const Fact& f = sp->facts[(size_t)(r / per_unit)];
  r %= per_unit;
  out->N = f.N; out->T = f.T; out->K = f.K; out->D = f.D;
  const u32 vt = (u32)(r / d.n_codes);
  u32 code = (u32)(r % d.n_codes);
  out->act_variant = vt / d.nt;
  out->tpa_variant = vt % d.nt;
  u32 full = 0, weight = 1;
  for (int s = 0; s < 4; ++s) {
    full += weight * sp->modes[code % d.nm];
    code /= d.nm;
    weight *= 5;
  }
  out->code_dp = (uint16_t)full;
  out->code_tp = out->tpa_variant == 0 ? PS_CODE_TP_SEQPAR : PS_CODE_TP;
  out->code_pp = PS_CODE_PP;
  out->pad = 0;
  return PS_OK;
}

// ------------------------------------------------------------------ batch evaluation
int ps_eval_batch(ps_ctx* ctx, const ps_space* sp, uint64_t first, uint64_t count,
                  const ps_filter* filter, ps_out_soa out, uint64_t* d_idx_out, uint64_t* d_n_out) {
  if (!ctx || !sp) return PS_E_NULLPTR;
  if (sp->ctx != ctx) return PS_E_RANGE;
  const u64 size = ps_space_size(sp);
  if (first > size || count > size - first) return PS_E_BADINDEX;
  if (filter && !d_n_out) return PS_E_NULLPTR;
  if (!aligned(out.mem, 8) || !aligned(out.comm_paper, 8) || !aligned(out.comm_ext, 8) ||
      !aligned(out.host, 8) || !aligned(out.flags, 4) || !aligned(d_idx_out, 8) || !aligned(d_n_out, 8))
    return PS_E_ALIGN;
  if (filter && (filter->comm_kind > PS_COMM_PAPER_PLUS_EXT || (filter->require_flags & ~KNOWN_FLAGS)))
    return PS_E_RANGE;
  int rc = pending_device_error(ctx);
  if (rc != PS_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  if (count == 0) {
    if (filter) CUDA_OK(cudaMemsetAsync(d_n_out, 0, sizeof(u64), ctx->stream));
    return PS_OK;
  }
  EvalArgs a;
  memset(&a, 0, sizeof(a));
  a.first = first;
  a.count = count;
  a.first_group = first / sp->dev.n_codes;
  const u64 last_group = (first + count - 1) / sp->dev.n_codes;
  const u64 n_groups = last_group - a.first_group + 1;
  if (n_groups > (u64)0x7fffffff) return PS_E_RANGE;
  a.n_tiles = (u32)n_groups;
  a.out = out;
  a.idx_out = d_idx_out;
  a.n_out = d_n_out;
  a.status = ctx->d_status;
  if (!filter) {
    CUDA_OK(launch_eval_materialise(sp->dev, a, ctx->stream));
  } else {
    a.has_filter = 1;
    a.cap_bytes = filter->cap_bytes;
    a.host_cap = filter->host_cap;
    a.require_flags = filter->require_flags & ~(u32)PS_F_FEASIBLE;
    // per group a count and a place in the list of groups with survivors, the list's length,
    // per run of groups an offset
    const size_t cnt_bytes = (sizeof(u32) * n_groups + 15) & ~size_t(15);
    rc = ensure_scratch(ctx, 2 * cnt_bytes + 16 + sizeof(u64) * n_groups);
    if (rc != PS_OK) return rc;
    char* base = static_cast<char*>(ctx->scratch);
    a.tile_count = reinterpret_cast<u32*>(base);
    a.nonempty = reinterpret_cast<u32*>(base + cnt_bytes);
    a.tile_offset = reinterpret_cast<u64*>(base + 2 * cnt_bytes + 16);
    // the list's length: one of the context's two counters, zero by now (the previous
    // compaction's scan cleared it); this call's scan clears the other
    a.n_nonempty = ctx->d_status + 2 + (ctx->compact_calls & 1u);
    a.n_nonempty_other = ctx->d_status + 2 + ((ctx->compact_calls + 1) & 1u);
    ++ctx->compact_calls;
    eval_plan_runs(a);
    CUDA_OK(launch_eval_count(sp->dev, a, ctx->stream));
    CUDA_OK(launch_tile_scan(a, ctx->stream));
    CUDA_OK(launch_eval_write(sp->dev, a, ctx->stream));
  }
  return enqueue_status_copy(ctx);
}

// ------------------------------------------------------------------ sweeps
int ps_sweep_pareto(ps_ctx* ctx, const ps_space* sp, const ps_filter* filter,
                    const uint64_t* caps_bytes, uint32_t n_caps, uint32_t reduce_kind,
                    uint32_t max_entries, ps_front_entry* d_out, uint32_t* d_counts) {
  if (!ctx || !sp || !filter || !caps_bytes || !d_out || !d_counts) return PS_E_NULLPTR;
  if (sp->ctx != ctx) return PS_E_RANGE;
  if (n_caps < 1 || n_caps > PS_MAX_CAPS || max_entries < 1) return PS_E_RANGE;
  if (reduce_kind != PS_REDUCE_PARETO && reduce_kind != PS_REDUCE_TOPK) return PS_E_RANGE;
  if (reduce_kind == PS_REDUCE_TOPK && max_entries > PS_TOPK_MAX) return PS_E_RANGE;
  if (filter->comm_kind > PS_COMM_PAPER_PLUS_EXT || (filter->require_flags & ~KNOWN_FLAGS)) return PS_E_RANGE;
  if (!aligned(d_out, 8) || !aligned(d_counts, 4)) return PS_E_ALIGN;
  int rc = pending_device_error(ctx);
  if (rc != PS_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;

  // top-k over a table of many models, in the fast case (powers of two, byte counts exact in a
  // double, every capacity below 2^53, nothing skipped): smaller blocks
  bool many = reduce_kind == PS_REDUCE_TOPK && !filter->skip_rejected && sp->dev.all_pow2 && sp->dev.all_small &&
              sp->dev.repl == 1 &&
              (u64)sp->dev.n_models >= (u64)SWEEP_TOPK_MANY_WAVES * ctx->sm_count * SWEEP_BLOCKS_TOPK_MANY;
  for (u32 c = 0; c < n_caps; ++c) many = many && caps_bytes[c] < ((u64)1 << 53) - 1;
  const u32 n_chunks = pick_chunks(ctx, sp, (int)reduce_kind, many);
  const size_t slots = (size_t)sp->dev.n_models * n_chunks * sweep_warps((int)reduce_kind, many);   // one list per warp
  const size_t partial_bytes = slots * SWEEP_LIST_CAP * sizeof(PartialEntry);
  const size_t lengths_bytes = (slots * sizeof(uint2) + 15) & ~size_t(15);
  rc = ensure_scratch(ctx, partial_bytes + lengths_bytes + sizeof(u32) * (size_t)sp->dev.n_models);
  if (rc != PS_OK) return rc;
  SweepArgs s;
  memset(&s, 0, sizeof(s));
  s.host_cap = filter->host_cap;
  s.require_flags = filter->require_flags & ~(u32)PS_F_FEASIBLE;
  s.comm_kind = filter->comm_kind;
  s.k_keep = reduce_kind == PS_REDUCE_TOPK ? max_entries : 0;
  s.skip_rejected = filter->skip_rejected ? 1u : 0u;
  s.many_models = many ? 1u : 0u;
  s.partial = static_cast<PartialEntry*>(ctx->scratch);
  s.partial_n = reinterpret_cast<uint2*>(static_cast<char*>(ctx->scratch) + partial_bytes);
  s.status = ctx->d_status;
  MergeArgs m;
  memset(&m, 0, sizeof(m));
  m.partial = s.partial;
  m.partial_n = s.partial_n;
  m.n_lists = n_chunks * sweep_warps((int)reduce_kind, many);
  m.host_cap = filter->host_cap;
  m.require_flags = s.require_flags;
  m.n_caps_total = n_caps;
  m.max_entries = max_entries;
  m.k_keep = s.k_keep;
  m.comm_kind = filter->comm_kind;
  m.out = d_out;
  m.counts = d_counts;
  m.slow_path = reinterpret_cast<u32*>(static_cast<char*>(ctx->scratch) + partial_bytes + lengths_bytes);
  m.status = ctx->d_status;
  if (reduce_kind == PS_REDUCE_PARETO) {
    u64 cap_max = 0;
    for (u32 c = 0; c < n_caps; ++c) { m.caps[c] = caps_bytes[c]; if (caps_bytes[c] > cap_max) cap_max = caps_bytes[c]; }
    s.cap_max = cap_max;
    m.cap_max = cap_max;
    m.n_caps = n_caps;
    CUDA_OK(launch_sweep(PS_REDUCE_PARETO, sp->dev, s, n_chunks, ctx->stream));
    CUDA_OK(launch_sweep_merge(PS_REDUCE_PARETO, sp->dev, m, ctx->stream));
  } else {
    for (u32 c = 0; c < n_caps; ++c) {
      s.cap_max = caps_bytes[c];
      m.caps[0] = caps_bytes[c];
      m.n_caps = 1;
      m.cap_index = c;
      m.cap_max = caps_bytes[c];
      CUDA_OK(launch_sweep(PS_REDUCE_TOPK, sp->dev, s, n_chunks, ctx->stream));
      CUDA_OK(launch_sweep_merge(PS_REDUCE_TOPK, sp->dev, m, ctx->stream));
    }
  }
  return enqueue_status_copy(ctx);
}

// ------------------------------------------------------------------ one composition
int ps_check_composition(ps_ctx* ctx, const ps_model_shape* shape, uint32_t N, uint32_t T,
                         uint32_t K, uint32_t D, uint16_t code_tp, uint16_t code_pp,
                         uint16_t code_dp, uint32_t act_variant, uint64_t cap_bytes,
                         uint32_t tp_max_valid, uint32_t tp_coll_per_layer, uint32_t comm_kind,
                         ps_front_entry* h_out) {
  if (!ctx || !shape || !h_out) return PS_E_NULLPTR;
  if (N < 1 || N > (1u << 24) || T < 1 || T > (1u << 24) || K < 1 || K > (1u << 24) || D < 1 ||
      D > (1u << 24))
    return PS_E_RANGE;
  if (code_tp > 624 || code_pp > 624 || code_dp > 624 || act_variant > 1 ||
      comm_kind > PS_COMM_PAPER_PLUS_EXT)
    return PS_E_RANGE;
  if (!shape_in_range(*shape, tp_coll_per_layer)) return PS_E_RANGE;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  int rc = ensure_scratch(ctx, 1024);
  if (rc != PS_OK) return rc;
  char* base = static_cast<char*>(ctx->scratch);
  ps_model_shape* d_shape = reinterpret_cast<ps_model_shape*>(base);
  ModelRec* d_rec = reinterpret_cast<ModelRec*>(base + 256);
  ps_front_entry* d_out = reinterpret_cast<ps_front_entry*>(base + 512);
  CUDA_OK(cudaMemcpyAsync(d_shape, shape, sizeof(ps_model_shape), cudaMemcpyHostToDevice, ctx->stream));
  CUDA_OK(launch_model_derive(d_shape, d_rec, 1, ctx->d_status, ctx->stream));
  // Table 2: tensor axis (S,S,S,S) or (S,S,S,R), pipeline axis (S,S,S,R); an axis
  // of degree 1 is absent.  Activation mode of the tensor axis: digit 3 of its code.
  const bool tp_form = (T == 1) || code_tp == PS_CODE_TP_SEQPAR || code_tp == PS_CODE_TP;
  const bool pp_form = (K == 1) || code_pp == PS_CODE_PP;
  const u32 tau = ((code_tp / 125) % 5 == PS_MODE_S) ? 0 : 1;
  CUDA_OK(launch_check_point(d_rec, Fact{N, T, K, D}, act_variant, tau, code_dp, tp_max_valid,
                             tp_coll_per_layer, (tp_form && pp_form) ? 1 : 0, comm_kind, cap_bytes,
                             d_out, ctx->stream));
  CUDA_OK(cudaMemcpyAsync(h_out, d_out, sizeof(ps_front_entry), cudaMemcpyDeviceToHost, ctx->stream));
  CUDA_OK(cudaStreamSynchronize(ctx->stream));
  return PS_OK;
}

// ------------------------------------------------------------------ Algorithm 1
int ps_select(ps_ctx* ctx, const ps_select_query* d_queries, uint64_t n, uint32_t headroom_num,
              uint32_t headroom_den, uint32_t layer_num, uint32_t layer_den, uint32_t tp_degree,
              ps_select_result* d_out) {
  if (!ctx || (n && (!d_queries || !d_out))) return PS_E_NULLPTR;
  if (!aligned(d_queries, 16) || !aligned(d_out, 16)) return PS_E_ALIGN;
  if (headroom_den < 1 || layer_den < 1 || tp_degree < 1 || headroom_num > (1u << 16) ||
      headroom_den > (1u << 16) || layer_num > (1u << 16) || layer_den > (1u << 16) ||
      n > ((u64)1 << 38))
    return PS_E_RANGE;
  if (n == 0) return PS_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(launch_select(d_queries, n, headroom_num, headroom_den, layer_num, layer_den, tp_degree, d_out,
                        ctx->stream));
  return PS_OK;
}

int ps_select_compare(ps_ctx* ctx, const ps_space* sp, uint32_t n_index, uint64_t device_bytes,
                      uint32_t fast_interconnect, uint32_t headroom_num, uint32_t headroom_den,
                      uint32_t layer_num, uint32_t layer_den, uint32_t tp_degree, const ps_filter* filter,
                      const ps_front_entry* d_frontier, const uint32_t* d_counts, uint32_t n_caps,
                      uint32_t cap_index, uint32_t max_entries, ps_select_compare_result* d_out) {
  if (!ctx || !sp || !filter || !d_frontier || !d_counts || !d_out) return PS_E_NULLPTR;
  if (sp->ctx != ctx) return PS_E_RANGE;
  if (!aligned(d_frontier, 8) || !aligned(d_counts, 4) || !aligned(d_out, 8)) return PS_E_ALIGN;
  if (n_index >= sp->n_values.size() || n_caps < 1 || n_caps > PS_MAX_CAPS || cap_index >= n_caps || max_entries < 1 ||
      headroom_den < 1 || layer_den < 1 || tp_degree < 1 || headroom_num > (1u << 16) || headroom_den > (1u << 16) ||
      layer_num > (1u << 16) || layer_den > (1u << 16) || device_bytes > ((u64)1 << 50) ||
      filter->comm_kind > PS_COMM_PAPER_PLUS_EXT || (filter->require_flags & ~KNOWN_FLAGS))
    return PS_E_RANGE;
  int rc = pending_device_error(ctx);
  if (rc != PS_OK) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(launch_select_compare(sp->dev, sp->fact_begin[n_index], sp->fact_begin[n_index + 1], sp->n_values[n_index],
                                device_bytes, fast_interconnect, headroom_num, headroom_den, layer_num, layer_den,
                                tp_degree, filter->host_cap, filter->require_flags & ~(u32)PS_F_FEASIBLE,
                                filter->comm_kind, d_frontier, d_counts, n_caps, cap_index, max_entries, d_out,
                                ctx->stream));
  return PS_OK;
}

// ------------------------------------------------------------------ verification protocol
int ps_verify_batch(ps_ctx* ctx, const ps_verify_shape* shape, const ps_verify_case* d_cases, uint64_t n,
                    const double* d_data, uint64_t data_len, ps_verify_result* d_out, double* d_theta_out) {
  if (!ctx || !shape || (n && (!d_cases || !d_data || !d_out))) return PS_E_NULLPTR;
  if (!aligned(d_cases, 8) || !aligned(d_data, 8) || !aligned(d_out, 8) || !aligned(d_theta_out, 8)) return PS_E_ALIGN;
  const ps_verify_shape& s = *shape;
  if (s.units < 1 || s.units > 8 || s.h < 1 || s.h > 32 || s.b < 1 || s.b > 4 || s.accum < 1 || s.accum > 4 ||
      s.steps < 1 || s.steps > 16 || s.gather_buffers < 1 || s.gather_buffers > 2)
    return PS_E_RANGE;
  if (s.w_theta < 1 || s.w_theta > 16 || s.w_grad < 1 || s.w_grad > 16 || s.w_omega < 3 || s.w_omega > 48 ||
      s.w_omega % 3 != 0)
    return PS_E_RANGE;
  if (!(s.lr > 0) || !(s.beta1 >= 0 && s.beta1 < 1) || !(s.beta2 >= 0 && s.beta2 < 1) || !(s.eps > 0) ||
      !(s.rtol >= 0) || !(s.atol >= 0) || n > ((u64)1 << 32))
    return PS_E_RANGE;
  int rc = pending_device_error(ctx);
  if (rc != PS_OK) return rc;
  if (n == 0) return PS_OK;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  rc = ensure_scratch(ctx, sizeof(double) * verify_workspace_doubles(s) * (size_t)n);
  if (rc != PS_OK) return rc;
  CUDA_OK(launch_verify(s, d_cases, n, d_data, data_len, static_cast<double*>(ctx->scratch), d_theta_out, d_out,
                        ctx->d_status, ctx->stream));
  return enqueue_status_copy(ctx);
}

// ------------------------------------------------------------------ measurement
int ps_int_peak(ps_ctx* ctx, uint32_t blocks, uint32_t iters, uint32_t* d_sink, uint64_t* thread_ops) {
  if (!ctx || !d_sink || !thread_ops) return PS_E_NULLPTR;
  if (blocks < 1 || blocks > (1u << 20) || iters < 1) return PS_E_RANGE;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  CUDA_OK(launch_int_peak(blocks, iters, d_sink, ctx->stream));
  *thread_ops = (u64)blocks * 256 * iters * 128;   // 8 rounds x 8 chains x 2 operations
  return PS_OK;
}

}  // extern "C"

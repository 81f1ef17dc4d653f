// ps_eval_compact_noalloc: the filter-and-compact path of ps_eval_batch for
// callers that must not allocate device memory.  The per-group survivor counts
// and the prefix sums over runs of groups live in a fixed array that is part of
// the library image instead of in the context's growable scratch.
#include <cuda_runtime.h>
#include <string.h>
#include <mutex>

#include "ps.h"
#include "ps_device.cuh"
#include "ps_internal.h"

namespace {

constexpr size_t COUNT_BYTES = sizeof(u32) * (size_t)PS_NOALLOC_MAX_GROUPS;
constexpr size_t LENGTH_BYTES = 256;
constexpr size_t OFFSET_BYTES = sizeof(u64) * (size_t)PS_NOALLOC_MAX_GROUPS;

// 2 MiB on every GPU that loads the library, for the life of the process:
// [0, COUNT_BYTES) survivor count of each group, then the list of groups that
// have survivors, its length, and the exclusive prefix sums (one per run of
// groups, so at most one per group).
static __device__ __align__(256) unsigned char g_fixed_scratch[2 * COUNT_BYTES + LENGTH_BYTES + OFFSET_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_setup_lock;
void* g_scratch_addr[MAX_DEVICES];   // device address of g_fixed_scratch, per device
bool g_scratch_ready[MAX_DEVICES];

// The array's name is only a handle on the host; the address a kernel can use
// has to be asked for, once per device, while that device is current.
int fixed_scratch_for(int device, void** out) {
  if (device < 0 || device >= MAX_DEVICES) return PS_E_RANGE;
  std::lock_guard<std::mutex> hold(g_setup_lock);
  if (!g_scratch_ready[device]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_fixed_scratch) != cudaSuccess || p == nullptr) return PS_E_CUDA;
    g_scratch_addr[device] = p;
    g_scratch_ready[device] = true;
  }
  *out = g_scratch_addr[device];
  return PS_OK;
}

struct CurrentDevice {
  int prev;
  bool ok;
  explicit CurrentDevice(int dev) : prev(-1), ok(false) {
    if (cudaGetDevice(&prev) != cudaSuccess) return;
    ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
  }
  ~CurrentDevice() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

bool is_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" int ps_eval_compact_noalloc(ps_ctx* ctx, const ps_space* sp, uint64_t first,
                                       uint64_t count, const ps_filter* filter, ps_out_soa out,
                                       uint64_t* d_idx_out, uint64_t* d_n_out) {
  if (!ctx || !sp || !filter || !d_n_out) return PS_E_NULLPTR;
  if (sp->ctx != ctx) return PS_E_RANGE;
  const u64 size = sp->dev.ppm * sp->dev.n_models;
  if (first > size || count > size - first) return PS_E_BADINDEX;
  if (!is_aligned(out.mem, 8) || !is_aligned(out.comm_paper, 8) || !is_aligned(out.comm_ext, 8) ||
      !is_aligned(out.host, 8) || !is_aligned(out.flags, 4) || !is_aligned(d_idx_out, 8) ||
      !is_aligned(d_n_out, 8))
    return PS_E_ALIGN;
  if (filter->comm_kind > PS_COMM_PAPER_PLUS_EXT || (filter->require_flags & ~((PS_F_PAPER_PRICED << 1) - 1u)))
    return PS_E_RANGE;
  const u32 seen = *ctx->h_status & ~(u32)ST_TRUNCATED;   // a kernel-reported problem of an earlier call
  if (seen) return PS_E_DEVICE;
  CurrentDevice guard(ctx->device);
  if (!guard.ok) return PS_E_CUDA;
  if (count == 0) {
    if (cudaMemsetAsync(d_n_out, 0, sizeof(u64), ctx->stream) != cudaSuccess) return PS_E_CUDA;
    return PS_OK;
  }
  EvalArgs a;
  memset(&a, 0, sizeof(a));
  a.first = first;
  a.count = count;
  a.first_group = first / sp->dev.n_codes;
  const u64 n_groups = (first + count - 1) / sp->dev.n_codes - a.first_group + 1;
  if (n_groups > (u64)PS_NOALLOC_MAX_GROUPS) return PS_E_NOALLOC_LIMIT;
  void* base = nullptr;
  const int rc = fixed_scratch_for(ctx->device, &base);
  if (rc != PS_OK) return rc;
  a.n_tiles = (u32)n_groups;
  a.out = out;
  a.idx_out = d_idx_out;
  a.n_out = d_n_out;
  a.status = ctx->d_status;
  a.has_filter = 1;
  a.cap_bytes = filter->cap_bytes;
  a.host_cap = filter->host_cap;
  a.require_flags = filter->require_flags & ~(u32)PS_F_FEASIBLE;
  unsigned char* bytes = static_cast<unsigned char*>(base);
  a.tile_count = reinterpret_cast<u32*>(bytes);
  a.nonempty = reinterpret_cast<u32*>(bytes + COUNT_BYTES);
  a.n_nonempty = ctx->d_status + 2 + (ctx->compact_calls & 1u);          // the context's alternating list lengths
  a.n_nonempty_other = ctx->d_status + 2 + ((ctx->compact_calls + 1) & 1u);
  ++ctx->compact_calls;
  a.tile_offset = reinterpret_cast<u64*>(bytes + 2 * COUNT_BYTES + LENGTH_BYTES);
  eval_plan_runs(a);
  // The array still holds the previous call's numbers.  Every word this call
  // reads is written earlier in this call (the count pass stores a count for
  // each group and a total for each run of groups, the scan turns the totals
  // into offsets); the counts are cleared anyway so that a stale value can
  // never be mistaken for a fresh one.
  if (cudaMemsetAsync(a.tile_count, 0, sizeof(u32) * n_groups, ctx->stream) != cudaSuccess) return PS_E_CUDA;
  if (launch_eval_count(sp->dev, a, ctx->stream) != cudaSuccess) return PS_E_CUDA;
  if (launch_tile_scan(a, ctx->stream) != cudaSuccess) return PS_E_CUDA;
  if (launch_eval_write(sp->dev, a, ctx->stream) != cudaSuccess) return PS_E_CUDA;
  if (cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(u32), cudaMemcpyDeviceToHost, ctx->stream) != cudaSuccess)
    return PS_E_CUDA;
  return PS_OK;
}

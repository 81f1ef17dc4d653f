// Host-visible declarations shared by the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include "ps.h"
#include "ps_device.cuh"

// ---- the opaque handles of ps.h
#include <vector>
struct ps_ctx {
  int device;
  cudaStream_t stream;
  void* scratch;
  size_t scratch_bytes;
  u32* d_status;      // 16 bytes: the status word, then (at +2) the two list lengths of the compaction
  u32* h_status;      // pinned
  u32 compact_calls;  // compactions enqueued so far (picks which list length a call uses)
  int sm_count;
};

struct ps_space {
  ps_ctx* ctx;
  ps_space_desc desc;             // pointers inside are not kept
  std::vector<u32> n_values;
  std::vector<Fact> facts;        // all N concatenated
  std::vector<u32> fact_begin;    // per N, offset into facts (n_n + 1 entries)
  std::vector<u32> modes;         // allowed modes ascending
  ps_model_shape* d_shapes;
  ModelRec* d_recs;
  Fact* d_facts;
  u32* d_order;                   // see SpaceDev::order
  std::vector<u32> order;
  SpaceDev dev;
};

// ---- sweep
// Block shapes of the sweep: warps per block and the resident blocks per SM the
// kernel is compiled for (which sets its register budget).  The top-k sweep is
// fastest with eight blocks of three warps (24 warps of 80 registers; 1184 resident
// blocks, so that a thousand models run as one wave): few and long lists per model.
// The Pareto sweep is fastest with four blocks of four warps (16 warps of 128
// registers): since its reduction pass became short, what it gains from registers
// outweighs what larger blocks gain from sharing a coarse staircase (2 x 10 warps of
// 96 registers: +6 %; 2 x 8: +2.5 %; 3 x 5, 8 x 2, 1 x 16: +3 to +10 %).
#ifndef SWEEP_WARPS_TOPK
#define SWEEP_WARPS_TOPK 3
#endif
#ifndef SWEEP_BLOCKS_TOPK
#define SWEEP_BLOCKS_TOPK 8
#endif
#ifndef SWEEP_WARPS_PARETO
#define SWEEP_WARPS_PARETO 4
#endif
#ifndef SWEEP_BLOCKS_PARETO
#define SWEEP_BLOCKS_PARETO 4
#endif
// A table of many models (at least SWEEP_TOPK_MANY_WAVES full waves of the smaller blocks) is
// swept for top-k with blocks of two warps, nine resident per SM: -3.7 % on four thousand
// models; on a thousand models the GPU is then short of warps (+10 %), so those keep three.
// Compiled for the fast case without skipping only (see launch_sweep_t).
#ifndef SWEEP_WARPS_TOPK_MANY
#define SWEEP_WARPS_TOPK_MANY 2
#endif
#ifndef SWEEP_BLOCKS_TOPK_MANY
#define SWEEP_BLOCKS_TOPK_MANY 9
#endif
#ifndef SWEEP_TOPK_MANY_WAVES
#define SWEEP_TOPK_MANY_WAVES 2
#endif
static inline int sweep_warps(int kind, bool many = false) {
  return kind == PS_REDUCE_PARETO ? SWEEP_WARPS_PARETO : (many ? SWEEP_WARPS_TOPK_MANY : SWEEP_WARPS_TOPK);
}
static inline int sweep_blocks_per_sm(int kind, bool many = false) {
  return kind == PS_REDUCE_PARETO ? SWEEP_BLOCKS_PARETO : (many ? SWEEP_BLOCKS_TOPK_MANY : SWEEP_BLOCKS_TOPK);
}
#define SWEEP_LIST_CAP 128        /* entries of a warp's list and of a block's partial list */
#define SWEEP_MAX_CHUNKS 16       /* blocks per model                                        */
#define MERGE_CAP (5 * SWEEP_LIST_CAP)    /* entries the merge kernel combines at a time: what it
                                     has kept plus as many of the warps' lists as fit      */
#define PS_MAX_CAPS 8

struct PartialEntry {
  u64 a, b;   // Pareto: (mem, comm); top-k: (comm, mem)
  u32 i;      // point index within the model
  u32 pad;
};

struct SweepArgs {
  u64 cap_max;          // survivors need mem <= cap_max
  u64 host_cap;
  u32 require_flags;    // without PS_F_FEASIBLE
  u32 comm_kind;
  u32 k_keep;           // top-k: entries kept
  u32 skip_rejected;    // do not evaluate factorisations whose composition bits miss a required flag
  u32 many_models;      // top-k: the blocks of two warps (the host has checked that the fast case applies)
  u32 pad;
  PartialEntry* partial;   // [n_models * n_chunks * warps][SWEEP_LIST_CAP]: one list per warp
  uint2* partial_n;        // [n_models * n_chunks * warps]: (entries, survivors)
  u32* status;
};

struct MergeArgs {
  const PartialEntry* partial;
  const uint2* partial_n;
  u64 caps[PS_MAX_CAPS];
  u64 cap_max, host_cap;  // the filter again, for the slow exact path
  u32 require_flags;
  u32 n_lists;          // partial lists per model: blocks per model x warps per block
  u32 n_caps;           // capacities this launch emits
  u32 n_caps_total;     // capacities of the output layout
  u32 cap_index;        // top-k: which capacity this launch is for
  u32 max_entries;
  u32 k_keep;
  u32 comm_kind;
  ps_front_entry* out;
  u32* counts;
  u32* slow_path;       // Pareto, [n_models]: set by the merge for a model whose frontier outgrew the lists
  u32* status;
};

cudaError_t launch_sweep(int kind, const SpaceDev& sp, const SweepArgs& a, u32 n_chunks,
                         cudaStream_t stream);
cudaError_t launch_sweep_merge(int kind, const SpaceDev& sp, const MergeArgs& a, cudaStream_t stream);

// ---- batch evaluation
/* Block shape of the window kernels: four resident blocks of four warps (128 registers a thread
   either way).  Against two blocks of eight warps: materialise -5 % (625 codes a group) to -13 %
   (256 codes), sparse compaction -3 % to -8 %; short blocks spread the warps' set-up and store
   phases better. */
#ifndef EVAL_THREADS
#define EVAL_THREADS 128
#endif
#ifndef EVAL_MIN_BLOCKS
#define EVAL_MIN_BLOCKS 4
#endif
#define EVAL_GROUPS_PER_TILE 8    /* a tile = this many consecutive groups of n_codes points */

struct EvalArgs {
  u64 first, count;         // the window
  u64 first_group;          // global group index of the tile 0's first group
  u32 n_tiles;
  // filter (compaction modes)
  u64 cap_bytes, host_cap;
  u32 require_flags;        // without PS_F_FEASIBLE
  u32 has_filter;
  ps_out_soa out;
  u64* idx_out;
  u64* n_out;
  // compaction scratch
  // compaction: the count pass walks the groups in n_runs runs of run_len
  // consecutive groups (one warp per run) -- set by eval_plan_runs
  u32 n_runs, run_len;
  u32* tile_count;          // [n_tiles] survivors of each group
  u32* nonempty;            // [n_tiles] the groups that have survivors, in any order
  u32* n_nonempty;          // how many (zero before the count pass)
  u32* n_nonempty_other;    // the next compaction's counter: the scan kernel clears it, so that no
                            // call needs a memset of its own (calls alternate between two counters)
  u64* tile_offset;         // [n_runs <= n_tiles] survivors of each run, then (scan) of all runs before it
  u32* status;
};

void eval_plan_runs(EvalArgs& a);   // fills n_runs, run_len from n_tiles (current device)
cudaError_t launch_eval_materialise(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream);
cudaError_t launch_eval_count(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream);
cudaError_t launch_tile_scan(const EvalArgs& a, cudaStream_t stream);
cudaError_t launch_eval_write(const SpaceDev& sp, const EvalArgs& a, cudaStream_t stream);

// ---- small kernels
cudaError_t launch_model_derive(const ps_model_shape* d_shapes, ModelRec* d_recs, u32 n,
                                u32* status, cudaStream_t stream);
cudaError_t launch_check_point(const ModelRec* d_rec, Fact f, u32 v, u32 tau, u32 code_dp,
                               u32 tp_max_valid, u32 tp_coll, u32 axis_form, u32 comm_kind,
                               u64 cap_bytes, ps_front_entry* d_out, cudaStream_t stream);
cudaError_t launch_select(const ps_select_query* d_q, u64 n, u32 head_num, u32 head_den, u32 layer_num,
                          u32 layer_den, u32 tp_degree, ps_select_result* d_out, cudaStream_t stream);
cudaError_t launch_int_peak(u32 blocks, u32 iters, u32* d_sink, cudaStream_t stream);

// ---- brute-force verifier
size_t verify_workspace_doubles(const ps_verify_shape& s);     // per case
cudaError_t launch_verify(const ps_verify_shape& s, const ps_verify_case* d_cases, u64 n, const double* d_data,
                          u64 data_len, double* d_ws, double* d_theta_out, ps_verify_result* d_out, u32* status,
                          cudaStream_t stream);

cudaError_t launch_select_compare(const SpaceDev& sp, u32 unit_begin, u32 unit_end, u32 N, u64 device_bytes, u32 fast,
                                  u32 head_num, u32 head_den, u32 layer_num, u32 layer_den, u32 tp_degree,
                                  u64 host_cap, u32 require_flags, u32 comm_kind, const ps_front_entry* d_frontier,
                                  const u32* d_counts, u32 n_caps, u32 cap_index, u32 max_entries,
                                  ps_select_compare_result* d_out, cudaStream_t stream);

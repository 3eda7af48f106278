// Internal declarations shared by the translation units of libtalon (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "talon.h"

namespace talon {

// ---- device status bits (ctx->d_status) -----------------------------------------------
constexpr int STATUS_NONFINITE = 1;
constexpr int STATUS_TIMEOUT = 2;
constexpr int STATUS_CAPACITY = 4;

// ---- expansion geometry -----------------------------------------------------------------
constexpr int EXP_THREADS = 256;           // threads per CTA of the row-streaming kernels
constexpr int EXP_WARPS = EXP_THREADS / 32;
constexpr int EXP_VEC = 4;                 // floats per 128-bit load
constexpr int EXP_UNROLL = 4;              // 128-bit loads in flight per thread
constexpr int EXP_TILE = EXP_THREADS * EXP_VEC * EXP_UNROLL;   // 4096 elements per CTA step
constexpr int EXP_CHUNK_ALIGN = EXP_THREADS * EXP_VEC;         // chunk boundaries: 1024 elements
constexpr int EXP_MAX_SPLITS = 32;         // a row is cut into at most this many chunks
constexpr int EXP_CTAS_PER_SM = 4;
constexpr int MAX_BUDGET = 128;
constexpr int MAX_BATCH = 1024;
constexpr int SEL_THREADS = 512;
// fused expansion kernel (k <= 32)
constexpr int FX_QCAP = 128;               // keys a warp's candidate buffer can hold
constexpr int FX_SURV = 64;                // keys of a row that may pass the merge bound before the slow path
constexpr int FX_MAX_SPLITS = 16;          // chunks per row, at most (one lane per chunk in the merge)

// Order-preserving map fp32 -> u32 (larger float <=> larger integer; -inf > 0).
__host__ __device__ inline uint32_t f32_ord(float f) {
#ifdef __CUDA_ARCH__
  uint32_t b = __float_as_uint(f);
#else
  union { float f; uint32_t u; } c; c.f = f; uint32_t b = c.u;
#endif
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__host__ __device__ inline float f32_unord(uint32_t o) {
  uint32_t b = (o & 0x80000000u) ? (o & 0x7FFFFFFFu) : ~o;
#ifdef __CUDA_ARCH__
  return __uint_as_float(b);
#else
  union { float f; uint32_t u; } c; c.u = b; return c.f;
#endif
}
// A candidate key: larger key = larger logit, then lower token id.  Key 0 means "empty".
__host__ __device__ inline uint64_t cand_key(float logit, uint32_t tok) {
  return ((uint64_t)f32_ord(logit) << 32) | (uint64_t)(0xFFFFFFFFu - tok);
}
__host__ __device__ inline float key_logit(uint64_t k) { return f32_unord((uint32_t)(k >> 32)); }
__host__ __device__ inline uint32_t key_tok(uint64_t k) { return 0xFFFFFFFFu - (uint32_t)k; }

// How one expansion layer is cut into work items.  Computed identically (from device data)
// by every CTA of the streaming kernel and by the selection kernel.
struct LayerGeom {
  int total_rows;   // frontier rows over all sequences
  int splits;       // chunks per row
  int chunk_len;    // elements per chunk (multiple of EXP_CHUNK_ALIGN)
};

__host__ __device__ inline LayerGeom make_geom(int total_rows, int vocab, int target_items,
                                               int max_splits = EXP_MAX_SPLITS, int min_chunk = EXP_CHUNK_ALIGN) {
  LayerGeom g;
  g.total_rows = total_rows;
  int want = total_rows > 0 ? (target_items + total_rows - 1) / total_rows : 1;
  if (want < 1) want = 1;
  if (want > max_splits) want = max_splits;
  int len = (vocab + want - 1) / want;
  len = ((len + EXP_CHUNK_ALIGN - 1) / EXP_CHUNK_ALIGN) * EXP_CHUNK_ALIGN;
  if (len < min_chunk) len = min_chunk;
  g.chunk_len = len;
  g.splits = (vocab + len - 1) / len;
  return g;
}

}  // namespace talon

namespace talon {
// A whole step captured as a CUDA graph, keyed by every argument of the call that made it.
constexpr int STEP_GRAPH_SLOTS = 64;
constexpr int STEP_GRAPH_WORDS = 36;
struct StepGraph {
  unsigned long long args[STEP_GRAPH_WORDS];
  cudaGraphExec_t exec;      // null: arguments seen once, nothing captured yet
  long long launches;        // kernels one replay launches
  int layers_run;            // host-side depth counter after the step
  unsigned long long last_use;
  bool used;
};
}  // namespace talon

// The context: parameters, host-side counters, and the device workspace.
struct talon_ctx {
  talon_params p;
  int device;
  int sm_count;
  int W;                  // mask words per node
  int k_cap;              // per-parent candidate cap actually used (cand_topk or N-1)
  int k_slots;            // ceil(k_cap / 32): list registers per lane
  int key_stride;         // keys stored per row / per item (k_cap rounded up to 4)
  int B;                  // batch of the current reset
  int layers_run;         // expand calls since reset
  int64_t launches;
  double log_mu;

  int *d_status;
  int32_t *d_prefix_len;          // [batch_max]
  // expansion workspace
  int exp_grid;                   // CTAs of the streaming kernel at full width
  int rows_cap;                   // batch_max * (N-1)
  int items_cap;                  // exp_grid + rows_cap
  unsigned long long *d_part_keys;   // [items_cap, key_stride]  per-chunk top-k
  float2 *d_part_ms;                 // [items_cap]              per-chunk (max, sum exp)
  unsigned long long *d_row_keys;    // [rows_cap, key_stride]   per-row top-k
  double *d_row_lse;                 // [rows_cap]               per-row log-sum-exp
  double *d_row_score;               // [rows_cap, key_stride]   per-row candidate scores (fused kernel, wide frontiers)
  unsigned int *d_row_count;         // [rows_cap]               chunks finished per row
  unsigned int *d_seq_count;         // [batch_max]              chunks finished per sequence (fused kernel)
  int fused_grid;                    // CTAs of the fused kernel at full width
  int attn_cluster;                  // key ranges of the tensor-core attention merge inside a cluster (1) or in a second kernel (0)
  long long attn_cluster_min_rows;   // automatic mode: least rows x key ranges for the merge inside the cluster
  int attn_cluster_cap;              // more key ranges than eight are cut back to eight up to this many
  int attn_cluster_ok[9];            // per cluster size: -1 not asked yet, 0 the device cannot place it, 1 it can
  int attn_force_splits;             // > 0: key ranges per (sequence, head, query tiles), for experiments
  int argmax_oversplit;              // target argmax: chunk rounds per CTA when the rows outnumber the grid
  int expand_max_split;              // fused kernel: chunks a row is cut into at most when the grid has room
  int attn_min_tiles;                // split-KV: key tiles a CTA should at least own
  int pdl;                           // programmatic stream serialization: 1 on, 0 off, -1 on for small batches
  // verification workspace
  unsigned long long *d_argmax;      // [batch_max * N] packed (logit, token) maxima
  int32_t *d_target_tok;             // [batch_max * N]
  unsigned int *d_walk_count;        // [batch_max] argmax chunks finished per sequence (zero between calls)
  float2 *d_samp_ms;                 // [batch_max * N, EXP_MAX_SPLITS] per-chunk (max, sum) of target rows
  float *d_attn_o;                   // split-KV partial outputs
  float2 *d_attn_ml;                 // split-KV partial (max, sum)
  size_t attn_o_elems, attn_ml_elems;
  // host-step staging (allocated on first use)
  struct HostStage *stage;
  // per-kernel timing (off unless talon_timing_enable was called)
  cudaEvent_t *ev;                   // [2 * ev_cap] start/stop pairs
  int *ev_kernel;                    // [ev_cap] kernel id of each pair
  int ev_cap, ev_used;
  unsigned ev_mask;                  // kernel families that are timed
  int ev_paused;                     // 1: launches are not bracketed for now
  // talon_step replays (see talon_step)
  int step_graph;                    // 0: never capture
  unsigned long long step_tick;
  talon::StepGraph *graphs;          // [STEP_GRAPH_SLOTS], allocated on first use
};

namespace talon {

// Programmatic dependent launch.  Every kernel of the library starts with pdl_enter(): it lets
// the next kernel of the stream be scheduled at once and then waits until the previous kernel
// has completed and its memory is visible, so only launch latency overlaps, never data.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Launches `kernel` so that it may be scheduled while its predecessor in the stream drains
// (the kernel itself waits in pdl_enter()); a plain launch when ctx->pdl is off.  In automatic mode
// (-1) it is used for batches of at most PDL_AUTO_BATCH sequences: there the grids are small and the
// overlapped launch latency is a gain, while at larger batches the early-scheduled CTAs of the next
// kernel take SM slots from the running one.
constexpr int PDL_AUTO_BATCH = 4;
// `chain` marks the launches of a chain of short dependent kernels (the expansion layers): there
// the overlap of launch latency pays at every batch size (a layer that finds every tree full costs
// little more than its launch), while behind the long verification kernels it does not.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_pdl(const talon_ctx *c, bool chain, void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                     size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (c->pdl == 1 || (c->pdl < 0 && (c->B <= PDL_AUTO_BATCH || chain))) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(const talon_ctx *c, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t st, Args &&...args) {
  return launch_kernel_pdl(c, false, kernel, grid, block, smem, st, static_cast<Args &&>(args)...);
}

// Brackets one kernel launch with a pair of CUDA events on the launching stream when timing
// is on; does nothing otherwise.  Pairs beyond the capacity are silently not timed.
struct LaunchTimer {
  talon_ctx *c;
  cudaStream_t st;
  int slot;
  LaunchTimer(talon_ctx *ctx, int kernel, cudaStream_t stream) : c(ctx), st(stream), slot(-1) {
    if (c->ev && !c->ev_paused && ((c->ev_mask >> kernel) & 1u) && c->ev_used < c->ev_cap) {
      slot = c->ev_used++;
      c->ev_kernel[slot] = kernel;
      cudaEventRecord(c->ev[2 * slot], st);
    }
  }
  ~LaunchTimer() {
    if (slot >= 0) cudaEventRecord(c->ev[2 * slot + 1], st);
  }
};

// launchers implemented in the .cu files (all asynchronous on `st`)
talon_status launch_reset(talon_ctx *c, const talon_tree *t, const int32_t *root_tok,
                          const int32_t *prefix_len, int B, cudaStream_t st);
talon_status launch_expand(talon_ctx *c, const talon_tree *t, const float *logits,
                           int64_t row_stride, int rows_per_seq, int layout, cudaStream_t st);
talon_status launch_build(talon_ctx *c, const talon_tree *t, uint8_t *dense, cudaStream_t st);
talon_status launch_prune(talon_ctx *c, const talon_tree *t, int keep, cudaStream_t st);
talon_status launch_attention(talon_ctx *c, const talon_tree *t, const void *q, const void *kp,
                              const void *vp, const void *kt, const void *vt,
                              const int64_t *kv_start, const int32_t *block_table, int bt_stride, int64_t kv_tokens,
                              int64_t stride_t, int64_t stride_h,
                              int max_prefix_len, float sm_scale, void *out, cudaStream_t st);
bool attention_tc_supported(const talon_ctx *c, int64_t stride_t, int64_t stride_h, float sm_scale);
talon_status launch_attention_tc(talon_ctx *c, const talon_tree *t, const void *q, const void *kp, const void *vp,
                                 const void *kt, const void *vt, const int64_t *kv_start, const int32_t *block_table,
                                 int bt_stride, int64_t stride_t, int64_t stride_h, int64_t kv_tokens, int max_prefix_len, float sm_scale, void *out,
                                 int splits, int m_blocks, cudaStream_t st, int *merged_in_kernel);
talon_status launch_accept(talon_ctx *c, const talon_tree *t, const float *target_logits,
                           int64_t row_stride, int32_t *target_tok, int32_t *accept_len,
                           int32_t *accept_nodes, int32_t *bonus_tok, cudaStream_t st, bool close_tree = false);
talon_status launch_accept_sample(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                                  double temperature, const double *u_accept, const double *u_sample,
                                  int32_t *accept_len, int32_t *accept_nodes, int32_t *out_tok, cudaStream_t st);
talon_status launch_commit(talon_ctx *c, const talon_tree *t, const int32_t *accept_len, const int32_t *accept_nodes,
                           const int32_t *next_tok, const void *k_tree, const void *v_tree, void *k_prefix,
                           void *v_prefix, const int64_t *kv_start, const int64_t *kv_limit, const int32_t *block_table,
                           int bt_stride, const int32_t *n_blocks, int64_t kv_tokens, int64_t stride_t, int64_t stride_h,
                           int32_t *prefix_len, int32_t *root_tok, int64_t *counters, cudaStream_t st);
size_t attention_workspace_elems(const talon_ctx *c, size_t *ml_elems);
talon_status expand_fused_setup(talon_ctx *c);
talon_status launch_expand_fused(talon_ctx *c, const talon_tree *t, const float *logits, int64_t row_stride,
                                 int rows_per_seq, int layout, int rows_bound, cudaStream_t st);

}  // namespace talon

// After a verified step (generation loop of the paper's Section 5.3): the accepted tokens join
// the sequence.
//
//   commit_gather_kernel : one CTA per (sequence, accepted position): the key and value rows of
//                          accepted node j (all kv heads, 128-bit copies) go from the tree's K/V
//                          to the prefix cache at token prefix_len + j, root first.
//   commit_update_kernel : one thread per sequence: prefix_len += accepted + 1, the correction
//                          token becomes the next root, and the counts of Section 5.3 advance
//                          (N_p by one target pass, N_q by one draft pass per expanded layer of
//                          Algorithm 2, L by the tokens produced).
//
// A sequence whose block of the cache has no room for its accepted tokens is left untouched and
// the CAPACITY status is set.
#include "talon_internal.cuh"

namespace talon {

namespace {

constexpr int COMMIT_PAGE = 128;          // tokens per page of a paged cache (one key tile of the attention)

struct CommitArgs {
  talon_tree t;
  int lo_stride;
  int B, N, max_depth, layers_run, n_kv_heads, head_dim;
  const int32_t *accept_len, *accept_nodes, *next_tok;
  const uint4 *k_tree, *v_tree;       // [B, N, Hkv, Dh] bf16
  uint4 *k_prefix, *v_prefix;
  const int64_t *kv_start, *kv_limit;
  const int32_t *block_table, *n_blocks;   // paged cache: [B, bt_stride] page numbers, [B] pages a sequence owns
  int bt_stride;
  int64_t kv_tokens, stride_t, stride_h;   // elements
  int32_t *prefix_len, *root_tok;
  int64_t *counters;                  // [B, 3] or null
  int *status;
};

// first token past the block of sequence b
__device__ __forceinline__ int64_t block_end(const CommitArgs &a, int b) {
  const int64_t lim = a.kv_limit ? a.kv_limit[b] : a.kv_tokens;
  return lim < a.kv_tokens ? lim : a.kv_tokens;
}

__device__ __forceinline__ bool fits(const CommitArgs &a, int b, int len) {
  if (len < 0 || len > a.max_depth) return false;
  if (a.block_table) return (int64_t)a.prefix_len[b] + len + 1 <= (int64_t)a.n_blocks[b] * COMMIT_PAGE;
  return a.kv_start[b] + a.prefix_len[b] + len + 1 <= block_end(a, b);
}

// cache token that holds token `pos` of sequence b
__device__ __forceinline__ int64_t cache_token(const CommitArgs &a, int b, int pos) {
  if (a.block_table)
    return (int64_t)a.block_table[(size_t)b * a.bt_stride + pos / COMMIT_PAGE] * COMMIT_PAGE + pos % COMMIT_PAGE;
  return a.kv_start[b] + pos;
}

__global__ void commit_gather_kernel(CommitArgs a) {
  pdl_enter();
  const int b = blockIdx.y, j = blockIdx.x;
  const int len = a.accept_len[b];
  if (j > len || !fits(a, b, len)) return;
  const int node = a.accept_nodes[(size_t)b * (a.max_depth + 1) + j];
  if (node < 0 || node >= a.N) return;                      // a malformed path never indexes outside the tree
  const int vec_per_head = a.head_dim / 8;                  // 16-byte units per head row
  const int vecs = a.n_kv_heads * vec_per_head;
  const int64_t tok = cache_token(a, b, a.prefix_len[b] + j);
  const size_t src = ((size_t)b * a.N + node) * vecs;
  for (int i = threadIdx.x; i < 2 * vecs; i += blockDim.x) {
    const int which = i >= vecs, r = which ? i - vecs : i;
    const int h = r / vec_per_head, x = r - h * vec_per_head;
    const int64_t dst = (tok * a.stride_t + h * a.stride_h) / 8 + x;
    if (which) a.v_prefix[dst] = a.v_tree[src + r];
    else a.k_prefix[dst] = a.k_tree[src + r];
  }
}

__global__ void commit_update_kernel(CommitArgs a) {
  pdl_enter();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= a.B) return;
  const int len = a.accept_len[b];
  if (!fits(a, b, len)) {
    atomicOr(a.status, STATUS_CAPACITY);
    return;
  }
  a.prefix_len[b] += len + 1;
  a.root_tok[b] = a.next_tok[b];
  if (a.counters) {
    int passes = 0;                  // layers that had a frontier and budget left when their turn came
    const int *lo = a.t.layer_off + (size_t)b * a.lo_stride;
    for (int d = 0; d < a.layers_run && d < a.max_depth; ++d)
      passes += (lo[d + 1] > lo[d] && lo[d + 1] < a.N) ? 1 : 0;
    a.counters[3 * b + 0] += 1;
    a.counters[3 * b + 1] += passes;
    a.counters[3 * b + 2] += len + 1;
  }
}

}  // namespace

talon_status launch_commit(talon_ctx *c, const talon_tree *t, const int32_t *accept_len, const int32_t *accept_nodes,
                           const int32_t *next_tok, const void *k_tree, const void *v_tree, void *k_prefix,
                           void *v_prefix, const int64_t *kv_start, const int64_t *kv_limit, const int32_t *block_table,
                           int bt_stride, const int32_t *n_blocks, int64_t kv_tokens, int64_t stride_t, int64_t stride_h,
                           int32_t *prefix_len, int32_t *root_tok, int64_t *counters, cudaStream_t st) {
  CommitArgs a;
  a.t = *t; a.lo_stride = c->p.max_depth + 2;
  a.B = c->B; a.N = c->p.budget; a.max_depth = c->p.max_depth; a.layers_run = c->layers_run;
  a.n_kv_heads = c->p.n_kv_heads; a.head_dim = c->p.head_dim;
  a.accept_len = accept_len; a.accept_nodes = accept_nodes; a.next_tok = next_tok;
  a.k_tree = static_cast<const uint4 *>(k_tree); a.v_tree = static_cast<const uint4 *>(v_tree);
  a.k_prefix = static_cast<uint4 *>(k_prefix); a.v_prefix = static_cast<uint4 *>(v_prefix);
  a.kv_start = kv_start; a.kv_limit = kv_limit; a.block_table = block_table; a.n_blocks = n_blocks; a.bt_stride = bt_stride;
  a.kv_tokens = kv_tokens; a.stride_t = stride_t; a.stride_h = stride_h;
  a.prefix_len = prefix_len; a.root_tok = root_tok; a.counters = counters; a.status = c->d_status;
  {
    LaunchTimer lt(c, TALON_K_COMMIT, st);
    launch_kernel(c, commit_gather_kernel, dim3(c->p.max_depth + 1, c->B), dim3(256), 0, st, a);
    launch_kernel(c, commit_update_kernel, dim3((c->B + 127) / 128), dim3(128), 0, st, a);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 2;
  return TALON_OK;
}

}  // namespace talon

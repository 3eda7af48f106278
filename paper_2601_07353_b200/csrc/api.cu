// C ABI of libtalon: argument checks, context life cycle, and the host-buffer step.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "talon_internal.cuh"

namespace talon {
talon_status expand_setup(talon_ctx *c);
talon_status attention_mma_setup();
talon_status attention_tc_setup();
}  // namespace talon

// Device staging for talon_step_host.
struct HostStage {
  int batch = 0;
  int64_t prefix_tokens = 0;
  float *draft = nullptr, *target = nullptr;
  void *q = nullptr, *kp = nullptr, *vp = nullptr, *kt = nullptr, *vt = nullptr, *out = nullptr;
  int32_t *root = nullptr, *plen = nullptr;
  int64_t *kv_start = nullptr;
  talon_tree tree{};
  int32_t *accept_len = nullptr, *accept_nodes = nullptr, *bonus = nullptr;
  int64_t *h_kv_start = nullptr;   // pinned host scratch
};

#define TALON_CUDA_OK(expr)                                                              \
  do {                                                                                   \
    cudaError_t e_ = (expr);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      std::fprintf(stderr, "talon: %s failed: %s\n", #expr, cudaGetErrorString(e_));     \
      return TALON_ERR_CUDA;                                                             \
    }                                                                                    \
  } while (0)

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static bool tree_complete(const talon_tree *t) {
  return t && t->n_nodes && t->token && t->parent && t->depth && t->position && t->layer_off && t->score &&
         t->mask;
}

static void free_stage(HostStage *s) {
  if (!s) return;
  cudaFree(s->draft); cudaFree(s->target); cudaFree(s->q); cudaFree(s->kp); cudaFree(s->vp);
  cudaFree(s->kt); cudaFree(s->vt); cudaFree(s->out); cudaFree(s->root); cudaFree(s->plen);
  cudaFree(s->kv_start);
  cudaFree(s->tree.n_nodes); cudaFree(s->tree.token); cudaFree(s->tree.parent); cudaFree(s->tree.depth);
  cudaFree(s->tree.position); cudaFree(s->tree.layer_off); cudaFree(s->tree.score); cudaFree(s->tree.mask);
  cudaFree(s->accept_len); cudaFree(s->accept_nodes); cudaFree(s->bonus);
  if (s->h_kv_start) cudaFreeHost(s->h_kv_start);
  delete s;
}

extern "C" {

const char *talon_status_string(talon_status s) {
  switch (s) {
    case TALON_OK: return "ok";
    case TALON_ERR_INVALID_ARG: return "invalid argument";
    case TALON_ERR_CAPACITY: return "capacity exceeded";
    case TALON_ERR_CUDA: return "CUDA runtime error";
    case TALON_ERR_TIMEOUT: return "device-side wait timed out";
    case TALON_ERR_NONFINITE: return "non-finite logits";
    case TALON_ERR_UNSUPPORTED: return "unsupported configuration";
  }
  return "unknown status";
}

talon_status talon_create(talon_ctx **out_ctx, const talon_params *p, int device) {
  if (!out_ctx || !p) return TALON_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  if (p->batch_max < 1 || p->batch_max > talon::MAX_BATCH) return TALON_ERR_INVALID_ARG;
  if (p->vocab < 2 || p->vocab >= (1 << 24)) return TALON_ERR_INVALID_ARG;
  if (p->budget < 2 || p->budget > talon::MAX_BUDGET) return TALON_ERR_INVALID_ARG;
  if (p->root_topk < 1 || p->root_topk > 128) return TALON_ERR_INVALID_ARG;
  if (p->cand_topk < 0 || p->cand_topk > 128) return TALON_ERR_INVALID_ARG;
  if (p->max_depth < 1 || p->max_depth > 126) return TALON_ERR_INVALID_ARG;
  if (p->init_layers < 0) return TALON_ERR_INVALID_ARG;
  if (!(p->mu > 0.0) || !(p->mu <= 1.0)) return TALON_ERR_INVALID_ARG;
  if (p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_q_heads % p->n_kv_heads) return TALON_ERR_INVALID_ARG;
  if (p->head_dim != 128) return TALON_ERR_UNSUPPORTED;

  int n_dev = 0;
  TALON_CUDA_OK(cudaGetDeviceCount(&n_dev));
  if (device < 0 || device >= n_dev) return TALON_ERR_INVALID_ARG;
  TALON_CUDA_OK(cudaSetDevice(device));
  cudaDeviceProp prop;
  TALON_CUDA_OK(cudaGetDeviceProperties(&prop, device));
  if (prop.major < 10) {
    std::fprintf(stderr, "talon: built for sm_100a, device reports sm_%d%d\n", prop.major, prop.minor);
    return TALON_ERR_UNSUPPORTED;
  }

  talon_ctx *c = new (std::nothrow) talon_ctx();
  if (!c) return TALON_ERR_CUDA;
  std::memset(c, 0, sizeof(*c));
  c->p = *p;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->W = (p->budget + 63) / 64;
  int k = p->cand_topk == 0 ? p->budget - 1 : p->cand_topk;
  if (k > p->budget - 1) k = p->budget - 1;      // a parent never places more than N-1 children
  if (k > p->vocab) k = p->vocab;
  if (k < 1) k = 1;
  c->k_cap = k;
  c->k_slots = k <= 32 ? 1 : (k <= 64 ? 2 : 4);
  c->key_stride = (k + 3) & ~3;
  c->log_mu = std::log(p->mu);
  {
    // Programmatic dependent launch: measured on B200 it gains about 3 % at batch 1 and loses
    // 3-10 % at batch 16, so by default it is used for small batches only (TALON_PDL=1 / 0 forces it).
    const char *mt = std::getenv("TALON_ATTN_MIN_TILES");
    c->attn_min_tiles = mt ? std::atoi(mt) : 2;
    if (c->attn_min_tiles < 1) c->attn_min_tiles = 1;
    const char *ms = std::getenv("TALON_EXPAND_MAX_SPLIT");
    c->expand_max_split = ms ? std::atoi(ms) : talon::FX_MAX_SPLITS - 1;
    if (c->expand_max_split < 1) c->expand_max_split = 1;
    if (c->expand_max_split > talon::FX_MAX_SPLITS - 1) c->expand_max_split = talon::FX_MAX_SPLITS - 1;
    const char *ac = std::getenv("TALON_ATTN_CLUSTER");
    c->attn_cluster = ac ? std::atoi(ac) : 1;
    for (int i = 0; i < 9; ++i) c->attn_cluster_ok[i] = -1;
    const char *cc = std::getenv("TALON_ATTN_CLUSTER_CAP");
    c->attn_cluster_cap = cc ? std::atoi(cc) : 32;
    const char *cr = std::getenv("TALON_ATTN_CLUSTER_MIN_ROWS");
    c->attn_cluster_min_rows = cr ? std::atoll(cr) : 8192;
    const char *fs = std::getenv("TALON_ATTN_SPLITS");
    c->attn_force_splits = fs ? std::atoi(fs) : 0;
    const char *ao = std::getenv("TALON_ARGMAX_OVERSPLIT");
    c->argmax_oversplit = ao ? std::atoi(ao) : 4;
    if (c->argmax_oversplit < 1) c->argmax_oversplit = 1;
    const char *e = std::getenv("TALON_PDL");
    c->pdl = !e ? -1 : (e[0] == '1' ? 1 : 0);
    const char *g = std::getenv("TALON_STEP_GRAPH");
    c->step_graph = (g && g[0] == '0') ? 0 : 1;
  }
  c->exp_grid = c->sm_count * talon::EXP_CTAS_PER_SM;
  c->rows_cap = p->batch_max * (p->budget - 1);
  if (c->rows_cap < p->batch_max * p->budget) c->rows_cap = p->batch_max * p->budget;
  c->items_cap = c->exp_grid + c->rows_cap;

  const size_t nrow = (size_t)p->batch_max * p->budget;
  bool ok = true;
  auto alloc = [&](void **ptr, size_t bytes) {
    if (ok && cudaMalloc(ptr, bytes ? bytes : 16) != cudaSuccess) ok = false;
  };
  alloc((void **)&c->d_status, sizeof(int));
  alloc((void **)&c->d_prefix_len, sizeof(int32_t) * p->batch_max);
  alloc((void **)&c->d_part_keys, sizeof(unsigned long long) * (size_t)c->items_cap * c->key_stride);
  alloc((void **)&c->d_part_ms, sizeof(float2) * (size_t)c->items_cap);
  alloc((void **)&c->d_row_keys, sizeof(unsigned long long) * (size_t)c->rows_cap * c->key_stride);
  alloc((void **)&c->d_row_lse, sizeof(double) * (size_t)c->rows_cap);
  alloc((void **)&c->d_row_score, sizeof(double) * (size_t)c->rows_cap * c->key_stride);
  alloc((void **)&c->d_row_count, sizeof(unsigned int) * (size_t)c->rows_cap);
  alloc((void **)&c->d_seq_count, sizeof(unsigned int) * (size_t)p->batch_max);
  alloc((void **)&c->d_argmax, sizeof(unsigned long long) * nrow);
  alloc((void **)&c->d_target_tok, sizeof(int32_t) * nrow);
  alloc((void **)&c->d_walk_count, sizeof(unsigned int) * (size_t)p->batch_max);
  alloc((void **)&c->d_samp_ms, sizeof(float2) * nrow * talon::EXP_MAX_SPLITS);
  c->attn_o_elems = talon::attention_workspace_elems(c, &c->attn_ml_elems);
  alloc((void **)&c->d_attn_o, sizeof(float) * c->attn_o_elems);
  alloc((void **)&c->d_attn_ml, sizeof(float2) * c->attn_ml_elems);
  if (ok) {
    ok = cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess &&
         cudaMemset(c->d_row_count, 0, sizeof(unsigned int) * (size_t)c->rows_cap) == cudaSuccess &&
         cudaMemset(c->d_argmax, 0, sizeof(unsigned long long) * nrow) == cudaSuccess &&
         cudaMemset(c->d_seq_count, 0, sizeof(unsigned int) * (size_t)p->batch_max) == cudaSuccess &&
         cudaMemset(c->d_walk_count, 0, sizeof(unsigned int) * (size_t)p->batch_max) == cudaSuccess &&
         cudaMemset(c->d_part_keys, 0, sizeof(unsigned long long) * (size_t)c->items_cap * c->key_stride) == cudaSuccess &&
         talon::expand_setup(c) == TALON_OK && talon::attention_mma_setup() == TALON_OK &&
         talon::attention_tc_setup() == TALON_OK &&
         (c->k_cap > 32 || talon::expand_fused_setup(c) == TALON_OK);
  }
  if (!ok) {
    std::fprintf(stderr, "talon: context creation failed: %s\n", cudaGetErrorString(cudaGetLastError()));
    talon_destroy(c);
    return TALON_ERR_CUDA;
  }
  *out_ctx = c;
  return TALON_OK;
}

talon_status talon_destroy(talon_ctx *c) {
  if (!c) return TALON_OK;
  cudaSetDevice(c->device);
  cudaFree(c->d_status); cudaFree(c->d_prefix_len); cudaFree(c->d_part_keys); cudaFree(c->d_part_ms);
  cudaFree(c->d_row_keys); cudaFree(c->d_row_lse); cudaFree(c->d_row_score); cudaFree(c->d_row_count); cudaFree(c->d_seq_count); cudaFree(c->d_argmax);
  cudaFree(c->d_target_tok); cudaFree(c->d_walk_count); cudaFree(c->d_samp_ms); cudaFree(c->d_attn_o); cudaFree(c->d_attn_ml);
  free_stage(c->stage);
  talon_timing_enable(c, 0, 0u);
  if (c->graphs) {
    for (int i = 0; i < talon::STEP_GRAPH_SLOTS; ++i)
      if (c->graphs[i].exec) cudaGraphExecDestroy(c->graphs[i].exec);
    delete[] c->graphs;
  }
  delete c;
  return TALON_OK;
}

talon_status talon_reset(talon_ctx *c, const talon_tree *t, const int32_t *root_tok, const int32_t *prefix_len,
                         int32_t B, void *stream) {
  if (!c || !tree_complete(t) || !root_tok || !prefix_len) return TALON_ERR_INVALID_ARG;
  if (B < 1) return TALON_ERR_INVALID_ARG;
  if (B > c->p.batch_max) return TALON_ERR_CAPACITY;
  c->B = B;
  c->layers_run = 0;
  return talon::launch_reset(c, t, root_tok, prefix_len, B, (cudaStream_t)stream);
}

talon_status talon_expand_layer(talon_ctx *c, const talon_tree *t, const float *logits, int64_t row_stride,
                                int32_t rows_per_seq, int32_t layout, void *stream) {
  if (!c || !tree_complete(t) || !logits) return TALON_ERR_INVALID_ARG;
  if (c->B < 1) return TALON_ERR_INVALID_ARG;                      // no reset yet
  if (layout != TALON_ROWS_BY_NODE && layout != TALON_ROWS_PACKED) return TALON_ERR_INVALID_ARG;
  if (row_stride < c->p.vocab || (row_stride & 3) || !aligned16(logits)) return TALON_ERR_INVALID_ARG;
  if (rows_per_seq < 1 || (layout == TALON_ROWS_BY_NODE && rows_per_seq < c->p.budget)) return TALON_ERR_INVALID_ARG;
  if (c->layers_run >= c->p.max_depth) return TALON_OK;            // depth stop: nothing to do
  talon_status s = talon::launch_expand(c, t, logits, row_stride, rows_per_seq, layout, (cudaStream_t)stream);
  if (s == TALON_OK) c->layers_run += 1;
  return s;
}

int32_t talon_layers_run(const talon_ctx *c) { return c ? c->layers_run : -1; }

talon_status talon_build_tree(talon_ctx *c, const talon_tree *t, uint8_t *dense_mask, void *stream) {
  if (!c || !tree_complete(t)) return TALON_ERR_INVALID_ARG;
  if (c->B < 1) return TALON_ERR_INVALID_ARG;
  return talon::launch_build(c, t, dense_mask, (cudaStream_t)stream);
}

talon_status talon_prune_tree(talon_ctx *c, const talon_tree *t, int32_t keep, void *stream) {
  if (!c || !tree_complete(t)) return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || keep < 1) return TALON_ERR_INVALID_ARG;
  return talon::launch_prune(c, t, keep, (cudaStream_t)stream);
}

talon_status talon_tree_attention(talon_ctx *c, const talon_tree *t, const void *q, const void *k_prefix,
                                  const void *v_prefix, const void *k_tree, const void *v_tree,
                                  const int64_t *kv_start, int64_t kv_tokens, int64_t kv_stride_t,
                                  int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale, void *out,
                                  void *stream) {
  if (!c || !tree_complete(t) || !q || !k_tree || !v_tree || !kv_start || !out) return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || max_prefix_len < 0 || kv_tokens < 0 || kv_tokens > 0x7FFFFFFFll) return TALON_ERR_INVALID_ARG;
  if (max_prefix_len > kv_tokens) return TALON_ERR_INVALID_ARG;
  if (max_prefix_len > 0 && (!k_prefix || !v_prefix)) return TALON_ERR_INVALID_ARG;
  if ((kv_stride_t & 7) || (kv_stride_h & 7) || kv_stride_t < 0 || kv_stride_h < 0) return TALON_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_prefix) || !aligned16(v_prefix) || !aligned16(k_tree) || !aligned16(v_tree) ||
      !aligned16(out))
    return TALON_ERR_INVALID_ARG;
  if (!(sm_scale == sm_scale)) return TALON_ERR_INVALID_ARG;
  return talon::launch_attention(c, t, q, k_prefix ? k_prefix : k_tree, v_prefix ? v_prefix : v_tree, k_tree,
                                 v_tree, kv_start, nullptr, 0, kv_tokens, kv_stride_t, kv_stride_h, max_prefix_len,
                                 sm_scale, out, (cudaStream_t)stream);
}

talon_status talon_tree_attention_paged(talon_ctx *c, const talon_tree *t, const void *q, const void *k_pages,
                                        const void *v_pages, const void *k_tree, const void *v_tree,
                                        const int32_t *block_table, int32_t table_stride, int64_t n_pages,
                                        int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len,
                                        float sm_scale, void *out, void *stream) {
  if (!c || !tree_complete(t) || !q || !k_tree || !v_tree || !block_table || !out) return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || max_prefix_len < 0 || n_pages < 0 || n_pages * TALON_PAGE_TOKENS > 0x7FFFFFFFll) return TALON_ERR_INVALID_ARG;
  if (table_stride < (max_prefix_len + TALON_PAGE_TOKENS - 1) / TALON_PAGE_TOKENS) return TALON_ERR_INVALID_ARG;
  if (max_prefix_len > 0 && (!k_pages || !v_pages || n_pages < 1)) return TALON_ERR_INVALID_ARG;
  if ((kv_stride_t & 7) || (kv_stride_h & 7) || kv_stride_t < 0 || kv_stride_h < 0) return TALON_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k_tree) || !aligned16(v_tree) ||
      !aligned16(out))
    return TALON_ERR_INVALID_ARG;
  if (!(sm_scale == sm_scale)) return TALON_ERR_INVALID_ARG;
  return talon::launch_attention(c, t, q, k_pages ? k_pages : k_tree, v_pages ? v_pages : v_tree, k_tree, v_tree,
                                 nullptr, block_table, table_stride, n_pages * TALON_PAGE_TOKENS, kv_stride_t,
                                 kv_stride_h, max_prefix_len, sm_scale, out, (cudaStream_t)stream);
}

// close_tree: the walk also does talon_build_tree's writes (used inside a whole step)
static talon_status accept_checked(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                                   int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes,
                                   int32_t *bonus_tok, void *stream, bool close_tree) {
  if (!c || !tree_complete(t) || !target_logits || !accept_len || !accept_nodes || !bonus_tok)
    return TALON_ERR_INVALID_ARG;
  if (c->B < 1) return TALON_ERR_INVALID_ARG;
  if (row_stride < c->p.vocab || (row_stride & 3) || !aligned16(target_logits)) return TALON_ERR_INVALID_ARG;
  return talon::launch_accept(c, t, target_logits, row_stride, target_tok, accept_len, accept_nodes, bonus_tok,
                              (cudaStream_t)stream, close_tree);
}

talon_status talon_accept(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                          int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                          void *stream) {
  return accept_checked(c, t, target_logits, row_stride, target_tok, accept_len, accept_nodes, bonus_tok, stream, false);
}

talon_status talon_close_and_accept(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                                    int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes,
                                    int32_t *bonus_tok, void *stream) {
  return accept_checked(c, t, target_logits, row_stride, target_tok, accept_len, accept_nodes, bonus_tok, stream, true);
}

talon_status talon_accept_sample(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                                 double temperature, const double *u_accept, const double *u_sample,
                                 int32_t *accept_len, int32_t *accept_nodes, int32_t *out_tok, void *stream) {
  if (!c || !tree_complete(t) || !target_logits || !u_accept || !u_sample || !accept_len || !accept_nodes || !out_tok)
    return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || !(temperature > 0.0) || !std::isfinite(temperature)) return TALON_ERR_INVALID_ARG;
  if (row_stride < c->p.vocab || (row_stride & 3) || !aligned16(target_logits)) return TALON_ERR_INVALID_ARG;
  return talon::launch_accept_sample(c, t, target_logits, row_stride, temperature, u_accept, u_sample, accept_len,
                                     accept_nodes, out_tok, (cudaStream_t)stream);
}

talon_status talon_commit(talon_ctx *c, const talon_tree *t, const int32_t *accept_len, const int32_t *accept_nodes,
                          const int32_t *next_tok, const void *k_tree, const void *v_tree, void *k_prefix,
                          void *v_prefix, const int64_t *kv_start, const int64_t *kv_limit, int64_t kv_tokens,
                          int64_t kv_stride_t, int64_t kv_stride_h, int32_t *prefix_len, int32_t *root_tok,
                          int64_t *counters, void *stream) {
  if (!c || !tree_complete(t) || !accept_len || !accept_nodes || !next_tok || !k_tree || !v_tree || !k_prefix ||
      !v_prefix || !kv_start || !prefix_len || !root_tok)
    return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || kv_tokens < 0 || kv_tokens > 0x7FFFFFFFll) return TALON_ERR_INVALID_ARG;
  if ((kv_stride_t & 7) || (kv_stride_h & 7) || kv_stride_t < 0 || kv_stride_h < 0) return TALON_ERR_INVALID_ARG;
  if (!aligned16(k_prefix) || !aligned16(v_prefix) || !aligned16(k_tree) || !aligned16(v_tree))
    return TALON_ERR_INVALID_ARG;
  return talon::launch_commit(c, t, accept_len, accept_nodes, next_tok, k_tree, v_tree, k_prefix, v_prefix, kv_start,
                              kv_limit, nullptr, 0, nullptr, kv_tokens, kv_stride_t, kv_stride_h, prefix_len, root_tok,
                              counters, (cudaStream_t)stream);
}

talon_status talon_commit_paged(talon_ctx *c, const talon_tree *t, const int32_t *accept_len,
                                const int32_t *accept_nodes, const int32_t *next_tok, const void *k_tree,
                                const void *v_tree, void *k_pages, void *v_pages, const int32_t *block_table,
                                int32_t table_stride, const int32_t *n_blocks, int64_t n_pages, int64_t kv_stride_t,
                                int64_t kv_stride_h, int32_t *prefix_len, int32_t *root_tok, int64_t *counters,
                                void *stream) {
  if (!c || !tree_complete(t) || !accept_len || !accept_nodes || !next_tok || !k_tree || !v_tree || !k_pages ||
      !v_pages || !block_table || !n_blocks || !prefix_len || !root_tok)
    return TALON_ERR_INVALID_ARG;
  if (c->B < 1 || n_pages < 1 || n_pages * TALON_PAGE_TOKENS > 0x7FFFFFFFll || table_stride < 1) return TALON_ERR_INVALID_ARG;
  if ((kv_stride_t & 7) || (kv_stride_h & 7) || kv_stride_t < 0 || kv_stride_h < 0) return TALON_ERR_INVALID_ARG;
  if (!aligned16(k_pages) || !aligned16(v_pages) || !aligned16(k_tree) || !aligned16(v_tree)) return TALON_ERR_INVALID_ARG;
  return talon::launch_commit(c, t, accept_len, accept_nodes, next_tok, k_tree, v_tree, k_pages, v_pages, nullptr, nullptr,
                              block_table, table_stride, n_blocks, n_pages * TALON_PAGE_TOKENS, kv_stride_t, kv_stride_h,
                              prefix_len, root_tok, counters, (cudaStream_t)stream);
}

static talon_status step_enqueue(talon_ctx *c, const talon_tree *t, int32_t B, const int32_t *root_tok,
                                 const int32_t *prefix_len, const float *draft_logits, int64_t draft_row_stride,
                                 int32_t n_layers, const void *q, const void *k_prefix, const void *v_prefix,
                                 const void *k_tree, const void *v_tree, const int64_t *kv_start, int64_t kv_tokens,
                                 int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale,
                                 void *out, const float *target_logits, int64_t target_row_stride,
                                 int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                                 void *stream);

talon_status talon_loop(talon_ctx *c, const talon_tree *t, int32_t B, int32_t n_steps, int32_t *root_tok,
                        int32_t *prefix_len, const float *draft_logits, int64_t draft_row_stride,
                        int64_t draft_step_stride, int32_t n_layers, const void *q, int64_t q_step_stride,
                        void *k_prefix, void *v_prefix, const void *k_tree, const void *v_tree,
                        int64_t kv_tree_step_stride, const int64_t *kv_start, const int64_t *kv_limit, int64_t kv_tokens,
                        int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale, void *out,
                        const float *target_logits, int64_t target_row_stride, int64_t target_step_stride,
                        int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                        int64_t result_step_stride, int64_t *counters, void *stream) {
  if (!c || n_steps < 1 || !root_tok || !prefix_len || !counters) return TALON_ERR_INVALID_ARG;
  if (n_layers < 0 || n_layers > c->p.max_depth) return TALON_ERR_INVALID_ARG;
  if (draft_step_stride < 0 || q_step_stride < 0 || kv_tree_step_stride < 0 || target_step_stride < 0 ||
      result_step_stride < 0 || (q_step_stride & 7) || (kv_tree_step_stride & 7) || (draft_step_stride & 3) ||
      (target_step_stride & 3))
    return TALON_ERR_INVALID_ARG;
  const char *qb = static_cast<const char *>(q), *ktb = static_cast<const char *>(k_tree), *vtb = static_cast<const char *>(v_tree);
  for (int s = 0; s < n_steps; ++s) {
    // step s reads its own slice of the stand-ins for the two model forwards; the tree, the cache,
    // the prefix lengths and the roots are the state the steps hand on to one another on the device
    const void *qs = qb + 2 * q_step_stride * s, *kts = ktb + 2 * kv_tree_step_stride * s, *vts = vtb + 2 * kv_tree_step_stride * s;
    int32_t *al = accept_len + result_step_stride * s, *an = accept_nodes + result_step_stride * (c->p.max_depth + 1) * s;
    int32_t *bt = bonus_tok + result_step_stride * s;
    talon_status r = step_enqueue(c, t, B, root_tok, prefix_len, draft_logits + draft_step_stride * s, draft_row_stride,
                                  n_layers, qs, k_prefix, v_prefix, kts, vts, kv_start, kv_tokens, kv_stride_t, kv_stride_h,
                                  max_prefix_len, sm_scale, out, target_logits + target_step_stride * s, target_row_stride,
                                  target_tok, al, an, bt, stream);
    if (r == TALON_OK)
      r = talon_commit(c, t, al, an, bt, kts, vts, k_prefix, v_prefix, kv_start, kv_limit, kv_tokens, kv_stride_t,
                       kv_stride_h, prefix_len, root_tok, counters, stream);
    if (r != TALON_OK) return r;
  }
  return TALON_OK;
}

talon_status talon_loop_metrics(const int64_t *counters, int32_t B, double cost_ratio, double *delta, double *tau,
                                double *speedup) {
  if (!counters || B < 1 || !delta || !tau || !speedup || !(cost_ratio >= 0.0)) return TALON_ERR_INVALID_ARG;
  long long n_p = 0, n_q = 0, len = 0;
  for (int b = 0; b < B; ++b) { n_p += counters[3 * b]; n_q += counters[3 * b + 1]; len += counters[3 * b + 2]; }
  if (n_p <= 0) return TALON_ERR_INVALID_ARG;
  *delta = (double)n_q / (double)n_p;                  // Eq. 6: draft passes per verification pass
  *tau = (double)len / (double)n_p;                    // mean accepted tokens per verification pass
  *speedup = *tau / (1.0 + cost_ratio * *delta);       // Eq. 7
  return TALON_OK;
}

talon_status talon_poll_status(talon_ctx *c, void *stream) {
  if (!c) return TALON_ERR_INVALID_ARG;
  int word = 0;
  TALON_CUDA_OK(cudaMemcpyAsync(&word, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  TALON_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  if (word & talon::STATUS_TIMEOUT) return TALON_ERR_TIMEOUT;
  if (word & talon::STATUS_CAPACITY) return TALON_ERR_CAPACITY;
  if (word & talon::STATUS_NONFINITE) return TALON_ERR_NONFINITE;
  return TALON_OK;
}

int64_t talon_launch_count(const talon_ctx *c) { return c ? c->launches : -1; }

const char *talon_kernel_name(int32_t k) {
  switch (k) {
    case TALON_K_RESET: return "reset";
    case TALON_K_EXPAND_ROWS: return "expand_rows";
    case TALON_K_SELECT: return "select_layer";
    case TALON_K_BUILD: return "build_tree";
    case TALON_K_ATTENTION: return "tree_attention";
    case TALON_K_COMBINE: return "attention_combine";
    case TALON_K_ARGMAX: return "target_argmax";
    case TALON_K_WALK: return "accept_walk";
    case TALON_K_ROWSTATS: return "target_softmax_stats";
    case TALON_K_SAMPLE: return "accept_sample";
    case TALON_K_COMMIT: return "commit";
  }
  return "unknown";
}

talon_status talon_timing_enable(talon_ctx *c, int32_t max_launches, uint32_t kernel_mask) {
  if (!c || max_launches < 0) return TALON_ERR_INVALID_ARG;
  cudaSetDevice(c->device);
  if (c->ev) {
    cudaDeviceSynchronize();
    for (int i = 0; i < 2 * c->ev_cap; ++i) cudaEventDestroy(c->ev[i]);
    delete[] c->ev;
    delete[] c->ev_kernel;
    c->ev = nullptr; c->ev_kernel = nullptr; c->ev_cap = c->ev_used = 0;
  }
  if (max_launches == 0) return TALON_OK;
  c->ev = new (std::nothrow) cudaEvent_t[2 * (size_t)max_launches];
  c->ev_kernel = new (std::nothrow) int[max_launches];
  if (!c->ev || !c->ev_kernel) return TALON_ERR_CUDA;
  for (int i = 0; i < 2 * max_launches; ++i) TALON_CUDA_OK(cudaEventCreate(&c->ev[i]));
  c->ev_cap = max_launches;
  c->ev_used = 0;
  c->ev_paused = 0;
  c->ev_mask = kernel_mask ? kernel_mask : 0xFFFFFFFFu;
  return TALON_OK;
}

talon_status talon_timing_pause(talon_ctx *c, int32_t paused) {
  if (!c) return TALON_ERR_INVALID_ARG;
  c->ev_paused = paused ? 1 : 0;
  return TALON_OK;
}

talon_status talon_timing_read(talon_ctx *c, void *stream, double *ms, int64_t *launches) {
  if (!c || !ms || !launches) return TALON_ERR_INVALID_ARG;
  for (int k = 0; k < TALON_N_KERNELS; ++k) { ms[k] = 0.0; launches[k] = 0; }
  if (!c->ev) return TALON_OK;
  TALON_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
  for (int i = 0; i < c->ev_used; ++i) {
    float t = 0.f;
    TALON_CUDA_OK(cudaEventElapsedTime(&t, c->ev[2 * i], c->ev[2 * i + 1]));
    const int k = c->ev_kernel[i];
    if (k >= 0 && k < TALON_N_KERNELS) { ms[k] += t; launches[k] += 1; }
  }
  c->ev_used = 0;
  return TALON_OK;
}

// The launches of one step, in order, on `stream`.
static talon_status step_enqueue(talon_ctx *c, const talon_tree *t, int32_t B, const int32_t *root_tok,
                                 const int32_t *prefix_len, const float *draft_logits, int64_t draft_row_stride,
                                 int32_t n_layers, const void *q, const void *k_prefix, const void *v_prefix,
                                 const void *k_tree, const void *v_tree, const int64_t *kv_start, int64_t kv_tokens,
                                 int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale,
                                 void *out, const float *target_logits, int64_t target_row_stride,
                                 int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok,
                                 void *stream) {
  talon_status r = talon_reset(c, t, root_tok, prefix_len, B, stream);
  for (int d = 0; r == TALON_OK && d < n_layers; ++d)
    r = talon_expand_layer(c, t, draft_logits, draft_row_stride, c->p.budget, TALON_ROWS_BY_NODE, stream);
  // (no separate closing launch: the attention needs only sizes and mask rows, and the accept walk
  // writes positions and sentinel slots before it walks)
  if (r == TALON_OK)
    r = talon_tree_attention(c, t, q, k_prefix, v_prefix, k_tree, v_tree, kv_start, kv_tokens, kv_stride_t, kv_stride_h,
                             max_prefix_len, sm_scale, out, stream);
  if (r == TALON_OK)
    r = accept_checked(c, t, target_logits, target_row_stride, target_tok, accept_len, accept_nodes, bonus_tok,
                       stream, true);
  return r;
}

talon_status talon_step(talon_ctx *c, const talon_tree *t, int32_t B, const int32_t *root_tok,
                        const int32_t *prefix_len, const float *draft_logits, int64_t draft_row_stride,
                        int32_t n_layers, const void *q, const void *k_prefix, const void *v_prefix,
                        const void *k_tree, const void *v_tree, const int64_t *kv_start, int64_t kv_tokens,
                        int64_t kv_stride_t, int64_t kv_stride_h, int32_t max_prefix_len, float sm_scale, void *out,
                        const float *target_logits, int64_t target_row_stride, int32_t *target_tok,
                        int32_t *accept_len, int32_t *accept_nodes, int32_t *bonus_tok, void *stream) {
  if (!c) return TALON_ERR_INVALID_ARG;
  if (n_layers < 0 || n_layers > c->p.max_depth) return TALON_ERR_INVALID_ARG;
#define TALON_STEP_ARGS                                                                                              \
  c, t, B, root_tok, prefix_len, draft_logits, draft_row_stride, n_layers, q, k_prefix, v_prefix, k_tree, v_tree,    \
      kv_start, kv_tokens, kv_stride_t, kv_stride_h, max_prefix_len, sm_scale, out, target_logits, target_row_stride, \
      target_tok, accept_len, accept_nodes, bonus_tok, stream
  cudaStream_t st = (cudaStream_t)stream;
  // A step is a chain of small dependent kernels, so a caller that repeats it pays mostly for
  // launches.  From the second call with the very same arguments the launches are captured once
  // into a CUDA graph and replayed from then on: the same kernels on the same memory, one
  // submission.  Not on the legacy default stream (it cannot be captured), not while the stream is
  // already being captured by the caller, and not while launches are being timed with events.
  const bool timing = c->ev && !c->ev_paused;
  if (!c->step_graph || !t || st == nullptr || st == cudaStreamLegacy || timing) return step_enqueue(TALON_STEP_ARGS);
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) {
    cudaGetLastError();
    return step_enqueue(TALON_STEP_ARGS);
  }
  if (!c->graphs) {
    c->graphs = new (std::nothrow) talon::StepGraph[talon::STEP_GRAPH_SLOTS];
    if (!c->graphs) return step_enqueue(TALON_STEP_ARGS);
    std::memset(c->graphs, 0, sizeof(talon::StepGraph) * talon::STEP_GRAPH_SLOTS);
  }
  unsigned long long key[talon::STEP_GRAPH_WORDS];
  std::memset(key, 0, sizeof(key));
  {
    int n = 0;
    auto put = [&](const void *p) { key[n++] = (unsigned long long)reinterpret_cast<uintptr_t>(p); };
    auto puti = [&](long long v) { key[n++] = (unsigned long long)v; };
    put(t->n_nodes); put(t->token); put(t->parent); put(t->depth); put(t->position); put(t->layer_off);
    put(t->score); put(t->mask);
    puti(B); put(root_tok); put(prefix_len); put(draft_logits); puti(draft_row_stride); puti(n_layers);
    put(q); put(k_prefix); put(v_prefix); put(k_tree); put(v_tree); put(kv_start); puti(kv_tokens);
    puti(kv_stride_t); puti(kv_stride_h); puti(max_prefix_len);
    unsigned int bits; std::memcpy(&bits, &sm_scale, 4); puti(bits);
    put(out); put(target_logits); puti(target_row_stride); put(target_tok); put(accept_len); put(accept_nodes);
    put(bonus_tok); put(stream);
  }
  talon::StepGraph *hit = nullptr, *victim = &c->graphs[0];
  for (int i = 0; i < talon::STEP_GRAPH_SLOTS; ++i) {
    talon::StepGraph *g = &c->graphs[i];
    if (g->used && std::memcmp(g->args, key, sizeof(key)) == 0) { hit = g; break; }
    if (!g->used || (victim->used && g->last_use < victim->last_use)) victim = g;
  }
  c->step_tick += 1;
  if (!hit) {                      // first sighting: remember the arguments, run the plain way
    if (victim->exec) cudaGraphExecDestroy(victim->exec);
    std::memset(victim, 0, sizeof(*victim));
    std::memcpy(victim->args, key, sizeof(key));
    victim->used = true;
    victim->last_use = c->step_tick;
    return step_enqueue(TALON_STEP_ARGS);
  }
  hit->last_use = c->step_tick;
  if (!hit->exec) {                // second sighting: capture
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      cudaGetLastError();
      c->step_graph = 0;           // this stream or driver cannot capture: stop trying
      return step_enqueue(TALON_STEP_ARGS);
    }
    const long long before = c->launches;
    const talon_status r = step_enqueue(TALON_STEP_ARGS);
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(st, &graph);
    cudaGraphExec_t exec = nullptr;
    if (r == TALON_OK && e == cudaSuccess && graph && cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
      hit->exec = exec;
      hit->launches = c->launches - before;
      hit->layers_run = c->layers_run;
      c->launches = before;        // nothing has run yet: the replay below counts
    } else {
      // nothing ran: clean up and do the step the plain way, which also reports a bad argument
      cudaGetLastError();
      c->launches = before;
      hit->used = false;
      if (graph) cudaGraphDestroy(graph);
      if (r == TALON_OK) c->step_graph = 0;      // the capture itself failed: stop trying
      return step_enqueue(TALON_STEP_ARGS);
    }
    cudaGraphDestroy(graph);
  }
  if (cudaGraphLaunch(hit->exec, st) != cudaSuccess) return TALON_ERR_CUDA;
  c->B = B;
  c->layers_run = hit->layers_run;
  c->launches += hit->launches;
  return TALON_OK;
#undef TALON_STEP_ARGS
}

talon_status talon_step_host(talon_ctx *c, int32_t B, const int32_t *root_tok, const int32_t *prefix_len,
                             const float *draft_logits, const float *target_logits, const void *q,
                             const void *k_prefix, const void *v_prefix, const void *k_tree, const void *v_tree,
                             float sm_scale, void *out_attn, int32_t *n_nodes, int32_t *token, int32_t *parent,
                             int32_t *depth, int32_t *position, int32_t *accept_len, int32_t *accept_nodes,
                             int32_t *bonus_tok, void *stream) {
  if (!c || !root_tok || !prefix_len || !draft_logits || !target_logits || !q || !k_tree || !v_tree ||
      !accept_len || !accept_nodes || !bonus_tok)
    return TALON_ERR_INVALID_ARG;
  if (B < 1) return TALON_ERR_INVALID_ARG;
  if (B > c->p.batch_max) return TALON_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  const talon_params &p = c->p;
  const size_t N = p.budget, V = p.vocab, Dh = p.head_dim;
  if (V & 3) return TALON_ERR_UNSUPPORTED;        // dense [B,N,V] rows must stay 16-byte aligned

  int64_t tokens = 0;
  int max_len = 0;
  for (int b = 0; b < B; ++b) {
    if (prefix_len[b] < 0) return TALON_ERR_INVALID_ARG;
    tokens += prefix_len[b];
    if (prefix_len[b] > max_len) max_len = prefix_len[b];
  }
  if (tokens > 0 && (!k_prefix || !v_prefix)) return TALON_ERR_INVALID_ARG;
  TALON_CUDA_OK(cudaSetDevice(c->device));

  HostStage *s = c->stage;
  if (!s || s->prefix_tokens < tokens) {
    TALON_CUDA_OK(cudaStreamSynchronize(st));
    free_stage(s);
    c->stage = nullptr;
    s = new (std::nothrow) HostStage();
    if (!s) return TALON_ERR_CUDA;
    c->stage = s;
    const size_t bm = p.batch_max, W = c->W;
    s->batch = p.batch_max;
    s->prefix_tokens = tokens > 0 ? tokens : 1;
    TALON_CUDA_OK(cudaMalloc((void **)&s->draft, bm * N * V * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->target, bm * N * V * 4));
    TALON_CUDA_OK(cudaMalloc(&s->q, bm * N * p.n_q_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc(&s->out, bm * N * p.n_q_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc(&s->kp, (size_t)s->prefix_tokens * p.n_kv_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc(&s->vp, (size_t)s->prefix_tokens * p.n_kv_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc(&s->kt, bm * N * p.n_kv_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc(&s->vt, bm * N * p.n_kv_heads * Dh * 2));
    TALON_CUDA_OK(cudaMalloc((void **)&s->root, bm * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->plen, bm * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->kv_start, bm * 8));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.n_nodes, bm * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.token, bm * N * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.parent, bm * N * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.depth, bm * N * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.position, bm * N * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.layer_off, bm * (p.max_depth + 2) * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.score, bm * N * 8));
    TALON_CUDA_OK(cudaMalloc((void **)&s->tree.mask, bm * N * W * 8));
    TALON_CUDA_OK(cudaMalloc((void **)&s->accept_len, bm * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->accept_nodes, bm * (p.max_depth + 1) * 4));
    TALON_CUDA_OK(cudaMalloc((void **)&s->bonus, bm * 4));
    TALON_CUDA_OK(cudaMallocHost((void **)&s->h_kv_start, bm * 8));
  }

  {
    int64_t run = 0;
    for (int b = 0; b < B; ++b) { s->h_kv_start[b] = run; run += prefix_len[b]; }
  }
  const size_t rows = (size_t)B * N;
  const size_t kvrow = (size_t)p.n_kv_heads * Dh * 2;
#define H2D(dst, src, bytes) TALON_CUDA_OK(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st))
#define D2H(dst, src, bytes) TALON_CUDA_OK(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st))
  H2D(s->root, root_tok, (size_t)B * 4);
  H2D(s->plen, prefix_len, (size_t)B * 4);
  H2D(s->kv_start, s->h_kv_start, (size_t)B * 8);
  H2D(s->draft, draft_logits, rows * V * 4);
  H2D(s->target, target_logits, rows * V * 4);
  H2D(s->q, q, rows * p.n_q_heads * Dh * 2);
  if (tokens > 0) {
    H2D(s->kp, k_prefix, (size_t)tokens * kvrow);
    H2D(s->vp, v_prefix, (size_t)tokens * kvrow);
  }
  H2D(s->kt, k_tree, rows * kvrow);
  H2D(s->vt, v_tree, rows * kvrow);

  talon_status r = talon_reset(c, &s->tree, s->root, s->plen, B, stream);
  for (int d = 0; r == TALON_OK && d < p.max_depth; ++d)
    r = talon_expand_layer(c, &s->tree, s->draft, (int64_t)V, (int32_t)N, TALON_ROWS_BY_NODE, stream);
  if (r == TALON_OK) r = talon_build_tree(c, &s->tree, nullptr, stream);
  if (r == TALON_OK)
    r = talon_tree_attention(c, &s->tree, s->q, s->kp, s->vp, s->kt, s->vt, s->kv_start, s->prefix_tokens,
                             (int64_t)p.n_kv_heads * Dh, (int64_t)Dh, max_len, sm_scale, s->out, stream);
  if (r == TALON_OK)
    r = talon_accept(c, &s->tree, s->target, (int64_t)V, nullptr, s->accept_len, s->accept_nodes, s->bonus, stream);
  if (r != TALON_OK) return r;

  if (out_attn) D2H(out_attn, s->out, rows * p.n_q_heads * Dh * 2);
  if (n_nodes) D2H(n_nodes, s->tree.n_nodes, (size_t)B * 4);
  if (token) D2H(token, s->tree.token, rows * 4);
  if (parent) D2H(parent, s->tree.parent, rows * 4);
  if (depth) D2H(depth, s->tree.depth, rows * 4);
  if (position) D2H(position, s->tree.position, rows * 4);
  D2H(accept_len, s->accept_len, (size_t)B * 4);
  D2H(accept_nodes, s->accept_nodes, (size_t)B * (p.max_depth + 1) * 4);
  D2H(bonus_tok, s->bonus, (size_t)B * 4);
#undef H2D
#undef D2H
  return talon_poll_status(c, stream);
}

}  // extern "C"

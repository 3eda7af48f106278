// Greedy verification (Appendix B of the paper, steps 1-2 at temperature 0) for sm_100a.
//
//   target_argmax_kernel : t_i = argmax_w target_logits[b, i, w] for every tree node, one
//                          streaming pass with 128-bit loads.  Rows are cut into chunks so
//                          that a single sequence still fills the GPU; chunks meet in a
//                          64-bit atomicMax on a packed (logit, lowest-token-first) key.
//   accept_walk_kernel   : decodes the keys, then walks from the root along the child whose
//                          token equals the target's choice until none does.
// When every CTA of the argmax kernel has one chunk at most (small batches, where a launch costs
// as much as the work), the CTA that brings a sequence's last chunk does that sequence's walk
// itself and the second kernel is not launched.  Inside a whole step the walk's warp also closes
// the tree (positions, sentinel slots, the unused tail of the layer offsets), which saves the
// launch of the closing kernel: nothing between the last expansion layer and the walk reads those.
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

constexpr unsigned FULL = 0xFFFFFFFFu;

struct ArgmaxArgs {
  const float *logits;
  int64_t row_stride;
  const int32_t *n_nodes;
  int B, N, V;
  int splits, chunk_len;
  unsigned long long *best;   // [B*N], zero on entry
  int *status;
};

struct WalkArgs {
  talon_tree t;
  int lo_stride;
  int B, N, max_depth;
  unsigned long long *best;
  int32_t *target_tok;      // [B*N] workspace or caller buffer
  int32_t *accept_len, *accept_nodes, *bonus_tok;
  // closing pass folded into the walk (close_tree != 0)
  int close_tree, W, layers_run;
  const int32_t *prefix_len;
};

// The closing pass over the node slots of sequence b (what build_tree_kernel writes there):
// positions of the tree's nodes, sentinels in the unused slots.  The walk reads none of it.
__device__ __forceinline__ void close_slots(const WalkArgs &a, int b, int first, int step) {
  const size_t nb = (size_t)b * a.N;
  const int n = a.t.n_nodes[b];
  const int L = a.prefix_len[b];
  for (int i = first; i < a.N; i += step) {
    if (i < n) {
      a.t.position[nb + i] = L + a.t.depth[nb + i];
    } else {
      a.t.token[nb + i] = -1;
      a.t.parent[nb + i] = -1;
      a.t.depth[nb + i] = -1;
      a.t.position[nb + i] = -1;
      a.t.score[nb + i] = -CUDART_INF;
      for (int w = 0; w < a.W; ++w) a.t.mask[(nb + i) * a.W + w] = ((i >> 6) == w) ? (1ull << (i & 63)) : 0ull;
    }
  }
}

// One warp decodes the keys of sequence b and walks its tree.
__device__ __forceinline__ void accept_walk(const WalkArgs &a, int b, int lane) {
  const size_t nb = (size_t)b * a.N;
  const int n = a.t.n_nodes[b];
  if (a.close_tree) {
    // layers that were never launched: their offsets close at the tree's size (the walk reads them)
    for (int i = a.layers_run + 2 + lane; i < a.lo_stride; i += 32) a.t.layer_off[b * a.lo_stride + i] = n;
    __syncwarp();
  }
  for (int i = lane; i < a.N; i += 32) {
    const unsigned long long k = __ldcg(&a.best[nb + i]);
    a.best[nb + i] = 0ull;                                  // leave the workspace clean
    a.target_tok[nb + i] = (i < n && k != 0ull) ? (int32_t)key_tok(k) : -1;
  }
  __syncwarp();
  int cur = 0, len = 0;
  if (lane == 0) a.accept_nodes[(size_t)b * (a.max_depth + 1)] = 0;
  for (int d = 0; d < a.max_depth; ++d) {
    const int want = a.target_tok[nb + cur];
    const int lo = a.t.layer_off[b * a.lo_stride + d + 1];
    const int hi = a.t.layer_off[b * a.lo_stride + d + 2];
    int found = -1;
    for (int c0 = lo; c0 < hi; c0 += 32) {
      const int c = c0 + lane;
      const bool hit = c < hi && a.t.parent[nb + c] == cur && a.t.token[nb + c] == want;
      const unsigned m = __ballot_sync(FULL, hit);
      if (m) { found = c0 + __ffs(m) - 1; break; }
    }
    if (found < 0) break;
    cur = found;
    ++len;
    if (lane == 0) a.accept_nodes[(size_t)b * (a.max_depth + 1) + len] = cur;
  }
  for (int i = len + 1 + lane; i <= a.max_depth; i += 32) a.accept_nodes[(size_t)b * (a.max_depth + 1) + i] = -1;
  if (lane == 0) {
    a.accept_len[b] = len;
    a.bonus_tok[b] = a.target_tok[nb + cur];
  }
}

__global__ void __launch_bounds__(EXP_THREADS)
target_argmax_kernel(ArgmaxArgs a, WalkArgs wa, unsigned int *seq_done, int fold) {
  __shared__ unsigned long long s_key[EXP_WARPS];
  __shared__ int s_walk;
  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_items = a.B * a.N * a.splits;
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int row = item / a.splits, chunk = item - row * a.splits;
    const int b = row / a.N, i = row - b * a.N;
    if (i >= a.n_nodes[b]) continue;                       // unused node slot (CTA-uniform)
    const float *rowp = a.logits + (int64_t)row * a.row_stride;
    const int start = chunk * a.chunk_len;
    const int end = min(a.V, start + a.chunk_len);
    float bestv = -CUDART_INF_F;
    uint32_t besti = 0xFFFFFFFFu;
    bool bad = false;
    // the next tile is requested before the current one is worked on: a chunk of a few tiles is a
    // chain of DRAM round trips otherwise
    float nx[EXP_UNROLL][EXP_VEC];
    auto load = [&](int base) {
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u) {
        const int idx = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC;
        if (idx + EXP_VEC <= end) {
          const float4 x = __ldcs(reinterpret_cast<const float4 *>(rowp + idx));
          nx[u][0] = x.x; nx[u][1] = x.y; nx[u][2] = x.z; nx[u][3] = x.w;
        } else {
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) nx[u][e] = (idx + e < end) ? __ldcs(rowp + idx + e) : -CUDART_INF_F;
        }
      }
    };
    load(start);
    for (int base = start; base < end; base += EXP_TILE) {
      float v[EXP_UNROLL][EXP_VEC];
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) v[u][e] = nx[u][e];
      if (base + EXP_TILE < end) load(base + EXP_TILE);
      // the tile's maximum first (one max per element); only a tile that raises the thread's
      // maximum, or the thread's first tile, is searched for where that maximum sits
      float bm = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) {
          bad |= (v[u][e] != v[u][e]);
          bm = fmaxf(bm, v[u][e]);
        }
      if (bm > bestv || besti == 0xFFFFFFFFu) {
        // strict > keeps the earlier tile among equal maxima; inside the tile the first match in
        // (u, e) order is the thread's lowest index; a tile of -inf only still claims its first slot
        uint32_t first = 0xFFFFFFFFu;
#pragma unroll
        for (int u = EXP_UNROLL - 1; u >= 0; --u)
#pragma unroll
          for (int e = EXP_VEC - 1; e >= 0; --e) {
            const int idx = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e;
            if (idx < end && v[u][e] == bm) first = (uint32_t)idx;
          }
        if (first != 0xFFFFFFFFu) { bestv = bm; besti = first; }
      }
    }
    unsigned long long key = (besti == 0xFFFFFFFFu) ? 0ull : cand_key(bestv, besti);
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(FULL, key, o);
      key = other > key ? other : key;
    }
    if (__any_sync(FULL, bad) && lane == 0) atomicOr(a.status, STATUS_NONFINITE);
    __syncthreads();
    if (lane == 0) s_key[warp] = key;
    __syncthreads();
    if (tid == 0) {
      unsigned long long k = s_key[0];
      for (int w = 1; w < EXP_WARPS; ++w) k = s_key[w] > k ? s_key[w] : k;
      if (a.splits == 1) a.best[row] = k;
      else atomicMax(&a.best[row], k);
      if (fold) {
        // count the chunk in; whoever brings the sequence's last one walks its tree
        __threadfence();
        const unsigned target = (unsigned)(a.n_nodes[b] * a.splits);
        const unsigned prev = atomicAdd(&seq_done[b], 1u);
        s_walk = (prev + 1u == target) ? b : -1;
        if (prev + 1u == target) { seq_done[b] = 0u; __threadfence(); }
      }
    }
    if (fold) {
      __syncthreads();
      if (s_walk >= 0) {
        if (warp == 0) accept_walk(wa, s_walk, lane);
        else if (wa.close_tree) close_slots(wa, s_walk, tid - 32, EXP_THREADS - 32);   // beside the walk
      }
    }
  }
}

// one warp per sequence
__global__ void accept_walk_kernel(WalkArgs a) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= a.B) return;
  // the closing pass needs each node's depth: the loads are issued before the walk (a chain of
  // dependent L2 trips) and their results are used after it
  constexpr int PER = (MAX_BUDGET + 31) / 32;
  int dep[PER];
  int L = 0, n = 0;
  if (a.close_tree) {
    n = a.t.n_nodes[b];
    L = a.prefix_len[b];
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int i = lane + 32 * k;
      dep[k] = (i < n) ? a.t.depth[(size_t)b * a.N + i] : -1;
    }
  }
  accept_walk(a, b, lane);
  if (a.close_tree) {
    const size_t nb = (size_t)b * a.N;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int i = lane + 32 * k;
      if (i >= a.N) continue;
      if (i < n) {
        a.t.position[nb + i] = L + dep[k];
      } else {
        a.t.token[nb + i] = -1;
        a.t.parent[nb + i] = -1;
        a.t.depth[nb + i] = -1;
        a.t.position[nb + i] = -1;
        a.t.score[nb + i] = -CUDART_INF;
        for (int w = 0; w < a.W; ++w) a.t.mask[(nb + i) * a.W + w] = ((i >> 6) == w) ? (1ull << (i & 63)) : 0ull;
      }
    }
  }
}


talon_status launch_accept(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                           int32_t *target_tok, int32_t *accept_len, int32_t *accept_nodes,
                           int32_t *bonus_tok, cudaStream_t st, bool close_tree) {
  const int rows = c->B * c->p.budget;
  // Fewer rows than CTAs: as many chunks per row as keep rows x chunks within the grid (rounded
  // down), so that every CTA has one chunk and the last chunk's CTA can do the walk.
  LayerGeom g = make_geom(rows, c->p.vocab, rows <= c->exp_grid ? c->exp_grid - rows + 1 : c->exp_grid);
  // More rows than half the grid: with one chunk per CTA round the last round leaves most SMs
  // idle (960 rows on 592 CTAs are 1.6 rounds); finer chunks keep every CTA streaming to the end.
  if ((long long)rows * g.splits > c->exp_grid && c->argmax_oversplit > 1)
    g = make_geom(rows, c->p.vocab, c->exp_grid * c->argmax_oversplit);
  ArgmaxArgs aa;
  aa.logits = target_logits; aa.row_stride = row_stride; aa.n_nodes = t->n_nodes;
  aa.B = c->B; aa.N = c->p.budget; aa.V = c->p.vocab;
  aa.splits = g.splits; aa.chunk_len = g.chunk_len;
  aa.best = c->d_argmax; aa.status = c->d_status;
  WalkArgs wa;
  wa.t = *t; wa.lo_stride = c->p.max_depth + 2;
  wa.B = c->B; wa.N = c->p.budget; wa.max_depth = c->p.max_depth;
  wa.best = c->d_argmax; wa.target_tok = target_tok ? target_tok : c->d_target_tok;
  wa.accept_len = accept_len; wa.accept_nodes = accept_nodes; wa.bonus_tok = bonus_tok;
  wa.close_tree = close_tree ? 1 : 0; wa.W = c->W; wa.layers_run = c->layers_run; wa.prefix_len = c->d_prefix_len;
  long long items = (long long)rows * g.splits;
  int grid = c->exp_grid;
  if (items < grid) grid = (int)items;
  const int fold = items <= grid ? 1 : 0;       // one chunk per CTA at most: the last chunk's CTA walks
  {
    LaunchTimer lt(c, TALON_K_ARGMAX, st);
    launch_kernel(c, target_argmax_kernel, dim3(grid), dim3(EXP_THREADS), 0, st, aa, wa, c->d_walk_count, fold);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  if (fold) return TALON_OK;
  const int warps_per_block = 4;
  {
    LaunchTimer lt(c, TALON_K_WALK, st);
    launch_kernel(c, accept_walk_kernel, dim3((c->B + warps_per_block - 1) / warps_per_block), dim3(warps_per_block * 32), 0, st, wa);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  return TALON_OK;
}

}  // namespace talon

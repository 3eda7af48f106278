// Tree attention (verification forward of Appendix B) -- warp-MMA implementation.
//
// For sequence b and kv head h the g = Hq/Hkv query heads of all N tree nodes are packed
// into one [g*N, 128] query matrix (row r = node * g + head-in-group), so each K/V tile is
// read once for the whole group.  The key axis (L_b prefix keys followed by the N tree keys)
// is cut into 64-key tiles and the tiles are divided over `splits` CTAs (split-KV); every
// CTA keeps a running (max, sum, O) per query row and a second kernel merges the splits
// with the log-sum-exp rule.  Prefix keys are visible to every node; a tree key j is visible
// to node i iff bit j of the node's ancestor-mask row is set.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

constexpr int AT_THREADS = 256;
constexpr int AT_BM = 128;     // packed query rows per CTA (16 per warp)
constexpr int AT_BN = 64;      // keys per tile
constexpr int AT_D = 128;      // head dimension
constexpr int AT_TILE_BYTES = AT_BN * AT_D * 2;
constexpr int TC_MIN_TILES_PER_CTA = 4;   // split-KV of the tensor-core path: key tiles a CTA should at least own
constexpr int AT_SMEM = AT_BM * AT_D * 2 + 4 * AT_TILE_BYTES;   // Q + 2 stages of (K, V)

struct AttnArgs {
  const __nv_bfloat16 *q, *kp, *vp, *kt, *vt;
  const int64_t *kv_start;
  int64_t stride_t, stride_h;
  const int32_t *prefix_len, *n_nodes;
  const unsigned long long *mask;
  int B, N, W, Hq, Hkv, g;
  float scale_log2;
  int splits, m_blocks;
  __nv_bfloat16 *out;
  float *part_o;
  float2 *part_ml;
};

__device__ inline void cp_async16(void *smem, const void *gmem, bool pred) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
  const int sz = pred ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(sz));
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ inline void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ inline void ldsm_x4(unsigned &r0, unsigned &r1, unsigned &r2, unsigned &r3, const void *p) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ inline void ldsm_x4_t(unsigned &r0, unsigned &r1, unsigned &r2, unsigned &r3, const void *p) {
  const unsigned s = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(s));
}
__device__ inline void mma_bf16(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline unsigned pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<unsigned *>(&v);
}
// byte offset of 16-byte chunk c of row r in a [rows][128] bf16 tile, XOR-swizzled
__device__ inline int swz(int r, int c) { return r * 256 + ((c ^ (r & 7)) << 4); }

// copy a [64 keys][128] tile: key t0+row of a source with `nvalid` keys, `stride` elements apart
__device__ inline void load_kv_tile(unsigned char *dst, const __nv_bfloat16 *src, int64_t stride, int t0,
                                    int nvalid, int tid) {
#pragma unroll
  for (int i = 0; i < (AT_BN * 16) / AT_THREADS; ++i) {
    const int id = tid + i * AT_THREADS;
    const int row = id >> 4, c = id & 15;
    const bool ok = (t0 + row) < nvalid;
    const __nv_bfloat16 *g = ok ? src + (int64_t)(t0 + row) * stride + c * 8 : src;
    cp_async16(dst + swz(row, c), g, ok);
  }
}

__global__ void __launch_bounds__(AT_THREADS, 1)
tree_attention_mma_kernel(AttnArgs a) {
  pdl_enter();
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_q = smem;
  unsigned char *s_kv = smem + AT_BM * AT_D * 2;     // stage s: K at s*2*TILE, V at (s*2+1)*TILE

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mblk = blockIdx.x, split = blockIdx.y;
  const int bh = blockIdx.z, b = bh / a.Hkv, kvh = bh - b * a.Hkv;
  const int n = a.n_nodes[b];
  const int L = a.prefix_len[b];
  const int rows_valid = a.g * n;                // packed rows that hold real nodes
  const int rows_total = a.g * a.N;

  // ---- Q tile -> shared -> A fragments ----
#pragma unroll
  for (int i = 0; i < (AT_BM * 16) / AT_THREADS; ++i) {
    const int id = tid + i * AT_THREADS;
    const int rl = id >> 4, c = id & 15;
    const int r = mblk * AT_BM + rl;
    const bool ok = r < rows_valid;
    const int node = ok ? r / a.g : 0, qh = ok ? r - node * a.g : 0;
    const __nv_bfloat16 *gp = a.q + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * AT_D + c * 8;
    cp_async16(s_q + swz(rl, c), gp, ok);
  }
  cp_async_commit();

  const int nP = (L + AT_BN - 1) / AT_BN;
  const int nT = (a.N + AT_BN - 1) / AT_BN;
  const int tt = nP + nT;
  const int tps = (tt + a.splits - 1) / a.splits;
  const int t_begin = split * tps;
  const int t_end = min(tt, t_begin + tps);

  const __nv_bfloat16 *kp = a.kp + a.kv_start[b] * a.stride_t + (int64_t)kvh * a.stride_h;
  const __nv_bfloat16 *vp = a.vp + a.kv_start[b] * a.stride_t + (int64_t)kvh * a.stride_h;
  const int64_t tree_stride = (int64_t)a.Hkv * AT_D;
  const __nv_bfloat16 *kt = a.kt + ((int64_t)b * a.N * a.Hkv + kvh) * AT_D;
  const __nv_bfloat16 *vt = a.vt + ((int64_t)b * a.N * a.Hkv + kvh) * AT_D;

  auto issue_tile = [&](int tg, int stage) {
    unsigned char *ks = s_kv + (stage * 2) * AT_TILE_BYTES;
    unsigned char *vs = ks + AT_TILE_BYTES;
    if (tg < nP) {
      load_kv_tile(ks, kp, a.stride_t, tg * AT_BN, L, tid);
      load_kv_tile(vs, vp, a.stride_t, tg * AT_BN, L, tid);
    } else {
      load_kv_tile(ks, kt, tree_stride, (tg - nP) * AT_BN, a.N, tid);
      load_kv_tile(vs, vt, tree_stride, (tg - nP) * AT_BN, a.N, tid);
    }
  };
  if (t_begin < t_end) issue_tile(t_begin, 0);
  cp_async_commit();

  cp_async_wait<1>();      // Q has landed
  __syncthreads();
  unsigned qf[8][4];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk)
    ldsm_x4(qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3],
            s_q + swz(warp * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), kk * 2 + (lane >> 4)));

  // rows owned by this thread: r0 and r0 + 8
  const int r0 = mblk * AT_BM + warp * 16 + (lane >> 2);
  unsigned long long mrow[2][2] = {{0ull, 0ull}, {0ull, 0ull}};
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int r = r0 + h * 8;
    if (r < rows_valid) {
      const int node = r / a.g;
      for (int w = 0; w < a.W; ++w) mrow[h][w] = a.mask[((int64_t)b * a.N + node) * a.W + w];
    }
  }

  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) { oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f; }
  float m_i[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_i[2] = {0.f, 0.f};

  int it = 0;
  for (int tg = t_begin; tg < t_end; ++tg, ++it) {
    const int stage = it & 1;
    if (tg + 1 < t_end) {
      issue_tile(tg + 1, stage ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const unsigned char *ks = s_kv + (stage * 2) * AT_TILE_BYTES;
    const unsigned char *vs = ks + AT_TILE_BYTES;

    float sacc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
      for (int nj = 0; nj < 4; ++nj) {
        unsigned b0, b1, b2, b3;
        ldsm_x4(b0, b1, b2, b3, ks + swz(nj * 16 + (lane >> 4) * 8 + (lane & 7), kk * 2 + ((lane >> 3) & 1)));
        mma_bf16(sacc[2 * nj], qf[kk], b0, b1);
        mma_bf16(sacc[2 * nj + 1], qf[kk], b2, b3);
      }
    }

    // ---- scale, mask, online softmax (base-2 exponent domain) ----
    const bool tree_tile = tg >= nP;
    const int key0 = tree_tile ? (tg - nP) * AT_BN : tg * AT_BN;
    float rmax[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int h = c >> 1;
        const int key = key0 + nt * 8 + (lane & 3) * 2 + (c & 1);
        bool vis;
        if (tree_tile) vis = key < a.N && ((mrow[h][key >> 6] >> (key & 63)) & 1ull);
        else vis = key < L;
        const float x = vis ? sacc[nt][c] * a.scale_log2 : -CUDART_INF_F;
        sacc[nt][c] = x;
        rmax[h] = fmaxf(rmax[h], x);
      }
    }
    float alpha[2], muse[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xFFFFFFFFu, rmax[h], 1));
      rmax[h] = fmaxf(rmax[h], __shfl_xor_sync(0xFFFFFFFFu, rmax[h], 2));
      const float mnew = fmaxf(m_i[h], rmax[h]);
      muse[h] = (mnew == -CUDART_INF_F) ? 0.f : mnew;
      alpha[h] = exp2f(m_i[h] - muse[h]);
      m_i[h] = mnew;
    }
    float rsum[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int h = c >> 1;
        const float p = exp2f(sacc[nt][c] - muse[h]);
        sacc[nt][c] = p;
        rsum[h] += p;
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) l_i[h] = l_i[h] * alpha[h] + rsum[h];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      oacc[i][0] *= alpha[0]; oacc[i][1] *= alpha[0];
      oacc[i][2] *= alpha[1]; oacc[i][3] *= alpha[1];
    }

    // ---- O += P V ----
#pragma unroll
    for (int kk2 = 0; kk2 < 4; ++kk2) {
      unsigned pa[4];
      pa[0] = pack_bf16(sacc[2 * kk2][0], sacc[2 * kk2][1]);
      pa[1] = pack_bf16(sacc[2 * kk2][2], sacc[2 * kk2][3]);
      pa[2] = pack_bf16(sacc[2 * kk2 + 1][0], sacc[2 * kk2 + 1][1]);
      pa[3] = pack_bf16(sacc[2 * kk2 + 1][2], sacc[2 * kk2 + 1][3]);
#pragma unroll
      for (int dj = 0; dj < 8; ++dj) {
        unsigned b0, b1, b2, b3;
        ldsm_x4_t(b0, b1, b2, b3, vs + swz(kk2 * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), dj * 2 + (lane >> 4)));
        mma_bf16(oacc[2 * dj], pa, b0, b1);
        mma_bf16(oacc[2 * dj + 1], pa, b2, b3);
      }
    }
    __syncthreads();
  }
  cp_async_wait<0>();

#pragma unroll
  for (int h = 0; h < 2; ++h) {
    l_i[h] += __shfl_xor_sync(0xFFFFFFFFu, l_i[h], 1);
    l_i[h] += __shfl_xor_sync(0xFFFFFFFFu, l_i[h], 2);
  }

  if (a.splits == 1) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int r = r0 + h * 8;
      if (r >= rows_total) continue;
      const int node = r / a.g, qh = r - node * a.g;
      const bool live = r < rows_valid && l_i[h] > 0.f;
      const float inv = live ? 1.f / l_i[h] : 0.f;
      __nv_bfloat16 *op = a.out + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * AT_D + (lane & 3) * 2;
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(oacc[nt][2 * h] * inv, oacc[nt][2 * h + 1] * inv);
        *reinterpret_cast<__nv_bfloat162 *>(op + nt * 8) = v;
      }
    }
  } else {
    const int mpad = a.m_blocks * AT_BM;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int r = r0 + h * 8;
      const int64_t prow = ((int64_t)bh * a.splits + split) * mpad + r;
      float *op = a.part_o + prow * AT_D + (lane & 3) * 2;
#pragma unroll
      for (int nt = 0; nt < 16; ++nt)
        *reinterpret_cast<float2 *>(op + nt * 8) = make_float2(oacc[nt][2 * h], oacc[nt][2 * h + 1]);
      if ((lane & 3) == 0) a.part_ml[prow] = make_float2(m_i[h], l_i[h]);
    }
  }
}

// merge the split-KV partials: one warp per packed query row
__global__ void attention_combine_kernel(AttnArgs a) {
  pdl_enter();
  const int lane = threadIdx.x & 31;
  const int mpad = a.m_blocks * AT_BM;
  const int rows_total = a.g * a.N;
  const int64_t gw = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t total = (int64_t)a.B * a.Hkv * rows_total;
  if (gw >= total) return;
  const int bh = (int)(gw / rows_total), r = (int)(gw - (int64_t)bh * rows_total);
  const int b = bh / a.Hkv, kvh = bh - b * a.Hkv;
  const int node = r / a.g, qh = r - node * a.g;
  __nv_bfloat16 *op = a.out + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * AT_D + lane * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float lsum = 0.f;
  if (r < a.g * a.n_nodes[b]) {
    float mx = -CUDART_INF_F;
    for (int s = 0; s < a.splits; ++s) mx = fmaxf(mx, a.part_ml[((int64_t)bh * a.splits + s) * mpad + r].x);
    for (int s = 0; s < a.splits; ++s) {
      const int64_t prow = ((int64_t)bh * a.splits + s) * mpad + r;
      const float2 ml = a.part_ml[prow];
      if (ml.x == -CUDART_INF_F) continue;
      const float w = exp2f(ml.x - mx);
      const float4 o = *reinterpret_cast<const float4 *>(a.part_o + prow * AT_D + lane * 4);
      acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
      lsum += w * ml.y;
    }
  }
  const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
  const __nv_bfloat162 v0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
  const __nv_bfloat162 v1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  *reinterpret_cast<__nv_bfloat162 *>(op) = v0;
  *reinterpret_cast<__nv_bfloat162 *>(op + 2) = v1;
}

static int attn_m_blocks(const talon_ctx *c) {
  const int g = c->p.n_q_heads / c->p.n_kv_heads;
  return (g * c->p.budget + AT_BM - 1) / AT_BM;
}

size_t attention_workspace_elems(const talon_ctx *c, size_t *ml_elems) {
  const int mb = attn_m_blocks(c);
  long long ctas = 2LL * c->p.batch_max * c->p.n_kv_heads * mb;       // room for two key ranges per CTA slot
  if (ctas < 2LL * c->sm_count) ctas = 2LL * c->sm_count;
  *ml_elems = (size_t)ctas * AT_BM;
  return (size_t)ctas * AT_BM * AT_D;
}

talon_status attention_mma_setup() {
  return cudaFuncSetAttribute(tree_attention_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, AT_SMEM) ==
                 cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

talon_status launch_attention(talon_ctx *c, const talon_tree *t, const void *q, const void *kp, const void *vp,
                              const void *kt, const void *vt, const int64_t *kv_start, const int32_t *block_table,
                              int bt_stride, int64_t kv_tokens,
                              int64_t stride_t, int64_t stride_h, int max_prefix_len, float sm_scale, void *out,
                              cudaStream_t st) {
  AttnArgs a;
  a.q = (const __nv_bfloat16 *)q; a.kp = (const __nv_bfloat16 *)kp; a.vp = (const __nv_bfloat16 *)vp;
  a.kt = (const __nv_bfloat16 *)kt; a.vt = (const __nv_bfloat16 *)vt;
  a.kv_start = kv_start; a.stride_t = stride_t; a.stride_h = stride_h;
  a.prefix_len = c->d_prefix_len; a.n_nodes = t->n_nodes; a.mask = (const unsigned long long *)t->mask;
  a.B = c->B; a.N = c->p.budget; a.W = c->W; a.Hq = c->p.n_q_heads; a.Hkv = c->p.n_kv_heads;
  a.g = a.Hq / a.Hkv;
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.m_blocks = attn_m_blocks(c);
  a.out = (__nv_bfloat16 *)out; a.part_o = c->d_attn_o; a.part_ml = c->d_attn_ml;

  if (attention_tc_supported(c, stride_t, stride_h, sm_scale)) {
    // tensor-core path: CTAs own two 128-row query tiles and 128-key tiles
    const int pairs = (a.m_blocks + 1) / 2;
    const int ctas = pairs * c->B * a.Hkv;
    const int tiles = (max_prefix_len + 127) / 128 + (a.N + 127) / 128;
    int sp = 1;
    if (ctas < c->sm_count) {
      sp = c->sm_count / ctas;
      const int by_tiles = (tiles + c->attn_min_tiles - 1) / c->attn_min_tiles;
      if (sp > by_tiles) sp = by_tiles;
      if (sp < 1) sp = 1;
      // up to eight key ranges can merge inside one thread-block cluster, which saves the merge
      // kernel; a ninth range is worth less than that
      if (c->attn_cluster && sp > 8 && sp <= c->attn_cluster_cap &&
          (c->attn_cluster == 2 || (long long)c->B * a.Hkv * a.g * a.N * 8 >= c->attn_cluster_min_rows))
        sp = 8;
    } else if (ctas % c->sm_count) {
      // More CTAs than SMs and a ragged last wave: halving the key ranges can fill it (512 CTAs on
      // 148 SMs are 4 waves of 257 tiles, 1024 half CTAs are 7 waves of 129).  Cost model in key
      // tiles: waves x (tiles per CTA + 2 for the prologue and epilogue), plus what merging the
      // partial results costs, about one tile per 24 CTAs per SM.
      const long long sm = c->sm_count;
      auto cost = [&](int s) {
        const long long n = (long long)ctas * s;
        const long long waves = (n + sm - 1) / sm;
        return waves * ((tiles + s - 1) / s + 2) + (s > 1 ? n / (24 * sm) + 3 : 0);
      };
      if (tiles >= 32 && cost(2) < cost(1)) sp = 2;
    }
    if (c->attn_force_splits > 0) sp = c->attn_force_splits;
    while (sp > 1 && (size_t)a.m_blocks * c->B * a.Hkv * sp * AT_BM > c->attn_ml_elems) --sp;
    a.splits = sp;
    int merged = 0;
    talon_status r = launch_attention_tc(c, t, q, kp, vp, kt, vt, kv_start, block_table, bt_stride, stride_t, stride_h, kv_tokens,
                                         max_prefix_len, sm_scale, out, sp, a.m_blocks, st, &merged);
    if (r != TALON_OK) return r;
    if (sp > 1 && !merged) {
      const int64_t rows = (int64_t)c->B * a.Hkv * a.g * a.N;
      const int wpb = 8;
      LaunchTimer lt(c, TALON_K_COMBINE, st);
      launch_kernel(c, attention_combine_kernel, dim3((unsigned)((rows + wpb - 1) / wpb)), dim3(wpb * 32), 0, st, a);
      if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
      c->launches += 1;
    }
    return TALON_OK;
  }

  if (block_table) return TALON_ERR_UNSUPPORTED;     // the warp-MMA kernel reads contiguous blocks only
  const int base = a.m_blocks * c->B * a.Hkv;
  const int max_tiles = (max_prefix_len + AT_BN - 1) / AT_BN + (a.N + AT_BN - 1) / AT_BN;
  int splits = 1;
  if (base < c->sm_count) {
    splits = c->sm_count / base;
    if (splits > max_tiles) splits = max_tiles;
    if (splits < 1) splits = 1;
  }
  // stay inside the partial workspace sized at creation
  while (splits > 1 && (size_t)base * splits * AT_BM > c->attn_ml_elems) --splits;
  a.splits = splits;

  dim3 grid(a.m_blocks, splits, c->B * a.Hkv);
  {
    LaunchTimer lt(c, TALON_K_ATTENTION, st);
    launch_kernel(c, tree_attention_mma_kernel, grid, dim3(AT_THREADS), AT_SMEM, st, a);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  if (splits > 1) {
    const int64_t rows = (int64_t)c->B * a.Hkv * a.g * a.N;
    const int wpb = 8;
    LaunchTimer lt(c, TALON_K_COMBINE, st);
    launch_kernel(c, attention_combine_kernel, dim3((unsigned)((rows + wpb - 1) / wpb)), dim3(wpb * 32), 0, st, a);
    if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
    c->launches += 1;
  }
  return TALON_OK;
}

}  // namespace talon

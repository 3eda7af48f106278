// Sampling verification (Appendix B of the paper, steps 1-3, the temperature-1 setting) for sm_100a.
//
//   target_softmax_stats_kernel : step (1), the posterior's normaliser: one streaming pass over
//                                 the target logits of every tree node, per chunk the maximum and
//                                 the sum of 2^((z - max) log2(e) / T).  Same traffic as the greedy
//                                 arg-max pass: 4 V bytes per node, read once.
//   accept_sample_kernel        : one CTA per sequence.  Chunk statistics -> log-sum-exp per node;
//                                 warp 0 walks from the root and tries the children of the current
//                                 node one after the other (child with token w accepted when
//                                 u * unclaimed mass < p(w), else w is struck); the CTA then draws
//                                 the correction token from what is left of the posterior at the
//                                 last node by inverse CDF in token order (step 3): the chunk
//                                 statistics of that row say which chunk holds the target mass, so
//                                 only that chunk of the row is read again.
//
// The uniforms are inputs: one per node (consumed if the node is tried) and one per sequence.
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int SAMP_THREADS = 1024;
constexpr int SAMP_WARPS = SAMP_THREADS / 32;
constexpr int SAMP_GROUP = 128;                       // elements a warp takes with one 128-bit load per lane
constexpr int SAMP_MAX_GROUPS = 2048;                 // vocabulary <= 262144
constexpr int SAMP_GROUPS_PER_THREAD = SAMP_MAX_GROUPS / SAMP_THREADS;
constexpr int SAMP_MAX_NODES = 128;                    // the library's largest node budget

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

struct StatsArgs {
  const float *logits;
  int64_t row_stride;
  const int32_t *n_nodes;
  int B, N, V;
  int splits, chunk_len;
  float scale;              // log2(e) / T
  float2 *part;             // [B * N, splits] (max, sum relative to max)
  int *status;
};

__global__ void __launch_bounds__(EXP_THREADS)
target_softmax_stats_kernel(StatsArgs a) {
  __shared__ float s_m[EXP_WARPS], s_s[EXP_WARPS];
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
    float m = -CUDART_INF_F, s = 0.f;
    bool bad = false;
    // the next tile is requested before the current one is worked on
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
      float bm = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) {
          bad |= (v[u][e] != v[u][e]);
          bm = fmaxf(bm, v[u][e]);
        }
      if (bm > m) {
        s *= ex2_approx((m - bm) * a.scale);
        m = bm;
      }
      if (m > -CUDART_INF_F) {
        const float c = -m * a.scale;          // an infinite m (a +inf logit) gives NaN, reported below
        float acc = 0.f;
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) acc += ex2_approx(fmaf(v[u][e], a.scale, c));
        s += acc;
      }
    }
    float wm = m;
#pragma unroll
    for (int o = 16; o; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(FULL, wm, o));
    float ws = (m > -CUDART_INF_F || s != s) ? s * exp2f((m - wm) * a.scale) : 0.f;
#pragma unroll
    for (int o = 16; o; o >>= 1) ws += __shfl_xor_sync(FULL, ws, o);
    if (__any_sync(FULL, bad) && lane == 0) atomicOr(a.status, STATUS_NONFINITE);
    __syncthreads();
    if (lane == 0) { s_m[warp] = wm; s_s[warp] = ws; }
    __syncthreads();
    if (tid == 0) {
      float bm = s_m[0];
      for (int w = 1; w < EXP_WARPS; ++w) bm = fmaxf(bm, s_m[w]);
      float tot = 0.f;
      for (int w = 0; w < EXP_WARPS; ++w)
        tot += (s_m[w] > -CUDART_INF_F || s_s[w] != s_s[w]) ? s_s[w] * exp2f((s_m[w] - bm) * a.scale) : 0.f;
      a.part[(size_t)row * a.splits + chunk] = make_float2(bm, tot);
    }
  }
}

struct SampleArgs {
  talon_tree t;
  int lo_stride;
  int B, N, V, max_depth;
  const float *logits;
  int64_t row_stride;
  int splits, chunk_len;
  const float2 *part;
  float scale;              // log2(e) / T
  double inv_t;             // 1 / T
  const double *u_accept;   // [B, N]
  const double *u_sample;   // [B]
  int32_t *accept_len, *accept_nodes, *out_tok;
  int *status;
};

// Unnormalised posterior weight of a logit relative to the row maximum; the same expression
// wherever the inverse CDF needs it, so a token's weight is the same number every time.
__device__ __forceinline__ double weight(float z, float row_max, float scale) {
  return (double)ex2_approx((z - row_max) * scale);        // relative error 2^-22: far inside the stated 1e-6
}

__global__ void __launch_bounds__(SAMP_THREADS)
accept_sample_kernel(SampleArgs a) {
  __shared__ double s_logt[SAMP_MAX_NODES];       // log of the row's sum of exponentials
  __shared__ float s_max[SAMP_MAX_NODES];         // row maximum
  __shared__ int s_rej[SAMP_MAX_NODES];           // tokens struck at the last node
  __shared__ double s_gsum[SAMP_MAX_GROUPS];        // weight of each group of 128 tokens
  __shared__ double s_wtot[SAMP_WARPS];
  __shared__ double s_rejw[SAMP_MAX_NODES];         // their weights
  __shared__ int s_cur, s_nrej, s_bad, s_pick, s_chunk;
  __shared__ double s_resid, s_cw;

  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  const size_t nb = (size_t)b * a.N;
  const int n = a.t.n_nodes[b];
  int32_t *path = a.accept_nodes + (size_t)b * (a.max_depth + 1);
  if (tid == 0) { s_bad = 0; s_pick = -1; }
  __syncthreads();

  // ---- step (1): the normaliser of every node's posterior from the chunk statistics:
  // one warp per node, one lane per chunk (at most 32 chunks) ----
  for (int i = warp; i < n; i += SAMP_WARPS) {
    const float2 ms = lane < a.splits ? a.part[(nb + i) * a.splits + lane] : make_float2(-CUDART_INF_F, 0.f);
    float mx = ms.x;
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
    double t = 0.0;
    if (ms.y != ms.y) t = (double)ms.y;
    else if (ms.x > -CUDART_INF_F) t = (double)ms.y * (double)exp2f((ms.x - mx) * a.scale);
#pragma unroll
    for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(FULL, t, o);
    if (lane == 0) {
      if (!(t > 0.0) || !(t < CUDART_INF) || !(mx < CUDART_INF_F) || !(mx > -CUDART_INF_F)) s_bad = 1;
      s_max[i] = mx;
      s_logt[i] = log(t);
    }
  }
  __syncthreads();
  if (s_bad) {                  // a posterior that does not exist: nothing is accepted, no token
    if (tid == 0) {
      atomicOr(a.status, STATUS_NONFINITE);
      a.accept_len[b] = 0;
      a.out_tok[b] = -1;
      path[0] = 0;
    }
    for (int i = 1 + tid; i <= a.max_depth; i += SAMP_THREADS) path[i] = -1;
    return;
  }

  // ---- step (2): walk down while a child is accepted ----
  if (warp == 0) {
    int cur = 0, len = 0, nrej = 0;
    if (lane == 0) path[0] = 0;
    for (int d = 0; d < a.max_depth; ++d) {
      const int lo = a.t.layer_off[b * a.lo_stride + d + 1];
      const int hi = a.t.layer_off[b * a.lo_stride + d + 2];
      const float *rowp = a.logits + (int64_t)(nb + cur) * a.row_stride;
      const double lse_m = (double)s_max[cur], logt = s_logt[cur];
      double mass = 1.0;
      int found = -1;
      nrej = 0;
      for (int c0 = lo; c0 < hi && found < 0; c0 += 32) {
        const int c = c0 + lane;
        const bool kid = c < hi && a.t.parent[nb + c] == cur;
        int w = 0;
        double p = 0.0, u = 1.0;
        if (kid) {
          w = a.t.token[nb + c];
          p = exp(((double)rowp[w] - lse_m) * a.inv_t - logt);
          u = a.u_accept[nb + c];
        }
        unsigned m = __ballot_sync(FULL, kid);
        while (m) {                                   // the children in storage order
          const int j = __ffs(m) - 1;
          m &= m - 1;
          const double pj = __shfl_sync(FULL, p, j), uj = __shfl_sync(FULL, u, j);
          const int wj = __shfl_sync(FULL, w, j);
          if (uj * mass < pj) { found = c0 + j; break; }
          mass -= pj;
          if (lane == 0) s_rej[nrej] = wj;
          ++nrej;
        }
      }
      if (found < 0) break;
      cur = found;
      ++len;
      nrej = 0;
      if (lane == 0) path[len] = cur;
    }
    // a node at the depth cap has no children: nothing was struck there
    if (len == a.max_depth) nrej = 0;
    for (int i = len + 1 + lane; i <= a.max_depth; i += 32) path[i] = -1;
    if (lane == 0) {
      a.accept_len[b] = len;
      s_cur = cur;
      s_nrej = nrej;
    }
  }
  __syncthreads();

  // ---- step (3): the correction token from what is left of the posterior at the last node ----
  const int cur = s_cur, nrej = s_nrej;
  const float *rowp = a.logits + (int64_t)(nb + cur) * a.row_stride;
  const float rmax = s_max[cur];
  // (a) which chunk of the row holds the target mass: the chunk statistics already say how much
  // weight each chunk carries; the struck tokens are taken out of their chunks first
  if (warp == 0) {
    const float2 ms = lane < a.splits ? a.part[(nb + cur) * a.splits + lane] : make_float2(-CUDART_INF_F, 0.f);
    double wc = (ms.x > -CUDART_INF_F) ? (double)ms.y * (double)exp2f((ms.x - rmax) * a.scale) : 0.0;
    for (int r0 = 0; r0 < nrej; r0 += 32) {
      const int r = r0 + lane;
      const int w = r < nrej ? s_rej[r] : 0;
      const double wt = r < nrej ? weight(rowp[w], rmax, a.scale) : 0.0;
      if (r < nrej) s_rejw[r] = wt;
      for (int j = 0; j < min(32, nrej - r0); ++j) {          // in storage order, one after the other
        const int wj = __shfl_sync(FULL, w, j);
        const double tj = __shfl_sync(FULL, wt, j);
        if (lane == wj / a.chunk_len) wc -= tj;
      }
    }
    wc = fmax(wc, 0.0);
    double inc = wc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(FULL, inc, o);
      if (lane >= o) inc += t;
    }
    const double total = __shfl_sync(FULL, inc, 31);
    const double target = a.u_sample[b] * total;
    const double excl = inc - wc;
    const unsigned here = __ballot_sync(FULL, wc > 0.0 && excl <= target && target < inc);
    const unsigned any = __ballot_sync(FULL, wc > 0.0);
    int c;
    double resid, cw;
    if (here) {
      c = __ffs(here) - 1;
      resid = target - __shfl_sync(FULL, excl, c);
    } else {                       // rounding put the target at or past the total: the last chunk with weight
      c = any ? 31 - __clz(any) : -1;
      resid = CUDART_INF;
    }
    cw = c >= 0 ? __shfl_sync(FULL, wc, c) : 0.0;
    if (lane == 0) { s_chunk = c; s_resid = resid; s_cw = cw; }
  }
  __syncthreads();
  const int chunk = s_chunk;
  const double chunk_resid = s_resid, chunk_weight = s_cw;      // read before anybody reuses the slots
  if (chunk < 0) {                 // no weight at all (cannot happen with a finite row)
    if (tid == 0) a.out_tok[b] = -1;
    return;
  }
  // (b) weights of the chosen chunk's groups of 128 tokens: one 128-bit load per lane, all of a
  // warp's loads requested before any is used
  const int c_lo = chunk * a.chunk_len, c_hi = min(a.V, c_lo + a.chunk_len);
  const int groups = (c_hi - c_lo + SAMP_GROUP - 1) / SAMP_GROUP;
  for (int g0 = warp; g0 < groups; g0 += 4 * SAMP_WARPS) {
    float4 x[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int g = g0 + r * SAMP_WARPS;
      const int idx = c_lo + g * SAMP_GROUP + lane * 4;
      x[r] = make_float4(-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F);
      if (g < groups) {
        if (idx + 4 <= c_hi) x[r] = *reinterpret_cast<const float4 *>(rowp + idx);
        else {
          if (idx < c_hi) x[r].x = rowp[idx];
          if (idx + 1 < c_hi) x[r].y = rowp[idx + 1];
          if (idx + 2 < c_hi) x[r].z = rowp[idx + 2];
        }
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int g = g0 + r * SAMP_WARPS;
      double sum = weight(x[r].x, rmax, a.scale) + weight(x[r].y, rmax, a.scale) +
                   weight(x[r].z, rmax, a.scale) + weight(x[r].w, rmax, a.scale);
#pragma unroll
      for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
      if (lane == 0 && g < groups) s_gsum[g] = sum;
    }
  }
  __syncthreads();
  if (tid == 0)                                   // strike the rejected tokens of this chunk, in order
    for (int r = 0; r < nrej; ++r) {
      const int w = s_rej[r];
      if (w >= c_lo && w < c_hi) s_gsum[(w - c_lo) / SAMP_GROUP] -= s_rejw[r];
    }
  __syncthreads();
  // inclusive scan of the group weights in token order: thread t owns groups 2t, 2t+1
  double own[SAMP_GROUPS_PER_THREAD], local = 0.0;
#pragma unroll
  for (int r = 0; r < SAMP_GROUPS_PER_THREAD; ++r) {
    const int g = tid * SAMP_GROUPS_PER_THREAD + r;
    own[r] = g < groups ? fmax(s_gsum[g], 0.0) : 0.0;
    local += own[r];
  }
  double inc = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_wtot[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    double w = s_wtot[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double t = __shfl_up_sync(FULL, w, o);
      if (lane >= o) w += t;
    }
    s_wtot[lane] = w;                             // inclusive over warps
  }
  __syncthreads();
  // the target inside the chunk, on the scale of the weights just recomputed (the chunk statistic
  // and the recomputed total agree to rounding; the ratio keeps the relative position)
  const double total = s_wtot[SAMP_WARPS - 1];
  const double target = chunk_resid < CUDART_INF ? chunk_resid * (total / chunk_weight) : CUDART_INF;
  double excl = (warp ? s_wtot[warp - 1] : 0.0) + inc - local;
#pragma unroll
  for (int r = 0; r < SAMP_GROUPS_PER_THREAD; ++r) {
    if (own[r] > 0.0 && excl <= target && target < excl + own[r]) {
      s_pick = tid * SAMP_GROUPS_PER_THREAD + r;  // at most one group satisfies this
      s_resid = target - excl;
    }
    excl += own[r];
  }
  __syncthreads();
  if (warp != 0) return;
  int g = s_pick;
  double resid = s_resid;
  if (g < 0) {
    // rounding put the target at or past the total: the last group that has weight, and its end
    for (int q = lane; q < groups; q += 32)
      if (s_gsum[q] > 0.0) g = q;                 // ascending: the lane's highest group with weight
#pragma unroll
    for (int o = 16; o; o >>= 1) g = max(g, __shfl_xor_sync(FULL, g, o));
    resid = CUDART_INF;
  }
  if (g < 0) {                                    // no weight at all (cannot happen with a finite row)
    if (lane == 0) a.out_tok[b] = -1;
    return;
  }
  // inside the group: 4 tokens per lane in token order
  const int idx = c_lo + g * SAMP_GROUP + lane * 4;
  double wv[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    wv[e] = idx + e < c_hi ? weight(rowp[idx + e], rmax, a.scale) : 0.0;
    for (int r = 0; r < nrej; ++r)
      if (s_rej[r] == idx + e) wv[e] = 0.0;
  }
  const double lsum = wv[0] + wv[1] + wv[2] + wv[3];
  double linc = lsum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double t = __shfl_up_sync(FULL, linc, o);
    if (lane >= o) linc += t;
  }
  double run = linc - lsum;
  int tok = -1, last = -1;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (wv[e] > 0.0) {
      last = idx + e;
      if (tok < 0 && resid < run + wv[e]) tok = idx + e;
    }
    run += wv[e];
  }
  // the first token (lowest lane) whose cumulative weight passes the target; else the group's last
  const unsigned hit = __ballot_sync(FULL, tok >= 0);
  if (hit) {
    tok = __shfl_sync(FULL, tok, __ffs(hit) - 1);
  } else {
    const unsigned any = __ballot_sync(FULL, last >= 0);
    tok = any ? __shfl_sync(FULL, last, 31 - __clz(any)) : -1;
  }
  if (lane == 0) a.out_tok[b] = tok;
}

}  // namespace

talon_status launch_accept_sample(talon_ctx *c, const talon_tree *t, const float *target_logits, int64_t row_stride,
                                  double temperature, const double *u_accept, const double *u_sample,
                                  int32_t *accept_len, int32_t *accept_nodes, int32_t *out_tok, cudaStream_t st) {
  if (c->p.vocab > SAMP_MAX_GROUPS * SAMP_GROUP || c->p.budget > SAMP_MAX_NODES) return TALON_ERR_UNSUPPORTED;
  const int rows = c->B * c->p.budget;
  LayerGeom g = make_geom(rows, c->p.vocab, c->exp_grid);
  // (as in the greedy arg-max pass: finer chunks when the rows outnumber the grid)
  if ((long long)rows * g.splits > c->exp_grid && c->argmax_oversplit > 1)
    g = make_geom(rows, c->p.vocab, c->exp_grid * c->argmax_oversplit);
  StatsArgs sa;
  sa.logits = target_logits; sa.row_stride = row_stride; sa.n_nodes = t->n_nodes;
  sa.B = c->B; sa.N = c->p.budget; sa.V = c->p.vocab;
  sa.splits = g.splits; sa.chunk_len = g.chunk_len;
  sa.scale = (float)(1.4426950408889634 / temperature);
  sa.part = c->d_samp_ms; sa.status = c->d_status;
  long long items = (long long)rows * g.splits;
  int grid = c->exp_grid;
  if (items < grid) grid = (int)items;
  {
    LaunchTimer lt(c, TALON_K_ROWSTATS, st);
    launch_kernel(c, target_softmax_stats_kernel, dim3(grid), dim3(EXP_THREADS), 0, st, sa);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;

  SampleArgs wa;
  wa.t = *t; wa.lo_stride = c->p.max_depth + 2;
  wa.B = c->B; wa.N = c->p.budget; wa.V = c->p.vocab; wa.max_depth = c->p.max_depth;
  wa.logits = target_logits; wa.row_stride = row_stride;
  wa.splits = g.splits; wa.chunk_len = g.chunk_len; wa.part = c->d_samp_ms;
  wa.scale = sa.scale; wa.inv_t = 1.0 / temperature;
  wa.u_accept = u_accept; wa.u_sample = u_sample;
  wa.accept_len = accept_len; wa.accept_nodes = accept_nodes; wa.out_tok = out_tok;
  wa.status = c->d_status;
  {
    LaunchTimer lt(c, TALON_K_SAMPLE, st);
    launch_kernel(c, accept_sample_kernel, dim3(c->B), dim3(SAMP_THREADS), 0, st, wa);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 2;
  return TALON_OK;
}

}  // namespace talon

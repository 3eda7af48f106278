// Adaptive draft-tree expansion (Algorithm 2 of the paper; Eq. 2-5) for sm_100a.
//
//   expand_rows_kernel  : one pass over the fp32 logit rows of the frontier.  Per row it
//                         produces the softmax normaliser (max and sum of exponentials,
//                         i.e. the denominator of P_Md(w | x_<=v) in Eq. 3) and the k
//                         largest logits with their token ids, in a single read of the row.
//                         Rows are cut into chunks so that a frontier of one row still
//                         spreads over the whole GPU; the CTA that finishes the last chunk
//                         of a row merges that row's chunk results.
//   select_layer_kernel : one CTA per sequence.  Scores the pooled candidates with
//                         log p(u) = log p(v) + log P(w|v) (Eq. 2-3), applies Top-K (Eq. 5) or
//                         the gate p(u) >= mu * max p (Eq. 4), truncates to the remaining
//                         budget, and appends the survivors with parent links, depths and
//                         ancestor-mask rows.
//   reset / build       : tree initialisation and the closing pass (positions, sentinels).
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr float LOG2E_F = 1.4426950408889634f;

struct ExpandArgs {
  const float *logits;
  int64_t row_stride;
  int rows_per_seq;
  int layout;
  const int32_t *n_nodes;
  const int32_t *layer_off;
  int lo_stride;
  int B, N, V, d, k, key_stride, target_items;
  unsigned long long *part_keys;
  float2 *part_ms;
  unsigned long long *row_keys;
  double *row_lse;
  unsigned int *row_count;
  int *status;
};

// ---------------------------------------------------------------------------------------
// Frontier geometry: exclusive scan of the per-sequence frontier sizes (block-wide).
// s_base[b] = first packed row of sequence b, s_base[B] = total rows.
// ---------------------------------------------------------------------------------------
template <int THREADS>
__device__ void frontier_scan(const int32_t *n_nodes, const int32_t *layer_off, int lo_stride,
                              int B, int N, int d, int *s_base, int *s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int PER = (MAX_BATCH + THREADS - 1) / THREADS;
  int f[PER];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    int b = tid * PER + i;
    int v = 0;
    if (b < B && n_nodes[b] < N) {
      v = layer_off[b * lo_stride + d + 1] - layer_off[b * lo_stride + d];
      if (v < 0) v = 0;
    }
    f[i] = v;
    sum += v;
  }
  int inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = lane < THREADS / 32 ? s_warp[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(FULL, winc, o);
      if (lane >= o) winc += t;
    }
    if (lane < THREADS / 32) s_warp[lane] = winc - w;   // exclusive warp offsets
    if (lane == THREADS / 32 - 1) s_base[B] = winc;     // total
  }
  __syncthreads();
  int run = s_warp[warp] + inc - sum;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    int b = tid * PER + i;
    if (b < B) s_base[b] = run;
    run += f[i];
  }
  __syncthreads();
}

// largest b with s_base[b] <= row (rows of empty sequences are skipped automatically)
__device__ inline int seq_of_row(const int *s_base, int B, int row) {
  int lo = 0, hi = B;   // invariant: s_base[lo] <= row < s_base[hi]
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (s_base[mid] <= row) lo = mid; else hi = mid;
  }
  return lo;
}

// ---------------------------------------------------------------------------------------
// Warp-distributed sorted list of the best keys seen so far (position p lives in register
// p/32 of lane p%32, descending).  thr is the key at position k-1: only a key above it can
// enter.  Keys are unique (they embed the token id), so there are no equal keys.
// ---------------------------------------------------------------------------------------
template <int SLOTS>
struct WarpList {
  unsigned long long key[SLOTS];
  unsigned long long thr;

  __device__ void clear() {
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) key[s] = 0ull;
    thr = 0ull;
  }
  __device__ void insert(unsigned long long nk, int k, int lane) {
    if (nk <= thr) return;                       // warp-uniform
    int pos = 0;
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) pos += __popc(__ballot_sync(FULL, key[s] > nk));
#pragma unroll
    for (int s = SLOTS - 1; s >= 0; --s) {
      unsigned long long up = __shfl_up_sync(FULL, key[s], 1);
      if (s > 0) {
        unsigned long long carry = __shfl_sync(FULL, key[s - 1], 31);
        if (lane == 0) up = carry;
      }
      int p = s * 32 + lane;
      if (p > pos) key[s] = up;
      else if (p == pos) key[s] = nk;
    }
    unsigned long long t = 0ull;
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      unsigned long long c = __shfl_sync(FULL, key[s], (k - 1) & 31);
      if (s == ((k - 1) >> 5)) t = c;
    }
    thr = t;
  }
};

// Number of entries of a descending list of length k that are greater than `key`.
__device__ inline int count_greater(const unsigned long long *list, int k, unsigned long long key) {
  int lo = 0, hi = k;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (list[mid] > key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// Merge `nlists` descending lists of length k (shared memory, `stride` apart) into the k best,
// written to out[0..k).  Rank of a key = its own position + how many keys of the other lists
// beat it; keys are unique so ranks are too.  Empty slots (key 0) fill the tail.
__device__ void merge_sorted_lists(const unsigned long long *s_lists, int nlists, int stride, int k,
                                   unsigned long long *out) {
  for (int idx = threadIdx.x; idx < nlists * k; idx += blockDim.x) {
    int w = idx / k, p = idx - w * k;
    unsigned long long key = s_lists[w * stride + p];
    int rank = p;
    for (int o = 0; o < nlists; ++o)
      if (o != w) rank += count_greater(s_lists + o * stride, k, key);
    if (rank < k) out[rank] = key;
  }
}

// ---------------------------------------------------------------------------------------
// The streaming kernel.
// ---------------------------------------------------------------------------------------
template <int SLOTS>
__global__ void __launch_bounds__(EXP_THREADS)
expand_rows_kernel(ExpandArgs a) {
  constexpr int KCAP = 32 * SLOTS;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long *s_lists = reinterpret_cast<unsigned long long *>(smem_raw);   // [EXP_MAX_SPLITS][KCAP]
  __shared__ int s_base[MAX_BATCH + 1];
  __shared__ int s_warp[EXP_WARPS];
  __shared__ float s_m[EXP_WARPS];
  __shared__ double s_s[EXP_WARPS];
  __shared__ float s_bm;
  __shared__ int s_last;

  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  frontier_scan<EXP_THREADS>(a.n_nodes, a.layer_off, a.lo_stride, a.B, a.N, a.d, s_base, s_warp);
  const LayerGeom g = make_geom(s_base[a.B], a.V, a.target_items);
  const int n_items = g.total_rows * g.splits;
  const int k = a.k;

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int row = item / g.splits, chunk = item - row * g.splits;
    const int b = seq_of_row(s_base, a.B, row);
    const int j = row - s_base[b];
    const int node = a.layer_off[b * a.lo_stride + a.d] + j;
    int rsel = (a.layout == TALON_ROWS_BY_NODE) ? node : j;
    if (rsel >= a.rows_per_seq) {               // caller reserved too few rows: stay in bounds, report
      rsel = a.rows_per_seq - 1;
      if (tid == 0) atomicOr(a.status, STATUS_CAPACITY);
    }
    const int64_t lrow = (int64_t)b * a.rows_per_seq + rsel;
    const float *rowp = a.logits + lrow * a.row_stride;
    const int start = chunk * g.chunk_len;
    const int end = min(a.V, start + g.chunk_len);

    float m_t = -CUDART_INF_F, s_t = 0.f;
    WarpList<SLOTS> list;
    list.clear();
    float thr0 = -CUDART_INF_F, thr_f = -CUDART_INF_F;
    bool first = true;

    for (int base = start; base < end; base += EXP_TILE) {
      float v[EXP_UNROLL][EXP_VEC];
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u) {
        const int idx = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC;
        if (idx + EXP_VEC <= end) {
          const float4 x = __ldcs(reinterpret_cast<const float4 *>(rowp + idx));
          v[u][0] = x.x; v[u][1] = x.y; v[u][2] = x.z; v[u][3] = x.w;
        } else {
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) v[u][e] = (idx + e < end) ? __ldcs(rowp + idx + e) : -CUDART_INF_F;
        }
      }
      float bm = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) bm = fmaxf(bm, v[u][e]);

      if (first) {
        first = false;
        if (k <= 32) {
          // k distinct elements (k lane maxima) are >= the k-th largest lane maximum, so it
          // is a valid lower bound of this warp's k-th largest element.
          int rank = 0;
#pragma unroll
          for (int l = 0; l < 32; ++l) {
            const float o = __shfl_sync(FULL, bm, l);
            rank += (o > bm) || (o == bm && l < lane);
          }
          const unsigned pick = __ballot_sync(FULL, rank == k - 1);
          if (pick) thr0 = __shfl_sync(FULL, bm, __ffs(pick) - 1);
          thr_f = thr0;
        }
      }
      // running softmax normaliser of this thread's elements
      if (bm > m_t) {
        s_t *= exp2f((m_t - bm) * LOG2E_F);
        m_t = bm;
      }
      if (m_t > -CUDART_INF_F) {
        float acc = 0.f;
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) acc += exp2f((v[u][e] - m_t) * LOG2E_F);
        s_t += acc;
      }
      // top-k: almost never taken once the list is warm
      bool hit = false;
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) hit |= (v[u][e] >= thr_f);
      if (__any_sync(FULL, hit)) {
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u) {
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) {
            const int my_tok = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e;
            unsigned mk = __ballot_sync(FULL, v[u][e] >= thr_f && my_tok < end);
            while (mk) {
              const int src = __ffs(mk) - 1;
              mk &= mk - 1;
              const float val = __shfl_sync(FULL, v[u][e], src);
              const uint32_t tok = base + u * EXP_CHUNK_ALIGN + (warp * 32 + src) * EXP_VEC + e;
              list.insert(cand_key(val, tok), k, lane);
            }
            thr_f = list.thr ? fmaxf(thr0, key_logit(list.thr)) : thr0;
          }
        }
      }
    }

    // ---- CTA result of this chunk: 8 warp lists -> k keys, (max, sum) ----
    __syncthreads();   // s_lists / s_m may still be read by the previous item's merge
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) s_lists[warp * KCAP + s * 32 + lane] = list.key[s];
    float wm = m_t;
#pragma unroll
    for (int o = 16; o; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(FULL, wm, o));
    if (lane == 0) s_m[warp] = wm;
    __syncthreads();
    if (tid == 0) {
      float mm = s_m[0];
      for (int w = 1; w < EXP_WARPS; ++w) mm = fmaxf(mm, s_m[w]);
      s_bm = mm;
    }
    __syncthreads();
    const float bmx = s_bm;
    // thread partial rescaled to the block maximum; a NaN partial (NaN or +inf logit) propagates
    double part = (m_t > -CUDART_INF_F || s_t != s_t) ? (double)(s_t * exp2f((m_t - bmx) * LOG2E_F)) : 0.0;
#pragma unroll
    for (int o = 16; o; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
    if (lane == 0) s_s[warp] = part;

    const bool single = (g.splits == 1);
    unsigned long long *kout = single ? a.row_keys + (size_t)row * a.key_stride
                                      : a.part_keys + (size_t)item * a.key_stride;
    merge_sorted_lists(s_lists, EXP_WARPS, KCAP, k, kout);
    __syncthreads();
    if (tid == 0) {
      double tot = 0.0;
      for (int w = 0; w < EXP_WARPS; ++w) tot += s_s[w];
      if (single) {
        double lse = (double)bmx + log(tot);
        if (!(tot > 0.0) || !(bmx < CUDART_INF_F) || lse != lse) {
          lse = CUDART_NAN;
          atomicOr(a.status, STATUS_NONFINITE);
        }
        a.row_lse[row] = lse;
      } else {
        a.part_ms[item] = make_float2(bmx, (float)tot);
      }
    }
    if (single) continue;

    // ---- last chunk of the row merges the row ----
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned prev = atomicAdd(&a.row_count[row], 1u);
      s_last = (prev == (unsigned)g.splits - 1u);
      if (s_last) a.row_count[row] = 0u;          // ready for the next layer
    }
    __syncthreads();
    if (!s_last) continue;
    __threadfence();
    const size_t item0 = (size_t)row * g.splits;
    for (int idx = tid; idx < g.splits * k; idx += EXP_THREADS) {
      const int c = idx / k, p = idx - c * k;
      s_lists[c * KCAP + p] = __ldcg(a.part_keys + (item0 + c) * a.key_stride + p);
    }
    __syncthreads();
    merge_sorted_lists(s_lists, g.splits, KCAP, k, a.row_keys + (size_t)row * a.key_stride);
    if (warp == 0) {
      float2 ms = make_float2(-CUDART_INF_F, 0.f);
      if (lane < g.splits) ms = __ldcg(a.part_ms + item0 + lane);
      float mx = ms.x;
#pragma unroll
      for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
      double t = (lane < g.splits) ? ((ms.y != ms.y) ? (double)ms.y
                                                      : (ms.x > -CUDART_INF_F ? (double)ms.y * exp((double)ms.x - (double)mx) : 0.0))
                                    : 0.0;
#pragma unroll
      for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(FULL, t, o);
      if (lane == 0) {
        double lse = (double)mx + log(t);
        if (!(t > 0.0) || !(mx < CUDART_INF_F) || lse != lse) {
          lse = CUDART_NAN;
          atomicOr(a.status, STATUS_NONFINITE);
        }
        a.row_lse[row] = lse;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
// Selection: one CTA per sequence.
// ---------------------------------------------------------------------------------------
struct SelectArgs {
  talon_tree t;
  int lo_stride;
  int B, N, W, V, d, k, key_stride, target_items;
  int root_topk, init_layers;
  double log_mu;
  const unsigned long long *row_keys;
  const double *row_lse;
  int *status;
  int pool_cap;
};

__device__ inline unsigned long long f64_ord(double x) {
  unsigned long long b = (unsigned long long)__double_as_longlong(x);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}

// digit `pass` (0 = most significant byte) of the 96-bit composite (score, tie-break)
__device__ inline int composite_digit(unsigned long long hi, unsigned int lo, int pass) {
  if (pass < 8) return (int)((hi >> (56 - 8 * pass)) & 0xFF);
  return (int)((lo >> (24 - 8 * (pass - 8))) & 0xFF);
}

__global__ void __launch_bounds__(SEL_THREADS)
select_layer_kernel(SelectArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // pool arrays (pool_cap entries each)
  unsigned long long *c_ord = reinterpret_cast<unsigned long long *>(smem_raw);          // ordered score bits
  double *c_score = reinterpret_cast<double *>(c_ord + a.pool_cap);
  unsigned int *c_tie = reinterpret_cast<unsigned int *>(c_score + a.pool_cap);          // ~((j << 24) | tok)
  int *c_tok = reinterpret_cast<int *>(c_tie + a.pool_cap);
  unsigned char *c_state = reinterpret_cast<unsigned char *>(c_tok + a.pool_cap);       // bit0 eligible, bit1 alive, bit2 selected
  __shared__ int s_base[MAX_BATCH + 1];
  __shared__ int s_warp[SEL_THREADS / 32];
  __shared__ unsigned int s_hist[256];
  __shared__ unsigned long long s_anchor;
  __shared__ int s_cnt, s_need, s_bin, s_done, s_bad;
  __shared__ int s_rowcnt[MAX_BUDGET], s_rowoff[MAX_BUDGET];

  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x;
  frontier_scan<SEL_THREADS>(a.t.n_nodes, a.t.layer_off, a.lo_stride, a.B, a.N, a.d, s_base, s_warp);
  const int n = a.t.n_nodes[b];
  const int lo = a.t.layer_off[b * a.lo_stride + a.d];
  const int F = s_base[b + 1] - s_base[b];
  if (F <= 0) {          // full, finished or empty frontier: the layer is empty for this sequence
    if (tid == 0) a.t.layer_off[b * a.lo_stride + a.d + 2] = n;
    return;
  }
  const int R = a.N - n;                    // remaining budget
  const int ke = min(a.k, R);               // a parent can place at most R children
  const int C = F * ke;
  const int row0 = s_base[b];

  if (tid == 0) { s_anchor = 0ull; s_cnt = 0; s_bad = 0; }
  for (int i = tid; i < F; i += SEL_THREADS) s_rowcnt[i] = 0;
  __syncthreads();

  // ---- pool: log p(u) = log p(v) + (z_w - lse_v)   (Eq. 2-3) ----
  for (int c = tid; c < C; c += SEL_THREADS) {
    const int j = c / ke, i = c - j * ke;
    const unsigned long long key = a.row_keys[(size_t)(row0 + j) * a.key_stride + i];
    const double lse = a.row_lse[row0 + j];
    double s = -CUDART_INF;
    int tok = -1;
    if (lse != lse) s_bad = 1;
    if (key != 0ull) {
      tok = (int)key_tok(key);
      s = a.t.score[(size_t)b * a.N + lo + j] + ((double)key_logit(key) - lse);
    }
    const bool ok = (key != 0ull) && (s > -CUDART_INF) && (s == s);
    c_score[c] = s;
    c_tok[c] = tok;
    c_ord[c] = ok ? f64_ord(s) : 0ull;
    c_tie[c] = 0xFFFFFFFFu - (((unsigned)j << 24) | (unsigned)(tok & 0xFFFFFF));
    c_state[c] = ok ? 1 : 0;
    if (ok) atomicMax(&s_anchor, f64_ord(s));
  }
  __syncthreads();
  if (s_bad) {            // a frontier row was not finite: this sequence adds nothing
    if (tid == 0) a.t.layer_off[b * a.lo_stride + a.d + 2] = n;
    return;
  }

  // ---- eligibility: Top-K layers take every valid candidate, gated layers Eq. 4 ----
  const bool init = a.d < a.init_layers;
  double thr = -CUDART_INF;
  if (!init && s_anchor != 0ull) {
    const unsigned long long ab = s_anchor;
    const unsigned long long bits = (ab >> 63) ? (ab & 0x7FFFFFFFFFFFFFFFull) : ~ab;
    thr = a.log_mu + __longlong_as_double((long long)bits);
  }
  int local = 0;
  for (int c = tid; c < C; c += SEL_THREADS) {
    unsigned char st = c_state[c];
    if (st && !init && !(c_score[c] >= thr)) st = 0;
    c_state[c] = st ? 3 : 0;     // eligible + alive
    local += st ? 1 : 0;
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) local += __shfl_xor_sync(FULL, local, o);
  if (lane == 0 && local) atomicAdd(&s_cnt, local);
  __syncthreads();
  const int eligible = s_cnt;
  int want = init ? min(a.root_topk, R) : R;
  const int n_sel = min(eligible, want);

  if (eligible <= want) {
    for (int c = tid; c < C; c += SEL_THREADS) if (c_state[c]) c_state[c] = 5;   // all selected
  } else {
    // ---- radix select of the n_sel best composites (score desc, parent asc, token asc) ----
    if (tid == 0) { s_need = n_sel; s_done = 0; }
    __syncthreads();
    for (int pass = 0; pass < 12; ++pass) {
      if (tid < 256) s_hist[tid] = 0;
      __syncthreads();
      for (int c = tid; c < C; c += SEL_THREADS)
        if (c_state[c] & 2) atomicAdd(&s_hist[composite_digit(c_ord[c], c_tie[c], pass)], 1u);
      __syncthreads();
      if (warp == 0) {
        // bins 255 down to 0; lane l owns bins 255-8l .. 248-8l
        unsigned h[8];
        unsigned sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { h[i] = s_hist[255 - (lane * 8 + i)]; sum += h[i]; }
        unsigned inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          unsigned t = __shfl_up_sync(FULL, inc, o);
          if (lane >= o) inc += t;
        }
        unsigned run = inc - sum;          // keys in bins above this lane's bins
        const unsigned need = (unsigned)s_need;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          if (run < need && run + h[i] >= need) {
            s_bin = 255 - (lane * 8 + i);
            s_need = (int)(need - run);    // still to take from inside this bin
            s_done = (h[i] == need - run);
          }
          run += h[i];
        }
      }
      __syncthreads();
      const int bin = s_bin, done = s_done;
      for (int c = tid; c < C; c += SEL_THREADS) {
        unsigned char st = c_state[c];
        if (st & 2) {
          const int dg = composite_digit(c_ord[c], c_tie[c], pass);
          if (dg > bin) st = 5;                       // selected, no longer alive
          else if (dg < bin) st = 1;                  // out
          else if (done) st = 5;
          c_state[c] = st;
        }
      }
      __syncthreads();
      if (done) break;
    }
  }
  __syncthreads();

  // ---- append in storage order: (parent asc, token asc) ----
  for (int c = tid; c < C; c += SEL_THREADS)
    if (c_state[c] & 4) atomicAdd(&s_rowcnt[c / ke], 1);
  __syncthreads();
  if (warp == 0) {
    int v[4], sum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) { int jj = lane * 4 + i; v[i] = jj < F ? s_rowcnt[jj] : 0; sum += v[i]; }
    int inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int t = __shfl_up_sync(FULL, inc, o);
      if (lane >= o) inc += t;
    }
    int run = inc - sum;
#pragma unroll
    for (int i = 0; i < 4; ++i) { int jj = lane * 4 + i; if (jj < F) s_rowoff[jj] = run; run += v[i]; }
  }
  __syncthreads();
  for (int c = tid; c < C; c += SEL_THREADS) {
    if (!(c_state[c] & 4)) continue;
    const int j = c / ke;
    const int tok = c_tok[c];
    int r = 0;
    for (int i = 0; i < ke; ++i) {
      const int o = j * ke + i;
      r += ((c_state[o] & 4) && c_tok[o] < tok) ? 1 : 0;
    }
    const int node = n + s_rowoff[j] + r;
    const int par = lo + j;
    const size_t nb = (size_t)b * a.N;
    a.t.token[nb + node] = tok;
    a.t.parent[nb + node] = par;
    a.t.depth[nb + node] = a.d + 1;
    a.t.score[nb + node] = c_score[c];
    for (int w = 0; w < a.W; ++w) {
      unsigned long long m = a.t.mask[(nb + par) * a.W + w];
      if ((node >> 6) == w) m |= 1ull << (node & 63);
      a.t.mask[(nb + node) * a.W + w] = m;
    }
  }
  if (tid == 0) {
    a.t.n_nodes[b] = n + n_sel;
    a.t.layer_off[b * a.lo_stride + a.d + 2] = n + n_sel;
  }
}

// ---------------------------------------------------------------------------------------
// Reset and closing pass.
// ---------------------------------------------------------------------------------------
__global__ void reset_kernel(talon_tree t, const int32_t *root_tok, const int32_t *prefix_len,
                             int32_t *prefix_copy, int B, int N, int W, int lo_stride, int *status,
                             unsigned int *row_count, int rows_cap, unsigned int *seq_count) {
  pdl_enter();
  const int gid = blockIdx.x * blockDim.x + threadIdx.x;
  const int stride = gridDim.x * blockDim.x;
  if (gid == 0) *status = 0;
  for (int i = gid; i < rows_cap; i += stride) row_count[i] = 0u;
  for (int i = gid; i < B; i += stride) seq_count[i] = 0u;
  for (int b = gid; b < B; b += stride) {
    const size_t nb = (size_t)b * N;
    t.n_nodes[b] = 1;
    t.token[nb] = root_tok[b];
    t.parent[nb] = -1;
    t.depth[nb] = 0;
    t.score[nb] = 0.0;
    for (int w = 0; w < W; ++w) t.mask[nb * W + w] = (w == 0) ? 1ull : 0ull;
    t.layer_off[b * lo_stride] = 0;
    t.layer_off[b * lo_stride + 1] = 1;
    prefix_copy[b] = prefix_len[b];
  }
}

__global__ void build_tree_kernel(talon_tree t, const int32_t *prefix_len, uint8_t *dense, int B, int N,
                                  int W, int lo_stride, int layers_run) {
  pdl_enter();
  const int b = blockIdx.x;
  const int n = t.n_nodes[b];
  const size_t nb = (size_t)b * N;
  const int L = prefix_len[b];
  for (int i = threadIdx.x; i < N; i += blockDim.x) {
    if (i < n) {
      t.position[nb + i] = L + t.depth[nb + i];
    } else {
      t.token[nb + i] = -1;
      t.parent[nb + i] = -1;
      t.depth[nb + i] = -1;
      t.position[nb + i] = -1;
      t.score[nb + i] = -CUDART_INF;
      for (int w = 0; w < W; ++w) t.mask[(nb + i) * W + w] = ((i >> 6) == w) ? (1ull << (i & 63)) : 0ull;
    }
  }
  for (int i = layers_run + 2 + threadIdx.x; i < lo_stride; i += blockDim.x) t.layer_off[b * lo_stride + i] = n;
  if (dense) {
    __syncthreads();
    for (int e = threadIdx.x; e < N * N; e += blockDim.x) {
      const int i = e / N, j = e - i * N;
      dense[(size_t)b * N * N + e] = (uint8_t)((t.mask[(nb + i) * W + (j >> 6)] >> (j & 63)) & 1ull);
    }
  }
}

// Last step of Algorithm 1 (static tree construction): T <- Top-N(T by p(u)).  One CTA per
// sequence, one thread per node.  A node's rank is the number of nodes with a larger score, or
// the same score and a lower index, so a kept node's parent (score at least as large, index
// lower) is kept too; the survivors keep their order, parents and mask bits are renumbered, the
// layer offsets recounted.  Slots past the new size are left to talon_build_tree.
__global__ void __launch_bounds__(MAX_BUDGET)
prune_tree_kernel(talon_tree t, int B, int N, int W, int lo_stride, int keep) {
  __shared__ double s_score[MAX_BUDGET];
  __shared__ int s_new[MAX_BUDGET];          // new index of a kept node, -1 for a dropped one
  __shared__ int s_depth[MAX_BUDGET];
  __shared__ unsigned s_keep[MAX_BUDGET / 32];
  pdl_enter();
  const int b = blockIdx.x, i = threadIdx.x, lane = i & 31, warp = i >> 5;
  const int n = t.n_nodes[b];
  const size_t nb = (size_t)b * N;
  const bool live = i < n;
  const double sc = live ? t.score[nb + i] : -CUDART_INF;
  const int tok = live ? t.token[nb + i] : -1, par = live ? t.parent[nb + i] : -1, dep = live ? t.depth[nb + i] : -1;
  unsigned long long mk[2] = {0ull, 0ull};
  if (live)
    for (int w = 0; w < W; ++w) mk[w] = t.mask[(nb + i) * W + w];
  s_score[i] = sc;
  __syncthreads();
  int rank = 0;
  for (int j = 0; j < n; ++j) rank += (s_score[j] > sc || (s_score[j] == sc && j < i)) ? 1 : 0;
  const bool kept = live && rank < keep;
  const unsigned bal = __ballot_sync(0xFFFFFFFFu, kept);
  if (lane == 0) s_keep[warp] = bal;
  __syncthreads();
  int before = __popc(bal & ((1u << lane) - 1u));
  for (int w = 0; w < warp; ++w) before += __popc(s_keep[w]);
  int total = 0;
  for (int w = 0; w < MAX_BUDGET / 32; ++w) total += __popc(s_keep[w]);
  s_new[i] = kept ? before : -1;
  s_depth[i] = kept ? dep : 0x7FFFFFFF;
  __syncthreads();
  if (kept) {
    const int ni = before;
    t.token[nb + ni] = tok;
    t.parent[nb + ni] = par < 0 ? -1 : s_new[par];
    t.depth[nb + ni] = dep;
    t.score[nb + ni] = sc;
    unsigned long long nm[2] = {0ull, 0ull};
    for (int w = 0; w < W; ++w) {
      unsigned long long bits = mk[w];
      while (bits) {
        const int j = w * 64 + __ffsll((long long)bits) - 1;
        bits &= bits - 1ull;
        const int nj = s_new[j];
        if (nj >= 0) nm[nj >> 6] |= 1ull << (nj & 63);
      }
    }
    for (int w = 0; w < W; ++w) t.mask[(nb + ni) * W + w] = nm[w];
  }
  // layer_off[d] = kept nodes of depth < d (kept nodes stay sorted by depth)
  for (int d = i; d < lo_stride; d += MAX_BUDGET) {
    int c = 0;
    for (int j = 0; j < n; ++j) c += s_depth[j] < d ? 1 : 0;
    t.layer_off[b * lo_stride + d] = c;
  }
  if (i == 0) t.n_nodes[b] = total;
}

// ---------------------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------------------
talon_status launch_prune(talon_ctx *c, const talon_tree *t, int keep, cudaStream_t st) {
  LaunchTimer lt(c, TALON_K_BUILD, st);
  launch_kernel(c, prune_tree_kernel, dim3(c->B), dim3(MAX_BUDGET), 0, st, *t, c->B, c->p.budget, c->W,
                c->p.max_depth + 2, keep);
  c->launches += 1;
  return cudaGetLastError() == cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

static int frontier_upper_bound(const talon_ctx *c, int d) {
  // host-side bound on rows per sequence at layer d (the device knows the real sizes)
  long long f = 1;
  for (int i = 0; i < d; ++i) {
    long long w = (i < c->p.init_layers) ? c->p.root_topk : f * c->k_cap;
    f = w;
    if (f >= c->p.budget - 1) { f = c->p.budget - 1; break; }
  }
  if (f > c->p.budget - 1) f = c->p.budget - 1;
  if (f < 1) f = 1;
  return (int)f;
}

static size_t select_smem_bytes(int pool_cap) {
  return (size_t)pool_cap * (8 + 8 + 4 + 4 + 1) + 16;
}

static int pool_capacity(const talon_ctx *c) {
  // max over F of F * min(k, N-1-F)
  int best = 1;
  for (int f = 1; f <= c->p.budget - 1; ++f) {
    int r = c->p.budget - 1 - f;
    if (f == 1) r = c->p.budget - 1;
    int ke = c->k_cap < r ? c->k_cap : r;
    if (f * ke > best) best = f * ke;
  }
  return ((best + 15) / 16) * 16;
}

talon_status launch_reset(talon_ctx *c, const talon_tree *t, const int32_t *root_tok,
                          const int32_t *prefix_len, int B, cudaStream_t st) {
  const int threads = 256;
  int blocks = (c->rows_cap + threads - 1) / threads;
  if (blocks > 64) blocks = 64;
  if (blocks < 1) blocks = 1;
  LaunchTimer lt(c, TALON_K_RESET, st);
  launch_kernel(c, reset_kernel, dim3(blocks), dim3(threads), 0, st, *t, root_tok, prefix_len, c->d_prefix_len, B,
                c->p.budget, c->W, c->p.max_depth + 2, c->d_status, c->d_row_count, c->rows_cap, c->d_seq_count);
  c->launches += 1;
  return cudaGetLastError() == cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

talon_status launch_expand(talon_ctx *c, const talon_tree *t, const float *logits, int64_t row_stride,
                           int rows_per_seq, int layout, cudaStream_t st) {
  const int d = c->layers_run;
  const int fub = frontier_upper_bound(c, d);
  if (c->k_cap <= 32)
    return launch_expand_fused(c, t, logits, row_stride, rows_per_seq, layout, c->B * fub, st);
  long long max_items = (long long)c->B * fub * EXP_MAX_SPLITS;
  int grid = c->exp_grid;
  if (max_items < grid) grid = (int)max_items;
  if (grid < 1) grid = 1;

  ExpandArgs ea;
  ea.logits = logits; ea.row_stride = row_stride; ea.rows_per_seq = rows_per_seq; ea.layout = layout;
  ea.n_nodes = t->n_nodes; ea.layer_off = t->layer_off; ea.lo_stride = c->p.max_depth + 2;
  ea.B = c->B; ea.N = c->p.budget; ea.V = c->p.vocab; ea.d = d; ea.k = c->k_cap;
  ea.key_stride = c->key_stride; ea.target_items = grid;
  ea.part_keys = c->d_part_keys; ea.part_ms = c->d_part_ms; ea.row_keys = c->d_row_keys;
  ea.row_lse = c->d_row_lse; ea.row_count = c->d_row_count; ea.status = c->d_status;
  const size_t lists_bytes = (size_t)EXP_MAX_SPLITS * 32 * c->k_slots * sizeof(unsigned long long);
  {
    LaunchTimer lt(c, TALON_K_EXPAND_ROWS, st);
    switch (c->k_slots) {
      case 1: launch_kernel(c, expand_rows_kernel<1>, dim3(grid), dim3(EXP_THREADS), lists_bytes, st, ea); break;
      case 2: launch_kernel(c, expand_rows_kernel<2>, dim3(grid), dim3(EXP_THREADS), lists_bytes, st, ea); break;
      default: launch_kernel(c, expand_rows_kernel<4>, dim3(grid), dim3(EXP_THREADS), lists_bytes, st, ea); break;
    }
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;

  SelectArgs sa;
  sa.t = *t; sa.lo_stride = c->p.max_depth + 2;
  sa.B = c->B; sa.N = c->p.budget; sa.W = c->W; sa.V = c->p.vocab; sa.d = d; sa.k = c->k_cap;
  sa.key_stride = c->key_stride; sa.target_items = grid;
  sa.root_topk = c->p.root_topk; sa.init_layers = c->p.init_layers; sa.log_mu = c->log_mu;
  sa.row_keys = c->d_row_keys; sa.row_lse = c->d_row_lse; sa.status = c->d_status;
  sa.pool_cap = pool_capacity(c);
  {
    LaunchTimer lt(c, TALON_K_SELECT, st);
    launch_kernel(c, select_layer_kernel, dim3(c->B), dim3(SEL_THREADS), select_smem_bytes(sa.pool_cap), st, sa);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 2;
  return TALON_OK;
}

talon_status launch_build(talon_ctx *c, const talon_tree *t, uint8_t *dense, cudaStream_t st) {
  LaunchTimer lt(c, TALON_K_BUILD, st);
  launch_kernel(c, build_tree_kernel, dim3(c->B), dim3(128), 0, st, *t, c->d_prefix_len, dense, c->B, c->p.budget,
                c->W, c->p.max_depth + 2, c->layers_run);
  c->launches += 1;
  return cudaGetLastError() == cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

// one-time kernel attribute setup (dynamic shared memory above 48 KB)
talon_status expand_setup(talon_ctx *c) {
  const size_t lists_bytes = (size_t)EXP_MAX_SPLITS * 32 * c->k_slots * sizeof(unsigned long long);
  cudaError_t e = cudaSuccess;
  if (c->k_slots == 1) e = cudaFuncSetAttribute(expand_rows_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lists_bytes);
  else if (c->k_slots == 2) e = cudaFuncSetAttribute(expand_rows_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lists_bytes);
  else e = cudaFuncSetAttribute(expand_rows_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lists_bytes);
  if (e != cudaSuccess) return TALON_ERR_CUDA;
  e = cudaFuncSetAttribute(select_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)select_smem_bytes(pool_capacity(c)));
  return e == cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

}  // namespace talon

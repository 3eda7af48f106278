// Adaptive draft-tree expansion (Algorithm 2 of the paper; Eq. 2-5) as ONE kernel per layer,
// for per-parent candidate caps k <= 32 (the usual case: the paper's K is 10).
//
// Streaming phase.  The frontier's fp32 logit rows are cut into equal chunks, one CTA per chunk
// at a time.  In a single read of its chunk a CTA produces the chunk's share of the softmax
// normaliser of Eq. 3 (maximum and sum of exponentials) and the chunk's k largest logits with
// their token ids.
//   * A chunk of at most 4096 elements sits in registers (16 per thread).  The smallest of the
//     256/G maxima of G-lane groups bounds the chunk's k-th largest element from below (the
//     groups hold 256/G >= k different elements that large), so only elements at or above it
//     go to a shared pool, which is then ranked by counting.
//   * A longer chunk is streamed tile by tile; each warp keeps a sorted list of its best k
//     keys across its lanes plus a queue of elements that passed the current threshold, and a
//     full queue is folded into the list with a bitonic sort and merge.
//
// Selection phase.  The CTA that finishes the last chunk of a sequence merges that sequence's
// chunk results into per-row top-k lists and log-sum-exps, scores the pooled candidates with
// log p(u) = log p(v) + log P(w | v) (Eq. 2-3), applies Top-K (Eq. 5) or the confidence gate
// p(u) >= mu * max p (Eq. 4), truncates to the remaining budget, and appends the survivors with
// parent links, depths, scores and ancestor-mask rows.  Nothing returns to the host in between.
#include <cuda/atomic>
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr float LOG2E_F = 1.4426950408889634f;
typedef unsigned long long u64;

struct FusedArgs {
  const float *logits;
  int64_t row_stride;
  int rows_per_seq, layout;
  talon_tree t;
  int lo_stride;
  int B, N, W, V, d, k, key_stride, target_items, max_splits, items_cap;
  int root_topk, init_layers;
  double log_mu;
  u64 *part_keys;          // [items, key_stride]  per-chunk top-k, descending
  float2 *part_ms;         // [items]              per-chunk (max, sum of exp)
  unsigned int *seq_count; // [B]                  chunks finished per sequence (zero between layers)
  int *status;
};

// 2^x on the special-function unit (relative error about 2^-22, results below 2^-126 flush to 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// ---- bulk-copy ring: a longer chunk is brought in by the TMA engine, FX_RING tiles ahead ----
__device__ inline uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ inline void ring_bar_init(uint32_t bar) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
}
// Arms `bar` for `bytes` and starts the copy global -> shared (both 16-byte aligned, bytes a
// multiple of 16).  No multicast.
__device__ inline void ring_issue(uint32_t dst, const float *src, uint32_t bytes, uint32_t bar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(bar), "r"(bytes)
               : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Waits for the phase of `bar` with the given parity, for about two seconds at most.
__device__ inline bool ring_wait(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i) {
      uint32_t ok;
      // the hint lets the hardware park the thread until the phase completes (or ~20 us pass)
      asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.b32 %0, 1, 0, p;\n}"
                   : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
      if (ok) return true;
    }
    if (clock64() - t0 > 4000000000ll) return false;
  }
}

__device__ inline u64 shfl_u64(u64 v, int src) { return __shfl_sync(FULL, v, src); }
__device__ inline u64 shfl_xor_u64(u64 v, int m) { return __shfl_xor_sync(FULL, v, m); }
__device__ inline u64 umax64(u64 a, u64 b) { return a > b ? a : b; }
__device__ inline u64 umin64(u64 a, u64 b) { return a < b ? a : b; }

__device__ inline u64 warp_max_u64(u64 v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = umax64(v, shfl_xor_u64(v, o));
  return v;
}

// bitonic sort of one key per lane, descending by lane index
__device__ inline u64 warp_sort_desc(u64 x, int lane) {
#pragma unroll
  for (int sz = 2; sz <= 32; sz <<= 1) {
#pragma unroll
    for (int j = sz >> 1; j > 0; j >>= 1) {
      const u64 o = shfl_xor_u64(x, j);
      const bool keep_max = (((lane & j) == 0) == ((lane & sz) == 0));
      x = keep_max ? umax64(x, o) : umin64(x, o);
    }
  }
  return x;
}

// list (descending across lanes) <- the 32 largest of list U q, q unsorted
__device__ inline u64 warp_merge_desc(u64 list, u64 q, int lane) {
  q = warp_sort_desc(q, lane);
  u64 x = umax64(list, shfl_u64(q, 31 - lane));     // bitonic sequence holding the 32 largest
#pragma unroll
  for (int j = 16; j > 0; j >>= 1) {
    const u64 o = shfl_xor_u64(x, j);
    x = ((lane & j) == 0) ? umax64(x, o) : umin64(x, o);
  }
  return x;
}

// Folds the first 32 queued keys into the warp's list, moves the rest of the queue (up to
// FX_QCAP - 32 keys) to its front and raises the threshold to the list's k-th key.
__device__ __forceinline__ void fold_queue(u64 &list, int &qn, float &thr_f, u64 *queue, float thr0, int k,
                                           int lane) {
  list = warp_merge_desc(list, queue[lane], lane);
  const int rem = qn - 32;
  const u64 r0 = queue[32 + lane], r1 = queue[64 + lane], r2 = queue[96 + lane];
  __syncwarp();
  if (lane < rem) queue[lane] = r0;
  if (32 + lane < rem) queue[32 + lane] = r1;
  if (64 + lane < rem) queue[64 + lane] = r2;
  __syncwarp();
  qn = rem;
  const u64 kth = shfl_u64(list, k - 1);
  if (kth) thr_f = fmaxf(thr0, key_logit(kth));
}

// Makes a warp's threshold known to the other warps of the CTA (monotone: a maximum).
__device__ __forceinline__ void publish_thr(unsigned *thr_cta, float thr_f, int lane) {
  if (lane == 0 && thr_f > -CUDART_INF_F) atomicMax(thr_cta, f32_ord(thr_f));
}

// Folds a queue of fewer than 32 keys into the list (queue left empty).
__device__ __forceinline__ void flush_queue(u64 &list, int &qn, float &thr_f, const u64 *queue, float thr0, int k,
                                            int lane) {
  list = warp_merge_desc(list, lane < qn ? queue[lane] : 0ull, lane);
  qn = 0;
  const u64 kth = shfl_u64(list, k - 1);
  if (kth) thr_f = fmaxf(thr0, key_logit(kth));
}

// Exclusive scan of the per-sequence frontier sizes: s_base[b] = first packed row of sequence
// b, s_base[B] = total rows.  A sequence whose tree is full has no rows.
__device__ void frontier_bases(const FusedArgs &a, int *s_base, int *s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (a.B <= 32) {
    if (warp == 0) {
      int f = 0;
      if (lane < a.B && a.t.n_nodes[lane] < a.N) {
        f = a.t.layer_off[lane * a.lo_stride + a.d + 1] - a.t.layer_off[lane * a.lo_stride + a.d];
        f = max(f, 0);
      }
      int inc = f;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += t;
      }
      if (lane < a.B) s_base[lane] = inc - f;
      if (lane == a.B - 1) s_base[a.B] = inc;
    }
    __syncthreads();
    return;
  }
  constexpr int PER = (MAX_BATCH + EXP_THREADS - 1) / EXP_THREADS;
  int f[PER];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int b = tid * PER + i;
    int v = 0;
    if (b < a.B && a.t.n_nodes[b] < a.N) {
      v = a.t.layer_off[b * a.lo_stride + a.d + 1] - a.t.layer_off[b * a.lo_stride + a.d];
      v = max(v, 0);
    }
    f[i] = v;
    sum += v;
  }
  int inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < EXP_WARPS ? s_warp[lane] : 0;
    int winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL, winc, o);
      if (lane >= o) winc += t;
    }
    if (lane < EXP_WARPS) s_warp[lane] = winc - w;
    if (lane == EXP_WARPS - 1) s_base[a.B] = winc;
  }
  __syncthreads();
  int run = s_warp[warp] + inc - sum;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int b = tid * PER + i;
    if (b < a.B) s_base[b] = run;
    run += f[i];
  }
  __syncthreads();
}

__device__ inline int seq_of_row(const int *s_base, int B, int row) {
  int lo = 0, hi = B;   // s_base[lo] <= row < s_base[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s_base[mid] <= row) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ inline u64 f64_ord(double x) {
  const u64 b = (u64)__double_as_longlong(x);
  return (b >> 63) ? ~b : (b | 0x8000000000000000ull);
}
__device__ inline double f64_unord(u64 o) {
  const u64 b = (o >> 63) ? (o & 0x7FFFFFFFFFFFFFFFull) : ~o;
  return __longlong_as_double((long long)b);
}

// Chunks per row for this layer.  Every CTA of the grid is resident, so a layer takes
// ceil(items / grid) rounds of one chunk each: the cost of a candidate split count is
// rounds x (tiles per chunk + a fixed per-chunk overhead of about two tiles).  Chunks of one
// row are equal up to rounding to 4 elements (rows are 16-byte aligned), and a split row keeps
// at least 1024 elements per chunk so that every warp of a CTA holds some.  Lane l scores the
// split count l + 1; the warp keeps the cheapest (the smaller count on ties).
__device__ inline LayerGeom balanced_geom(int total_rows, int vocab, int grid, int max_splits, int items_cap) {
  const int lane = threadIdx.x & 31;
  unsigned best = 0xFFFFFFFFu;               // cost << 8 | splits
  if (total_rows > 0) {
    const int sp = lane + 1;
    int len = (((vocab + sp - 1) / sp) + 3) & ~3;
    const int eff = (vocab + len - 1) / len;
    const bool fits = sp == 1 || (sp <= max_splits && len >= 1024 && (long long)total_rows * eff <= items_cap);
    if (fits) {
      const int rounds = (total_rows * eff + grid - 1) / grid;
      const unsigned cost = (unsigned)rounds * (unsigned)(2 * ((len + EXP_TILE - 1) / EXP_TILE) + 4);
      best = (min(cost, 0xFFFFFFu) << 8) | (unsigned)eff;
    }
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) best = min(best, __shfl_xor_sync(FULL, best, o));
  LayerGeom g;
  g.total_rows = total_rows;
  g.splits = total_rows > 0 ? (int)(best & 0xFFu) : 1;
  g.chunk_len = (((vocab + g.splits - 1) / g.splits) + 3) & ~3;
  g.splits = (vocab + g.chunk_len - 1) / g.chunk_len;
  return g;
}

// Where a packed frontier row lives: sequence, index inside that sequence's frontier, tree
// node, frontier size and first packed row of the sequence.
struct RowLoc { int b, j, node, F, row0; };

// Frontier geometry of the layer.  For B <= 32 every warp holds it in registers (lane b = sequence
// b) and needs no shared memory or barrier; larger batches use a block-wide scan.
struct Frontier {
  int base_l, f_l, lo_l;     // B <= 32: this lane's sequence
  int total;
  bool in_regs;
  const int *s_base;
};

__device__ inline RowLoc locate_row(const FusedArgs &a, const Frontier &fr, int row) {
  RowLoc r;
  const int lane = threadIdx.x & 31;
  if (fr.in_regs) {
    // the last sequence whose first row is <= row (bases never decrease, empty sequences share
    // their base with the next one)
    const unsigned m = __ballot_sync(FULL, lane < a.B && fr.base_l <= row);
    r.b = 31 - __clz(m);
    r.row0 = __shfl_sync(FULL, fr.base_l, r.b);
    r.F = __shfl_sync(FULL, fr.f_l, r.b);
    r.j = row - r.row0;
    r.node = __shfl_sync(FULL, fr.lo_l, r.b) + r.j;
  } else {
    r.b = seq_of_row(fr.s_base, a.B, row);
    r.row0 = fr.s_base[r.b];
    r.F = fr.s_base[r.b + 1] - r.row0;
    r.j = row - r.row0;
    r.node = a.t.layer_off[r.b * a.lo_stride + a.d] + r.j;
  }
  return r;
}

// Shared-memory carve-up of the selection phase.
struct TailSmem {
  u64 *stage;        // [EXP_WARPS][32 k + FX_SURV]  chunk lists of the row a warp is merging, survivors
  u64 *row_keys;     // [N-1][k]               per-row top-k keys, descending
  double *score;     // [N-1][k]               log p(u) of each pooled candidate
  double *row_t;     // [N-1]                  sum of exponentials relative to row_m
  double *row_ps;    // [N-1]                  log p(v) of the row's parent
  u64 *row_mask;     // [N-1][W]               ancestor mask of the row's parent
  float *row_m;      // [N-1]
  int *row_cnt, *row_off;   // [N-1]
  unsigned char *state;     // [N-1][k]        bit0 eligible, bit2 selected
};

// Leaves a frontier row's maximum m and sum of exponentials t for the scoring phase, which takes
// the logarithm once per candidate, in parallel (one thread taking it here would hold up its whole
// warp).  m + log t is a finite number exactly when m is finite and 0 < t < inf; anything else
// (a NaN or +inf logit, a row of -inf only) flags the sequence.
__device__ __forceinline__ void finish_row(const FusedArgs &a, const TailSmem &sm, int j, float m, double t,
                                           int *s_bad) {
  if (!(t > 0.0) || !(t < CUDART_INF) || !(m < CUDART_INF_F) || !(m > -CUDART_INF_F)) {
    *s_bad = 1;
    atomicOr(a.status, STATUS_NONFINITE);
  }
  sm.row_m[j] = m;
  sm.row_t[j] = t;
  sm.row_cnt[j] = 0;
}

__device__ void select_tail(const FusedArgs &a, const TailSmem &sm, int b, int lo, int row0, int F, int S,
                            u64 *s_anchor, int *s_cnt, int *s_bad) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = a.k, ks = a.key_stride;
  const int n = a.t.n_nodes[b];
  const int R = a.N - n;
  const int ke = min(k, R);                 // a parent can place at most R children
  const size_t nb = (size_t)b * a.N;

  // ---- per row: chunk normalisers -> (max, sum); chunk lists -> the row's k best keys.
  // One warp per row, one lane per chunk (S <= 32). ----
  const int stage_words = 32 * k + FX_SURV;
  // Many rows means few chunks per row (their product is bounded by the grid): then all rows
  // are merged at once, one thread per key, instead of a row at a time per warp.  Up to two
  // rounds of the warp-per-row merge measured faster than the flat one (10 rows x 8 chunks:
  // 4 us per layer), hence the bound on F.
  const bool flat = S > 1 && S <= 8 && F > 2 * EXP_WARPS && F * S * k <= EXP_WARPS * stage_words;
  if (flat) {
    const size_t item0 = (size_t)row0 * S;
    u64 *st = sm.stage;                           // st[(j * S + c) * k + i]
    const int nkeys = F * S * k;
    // The compiler cannot move a global load above a store through a shared-memory pointer it
    // cannot tell apart, so every round of loads goes to registers before anything is stored:
    // one trip to L2 per round instead of one per load.
    auto key_at = [&](int idx) {
      const int jc = idx / k, i = idx - jc * k;
      return __ldcg(a.part_keys + (item0 + jc) * ks + i);
    };
    const u64 key_first = tid < nkeys ? key_at(tid) : 0ull;
    if (tid < F) {
      const int j = tid;
      float2 ms[8];
#pragma unroll
      for (int c = 0; c < 8; ++c)
        ms[c] = c < S ? __ldcg(a.part_ms + item0 + (size_t)j * S + c) : make_float2(-CUDART_INF_F, 0.f);
      const double ps = a.t.score[nb + lo + j];
      u64 mk[4];
#pragma unroll
      for (int w = 0; w < 4; ++w) mk[w] = w < a.W ? a.t.mask[(nb + lo + j) * a.W + w] : 0ull;
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int c = 0; c < 8; ++c) mx = fmaxf(mx, ms[c].x);
      double t = 0.0;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (ms[c].y != ms[c].y) t += (double)ms[c].y;                     // NaN or +inf logit in the chunk
        else if (ms[c].x > -CUDART_INF_F) t += (double)ms[c].y * (double)exp2f((ms[c].x - mx) * LOG2E_F);
      }
      sm.row_ps[j] = ps;
#pragma unroll
      for (int w = 0; w < 4; ++w)
        if (w < a.W) sm.row_mask[j * a.W + w] = mk[w];
      for (int w = 4; w < a.W; ++w) sm.row_mask[j * a.W + w] = a.t.mask[(nb + lo + j) * a.W + w];
      finish_row(a, sm, j, mx, t, s_bad);
    }
    if (tid < nkeys) st[tid] = key_first;
    for (int idx = tid + EXP_THREADS; idx < nkeys; idx += 2 * EXP_THREADS) {
      const u64 k0 = key_at(idx);
      const u64 k1 = idx + EXP_THREADS < nkeys ? key_at(idx + EXP_THREADS) : 0ull;
      st[idx] = k0;
      if (idx + EXP_THREADS < nkeys) st[idx + EXP_THREADS] = k1;
    }
    for (int idx = tid; idx < F * k; idx += EXP_THREADS) sm.row_keys[idx] = 0ull;
    __syncthreads();
    // a key's rank in its row: its place in its own list plus, for every other chunk of the
    // row, how many of that chunk's keys beat it (keys are unique; lists are descending)
    for (int idx = tid; idx < nkeys; idx += EXP_THREADS) {
      const u64 key = st[idx];
      if (key == 0ull) continue;
      const int jc = idx / k, i = idx - jc * k;
      const int j = jc / S, c = jc - j * S;
      int rank = i;
      for (int o = 0; o < S; ++o) {
        if (o == c) continue;
        const u64 *lst = st + (size_t)(j * S + o) * k;
        int l = 0, h = k;
        while (l < h) {
          const int mid = (l + h) >> 1;
          if (lst[mid] > key) l = mid + 1; else h = mid;
        }
        rank += l;
      }
      if (rank < k) sm.row_keys[(size_t)j * k + rank] = key;
    }
  }
  for (int j = flat ? F : warp; j < F; j += EXP_WARPS) {
    const size_t item0 = (size_t)(row0 + j) * S;
    u64 *st = sm.stage + warp * stage_words;       // st[i * 32 + c] = i-th best key of chunk c
    u64 *sv = st + 32 * k;                         // keys that reach the bound
    u64 *rk = sm.row_keys + (size_t)j * k;
    // Everything this row needs from global memory goes to registers before the first store
    // (a load cannot pass a store through a pointer the compiler cannot tell apart): one trip
    // to L2 for the row, not one per load.
    const float2 ms = (lane < S) ? __ldcg(a.part_ms + item0 + lane) : make_float2(-CUDART_INF_F, 0.f);
    const double ps = lane == 0 ? a.t.score[nb + lo + j] : 0.0;
    const u64 pmask = lane < a.W ? a.t.mask[(nb + lo + j) * a.W + lane] : 0ull;
    if (S == 1) {
      const u64 key = lane < k ? __ldcg(a.part_keys + item0 * ks + lane) : 0ull;
      if (lane < k) rk[lane] = key;
    } else {
      const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(a.part_keys + (item0 + min(lane, S - 1)) * ks);
      for (int i0 = 0; i0 < k; i0 += 16) {         // slots k..ks-1 of a list always hold zero
        ulonglong2 x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          x[u] = (lane < S && i0 + 2 * u < k) ? __ldcg(src + i0 / 2 + u) : make_ulonglong2(0ull, 0ull);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int i = i0 + 2 * u;
          if (lane < S && i < k) st[i * 32 + lane] = x[u].x;
          if (lane < S && i + 1 < k) st[(i + 1) * 32 + lane] = x[u].y;
        }
      }
    }
    if (lane == 0) sm.row_ps[j] = ps;
    if (lane < a.W) sm.row_mask[j * a.W + lane] = pmask;

    float mx = ms.x;
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
    double t = 0.0;
    if (ms.y != ms.y) t = (double)ms.y;                                   // NaN or +inf logit in the chunk
    else if (ms.x > -CUDART_INF_F) t = (double)ms.y * (double)exp2f((ms.x - mx) * LOG2E_F);
#pragma unroll
    for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(FULL, t, o);
    if (lane == 0) finish_row(a, sm, j, mx, t, s_bad);
    if (S == 1) continue;

    if (lane < k) rk[lane] = 0ull;
    // Two lower bounds of the row's k-th best key: the best k-th key of any one chunk, and the
    // k-th best of the chunk heads (k different chunks each hold a key at least that large).
    const u64 head = lane < S ? st[lane] : 0ull;
    u64 tau = lane < S ? st[(k - 1) * 32 + lane] : 0ull;
    if (S >= k) {
      int cnt = 0;
#pragma unroll 8
      for (int o = 0; o < 32; ++o) cnt += (shfl_u64(head, o) > head) ? 1 : 0;
      if (cnt == k - 1) tau = umax64(tau, head);
    }
    tau = warp_max_u64(tau);
    // keys that reach the bound: lists are sorted, so the scan over list positions stops at the
    // first position where no chunk has one
    int ns = 0;
    for (int i = 0; i < k; ++i) {
      const u64 key = lane < S ? st[i * 32 + lane] : 0ull;
      const bool ok = key != 0ull && key >= tau;
      const unsigned mk = __ballot_sync(FULL, ok);
      if (mk == 0u) break;
      const int pos = ns + __popc(mk & ((1u << lane) - 1u));
      if (ok && pos < FX_SURV) sv[pos] = key;
      ns += __popc(mk);
    }
    __syncwarp();
    if (ns <= FX_SURV) {
      // rank by counting (keys are unique)
      for (int i = lane; i < ns; i += 32) {
        const u64 key = sv[i];
        int r = 0;
        for (int o = 0; o < ns; ++o) r += (sv[o] > key) ? 1 : 0;
        if (r < k) rk[r] = key;
      }
    } else {
      // many keys at the bound (equal logits): pop the largest head k times
      int p = 0;
      for (int r = 0; r < k; ++r) {
        const u64 cand = (lane < S && p < k) ? st[p * 32 + lane] : 0ull;
        const u64 best = warp_max_u64(cand);
        if (best == 0ull) break;
        if (cand == best) ++p;
        if (lane == 0) rk[r] = best;
      }
    }
    __syncwarp();
  }
  __syncthreads();

  if (*s_bad) {            // a frontier row was not finite: this sequence adds nothing
    if (tid == 0) a.t.layer_off[b * a.lo_stride + a.d + 2] = n;
    return;
  }

  // ---- pool: log p(u) = log p(v) + (z_w - lse_v)   (Eq. 2-3) ----
  const int C = F * k;
  for (int c = tid; c < C; c += EXP_THREADS) {
    const int j = c / k, i = c - j * k;
    const u64 key = sm.row_keys[c];
    double s = -CUDART_INF;
    if (i < ke && key != 0ull) s = sm.row_ps[j] + ((double)key_logit(key) - ((double)sm.row_m[j] + log(sm.row_t[j])));
    const bool ok = (s > -CUDART_INF) && (s == s);
    if (!ok) s = -CUDART_INF;
    sm.score[c] = s;
    sm.state[c] = ok ? 1 : 0;
    if (ok && i == 0) atomicMax(s_anchor, f64_ord(s));        // rows are sorted: heads carry the maxima
  }
  __syncthreads();

  // ---- eligibility: Top-K layers take every candidate, gated layers Eq. 4 ----
  const bool init = a.d < a.init_layers;
  double thr = -CUDART_INF;
  if (!init && *s_anchor != 0ull) thr = a.log_mu + f64_unord(*s_anchor);
  int local = 0;
  for (int c = tid; c < C; c += EXP_THREADS) {
    unsigned char stt = sm.state[c];
    if (stt && !init && !(sm.score[c] >= thr)) stt = 0;
    sm.state[c] = stt;
    local += stt;
  }
#pragma unroll
  for (int o = 16; o; o >>= 1) local += __shfl_xor_sync(FULL, local, o);
  if (lane == 0 && local) atomicAdd(s_cnt, local);
  __syncthreads();
  const int eligible = *s_cnt;
  const int want = init ? min(a.root_topk, R) : R;
  const int n_sel = min(eligible, want);

  // ---- budget truncation: rank among all candidates by (score desc, parent asc, token asc).
  // Every row is sorted that way already, so a rank is a sum of binary searches. ----
  for (int c = tid; c < C; c += EXP_THREADS) {
    if (!sm.state[c]) continue;
    bool sel = true;
    if (eligible > want) {
      const int j = c / k, i = c - j * k;
      const double s = sm.score[c];
      int rank = i;
      for (int o = 0; o < F; ++o) {
        if (o == j) continue;
        const double *sc = sm.score + o * k;
        const bool before = o < j;
        int l = 0, h = ke;
        while (l < h) {
          const int mid = (l + h) >> 1;
          const double v = sc[mid];
          if (v > s || (v == s && before)) l = mid + 1; else h = mid;
        }
        rank += l;
      }
      sel = rank < want;
    }
    if (sel) {
      sm.state[c] = 5;
      atomicAdd(&sm.row_cnt[c / k], 1);
    }
  }
  __syncthreads();

  // ---- append in storage order: (parent asc, token asc) ----
  if (warp == 0) {
    int v[4], sum = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) { const int jj = lane * 4 + i; v[i] = jj < F ? sm.row_cnt[jj] : 0; sum += v[i]; }
    int inc = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL, inc, o);
      if (lane >= o) inc += t;
    }
    int run = inc - sum;
#pragma unroll
    for (int i = 0; i < 4; ++i) { const int jj = lane * 4 + i; if (jj < F) sm.row_off[jj] = run; run += v[i]; }
  }
  __syncthreads();
  for (int c = tid; c < C; c += EXP_THREADS) {
    if (!(sm.state[c] & 4)) continue;
    const int j = c / k;
    const int tok = (int)key_tok(sm.row_keys[c]);
    int r = 0;
    for (int i = 0; i < ke; ++i) {
      const int o = j * k + i;
      r += ((sm.state[o] & 4) && (int)key_tok(sm.row_keys[o]) < tok) ? 1 : 0;
    }
    const int node = n + sm.row_off[j] + r;
    a.t.token[nb + node] = tok;
    a.t.parent[nb + node] = lo + j;
    a.t.depth[nb + node] = a.d + 1;
    a.t.score[nb + node] = sm.score[c];
    for (int w = 0; w < a.W; ++w) {
      u64 m = sm.row_mask[j * a.W + w];
      if ((node >> 6) == w) m |= 1ull << (node & 63);
      a.t.mask[(nb + node) * a.W + w] = m;
    }
  }
  if (tid == 0) {
    a.t.n_nodes[b] = n + n_sel;
    a.t.layer_off[b * a.lo_stride + a.d + 2] = n + n_sel;
  }
}

// Per-warp state of the streamed top-k: a sorted list across the lanes (once something was
// folded), a queue in shared memory, and the threshold an element has to reach.
struct WarpTopk {
  u64 list;
  bool folded, first;
  int qn;
  float thr0, thr_f;
};

// One tile (16 elements per thread, already in registers) through the warp's threshold queue.
// bm is the thread's maximum over the tile.
__device__ __forceinline__ void topk_tile(const float (&v)[EXP_UNROLL][EXP_VEC], float bm, int base, int end, int k,
                                          u64 *queue, int *qcnt, unsigned *thr_cta, WarpTopk &w) {
  const int tid = threadIdx.x, lane = tid & 31;
  const bool was_first = w.first;
  if (w.first) {
    w.first = false;
    // k lane maxima are k distinct elements, so the k-th largest lane maximum is a lower
    // bound of this warp's k-th largest element: nothing below it needs to be looked at.
    int rank = 0;
#pragma unroll
    for (int l = 0; l < 32; ++l) {
      const float o = __shfl_sync(FULL, bm, l);
      rank += (o > bm) || (o == bm && l < lane);
    }
    const unsigned pick = __ballot_sync(FULL, rank == k - 1);
    if (pick) w.thr0 = __shfl_sync(FULL, bm, __ffs(pick) - 1);
    w.thr_f = w.thr0;
  }
  // A thread holds something at or above the threshold iff its maximum over the tile is: one
  // compare per tile.  The threshold is shared by the CTA's warps: whenever a warp sorts its
  // keys, its k-th best key is a lower bound of the chunk's k-th largest element for everybody.
  {
    const unsigned shared_thr = *thr_cta;
    if (shared_thr) w.thr_f = fmaxf(w.thr_f, f32_unord(shared_thr));
  }
  const bool hit = bm >= w.thr_f;
  const unsigned hm = __ballot_sync(FULL, hit);
  if (hm == 0u) return;
  if (__popc(hm) <= 6) {
    // a few lanes hold everything that reaches the threshold: only they look at their elements
    // (at most 6 x 16 new keys; fewer than 32 were waiting)
    if (lane == 0) *qcnt = w.qn;
    __syncwarp();
    if (hit) {
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) {
          const int tok = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e;
          if (v[u][e] >= w.thr_f && tok < end) queue[atomicAdd(qcnt, 1)] = cand_key(v[u][e], (uint32_t)tok);
        }
    }
    __syncwarp();
    w.qn = *qcnt;
    while (w.qn >= 32) { fold_queue(w.list, w.qn, w.thr_f, queue, w.thr0, k, lane); w.folded = true; publish_thr(thr_cta, w.thr_f, lane); }
    return;
  }
  int mine = 0;
#pragma unroll
  for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
    for (int e = 0; e < EXP_VEC; ++e)
      mine += (v[u][e] >= w.thr_f && base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e < end) ? 1 : 0;
  if (!__any_sync(FULL, mine > 0)) return;
  int inc = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  const int total = __shfl_sync(FULL, inc, 31);
  if (total <= 32) {
    int pos = w.qn + inc - mine;
#pragma unroll
    for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
      for (int e = 0; e < EXP_VEC; ++e) {
        const int tok = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e;
        if (v[u][e] >= w.thr_f && tok < end) queue[pos++] = cand_key(v[u][e], (uint32_t)tok);
      }
    w.qn += total;
    __syncwarp();
    if (w.qn >= 32) { fold_queue(w.list, w.qn, w.thr_f, queue, w.thr0, k, lane); w.folded = true; publish_thr(thr_cta, w.thr_f, lane); }
    else if (was_first && w.qn >= k) {
      // the first tile's bound is loose: sort what it let through so that the k-th best key of
      // this tile becomes the threshold for the next ones
      flush_queue(w.list, w.qn, w.thr_f, queue, w.thr0, k, lane);
      w.folded = true;
      publish_thr(thr_cta, w.thr_f, lane);
    }
  } else {
    // many elements at or above the threshold (equal logits, or a cold threshold): one
    // register slot at a time, folding whenever 32 keys are waiting
#pragma unroll
    for (int u = 0; u < EXP_UNROLL; ++u) {
#pragma unroll
      for (int e = 0; e < EXP_VEC; ++e) {
        const int tok = base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e;
        const bool ok = v[u][e] >= w.thr_f && tok < end;
        const unsigned mk = __ballot_sync(FULL, ok);
        if (mk == 0u) continue;
        if (ok) queue[w.qn + __popc(mk & ((1u << lane) - 1u))] = cand_key(v[u][e], (uint32_t)tok);
        w.qn += __popc(mk);
        __syncwarp();
        if (w.qn >= 32) { fold_queue(w.list, w.qn, w.thr_f, queue, w.thr0, k, lane); w.folded = true; publish_thr(thr_cta, w.thr_f, lane); }
      }
    }
  }
}

// The warp's best keys (list and queue) -> the CTA pool.
__device__ __forceinline__ void pool_from_warp(WarpTopk &w, u64 *queue, u64 *s_pool, int *s_pool_n, int k) {
  const int lane = threadIdx.x & 31;
  int cnt_w = w.qn;
  if (w.folded) {
    if (w.qn > 0) w.list = warp_merge_desc(w.list, lane < w.qn ? queue[lane] : 0ull, lane);
    cnt_w = __popc(__ballot_sync(FULL, lane < k && w.list != 0ull));
  }
  int pos = 0;
  if (lane == 0) pos = atomicAdd(s_pool_n, cnt_w);
  pos = __shfl_sync(FULL, pos, 0);
  if (lane < cnt_w) s_pool[pos + lane] = w.folded ? w.list : queue[lane];
}

__device__ __forceinline__ void load_tile(float (&v)[EXP_UNROLL][EXP_VEC], const float *rowp, int base, int end) {
  const int tid = threadIdx.x;
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
}

__global__ void __launch_bounds__(EXP_THREADS, 3)
expand_fused_kernel(FusedArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ u64 s_queue[EXP_WARPS][FX_QCAP];       // per-warp queues of keys above the threshold
  __shared__ u64 s_pool[FX_POOL];                   // the chunk's candidates, all warps
  __shared__ int s_base[MAX_BATCH + 1];
  __shared__ int s_warp[EXP_WARPS];
  __shared__ float s_m[EXP_WARPS], s_s[EXP_WARPS];
  __shared__ __align__(8) unsigned long long s_ring_bar[FX_RING];   // "tile landed" barriers
  __shared__ unsigned s_thr_cta;                    // ordered bits of the CTA-wide threshold (0: none yet)
  __shared__ int s_qn[EXP_WARPS];                   // queue fill, when lanes append on their own
  __shared__ float s_gmax[32];                      // maxima of lane groups (single-tile chunks)
  __shared__ u64 s_anchor;
  __shared__ int s_pool_n, s_last, s_cnt, s_bad;

  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = a.k;

  // ---- frontier geometry ----
  Frontier fr;
  fr.in_regs = a.B <= 32;
  fr.s_base = s_base;
  fr.base_l = fr.f_l = fr.lo_l = 0;
  if (fr.in_regs) {
    if (lane < a.B) {
      const int nn = a.t.n_nodes[lane];
      fr.lo_l = a.t.layer_off[lane * a.lo_stride + a.d];
      const int hi = a.t.layer_off[lane * a.lo_stride + a.d + 1];
      fr.f_l = nn < a.N ? max(hi - fr.lo_l, 0) : 0;
      if (fr.f_l == 0 && blockIdx.x == 0 && warp == 0)        // nothing to expand: close the layer
        a.t.layer_off[lane * a.lo_stride + a.d + 2] = nn;
    }
    int inc = fr.f_l;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(FULL, inc, o);
      if (lane >= o) inc += t;
    }
    fr.base_l = inc - fr.f_l;
    fr.total = __shfl_sync(FULL, inc, 31);
  } else {
    frontier_bases(a, s_base, s_warp);
    fr.total = s_base[a.B];
    if (blockIdx.x == 0)
      for (int b = tid; b < a.B; b += EXP_THREADS)
        if (s_base[b + 1] == s_base[b]) a.t.layer_off[b * a.lo_stride + a.d + 2] = a.t.n_nodes[b];
  }
  if (tid == 0) {
    s_pool_n = 0;
    s_thr_cta = 0u;
    for (int i = 0; i < FX_RING; ++i) ring_bar_init(smem_addr(&s_ring_bar[i]));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  unsigned ring_tiles = 0;         // tiles this CTA has taken from the ring so far (all threads agree)
  const LayerGeom g = balanced_geom(fr.total, a.V, a.target_items, a.max_splits, a.items_cap);
  const int n_items = fr.total * g.splits;
  // lanes per group whose maxima bound the k-th largest element of a single-tile chunk
  const int grp = k <= 8 ? 32 : (k <= 16 ? 16 : 8);
  __syncthreads();

  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int row = item / g.splits, chunk = item - row * g.splits;
    const RowLoc rl = locate_row(a, fr, row);
    int rsel = (a.layout == TALON_ROWS_BY_NODE) ? rl.node : rl.j;
    if (rsel >= a.rows_per_seq) {               // caller reserved too few rows: stay in bounds, report
      rsel = a.rows_per_seq - 1;
      if (tid == 0) atomicOr(a.status, STATUS_CAPACITY);
    }
    const float *rowp = a.logits + ((int64_t)rl.b * a.rows_per_seq + rsel) * a.row_stride;
    const int start = chunk * g.chunk_len;
    const int end = min(a.V, start + g.chunk_len);
    u64 *queue = s_queue[warp];
    float wm, ws;                    // this warp's maximum and sum of exponentials relative to it

    if (end - start <= EXP_TILE) {
      // ---- the whole chunk in registers ----
      float v[EXP_UNROLL][EXP_VEC];
      load_tile(v, rowp, start, end);
      float bm = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
        for (int e = 0; e < EXP_VEC; ++e) bm = fmaxf(bm, v[u][e]);
      float g8 = bm;
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) g8 = fmaxf(g8, __shfl_xor_sync(FULL, g8, o));
      const float g16 = fmaxf(g8, __shfl_xor_sync(FULL, g8, 8));
      wm = fmaxf(g16, __shfl_xor_sync(FULL, g16, 16));
      float acc = 0.f;
      if (wm > -CUDART_INF_F) {
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) acc += fast_exp2(fmaf(v[u][e], LOG2E_F, -wm * LOG2E_F));
      }
      ws = acc;
#pragma unroll
      for (int o = 16; o; o >>= 1) ws += __shfl_xor_sync(FULL, ws, o);
      if ((lane & (grp - 1)) == 0) s_gmax[(tid / grp)] = grp == 32 ? wm : (grp == 16 ? g16 : g8);
      if (lane == 0) { s_m[warp] = wm; s_s[warp] = ws; }
      __syncthreads();
      // the smallest group maximum: at least 256/grp >= k elements of the chunk reach it
      float tau = lane < EXP_THREADS / grp ? s_gmax[lane] : CUDART_INF_F;
#pragma unroll
      for (int o = 16; o; o >>= 1) tau = fminf(tau, __shfl_xor_sync(FULL, tau, o));
      // Only a thread whose own maximum reaches the bound holds candidates (about 8 H(8) = 22 of
      // the 256 do): those append to the CTA's pool themselves.  -inf never competes (probability
      // zero, and it is what the slots past `end` hold), so the bound is kept finite.
      const float tau_f = fmaxf(tau, -CUDART_MAX_NORMAL_F);
      if (bm >= tau_f) {
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e)
            if (v[u][e] >= tau_f) {
              const int pos = atomicAdd(&s_pool_n, 1);
              if (pos < FX_POOL)
                s_pool[pos] = cand_key(v[u][e], (uint32_t)(start + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e));
            }
      }
      __syncthreads();
      if (s_pool_n > FX_POOL) {
        // too many elements at the bound (equal logits, masked vocabulary, a tiny chunk): take
        // the per-warp queue route on the same registers
        __syncthreads();
        if (tid == 0) s_pool_n = 0;
        __syncthreads();
        WarpTopk w;
        w.list = 0ull; w.folded = false; w.first = true; w.qn = 0;
        w.thr0 = w.thr_f = -CUDART_INF_F;
        topk_tile(v, bm, start, end, k, queue, &s_qn[warp], &s_thr_cta, w);
        pool_from_warp(w, queue, s_pool, &s_pool_n, k);
        __syncthreads();
      }
    } else {
      // ---- a longer chunk, streamed tile by tile ----
      float m_t = -CUDART_INF_F, s_t = 0.f;
      WarpTopk w;
      w.list = 0ull; w.folded = false; w.first = true; w.qn = 0;
      w.thr0 = w.thr_f = -CUDART_INF_F;
      const int nt = (end - start + EXP_TILE - 1) / EXP_TILE;
      float *ring = reinterpret_cast<float *>(smem_raw);        // FX_RING tiles; the selection phase reuses it
      auto issue = [&](int t, unsigned slot_index) {
        const int base = start + t * EXP_TILE;
        const int n = min(EXP_TILE, end - base);
        const unsigned st = slot_index % FX_RING;
        // whole 16-byte units: the last one may reach into the row's stride padding
        ring_issue(smem_addr(ring + st * EXP_TILE), rowp + base, (uint32_t)(((n * 4) + 15) & ~15),
                   smem_addr(&s_ring_bar[st]));
      };
      if (tid == 0)
        for (int t = 0; t < nt && t < FX_RING; ++t) issue(t, ring_tiles + t);
      for (int t = 0; t < nt; ++t) {
        const int base = start + t * EXP_TILE;
        const unsigned st = ring_tiles % FX_RING;
        const bool landed = ring_wait(smem_addr(&s_ring_bar[st]), (ring_tiles / FX_RING) & 1u);
        float v[EXP_UNROLL][EXP_VEC];
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u) {
          const int off = u * EXP_CHUNK_ALIGN + tid * EXP_VEC;
          const float4 x = *reinterpret_cast<const float4 *>(ring + st * EXP_TILE + off);
          v[u][0] = x.x; v[u][1] = x.y; v[u][2] = x.z; v[u][3] = x.w;
        }
        if (base + EXP_TILE > end) {          // the chunk's last, partial tile: nothing past `end` counts
#pragma unroll
          for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
            for (int e = 0; e < EXP_VEC; ++e)
              if (base + u * EXP_CHUNK_ALIGN + tid * EXP_VEC + e >= end) v[u][e] = -CUDART_INF_F;
        }
        // every thread has its copy of the tile: the slot can take the tile FX_RING ahead
        if (!__syncthreads_and(landed)) {
          if (tid == 0) atomicOr(a.status, STATUS_TIMEOUT);
          return;
        }
        if (tid == 0 && t + FX_RING < nt) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          issue(t + FX_RING, ring_tiles + FX_RING);
        }
        ++ring_tiles;
        float bm = -CUDART_INF_F;
#pragma unroll
        for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
          for (int e = 0; e < EXP_VEC; ++e) bm = fmaxf(bm, v[u][e]);
        // running softmax normaliser of this thread's elements
        if (bm > m_t) {
          s_t *= fast_exp2((m_t - bm) * LOG2E_F);
          m_t = bm;
        }
        if (m_t > -CUDART_INF_F) {
          // exp(v - m) = 2^(v * log2e - m * log2e); an infinite m (a +inf logit) must give NaN
          const float c = -m_t * LOG2E_F;
          float acc = 0.f;
#pragma unroll
          for (int u = 0; u < EXP_UNROLL; ++u)
#pragma unroll
            for (int e = 0; e < EXP_VEC; ++e) acc += fast_exp2(fmaf(v[u][e], LOG2E_F, c));
          s_t += acc;
        }
        topk_tile(v, bm, base, end, k, queue, &s_qn[warp], &s_thr_cta, w);
      }
      pool_from_warp(w, queue, s_pool, &s_pool_n, k);
      wm = m_t;
#pragma unroll
      for (int o = 16; o; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(FULL, wm, o));
      // thread partial rescaled to the warp maximum; a NaN partial (NaN or +inf logit) propagates
      ws = (m_t > -CUDART_INF_F || s_t != s_t) ? s_t * exp2f((m_t - wm) * LOG2E_F) : 0.f;
#pragma unroll
      for (int o = 16; o; o >>= 1) ws += __shfl_xor_sync(FULL, ws, o);
      if (lane == 0) { s_m[warp] = wm; s_s[warp] = ws; }
      __syncthreads();
    }

    // ---- the chunk's k best keys: four lanes count each candidate's betters (keys are unique) ----
    const int nc = s_pool_n;
    for (int c0 = 0; c0 < nc; c0 += EXP_THREADS / 4) {
      const int ci = c0 + (tid >> 2), q = tid & 3;
      const u64 key = ci < nc ? s_pool[ci] : 0ull;
      int r = 0;
      for (int o = q; o < nc; o += 4) r += (s_pool[o] > key) ? 1 : 0;
      r += __shfl_xor_sync(FULL, r, 1);
      r += __shfl_xor_sync(FULL, r, 2);
      if (q == 0 && ci < nc && r < k) a.part_keys[(size_t)item * a.key_stride + r] = key;
    }
    if (tid >= nc && tid < k) a.part_keys[(size_t)item * a.key_stride + tid] = 0ull;
    if (warp == EXP_WARPS - 1) {
      const float mw = lane < EXP_WARPS ? s_m[lane] : -CUDART_INF_F;
      const float sw = lane < EXP_WARPS ? s_s[lane] : 0.f;
      float bmx = mw;
#pragma unroll
      for (int o = 4; o; o >>= 1) bmx = fmaxf(bmx, __shfl_xor_sync(FULL, bmx, o));
      float tot = (mw > -CUDART_INF_F || sw != sw) ? sw * exp2f((mw - bmx) * LOG2E_F) : 0.f;
#pragma unroll
      for (int o = 4; o; o >>= 1) tot += __shfl_xor_sync(FULL, tot, o);
      if (lane == 0) a.part_ms[item] = make_float2(bmx, tot);
    }

    // ---- the last chunk of a sequence runs that sequence's selection.  The barrier orders
    // this CTA's writes before thread 0's device-scope release; the last arrival acquires. ----
    __syncthreads();
    if (tid == 0) {
      s_pool_n = 0;
      s_thr_cta = 0u;
      s_anchor = 0ull; s_cnt = 0; s_bad = 0;        // the selection phase's accumulators
      cuda::atomic_ref<unsigned int, cuda::thread_scope_device> cnt(a.seq_count[rl.b]);
      const unsigned prev = cnt.fetch_add(1u, cuda::memory_order_acq_rel);
      s_last = (prev == (unsigned)(rl.F * g.splits) - 1u);
      if (s_last) cnt.store(0u, cuda::memory_order_relaxed);      // ready for the next layer
    }
    __syncthreads();
    if (!s_last) continue;
    TailSmem sm;
    const int rows_max = a.N - 1;
    unsigned char *p = smem_raw;
    sm.stage = reinterpret_cast<u64 *>(p);            p += sizeof(u64) * EXP_WARPS * (32 * k + FX_SURV);
    sm.row_keys = reinterpret_cast<u64 *>(p);         p += sizeof(u64) * rows_max * k;
    sm.score = reinterpret_cast<double *>(p);         p += sizeof(double) * rows_max * k;
    sm.row_t = reinterpret_cast<double *>(p);         p += sizeof(double) * rows_max;
    sm.row_ps = reinterpret_cast<double *>(p);        p += sizeof(double) * rows_max;
    sm.row_mask = reinterpret_cast<u64 *>(p);         p += sizeof(u64) * rows_max * a.W;
    sm.row_m = reinterpret_cast<float *>(p);          p += sizeof(float) * rows_max;
    sm.row_cnt = reinterpret_cast<int *>(p);          p += sizeof(int) * rows_max;
    sm.row_off = reinterpret_cast<int *>(p);          p += sizeof(int) * rows_max;
    sm.state = p;
    select_tail(a, sm, rl.b, rl.node - rl.j, rl.row0, rl.F, g.splits, &s_anchor, &s_cnt, &s_bad);
    __syncthreads();     // the next chunk's bulk copies land in the memory the selection phase just used
  }
}

size_t fused_smem_bytes(const talon_ctx *c) {
  const size_t rows = c->p.budget - 1, k = c->k_cap, W = c->W;
  const size_t tail = sizeof(u64) * EXP_WARPS * (32 * k + FX_SURV) + rows * k * (8 + 8 + 1) +
                      rows * (8 + 8 + 8 * W + 4 + 4 + 4) + 16;
  const size_t ring = sizeof(float) * FX_RING * EXP_TILE;       // the two phases share the space
  return tail > ring ? tail : ring;
}

}  // namespace

int fused_max_splits(int key_stride) {
  (void)key_stride;
  return FX_MAX_SPLITS;
}

talon_status expand_fused_setup(talon_ctx *c) {
  const size_t bytes = fused_smem_bytes(c);
  if (cudaFuncSetAttribute(expand_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) !=
      cudaSuccess)
    return TALON_ERR_CUDA;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, expand_fused_kernel, EXP_THREADS, bytes) !=
      cudaSuccess || per_sm < 1)
    return TALON_ERR_CUDA;
  if (per_sm > EXP_CTAS_PER_SM) per_sm = EXP_CTAS_PER_SM;
  c->fused_grid = c->sm_count * per_sm;
  return TALON_OK;
}

talon_status launch_expand_fused(talon_ctx *c, const talon_tree *t, const float *logits, int64_t row_stride,
                                 int rows_per_seq, int layout, int rows_bound, cudaStream_t st) {
  FusedArgs a;
  a.logits = logits; a.row_stride = row_stride; a.rows_per_seq = rows_per_seq; a.layout = layout;
  a.t = *t; a.lo_stride = c->p.max_depth + 2;
  a.B = c->B; a.N = c->p.budget; a.W = c->W; a.V = c->p.vocab; a.d = c->layers_run; a.k = c->k_cap;
  a.key_stride = c->key_stride;
  a.max_splits = fused_max_splits(c->key_stride);
  long long max_items = (long long)rows_bound * a.max_splits;
  int grid = c->fused_grid;
  if (max_items < grid) grid = (int)max_items;
  if (grid < 1) grid = 1;
  a.target_items = grid;
  a.items_cap = c->items_cap;
  a.root_topk = c->p.root_topk; a.init_layers = c->p.init_layers; a.log_mu = c->log_mu;
  a.part_keys = c->d_part_keys; a.part_ms = c->d_part_ms; a.seq_count = c->d_seq_count; a.status = c->d_status;
  {
    LaunchTimer lt(c, TALON_K_EXPAND_ROWS, st);
    launch_kernel(c, expand_fused_kernel, dim3(grid), dim3(EXP_THREADS), fused_smem_bytes(c), st, a);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  return TALON_OK;
}

}  // namespace talon

// Adaptive draft-tree expansion (Algorithm 2 of the paper; Eq. 2-5) as ONE kernel per layer,
// for per-parent candidate caps k <= 32 (the usual case: the paper's K is 10).
//
// Streaming phase.  The frontier's fp32 logit rows are cut into equal chunks, one CTA per chunk
// at a time, and a chunk into eight slices, one per warp.  A warp streams its slice on its own:
// 2 KB bulk copies (TMA, no multicast) into a private ring of shared-memory slots with private
// mbarriers, so no CTA-wide barrier sits on the streaming path.  In the single read of its slice
// a warp produces
//   * its share of the softmax normaliser of Eq. 3 (per-lane running maximum and sum of
//     exponentials), and
//   * an unsorted buffer of every element that reached the warp's threshold.  The threshold is a
//     lower bound of the row's k-th largest logit that only grows: the k-th largest of the 32
//     per-lane running maxima (k different elements that large have been seen), refreshed after
//     tiles 1, 2, 4, 8, ...; the smallest of the eight warps' ceil(k/8)-th largest lane maxima
//     (again k different elements); and, on gated layers, the running maximum plus ln(mu): by
//     Eq. 4 a candidate can only survive if its path score is within ln(mu) of the layer's best,
//     which is at least the best of its own row, so a logit more than |ln(mu)| below the row
//     maximum never matters.  Nothing is sorted while streaming; a buffer that fills up is cut
//     back to its k largest keys.
// At the end of a chunk the eight buffers meet in a CTA pool that is ranked by counting, and the
// chunk's k best keys and normaliser go to global memory.
//
// Selection phase.  Frontiers of at most eight rows: the CTA that finishes a sequence's last chunk
// merges that sequence's rows, one warp per row.  Wider frontiers: the CTA that finishes a row's
// last chunk merges that row (rows of one sequence finish all over the grid, so the merges run in
// parallel), and the CTA that finishes the sequence's last row collects the row results.  Either
// way that CTA then scores the pooled candidates with log p(u) = log p(v) + log P(w | v)
// (Eq. 2-3), applies Top-K (Eq. 5) or the confidence gate p(u) >= mu * max p (Eq. 4), truncates
// to the remaining budget, and appends the survivors with parent links, depths, scores and
// ancestor-mask rows.  Nothing returns to the host in between.
#include <cuda/atomic>
#include <math_constants.h>

#include "talon_internal.cuh"

namespace talon {

namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr float LOG2E_F = 1.4426950408889634f;
typedef unsigned long long u64;

constexpr int XS_WTILE = 512;                 // floats a warp takes per step: 16 per lane, one 2 KB copy
constexpr int XS_RING = 3;                    // copies in flight per warp
constexpr int XS_BUF = FX_QCAP;               // keys a warp's candidate buffer holds
constexpr int XS_POOL = 384;                  // keys the CTA pool holds
constexpr int XS_TWO_LEVEL = EXP_WARPS;       // frontiers wider than this merge their rows all over the grid
static_assert(XS_WTILE * EXP_WARPS == EXP_TILE, "a CTA step is eight warp tiles");
static_assert(XS_BUF >= 64 && XS_POOL >= EXP_WARPS * 32, "buffers must hold a cut-back list plus one ballot");

struct FusedArgs {
  const float *logits;
  int64_t row_stride;
  int rows_per_seq, layout;
  talon_tree t;
  int lo_stride;
  int B, N, W, V, d, k, key_stride, max_split, base_offset;
  int root_topk, init_layers;
  double log_mu;
  u64 *part_keys;          // [items, key_stride]  per-chunk top-k, descending
  float2 *part_ms;         // [items]              per-chunk (max, sum of exp)
  u64 *row_keys;           // [rows, key_stride]   per-row top-k (wide frontiers)
  double *row_score;       // [rows, key_stride]   log p(u) of those candidates; slot 0 NaN: row not finite
  unsigned int *row_count; // [rows]               chunks finished per row (zero between layers)
  unsigned int *seq_count; // [B]                  chunks or rows finished per sequence (zero between layers)
  int *status;
};

// 2^x on the special-function unit (relative error about 2^-22, results below 2^-126 flush to 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ u64 pack_f32x2(float lo, float hi) {
  u64 d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack_f32x2(u64 v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma_f32x2(u64 a, u64 b, u64 c) {
  u64 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ u64 add_f32x2(u64 a, u64 b) {
  u64 d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// ---- bulk-copy ring ----
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

// the same for one float per lane (NaN never appears: the inputs are maxima taken with fmaxf)
__device__ inline float warp_sort_desc_f32(float x, int lane) {
#pragma unroll
  for (int sz = 2; sz <= 32; sz <<= 1) {
#pragma unroll
    for (int j = sz >> 1; j > 0; j >>= 1) {
      const float o = __shfl_xor_sync(FULL, x, j);
      const bool keep_max = (((lane & j) == 0) == ((lane & sz) == 0));
      x = keep_max ? fmaxf(x, o) : fminf(x, o);
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

// Exclusive scan of the per-sequence frontier sizes: s_base[b] = first packed row of sequence
// b, s_base[B] = total rows.  A sequence whose tree is full has no rows.  The tree's size before
// this layer is layer_off[d + 1], which this launch never writes (n_nodes changes under it).
__device__ void frontier_bases(const FusedArgs &a, int *s_base, int *s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int PER = (MAX_BATCH + EXP_THREADS - 1) / EXP_THREADS;
  int f[PER];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < PER; ++i) {
    const int b = tid * PER + i;
    int v = 0;
    if (b < a.B) {
      const int lo = a.t.layer_off[b * a.lo_stride + a.d], hi = a.t.layer_off[b * a.lo_stride + a.d + 1];
      v = hi < a.N ? max(hi - lo, 0) : 0;
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

// How a layer is cut.  The frontier's rows are laid end to end on a line, `pitch` elements apart,
// and the CTAs of the grid take consecutive spans of `span` elements of that line (both multiples
// of four: rows are 16-byte aligned).
//   * Few rows (the grid holds at least two CTAs per row): a row is cut into S equal chunks, one
//     CTA each, S as large as the grid allows (at most FX_MAX_SPLITS - 1, at least 4096 elements
//     per chunk); pitch = S * span, so no span crosses a row.
//   * Many rows: pitch is the row length and every CTA takes the same share of the whole line, so
//     every CTA (and every SM) streams the same number of bytes whatever the number of rows; a span
//     that crosses a row boundary is worked off as one chunk per row it touches.
// Either way a row has at most FX_MAX_SPLITS chunks (one lane per chunk in the merge).  Chunk
// results live at index (CTA + packed row), which grows along the line; a row's chunks are
// consecutive there.
struct SpanGeom {
  unsigned span;       // elements of the line per CTA
  unsigned pitch;      // elements of the line per row (>= the row length)
  unsigned per_row;    // chunks per row when no span crosses a row, else 0
};

__device__ inline unsigned div_u64(unsigned long long a, unsigned b) {
  return a <= 0xFFFFFFFFull ? (unsigned)a / b : (unsigned)(a / b);
}

__device__ inline SpanGeom span_geom(int total_rows, int vocab, int grid, int max_split) {
  SpanGeom g;
  const unsigned vp = ((unsigned)vocab + 3u) & ~3u;
  const unsigned per_row = total_rows > 0 ? (unsigned)grid / (unsigned)total_rows : 1u;
  if (per_row >= 2u) {
    const unsigned S = max(1u, min(min(per_row, (unsigned)max_split), vp / 4096u));
    g.span = ((vp + S - 1u) / S + 3u) & ~3u;
    g.pitch = S * g.span;
    g.per_row = S;
  } else {
    const unsigned long long line = (unsigned long long)total_rows * vp;
    const unsigned span = (div_u64(line + grid - 1, (unsigned)grid) + 3u) & ~3u;
    const unsigned span_min = max(4096u, ((vp + FX_MAX_SPLITS - 2) / (FX_MAX_SPLITS - 1) + 3u) & ~3u);
    g.span = max(span, span_min);
    g.pitch = vp;
    g.per_row = 0u;
  }
  return g;
}

// First chunk-result index and number of chunks of packed row `row`.
__device__ inline void row_chunks(const SpanGeom &g, int row, int &item0, int &S) {
  if (g.per_row) {                       // equal chunks of whole rows: no division
    item0 = row * (int)g.per_row + row;
    S = (int)g.per_row;
    return;
  }
  const unsigned long long lo = (unsigned long long)row * g.pitch;
  const unsigned first = div_u64(lo, g.span), last = div_u64(lo + g.pitch - 1, g.span);
  item0 = (int)first + row;
  S = (int)(last - first) + 1;
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

// ---------------------------------------------------------------------------------------
// Streaming state of one warp
// ---------------------------------------------------------------------------------------
struct WarpStream {
  float m_t, s_t;        // this lane's running maximum and sum of exponentials relative to it
  float thr_f;           // an element below it cannot be among the row's k best (warp-uniform)
  u64 thr_key;           // after a cut-back: the buffer's k-th key; only larger keys enter (warp-uniform)
  int cnt;               // keys in the warp's buffer (warp-uniform)
};

// Cuts the warp's buffer back to its (at most) ke largest keys, sorted descending at the front,
// and raises the thresholds to the ke-th of them when there are that many.
struct CutBack { u64 thr_key; float thr_f; int cnt; };
__device__ __noinline__ CutBack cut_back_impl(u64 *buf, int ke, int n, float thr_f, u64 thr_key) {
  const int lane = threadIdx.x & 31;
  u64 list = 0ull;
  for (int off = 0; off < n; off += 32) list = warp_merge_desc(list, off + lane < n ? buf[off + lane] : 0ull, lane);
  __syncwarp();
  const bool keep = lane < ke && list != 0ull;
  if (keep) buf[lane] = list;
  CutBack r;
  r.cnt = __popc(__ballot_sync(FULL, keep));
  r.thr_key = thr_key;
  r.thr_f = thr_f;
  const u64 kth = shfl_u64(list, ke - 1);
  if (kth != 0ull) {
    r.thr_key = kth;
    r.thr_f = fmaxf(thr_f, key_logit(kth));
  }
  __syncwarp();
  return r;
}
__device__ __forceinline__ void cut_back(u64 *buf, int ke, WarpStream &w, int lane) {
  (void)lane;
  const CutBack r = cut_back_impl(buf, ke, w.cnt, w.thr_f, w.thr_key);
  w.cnt = r.cnt; w.thr_key = r.thr_key; w.thr_f = r.thr_f;
}

// Raises the warp's threshold from what it has seen so far (see the header of this file).
// s_wtop[w] holds warp w's (share_pos + 1)-th largest lane maximum, s_wmax[w] its largest.
__device__ __forceinline__ void refresh_threshold(WarpStream &w, int ke, int share_pos, bool gated, float ln_mu,
                                                  float *s_wtop, float *s_wmax, int lane, int warp, bool exact) {
  float cand, wmax, mine;
  if (share_pos == 0 && !exact) {
    // ke <= 8: the eight 4-lane groups hold eight different elements at least as large as the
    // smallest group maximum; the warp maximum is what the other warps get to see
    float g = fmaxf(w.m_t, __shfl_xor_sync(FULL, w.m_t, 1));
    g = fmaxf(g, __shfl_xor_sync(FULL, g, 2));
    float hi = g, lo = g;
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      hi = fmaxf(hi, __shfl_xor_sync(FULL, hi, o));
      lo = fminf(lo, __shfl_xor_sync(FULL, lo, o));
    }
    cand = lo; wmax = hi; mine = hi;
  } else {
    const float sorted = warp_sort_desc_f32(w.m_t, lane);
    cand = __shfl_sync(FULL, sorted, ke - 1);
    wmax = __shfl_sync(FULL, sorted, 0);
    mine = __shfl_sync(FULL, sorted, share_pos);
  }
  if (lane == 0) { s_wtop[warp] = mine; s_wmax[warp] = wmax; }
  __syncwarp();
  // eight warps x (share_pos + 1) lane maxima >= the smallest published value: at least ke elements
  float omin = lane < EXP_WARPS ? s_wtop[lane] : CUDART_INF_F;
  float omax = lane < EXP_WARPS ? s_wmax[lane] : -CUDART_INF_F;
#pragma unroll
  for (int o = 4; o; o >>= 1) {
    omin = fminf(omin, __shfl_xor_sync(FULL, omin, o));
    omax = fmaxf(omax, __shfl_xor_sync(FULL, omax, o));
  }
  omin = __shfl_sync(FULL, omin, 0);
  omax = fmaxf(wmax, __shfl_sync(FULL, omax, 0));
  cand = fmaxf(cand, omin);
  if (gated && omax > -CUDART_INF_F) {
    // fp32 rounding of the sum and of ln(mu), and the 1e-5 band around the gate, stay inside the slack
    cand = fmaxf(cand, omax + ln_mu - (1e-4f + 1e-6f * fabsf(omax)));
  }
  w.thr_f = fmaxf(w.thr_f, cand);
}

// Appends the elements of one tile that reach the threshold to the warp's buffer.  `slot` is the
// warp's copy of the tile in shared memory (still intact: it is refilled after this call), tok_tile
// the token id of its first element; lane l holds elements (i / 4) * 128 + l * 4 + i % 4 of it in v.
__device__ __forceinline__ void collect_tile(const float *slot, const float (&v)[16], int tok_tile, int ke, u64 *buf,
                                             WarpStream &w, int lane) {
  unsigned mm = 0u;
#pragma unroll
  for (int i = 0; i < 16; ++i)
    if (v[i] >= w.thr_f) mm |= 1u << i;
  const int c = __popc(mm);
  int inc = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(FULL, inc, o);
    if (lane >= o) inc += t;
  }
  const int total = __shfl_sync(FULL, inc, 31);
  if (w.cnt + total <= XS_BUF) {
    // the usual case: a handful of elements in a few lanes; each lane fetches its own from the
    // slot.  After a cut-back only keys above the buffer's k-th count: the others leave an empty
    // slot (key 0), which every reader of the buffer skips.
    int pos = w.cnt + inc - c;
    while (mm) {
      const int i = __ffs(mm) - 1;
      mm &= mm - 1u;
      const int e = (i >> 2) * 128 + lane * 4 + (i & 3);
      const u64 key = cand_key(slot[e], (uint32_t)(tok_tile + e));
      buf[pos++] = key > w.thr_key ? key : 0ull;
    }
    w.cnt += total;
    __syncwarp();
    if (w.cnt > XS_BUF - 32) cut_back(buf, ke, w, lane);
    return;
  }
  // More than the buffer holds (equal logits, a sorted row, a cold threshold): cut the buffer
  // back, then take the tile one register slot at a time, cutting back whenever a ballot's worth
  // might not fit.
  cut_back(buf, ke, w, lane);
#pragma unroll 1
  for (int i = 0; i < 16; ++i) {
    const int e = (i >> 2) * 128 + lane * 4 + (i & 3);
    const float x = slot[e];
    const u64 key = cand_key(x, (uint32_t)(tok_tile + e));
    bool ok = ((mm >> i) & 1u) && x >= w.thr_f && key > w.thr_key;
    unsigned mk = __ballot_sync(FULL, ok);
    if (mk == 0u) continue;
    if (w.cnt + __popc(mk) > XS_BUF) {
      cut_back(buf, ke, w, lane);
      ok = ok && x >= w.thr_f && key > w.thr_key;
      mk = __ballot_sync(FULL, ok);
    }
    if (ok) buf[w.cnt + __popc(mk & ((1u << lane) - 1u))] = key;
    w.cnt += __popc(mk);
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------------------
// Selection phase
// ---------------------------------------------------------------------------------------
// Shared-memory carve-up of the selection phase (it reuses the streaming ring).
struct TailSmem {
  u64 *stage;        // [EXP_WARPS][FX_MAX_SPLITS k + FX_SURV + k]  chunk lists of the row a warp is merging, survivors, result
  u64 *row_keys;     // [N-1][k]               per-row top-k keys, descending
  double *score;     // [N-1][k]               log p(u) of each pooled candidate
  u64 *row_mask;     // [N-1][W]               ancestor mask of the row's parent
  int *row_cnt, *row_off;   // [N-1]
  unsigned char *state;     // [N-1][k]        bit0 eligible, bit2 selected
};

__device__ inline int stage_words(int k) { return FX_MAX_SPLITS * k + FX_SURV + k; }

// One warp merges the S chunk results of the frontier row of tree node `node` (index into the
// [B, N] arrays).  Afterwards lane i < k holds the row's i-th best key and its score
// log p(v) + (z - lse) (Eq. 2-3; -inf for an empty slot or one past the ke children the budget
// still allows), and lane w < W word w of the parent's ancestor mask.  Returns false, for the whole warp, when the row's
// normaliser is not a positive finite number (a NaN or +inf logit, a row of -inf only).
__device__ __forceinline__ bool merge_row(const FusedArgs &a, size_t item0, int S, int k, int ke, size_t node, u64 *st,
                                          u64 &out_key, double &out_score, u64 &out_mask) {
  const int lane = threadIdx.x & 31;
  const int ks = a.key_stride;
  u64 *sv = st + FX_MAX_SPLITS * k;              // keys that reach the bound
  u64 *rk = sv + FX_SURV;                        // the row's k best keys
  // Everything this row needs from global memory goes to registers before the first store (a
  // load cannot pass a store through a pointer the compiler cannot tell apart): one trip to L2
  // for the row, not one per load.
  const float2 ms = (lane < S) ? __ldcg(a.part_ms + item0 + lane) : make_float2(-CUDART_INF_F, 0.f);
  const double ps = a.t.score[node];                                    // log p(v) of the row's parent
  out_mask = lane < a.W ? a.t.mask[node * a.W + lane] : 0ull;           // and its ancestor-mask row
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
        if (lane < S && i < k) st[i * FX_MAX_SPLITS + lane] = x[u].x;
        if (lane < S && i + 1 < k) st[(i + 1) * FX_MAX_SPLITS + lane] = x[u].y;
      }
    }
  }
  static_assert(FX_MAX_SPLITS <= 16, "the chunk statistics are reduced over 16 lanes");
  float mx = ms.x;                                                      // lanes >= S hold -inf and 0
#pragma unroll
  for (int o = 8; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
  mx = __shfl_sync(FULL, mx, 0);
  double t = 0.0;
  if (ms.y != ms.y) t = (double)ms.y;                                   // NaN or +inf logit in the chunk
  else if (ms.x > -CUDART_INF_F) t = (double)ms.y * (double)exp2f((ms.x - mx) * LOG2E_F);
#pragma unroll
  for (int o = 8; o; o >>= 1) t += __shfl_xor_sync(FULL, t, o);
  t = __shfl_sync(FULL, t, 0);
  const bool finite = (t > 0.0) && (t < CUDART_INF) && (mx < CUDART_INF_F) && (mx > -CUDART_INF_F);

  if (S > 1) {
    if (lane < k) rk[lane] = 0ull;
    __syncwarp();
    // Two lower bounds of the row's ke-th best key (chunk lists hold ke keys at most): the best
    // ke-th key of any one chunk, and the ke-th best of the chunk heads (ke different chunks each
    // hold a key at least that large).
    const u64 head = lane < S ? st[lane] : 0ull;
    u64 tau = lane < S ? st[(ke - 1) * FX_MAX_SPLITS + lane] : 0ull;
    if (S >= ke) {
      int cnt = 0;                                 // (lanes past the chunks hold 0 and count for nothing)
#pragma unroll
      for (int o = 0; o < FX_MAX_SPLITS; ++o) cnt += (shfl_u64(head, o) > head) ? 1 : 0;
      if (cnt == ke - 1) tau = umax64(tau, head);
    }
    tau = warp_max_u64(tau);
    // keys that reach the bound: lists are sorted, so the scan over list positions stops at the
    // first position where no chunk has one
    int ns = 0;
    for (int i = 0; i < ke; ++i) {
      const u64 key = lane < S ? st[i * FX_MAX_SPLITS + lane] : 0ull;
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
        if (r < ke) rk[r] = key;
      }
    } else {
      // many keys at the bound (equal logits): pop the largest head ke times
      int p = 0;
      for (int r = 0; r < ke; ++r) {
        const u64 cand = (lane < S && p < ke) ? st[p * FX_MAX_SPLITS + lane] : 0ull;
        const u64 best = warp_max_u64(cand);
        if (best == 0ull) break;
        if (cand == best) ++p;
        if (lane == 0) rk[r] = best;
      }
    }
  }
  __syncwarp();
  out_key = lane < k ? rk[lane] : 0ull;
  out_score = -CUDART_INF;
  if (finite && lane < ke && out_key != 0ull) {
    const double s = ps + ((double)key_logit(out_key) - ((double)mx + log(t)));
    if (s == s && s > -CUDART_INF) out_score = s;
  }
  __syncwarp();
  return finite;
}

// Gate, budget truncation and append for one sequence, from the pooled candidates in shared
// memory (sm.row_keys / sm.score: F rows of k, each row descending; sm.row_mask: the parents'
// mask rows).  n is the tree's size before the layer.
__device__ void select_and_append(const FusedArgs &a, const TailSmem &sm, int b, int lo, int F, int n,
                                  u64 *s_anchor, int *s_cnt) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = a.k;
  const int R = a.N - n;
  const int ke = min(k, R);                 // a parent can place at most R children
  const size_t nb = (size_t)b * a.N;
  const int C = F * k;

  // ---- eligibility: Top-K layers take every candidate, gated layers Eq. 4 ----
  const bool init = a.d < a.init_layers;
  double thr = -CUDART_INF;
  if (!init && *s_anchor != 0ull) thr = a.log_mu + f64_unord(*s_anchor);
  int local = 0;
  for (int c = tid; c < C; c += EXP_THREADS) {
    const double s = sm.score[c];
    unsigned char stt = (s > -CUDART_INF) ? 1 : 0;
    if (stt && !init && !(s >= thr)) stt = 0;
    sm.state[c] = stt;
    local += stt;
  }
  for (int j = tid; j < F; j += EXP_THREADS) sm.row_cnt[j] = 0;
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
#pragma unroll 4
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

__global__ void __launch_bounds__(EXP_THREADS, 3)
expand_fused_kernel(FusedArgs a) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ u64 s_buf[EXP_WARPS][XS_BUF];          // per-warp buffers of keys that reached the threshold
  __shared__ u64 s_pool[XS_POOL];                   // the chunk's candidates, all warps
  __shared__ int s_warp[EXP_WARPS];
  __shared__ float s_m[EXP_WARPS], s_s[EXP_WARPS];
  __shared__ __align__(8) u64 s_bar[EXP_WARPS][XS_RING];   // "tile landed" barriers, per warp
  __shared__ float s_wtop[EXP_WARPS];               // each warp's ceil(k/8)-th largest lane maximum
  __shared__ float s_wmax[EXP_WARPS];               // each warp's largest
  __shared__ u64 s_anchor;
  __shared__ int s_pool_n, s_last, s_last_seq, s_ecnt, s_bad, s_abort;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = a.k;
  if (lane == 0) {
    for (int i = 0; i < XS_RING; ++i) ring_bar_init(smem_addr(&s_bar[warp][i]));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_wtop[warp] = -CUDART_INF_F;
    s_wmax[warp] = -CUDART_INF_F;
  }
  if (tid == 0) {
    s_pool_n = 0; s_abort = 0;
    s_anchor = 0ull; s_ecnt = 0; s_bad = 0;
  }
  pdl_enter();

  // ---- frontier geometry (from layer_off[d], layer_off[d + 1]: never written by this launch) ----
  Frontier fr;
  fr.in_regs = a.B <= 32;
  // batches above 32 keep their frontier bases behind the ring (the launch adds the room)
  int *s_base = reinterpret_cast<int *>(smem_raw + a.base_offset);
  fr.s_base = s_base;
  fr.base_l = fr.f_l = fr.lo_l = 0;
  if (fr.in_regs) {
    if (lane < a.B) {
      fr.lo_l = a.t.layer_off[lane * a.lo_stride + a.d];
      const int hi = a.t.layer_off[lane * a.lo_stride + a.d + 1];
      fr.f_l = hi < a.N ? max(hi - fr.lo_l, 0) : 0;
      if (fr.f_l == 0 && blockIdx.x == 0 && warp == 0)        // nothing to expand: close the layer
        a.t.layer_off[lane * a.lo_stride + a.d + 2] = hi;
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
        if (s_base[b + 1] == s_base[b])
          a.t.layer_off[b * a.lo_stride + a.d + 2] = a.t.layer_off[b * a.lo_stride + a.d + 1];
  }
  const SpanGeom g = span_geom(fr.total, a.V, (int)gridDim.x, a.max_split);
  const unsigned long long line_end = (unsigned long long)fr.total * g.pitch;
  const bool gated = a.d >= a.init_layers;
  const float ln_mu = (float)a.log_mu;
  unsigned wt = 0;                 // tiles this warp has taken from its ring so far
  float *ring = reinterpret_cast<float *>(smem_raw) + warp * (XS_RING * XS_WTILE);
  u64 *buf = s_buf[warp];
  __syncthreads();

  unsigned long long pos = (unsigned long long)blockIdx.x * g.span;
  const unsigned long long span_end = min(line_end, pos + g.span);
  int row = pos < span_end ? (int)div_u64(pos, g.pitch) : 0;
  int start = pos < span_end ? (int)(pos - (unsigned long long)row * g.pitch) : 0;
  for (; pos < span_end; ++row, start = 0) {
    // ---- one chunk: elements [start, start + len) of packed row `row` ----
    const int len = (int)min((unsigned long long)(g.pitch - (unsigned)start), span_end - pos);
    pos += (unsigned)len;
    const int item = (int)blockIdx.x + row;
    const RowLoc rl = locate_row(a, fr, row);
    int rsel = (a.layout == TALON_ROWS_BY_NODE) ? rl.node : rl.j;
    if (rsel >= a.rows_per_seq) {               // caller reserved too few rows: stay in bounds, report
      rsel = a.rows_per_seq - 1;
      if (tid == 0) atomicOr(a.status, STATUS_CAPACITY);
    }
    const float *rowp = a.logits + ((int64_t)rl.b * a.rows_per_seq + rsel) * a.row_stride;
    const int end = min(a.V, start + len);        // (an empty chunk past the row's end still reports in)
    const int lo = rl.node - rl.j;               // first frontier node of the sequence
    const int n_before = lo + rl.F;              // the tree's size before this layer
    const int ke = min(k, a.N - n_before);       // a parent can place at most N - |T| children
    const int share_pos = (ke + EXP_WARPS - 1) / EXP_WARPS - 1;

    // ---- this warp's slice of the chunk ----
    // (a short chunk goes to fewer warps, a full tile each: thresholds need elements to work with)
    const int wlen = max(XS_WTILE, ((end - start + 4 * EXP_WARPS - 1) / (4 * EXP_WARPS)) * 4);
    const int ws = start + warp * wlen;
    const int we = min(end, ws + wlen);
    const int nt = ws < we ? (we - ws + XS_WTILE - 1) / XS_WTILE : 0;
    auto issue = [&](int t, unsigned slot_index) {
      const int base = ws + t * XS_WTILE;
      const int n = min(XS_WTILE, we - base);
      const unsigned sl = slot_index % XS_RING;
      // whole 16-byte units: the last one of a row may reach into the row's stride padding
      ring_issue(smem_addr(ring + sl * XS_WTILE), rowp + base, (uint32_t)(((n * 4) + 15) & ~15),
                 smem_addr(&s_bar[warp][sl]));
    };
    if (lane == 0)
      for (int t = 0; t < nt && t < XS_RING; ++t) issue(t, wt + t);
    WarpStream w;
    w.m_t = -CUDART_INF_F; w.s_t = 0.f;
    w.thr_f = -CUDART_MAX_NORMAL_F;              // -inf never competes (probability zero)
    w.thr_key = 0ull;
    w.cnt = 0;
    bool refreshed = false;
    for (int t = 0; t < nt; ++t) {
      const int base = ws + t * XS_WTILE;
      const unsigned sl = wt % XS_RING;
      if (!ring_wait(smem_addr(&s_bar[warp][sl]), (wt / XS_RING) & 1u)) {
        // The copy did not land in time: the launch is reported as timed out (the tree arrays are
        // undefined from here on) and the CTA leaves at the end of this chunk.  The copy gets one
        // more bounded wait so that it does not land in memory the CTA has already given back.
        if (lane == 0) { atomicOr(a.status, STATUS_TIMEOUT); s_abort = 1; }
        ring_wait(smem_addr(&s_bar[warp][sl]), (wt / XS_RING) & 1u);
      }
      float v[16];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float4 x = *reinterpret_cast<const float4 *>(ring + sl * XS_WTILE + u * 128 + lane * 4);
        v[4 * u + 0] = x.x; v[4 * u + 1] = x.y; v[4 * u + 2] = x.z; v[4 * u + 3] = x.w;
      }
      if (base + XS_WTILE > we) {             // the slice's last, partial tile: nothing past `we` counts
#pragma unroll
        for (int i = 0; i < 16; ++i)
          if (base + (i >> 2) * 128 + lane * 4 + (i & 3) >= we) v[i] = -CUDART_INF_F;
      }
      ++wt;
      float bm = max3(max3(v[0], v[1], v[2]), max3(v[3], v[4], v[5]), max3(v[6], v[7], v[8]));
      bm = max3(bm, max3(v[9], v[10], v[11]), max3(v[12], v[13], v[14]));
      bm = fmaxf(bm, v[15]);
      // running softmax normaliser of this lane's elements
      if (bm > w.m_t) {
        w.s_t *= fast_exp2((w.m_t - bm) * LOG2E_F);
        w.m_t = bm;
      }
      if (w.m_t > -CUDART_INF_F) {
        // exp(v - m) = 2^(v * log2e - m * log2e); an infinite m (a +inf logit) must give NaN
        const float c = -w.m_t * LOG2E_F;
        const u64 c2 = pack_f32x2(c, c), l2 = pack_f32x2(LOG2E_F, LOG2E_F);
        u64 acc0 = 0ull, acc1 = 0ull;              // two pairs of +0.0f
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
          float x0, x1, x2, x3;
          unpack_f32x2(fma_f32x2(pack_f32x2(v[i], v[i + 1]), l2, c2), x0, x1);
          unpack_f32x2(fma_f32x2(pack_f32x2(v[i + 2], v[i + 3]), l2, c2), x2, x3);
          acc0 = add_f32x2(acc0, pack_f32x2(fast_exp2(x0), fast_exp2(x1)));
          acc1 = add_f32x2(acc1, pack_f32x2(fast_exp2(x2), fast_exp2(x3)));
        }
        float s0, s1;
        unpack_f32x2(add_f32x2(acc0, acc1), s0, s1);
        w.s_t += s0 + s1;
      }
      refreshed = (t & (t + 1)) == 0 || t == 2;  // after tiles 1, 2, 3, 4, 8, 16, ... of the slice
      // (the first tile has nothing but its own lane maxima to go by: their exact ke-th largest)
      if (refreshed) refresh_threshold(w, ke, share_pos, gated, ln_mu, s_wtop, s_wmax, lane, warp, t == 0);
      if (__ballot_sync(FULL, bm >= w.thr_f) != 0u) {
        collect_tile(ring + sl * XS_WTILE, v, base, ke, buf, w, lane);
        __syncwarp();
      }
      // Every lane's loads from the slot have delivered their data (the vote needs every lane's
      // maximum, and what the collection read has gone into the buffer): the slot can take the
      // tile XS_RING ahead.
      if (lane == 0 && t + XS_RING < nt) issue(t + XS_RING, wt - 1 + XS_RING);
    }
    if (nt > 4 && !refreshed) refresh_threshold(w, ke, share_pos, gated, ln_mu, s_wtop, s_wmax, lane, warp, false);

    // ---- the warp's survivors -> the CTA pool; its normaliser -> shared memory ----
    {
      // a warp that could not build a threshold (a short slice) brings its ke best keys only, so
      // that eight warps never overflow the pool
      if (w.cnt > XS_POOL / EXP_WARPS) cut_back(buf, ke, w, lane);
      const int n = w.cnt;
      for (int i = lane; i < n; i += 32) {
        const u64 key = buf[i];
        if (key != 0ull && key_logit(key) >= w.thr_f) {
          const int pos = atomicAdd(&s_pool_n, 1);
          if (pos < XS_POOL) s_pool[pos] = key;
        }
      }
      float wm = w.m_t;
#pragma unroll
      for (int o = 16; o; o >>= 1) wm = fmaxf(wm, __shfl_xor_sync(FULL, wm, o));
      // lane partial rescaled to the warp maximum; a NaN partial (NaN or +inf logit) propagates
      float wsum = (w.m_t > -CUDART_INF_F || w.s_t != w.s_t) ? w.s_t * exp2f((w.m_t - wm) * LOG2E_F) : 0.f;
#pragma unroll
      for (int o = 16; o; o >>= 1) wsum += __shfl_xor_sync(FULL, wsum, o);
      if (lane == 0) { s_m[warp] = wm; s_s[warp] = wsum; }
    }
    __syncthreads();
    if (s_abort) return;
    if (s_pool_n > XS_POOL) {
      // the pool cannot hold every survivor (equal logits): each warp brings its ke best only
      __syncthreads();
      if (tid == 0) s_pool_n = 0;
      __syncthreads();
      cut_back(buf, ke, w, lane);
      const int n = w.cnt;
      int pos = 0;
      if (lane == 0) pos = atomicAdd(&s_pool_n, n);
      pos = __shfl_sync(FULL, pos, 0);
      if (lane < n) s_pool[pos + lane] = buf[lane];
      __syncthreads();
    }

    // ---- the chunk's ke best keys: four lanes count each candidate's betters (keys are unique) ----
    const int nc = s_pool_n;
    for (int c0 = 0; c0 < nc; c0 += EXP_THREADS / 4) {
      const int ci = c0 + (tid >> 2), q = tid & 3;
      const u64 key = ci < nc ? s_pool[ci] : 0ull;
      int r = 0;
#pragma unroll 4
      for (int o = q; o < nc; o += 4) r += (s_pool[o] > key) ? 1 : 0;
      r += __shfl_xor_sync(FULL, r, 1);
      r += __shfl_xor_sync(FULL, r, 2);
      if (q == 0 && ci < nc && r < ke) a.part_keys[(size_t)item * a.key_stride + r] = key;
    }
    if (tid < k && tid >= min(nc, ke)) a.part_keys[(size_t)item * a.key_stride + tid] = 0ull;
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

    // ---- hand-off.  The barrier orders this CTA's writes before thread 0's device-scope
    // release; the last arrival acquires.  Narrow frontiers count chunks per sequence, wide ones
    // chunks per row and then rows per sequence. ----
    const bool two_level = rl.F > XS_TWO_LEVEL;
    __syncthreads();
    if (lane == 0) { s_wtop[warp] = -CUDART_INF_F; s_wmax[warp] = -CUDART_INF_F; }
    if (tid == 0) {
      s_pool_n = 0;
      if (two_level && (unsigned)len == g.pitch) {
        s_last = 1;                                               // the row's only chunk
      } else {
        // the counters add up elements of the line: a row is done at pitch, a narrow frontier at F * pitch
        cuda::atomic_ref<unsigned int, cuda::thread_scope_device> c(two_level ? a.row_count[row] : a.seq_count[rl.b]);
        const unsigned target = two_level ? g.pitch : (unsigned)rl.F * g.pitch;
        const unsigned prev = c.fetch_add((unsigned)len, cuda::memory_order_acq_rel);
        s_last = (prev + (unsigned)len == target);
        if (s_last) c.store(0u, cuda::memory_order_relaxed);      // ready for the next layer
      }
    }
    __syncthreads();
    if (!s_last) continue;

    TailSmem sm;
    const int rows_max = a.N - 1;
    {
      unsigned char *p = smem_raw;
      sm.stage = reinterpret_cast<u64 *>(p);            p += sizeof(u64) * EXP_WARPS * stage_words(k);
      sm.row_keys = reinterpret_cast<u64 *>(p);         p += sizeof(u64) * rows_max * k;
      sm.score = reinterpret_cast<double *>(p);         p += sizeof(double) * rows_max * k;
      sm.row_mask = reinterpret_cast<u64 *>(p);         p += sizeof(u64) * rows_max * a.W;
      sm.row_cnt = reinterpret_cast<int *>(p);          p += sizeof(int) * rows_max;
      sm.row_off = reinterpret_cast<int *>(p);          p += sizeof(int) * rows_max;
      sm.state = p;
    }
    const size_t nb = (size_t)rl.b * a.N;
    if (two_level) {
      // ---- this CTA finished a row of a wide frontier: one warp merges it, publishes the result
      // and counts the row; the CTA that counts the sequence's last row goes on ----
      if (warp == 0) {
        u64 key, pmask; double sc;
        int item0, S;
        row_chunks(g, row, item0, S);
        const bool finite = merge_row(a, (size_t)item0, S, k, ke, nb + rl.node, sm.stage, key, sc, pmask);
        if (!finite) {
          sc = lane == 0 ? CUDART_NAN : -CUDART_INF;
          if (lane == 0) atomicOr(a.status, STATUS_NONFINITE);
        }
        if (lane < k) {
          a.row_keys[(size_t)row * a.key_stride + lane] = key;
          a.row_score[(size_t)row * a.key_stride + lane] = sc;
        }
        __syncwarp();
        if (lane == 0) {
          cuda::atomic_ref<unsigned int, cuda::thread_scope_device> c(a.seq_count[rl.b]);
          const unsigned prev = c.fetch_add(1u, cuda::memory_order_acq_rel);
          s_last_seq = (prev == (unsigned)rl.F - 1u);
          if (s_last_seq) c.store(0u, cuda::memory_order_relaxed);
        }
      }
      __syncthreads();
      if (!s_last_seq) continue;
      // ---- collect the sequence's row results and the parents' mask rows: four loads per thread
      // go to registers before the first store, so that they share one trip to L2 ----
      const int C = rl.F * k;
      for (int c0 = 0; c0 < C; c0 += 4 * EXP_THREADS) {
        u64 key[4]; double sc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c = c0 + u * EXP_THREADS + tid;
          const int j = c / k, i = c - j * k;
          key[u] = c < C ? __ldcg(a.row_keys + (size_t)(rl.row0 + j) * a.key_stride + i) : 0ull;
          sc[u] = c < C ? __ldcg(a.row_score + (size_t)(rl.row0 + j) * a.key_stride + i) : -CUDART_INF;
        }
        const int mi = c0 / 4 + tid;                 // the mask words ride along, EXP_THREADS per round
        const u64 mword = mi < rl.F * a.W ? a.t.mask[(nb + lo) * a.W + mi] : 0ull;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c = c0 + u * EXP_THREADS + tid;
          if (c >= C) continue;
          sm.row_keys[c] = key[u];
          if (sc[u] != sc[u]) { s_bad = 1; sm.score[c] = -CUDART_INF; }
          else {
            sm.score[c] = sc[u];
            // rows are sorted: heads carry the maxima
            if (c % k == 0 && sc[u] > -CUDART_INF) atomicMax(&s_anchor, f64_ord(sc[u]));
          }
        }
        if (mi < rl.F * a.W) sm.row_mask[mi] = mword;
      }
      for (int mi = (C + 4 * EXP_THREADS - 1) / (4 * EXP_THREADS) * EXP_THREADS + tid; mi < rl.F * a.W; mi += EXP_THREADS)
        sm.row_mask[mi] = a.t.mask[(nb + lo) * a.W + mi];
    } else {
      // ---- this CTA finished the sequence: one warp per row ----
      for (int j = warp; j < rl.F; j += EXP_WARPS) {
        u64 key, pmask; double sc;
        int item0, S;
        row_chunks(g, rl.row0 + j, item0, S);
        const bool finite = merge_row(a, (size_t)item0, S, k, ke, nb + lo + j, sm.stage + warp * stage_words(k), key, sc,
                                      pmask);
        if (!finite && lane == 0) { s_bad = 1; atomicOr(a.status, STATUS_NONFINITE); }
        if (lane < k) {
          sm.row_keys[j * k + lane] = key;
          sm.score[j * k + lane] = sc;
        }
        if (lane < a.W) sm.row_mask[j * a.W + lane] = pmask;
        if (lane == 0 && sc > -CUDART_INF) atomicMax(&s_anchor, f64_ord(sc));
      }
    }
    __syncthreads();
    if (s_bad) {             // a frontier row was not finite: this sequence adds nothing
      if (tid == 0) a.t.layer_off[rl.b * a.lo_stride + a.d + 2] = n_before;
    } else {
      select_and_append(a, sm, rl.b, lo, rl.F, n_before, &s_anchor, &s_ecnt);
    }
    __syncthreads();     // the next chunk's bulk copies land in the memory the selection phase just used
    if (tid == 0) { s_anchor = 0ull; s_ecnt = 0; s_bad = 0; }
  }
}

size_t fused_smem_bytes(const talon_ctx *c) {
  const size_t rows = c->p.budget - 1, k = c->k_cap, W = c->W;
  const size_t tail = sizeof(u64) * EXP_WARPS * (FX_MAX_SPLITS * k + FX_SURV + k) + rows * k * (8 + 8 + 1) +
                      rows * (8 * W + 4 + 4) + 16;
  const size_t ring = sizeof(float) * EXP_WARPS * XS_RING * XS_WTILE;       // the two phases share the space
  return ((tail > ring ? tail : ring) + 15) & ~(size_t)15;
}

// batches above 32 sequences keep the frontier bases in dynamic shared memory behind that
size_t fused_base_bytes(int B) { return B > 32 ? sizeof(int) * (MAX_BATCH + 1) : 0; }

}  // namespace

talon_status expand_fused_setup(talon_ctx *c) {
  const size_t bytes = fused_smem_bytes(c);
  if (cudaFuncSetAttribute(expand_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)(bytes + fused_base_bytes(c->p.batch_max))) !=
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
  a.max_split = c->expand_max_split;
  long long max_items = (long long)rows_bound * FX_MAX_SPLITS;
  int grid = c->fused_grid;
  if (max_items < grid) grid = (int)max_items;
  if (grid < 1) grid = 1;
  a.root_topk = c->p.root_topk; a.init_layers = c->p.init_layers; a.log_mu = c->log_mu;
  a.part_keys = c->d_part_keys; a.part_ms = c->d_part_ms; a.row_keys = c->d_row_keys; a.row_score = c->d_row_score;
  a.row_count = c->d_row_count; a.seq_count = c->d_seq_count; a.status = c->d_status;
  {
    LaunchTimer lt(c, TALON_K_EXPAND_ROWS, st);
    a.base_offset = (int)fused_smem_bytes(c);
    launch_kernel_pdl(c, true, expand_fused_kernel, dim3(grid), dim3(EXP_THREADS), fused_smem_bytes(c) + fused_base_bytes(c->B), st, a);
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  return TALON_OK;
}

}  // namespace talon

// Tree attention (verification forward of Appendix B) on the 5th-generation tensor cores.
//
// Work split.  For sequence b and kv head h the g = Hq/Hkv query heads of all N tree nodes are
// packed into one [g*N, 128] query matrix (row = node * g + head-in-group), so every K/V tile
// is read once for the whole group.  A CTA owns up to two 128-row query tiles and a range of
// 128-key tiles of the key axis (the L_b prefix keys, then the tree keys).  Several ranges per
// (b, h) are merged either inside the kernel -- the ranges form a thread-block cluster, leave
// their partial results in shared memory and every CTA merges a share of the rows through
// distributed shared memory -- or, for more than eight ranges or very few rows, by a second kernel
// from fp32 partials in global memory (split-KV).
//
// Roles inside a CTA (320 threads):
//   warps 0-3, 4-7  softmax of query tile 0 / 1: thread r owns row r.  It reads its row of
//                   S = Q K^T from tensor memory (tcgen05.ld), applies the ragged-length or
//                   ancestor-bitmask visibility, keeps a running maximum and sum, and writes
//                   P = exp2(S*scale - max) as bf16 back to tensor memory over S (tcgen05.st).
//                   The running maximum is only raised when it grows by more than 2^8, so the
//                   accumulator in tensor memory is rescaled rarely (the final division by the
//                   running sum makes any reference maximum exact).
//   warp 8          producer: TMA loads of Q (once) and of the K / V tiles into a ring of
//                   128-byte-swizzled shared-memory stages (no multicast).
//   warp 9          one thread issues tcgen05.mma: S_i = Q_i K^T (both operands in shared
//                   memory) and O_i += P_i V (P from tensor memory, V from shared memory), with
//                   tcgen05.commit arriving on mbarriers that the other roles wait on.
// Every wait is bounded: a role that gives up raises a flag that makes the other roles leave
// too, tensor memory is released, and the device status word reports a timeout.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include <cstdio>
#include <cstring>

#include "talon_internal.cuh"

namespace talon {

namespace {

constexpr int TC_BN = 128;                 // keys per tile
constexpr int TC_D = 128;                  // head dimension
constexpr int TC_MT = 128;                 // query rows per tile
constexpr int TC_STAGES = 2;               // K and V ring depth
constexpr int TC_THREADS = 320;
constexpr int TC_TILE_BYTES = TC_BN * TC_D * 2;      // 32 KB: one K, V or Q tile
constexpr int TC_HALF_BYTES = TC_BN * 64 * 2;        // 16 KB: the 64-element half of a tile
constexpr int TC_NBARS = 16;
constexpr int TC_SMEM = (2 + 2 * TC_STAGES) * TC_TILE_BYTES + 1024 + TC_NBARS * 8 + 64;
constexpr uint32_t TC_TMEM_COLS = 512;     // O0 | O1 | S0 | S1, 128 fp32 columns each
constexpr float TC_RESCALE_GAP = 8.f;      // raise the reference maximum only beyond 2^8
constexpr long long TC_WAIT_CYCLES = 4000000000ll;   // ~2 s: far beyond any legitimate wait
constexpr int TC_XO_PITCH = TC_D + 4;      // floats per row of the partial result a CTA leaves in shared memory
constexpr int TC_XO_BYTES = 2 * TC_MT * TC_XO_PITCH * 4;        // 256 rows; their (max, sum) pairs follow
static_assert(TC_XO_BYTES + 2 * TC_MT * 8 <= (2 + 2 * TC_STAGES) * TC_TILE_BYTES, "the partial result reuses the tile buffers");

// barrier slots
enum { B_Q = 0, B_KFULL = 1, B_VFULL = 3, B_KEMPTY = 5, B_VEMPTY = 7, B_SFULL = 9, B_PFULL = 11, B_ODONE = 13 };

struct TcArgs {
  const int64_t *kv_start;
  const int32_t *block_table;  // paged prefix: [B, bt_stride] page numbers (null: contiguous blocks at kv_start)
  int bt_stride;
  const int32_t *prefix_len, *n_nodes;
  const unsigned long long *mask;
  int B, N, W, Hq, Hkv, g;
  float scale_log2;
  int splits, m_blocks;
  int cluster_merge;           // the key ranges of a (sequence, head, tile pair) form a cluster and merge in shared memory
  __nv_bfloat16 *out;
  float *part_o;
  float2 *part_ml;
  int *status;
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ inline uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ inline void mbar_arrive(uint32_t bar) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.shared::cta.b64 st, [%0];\n}" ::"r"(bar) : "memory");
}
__device__ inline void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("{\n.reg .b64 st;\nmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n}" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ inline bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  // the hint lets the hardware park the thread until the phase completes (or ~20 us pass)
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.b32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(bar), "r"(parity), "r"(20000u) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity; gives up after TC_WAIT_CYCLES or when another
// role already gave up.  Returns false in that case.
__device__ inline bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > TC_WAIT_CYCLES) { *abort_flag = 1; return false; }
  }
}

__device__ inline void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ inline void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
               ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ inline void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ inline void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accum) {
  asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}"
               ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accum) : "memory");
}
__device__ inline void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr));
}
__device__ inline void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
               "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
               "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                 "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                 "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                 "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
               : "memory");
}
__device__ inline void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ inline void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle; 8-row groups 1024 bytes apart).
// K-major operand: rows of 64 bf16 (128 bytes); the leading offset is unused.
__device__ inline uint64_t desc_kmajor(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand (V: keys x d, d contiguous): the next 64-element block of d starts
// TC_HALF_BYTES further, the next group of 8 keys 1024 bytes further.
__device__ inline uint64_t desc_mnmajor(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)(TC_HALF_BYTES >> 4) << 16) | (64ull << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = 128.
constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_QK = idesc_base;                 // A and B K-major
constexpr uint32_t IDESC_PV = idesc_base | (1u << 16);    // B MN-major

__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Packed fp32 pairs (sm_100): one instruction for two lanes of a 64-bit register pair.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ inline uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}
// ---- distributed shared memory of a thread-block cluster ----
__device__ inline uint32_t cluster_map(uint32_t addr, uint32_t cta_rank) {     // my shared address, seen in CTA cta_rank
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta_rank));
  return r;
}
__device__ inline float4 cluster_ld_f4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ inline float2 cluster_ld_f2(uint32_t addr) {
  float2 v;
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
  return v;
}
// every thread of every CTA of the cluster; orders shared-memory writes before it against reads after it
__device__ inline void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace

__global__ void __launch_bounds__(TC_THREADS, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kp,
                         const __grid_constant__ CUtensorMap map_vp, const __grid_constant__ CUtensorMap map_kt,
                         const __grid_constant__ CUtensorMap map_vt, TcArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  __shared__ uint32_t s_tmem_base;
  __shared__ int s_abort;

  pdl_enter();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int mpair = blockIdx.x, split = blockIdx.y;
  const int bh = blockIdx.z, b = bh / a.Hkv, kvh = bh - b * a.Hkv;

  // carve shared memory: tiles need 1024-byte alignment for the 128-byte swizzle
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  const uint32_t q_smem = base;
  const uint32_t k_smem = base + 2 * TC_TILE_BYTES;
  const uint32_t v_smem = k_smem + TC_STAGES * TC_TILE_BYTES;
  const uint32_t bars = v_smem + TC_STAGES * TC_TILE_BYTES;
  unsigned char *gen_base = smem_dyn + (base - smem_u32(smem_dyn));      // generic pointer to `base`
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int n = a.n_nodes[b];
  const int L = a.prefix_len[b];
  const int rows_total = a.g * a.N;
  const int rows_valid = a.g * n;
  int nmt = (rows_total - mpair * 2 * TC_MT + TC_MT - 1) / TC_MT;       // query tiles of this CTA with rows
  nmt = nmt > 2 ? 2 : nmt;

  const int nP = (L + TC_BN - 1) / TC_BN;
  const int nT = (a.N + TC_BN - 1) / TC_BN;
  const int tt = nP + nT;
  const int tps = (tt + a.splits - 1) / a.splits;
  const int t_begin = split * tps;
  const int t_end = min(tt, t_begin + tps);
  const int nt = max(t_end - t_begin, 0);

  if (tid == 0) {
    s_abort = 0;
    mbar_init(bar(B_Q), 1);
    for (int s = 0; s < TC_STAGES; ++s) {
      mbar_init(bar(B_KFULL + s), 1);
      mbar_init(bar(B_VFULL + s), 1);
      mbar_init(bar(B_KEMPTY + s), 1);
      mbar_init(bar(B_VEMPTY + s), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(B_SFULL + i), 1);
      mbar_init(bar(B_PFULL + i), 128);
      mbar_init(bar(B_ODONE + i), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {          // this warp owns the tensor-memory allocation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem_base)),
                 "r"(TC_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem_base;
  volatile int *abort_flag = &s_abort;

  if (warp == 8) {
    // ================= producer =================
    if (lane == 0 && nt > 0) {
      const int nodes_per_tile = TC_MT / a.g;
      mbar_expect_tx(bar(B_Q), (uint32_t)nmt * TC_TILE_BYTES);
      for (int i = 0; i < nmt; ++i)
        for (int h = 0; h < 2; ++h)
          tma_load_4d(q_smem + i * TC_TILE_BYTES + h * TC_HALF_BYTES, &map_q, bar(B_Q), h * 64, kvh * a.g,
                      (mpair * 2 + i) * nodes_per_tile, b);
      // first cache token of prefix tile tg: a page of TC_BN tokens from the table, or the
      // sequence's contiguous block
      const long long tok0 = a.block_table ? 0ll : a.kv_start[b];
      auto tile_tok = [&](int tg) {
        return a.block_table ? (long long)a.block_table[(size_t)b * a.bt_stride + tg] * TC_BN : tok0 + (long long)tg * TC_BN;
      };
      bool ok = true;
      for (int it = 0; it < nt && ok; ++it) {
        const int s = it % TC_STAGES;
        const uint32_t par = ((it / TC_STAGES) & 1) ^ 1;
        const int tg = t_begin + it;
        ok = mbar_wait(bar(B_KEMPTY + s), par, abort_flag);
        if (!ok) break;
        mbar_expect_tx(bar(B_KFULL + s), TC_TILE_BYTES);
        for (int h = 0; h < 2; ++h) {
          const uint32_t dst = k_smem + s * TC_TILE_BYTES + h * TC_HALF_BYTES;
          if (tg < nP) tma_load_3d(dst, &map_kp, bar(B_KFULL + s), h * 64, kvh, (int)tile_tok(tg));
          else tma_load_4d(dst, &map_kt, bar(B_KFULL + s), h * 64, kvh, (tg - nP) * TC_BN, b);
        }
        ok = mbar_wait(bar(B_VEMPTY + s), par, abort_flag);
        if (!ok) break;
        mbar_expect_tx(bar(B_VFULL + s), TC_TILE_BYTES);
        for (int h = 0; h < 2; ++h) {
          const uint32_t dst = v_smem + s * TC_TILE_BYTES + h * TC_HALF_BYTES;
          if (tg < nP) tma_load_3d(dst, &map_vp, bar(B_VFULL + s), h * 64, kvh, (int)tile_tok(tg));
          else tma_load_4d(dst, &map_vt, bar(B_VFULL + s), h * 64, kvh, (tg - nP) * TC_BN, b);
        }
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ================= MMA issue =================
    if (lane == 0 && nt > 0) {
      bool ok = mbar_wait(bar(B_Q), 0, abort_flag);
      auto issue_qk = [&](int i, int s) {
#pragma unroll
        for (int kk = 0; kk < TC_D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * TC_HALF_BYTES + (kk & 3) * 32;
          tc_mma_ss(tmem + 256 + 128 * i, desc_kmajor(q_smem + i * TC_TILE_BYTES + off),
                    desc_kmajor(k_smem + s * TC_TILE_BYTES + off), IDESC_QK, kk > 0 ? 1u : 0u);
        }
      };
      auto issue_pv = [&](int i, int s, bool accumulate) {
#pragma unroll
        for (int kk = 0; kk < TC_BN / 16; ++kk)
          tc_mma_ts(tmem + 128 * i, tmem + 256 + 128 * i + kk * 8, desc_mnmajor(v_smem + s * TC_TILE_BYTES + kk * 2048),
                    IDESC_PV, (accumulate || kk > 0) ? 1u : 0u);
      };
      if (ok) ok = mbar_wait(bar(B_KFULL + 0), 0, abort_flag);
      if (ok) {
        tc_fence_after();
        for (int i = 0; i < nmt; ++i) {
          issue_qk(i, 0);
          tc_commit(bar(B_SFULL + i));
        }
        tc_commit(bar(B_KEMPTY + 0));
      }
      for (int it = 0; it < nt && ok; ++it) {
        const int s = it % TC_STAGES;
        ok = mbar_wait(bar(B_VFULL + s), (it / TC_STAGES) & 1, abort_flag);
        for (int i = 0; i < nmt && ok; ++i) {
          ok = mbar_wait(bar(B_PFULL + i), it & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_pv(i, s, it > 0);
          tc_commit(bar(B_ODONE + i));
          if (i == nmt - 1) tc_commit(bar(B_VEMPTY + s));
          if (it + 1 < nt) {
            const int s2 = (it + 1) % TC_STAGES;
            if (i == 0) {
              ok = mbar_wait(bar(B_KFULL + s2), ((it + 1) / TC_STAGES) & 1, abort_flag);
              if (!ok) break;
              tc_fence_after();
            }
            issue_qk(i, s2);
            tc_commit(bar(B_SFULL + i));
            if (i == nmt - 1) tc_commit(bar(B_KEMPTY + s2));
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ================= softmax + epilogue: warps 0-3 own query tile 0, warps 4-7 tile 1 =================
    const int i = warp >> 2;
    const int quarter = warp & 3;
    const int r_local = quarter * 32 + lane;
    const int R = (mpair * 2 + i) * TC_MT + r_local;            // packed query row
    const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16);
    const uint32_t t_S = t_lane + 256 + 128 * i;
    const uint32_t t_O = t_lane + 128 * i;
    const bool row_valid = R < rows_valid;
    unsigned long long mrow[2] = {0ull, 0ull};
    if (row_valid)
      for (int w = 0; w < a.W; ++w) mrow[w] = a.mask[((int64_t)b * a.N + R / a.g) * a.W + w];

    float m_used = -CUDART_INF_F, l_run = 0.f;
    bool ok = (i < nmt) && nt > 0;
    for (int it = 0; it < nt && ok; ++it) {
      const int tg = t_begin + it;
      const bool tree_tile = tg >= nP;
      const int kvalid = tree_tile ? min(n - (tg - nP) * TC_BN, TC_BN) : min(L - tg * TC_BN, TC_BN);
      const int s = it % TC_STAGES;
      // keys beyond the valid range may hold anything: tile 0's warps clear their V rows so that
      // a zero probability times stale memory cannot produce a NaN
      if (i == 0 && kvalid < TC_BN) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(B_VFULL + s), (it / TC_STAGES) & 1, abort_flag));
        if (!ok) break;
        const int zr = max(kvalid, 0) + r_local;
        if (zr < TC_BN) {
          uint4 *p0 = reinterpret_cast<uint4 *>(gen_base + (2 + TC_STAGES) * TC_TILE_BYTES + s * TC_TILE_BYTES + zr * 128);
          uint4 *p1 = reinterpret_cast<uint4 *>(reinterpret_cast<unsigned char *>(p0) + TC_HALF_BYTES);
#pragma unroll
          for (int c = 0; c < 8; ++c) { p0[c] = make_uint4(0, 0, 0, 0); p1[c] = make_uint4(0, 0, 0, 0); }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      }
      ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(B_SFULL + i), it & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();

      const bool masked = tree_tile || kvalid < TC_BN;
      const unsigned long long vis0 = tree_tile ? mrow[0] : ~0ull, vis1 = tree_tile ? mrow[1] : ~0ull;
      // keys c of this tile the row may see: c < kvalid and (tree tile) ancestor bit c
      unsigned long long see0 = vis0, see1 = vis1;
      if (kvalid < 64) { see0 &= kvalid <= 0 ? 0ull : (~0ull >> (64 - kvalid)); see1 = 0ull; }
      else if (kvalid < 128) see1 &= kvalid == 64 ? 0ull : (~0ull >> (128 - kvalid));
      if (tree_tile && (tg - nP) > 0) { see0 = 0ull; see1 = 0ull; }     // N <= 128: there is one tree tile

      // ---- the row of S: one read from tensor memory, held in registers ----
      uint32_t r[4][32];
      tc_ld32(t_S + 0, r[0]);
      tc_ld32(t_S + 32, r[1]);
      tc_ld32(t_S + 64, r[2]);
      tc_ld32(t_S + 96, r[3]);
      tc_wait_ld();
      if (masked) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint32_t bits = (uint32_t)((q < 2 ? see0 : see1) >> ((q & 1) * 32));
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (!((bits >> c) & 1u)) r[q][c] = 0xFF800000u;            // -inf: exp2 gives an exact 0
        }
      }
      // row maximum, four independent chains
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int c = 0; c < 32; c += 2) mx4[q] = max3(mx4[q], __uint_as_float(r[q][c]), __uint_as_float(r[q][c + 1]));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float mx_x = mx * a.scale_log2;
      float alpha = 1.f;
      if (m_used == -CUDART_INF_F) m_used = mx_x;
      else if (mx_x > m_used + TC_RESCALE_GAP) {
        alpha = fast_exp2(m_used - mx_x);
        l_run *= alpha;
        m_used = mx_x;
      }
      const float m_eff = (m_used == -CUDART_INF_F) ? 0.f : m_used;

      // ---- P = exp2(S * scale - max) as bf16 over S; row sum in four packed chains ----
      const unsigned long long scale2 = pack_f32x2(a.scale_log2, a.scale_log2);
      const unsigned long long nmax2 = pack_f32x2(-m_eff, -m_eff);
      unsigned long long sum2[4] = {0ull, 0ull, 0ull, 0ull};          // four pairs of 0.f
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t pk[32];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
#pragma unroll
          for (int c = 0; c < 32; c += 2) {
            const unsigned long long x2 =
                fma_f32x2(pack_f32x2(__uint_as_float(r[half * 2 + q][c]), __uint_as_float(r[half * 2 + q][c + 1])), scale2, nmax2);
            float x0, x1;
            unpack_f32x2(x2, x0, x1);
            const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
            sum2[(c >> 1) & 3] = add_f32x2(sum2[(c >> 1) & 3], pack_f32x2(p0, p1));
            pk[q * 16 + (c >> 1)] = pack_bf16x2(p0, p1);
          }
        }
        tc_st32(t_S + half * 32, pk);
      }
      float sum4[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        float lo, hi;
        unpack_f32x2(sum2[q], lo, hi);
        sum4[q] = lo + hi;
      }
      l_run += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);

      // ---- rare: the reference maximum moved, rescale the accumulator of this row's warp ----
      if (it > 0 && __any_sync(0xFFFFFFFFu, alpha != 1.f)) {
        ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(B_ODONE + i), (it - 1) & 1, abort_flag));
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int c0 = 0; c0 < TC_D; c0 += 32) {
            uint32_t r[32];
            tc_ld32(t_O + c0, r);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) r[c] = __float_as_uint(__uint_as_float(r[c]) * alpha);
            tc_st32(t_O + c0, r);
          }
        }
      }
      tc_wait_st();
      tc_fence_before();
      mbar_arrive(bar(B_PFULL + i));
    }

    // ---- epilogue: O / l (or the partial result of this key range) ----
    // tcgen05.ld is a warp-wide instruction: every lane of a warp that holds any row takes part
    // in the loads, and only the stores are per lane.
    if (ok) ok = __all_sync(0xFFFFFFFFu, mbar_wait(bar(B_ODONE + i), (nt - 1) & 1, abort_flag));
    const bool in_range = R < rows_total;
    if (a.cluster_merge) {
      // The key ranges of this (sequence, head, tile pair) are the CTAs of one cluster: each leaves
      // its partial result in its own shared memory (the tile buffers are free once both query
      // tiles' MMAs have finished, hence the barrier over the 256 softmax threads) and the merge
      // reads them from there after the cluster barrier at the end of the kernel.
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const int rr = i * TC_MT + r_local;
      float *xo = reinterpret_cast<float *>(gen_base) + (size_t)rr * TC_XO_PITCH;
      float2 *xml = reinterpret_cast<float2 *>(gen_base + TC_XO_BYTES);
      const bool dump = ok && __any_sync(0xFFFFFFFFu, in_range);     // warp-uniform; rows past the last are never read
      if (dump) {
        tc_fence_after();
#pragma unroll
        for (int c0 = 0; c0 < TC_D; c0 += 32) {
          uint32_t r[32];
          tc_ld32(t_O + c0, r);
          tc_wait_ld();
#pragma unroll
          for (int c = 0; c < 8; ++c)
            reinterpret_cast<uint4 *>(xo + c0)[c] = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
        }
      }
      xml[rr] = (ok && row_valid) ? make_float2(m_used, l_run) : make_float2(-CUDART_INF_F, 0.f);
    } else if (ok && __any_sync(0xFFFFFFFFu, in_range)) {
      tc_fence_after();
      const int node = in_range ? R / a.g : 0, qh = in_range ? R - node * a.g : 0;
      if (a.splits == 1) {
        const bool live = row_valid && l_run > 0.f;
        const float inv = live ? 1.f / l_run : 0.f;
        __nv_bfloat16 *op = a.out + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * TC_D;
#pragma unroll
        for (int c0 = 0; c0 < TC_D; c0 += 32) {
          uint32_t r[32];
          tc_ld32(t_O + c0, r);
          tc_wait_ld();
          uint32_t o[16];
#pragma unroll
          for (int c = 0; c < 16; ++c)
            o[c] = live ? pack_bf16x2(__uint_as_float(r[2 * c]) * inv, __uint_as_float(r[2 * c + 1]) * inv) : 0u;
          if (in_range) {
#pragma unroll
            for (int c = 0; c < 4; ++c)
              reinterpret_cast<uint4 *>(op + c0)[c] = make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
          }
        }
      } else {
        const int mpad = a.m_blocks * TC_MT;
        const int64_t prow = ((int64_t)bh * a.splits + split) * mpad + (in_range ? R : 0);
        float *op = a.part_o + prow * TC_D;
#pragma unroll
        for (int c0 = 0; c0 < TC_D; c0 += 32) {
          uint32_t r[32];
          tc_ld32(t_O + c0, r);
          tc_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int c = 0; c < 8; ++c)
              reinterpret_cast<uint4 *>(op + c0)[c] = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
          }
        }
        if (row_valid) a.part_ml[prow] = make_float2(m_used, l_run);
      }
    } else if (nt == 0 && i < nmt && R < rows_total) {
      // an empty key range (more splits than tiles): contribute nothing
      if (a.splits == 1) {
        const int node = R / a.g, qh = R - node * a.g;
        uint4 *op = reinterpret_cast<uint4 *>(a.out + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * TC_D);
#pragma unroll
        for (int c = 0; c < 16; ++c) op[c] = make_uint4(0, 0, 0, 0);
      } else if (row_valid) {
        const int mpad = a.m_blocks * TC_MT;
        a.part_ml[((int64_t)bh * a.splits + split) * mpad + R] = make_float2(-CUDART_INF_F, 0.f);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (a.cluster_merge) {
    // ---- merge of the cluster's partial results: CTA c takes every splits-th share of the 256
    // packed rows, one warp per row, lane l the output columns 4l..4l+3 ----
    cluster_sync_all();
    if (warp < 8) {
      const int S = a.splits;
      const int share = (2 * TC_MT + S - 1) / S;
      const int r_lo = split * share, r_hi = min(2 * TC_MT, r_lo + share);
      const uint32_t xo0 = smem_u32(gen_base), xml0 = smem_u32(gen_base + TC_XO_BYTES);
      for (int rr = r_lo + warp; rr < r_hi; rr += 8) {
        const int Rm = mpair * 2 * TC_MT + rr;
        if (Rm >= rows_total) break;
        const float2 ml = lane < S ? cluster_ld_f2(cluster_map(xml0 + (uint32_t)rr * 8u, (uint32_t)lane))
                                   : make_float2(-CUDART_INF_F, 0.f);
        float gm = ml.x;
#pragma unroll
        for (int o = 16; o; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xFFFFFFFFu, gm, o));
        const float w = (ml.x == -CUDART_INF_F) ? 0.f : fast_exp2(ml.x - gm);    // an empty range has no row to read
        float lsum = w * ml.y;
#pragma unroll
        for (int o = 16; o; o >>= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, o);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        const uint32_t row_off = xo0 + ((uint32_t)rr * TC_XO_PITCH + (uint32_t)lane * 4u) * 4u;
        for (int s0 = 0; s0 < S; s0 += 4) {        // the loads of four ranges go out before any is used
          float ws[4];
          float4 o4[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int sidx = s0 + u;
            ws[u] = __shfl_sync(0xFFFFFFFFu, w, sidx & 31);
            if (sidx >= S) ws[u] = 0.f;
            o4[u] = ws[u] != 0.f ? cluster_ld_f4(cluster_map(row_off, (uint32_t)sidx)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            acc.x += ws[u] * o4[u].x; acc.y += ws[u] * o4[u].y; acc.z += ws[u] * o4[u].z; acc.w += ws[u] * o4[u].w;
          }
        }
        const float inv = lsum > 0.f ? 1.f / lsum : 0.f;
        const int node = Rm / a.g, qh = Rm - node * a.g;
        uint2 packed;
        packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
        packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2 *>(a.out + (((int64_t)b * a.N + node) * a.Hq + kvh * a.g + qh) * TC_D + lane * 4) = packed;
      }
    }
    cluster_sync_all();                    // nobody leaves while a peer may still read its shared memory
  }
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TC_TMEM_COLS) : "memory");
  }
  if (tid == 0 && s_abort) atomicOr(a.status, STATUS_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool encode_bf16(CUtensorMap *m, const void *ptr, int rank, const cuuint64_t *dims, const cuuint64_t *strides_bytes,
                 const cuuint32_t *box) {
  const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(ptr), dims,
                        strides_bytes, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) std::fprintf(stderr, "talon: cuTensorMapEncodeTiled failed (%d)\n", (int)r);
  return r == CUDA_SUCCESS;
}

}  // namespace

bool attention_tc_supported(const talon_ctx *c, int64_t stride_t, int64_t stride_h, float sm_scale) {
  const int g = c->p.n_q_heads / c->p.n_kv_heads;
  if (c->p.head_dim != 128 || c->p.budget > 128) return false;
  if (g < 1 || g > 128 || (128 % g) != 0) return false;
  if (!(sm_scale > 0.f)) return false;                     // the lazy maximum assumes a positive scale
  if (stride_t < 128 || stride_h < 1) return false;
  return encode_fn() != nullptr;
}

talon_status attention_tc_setup() {
  return cudaFuncSetAttribute(tree_attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM) ==
                 cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

talon_status launch_attention_tc(talon_ctx *c, const talon_tree *t, const void *q, const void *kp, const void *vp,
                                 const void *kt, const void *vt, const int64_t *kv_start, const int32_t *block_table,
                                 int bt_stride, int64_t stride_t,
                                 int64_t stride_h, int64_t kv_tokens, int max_prefix_len, float sm_scale, void *out,
                                 int splits, int m_blocks, cudaStream_t st, int *merged_in_kernel) {
  *merged_in_kernel = 0;
  const int N = c->p.budget, Hq = c->p.n_q_heads, Hkv = c->p.n_kv_heads, g = Hq / Hkv, B = c->B;
  CUtensorMap mq, mkp, mvp, mkt, mvt;
  {
    const cuuint64_t dims[4] = {128, (cuuint64_t)Hq, (cuuint64_t)N, (cuuint64_t)B};
    const cuuint64_t str[3] = {256, (cuuint64_t)Hq * 256, (cuuint64_t)N * Hq * 256};
    const cuuint32_t box[4] = {64, (cuuint32_t)g, (cuuint32_t)(128 / g), 1};
    if (!encode_bf16(&mq, q, 4, dims, str, box)) return TALON_ERR_CUDA;
  }
  {
    const cuuint64_t dims[3] = {128, (cuuint64_t)Hkv, (cuuint64_t)(kv_tokens > 0 ? kv_tokens : 1)};
    const cuuint64_t str[2] = {(cuuint64_t)stride_h * 2, (cuuint64_t)stride_t * 2};
    const cuuint32_t box[3] = {64, 1, TC_BN};
    if (!encode_bf16(&mkp, kp, 3, dims, str, box) || !encode_bf16(&mvp, vp, 3, dims, str, box)) return TALON_ERR_CUDA;
  }
  {
    const cuuint64_t dims[4] = {128, (cuuint64_t)Hkv, (cuuint64_t)N, (cuuint64_t)B};
    const cuuint64_t str[3] = {256, (cuuint64_t)Hkv * 256, (cuuint64_t)N * Hkv * 256};
    const cuuint32_t box[4] = {64, 1, TC_BN, 1};
    if (!encode_bf16(&mkt, kt, 4, dims, str, box) || !encode_bf16(&mvt, vt, 4, dims, str, box)) return TALON_ERR_CUDA;
  }
  TcArgs a;
  a.kv_start = kv_start; a.block_table = block_table; a.bt_stride = bt_stride;
  a.prefix_len = c->d_prefix_len; a.n_nodes = t->n_nodes;
  a.mask = (const unsigned long long *)t->mask;
  a.B = B; a.N = N; a.W = c->W; a.Hq = Hq; a.Hkv = Hkv; a.g = g;
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.splits = splits; a.m_blocks = m_blocks;
  a.out = (__nv_bfloat16 *)out; a.part_o = c->d_attn_o; a.part_ml = c->d_attn_ml; a.status = c->d_status;
  (void)max_prefix_len;
  dim3 grid((m_blocks + 1) / 2, splits, B * Hkv);
  // Two to eight key ranges: they are launched as one thread-block cluster and merge their partial
  // results through distributed shared memory, if the device can place such a cluster (asked once
  // per cluster size; a cluster of full-SM CTAs needs that many SMs free in one GPC).
  a.cluster_merge = 0;
  // (few rows: the second kernel is cheaper than a cluster launch and two cluster barriers)
  const long long merge_rows = (long long)B * Hkv * g * N * splits;
  if ((c->attn_cluster == 2 || (c->attn_cluster == 1 && merge_rows >= c->attn_cluster_min_rows)) && splits >= 2 &&
      splits <= 8) {
    cudaLaunchConfig_t q = {};
    q.gridDim = grid; q.blockDim = dim3(TC_THREADS); q.dynamicSmemBytes = TC_SMEM; q.stream = st;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = 1; qa[0].val.clusterDim.y = (unsigned)splits; qa[0].val.clusterDim.z = 1;
    q.attrs = qa; q.numAttrs = 1;
    if (c->attn_cluster_ok[splits] < 0) {
      int n = 0;
      const cudaError_t e = cudaOccupancyMaxActiveClusters(&n, tree_attention_tc_kernel, &q);
      if (e != cudaSuccess) cudaGetLastError();
      c->attn_cluster_ok[splits] = (e == cudaSuccess && n >= 1) ? 1 : 0;
    }
    a.cluster_merge = c->attn_cluster_ok[splits];
  }
  {
    LaunchTimer lt(c, TALON_K_ATTENTION, st);
    if (a.cluster_merge) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = grid; cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = TC_SMEM; cfg.stream = st;
      cudaLaunchAttribute attr[2];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = (unsigned)splits; attr[0].val.clusterDim.z = 1;
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = (c->pdl == 1 || (c->pdl < 0 && c->B <= PDL_AUTO_BATCH)) ? 2 : 1;
      cudaLaunchKernelEx(&cfg, tree_attention_tc_kernel, mq, mkp, mvp, mkt, mvt, a);
      *merged_in_kernel = 1;
    } else {
      launch_kernel(c, tree_attention_tc_kernel, grid, dim3(TC_THREADS), TC_SMEM, st, mq, mkp, mvp, mkt, mvt, a);
    }
  }
  if (cudaGetLastError() != cudaSuccess) return TALON_ERR_CUDA;
  c->launches += 1;
  return TALON_OK;
}

}  // namespace talon

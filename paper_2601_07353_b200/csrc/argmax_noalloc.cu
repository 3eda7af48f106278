// Target argmax without any allocation, for callers that must not call cudaMalloc.
//
// The ordinary route (talon_accept) keeps its per-row scratch keys in the context's workspace,
// which talon_create allocates.  A caller that runs inside a memory pool it may not grow, or in
// a phase of a serving process where allocation is forbidden (allocation synchronises the device
// and can fail late), cannot create a context.  This file gives that caller the argmax step of
// the verification alone, with the scratch in a fixed array that is part of the library image.
#include <math_constants.h>

#include <cstdio>
#include <mutex>

#include "talon_internal.cuh"

namespace talon {
namespace {

constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr int NA_THREADS = 256;
constexpr int NA_MAX_DEVICES = 64;

// One packed (logit, lowest-token-first) key per row.  Every GPU that loads the library holds
// these TALON_NOALLOC_MAX_ROWS * 8 bytes until the process exits.  All calls share the array.
static __device__ __align__(256) unsigned long long g_argmax_scratch[TALON_NOALLOC_MAX_ROWS];

__global__ void noalloc_clear_kernel(int n_rows) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_rows) g_argmax_scratch[i] = 0ull;
}

// One CTA per (row, chunk); chunks of a row meet in a 64-bit atomicMax on the row's key.
__global__ void __launch_bounds__(NA_THREADS)
noalloc_argmax_kernel(const float *logits, int64_t row_stride, int V, int n_rows, int splits, int chunk_len,
                      unsigned long long *best) {
  __shared__ unsigned long long s_key[NA_THREADS / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long n_items = (long long)n_rows * splits;
  for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int row = (int)(item / splits), chunk = (int)(item - (long long)row * splits);
    const float *rowp = logits + (int64_t)row * row_stride;
    const int start = chunk * chunk_len;
    const int end = min(V, start + chunk_len);
    float bestv = -CUDART_INF_F;
    uint32_t besti = 0xFFFFFFFFu;
    for (int idx = start + tid * 4; idx < end; idx += NA_THREADS * 4) {
      float x[4];
      if (idx + 4 <= end) {
        const float4 q = __ldcs(reinterpret_cast<const float4 *>(rowp + idx));
        x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = (idx + e < end) ? __ldcs(rowp + idx + e) : -CUDART_INF_F;
      }
#pragma unroll
      for (int e = 0; e < 4; ++e)   // strict > keeps the lowest index among equal values; a NaN never competes
        if (idx + e < end && x[e] == x[e] && (x[e] > bestv || besti == 0xFFFFFFFFu)) {
          bestv = x[e];
          besti = (uint32_t)(idx + e);
        }
    }
    unsigned long long key = (besti == 0xFFFFFFFFu) ? 0ull : cand_key(bestv, besti);
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(FULL, key, o);
      key = other > key ? other : key;
    }
    __syncthreads();
    if (lane == 0) s_key[warp] = key;
    __syncthreads();
    if (tid == 0) {
      unsigned long long kk = s_key[0];
      for (int w = 1; w < NA_THREADS / 32; ++w) kk = s_key[w] > kk ? s_key[w] : kk;
      atomicMax(&best[row], kk);
    }
  }
}

__global__ void noalloc_decode_kernel(int n_rows, int32_t *target_tok) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_rows) {
    const unsigned long long kk = g_argmax_scratch[i];
    target_tok[i] = kk != 0ull ? (int32_t)key_tok(kk) : -1;
  }
}

// per-device set-up, done by the first call on that device
struct DeviceSlot {
  bool ready;
  unsigned long long *scratch;   // device address of g_argmax_scratch on this device
  int sm_count;
};
DeviceSlot g_slots[NA_MAX_DEVICES];
std::mutex g_slots_lock;       // two host threads may make the first call on a device at once

}  // namespace
}  // namespace talon

extern "C" talon_status talon_target_argmax_noalloc(const float *target_logits, int64_t row_stride, int32_t vocab,
                                                    int32_t n_rows, int32_t *target_tok, void *stream) {
  using namespace talon;
  if (!target_logits || !target_tok) return TALON_ERR_INVALID_ARG;
  if (vocab < 1 || vocab >= (1 << 24) || n_rows < 0) return TALON_ERR_INVALID_ARG;
  if (n_rows > TALON_NOALLOC_MAX_ROWS) {
    std::fprintf(stderr, "talon_target_argmax_noalloc: %d rows exceed the fixed scratch of %d rows\n", n_rows,
                 TALON_NOALLOC_MAX_ROWS);
    return TALON_ERR_CAPACITY;
  }
  if (row_stride < vocab || (row_stride & 3) || (reinterpret_cast<uintptr_t>(target_logits) & 15u))
    return TALON_ERR_INVALID_ARG;
  if (n_rows == 0) return TALON_OK;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return TALON_ERR_CUDA;
  DeviceSlot &slot = g_slots[dev];
  {
    std::lock_guard<std::mutex> hold(g_slots_lock);
    if (!slot.ready) {
    // In host code the array's name is only a handle: the device address has to be asked for,
    // with the device that will run the kernels current.
    void *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_argmax_scratch);
    if (e != cudaSuccess || !p) {
      std::fprintf(stderr, "talon_target_argmax_noalloc: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return TALON_ERR_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return TALON_ERR_CUDA;
    slot.scratch = static_cast<unsigned long long *>(p);
    slot.sm_count = sms;
    slot.ready = true;
    }
  }
  cudaStream_t st = (cudaStream_t)stream;
  // chunks per row: enough items to fill the GPU, chunks a multiple of 1024 elements
  const int target_items = slot.sm_count * 8;
  int want = (target_items + n_rows - 1) / n_rows;
  if (want < 1) want = 1;
  if (want > 32) want = 32;
  int len = (vocab + want - 1) / want;
  len = ((len + 1023) / 1024) * 1024;
  const int splits = (vocab + len - 1) / len;
  long long items = (long long)n_rows * splits;
  int grid = target_items;
  if (items < grid) grid = (int)items;
  noalloc_clear_kernel<<<(n_rows + 255) / 256, 256, 0, st>>>(n_rows);
  noalloc_argmax_kernel<<<grid, NA_THREADS, 0, st>>>(target_logits, row_stride, vocab, n_rows, splits, len,
                                                       slot.scratch);
  noalloc_decode_kernel<<<(n_rows + 255) / 256, 256, 0, st>>>(n_rows, target_tok);
  return cudaGetLastError() == cudaSuccess ? TALON_OK : TALON_ERR_CUDA;
}

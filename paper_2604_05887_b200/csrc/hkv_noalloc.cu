// hkv_topk_chunks_noalloc: chunk scoring + exact top-k for ONE dynamic head with the float32 score
// scratch in a fixed device array of this library instead of caller-provided memory.  For callers
// that hold no allocator at the point of the call (a plugin running inside another runtime's
// callback, a real-time loop that must not touch the CUDA memory manager): they pass only inputs
// and outputs.  The array is part of the library image on every GPU that loads it.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>

#include "hkv_device.cuh"
#include "hkv_internal.h"

namespace hkv {
namespace {

constexpr int kNoAllocThreads = 256;
constexpr int kMaxDevices = 64;

// The scratch: one float32 score per chunk mean.  All calls on a device share it.
static __device__ __align__(256) float g_noalloc_scores[HKV_NOALLOC_MAX_CHUNKS];

// One CTA: score_c = <sum_g q_g, mean_c> in float32, then radix selection of the k largest with ties
// to the lower chunk id, ids written in ascending order.  `scores` is the scratch (every entry below
// n_chunks is overwritten before it is read, so nothing has to be cleared between calls).
__global__ void __launch_bounds__(kNoAllocThreads)
    topk_chunks_kernel(const __nv_bfloat16* q, const uint4* means, int G, int n_chunks, int k, float* scores,
                       int32_t* out_ids) {
  __shared__ float qsum[kHeadDim];
  __shared__ int hist[256];
  __shared__ int wsum[96];
  __shared__ int bc[4];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < kHeadDim) {
    float s = 0.f;
    for (int g = 0; g < G; ++g) s += __bfloat162float(q[g * kHeadDim + tid]);
    qsum[tid] = s;
  }
  __syncthreads();
  {
    // 16 lanes per chunk mean (16 B each), two means per warp pass
    const int sub = lane & 15, half = lane >> 4;
    float qv[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) qv[j] = qsum[sub * 8 + j];
    for (int c0 = warp * 2; c0 < n_chunks; c0 += (kNoAllocThreads / 32) * 2) {
      const int c = c0 + half;
      float acc = 0.f;
      if (c < n_chunks) {
        const uint4 m = means[static_cast<size_t>(c) * 16 + sub];
        acc = fmaf(bf16_lo(m.x), qv[0], acc); acc = fmaf(bf16_hi(m.x), qv[1], acc);
        acc = fmaf(bf16_lo(m.y), qv[2], acc); acc = fmaf(bf16_hi(m.y), qv[3], acc);
        acc = fmaf(bf16_lo(m.z), qv[4], acc); acc = fmaf(bf16_hi(m.z), qv[5], acc);
        acc = fmaf(bf16_lo(m.w), qv[6], acc); acc = fmaf(bf16_hi(m.w), qv[7], acc);
      }
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
      if (c < n_chunks && sub == 0) scores[c] = acc;
    }
  }
  __threadfence_block();
  __syncthreads();
  if (k >= n_chunks) {
    for (int i = tid; i < n_chunks; i += kNoAllocThreads) out_ids[i] = i;
    return;
  }
  block_select_emit(
      n_chunks, k, [&](int i) { return float_key(scores[i]); }, [](int) { return false; },
      [&](int pos, int i) { out_ids[pos] = i; }, hist, wsum, bc);
}

// Device address of the scratch on each device, resolved once per device (host code cannot use the
// array's name as a pointer: on the host it is only a handle for the runtime's symbol table).
std::atomic<float*> g_scratch_addr[kMaxDevices];   // zero-initialised; host threads may race to fill an entry with the same value

}  // namespace
}  // namespace hkv

extern "C" hkv_status hkv_topk_chunks_noalloc(const void* q, const void* means, int32_t group, int32_t n_chunks,
                                              int32_t k, int32_t* out_ids, void* stream) {
  using namespace hkv;
  if (!q || !means || !out_ids) return HKV_ERR_INVALID_ARG;
  if (group < 1 || group > kMaxGroup) return HKV_ERR_UNSUPPORTED;
  if (n_chunks < 1 || k < 1) return HKV_ERR_SHAPE;
  if (n_chunks > HKV_NOALLOC_MAX_CHUNKS) return HKV_ERR_WORKSPACE;   // beyond the built-in scratch
  if ((reinterpret_cast<uintptr_t>(means) & 15) || (reinterpret_cast<uintptr_t>(q) & 1)) return HKV_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return HKV_ERR_CUDA; }
  float* scratch = g_scratch_addr[dev].load(std::memory_order_acquire);
  if (!scratch) {
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&scratch), g_noalloc_scores) != cudaSuccess || !scratch) {
      cudaGetLastError();
      return HKV_ERR_CUDA;
    }
    g_scratch_addr[dev].store(scratch, std::memory_order_release);
  }
  topk_chunks_kernel<<<1, kNoAllocThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(q), static_cast<const uint4*>(means), group, n_chunks, std::min(k, n_chunks),
      scratch, out_ids);
  if (cudaGetLastError() != cudaSuccess) return HKV_ERR_CUDA;
  return HKV_OK;
}

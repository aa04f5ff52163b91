// amk_argmax_static: the greedy-token selection of the LM-head tail (block candidates, last-arriving block
// reduces them) as a stand-alone kernel whose scratch memory is a fixed array inside the library image, so
// the call needs no caller buffer and allocates nothing.  The scratch array, the set-up that looks up its
// address and the kernel are all in this file.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>
#include <stdio.h>

#include <mutex>

#include "amk.h"

namespace {

constexpr int kThreads = 256;
constexpr int kPerBlock = 2048;                                     // elements one block scans
constexpr int kMaxBlocks = AMK_ARGMAX_STATIC_MAX_N / kPerBlock;     // 512
constexpr int kCandBase = 32;                                       // word 0: arrival counter; 1..31 unused
constexpr int kScratchWords = kCandBase + kMaxBlocks;               // 544 words = 4352 bytes
static_assert(AMK_ARGMAX_STATIC_MAX_N % kPerBlock == 0, "whole blocks");

// Word 0 counts the blocks that have published their candidate.  It must be zero when the kernel starts: every
// call clears it on its own stream before the launch (so a call never inherits a count from a launch that did
// not run to its end), and the block that arrives last puts it back to zero as well.
// Words kCandBase + b hold block b's candidate {value bits, index}; they are written before they are read in
// every call and need no initial value.
static __device__ __align__(256) unsigned long long scratch[kScratchWords];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned long long* g_scratch_of_device[kMaxDevices];   // looked up once per device, under g_mu

__device__ __forceinline__ bool better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

__global__ void __launch_bounds__(kThreads) argmax_static_kernel(const float* __restrict__ x, int n,
                                                                 int* __restrict__ out, unsigned long long* s) {
  __shared__ float sv[kThreads / 32];
  __shared__ int si[kThreads / 32];
  __shared__ bool last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float bv = -CUDART_INF_F;
  int bi = 0x7fffffff;
  const int base = blockIdx.x * kPerBlock;
  for (int i = base + threadIdx.x; i < min(base + kPerBlock, n); i += kThreads) {
    const float v = x[i];
    if (better(v, i, bv, bi)) { bv = v; bi = i; }
  }
  auto warp_reduce = [&]() {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
  };
  auto block_reduce = [&]() {   // result valid in warp 0
    warp_reduce();
    if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
    __syncthreads();
    if (warp == 0) {
      bv = lane < kThreads / 32 ? sv[lane] : -CUDART_INF_F;
      bi = lane < kThreads / 32 ? si[lane] : 0x7fffffff;
      warp_reduce();
    }
  };
  block_reduce();
  if (threadIdx.x == 0) {
    __stcg(s + kCandBase + blockIdx.x, (unsigned long long)__float_as_uint(bv) | ((unsigned long long)(unsigned)bi << 32));
    __threadfence();
    last = atomicAdd((unsigned*)s, 1u) == gridDim.x - 1;
  }
  __syncthreads();
  if (!last) return;
  __threadfence();
  bv = -CUDART_INF_F;
  bi = 0x7fffffff;
  for (int b = threadIdx.x; b < (int)gridDim.x; b += kThreads) {
    const unsigned long long w = __ldcg(s + kCandBase + b);
    const float v = __uint_as_float((unsigned)w);
    const int i = (int)(unsigned)(w >> 32);
    if (better(v, i, bv, bi)) { bv = v; bi = i; }
  }
  __syncthreads();   // sv / si are reused
  block_reduce();
  if (threadIdx.x == 0) {
    // NaN elements compare false and are never chosen; a vector of nothing but NaNs has no candidate: index 0
    *out = (bi == 0x7fffffff) ? 0 : bi;
    *(unsigned*)s = 0u;   // the next call starts from zero again
  }
}

void say(char* msg, size_t n, const char* fmt, long long a, long long b) {
  if (msg && n) snprintf(msg, n, fmt, a, b);
}

}  // namespace

extern "C" amk_status amk_argmax_static(const float* x, int64_t n, int32_t* token, char* msg, size_t msg_bytes,
                                        void* cuda_stream) {
  if (msg && msg_bytes) msg[0] = 0;
  if (!x || !token) {
    say(msg, msg_bytes, "amk_argmax_static: NULL pointer", 0, 0);
    return AMK_ERR_INVALID_ARG;
  }
  if (n < 1) {
    say(msg, msg_bytes, "amk_argmax_static: n = %lld, need at least 1 element", (long long)n, 0);
    return AMK_ERR_INVALID_ARG;
  }
  if (n > AMK_ARGMAX_STATIC_MAX_N) {
    say(msg, msg_bytes, "amk_argmax_static: n = %lld exceeds AMK_ARGMAX_STATIC_MAX_N = %lld (fixed scratch size)",
        (long long)n, (long long)AMK_ARGMAX_STATIC_MAX_N);
    return AMK_ERR_UNSUPPORTED;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    say(msg, msg_bytes, "amk_argmax_static: no usable current device (index %lld, table holds %lld)", dev, kMaxDevices);
    return AMK_ERR_CUDA;
  }
  unsigned long long* ptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    ptr = g_scratch_of_device[dev];
    if (!ptr) {   // set-up: once per device
      const cudaError_t e = cudaGetSymbolAddress((void**)&ptr, scratch);
      if (e != cudaSuccess || !ptr) {
        say(msg, msg_bytes, "amk_argmax_static: cudaGetSymbolAddress failed (error %lld) on device %lld", (long long)e, dev);
        return AMK_ERR_CUDA;
      }
      g_scratch_of_device[dev] = ptr;
    }
  }
  // both buffers must be device memory of the current device: the scratch used is this device's
  for (int k = 0; k < 2; k++) {
    cudaPointerAttributes at;
    const void* q = k ? (const void*)token : (const void*)x;
    const cudaError_t e = cudaPointerGetAttributes(&at, q);
    if (e != cudaSuccess) (void)cudaGetLastError();
    if (e != cudaSuccess || (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged) ||
        (at.type == cudaMemoryTypeDevice && at.device != dev)) {
      say(msg, msg_bytes, "amk_argmax_static: argument %lld is not device memory of the current device %lld", k, dev);
      return AMK_ERR_INVALID_ARG;
    }
  }
  if (((uintptr_t)x | (uintptr_t)token) & 3u) {
    say(msg, msg_bytes, "amk_argmax_static: pointers must be 4-byte aligned", 0, 0);
    return AMK_ERR_INVALID_ARG;
  }
  const int blocks = (int)((n + kPerBlock - 1) / kPerBlock);
  {
    const cudaError_t e = cudaMemsetAsync(ptr, 0, sizeof(unsigned long long), (cudaStream_t)cuda_stream);
    if (e != cudaSuccess) {
      say(msg, msg_bytes, "amk_argmax_static: clearing the arrival counter failed (error %lld)", (long long)e, 0);
      return AMK_ERR_CUDA;
    }
  }
  argmax_static_kernel<<<blocks, kThreads, 0, (cudaStream_t)cuda_stream>>>(x, (int)n, token, ptr);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    say(msg, msg_bytes, "amk_argmax_static: launch failed (error %lld)", (long long)e, 0);
    return AMK_ERR_CUDA;
  }
  return AMK_OK;
}

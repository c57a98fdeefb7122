// pe_select_best: arg-min of the makespan (Eq. 1) over the candidates that pass the status mask.
#include <atomic>
#include <climits>

#include "pe.h"
#include <cuda_runtime.h>

namespace pe {

// key = makespan << 32 | index: the 64-bit minimum is the smallest makespan, ties to the smallest index
constexpr unsigned long long kNoKey = ~0ull;

// The four result words double as the running state: [0] minimum key, [2] qualifying candidates,
// [3] blocks finished; the last block to finish turns [0] into {index, makespan} in [0], [1].
__global__ void pe_select_init_kernel(unsigned long long* r) {
  r[0] = kNoKey;
  r[1] = 0ull;
  r[2] = 0ull;
  r[3] = 0ull;
}

__global__ void __launch_bounds__(256) pe_select_kernel(int64_t K, const int32_t* __restrict__ makespan,
                                                        const uint32_t* __restrict__ status, uint32_t reject_mask,
                                                        unsigned long long* scratch) {
  unsigned long long best = kNoKey;
  unsigned long long count = 0;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < K; c += (int64_t)gridDim.x * blockDim.x) {
    if ((status[c] & reject_mask) == 0) {
      ++count;
      const unsigned long long key = ((unsigned long long)(unsigned)makespan[c] << 32) | (unsigned long long)c;
      best = key < best ? key : best;
    }
  }
  for (int off = 16; off > 0; off >>= 1) {
    const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, best, off);
    best = o < best ? o : best;
    count += __shfl_xor_sync(0xFFFFFFFFu, count, off);
  }
  __shared__ unsigned long long s_best[8], s_count[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { s_best[warp] = best; s_count[warp] = count; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w) {
      best = s_best[w] < best ? s_best[w] : best;
      count += s_count[w];
    }
    if (best != kNoKey) atomicMin(&scratch[0], best);
    if (count) atomicAdd(&scratch[2], count);
    __threadfence();
    const unsigned long long done = atomicAdd(&scratch[3], 1ull) + 1ull;
    if (done == gridDim.x) {  // the last block publishes the result
      __threadfence();
      const unsigned long long m = atomicMin(&scratch[0], kNoKey);  // atomic read
      int64_t* result = reinterpret_cast<int64_t*>(scratch);
      result[0] = m == kNoKey ? -1 : (int64_t)(m & 0xFFFFFFFFull);
      result[1] = m == kNoKey ? (int64_t)INT32_MAX : (int64_t)(m >> 32);
    }
  }
}

}  // namespace pe

extern "C" int pe_select_best(int64_t K, const int32_t* makespan, const uint32_t* status, uint32_t reject_mask,
                              int64_t* result, void* cuda_stream) {
  if (K < 0 || !result || (K > 0 && (!makespan || !status))) return PE_ERR_INVALID_ARG;
  if (K > 0xFFFFFFFFll) return PE_ERR_INVALID_ARG;  // the index shares a 64-bit key with the makespan
  // run on the device that owns `result` (the other arrays must live there too)
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, result) != cudaSuccess ||
      (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)) {
    cudaGetLastError();
    return PE_ERR_INVALID_ARG;
  }
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != attr.device && cudaSetDevice(attr.device) != cudaSuccess) return PE_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  unsigned long long* scratch = reinterpret_cast<unsigned long long*>(result);
  pe::pe_select_init_kernel<<<1, 1, 0, stream>>>(scratch);
  int blocks = (int)((K + 255) / 256);
  if (blocks > 1184) blocks = 1184;  // 148 SMs x 8 resident blocks: a grid-stride loop covers the rest
  if (blocks < 1) blocks = 1;
  pe::pe_select_kernel<<<blocks, 256, 0, stream>>>(K, makespan, status, reject_mask, scratch);
  const int ret = cudaGetLastError() == cudaSuccess ? PE_OK : PE_ERR_CUDA;
  if (prev != attr.device) cudaSetDevice(prev);
  return ret;
}

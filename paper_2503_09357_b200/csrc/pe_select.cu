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

// ============================================================================================
// pe_select_topk: the k best qualifying candidates (smallest makespan, ties to the smallest index).
//
// Radix select on the makespan (three passes over 11 + 11 + 10 bits) finds the value T of the k-th best
// and how many candidates are strictly better; an ordered compaction (per-block counts, a scan over
// the blocks, a write pass) then lists, by increasing index, every candidate better than T and the
// first (k - better) candidates equal to T.  State lives in the caller's workspace:
//   words [0..7]   : prefix (bits of T fixed so far), remaining rank, qualifying count, result count
//   words [8..]    : histogram (2048 bins), then per-block (better, equal) counts and their scans
// ============================================================================================
namespace pe {

constexpr int kTopkBins = 2048;
constexpr int kTopkBlock = 256;
constexpr int kTopkPerBlock = 4096;   // candidates per block of the compaction passes

struct TopkState {
  unsigned int prefix;      // high bits of T found so far
  unsigned int remaining;   // rank still to resolve inside the current prefix (1-based)
  unsigned int qualifying;  // candidates that pass the mask
  unsigned int take_equal;  // how many candidates equal to T belong to the result
  unsigned int threshold;   // T
  unsigned int none;        // 1 when fewer than k qualify: everything qualifying is taken
  unsigned int pad[2];
};

__global__ void pe_topk_init_kernel(TopkState* s, unsigned int* hist, unsigned int k) {
  for (int b = threadIdx.x; b < kTopkBins; b += blockDim.x) hist[b] = 0;
  if (threadIdx.x == 0) {
    s->prefix = 0; s->remaining = k; s->qualifying = 0; s->take_equal = 0; s->threshold = 0; s->none = 0;
  }
}

// histogram of the `bits` bits at `shift` over the qualifying candidates whose higher bits equal the prefix
__global__ void __launch_bounds__(kTopkBlock) pe_topk_hist_kernel(int64_t K, const int32_t* __restrict__ makespan,
                                                                  const uint32_t* __restrict__ status,
                                                                  uint32_t reject_mask, const TopkState* s,
                                                                  unsigned int* hist, int shift, int bits, int first) {
  __shared__ unsigned int sh[kTopkBins];
  for (int b = threadIdx.x; b < kTopkBins; b += blockDim.x) sh[b] = 0;
  __syncthreads();
  const unsigned int prefix = s->prefix;
  const unsigned int mask = (1u << bits) - 1u;
  unsigned int qual = 0;
  for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < K; c += (int64_t)gridDim.x * blockDim.x) {
    if ((status[c] & reject_mask) != 0) continue;
    ++qual;
    const unsigned int v = (unsigned int)makespan[c];
    const int hi = shift + bits;
    if (hi < 32 && (v >> hi) != (prefix >> hi)) continue;
    atomicAdd(&sh[(v >> shift) & mask], 1u);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kTopkBins; b += blockDim.x)
    if (sh[b]) atomicAdd(&hist[b], sh[b]);
  if (first) {
    for (int off = 16; off > 0; off >>= 1) qual += __shfl_xor_sync(0xFFFFFFFFu, qual, off);
    if ((threadIdx.x & 31) == 0 && qual) atomicAdd(const_cast<unsigned int*>(&s->qualifying), qual);
  }
}

// one block: find the bin that holds the remaining-th smallest, fix its bits in the prefix, clear the histogram
__global__ void __launch_bounds__(kTopkBlock) pe_topk_pick_kernel(TopkState* s, unsigned int* hist, int shift, int bits,
                                                                  int first, int last) {
  __shared__ unsigned int part[kTopkBlock];
  __shared__ unsigned int chosen_bin, chosen_below;
  const int nb = 1 << bits;
  const int per = (nb + kTopkBlock - 1) / kTopkBlock;   // consecutive bins per thread
  if (first && threadIdx.x == 0 && s->qualifying < s->remaining) s->none = 1;
  __syncthreads();
  const bool none = s->none != 0;
  unsigned int mine = 0;
  for (int q = 0; q < per; ++q) {
    const int b = threadIdx.x * per + q;
    if (b < nb) mine += hist[b];
  }
  part[threadIdx.x] = mine;
  __syncthreads();
  if (threadIdx.x == 0 && !none) {
    unsigned int below = 0, rem = s->remaining;
    int t = 0;
    while (t < kTopkBlock - 1 && below + part[t] < rem) { below += part[t]; ++t; }
    int b = t * per;
    while (b < nb - 1 && below + hist[b] < rem) { below += hist[b]; ++b; }
    chosen_bin = (unsigned int)b;
    chosen_below = below;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    if (none) {
      s->threshold = 0xFFFFFFFFu;   // everything that qualifies is better than T
      s->take_equal = 0;
    } else {
      s->prefix |= chosen_bin << shift;
      s->remaining -= chosen_below;
      if (last) { s->threshold = s->prefix; s->take_equal = s->remaining; }
    }
  }
  __syncthreads();
  for (int b = threadIdx.x; b < kTopkBins; b += blockDim.x) hist[b] = 0;
}

// per block of kTopkPerBlock candidates: how many are better than T, how many equal
__global__ void __launch_bounds__(kTopkBlock) pe_topk_count_kernel(int64_t K, const int32_t* __restrict__ makespan,
                                                                   const uint32_t* __restrict__ status,
                                                                   uint32_t reject_mask, const TopkState* s,
                                                                   unsigned int* blk) {
  const unsigned int T = s->threshold;
  unsigned int better = 0, equal = 0;
  const int64_t base = (int64_t)blockIdx.x * kTopkPerBlock;
  for (int q = threadIdx.x; q < kTopkPerBlock; q += kTopkBlock) {
    const int64_t c = base + q;
    if (c < K && (status[c] & reject_mask) == 0) {
      const unsigned int v = (unsigned int)makespan[c];
      better += v < T;
      equal += v == T;
    }
  }
  for (int off = 16; off > 0; off >>= 1) {
    better += __shfl_xor_sync(0xFFFFFFFFu, better, off);
    equal += __shfl_xor_sync(0xFFFFFFFFu, equal, off);
  }
  __shared__ unsigned int sb[kTopkBlock / 32], se[kTopkBlock / 32];
  if ((threadIdx.x & 31) == 0) { sb[threadIdx.x >> 5] = better; se[threadIdx.x >> 5] = equal; }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int b = 0, e = 0;
    for (int w = 0; w < kTopkBlock / 32; ++w) { b += sb[w]; e += se[w]; }
    blk[2 * blockIdx.x] = b;
    blk[2 * blockIdx.x + 1] = e;
  }
}

// one block: exclusive scan of the per-block counts, in place
__global__ void __launch_bounds__(kTopkBlock) pe_topk_scan_kernel(unsigned int* blk, int nblocks) {
  __shared__ unsigned int sb[kTopkBlock], se[kTopkBlock];
  __shared__ unsigned int carry_b, carry_e;
  if (threadIdx.x == 0) { carry_b = 0; carry_e = 0; }
  __syncthreads();
  for (int base = 0; base < nblocks; base += kTopkBlock) {
    const int i = base + threadIdx.x;
    const unsigned int b = i < nblocks ? blk[2 * i] : 0u, e = i < nblocks ? blk[2 * i + 1] : 0u;
    sb[threadIdx.x] = b; se[threadIdx.x] = e;
    __syncthreads();
    for (int off = 1; off < kTopkBlock; off <<= 1) {   // inclusive scan of the chunk
      const unsigned int pb = threadIdx.x >= off ? sb[threadIdx.x - off] : 0u;
      const unsigned int pe_ = threadIdx.x >= off ? se[threadIdx.x - off] : 0u;
      __syncthreads();
      sb[threadIdx.x] += pb; se[threadIdx.x] += pe_;
      __syncthreads();
    }
    if (i < nblocks) { blk[2 * i] = carry_b + sb[threadIdx.x] - b; blk[2 * i + 1] = carry_e + se[threadIdx.x] - e; }
    __syncthreads();
    if (threadIdx.x == 0) { carry_b += sb[kTopkBlock - 1]; carry_e += se[kTopkBlock - 1]; }
    __syncthreads();
  }
}

// A candidate is taken if it is better than T, or equal to T with fewer than take_equal equal ones before it.
// Its place in the output is the number of taken candidates before it, which is
// better_before + min(equal_before, take_equal): the list comes out ordered by candidate index.
__global__ void __launch_bounds__(kTopkBlock) pe_topk_write_kernel(int64_t K, const int32_t* __restrict__ makespan,
                                                                   const uint32_t* __restrict__ status,
                                                                   uint32_t reject_mask, const TopkState* s,
                                                                   const unsigned int* blk, int32_t k,
                                                                   int32_t* out_index, int32_t* out_count) {
  constexpr int kPer = kTopkPerBlock / kTopkBlock;   // consecutive candidates per thread
  const unsigned int T = s->threshold, take_equal = s->take_equal;
  const int64_t first = (int64_t)blockIdx.x * kTopkPerBlock + (int64_t)threadIdx.x * kPer;
  unsigned int flag_b = 0, flag_e = 0, nb = 0, ne = 0;
  for (int q = 0; q < kPer; ++q) {
    const int64_t c = first + q;
    if (c < K && (status[c] & reject_mask) == 0) {
      const unsigned int v = (unsigned int)makespan[c];
      if (v < T) { flag_b |= 1u << q; ++nb; }
      if (v == T) { flag_e |= 1u << q; ++ne; }
    }
  }
  // exclusive scan of (nb, ne) over the block's threads
  unsigned int pb = nb, pe_ = ne;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned int ub = __shfl_up_sync(0xFFFFFFFFu, pb, off), ue = __shfl_up_sync(0xFFFFFFFFu, pe_, off);
    if (lane >= off) { pb += ub; pe_ += ue; }
  }
  __shared__ unsigned int wb[kTopkBlock / 32], we[kTopkBlock / 32];
  if (lane == 31) { wb[warp] = pb; we[warp] = pe_; }
  __syncthreads();
  unsigned int before_b = blk[2 * blockIdx.x] + pb - nb, before_e = blk[2 * blockIdx.x + 1] + pe_ - ne;
  for (int w = 0; w < warp; ++w) { before_b += wb[w]; before_e += we[w]; }
  for (int q = 0; q < kPer; ++q) {
    const bool isb = (flag_b >> q) & 1u, ise = (flag_e >> q) & 1u;
    if (isb || (ise && before_e < take_equal)) {
      const unsigned int at = before_b + (before_e < take_equal ? before_e : take_equal);
      if (at < (unsigned int)k) out_index[at] = (int32_t)(first + q);
    }
    before_b += isb;
    before_e += ise;
  }
  if (blockIdx.x == gridDim.x - 1 && threadIdx.x == kTopkBlock - 1) {   // the totals end here
    const unsigned int total = before_b + (before_e < take_equal ? before_e : take_equal);
    *out_count = (int32_t)(total < (unsigned int)k ? total : (unsigned int)k);
  }
}

__global__ void pe_topk_fill_kernel(int32_t* out_index, int32_t k) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < k; i += gridDim.x * blockDim.x) out_index[i] = -1;
}

static size_t topk_blocks(int64_t K) { return (size_t)((K + kTopkPerBlock - 1) / kTopkPerBlock); }

}  // namespace pe

extern "C" size_t pe_select_topk_workspace_bytes(int64_t K) {
  if (K < 0) return 0;
  return sizeof(pe::TopkState) + sizeof(unsigned int) * (pe::kTopkBins + 2 * (pe::topk_blocks(K) + 1));
}

extern "C" int pe_select_topk(int64_t K, const int32_t* makespan, const uint32_t* status, uint32_t reject_mask,
                              int32_t k, int32_t* out_index, int32_t* out_count, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  if (K < 0 || k < 0 || !out_count || (k > 0 && !out_index) || (K > 0 && (!makespan || !status))) return PE_ERR_INVALID_ARG;
  if (K > 0x7FFFFFFFll) return PE_ERR_INVALID_ARG;   // indices are int32
  if (!workspace || workspace_bytes < pe_select_topk_workspace_bytes(K) || ((uintptr_t)workspace & 15u))
    return PE_ERR_WORKSPACE;
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, out_count) != cudaSuccess ||
      (attr.type != cudaMemoryTypeDevice && attr.type != cudaMemoryTypeManaged)) {
    cudaGetLastError();
    return PE_ERR_INVALID_ARG;
  }
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != attr.device && cudaSetDevice(attr.device) != cudaSuccess) return PE_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  pe::TopkState* st = static_cast<pe::TopkState*>(workspace);
  unsigned int* hist = reinterpret_cast<unsigned int*>(st + 1);
  unsigned int* blk = hist + pe::kTopkBins;
  const int nblocks = (int)pe::topk_blocks(K);
  int grid = (int)((K + pe::kTopkBlock - 1) / pe::kTopkBlock);
  if (grid > 1184) grid = 1184;
  if (grid < 1) grid = 1;
  if (k > 0) pe::pe_topk_fill_kernel<<<(k + 255) / 256 > 256 ? 256 : (k + 255) / 256, 256, 0, stream>>>(out_index, k);
  pe::pe_topk_init_kernel<<<1, 256, 0, stream>>>(st, hist, (unsigned int)k);
  const int shifts[3] = {21, 10, 0}, bits[3] = {11, 11, 10};
  for (int p = 0; p < 3; ++p) {
    pe::pe_topk_hist_kernel<<<grid, pe::kTopkBlock, 0, stream>>>(K, makespan, status, reject_mask, st, hist, shifts[p],
                                                                 bits[p], p == 0);
    pe::pe_topk_pick_kernel<<<1, pe::kTopkBlock, 0, stream>>>(st, hist, shifts[p], bits[p], p == 0, p == 2);
  }
  if (nblocks > 0) {
    pe::pe_topk_count_kernel<<<nblocks, pe::kTopkBlock, 0, stream>>>(K, makespan, status, reject_mask, st, blk);
    pe::pe_topk_scan_kernel<<<1, pe::kTopkBlock, 0, stream>>>(blk, nblocks);
    pe::pe_topk_write_kernel<<<nblocks, pe::kTopkBlock, 0, stream>>>(K, makespan, status, reject_mask, st, blk, k,
                                                                      out_index, out_count);
  } else {
    cudaMemsetAsync(out_count, 0, sizeof(int32_t), stream);
  }
  const int ret = cudaGetLastError() == cudaSuccess ? PE_OK : PE_ERR_CUDA;
  if (prev != attr.device) cudaSetDevice(prev);
  return ret;
}

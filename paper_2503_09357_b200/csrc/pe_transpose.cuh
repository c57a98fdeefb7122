// Tiled transposition between the candidate-interleaved arrays of the interface ([rows][K]) and
// candidate-major staging copies ([K][rows padded]).  A block of pe_eval_team_kernel works on one
// candidate; with the interleaved layout every one of its loads and stores would touch its own
// 32-byte sector (2 or 4 useful bytes each), with the staging copy it moves whole lines.  The
// transposition itself reads and writes 128 contiguous bytes per warp instruction on both sides.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace pe {

// in:  [R][in_ld] elements of S bytes, columns 0..C-1 used; out: [C][out_ld], columns 0..R-1 written
// (and zeros up to the next multiple of 4 / S).  C * S, in_ld * S and out_ld * S must be multiples of 4
// and both bases 4-byte aligned.  One block moves a tile of 32*G rows by 32*G columns (G = 4 / S
// elements per 32-bit word) through shared memory; word (r, cw) of the tile is kept at column
// (cw + r / G) mod 32, which makes both the row-wise writes and the G-rows-per-lane reads free of bank
// conflicts.  grid = (ceil(C / (32 G)), ceil(R / (32 G))), 256 threads.
template <int S>
__global__ void __launch_bounds__(256) pe_transpose_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out,
                                                           int64_t R, int64_t C, int64_t in_ld, int64_t out_ld) {
  constexpr int G = 4 / S;
  constexpr int TR = 32 * G;   // tile rows = tile columns (elements)
  __shared__ uint32_t tile[TR][32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t r0 = (int64_t)blockIdx.y * TR, c0 = (int64_t)blockIdx.x * TR;
  const uint32_t* in_w = reinterpret_cast<const uint32_t*>(in);
  uint32_t* out_w = reinterpret_cast<uint32_t*>(out);
  const int64_t in_ldw = in_ld / G, out_ldw = out_ld / G;   // row pitches in words
  const int64_t cw0 = c0 / G, rw0 = r0 / G;
  const int64_t Cw = C / G;                                  // words per input row
  const int64_t Rw = (R + G - 1) / G;                        // words per output row
  // load: row r of the tile, lanes over the 32 words of the row
  for (int r = warp; r < TR; r += 8) {
    const int64_t rr = r0 + r;
    uint32_t w = 0;
    if (rr < R && cw0 + lane < Cw) w = in_w[rr * in_ldw + cw0 + lane];
    tile[r][(lane + r / G) & 31] = w;
  }
  __syncthreads();
  // store: word column cw of the tile holds G input columns; lane t owns input rows G t .. G t + G - 1
  for (int cw = warp; cw < 32; cw += 8) {
    uint32_t v[G];
#pragma unroll
    for (int q = 0; q < G; ++q) v[q] = tile[G * lane + q][(cw + lane) & 31];
    uint32_t o[G];
    if constexpr (G == 1) {
      o[0] = v[0];
    } else if constexpr (G == 2) {   // 2 x 2 halfwords
      o[0] = __byte_perm(v[0], v[1], 0x5410);
      o[1] = __byte_perm(v[0], v[1], 0x7632);
    } else {                         // 4 x 4 bytes
      const uint32_t t0 = __byte_perm(v[0], v[1], 0x5140), t1 = __byte_perm(v[2], v[3], 0x5140);
      const uint32_t t2 = __byte_perm(v[0], v[1], 0x7362), t3 = __byte_perm(v[2], v[3], 0x7362);
      o[0] = __byte_perm(t0, t1, 0x5410);
      o[1] = __byte_perm(t0, t1, 0x7632);
      o[2] = __byte_perm(t2, t3, 0x5410);
      o[3] = __byte_perm(t2, t3, 0x7632);
    }
#pragma unroll
    for (int q = 0; q < G; ++q) {
      const int64_t cc = c0 + (int64_t)G * cw + q;   // input column = output row
      if (cc < C && rw0 + lane < Rw) out_w[cc * out_ldw + rw0 + lane] = o[q];
    }
  }
}

}  // namespace pe

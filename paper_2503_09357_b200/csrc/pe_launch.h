// Internal: launch plan and the launchers of the compact-graph kernels (each family of
// kernel instantiations lives in its own translation unit so that they compile in parallel).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "pe_graph.h"

namespace pe {

struct Plan {
  int variant = 0;        // PE_VARIANT_* value
  int threads = 0;        // block size
  size_t smem = 0;        // dynamic shared memory per block
  bool graph_smem = false;  // graph blob staged into shared memory
  size_t workspace = 0;   // bytes of caller workspace
  size_t ws_x_off = 0;    // offset of the machine-state array inside the workspace (generic GLOBAL, by-pos)
  size_t ws_c_off = 0;    // generic GLOBAL with PE_COMM_EXCLUSIVE: offset of the per-channel array inside the workspace
  int warp_words = 0;     // WARP: 32-bit words of shared memory per candidate
  bool compact = false;   // SHARED / GLOBAL / WARP: the compact-graph kernels
  bool exclusive = false; // SHARED (compact): PE_COMM_EXCLUSIVE, one more word per machine pair and candidate
  bool state16 = false;   // SHARED (compact): 16-bit state words, end << jbits | machine
  int jbits = 8;          // bits of the machine field of a state word
  bool slab = false;      // WARP (compact): order entries and times go through shared tiles, a slab at a time
  // TEAM: inputs and times go through candidate-major staging copies in the workspace, a chunk of candidates at a time
  bool staged = false;
  int64_t team_chunk = 0;   // candidates per chunk (multiple of 4)
  int64_t team_vp = 0;      // row length of the staging copies: V rounded up to a multiple of 64
  size_t team_off_order = 0, team_off_assign = 0, team_off_start = 0, team_off_finish = 0;   // offsets in a half
  size_t team_half = 0;     // bytes of one half of the workspace (two chunks are in flight)
};

// Raise a kernel's dynamic shared-memory limit to at least `bytes` on the current device.  The attribute
// belongs to the function, not to a launch, and several host threads may launch the same kernel with
// different sizes: the limit is therefore only ever raised, under a lock, so a launch that was prepared
// with a smaller size can never find the limit lowered underneath it.
bool raise_smem_limit(const void* func, size_t bytes);

template <typename Kern>
static bool set_smem(Kern kern, size_t bytes) {
  return raise_smem_limit(reinterpret_cast<const void*>(kern), bytes);
}

// pe_eval_lane_kernel: state in shared memory (plan variant SHARED) or in `gstate` (GLOBAL).
int launch_lane(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                uint32_t flags, const pe_outputs& out, uint32_t* gstate, unsigned grid, cudaStream_t stream);

// pe_eval_warp2_kernel (plan variant WARP over the compact encoding).
int launch_warp2(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                 uint32_t flags, const pe_outputs& out, unsigned grid, cudaStream_t stream);

// pe_eval_team_kernel (plan variant TEAM: one block of plan.threads / 32 warps per candidate).
// Adds the number of kernels it launched to *launches.
int launch_team(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                uint32_t flags, const pe_outputs& out, void* workspace, cudaStream_t stream, int64_t* launches);

}  // namespace pe

// Launcher of pe_eval_team_kernel (instantiated in pe_team_nw*.cu), with the staging transpositions around it.
#include "pe_team_launch.h"
#include "pe_transpose.cuh"

#include <mutex>

namespace pe {

namespace {

template <bool BY_POS>
int launch1(const TeamCall& t) {
  switch (t.p->threads / 32) {
    case 2: return launch_team_nw2(t, BY_POS);
    case 4: return launch_team_nw4(t, BY_POS);
    case 6: return launch_team_nw6(t, BY_POS);
    default: return PE_ERR_UNSUPPORTED;
  }
}

// out[C][out_ld] = transposed in[R][in_ld] (element size S)
template <int S>
void transpose(const void* in, void* out, int64_t R, int64_t C, int64_t in_ld, int64_t out_ld, cudaStream_t stream) {
  constexpr int TR = 32 * (4 / S);
  const dim3 grid((unsigned)((C + TR - 1) / TR), (unsigned)((R + TR - 1) / TR));
  pe_transpose_kernel<S><<<grid, 256, 0, stream>>>(static_cast<const uint8_t*>(in), static_cast<uint8_t*>(out), R, C, in_ld,
                                                   out_ld);
}

}  // namespace

int launch_team(const pe_graph* g, const Plan& p, bool by_pos, int64_t K, const uint8_t* assign, const uint16_t* order,
                uint32_t flags, const pe_outputs& out, void* workspace, cudaStream_t stream, int64_t* launches) {
  TeamCall t;
  t.g = g; t.p = &p; t.K = K; t.flags = flags; t.stream = stream;
  if (!p.staged) {
    t.kc = K; t.assign = assign; t.order = order; t.out = out;
    t.sd.in_row = (size_t)K; t.sd.in_cand = 1; t.sd.out_row = (size_t)K; t.sd.out_cand = 1;
    *launches += 1;
    return by_pos ? launch1<true>(t) : launch1<false>(t);
  }
  // staged: chunks of candidates go through candidate-major copies in the workspace.  Consecutive chunks
  // use the two halves of the workspace and the graph's two side streams, so the transpositions of one
  // chunk run while the other is evaluated, and the tail of one evaluation overlaps the head of the next.
  const int64_t V = g->V, Vp = p.team_vp;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  const bool times = out.start != nullptr;
  const bool fork = K > p.team_chunk;
  pe_graph* gm = const_cast<pe_graph*>(g);
  std::unique_lock<std::mutex> lock(gm->team_mutex, std::defer_lock);
  bool ok = true;
  if (fork) {
    lock.lock();
    ok = cudaEventRecord(gm->team_fork, stream) == cudaSuccess &&
         cudaStreamWaitEvent(gm->team_stream[0], gm->team_fork, 0) == cudaSuccess &&
         cudaStreamWaitEvent(gm->team_stream[1], gm->team_fork, 0) == cudaSuccess;
  }
  int rc = ok ? PE_OK : PE_ERR_CUDA;
  int q = 0;
  for (int64_t c0 = 0; c0 < K && rc == PE_OK; c0 += p.team_chunk, ++q) {
    const int64_t kc = K - c0 < p.team_chunk ? K - c0 : p.team_chunk;
    uint8_t* half = ws + (size_t)(q & 1) * p.team_half;
    uint16_t* ord_t = reinterpret_cast<uint16_t*>(half + p.team_off_order);
    uint8_t* asg_t = half + p.team_off_assign;
    int32_t* start_t = reinterpret_cast<int32_t*>(half + p.team_off_start);
    int32_t* finish_t = reinterpret_cast<int32_t*>(half + p.team_off_finish);
    t.stream = fork ? gm->team_stream[q & 1] : stream;
    transpose<2>(order + c0, ord_t, V, kc, K, Vp, t.stream);
    transpose<1>(assign + c0, asg_t, V, kc, K, Vp, t.stream);
    t.kc = kc; t.assign = asg_t; t.order = ord_t;
    t.out.start = times ? start_t : nullptr;
    t.out.finish = times ? finish_t : nullptr;
    t.out.makespan = out.makespan ? out.makespan + c0 : nullptr;
    t.out.status = out.status ? out.status + c0 : nullptr;
    t.out.busy = out.busy ? out.busy + c0 : nullptr;
    t.out.peak_mem = out.peak_mem ? out.peak_mem + c0 : nullptr;
    t.sd.in_row = 1; t.sd.in_cand = (size_t)Vp; t.sd.out_row = 1; t.sd.out_cand = (size_t)Vp;
    rc = by_pos ? launch1<true>(t) : launch1<false>(t);
    if (rc != PE_OK) break;
    *launches += 3;
    if (times) {
      transpose<4>(start_t, out.start + c0, kc, V, Vp, K, t.stream);
      transpose<4>(finish_t, out.finish + c0, kc, V, Vp, K, t.stream);
      *launches += 2;
    }
  }
  if (fork) {   // join, also after an error: nothing of this call may stay unordered on the side streams
    for (int b = 0; b < 2; ++b)
      if (cudaEventRecord(gm->team_join[b], gm->team_stream[b]) != cudaSuccess ||
          cudaStreamWaitEvent(stream, gm->team_join[b], 0) != cudaSuccess)
        rc = rc == PE_OK ? PE_ERR_CUDA : rc;
  }
  return rc;
}

}  // namespace pe

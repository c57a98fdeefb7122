// Host side of the library: description checks, by-predecessor CSR, upload, teardown.
#include <climits>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "pe_device.cuh"
#include "pe_graph.h"

namespace {

inline uint32_t align16(uint64_t x) { return (uint32_t)((x + 15u) & ~(uint64_t)15u); }

// Ranges, acyclicity and overflow bounds; fills the bounds when asked.
int check_desc(const pe_graph_desc* d, int64_t* time_bound, int64_t* mem_bound, int32_t* max_indeg) {
  if (!d) return PE_ERR_INVALID_ARG;
  const int32_t V = d->num_ops, E = d->num_edges, D = d->num_devices, L = d->num_link_classes;
  if (V < 1 || E < 0 || D < 1 || D > 255 || L < 1 || L > 254) return PE_ERR_INVALID_ARG;
  if (!d->dur || (E > 0 && (!d->edge_src || !d->edge_dst))) return PE_ERR_INVALID_ARG;
  if ((int64_t)E * L > (int64_t)INT32_MAX) return PE_ERR_INVALID_ARG;

  int64_t tsum = 0, msum = 0;
  for (int32_t i = 0; i < V; ++i) {
    if (d->dur[i] < 0) return PE_ERR_RANGE;
    int64_t longest = d->dur[i];
    if (d->dur_by_machine) {   // heterogeneous machines: the bound takes the slowest machine
      longest = 0;
      for (int32_t j = 0; j < D; ++j) {
        const int32_t t = d->dur_by_machine[(size_t)i * D + j];
        if (t < 0) return PE_ERR_RANGE;
        if (t > longest) longest = t;
      }
    }
    tsum += longest;
    if (d->mem_delta) msum += d->mem_delta[i] < 0 ? -(int64_t)d->mem_delta[i] : (int64_t)d->mem_delta[i];
    if (d->mem_weight) {
      if (d->mem_weight[i] < 0) return PE_ERR_RANGE;
      msum += d->mem_weight[i];
    }
  }
  std::vector<int32_t> indeg(V, 0), succ_ptr(V + 1, 0);
  for (int32_t b = 0; b < E; ++b) {
    const int32_t p = d->edge_src[b], i = d->edge_dst[b];
    if (p < 0 || p >= V || i < 0 || i >= V) return PE_ERR_RANGE;
    if (p == i) return PE_ERR_CYCLE;
    indeg[i]++;
    succ_ptr[p + 1]++;
    if (d->comm) {
      int32_t mx = 0;
      for (int32_t l = 0; l < L; ++l) {
        const int32_t cst = d->comm[(size_t)b * L + l];
        if (cst < 0) return PE_ERR_RANGE;
        if (cst > mx) mx = cst;
      }
      tsum += mx;
    }
  }
  if (d->link_class)
    for (int32_t a = 0; a < D * D; ++a)
      if (d->link_class[a] != 0xFF && d->link_class[a] >= L) return PE_ERR_RANGE;
  if (tsum > (int64_t)INT32_MAX || msum > (int64_t)INT32_MAX) return PE_ERR_OVERFLOW;

  // acyclic iff Kahn's algorithm removes every operator
  int32_t mdeg = 0;
  for (int32_t i = 0; i < V; ++i) {
    succ_ptr[i + 1] += succ_ptr[i];
    if (indeg[i] > mdeg) mdeg = indeg[i];
  }
  std::vector<int32_t> succ(E), fill(succ_ptr.begin(), succ_ptr.end() - 1), deg(indeg), stack;
  for (int32_t b = 0; b < E; ++b) succ[fill[d->edge_src[b]]++] = d->edge_dst[b];
  for (int32_t i = 0; i < V; ++i)
    if (deg[i] == 0) stack.push_back(i);
  int32_t removed = 0;
  while (!stack.empty()) {
    const int32_t i = stack.back();
    stack.pop_back();
    ++removed;
    for (int32_t q = succ_ptr[i]; q < succ_ptr[i + 1]; ++q)
      if (--deg[succ[q]] == 0) stack.push_back(succ[q]);
  }
  if (removed != V) return PE_ERR_CYCLE;

  if (time_bound) *time_bound = tsum;
  if (mem_bound) *mem_bound = msum;
  if (max_indeg) *max_indeg = mdeg;
  return PE_OK;
}

}  // namespace

extern "C" int pe_graph_validate(const pe_graph_desc* desc) { return check_desc(desc, nullptr, nullptr, nullptr); }

extern "C" int pe_graph_create(const pe_graph_desc* d, int cuda_device, pe_graph** out) {
  if (!out) return PE_ERR_INVALID_ARG;
  *out = nullptr;
  int64_t tb = 0, mb = 0;
  int32_t mdeg = 0;
  const int rc = check_desc(d, &tb, &mb, &mdeg);
  if (rc != PE_OK) return rc;
  const int32_t V = d->num_ops, E = d->num_edges, D = d->num_devices, L = d->num_link_classes;

  pe_graph* g = new (std::nothrow) pe_graph();
  if (!g) return PE_ERR_INVALID_ARG;
  g->V = V; g->E = E; g->D = D; g->L = L;
  g->device = cuda_device;
  g->has_weight = d->mem_weight != nullptr;
  g->hetero = d->dur_by_machine != nullptr;
  g->time_bound = tb; g->mem_bound = mb; g->max_indeg = mdeg;
  g->d_blob = nullptr; g->d_error = nullptr;

  PeBlobLayout& lay = g->lay;
  uint64_t at = 0;
  lay.ops = (uint32_t)at;    at = align16(at + (uint64_t)V * sizeof(PeOpRec));
  lay.pred = (uint32_t)at;   at = align16(at + (uint64_t)E * 4);
  lay.comm = (uint32_t)at;   at = align16(at + (uint64_t)E * L * 4);
  lay.weight = (uint32_t)at; at = align16(at + (g->has_weight ? (uint64_t)V * 4 : 0));
  lay.cls = (uint32_t)at;    at = align16(at + (uint64_t)D * D);
  lay.cap = (uint32_t)at;    at = align16(at + (uint64_t)D * 4);
  lay.durm = (uint32_t)at;   at = align16(at + (g->hetero ? (uint64_t)V * D * 4 : 0));
  if (at > 0x7FFFFFF0ull) { delete g; return PE_ERR_INVALID_ARG; }
  lay.bytes = (uint32_t)at;

  // by-predecessor CSR: incoming edges of operator i occupy slots edge_begin .. edge_begin + indeg
  std::vector<uint8_t> blob(lay.bytes, 0);
  PeOpRec* ops = (PeOpRec*)(blob.data() + lay.ops);
  int32_t* pred = (int32_t*)(blob.data() + lay.pred);
  int32_t* comm = (int32_t*)(blob.data() + lay.comm);
  for (int32_t i = 0; i < V; ++i) {
    ops[i].indeg = 0;
    ops[i].dur = d->dur[i];
    ops[i].mem_delta = d->mem_delta ? d->mem_delta[i] : 0;
  }
  for (int32_t b = 0; b < E; ++b) ops[d->edge_dst[b]].indeg++;
  int32_t run = 0;
  for (int32_t i = 0; i < V; ++i) { ops[i].edge_begin = run; run += ops[i].indeg; }
  {
    std::vector<int32_t> fill(V);
    for (int32_t i = 0; i < V; ++i) fill[i] = ops[i].edge_begin;
    for (int32_t b = 0; b < E; ++b) {
      const int32_t q = fill[d->edge_dst[b]]++;
      pred[q] = d->edge_src[b];
      for (int32_t l = 0; l < L; ++l) comm[(size_t)q * L + l] = d->comm ? d->comm[(size_t)b * L + l] : 0;
    }
  }
  if (g->has_weight) std::memcpy(blob.data() + lay.weight, d->mem_weight, (size_t)V * 4);
  if (d->link_class) std::memcpy(blob.data() + lay.cls, d->link_class, (size_t)D * D);
  if (g->hetero) std::memcpy(blob.data() + lay.durm, d->dur_by_machine, (size_t)V * D * 4);
  int32_t* cap = (int32_t*)(blob.data() + lay.cap);
  for (int32_t j = 0; j < D; ++j) cap[j] = d->mem_capacity ? d->mem_capacity[j] : INT32_MAX;

  // compact encoding, when every value fits its field
  bool no_channel = false;
  if (d->link_class)
    for (int32_t a = 0; a < D * D; ++a) no_channel = no_channel || d->link_class[a] == 0xFF;
  bool narrow = V <= 65535 && L <= 2 && mdeg <= 255 && E < (1 << 24) && !g->hetero;   // (the compact record has one duration)
  for (int32_t i = 0; narrow && i < V; ++i)
    narrow = ops[i].dur <= 65535 && ops[i].mem_delta >= -128 && ops[i].mem_delta <= 127;
  for (int64_t q = 0; narrow && q < (int64_t)E * L; ++q) narrow = comm[q] <= 65535;
  std::vector<uint8_t> nblob;
  g->narrow_ok = narrow;
  g->d_nblob = nullptr;
  std::memset(&g->nview, 0, sizeof(g->nview));
  if (narrow) {
    PeNarrowView& nv = g->nview;
    nv.V = V; nv.E = E; nv.D = D; nv.L = L;
    nv.has_weight = g->has_weight ? 1 : 0;
    nv.need_cls = (L > 1 || no_channel) ? 1 : 0;
    nv.max_indeg = mdeg;
    uint64_t nat = 0;
    nv.ops = (uint32_t)nat;    nat = align16(nat + (uint64_t)V * 16);
    nv.edges = (uint32_t)nat;  nat = align16(nat + (uint64_t)E * 4 * L);
    nv.weight = (uint32_t)nat; nat = align16(nat + (g->has_weight ? (uint64_t)V * 4 : 0));
    nv.cls = (uint32_t)nat;    nat = align16(nat + (uint64_t)D * D);
    nv.cap = (uint32_t)nat;    nat = align16(nat + (uint64_t)D * 4);
    nv.bytes = (uint32_t)nat;
    nblob.assign(nv.bytes, 0);
    uint32_t* nops = (uint32_t*)(nblob.data() + nv.ops);
    uint32_t* nedges = (uint32_t*)(nblob.data() + nv.edges);
    for (int32_t q = 0; q < E; ++q) {
      const uint32_t lo = ((uint32_t)comm[(size_t)q * L] << 16) | (uint32_t)pred[q];
      if (L == 1) nedges[q] = lo;
      else { nedges[2 * (size_t)q] = lo; nedges[2 * (size_t)q + 1] = (uint32_t)comm[(size_t)q * L + 1]; }
    }
    for (int32_t i = 0; i < V; ++i) {
      uint32_t* r = nops + 4 * (size_t)i;
      const int32_t b = ops[i].edge_begin, n = ops[i].indeg;
      r[1] = ((uint32_t)n << 24) | ((uint32_t)(uint8_t)(int8_t)ops[i].mem_delta << 16) | (uint32_t)ops[i].dur;
      // a missing inline edge points at the sentinel operator V (always "ended at 0", zero delay)
      const uint32_t none = (uint32_t)V;
      if (L == 1) {
        r[2] = n > 0 ? nedges[b] : none;
        r[3] = n > 1 ? nedges[b + 1] : none;
        r[0] = n > 3 ? (uint32_t)b : (n > 2 ? nedges[b + 2] : none);
      } else {
        r[2] = n > 0 ? nedges[2 * (size_t)b] : none;
        r[3] = n > 0 ? nedges[2 * (size_t)b + 1] : 0u;
        r[0] = (uint32_t)b;
      }
    }
    if (g->has_weight) std::memcpy(nblob.data() + nv.weight, d->mem_weight, (size_t)V * 4);
    if (d->link_class) std::memcpy(nblob.data() + nv.cls, d->link_class, (size_t)D * D);
    std::memcpy(nblob.data() + nv.cap, cap, (size_t)D * 4);
  }

  // forward view (successor lists) for priority-list decoding
  std::vector<uint8_t> fblob;
  g->fwd_ok = V <= 65536 && mdeg <= 255;
  g->d_fwd = nullptr;
  std::memset(&g->fview, 0, sizeof(g->fview));
  if (g->fwd_ok) {
    PeFwdView& fv = g->fview;
    fv.V = V; fv.E = E;
    uint64_t fat = 0;
    fv.ptr = (uint32_t)fat;   fat = align16(fat + (uint64_t)(V + 1) * 4);
    fv.succ = (uint32_t)fat;  fat = align16(fat + (uint64_t)E * 2);
    fv.indeg = (uint32_t)fat; fat = align16(fat + (uint64_t)V);
    fv.bytes = (uint32_t)fat;
    fblob.assign(fv.bytes, 0);
    uint32_t* fptr = (uint32_t*)(fblob.data() + fv.ptr);
    uint16_t* fsucc = (uint16_t*)(fblob.data() + fv.succ);
    uint8_t* findeg = fblob.data() + fv.indeg;
    for (int32_t b = 0; b < E; ++b) fptr[d->edge_src[b] + 1]++;
    for (int32_t i = 0; i < V; ++i) { fptr[i + 1] += fptr[i]; findeg[i] = (uint8_t)ops[i].indeg; }
    std::vector<uint32_t> ffill(fptr, fptr + V);
    for (int32_t b = 0; b < E; ++b) fsucc[ffill[d->edge_src[b]]++] = (uint16_t)d->edge_dst[b];
  }

  cudaDeviceProp prop;
  int prev = -1;
  bool ok = cudaGetDevice(&prev) == cudaSuccess && cudaSetDevice(cuda_device) == cudaSuccess &&
            cudaGetDeviceProperties(&prop, cuda_device) == cudaSuccess;
  if (ok) {
    g->sm_count = prop.multiProcessorCount;
    g->smem_optin = prop.sharedMemPerBlockOptin;
    g->smem_per_sm = prop.sharedMemPerMultiprocessor;
    ok = cudaMalloc((void**)&g->d_blob, lay.bytes) == cudaSuccess &&
         cudaMalloc((void**)&g->d_error, 256) == cudaSuccess &&
         cudaMemcpy(g->d_blob, blob.data(), lay.bytes, cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemset(g->d_error, 0, 256) == cudaSuccess;
    if (ok && narrow)
      ok = cudaMalloc((void**)&g->d_nblob, nblob.size()) == cudaSuccess &&
           cudaMemcpy(g->d_nblob, nblob.data(), nblob.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    if (ok && g->fwd_ok)
      ok = cudaMalloc((void**)&g->d_fwd, fblob.size()) == cudaSuccess &&
           cudaMemcpy(g->d_fwd, fblob.data(), fblob.size(), cudaMemcpyHostToDevice) == cudaSuccess;
    if (ok) {
      ok = cudaStreamCreateWithFlags(&g->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
           cudaStreamCreateWithFlags(&g->copy_out, cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&g->ev_begin, cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&g->ev_end, cudaEventDisableTiming) == cudaSuccess &&
           cudaStreamCreateWithFlags(&g->team_stream[0], cudaStreamNonBlocking) == cudaSuccess &&
           cudaStreamCreateWithFlags(&g->team_stream[1], cudaStreamNonBlocking) == cudaSuccess &&
           cudaEventCreateWithFlags(&g->team_fork, cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&g->team_join[0], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&g->team_join[1], cudaEventDisableTiming) == cudaSuccess;
      for (int q = 0; ok && q < pe_graph::kMaxChunks; ++q)
        ok = cudaEventCreateWithFlags(&g->ev_in[q], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&g->ev_done[q], cudaEventDisableTiming) == cudaSuccess;
    }
  }
  if (prev >= 0) cudaSetDevice(prev);
  if (!ok) {
    cudaGetLastError();
    if (g->d_blob) cudaFree(g->d_blob);
    if (g->d_error) cudaFree(g->d_error);
    if (g->d_nblob) cudaFree(g->d_nblob);
    if (g->d_fwd) cudaFree(g->d_fwd);
    if (g->copy_in) cudaStreamDestroy(g->copy_in);
    if (g->copy_out) cudaStreamDestroy(g->copy_out);
    if (g->ev_begin) cudaEventDestroy(g->ev_begin);
    if (g->ev_end) cudaEventDestroy(g->ev_end);
    for (int q = 0; q < 2; ++q) {
      if (g->team_stream[q]) cudaStreamDestroy(g->team_stream[q]);
      if (g->team_join[q]) cudaEventDestroy(g->team_join[q]);
    }
    if (g->team_fork) cudaEventDestroy(g->team_fork);
    for (int q = 0; q < pe_graph::kMaxChunks; ++q) {
      if (g->ev_in[q]) cudaEventDestroy(g->ev_in[q]);
      if (g->ev_done[q]) cudaEventDestroy(g->ev_done[q]);
    }
    cudaGetLastError();
    delete g;
    return PE_ERR_CUDA;
  }
  *out = g;
  return PE_OK;
}

extern "C" int pe_destroy(pe_graph* g) {
  if (!g) return PE_OK;
  int prev = -1;
  cudaGetDevice(&prev);
  cudaSetDevice(g->device);
  cudaStreamDestroy(g->copy_in);
  cudaStreamDestroy(g->copy_out);
  cudaEventDestroy(g->ev_begin);
  cudaEventDestroy(g->ev_end);
  for (int q = 0; q < 2; ++q) { cudaStreamDestroy(g->team_stream[q]); cudaEventDestroy(g->team_join[q]); }
  cudaEventDestroy(g->team_fork);
  for (int q = 0; q < pe_graph::kMaxChunks; ++q) { cudaEventDestroy(g->ev_in[q]); cudaEventDestroy(g->ev_done[q]); }
  bool ok = cudaFree(g->d_blob) == cudaSuccess && cudaFree(g->d_error) == cudaSuccess;
  if (g->d_nblob) ok = cudaFree(g->d_nblob) == cudaSuccess && ok;
  if (g->d_fwd) ok = cudaFree(g->d_fwd) == cudaSuccess && ok;
  if (prev >= 0) cudaSetDevice(prev);
  delete g;
  return ok ? PE_OK : PE_ERR_CUDA;
}

extern "C" int pe_graph_poll_error(pe_graph* g, void* cuda_stream) {
  if (!g) return PE_ERR_INVALID_ARG;
  int word = 0;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return PE_ERR_CUDA;
  if (cudaMemcpy(&word, g->d_error, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return PE_ERR_CUDA;
  if (word != 0 && cudaMemset(g->d_error, 0, sizeof(int)) != cudaSuccess) return PE_ERR_CUDA;
  return word;
}

// Self-test of the bounded wait: the barrier is told to expect bytes that no copy will ever bring, so the
// wait runs out after `limit` polls, the error word is set and the block returns - nothing is in flight.
__global__ void pe_selftest_wait_kernel(int* err, int limit) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) pe::mbar_init(&bar, 1);
  __syncthreads();
  if (threadIdx.x == 0) pe::mbar_expect_tx(&bar, 16);
  __syncthreads();
  if (!pe::mbar_wait_bounded(&bar, 0, limit)) atomicExch(err, PE_ERR_TIMEOUT);
}

extern "C" int pe_selftest_wait_timeout(pe_graph* g, void* cuda_stream) {
  if (!g) return PE_ERR_INVALID_ARG;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return PE_ERR_CUDA;
  if (prev != g->device && cudaSetDevice(g->device) != cudaSuccess) return PE_ERR_CUDA;
  pe_selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(g->d_error, 1024);
  const int ret = cudaGetLastError() == cudaSuccess ? PE_OK : PE_ERR_CUDA;
  if (prev != g->device) cudaSetDevice(prev);
  return ret;
}

extern "C" const char* pe_strerror(int code) {
  switch (code) {
    case PE_OK: return "ok";
    case PE_ERR_INVALID_ARG: return "invalid argument";
    case PE_ERR_CYCLE: return "operator graph has a cycle";
    case PE_ERR_RANGE: return "value out of range (negative duration/communication/weight, edge endpoint or link class)";
    case PE_ERR_OVERFLOW: return "time or memory bound does not fit in int32";
    case PE_ERR_CUDA: return "CUDA runtime call failed";
    case PE_ERR_WORKSPACE: return "workspace missing or too small";
    case PE_ERR_TIMEOUT: return "bounded device-side wait expired";
    case PE_ERR_UNSUPPORTED: return "kernel variant cannot run this problem size";
    case PE_ERR_SCRATCH_LIMIT: return "batch needs more scratch than the built-in no-allocation array holds";
    default: return "unknown error code";
  }
}

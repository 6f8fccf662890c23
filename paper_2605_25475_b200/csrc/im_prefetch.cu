// L2 warm-up for the latency-bound kernels of the next layer call.
//
// A decode step visits the layers in order and streams ~350 MB per layer through the 126 MB L2, so
// by the time a layer comes round again (one step later) none of its weights, indexer keys, counters
// or pending memory terms are cached, and its small kernels pay a DRAM (and page-walk) round trip for
// every dependent load.  None of that data depends on the output of the previous layer, so while the
// attention kernel of layer l streams K/V (with an evict-first policy), this kernel prefetches what
// layer (l + 1) mod n_layers will read for the same sequences, with an evict-last policy.
#include "im_internal.cuh"

namespace {

__device__ __forceinline__ void prefetch_range(const void* base, size_t bytes, size_t tid, size_t nthreads) {
  const char* p = static_cast<const char*>(base);
  for (size_t off = tid * 128; off < bytes; off += nthreads * 128)
    asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(p + off));
}

// grid = (PF_BLOCKS, 1 + n_seq): y == 0 prefetches the weights of `w`, y == 1 + i the index state of
// call sequence i in layer `call.layer` (the caller passes the NEXT layer in both).  block = 256.
constexpr int PF_BLOCKS = 8;
__global__ void __launch_bounds__(256) k_prefetch_layer(ImDims p, ImState st, ImWeights w, ImCall call) {
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t nth = (size_t)gridDim.x * blockDim.x;
  if (blockIdx.y == 0) {
    prefetch_range(w.Uq, (size_t)p.HI * p.dI * p.D * 2, tid, nth);
    prefetch_range(w.Uk, (size_t)p.dI * p.D * 2, tid, nth);
    prefetch_range(w.G, (size_t)p.HI * p.D * 2, tid, nth);
    if (p.mem) {
      prefetch_range(w.Wt, (size_t)p.dM * p.D * 2, tid, nth);
      prefetch_range(w.wg, (size_t)p.D * 2, tid, nth);
      prefetch_range(w.Wfh, (size_t)p.dM * p.Dkv * 2, tid, nth);
      prefetch_range(w.Wfl, (size_t)p.dM * p.Dkv * 2, tid, nth);
      prefetch_range(w.bg, 4, tid, nth);
    }
    return;
  }
  const int i = blockIdx.y - 1;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = max(0, min(ctr[CTR_N], p.cap));
  prefetch_range(st.kidx + u * p.cap * p.dI, (size_t)n * p.dI * 2, tid, nth);
  prefetch_range(st.imp + u * p.cap, (size_t)n * 4, tid, nth);
  prefetch_range(st.pos + u * p.cap, (size_t)n * 4, tid, nth);
  if (p.mem) {
    const int np = max(0, min(ctr[CTR_NPEND], p.F));
    prefetch_range(st.bvec + u * p.dM, (size_t)p.dM * 4, tid, nth);
    prefetch_range(st.pend_phi + u * p.F * p.dM, (size_t)np * p.dM * 4, tid, nth);
    prefetch_range(st.pend_v + u * p.F * p.Dkv, (size_t)np * p.Dkv * 2, tid, nth);
    prefetch_range(st.pend_w + u * p.F, (size_t)np * 4, tid, nth);
    prefetch_range(st.cscale + u, 4, tid, nth);
  }
}

// The memory matrices of layer `call.layer` (the NEXT layer) for the call's sequences, requested into L2 as bulk
// prefetches of 4 KB, the first `eighths` eighths of each matrix.  grid = ceil(n_seq / per_block), block = 512.  An
// SM's copy engine takes these requests at a bounded rate, so the number of blocks paces the whole prefetch: it is
// meant to trickle in next to the merge kernel and the next call's projections, not to compete with them
// (measured on the 32-layer benchmark: one block per sequence 2.24 ms per step, eight 2.33 ms).
__global__ void __launch_bounds__(512) k_prefetch_memory(ImDims p, ImState st, ImCall call, int eighths, int per_block) {
  const size_t bytes = (size_t)p.dM * p.Dkv * 4 / 8 * eighths;
  for (int i = blockIdx.x * per_block; i < min(call.n_seq, (blockIdx.x + 1) * per_block); ++i) {
    const size_t u = (size_t)call.layer * p.S + call.seq[i];
    const char* base = reinterpret_cast<const char*>(st.Mhat + u * p.dM * p.Dkv);
    for (size_t off = (size_t)threadIdx.x * 4096; off + 4096 <= bytes; off += (size_t)blockDim.x * 4096)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(base + off), "r"(4096) : "memory");
  }
}

// Marks the id of the SM a block runs on in a 256-bit map (ids beyond 255: bit 31 of word 8).  Blocks of 1024 threads
// that nap for a while, several waves of them, so that every SM gets one.
__global__ void __launch_bounds__(1024) k_probe_sm_ids(uint32_t* map) {
  if (threadIdx.x == 0) {
    unsigned smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    if (smid < 256u) atomicOr(map + (smid >> 5), 1u << (smid & 31u));
    else atomicOr(map + 8, 0x80000000u);
    __nanosleep(8000);
  }
  __syncthreads();
}

}  // namespace

// The ids (%smid) of the device's SMs, ascending, as blocks of a probe kernel report them; `map` is device scratch of
// at least 64 bytes.  *n = 0 if the ids do not number n_sm distinct values below 256 (the caller then does without).
cudaError_t im_probe_sm_ids(void* map, int n_sm, int* ids, int* n, cudaStream_t stream) {
  *n = 0;
  cudaError_t e = cudaMemsetAsync(map, 0, 64, stream);
  if (e != cudaSuccess) return e;
  k_probe_sm_ids<<<8 * n_sm, 1024, 0, stream>>>(static_cast<uint32_t*>(map));
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  uint32_t host[16];
  if ((e = cudaMemcpyAsync(host, map, 64, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return e;
  if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return e;
  if (host[8]) return cudaSuccess;
  int k = 0;
  for (int s = 0; s < 256; ++s)
    if ((host[s >> 5] >> (s & 31)) & 1u) {
      if (k < n_sm) ids[k] = s;
      ++k;
    }
  if (k == n_sm) *n = k;
  return cudaSuccess;
}

// `call.layer` names the layer to warm up.  Needs 16-byte aligned matrices whose eighth is a multiple of 4 KB.
cudaError_t im_launch_prefetch_memory(const ImLaunch& L, const ImCall& call, int eighths, int per_block) {
  if (!L.p.mem || eighths <= 0 || ((size_t)L.p.dM * L.p.Dkv * 4 / 8) % 4096) return cudaSuccess;
  if (per_block <= 0) per_block = 1;
  k_prefetch_memory<<<(call.n_seq + per_block - 1) / per_block, 512, 0, L.stream>>>(L.p, L.st, call, eighths > 8 ? 8 : eighths, per_block);
  ++*L.launches;
  return cudaGetLastError();
}

// `L.w` and `call.layer` must describe the layer to warm up (not the one being computed).
cudaError_t im_launch_prefetch_layer(const ImLaunch& L, const ImCall& call) {
  dim3 grid(PF_BLOCKS, 1 + call.n_seq);
  k_prefetch_layer<<<grid, 256, 0, L.stream>>>(L.p, L.st, L.w, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_prefetch_prepare_decode() { return im_prefer_max_smem(k_prefetch_layer); }

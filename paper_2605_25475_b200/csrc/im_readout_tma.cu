// a6, the part of the memory readout (Eq. 5) that streams the state: per sequence and column
//   rsum[col] = sum over all d_M rows m of phi(q)[m] * Mhat[m][col]
// as a persistent kernel fed by bulk copies.
//
// The kernel runs next to the streaming attention kernel, whose CTAs keep a ring of TMA copies in flight.  The
// memory system serves the requests queued on an SM roughly in proportion to the bytes each requester has in flight
// there: a readout built on plain loads (k_readout_cols) holds a few tens of KB per SM against the attention ring's
// 128-192 KB and falls behind.  Here the rows of Mhat come through a ring of 32 KB stages of their own (one untiled
// bulk copy each: 32 KB of Mhat are contiguous), so the readout's share is set by the depth of its ring.
//   * Mhat of a sequence is [d_M][D_kv] float32, row-major: a chunk is RC = 8192 / D_kv consecutive rows = 32 KB.
//     All chunks of all sequences of the call are cut into equal contiguous runs, one per CTA.
//   * warp 8 (one lane) requests chunks as stages come free; warps 0-7 consume: thread t owns the float4 column
//     t % (D_kv / 4) of the rows r = t / (D_kv / 4) (mod the number of such row groups) of every chunk and keeps one
//     float4 of partial sums per sequence of its run.
//   * at the end of a sequence's chunks within the run the row groups are added through shared memory and the CTA
//     writes one partial vector; the merge kernel adds the partial vectors of a sequence in CTA order (slot = CTA
//     index + sequence index: consecutive sequences share at most one CTA).
// Every wait is bounded; a wait that runs out sets ST_TIMEOUT and an abort flag that the other role polls, and the
// producer waits (bounded) for every copy it has in flight before the CTA ends.
#include "im_internal.cuh"

namespace {

constexpr int RO_CHUNK = 32 * 1024;          // bytes per stage
constexpr int RO_CONSUMERS = 256;
constexpr int RO_THREADS = RO_CONSUMERS + 32;
constexpr int RO_MAX_STAGES = 6;
constexpr uint32_t WAIT_LIMIT = IM_WAIT_LIMIT;

struct RoShared {
  unsigned long long full[RO_MAX_STAGES], empty[RO_MAX_STAGES];
  int abort;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit = WAIT_LIMIT) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if (abort_flag && (it & 63) == 63 && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
      ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
      : "memory");
}

// grid = CTAs, block = RO_THREADS, dynamic smem = stages * 32 KB (128-byte aligned) | phi [d_M] | red [RO_CONSUMERS] float4 | RoShared
__global__ void __launch_bounds__(RO_THREADS, 1)
k_readout_stream(ImDims p, ImState st, ImScratch sc, ImCall call, int stages) {
  extern __shared__ __align__(128) unsigned char smem[];
  float* s_phi = reinterpret_cast<float*>(smem + (size_t)stages * RO_CHUNK);
  float4* s_red = reinterpret_cast<float4*>(s_phi + ((p.dM + 3) & ~3));
  RoShared* sh = reinterpret_cast<RoShared*>(s_red + RO_CONSUMERS);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh->abort;
  const int C4 = p.Dkv / 4;              // float4 columns of a row (divides RO_CONSUMERS: checked by the launcher)
  const int G = RO_CONSUMERS / C4;       // row groups
  const int RC = RO_CHUNK / (p.Dkv * 4); // rows per chunk (divides d_M: checked by the launcher)
  const int CS = p.dM / RC;              // chunks per sequence
  const long long total = (long long)call.n_seq * CS;
  const long long qrun = (total + gridDim.x - 1) / gridDim.x;
  const long long run0 = min(total, (long long)blockIdx.x * qrun), run1 = min(total, run0 + qrun);
  if (tid == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), RO_CONSUMERS / 32);
    }
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (warp == RO_CONSUMERS / 32) {
    // ================= producer (one lane)
    long long issued = run0;
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      for (; issued < run1; ++issued) {
        const long long k = issued - run0;
        const int s = (int)(k % stages);
        if (k >= stages && !mbar_wait(smem_u32(&sh->empty[s]), (uint32_t)(((k / stages) - 1) & 1), abort_flag)) { ok = false; break; }
        const int i = (int)(issued / CS), c = (int)(issued % CS);
        const size_t u = (size_t)call.layer * p.S + call.seq[i];
        const float* src = st.Mhat + u * p.dM * (size_t)p.Dkv + (size_t)c * RC * p.Dkv;
        const uint32_t bar = smem_u32(&sh->full[s]);
        mbar_expect_tx(bar, RO_CHUNK);
        bulk_load(smem_u32(smem + (size_t)s * RO_CHUNK), src, RO_CHUNK, bar, pol);
      }
      if (!ok) {
        sh->abort = 1;
        atomicOr(st.status, ST_TIMEOUT);
      }
      // every copy requested must have landed before the CTA ends (after a normal run these return at once)
      for (long long j = max(run0, issued - stages); j < issued; ++j)
        if (!mbar_wait(smem_u32(&sh->full[(j - run0) % stages]), (uint32_t)(((j - run0) / stages) & 1), nullptr)) atomicOr(st.status, ST_TIMEOUT);
    }
  } else {
    // ================= consumers: thread t owns float4 column col4 of the rows grp, grp + G, ... of every chunk
    const int col4 = tid % C4, grp = tid / C4;
    const ImRows r = im_rows(p);
    long long j = run0;
    bool fail = false;
    while (j < run1) {
      const int i = (int)(j / CS);
      const long long seq_end = min(run1, (long long)(i + 1) * CS);
      // phi(q) of the sequence (K-split partials of the projection summed in a fixed order)
      asm volatile("bar.sync 1, %0;" ::"n"(RO_CONSUMERS) : "memory");  // the previous sequence's readers of s_phi / s_red are done
      for (int m = tid; m < p.dM; m += RO_CONSUMERS) s_phi[m] = im_raw_sum(p, sc, call, i, r.theta + m);
      asm volatile("bar.sync 1, %0;" ::"n"(RO_CONSUMERS) : "memory");
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (; j < seq_end; ++j) {
        const long long k = j - run0;
        const int s = (int)(k % stages);
        if (!fail && !mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((k / stages) & 1), abort_flag, p.wait_limit)) {
          fail = true;
          sh->abort = 1;
        }
        if (!fail) {
          const float4* rows = reinterpret_cast<const float4*>(smem + (size_t)s * RO_CHUNK);
          const float* ph = s_phi + (int)(j % CS) * RC;
          for (int rr = grp; rr < RC; rr += G) {
            const float f = ph[rr];
            const float4 v = rows[(size_t)rr * C4 + col4];
            acc.x = fmaf(f, v.x, acc.x); acc.y = fmaf(f, v.y, acc.y);
            acc.z = fmaf(f, v.z, acc.z); acc.w = fmaf(f, v.w, acc.w);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sh->empty[s]));
      }
      // ---- the sequence's chunks of this run are done: add the row groups, write the partial vector
      s_red[tid] = acc;
      asm volatile("bar.sync 1, %0;" ::"n"(RO_CONSUMERS) : "memory");
      if (tid < C4) {
        float4 sum = s_red[tid];
        for (int g = 1; g < G; ++g) {
          const float4 o = s_red[g * C4 + tid];
          sum.x += o.x; sum.y += o.y; sum.z += o.z; sum.w += o.w;
        }
        reinterpret_cast<float4*>(sc.rpart + (size_t)((long long)blockIdx.x + i) * p.Dkv)[tid] = sum;
      }
    }
    if (fail && lane == 0) atomicOr(st.status, ST_TIMEOUT);
  }
  (void)ok;
}

}  // namespace

// shapes the streaming readout takes: the float4 columns of a row divide the consumer threads, whole chunks per sequence
bool im_readout_stream_supported(const ImDims& p) {
  if (p.Dkv % 4 || p.Dkv * 4 > RO_CHUNK) return false;
  const int C4 = p.Dkv / 4;
  if (C4 > RO_CONSUMERS || RO_CONSUMERS % C4) return false;
  const int RC = RO_CHUNK / (p.Dkv * 4);
  return RO_CHUNK % (p.Dkv * 4) == 0 && p.dM % RC == 0;
}

// chunks per sequence (the merge kernel rebuilds the runs from it)
int im_readout_stream_chunks(const ImDims& p) { return p.dM / (RO_CHUNK / (p.Dkv * 4)); }

static size_t ro_smem_bytes(const ImDims& p, int stages) {
  return (size_t)stages * RO_CHUNK + (size_t)((p.dM + 3) & ~3) * 4 + (size_t)RO_CONSUMERS * 16 + sizeof(RoShared) + 16;
}

cudaError_t im_readout_stream_prepare(const ImDims& p) {
  cudaError_t e = cudaFuncSetAttribute(k_readout_stream, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)ro_smem_bytes(p, RO_MAX_STAGES));
  if (e == cudaSuccess) e = im_prefer_max_smem(k_readout_stream);
  return e;
}

cudaError_t im_launch_readout_stream(const ImLaunch& L, const ImCall& call, int grid, int stages) {
  stages = stages < 1 ? 1 : (stages > RO_MAX_STAGES ? RO_MAX_STAGES : stages);
  const long long total = (long long)call.n_seq * im_readout_stream_chunks(L.p);
  const int blocks = (int)(total < grid ? total : grid);
  k_readout_stream<<<blocks < 1 ? 1 : blocks, RO_THREADS, ro_smem_bytes(L.p, stages), L.stream>>>(L.p, L.st, L.sc, call, stages);
  ++*L.launches;
  return cudaGetLastError();
}

// Chunked-prefill indexer scoring (Sec. 3.1: A_{s,t} = sum_h alpha_{s,h} act(q_{s,h} . k_t), pooled over
// the chunk's queries s by max under the causal mask) as a dense contraction on the 5th-generation
// tensor cores: tcgen05.mma with the accumulator in tensor memory.
//
// Mapping.  One CTA owns 128 cached keys (the M dimension = the 128 TMEM lanes) and walks over tiles of
// 32 queries.  A tile's N dimension is 32 queries x 8 head slots = 256 accumulator columns, so the sum
// over indexer heads and the max over queries are both register-local to the thread that owns a key:
// no shuffles, one atomic max per key at the end.  The reduction dimension is d_I (8 or 16, padded to 16).
// The query features are float32; to keep the scores within 1e-5 of a float32 evaluation each feature is
// split into three bf16 terms (q = q1 + q2 + q3 exactly to 2^-24), which costs three K = 16 MMAs per tile
// against the same key operand.  bf16 x bf16 products are exact in the float32 accumulator.
//
// Operands.  The append kernel writes, per sequence and 32-query tile, one 25,600-byte record that is
// already in the shared-memory layout of a K-major operand without swizzle (core matrices of 8 rows x 16
// bytes; the 8 head slots of one query are one core-matrix row group): 3 x 8 KB of features followed by
// 1 KB of alpha.  A record is fetched with one bulk copy that completes on an mbarrier.  The key tile is
// written once per CTA with plain stores.
//
// Roles.  Warps 0-7: epilogue (warp w reads TMEM lanes 32 (w mod 4) .., columns 128 (w div 4) ..);
// warp 8 lane 0: bulk copies and MMA issue.  Ring of 5 records, two accumulators of 256 columns.
// Every mbarrier wait is bounded; a wait that runs out sets ST_TIMEOUT and an abort flag that ends all
// roles, after which the CTA still frees its tensor memory and returns.
#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int TC_KEYS = 128;
constexpr int TC_N = IM_TC_QT * IM_TC_HP;             // 256 accumulator columns per tile
constexpr int TC_SPLIT_BYTES = TC_N * 32;             // one bf16 term of the features: 256 rows x 16 bf16
constexpr int TC_ALPHA_OFF = 3 * TC_SPLIT_BYTES;      // 24,576
constexpr int TC_STAGES = 5;
constexpr int TC_A_BYTES = TC_KEYS * 32;
constexpr int TC_THREADS = 288;
constexpr int TC_TMEM_COLS = 512;
constexpr uint32_t TC_WAIT_LIMIT = 1u << 22;
static_assert(TC_ALPHA_OFF + IM_TC_QT * IM_TC_HP * 4 == IM_TC_TILE_BYTES, "record size");

struct TcShared {
  unsigned long long full[TC_STAGES], empty[TC_STAGES], tfull[2], tempty[2];
  uint32_t tmem;
  int abort, cmin, cmax;
  float best[2][TC_KEYS];
};
constexpr int TC_SMEM = TC_A_BYTES + TC_STAGES * IM_TC_TILE_BYTES + (int)sizeof(TcShared);

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
// bounded wait; gives up early when another role has already given up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < TC_WAIT_LIMIT; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if ((it & 63) == 63 && *abort_flag) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

// shared-memory operand descriptor: K-major, no swizzle; the two 8-element K groups of a row group are
// 128 bytes apart (leading offset), consecutive 8-row groups 256 bytes apart (stride offset)
__device__ __forceinline__ uint64_t operand_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)(128u >> 4) << 16;          // leading-dimension byte offset
  d |= (uint64_t)(256u >> 4) << 32;          // stride-dimension byte offset
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  return d;                                  // base offset 0, relative offsets, swizzle mode 0 (none)
}
// instruction descriptor: D float32, A and B bf16, both K-major, N = 256, M = 128, dense
constexpr uint32_t TC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TC_N >> 3) << 17) | ((uint32_t)(TC_KEYS >> 4) << 24);

__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(TC_IDESC), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive accumulator columns of this thread's lane (load and its completion wait in one
// statement, so that no use of the registers can be scheduled between them)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int k = 0; k < 32; ++k) v[k] = __uint_as_float(r[k]);
}

// the same load without the wait, and the pieces to use several of them at once: issue the loads, wait once,
// then pass every destination register through an empty volatile statement placed after the wait, so that the
// compiler cannot schedule a use of a loaded value before the wait
#define IM_R32(r) "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]), \
    "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]), "+r"(r[17]),      \
    "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]),      \
    "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32_landed(uint32_t* r) { asm volatile("" : IM_R32(r)::"memory"); }

// imp = max(imp, v) for any mixture of signs (non-negative floats order as signed integers, negative
// ones in reverse as unsigned integers); the result does not depend on the order of the updates
__device__ __forceinline__ void atomic_max_float(float* addr, float v) {
  if (!(__float_as_uint(v) >> 31)) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
  else atomicMin(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

// grid = (query segments, key tiles, n_seq), block = 288, one CTA per SM (shared memory).
template <bool RELU>
__global__ void __launch_bounds__(TC_THREADS, 1) k_prefill_score_tc(ImDims p, ImState st, ImScratch sc, ImCall call) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* s_a = smem;
  uint8_t* s_stage = smem + TC_A_BYTES;
  TcShared* sh = reinterpret_cast<TcShared*>(smem + TC_A_BYTES + TC_STAGES * IM_TC_TILE_BYTES);
  const int i = blockIdx.z, seg = blockIdx.x, nseg = gridDim.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n0 = ctr[CTR_N], T = ctr[CTR_T], C = call.C;
  const int n1 = n0 + C;
  if (n0 < 0 || n1 > p.cap) return;  // flagged by the append kernel
  const int e0 = blockIdx.y * TC_KEYS;
  if (e0 >= n1) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh->abort;

  if (tid == 0) {
    for (int s = 0; s < TC_STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 8);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tfull[a]), 1);
      mbar_init(smem_u32(&sh->tempty[a]), 8);
    }
    sh->abort = 0;
    sh->cmin = 0x7fffffff;
    sh->cmax = -0x7fffffff;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 8) {  // tensor memory: both accumulators, whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem)),
                 "r"((uint32_t)TC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    tc_fence_before();
  }
  if (tid < TC_KEYS) {  // key operand: row tid of the tile, two 16-byte K groups
    const int e = e0 + tid;
    const bool live = e < n1;
    uint4 g0 = make_uint4(0, 0, 0, 0), g1 = g0;
    int cm = 0x7fffffff, cx = -0x7fffffff;
    if (live) {
      const uint4* row = reinterpret_cast<const uint4*>(st.kidx + (u * p.cap + e) * p.dI);
      g0 = row[0];
      if (p.dI == 16) g1 = row[1];
      cm = cx = st.pos[u * p.cap + e] - T;  // index of the first chunk query that may see this key
    }
    uint8_t* dst = s_a + (tid >> 3) * 256 + (tid & 7) * 16;
    *reinterpret_cast<uint4*>(dst) = g0;
    *reinterpret_cast<uint4*>(dst + 128) = g1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      cm = min(cm, __shfl_xor_sync(0xffffffffu, cm, o));
      cx = max(cx, __shfl_xor_sync(0xffffffffu, cx, o));
    }
    if (lane == 0) {
      atomicMin(&sh->cmin, cm);
      atomicMax(&sh->cmax, cx);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the MMA reads the tile through the async proxy
  }
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem;
  const int n_qt = (C + IM_TC_QT - 1) / IM_TC_QT;
  const int j_first = max(0, sh->cmin) / IM_TC_QT;  // earlier tiles cannot see any key of this CTA
  const int cmax = sh->cmax;
  const int j0 = j_first + seg;
  const int nt = j0 < n_qt ? (n_qt - j0 + nseg - 1) / nseg : 0;  // tiles j0, j0 + nseg, ...
  const uint8_t* records = sc.qpack + (size_t)i * n_qt * IM_TC_TILE_BYTES;

  if (warp == 8) {
    if (lane == 0) {
      const uint64_t adesc = operand_desc(smem_u32(s_a));
      int issued = 0, consumed = 0;
      bool ok = true;
      constexpr int AHEAD = TC_STAGES - 1;
      for (int it = 0; it < nt + AHEAD && ok; ++it) {
        if (it < nt) {
          const int s = it % TC_STAGES, use = it / TC_STAGES;
          if (use > 0 && !mbar_wait(smem_u32(&sh->empty[s]), (uint32_t)((use - 1) & 1), abort_flag)) { ok = false; break; }
          const uint32_t bar = smem_u32(&sh->full[s]);
          mbar_expect_tx(bar, IM_TC_TILE_BYTES);
          bulk_load(smem_u32(s_stage + s * IM_TC_TILE_BYTES), records + (size_t)(j0 + it * nseg) * IM_TC_TILE_BYTES,
                    IM_TC_TILE_BYTES, bar);
          ++issued;
        }
        const int k = it - AHEAD;
        if (k >= 0) {
          const int s = k % TC_STAGES, a = k & 1;
          if (!mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((k / TC_STAGES) & 1), abort_flag)) { ok = false; break; }
          ++consumed;
          if (k >= 2 && !mbar_wait(smem_u32(&sh->tempty[a]), (uint32_t)(((k >> 1) - 1) & 1), abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t b0 = smem_u32(s_stage + s * IM_TC_TILE_BYTES);
#pragma unroll
          for (int sp = 0; sp < 3; ++sp)
            mma_bf16(tmem + (uint32_t)(a * TC_N), adesc, operand_desc(b0 + sp * TC_SPLIT_BYTES), sp > 0 ? 1u : 0u);
          mma_commit(smem_u32(&sh->tfull[a]));
        }
      }
      if (!ok) {
        sh->abort = 1;
        atomicOr(st.status, ST_TIMEOUT);
        // copies still in flight write into this CTA's shared memory: give them their time to land
        volatile int never = 0;
        for (int l = consumed; l < issued; ++l)
          mbar_wait(smem_u32(&sh->full[l % TC_STAGES]), (uint32_t)((l / TC_STAGES) & 1), &never);
      }
    }
    __syncwarp();
  } else {
    const int half = warp >> 2, lane_base = (warp & 3) * 32;
    const int e = e0 + lane_base + lane;
    const int cmin_e = e < n1 ? st.pos[u * p.cap + e] - T : 0x7fffffff;
    float best = NEG_INF, chk = 0.f;
    bool ok = true;
    for (int k = 0; k < nt; ++k) {
      const int jt = j0 + k * nseg, s = k % TC_STAGES, a = k & 1;
      // the record's barrier first (it completed before the MMA was issued): acquires alpha for this thread
      if (!mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((k / TC_STAGES) & 1), abort_flag)) { ok = false; break; }
      if (!mbar_wait(smem_u32(&sh->tfull[a]), (uint32_t)((k >> 1) & 1), abort_flag)) { ok = false; break; }
      tc_fence_after();
      const float4* al = reinterpret_cast<const float4*>(s_stage + s * IM_TC_TILE_BYTES + TC_ALPHA_OFF) + half * 32;
      const int sbase = jt * IM_TC_QT + half * 16;
      const bool masked = jt * IM_TC_QT < cmax;  // some key of the CTA is newer than the tile's first query
      const uint32_t taddr = tmem + ((uint32_t)lane_base << 16) + (uint32_t)(a * TC_N + half * 128);
      // the warp's 128 accumulator columns of the tile in one round trip
      uint32_t rv[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32_issue(taddr + c * 32, rv[c]);
      tmem_ld_wait();
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32_landed(rv[c]);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        if (sbase + c * 4 >= C) break;
        float v[32];
#pragma unroll
        for (int k = 0; k < 32; ++k) v[k] = __uint_as_float(rv[c][k]);
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
          const int sq = sbase + c * 4 + qq;
          if (sq < C) {
            const float4 a0 = al[(c * 4 + qq) * 2], a1 = al[(c * 4 + qq) * 2 + 1];
            const float* z = v + qq * 8;
            float A;
            if (RELU) {
              A = a0.x * fmaxf(z[0], 0.f);
              A = fmaf(a0.y, fmaxf(z[1], 0.f), A);
              A = fmaf(a0.z, fmaxf(z[2], 0.f), A);
              A = fmaf(a0.w, fmaxf(z[3], 0.f), A);
              A = fmaf(a1.x, fmaxf(z[4], 0.f), A);
              A = fmaf(a1.y, fmaxf(z[5], 0.f), A);
              A = fmaf(a1.z, fmaxf(z[6], 0.f), A);
              A = fmaf(a1.w, fmaxf(z[7], 0.f), A);
            } else {
              A = a0.x * z[0];
              A = fmaf(a0.y, z[1], A);
              A = fmaf(a0.z, z[2], A);
              A = fmaf(a0.w, z[3], A);
              A = fmaf(a1.x, z[4], A);
              A = fmaf(a1.y, z[5], A);
              A = fmaf(a1.z, z[6], A);
              A = fmaf(a1.w, z[7], A);
            }
            chk = fmaf(A, 0.f, chk);  // NaN as soon as one score is not finite
            if (masked && sq < cmin_e) A = NEG_INF;
            best = fmaxf(best, A);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(smem_u32(&sh->tempty[a]));
        mbar_arrive(smem_u32(&sh->empty[s]));
      }
    }
    if (!ok && lane == 0) {
      sh->abort = 1;
      atomicOr(st.status, ST_TIMEOUT);
    }
    sh->best[half][lane_base + lane] = best;
    if (chk != chk) atomicOr(st.status, ST_NONFINITE);
  }
  tc_fence_before();
  __syncthreads();
  if (tid < TC_KEYS) {
    const int e = e0 + tid;
    const float b = fmaxf(sh->best[0][tid], sh->best[1][tid]);
    if (e < n1 && b > NEG_INF && !sh->abort) atomic_max_float(st.imp + u * p.cap + e, b);
  }
  if (warp == 8) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TC_TMEM_COLS) : "memory");
  }
}

}  // namespace

bool im_score_tc_supported(const ImDims& p) {
  return p.HI >= 1 && p.HI <= IM_TC_HP && (p.dI == 8 || p.dI == 16) && (p.act == 0 || p.act == 1);
}

cudaError_t im_score_tc_prepare() {
  cudaError_t e = cudaFuncSetAttribute(k_prefill_score_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_prefill_score_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM);
}

cudaError_t im_launch_prefill_score_tc(const ImLaunch& L, const ImCall& call, int n_max, int n_sm) {
  const int k_tiles = (n_max + TC_KEYS - 1) / TC_KEYS;
  const int n_qt = (call.C + IM_TC_QT - 1) / IM_TC_QT;
  int nseg = (2 * n_sm + k_tiles * call.n_seq - 1) / (k_tiles * call.n_seq);
  nseg = std::max(1, std::min(nseg, n_qt));
  dim3 grid(nseg, k_tiles, call.n_seq);
  if (L.p.act == 0) k_prefill_score_tc<true><<<grid, TC_THREADS, TC_SMEM, L.stream>>>(L.p, L.st, L.sc, call);
  else k_prefill_score_tc<false><<<grid, TC_THREADS, TC_SMEM, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

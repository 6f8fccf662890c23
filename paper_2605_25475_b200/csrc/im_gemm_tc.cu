// The skinny GEMMs of chunked prefill on the 5th-generation tensor cores (tcgen05.mma, accumulator in tensor
// memory): out[v][row0 + r] = sum_k (W[r][k] + W2[r][k]) * in[v][k] for thousands of vectors v (the chunk's tokens
// or its evicted keys) - a0 projections and phi of the evicted keys (Sec. 3.1, Eq. 5-7 operands).  Same
// arguments as k_skinny_gemm (ImGemmArgs, one K split).
//
// A CTA owns 128 vectors (the M dimension = the TMEM lanes) and up to 128 weight rows of one job (N, rounded
// up to 16).  Both operands are K-major in global memory; four producer warps bring 64-wide K tiles into a
// 4-stage ring with 16-byte cp.async copies, laid out as the K-major no-swizzle operand layout with the
// 8-element K groups as the outer dimension: byte (kgroup * (128 * 16 + 16) + row * 16), i.e. 8 rows x 16 bytes
// are contiguous (one core matrix), consecutive 8-row groups 128 bytes apart, consecutive K groups 2064 bytes
// apart (the 16 bytes of padding spread the copies of one row over the banks).  A stage is handed to the MMA
// thread through an mbarrier after cp.async.wait_group and a proxy fence; tcgen05.commit releases it.  A second
// weight term is a second pass over K into the same accumulator.  The producer warps then read the
// accumulator with tcgen05.ld and store float32.  Every wait is bounded (ST_TIMEOUT).
#include <cuda.h>

#include "im_internal.cuh"

namespace {

constexpr int GM = 128;              // vectors per CTA
constexpr int GN = 128;              // weight rows per CTA
constexpr int GK = 64;               // K elements per stage
constexpr int G_STAGES = 4;
constexpr int G_LAG = 2;             // stages whose copies may still be in flight behind the producer
constexpr int G_PLANE = GM * 16 + 16;           // one K group of one operand: 128 rows x 16 bytes + padding
constexpr int G_OPER = (GK / 8) * G_PLANE;      // one operand of one stage
constexpr int G_STAGE = 2 * G_OPER;
constexpr int G_THREADS = 160;
constexpr uint32_t G_WAIT_LIMIT = 1u << 22;
static_assert(GM == GN, "the two operands share the plane size");

struct GShared {
  unsigned long long full[G_STAGES], empty[G_STAGES], acc;
  uint32_t tmem;
  int abort;
};
constexpr int G_SMEM = G_STAGES * G_STAGE + (int)sizeof(GShared);

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < G_WAIT_LIMIT; ++it) {
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
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;  // src-size 0: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
// K-major, no swizzle: K groups G_PLANE bytes apart (leading offset), 8-row groups 128 bytes apart (stride offset)
__device__ __forceinline__ uint64_t operand_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((uint32_t)G_PLANE >> 4) << 16;
  d |= (uint64_t)(128u >> 4) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  return d;
}
// Called by a whole (converged) warp: one elected lane issues.  The operands then stay warp-uniform values; issued
// from inside an `if (lane == 0)` they were per-thread values moved to uniform registers before every instruction.
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar)
      : "memory");
}
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
// epilogue of one thread: 32 consecutive weight rows (c0 ..) of vector v
__device__ __forceinline__ void store_columns(const ImGemmArgs& a, const ImGemmJob& job, int r0, int n_rows, int c0,
                                              long long v, const float* acc, float* out, const int32_t* gate) {
  if (v >= a.NV) return;
  if (gate && *gate <= a.gate_min) return;
  if (a.out_t) {
    float* o = out + (size_t)(job.row0 + r0 + c0) * a.out_outer + v;
    if (a.rmw) {
      // read-modify-write: all 32 old values are requested before the first store (a store between two loads
      // would keep the compiler from overlapping them: it cannot know that the addresses differ)
      float old[32];
#pragma unroll
      for (int c = 0; c < 32; ++c) old[c] = c0 + c < n_rows ? o[(size_t)c * a.out_outer] : 0.f;
#pragma unroll
      for (int c = 0; c < 32; ++c)
        if (c0 + c < n_rows) o[(size_t)c * a.out_outer] = fmaf(a.beta, old[c], a.alpha * acc[c]);
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c)
        if (c0 + c < n_rows) o[(size_t)c * a.out_outer] = acc[c];
    }
  } else {
    float* o = out + (v / a.out_cnt) * a.out_outer + (v % a.out_cnt) * a.out_inner + job.row0 + r0 + c0;
#pragma unroll
    for (int c = 0; c < 32; ++c)
      if (c0 + c < n_rows) o[c] = a.rmw ? fmaf(a.beta, o[c], a.alpha * acc[c]) : acc[c];
  }
}
__device__ __forceinline__ const bf16* vec_ptr(const ImGemmArgs& a, int sel, long long v) {
  return a.in[sel] + (v / a.in_cnt[sel]) * a.in_outer[sel] + (v % a.in_cnt[sel]) * a.in_inner[sel];
}

// grid = (ceil(NV / 128), sum over jobs of ceil(rows / 128)), block = 160: warps 0-3 copy and run the epilogue,
// warp 4 allocates tensor memory and its lane 0 issues the MMAs.
__global__ void __launch_bounds__(G_THREADS, 1) k_tc_gemm(ImGemmArgs a, int32_t* status) {
  extern __shared__ __align__(128) uint8_t smem[];
  GShared* sh = reinterpret_cast<GShared*>(smem + G_STAGES * G_STAGE);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int tile = blockIdx.y, j = 0;
  while (j + 1 < a.n_jobs && tile >= (a.job[j].rows + GN - 1) / GN) {
    tile -= (a.job[j].rows + GN - 1) / GN;
    ++j;
  }
  const ImGemmJob job = a.job[j];
  const int r0 = tile * GN;                                   // first weight row of the CTA
  const int n_rows = min(GN, job.rows - r0);
  const int n_cols = (n_rows + 15) & ~15;                     // MMA N
  const long long v0 = (long long)blockIdx.x * GM;
  const int KT = a.K / GK;                                    // K is a multiple of 64 (checked by the launcher)
  const int KTOT = KT * (job.W2 ? 2 : 1);
  volatile int* abort_flag = &sh->abort;
  if (tid == 0) {
    for (int s = 0; s < G_STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 128);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->acc), 1);
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem)), "r"(128u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh->tmem;
  bool ok = true;

  if (warp < 4) {
    // ---- producer: thread t copies K group (t & 7) of rows (t >> 3) + 16 it, it = 0..7, of both operands
    const int kg = tid & 7, rb = tid >> 3;
    const bf16* pa[8];
    const bf16* pb[8];
    const long long w2_off = job.W2 ? job.W2 - job.W : 0;  // second term: the same rows of the other matrix
    bool va[8], vb[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int r = rb + 16 * it;
      va[it] = v0 + r < a.NV;
      pa[it] = vec_ptr(a, job.in_sel, va[it] ? v0 + r : 0) + kg * 8;
      vb[it] = r < n_rows;
      const size_t off = (size_t)(vb[it] ? r0 + r : 0) * a.K + kg * 8;
      pb[it] = job.W + off;
    }
    auto publish = [&](int kt) {  // the copies of tile kt have landed: make them visible to the tensor core, hand over
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(smem_u32(&sh->full[kt % G_STAGES]));
    };
    for (int kt = 0; kt < KTOT && ok; ++kt) {
      const int s = kt % G_STAGES;
      if (kt >= G_STAGES && !mbar_wait(smem_u32(&sh->empty[s]), (uint32_t)(((kt / G_STAGES) - 1) & 1), abort_flag)) {
        ok = false;
        break;
      }
      const int term = kt / KT, k0 = (kt % KT) * GK;
      const uint32_t sa = smem_u32(smem + (size_t)s * G_STAGE) + kg * G_PLANE + rb * 16;
      const uint32_t sb = sa + G_OPER;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        cp_async16(sa + it * 256, pa[it] + k0, va[it]);
        cp_async16(sb + it * 256, pb[it] + term * w2_off + k0, vb[it]);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      if (kt >= G_LAG) {
        asm volatile("cp.async.wait_group %0;" ::"n"(G_LAG) : "memory");
        publish(kt - G_LAG);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    if (ok)
      for (int kt = max(0, KTOT - G_LAG); kt < KTOT; ++kt) publish(kt);
    // ---- epilogue: lane = vector, 32 accumulator columns (weight rows) at a time
    if (ok && !mbar_wait(smem_u32(&sh->acc), 0u, abort_flag)) ok = false;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long v = v0 + warp * 32 + lane;
      for (int c0 = 0; c0 < n_cols; c0 += 32) {
        float acc[32];
        tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, acc);
        store_columns(a, job, r0, n_rows, c0, v, acc, a.out, a.gate);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
  } else {
    // ---- MMA issue (whole warp, one elected lane issues): four K = 16 steps per stage
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(GM >> 4) << 24);
    for (int kt = 0; kt < KTOT; ++kt) {
      const int s = kt % G_STAGES;
      if (!mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((kt / G_STAGES) & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t sa = smem_u32(smem + (size_t)s * G_STAGE), sb = sa + G_OPER;
#pragma unroll
      for (int ks = 0; ks < GK / 16; ++ks)
        mma_bf16(tmem, operand_desc(sa + ks * 2 * G_PLANE), operand_desc(sb + ks * 2 * G_PLANE), idesc, (kt | ks) ? 1u : 0u);
      mma_commit(smem_u32(&sh->empty[s]));
    }
    if (ok) mma_commit(smem_u32(&sh->acc));
  }
  if (!ok && lane == 0) {
    sh->abort = 1;
    atomicOr(status, ST_TIMEOUT);
  }
  __syncthreads();
  if (warp == 4) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
  }
}


// ------------------------------------------------------------------------------------------------
// The same product with both operands brought in by TMA (2-D tensor maps over [rows][K], box 64 x 128,
// 128-byte swizzle) for one job whose vectors are uniformly strided in memory.  Shared-memory operand
// descriptors of the swizzled K-major layout: 8-row groups 1024 bytes apart, a K = 16 step advances the start
// address by 32 bytes inside the 128-byte rows.  block = 192: warp 0 lane 0 issues the copies, warp 1 owns
// tensor memory and its lane 0 issues the MMAs, warps 2-5 run the epilogue.  6 stages of 32 KB.
constexpr int T_STAGES = 6;
constexpr int T_TILE = GM * GK * 2;  // one operand of one stage: 16 KB
constexpr int T_STAGE = 2 * T_TILE;
constexpr int T_THREADS = 192;
struct TShared {
  unsigned long long full[T_STAGES], empty[T_STAGES], acc;
  uint32_t tmem;
  int abort;
};
constexpr int T_SMEM = T_STAGES * T_STAGE + (int)sizeof(TShared) + 1024;  // + slack to align the ring to 1024 bytes

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint64_t operand_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                    // leading offset: not used by this layout
  d |= (uint64_t)(1024u >> 4) << 32;         // stride offset: 8 rows x 128 bytes
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}

__global__ void __launch_bounds__(T_THREADS, 1)
k_tc_gemm_tma(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB0,
              const __grid_constant__ CUtensorMap mapB1, ImGemmArgs a, int j, int32_t* status,
              const __grid_constant__ ImGemmBatch bt) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  TShared* sh = reinterpret_cast<TShared*>(smem + T_STAGES * T_STAGE);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const ImGemmJob job = a.job[j];
  const int r0 = blockIdx.y * GN;
  const int n_rows = min(GN, job.rows - r0);
  const int n_cols = (n_rows + 15) & ~15;
  const long long v0 = (long long)blockIdx.x * GM;
  // K split (not with a batched launch): this CTA's share of the K tiles and the partial buffer it writes
  const int nks = (bt.n <= 1 && a.tc_ksplit > 1) ? a.tc_ksplit : 1;
  const int ksi = nks > 1 ? (int)blockIdx.z : 0;
  const int KT = a.K / GK / nks;          // K tiles of this CTA per weight term
  const int kt0 = ksi * KT;
  const int KTOT = KT * (job.W2 ? 2 : 1);
  // batched launch: this CTA's product
  const int zb = bt.n > 1 ? (int)blockIdx.z : 0;
  const long long zu = bt.n > 1 ? (long long)bt.unit0 + bt.seq[zb] : 0;
  const int ya = (int)(v0 + zb * bt.zA_rows), yb = (int)(r0 + zb * bt.zB_rows);
  float* out_z = nks > 1 ? a.part + (long long)ksi * a.part_stride : a.out + zu * bt.z_out;
  const int32_t* gate_z = a.gate ? a.gate + zu * bt.z_gate : nullptr;
  volatile int* abort_flag = &sh->abort;
  if (tid == 0) {
    for (int s = 0; s < T_STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->acc), 1);
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem)), "r"(128u)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh->tmem;
  bool ok = true;
  if (warp == 0) {
    if (lane == 0) {
      for (int kt = 0; kt < KTOT; ++kt) {
        const int s = kt % T_STAGES;
        if (kt >= T_STAGES && !mbar_wait(smem_u32(&sh->empty[s]), (uint32_t)(((kt / T_STAGES) - 1) & 1), abort_flag)) {
          ok = false;
          break;
        }
        const uint32_t bar = smem_u32(&sh->full[s]);
        const uint32_t sa = smem_u32(smem + (size_t)s * T_STAGE);
        const int k0 = (kt0 + kt % KT) * GK;
        mbar_expect_tx(bar, T_STAGE);
        tma_load_2d(sa, &mapA, k0, ya, bar);
        tma_load_2d(sa + T_TILE, kt < KT ? &mapB0 : &mapB1, k0, yb, bar);
      }
    }
  } else if (warp == 1) {
    {  // MMA issue: whole warp, one elected lane issues
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(GM >> 4) << 24);
      for (int kt = 0; kt < KTOT; ++kt) {
        const int s = kt % T_STAGES;
        if (!mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((kt / T_STAGES) & 1), abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = smem_u32(smem + (size_t)s * T_STAGE), sb = sa + T_TILE;
#pragma unroll
        for (int ks = 0; ks < GK / 16; ++ks)
          mma_bf16(tmem, operand_desc_sw128(sa + ks * 32), operand_desc_sw128(sb + ks * 32), idesc, (kt | ks) ? 1u : 0u);
        mma_commit(smem_u32(&sh->empty[s]));
      }
      if (ok) mma_commit(smem_u32(&sh->acc));
    }
  } else {
    const int qd = warp & 3;  // the TMEM lane quarter this warp may read
    if (!mbar_wait(smem_u32(&sh->acc), 0u, abort_flag)) ok = false;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long v = v0 + qd * 32 + lane;
      for (int c0 = 0; c0 < n_cols; c0 += 32) {
        float acc[32];
        tmem_ld32(tmem + ((uint32_t)(qd * 32) << 16) + (uint32_t)c0, acc);
        store_columns(a, job, r0, n_rows, c0, v, acc, out_z, gate_z);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
  }
  if (!ok && lane == 0) {
    sh->abort = 1;
    atomicOr(status, ST_TIMEOUT);
    // copies that this CTA still has in flight write into its shared memory: give them time to land (bounded)
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(128u) : "memory");
  }
}

// out = sum over the K splits of the partial buffers, in split order, for the rows of job j (vectors x rows, any
// output layout: the partial buffers are laid out like `out`).  grid = ceil(NV * rows / 256), block = 256.
__global__ void __launch_bounds__(256) k_ksplit_reduce(ImGemmArgs a, int j) {
  const ImGemmJob job = a.job[j];
  const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
  if (idx >= a.NV * (long long)job.rows) return;
  const long long v = idx / job.rows;
  const int r = (int)(idx % job.rows);
  const long long off = a.out_t ? (long long)(job.row0 + r) * a.out_outer + v
                                : (v / a.out_cnt) * a.out_outer + (v % a.out_cnt) * a.out_inner + job.row0 + r;
  float s = 0.f;
  for (int k = 0; k < a.tc_ksplit; ++k) s += a.part[(long long)k * a.part_stride + off];
  a.out[off] = s;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [rows][K] bf16, row stride `stride` elements, box 64 x 128, 128-byte swizzle
bool encode_rows_map(CUtensorMap* m, const void* base, long long rows, long long K, long long stride) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return false;
    enc = (EncodeTiledFn)fn;
  }
  if (((uintptr_t)base & 15) || (stride * 2) % 16 || rows < 1) return false;
  // A map is a function of (base, rows, K, stride) alone, and a chunked prefill asks for the same dozen again in every
  // call (weights; the caller's input buffers where it reuses them): the last few are kept per host thread.
  struct Memo { const void* base; long long rows, K, stride; CUtensorMap map; };
  constexpr int N_MEMO = 32;
  thread_local Memo memo[N_MEMO];
  thread_local int n_memo = 0, next_memo = 0;
  for (int k = 0; k < n_memo; ++k)
    if (memo[k].base == base && memo[k].rows == rows && memo[k].K == K && memo[k].stride == stride) {
      *m = memo[k].map;
      return true;
    }
  const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)stride * 2};
  const cuuint32_t box[2] = {(cuuint32_t)GK, (cuuint32_t)GM};
  const cuuint32_t estr[2] = {1, 1};
  if (enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  Memo& e = memo[next_memo];
  e.base = base; e.rows = rows; e.K = K; e.stride = stride; e.map = *m;
  next_memo = (next_memo + 1) % N_MEMO;
  if (n_memo < N_MEMO) ++n_memo;
  return true;
}

}  // namespace

bool im_tc_gemm_usable(const ImGemmArgs& a) {
  if (a.ksplit != 1 || a.K < GK || a.K % GK || a.NV < GM) return false;
  for (int j = 0; j < a.n_jobs; ++j)
    if (a.job[j].rows < 1) return false;
  return true;
}

cudaError_t im_launch_tc_gemm(const ImLaunch& L, const ImGemmArgs& a) {
  static bool attr_done_dev[64] = {};
  bool* attr_done = im_device_flag(attr_done_dev);
  if (!attr_done || !*attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_tc_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM);
    if (e != cudaSuccess) return e;
    if (attr_done) *attr_done = true;
  }
  // vectors at a uniform stride: both operands by TMA, one launch per job
  bool uniform = true;
  long long vstride[4] = {0, 0, 0, 0};
  for (int j = 0; j < a.n_jobs && uniform; ++j) {
    const int s = a.job[j].in_sel;
    if (a.in_cnt[s] == 1) vstride[j] = a.in_outer[s];
    else if (a.in_outer[s] == (long long)a.in_cnt[s] * a.in_inner[s]) vstride[j] = a.in_inner[s];
    else uniform = false;
  }
  if (uniform) {
    static bool tma_attr_done_dev[64] = {};
    bool* tma_attr_done = im_device_flag(tma_attr_done_dev);
    if (!tma_attr_done || !*tma_attr_done) {
      cudaError_t e = cudaFuncSetAttribute(k_tc_gemm_tma, cudaFuncAttributeMaxDynamicSharedMemorySize, T_SMEM);
      if (e != cudaSuccess) return e;
      if (tma_attr_done) *tma_attr_done = true;
    }
    CUtensorMap mA[4], mB0[4], mB1[4];
    bool enc_ok = true;
    static const ImGemmBatch no_batch = {};
    const ImGemmBatch& bt = a.batch ? *a.batch : no_batch;
    const int nb = bt.n > 1 ? bt.n : 1;
    for (int j = 0; j < a.n_jobs && enc_ok; ++j) {
      const ImGemmJob& jb = a.job[j];
      // a batched launch addresses batch b's operands zA_rows / zB_rows rows further down the same maps; the second
      // weight term starts (W2 - W) / K rows into the first batch's block
      const long long rowsA = nb > 1 ? (nb - 1) * bt.zA_rows + a.NV : a.NV;
      const long long rowsB = nb > 1 ? (nb - 1) * bt.zB_rows + jb.rows : jb.rows;
      enc_ok = encode_rows_map(&mA[j], a.in[jb.in_sel], rowsA, a.K, vstride[j]) &&
               encode_rows_map(&mB0[j], jb.W, rowsB, a.K, a.K) &&
               encode_rows_map(&mB1[j], jb.W2 ? jb.W2 : jb.W, rowsB, a.K, a.K);
    }
    if (enc_ok) {
      for (int j = 0; j < a.n_jobs; ++j) {
        const int nks = (nb == 1 && a.tc_ksplit > 1 && !a.rmw && a.part && (a.K / GK) % a.tc_ksplit == 0) ? a.tc_ksplit : 1;
        ImGemmArgs aj = a;
        aj.tc_ksplit = nks;
        dim3 grid((unsigned)((a.NV + GM - 1) / GM), (unsigned)((a.job[j].rows + GN - 1) / GN), (unsigned)(nb * nks));
        k_tc_gemm_tma<<<grid, T_THREADS, T_SMEM, L.stream>>>(mA[j], mB0[j], mB1[j], aj, j, L.st.status, bt);
        ++*L.launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (nks > 1) {
          const long long total = a.NV * (long long)a.job[j].rows;
          k_ksplit_reduce<<<(unsigned)((total + 255) / 256), 256, 0, L.stream>>>(aj, j);
          ++*L.launches;
          if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
      }
      return cudaSuccess;
    }
  }
  if (a.batch && a.batch->n > 1) return cudaErrorNotSupported;  // the batched form exists for the TMA variant only
  int tiles = 0;
  for (int j = 0; j < a.n_jobs; ++j) tiles += (a.job[j].rows + GN - 1) / GN;
  dim3 grid((unsigned)((a.NV + GM - 1) / GM), tiles);
  k_tc_gemm<<<grid, G_THREADS, G_SMEM, L.stream>>>(a, L.st.status);
  ++*L.launches;
  return cudaGetLastError();
}

// Layer outputs of a prefill chunk's own queries (Eq. 4-5 during chunked prefill): the flash attention of
// im_chunk_attn.cu on the 5th-generation tensor cores, for head_dim 128.
//
// A CTA owns 128 rows = floor(128 / G_q) queries x G_q heads of one KV head; row r is TMEM lane r.  Per tile of 64 keys:
//   S = Q K^T      tcgen05.mma, M = 128 rows, N = 64 keys, K = d = 128 (8 steps); Q and the K tile K-major in shared
//                  memory (128-byte swizzle; the K/V tiles come by TMA through the tensor maps of the decode
//                  attention kernel, two 32-row boxes per 64-column half), S in tensor memory (double buffered)
//   softmax        two threads per row (32 keys each) read their scores with tcgen05.ld, mask (causal by chunk
//                  index), exchange the maxima, keep the running maximum and sum (base 2), and write P as two bf16
//                  terms (upper 16 bits + rounded remainder: 2^-16) into TENSOR memory with tcgen05.st, two values per
//                  32-bit column, row = lane: the layout of an A operand read from tensor memory
//   O += P V       tcgen05.mma with A = P from tensor memory, N = d = 128, K = 64 keys (4 steps, both P terms),
//                  accumulating in tensor memory over the tiles; V is used as it lies in the cache ([key][d], i.e.
//                  MN-major for this product: 8-key groups 1024 bytes apart, the two 64-column halves 8 KB apart)
//   rescale        P is formed relative to a reference maximum that is only raised when a row's maximum has
//                  grown by more than 2^8 (or is seen for the first time): then the warp waits for the previous
//                  P V product, multiplies its O rows in tensor memory (tcgen05.ld / st) and its row sums by
//                  2^(m_ref_old - m_ref_new).  Between such events P (<= 2^8) and O need no correction, so the
//                  softmax of tile j + 1 overlaps with the P V product of tile j (P is double buffered).
// Tensor memory (512 columns): S 0..127, O 128..255, P 256..383.
// Warps 0-7: softmax / rescale / epilogue (two groups of four: each row's 64 keys of a tile and its 128 output
// columns are split between two threads); warp 8 lane 0: TMA; warp 9: tensor memory owner and MMA issue.  The whole
// of warp 9 runs the issue loop and one elected lane issues each instruction: with the loop inside an
// `if (lane == 0)` the operand descriptors were per-thread values that had to be moved to uniform registers for every
// instruction, and the issue itself (70-90 cycles per MMA of 32-64 cycles) bounded the kernel.
// Every wait is bounded (ST_TIMEOUT).
#include <cuda.h>

#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int DH = 128;
constexpr int KT = 64;                      // keys per tile
constexpr int ROWS = 128;
constexpr int STAGES = 5;
constexpr int HALF_BYTES = KT * 128;        // one 64-column half of a K or V tile: 64 rows x 128 bytes
constexpr int KV_TILE = 2 * HALF_BYTES;     // 16 KB
constexpr int STAGE_BYTES = 2 * KV_TILE;    // K + V
constexpr int Q_BYTES = ROWS * DH * 2;      // 32 KB: two halves of 128 rows x 128 bytes
constexpr int THREADS = 320;                // warps 0-7: softmax (two groups of four), 8: TMA, 9: tensor memory / MMA
constexpr uint32_t WAIT_LIMIT = 1u << 22;
constexpr int TMEM_COLS = 512;              // S: 2 x 64, O: 128, P: 2 buffers x 2 terms x 32 (bf16 pairs); a power of two
constexpr int P_COL = 256;                  // first column of P; buffer b, term t at P_COL + 64 b + 32 t

struct Shared {
  unsigned long long full[STAGES], empty[STAGES], sfull[2], sempty[2], pfull[2], pvdone[2];
  unsigned long long xch[2][4];   // row statistics of the two softmax groups exchanged: [tile parity][lane quarter]
  float stat[2][2][ROWS];         // [tile parity][group][row]
  uint32_t tmem;
  int abort;
};
constexpr int SMEM_BYTES = Q_BYTES + STAGES * STAGE_BYTES + (int)sizeof(Shared) + 1024;

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
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
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
// shared-memory operand descriptor, 128-byte swizzle: lbo / sbo in bytes
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;  // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the same with the A operand in tensor memory (row = lane, two bf16 per 32-bit column along K)
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate)
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
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n\t"
      "tcgen05.wait::st.sync.aligned;" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
      "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
      "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
      "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
      "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
      "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
// 2^x, x <= 8 here; -inf gives 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// grid = (ceil(C / QB), Hkv, n_seq) with QB = 128 / Gq queries per CTA; block = 320.
template <typename OutT>
__global__ void __launch_bounds__(THREADS, 1)
k_chunk_attention_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, ImDims p, ImState st,
                     ImScratch sc, ImCall call, const bf16* __restrict__ q, OutT* __restrict__ out) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;                       // [2 halves][128 rows][128 bytes]
  uint8_t* s_kv = smem + Q_BYTES;            // [STAGES][K: 2 halves x 64 rows x 128 bytes | V: the same]
  Shared* sh = reinterpret_cast<Shared*>(s_kv + STAGES * STAGE_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.y, i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int n0 = st.ctr[u * CTR_STRIDE + CTR_N];  // entries cached before the chunk (the counters advance later)
  const int C = call.C;
  if (n0 < 0 || n0 + C > p.cap) return;  // flagged by the append kernel
  const int QB = ROWS / p.Gq;
  const int s0 = blockIdx.x * QB;
  if (s0 >= C) return;
  const int s_last = min(C, s0 + QB) - 1;
  const int n_keys = n0 + s_last + 1;  // slots the block's last query sees
  const int nt = (n_keys + KT - 1) / KT;
  volatile int* abort_flag = &sh->abort;
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->sfull[b]), 1);
      mbar_init(smem_u32(&sh->sempty[b]), 2 * ROWS);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->pfull[b]), 2 * ROWS);
      mbar_init(smem_u32(&sh->pvdone[b]), 1);
      for (int qd = 0; qd < 4; ++qd) mbar_init(smem_u32(&sh->xch[b][qd]), 64);
    }
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  // ---- Q tile: thread r writes row r (query s0 + r / Gq, head r % Gq) into the swizzled K-major layout
  int lim = 0;          // this row sees slots [0, lim)
  bool row_ok = false;
  int s_row = s0, hh = 0;
  const int row = tid & (ROWS - 1);  // softmax threads: the row (both groups), TMEM lane
  if (tid < 2 * ROWS) {
    const int sl = row / p.Gq;
    hh = row % p.Gq;
    s_row = s0 + sl;
    row_ok = sl < QB && s_row < C;
    lim = row_ok ? n0 + s_row + 1 : 0;
  }
  if (tid < ROWS) {
    const uint4* src = reinterpret_cast<const uint4*>(q + (((size_t)i * C + (row_ok ? s_row : s0)) * p.H + (size_t)h * p.Gq + (row_ok ? hh : 0)) * DH);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const uint4 v = row_ok ? src[c] : make_uint4(0u, 0u, 0u, 0u);
      uint8_t* dst = s_q + (c >> 3) * (ROWS * 128) + (tid >> 3) * 1024 + (tid & 7) * 128 + (((c & 7) ^ (tid & 7)) << 4);
      *reinterpret_cast<uint4*>(dst) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh->tmem;
  const uint32_t t_o = tmem + 128;  // O columns; S buffers at columns 0 and 64
  bool ok = true;

  if (warp == 8) {
    if (lane == 0) {  // ---- TMA: K and V tiles of 64 keys, two 32-row boxes per 64-column half
      const int row_base = (int)((u * p.Hkv + h) * (size_t)p.cap);
      for (int j = 0; j < nt; ++j) {
        const int s = j % STAGES;
        if (j >= STAGES && !mbar_wait(smem_u32(&sh->empty[s]), (uint32_t)(((j / STAGES) - 1) & 1), abort_flag)) { ok = false; break; }
        const uint32_t bar = smem_u32(&sh->full[s]);
        const uint32_t dk = smem_u32(s_kv + (size_t)s * STAGE_BYTES), dv = dk + KV_TILE;
        mbar_expect_tx(bar, STAGE_BYTES);
#pragma unroll
        for (int hf = 0; hf < 2; ++hf)
#pragma unroll
          for (int b = 0; b < 2; ++b) {
            tma_load_2d(dk + hf * HALF_BYTES + b * 4096, &tmK, hf * 64, row_base + j * KT + b * 32, bar);
            tma_load_2d(dv + hf * HALF_BYTES + b * 4096, &tmV, hf * 64, row_base + j * KT + b * 32, bar);
          }
      }
    }
  } else if (warp == 9) {
    {  // ---- MMA issue: the whole warp runs the loop (descriptors stay warp-uniform), one elected lane issues
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
      const uint32_t qa = smem_u32(s_q);
      auto issue_s = [&](int j) -> bool {  // S(j) = Q K_j^T into S buffer j & 1
        const int s = j % STAGES, b = j & 1;
        if (!mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((j / STAGES) & 1), abort_flag)) return false;
        if (j >= 2 && !mbar_wait(smem_u32(&sh->sempty[b]), (uint32_t)(((j >> 1) - 1) & 1), abort_flag)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t ka = smem_u32(s_kv + (size_t)s * STAGE_BYTES);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
          mma_bf16(tmem + (uint32_t)(b * KT), desc_sw128(qa + (ks >> 2) * (ROWS * 128) + (ks & 3) * 32, 16, 1024),
                   desc_sw128(ka + (ks >> 2) * HALF_BYTES + (ks & 3) * 32, 16, 1024), idesc_s, ks ? 1u : 0u);
        mma_commit(smem_u32(&sh->sfull[b]));
        return true;
      };
      ok = issue_s(0);
      for (int j = 0; j < nt && ok; ++j) {
        if (j + 1 < nt && !issue_s(j + 1)) { ok = false; break; }
        const int s = j % STAGES, b = j & 1;
        if (!mbar_wait(smem_u32(&sh->pfull[b]), (uint32_t)((j >> 1) & 1), abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t va = smem_u32(s_kv + (size_t)s * STAGE_BYTES) + KV_TILE;
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int ks = 0; ks < KT / 16; ++ks)
            mma_bf16_ts(t_o, tmem + (uint32_t)(P_COL + 64 * b + 32 * term + 8 * ks), desc_sw128(va + ks * 2048, HALF_BYTES, 1024),
                        idesc_o, (j | term | ks) ? 1u : 0u);
        mma_commit(smem_u32(&sh->pvdone[b]));
        mma_commit(smem_u32(&sh->empty[s]));
      }
    }
  } else {
    // ---- softmax, rescale, epilogue.  Two groups of four warps: thread (group g, row r) owns keys 32 g .. 32 g + 31
    // of every tile of row r = TMEM lane r (warps w and w + 4 may both read lane quarter w) and, for the rescale and
    // the epilogue, columns 64 g .. 64 g + 63 of O.  The two threads of a row exchange their maxima (and at the end
    // their sums) through shared memory and an mbarrier per lane quarter, and take every decision alike.
    const int grp = warp >> 2, qd = warp & 3;
    const uint32_t lane_addr = (uint32_t)(qd * 32) << 16;
    const float sl2 = p.scale * 1.4426950408889634f;  // softmax in base 2
    float m_ref = NEG_INF, l = 0.f;                    // reference maximum of P and O, this thread's share of the row sum
    for (int j = 0; j < nt; ++j) {
      const int b = j & 1;
      if (!mbar_wait(smem_u32(&sh->sfull[b]), (uint32_t)((j >> 1) & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float sv[32];
      tmem_ld32(tmem + lane_addr + (uint32_t)(b * KT + grp * 32), sv);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(smem_u32(&sh->sempty[b]));
      const int key0 = j * KT + grp * 32;
      float tm = NEG_INF;
      if (key0 + 32 > lim) {  // only the row's last tiles need the causal mask
#pragma unroll
        for (int k = 0; k < 32; ++k) sv[k] = key0 + k < lim ? sv[k] : NEG_INF;
      }
#pragma unroll
      for (int k = 0; k < 32; ++k) tm = fmaxf(tm, sv[k]);
      sh->stat[b][grp][row] = tm;
      mbar_arrive(smem_u32(&sh->xch[b][qd]));
      if (!mbar_wait(smem_u32(&sh->xch[b][qd]), (uint32_t)((j >> 1) & 1), abort_flag)) { ok = false; break; }
      tm = fmaxf(tm, sh->stat[b][grp ^ 1][row]);
      tm *= sl2;  // the scale is positive: the maximum of the scaled scores
      // raise the reference only for a first maximum or a jump of more than 8 (P stays below 2^8 otherwise)
      const bool raise = tm > NEG_INF && (m_ref == NEG_INF || tm > m_ref + 8.0f);
      if (__any_sync(0xffffffffu, raise)) {
        const float corr = raise ? exp2f(m_ref - tm) : 1.0f;  // 0 for a first maximum: nothing accumulated yet
        if (raise) {
          m_ref = tm;
          l *= corr;
        }
        if (j >= 1) {  // O holds the products up to tile j - 1: wait for the last one, then scale this thread's half row
          if (!mbar_wait(smem_u32(&sh->pvdone[(j - 1) & 1]), (uint32_t)(((j - 1) >> 1) & 1), abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int c0 = 0; c0 < DH / 2; c0 += 32) {
            float t[32];
            tmem_ld32(t_o + lane_addr + (uint32_t)(grp * (DH / 2) + c0), t);
#pragma unroll
            for (int c = 0; c < 32; ++c) t[c] *= corr;
            tmem_st32(t_o + lane_addr + (uint32_t)(grp * (DH / 2) + c0), t);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
      }
      // P buffer b was last read by the product of tile j - 2
      if (j >= 2 && !mbar_wait(smem_u32(&sh->pvdone[b]), (uint32_t)(((j >> 1) - 1) & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const float e = m_ref == NEG_INF ? 0.f : m_ref;
      uint32_t hi[16], lo[16];
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        const float p0 = ex2(fmaf(sv[2 * k], sl2, -e)), p1 = ex2(fmaf(sv[2 * k + 1], sl2, -e));
        l += p0 + p1;
        // bf16 split on the integer pipe: first term = the upper 16 bits, second = the remainder rounded half up
        const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
        hi[k] = __byte_perm(b0, b1, 0x7632);
        const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u), r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
        lo[k] = __byte_perm(__float_as_uint(r0) + 0x8000u, __float_as_uint(r1) + 0x8000u, 0x7632);
      }
      const uint32_t t_p = tmem + lane_addr + (uint32_t)(P_COL + 64 * b + 16 * grp);
      tmem_st16(t_p, hi);
      tmem_st16(t_p + 32, lo);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(smem_u32(&sh->pfull[b]));
    }
    // ---- epilogue: O / l + gated readout; the row sum is the two threads' shares added
    if (ok) {
      const int b = nt & 1;  // the exchange barrier of the parity after the last tile: used (nt - b + 1) / 2 times so far
      sh->stat[b][grp][row] = l;
      mbar_arrive(smem_u32(&sh->xch[b][qd]));
      if (!mbar_wait(smem_u32(&sh->xch[b][qd]), (uint32_t)((nt >> 1) & 1), abort_flag)) ok = false;
      l += sh->stat[b][grp ^ 1][row];
    }
    if (ok && !mbar_wait(smem_u32(&sh->pvdone[(nt - 1) & 1]), (uint32_t)(((nt - 1) >> 1) & 1), abort_flag)) ok = false;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      const float* mr = sc.mch + ((size_t)i * C + (row_ok ? s_row : 0)) * p.Dkv + h * DH;
      OutT* op = out + (((size_t)i * C + (row_ok ? s_row : 0)) * p.H + (size_t)h * p.Gq + hh) * DH;
#pragma unroll
      for (int c1 = 0; c1 < DH / 2; c1 += 32) {
        const int c0 = grp * (DH / 2) + c1;
        float t[32];
        tmem_ld32(t_o + lane_addr + (uint32_t)c0, t);  // (warp-collective: rows out of range load too, and skip the store)
        if (row_ok) {
#pragma unroll
          for (int c = 0; c < 32; c += 8) {
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = t[c + k] * inv + (p.mem ? mr[c0 + c + k] : 0.f);
            if constexpr (sizeof(OutT) == 2) {
              *reinterpret_cast<uint4*>(op + c0 + c) =
                  make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]), pack_bf16(v[6], v[7]));
            } else {
#pragma unroll
              for (int k = 0; k < 8; ++k) op[c0 + c + k] = v[k];
            }
          }
        }
      }
    }
  }
  if (!ok && lane == 0) {
    sh->abort = 1;
    atomicOr(st.status, ST_TIMEOUT);
    // copies that this CTA still has in flight write into its shared memory: give them time to land (bounded)
    for (int k = 0; k < 64; ++k) __nanosleep(1000);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 9) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

bool im_chunk_attn_tc_supported(const ImDims& p) { return p.d == DH && p.Gq <= 8; }

cudaError_t im_chunk_attn_tc_prepare() {
  cudaError_t e = cudaFuncSetAttribute(k_chunk_attention_tc<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_chunk_attention_tc<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

cudaError_t im_launch_chunk_attention_tc(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                         const void* q, void* out) {
  const ImDims& p = L.p;
  const int QB = ROWS / p.Gq;
  dim3 grid((call.C + QB - 1) / QB, p.Hkv, call.n_seq);
  const CUtensorMap& mk = *(const CUtensorMap*)mapK;
  const CUtensorMap& mv = *(const CUtensorMap*)mapV;
  if (p.out_f32) k_chunk_attention_tc<float><<<grid, THREADS, SMEM_BYTES, L.stream>>>(mk, mv, p, L.st, L.sc, call, (const bf16*)q, (float*)out);
  else k_chunk_attention_tc<bf16><<<grid, THREADS, SMEM_BYTES, L.stream>>>(mk, mv, p, L.st, L.sc, call, (const bf16*)q, (bf16*)out);
  ++*L.launches;
  return cudaGetLastError();
}

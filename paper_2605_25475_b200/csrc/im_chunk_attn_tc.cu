// Layer outputs of a prefill chunk's own queries (Eq. 4-5 during chunked prefill): the flash attention of
// im_chunk_attn.cu on the 5th-generation tensor cores, for head_dim 128.
//
// A CTA owns two Q tiles of 128 rows each = 2 floor(128 / G_q) queries x G_q heads of one KV head; row r of tile g is
// TMEM lane r and belongs to softmax thread (g, r).  Per tile of 64 keys and per Q tile g:
//   S_g = Q_g K^T  tcgen05.mma, M = 128 rows, N = 64 keys, K = d = 128 (8 steps); Q_g and the K tile K-major in shared
//                  memory (128-byte swizzle; the K/V tiles come by TMA through the tensor maps of the decode
//                  attention kernel, two 32-row boxes per 64-column half, and serve both Q tiles), S_g in tensor memory
//   softmax        thread (g, r) reads its 64 scores with tcgen05.ld, masks (causal by chunk index), keeps the running
//                  maximum and sum (base 2), and writes P as two bf16 terms (upper 16 bits + rounded remainder: 2^-16)
//                  into TENSOR memory with tcgen05.st, two values per 32-bit column, row = lane: the layout of an A
//                  operand read from tensor memory.  The split is integer arithmetic: the conversion instruction
//                  shares the transcendental unit with ex2.
//   O_g += P_g V   tcgen05.mma with A = P_g from tensor memory, N = d = 128, K = 64 keys (4 steps, both P terms),
//                  accumulating in tensor memory over the tiles; V is used as it lies in the cache ([key][d], i.e.
//                  MN-major for this product: 8-key groups 1024 bytes apart, the two 64-column halves 8 KB apart)
//   rescale        P is formed relative to a reference maximum that is only raised when a row's maximum has
//                  grown by more than 2^8 (or is seen for the first time): then the warp waits for the previous
//                  P V product, multiplies its O rows in tensor memory (tcgen05.ld / st) and its row sums by
//                  2^(m_ref_old - m_ref_new).  Between such events P (<= 2^8) and O need no correction.
// Tensor memory (512 columns): S_g at 64 g, P_g at 128 + 64 g, O_g at 256 + 128 g.  The two Q tiles are independent
// but for the K/V tiles they share: while the threads of one are in their exponentials, the other's loads, maxima
// and barrier round trips and both tiles' products run.  (One Q tile per CTA, with its rows' keys or its tiles dealt
// to two warp groups, needs an exchange of maxima per tile and was no faster than one thread per row.)
// Warps 0-3 / 4-7: softmax, rescale, epilogue of Q tile 0 / 1; warp 8 lane 0: TMA; warp 9: tensor memory owner and
// MMA issue.  The whole of warp 9 runs the issue loop and one elected lane issues each instruction: with the loop
// inside an `if (lane == 0)` the operand descriptors were per-thread values that had to be moved to uniform registers
// for every instruction, and the issue itself (70-90 cycles per MMA of 32-64 cycles) bounded the kernel.
// Every wait is bounded (ST_TIMEOUT).
#include <cuda.h>

#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int DH = 128;
constexpr int KT = 64;                      // keys per tile
constexpr int ROWS = 128;
constexpr int STAGES = 4;
constexpr int HALF_BYTES = KT * 128;        // one 64-column half of a K or V tile: 64 rows x 128 bytes
constexpr int KV_TILE = 2 * HALF_BYTES;     // 16 KB
constexpr int STAGE_BYTES = 2 * KV_TILE;    // K + V
constexpr int Q_BYTES = ROWS * DH * 2;      // 32 KB per Q tile: two halves of 128 rows x 128 bytes
constexpr int QTILES = 2;                   // Q tiles (row groups of 128) per CTA
constexpr int THREADS = 320;                // warps 0-7: softmax (two groups of four), 8: TMA, 9: tensor memory / MMA
constexpr uint32_t WAIT_LIMIT = IM_WAIT_LIMIT;
constexpr int TMEM_COLS = 512;              // per Q tile g: S 64, P 2 terms x 32 (bf16 pairs), O 128
constexpr int S_COL = 0;                    // S of tile g at S_COL + 64 g
constexpr int P_COL = 128;                  // P of tile g, term t at P_COL + 64 g + 32 t
constexpr int O_COL = 256;                  // O of tile g at O_COL + 128 g

struct Shared {
  unsigned long long full[STAGES], empty[STAGES], sfull[2], sempty[2], pfull[2], pvdone[2];
  uint32_t tmem;
  int abort;
};
constexpr int SMEM_BYTES = QTILES * Q_BYTES + STAGES * STAGE_BYTES + (int)sizeof(Shared) + 1024;

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

// grid = (Hkv, ceil(C / (2 QB)), n_seq) with QB = 128 / Gq queries per Q tile; block = 320.  Blocks are dispatched in
// the order of their linear index (x fastest), so the query block is the slower dimension and counts down: block y
// handles the queries from (gridDim.y - 1 - y) * 2 QB, and the blocks with the most keys (the latest queries) of all
// heads start first.  With the shortest first, the last long blocks ran alone at the end (215 us against 186 us).
template <typename OutT>
__global__ void __launch_bounds__(THREADS, 1)
k_chunk_attention_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, ImDims p, ImState st,
                     ImScratch sc, ImCall call, const bf16* __restrict__ q, OutT* __restrict__ out) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;                       // [2 Q tiles][2 halves][128 rows][128 bytes]
  uint8_t* s_kv = smem + QTILES * Q_BYTES;   // [STAGES][K: 2 halves x 64 rows x 128 bytes | V: the same]
  Shared* sh = reinterpret_cast<Shared*>(s_kv + STAGES * STAGE_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x, i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int n0 = st.ctr[u * CTR_STRIDE + CTR_NNEXT];  // entries cached before the chunk (set by the append kernel; CTR_N advances meanwhile)
  const int C = call.C;
  if (n0 < 0 || n0 + C > p.cap) return;  // flagged by the append kernel
  const int QB = ROWS / p.Gq;
  const int s0 = (int)(gridDim.y - 1 - blockIdx.y) * QTILES * QB;
  if (s0 >= C) return;
  const int s_last = min(C, s0 + QTILES * QB) - 1;
  const int n_keys = n0 + s_last + 1;  // slots the block's last query sees
  const int nt = (n_keys + KT - 1) / KT;
  volatile int* abort_flag = &sh->abort;
  if (tid == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int g = 0; g < QTILES; ++g) {
      mbar_init(smem_u32(&sh->sfull[g]), 1);
      mbar_init(smem_u32(&sh->sempty[g]), ROWS);
      mbar_init(smem_u32(&sh->pfull[g]), ROWS);
      mbar_init(smem_u32(&sh->pvdone[g]), 1);
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
  // ---- Q tiles: softmax thread (g, r) writes row r of tile g (query s0 + (128 g + r) / Gq, head (128 g + r) % Gq) into
  // the swizzled K-major layout
  int lim = 0;          // this row sees slots [0, lim)
  bool row_ok = false;
  int s_row = s0, hh = 0;
  const int grp = warp >> 2;         // softmax warps: the Q tile
  const int row = tid & (ROWS - 1);  // softmax threads: the row within the tile = TMEM lane
  if (tid < QTILES * ROWS) {
    const int sl = tid / p.Gq;
    hh = tid % p.Gq;
    s_row = s0 + sl;
    row_ok = sl < QTILES * QB && s_row < C;
    lim = row_ok ? n0 + s_row + 1 : 0;
    const uint4* src = reinterpret_cast<const uint4*>(q + (((size_t)i * C + (row_ok ? s_row : s0)) * p.H + (size_t)h * p.Gq + (row_ok ? hh : 0)) * DH);
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const uint4 v = row_ok ? src[c] : make_uint4(0u, 0u, 0u, 0u);
      uint8_t* dst = s_q + grp * Q_BYTES + (c >> 3) * (ROWS * 128) + (row >> 3) * 1024 + (row & 7) * 128 + (((c & 7) ^ (row & 7)) << 4);
      *reinterpret_cast<uint4*>(dst) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh->tmem;
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
    {  // ---- MMA issue: the whole warp runs the loop (descriptors stay warp-uniform), one elected lane issues.
      // Order in the tensor pipe: S_0(0) S_1(0) | S_0(1) PV_0(0) S_1(1) PV_1(0) | S_0(2) PV_0(1) ...: the score tile
      // j + 1 of a Q tile is issued as soon as its softmax threads have read tile j, ahead of the P V product of tile j
      // (which waits for their P), so that they find it when they come back.
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(KT >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
      const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(ROWS >> 4) << 24);
      const uint32_t qa = smem_u32(s_q);
      auto issue_s = [&](int j, int g) -> bool {  // S_g(j) = Q_g K_j^T
        const int s = j % STAGES;
        if (g == 0 && !mbar_wait(smem_u32(&sh->full[s]), (uint32_t)((j / STAGES) & 1), abort_flag, p.wait_limit)) return false;
        if (j >= 1 && !mbar_wait(smem_u32(&sh->sempty[g]), (uint32_t)((j - 1) & 1), abort_flag)) return false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t ka = smem_u32(s_kv + (size_t)s * STAGE_BYTES);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
          mma_bf16(tmem + (uint32_t)(S_COL + g * KT), desc_sw128(qa + g * Q_BYTES + (ks >> 2) * (ROWS * 128) + (ks & 3) * 32, 16, 1024),
                   desc_sw128(ka + (ks >> 2) * HALF_BYTES + (ks & 3) * 32, 16, 1024), idesc_s, ks ? 1u : 0u);
        mma_commit(smem_u32(&sh->sfull[g]));
        return true;
      };
      ok = issue_s(0, 0) && issue_s(0, 1);
      for (int j = 0; j < nt && ok; ++j) {
        const int s = j % STAGES;
        const uint32_t va = smem_u32(s_kv + (size_t)s * STAGE_BYTES) + KV_TILE;
        for (int g = 0; g < QTILES && ok; ++g) {
          if (j + 1 < nt && !issue_s(j + 1, g)) { ok = false; break; }
          if (!mbar_wait(smem_u32(&sh->pfull[g]), (uint32_t)(j & 1), abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int term = 0; term < 2; ++term)
#pragma unroll
            for (int ks = 0; ks < KT / 16; ++ks)
              mma_bf16_ts(tmem + (uint32_t)(O_COL + g * DH), tmem + (uint32_t)(P_COL + 64 * g + 32 * term + 8 * ks),
                          desc_sw128(va + ks * 2048, HALF_BYTES, 1024), idesc_o, (j | term | ks) ? 1u : 0u);
          mma_commit(smem_u32(&sh->pvdone[g]));
        }
        if (ok) mma_commit(smem_u32(&sh->empty[s]));
      }
    }
  } else {
    // ---- softmax, rescale, epilogue: warps 4 g .. 4 g + 3 own Q tile g, thread = row = TMEM lane (warp w reads lane
    // quarter w % 4).  The two groups share nothing but the K/V tiles, so one group's loads, maxima and waits overlap
    // with the other's exponentials and with the tensor pipe.
    const int g = grp, qd = warp & 3;
    const uint32_t lane_addr = (uint32_t)(qd * 32) << 16;
    const uint32_t t_s = tmem + lane_addr + (uint32_t)(S_COL + g * KT);
    const uint32_t t_p = tmem + lane_addr + (uint32_t)(P_COL + 64 * g);
    const uint32_t t_o = tmem + lane_addr + (uint32_t)(O_COL + g * DH);
    const float sl2 = p.scale * 1.4426950408889634f;  // softmax in base 2
    float m_ref = NEG_INF, l = 0.f;                    // reference maximum of P and O, row sum
    for (int j = 0; j < nt; ++j) {
      if (!mbar_wait(smem_u32(&sh->sfull[g]), (uint32_t)(j & 1), abort_flag)) { ok = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float sv[KT];
      tmem_ld32(t_s, sv);
      tmem_ld32(t_s + 32, sv + 32);
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(smem_u32(&sh->sempty[g]));
      const int key0 = j * KT;
      if (key0 + KT > lim) {  // only the row's last tiles need the causal mask
#pragma unroll
        for (int k = 0; k < KT; ++k) sv[k] = key0 + k < lim ? sv[k] : NEG_INF;
      }
      float t0 = sv[0], t1 = sv[1], t2 = sv[2], t3 = sv[3];
#pragma unroll
      for (int k = 4; k < KT; k += 4) {
        t0 = fmaxf(t0, sv[k]);
        t1 = fmaxf(t1, sv[k + 1]);
        t2 = fmaxf(t2, sv[k + 2]);
        t3 = fmaxf(t3, sv[k + 3]);
      }
      const float tm = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3)) * sl2;  // the scale is positive: the maximum of the scaled scores
      // raise the reference only for a first maximum or a jump of more than 8 (P stays below 2^8 otherwise)
      const bool raise = tm > NEG_INF && (m_ref == NEG_INF || tm > m_ref + 8.0f);
      bool pv_waited = false;
      if (__any_sync(0xffffffffu, raise)) {
        const float corr = raise ? exp2f(m_ref - tm) : 1.0f;  // 0 for a first maximum: nothing accumulated yet
        if (raise) {
          m_ref = tm;
          l *= corr;
        }
        if (j >= 1) {  // O holds the products up to tile j - 1: wait for the last one, then scale the row
          if (!mbar_wait(smem_u32(&sh->pvdone[g]), (uint32_t)((j - 1) & 1), abort_flag)) { ok = false; break; }
          pv_waited = true;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
          for (int c0 = 0; c0 < DH; c0 += 32) {
            float t[32];
            tmem_ld32(t_o + (uint32_t)c0, t);
#pragma unroll
            for (int c = 0; c < 32; ++c) t[c] *= corr;
            tmem_st32(t_o + (uint32_t)c0, t);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
      }
      const float e = m_ref == NEG_INF ? 0.f : m_ref;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
          const float p0 = ex2(fmaf(sv[32 * hf + 2 * k], sl2, -e)), p1 = ex2(fmaf(sv[32 * hf + 2 * k + 1], sl2, -e));
          l += p0 + p1;
          // bf16 split on the integer pipe (the conversion instruction shares the transcendental unit with ex2):
          // first term = the upper 16 bits, second = the remainder rounded half up
          const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
          hi[k] = __byte_perm(b0, b1, 0x7632);
          const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u), r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
          lo[k] = __byte_perm(__float_as_uint(r0) + 0x8000u, __float_as_uint(r1) + 0x8000u, 0x7632);
        }
        if (hf == 0 && j >= 1 && !pv_waited) {  // P is single buffered: the product of tile j - 1 has to be through with it
          if (!mbar_wait(smem_u32(&sh->pvdone[g]), (uint32_t)((j - 1) & 1), abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        }
        tmem_st16(t_p + (uint32_t)(16 * hf), hi);
        tmem_st16(t_p + (uint32_t)(32 + 16 * hf), lo);
      }
      if (!ok) break;
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(smem_u32(&sh->pfull[g]));
    }
    // ---- epilogue: O / l + gated readout
    if (ok && !mbar_wait(smem_u32(&sh->pvdone[g]), (uint32_t)((nt - 1) & 1), abort_flag)) ok = false;
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const float inv = l > 0.f ? 1.0f / l : 0.f;
      const float* mr = sc.mch + ((size_t)i * C + (row_ok ? s_row : 0)) * p.Dkv + h * DH;
      OutT* op = out + (((size_t)i * C + (row_ok ? s_row : 0)) * p.H + (size_t)h * p.Gq + hh) * DH;
#pragma unroll
      for (int c0 = 0; c0 < DH; c0 += 32) {
        float t[32];
        tmem_ld32(t_o + (uint32_t)c0, t);  // (warp-collective: rows out of range load too, and skip the store)
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
  dim3 grid(p.Hkv, (call.C + QTILES * QB - 1) / (QTILES * QB), call.n_seq);
  const CUtensorMap& mk = *(const CUtensorMap*)mapK;
  const CUtensorMap& mv = *(const CUtensorMap*)mapV;
  if (p.out_f32) k_chunk_attention_tc<float><<<grid, THREADS, SMEM_BYTES, L.stream>>>(mk, mv, p, L.st, L.sc, call, (const bf16*)q, (float*)out);
  else k_chunk_attention_tc<bf16><<<grid, THREADS, SMEM_BYTES, L.stream>>>(mk, mv, p, L.st, L.sc, call, (const bf16*)q, (bf16*)out);
  ++*L.launches;
  return cudaGetLastError();
}

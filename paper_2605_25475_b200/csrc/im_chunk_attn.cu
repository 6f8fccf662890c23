// Layer outputs of a prefill chunk's own queries (Eq. 4-5 during chunked prefill, Sec. 4 schedule): query s
// of the chunk attends to every entry cached when the chunk arrived plus the chunk's tokens up to itself, and
// adds g(q_s) m(q_s) read from the memory as the previous evict steps left it.  Runs after the chunk has been
// appended to the cache and before it is compressed.
//
//   k_chunk_readout    m(q_s) for every chunk query: [C x d_M] x [d_M x D_kv] as three tf32 products (mma.sync), gate applied
//   k_chunk_attention  flash attention, queries on the M dimension of mma.sync m16n8k16: a CTA owns
//                      128 rows = floor(128 / G_q) queries x G_q heads of one KV head (row = query * G_q + head),
//                      8 warps x 16 rows, K/V tiles of 32 keys brought in by TMA (the tensor maps of the decode
//                      attention kernel) into a 4-stage ring shared by the warps; softmax in base 2; P as two
//                      bf16 terms (2^-17) for the P V product; epilogue adds the readout and stores.
#include <cuda.h>

#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int TILE = IM_ATTN_TILE;  // keys per tile
constexpr int CA_WARPS = 8;
constexpr int CA_ROWS = CA_WARPS * 16;
constexpr int CA_STAGES = 4;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(x), "r"(y), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two floats -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ------------------------------------------------------------------------------------------------
// mch[i][s][col] = g(q_s) * cscale * (sum_m phi_s[m] Mhat[m][col]) / (eps + sum_m phi_s[m]^2 b[m])   (Eq. 5,
// gate of Eq. 4).  The pending list is empty here (the call folds it first).  phi_s and the gate logit are
// rows [0, dM) and dM of the chunk's memory-side projection, which the call writes behind the indexer-side
// block of the projection scratch.  A float32 product ([C x d_M] x [d_M x D_kv], 2.1 GFLOP per 2048-token chunk) on
// the tensor cores as three tf32 products: x = hi + lo with hi the upper 19 bits of x (what a tf32 operand keeps)
// and lo the exact remainder, and phi Mhat ~ hi hi + hi lo + lo hi (the dropped lo lo term and the truncation of lo
// are 2^-20 of a product).  64 queries x 128 columns per block, 8 warps of 32 queries x 32 columns (2 x 4
// mma.sync.m16n8k8 tiles each), K slices of 16 staged through registers into shared memory while the previous slice
// is multiplied; rows padded by 8 floats so that a warp's fragment loads (4 k x 8 rows) touch 32 different banks.
// The loop is bound by the latency of the next slice's loads, not by the arithmetic (the float32 FMA version of the
// same loop took the same 78 us): hence the small tile, two or three blocks per SM.  The denominators are summed by
// the staging threads (each holds 4 queries x 1 m per slice) in float32.
// grid = (ceil(Dkv / 128), ceil(C / 64), n_seq), block = 256.
constexpr int CR_T = 128, CR_TQ = 64, CR_K = 16, CR_LD = CR_T + 8, CR_LDQ = CR_TQ + 8;
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// x = hi + lo, both with the low 13 mantissa bits clear
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  hi = __float_as_uint(x) & 0xffffe000u;
  lo = __float_as_uint(x - __uint_as_float(hi)) & 0xffffe000u;
}
__global__ void __launch_bounds__(256, 3) k_chunk_readout(ImDims p, ImState st, ImWeights w, ImScratch sc, ImCall call) {
  __shared__ __align__(16) float s_a[2][CR_K][CR_LDQ];  // [m][query]
  __shared__ __align__(16) float s_b[2][CR_K][CR_LD];  // [m][col]
  __shared__ float s_den[CR_TQ];
  const int i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const float* proj = sc.raw + (size_t)p.S * p.max_chunk * p.R3;  // [n_seq * C][dM + 1]
  const int ps = p.dM + 1;
  const int q0 = blockIdx.y * CR_TQ, col0 = blockIdx.x * CR_T;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int wq = (warp & 1) * 32, wc = (warp >> 1) * 32;  // the warp's 32 queries x 32 columns of the tile
  const float* Mh = st.Mhat + u * p.dM * p.Dkv;
  const float* bv = st.bvec + u * p.dM;
  // staging roles: A - thread t loads m = t & 15 of queries (t >> 4) + 16 j, j < 4 (16 consecutive floats of a
  // projection row per 16 threads); B - thread t loads float4 (t & 31) of rows (t >> 5) and (t >> 5) + 8
  const int am = tid & 15, as = tid >> 4;
  const int bc = (tid & 31) * 4, bm = tid >> 5;
  const bool b_vec = (p.Dkv & 3) == 0;
  float ra[4], den[4];
  float4 rb[2];
#pragma unroll
  for (int j = 0; j < 4; ++j) den[j] = 0.f;
  auto fetch = [&](int m0) {
    const int m = m0 + am;
    const float bm_ = m < p.dM ? bv[m] : 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int s = q0 + as + 16 * j;
      ra[j] = (s < call.C && m < p.dM) ? proj[((size_t)i * call.C + s) * ps + m] : 0.f;
      den[j] = fmaf(ra[j] * ra[j], bm_, den[j]);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int mm = m0 + bm + 8 * j, c = col0 + bc;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (mm < p.dM) {
        const float* src = Mh + (size_t)mm * p.Dkv + c;
        if (b_vec && c + 3 < p.Dkv) v = *reinterpret_cast<const float4*>(src);
        else {
          if (c < p.Dkv) v.x = src[0];
          if (c + 1 < p.Dkv) v.y = src[1];
          if (c + 2 < p.Dkv) v.z = src[2];
          if (c + 3 < p.Dkv) v.w = src[3];
        }
      }
      rb[j] = v;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int j = 0; j < 4; ++j) s_a[buf][am][as + 16 * j] = ra[j];
#pragma unroll
    for (int j = 0; j < 2; ++j) *reinterpret_cast<float4*>(&s_b[buf][bm + 8 * j][bc]) = rb[j];
  };
  float acc[2][4][4];
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int ni = 0; ni < 4; ++ni)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mi][ni][e] = 0.f;
  fetch(0);
  stash(0);
  __syncthreads();
  const int nk = (p.dM + CR_K - 1) / CR_K;
  for (int kb = 0; kb < nk; ++kb) {
    const int buf = kb & 1;
    if (kb + 1 < nk) fetch((kb + 1) * CR_K);
#pragma unroll
    for (int kk = 0; kk < CR_K; kk += 8) {
      // fragments: A (query row, m): a0 (g, t), a1 (g + 8, t), a2 (g, t + 4), a3 (g + 8, t + 4); B (m, column): b0 (t, g),
      // b1 (t + 4, g)
      uint32_t bh[4][2], bl[4][2];
#pragma unroll
      for (int ni = 0; ni < 4; ++ni) {
        split_tf32(s_b[buf][kk + t][wc + ni * 8 + g], bh[ni][0], bl[ni][0]);
        split_tf32(s_b[buf][kk + t + 4][wc + ni * 8 + g], bh[ni][1], bl[ni][1]);
      }
#pragma unroll
      for (int mi = 0; mi < 2; ++mi) {
        uint32_t ah[4], al[4];
        const int qr = wq + mi * 16 + g;
        split_tf32(s_a[buf][kk + t][qr], ah[0], al[0]);
        split_tf32(s_a[buf][kk + t][qr + 8], ah[1], al[1]);
        split_tf32(s_a[buf][kk + t + 4][qr], ah[2], al[2]);
        split_tf32(s_a[buf][kk + t + 4][qr + 8], ah[3], al[3]);
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
          mma_tf32(acc[mi][ni], al, bh[ni]);
          mma_tf32(acc[mi][ni], ah, bl[ni]);
          mma_tf32(acc[mi][ni], ah, bh[ni]);
        }
      }
    }
    if (kb + 1 < nk) stash(buf ^ 1);  // (the other buffer: last read before the barrier that ended slice kb - 1)
    __syncthreads();
  }
  // denominators: the 16 threads with the same query set (tid >> 4) hold one m each per slice
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    float d = den[j];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
    if (am == 0) s_den[as + 16 * j] = d;
  }
  __syncthreads();
  const float cs = st.cscale[u];
  // C fragment: c0, c1 (row g, columns 2 t, 2 t + 1), c2, c3 (row g + 8)
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int row = wq + mi * 16 + g + 8 * hf, s = q0 + row;
      if (s >= call.C) continue;
      const float logit = proj[((size_t)i * call.C + s) * ps + p.dM] + w.bg[0];
      const float f = cs / (1.0f + expf(-logit)) / (p.eps + s_den[row]);
      float* dst = sc.mch + ((size_t)i * call.C + s) * p.Dkv;
#pragma unroll
      for (int ni = 0; ni < 4; ++ni) {
        const int col = col0 + wc + ni * 8 + 2 * t;
        if (col < p.Dkv) dst[col] = f * acc[mi][ni][2 * hf];
        if (col + 1 < p.Dkv) dst[col + 1] = f * acc[mi][ni][2 * hf + 1];
      }
    }
}

// ------------------------------------------------------------------------------------------------
// grid = (ceil(C / QB), Hkv, n_seq) with QB = 128 / Gq queries per CTA; block = 256.
// Dynamic shared memory: CA_STAGES x (K tile + V tile) (1024-byte aligned), then the barriers.
template <int DH, typename OutT>
__global__ void __launch_bounds__(CA_WARPS * 32, 1)
k_chunk_attention(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, ImDims p, ImState st,
                  ImScratch sc, ImCall call, const bf16* __restrict__ q, OutT* __restrict__ out) {
  constexpr int KS = DH / 16;                // k-steps of S = Q K^T
  constexpr int DN = DH / 8;                 // 8-column tiles of O
  constexpr int NT = TILE / 8;               // 8-key tiles of S
  constexpr int BOXES = DH / 64;             // 128-byte column boxes per row
  constexpr int TILE_BYTES = TILE * DH * 2;
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  extern __shared__ __align__(1024) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)CA_STAGES * STAGE_BYTES);
  uint64_t* empty = full + CA_STAGES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int h = blockIdx.y, i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int n0 = st.ctr[u * CTR_STRIDE + CTR_NNEXT];  // entries cached before the chunk (set by the append kernel; CTR_N advances meanwhile)
  const int C = call.C;
  if (n0 < 0 || n0 + C > p.cap) return;  // flagged by the append kernel
  const int QB = CA_ROWS / p.Gq;
  const int s0 = blockIdx.x * QB;
  if (s0 >= C) return;
  const int s_last = min(C, s0 + QB) - 1;
  const int n_keys = n0 + s_last + 1;  // slots the block's last query sees
  const int nt_tiles = (n_keys + TILE - 1) / TILE;
  if (threadIdx.x == 0) {
    for (int s = 0; s < CA_STAGES; ++s) {
      mbar_init(smem_u32(&full[s]), 1);
      mbar_init(smem_u32(&empty[s]), CA_WARPS);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  const int row_base = (int)((u * p.Hkv + h) * (size_t)p.cap);
  auto issue = [&](int j) {  // thread 0 only
    const int s = j % CA_STAGES;
    const uint32_t bar = smem_u32(&full[s]);
    const uint32_t dst = smem_u32(smem + (size_t)s * STAGE_BYTES);
    mbar_expect_tx(bar, STAGE_BYTES);
#pragma unroll
    for (int b = 0; b < BOXES; ++b) {
      tma_load_2d(dst + b * (TILE * 128), &tmK, b * 64, row_base + j * TILE, bar);
      tma_load_2d(dst + TILE_BYTES + b * (TILE * 128), &tmV, b * 64, row_base + j * TILE, bar);
    }
  };
  if (threadIdx.x == 0)
    for (int j = 0; j < CA_STAGES && j < nt_tiles; ++j) issue(j);

  // ---- this thread's two rows: (query, head of the group)
  const int rowA = warp * 16 + g, rowB = rowA + 8;
  const int slA = rowA / p.Gq, slB = rowB / p.Gq;
  const int sA = s0 + slA, sB = s0 + slB;
  const bool okA = slA < QB && sA < C, okB = slB < QB && sB < C;
  const int limA = okA ? n0 + sA + 1 : 0, limB = okB ? n0 + sB + 1 : 0;  // visible slots: [0, lim)
  uint32_t qa[KS][4];
  {
    const bf16* qA = q + (((size_t)i * C + (okA ? sA : s0)) * p.H + (size_t)h * p.Gq + (okA ? rowA % p.Gq : 0)) * DH;
    const bf16* qB = q + (((size_t)i * C + (okB ? sB : s0)) * p.H + (size_t)h * p.Gq + (okB ? rowB % p.Gq : 0)) * DH;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qa[ks][0] = *reinterpret_cast<const uint32_t*>(qA + ks * 16 + 2 * t);
      qa[ks][1] = *reinterpret_cast<const uint32_t*>(qB + ks * 16 + 2 * t);
      qa[ks][2] = *reinterpret_cast<const uint32_t*>(qA + ks * 16 + 8 + 2 * t);
      qa[ks][3] = *reinterpret_cast<const uint32_t*>(qB + ks * 16 + 8 + 2 * t);
    }
  }
  float o[DN][4];
#pragma unroll
  for (int dn = 0; dn < DN; ++dn) o[dn][0] = o[dn][1] = o[dn][2] = o[dn][3] = 0.f;
  float mA = NEG_INF, mB = NEG_INF, lA = 0.f, lB = 0.f;  // l: this thread's share of the row sums
  const float sl2 = p.scale * 1.4426950408889634f;        // softmax in base 2
  // the warp's rows see no key at or beyond this slot: later tiles are waited for and released, not computed
  int warp_lim = max(limA, limB);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) warp_lim = max(warp_lim, __shfl_xor_sync(0xffffffffu, warp_lim, off));
  bool ok = true;
  for (int j = 0; j < nt_tiles; ++j) {
    const int s = j % CA_STAGES;
    // every warp waits for every tile, also for the tiles it has nothing to compute on: an arrival on the
    // stage's release barrier counts for whatever phase is current, so no warp may run a whole ring ahead
    if (!mbar_wait(smem_u32(&full[s]), (uint32_t)((j / CA_STAGES) & 1))) { ok = false; break; }
    if (j * TILE < warp_lim) {
      const uint32_t Ks = smem_u32(smem + (size_t)s * STAGE_BYTES), Vs = Ks + TILE_BYTES;
      // ---- S = Q K^T : [16 rows] x [32 keys]
      float sacc[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
        const int r = nt * 8 + (lane & 7);
#pragma unroll
        for (int ks = 0; ks < KS; ks += 2) {
          const int c = 2 * ks + (lane >> 3);
          const uint32_t addr = Ks + (c >> 3) * (TILE * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4(addr, b0, b1, b2, b3);
          mma_bf16(sacc[nt], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
          mma_bf16(sacc[nt], qa[ks + 1][0], qa[ks + 1][1], qa[ks + 1][2], qa[ks + 1][3], b2, b3);
        }
      }
      // ---- causal mask and online softmax: elements 0,1 belong to row A, 2,3 to row B; keys 8 nt + 2t (+1)
      const int key0 = j * TILE;
      float tmA = NEG_INF, tmB = NEG_INF;
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const int k0 = key0 + nt * 8 + 2 * t;
        sacc[nt][0] = k0 < limA ? sacc[nt][0] * sl2 : NEG_INF;
        sacc[nt][1] = k0 + 1 < limA ? sacc[nt][1] * sl2 : NEG_INF;
        sacc[nt][2] = k0 < limB ? sacc[nt][2] * sl2 : NEG_INF;
        sacc[nt][3] = k0 + 1 < limB ? sacc[nt][3] * sl2 : NEG_INF;
        tmA = fmaxf(tmA, fmaxf(sacc[nt][0], sacc[nt][1]));
        tmB = fmaxf(tmB, fmaxf(sacc[nt][2], sacc[nt][3]));
      }
      tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 1));
      tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 2));
      tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 1));
      tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 2));
      const float mnA = fmaxf(mA, tmA), mnB = fmaxf(mB, tmB);
      // a row that has seen no key yet keeps the factor 1 (its sums are zero anyway)
      const float cA = mnA == NEG_INF ? 1.f : exp2f(mA - mnA), cB = mnB == NEG_INF ? 1.f : exp2f(mB - mnB);
      const float eA = mnA == NEG_INF ? 0.f : mnA, eB = mnB == NEG_INF ? 0.f : mnB;
      mA = mnA;
      mB = mnB;
      lA *= cA;
      lB *= cB;
#pragma unroll
      for (int dn = 0; dn < DN; ++dn) { o[dn][0] *= cA; o[dn][1] *= cA; o[dn][2] *= cB; o[dn][3] *= cB; }
      uint32_t ph[NT][2], pl[NT][2];  // P as A fragments, high and low bf16 terms
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const float p0 = exp2f(sacc[nt][0] - eA), p1 = exp2f(sacc[nt][1] - eA);
        const float p2 = exp2f(sacc[nt][2] - eB), p3 = exp2f(sacc[nt][3] - eB);
        lA += p0 + p1;
        lB += p2 + p3;
        ph[nt][0] = pack_bf16(p0, p1);
        ph[nt][1] = pack_bf16(p2, p3);
        pl[nt][0] = pack_bf16(p0 - __uint_as_float(ph[nt][0] << 16), p1 - __uint_as_float(ph[nt][0] & 0xffff0000u));
        pl[nt][1] = pack_bf16(p2 - __uint_as_float(ph[nt][1] << 16), p3 - __uint_as_float(ph[nt][1] & 0xffff0000u));
      }
      // ---- O += P V : [16 rows] x [DH]
#pragma unroll
      for (int kk = 0; kk < TILE / 16; ++kk) {
        const int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int dn = 0; dn < DN; dn += 2) {
          const int c = dn + (lane >> 4);
          const uint32_t addr = Vs + (c >> 3) * (TILE * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(addr, b0, b1, b2, b3);
          mma_bf16(o[dn], ph[2 * kk][0], ph[2 * kk][1], ph[2 * kk + 1][0], ph[2 * kk + 1][1], b0, b1);
          mma_bf16(o[dn], pl[2 * kk][0], pl[2 * kk][1], pl[2 * kk + 1][0], pl[2 * kk + 1][1], b0, b1);
          mma_bf16(o[dn + 1], ph[2 * kk][0], ph[2 * kk][1], ph[2 * kk + 1][0], ph[2 * kk + 1][1], b2, b3);
          mma_bf16(o[dn + 1], pl[2 * kk][0], pl[2 * kk][1], pl[2 * kk + 1][0], pl[2 * kk + 1][1], b2, b3);
        }
      }
    }
    // ---- the warp is done with the stage; thread 0 refills it once every warp is
    __syncwarp();
    if (lane == 0) mbar_arrive(smem_u32(&empty[s]));
    if (threadIdx.x == 0 && j + CA_STAGES < nt_tiles) {
      if (!mbar_wait(smem_u32(&empty[s]), (uint32_t)((j / CA_STAGES) & 1))) { ok = false; break; }
      issue(j + CA_STAGES);
    }
  }
  if (!ok) {
    if (lane == 0) {
      atomicOr(st.status, ST_TIMEOUT);
      // copies that this CTA still has in flight write into its shared memory: give them time to land (bounded)
      for (int k = 0; k < 64; ++k) __nanosleep(1000);
    }
    return;
  }
  // ---- normalise, add the gated readout, store
  lA += __shfl_xor_sync(0xffffffffu, lA, 1);
  lA += __shfl_xor_sync(0xffffffffu, lA, 2);
  lB += __shfl_xor_sync(0xffffffffu, lB, 1);
  lB += __shfl_xor_sync(0xffffffffu, lB, 2);
  const float iA = lA > 0.f ? 1.0f / lA : 0.f, iB = lB > 0.f ? 1.0f / lB : 0.f;
  const float* mrA = sc.mch + ((size_t)i * C + (okA ? sA : 0)) * p.Dkv + h * DH;
  const float* mrB = sc.mch + ((size_t)i * C + (okB ? sB : 0)) * p.Dkv + h * DH;
  OutT* oA = out + (((size_t)i * C + (okA ? sA : 0)) * p.H + (size_t)h * p.Gq + rowA % p.Gq) * DH;
  OutT* oB = out + (((size_t)i * C + (okB ? sB : 0)) * p.H + (size_t)h * p.Gq + rowB % p.Gq) * DH;
#pragma unroll
  for (int dn = 0; dn < DN; ++dn) {
    const int c = dn * 8 + 2 * t;
    if (okA) {
      const float v0 = o[dn][0] * iA + (p.mem ? mrA[c] : 0.f), v1 = o[dn][1] * iA + (p.mem ? mrA[c + 1] : 0.f);
      if constexpr (sizeof(OutT) == 2) *reinterpret_cast<uint32_t*>(oA + c) = pack_bf16(v0, v1);
      else { oA[c] = v0; oA[c + 1] = v1; }
    }
    if (okB) {
      const float v0 = o[dn][2] * iB + (p.mem ? mrB[c] : 0.f), v1 = o[dn][3] * iB + (p.mem ? mrB[c + 1] : 0.f);
      if constexpr (sizeof(OutT) == 2) *reinterpret_cast<uint32_t*>(oB + c) = pack_bf16(v0, v1);
      else { oB[c] = v0; oB[c + 1] = v1; }
    }
  }
}

int chunk_attn_smem(const ImDims& p) { return CA_STAGES * 2 * TILE * p.d * 2 + 2 * CA_STAGES * 8; }

}  // namespace

cudaError_t im_chunk_attn_prepare(const ImDims& p) {
  const int smem = chunk_attn_smem(p);
  cudaError_t e = cudaSuccess;
  if (p.d == 64) {
    e = cudaFuncSetAttribute(k_chunk_attention<64, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_chunk_attention<64, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  } else {
    e = cudaFuncSetAttribute(k_chunk_attention<128, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_chunk_attention<128, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  }
  return e;
}

cudaError_t im_launch_chunk_readout(const ImLaunch& L, const ImCall& call) {
  dim3 grid((L.p.Dkv + CR_T - 1) / CR_T, (call.C + CR_TQ - 1) / CR_TQ, call.n_seq);
  k_chunk_readout<<<grid, 256, 0, L.stream>>>(L.p, L.st, L.w, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_chunk_attention(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                      const void* q, void* out) {
  const ImDims& p = L.p;
  const int QB = CA_ROWS / p.Gq;
  dim3 grid((call.C + QB - 1) / QB, p.Hkv, call.n_seq);
  const int smem = chunk_attn_smem(p);
  const CUtensorMap& mk = *(const CUtensorMap*)mapK;
  const CUtensorMap& mv = *(const CUtensorMap*)mapV;
  const bf16* qp = (const bf16*)q;
  if (p.d == 64) {
    if (p.out_f32) k_chunk_attention<64, float><<<grid, CA_WARPS * 32, smem, L.stream>>>(mk, mv, p, L.st, L.sc, call, qp, (float*)out);
    else k_chunk_attention<64, bf16><<<grid, CA_WARPS * 32, smem, L.stream>>>(mk, mv, p, L.st, L.sc, call, qp, (bf16*)out);
  } else {
    if (p.out_f32) k_chunk_attention<128, float><<<grid, CA_WARPS * 32, smem, L.stream>>>(mk, mv, p, L.st, L.sc, call, qp, (float*)out);
    else k_chunk_attention<128, bf16><<<grid, CA_WARPS * 32, smem, L.stream>>>(mk, mv, p, L.st, L.sc, call, qp, (bf16*)out);
  }
  ++*L.launches;
  return cudaGetLastError();
}

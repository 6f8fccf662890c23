// Skinny GEMMs of the path (a0 projections, phi of evicted keys): out[v][r] = sum_k W[r][k] * in[v][k]
// with a handful to a few thousand weight rows and 1 .. 65536 input vectors, bf16 operands, float32
// accumulation on mma.sync m16n8k16.  Weight-streaming bound in decode (every weight byte is read
// once per call), so the grid is (16-row tiles) x (K splits) to spread the stream over the SMs; the
// K-split partial sums are added by the consumer in a fixed order (deterministic).
// Also here: the float64 indexer-key projection, split over K the same way.
#include "im_internal.cuh"

namespace {

constexpr int KC_MAX = 512;  // K elements staged per round (ImGemmArgs::kc, a multiple of 16, at most this)
// A staged row takes kc * 2 + 16 bytes: consecutive rows shift by one 16-byte bank group (conflict-free ldmatrix).
constexpr int VB = 32;                  // vectors per CTA (4 warps x 8)

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int sz = valid ? 16 : 0;  // src-size 0: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ const bf16* vec_ptr(const ImGemmArgs& a, int sel, long long v) {
  return a.in[sel] + (v / a.in_cnt[sel]) * a.in_outer[sel] + (v % a.in_cnt[sel]) * a.in_inner[sel];
}

// grid = (row tiles over all jobs, ksplit, ceil(NV / 32)), block = 128.
// Dynamic smem: two stages of (16 weight rows [+ 16 rows of the second term] + 32 vector rows) x ROW_BYTES;
// the cp.async copies of round r+1 are in flight while round r is multiplied.
__global__ void __launch_bounds__(128) k_skinny_gemm(ImGemmArgs a) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int KC = a.kc, ROW_BYTES = a.kc * 2 + 16;
  const int stage_rows = a.any_w2 ? 64 : 48;
  const int offB = a.any_w2 ? 32 : 16;  // row offset of the vector tile inside a stage
  int tile = blockIdx.x, j = 0;
  while (j + 1 < a.n_jobs && tile >= (a.job[j].rows + 15) / 16) {
    tile -= (a.job[j].rows + 15) / 16;
    ++j;
  }
  const ImGemmJob job = a.job[j];
  const int r0 = tile * 16;
  const int ks = blockIdx.y;
  const int kspan = a.K / a.ksplit;
  const int kbeg = ks * kspan;
  const long long v0 = (long long)blockIdx.z * VB;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rounds = (kspan + KC - 1) / KC;
  // warp w stages rows w, w+4, ...; one row pointer per row, lanes stride over its 16-byte chunks
  auto issue = [&](int rd) {
    unsigned char* st = smem + (size_t)(rd & 1) * stage_rows * ROW_BYTES;
    const int k0 = rd * KC;
    const int chunks = min(KC, kspan - k0) / 8;
    for (int r = warp; r < 16; r += 4) {
      const bool valid = r0 + r < job.rows;
      const size_t off = (size_t)(valid ? r0 + r : 0) * a.K + kbeg + k0;
      for (int c = lane; c < chunks; c += 32) {
        cp_async16(smem_u32(st + r * ROW_BYTES + c * 16), job.W + off + c * 8, valid);
        if (job.W2) cp_async16(smem_u32(st + (16 + r) * ROW_BYTES + c * 16), job.W2 + off + c * 8, valid);
      }
    }
    for (int r = warp; r < VB; r += 4) {
      const bool valid = v0 + r < a.NV;
      const bf16* src = vec_ptr(a, job.in_sel, valid ? v0 + r : 0) + kbeg + k0;
      for (int c = lane; c < chunks; c += 32) cp_async16(smem_u32(st + (offB + r) * ROW_BYTES + c * 16), src + c * 8, valid);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  issue(0);
  if (rounds > 1) issue(1);
  for (int rd = 0; rd < rounds; ++rd) {
    if (rd + 1 < rounds) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    const uint32_t stg = smem_u32(smem + (size_t)(rd & 1) * stage_rows * ROW_BYTES);
    const int kc = min(KC, kspan - rd * KC);  // multiple of 16
    // A fragment rows: lanes 0-7 rows 0-7 (k 0-7), 8-15 rows 8-15 (k 0-7), 16-23 rows 0-7 (k 8-15), 24-31 rows 8-15 (k 8-15)
    const uint32_t aBase = stg + ((lane & 7) + ((lane >> 3) & 1) * 8) * ROW_BYTES + (lane >> 4) * 16;
    // B fragment rows (= vectors): lanes 0-7 k 0-7, lanes 8-15 k 8-15 (the other lanes' addresses are ignored by .x2)
    const uint32_t bBase = stg + (offB + warp * 8 + (lane & 7)) * ROW_BYTES + ((lane >> 3) & 1) * 16;
    for (int kk = 0; kk < kc; kk += 16) {
      uint32_t a0, a1, a2, a3, b0, b1;
      ldsm_x4(aBase + kk * 2, a0, a1, a2, a3);
      ldsm_x2(bBase + kk * 2, b0, b1);
      mma_bf16(acc, a0, a1, a2, a3, b0, b1);
      if (job.W2) {
        ldsm_x4(aBase + 16 * ROW_BYTES + kk * 2, a0, a1, a2, a3);
        mma_bf16(acc, a0, a1, a2, a3, b0, b1);
      }
    }
    __syncthreads();  // everyone is done with this stage before it is refilled
    if (rd + 2 < rounds) issue(rd + 2);
  }
  // C fragment: rows g / g+8 (weight rows), columns 2t / 2t+1 (vectors of this warp)
  const long long vA = v0 + warp * 8 + 2 * t, vB = vA + 1;
  float* outk = a.out + (size_t)ks * a.ks_stride;
  const int rA = r0 + g, rB = r0 + g + 8;
  if (vA < a.NV) {
    float* o = outk + (vA / a.out_cnt) * a.out_outer + (vA % a.out_cnt) * a.out_inner + job.row0;
    if (rA < job.rows) o[rA] = acc[0];
    if (rB < job.rows) o[rB] = acc[2];
  }
  if (vB < a.NV) {
    float* o = outk + (vB / a.out_cnt) * a.out_outer + (vB % a.out_cnt) * a.out_inner + job.row0;
    if (rA < job.rows) o[rA] = acc[1];
    if (rB < job.rows) o[rB] = acc[3];
  }
}

// ------------------------------------------------------------------------------------------------
// Decode variant for at most a few dozen vectors: the same product with the MMA fragments loaded straight
// from global memory, no shared-memory staging.  It has to run next to the attention kernel, whose CTAs
// leave about 30 KB of shared memory per SM, and it is latency bound: what counts is how many weight bytes
// a warp has in flight.  The contraction index may be permuted as long as both operands use the same
// permutation, so a thread takes 8 consecutive k (one 16-byte load) of its fragment row and feeds them to
// two k-steps: k-step s of a 32-wide chunk uses elements 4s .. 4s+3 of every thread's vector.  A warp
// issues all loads of up to 4 chunks before the first MMA.
// grid = (row tiles over all jobs, ksplit, ceil(NV / 32)), block = 256: the warps take the 32-wide chunks of
// the K split round-robin and their accumulators are added through shared memory in warp order.
// 16-byte read-only load that the compiler may neither reorder nor delay: the point of the direct variant is
// that all loads of a batch are in flight together
__device__ __forceinline__ uint4 ldg128_now(const void* p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void dmma_884(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1]) : "d"(a), "d"(b));
}
__device__ __forceinline__ double bf16_elem(const uint4& v, int s) {
  const uint32_t w = s < 2 ? v.x : s < 4 ? v.y : s < 6 ? v.z : v.w;
  return (double)((s & 1) ? __uint_as_float(w & 0xffff0000u) : __uint_as_float(w << 16));
}
// One block's share of the float64 key projection (see k_proj_key_mma): block (bx, by) of a (ceil(NV / 8), ksplit)
// grid, W warps, `red` = W * NT * 64 doubles of shared memory.
template <int NT, int W>
__device__ __forceinline__ void proj_key_mma_block(int D, int dI, const bf16* __restrict__ Uk, const bf16* __restrict__ x, int NV,
                                                   int ksplit, double* __restrict__ keyp, int bx, int by, double* red) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 2, q = lane & 3;
  const long long v0 = (long long)bx * 8;
  const int kspan = D / (W * ksplit), kbeg = (by * W + warp) * kspan;  // a multiple of 32 (checked by the launcher)
  keyp += (size_t)by * NV * dI;
  const bf16* xrow = x + (size_t)min(v0 + r, (long long)NV - 1) * D + kbeg + 8 * q;
  const bf16* urow = Uk + (size_t)r * D + kbeg + 8 * q;
  double c[NT][2];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) c[nt][0] = c[nt][1] = 0.0;
  // the loads of four 32-wide chunks are requested before the first of them is converted and multiplied: the loop is
  // bound by the latency of its load -> convert -> mma chains, not by arithmetic
  constexpr int PF = 4;
  for (int kb0 = 0; kb0 < kspan; kb0 += 32 * PF) {
    uint4 xa[PF], ub[PF][NT];
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      const int kb = min(kb0 + 32 * i, kspan - 32);  // (a chunk past the end is loaded again and skipped below)
      xa[i] = *reinterpret_cast<const uint4*>(xrow + kb);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) ub[i][nt] = *reinterpret_cast<const uint4*>(urow + (size_t)nt * 8 * D + kb);
    }
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      if (kb0 + 32 * i >= kspan) break;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const double a = bf16_elem(xa[i], s);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) dmma_884(c[nt], a, bf16_elem(ub[i][nt], s));
      }
    }
  }
  // C fragment: row r (vector), columns 2 q and 2 q + 1 (weight row of the n-tile)
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    red[(warp * NT + nt) * 64 + r * 8 + 2 * q] = c[nt][0];
    red[(warp * NT + nt) * 64 + r * 8 + 2 * q + 1] = c[nt][1];
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < NT * 64; idx += 32 * W) {
    const int nt = idx >> 6, e = idx & 63;
    const long long v = v0 + (e >> 3);
    if (v < NV) {
      double sum = red[nt * 64 + e];
#pragma unroll
      for (int w = 1; w < W; ++w) sum += red[(w * NT + nt) * 64 + e];
      keyp[(size_t)v * dI + nt * 8 + (e & 7)] = sum;
    }
  }
}

constexpr int DG_DEPTH = 4;   // 32-wide chunks whose loads (weights and vectors) a warp has in flight
constexpr int DG_WARPS = 8;
template <bool TWO>  // TWO: the jobs have a second weight term
__global__ void __launch_bounds__(DG_WARPS * 32) k_direct_gemm(ImGemmArgs a) {
  // the warps' partial tiles are added through shared memory in two rounds of four warps (half the buffer: the block
  // fits next to a streaming attention CTA that leaves 12 KB of an SM's shared memory), in warp order: deterministic
  constexpr int RED_BYTES = (DG_WARPS / 2) * 16 * 33 * 4 > DG_WARPS * 2 * 64 * 8 ? (DG_WARPS / 2) * 16 * 33 * 4 : DG_WARPS * 2 * 64 * 8;
  __shared__ __align__(16) unsigned char red_raw[RED_BYTES];  // the float tiles below, or the key projection's doubles
  float (*red)[16][33] = reinterpret_cast<float (*)[16][33]>(red_raw);
  // a kernel launched as programmatic dependent of this one may start its own preamble now
  asm volatile("griddepcontrol.launch_dependents;");
  IM_MARK_GEMM(a, 0);
  if ((int)blockIdx.x >= a.tiles) {
    // the float64 indexer-key projection of the same vectors, in the same launch (blocks behind the tiles' blocks)
    if (blockIdx.z == 0) {
      const int kid = ((int)blockIdx.x - a.tiles) * (int)gridDim.y + (int)blockIdx.y;
      const int nbx = (a.key_nv + 7) / 8;
      if (kid < nbx * a.key_ksplit) {
        double* redd = reinterpret_cast<double*>(red_raw);
        if (a.key_dI == 8) proj_key_mma_block<1, DG_WARPS>(a.K, 8, a.key_W, a.key_x, a.key_nv, a.key_ksplit, a.key_out, kid % nbx, kid / nbx, redd);
        else proj_key_mma_block<2, DG_WARPS>(a.K, 16, a.key_W, a.key_x, a.key_nv, a.key_ksplit, a.key_out, kid % nbx, kid / nbx, redd);
      }
    }
    return;
  }
  int tile = blockIdx.x, j = 0;
  while (j + 1 < a.n_jobs && tile >= (a.job[j].rows + 15) / 16) {
    tile -= (a.job[j].rows + 15) / 16;
    ++j;
  }
  const ImGemmJob job = a.job[j];
  const int r0 = tile * 16;
  const int ks = blockIdx.y;
  const int kspan = a.K / a.ksplit;  // a multiple of 32 (checked by the launcher)
  const int kbeg = ks * kspan;
  const long long v0 = (long long)blockIdx.z * VB;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_chunks = kspan / 32;
  // fragment rows of this thread (clamped: results of rows / vectors out of range are not stored)
  const int rowA = min(r0 + g, job.rows - 1), rowB = min(r0 + g + 8, job.rows - 1);
  const bf16* xb[4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) xb[nt] = vec_ptr(a, job.in_sel, min(v0 + nt * 8 + g, (long long)a.NV - 1)) + kbeg + 8 * t;
#ifdef IM_TRACE
  if (a.trace_skip & 4)  // timing experiment: the vectors are read from the (L2-resident) weights instead
    for (int nt = 0; nt < 4; ++nt) xb[nt] = job.W + (size_t)min(nt * 8 + g, job.rows - 1) * a.K + kbeg + 8 * t;
#endif
  float acc[4][4];
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  for (int c0 = warp; c0 < n_chunks; c0 += DG_WARPS * DG_DEPTH) {
    // weights (the long round trip) first, then the vectors (L2: every block reads the same few vectors)
    uint4 fa[TWO ? 2 : 1][DG_DEPTH], fb[TWO ? 2 : 1][DG_DEPTH];
#pragma unroll
    for (int term = 0; term < (TWO ? 2 : 1); ++term) {
      const bf16* W = term ? job.W2 : job.W;
      const bf16* wa = W + (size_t)rowA * a.K + kbeg + 8 * t;
      const bf16* wb = W + (size_t)rowB * a.K + kbeg + 8 * t;
#pragma unroll
      for (int d = 0; d < DG_DEPTH; ++d) {
        const int c = c0 + DG_WARPS * d;
#ifdef IM_TRACE
        if (a.trace_skip & 1) { fa[term][d] = zero4; fb[term][d] = zero4; continue; }
#endif
        fa[term][d] = c < n_chunks ? ldg128_now(wa + c * 32) : zero4;
        fb[term][d] = c < n_chunks ? ldg128_now(wb + c * 32) : zero4;
      }
    }
    // (the vectors may be the output of the kernel this one was launched behind as a programmatic dependent)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    uint4 fx[DG_DEPTH][4];
#pragma unroll
    for (int d = 0; d < DG_DEPTH; ++d) {
      const int c = c0 + DG_WARPS * d;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
#ifdef IM_TRACE
        if (a.trace_skip & 2) { fx[d][nt] = zero4; continue; }
#endif
        fx[d][nt] = c < n_chunks ? ldg128_now(xb[nt] + c * 32) : zero4;
      }
    }
    asm volatile("" ::: "memory");  // every load of the batch is issued before the first MMA: one round trip
#pragma unroll
    for (int d = 0; d < DG_DEPTH; ++d) {
      const uint4* x = fx[d];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        mma_bf16(acc[nt], fa[0][d].x, fb[0][d].x, fa[0][d].y, fb[0][d].y, x[nt].x, x[nt].y);
        mma_bf16(acc[nt], fa[0][d].z, fb[0][d].z, fa[0][d].w, fb[0][d].w, x[nt].z, x[nt].w);
      }
      if (TWO) {
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          mma_bf16(acc[nt], fa[TWO ? 1 : 0][d].x, fb[TWO ? 1 : 0][d].x, fa[TWO ? 1 : 0][d].y, fb[TWO ? 1 : 0][d].y, x[nt].x, x[nt].y);
          mma_bf16(acc[nt], fa[TWO ? 1 : 0][d].z, fb[TWO ? 1 : 0][d].z, fa[TWO ? 1 : 0][d].w, fb[TWO ? 1 : 0][d].w, x[nt].z, x[nt].w);
        }
      }
    }
  }
  IM_MARK_GEMM(a, 1);
  // C fragment: rows g / g+8, columns 8 nt + 2t / + 1
  constexpr int ITEMS = 16 * VB / (DG_WARPS * 32);  // outputs per thread
  float sum[ITEMS];
#pragma unroll
  for (int k = 0; k < ITEMS; ++k) sum[k] = 0.f;
#pragma unroll
  for (int round = 0; round < 2; ++round) {
    if ((warp >> 2) == round) {
      const int w = warp & 3;
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        red[w][g][nt * 8 + 2 * t] = acc[nt][0];
        red[w][g][nt * 8 + 2 * t + 1] = acc[nt][1];
        red[w][g + 8][nt * 8 + 2 * t] = acc[nt][2];
        red[w][g + 8][nt * 8 + 2 * t + 1] = acc[nt][3];
      }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < ITEMS; ++k) {
      const int idx = threadIdx.x + k * DG_WARPS * 32;
      const int r = idx & 15, vl = idx >> 4;
#pragma unroll
      for (int w = 0; w < DG_WARPS / 2; ++w) sum[k] += red[w][r][vl];
    }
    __syncthreads();
  }
  IM_MARK_GEMM(a, 2);
  float* outk = a.out + (size_t)ks * a.ks_stride;
#pragma unroll
  for (int k = 0; k < ITEMS; ++k) {
    const int idx = threadIdx.x + k * DG_WARPS * 32;
    const int r = idx & 15, vl = idx >> 4;
    const long long v = v0 + vl;
    if (v < a.NV && r0 + r < job.rows)
      outk[(v / a.out_cnt) * a.out_outer + (v % a.out_cnt) * a.out_inner + job.row0 + r0 + r] = sum[k];
  }
  IM_MARK_GEMM(a, 3);
}

// ------------------------------------------------------------------------------------------------
// Indexer key projection U_k x in float64 (the cached key is a quantised code: the value that gets
// rounded to bf16 must not depend on the summation order).  K is split over blockIdx.x; one warp
// per vector.  keyp[ks][v][r] receives the partial sums.
// grid = (ksplit, ceil(NV / 8)), block = 256.
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__global__ void __launch_bounds__(256) k_proj_key_split(ImDims p, const bf16* __restrict__ Uk, const bf16* __restrict__ x,
                                                         int NV, int ksplit, double* __restrict__ keyp) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ks = blockIdx.x;
  const long long v = (long long)blockIdx.y * 8 + warp;
  if (v >= NV) return;
  const int kspan = p.D / ksplit, kbeg = ks * kspan;  // kspan is a multiple of 8
  const uint4* x4 = reinterpret_cast<const uint4*>(x + (size_t)v * p.D + kbeg);
  double* dst = keyp + ((size_t)ks * NV + v) * p.dI;
  for (int rb = 0; rb < p.dI; rb += 8) {  // 8 rows at a time: their loads are in flight together
    double acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.0;
    for (int c = lane; c < kspan / 8; c += 32) {
      const uint4 b = x4[c];
      uint4 a[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        a[j] = rb + j < p.dI ? reinterpret_cast<const uint4*>(Uk + (size_t)(rb + j) * p.D + kbeg)[c] : make_uint4(0, 0, 0, 0);
      const uint32_t bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t aw[4] = {a[j].x, a[j].y, a[j].z, a[j].w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          // a product of two bf16 values is exact in float32
          acc[j] += (double)(__uint_as_float(aw[k] << 16) * __uint_as_float(bw[k] << 16));
          acc[j] += (double)(__uint_as_float(aw[k] & 0xffff0000u) * __uint_as_float(bw[k] & 0xffff0000u));
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const double s = warp_sum_d(acc[j]);
      if (lane == 0 && rb + j < p.dI) dst[rb + j] = s;
    }
  }
}

// The same projection for the thousands of vectors of a prefill chunk, on the float64 tensor-core path
// (mma.sync m8n8k4 f64): a warp takes 8 vectors x all d_I rows over 1 / W of the K range, the W warps of a
// block add their 8 x 8 tiles through shared memory in warp order (W = 8 for prefill chunks: the kernel is bound by
// the latency of its load -> convert -> mma chains, and 256 blocks of 4 warps leave an SM 7 warps to hide it).  Lane (r, q) = (lane / 4, lane % 4) loads 8
// consecutive k of row r (vector r for A, weight row r of the n-tile for B) starting at 8 q inside a 32-wide
// chunk; k-step s multiplies element s of every lane's vector: the contraction index is permuted identically for
// both operands.  Every product and sum is formed in float64.
// grid = (ceil(NV / 8), ksplit), block = 32 W; D a multiple of 32 W ksplit, d_I = 8 NT.  Block (., ks) takes the ks-th
// part of the K range and writes the partial sums keyp[ks][v][.] (decode: the few vectors of a step would leave all
// but a handful of SMs idle, and the consumer adds the parts in split order).
template <int NT, int W>
__global__ void __launch_bounds__(32 * W) k_proj_key_mma(ImDims p, const bf16* __restrict__ Uk, const bf16* __restrict__ x,
                                                       int NV, int ksplit, double* __restrict__ keyp) {
  __shared__ double red[W * NT * 64];
  proj_key_mma_block<NT, W>(p.D, p.dI, Uk, x, NV, ksplit, keyp, blockIdx.x, blockIdx.y, red);
}

}  // namespace

cudaError_t im_launch_gemm(const ImLaunch& L, const ImGemmArgs& a_in) {
  static bool attr_done_dev[64] = {};
  bool* attr_done = im_device_flag(attr_done_dev);
  if (!attr_done || !*attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_skinny_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 64 * (KC_MAX * 2 + 16));
    if (e != cudaSuccess) return e;
    if (attr_done) *attr_done = true;
  }
  ImGemmArgs a = a_in;
  if (a.tensor && im_tc_gemm_usable(a)) return im_launch_tc_gemm(L, a);
  int n_w2 = 0;
  for (int j = 0; j < a.n_jobs; ++j) n_w2 += a.job[j].W2 != nullptr;
  if (a.direct && a.ksplit > 0 && a.K % a.ksplit == 0 && (a.K / a.ksplit) % 32 == 0 && a.NV > 0 &&
      (n_w2 == 0 || n_w2 == a.n_jobs)) {
    int tiles = 0;
    for (int j = 0; j < a.n_jobs; ++j) tiles += (a.job[j].rows + 15) / 16;
    a.tiles = tiles;
    int key_cols = 0;  // columns of blocks behind the tiles' for the key projection riding along
    if (a.key_W) {
      if ((a.key_dI != 8 && a.key_dI != 16) || a.key_ksplit < 1 || a.K % (32 * DG_WARPS * a.key_ksplit)) return cudaErrorInvalidValue;
      key_cols = (((a.key_nv + 7) / 8) * a.key_ksplit + a.ksplit - 1) / a.ksplit;
    }
    dim3 grid(tiles + key_cols, a.ksplit, (unsigned)((a.NV + VB - 1) / VB));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(DG_WARPS * 32);
    cfg.dynamicSmemBytes = (size_t)std::max(0, a.smem_floor);
    cfg.stream = L.stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = a.programmatic ? 1 : 0;
    const cudaError_t e = n_w2 ? cudaLaunchKernelEx(&cfg, k_direct_gemm<true>, a) : cudaLaunchKernelEx(&cfg, k_direct_gemm<false>, a);
    ++*L.launches;
    return e != cudaSuccess ? e : cudaGetLastError();
  }
  a.any_w2 = 0;
  for (int j = 0; j < a.n_jobs; ++j) a.any_w2 |= a.job[j].W2 != nullptr;
  if (a.kc <= 0 || a.kc > KC_MAX || a.kc % 16) a.kc = KC_MAX;
  const int smem = 2 * (a.any_w2 ? 64 : 48) * (a.kc * 2 + 16);
  int tiles = 0;
  for (int j = 0; j < a.n_jobs; ++j) tiles += (a.job[j].rows + 15) / 16;
  dim3 grid(tiles, a.ksplit, (unsigned)((a.NV + VB - 1) / VB));
  k_skinny_gemm<<<grid, 128, smem, L.stream>>>(a);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_proj_key_split(const ImLaunch& L, const void* x, int NV, int ksplit) {
  // float64 tensor-core path: prefill chunks whole, decode steps with the K range cut over `ksplit` blocks
  if ((ksplit > 1 || NV >= 64) && L.p.D % (128 * ksplit) == 0 && (L.p.dI == 8 || L.p.dI == 16)) {
    dim3 grid((NV + 7) / 8, ksplit);
    const bool wide = ksplit == 1 && L.p.D % 256 == 0;  // prefill chunks
    if (L.p.dI == 8) {
      if (wide) k_proj_key_mma<1, 8><<<grid, 256, 0, L.stream>>>(L.p, L.w.Uk, (const bf16*)x, NV, ksplit, L.sc.keyp);
      else k_proj_key_mma<1, 4><<<grid, 128, 0, L.stream>>>(L.p, L.w.Uk, (const bf16*)x, NV, ksplit, L.sc.keyp);
    } else {
      if (wide) k_proj_key_mma<2, 8><<<grid, 256, 0, L.stream>>>(L.p, L.w.Uk, (const bf16*)x, NV, ksplit, L.sc.keyp);
      else k_proj_key_mma<2, 4><<<grid, 128, 0, L.stream>>>(L.p, L.w.Uk, (const bf16*)x, NV, ksplit, L.sc.keyp);
    }
    ++*L.launches;
    return cudaGetLastError();
  }
  dim3 grid(ksplit, (NV + 7) / 8);
  k_proj_key_split<<<grid, 256, 0, L.stream>>>(L.p, L.w.Uk, (const bf16*)x, NV, ksplit, L.sc.keyp);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_gemm_prepare_decode() {
  cudaError_t e = im_prefer_max_smem(k_direct_gemm<false>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_direct_gemm<true>);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_direct_gemm<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_SMEM_HEAD);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_direct_gemm<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_SMEM_SIDE);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_skinny_gemm);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_proj_key_split);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_proj_key_mma<1, 4>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_proj_key_mma<2, 4>);
  return e;
}

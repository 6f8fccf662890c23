// Latent-memory write (a3, Eq. 6-7).
//
// State representation: the true fast-weight state is
//     M = cscale * ( Mhat + sum_p pend_w[p] * pend_phi[p] (x) pend_v[p] ),
// i.e. a scalar decay factor, the materialised matrix and a short list (at most F entries) of
// rank-one terms that have not been folded in yet.  An evict step with few evicted pairs only
// appends to the list (O(d_M + D_kv) bytes instead of a read-modify-write of the whole matrix) and
// the readout adds the listed terms exactly.  When the list cannot take the evicted set of the
// coming compression, it is folded into Mhat first (cscale returns to 1); an evicted set larger
// than F is accumulated into Mhat directly.  b is small and is updated in place.  All of this is
// Eq. 6-7 re-associated.
//
// Kernel order inside one call: k_mem_fold, k_mem_fold_commit (both before the counters of the
// call change), ..., selection, gather, phi of the evicted keys (skinny GEMM), k_mem_small,
// k_mem_accumulate (large sets only).
#include "im_internal.cuh"

namespace {

// does the coming compression of this sequence need the pending list folded first?
__device__ __forceinline__ bool fold_needed(const ImDims& p, const ImCall& call, const int32_t* ctr, float cscale) {
  if (!p.mem) return false;
  if (call.fold_all) return ctr[CTR_NPEND] > 0 || cscale != 1.0f;
  // (the phase of the interval comes from the host, not from the counter the decode front kernel advances, so
  // that the fold kernels and the front kernel do not depend on one another)
  const int ne = im_upcoming_evictions(p, call.prefill || call.due, call.C, ctr[CTR_N]);
  const int np = ctr[CTR_NPEND];
  if (ne <= 0) return false;
  if (ne > p.F) return np > 0 || cscale != 1.0f;  // a large set is accumulated into Mhat with cscale == 1
  return np + ne > p.F;
}

// Mhat <- cscale * (Mhat + sum_p w_p phi_p v_p^T).  grid = (stripes of 64 rows, n_seq), block = 256.  A block owns a
// stripe of 64 rows of one sequence's Mhat.  Per FOLD_ENT listed entries it stages w_p phi_p of its rows and v_p of up to
// FOLD_COLS columns in shared memory ONCE, then walks the stripe in 64 x 64 tiles, each thread a 4 x 4 micro tile whose rows it
// reads and writes as 16-byte words, the next tile's rows requested before the current tile is updated: between the
// staging and the end of the stripe the kernel only streams Mhat.  (Its first form staged per tile, with two block
// barriers and a round trip of small loads each, and read Mhat in 4-byte words: next to the streaming kernels of a
// decode step, where every request queues behind theirs, the 32 layers' folds of a step took 1.7 ms; this form 1.2 ms.)
// Blocks of sequences that need no fold leave at once (the kernel is part of every decode step so that a captured
// launch sequence stays valid).
constexpr int FOLD_COLS = 512;  // columns of v_p staged at a time
constexpr int FOLD_ENT = 32;    // listed entries folded per pass over a stripe (a list of up to FOLD_ENT entries: one pass)
__global__ void __launch_bounds__(256) k_mem_fold(ImDims p, ImState st, ImCall call) {
  __shared__ float s_a[FOLD_ENT][64 + 4];        // [entry][m]   w_p * phi_p
  __shared__ bf16 s_v[FOLD_ENT][FOLD_COLS + 8];  // [entry][col] v_p
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const float c = st.cscale[u];
  if (!fold_needed(p, call, ctr, c)) return;
  const int np = min(ctr[CTR_NPEND], p.F);
  const int stripes = (p.dM + 63) / 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float* Mh = st.Mhat + u * p.dM * p.Dkv;
  const bool wide = (p.Dkv & 7) == 0 && (p.dM & 3) == 0;  // 16-byte words throughout
  // rows a thread owns in a stripe: ty, ty + 16, ty + 32, ty + 48 (a warp's loads then cover two whole 256-byte row pieces)
  auto load_tile = [&](float (&acc)[4][4], int m0, int col0) {
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int m = m0 + a * 16 + ty;
      if (wide && col0 + tx * 4 + 3 < p.Dkv) {
        float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
        if (m < p.dM) w = *reinterpret_cast<const float4*>(Mh + (size_t)m * p.Dkv + col0 + tx * 4);
        acc[a][0] = w.x; acc[a][1] = w.y; acc[a][2] = w.z; acc[a][3] = w.w;
      } else {
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int col = col0 + tx * 4 + b;
          acc[a][b] = (m < p.dM && col < p.Dkv) ? Mh[(size_t)m * p.Dkv + col] : 0.f;
        }
      }
    }
  };
  for (int stripe = blockIdx.x; stripe < stripes; stripe += gridDim.x) {
    const int m0 = stripe * 64;
    for (int cb = 0; cb < p.Dkv; cb += FOLD_COLS) {
      const int ncol = min(FOLD_COLS, p.Dkv - cb);
      for (int k0 = 0; k0 < np || k0 == 0; k0 += FOLD_ENT) {
        const int lim = max(0, min(FOLD_ENT, np - k0));
        const bool last = k0 + FOLD_ENT >= np;  // (the scale is applied with the last entries)
        __syncthreads();
        for (int k = threadIdx.x; k < lim * 64; k += blockDim.x) {
          const int e = k / 64, j = k % 64;
          s_a[e][j] = m0 + j < p.dM ? st.pend_w[u * p.F + k0 + e] * st.pend_phi[(u * p.F + k0 + e) * p.dM + m0 + j] : 0.f;
        }
        if (wide) {
          for (int k = threadIdx.x; k < lim * (ncol / 8); k += blockDim.x) {
            const int e = k / (ncol / 8), j = (k % (ncol / 8)) * 8;
            *reinterpret_cast<uint4*>(&s_v[e][j]) = *reinterpret_cast<const uint4*>(st.pend_v + (u * p.F + k0 + e) * p.Dkv + cb + j);
          }
        } else {
          for (int k = threadIdx.x; k < lim * ncol; k += blockDim.x) {
            const int e = k / ncol, j = k % ncol;
            s_v[e][j] = st.pend_v[(u * p.F + k0 + e) * p.Dkv + cb + j];
          }
        }
        __syncthreads();
        float cur[4][4], nxt[4][4];
        load_tile(cur, m0, cb);
        for (int c0 = 0; c0 < ncol; c0 += 64) {
          if (c0 + 64 < ncol) load_tile(nxt, m0, cb + c0 + 64);
          for (int e = 0; e < lim; ++e) {
            float bv[4];
#pragma unroll
            for (int b = 0; b < 4; ++b) bv[b] = c0 + tx * 4 + b < ncol ? __bfloat162float(s_v[e][c0 + tx * 4 + b]) : 0.f;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
              const float av = s_a[e][a * 16 + ty];
#pragma unroll
              for (int b = 0; b < 4; ++b) cur[a][b] = fmaf(av, bv[b], cur[a][b]);
            }
          }
          const float sc_ = last ? c : 1.0f;
#pragma unroll
          for (int a = 0; a < 4; ++a) {
            const int m = m0 + a * 16 + ty, col = cb + c0 + tx * 4;
            if (m >= p.dM) continue;
            if (wide && col + 3 < p.Dkv) {
              *reinterpret_cast<float4*>(Mh + (size_t)m * p.Dkv + col) =
                  make_float4(sc_ * cur[a][0], sc_ * cur[a][1], sc_ * cur[a][2], sc_ * cur[a][3]);
            } else {
#pragma unroll
              for (int b = 0; b < 4; ++b)
                if (col + b < p.Dkv) Mh[(size_t)m * p.Dkv + col + b] = sc_ * cur[a][b];
            }
          }
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) cur[a][b] = nxt[a][b];
        }
      }
    }
  }
}

// The same fold with the rank-one terms added by the tensor cores, for shapes whose d_M and D_kv are multiples of 64.
// Per element the fold is one multiply-add per listed entry: 17 GFLOP for the 32 layers x 32 sequences of the decode
// benchmark at 16 entries, which the FFMA form above spends on the few SMs the streaming kernels leave it (a quarter
// of a fold step's extra time, and all of what a longer list adds).  Here a warp owns 16 rows x FOLDT_W columns of the
// block's 64 x 2 FOLDT_W tile as FOLDT_NJ m16n8 accumulators that it loads from and stores to Mhat directly in the accumulator
// layout (8-byte words: a warp's access covers whole 32-byte sectors), A = w_p phi_p of its rows as THREE bf16 terms
// (hi + mid + lo reproduce the float32 value to 2^-24), B = v_p, which is bf16 as stored, through ldmatrix.trans from
// the staged [entry][column] rows: the products are exact and the sums are float32, so the result differs from the
// FFMA form by rounding order only.  Entries are staged FOLDT_ENT at a time (a list of up to 32: one pass over Mhat).
constexpr int FOLDT_COLS = 512;
constexpr int FOLDT_ENT = 32;
#ifndef FOLDT_NJ
#define FOLDT_NJ 4        /* m16n8 accumulators per warp and step */
#define FOLDT_BLOCKS 3    /* blocks per SM the register budget allows */
#endif
constexpr int FOLDT_W = FOLDT_NJ * 8;  // columns of a warp's step
__device__ __forceinline__ void fold_ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void fold_mma(float2& c01, float2& c23, const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c01.x), "+f"(c01.y), "+f"(c23.x), "+f"(c23.y)
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// x0, x1 -> three packed bf16 pairs (x0 in the low half) whose sum is x to 2^-24
__device__ __forceinline__ void fold_split3(float x0, float x1, uint32_t& hi, uint32_t& mid, uint32_t& lo) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
  const float r0 = x0 - __bfloat162float(h0), r1 = x1 - __bfloat162float(h1);
  const __nv_bfloat16 m0 = __float2bfloat16_rn(r0), m1 = __float2bfloat16_rn(r1);
  const float q0 = r0 - __bfloat162float(m0), q1 = r1 - __bfloat162float(m1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(q0), l1 = __float2bfloat16_rn(q1);
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  mid = (uint32_t)__bfloat16_as_ushort(m0) | ((uint32_t)__bfloat16_as_ushort(m1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}
__global__ void __launch_bounds__(256, FOLDT_BLOCKS) k_mem_fold_tc(ImDims p, ImState st, ImCall call) {
  __shared__ __align__(16) float s_a[FOLDT_ENT][64 + 4];        // [entry][m]   w_p * phi_p
  __shared__ __align__(16) bf16 s_v[FOLDT_ENT][FOLDT_COLS + 8];  // [entry][col] v_p
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const float c = st.cscale[u];
  if (!fold_needed(p, call, ctr, c)) return;
  const int np = min(ctr[CTR_NPEND], p.F);
  const int stripes = p.dM / 64;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wr = warp & 3, wc = warp >> 2;  // the warp's 16-row slab of the stripe; which FOLDT_W columns of a 2 FOLDT_W-column step
  float* Mh = st.Mhat + u * p.dM * p.Dkv;
  for (int stripe = blockIdx.x; stripe < stripes; stripe += gridDim.x) {
    const int m0 = stripe * 64;
    float* rowp = Mh + (size_t)(m0 + wr * 16 + g) * p.Dkv + 2 * t;  // the thread's upper row; the lower one is 8 rows on
    for (int cb = 0; cb < p.Dkv; cb += FOLDT_COLS) {
      const int ncol = min(FOLDT_COLS, p.Dkv - cb);
      const int ngroups = ncol / FOLDT_W;
      for (int k0 = 0; k0 < np || k0 == 0; k0 += FOLDT_ENT) {
        const int lim = max(0, min(FOLDT_ENT, np - k0));
        const int limr = (lim + 15) & ~15;            // entries staged: whole k-steps, zeros past the list's end
        const bool last = k0 + FOLDT_ENT >= np;       // (the scale is applied with the last entries)
        __syncthreads();
        for (int k = threadIdx.x; k < limr * 64; k += blockDim.x) {
          const int e = k / 64, j = k % 64;
          s_a[e][j] = e < lim ? st.pend_w[u * p.F + k0 + e] * st.pend_phi[(u * p.F + k0 + e) * p.dM + m0 + j] : 0.f;
        }
        for (int k = threadIdx.x; k < limr * (ncol / 8); k += blockDim.x) {
          const int e = k / (ncol / 8), j = (k % (ncol / 8)) * 8;
          *reinterpret_cast<uint4*>(&s_v[e][j]) =
              e < lim ? *reinterpret_cast<const uint4*>(st.pend_v + (u * p.F + k0 + e) * p.Dkv + cb + j) : make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        // A of the warp's rows: [k-step][term][register]
        uint32_t af[FOLDT_ENT / 16][3][4];
#pragma unroll
        for (int ks = 0; ks < FOLDT_ENT / 16; ++ks)
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            af[ks][0][r] = af[ks][1][r] = af[ks][2][r] = 0u;
            if (ks * 16 < limr) {
              const int row = wr * 16 + g + (r & 1) * 8, kk = ks * 16 + 2 * t + (r >> 1) * 8;
              fold_split3(s_a[kk][row], s_a[kk + 1][row], af[ks][0][r], af[ks][1][r], af[ks][2][r]);
            }
          }
        // ldmatrix row address of this lane: entry (lane & 7) + 8 * ((lane >> 3) & 1) of a k-step, 8 columns on for lanes 16-31
        const uint32_t sv_lane = (uint32_t)__cvta_generic_to_shared(&s_v[(lane & 7) + ((lane >> 3) & 1) * 8][(lane >> 4) * 8]);
        float2 cur[2 * FOLDT_NJ], nxt[2 * FOLDT_NJ];
        auto load_group = [&](float2 (&a)[2 * FOLDT_NJ], int grp) {
          const float* q = rowp + cb + grp * FOLDT_W;
#pragma unroll
          for (int j = 0; j < FOLDT_NJ; ++j) {
            a[2 * j] = *reinterpret_cast<const float2*>(q + j * 8);
            a[2 * j + 1] = *reinterpret_cast<const float2*>(q + (size_t)8 * p.Dkv + j * 8);
          }
        };
        int grp = wc;
        if (grp < ngroups) load_group(cur, grp);
        for (; grp < ngroups; grp += 2) {
          if (grp + 2 < ngroups) load_group(nxt, grp + 2);
#pragma unroll
          for (int ks = 0; ks < FOLDT_ENT / 16; ++ks) {
            if (ks * 16 < limr) {
#pragma unroll
              for (int jp = 0; jp < FOLDT_NJ / 2; ++jp) {
                uint32_t b0, b1, b2, b3;
                fold_ldsm_x4_t(sv_lane + (uint32_t)((ks * 16 * (FOLDT_COLS + 8) + grp * FOLDT_W + jp * 16) * 2), b0, b1, b2, b3);
#pragma unroll
                for (int term = 2; term >= 0; --term) {
                  fold_mma(cur[4 * jp], cur[4 * jp + 1], af[ks][term], b0, b1);
                  fold_mma(cur[4 * jp + 2], cur[4 * jp + 3], af[ks][term], b2, b3);
                }
              }
            }
          }
          const float sc_ = last ? c : 1.0f;
          float* q = rowp + cb + grp * FOLDT_W;
#pragma unroll
          for (int j = 0; j < FOLDT_NJ; ++j) {
            *reinterpret_cast<float2*>(q + j * 8) = make_float2(sc_ * cur[2 * j].x, sc_ * cur[2 * j].y);
            *reinterpret_cast<float2*>(q + (size_t)8 * p.Dkv + j * 8) = make_float2(sc_ * cur[2 * j + 1].x, sc_ * cur[2 * j + 1].y);
          }
#pragma unroll
          for (int j = 0; j < 2 * FOLDT_NJ; ++j) cur[j] = nxt[j];
        }
      }
    }
  }
}

// after every block of k_mem_fold has read cscale / the list: cscale <- 1, list emptied.
// grid = n_seq, block = 32.
__global__ void k_mem_fold_commit(ImDims p, ImState st, ImCall call) {
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  if (threadIdx.x == 0 && fold_needed(p, call, ctr, st.cscale[u])) {
    st.cscale[u] = 1.0f;
    ctr[CTR_NPEND] = 0;
  }
}

// phi of evicted entry e of call sequence i (see ImCall::phi_large)
__device__ __forceinline__ float phi_at(const ImDims& p, const ImScratch& sc, const ImCall& call, int i, int e, int m) {
  if (call.phi_large) return sc.phi[((size_t)i * p.tail + e) * p.dM + m];
  float s = 0.f;
  for (int ks = 0; ks < call.ksplit_phi; ++ks) s += sc.phip[(((size_t)ks * call.n_seq + i) * p.F + e) * p.dM + m];
  return s;
}

// b <- lambda b + eta sum_e phi_e^2 (Eq. 7), decay scale, and for sets of at most F entries the
// append to the pending list.  grid = n_seq, block = 256.
__global__ void __launch_bounds__(256) k_mem_small(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int i = blockIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int ne = min(ctr[CTR_NEVICT], p.tail);
  if (ne <= 0) return;
  const int np = min(ctr[CTR_NPEND], p.F);
  if (ne > p.F) return;  // large sets: b and Mhat are updated by k_mem_accumulate; cscale stays 1
  const float c_new = p.lambda * st.cscale[u];
  for (int m = threadIdx.x; m < p.dM; m += blockDim.x) {
    float s = 0.f;
    for (int e = 0; e < ne; ++e) {
      const float f = phi_at(p, sc, call, i, e, m);
      s = fmaf(f, f, s);
      if (np + e < p.F) st.pend_phi[(u * p.F + np + e) * p.dM + m] = f;
    }
    st.bvec[u * p.dM + m] = p.lambda * st.bvec[u * p.dM + m] + p.eta * s;
  }
  if (np + ne > p.F) {
    if (threadIdx.x == 0) atomicOr(st.status, ST_COUNT);  // the fold kernel should have made room
    return;
  }
  const int dv = p.Dkv / 8;
  for (int k = threadIdx.x; k < ne * dv; k += blockDim.x) {
    const int e = k / dv, c = k % dv;
    reinterpret_cast<uint4*>(st.pend_v + (u * p.F + np + e) * p.Dkv)[c] =
        reinterpret_cast<const uint4*>(sc.evV + ((size_t)i * p.tail + e) * p.Dkv)[c];
  }
  for (int e = threadIdx.x; e < ne; e += blockDim.x) st.pend_w[u * p.F + np + e] = p.eta / c_new;
  __syncthreads();
  if (threadIdx.x == 0) {
    st.cscale[u] = c_new;
    ctr[CTR_NPEND] = np + ne;
  }
}

// Evicted sets larger than F: Mhat <- lambda * Mhat + eta * sum_e phi_e v_e^T (the list is empty and
// cscale is 1 after the fold), and b <- lambda b + eta sum_e phi_e^2 by the blocks of the first tile column
// (they stage every phi row of their 64 memory rows anyway).  grid = (ceil(Dkv/64), ceil(dM/64), n_seq), block = 256.
__global__ void __launch_bounds__(256) k_mem_accumulate(ImDims p, ImState st, ImScratch sc, ImCall call) {
  __shared__ float s_a[16][64 + 4];
  __shared__ float s_b[16][64 + 4];
  const int i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(st.ctr[u * CTR_STRIDE + CTR_NEVICT], p.tail);
  if (ne <= p.F) return;
  const int m0 = blockIdx.y * 64, col0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  float bsum = 0.f;
  const float* phi = sc.phi + (size_t)i * p.tail * p.dM;
  const bf16* V = sc.evV + (size_t)i * p.tail * p.Dkv;
  for (int k0 = 0; k0 < ne; k0 += 16) {
    __syncthreads();
    for (int k = threadIdx.x; k < 16 * 64; k += blockDim.x) {
      const int e = k / 64, j = k % 64;
      float av = 0.f, bv = 0.f;
      if (k0 + e < ne) {
        if (m0 + j < p.dM) av = phi[(size_t)(k0 + e) * p.dM + m0 + j];
        if (col0 + j < p.Dkv) bv = __bfloat162float(V[(size_t)(k0 + e) * p.Dkv + col0 + j]);
      }
      s_a[e][j] = av;
      s_b[e][j] = bv;
    }
    __syncthreads();
    const int lim = min(16, ne - k0);
    if (blockIdx.x == 0 && threadIdx.x < 64)
      for (int e = 0; e < lim; ++e) bsum = fmaf(s_a[e][threadIdx.x], s_a[e][threadIdx.x], bsum);
    for (int e = 0; e < lim; ++e) {
      float av[4], bv[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) av[a] = s_a[e][ty * 4 + a];
#pragma unroll
      for (int b = 0; b < 4; ++b) bv[b] = s_b[e][tx * 4 + b];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(av[a], bv[b], acc[a][b]);
    }
  }
  if (blockIdx.x == 0 && threadIdx.x < 64 && m0 + threadIdx.x < p.dM) {
    float* bp = st.bvec + u * p.dM + m0 + threadIdx.x;
    *bp = p.lambda * *bp + p.eta * bsum;
  }
  float* Mh = st.Mhat + u * p.dM * p.Dkv;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int m = m0 + ty * 4 + a, col = col0 + tx * 4 + b;
      if (m < p.dM && col < p.Dkv) Mh[(size_t)m * p.Dkv + col] = p.lambda * Mh[(size_t)m * p.Dkv + col] + p.eta * acc[a][b];
    }
}

// ---- large evicted sets on the tensor cores: Mhat <- lambda Mhat + eta Phi^T V as a GEMM over the evicted
// entries.  The GEMM kernels want both operands K-major (K = evicted entry), so phi (float32, [e][m]) and the
// evicted values ([e][col]) of one sequence are transposed first; phi becomes two bf16 terms (hi + lo
// reproduces the float32 value to 2^-17).  Entries at or beyond the sequence's evicted count are zero.
// grid = (KE / 32, (dM + Dkv) / 32, sequences), block = (32, 8); sequence i0 + blockIdx.z goes to block blockIdx.z
// of phiT / vT.
__global__ void __launch_bounds__(256) k_mem_pack(ImDims p, ImState st, ImScratch sc, ImCall call, int i0, int KE) {
  __shared__ float tile[32][33];
  const int i = i0 + blockIdx.z;
  bf16* phiT = sc.phiT + (size_t)blockIdx.z * 2 * p.dM * KE;
  bf16* vT = sc.vT + (size_t)blockIdx.z * p.Dkv * KE;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(st.ctr[u * CTR_STRIDE + CTR_NEVICT], p.tail);
  const int e0 = blockIdx.x * 32, tx = threadIdx.x, ty = threadIdx.y;
  const int mt = (p.dM + 31) / 32;
  const bool is_phi = (int)blockIdx.y < mt;
  const int c0 = (is_phi ? blockIdx.y : blockIdx.y - mt) * 32;
  const int width = is_phi ? p.dM : p.Dkv;
  for (int r = ty; r < 32; r += 8) {  // rows = entries, threads along the contiguous column index
    const int e = e0 + r, c = c0 + tx;
    float v = 0.f;
    if (e < ne && c < width)
      v = is_phi ? sc.phi[((size_t)i * p.tail + e) * p.dM + c] : __bfloat162float(sc.evV[((size_t)i * p.tail + e) * p.Dkv + c]);
    tile[r][tx] = v;
  }
  __syncthreads();
  if (is_phi && ty == 0 && c0 + tx < width) {
    // sum of phi^2 over this block's 32 entries for column c0 + tx (Eq. 7), in a fixed order; k_mem_bsum adds the
    // blocks' sums
    float s2 = 0.f;
#pragma unroll 8
    for (int r = 0; r < 32; ++r) s2 = fmaf(tile[r][tx], tile[r][tx], s2);
    sc.bpart[((size_t)blockIdx.z * (KE / 32) + blockIdx.x) * p.dM + c0 + tx] = s2;
  }
  for (int r = ty; r < 32; r += 8) {  // rows = columns of the source, threads along the entries
    const int c = c0 + r, e = e0 + tx;
    if (c >= width || e >= KE) continue;
    const float v = tile[tx][r];
    const bf16 hi = __float2bfloat16_rn(v);
    if (is_phi) {
      phiT[(size_t)c * KE + e] = hi;
      phiT[((size_t)p.dM + c) * KE + e] = __float2bfloat16_rn(v - __bfloat162float(hi));
    } else {
      vT[(size_t)c * KE + e] = hi;
    }
  }
}

// b <- lambda b + eta sum_e phi_e^2 (Eq. 7) for the sequences whose evicted set is larger than the pending list,
// from the sums over 32 entries that k_mem_pack left (block `slot` of the packed operands holds sequence i0 + slot).
// grid = (ceil(dM / 32), sequences), block = (32, 8): eight partial sums per row, added in a fixed order.
__global__ void __launch_bounds__(256) k_mem_bsum(ImDims p, ImState st, ImScratch sc, ImCall call, int i0, int KE) {
  __shared__ float part[8][32];
  const int i = i0 + blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(st.ctr[u * CTR_STRIDE + CTR_NEVICT], p.tail);
  if (ne <= p.F) return;
  const int m = blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (m < p.dM)
    for (int j = threadIdx.y; j < KE / 32; j += 8) s += sc.bpart[((size_t)blockIdx.y * (KE / 32) + j) * p.dM + m];
  part[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && m < p.dM) {
    for (int k = 1; k < 8; ++k) s += part[k][threadIdx.x];
    st.bvec[u * p.dM + m] = p.lambda * st.bvec[u * p.dM + m] + p.eta * s;
  }
}

}  // namespace

cudaError_t im_launch_mem_fold(const ImLaunch& L, const ImCall& call) {
  const ImDims& p = L.p;
  dim3 grid((p.dM + 63) / 64, call.n_seq);
  if (!call.fold_ffma && p.dM % 64 == 0 && p.Dkv % 64 == 0) k_mem_fold_tc<<<grid, 256, 0, L.stream>>>(p, L.st, call);
  else k_mem_fold<<<grid, 256, 0, L.stream>>>(p, L.st, call);
  ++*L.launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  k_mem_fold_commit<<<call.n_seq, 32, 0, L.stream>>>(p, L.st, call);
  ++*L.launches;
  return cudaGetLastError();
}

// after phi of the evicted keys is available (ImCall::phi_large says where)
cudaError_t im_launch_mem_update(const ImLaunch& L, const ImCall& call, int ne_max, const int* ne_host) {
  const ImDims& p = L.p;
  k_mem_small<<<call.n_seq, 256, 0, L.stream>>>(p, L.st, L.sc, call);
  ++*L.launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || ne_max <= p.F) return e;
  // evicted sets larger than the pending list: Phi^T V on the tensor cores, one sequence at a time
  const int KE = (ne_max + 63) / 64 * 64;
  ImGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.tensor = 1;
  g.NV = p.Dkv;  // the GEMM's "vectors" are the columns of Mhat (rows of V^T), its "weight rows" the rows of Phi^T
  g.K = KE;
  g.ksplit = 1;
  g.in[0] = L.sc.vT;
  g.in_cnt[0] = 1;
  g.in_outer[0] = KE;
  g.job[0] = {L.sc.phiT, L.sc.phiT ? L.sc.phiT + (size_t)p.dM * KE : nullptr, p.dM, 0, 0};
  g.n_jobs = 1;
  g.out_t = 1;
  g.out_outer = p.Dkv;
  g.out_cnt = 1;
  g.rmw = 1;
  g.alpha = p.eta;
  g.beta = p.lambda;
  g.gate_min = p.F;
  if (L.sc.phiT && call.phi_large && ne_host && im_tc_gemm_usable(g)) {
    // all sequences of the call in one batched launch when their packed operands fit the scratch arrays
    if (call.n_seq > 1 && (long long)call.n_seq * KE <= L.sc.pack_k) {
      dim3 gp(KE / 32, (p.dM + 31) / 32 + (p.Dkv + 31) / 32, call.n_seq);
      k_mem_pack<<<gp, dim3(32, 8), 0, L.stream>>>(p, L.st, L.sc, call, 0, KE);
      ++*L.launches;
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      dim3 gb((p.dM + 31) / 32, call.n_seq);
      k_mem_bsum<<<gb, dim3(32, 8), 0, L.stream>>>(p, L.st, L.sc, call, 0, KE);
      ++*L.launches;
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      ImGemmBatch bt;
      memset(&bt, 0, sizeof(bt));
      bt.n = call.n_seq;
      bt.unit0 = call.layer * p.S;
      for (int i = 0; i < call.n_seq; ++i) bt.seq[i] = call.seq[i];
      bt.zA_rows = p.Dkv;
      bt.zB_rows = 2 * (long long)p.dM;
      bt.z_out = (long long)p.dM * p.Dkv;
      bt.z_gate = CTR_STRIDE;
      g.batch = &bt;
      g.out = L.st.Mhat;
      g.gate = L.st.ctr + CTR_NEVICT;
      return im_launch_tc_gemm(L, g);
    }
    for (int i = 0; i < call.n_seq; ++i) {
      if (ne_host[i] <= p.F) continue;
      const size_t u = (size_t)call.layer * p.S + call.seq[i];
      dim3 gp(KE / 32, (p.dM + 31) / 32 + (p.Dkv + 31) / 32);
      k_mem_pack<<<gp, dim3(32, 8), 0, L.stream>>>(p, L.st, L.sc, call, i, KE);
      ++*L.launches;
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      k_mem_bsum<<<dim3((p.dM + 31) / 32, 1), dim3(32, 8), 0, L.stream>>>(p, L.st, L.sc, call, i, KE);
      ++*L.launches;
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      g.out = L.st.Mhat + u * p.dM * p.Dkv;
      g.gate = L.st.ctr + u * CTR_STRIDE + CTR_NEVICT;
      if ((e = im_launch_tc_gemm(L, g)) != cudaSuccess) return e;
    }
    return cudaSuccess;
  }
  dim3 grid((p.Dkv + 63) / 64, (p.dM + 63) / 64, call.n_seq);
  k_mem_accumulate<<<grid, 256, 0, L.stream>>>(p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_memory_prepare_decode() {
  cudaError_t e = im_prefer_max_smem(k_mem_fold);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_mem_fold_tc);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_mem_fold_commit);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_mem_small);
  return e;
}

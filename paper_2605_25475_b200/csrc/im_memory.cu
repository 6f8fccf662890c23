// Latent-memory write (a3, Eq. 6-7) and cache compaction (a4).
//
// State representation: the true fast-weight state is
//     M = cscale * ( Mhat + sum_p pend_w[p] * pend_phi[p] (x) pend_v[p] ),
// i.e. a scalar decay factor, the materialised matrix and a short list of rank-one terms that have
// not been folded in yet.  An evict step with few evicted pairs only appends to the list (O(d_M)
// bytes instead of a read-modify-write of the whole matrix); when the list cannot take the evicted
// set, everything is folded into Mhat in one pass and cscale returns to 1.  b is small and is
// updated in place.  All of this is Eq. 6-7 re-associated.
#include "im_internal.cuh"

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// phi_e = Wfold . k_e for the evicted entries (phi(k) of Eq. 6 on the model-space key, folded to KV
// space).  grid = (ceil(ne_max / 8), n_seq), block = 256: 8 entries staged, warps stride over rows.
constexpr int PHI_E = 8;
__global__ void k_phi_evicted(ImDims p, ImState st, ImWeights w, ImScratch sc, ImCall call) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  bf16* s_k = reinterpret_cast<bf16*>(smem_raw);  // [PHI_E][Dkv]
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int ne = min(ctr[CTR_NEVICT], p.tail);
  const int e0 = blockIdx.x * PHI_E;
  if (e0 >= ne) return;
  const int cnt = min(PHI_E, ne - e0);
  const int dv = p.d / 8;
  for (int k = threadIdx.x; k < PHI_E * p.Hkv * dv; k += blockDim.x) {
    const int e = k / (p.Hkv * dv), rem = k % (p.Hkv * dv), h = rem / dv, c = rem % dv;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (e < cnt) {
      const int slot = st.ev_slot[u * p.tail + e0 + e];
      val = reinterpret_cast<const uint4*>(st.Kc + ((u * p.Hkv + h) * p.cap + slot) * p.d)[c];
    }
    reinterpret_cast<uint4*>(s_k + (size_t)e * p.Dkv + h * p.d)[c] = val;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int m = warp; m < p.dM; m += nw) {
    const float* wr = w.Wfold + (size_t)m * p.Dkv;
    float acc[PHI_E];
#pragma unroll
    for (int e = 0; e < PHI_E; ++e) acc[e] = 0.f;
    for (int c = lane; c < p.Dkv; c += 32) {
      const float wv = wr[c];
#pragma unroll
      for (int e = 0; e < PHI_E; ++e) acc[e] = fmaf(wv, __bfloat162float(s_k[(size_t)e * p.Dkv + c]), acc[e]);
    }
#pragma unroll
    for (int e = 0; e < PHI_E; ++e) {
      const float s = warp_sum(acc[e]);
      if (lane == 0 && e < cnt) sc.phi[((size_t)i * p.tail + e0 + e) * p.dM + m] = s;
    }
  }
}

// Full fold: Mhat <- lambda*c*(Mhat + sum_p w_p phi_p v_p^T) + eta * sum_e phi_e v_e^T for the
// sequences whose evict step was flagged direct.  Tiled like a small SGEMM:
// grid = (ceil(Dkv/64), ceil(dM/64), n_seq), block = 256, each thread a 4x4 micro tile.
__global__ void k_mem_direct(ImDims p, ImState st, ImScratch sc, ImCall call) {
  __shared__ float s_a[16][64 + 4];  // [entry][m]
  __shared__ float s_b[16][64 + 4];  // [entry][col]
  const int i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  if (!ctr[CTR_DIRECT]) return;
  const int ne = min(ctr[CTR_NEVICT], p.tail);
  const int np = min(ctr[CTR_NPEND], p.F);
  const float c_new = p.lambda * st.cscale[u];
  const int m0 = blockIdx.y * 64, col0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // micro tile: rows m0+ty*4.., cols col0+tx*4..
  float acc[4][4];
  float* Mh = st.Mhat + u * p.dM * p.Dkv;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int m = m0 + ty * 4 + a, col = col0 + tx * 4 + b;
      acc[a][b] = (m < p.dM && col < p.Dkv) ? Mh[(size_t)m * p.Dkv + col] : 0.f;
    }
  // phase 0: pending rank-one terms (coefficient pend_w), then scale by c_new;
  // phase 1: the evicted set of this step (coefficient eta)
  for (int phase = 0; phase < 2; ++phase) {
    const int cnt = phase == 0 ? np : ne;
    for (int k0 = 0; k0 < cnt; k0 += 16) {
      __syncthreads();
      for (int k = threadIdx.x; k < 16 * 64; k += blockDim.x) {
        const int e = k / 64, j = k % 64;
        float av = 0.f, bv = 0.f;
        if (k0 + e < cnt) {
          const int m = m0 + j, col = col0 + j;
          if (phase == 0) {
            if (m < p.dM) av = st.pend_w[u * p.F + k0 + e] * st.pend_phi[(u * p.F + k0 + e) * p.dM + m];
            if (col < p.Dkv) bv = __bfloat162float(st.pend_v[(u * p.F + k0 + e) * p.Dkv + col]);
          } else {
            if (m < p.dM) av = p.eta * sc.phi[((size_t)i * p.tail + k0 + e) * p.dM + m];
            if (col < p.Dkv) {
              const int slot = st.ev_slot[u * p.tail + k0 + e];
              const int h = col / p.d, c = col % p.d;
              bv = __bfloat162float(st.Vc[((u * p.Hkv + h) * p.cap + slot) * p.d + c]);
            }
          }
        }
        s_a[e][j] = av;
        s_b[e][j] = bv;
      }
      __syncthreads();
      const int lim = min(16, cnt - k0);
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
    if (phase == 0) {
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] *= c_new;
    }
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int m = m0 + ty * 4 + a, col = col0 + tx * 4 + b;
      if (m < p.dM && col < p.Dkv) Mh[(size_t)m * p.Dkv + col] = acc[a][b];
    }
}

// b <- lambda b + eta sum_e phi_e^2 (Eq. 7); for non-direct steps append the evicted pairs to the
// pending list and advance the decay scale.  grid = n_seq, block = 256.
__global__ void k_mem_small(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int i = blockIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int ne = min(ctr[CTR_NEVICT], p.tail);
  if (ne <= 0) return;
  const int np = min(ctr[CTR_NPEND], p.F);
  const bool direct = ctr[CTR_DIRECT] != 0;
  const float c_new = p.lambda * st.cscale[u];
  const float* phi = sc.phi + (size_t)i * p.tail * p.dM;
  for (int m = threadIdx.x; m < p.dM; m += blockDim.x) {
    float s = 0.f;
    for (int e = 0; e < ne; ++e) {
      const float f = phi[(size_t)e * p.dM + m];
      s = fmaf(f, f, s);
    }
    st.bvec[u * p.dM + m] = p.lambda * st.bvec[u * p.dM + m] + p.eta * s;
  }
  if (direct) return;  // k_mem_direct folds M; the compaction kernel resets cscale / the list
  for (int k = threadIdx.x; k < ne * p.dM; k += blockDim.x) {
    const int e = k / p.dM, m = k % p.dM;
    st.pend_phi[(u * p.F + np + e) * p.dM + m] = phi[(size_t)e * p.dM + m];
  }
  for (int k = threadIdx.x; k < ne * p.Dkv; k += blockDim.x) {
    const int e = k / p.Dkv, col = k % p.Dkv;
    const int slot = st.ev_slot[u * p.tail + e];
    const int h = col / p.d, c = col % p.d;
    st.pend_v[(u * p.F + np + e) * p.Dkv + col] = st.Vc[((u * p.Hkv + h) * p.cap + slot) * p.d + c];
  }
  for (int e = threadIdx.x; e < ne; e += blockDim.x) st.pend_w[u * p.F + np + e] = p.eta / c_new;
  __syncthreads();
  if (threadIdx.x == 0) {
    st.cscale[u] = c_new;
    ctr[CTR_NPEND] = np + ne;
  }
}

// exclusive prefix sum of one int per thread over the block; returns the total
__device__ int block_exclusive_scan(int v, int* out_excl, int* s_tmp /*[33]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) s_tmp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    int wv = lane < nw ? s_tmp[lane] : 0;
    int wi = wv;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < nw) s_tmp[lane] = wi - wv;
    if (lane == nw - 1) s_tmp[32] = wi;
  }
  __syncthreads();
  *out_excl = incl - v + s_tmp[warp];
  const int total = s_tmp[32];
  __syncthreads();
  return total;
}

// a4: the retained entries end in slots [0, B): the k-th evicted slot below B receives the k-th
// retained entry found at or above B (both ascending).  grid = n_seq, block = 256.
__global__ void k_compact(ImDims p, ImState st, ImScratch sc, ImCall call) {
  __shared__ int s_tmp[33];
  const int i = blockIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int ne = min(ctr[CTR_NEVICT], p.tail);
  if (ne <= 0) return;
  const int n = ctr[CTR_N];
  if (n != p.B + ne) {
    if (threadIdx.x == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  const int32_t* evs = st.ev_slot + u * p.tail;
  const uint8_t* keep = st.keep + u * p.cap;
  int32_t* surv = sc.moves + ((size_t)i * 2 + 1) * p.tail;
  // survivors among the tail slots [B, n), in ascending order
  const int per = (ne + blockDim.x - 1) / blockDim.x;
  const int t0 = min(ne, (int)threadIdx.x * per), t1 = min(ne, t0 + per);
  int cnt = 0;
  for (int t = t0; t < t1; ++t) cnt += keep[p.B + t] ? 1 : 0;
  int off;
  const int nh = block_exclusive_scan(cnt, &off, s_tmp);  // survivors above B == holes below B
  for (int t = t0; t < t1; ++t)
    if (keep[p.B + t]) surv[off++] = p.B + t;
  __syncthreads();
  // the evicted list is ascending, so its first nh entries are exactly the holes below B
  const int dv = p.d / 8;
  for (int k = threadIdx.x; k < nh * p.Hkv * dv; k += blockDim.x) {
    const int j = k / (p.Hkv * dv), rem = k % (p.Hkv * dv), h = rem / dv, c = rem % dv;
    const int dst = evs[j], src = surv[j];
    const size_t base = (u * p.Hkv + h) * p.cap;
    reinterpret_cast<uint4*>(st.Kc + (base + dst) * p.d)[c] = reinterpret_cast<const uint4*>(st.Kc + (base + src) * p.d)[c];
    reinterpret_cast<uint4*>(st.Vc + (base + dst) * p.d)[c] = reinterpret_cast<const uint4*>(st.Vc + (base + src) * p.d)[c];
  }
  for (int k = threadIdx.x; k < nh * p.dI; k += blockDim.x) {
    const int j = k / p.dI, c = k % p.dI;
    st.kidx[(u * p.cap + evs[j]) * p.dI + c] = st.kidx[(u * p.cap + surv[j]) * p.dI + c];
  }
  for (int j = threadIdx.x; j < nh; j += blockDim.x) {
    if (evs[j] >= p.B) atomicOr(st.status, ST_COUNT);
    st.pos[u * p.cap + evs[j]] = st.pos[u * p.cap + surv[j]];
  }
  if (threadIdx.x == 0) {
    ctr[CTR_N] = p.B;
    if (ctr[CTR_DIRECT]) {
      st.cscale[u] = 1.0f;
      ctr[CTR_NPEND] = 0;
      ctr[CTR_DIRECT] = 0;
    }
  }
}

}  // namespace

cudaError_t im_launch_memory_write(const ImLaunch& L, const ImCall& call, int ne_max, bool direct) {
  const ImDims& p = L.p;
  {
    dim3 grid((ne_max + PHI_E - 1) / PHI_E, call.n_seq);
    const size_t smem = (size_t)PHI_E * p.Dkv * 2;
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(k_phi_evicted, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    k_phi_evicted<<<grid, 256, smem, L.stream>>>(p, L.st, L.w, L.sc, call);
    ++*L.launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (direct) {
    dim3 grid((p.Dkv + 63) / 64, (p.dM + 63) / 64, call.n_seq);
    k_mem_direct<<<grid, 256, 0, L.stream>>>(p, L.st, L.sc, call);
    ++*L.launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  k_mem_small<<<call.n_seq, 256, 0, L.stream>>>(p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_compact(const ImLaunch& L, const ImCall& call) {
  k_compact<<<call.n_seq, 256, 0, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

// a5-a6: attention over the retained entries (split over the key axis), merge of the partials,
// memory readout (Eq. 5) and the gated residual fuse (Eq. 4).
#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int SPLIT_LEN = 256;  // keys per split (ImDims::max_splits is derived from the same value)

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Partial attention of one query head over one split of the retained entries.
// grid = (splits, H, n_seq), block = 128 (4 warps striding over keys; lanes stride over d).
// part[((i*H + j)*max_splits + s)*(d+2) + ..] = unnormalised acc[d], running max, running sum.
__global__ void k_attn_partial(ImDims p, ImState st, ImScratch sc, ImCall call, const bf16* __restrict__ q) {
  __shared__ float s_acc[4][256];
  __shared__ float s_m[4], s_l[4];
  const int s = blockIdx.x, j = blockIdx.y, i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int n = min(st.ctr[u * CTR_STRIDE + CTR_N], p.cap);
  const int t0 = s * SPLIT_LEN;
  if (t0 >= n) return;
  const int t1 = min(n, t0 + SPLIT_LEN);
  const int g = j / p.Gq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bf16* Kb = st.Kc + (u * p.Hkv + g) * (size_t)p.cap * p.d;
  const bf16* Vb = st.Vc + (u * p.Hkv + g) * (size_t)p.cap * p.d;
  float qr[8], acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c = lane + 32 * k;
    qr[k] = c < p.d ? __bfloat162float(q[((size_t)i * p.H + j) * p.d + c]) : 0.f;
    acc[k] = 0.f;
  }
  float m = NEG_INF, l = 0.f;
  for (int t = t0 + warp; t < t1; t += 4) {
    const bf16* kr = Kb + (size_t)t * p.d;
    float dot = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      if (c < p.d) dot = fmaf(qr[k], __bfloat162float(kr[c]), dot);
    }
    dot = warp_sum(dot) * p.scale;
    const float m_new = fmaxf(m, dot);
    const float corr = __expf(m - m_new);   // exp(-inf) = 0 on the first key
    const float pr = __expf(dot - m_new);
    l = l * corr + pr;
    const bf16* vr = Vb + (size_t)t * p.d;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      if (c < p.d) acc[k] = fmaf(pr, __bfloat162float(vr[c]), acc[k] * corr);
    }
    m = m_new;
  }
  if (lane == 0) {
    s_m[warp] = m;
    s_l[warp] = l;
  }
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c = lane + 32 * k;
    if (c < p.d) s_acc[warp][c] = acc[k];
  }
  __syncthreads();
  float M = NEG_INF;
  for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w]);
  float* dst = sc.part + (((size_t)i * p.H + j) * p.max_splits + s) * (p.d + 2);
  for (int c = threadIdx.x; c < p.d; c += blockDim.x) {
    float a = 0.f;
    for (int w = 0; w < 4; ++w)
      if (s_m[w] > NEG_INF) a = fmaf(s_acc[w][c], __expf(s_m[w] - M), a);
    dst[c] = a;
  }
  if (threadIdx.x == 0) {
    float L = 0.f;
    for (int w = 0; w < 4; ++w)
      if (s_m[w] > NEG_INF) L = fmaf(s_l[w], __expf(s_m[w] - M), L);
    dst[p.d] = M;
    dst[p.d + 1] = L;
  }
}

// Merge of the split partials of one query head + readout + fuse.
// grid = (H, n_seq), block = 256.
template <typename OutT>
__global__ void k_attn_merge(ImDims p, ImState st, ImWeights w, ImScratch sc, ImCall call, OutT* __restrict__ out) {
  __shared__ float s_red[256];
  __shared__ float s_dot[64];
  __shared__ float s_scalar[2];
  const int j = blockIdx.x, i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = min(ctr[CTR_N], p.cap);
  const int ns = (n + SPLIT_LEN - 1) / SPLIT_LEN;
  const int g = j / p.Gq;
  const int tid = threadIdx.x;
  const float* part = sc.part + ((size_t)i * p.H + j) * p.max_splits * (p.d + 2);
  float M = NEG_INF;
  for (int s = 0; s < ns; ++s) M = fmaxf(M, part[(size_t)s * (p.d + 2) + p.d]);
  float Lsum = 0.f;
  for (int s = 0; s < ns; ++s) Lsum = fmaf(part[(size_t)s * (p.d + 2) + p.d + 1], __expf(part[(size_t)s * (p.d + 2) + p.d] - M), Lsum);
  float o = 0.f;
  if (tid < p.d) {
    for (int s = 0; s < ns; ++s)
      o = fmaf(part[(size_t)s * (p.d + 2) + tid], __expf(part[(size_t)s * (p.d + 2) + p.d] - M), o);
    o = ns > 0 ? o / Lsum : 0.f;
  }
  float res = o;
  if (p.mem) {
    const ImRows r = im_rows(p);
    extern __shared__ float phiq[];  // [dM] phi(q), summed over the K-split partials
    for (int m = tid; m < p.dM; m += blockDim.x) phiq[m] = im_raw_sum(p, sc, call, i, r.theta + m);
    __syncthreads();
    const int np = min(ctr[CTR_NPEND], p.F);
    // den = sum_m phi_q[m]^2 b[m] + eps
    float part_den = 0.f;
    for (int m = tid; m < p.dM; m += blockDim.x) part_den = fmaf(phiq[m] * phiq[m], st.bvec[u * p.dM + m], part_den);
    s_red[tid] = part_den;
    __syncthreads();
    if (tid < 32) {
      float v = 0.f;
      for (int k = tid; k < 256; k += 32) v += s_red[k];
      v = warp_sum(v);
      if (tid == 0) s_scalar[0] = v + p.eps;
    }
    __syncthreads();
    // phi_q . phi_p for the pending rank-one terms
    const int warp = tid >> 5, lane = tid & 31;
    for (int pp = warp; pp < np; pp += 8) {
      const float* ph = st.pend_phi + (u * p.F + pp) * p.dM;
      float v = 0.f;
      for (int m = lane; m < p.dM; m += 32) v = fmaf(phiq[m], ph[m], v);
      v = warp_sum(v);
      if (lane == 0) s_dot[pp] = v * st.pend_w[u * p.F + pp];
    }
    __syncthreads();
    if (tid < p.d) {
      const int col = g * p.d + tid;
      const float* Mh = st.Mhat + u * p.dM * p.Dkv;
      float mv = 0.f;
      for (int m = 0; m < p.dM; ++m) mv = fmaf(phiq[m], Mh[(size_t)m * p.Dkv + col], mv);
      for (int pp = 0; pp < np; ++pp) mv = fmaf(s_dot[pp], __bfloat162float(st.pend_v[(u * p.F + pp) * p.Dkv + col]), mv);
      mv = st.cscale[u] * mv / s_scalar[0];
      const float gate = 1.0f / (1.0f + expf(-(im_raw_sum(p, sc, call, i, r.wg) + w.bg[0])));
      res = fmaf(gate, mv, o);
    }
  }
  if (tid < p.d) {
    const size_t idx = ((size_t)i * p.H + j) * p.d + tid;
    if constexpr (sizeof(OutT) == 2) out[idx] = __float2bfloat16_rn(res);
    else out[idx] = res;
  }
}

}  // namespace

cudaError_t im_launch_attention(const ImLaunch& L, const ImCall& call, const void* q, void* out, int n_max) {
  const ImDims& p = L.p;
  dim3 grid((n_max + SPLIT_LEN - 1) / SPLIT_LEN, p.H, call.n_seq);
  k_attn_partial<<<grid, 128, 0, L.stream>>>(p, L.st, L.sc, call, (const bf16*)q);
  ++*L.launches;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  dim3 grid2(p.H, call.n_seq);
  if (p.out_f32) k_attn_merge<float><<<grid2, 256, (size_t)p.dM * 4, L.stream>>>(p, L.st, L.w, L.sc, call, (float*)out);
  else k_attn_merge<bf16><<<grid2, 256, (size_t)p.dM * 4, L.stream>>>(p, L.st, L.w, L.sc, call, (bf16*)out);
  ++*L.launches;
  return cudaGetLastError();
}

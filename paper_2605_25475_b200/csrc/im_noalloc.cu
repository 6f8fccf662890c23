// im_attention_noalloc: split softmax attention for one query token whose scratch (the per-split
// partial results) lives in a fixed device array that is part of the library image, so the call
// needs no allocation from anyone.  See include/indexmem.h for the contract.
#include <math.h>
#include <stdio.h>

#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int SPLIT = 256;                               // keys per split
constexpr size_t SCRATCH_FLOATS = IM_NOALLOC_MAX_FLOATS; // 4 MiB of partials

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) float g_noalloc_scratch[SCRATCH_FLOATS];

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// partial attention of query head j over split s.  grid = (splits, H), block = 128.
// part[(j * splits + s) * (d + 2) + ..] = unnormalised acc[d], running max, running sum.
__global__ void k_noalloc_partial(const bf16* __restrict__ q, const bf16* __restrict__ K, const bf16* __restrict__ V,
                                  int Gq, int d, int n, float scale, float* __restrict__ part) {
  __shared__ float s_acc[4][256];
  __shared__ float s_m[4], s_l[4];
  const int s = blockIdx.x, j = blockIdx.y, splits = gridDim.x;
  const int t0 = s * SPLIT, t1 = min(n, t0 + SPLIT);
  const int g = j / Gq;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bf16* Kb = K + (size_t)g * n * d;
  const bf16* Vb = V + (size_t)g * n * d;
  float qr[8], acc[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c = lane + 32 * k;
    qr[k] = c < d ? __bfloat162float(q[(size_t)j * d + c]) : 0.f;
    acc[k] = 0.f;
  }
  float m = NEG_INF, l = 0.f;
  for (int t = t0 + warp; t < t1; t += 4) {
    float dot = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      if (c < d) dot = fmaf(qr[k], __bfloat162float(Kb[(size_t)t * d + c]), dot);
    }
    dot = warp_sum(dot) * scale;
    const float m_new = fmaxf(m, dot);
    const float corr = __expf(m - m_new);
    const float pr = __expf(dot - m_new);
    l = l * corr + pr;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int c = lane + 32 * k;
      if (c < d) acc[k] = fmaf(pr, __bfloat162float(Vb[(size_t)t * d + c]), acc[k] * corr);
    }
    m = m_new;
  }
  if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int c = lane + 32 * k;
    if (c < d) s_acc[warp][c] = acc[k];
  }
  __syncthreads();
  float M = NEG_INF;
  for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w]);
  float* dst = part + ((size_t)j * splits + s) * (d + 2);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float a = 0.f;
    for (int w = 0; w < 4; ++w)
      if (s_m[w] > NEG_INF) a = fmaf(s_acc[w][c], __expf(s_m[w] - M), a);
    dst[c] = a;
  }
  if (threadIdx.x == 0) {
    float L = 0.f;
    for (int w = 0; w < 4; ++w)
      if (s_m[w] > NEG_INF) L = fmaf(s_l[w], __expf(s_m[w] - M), L);
    dst[d] = M;
    dst[d + 1] = L;
  }
}

// merge of the splits of one query head.  grid = H, block = 256.
__global__ void k_noalloc_merge(const float* __restrict__ part, int splits, int d, bf16* __restrict__ out) {
  const int j = blockIdx.x, c = threadIdx.x;
  const float* ps = part + (size_t)j * splits * (d + 2);
  float M = NEG_INF;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, ps[(size_t)s * (d + 2) + d]);
  float L = 0.f, o = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float e = __expf(ps[(size_t)s * (d + 2) + d] - M);
    L = fmaf(ps[(size_t)s * (d + 2) + d + 1], e, L);
    if (c < d) o = fmaf(ps[(size_t)s * (d + 2) + c], e, o);
  }
  if (c < d) out[(size_t)j * d + c] = __float2bfloat16_rn(o / L);
}

// device address of the scratch array, looked up once per device (the array's name is only a
// host-side handle in host code; kernels must be given the address that the runtime reports).
// Host threads that make their first call on a device at the same time each look the address up
// and store the same value: the cache needs no lock.
constexpr int MAX_DEVICES = 64;
float* g_scratch_addr[MAX_DEVICES] = {};

}  // namespace

extern "C" int im_attention_noalloc(const void* q, const void* k, const void* v, int n_q_heads, int n_kv_heads,
                                    int head_dim, int n, float softmax_scale, void* out, void* cuda_stream) {
  if (!q || !k || !v || !out) return im_fail_message(IM_ERR_ARG, "im_attention_noalloc: null tensor");
  if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads || head_dim < 1 || head_dim > 256 || n < 1)
    return im_fail_message(IM_ERR_ARG, "im_attention_noalloc: bad shape");
  if (n_q_heads > 65535)  // the query heads ride on the grid's y axis
    return im_fail_message(IM_ERR_ARG, "im_attention_noalloc: more than 65535 query heads");
  const int splits = (n + SPLIT - 1) / SPLIT;
  const size_t need = (size_t)n_q_heads * splits * (head_dim + 2);
  if (need > SCRATCH_FLOATS) {
    char msg[200];
    snprintf(msg, sizeof(msg), "im_attention_noalloc: needs %zu scratch floats (heads * ceil(n/256) * (d+2)), the built-in array holds %zu",
             need, (size_t)SCRATCH_FLOATS);
    return im_fail_message(IM_ERR_CAPACITY, msg);
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return im_fail_message(IM_ERR_CUDA, "im_attention_noalloc: no usable CUDA device");
  if (!g_scratch_addr[dev]) {  // first call on this device: resolve the array's device address
    float* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || !ptr) return im_fail_message(IM_ERR_CUDA, cudaGetErrorString(e));
    g_scratch_addr[dev] = ptr;
  }
  float* scratch = g_scratch_addr[dev];
  const float scale = softmax_scale != 0.f ? softmax_scale : 1.0f / sqrtf((float)head_dim);
  cudaStream_t s = (cudaStream_t)cuda_stream;
  dim3 grid(splits, n_q_heads);
  k_noalloc_partial<<<grid, 128, 0, s>>>((const bf16*)q, (const bf16*)k, (const bf16*)v, n_q_heads / n_kv_heads,
                                         head_dim, n, scale, scratch);
  e = cudaGetLastError();
  if (e == cudaSuccess) {
    k_noalloc_merge<<<n_q_heads, 256, 0, s>>>(scratch, splits, head_dim, (bf16*)out);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) return im_fail_message(IM_ERR_CUDA, cudaGetErrorString(e));
  return IM_OK;
}

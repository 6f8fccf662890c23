// Block-level building blocks of the budgeted selection (a2), shared by the kernels that select one row per thread
// block: the shared-row selection of a sequence (im_index.cu) and the selection per KV head (im_perhead.cu).
#pragma once
#include "im_internal.cuh"

// ------------------------------------------------------------------------------------------------
// a2: budgeted selection of one row (one thread block).  Radix select of the k-th largest 64-bit
// key (score image, ~position), eight passes of eight bits; keys are distinct, so exactly k entries
// compare >= the threshold.
struct SelectShared {
  uint32_t hist[256];
  uint32_t digit, remaining, single;
  unsigned long long found;
};

// Key of rank k (k-th largest; keys are distinct) among n entries, by an 8-pass radix select over the 64-bit key,
// most significant byte first.  Up to SEL_KPT keys per thread stay in registers over the passes (n beyond that:
// re-read from memory); the digit of a pass is found by warp 0 (lane l sums the 8 bins 255 - 8 l down to
// 248 - 8 l, a prefix over the lanes locates the lane, which then walks its own bins).  As soon as the chosen bin
// holds a single key that key is the answer: with distinct scores that is after two or three passes, not eight.
constexpr int SEL_KPT = 8;
static __device__ uint64_t block_kth_largest_key(const float* __restrict__ score, const int32_t* __restrict__ pos, int n,
                                          int k, int n_sink, SelectShared* sh) {
  uint64_t prefix = 0, mask = 0;
  const bool cached = n <= SEL_KPT * (int)blockDim.x;
  uint64_t kreg[SEL_KPT];
  if (cached) {
#pragma unroll
    for (int j = 0; j < SEL_KPT; ++j) {
      const int t = threadIdx.x + j * blockDim.x;
      kreg[j] = t < n ? im_select_key(score[t], pos[t], n_sink) : 0ull;
    }
  }
  if (threadIdx.x == 0) sh->remaining = (uint32_t)k;
  for (int shift = 56; shift >= 0; shift -= 8) {
    for (int b = threadIdx.x; b < 256; b += blockDim.x) sh->hist[b] = 0;
    __syncthreads();
    if (cached) {
#pragma unroll
      for (int j = 0; j < SEL_KPT; ++j) {
        const int t = threadIdx.x + j * blockDim.x;
        if (t < n && (kreg[j] & mask) == prefix) atomicAdd(&sh->hist[(uint32_t)(kreg[j] >> shift) & 255u], 1u);
      }
    } else {
      for (int t = threadIdx.x; t < n; t += blockDim.x) {
        const uint64_t key = im_select_key(score[t], pos[t], n_sink);
        if ((key & mask) == prefix) atomicAdd(&sh->hist[(uint32_t)(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      const int lane = threadIdx.x;
      const uint32_t rem = sh->remaining;
      uint32_t mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += sh->hist[255 - 8 * lane - j];
      uint32_t incl = mine;  // entries in the bins of lanes 0 .. lane (the highest bins)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const uint32_t hit = __ballot_sync(0xffffffffu, incl >= rem);
      // the rank lies in the bins of the first lane whose prefix reaches it (bin 0 takes what is left otherwise)
      const int owner = hit ? __ffs(hit) - 1 : 31;
      if (lane == owner) {
        uint32_t cum = incl - mine;
        int b = 255 - 8 * lane;
        const int b_last = lane == 31 ? 0 : 255 - 8 * lane - 7;
        for (; b > b_last; --b) {
          const uint32_t c = sh->hist[b];
          if (cum + c >= rem) break;
          cum += c;
        }
        sh->digit = (uint32_t)b;
        sh->remaining = rem - cum;
        sh->single = sh->hist[b] == 1u ? 1u : 0u;
      }
    }
    __syncthreads();
    prefix |= (uint64_t)sh->digit << shift;
    mask |= 0xFFull << shift;
    if (sh->single) {  // (block uniform) exactly one key carries this prefix: find it
      if (cached) {
#pragma unroll
        for (int j = 0; j < SEL_KPT; ++j) {
          const int t = threadIdx.x + j * blockDim.x;
          if (t < n && (kreg[j] & mask) == prefix) sh->found = kreg[j];
        }
      } else {
        for (int t = threadIdx.x; t < n; t += blockDim.x) {
          const uint64_t key = im_select_key(score[t], pos[t], n_sink);
          if ((key & mask) == prefix) sh->found = key;
        }
      }
      __syncthreads();
      const uint64_t key = sh->found;
      __syncthreads();  // (before a later call of this function writes the structure again)
      return key;
    }
    __syncthreads();
  }
  return prefix;
}

// exclusive prefix sum of one int per thread over the block (blockDim.x <= 1024); returns the total
static __device__ int block_exclusive_scan(int v, int* out_excl, int* s_tmp /*[33]*/) {
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
    int w = lane < nw ? s_tmp[lane] : 0;
    int wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += t;
    }
    if (lane < nw) s_tmp[lane] = wi - w;
    if (lane == nw - 1) s_tmp[32] = wi;
  }
  __syncthreads();
  *out_excl = incl - v + s_tmp[warp];
  const int total = s_tmp[32];
  __syncthreads();
  return total;
}


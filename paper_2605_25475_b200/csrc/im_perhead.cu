// A retained set per KV head (Sec. 2.2: S = f(.) in R^{B x H_kv x L}, I = TopK(S, L'), [K', V'] = Gather(K, V, I)).
//
// With a scorer that has a head axis - Knorm, S_t = ||K_t||_2 (Sec. 2.2), or scores handed in by the caller (the memory
// module on top of another eviction policy, Sec. 5 ablation) - every KV head of a sequence keeps its own B token
// positions.  The K / V cache already is one slab per (sequence, KV head), so attention needs nothing new: all heads
// hold the same NUMBER of entries (same budget, same evicted count per compression), only the positions in their
// slots differ.  What this file adds is the bookkeeping per head (position and score per slot, selection, hole
// filling) and the evict step's memory write: Alg. 1 sums the evicted values "across heads per token", read here as
// one model-space pair per token that loses at least one head slice in the step, holding the evicted slices at their
// heads' places and zeros at the heads that keep the token.  In KV space that is a row [H_kv * d] with the slices of
// the evicting heads; rows are formed by grouping the evicted (head, slot) pairs of a sequence by position.
//
// These calls run in order on the caller's stream (no side streams); the memory write accumulates straight into Mhat
// (no pending list), so the state is M = Mhat, cscale = 1.
#include "im_internal.cuh"
#include "im_select.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();

__device__ __forceinline__ size_t hrow(const ImDims& p, size_t u, int h) { return (u * p.Hkv + h) * (size_t)p.cap; }

// append C tokens (decode: C = 1): K / V slices into the slabs, position and score per head.
// grid = (C, n_seq), block = 128.  Counters advance in k_ph_commit.
__global__ void k_ph_append(ImDims p, ImState st, ImCall call, const bf16* __restrict__ K, const bf16* __restrict__ V) {
  const int c = blockIdx.x, i = blockIdx.y, tid = threadIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = ctr[CTR_N], T = ctr[CTR_T];
  if (n < 0 || n + call.C > p.cap) {
    if (tid == 0 && c == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  const int slot = n + c;
  const int dv = p.d / 8;
  for (int k = tid; k < p.Hkv * dv; k += blockDim.x) {
    const int h = k / dv, cc = k % dv;
    const size_t src = ((size_t)i * call.C + c) * p.Dkv + h * p.d;
    const size_t row = (hrow(p, u, h) + slot) * p.d;
    reinterpret_cast<uint4*>(st.Kc + row)[cc] = reinterpret_cast<const uint4*>(K + src)[cc];
    reinterpret_cast<uint4*>(st.Vc + row)[cc] = reinterpret_cast<const uint4*>(V + src)[cc];
  }
  // one warp per head (round robin): Knorm of the head's key slice in float32
  const int warp = tid >> 5, lane = tid & 31;
  for (int h = warp; h < p.Hkv; h += blockDim.x >> 5) {
    float s = NEG_INF;
    if (p.scorer == 1) {
      float sq = 0.f;
      const bf16* kr = K + ((size_t)i * call.C + c) * p.Dkv + h * p.d;
      for (int k = lane; k < p.d; k += 32) {
        const float x = __bfloat162float(kr[k]);
        sq = fmaf(x, x, sq);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      s = sqrtf(sq);
    }
    if (lane == 0) {
      st.hpos[hrow(p, u, h) + slot] = T + c;
      st.hscore[hrow(p, u, h) + slot] = s;
    }
  }
}

// counters after the append.  decode: C = 1 and the interval counter advances; prefill: the interval restarts in
// the selection.  grid = n_seq, block = 32.
__global__ void k_ph_commit(ImDims p, ImState st, ImCall call) {
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  if (threadIdx.x == 0) {
    const int n0 = ctr[CTR_N];
    if (n0 < 0 || n0 + call.C > p.cap) return;
    ctr[CTR_N] = n0 + call.C;
    ctr[CTR_T] = ctr[CTR_T] + call.C;
    ctr[CTR_NEVICT] = 0;
    if (!call.prefill) ctr[CTR_SINCE] = ctr[CTR_SINCE] + 1;
  }
}

// scores handed in by the caller: ext[i][h][position] -> score of the slot that holds that position.
// grid = (Hkv, n_seq), block = 256.
__global__ void k_ph_scores_in(ImDims p, ImState st, ImCall call, const float* __restrict__ ext, long long n_pos) {
  const int h = blockIdx.x, i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int n = st.ctr[u * CTR_STRIDE + CTR_N];
  if (n < 0 || n > p.cap) return;
  const float* row = ext + ((size_t)i * p.Hkv + h) * n_pos;
  bool bad = false;
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    const int ps = st.hpos[hrow(p, u, h) + t];
    if (ps < 0 || ps >= n_pos) { bad = true; continue; }
    const float s = row[ps];
    bad |= s != s;
    st.hscore[hrow(p, u, h) + t] = s;
  }
  if (bad) atomicOr(st.status, ST_NONFINITE);
}

// a2 per (sequence, KV head): keep the B best of the head's n entries (score descending, position ascending, sinks
// first), list the evicted slots in ascending slot order and the retained entries above the budget that will fill
// the holes.  grid = (Hkv, n_seq), block = 1024.
__global__ void k_ph_select(ImDims p, ImState st, ImScratch sc, ImCall call) {
  __shared__ SelectShared sh;
  __shared__ int s_tmp[33];
  const int h = blockIdx.x, i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = ctr[CTR_N];
  if (n < 0 || n > p.cap) {
    if (threadIdx.x == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  const size_t r0 = hrow(p, u, h);
  const float* score = st.hscore + r0;
  const int32_t* pos = st.hpos + r0;
  uint8_t* keep = st.hkeep + r0;
  const size_t e0 = (u * p.Hkv + h) * (size_t)p.tail;                     // this row's evicted lists
  const size_t s0 = ((size_t)i * p.Hkv + h) * (size_t)p.tail;            // this row's survivors (per call)
  for (int t = threadIdx.x; t < n; t += blockDim.x) {  // what the selection saw (parity export)
    st.hsel_pos[r0 + t] = pos[t];
    st.hsel_score[r0 + t] = score[t];
  }
  int ne = 0, nh = 0;
  if (n > p.B) {
    ne = n - p.B;
    const uint64_t thr = block_kth_largest_key(score, pos, n, p.B, p.n_sink, &sh);
    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int t0 = min(n, (int)threadIdx.x * per), t1 = min(n, t0 + per);
    int cnt = 0;
    for (int t = t0; t < t1; ++t) {
      const bool k = im_select_key(score[t], pos[t], p.n_sink) >= thr;
      keep[t] = k ? 1 : 0;
      cnt += k ? 0 : 1;
    }
    int off;
    const int total = block_exclusive_scan(cnt, &off, s_tmp);
    if (total != ne && threadIdx.x == 0) atomicOr(st.status, ST_COUNT);
    for (int t = t0; t < t1; ++t)
      if (!keep[t] && off < p.tail) {
        st.hev_slot[e0 + off] = t;
        st.hev_pos[e0 + off] = pos[t];
        ++off;
      }
    __syncthreads();
    const int tl = n - p.B;
    const int per2 = (tl + blockDim.x - 1) / blockDim.x;
    const int a0 = min(tl, (int)threadIdx.x * per2), a1 = min(tl, a0 + per2);
    int cnt2 = 0;
    for (int t = a0; t < a1; ++t) cnt2 += keep[p.B + t] ? 1 : 0;
    int off2;
    nh = block_exclusive_scan(cnt2, &off2, s_tmp);
    for (int t = a0; t < a1; ++t)
      if (keep[p.B + t]) sc.hsurv[s0 + off2++] = p.B + t;
  }
  if (threadIdx.x == 0) sc.hnhole[(size_t)i * p.Hkv + h] = nh;
}

// counters after the selection of all heads.  grid = n_seq, block = 32.
__global__ void k_ph_select_commit(ImDims p, ImState st, ImCall call) {
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  if (threadIdx.x == 0) {
    const int n = ctr[CTR_N];
    if (n < 0 || n > p.cap) return;
    const int ne = n > p.B ? n - p.B : 0;
    ctr[CTR_SINCE] = 0;
    ctr[CTR_NSEL] = n;
    ctr[CTR_NEVICT] = ne;
    ctr[CTR_N] = n - ne;
    if (ne > 0) ctr[CTR_EVSTEPS] = ctr[CTR_EVSTEPS] + 1;
  }
}

// Group the evicted (head, slot) pairs of a sequence by token position: the pairs are sorted by (position, head)
// with a bitonic network in shared memory, every distinct position gets a row number (ascending position), and
// hrowmap[i][h][e] receives the row of evicted entry e of head h.  hntok[i] = number of rows.
// grid = n_seq, block = 1024, dynamic smem = NP * 8 bytes, NP = the pair count rounded up to a power of two.
__global__ void k_ph_group(ImDims p, ImState st, ImScratch sc, ImCall call, int NP) {
  extern __shared__ unsigned long long s_key[];  // (position << 32) | (head << 20) | evicted index; ~0 pads
  __shared__ int s_tmp[33];
  const int i = blockIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(max(st.ctr[u * CTR_STRIDE + CTR_NEVICT], 0), p.tail);
  const int N = ne * p.Hkv;
  for (int k = threadIdx.x; k < NP; k += blockDim.x) {
    unsigned long long key = ~0ull;
    if (k < N) {
      const int h = k / ne, e = k % ne;
      const int ps = st.hev_pos[(u * p.Hkv + h) * (size_t)p.tail + e];
      key = ((unsigned long long)(uint32_t)ps << 32) | ((unsigned long long)h << 20) | (unsigned long long)e;
    }
    s_key[k] = key;
  }
  __syncthreads();
  for (int size = 2; size <= NP; size <<= 1)
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int k = threadIdx.x; k < NP / 2; k += blockDim.x) {
        const int lo = (k / stride) * 2 * stride + (k % stride), hi = lo + stride;
        const bool up = ((lo & size) == 0);
        const unsigned long long a = s_key[lo], b = s_key[hi];
        if ((a > b) == up) { s_key[lo] = b; s_key[hi] = a; }
      }
      __syncthreads();
    }
  // row of a pair = number of position changes before it
  const int per = (NP + blockDim.x - 1) / blockDim.x;
  const int k0 = min(NP, (int)threadIdx.x * per), k1 = min(NP, k0 + per);
  int cnt = 0;
  for (int k = k0; k < k1; ++k)
    if (k < N && (k == 0 || (s_key[k] >> 32) != (s_key[k - 1] >> 32))) ++cnt;
  int off;
  const int total = block_exclusive_scan(cnt, &off, s_tmp);
  for (int k = k0; k < k1; ++k) {
    if (k >= N) break;
    if (k == 0 || (s_key[k] >> 32) != (s_key[k - 1] >> 32)) ++off;
    const int h = (int)((s_key[k] >> 20) & 0xfff), e = (int)(s_key[k] & 0xfffff);
    sc.hrowmap[((size_t)i * p.Hkv + h) * p.tail + e] = off - 1;
  }
  if (threadIdx.x == 0) sc.hntok[i] = total;
}

// Assemble the rows: row r of sequence i in KV space [Hkv * d], the evicted slices at their heads' places, zeros
// elsewhere.  Two launches: this kernel with zero = 1 clears the rows, then with zero = 0 scatters the slices.
// grid = (rows, n_seq), block = 128.
__global__ void k_ph_assemble(ImDims p, ImState st, ImScratch sc, ImCall call, int zero) {
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(max(st.ctr[u * CTR_STRIDE + CTR_NEVICT], 0), p.tail);
  const int dv = p.d / 8;
  if (zero) {
    const int r = blockIdx.x;
    if (r >= ne * p.Hkv) return;
    uint4* kd = reinterpret_cast<uint4*>(sc.evK + ((size_t)i * p.evr + r) * p.Dkv);
    uint4* vd = reinterpret_cast<uint4*>(sc.evV + ((size_t)i * p.evr + r) * p.Dkv);
    for (int k = threadIdx.x; k < p.Hkv * dv; k += blockDim.x) kd[k] = vd[k] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const int pair = blockIdx.x;  // (head, evicted index)
  if (pair >= ne * p.Hkv) return;
  const int h = pair / ne, e = pair % ne;
  const int slot = st.hev_slot[(u * p.Hkv + h) * (size_t)p.tail + e];
  const int r = sc.hrowmap[((size_t)i * p.Hkv + h) * p.tail + e];
  if (slot < 0 || slot >= p.cap || r < 0 || r >= p.evr) return;
  const uint4* ks = reinterpret_cast<const uint4*>(st.Kc + (hrow(p, u, h) + slot) * p.d);
  const uint4* vs = reinterpret_cast<const uint4*>(st.Vc + (hrow(p, u, h) + slot) * p.d);
  uint4* kd = reinterpret_cast<uint4*>(sc.evK + ((size_t)i * p.evr + r) * p.Dkv + h * p.d);
  uint4* vd = reinterpret_cast<uint4*>(sc.evV + ((size_t)i * p.evr + r) * p.Dkv + h * p.d);
  for (int k = threadIdx.x; k < dv; k += blockDim.x) { kd[k] = ks[k]; vd[k] = vs[k]; }
}

// Eq. 6-7 over the assembled rows, straight into the state: Mhat <- lambda Mhat + eta sum_r phi_r v_r^T,
// b <- lambda b + eta sum_r phi_r^2 (rows beyond the token count are zero and add nothing).  Only sequences that
// evict decay.  grid = (ceil(Dkv / 64), ceil(dM / 16), n_seq), block = 256: thread = (4 columns, 1 of 16 rows).
__global__ void __launch_bounds__(256) k_ph_mem_write(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int i = blockIdx.z;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(max(st.ctr[u * CTR_STRIDE + CTR_NEVICT], 0), p.tail);
  if (ne <= 0) return;
  const int nt = min(sc.hntok[i], p.evr);
  const int m = blockIdx.y * 16 + (threadIdx.x >> 4);
  const int c0 = blockIdx.x * 64 + (threadIdx.x & 15) * 4;
  if (m >= p.dM) return;
  const float* phi = sc.phi + (size_t)i * p.evr * p.dM;
  const bf16* V = sc.evV + (size_t)i * p.evr * p.Dkv;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, sq = 0.f;
  for (int r = 0; r < nt; ++r) {
    const float f = phi[(size_t)r * p.dM + m];
    sq = fmaf(f, f, sq);
    if (c0 < p.Dkv) {
      const uint2 w = *reinterpret_cast<const uint2*>(V + (size_t)r * p.Dkv + c0);
      a0 = fmaf(f, __uint_as_float(w.x << 16), a0);
      a1 = fmaf(f, __uint_as_float(w.x & 0xffff0000u), a1);
      a2 = fmaf(f, __uint_as_float(w.y << 16), a2);
      a3 = fmaf(f, __uint_as_float(w.y & 0xffff0000u), a3);
    }
  }
  if (c0 < p.Dkv) {
    float4* dst = reinterpret_cast<float4*>(st.Mhat + (u * p.dM + m) * (size_t)p.Dkv + c0);
    float4 o = *dst;
    o.x = p.lambda * o.x + p.eta * a0;
    o.y = p.lambda * o.y + p.eta * a1;
    o.z = p.lambda * o.z + p.eta * a2;
    o.w = p.lambda * o.w + p.eta * a3;
    *dst = o;
  }
  if (blockIdx.x == 0 && (threadIdx.x & 15) == 0) st.bvec[u * p.dM + m] = p.lambda * st.bvec[u * p.dM + m] + p.eta * sq;
}

// a4 per (sequence, KV head): the k-th hole below the budget receives the k-th retained entry above it (K, V,
// position, score).  After the assembly has read the evicted slots.  grid = (Hkv, n_seq), block = 256.
__global__ void k_ph_move(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int h = blockIdx.x, i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(max(st.ctr[u * CTR_STRIDE + CTR_NEVICT], 0), p.tail);
  const int nh = min(sc.hnhole[(size_t)i * p.Hkv + h], ne);
  if (nh <= 0) return;
  const int32_t* evs = st.hev_slot + (u * p.Hkv + h) * (size_t)p.tail;
  const int32_t* surv = sc.hsurv + ((size_t)i * p.Hkv + h) * (size_t)p.tail;
  const size_t r0 = hrow(p, u, h);
  const int dv = p.d / 8;
  for (int k = threadIdx.x; k < nh * dv; k += blockDim.x) {
    const int j = k / dv, c = k % dv;
    reinterpret_cast<uint4*>(st.Kc + (r0 + evs[j]) * p.d)[c] = reinterpret_cast<const uint4*>(st.Kc + (r0 + surv[j]) * p.d)[c];
    reinterpret_cast<uint4*>(st.Vc + (r0 + evs[j]) * p.d)[c] = reinterpret_cast<const uint4*>(st.Vc + (r0 + surv[j]) * p.d)[c];
  }
  for (int j = threadIdx.x; j < nh; j += blockDim.x) {
    st.hpos[r0 + evs[j]] = st.hpos[r0 + surv[j]];
    st.hscore[r0 + evs[j]] = st.hscore[r0 + surv[j]];
  }
}

}  // namespace

#define PH_LAUNCH(stmt)                                  \
  do {                                                   \
    stmt;                                                \
    ++*L.launches;                                       \
    cudaError_t e_ = cudaGetLastError();                 \
    if (e_ != cudaSuccess) return e_;                    \
  } while (0)

cudaError_t im_perhead_prepare(const ImDims& p) {
  return cudaFuncSetAttribute(k_ph_group, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_PH_MAX_PAIRS * 8);
}

// append (and commit the counters of) the call's tokens
cudaError_t im_ph_launch_append(const ImLaunch& L, const ImCall& call, const void* k, const void* v) {
  PH_LAUNCH((k_ph_append<<<dim3(call.C, call.n_seq), 128, 0, L.stream>>>(L.p, L.st, call, (const bf16*)k, (const bf16*)v)));
  PH_LAUNCH((k_ph_commit<<<call.n_seq, 32, 0, L.stream>>>(L.p, L.st, call)));
  return cudaSuccess;
}

// the compression of the call: scores from the caller (if any), selection per head, the rows of the memory write
// (grouping + assembly; phi and the write itself follow in the caller, which owns the GEMM), hole filling.
// ne_max: the largest evicted count per head among the call's sequences (host mirror).
cudaError_t im_ph_launch_select(const ImLaunch& L, const ImCall& call, const float* ext, long long n_pos) {
  const ImDims& p = L.p;
  if (ext) PH_LAUNCH((k_ph_scores_in<<<dim3(p.Hkv, call.n_seq), 256, 0, L.stream>>>(p, L.st, call, ext, n_pos)));
  PH_LAUNCH((k_ph_select<<<dim3(p.Hkv, call.n_seq), 1024, 0, L.stream>>>(p, L.st, L.sc, call)));
  PH_LAUNCH((k_ph_select_commit<<<call.n_seq, 32, 0, L.stream>>>(p, L.st, call)));
  return cudaSuccess;
}

cudaError_t im_ph_launch_assemble(const ImLaunch& L, const ImCall& call, int ne_max) {
  const ImDims& p = L.p;
  const int N = ne_max * p.Hkv;
  int NP = 2;
  while (NP < N) NP <<= 1;
  PH_LAUNCH((k_ph_group<<<call.n_seq, 1024, (size_t)NP * 8, L.stream>>>(p, L.st, L.sc, call, NP)));
  PH_LAUNCH((k_ph_assemble<<<dim3(N, call.n_seq), 128, 0, L.stream>>>(p, L.st, L.sc, call, 1)));
  PH_LAUNCH((k_ph_assemble<<<dim3(N, call.n_seq), 128, 0, L.stream>>>(p, L.st, L.sc, call, 0)));
  return cudaSuccess;
}

cudaError_t im_ph_launch_mem_write(const ImLaunch& L, const ImCall& call) {
  const ImDims& p = L.p;
  dim3 grid((p.Dkv + 63) / 64, (p.dM + 15) / 16, call.n_seq);
  PH_LAUNCH((k_ph_mem_write<<<grid, 256, 0, L.stream>>>(p, L.st, L.sc, call)));
  return cudaSuccess;
}

cudaError_t im_ph_launch_move(const ImLaunch& L, const ImCall& call) {
  PH_LAUNCH((k_ph_move<<<dim3(L.p.Hkv, call.n_seq), 256, 0, L.stream>>>(L.p, L.st, L.sc, call)));
  return cudaSuccess;
}

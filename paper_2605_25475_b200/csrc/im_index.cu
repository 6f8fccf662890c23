// Indexer side of the path: projections (a0), append, indexer scores pooled by max (a1), budgeted
// selection (a2), plus weight initialisation.  Symbols follow Sec. 3.1 of the paper.
#include "im_internal.cuh"
#include "im_select.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();

// RMSNorm of one token's raw q features per indexer head, in place, and alpha = G x / sqrt(H_I d_I)
// (Sec. 3.1).  Executed by one warp; lanes stride over heads.
__device__ void finalize_features(const ImDims& p, float* raw, int lane) {
  const ImRows r = im_rows(p);
  for (int h = lane; h < p.HI; h += 32) {
    float* y = raw + r.uq + h * p.dI;
    float ms = 0.f;
    for (int i = 0; i < p.dI; ++i) ms = fmaf(y[i], y[i], ms);
    const float inv = 1.0f / sqrtf(ms / (float)p.dI + p.norm_eps);
    for (int i = 0; i < p.dI; ++i) y[i] *= inv;
  }
  const float gs = 1.0f / sqrtf((float)p.HI * (float)p.dI);
  for (int h = lane; h < p.HI; h += 32) raw[r.g + h] *= gs;
}

// A_{s,t} = sum_h alpha_h * act(q_h . k_t)   (Sec. 3.1), q/alpha in shared memory, k in registers
__device__ __forceinline__ float index_score(const ImDims& p, const float* __restrict__ qf,
                                             const float* __restrict__ alpha, const float* __restrict__ k) {
  float A = 0.f;
  for (int h = 0; h < p.HI; ++h) {
    float z = 0.f;
    for (int i = 0; i < p.dI; ++i) z = fmaf(qf[h * p.dI + i], k[i], z);
    if (p.act == 0) z = fmaxf(z, 0.f);
    A = fmaf(alpha[h], z, A);
  }
  return A;
}

// prefill: finalise the features of every chunk token, append K/V/kidx/pos.
// grid = (C, n_seq), block = 128.  The counters are advanced by k_prefill_commit (CTR_NNEXT keeps the old count).
__global__ void k_prefill_append(ImDims p, ImState st, ImScratch sc, ImCall call, const bf16* __restrict__ K,
                                 const bf16* __restrict__ V) {
  const int c = blockIdx.x, i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = ctr[CTR_N], T = ctr[CTR_T];
  const int tid = threadIdx.x;
  if (n < 0 || n + call.C > p.cap) {
    if (tid == 0 && c == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  // the entry count of before the chunk, for the kernels that form the chunk's layer outputs while the counters advance
  if (tid == 0 && c == 0) st.ctr[u * CTR_STRIDE + CTR_NNEXT] = n;
  const ImRows r = im_rows(p);
  float* raw = sc.raw + ((size_t)i * call.C + c) * p.R3;
  const bool follow = call.lead >= 0;  // the layer reuses another layer's scores: no indexer features, no indexer key
  if (tid < 32 && !follow) finalize_features(p, raw, tid);
  __syncthreads();
  if (call.pack && !follow) {
    // operand record of the tensor-core scoring: the token's features as three bf16 terms (their sum is the
    // float32 value to 2^-24), each 16-byte row (8 features of one head slot) at its place in the
    // shared-memory layout of a K-major operand without swizzle; alpha follows the three terms
    const int n_qt = (call.C + IM_TC_QT - 1) / IM_TC_QT;
    uint8_t* rec = sc.qpack + ((size_t)i * n_qt + c / IM_TC_QT) * IM_TC_TILE_BYTES;
    const int sq = c % IM_TC_QT;
    if (tid < 48) {
      const int term = tid >> 4, kg = (tid >> 3) & 1, h = tid & 7;
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      if (h < p.HI && kg * 8 < p.dI) {
        const float* y = raw + r.uq + h * p.dI + kg * 8;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float x0 = y[j];
          const bf16 t0 = __float2bfloat16_rn(x0);
          const float x1 = x0 - __bfloat162float(t0);
          const bf16 t1 = __float2bfloat16_rn(x1);
          const bf16 t2 = __float2bfloat16_rn(x1 - __bfloat162float(t1));
          const bf16 t = term == 0 ? t0 : (term == 1 ? t1 : t2);
          w[j >> 1] |= (uint32_t)__bfloat16_as_ushort(t) << (16 * (j & 1));
        }
      }
      *reinterpret_cast<uint4*>(rec + term * (IM_TC_QT * IM_TC_HP * 32) + sq * 256 + kg * 128 + h * 16) =
          make_uint4(w[0], w[1], w[2], w[3]);
    } else if (tid >= 64 && tid < 64 + IM_TC_HP) {
      const int h = tid - 64;
      reinterpret_cast<float*>(rec + 3 * (IM_TC_QT * IM_TC_HP * 32))[sq * IM_TC_HP + h] = h < p.HI ? raw[r.g + h] : 0.f;
    }
  }
  const int slot = n + c;
  bf16* kid = st.kidx + (u * p.cap + slot) * p.dI;
  // k = bf16(RMSNorm(U_k x)) from the float64 projection (one K split in prefill)
  if (!follow && tid >= 32 && tid < 32 + p.dI) {
    const double* ud = sc.keyp + ((size_t)i * call.C + c) * p.dI;
    double ms = 0.0;
    for (int j = 0; j < p.dI; ++j) ms += ud[j] * ud[j];
    const double inv = 1.0 / sqrt(ms / (double)p.dI + (double)p.norm_eps);
    kid[tid - 32] = __double2bfloat16(ud[tid - 32] * inv);
  }
  const int dv = p.d / 8;
  for (int k = tid; k < p.Hkv * dv; k += blockDim.x) {
    const int h = k / dv, cc = k % dv;
    const size_t src = ((size_t)i * call.C + c) * p.Dkv + h * p.d;
    const size_t row = ((u * p.Hkv + h) * p.cap + slot) * p.d;
    reinterpret_cast<uint4*>(st.Kc + row)[cc] = reinterpret_cast<const uint4*>(K + src)[cc];
    reinterpret_cast<uint4*>(st.Vc + row)[cc] = reinterpret_cast<const uint4*>(V + src)[cc];
  }
  if (tid == 0) {
    st.pos[u * p.cap + slot] = T + c;
    st.imp[u * p.cap + slot] = NEG_INF;
  }
}

// prefill a1: imp_t = max(imp_t, max over chunk queries s with pos_s >= pos_t of A_{s,t}).
// grid = (ceil(n_max / 32), n_seq), block = 256 = 32 entries x 8 query lanes.
constexpr int PS_QT = 32;  // queries staged per tile
__global__ void k_prefill_score(ImDims p, ImState st, ImScratch sc, ImCall call) {
  extern __shared__ float smem[];
  const int nq = p.HI * p.dI;
  float* s_q = smem;                       // [PS_QT][nq]
  float* s_a = s_q + PS_QT * nq;           // [PS_QT][HI]
  float* s_max = s_a + PS_QT * p.HI;       // [8][32]
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n0 = ctr[CTR_N], T = ctr[CTR_T];
  const int n1 = n0 + call.C;
  if (n0 < 0 || n1 > p.cap) return;  // flagged by the append kernel
  const int e0 = blockIdx.x * 32;
  if (e0 >= n1) return;
  const int el = threadIdx.x & 31, ql = threadIdx.x >> 5;
  const int e = e0 + el;
  const bool live = e < n1;
  const ImRows r = im_rows(p);
  float kk[64];
  int epos = 0x7fffffff;
  if (live) {
    const bf16* row = st.kidx + (u * p.cap + e) * p.dI;
    for (int k = 0; k < p.dI; ++k) kk[k] = __bfloat162float(row[k]);
    epos = st.pos[u * p.cap + e];
  } else {
    for (int k = 0; k < p.dI; ++k) kk[k] = 0.f;
  }
  float best = NEG_INF;
  bool bad = false;
  // queries before the oldest entry of this block cannot see it: skip whole tiles
  int min_pos = epos;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) min_pos = min(min_pos, __shfl_xor_sync(0xffffffffu, min_pos, o));
  int c_first = max(0, min_pos - T);
  c_first = (c_first / PS_QT) * PS_QT;
  for (int c0 = c_first; c0 < call.C; c0 += PS_QT) {
    const int cn = min(PS_QT, call.C - c0);
    __syncthreads();
    for (int k = threadIdx.x; k < cn * nq; k += blockDim.x) {
      const int cc = k / nq, j = k % nq;
      s_q[cc * nq + j] = sc.raw[((size_t)i * call.C + c0 + cc) * p.R3 + r.uq + j];
    }
    for (int k = threadIdx.x; k < cn * p.HI; k += blockDim.x) {
      const int cc = k / p.HI, j = k % p.HI;
      s_a[cc * p.HI + j] = sc.raw[((size_t)i * call.C + c0 + cc) * p.R3 + r.g + j];
    }
    __syncthreads();
    if (live) {
      for (int cc = ql; cc < cn; cc += 8) {
        if (T + c0 + cc < epos) continue;  // causal mask
        const float A = index_score(p, s_q + cc * nq, s_a + cc * p.HI, kk);
        bad |= !isfinite(A);
        best = fmaxf(best, A);
      }
    }
  }
  __syncthreads();
  s_max[ql * 32 + el] = best;
  __syncthreads();
  if (ql == 0 && live) {
    for (int k = 1; k < 8; ++k) best = fmaxf(best, s_max[k * 32 + el]);
    st.imp[u * p.cap + e] = fmaxf(st.imp[u * p.cap + e], best);
  }
  if (bad) atomicOr(st.status, ST_NONFINITE);
}

// advance the counters after the chunk has been appended and scored.  grid = n_seq, block = 32.
__global__ void k_prefill_commit(ImDims p, ImState st, ImCall call) {
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  if (threadIdx.x == 0) {
    const int n0 = ctr[CTR_N];
    if (n0 < 0 || n0 + call.C > p.cap) return;
    ctr[CTR_N] = n0 + call.C;
    ctr[CTR_T] = ctr[CTR_T] + call.C;
    ctr[CTR_NEVICT] = 0;
  }
}

// A layer that reuses the scores of the leading layer of its group (App. B, IndexCache-style reuse): its pooled
// importances are those the leading layer's latest selection saw, slot by slot.  The two layers have made the same
// calls, so their slot layouts agree; the kernel checks it position by position (ST_LAYOUT otherwise).
// grid = n_seq, block = 256; after k_prefill_commit (CTR_N counts the appended chunk).
__global__ void k_follow_scores(ImDims p, ImState st, ImCall call) {
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  const size_t ul = (size_t)call.lead * p.S + call.seq[blockIdx.x];
  const int n = st.ctr[u * CTR_STRIDE + CTR_N];
  if (n < 0 || n > p.cap) return;  // flagged elsewhere
  bool bad = n != st.ctr[ul * CTR_STRIDE + CTR_NSEL];
  for (int t = threadIdx.x; t < n && !bad; t += blockDim.x) {
    bad |= st.sel_pos[ul * p.cap + t] != st.pos[u * p.cap + t];
    st.imp[u * p.cap + t] = st.sel_imp[ul * p.cap + t];
  }
  if (bad) atomicOr(st.status, ST_LAYOUT);
}

// Compression of every sequence in the call (Sec. 4 schedule): restart pooling; if over budget,
// flag the retained entries and list the evicted slots in ascending slot order.
// grid = n_seq, block = 1024.
__global__ void k_select(ImDims p, ImState st, ImScratch sc, ImCall call) {
  __shared__ SelectShared sh;
  __shared__ int s_tmp[33];
  const size_t u = (size_t)call.layer * p.S + call.seq[blockIdx.x];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const int n = ctr[CTR_N];
  float* imp = st.imp + u * p.cap;
  const int32_t* pos = st.pos + u * p.cap;
  uint8_t* keep = st.keep + u * p.cap;
  if (n < 0 || n > p.cap) {
    if (threadIdx.x == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  int ne = 0;
  if (threadIdx.x == 0) sc.nhole[blockIdx.x] = 0;
  // keep what the selection saw (debug/parity export)
  for (int t = threadIdx.x; t < n; t += blockDim.x) {
    st.sel_pos[u * p.cap + t] = pos[t];
    st.sel_imp[u * p.cap + t] = imp[t];
  }
  if (n > p.B) {
    ne = n - p.B;
    const uint64_t thr = block_kth_largest_key(imp, pos, n, p.B, p.n_sink, &sh);
    // ordered list of the evicted slots: each thread owns a contiguous run of slots
    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int t0 = min(n, (int)threadIdx.x * per), t1 = min(n, t0 + per);
    int cnt = 0;
    for (int t = t0; t < t1; ++t) {
      const bool k = im_select_key(imp[t], pos[t], p.n_sink) >= thr;
      keep[t] = k ? 1 : 0;
      cnt += k ? 0 : 1;
    }
    int off;
    const int total = block_exclusive_scan(cnt, &off, s_tmp);
    if (total != ne && threadIdx.x == 0) atomicOr(st.status, ST_COUNT);
    int32_t* evs = st.ev_slot + u * p.tail;
    int32_t* evp = st.ev_pos + u * p.tail;
    for (int t = t0; t < t1; ++t)
      if (!keep[t] && off < p.tail) {
        evs[off] = t;
        evp[off] = pos[t];
        ++off;
      }
    __syncthreads();
    // retained entries at or above the budget, ascending: they fill the evicted slots below it
    const int tl = n - p.B;  // == ne slots in [B, n)
    const int per2 = (tl + blockDim.x - 1) / blockDim.x;
    const int a0 = min(tl, (int)threadIdx.x * per2), a1 = min(tl, a0 + per2);
    int cnt2 = 0;
    for (int t = a0; t < a1; ++t) cnt2 += keep[p.B + t] ? 1 : 0;
    int off2;
    const int nh = block_exclusive_scan(cnt2, &off2, s_tmp);
    int32_t* surv = sc.surv + (size_t)blockIdx.x * p.tail;
    for (int t = a0; t < a1; ++t)
      if (keep[p.B + t]) surv[off2++] = p.B + t;
    if (threadIdx.x == 0) sc.nhole[blockIdx.x] = nh;
    __syncthreads();
  }
  for (int t = threadIdx.x; t < n; t += blockDim.x) imp[t] = NEG_INF;
  if (threadIdx.x == 0) {
    ctr[CTR_SINCE] = 0;
    ctr[CTR_NSEL] = n;
    ctr[CTR_NEVICT] = ne;
    ctr[CTR_N] = n - ne;  // the gather / move kernels that follow work from the lists, not from the count
    if (ne > 0) ctr[CTR_EVSTEPS] = ctr[CTR_EVSTEPS] + 1;
  }
}

// Row-generic selection without a context.  grid = rows, block = 256.
__global__ void k_topb(const float* __restrict__ scores, const int32_t* __restrict__ pos, int n, int B, int n_sink,
                       uint8_t* __restrict__ keep, int32_t* __restrict__ n_evict) {
  __shared__ SelectShared sh;
  const size_t row = blockIdx.x;
  const float* s = scores + row * n;
  const int32_t* ps = pos + row * n;
  uint8_t* k = keep + row * n;
  if (n <= B) {
    for (int t = threadIdx.x; t < n; t += blockDim.x) k[t] = 1;
    if (threadIdx.x == 0) n_evict[row] = 0;
    return;
  }
  if (B == 0) {
    for (int t = threadIdx.x; t < n; t += blockDim.x) k[t] = 0;
    if (threadIdx.x == 0) n_evict[row] = n;
    return;
  }
  const uint64_t thr = block_kth_largest_key(s, ps, n, B, n_sink, &sh);
  for (int t = threadIdx.x; t < n; t += blockDim.x) k[t] = im_select_key(s[t], ps[t], n_sink) >= thr ? 1 : 0;
  if (threadIdx.x == 0) n_evict[row] = n - B;
}

// ------------------------------------------------------------------------------------------------
// Seeded N(0, std^2) bf16 init: counter-based (splitmix64 of (seed, layer, tensor, index)) + Box-Muller.
__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
__global__ void k_init_normal(bf16* __restrict__ dst, size_t n, uint64_t key, float std) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t r = splitmix64(key ^ splitmix64(i));
  const float u1 = ((float)((r >> 40) + 1)) * (1.0f / 16777216.0f);   // (0, 1]
  const float u2 = ((float)((r >> 8) & 0xFFFFFFu)) * (1.0f / 16777216.0f);
  const float z = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
  dst[i] = __float2bfloat16_rn(z * std);
}

// Wfold[m][g*d + c] = sum over the query heads j of group g of Wt[m][j*d + c]   (float32)
__global__ void k_fold_theta(ImDims p, const bf16* __restrict__ Wt, bf16* __restrict__ Wfh, bf16* __restrict__ Wfl) {
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)p.dM * p.Dkv) return;
  const int m = (int)(idx / p.Dkv), col = (int)(idx % p.Dkv);
  const int g = col / p.d, c = col % p.d;
  float s = 0.f;
  for (int j = g * p.Gq; j < (g + 1) * p.Gq; ++j) s += __bfloat162float(Wt[(size_t)m * p.D + j * p.d + c]);
  const bf16 hi = __float2bfloat16_rn(s);
  Wfh[idx] = hi;
  Wfl[idx] = __float2bfloat16_rn(s - __bfloat162float(hi));
}

}  // namespace

// ------------------------------------------------------------------------------------------------ launchers
cudaError_t im_launch_prefill_append(const ImLaunch& L, const ImCall& call, const void* k, const void* v) {
  dim3 grid(call.C, call.n_seq);
  k_prefill_append<<<grid, 128, 0, L.stream>>>(L.p, L.st, L.sc, call, (const bf16*)k, (const bf16*)v);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_prefill_score(const ImLaunch& L, const ImCall& call, int n_max) {
  dim3 grid((n_max + 31) / 32, call.n_seq);
  const size_t smem = ((size_t)PS_QT * (L.p.HI * L.p.dI + L.p.HI) + 256) * 4;
  k_prefill_score<<<grid, 256, smem, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_follow_scores(const ImLaunch& L, const ImCall& call) {
  k_follow_scores<<<call.n_seq, 256, 0, L.stream>>>(L.p, L.st, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_prefill_commit(const ImLaunch& L, const ImCall& call) {
  k_prefill_commit<<<call.n_seq, 32, 0, L.stream>>>(L.p, L.st, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_select(const ImLaunch& L, const ImCall& call) {
  k_select<<<call.n_seq, 1024, 0, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_topb(const float* scores, const int32_t* pos, int rows, int n, int budget, int n_sink,
                           uint8_t* keep, int32_t* n_evict, cudaStream_t stream) {
  k_topb<<<rows, 256, 0, stream>>>(scores, pos, n, budget, n_sink, keep, n_evict);
  return cudaGetLastError();
}

cudaError_t im_launch_init_weights(const ImDims& p, const ImWeights& w, int layer, uint64_t seed, float std,
                                   cudaStream_t stream) {
  struct T { bf16* ptr; size_t n; } ts[5] = {{w.Uq, (size_t)p.HI * p.dI * p.D}, {w.Uk, (size_t)p.dI * p.D},
                                             {w.G, (size_t)p.HI * p.D}, {w.Wt, (size_t)p.dM * p.D}, {w.wg, (size_t)p.D}};
  for (int t = 0; t < 5; ++t) {
    const uint64_t key = seed * 0x9E3779B97F4A7C15ull + ((uint64_t)layer << 8) + (uint64_t)t;
    k_init_normal<<<(unsigned)((ts[t].n + 255) / 256), 256, 0, stream>>>(ts[t].ptr, ts[t].n, key, std);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaMemsetAsync(w.bg, 0, 4, stream);
}

cudaError_t im_launch_fold_theta(const ImDims& p, const ImWeights& w, cudaStream_t stream) {
  const size_t n = (size_t)p.dM * p.Dkv;
  k_fold_theta<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(p, w.Wt, w.Wfh, w.Wfl);
  return cudaGetLastError();
}

// Decode front end of one layer call, one thread block per sequence: finish the indexer features
// from the K-split projection partials, append the token, score every cached entry with the new
// query (a1), and - when the compression is due and small - select (a2), gather the evicted pairs
// for the memory write and compact the cache (a4) in the same kernel.  Also the stand-alone gather
// and move kernels used after k_select when the evicted set is large (prefill).
#include "im_internal.cuh"

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int FRONT_THREADS = 512;

struct FrontShared {
  double kd[64];             // indexer key before normalisation (float64)
  float alpha[64];
  float knew[64];            // the new token's cached (rounded) indexer key
  unsigned long long wmin[FRONT_THREADS / 32];
  int wslot[FRONT_THREADS / 32];
  int ev[IM_FRONT_MAX_NE];   // evicted slots, ascending after the sort
  int evpos[IM_FRONT_MAX_NE];// their positions
  int surv[IM_FRONT_MAX_NE]; // retained entries found at or above the budget, ascending
  int nh;
};

// grid = n_seq, block = FRONT_THREADS, dynamic smem = keys of the selection (8 bytes per entry) when
// do_select (`key_slots` of them), followed by the q features [HI][dI] (float32).
template <int DI>  // d_I known at compile time (8, 16) keeps the key and the dot products in registers; 0: generic
__global__ void __maxnreg__(80)
k_decode_front(ImDims p, ImState st, ImScratch sc, ImCall call, const bf16* __restrict__ k_new,
               const bf16* __restrict__ v_new, int do_select, int key_slots) {
  extern __shared__ __align__(16) unsigned long long s_key[];
  __shared__ FrontShared sh;
  // a kernel launched as programmatic dependent of this one (phi of the evicted keys) may request its weights now
  asm volatile("griddepcontrol.launch_dependents;");
  float* s_q = reinterpret_cast<float*>(s_key + key_slots);                         // [HI][dI], 16-byte aligned
  double* s_pk = reinterpret_cast<double*>(s_q + ((p.HI * p.dI + 3) & ~3));         // [ksplit_key][dI] key partials
  float* s_pf = reinterpret_cast<float*>(s_pk + IM_KSPLIT_KEY * p.dI);              // [ksplit][HI dI + HI] partials
  const int i = blockIdx.x, tid = threadIdx.x;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  int32_t* ctr = st.ctr + u * CTR_STRIDE;
  const ImRows r = im_rows(p);
  const int nq = p.HI * p.dI;
  const int dI = DI > 0 ? DI : p.dI;
  float* imp = st.imp + u * p.cap;
  int32_t* pos = st.pos + u * p.cap;
  // A layer that reuses the scores of the leading layer of its group (App. B) computes no indexer features and caches
  // no indexer key: the pooled importances are those the leading layer's selection saw in this step, slot by slot.
  const bool follow = call.lead >= 0;
  const size_t ul = follow ? (size_t)call.lead * p.S + call.seq[i] : u;
  IM_MARK(sc, call.layer, 0, 0);
  // ---- issue the loads of the first batch of cached entries (they depend on nothing of this call)
  constexpr int EPT = 4;
  int n_lim = p.cap;  // entries a batch may read: the capacity until the count is known
  uint4 kraw[EPT][DI > 0 ? DI / 8 : 1];
  float imp_old[EPT];
  int pos_old[EPT];
  auto load_batch = [&](int b0) {
#pragma unroll
    for (int e = 0; e < EPT; ++e) {
      const int t = b0 + e * FRONT_THREADS + tid;
      imp_old[e] = NEG_INF;
      pos_old[e] = 0;
      if (t < n_lim) {  // (entries at or beyond the count are read but never used; slot n is the token being appended)
        if (DI > 0 && !follow) {
          const uint4* row = reinterpret_cast<const uint4*>(st.kidx + (u * p.cap + t) * dI);
#pragma unroll
          for (int c = 0; c < (DI > 0 ? DI / 8 : 1); ++c) kraw[e][c] = im_ld_now_u4(row + c);
        }
        imp_old[e] = follow ? NEG_INF : im_ld_now_f32(imp + t);
        pos_old[e] = im_ld_now_s32(pos + t);
      }
    }
  };
  // the first batch goes out before the entry count is known: its addresses do not depend on it
  load_batch(0);
  const int n = ctr[CTR_N], T = ctr[CTR_T], since = ctr[CTR_SINCE];
  if (n < 0 || n >= p.cap) {  // never write out of bounds: flag and leave
    if (tid == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  n_lim = n;
  IM_MARK(sc, call.layer, 0, 1);
  // the new token's K / V rows (copied into slot n below): requested now, stored after the first barrier
  const int dv = p.d / 8;
  const bool kv_here = tid < p.Hkv * dv;
  uint4 knew_c = make_uint4(0u, 0u, 0u, 0u), vnew_c = knew_c;
  if (kv_here) {
    const int h = tid / dv, c = tid % dv;
    knew_c = reinterpret_cast<const uint4*>(k_new + (size_t)i * p.Dkv + h * p.d)[c];
    vnew_c = reinterpret_cast<const uint4*>(v_new + (size_t)i * p.Dkv + h * p.d)[c];
  }
  // ---- finish the projections: sum the K-split partials in a fixed order.  Launched as programmatic dependent of
  // the projection kernel this block may have come this far while that kernel still runs: wait for its partial sums.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  IM_MARK(sc, call.layer, 0, 2);
  if (!follow) {
    // every partial is requested before the first one is used (one memory round trip), staged in shared memory,
    // then added in K-split order
    const int nrow = nq + p.HI, n_pf = call.ksplit * nrow, n_pk = call.ksplit_key * p.dI;
    auto raw_at = [&](int k) {
      const int ks = k / nrow, row = k % nrow;
      return sc.raw[((size_t)ks * call.n_seq + i) * p.R5 + (row < nq ? r.uq + row : r.g + (row - nq))];
    };
    auto key_at = [&](int k) { return sc.keyp[((size_t)(k / p.dI) * call.n_seq + i) * p.dI + k % p.dI]; };
    for (int k0 = tid; k0 < max(n_pf, n_pk); k0 += 2 * FRONT_THREADS) {
      const int k1 = k0 + FRONT_THREADS;
      const float f0 = k0 < n_pf ? raw_at(k0) : 0.f, f1 = k1 < n_pf ? raw_at(k1) : 0.f;
      const double d0 = k0 < n_pk ? key_at(k0) : 0.0, d1 = k1 < n_pk ? key_at(k1) : 0.0;
      if (k0 < n_pf) s_pf[k0] = f0;
      if (k1 < n_pf) s_pf[k1] = f1;
      if (k0 < n_pk) s_pk[k0] = d0;
      if (k1 < n_pk) s_pk[k1] = d1;
    }
    __syncthreads();
    for (int k = tid; k < nrow; k += FRONT_THREADS) {
      float v = 0.f;
      for (int ks = 0; ks < call.ksplit; ++ks) v += s_pf[ks * nrow + k];
      if (k < nq) s_q[k] = v;
      else sh.alpha[k - nq] = v * (1.0f / sqrtf((float)p.HI * (float)p.dI));
    }
    for (int k = tid; k < p.dI; k += FRONT_THREADS) {
      double v = 0.0;
      for (int ks = 0; ks < call.ksplit_key; ++ks) v += s_pk[ks * p.dI + k];
      sh.kd[k] = v;
    }
  }
  __syncthreads();
  // RMSNorm of the q features per indexer head (float32) and of the key (float64, then bf16)
  for (int h = tid; h < (follow ? 0 : p.HI); h += FRONT_THREADS) {
    float* y = s_q + h * p.dI;
    float ms = 0.f;
    for (int k = 0; k < p.dI; ++k) ms = fmaf(y[k], y[k], ms);
    const float inv = 1.0f / sqrtf(ms / (float)p.dI + p.norm_eps);
    for (int k = 0; k < p.dI; ++k) y[k] *= inv;
  }
  if (!follow && tid >= 64 && tid < 64 + p.dI) {
    const int k = tid - 64;
    double ms = 0.0;
    for (int j = 0; j < p.dI; ++j) ms += sh.kd[j] * sh.kd[j];
    const double inv = 1.0 / sqrt(ms / (double)p.dI + (double)p.norm_eps);
    const bf16 b = __double2bfloat16(sh.kd[k] * inv);
    st.kidx[(u * p.cap + n) * p.dI + k] = b;
    sh.knew[k] = __bfloat162float(b);
  }
  // ---- append K / V / position in slot n
  if (kv_here) {
    const int h = tid / dv, c = tid % dv;
    const size_t row = ((u * p.Hkv + h) * p.cap + n) * p.d;
    reinterpret_cast<uint4*>(st.Kc + row)[c] = knew_c;
    reinterpret_cast<uint4*>(st.Vc + row)[c] = vnew_c;
  }
  for (int k = tid + FRONT_THREADS; k < p.Hkv * dv; k += FRONT_THREADS) {  // (more chunks than threads)
    const int h = k / dv, c = k % dv;
    const size_t row = ((u * p.Hkv + h) * p.cap + n) * p.d;
    reinterpret_cast<uint4*>(st.Kc + row)[c] = reinterpret_cast<const uint4*>(k_new + (size_t)i * p.Dkv + h * p.d)[c];
    reinterpret_cast<uint4*>(st.Vc + row)[c] = reinterpret_cast<const uint4*>(v_new + (size_t)i * p.Dkv + h * p.d)[c];
  }
  if (tid == 0) st.pos[u * p.cap + n] = T;
  __syncthreads();
  IM_MARK(sc, call.layer, 0, 4);
  // ---- a1: A_t = sum_h alpha_h act(q_h . k_t), pooled by max into the importance.
  // Entries are handled in batches of EPT per thread; the loads of a batch are all issued before its
  // arithmetic (the first batch was issued before the feature finalisation above).
  const int n1 = n + 1;
  const bool due = (since + 1 == p.tau);
  const bool select_here = do_select && due;
  bool bad = false, layout_bad = false;
  for (int b0 = 0; b0 < n1; b0 += EPT * FRONT_THREADS) {
    if (b0 > 0) load_batch(b0);
    auto publish = [&](int e, int t, float pooled) {  // what the selection sees (parity export), then the pooling restarts
      const int ps = (t == n) ? T : pos_old[e];
      if (due) {
        st.sel_pos[u * p.cap + t] = ps;
        st.sel_imp[u * p.cap + t] = pooled;
      }
      if (select_here) {
        s_key[t] = im_select_key(pooled, ps, p.n_sink);
        imp[t] = NEG_INF;
      } else {
        imp[t] = pooled;
      }
    };
    if (follow) {
#pragma unroll
      for (int e = 0; e < EPT; ++e) {
        const int t = b0 + e * FRONT_THREADS + tid;
        if (t >= n1) continue;
        // the leading layer scored the same entries in the same slots (checked: same position in the same slot)
        const int ps = (t == n) ? T : pos_old[e];
        if (due) {
          const float pooled = st.sel_imp[ul * p.cap + t];
          if (st.sel_pos[ul * p.cap + t] != ps) layout_bad = true;
          publish(e, t, pooled);
        }
      }
      continue;
    }
    // two entries at a time: a head's query features are read from shared memory once (as 16-byte words) for both
#pragma unroll
    for (int e0 = 0; e0 < EPT; e0 += 2) {
      constexpr int KD = DI > 0 ? DI : 64;
      float kk[2][KD];
      int tt[2];
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int e = e0 + j, t = b0 + e * FRONT_THREADS + tid;
        tt[j] = t;
        if (t == n) {
#pragma unroll
          for (int k = 0; k < dI; ++k) kk[j][k] = sh.knew[k];
        } else if (DI > 0) {
#pragma unroll
          for (int c = 0; c < (DI > 0 ? DI / 8 : 1); ++c) {
            const uint32_t ww[4] = {kraw[e][c].x, kraw[e][c].y, kraw[e][c].z, kraw[e][c].w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              kk[j][c * 8 + 2 * k] = __uint_as_float(ww[k] << 16);
              kk[j][c * 8 + 2 * k + 1] = __uint_as_float(ww[k] & 0xffff0000u);
            }
          }
        } else if (t < n1) {
          const bf16* row = st.kidx + (u * p.cap + t) * dI;
          for (int k = 0; k < dI; ++k) kk[j][k] = __bfloat162float(row[k]);
        }
      }
      if (tt[0] >= n1) continue;  // (then tt[1] >= n1 as well)
      if (b0 == 0) IM_MARK(sc, call.layer, 0, 10 + e0);
      float A[2] = {0.f, 0.f};
      for (int h = 0; h < p.HI; ++h) {
        float z[2] = {0.f, 0.f};
        if (DI > 0) {
          const float4* q4 = reinterpret_cast<const float4*>(s_q + h * dI);
#pragma unroll
          for (int c = 0; c < (DI > 0 ? DI / 4 : 1); ++c) {
            const float4 qv = q4[c];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              z[j] = fmaf(qv.x, kk[j][4 * c], z[j]);
              z[j] = fmaf(qv.y, kk[j][4 * c + 1], z[j]);
              z[j] = fmaf(qv.z, kk[j][4 * c + 2], z[j]);
              z[j] = fmaf(qv.w, kk[j][4 * c + 3], z[j]);
            }
          }
        } else {
          for (int k = 0; k < dI; ++k) {
            const float qv = s_q[h * dI + k];
            z[0] = fmaf(qv, kk[0][k], z[0]);
            z[1] = fmaf(qv, kk[1][k], z[1]);
          }
        }
        const float al = sh.alpha[h];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          if (p.act == 0) z[j] = fmaxf(z[j], 0.f);
          A[j] = fmaf(al, z[j], A[j]);
        }
      }
      if (b0 == 0) IM_MARK(sc, call.layer, 0, 11 + e0);
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int e = e0 + j, t = tt[j];
        if (t >= n1) continue;
        bad |= !isfinite(A[j]);
        publish(e, t, fmaxf((t == n) ? NEG_INF : imp_old[e], A[j]));
      }
    }
  }
  if (bad) atomicOr(st.status, ST_NONFINITE);
  if (layout_bad) atomicOr(st.status, ST_LAYOUT);
  IM_MARK(sc, call.layer, 0, 5);
  if (!select_here) {
    // either not due, or the selection runs in the kernels that follow (they read imp / pos)
    if (tid == 0) {
      ctr[call.defer ? CTR_NNEXT : CTR_N] = n1;
      ctr[CTR_T] = T + 1;
      ctr[CTR_SINCE] = since + 1;
      ctr[CTR_NEVICT] = 0;
    }
    return;
  }
  __syncthreads();
  // ---- a2: the ne entries with the smallest keys leave (keys are distinct)
  const int ne = n1 > p.B ? n1 - p.B : 0;
  if (ne > IM_FRONT_MAX_NE) {  // the host never asks for this
    if (tid == 0) atomicOr(st.status, ST_COUNT);
    return;
  }
  for (int e = 0; e < ne; ++e) {
    unsigned long long best = ~0ull;
    int slot = -1;
    for (int t = tid; t < n1; t += FRONT_THREADS) {
      const unsigned long long k = s_key[t];
      if (k < best) { best = k; slot = t; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int os = __shfl_xor_sync(0xffffffffu, slot, o);
      if (ob < best) { best = ob; slot = os; }
    }
    if ((tid & 31) == 0) { sh.wmin[tid >> 5] = best; sh.wslot[tid >> 5] = slot; }
    __syncthreads();
    if (tid == 0) {
      for (int w = 1; w < FRONT_THREADS / 32; ++w)
        if (sh.wmin[w] < best) { best = sh.wmin[w]; slot = sh.wslot[w]; }
      sh.ev[e] = slot;
      sh.evpos[e] = (int)(0xFFFFFFFFu - (uint32_t)best);  // the key's low word is ~position
      s_key[slot] = ~0ull;                                 // taken: the largest possible value
    }
    __syncthreads();
  }
  IM_MARK(sc, call.layer, 0, 6);
  if (tid == 0) {
    // ascending slot order; holes below the budget pair with the retained entries above it
    for (int a = 1; a < ne; ++a) {
      const int v = sh.ev[a], vp = sh.evpos[a];
      int b = a - 1;
      while (b >= 0 && sh.ev[b] > v) { sh.ev[b + 1] = sh.ev[b]; sh.evpos[b + 1] = sh.evpos[b]; --b; }
      sh.ev[b + 1] = v;
      sh.evpos[b + 1] = vp;
    }
    int nh = 0, ns = 0;
    for (int a = 0; a < ne; ++a) nh += sh.ev[a] < p.B ? 1 : 0;
    for (int t = p.B; t < n1; ++t) {
      bool gone = false;
      for (int a = 0; a < ne; ++a) gone |= sh.ev[a] == t;
      if (!gone) sh.surv[ns++] = t;
    }
    if (ns != nh) atomicOr(st.status, ST_COUNT);
    sh.nh = min(nh, ns);
    for (int a = 0; a < ne; ++a) {
      st.ev_slot[u * p.tail + a] = sh.ev[a];
      st.ev_pos[u * p.tail + a] = sh.evpos[a];
    }
    if (call.defer) {  // the moves are made by the merge kernel, after the attention kernel has read the cache
      sc.nhole[i] = sh.nh;
      for (int a = 0; a < sh.nh; ++a) sc.surv[(size_t)i * p.tail + a] = sh.surv[a];
    }
  }
  __syncthreads();
  IM_MARK(sc, call.layer, 0, 7);
  // ---- gather the evicted pairs for the memory write (a3) and, in the same pass, a4: a hole below
  // the budget (the first nh evicted slots) receives the retained entry found above it.  A thread
  // reads the evicted chunk before it overwrites it; the sources of the moves are never written.
  const int nh = call.defer ? 0 : sh.nh;
  for (int k = tid; k < ne * p.Hkv * dv; k += FRONT_THREADS) {
    const int e = k / (p.Hkv * dv), rem = k % (p.Hkv * dv), h = rem / dv, c = rem % dv;
    const size_t base = (u * p.Hkv + h) * p.cap;
    uint4* krow = reinterpret_cast<uint4*>(st.Kc + (base + sh.ev[e]) * p.d) + c;
    uint4* vrow = reinterpret_cast<uint4*>(st.Vc + (base + sh.ev[e]) * p.d) + c;
    const uint4 ke = *krow, ve = *vrow;
    uint4 ks = ke, vs = ve;
    if (e < nh) {
      ks = reinterpret_cast<const uint4*>(st.Kc + (base + sh.surv[e]) * p.d)[c];
      vs = reinterpret_cast<const uint4*>(st.Vc + (base + sh.surv[e]) * p.d)[c];
    }
    const size_t dst = ((size_t)i * p.tail + e) * p.Dkv + h * p.d;
    reinterpret_cast<uint4*>(sc.evK + dst)[c] = ke;
    reinterpret_cast<uint4*>(sc.evV + dst)[c] = ve;
    if (e < nh) { *krow = ks; *vrow = vs; }
  }
  IM_MARK(sc, call.layer, 0, 8);
  for (int k = tid; k < nh * p.dI; k += FRONT_THREADS) {
    const int j = k / p.dI, c = k % p.dI;
    st.kidx[(u * p.cap + sh.ev[j]) * p.dI + c] = st.kidx[(u * p.cap + sh.surv[j]) * p.dI + c];
  }
  for (int j = tid; j < nh; j += FRONT_THREADS) pos[sh.ev[j]] = (sh.surv[j] == n) ? T : pos[sh.surv[j]];
  if (tid == 0) {
    ctr[call.defer ? CTR_NNEXT : CTR_N] = n1 - ne;
    ctr[CTR_T] = T + 1;
    ctr[CTR_SINCE] = 0;
    ctr[CTR_NSEL] = n1;
    ctr[CTR_NEVICT] = ne;
    if (ne > 0) ctr[CTR_EVSTEPS] = ctr[CTR_EVSTEPS] + 1;
  }
  IM_MARK(sc, call.layer, 0, 9);
}

// Stand-alone versions for large evicted sets (after k_select): gather the evicted pairs, then move
// the retained entries from above the budget into the holes.  Two kernels: every gather must be done
// before a move overwrites an evicted slot.
// grid = (ceil(ne_max / 4), n_seq), block = 256.
__global__ void __launch_bounds__(256) k_gather_evicted(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(st.ctr[u * CTR_STRIDE + CTR_NEVICT], p.tail);
  const int e0 = blockIdx.x * 4;
  if (e0 >= ne) return;
  const int cnt = min(4, ne - e0);
  const int dv = p.d / 8;
  for (int k = threadIdx.x; k < cnt * p.Hkv * dv; k += blockDim.x) {
    const int e = e0 + k / (p.Hkv * dv), rem = k % (p.Hkv * dv), h = rem / dv, c = rem % dv;
    const int slot = st.ev_slot[u * p.tail + e];
    const size_t row = ((u * p.Hkv + h) * p.cap + slot) * p.d;
    const size_t dst = ((size_t)i * p.tail + e) * p.Dkv + h * p.d;
    reinterpret_cast<uint4*>(sc.evK + dst)[c] = reinterpret_cast<const uint4*>(st.Kc + row)[c];
    reinterpret_cast<uint4*>(sc.evV + dst)[c] = reinterpret_cast<const uint4*>(st.Vc + row)[c];
  }
}

__global__ void __launch_bounds__(256) k_move_survivors(ImDims p, ImState st, ImScratch sc, ImCall call) {
  const int i = blockIdx.y;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int ne = min(st.ctr[u * CTR_STRIDE + CTR_NEVICT], p.tail);
  if (ne <= 0) return;
  const int nh = min(sc.nhole[i], ne);
  const int j0 = blockIdx.x * 4;
  if (j0 >= nh) return;
  const int cnt = min(4, nh - j0);
  const int dv = p.d / 8;
  const int32_t* evs = st.ev_slot + u * p.tail;
  const int32_t* surv = sc.surv + (size_t)i * p.tail;
  for (int k = threadIdx.x; k < cnt * p.Hkv * dv; k += blockDim.x) {
    const int j = j0 + k / (p.Hkv * dv), rem = k % (p.Hkv * dv), h = rem / dv, c = rem % dv;
    const size_t base = (u * p.Hkv + h) * p.cap;
    reinterpret_cast<uint4*>(st.Kc + (base + evs[j]) * p.d)[c] = reinterpret_cast<const uint4*>(st.Kc + (base + surv[j]) * p.d)[c];
    reinterpret_cast<uint4*>(st.Vc + (base + evs[j]) * p.d)[c] = reinterpret_cast<const uint4*>(st.Vc + (base + surv[j]) * p.d)[c];
  }
  for (int k = threadIdx.x; k < cnt * p.dI; k += blockDim.x) {
    const int j = j0 + k / p.dI, c = k % p.dI;
    st.kidx[(u * p.cap + evs[j]) * p.dI + c] = st.kidx[(u * p.cap + surv[j]) * p.dI + c];
  }
  for (int j = j0 + threadIdx.x; j < j0 + cnt; j += blockDim.x) st.pos[u * p.cap + evs[j]] = st.pos[u * p.cap + surv[j]];
}

}  // namespace

// `started`: an event (timing disabled) that triggers once every block of the kernel has begun to run; a stream that
// waits for it launches its next kernel when this kernel's blocks are resident, not when they have ended.
// `programmatic`: the kernel before this one in the stream releases its dependents early; this kernel's blocks then read
// the cache, the counters and the new token's K / V while it still runs, and wait for it before they read its output.
cudaError_t im_launch_decode_front(const ImLaunch& L, const ImCall& call, const void* k_new, const void* v_new,
                                   int do_select, int n_max, int smem_floor, cudaEvent_t started, int programmatic) {
  static bool attr_done_dev[64] = {};
  bool* attr_done = im_device_flag(attr_done_dev);
  if (!attr_done || !*attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_front<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_SMEM_FRONT);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_decode_front<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_SMEM_FRONT);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(k_decode_front<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, IM_SMEM_FRONT);
    if (e != cudaSuccess) return e;
    if (attr_done) *attr_done = true;
  }
  const int key_slots = do_select ? (n_max + 1) & ~1 : 0;  // (even: what follows the keys is 16-byte aligned)
  size_t smem = (size_t)key_slots * 8 + (size_t)((L.p.HI * L.p.dI + 3) & ~3) * 4 + (size_t)IM_KSPLIT_KEY * L.p.dI * 8 +
                (size_t)IM_KSPLIT * (L.p.HI * L.p.dI + L.p.HI) * 4;
  if (smem < (size_t)smem_floor) smem = (size_t)smem_floor;  // keeps the streaming kernels' blocks off this block's SM
  const bf16* kn = (const bf16*)k_new;
  const bf16* vn = (const bf16*)v_new;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(call.n_seq);
  cfg.blockDim = dim3(FRONT_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = L.stream;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (started) {
    attr[na].id = cudaLaunchAttributeProgrammaticEvent;
    attr[na].val.programmaticEvent.event = started;
    attr[na].val.programmaticEvent.flags = 0;
    attr[na].val.programmaticEvent.triggerAtBlockStart = 1;
    ++na;
  }
  if (programmatic) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  cudaError_t e;
  if (L.p.dI == 16) e = cudaLaunchKernelEx(&cfg, k_decode_front<16>, L.p, L.st, L.sc, call, kn, vn, do_select, key_slots);
  else if (L.p.dI == 8) e = cudaLaunchKernelEx(&cfg, k_decode_front<8>, L.p, L.st, L.sc, call, kn, vn, do_select, key_slots);
  else e = cudaLaunchKernelEx(&cfg, k_decode_front<0>, L.p, L.st, L.sc, call, kn, vn, do_select, key_slots);
  ++*L.launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

// gather of the evicted pairs / move of the retained entries into the holes: every gather must be done before a
// move overwrites an evicted slot (stream order, or an event between the two launches)
cudaError_t im_launch_gather(const ImLaunch& L, const ImCall& call, int ne_max) {
  dim3 grid((ne_max + 3) / 4, call.n_seq);
  k_gather_evicted<<<grid, 256, 0, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}
cudaError_t im_launch_move(const ImLaunch& L, const ImCall& call, int ne_max) {
  dim3 grid((ne_max + 3) / 4, call.n_seq);
  k_move_survivors<<<grid, 256, 0, L.stream>>>(L.p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}
cudaError_t im_launch_gather_move(const ImLaunch& L, const ImCall& call, int ne_max) {
  const cudaError_t e = im_launch_gather(L, call, ne_max);
  return e != cudaSuccess ? e : im_launch_move(L, call, ne_max);
}

cudaError_t im_front_prepare_decode() {
  cudaError_t e = im_prefer_max_smem(k_decode_front<0>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_decode_front<8>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_decode_front<16>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_move_survivors);
  return e;
}

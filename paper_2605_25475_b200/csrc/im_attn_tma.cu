// a5-a6, B200 path: attention over the retained entries as a persistent, TMA-fed flash-decode
// kernel; the memory readout (Eq. 5) as a streaming GEMV; one merge kernel that fuses both (Eq. 4).
//
// Attention kernel.  HBM-bound (every retained K/V byte is read once per step), so the design is
// about keeping loads in flight, not about FLOPs:
//   * the retained entries of a (sequence, KV head) row form tiles of 32 keys; all tiles of all rows
//     are cut into equal contiguous runs, one run per warp (stream-K style: perfect balance for any
//     mix of lengths, at most one partial result per row boundary inside a run);
//   * every warp owns a private ring of 16 KB stages (K tile + V tile), filled by TMA tensor copies
//     (128-byte swizzle) that its lane 0 issues, completion on one mbarrier per stage.  No CTA-wide
//     barrier exists in the main loop;
//   * the math runs on mma.sync m16n8k16 with the KEYS on the M axis and the G_q query heads of the
//     KV head (padded to 8) on N: S^T = K Q^T, then O^T += V^T P^T.  P^T is moved from the
//     accumulator layout to the B-operand layout with movmatrix.  P is split into two bf16 terms so
//     that the product is accurate to 2^-17, not 2^-9.
#include <cuda.h>

#include <algorithm>

#include "im_internal.cuh"


namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int TILE = IM_ATTN_STREAM_TILE;  // keys per tile (48-key tiles with 6 KB boxes and a 192 KB ring measured slower
                                           // in the full step: the readout kernel next to it then falls behind)
constexpr int STAGES = 2;                // ring depth per warp
constexpr int WARPS = IM_ATTN_WARPS;     // consumer warps per CTA (each also issues its own TMA)
constexpr uint32_t WAIT_LIMIT = IM_WAIT_LIMIT;  // try_wait attempts before a warp gives up and flags ST_TIMEOUT

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// bounded wait: returns false if the phase did not complete within `limit` attempts
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = WAIT_LIMIT) {
  for (uint32_t it = 0; it < limit; ++it) {
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
// L2 policy for data that is read once per step (the K/V stream, Mhat): evict first, so that the
// small working set prefetched for the next layer's latency-bound kernels stays resident.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(pol)
      : "memory");
}
// one copy for a whole tile of a cache with 256-byte rows: box (64 columns, rows, 2 halves), see im_attn_make_maps
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar, uint64_t pol) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(pol)
      : "memory");
}
__device__ __forceinline__ float4 ldg_stream(const float4* ptr, uint64_t pol) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0,%1,%2,%3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(pol));
  return v;
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t movm_t(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
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

// tiles of sequence i (all KV heads have the same count)
__device__ __forceinline__ int tiles_of(int n) { return (n + TILE - 1) / TILE; }

// ------------------------------------------------------------------------------------------------
// Persistent attention kernel.  grid = #SMs (or fewer), block = WARPS * 32.
// Shared memory: per warp STAGES x 16 KB (1024-byte aligned), then barriers and the per-sequence
// prefix of tile counts.
// DYN (pipelined stack calls): the tiles are cut into call.att_chunks equal runs and a warp takes runs from a
// counter until none is left, instead of owning the one run its index names.  With layers overlapping, a block of
// this kernel may find its SM busy for a while with blocks of a neighbouring layer's small kernels; with fixed runs
// the whole kernel, and every layer behind it, would wait for that one block.  The merge kernel only needs to know
// how the tiles were cut (run r writes partial slot r + row), not who computed a run.
template <int DH, bool DYN>
__global__ void __launch_bounds__(WARPS * 32, 1)
k_attn_stream(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, ImDims p, ImState st,
              ImScratch sc, ImCall call, const bf16* __restrict__ q) {
  static_assert(DH == 64 || DH == 128, "head dims with a fast path");
  constexpr int KSTEPS = DH / 16;            // k-steps of the S = K Q^T product
  constexpr int DT = DH / 16;                // 16-row tiles of O^T
  constexpr int BOXES = DH / 64;             // 128-byte column boxes per row
  constexpr int TILE_BYTES = TILE * DH * 2;  // one K (or V) tile
  constexpr int STAGE_BYTES = 2 * TILE_BYTES;
  extern __shared__ __align__(1024) unsigned char smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  unsigned char* ring = smem + (size_t)warp * STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)WARPS * STAGES * STAGE_BYTES);
  // (sized by the call's sequences, not by the most a call may have: next to this block and a readout block an SM has
  // some 25 KB of shared memory left, which the small kernels of the layers in flight need every KB of)
  long long* s_pref = reinterpret_cast<long long*>(bars + WARPS * STAGES);  // [n_seq + 1]
  int* s_n = reinterpret_cast<int*>(s_pref + call.n_seq + 1);               // [n_seq]
  int* s_misc = s_n + call.n_seq;                                           // [1 + WARPS * 4] (DYN)
  int* s_fifo = s_misc + 1 + warp * 4;  // runs this warp's producer side has taken, in order (-1: none left)

  // Pipelined stack call: the block claims a worker id (blocks on SMs that are set aside for the call's small
  // kernels, and blocks beyond the worker count, leave).  Nothing that this kernel reads or writes belongs to the
  // kernel ahead of it in its stream (the attention kernel of the previous layer, with a scratch set of its own), so
  // a programmatic dependent never waits for it.
  int wid = blockIdx.x;
  if (DYN) {
    if (threadIdx.x == 0) s_misc[0] = im_claim_worker(call, sc.claim, call.att_workers);
    __syncthreads();
    wid = s_misc[0];
    if (wid < 0) {
      if (threadIdx.x == 0) im_claim_exit(sc.claim);
      return;
    }
    __syncthreads();
  }
  int next_run = 0;  // DYN, lane 0: the run this warp's producer side starts next
  if (DYN && lane == 0) next_run = atomicAdd(sc.claim + 3, 1);
  // (launched behind the merge kernel of a call on the SAME layer, which advances the counters and fills the holes of
  // this very cache: nothing of it may be read before that kernel has ended)
  if (!call.early_cache) asm volatile("griddepcontrol.wait;" ::: "memory");
  // ---- tile prefix over the sequences of the call (every CTA computes the same table)
  for (int i = threadIdx.x; i < call.n_seq; i += blockDim.x) {
    const size_t u = (size_t)call.layer * p.S + call.seq[i];
    s_n[i] = max(0, min(st.ctr[u * CTR_STRIDE + CTR_N], p.cap));
  }
  if (lane == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(smem_u32(&bars[warp * STAGES + s]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    long long acc = 0;
    for (int i = 0; i < call.n_seq; ++i) {
      s_pref[i] = acc;
      acc += (long long)tiles_of(s_n[i]) * p.Hkv;
    }
    s_pref[call.n_seq] = acc;
  }
  __syncthreads();
  const long long total = s_pref[call.n_seq];
  const long long WT = DYN ? (long long)call.att_chunks : (long long)gridDim.x * WARPS;  // runs the tiles are cut into
  const long long qrun = (total + WT - 1) / WT;

  // position of global tile `tile`: sequence i_, KV head h_, tile tt_ of nt_
  auto locate = [&](long long tile, int& i_, int& h_, int& tt_, int& nt_) {
    int lo = 0, hi = call.n_seq;  // last i with s_pref[i] <= tile
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_pref[mid] <= tile) lo = mid; else hi = mid;
    }
    i_ = lo;
    while (i_ < call.n_seq - 1 && tiles_of(s_n[i_]) == 0) ++i_;  // empty sequences own no tiles
    nt_ = max(1, tiles_of(s_n[i_]));
    h_ = (int)((tile - s_pref[i_]) / nt_);
    tt_ = (int)((tile - s_pref[i_]) % nt_);
  };

  const uint64_t pol = policy_evict_first();
  // ---- producer side (lane 0): runs STAGES tiles ahead of the consumer side.  The k-th tile this warp requests goes
  // to stage k % STAGES, whichever run it belongs to.
  long long p_pos = 0, p_end = 0;  // next tile to request, end of the producer's current run
  long long n_issued = 0;          // tiles requested so far
  int pi = 0, ph = 0, ptt = 0, pnt = 1, n_pushed = 0;
  bool p_done = false, released = false;
  auto take_run = [&]() {  // the producer's next run (DYN: from the counter, recorded for the consumer side)
    long long r = -1;
    if (DYN) {
      // (the run was taken from the counter when the previous one was started, and the one after it is taken now:
      // the add's round trip, microseconds while the streams keep the memory system busy, is off the warp's path)
      const int c = next_run;
      next_run = atomicAdd(sc.claim + 3, 1);
      if (c < WT && (long long)c * qrun < total) r = c;
      s_fifo[n_pushed & 3] = (int)r;
      ++n_pushed;
    } else if (n_pushed == 0) {
      const long long w = (long long)wid * WARPS + warp;
      if (w * qrun < total) r = w;
      ++n_pushed;
    }
    if (r < 0) { p_done = true; return; }
    p_pos = r * qrun;
    p_end = min(total, p_pos + qrun);
    locate(p_pos, pi, ph, ptt, pnt);
  };
  auto issue = [&]() {  // lane 0 only: request the next tile, if one is left
    if (!p_done && p_pos == p_end) take_run();
    if (p_done) {
      // nothing left to request: a kernel launched as programmatic dependent (the merge, or the next layer's attention
      // kernel) may become resident and run what does not read this kernel's output
      if (!released) asm volatile("griddepcontrol.launch_dependents;");
      released = true;
      return;
    }
    const int s = (int)(n_issued % STAGES);
    const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
    const uint32_t dst = smem_u32(ring + (size_t)s * STAGE_BYTES);
    const size_t u = (size_t)call.layer * p.S + call.seq[pi];
    const int row = (int)((u * p.Hkv + ph) * (size_t)p.cap) + ptt * TILE;
    mbar_expect_tx(bar, STAGE_BYTES);
    if (BOXES == 1) {
      tma_load_2d(dst, &tmK, 0, row, bar, pol);
      tma_load_2d(dst + TILE_BYTES, &tmV, 0, row, bar, pol);
    } else {
      // (one copy per tile and cache: the 128-byte halves of the rows are the map's third dimension, and the box lands
      // in shared memory half by half, each half the 128-byte-swizzled rows that two 2-D boxes would leave; an SM's
      // copy unit takes requests at a bounded rate, and with 4 KB boxes that rate, not the memory, bounded the kernel)
      tma_load_3d(dst, &tmK, 0, row, 0, bar, pol);
      tma_load_3d(dst + TILE_BYTES, &tmV, 0, row, 0, bar, pol);
    }
    ++n_issued;
    ++p_pos;
    // advance the producer iterator
    if (++ptt == pnt) {
      ptt = 0;
      if (++ph == p.Hkv) {
        ph = 0;
        do { ++pi; } while (pi < call.n_seq && tiles_of(s_n[pi]) == 0);
        pnt = pi < call.n_seq ? tiles_of(s_n[pi]) : 1;
      }
    }
    if (!DYN && p_pos == p_end) {  // (a fixed run: its last tile is requested)
      asm volatile("griddepcontrol.launch_dependents;");
      released = true;
      p_done = true;
    }
  };
  if (lane == 0) {
    for (int k = 0; k < STAGES; ++k) issue();
  }
  if (!DYN) im_warm_inputs(call, wid, threadIdx.x, blockDim.x);  // (the first CTAs: one input tensor each)
  // Launched as a programmatic dependent (of the previous call's merge kernel, or of whatever precedes the call in
  // the caller's stream) the kernel may have come this far before that kernel has ended: the cache of this layer,
  // which the first tiles are being fetched from, is not that kernel's business, but the query rows may be its
  // output and the partials and entry counts of this call overwrite what the previous call's merge still reads.
  if (!DYN) asm volatile("griddepcontrol.wait;" ::: "memory");
  // DYN: the kernel is launched as programmatic dependent so that its blocks follow those of the previous layer's
  // attention kernel without a gap.  Among the launch's other prerequisites is the layer that used this lane's scratch
  // set before (the stream waits for its event), and a prerequisite that releases its dependents early - that layer's
  // merge kernel does - may still be running when this kernel starts.  So nothing is written to the scratch set before
  // `griddepcontrol.wait` has returned; a warp calls it just ahead of its first store, a run's worth of streaming into
  // the kernel, when it returns at once.
  bool scratch_free = !DYN;
  if (!DYN && wid == 0)  // what the merge kernel rebuilds the tile bookkeeping from
    for (int k = threadIdx.x; k < call.n_seq; k += blockDim.x) sc.n_att[k] = s_n[k];

  const float sl2 = p.scale * 1.4426950408889634f;  // softmax in base 2
  bool ok = true;
  long long n_done = 0;  // tiles consumed so far (tile k sits in stage k % STAGES)
  int n_popped = 0;
  while (ok) {
    // ---- the consumer side's next run
    long long run_id = -1;
    if (DYN) {
      __syncwarp();  // (the producer side, lane 0, has recorded the run before it requested the run's first tile)
      run_id = s_fifo[n_popped & 3];
    } else if (n_popped == 0) {
      const long long w = (long long)wid * WARPS + warp;
      if (w * qrun < total) run_id = w;
    }
    ++n_popped;
    if (run_id < 0) break;
    const long long run0 = run_id * qrun, run1 = min(total, run0 + qrun);
    int i, h, tt, nt;
    locate(run0, i, h, tt, nt);
  long long j = run0;
  while (j < run1 && ok) {
    // ---- one (sequence, KV head) segment of the run
    const int n = s_n[i];
    const long long row_id = (long long)i * p.Hkv + h;
    // Q^T as B fragments: head g of the group (zero for the padding heads)
    uint32_t qf[KSTEPS][2];
    {
      const bf16* qrow = q + ((size_t)i * p.H + (size_t)h * p.Gq + g) * DH;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ++ks) {
        qf[ks][0] = g < p.Gq ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t) : 0u;
        qf[ks][1] = g < p.Gq ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t + 8) : 0u;
      }
    }
    float o[DT][4];
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) o[dt][0] = o[dt][1] = o[dt][2] = o[dt][3] = 0.f;
    float m0 = NEG_INF, m1 = NEG_INF, l0 = 0.f, l1 = 0.f;  // heads 2t, 2t+1 (l: this thread's share)

    for (; tt < nt && j < run1; ++tt, ++j) {
      const int s = (int)(n_done % STAGES);
      const uint32_t bar = smem_u32(&bars[warp * STAGES + s]);
      // (the outcome is made warp-uniform: the lanes poll on their own and could disagree at the limit)
      if (!__all_sync(0xffffffffu, mbar_wait(bar, (uint32_t)((n_done / STAGES) & 1), p.wait_limit))) { ok = false; break; }
      ++n_done;
      const uint32_t Ks = smem_u32(ring + (size_t)s * STAGE_BYTES), Vs = Ks + TILE_BYTES;
      // ---- S^T = K Q^T : [32 keys] x [8 heads]
      float sacc[TILE / 16][4];
#pragma unroll
      for (int mt = 0; mt < TILE / 16; ++mt) {
        sacc[mt][0] = sacc[mt][1] = sacc[mt][2] = sacc[mt][3] = 0.f;
        const int r = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
          const int c = ks * 2 + (lane >> 4);
          const uint32_t addr = Ks + (c >> 3) * (TILE * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          uint32_t a0, a1, a2, a3;
          ldsm_x4(addr, a0, a1, a2, a3);
          mma_bf16(sacc[mt], a0, a1, a2, a3, qf[ks][0], qf[ks][1]);
        }
      }
      // ---- online softmax (base 2); keys beyond n are masked
      const int key0 = tt * TILE;
      float tmax0 = NEG_INF, tmax1 = NEG_INF;
#pragma unroll
      for (int mt = 0; mt < TILE / 16; ++mt) {
        const bool v0 = key0 + mt * 16 + g < n, v1 = key0 + mt * 16 + g + 8 < n;
        sacc[mt][0] = v0 ? sacc[mt][0] * sl2 : NEG_INF;
        sacc[mt][1] = v0 ? sacc[mt][1] * sl2 : NEG_INF;
        sacc[mt][2] = v1 ? sacc[mt][2] * sl2 : NEG_INF;
        sacc[mt][3] = v1 ? sacc[mt][3] * sl2 : NEG_INF;
        tmax0 = fmaxf(tmax0, fmaxf(sacc[mt][0], sacc[mt][2]));
        tmax1 = fmaxf(tmax1, fmaxf(sacc[mt][1], sacc[mt][3]));
      }
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, off));
        tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, off));
      }
      const float mn0 = fmaxf(m0, tmax0), mn1 = fmaxf(m1, tmax1);
      // every tile holds at least one valid key, so mn0/mn1 are finite
      const float c0 = exp2f(m0 - mn0), c1 = exp2f(m1 - mn1);
      m0 = mn0; m1 = mn1;
      l0 *= c0; l1 *= c1;
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        o[dt][0] *= c0; o[dt][1] *= c1; o[dt][2] *= c0; o[dt][3] *= c1;
      }
      uint32_t ph_[TILE / 16][2], pl_[TILE / 16][2];  // P^T as B fragments, high and low bf16 terms
#pragma unroll
      for (int mt = 0; mt < TILE / 16; ++mt) {
        const float p0 = exp2f(sacc[mt][0] - mn0), p1 = exp2f(sacc[mt][1] - mn1);
        const float p2 = exp2f(sacc[mt][2] - mn0), p3 = exp2f(sacc[mt][3] - mn1);
        l0 += p0 + p2;
        l1 += p1 + p3;
        const uint32_t hi01 = pack_bf16(p0, p1), hi23 = pack_bf16(p2, p3);
        const uint32_t lo01 = pack_bf16(p0 - __uint_as_float(hi01 << 16), p1 - __uint_as_float(hi01 & 0xffff0000u));
        const uint32_t lo23 = pack_bf16(p2 - __uint_as_float(hi23 << 16), p3 - __uint_as_float(hi23 & 0xffff0000u));
        ph_[mt][0] = movm_t(hi01); ph_[mt][1] = movm_t(hi23);
        pl_[mt][0] = movm_t(lo01); pl_[mt][1] = movm_t(lo23);
      }
      // ---- O^T += V^T P^T : [DH] x [8 heads]
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
#pragma unroll
        for (int kt = 0; kt < TILE / 16; ++kt) {
          const int r = kt * 16 + (lane & 7) + (lane >> 4) * 8;
          const int c = dt * 2 + ((lane >> 3) & 1);
          const uint32_t addr = Vs + (c >> 3) * (TILE * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
          uint32_t a0, a1, a2, a3;
          ldsm_x4_t(addr, a0, a1, a2, a3);
          mma_bf16(o[dt], a0, a1, a2, a3, ph_[kt][0], ph_[kt][1]);
          mma_bf16(o[dt], a0, a1, a2, a3, pl_[kt][0], pl_[kt][1]);
        }
      }
      // ---- the stage is free again: refill it
      __syncwarp();
      if (lane == 0) issue();
    }
    if (!ok) break;
    // ---- segment finished: write the partial (unnormalised O, max, sum) of this row
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, off);
      l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
    if (!scratch_free) {  // (warp uniform)
      asm volatile("griddepcontrol.wait;" ::: "memory");
      scratch_free = true;
      if (wid == 0 && warp == 0)
        for (int k = lane; k < call.n_seq; k += 32) sc.n_att[k] = s_n[k];
    }
    {
      // Rows are served by consecutive runs and consecutive rows share at most one run, so
      // (run index + row index) is a collision-free slot id below WT + rows.
      const long long slot = run_id + row_id;
      float* dst = sc.part + (size_t)slot * p.Gq * (DH + 2);
      const int hh0 = 2 * t, hh1 = 2 * t + 1;
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        if (hh0 < p.Gq) {
          dst[(size_t)hh0 * (DH + 2) + dt * 16 + g] = o[dt][0];
          dst[(size_t)hh0 * (DH + 2) + dt * 16 + g + 8] = o[dt][2];
        }
        if (hh1 < p.Gq) {
          dst[(size_t)hh1 * (DH + 2) + dt * 16 + g] = o[dt][1];
          dst[(size_t)hh1 * (DH + 2) + dt * 16 + g + 8] = o[dt][3];
        }
      }
      if (g == 0) {
        if (hh0 < p.Gq) { dst[(size_t)hh0 * (DH + 2) + DH] = m0; dst[(size_t)hh0 * (DH + 2) + DH + 1] = l0; }
        if (hh1 < p.Gq) { dst[(size_t)hh1 * (DH + 2) + DH] = m1; dst[(size_t)hh1 * (DH + 2) + DH + 1] = l1; }
      }
    }
    // ---- next row
    if (tt == nt) {
      tt = 0;
      if (++h == p.Hkv) {
        h = 0;
        do { ++i; } while (i < call.n_seq && tiles_of(s_n[i]) == 0);
        if (i >= call.n_seq) break;
        nt = tiles_of(s_n[i]);
      }
    }
  }
    if (!DYN) break;
  }
  if (!ok && lane == 0) {
    // The warp gives up.  The copies it has requested and not consumed (tiles n_done .. n_issued - 1 of its own count)
    // still write into this CTA's shared memory, which the SM hands to another CTA when this one ends: wait for each
    // of them, with the full limit, before returning.
    atomicOr(st.status, ST_TIMEOUT);
    for (long long t2 = n_done; t2 < n_issued; ++t2)
      mbar_wait(smem_u32(&bars[warp * STAGES + (int)(t2 % STAGES)]), (uint32_t)((t2 / STAGES) & 1));
  }
  if (DYN) {
    __syncthreads();
    if (threadIdx.x == 0) im_claim_exit(sc.claim);
  }
}

// ------------------------------------------------------------------------------------------------
// Readout numerators (Eq. 5): rsum[i][col] = sum over all dM rows m of phi_q[m] * Mhat[m][col].
// The kernel runs next to the attention kernel and shares an SM with one of its CTAs: a persistent grid of
// 256-thread blocks, at most one per SM.  A block owns a contiguous run of items; an item is a 64-column slice
// (256 bytes of every row) of one sequence's Mhat over all its rows, so that no partial sums go through memory
// and the merge kernel reads one number per column.  A half warp reads one row slice per load, the 16 half warps
// of the block take 16 consecutive rows per round, and every thread keeps DEPTH loads in flight across round,
// batch and item boundaries (a consumed register is re-requested at once).  The loop body between two loads has
// no branch: with branches there the compiler waits for every load in flight at each of them.
// Two variants: DEPTH 32 (128 KB in flight per SM, 42 K registers: with an attention CTA it fills the SM's register
// file, so it is used where the front kernel runs on SMs of its own and has ended before this kernel starts) and
// DEPTH 8 (16 K registers: leaves room for a front block on the same SM).
// grid = min(blocks wanted, items), block = RC_THREADS, smem = dM rounded up to RC_RPR * DEPTH floats.
constexpr int RC_COLS = 64;
constexpr int RC_THREADS = 256;
constexpr int RC_RPR = RC_THREADS / 16;  // rows per round
// DYN (pipelined stack calls): a block claims a worker id and then takes items from a counter, always one item
// ahead of the one it works on (the first loads of the next item are requested while the current one is added up),
// instead of owning the run of items its index names; see k_attn_stream for why.
template <int RC_DEPTH, bool DYN>
__device__ __forceinline__ void readout_cols_body(const ImDims& p, const ImState& st, const ImScratch& sc, const ImCall& call) {
  extern __shared__ float s_phi[];  // phi(q) of the current sequence, zero beyond dM
  __shared__ float4 s_red[RC_RPR][RC_COLS / 4];
  __shared__ int s_take[2];
  const int tid = threadIdx.x;
  const int rsub = tid >> 4, c4 = tid & 15;  // row within a round, float4 within the slice
  const int nsl = p.Dkv / RC_COLS;
  const int total = call.n_seq * nsl;
  int t = 0, t_next = 0, t_end = total;  // current item, the one after it, end of the items (of this block's run)
  if (DYN) {
    if (tid == 0) {
      const int wid = im_claim_worker(call, sc.claim + 4, call.ro_claim);
      s_take[0] = wid < 0 ? total : atomicAdd(sc.claim + 7, 1);
      s_take[1] = wid < 0 ? total : atomicAdd(sc.claim + 7, 1);
    }
    __syncthreads();
    t = s_take[0];
    t_next = s_take[1];
  } else {
    t = (int)((long long)blockIdx.x * total / gridDim.x);
    t_end = (int)((long long)(blockIdx.x + 1) * total / gridDim.x);
    t_next = t + 1;
  }
  if (t >= t_end) {
    if (DYN && tid == 0) im_claim_exit(sc.claim + 4);
    return;
  }
  const int nb = (p.dM + RC_RPR * RC_DEPTH - 1) / (RC_RPR * RC_DEPTH);  // batches of RC_DEPTH rounds per item
  const uint64_t pol = policy_evict_first();
  const ImRows r = im_rows(p);
  const size_t row_f4 = (size_t)p.Dkv / 4;
  // first load of (item t, batch b) for this thread; round k of the batch is k * RC_RPR rows further
  auto batch_ptr = [&](int t, int b) {
    const size_t u = (size_t)call.layer * p.S + call.seq[t / nsl];
    return reinterpret_cast<const float4*>(st.Mhat + u * p.dM * (size_t)p.Dkv + (size_t)(t % nsl) * RC_COLS) + c4;
  };
  float4 v[RC_DEPTH];
  {
    const float4* src = batch_ptr(t, 0);
#pragma unroll
    for (int k = 0; k < RC_DEPTH; ++k) v[k] = ldg_stream(src + (size_t)min(k * RC_RPR + rsub, p.dM - 1) * row_f4, pol);
  }
  int cur = -1;
  while (t < t_end) {
    const int i = t / nsl;
    if (i != cur) {  // (block uniform)
      if (cur >= 0) __syncthreads();
      for (int m = tid; m < nb * RC_RPR * RC_DEPTH; m += RC_THREADS)
        s_phi[m] = m < p.dM ? im_raw_sum(p, sc, call, i, r.theta + m) : 0.f;
      cur = i;
      __syncthreads();
    }
    if (DYN && tid == 0) s_take[0] = t_next < total ? atomicAdd(sc.claim + 7, 1) : total;  // the item after the next
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int b = 0; b < nb; ++b) {
      const bool more = b + 1 < nb || t_next < t_end;
      const float4* src = more ? (b + 1 < nb ? batch_ptr(t, b + 1) : batch_ptr(t_next, 0)) : nullptr;
      const int row_next = b + 1 < nb ? (b + 1) * RC_RPR * RC_DEPTH + rsub : rsub;
      const float* ph = s_phi + b * RC_RPR * RC_DEPTH + rsub;
#pragma unroll
      for (int k = 0; k < RC_DEPTH; ++k) {
        const float f = ph[k * RC_RPR];
        acc.x = fmaf(f, v[k].x, acc.x); acc.y = fmaf(f, v[k].y, acc.y);
        acc.z = fmaf(f, v[k].z, acc.z); acc.w = fmaf(f, v[k].w, acc.w);
        if (more) v[k] = ldg_stream(src + (size_t)min(row_next + k * RC_RPR, p.dM - 1) * row_f4, pol);
      }
    }
    s_red[rsub][c4] = acc;
    __syncthreads();
    if (tid < RC_COLS / 4) {
      float4 sum = s_red[0][tid];
#pragma unroll
      for (int j = 1; j < RC_RPR; ++j) {
        const float4 o = s_red[j][tid];
        sum.x += o.x; sum.y += o.y; sum.z += o.z; sum.w += o.w;
      }
      reinterpret_cast<float4*>(sc.rpart + (size_t)i * p.Dkv + (size_t)(t % nsl) * RC_COLS)[tid] = sum;
    }
    const int t_after = DYN ? s_take[0] : t_next + 1;  // (written by thread 0 before the barrier above)
    __syncthreads();
    t = t_next;
    t_next = t_after;
  }
  if (DYN && tid == 0) im_claim_exit(sc.claim + 4);
}

__global__ void __maxnreg__(168) k_readout_cols(ImDims p, ImState st, ImScratch sc, ImCall call) {
  readout_cols_body<32, false>(p, st, sc, call);
}
__global__ void __maxnreg__(168) k_readout_cols_dyn(ImDims p, ImState st, ImScratch sc, ImCall call) {
  readout_cols_body<32, true>(p, st, sc, call);
}
__global__ void __maxnreg__(64) k_readout_cols_light(ImDims p, ImState st, ImScratch sc, ImCall call) {
  readout_cols_body<8, false>(p, st, sc, call);
}

// ------------------------------------------------------------------------------------------------
// Readout, the part that does not go through Mhat (Eq. 5 and the gate of Eq. 4), once per sequence.  With
// s = cscale / (sum_m phi_q[m]^2 b[m] + eps):
//   mres[i][col]     = s * sum_p w_p (phi_q . phi_p) v_p[col]      (pending rank-one terms)
//   mres[i][Dkv]     = g(q)
//   mres[i][Dkv + 2] = s                                             (the merge kernel adds s * phi(q)^T Mhat[col])
// It does not read the output of k_readout_cols and may run next to it.  Without deferred compaction it runs
// after the memory write of the call (it reads the pending list, b and cscale).  With it (call.defer) it runs
// BEFORE the write with s = cscale, leaving the denominator sum apart in mres[i][Dkv + 1]; the merge kernel
// then adds the terms of the entries written in this call, so that the readout does not wait for the selection.
// grid = n_seq, block = 256, smem = dM floats.
__global__ void __launch_bounds__(256) k_readout_finish(ImDims p, ImState st, ImWeights w, ImScratch sc, ImCall call) {
  extern __shared__ float phiq[];  // [dM] phi(q), summed over the K-split partials
  __shared__ float s_dot[64];
  __shared__ float s_red[8];
  const int i = blockIdx.x, tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const ImRows r = im_rows(p);
  for (int m = tid; m < p.dM; m += 256) phiq[m] = im_raw_sum(p, sc, call, i, r.theta + m);
  __syncthreads();
  const int np = min(st.ctr[u * CTR_STRIDE + CTR_NPEND], p.F);
  float part_den = 0.f;
  for (int m = tid; m < p.dM; m += 256) part_den = fmaf(phiq[m] * phiq[m], st.bvec[u * p.dM + m], part_den);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) part_den += __shfl_xor_sync(0xffffffffu, part_den, off);
  if (lane == 0) s_red[warp] = part_den;
  // phi_q . phi_p, two pending entries per warp at a time so that their loads overlap
  for (int pp = warp; pp < np; pp += 16) {
    const float* ph0 = st.pend_phi + (u * p.F + pp) * p.dM;
    const bool two = pp + 8 < np;
    const float* ph1 = st.pend_phi + (u * p.F + (two ? pp + 8 : pp)) * p.dM;
    float v0 = 0.f, v1 = 0.f;
    for (int m = lane; m < p.dM; m += 32) {
      v0 = fmaf(phiq[m], ph0[m], v0);
      v1 = fmaf(phiq[m], ph1[m], v1);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      v0 += __shfl_xor_sync(0xffffffffu, v0, off);
      v1 += __shfl_xor_sync(0xffffffffu, v1, off);
    }
    if (lane == 0) {
      s_dot[pp] = v0 * st.pend_w[u * p.F + pp];
      if (two) s_dot[pp + 8] = v1 * st.pend_w[u * p.F + pp + 8];
    }
  }
  __syncthreads();
  float den = p.eps;
  for (int k = 0; k < 8; ++k) den += s_red[k];
  // deferred compaction: numerator and denominator sum over the state from before the call's memory write
  const float scale = call.defer ? st.cscale[u] : st.cscale[u] / den;
  float* dst = sc.mres + (size_t)i * IM_MRES_ROW(p);
  for (int m = tid; m < p.dM; m += 256) sc.phiq[(size_t)i * p.dM + m] = phiq[m];
  for (int col = tid; col < p.Dkv; col += 256) {
    float mv = 0.f;
    for (int pp = 0; pp < np; ++pp) mv = fmaf(s_dot[pp], __bfloat162float(st.pend_v[(u * p.F + pp) * p.Dkv + col]), mv);
    dst[col] = scale * mv;
  }
  if (tid == 0) {
    dst[p.Dkv] = 1.0f / (1.0f + expf(-(im_raw_sum(p, sc, call, i, r.wg) + w.bg[0])));
    dst[p.Dkv + 1] = den - p.eps;
    dst[p.Dkv + 2] = scale;  // coefficient of phi(q)^T Mhat, which the merge kernel adds
  }
}

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// one more key for a running (base 2) softmax state of one query head spread over a warp
template <int CPL>
__device__ __forceinline__ void softmax_push(float s, const float (&v)[CPL], float& M, float& L, float (&res)[CPL]) {
  const float Mn = fmaxf(M, s);
  const float eo = exp2f(M - Mn), en = exp2f(s - Mn);
  L = L * eo + en;
#pragma unroll
  for (int k = 0; k < CPL; ++k) res[k] = res[k] * eo + en * v[k];
  M = Mn;
}

// Merge: softmax-merge of the attention partials of one (sequence, KV head) row, add the gated
// memory readout (Eq. 4), store.
// grid = (Hkv, n_seq), block = 32 * max(Gq, DH / 32): warp hh merges query head hh of the group
// (each lane DH/32 output columns), all heads in parallel.
//
// Deferred compaction (call.defer): the partials cover the entries cached before the call, i.e. without the
// new token and with the entries the selection has evicted meanwhile.  The attention over the retained set
// (Eq. 4) is recovered exactly: the new token's term is added, the evicted entries' terms
// exp(s_e) (1, v_e) are taken out of the sums again.  Taking out is safe in float32 while the evicted
// entries hold at most 90 % of the softmax mass (the error of the remainder grows by at most 10); beyond
// that the block's warps together recompute, from the cache, which is still uncompacted, the partials of that
// head whose key range holds an evicted entry.
template <int DH, typename OutT>
__global__ void __launch_bounds__(256, 1) k_attn_merge_rows(ImDims p, ImState st, ImScratch sc, ImCall call, int n_workers, int tile,
                                                          int ro_workers, int ro_cs, OutT* __restrict__ out, const bf16* __restrict__ q,
                                                          const bf16* __restrict__ k_new, const bf16* __restrict__ v_new) {
  constexpr int CPL = DH / 32;  // columns per lane
  __shared__ float s_q[8][DH];       // redo path: the query rows of the heads to redo
  __shared__ float s_st[8][DH + 2];  // redo path: the warps' softmax states of a key range
  __shared__ int s_redo[8];
  __shared__ float s_dot[IM_FRONT_MAX_NE][8], s_sq[IM_FRONT_MAX_NE][8];  // readout terms of this call's write, per warp
  // the next call's attention kernel may become resident and start fetching its first tiles
  asm volatile("griddepcontrol.launch_dependents;");
  const int h = blockIdx.x, i = blockIdx.y, tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31, nwarps = blockDim.x >> 5;
  const size_t u = (size_t)call.layer * p.S + call.seq[i];
  const int hh0 = min(warp, p.Gq - 1);  // the head this warp merges first (usually its only one)
  IM_MARK(sc, call.layer, 1, 0);
  // ---- every load whose address depends on no other load is issued here, ahead of its use: this kernel is
  // on the critical path of the call and a dependent chain of loads costs a memory round trip per link
  const int ne_raw = st.ctr[u * CTR_STRIDE + CTR_NEVICT];
  const int ev_l = lane < IM_FRONT_MAX_NE ? st.ev_slot[u * p.tail + min(lane, p.tail - 1)] : -1;
  // (deferred compaction) the moves the front kernel listed, and the entry counts the attention kernel ran over: the
  // counts of before the call, which the front kernel left as CTR_NNEXT + CTR_NEVICT - 1 (CTR_N itself is advanced by
  // this kernel further down)
  const int nh_raw = call.defer ? sc.nhole[i] : 0;
  const int surv_l = (call.defer && lane < IM_FRONT_MAX_NE) ? sc.surv[(size_t)i * p.tail + min(lane, p.tail - 1)] : 0;
  auto count_before = [&](int k) {
    const int32_t* c = st.ctr + ((size_t)call.layer * p.S + call.seq[k]) * CTR_STRIDE;
    return max(0, min(c[CTR_NNEXT] + c[CTR_NEVICT] - 1, p.cap));
  };
  int na_lane = (call.defer && lane < call.n_seq) ? count_before(lane) : 0;
  const float* mr = sc.mres + (size_t)i * IM_MRES_ROW(p);
  // phi(q)^T Mhat: one vector per sequence (k_readout_cols), or - ro_workers > 0 - the partial vectors of the CTAs of
  // k_readout_stream whose runs of ro_cs chunks per sequence hold chunks of this sequence, added in CTA order
  const float* rs = sc.rpart + (size_t)i * p.Dkv;
  int rw0 = 0, rw1 = 0;
  if (ro_workers > 0) {
    const long long rq = ((long long)call.n_seq * ro_cs + ro_workers - 1) / ro_workers;
    rw0 = (int)(((long long)i * ro_cs) / rq);
    rw1 = (int)(((long long)(i + 1) * ro_cs - 1) / rq);
    rs = sc.rpart + (size_t)(rw0 + i) * p.Dkv;
  }
  float pf0[4], pq0[4];
  float gate = 0.f, c_hat = 0.f, den_old = 0.f, mcol[CPL], qv[CPL], kn[CPL], vn[CPL], ek0[CPL], ev0[CPL];
  {
    const bf16* qrow = q + ((size_t)i * p.H + (size_t)h * p.Gq + hh0) * DH;
    const bf16* kr = k_new + (size_t)i * p.Dkv + h * DH;
    const bf16* vr = v_new + (size_t)i * p.Dkv + h * DH;
    const bf16* ekr = sc.evK + (size_t)i * p.tail * p.Dkv + h * DH;
    const bf16* evr = sc.evV + (size_t)i * p.tail * p.Dkv + h * DH;
    if (p.mem) { gate = mr[p.Dkv]; c_hat = mr[p.Dkv + 2]; den_old = mr[p.Dkv + 1]; }
    if (p.mem && call.defer) {  // slot 0 of the evicted entries' phi is read before the evicted count is known
      float pk[4][IM_KSPLIT];  // (all requested before the first sum: one round trip)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int m = tid + j * blockDim.x;
        pq0[j] = m < p.dM ? sc.phiq[(size_t)i * p.dM + m] : 0.f;
#pragma unroll
        for (int ks = 0; ks < IM_KSPLIT; ++ks)
          pk[j][ks] = (m < p.dM && ks < call.ksplit_phi) ? sc.phip[((size_t)ks * call.n_seq + i) * p.F * p.dM + m] : 0.f;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        pf0[j] = 0.f;
#pragma unroll
        for (int ks = 0; ks < IM_KSPLIT; ++ks) pf0[j] += pk[j][ks];
      }
    }
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
      const int c = lane + 32 * k;
      float rv = p.mem ? rs[h * DH + c] : 0.f;
      for (int w = rw0 + 1; w <= rw1; ++w) rv += rs[(size_t)(w - rw0) * p.Dkv + h * DH + c];
      mcol[k] = p.mem ? fmaf(c_hat, rv, mr[h * DH + c]) : 0.f;
      qv[k] = __bfloat162float(qrow[c]);
      kn[k] = __bfloat162float(kr[c]);
      vn[k] = __bfloat162float(vr[c]);
      ek0[k] = call.defer ? __bfloat162float(ekr[c]) : 0.f;
      ev0[k] = call.defer ? __bfloat162float(evr[c]) : 0.f;
    }
  }
  // ---- deferred compaction: Eq. 5 over the memory AFTER this call's write (Eq. 6-7), M' = lambda M + eta sum_e
  // phi_e v_e^T, b' = lambda b + eta sum_e phi_e^2 (applied only if something was evicted), from the parts of
  // before the write: with P = s (phi(q)^T Mhat + pending terms) and the denominator sum D that k_readout_finish
  // left,  m[col] = (decay P[col] + eta sum_e (phi_q . phi_e) v_e[col]) / (eps + decay D + eta sum_e sum_m
  // phi_q[m]^2 phi_e[m]^2).  Needs phi of the evicted keys (K-split partials), not the state update itself.
  if (p.mem && call.defer) {  // (block uniform)
    const int ne_m = max(0, min(ne_raw, min(IM_FRONT_MAX_NE, p.F)));
    const float* pq = sc.phiq + (size_t)i * p.dM;
    for (int e = 0; e < ne_m; ++e) {
      float dot = 0.f, sq = 0.f;
      int m_first = tid;
      if (e == 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          dot = fmaf(pq0[j], pf0[j], dot);
          sq = fmaf(pq0[j] * pq0[j], pf0[j] * pf0[j], sq);
        }
        m_first = tid + 4 * blockDim.x;
      }
      for (int m = m_first; m < p.dM; m += blockDim.x) {
        float f = 0.f;
        for (int ks = 0; ks < call.ksplit_phi; ++ks) f += sc.phip[(((size_t)ks * call.n_seq + i) * p.F + e) * p.dM + m];
        const float qf = pq[m];
        dot = fmaf(qf, f, dot);
        sq = fmaf(qf * qf, f * f, sq);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        dot += __shfl_xor_sync(0xffffffffu, dot, o);
        sq += __shfl_xor_sync(0xffffffffu, sq, o);
      }
      if (lane == 0) { s_dot[e][warp] = dot; s_sq[e][warp] = sq; }
    }
    __syncthreads();
    const float decay = ne_m > 0 ? p.lambda : 1.0f;
    float den = p.eps + decay * den_old;
    for (int e = 0; e < ne_m; ++e) {
      float sq = 0.f;
      for (int w = 0; w < nwarps; ++w) sq += s_sq[e][w];
      den = fmaf(p.eta, sq, den);
    }
#pragma unroll
    for (int k = 0; k < CPL; ++k) mcol[k] *= decay;
    for (int e = 0; e < ne_m; ++e) {
      float dot = 0.f;
      for (int w = 0; w < nwarps; ++w) dot += s_dot[e][w];
      const bf16* evr = sc.evV + ((size_t)i * p.tail + e) * p.Dkv + h * DH;
#pragma unroll
      for (int k = 0; k < CPL; ++k)
        mcol[k] = fmaf(p.eta * dot, e == 0 ? ev0[k] : __bfloat162float(evr[lane + 32 * k]), mcol[k]);
    }
    const float inv = 1.0f / den;
#pragma unroll
    for (int k = 0; k < CPL; ++k) mcol[k] *= inv;
  }
  // ---- a4 with deferred compaction: this block fills the holes of head h's slabs (block h == 0 also those of the
  // index-key and position arrays).  The retained entries above the budget are read here, the holes are overwritten
  // once the attention kernel, which streams the evicted entries like any other, has ended.
  constexpr int MV = 4, DV = DH / 8;
  IM_MARK(sc, call.layer, 1, 1);
  uint4 mv[MV];
  bf16 mx[MV];
  int n_mv = 0, n_mx = 0, nh = 0, pos_surv = 0, n_next = 0;
  int hole[MV], hole_x[MV], hole_p = 0;
  bf16* Kw = st.Kc + (u * p.Hkv + h) * (size_t)p.cap * DH;
  bf16* Vw = st.Vc + (u * p.Hkv + h) * (size_t)p.cap * DH;
  if (call.defer) {
    const int ne_c = min(ne_raw, min(p.tail, IM_FRONT_MAX_NE));
    nh = ne_c > 0 ? max(0, min(nh_raw, ne_c)) : 0;
    n_mv = nh * 2 * DV;
    n_mx = h == 0 ? nh * p.dI : 0;
#pragma unroll
    for (int r = 0; r < MV; ++r) {
      const int k = tid + r * blockDim.x;
      const int j = min(k / (2 * DV), IM_FRONT_MAX_NE - 1), rem = k % (2 * DV);
      const int sj = __shfl_sync(0xffffffffu, surv_l, j), ej = __shfl_sync(0xffffffffu, ev_l, j);
      if (k < n_mv) {
        mv[r] = reinterpret_cast<const uint4*>((rem < DV ? Kw : Vw) + (size_t)sj * DH)[rem % DV];
        hole[r] = ej;
      }
      const int jx = min(k / p.dI, IM_FRONT_MAX_NE - 1);
      const int sx = __shfl_sync(0xffffffffu, surv_l, jx), ex = __shfl_sync(0xffffffffu, ev_l, jx);
      if (k < n_mx) {
        mx[r] = st.kidx[(u * p.cap + sx) * p.dI + k % p.dI];
        hole_x[r] = ex;
      }
    }
    if (h == 0 && warp == 0) {
      if (lane < nh) pos_surv = st.pos[u * p.cap + surv_l];
      hole_p = ev_l;
    }
    if (h == 0 && tid == 0) n_next = st.ctr[u * CTR_STRIDE + CTR_NNEXT];
  }
  // ---- the tile bookkeeping of the attention kernel, rebuilt (lanes stride over the sequences).  With deferred
  // compaction it needs nothing that the attention kernel writes and runs ahead of the wait.
  long long pref = 0, total = 0;
  int nt_i = 0, n_old = 0;
  auto bookkeeping = [&]() {
    for (int k0 = 0; k0 < call.n_seq; k0 += 32) {
      const int k = k0 + lane;
      int na = 0;
      if (k0 == 0) na = na_lane;
      else if (k < call.n_seq) na = call.defer ? count_before(k) : sc.n_att[k];
      const int nk = (na + tile - 1) / tile;
      // inclusive prefix over the 32 lanes
      long long incl = (long long)nk * p.Hkv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      if (i >= k0 && i < k0 + 32) {
        pref = total + __shfl_sync(0xffffffffu, incl, i - k0) - (long long)__shfl_sync(0xffffffffu, nk, i - k0) * p.Hkv;
        nt_i = __shfl_sync(0xffffffffu, nk, i - k0);
        n_old = __shfl_sync(0xffffffffu, na, i - k0);
      }
      total += __shfl_sync(0xffffffffu, incl, 31);
    }
  };
  if (call.defer) bookkeeping();
  IM_MARK(sc, call.layer, 1, 2);
  // ---- everything below reads what the attention kernel has written.  When this kernel was launched as its
  // programmatic dependent it may have started before that kernel ended: wait for it (and its writes) here.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (call.defer) {
    // (the recomputation below reads the slabs too: never a hole with a weight, and no entry that is moved away)
#pragma unroll
    for (int r = 0; r < MV; ++r) {
      const int k = tid + r * blockDim.x;
      if (k < n_mv) {
        const int rem = k % (2 * DV);
        reinterpret_cast<uint4*>((rem < DV ? Kw : Vw) + (size_t)hole[r] * DH)[rem % DV] = mv[r];
      }
      if (k < n_mx) st.kidx[(u * p.cap + hole_x[r]) * p.dI + k % p.dI] = mx[r];
    }
    for (int k = tid + MV * blockDim.x; k < n_mx; k += blockDim.x) {  // (index keys wider than MV elements per thread)
      const int32_t* evs = st.ev_slot + u * p.tail;
      const int32_t* surv = sc.surv + (size_t)i * p.tail;
      st.kidx[(u * p.cap + evs[k / p.dI]) * p.dI + k % p.dI] = st.kidx[(u * p.cap + surv[k / p.dI]) * p.dI + k % p.dI];
    }
    if (h == 0 && warp == 0 && lane < nh) st.pos[u * p.cap + hole_p] = pos_surv;
    // the entry count the call leaves (nothing that runs next to this kernel reads it: the merge below works from
    // the attention kernel's snapshot)
    if (h == 0 && tid == 0) st.ctr[u * CTR_STRIDE + CTR_N] = n_next;
  }
  IM_MARK(sc, call.layer, 1, 3);
  if (!call.defer) {
    na_lane = lane < call.n_seq ? sc.n_att[lane] : 0;
    bookkeeping();
  }
  n_old = max(0, min(n_old, p.cap - 1));  // with deferred compaction: the slot of the new token
  const long long WT = n_workers;  // runs the attention kernel cut the tiles into (warps or CTAs)
  const long long qrun = (total + WT - 1) / WT;
  const long long row_first = pref + (long long)h * nt_i, row_last = row_first + nt_i - 1;
  const long long row_id = (long long)i * p.Hkv + h;
  const int ne = call.defer ? max(0, min(ne_raw, IM_FRONT_MAX_NE)) : 0;
  const float sl2 = p.scale * 1.4426950408889634f;
  // ---- one warp per query head of the group (the block has at least Gq warps)
  const bf16* Kb = st.Kc + (u * p.Hkv + h) * (size_t)p.cap * DH;
  const bf16* Vb = st.Vc + (u * p.Hkv + h) * (size_t)p.cap * DH;
  const bool has_head = warp < p.Gq;
  const int hh = hh0;
  const long long w0 = nt_i > 0 ? row_first / qrun : 0, w1 = nt_i > 0 ? row_last / qrun : -1;
  // keys of partial wv of this row: the tiles of the row that fall into run wv
  auto partial_keys = [&](long long wv, int& key0, int& key1) {
    const int lt0 = (int)(max(wv * qrun, row_first) - row_first);
    const int lt1 = (int)(min((wv + 1) * qrun - 1, row_last) - row_first);
    key0 = lt0 * tile;
    key1 = min((lt1 + 1) * tile, n_old);
  };
  auto merge_stored = [&](long long wv, int head, float& M, float& L, float (&res)[CPL]) {
    const float* ps = sc.part + ((size_t)(wv + row_id) * p.Gq + head) * (DH + 2);
    const float mw = ps[DH], lw = ps[DH + 1];
    float a[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) a[k] = ps[lane + 32 * k];
    const float Mn = fmaxf(M, mw);
    const float eo = exp2f(M - Mn), en = exp2f(mw - Mn);  // exp2(-inf) = 0 for the first contributor
    L = L * eo + lw * en;
#pragma unroll
    for (int k = 0; k < CPL; ++k) res[k] = res[k] * eo + a[k] * en;
    M = Mn;
  };
  // the stored partials wa .. wb of a head, four at a time: their loads are all requested before the first is added
  auto merge_stored_range = [&](long long wa, long long wb, int head, float& M, float& L, float (&res)[CPL]) {
    for (long long w4 = wa; w4 <= wb; w4 += 4) {
      float a[4][CPL], mw[4], lw[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float* ps = sc.part + ((size_t)(min(w4 + j, wb) + row_id) * p.Gq + head) * (DH + 2);
        mw[j] = ps[DH];
        lw[j] = ps[DH + 1];
#pragma unroll
        for (int k = 0; k < CPL; ++k) a[j][k] = ps[lane + 32 * k];
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (w4 + j > wb) break;
        const float Mn = fmaxf(M, mw[j]);
        const float eo = exp2f(M - Mn), en = exp2f(mw[j] - Mn);  // exp2(-inf) = 0 for the first contributor
        L = L * eo + lw[j] * en;
#pragma unroll
        for (int k = 0; k < CPL; ++k) res[k] = res[k] * eo + a[j][k] * en;
        M = Mn;
      }
    }
  };
  bool new_kept = true;
  for (int a = 0; a < ne; ++a) new_kept &= __shfl_sync(0xffffffffu, ev_l, a) != n_old;
  auto push_new = [&](float& M, float& L, float (&res)[CPL]) {
    if (!new_kept) return;
    float dot = 0.f;
#pragma unroll
    for (int k = 0; k < CPL; ++k) dot = fmaf(qv[k], kn[k], dot);
    softmax_push<CPL>(warp_sum_f(dot) * sl2, vn, M, L, res);
  };
  auto store_head = [&](float L, float (&res)[CPL]) {
    if (L > 0.f) {
      const float inv = 1.0f / L;
#pragma unroll
      for (int k = 0; k < CPL; ++k) res[k] *= inv;
    }
    const size_t base = ((size_t)i * p.H + (size_t)h * p.Gq + hh) * DH;
#pragma unroll
    for (int k = 0; k < CPL; ++k) {
      const float v = res[k] + gate * mcol[k];  // Eq. 4: attention over the retained set + gated memory readout
      if constexpr (sizeof(OutT) == 2) out[base + lane + 32 * k] = __float2bfloat16_rn(v);
      else out[base + lane + 32 * k] = v;
    }
  };
  // Pass 0 merges the stored partials and, with deferred compaction, takes the evicted entries' terms out of the
  // sums.  A head whose evicted entries hold more than 90 % of the mass is redone below.
  bool redo = false;
  if (has_head) {
    float res[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) res[k] = 0.f;
    float M = NEG_INF, L = 0.f;
    merge_stored_range(w0, w1, hh, M, L, res);
    if (call.defer) {
      push_new(M, L, res);
      float Lsub = 0.f, sub[CPL];
#pragma unroll
      for (int k = 0; k < CPL; ++k) sub[k] = 0.f;
      for (int a = 0; a < ne; ++a) {
        if (__shfl_sync(0xffffffffu, ev_l, a) >= n_old) continue;  // the new token itself: it was never added
        float ke[CPL], ve[CPL];
        if (a == 0) {
#pragma unroll
          for (int k = 0; k < CPL; ++k) { ke[k] = ek0[k]; ve[k] = ev0[k]; }
        } else {
          const bf16* kr = sc.evK + ((size_t)i * p.tail + a) * p.Dkv + h * DH;
          const bf16* vr = sc.evV + ((size_t)i * p.tail + a) * p.Dkv + h * DH;
#pragma unroll
          for (int k = 0; k < CPL; ++k) { ke[k] = __bfloat162float(kr[lane + 32 * k]); ve[k] = __bfloat162float(vr[lane + 32 * k]); }
        }
        float dot = 0.f;
#pragma unroll
        for (int k = 0; k < CPL; ++k) dot = fmaf(qv[k], ke[k], dot);
        const float w = exp2f(warp_sum_f(dot) * sl2 - M);
        Lsub += w;
#pragma unroll
        for (int k = 0; k < CPL; ++k) sub[k] = fmaf(w, ve[k], sub[k]);
      }
      if (Lsub <= 0.9f * L) {
        L -= Lsub;
#pragma unroll
        for (int k = 0; k < CPL; ++k) res[k] -= sub[k];
      } else {
        redo = true;  // the evicted entries dominate this head's softmax
        if (lane == 0) atomicAdd(st.status + 1, 1);
#pragma unroll
        for (int k = 0; k < CPL; ++k) s_q[warp][lane + 32 * k] = qv[k];
      }
    }
    if (!redo) store_head(L, res);
  }
  IM_MARK(sc, call.layer, 1, 4);
  if (!call.defer) return;  // (block uniform)
  if (lane == 0) s_redo[warp] = redo ? 1 : 0;
  __syncthreads();
  // Redo of a head, by all warps of the block: the partials whose key range holds an evicted entry are recomputed
  // from the cache, which is still uncompacted, without that entry (the others are exact already).  The 32-key
  // rounds of such a range go round-robin over the warps; within a round a lane forms its key's whole dot product
  // (q from shared memory; 16 independent 16-byte loads), then the warp adds the 32 weighted V rows, lane l holding
  // columns CPL l .. CPL l + CPL - 1 (32 independent loads).  The warps' softmax states are merged in warp order by
  // the warp that owns the head, like stored partials.
  for (int hq = 0; hq < p.Gq; ++hq) {
    if (!s_redo[hq]) continue;  // (block uniform)
    const bool owner = warp == hq;
    float res[CPL];
#pragma unroll
    for (int k = 0; k < CPL; ++k) res[k] = 0.f;
    float M = NEG_INF, L = 0.f;
    for (long long wv = w0; wv <= w1; ++wv) {
      int key0, key1;
      partial_keys(wv, key0, key1);
      bool dirty = false;
      for (int a = 0; a < ne; ++a) {
        const int sl = __shfl_sync(0xffffffffu, ev_l, a);
        dirty |= sl >= key0 && sl < key1;
      }
      if (!dirty) {
        if (owner) merge_stored(wv, hq, M, L, res);
        continue;
      }
      const float* sq = s_q[hq];
      float Mr = NEG_INF, Lr = 0.f, racc[CPL];
#pragma unroll
      for (int k = 0; k < CPL; ++k) racc[k] = 0.f;
      for (int t0 = key0 + 32 * warp; t0 < key1; t0 += 32 * nwarps) {
        const int tk = t0 + lane;
        bool valid = tk < key1;
        for (int a = 0; a < ne; ++a) valid &= __shfl_sync(0xffffffffu, ev_l, a) != tk;
        const uint4* kr = reinterpret_cast<const uint4*>(Kb + (size_t)min(tk, key1 - 1) * DH);
        uint4 kw[DH / 8];
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) kw[c] = kr[c];
        uint2 vw[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const bf16* vr = Vb + (size_t)min(t0 + j, key1 - 1) * DH + CPL * lane;
          if (CPL == 4) vw[j] = *reinterpret_cast<const uint2*>(vr);
          else { vw[j].x = *reinterpret_cast<const uint32_t*>(vr); vw[j].y = 0u; }
        }
        float sd = 0.f;
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
          const uint32_t ww[4] = {kw[c].x, kw[c].y, kw[c].z, kw[c].w};
#pragma unroll
          for (int e2 = 0; e2 < 4; ++e2) {
            sd = fmaf(sq[c * 8 + 2 * e2], __uint_as_float(ww[e2] << 16), sd);
            sd = fmaf(sq[c * 8 + 2 * e2 + 1], __uint_as_float(ww[e2] & 0xffff0000u), sd);
          }
        }
        sd = valid ? sd * sl2 : NEG_INF;
        float mb = sd;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, o));
        if (mb == NEG_INF) continue;  // (warp-uniform) nothing left in this round
        const float Mn = fmaxf(Mr, mb);
        const float eo = exp2f(Mr - Mn);
        const float pl = valid ? exp2f(sd - Mn) : 0.f;
        Lr = Lr * eo + warp_sum_f(pl);
#pragma unroll
        for (int k = 0; k < CPL; ++k) racc[k] *= eo;
        Mr = Mn;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float pj = __shfl_sync(0xffffffffu, pl, j);
          racc[0] = fmaf(pj, __uint_as_float(vw[j].x << 16), racc[0]);
          racc[1] = fmaf(pj, __uint_as_float(vw[j].x & 0xffff0000u), racc[1]);
          if (CPL == 4) {
            racc[2] = fmaf(pj, __uint_as_float(vw[j].y << 16), racc[2]);
            racc[3] = fmaf(pj, __uint_as_float(vw[j].y & 0xffff0000u), racc[3]);
          }
        }
      }
      // this warp's state of the range: columns CPL l + k -> l + 32 k through shared memory
      float* stw = s_st[warp];
#pragma unroll
      for (int k = 0; k < CPL; ++k) stw[CPL * lane + k] = racc[k];
      if (lane == 0) { stw[DH] = Mr; stw[DH + 1] = Lr; }
      __syncthreads();
      if (owner) {
        for (int w = 0; w < nwarps; ++w) {
          const float Mw = s_st[w][DH], Lw = s_st[w][DH + 1];
          if (!(Lw > 0.f)) continue;
          const float Mn = fmaxf(M, Mw);
          const float eo = exp2f(M - Mn), en = exp2f(Mw - Mn);
          L = L * eo + Lw * en;
#pragma unroll
          for (int k = 0; k < CPL; ++k) res[k] = res[k] * eo + s_st[w][lane + 32 * k] * en;
          M = Mn;
        }
      }
      __syncthreads();
    }
    if (owner) {
      push_new(M, L, res);
      store_head(L, res);
    }
  }
  IM_MARK(sc, call.layer, 1, 5);
}


typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// Encodes the tensor maps of the K and V caches: 2-D [rows = units * Hkv * cap, cols = d] bf16,
// box = 64 columns x box_rows rows, 128-byte swizzle.  Returns false if the fast path is unavailable.
bool im_attn_fast_supported(const ImDims& p) { return (p.d == 64 || p.d == 128) && p.Gq <= 8 && p.Dkv % 4 == 0; }

// halves3d (head_dim 128 only): the 256-byte rows as two 128-byte halves on a third dimension, dims (64 columns, rows,
// 2 halves) with strides (256, 128) bytes and box (64, box_rows, 2): one copy brings a whole tile, laid out in shared
// memory as the two 2-D boxes of its halves would be.
cudaError_t im_attn_make_maps(const ImDims& p, const ImState& st, void* mapK, void* mapV, int box_rows, int halves3d) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (!fn || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  EncodeTiledFn enc = (EncodeTiledFn)fn;
  const cuuint64_t rows = (cuuint64_t)p.L * p.S * p.Hkv * p.cap;
  const cuuint64_t dims[2] = {(cuuint64_t)p.d, rows};
  const cuuint64_t strides[1] = {(cuuint64_t)p.d * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  void* bases[2] = {st.Kc, st.Vc};
  void* maps[2] = {mapK, mapV};
  const cuuint64_t dims3[3] = {64, rows, 2};
  const cuuint64_t strides3[2] = {(cuuint64_t)p.d * 2, 128};
  const cuuint32_t box3[3] = {64, (cuuint32_t)box_rows, 2};
  const cuuint32_t estr3[3] = {1, 1, 1};
  if (halves3d && p.d != 128) return cudaErrorInvalidValue;
  for (int k = 0; k < 2; ++k) {
    CUresult r = halves3d
        ? enc((CUtensorMap*)maps[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, bases[k], dims3, strides3, box3, estr3,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE)
        : enc((CUtensorMap*)maps[k], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bases[k], dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  return cudaSuccess;
}

size_t im_attn_smem_bytes(const ImDims& p, int n_seq) {
  const size_t stage = (size_t)2 * TILE * p.d * 2;
  return (size_t)WARPS * STAGES * stage + (size_t)WARPS * STAGES * 8 + (size_t)(n_seq + 1) * 8 + (size_t)n_seq * 4 + (1 + WARPS * 4) * 4 + 64;
}

cudaError_t im_attn_prepare(const ImDims& p) {
  const int smem = (int)im_attn_smem_bytes(p, IM_MAX_CALL_SEQS);
  cudaError_t e = cudaFuncSetAttribute(k_attn_stream<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_attn_stream<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_attn_stream<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_attn_stream<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_stream<64, false>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_stream<128, false>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_stream<64, true>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_stream<128, true>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_readout_cols);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_readout_cols_dyn);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_readout_cols_light);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_readout_finish);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_merge_rows<64, bf16>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_merge_rows<64, float>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_merge_rows<128, bf16>);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_merge_rows<128, float>);
  return e;
}

cudaError_t im_launch_readout(const ImLaunch& L, const ImCall& call, int grid, int light) {
  const ImDims& p = L.p;
  const int depth = light ? 8 : 32;
  const int nb = (p.dM + RC_RPR * depth - 1) / (RC_RPR * depth);
  const int items = call.n_seq * (p.Dkv / RC_COLS);
  const size_t smem = (size_t)nb * RC_RPR * depth * 4;
  const int blocks = std::max(1, std::min(grid, items));
  if (call.stack) k_readout_cols_dyn<<<blocks, RC_THREADS, smem, L.stream>>>(p, L.st, L.sc, call);
  else if (light) k_readout_cols_light<<<blocks, RC_THREADS, smem, L.stream>>>(p, L.st, L.sc, call);
  else k_readout_cols<<<blocks, RC_THREADS, smem, L.stream>>>(p, L.st, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_readout_finish(const ImLaunch& L, const ImCall& call) {
  k_readout_finish<<<call.n_seq, 256, (size_t)L.p.dM * 4, L.stream>>>(L.p, L.st, L.w, L.sc, call);
  ++*L.launches;
  return cudaGetLastError();
}

cudaError_t im_launch_attention_fast(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                     const void* q, int n_ctas, int programmatic) {
  const ImDims& p = L.p;
  const CUtensorMap& mk = *(const CUtensorMap*)mapK;
  const CUtensorMap& mv = *(const CUtensorMap*)mapV;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(WARPS * 32);
  cfg.dynamicSmemBytes = im_attn_smem_bytes(p, call.n_seq);
  cfg.stream = L.stream;
  // programmatic: the kernel may start while the kernel before it in the stream is still running (it waits for it,
  // griddepcontrol.wait, before it touches anything but this layer's cache)
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  cudaError_t e;
  if (call.stack) {
    if (p.d == 64) e = cudaLaunchKernelEx(&cfg, k_attn_stream<64, true>, mk, mv, p, L.st, L.sc, call, (const bf16*)q);
    else e = cudaLaunchKernelEx(&cfg, k_attn_stream<128, true>, mk, mv, p, L.st, L.sc, call, (const bf16*)q);
  } else {
    if (p.d == 64) e = cudaLaunchKernelEx(&cfg, k_attn_stream<64, false>, mk, mv, p, L.st, L.sc, call, (const bf16*)q);
    else e = cudaLaunchKernelEx(&cfg, k_attn_stream<128, false>, mk, mv, p, L.st, L.sc, call, (const bf16*)q);
  }
  ++*L.launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t im_launch_attention_merge(const ImLaunch& L, const ImCall& call, void* out, int n_workers, int tile, int ro_workers,
                                      const void* q, const void* k_new, const void* v_new, int programmatic) {
  const int ro_cs = ro_workers > 0 ? im_readout_stream_chunks(L.p) : 0;
  const bf16* qp = (const bf16*)q;
  const bf16* kp = (const bf16*)k_new;
  const bf16* vp = (const bf16*)v_new;
  const ImDims& p = L.p;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.Hkv, call.n_seq);
  cfg.blockDim = dim3(32 * std::max(p.Gq, p.d / 32));
  cfg.stream = L.stream;
  // programmatic: the kernel before this one in the stream is the attention kernel, which releases its dependents
  // when its last tiles are requested; this kernel waits for it (griddepcontrol.wait) before it reads its output
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  cudaError_t e;
  if (p.d == 64) {
    if (p.out_f32) e = cudaLaunchKernelEx(&cfg, k_attn_merge_rows<64, float>, p, L.st, L.sc, call, n_workers, tile, ro_workers, ro_cs, (float*)out, qp, kp, vp);
    else e = cudaLaunchKernelEx(&cfg, k_attn_merge_rows<64, bf16>, p, L.st, L.sc, call, n_workers, tile, ro_workers, ro_cs, (bf16*)out, qp, kp, vp);
  } else {
    if (p.out_f32) e = cudaLaunchKernelEx(&cfg, k_attn_merge_rows<128, float>, p, L.st, L.sc, call, n_workers, tile, ro_workers, ro_cs, (float*)out, qp, kp, vp);
    else e = cudaLaunchKernelEx(&cfg, k_attn_merge_rows<128, bf16>, p, L.st, L.sc, call, n_workers, tile, ro_workers, ro_cs, (bf16*)out, qp, kp, vp);
  }
  ++*L.launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

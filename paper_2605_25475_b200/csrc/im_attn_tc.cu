// a5, B200 path for head_dim 128: attention over the retained entries as a persistent, warp-specialised
// flash-decode kernel on the 5th-generation tensor cores.
//
// The kernel is HBM-bound (every retained K/V byte is read once per step); its job is to keep as many bytes in
// flight per SM as the shared memory holds and to keep the arithmetic out of the way of the loads:
//   * the retained entries of a (sequence, KV head) row form tiles of 128 keys; all tiles of all rows are cut into
//     equal contiguous runs, one run per CTA (stream-K: perfect balance for any mix of lengths, at most one partial
//     result per row boundary inside a run);
//   * warp 4 (one lane) feeds a CTA-wide ring of 64 KB stages (K tile + V tile) with TMA tensor copies, 128-byte
//     swizzle, as many 32-row boxes as the tile has entries, and re-arms a stage the moment its products are done;
//   * warp 5 issues tcgen05.mma with the KEYS on the M axis (= the 128 TMEM lanes) and the G_q query heads of the
//     KV head on N (16 columns, the heads in the first G_q): S^T = K Q^T (A = the K tile as cached, K-major), then
//     O^T += V^T P^T (A = the V tile as cached, i.e. MN-major; B = P^T written to shared memory by the softmax
//     threads).  The products are asynchronous: nothing in this kernel waits for arithmetic except the thread that
//     needs its result;
//   * warps 0-3 are the softmax: thread t owns key t of the tile (TMEM lane t), reads its G_q scores with
//     tcgen05.ld, forms P = 2^(s - m_ref) against a reference maximum per head that all threads share and that is
//     raised only when some score exceeds it by more than 2^8 (one barrier.red.or over the 128 threads per tile
//     decides; the raise itself - maxima through shared memory, O^T rescaled in tensor memory - is rare), splits P
//     into two bf16 terms (2^-17) and stores them for the second product.
// Columns of B beyond the G_q heads are never initialised: a column of the accumulator depends on its own column
// of B alone, and those columns are not read.
// Every wait is bounded; a wait that runs out sets ST_TIMEOUT and an abort flag that the other roles poll, the
// producer then waits (again bounded) for every copy it has in flight, and the CTA frees its tensor memory.
#include <cuda.h>

#include <algorithm>

#include "im_internal.cuh"

// Development aid (off in the library build): with IM_ATTN_TRACE defined, one CTA records the SM clock at the steps
// of every tile's way through the pipeline into im_attn_trace[tile][step].
#ifdef IM_ATTN_TRACE
__device__ long long im_attn_trace[512][12];
__device__ unsigned long long im_attn_span[1024][2];  // per CTA: global timer (ns) at entry and exit
__device__ __forceinline__ unsigned long long im_gtimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define TRACE(k, step)                                                                 \
  do {                                                                                 \
    if (blockIdx.x == IM_ATTN_TRACE && (k) < 512) im_attn_trace[(k)][(step)] = clock64(); \
  } while (0)
#else
#define TRACE(k, step) \
  do {                 \
  } while (0)
#endif

namespace {

constexpr float NEG_INF = -__builtin_huge_valf();
constexpr int DH = 128;
constexpr int KT = IM_ATTN_TC_TILE;          // keys per tile = TMEM lanes
constexpr int BOX = IM_ATTN_TILE;            // rows per TMA box (the tensor maps of the cache: 64 columns x 32 rows)
constexpr int SLOTS = 2;                     // tiles in each of the two rings (K tiles, V tiles)
constexpr int HALF_BYTES = KT * 128;         // one 64-column half of a K or V tile: 128 rows x 128 bytes
constexpr int KV_TILE = 2 * HALF_BYTES;      // 32 KB
constexpr int RING_BYTES = 2 * SLOTS * KV_TILE;
constexpr int NCOL = 16;                     // accumulator columns (N of both products)
constexpr int OP_HALF = 8 * 128;             // one 64-element half of a B operand held as 8 rows x 128 bytes
constexpr int Q_BYTES = 2 * OP_HALF;         // Q^T of one segment: rows = heads, 128 elements per row
constexpr int P_BYTES = 2 * OP_HALF;         // one bf16 term of P^T of one tile: rows = heads, 128 keys per row
constexpr int THREADS = 192;                 // warps 0-3 softmax, 4 TMA, 5 tensor memory / MMA issue
constexpr uint32_t WAIT_LIMIT = IM_WAIT_LIMIT;
constexpr int TMEM_COLS = 64;                // S^T double buffered at 0 / 16, O^T at 32
constexpr int S_COL = 0, O_COL = 32;

struct Shared {
  unsigned long long fullK[SLOTS], emptyK[SLOTS], fullV[SLOTS], emptyV[SLOTS], sfull[2], sempty[2], pfull[2], pvdone[2];
  uint32_t tmem;
  int abort;
  int ragged;                            // some sequence of the call has a last tile that is not full
  float red[4][8];                       // per softmax warp: tile maxima / row sums of the G_q heads
  long long pref[IM_MAX_CALL_SEQS + 1];  // tiles before sequence i (all KV heads)
  int n[IM_MAX_CALL_SEQS];               // entries per sequence
};
// ring | Q^T x 2 | P^T x 2 buffers x 2 terms | Shared
constexpr int OPS_BYTES = 2 * Q_BYTES + 4 * P_BYTES + OP_HALF;  // + one half: the descriptors of the last buffer read 16 rows
constexpr int SMEM_BYTES = RING_BYTES + OPS_BYTES + (int)sizeof(Shared);

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// bounded wait; gives up early when another role of the CTA has given up
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit = WAIT_LIMIT) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if ((it & 63) == 63 && *abort_flag) return false;
  }
  return false;
}
// the same without the early exit: the drain of copies in flight keeps the full limit
__device__ __forceinline__ bool mbar_wait_full(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}
// one look at a barrier: has the phase completed?
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return done != 0;
}
// the same by a whole warp  (warp-uniform: completion is final, so one lane
// that has seen it speaks for all)
__device__ __forceinline__ bool mbar_test_warp(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(done)
      : "r"(bar), "r"(parity)
      : "memory");
  return __any_sync(0xffffffffu, done != 0);
}
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
// shared-memory operand descriptor, 128-byte swizzle: lbo / sbo in bytes
__device__ __forceinline__ uint64_t desc_sw128(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of this architecture
  d |= (uint64_t)2 << 61;  // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a), "l"(b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .pred q;\n\t"
      "elect.sync _|q, 0xffffffff;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t r[8];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int k = 0; k < 8; ++k) v[k] = __uint_as_float(r[k]);
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n\t"
      "tcgen05.wait::st.sync.aligned;" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7]))
      : "memory");
}
// 2^x; -inf gives 0
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// OR of a predicate over the 128 softmax threads (named barrier 1), every thread gets the result
__device__ __forceinline__ bool softmax_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %1, 0;\n\t"
      "barrier.cta.red.or.pred.aligned q, 1, 128, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void softmax_sync() { asm volatile("barrier.cta.sync.aligned 1, 128;" ::: "memory"); }

__device__ __forceinline__ int tiles_of(int n) { return (n + KT - 1) / KT; }

// Position of a run in the row structure: sequence i, KV head h, tile tt of nt.
struct Cursor {
  int i, h, tt, nt;
};
__device__ __forceinline__ void cursor_next_row(Cursor& c, const Shared* sh, int n_seq, int Hkv) {
  c.tt = 0;
  if (++c.h == Hkv) {
    c.h = 0;
    do { ++c.i; } while (c.i < n_seq && tiles_of(sh->n[c.i]) == 0);
    c.nt = c.i < n_seq ? tiles_of(sh->n[c.i]) : 1;
  }
}

// grid = CTAs (at most one per SM), block = 192.
__global__ void __launch_bounds__(THREADS, 1)
k_attn_stream_tc(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmK128, const __grid_constant__ CUtensorMap tmV128, ImDims p, ImState st,
                 ImScratch sc, ImCall call, const bf16* __restrict__ q) {
  extern __shared__ __align__(1024) uint8_t smem[];
  uint8_t* s_k = smem;                              // [SLOTS][2 halves][128 rows x 128 bytes]
  uint8_t* s_v = smem + SLOTS * KV_TILE;            // the same
  uint8_t* s_q = smem + RING_BYTES;                 // [2][2 halves][8 rows x 128 bytes]
  uint8_t* s_p = s_q + 2 * Q_BYTES;                 // [2 buffers][2 terms][2 halves][8 rows x 128 bytes]
  Shared* sh = reinterpret_cast<Shared*>(s_q + OPS_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = &sh->abort;
  if (tid == 0) TRACE(500, 0);
#ifdef IM_ATTN_TRACE
  if (tid == 0) im_attn_span[blockIdx.x][0] = im_gtimer();
#endif

  // (behind the merge kernel of a call on the same layer nothing of this cache may be read before that kernel has ended)
  if (!call.early_cache) asm volatile("griddepcontrol.wait;" ::: "memory");
  // ---- tile prefix over the sequences of the call (every CTA computes the same table)
  for (int i = tid; i < call.n_seq; i += THREADS) {
    const size_t u = (size_t)call.layer * p.S + call.seq[i];
    sh->n[i] = max(0, min(st.ctr[u * CTR_STRIDE + CTR_N], p.cap));
  }
  if (tid == 0) {
    for (int s = 0; s < SLOTS; ++s) {
      mbar_init(smem_u32(&sh->fullK[s]), 1);
      mbar_init(smem_u32(&sh->emptyK[s]), 1);
      mbar_init(smem_u32(&sh->fullV[s]), 1);
      mbar_init(smem_u32(&sh->emptyV[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&sh->sfull[b]), 1);
      mbar_init(smem_u32(&sh->sempty[b]), KT);
      mbar_init(smem_u32(&sh->pfull[b]), KT);
      mbar_init(smem_u32(&sh->pvdone[b]), 1);
    }
    sh->abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (tid == 0) {
    long long acc = 0;
    int ragged = 0;
    for (int i = 0; i < call.n_seq; ++i) {
      sh->pref[i] = acc;
      acc += (long long)tiles_of(sh->n[i]) * p.Hkv;
      ragged |= sh->n[i] % KT;
    }
    sh->pref[call.n_seq] = acc;
    sh->ragged = ragged;
  }
  __syncthreads();
  // Rows whose last tile is ragged leave the rest of a ring stage as it is.  Those rows of the stage must hold finite
  // numbers (they are multiplied by P = 0): cache data of an earlier tile is, uninitialised shared memory need not
  // be, so the ring starts as zeros whenever some row of the call has a ragged tail.
  if (sh->ragged) {
    for (int k = tid; k < RING_BYTES / 16; k += THREADS) reinterpret_cast<uint4*>(smem)[k] = make_uint4(0u, 0u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (tid == 0) TRACE(500, 1);
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh->tmem;
  if (tid == 0) TRACE(500, 2);
  const long long total = sh->pref[call.n_seq];
  const long long qrun = (total + gridDim.x - 1) / gridDim.x;
  const long long run0 = min(total, (long long)blockIdx.x * qrun), run1 = min(total, run0 + qrun);
  const bool has_work = run0 < run1;

  // ---- position of the first tile of the run
  Cursor c0 = {0, 0, 0, 1};
  if (has_work) {
    int lo = 0, hi = call.n_seq;  // last i with pref[i] <= run0
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (sh->pref[mid] <= run0) lo = mid; else hi = mid;
    }
    c0.i = lo;
    while (c0.i < call.n_seq - 1 && tiles_of(sh->n[c0.i]) == 0) ++c0.i;  // empty sequences own no tiles
    c0.nt = max(1, tiles_of(sh->n[c0.i]));
    c0.h = (int)((run0 - sh->pref[c0.i]) / c0.nt);
    c0.tt = (int)((run0 - sh->pref[c0.i]) % c0.nt);
  }
  bool ok = true;

  if (warp == 4) {
    // ================= TMA producer (one lane).  K tiles and V tiles go through rings of their own: a K slot is
    // free again as soon as the tile's first product has run, long before the V slot of the same tile, and every
    // microsecond a slot is held is a microsecond in which it holds no load in flight.
    long long jk = run0, jv = run0;  // next K / V tile to request
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      Cursor ck = c0, cv = c0;
      auto issue = [&](long long j, Cursor& c, bool is_v) {
        const int s = (int)((j - run0) % SLOTS);
        const uint32_t bar = smem_u32(is_v ? &sh->fullV[s] : &sh->fullK[s]);
        const uint32_t dst = smem_u32((is_v ? s_v : s_k) + (size_t)s * KV_TILE);
        const size_t u = (size_t)call.layer * p.S + call.seq[c.i];
        const int row = (int)((u * p.Hkv + c.h) * (size_t)p.cap) + c.tt * KT;
        const int left = sh->n[c.i] - c.tt * KT;
        TRACE(j - run0, is_v ? 7 : 0);
        if (left >= KT) {
          // a full tile: one 128-row box per 64-column half (a box is one request to the copy engine, and the
          // engine's request rate, not the memory, bounds a stream of 4 KB boxes)
          mbar_expect_tx(bar, (uint32_t)KV_TILE);
#pragma unroll
          for (int hf = 0; hf < 2; ++hf) tma_load_2d(dst + hf * HALF_BYTES, is_v ? &tmV128 : &tmK128, hf * 64, row, bar, pol);
        } else {
          // the ragged last tile of a row: as many 32-row boxes as hold entries (1..4), so that no slot beyond the
          // row's entries (uninitialised memory, or another row) is ever read
          const int nb = (left + BOX - 1) / BOX;
          mbar_expect_tx(bar, (uint32_t)nb * 2u * (BOX * 128));
          for (int b = 0; b < nb; ++b) {
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
              tma_load_2d(dst + hf * HALF_BYTES + b * (BOX * 128), is_v ? &tmV : &tmK, hf * 64, row + b * BOX, bar, pol);
          }
        }
        if (++c.tt == c.nt) cursor_next_row(c, sh, call.n_seq, p.Hkv);
      };
      // the first tiles are requested before the dependency wait: they come from this layer's cache alone
      for (int k = 0; k < SLOTS && jk < run1; ++k) {
        issue(jk++, ck, false);
        issue(jv++, cv, true);
      }
      if (jv == run1) asm volatile("griddepcontrol.launch_dependents;");
      asm volatile("griddepcontrol.wait;" ::: "memory");
      uint32_t idle = 0;
      while (jv < run1) {
        bool progressed = false;
        if (jk < run1) {
          const long long k = jk - run0;
          if (mbar_test(smem_u32(&sh->emptyK[k % SLOTS]), (uint32_t)(((k / SLOTS) - 1) & 1))) {
            issue(jk++, ck, false);
            progressed = true;
          }
        }
        {
          const long long k = jv - run0;
          if (jv < jk && mbar_test(smem_u32(&sh->emptyV[k % SLOTS]), (uint32_t)(((k / SLOTS) - 1) & 1))) {
            issue(jv++, cv, true);
            progressed = true;
            // the last tile of this CTA's run is requested: a kernel launched as programmatic dependent (the merge) may
            // become resident and run the part of its prologue that does not read this kernel's output
            if (jv == run1) asm volatile("griddepcontrol.launch_dependents;");
          }
        }
        if (progressed) idle = 0;
        else {
          if (++idle >= WAIT_LIMIT || ((idle & 63) == 0 && *abort_flag)) { ok = false; break; }
          __nanosleep(40);
        }
      }
      if (!ok) {
        sh->abort = 1;
        atomicOr(st.status, ST_TIMEOUT);
      }
    }
    // Before the CTA ends, every copy this lane has requested must have landed (shared memory of an ended CTA may be
    // given to the next one).  After a normal run these waits return at once; after a give-up, of this role or of
    // another, each gets the full limit.
    if (lane == 0) {
      for (long long j = max(run0, jk - SLOTS); j < jk; ++j)
        if (!mbar_wait_full(smem_u32(&sh->fullK[(j - run0) % SLOTS]), (uint32_t)(((j - run0) / SLOTS) & 1))) atomicOr(st.status, ST_TIMEOUT);
      for (long long j = max(run0, jv - SLOTS); j < jv; ++j)
        if (!mbar_wait_full(smem_u32(&sh->fullV[(j - run0) % SLOTS]), (uint32_t)(((j - run0) / SLOTS) & 1))) atomicOr(st.status, ST_TIMEOUT);
    }
  } else if (warp == 5) {
    // ================= MMA issue: the whole warp runs the loop (descriptors stay warp-uniform), one elected lane issues
    asm volatile("griddepcontrol.wait;" ::: "memory");  // q may be the previous kernel's output
    if (has_work) {
      // instruction descriptors: f32 accumulators, bf16 operands, N = 16, M = 128; the second product reads A = V^T
      // MN-major (the tile lies [key][d] in shared memory)
      const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NCOL >> 3) << 17) | ((uint32_t)(KT >> 4) << 24);
      const uint32_t idesc_o = idesc_s | (1u << 15);
      Cursor c = c0;
      int seg = 0;                 // segments (rows) met so far: parity selects the Q^T buffer
      bool seg_first = true;       // the tile whose first product comes next is the first of its segment within this run
      // The two products of a tile are issued when their inputs are there, whichever comes first: the second product
      // of tile jp as soon as its P is stored (it frees the tile's ring stage, so it goes first), the first product
      // of tile js as soon as the tile has landed and the score buffer of tile js - 2 has been read.  Neither waits
      // for the other: with the products in one fixed order the release of a stage waited for the NEXT tile's load.
      long long js = run0, jp = run0;
      uint32_t firsts = 0;  // bit (k & 31): tile k of the run starts a segment (the window js - jp stays below 8)
      uint32_t idle = 0;
      while (jp < run1) {
        bool progressed = false;
        if (jp < js) {
          const long long k = jp - run0;
          const int b = (int)(k & 1), s = (int)(k % SLOTS);
          if (mbar_test_warp(smem_u32(&sh->pfull[b]), (uint32_t)((k >> 1) & 1)) &&
              mbar_test_warp(smem_u32(&sh->fullV[s]), (uint32_t)((k / SLOTS) & 1))) {  // O^T (+)= V^T P^T of tile jp
            if (lane == 0) TRACE(k, 5);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const bool first = (firsts >> (k & 31)) & 1u;
            const uint32_t va = smem_u32(s_v + (size_t)s * KV_TILE);
            const uint32_t pa = smem_u32(s_p + (size_t)b * 2 * P_BYTES);
#pragma unroll
            for (int term = 0; term < 2; ++term)
#pragma unroll
              for (int ks = 0; ks < KT / 16; ++ks)
                mma_bf16(tmem + O_COL, desc_sw128(va + ks * 2048, HALF_BYTES, 1024),
                         desc_sw128(pa + term * P_BYTES + (ks >> 2) * OP_HALF + (ks & 3) * 32, 16, 1024), idesc_o,
                         (first && term == 0 && ks == 0) ? 0u : 1u);
            mma_commit(smem_u32(&sh->pvdone[b]));
            mma_commit(smem_u32(&sh->emptyV[s]));
            if (lane == 0) TRACE(k, 6);
            ++jp;
            progressed = true;
          }
        }
        if (js < run1) {
          const long long k = js - run0;
          const int b = (int)(k & 1), s = (int)(k % SLOTS);
          if ((k < 2 || mbar_test_warp(smem_u32(&sh->sempty[b]), (uint32_t)(((k >> 1) - 1) & 1))) &&
              mbar_test_warp(smem_u32(&sh->fullK[s]), (uint32_t)((k / SLOTS) & 1))) {  // S^T = K Q^T of tile js
            if (lane == 0) TRACE(k, 1);
            if (seg_first) {
              // Q^T of the segment: row g = head g of the group, 16-byte chunk ch of row g at the swizzled place.  The
              // buffer of this parity was last read by first products of tiles at least two back, which are complete
              // (the softmax threads have read the scores of tile js - 2)
              uint8_t* qb = s_q + (seg & 1) * Q_BYTES;
              for (int e = lane; e < p.Gq * 16; e += 32) {
                const int g = e >> 4, ch = e & 15;
                const uint4 v = *reinterpret_cast<const uint4*>(q + ((size_t)c.i * p.H + (size_t)c.h * p.Gq + g) * DH + ch * 8);
                *reinterpret_cast<uint4*>(qb + (ch >> 3) * OP_HALF + g * 128 + (((ch & 7) ^ (g & 7)) << 4)) = v;
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
              __syncwarp();
            }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t ka = smem_u32(s_k + (size_t)s * KV_TILE);
            const uint32_t qa = smem_u32(s_q + (seg & 1) * Q_BYTES);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
              mma_bf16(tmem + (uint32_t)(S_COL + b * NCOL), desc_sw128(ka + (ks >> 2) * HALF_BYTES + (ks & 3) * 32, 16, 1024),
                       desc_sw128(qa + (ks >> 2) * OP_HALF + (ks & 3) * 32, 16, 1024), idesc_s, ks ? 1u : 0u);
            mma_commit(smem_u32(&sh->sfull[b]));
            mma_commit(smem_u32(&sh->emptyK[s]));
            if (lane == 0) TRACE(k, 2);
            firsts = (firsts & ~(1u << (k & 31))) | ((seg_first ? 1u : 0u) << (k & 31));
            seg_first = false;
            if (++c.tt == c.nt) {
              cursor_next_row(c, sh, call.n_seq, p.Hkv);
              ++seg;
              seg_first = true;
            }
            ++js;
            progressed = true;
          }
        }
        if (progressed) idle = 0;
        else {
          if (idle >= p.wait_limit || ((idle & 63) == 63 && *abort_flag)) { ok = false; break; }  // (warp uniform)
          ++idle;
          __nanosleep(40);  // this warp shares its scheduler with a softmax warp: do not spin at full rate
        }
      }
      if (!ok && lane == 0) {
        sh->abort = 1;
        atomicOr(st.status, ST_TIMEOUT);
      }
    }
  } else {
    // ================= softmax (warps 0-3): thread t = key t of the tile = TMEM lane t
    // A wait that runs out does not leave the loop on its own (the other threads would wait for this one at the next
    // named barrier): it is recorded in `fail`, the abort flag makes every later wait of the CTA return at once,
    // and the threads leave together where the per-tile reduction shows the failure to all of them.
    im_warm_inputs(call, blockIdx.x, tid, KT);  // (the first CTAs: one input tensor each)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (blockIdx.x == 0)  // what the merge kernel rebuilds the tile bookkeeping from
      for (int k = tid; k < call.n_seq; k += KT) sc.n_att[k] = sh->n[k];
    if (has_work) {
      const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
      const float sl2 = p.scale * 1.4426950408889634f;  // softmax in base 2
      Cursor c = c0;
      long long j = run0;
      bool fail = false;
      auto wait = [&](unsigned long long* bar, uint32_t parity) {
        const bool got = mbar_wait(smem_u32(bar), parity, abort_flag, p.wait_limit);
        if (!got) { fail = true; sh->abort = 1; }
        return got;
      };
      while (j < run1 && ok) {
        // ---- one (sequence, KV head) segment of the run
        const int n = sh->n[c.i];
        const long long row_id = (long long)c.i * p.Hkv + c.h;
        float m_ref[8], l[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) { m_ref[g] = NEG_INF; l[g] = 0.f; }
        bool seg_first = true;
        for (; c.tt < c.nt && j < run1; ++c.tt, ++j) {
          const int b = (int)((j - run0) & 1);
          const uint32_t par = (uint32_t)(((j - run0) >> 1) & 1);
          float x[8];
#pragma unroll
          for (int g = 0; g < 8; ++g) x[g] = NEG_INF;
          if (wait(&sh->sfull[b], par)) {
            if (tid == 0) TRACE(j - run0, 3);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            tmem_ld8(tmem + lane_addr + (uint32_t)(S_COL + b * NCOL), x);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          }
          mbar_arrive(smem_u32(&sh->sempty[b]));
          if (tid == 0) TRACE(j - run0, 8);
          const bool valid = c.tt * KT + tid < n;
          bool exceed = false;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            x[g] = (valid && g < p.Gq) ? x[g] * sl2 : NEG_INF;
            exceed |= x[g] > m_ref[g] + 8.0f;  // (-inf + 8 = -inf: any finite score exceeds an unset reference)
          }
          const bool any_ex = softmax_any(exceed || fail);
          if (tid == 0) TRACE(j - run0, 9);
          if (any_ex) {
            if (softmax_any(fail)) { ok = false; break; }  // (uniform over the 128 threads)
            // ---- raise the references (rare): tile maxima per head through shared memory, then scale what has been
            // accumulated against the old references: the row sums here, O^T in tensor memory
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              float v = x[g];
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
              if (lane == 0) sh->red[warp][g] = v;
            }
            softmax_sync();
            float corr[8];
            bool any_scale = false;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const float tm = fmaxf(fmaxf(sh->red[0][g], sh->red[1][g]), fmaxf(sh->red[2][g], sh->red[3][g]));
              corr[g] = 1.0f;
              if (tm > m_ref[g] + 8.0f) {
                corr[g] = m_ref[g] == NEG_INF ? 0.f : ex2(m_ref[g] - tm);
                any_scale |= m_ref[g] != NEG_INF;
                m_ref[g] = tm;
                l[g] *= corr[g];
              }
            }
            softmax_sync();  // red is free again
            if (any_scale && !seg_first) {
              // O^T holds the products up to tile j - 1: wait for the last one, then scale the columns.  Thread t
              // owns row t (output column d = t of the head) of all 8 accumulator columns in use.
              const int bp = (int)((j - 1 - run0) & 1);
              if (wait(&sh->pvdone[bp], (uint32_t)(((j - 1 - run0) >> 1) & 1))) {
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                float o[8];
                tmem_ld8(tmem + lane_addr + O_COL, o);
#pragma unroll
                for (int g = 0; g < 8; ++g) o[g] *= corr[g];
                tmem_st8(tmem + lane_addr + O_COL, o);
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
              }
            }
          }
          // ---- P = 2^(x - m_ref) as two bf16 terms, stored as column t of row g of the B operand; the buffer was
          // last read by the second product of tile j - 2
          if (j - run0 >= 2) wait(&sh->pvdone[b], (uint32_t)((((j - run0) >> 1) - 1) & 1));
          uint8_t* pb = s_p + (size_t)b * 2 * P_BYTES + (tid >> 6) * OP_HALF;
          const int ch = (tid & 63) >> 3, within = (tid & 7) * 2;  // 16-byte chunk of the 128-byte row, byte offset in it
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            if (g < p.Gq) {
              const float pv = m_ref[g] == NEG_INF ? 0.f : ex2(x[g] - m_ref[g]);
              l[g] += pv;
              const uint32_t bits = __float_as_uint(pv);
              const float rem = pv - __uint_as_float(bits & 0xffff0000u);
              const uint16_t hi = (uint16_t)(bits >> 16);
              const uint16_t lo = (uint16_t)((__float_as_uint(rem) + 0x8000u) >> 16);
              uint8_t* dst = pb + g * 128 + ((ch ^ (g & 7)) << 4) + within;
              *reinterpret_cast<uint16_t*>(dst) = hi;
              *reinterpret_cast<uint16_t*>(dst + P_BYTES) = lo;
            }
          }
          if (tid == 0) TRACE(j - run0, 10);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          mbar_arrive(smem_u32(&sh->pfull[b]));
          if (tid == 0) TRACE(j - run0, 4);
          seg_first = false;
        }
        if (!ok) break;
        // ---- segment finished: wait for its last second product, write the partial (unnormalised O, reference, sum)
        // of this row.  Thread t holds output column d = t of every head.
        {
          const long long jl = j - 1;
          const int bl = (int)((jl - run0) & 1);
          float o[8];
#pragma unroll
          for (int g = 0; g < 8; ++g) o[g] = 0.f;
          if (wait(&sh->pvdone[bl], (uint32_t)(((jl - run0) >> 1) & 1))) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            tmem_ld8(tmem + lane_addr + O_COL, o);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          }
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            float v = l[g];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == 0) sh->red[warp][g] = v;
          }
          softmax_sync();
          // Rows are served by consecutive CTAs and consecutive rows share at most one CTA, so (CTA index + row
          // index) is a collision-free slot id below CTAs + rows.
          float* dst = sc.part + (size_t)((long long)blockIdx.x + row_id) * p.Gq * (DH + 2);
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            if (g < p.Gq) {
              dst[(size_t)g * (DH + 2) + tid] = o[g];
              if (tid == g) {
                dst[(size_t)g * (DH + 2) + DH] = m_ref[g];
                dst[(size_t)g * (DH + 2) + DH + 1] = sh->red[0][g] + sh->red[1][g] + sh->red[2][g] + sh->red[3][g];
              }
            }
          }
          softmax_sync();  // red is free again
        }
        if (c.tt == c.nt) {
          cursor_next_row(c, sh, call.n_seq, p.Hkv);
          if (c.i >= call.n_seq) break;
        }
      }
      if (softmax_any(fail)) ok = false;
      if (!ok && tid == 0) atomicOr(st.status, ST_TIMEOUT);
    }
  }
  if (tid == 0) TRACE(500, 3);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0) TRACE(500, 4);
#ifdef IM_ATTN_TRACE
  if (tid == 0) im_attn_span[blockIdx.x][1] = im_gtimer();
#endif
  if (warp == 5) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)TMEM_COLS) : "memory");
  }
}

}  // namespace

bool im_attn_tc_supported(const ImDims& p) { return p.d == DH && p.Gq <= 8 && p.Dkv % 4 == 0; }

cudaError_t im_attn_tc_prepare() {
  cudaError_t e = cudaFuncSetAttribute(k_attn_stream_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
  if (e == cudaSuccess) e = im_prefer_max_smem(k_attn_stream_tc);
  return e;
}

cudaError_t im_launch_attention_tc(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                   const void* mapK128, const void* mapV128, const void* q, int n_ctas, int programmatic) {
  const CUtensorMap& mk = *(const CUtensorMap*)mapK;
  const CUtensorMap& mv = *(const CUtensorMap*)mapV;
  const CUtensorMap& mk128 = *(const CUtensorMap*)mapK128;
  const CUtensorMap& mv128 = *(const CUtensorMap*)mapV128;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
  cfg.stream = L.stream;
  // programmatic: the kernel may start while the kernel before it in the stream is still running (it waits for it,
  // griddepcontrol.wait, before it touches anything but this layer's cache)
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = programmatic ? 1 : 0;
  cudaError_t e = cudaLaunchKernelEx(&cfg, k_attn_stream_tc, mk, mv, mk128, mv128, L.p, L.st, L.sc, call, (const bf16*)q);
  ++*L.launches;
  return e != cudaSuccess ? e : cudaGetLastError();
}

// Internal declarations shared by the translation units of libindexmem (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "indexmem.h"

typedef __nv_bfloat16 bf16;

#define IM_MAX_CALL_SEQS 256 /* sequences per hot call (the id list travels as a kernel parameter) */
#define IM_SLOT_ALIGN 64     /* slot capacity is a multiple of the attention tile */
#define IM_ATTN_TILE 32      /* rows of the small TMA box of the cache's tensor maps (32 rows x 128 bytes) */
#define IM_ATTN_MIN_RUN 4 /* tiles a warp of the streaming attention kernel should at least get (bounds the grid of small calls) */
#ifndef IM_ATTN_STREAM_TILE
#define IM_ATTN_STREAM_TILE 32 /* keys per tile (= rows of a TMA box) of the mma.sync streaming attention kernel */
#endif
#define IM_ATTN_WARPS 4      /* warps per CTA of the streaming attention kernel */
#define IM_ATTN_TC_TILE 128  /* keys per tile of the tensor-core streaming attention kernel (= the TMEM lanes) */
#define IM_ATTN_MAX_CTAS 512 /* upper bound of its grid (one CTA per SM) */
#define IM_TC_QT 32          /* queries per tile of the tensor-core prefill scoring */
#define IM_TC_HP 8           /* head slots per query in its operand (indexer heads, zero padded) */
#define IM_TC_TILE_BYTES 25600 /* one tile record: 3 bf16 terms x (256 rows x 32 bytes) + 256 alpha floats */

// per-(layer, sequence) device counters
enum { CTR_N = 0, CTR_T = 1, CTR_SINCE = 2, CTR_EVSTEPS = 3, CTR_NEVICT = 4, CTR_NPEND = 5, CTR_NNEXT = 6, CTR_NSEL = 7, CTR_STRIDE = 8 };

// CTR_NNEXT: in a decode call with deferred compaction, the entry count the call will leave; CTR_N keeps the
// count from before the call until the call's last kernel (the attention and merge kernels read it).

// device status bits (sticky)
enum { ST_NONFINITE = 1, ST_COUNT = 2, ST_TIMEOUT = 4, ST_LAYOUT = 8 };

struct ImDims {
  int L, S;                   // layers, sequences per layer
  int H, Hkv, d, D, Dkv, Gq;  // attention shape
  int HI, dI, dM;             // indexer / memory widths
  int B, tau, cap, tail;      // budget, interval, slots per sequence, tail = cap - B
  int n_sink, act, mem, F, out_f32, max_chunk, chunk_out;
  int share;                  // >= 2: layers l with l % share != 0 reuse the scores of layer l - l % share
  int scorer;                 // 0 indexer (one row per sequence); a retained set per KV head: 1 Knorm, 2 caller's scores
  int evr;                    // rows per sequence of the evicted-pair scratch (evK / evV / phi): tail, per head tail * Hkv
  int R3, R5;                 // projection rows: indexer only / indexer + memory
  int max_splits;             // attention splits per (sequence, KV head)
  float scale, lambda, eta, eps, norm_eps;
  uint32_t wait_limit;        // attempts of a consumer's bounded wait for data to arrive (IM_OPT_WAIT_LIMIT; the waits for
                              // a CTA's own copies to land before it ends always get the full IM_WAIT_LIMIT)
};
#define IM_WAIT_LIMIT (1u << 22)

// projection row offsets inside one raw output vector
struct ImRows {
  int uq, uk, g, theta, wg;
};
__host__ __device__ inline ImRows im_rows(const ImDims& p) {
  ImRows r;
  r.uq = 0;
  r.uk = p.HI * p.dI;
  r.g = r.uk + p.dI;
  r.theta = r.g + p.HI;
  r.wg = r.theta + p.dM;
  return r;
}

// device state, unit u = layer * S + seq
struct ImState {
  bf16* Kc;         // [U][Hkv][cap][d]
  bf16* Vc;         // [U][Hkv][cap][d]
  bf16* kidx;       // [U][cap][dI]
  int32_t* pos;     // [U][cap]
  float* imp;       // [U][cap]
  uint8_t* keep;    // [U][cap]   flags of the last selection
  int32_t* sel_pos; // [U][cap]   positions / importance of the candidates of the last selection
  float* sel_imp;   // [U][cap]
  int32_t* ev_slot; // [U][tail]  slots evicted by the last compression, ascending
  int32_t* ev_pos;  // [U][tail]  their positions
  float* Mhat;      // [U][dM][Dkv]
  float* bvec;      // [U][dM]
  float* cscale;    // [U]        M = cscale * (Mhat + sum_p pend_w[p] phi_p v_p^T)
  float* pend_phi;  // [U][F][dM]
  bf16* pend_v;     // [U][F][Dkv]
  float* pend_w;    // [U][F]
  int32_t* ctr;     // [U][CTR_STRIDE]
  int32_t* status;  // [1]
  // a retained set per KV head (ImDims::scorer != 0): row = (u * Hkv + h)
  int32_t* hpos;       // [U][Hkv][cap]  position held by a slot of the head's slab
  float* hscore;       // [U][Hkv][cap]  the head's score of that entry
  int32_t* hsel_pos;   // [U][Hkv][cap]  what the head's latest selection chose among
  float* hsel_score;   // [U][Hkv][cap]
  int32_t* hev_slot;   // [U][Hkv][tail] slots the head evicted in the latest compression, ascending
  int32_t* hev_pos;    // [U][Hkv][tail] their positions
  uint8_t* hkeep;      // [U][Hkv][cap]
};

struct ImWeights {  // one layer
  bf16* Uq;
  bf16* Uk;
  bf16* G;
  bf16* Wt;
  bf16* wg;
  float* bg;
  // Linear_theta folded over each query-head group, [dM][Dkv]: Wfold[m][g*d+c] = sum_{j in group g} Wt[m][j*d+c],
  // kept as two bf16 terms (Wfh + Wfl reproduces the float32 sum to 2^-17) so that it can feed the tensor cores
  bf16* Wfh;
  bf16* Wfl;
};

struct ImScratch {   // per call, shared by all layers, stream ordered
  float* raw;        // projection outputs: prefill [n_seq * C][R3]; decode K-split partials [IM_KSPLIT][n_seq][R5]
  double* keyp;      // indexer-key projection in float64: prefill [n_seq * C][dI]; decode partials [IM_KSPLIT_KEY][n_seq][dI]
  bf16* evK;         // [max_seqs][tail][Dkv]  evicted keys of the last compression, gathered
  bf16* evV;         // [max_seqs][tail][Dkv]  evicted values
  float* phi;        // [max_seqs][tail][dM]   phi of the evicted keys (evict steps with more than F entries)
  float* phip;       // [IM_KSPLIT][max_seqs][F][dM] K-split partials of phi for evict steps with at most F entries
  int32_t* surv;     // [max_seqs][tail]       compaction: retained entries found above the budget, ascending
  int32_t* nhole;    // [max_seqs]             compaction: number of evicted slots below the budget
  float* part;       // attention partials (acc[d], max, sum): generic kernel [max_seqs][H][max_splits][d + 2];
                     // streaming kernel [warps + rows][Gq][d + 2]
  float* rpart;      // readout numerators phi(q)^T Mhat: [max_seqs][Dkv] (k_readout_cols), or partial vectors
                     // [CTAs + max_seqs][Dkv] (k_readout_stream)
  float* mres;       // [max_seqs][IM_MRES_ROW] per column the part of the memory readout (Eq. 5) that does not go
                     // through Mhat (pending list, entries written in this call), then the gate g(q), the denominator
                     // sum, and the coefficient c of the Mhat part: m(q)[col] = mres[col] + c * rpart[col]
  float* phiq;       // [max_seqs][dM] phi(q) of the call (K-split partials summed)
  int32_t* n_att;    // [max_seqs] entries per sequence the streaming attention kernel of the call ran over
  bf16* phiT;        // [seq][2][dM][KE] phi of the evicted keys, transposed, as two bf16 terms (KE = evicted count rounded
                     // up to 64); room for pack_k entries in all (one sequence's tail at least)
  bf16* vT;          // [seq][Dkv][KE] the evicted values, transposed
  long long pack_k;  // entries phiT / vT have room for
  float* gpart;      // partial results of K-split tensor-core projections: IM_TC_KSPLIT x [gpart_vecs][R3]
  long long gpart_vecs;
  float* bpart;      // [pack_k / 32][dM] sums of phi^2 over the 32 entries of a block of the packed operands
  float* mch;        // [max_seqs][max_chunk][Dkv] gated memory readout of a chunk's own queries (im_prefill_chunk_attend)
  uint8_t* qpack;    // [n_seq][ceil(C / IM_TC_QT)][IM_TC_TILE_BYTES] query operand of the tensor-core prefill scoring
  // a retained set per KV head
  int32_t* hsurv;    // [max_seqs][Hkv][tail] retained entries above the budget, ascending, per head
  int32_t* hnhole;   // [max_seqs][Hkv]       holes below the budget per head
  int32_t* hrowmap;  // [max_seqs][Hkv][tail] row of the memory write that an evicted (head, entry) pair belongs to
  int32_t* hntok;    // [max_seqs]            rows (tokens that lose a slice) of the evict step
  int32_t* claim;    // [8] worker claiming of the persistent streaming kernels in a pipelined stack call (im_claim_worker):
                     // (arrivals and ids, -, blocks ended, next piece of work) of the attention kernel at [0..3], of the readout
                     // kernel at [4..7]; zero between launches
#ifdef IM_TRACE
  unsigned long long* trace;  // [n_layers][IM_TRACE_KERNELS][IM_TRACE_MARKS] nanosecond time stamps (development builds)
#endif
};

// Development aid, compiled out of the library build: with IM_TRACE defined, thread 0 of block (0, 0) of an instrumented
// kernel writes the global nanosecond timer at its marks; im_trace_read() copies the stamps to the host.
#define IM_TRACE_KERNELS 8
#define IM_TRACE_MARKS 16
#ifdef IM_TRACE
#define IM_MARK(sc_, layer_, kern_, mark_)                                                                      \
  do {                                                                                                          \
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {                                               \
      unsigned long long t_;                                                                                    \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                                    \
      (sc_).trace[((size_t)(layer_) * IM_TRACE_KERNELS + (kern_)) * IM_TRACE_MARKS + (mark_)] = t_;             \
    }                                                                                                           \
  } while (0)
#else
#define IM_MARK(sc_, layer_, kern_, mark_) do {} while (0)
#endif

struct ImCall {
  int layer, n_seq, C;
  int prefill;    // 1: im_prefill_chunk (always compresses), 0: im_decode_step (compresses every tau-th token)
  int defer;      // decode: 1 = the attention kernel runs over the entries cached before the call while the front
                  // kernel appends / scores / selects; the merge adds the new token and takes the evicted entries
                  // out again, and the holes are filled (and CTR_N advanced) by the call's last kernel
  int due;        // decode: 1 = this call compresses (the host checks that all its sequences are at that phase of the
                  // interval); prefill calls always do
  int fold_all;   // prefill with outputs: fold the pending list of every sequence first (the chunk readout reads Mhat alone)
  int pack;       // prefill: 1 = the append kernel also writes the operand records of the tensor-core scoring
  int phi_large;  // 1: phi of the evicted keys lives in ImScratch::phi, 0: in the K-split partials phip
  int ksplit, ksplit_key, ksplit_phi;  // K splits of the projections / key projection / phi partials of this call
  int lead;       // >= 0: the layer whose pooled importances this call's layer reuses instead of scoring with an
                  // indexer of its own (App. B); that layer has already made this call for the same sequences
  // decode: the call's input tensors (x, q_pre, q, k_new, v_new; null entries are skipped) and their size in bytes.
  // The attention kernel, which may start before the kernel ahead of it in the stream has ended, requests them into L2
  // at once: where the caller keeps them resident in HBM the call's latency-bound kernels would each pay a DRAM round
  // trip behind the streams' queued requests (about 7 us against 2 us for a line found in L2).  A line that its
  // producer has yet to write is simply written later: L2 is where the device's writes meet.
  const void* warm[5];
  unsigned warm_bytes[5];
  // decode: 1 = the attention kernel may read this layer's counters and cache before the kernel ahead of it in the
  // stream has ended (that kernel is the merge of a call on another layer); 0 = it waits for that kernel first
  int early_cache;
  // Pipelined stack call (im_decode_stack): the layers of the call overlap, so the occupancy rules that keep the
  // streaming kernels off the SMs set aside for the chain of small kernels no longer hold (a streaming kernel of the
  // next layer starts when SMs of either kind happen to be free).  The split is made by SM id instead: the persistent
  // streaming kernels are launched with one block per SM, a block reads %smid and claims a worker id only on an SM
  // whose bit is set in sm_stream; see im_claim_worker.
  int stack;                        // 1 = the streaming kernels claim their worker ids
  int att_workers, ro_claim;        // blocks of the attention / readout kernel of the call that are to work
  int att_chunks;                   // runs the attention kernel's tiles are cut into (taken from a counter)
  int fold_ffma;                    // 1 = the fold of the pending list by the FFMA kernel whatever the shape (IM_OPT_FOLD_TENSOR 0)
  unsigned long long sm_stream[4];  // bit s set: SM s runs streaming blocks
  int seq[IM_MAX_CALL_SEQS];
};
#define IM_STACK_LANES 3     /* layers of a pipelined stack call in flight (scratch sets, stream sets) */
#define IM_CLAIM_POLLS 12    /* one-microsecond naps of a block that stays off the workers' SMs until the workers are placed */
__device__ __forceinline__ void im_warm_inputs(const ImCall& call, int part, int tid, int nthreads) {
  if (part >= 5 || !call.warm[part]) return;
  const char* b = static_cast<const char*>(call.warm[part]);
  for (size_t off = (size_t)tid * 128; off < call.warm_bytes[part]; off += (size_t)nthreads * 128)
    asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(b + off));
}

// Worker claiming (ImCall::stack).  The grid has at least n_workers blocks; tk[0] holds (blocks arrived << 16 | ids
// claimed) and tk[2] the blocks that have ended, both zero when the launch starts.  Called by one thread of a block, it
// returns the block's worker id in [0, n_workers) or -1 (the block has nothing to do).  A block on a streaming SM
// arrives and claims in one atomic add and works if its id is below n_workers.  A block on another SM arrives with an
// add of its own and leaves without an id, but only if, by the counts that add returned, the blocks still to come
// could claim every id that is left; otherwise it claims like a streaming block.  The count of blocks to come thus
// never falls below the count of ids left (a claim lowers both; a block leaves only where the inequality holds
// after its arrival, and it judges by a claim count that can only be too low): whatever the block scheduler does,
// every id is claimed by exactly one block, and the SM split only decides where.  No add is ever retried: a
// compare-and-swap loop here cost every launch 60 us, one memory round trip per block, one block after the other.
// A block that leaves stays resident for a moment (until the ids are gone, IM_CLAIM_POLLS naps at most) so that the
// blocks still queued are not all dispatched to its SM, one after the other, while the workers' SMs are still busy
// with the previous launch.  Every block, with or without an id, ends with im_claim_exit; the last one clears the
// counters.
__device__ __forceinline__ int im_claim_worker(const ImCall& call, int32_t* tk, int n_workers) {
  unsigned smid;
  asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
  const bool streaming = smid < 256u && ((call.sm_stream[smid >> 6] >> (smid & 63u)) & 1ull);
  unsigned* word = reinterpret_cast<unsigned*>(tk);
  if (streaming) {
    const int id = (int)(atomicAdd(word, (1u << 16) + 1u) & 0xffffu);
    return id < n_workers ? id : -1;
  }
  const unsigned old = atomicAdd(word, 1u << 16);
  const int arrived = (int)(old >> 16), claimed = (int)(old & 0xffffu);
  if (claimed >= n_workers) return -1;
  if ((int)gridDim.x - 1 - arrived >= n_workers - claimed) {
    for (int it = 0; it < IM_CLAIM_POLLS; ++it) {
      __nanosleep(1000);
      if ((int)(*reinterpret_cast<volatile unsigned*>(word) & 0xffffu) >= n_workers) break;
    }
    return -1;
  }
  const int id = (int)(atomicAdd(word, 1u) & 0xffffu);
  return id < n_workers ? id : -1;
}
__device__ __forceinline__ void im_claim_exit(int32_t* tk) {
  if (atomicAdd(tk + 2, 1) == (int)gridDim.x - 1) {
    tk[0] = 0;
    tk[2] = 0;
    tk[3] = 0;  // (the kernel's work counter)
  }
}

// Skinny GEMM arguments: out[v][row0 + r] (+)= sum_k (W[r][k] + W2[r][k]) * in[v][k].
// Vector v of input set s starts at in[s] + (v / in_cnt[s]) * in_outer[s] + (v % in_cnt[s]) * in_inner[s]
// (elements); its outputs at out + (v / out_cnt) * out_outer + (v % out_cnt) * out_inner + ks * ks_stride.
struct ImGemmJob {
  const bf16* W;   // [rows][K]
  const bf16* W2;  // optional second term of the weights (nullptr: none)
  int rows, row0, in_sel;
};
// Batched launch of the tensor-core TMA variant: n independent products, blockIdx.z = b.  Batch b reads its vectors
// zA_rows rows and its weights zB_rows rows further down the operand arrays and writes to out + u * z_out with
// u = unit0 + seq[b] (its gate is gate[u * z_gate]).  Travels as a kernel parameter of that variant alone.
struct ImGemmBatch {
  int n, unit0;
  long long zA_rows, zB_rows, z_out, z_gate;
  int seq[IM_MAX_CALL_SEQS];
};
struct ImGemmArgs {
  ImGemmJob job[4];
  int n_jobs;
  const bf16* in[3];
  long long in_outer[3], in_inner[3];
  int in_cnt[3];
  float* out;
  long long out_outer, out_inner, ks_stride;
  int out_cnt;
  int NV, K, ksplit;
  int kc;      // K elements staged per round (0: the maximum, 512); small values keep the shared-memory footprint low
  int tensor;  // 1: thousands of vectors (prefill) - the tcgen05 variant where it applies (im_tc_gemm_usable)
  int direct;  // 1: few vectors (decode) - the variant without shared-memory staging, if the K split is a multiple of 32
  int any_w2;  // set by the launcher: some job has a second weight term (decides the smem layout)
  int smem_floor;  // direct variant: dynamic shared memory to ask for although the kernel uses none (IM_SMEM_SIDE)
  // direct variant: the float64 indexer-key projection of key_nv vectors (rows of key_x, K elements each) rides along in
  // the same launch if key_W is set: key_out[ks][v][key_dI] receives key_ksplit partial sums (K a multiple of
  // 256 key_ksplit, key_dI 8 or 16); `tiles` is set by the launcher
  const bf16* key_W;
  const bf16* key_x;
  double* key_out;
  int key_nv, key_ksplit, key_dI, tiles;
  int programmatic;  // direct variant: launched as programmatic dependent of the kernel ahead of it in the stream, whose
                     // output the vectors are: the weights are requested while that kernel still runs
  // tensor-core TMA variant only: tc_ksplit > 1 cuts the K range over that many CTAs per output tile (launches of
  // few tiles are bound by the K loop of one CTA); split s writes to part + s * part_stride in the layout of `out`,
  // and a second kernel adds the splits into `out` in a fixed order.  Not with rmw or a batched launch.
  int tc_ksplit;
  float* part;
  long long part_stride;
  const struct ImGemmBatch* batch;  // host pointer, tensor-core TMA variant only: several products in one launch
  // tensor-core variant only:
  int out_t;            // 1: the result goes to out[(row0 + r) * out_outer + v] (vectors contiguous) instead
  int rmw;              // 1: out = beta * out + alpha * result
  float alpha, beta;
  const int32_t* gate;  // if set, nothing is stored unless *gate > gate_min (a device-side counter decides)
  int gate_min;
#ifdef IM_TRACE
  ImScratch trace_sc;  // development builds: where IM_MARK writes (trace_sc.trace == nullptr: nowhere)
  int trace_layer, trace_kern, trace_skip;
#endif
};
#ifdef IM_TRACE
#define IM_MARK_GEMM(a_, mark_) do { if ((a_).trace_sc.trace && blockIdx.z == 0) IM_MARK((a_).trace_sc, (a_).trace_layer, (a_).trace_kern, mark_); } while (0)
#define IM_TRACE_GEMM(g_, L_, layer_, kern_) do { (g_).trace_sc = (L_).sc; (g_).trace_layer = (layer_); (g_).trace_kern = (kern_); } while (0)
#define IM_TRACE_GEMM_OFF(g_) do { (g_).trace_sc.trace = nullptr; } while (0)
#else
#define IM_MARK_GEMM(a_, mark_) do {} while (0)
#define IM_TRACE_GEMM(g_, L_, layer_, kern_) do {} while (0)
#define IM_TRACE_GEMM_OFF(g_) do {} while (0)
#endif

#define IM_NOALLOC_MAX_FLOATS (1u << 20) /* floats in the built-in scratch array of im_attention_noalloc (4 MiB) */
#define IM_KSPLIT 4       /* K splits of the decode projections (partials summed by the consumer) */
#define IM_KSPLIT_KEY 16  /* K splits of the float64 indexer-key projection in decode */
#define IM_FRONT_MAX_N 6144 /* entries the fused decode front kernel can select among (keys in shared memory) */
#define IM_FRONT_MAX_NE 16  /* evicted entries per sequence the fused decode front kernel handles */

struct ImLaunch {
  ImDims p;
  ImState st;
  ImWeights w;
  ImScratch sc;
  cudaStream_t stream;
  int64_t* launches;
};

// Function attributes (dynamic shared-memory limits) are a per-device setting: launchers that set them lazily keep
// one flag per device.  Returns the current device's flag (nullptr if the device id is out of range).
inline bool* im_device_flag(bool (&flags)[64]) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  return &flags[dev];
}

// An SM changes its shared-memory carveout only while it is idle.  The streaming attention kernel needs the largest
// one; every kernel that runs next to it or shortly before it asks for the same, so that attention CTAs never wait
// for resident blocks of a kernel with a smaller carveout to drain.
template <typename F>
inline cudaError_t im_prefer_max_smem(F* kernel) {
  return cudaFuncSetAttribute(reinterpret_cast<const void*>(kernel), cudaFuncAttributePreferredSharedMemoryCarveout,
                              (int)cudaSharedmemCarveoutMaxShared);
}
cudaError_t im_gemm_prepare_decode();
cudaError_t im_memory_prepare_decode();
cudaError_t im_front_prepare_decode();
cudaError_t im_prefetch_prepare_decode();

#define IM_MRES_ROW(p) ((p).Dkv + 4)
#define IM_PH_MAX_PAIRS 16384 /* evicted (head, entry) pairs per sequence and evict step in per-head mode (sorted in shared memory) */
// a retained set per KV head (im_perhead.cu)
cudaError_t im_perhead_prepare(const ImDims& p);
cudaError_t im_ph_launch_append(const ImLaunch& L, const ImCall& call, const void* k, const void* v);
cudaError_t im_ph_launch_select(const ImLaunch& L, const ImCall& call, const float* ext, long long n_pos);
cudaError_t im_ph_launch_assemble(const ImLaunch& L, const ImCall& call, int ne_max);
cudaError_t im_ph_launch_mem_write(const ImLaunch& L, const ImCall& call);
cudaError_t im_ph_launch_move(const ImLaunch& L, const ImCall& call);
#define IM_TC_KSPLIT 4  /* K splits of the prefill projections on the tensor cores (chunks of up to 8192 vectors) */

// Decode calls of few sequences split the SMs between the two kinds of work of a call: the streaming kernels
// (attention over the cache, readout over Mhat), bound by HBM bandwidth, and the chain of small kernels that
// decides what the call evicts (front kernel, phi of the evicted keys), bound by memory latency, which runs
// several times slower on an SM whose load queues a streaming block keeps full.  The split is made by the
// occupancy rules alone: a front block asks for so much shared memory that no attention CTA fits next to it,
// and the attention grid is n_res blocks short of the SM count (n_res = number of front blocks), so that
// wherever its CTAs land, n_res SMs are left to the front kernel.  The readout kernel, whose blocks would settle
// on just those SMs (the emptiest), starts when the front kernel has ended; the phi GEMM that follows the front
// kernel asks for more shared memory than an SM with an attention CTA has left and ends up on the SMs the front
// kernel has just freed.
#define IM_SMEM_FRONT (192 * 1024)   /* front block: excludes attention CTAs (>= 64 KB of shared memory each) */
#define IM_SMEM_SIDE (38 * 1024)     /* phi GEMM block (+ 17 KB static): four per free SM, at most one next to an attention CTA */
#define IM_PREFETCH_MEM_EIGHTHS 4   /* eighths of the next layer's memory matrices requested into L2 at the end of a decode call */
#define IM_SMEM_HEAD (100 * 1024)    /* indexer projection block, which heads the call's longest chain: two per free SM, none next
                                        to an attention CTA (which leaves 96 KB of an SM's shared memory) */
inline int im_reserved_sms(int n_sm, int n_seq) { return n_seq <= n_sm / 4 ? n_seq : 0; }

// records `msg` as the calling thread's last error and returns `code` (defined next to im_last_error)
int im_fail_message(int code, const char* msg);

// ---- kernels' host launchers (each returns the cudaError of the launch)
cudaError_t im_launch_gemm(const ImLaunch& L, const ImGemmArgs& a);
// tensor-core (tcgen05) variant for thousands of vectors and one K split (prefill)
bool im_tc_gemm_usable(const ImGemmArgs& a);
cudaError_t im_launch_tc_gemm(const ImLaunch& L, const ImGemmArgs& a);
cudaError_t im_launch_proj_key_split(const ImLaunch& L, const void* x, int NV, int ksplit);
cudaError_t im_launch_decode_front(const ImLaunch& L, const ImCall& call, const void* k_new, const void* v_new,
                                   int do_select, int n_max, int smem_floor, cudaEvent_t started = nullptr, int programmatic = 0);
cudaError_t im_launch_prefetch_layer(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_prefetch_memory(const ImLaunch& L, const ImCall& call, int eighths, int per_block = 1);
cudaError_t im_probe_sm_ids(void* map, int n_sm, int* ids, int* n, cudaStream_t stream);
cudaError_t im_launch_gather_move(const ImLaunch& L, const ImCall& call, int ne_max);
cudaError_t im_launch_gather(const ImLaunch& L, const ImCall& call, int ne_max);
cudaError_t im_launch_move(const ImLaunch& L, const ImCall& call, int ne_max);
cudaError_t im_launch_mem_fold(const ImLaunch& L, const ImCall& call);
// ne_host: per call sequence, the number of entries the compression of this call evicts (host mirror)
cudaError_t im_launch_mem_update(const ImLaunch& L, const ImCall& call, int ne_max, const int* ne_host);
cudaError_t im_launch_prefill_append(const ImLaunch& L, const ImCall& call, const void* k, const void* v);
cudaError_t im_launch_prefill_score(const ImLaunch& L, const ImCall& call, int n_max);
// tensor-core (tcgen05) version of the prefill scoring; needs ImCall::pack set for the append kernel
bool im_score_tc_supported(const ImDims& p);
cudaError_t im_score_tc_prepare();
cudaError_t im_launch_prefill_score_tc(const ImLaunch& L, const ImCall& call, int n_max, int n_sm);
cudaError_t im_launch_prefill_commit(const ImLaunch& L, const ImCall& call);
// a layer that reuses another layer's scores: copy the pooled importances that layer's selection saw (slot by slot; the
// two layers' slot layouts agree, which the kernel checks position by position)
cudaError_t im_launch_follow_scores(const ImLaunch& L, const ImCall& call);
// layer outputs of a prefill chunk's own queries
cudaError_t im_chunk_attn_prepare(const ImDims& p);
cudaError_t im_launch_chunk_readout(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_chunk_attention(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                      const void* q, void* out);
bool im_chunk_attn_tc_supported(const ImDims& p);
cudaError_t im_chunk_attn_tc_prepare();
cudaError_t im_launch_chunk_attention_tc(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                         const void* q, void* out);
cudaError_t im_launch_select(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_attention(const ImLaunch& L, const ImCall& call, const void* q, void* out, int n_max);
bool im_attn_fast_supported(const ImDims& p);
cudaError_t im_attn_make_maps(const ImDims& p, const ImState& st, void* mapK, void* mapV, int box_rows, int halves3d = 0);
// tcgen05 version of the streaming attention kernel (head_dim 128): one run of 128-key tiles per CTA; mapK / mapV
// with 32-row boxes (ragged last tile of a row), mapK128 / mapV128 with 128-row boxes (full tiles)
bool im_attn_tc_supported(const ImDims& p);
cudaError_t im_attn_tc_prepare();
cudaError_t im_launch_attention_tc(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                   const void* mapK128, const void* mapV128, const void* q, int n_ctas, int programmatic);
cudaError_t im_attn_prepare(const ImDims& p);
// grid blocks (at most one per SM wanted); light: the variant that leaves room for a front block on its SM
cudaError_t im_launch_readout(const ImLaunch& L, const ImCall& call, int grid, int light);
cudaError_t im_launch_readout_finish(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_attention_fast(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                     const void* q, int n_ctas, int programmatic);
// n_workers / tile: the runs the attention kernel of the call cut the tiles into, and its tile size; ro_workers: CTAs
// of the streaming readout kernel whose partial vectors are to be added (0: one vector per sequence from k_readout_cols)
cudaError_t im_launch_attention_merge(const ImLaunch& L, const ImCall& call, void* out, int n_workers, int tile, int ro_workers,
                                      const void* q, const void* k_new, const void* v_new, int programmatic);
// phi(q)^T Mhat as a persistent kernel fed by bulk copies (ring of `stages` 32 KB stages per CTA)
bool im_readout_stream_supported(const ImDims& p);
int im_readout_stream_chunks(const ImDims& p);
cudaError_t im_readout_stream_prepare(const ImDims& p);
cudaError_t im_launch_readout_stream(const ImLaunch& L, const ImCall& call, int grid, int stages);

cudaError_t im_launch_topb(const float* scores, const int32_t* pos, int rows, int n, int budget, int n_sink,
                           uint8_t* keep, int32_t* n_evict, cudaStream_t stream);
cudaError_t im_launch_init_weights(const ImDims& p, const ImWeights& w, int layer, uint64_t seed, float std,
                                   cudaStream_t stream);
cudaError_t im_launch_fold_theta(const ImDims& p, const ImWeights& w, cudaStream_t stream);

// Evict-step bookkeeping shared by the memory kernels: number of entries the compression of this
// call will evict for a sequence whose counters are still those from before the call.
__host__ __device__ inline int im_upcoming_evictions(const ImDims& p, int due, int C, int n) {
  const int over = n + C - p.B;
  return (due && over > 0) ? over : 0;
}

// decode: projection row `row` of call sequence i, summed over the K-split partials in a fixed order
__device__ __forceinline__ float im_raw_sum(const ImDims& p, const ImScratch& sc, const ImCall& call, int i, int row) {
  float s = 0.f;
  for (int ks = 0; ks < call.ksplit; ++ks) s += sc.raw[((size_t)ks * call.n_seq + i) * p.R5 + row];
  return s;
}

// Loads that the compiler may neither reorder nor delay to their first use: for values that are requested long before
// they are needed, so that the round trip overlaps what lies in between.
__device__ __forceinline__ uint4 im_ld_now_u4(const void* p) {
  uint4 v;
  asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ float im_ld_now_f32(const float* p) {
  float v;
  asm volatile("ld.volatile.global.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ int im_ld_now_s32(const int32_t* p) {
  int v;
  asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

// ---- small device helpers
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

// Selection key: larger is better.  High word: order-preserving image of the score (sinks above
// everything, -0.0 folded onto +0.0); low word: ~position, so that the lower position wins ties.
__device__ __forceinline__ uint64_t im_select_key(float s, int pos, int n_sink) {
  uint32_t ks;
  if (pos < n_sink) {
    ks = 0xFFFFFFFFu;
  } else {
    uint32_t b = __float_as_uint(s + 0.0f);
    ks = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
  }
  return ((uint64_t)ks << 32) | (uint64_t)(0xFFFFFFFFu - (uint32_t)pos);
}

// Internal declarations shared by the translation units of libindexmem (not part of the ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "indexmem.h"

typedef __nv_bfloat16 bf16;

#define IM_MAX_CALL_SEQS 256 /* sequences per hot call (the id list travels as a kernel parameter) */
#define IM_SLOT_ALIGN 64     /* slot capacity is a multiple of the attention tile */
#define IM_ATTN_TILE 32      /* keys per attention tile (one TMA box is 32 rows x 128 bytes) */
#define IM_ATTN_WARPS 4      /* warps per CTA of the streaming attention kernel */
#define IM_ATTN_MAX_CTAS 512 /* upper bound of its grid (one CTA per SM) */
#define IM_READOUT_ROWS 32   /* rows of M per readout partial */

// per-(layer, sequence) device counters
enum { CTR_N = 0, CTR_T = 1, CTR_SINCE = 2, CTR_EVSTEPS = 3, CTR_NEVICT = 4, CTR_NPEND = 5, CTR_DIRECT = 6, CTR_NSEL = 7, CTR_STRIDE = 8 };

// device status bits (sticky)
enum { ST_NONFINITE = 1, ST_COUNT = 2, ST_TIMEOUT = 4 };

struct ImDims {
  int L, S;                   // layers, sequences per layer
  int H, Hkv, d, D, Dkv, Gq;  // attention shape
  int HI, dI, dM;             // indexer / memory widths
  int B, tau, cap, tail;      // budget, interval, slots per sequence, tail = cap - B
  int n_sink, act, mem, F, out_f32, max_chunk;
  int R3, R5;                 // projection rows: indexer only / indexer + memory
  int max_splits;             // attention splits per (sequence, KV head)
  float scale, lambda, eta, eps, norm_eps;
};

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
};

struct ImWeights {  // one layer
  bf16* Uq;
  bf16* Uk;
  bf16* G;
  bf16* Wt;
  bf16* wg;
  float* bg;
  float* Wfold;  // [dM][Dkv] float32: Linear_theta folded over each query-head group
};

struct ImScratch {   // per call, shared by all layers, stream ordered
  float* raw;        // [max_seqs * max(1,max_chunk)][R5 or R3] projection outputs (qf / alpha are finalised in place)
  bf16* kidx_new;    // [max_seqs * max(1,max_chunk)][dI] indexer keys of the call's tokens
  float* phi;        // [max_seqs][tail][dM]   phi of the evicted keys
  int32_t* moves;    // [max_seqs][2][tail]    compaction: hole slots, survivor slots
  float* part;       // attention partials (acc[d], max, sum): generic kernel [max_seqs][H][max_splits][d + 2];
                     // streaming kernel [warps + rows][Gq][d + 2]
  float* rpart;      // [max_seqs][ceil(dM / IM_READOUT_ROWS)][Dkv] readout partials
};

struct ImCall {
  int layer, n_seq, C;
  int seq[IM_MAX_CALL_SEQS];
};

struct ImProjJob {
  const bf16* W;   // [rows][Dn]
  const bf16* in;  // [NV][Dn]
  int rows, row0;  // rows of this job, first output row
};
struct ImProjJobs {
  ImProjJob job[5];
  int n_jobs, total_rows, Dn, NV, out_stride;
};

struct ImLaunch {
  ImDims p;
  ImState st;
  ImWeights w;
  ImScratch sc;
  cudaStream_t stream;
  int64_t* launches;
};

// ---- kernels' host launchers (each returns the cudaError of the launch)
cudaError_t im_launch_proj(const ImLaunch& L, const ImProjJobs& jobs, float* out);
cudaError_t im_launch_proj_key(const ImLaunch& L, const void* x, int NV);
cudaError_t im_launch_decode_index(const ImLaunch& L, const ImCall& call, const void* k_new, const void* v_new);
cudaError_t im_launch_prefill_append(const ImLaunch& L, const ImCall& call, const void* k, const void* v);
cudaError_t im_launch_prefill_score(const ImLaunch& L, const ImCall& call, int n_max);
cudaError_t im_launch_select(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_memory_write(const ImLaunch& L, const ImCall& call, int ne_max, bool direct);
cudaError_t im_launch_compact(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_attention(const ImLaunch& L, const ImCall& call, const void* q, void* out, int n_max);
bool im_attn_fast_supported(const ImDims& p);
cudaError_t im_attn_make_maps(const ImDims& p, const ImState& st, void* mapK, void* mapV);
cudaError_t im_attn_prepare(const ImDims& p);
cudaError_t im_launch_readout(const ImLaunch& L, const ImCall& call);
cudaError_t im_launch_attention_fast(const ImLaunch& L, const ImCall& call, const void* mapK, const void* mapV,
                                     const void* q, void* out, int n_ctas);
cudaError_t im_launch_topb(const float* scores, const int32_t* pos, int rows, int n, int budget, int n_sink,
                           uint8_t* keep, int32_t* n_evict, cudaStream_t stream);
cudaError_t im_launch_init_weights(const ImDims& p, const ImWeights& w, int layer, uint64_t seed, float std,
                                   cudaStream_t stream);
cudaError_t im_launch_fold_theta(const ImDims& p, const ImWeights& w, cudaStream_t stream);

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

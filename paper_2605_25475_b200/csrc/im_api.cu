// Host side of libindexmem: configuration, workspace layout, the C ABI and the order of the
// kernels inside the two hot calls.  Every step of the path runs in the kernels of the other
// translation units; nothing here computes on the CPU except argument checks, host mirrors of the
// per-sequence counters (they are deterministic functions of the call history) and the
// non-hot-path state export/import.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "im_internal.cuh"

namespace {

thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

#define CK(call)                                                                              \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess) return fail(IM_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

int im_fail_message(int code, const char* msg) { return fail(code, "%s", msg); }

namespace {

struct Layout {
  ImState st;
  ImScratch sc;
  ImScratch lane[IM_STACK_LANES];  // decode scratch of the layers in flight in a pipelined stack call (see carve)
  int32_t* claims;                 // the lanes' claim counters, IM_STACK_LANES x 8 (zeroed at create)
  std::vector<ImWeights> w;
  size_t state_begin, state_end;  // byte range holding per-unit state (zeroed at create)
  size_t total;
};

bool resolve(const im_config* in, im_config* c, ImDims* p) {
  if (!in) return false;
  *c = *in;
  if (c->n_layers < 1 || c->max_seqs < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1) return false;
  if (c->n_q_heads % c->n_kv_heads) return false;
  if (c->head_dim < 16 || c->head_dim % 16 || c->head_dim > 256) return false;
  if (c->n_index_heads == 0) c->n_index_heads = std::max(1, c->n_q_heads / 4);
  if (c->index_dim == 0) c->index_dim = std::max(1, c->head_dim / 8);
  if (c->mem_dim == 0) c->mem_dim = std::max(1, c->n_q_heads * c->head_dim / 8);
  if (c->n_index_heads < 1 || c->n_index_heads > 64 || c->index_dim < 1 || c->index_dim > 64) return false;
  if (c->mem_dim < 1) return false;
  if (c->compress_interval < 1) return false;
  if (c->max_chunk < 0) return false;
  if (c->n_sink < 0 || c->budget <= c->n_sink || c->budget < 1) return false;
  if (c->act != 0 && c->act != 1) return false;
  if (c->pending_slots == 0) c->pending_slots = 32;
  if (c->pending_slots < 1 || c->pending_slots > 64) return false;
  if (c->softmax_scale == 0.f) c->softmax_scale = 1.0f / sqrtf((float)c->head_dim);
  if (c->lambda == 0.f) c->lambda = 1.f;
  if (c->eta == 0.f) c->eta = 1.f;
  if (c->eps == 0.f) c->eps = 1e-6f;
  if (c->norm_eps == 0.f) c->norm_eps = 1e-6f;
  if (c->init_std == 0.f) c->init_std = 0.02f;
  if (!(c->lambda > 0.f && c->lambda <= 1.f) || !(c->eta > 0.f) || !(c->eps > 0.f)) return false;
  long long cap = (long long)c->budget + std::max(c->compress_interval, std::max(c->max_chunk, 1));
  cap = (cap + IM_SLOT_ALIGN - 1) / IM_SLOT_ALIGN * IM_SLOT_ALIGN;
  if (cap > (1ll << 30)) return false;
  ImDims& q = *p;
  q.L = c->n_layers; q.S = c->max_seqs;
  q.H = c->n_q_heads; q.Hkv = c->n_kv_heads; q.d = c->head_dim;
  q.D = q.H * q.d; q.Dkv = q.Hkv * q.d; q.Gq = q.H / q.Hkv;
  q.HI = c->n_index_heads; q.dI = c->index_dim; q.dM = c->mem_dim;
  q.B = c->budget; q.tau = c->compress_interval; q.cap = (int)cap; q.tail = q.cap - q.B;
  q.n_sink = c->n_sink; q.act = c->act; q.mem = c->enable_memory ? 1 : 0; q.F = c->pending_slots;
  q.out_f32 = c->out_f32 ? 1 : 0; q.max_chunk = std::max(c->max_chunk, 1);
  q.chunk_out = c->chunk_outputs ? 1 : 0;
  if (c->score_share < 0 || c->score_share > c->n_layers) return false;
  q.share = c->score_share >= 2 ? c->score_share : 0;
  if (c->scorer < 0 || c->scorer > 2) return false;
  if (c->scorer && (q.share || c->chunk_outputs || c->n_kv_heads > 4096)) return false;  // per-head sets: neither score reuse nor chunk outputs
  q.scorer = c->scorer;
  q.evr = q.tail * (q.scorer ? q.Hkv : 1);
  q.R3 = q.HI * q.dI + q.dI + q.HI;
  q.R5 = q.R3 + q.dM + 1;
  q.max_splits = (q.cap + 255) / 256;
  q.scale = c->softmax_scale; q.lambda = c->lambda; q.eta = c->eta; q.eps = c->eps; q.norm_eps = c->norm_eps;
  if (q.Gq > 16) return false;
  p->wait_limit = IM_WAIT_LIMIT;
  return true;
}

// Carves the workspace.  base == nullptr: only sizes are computed.
void carve(const ImDims& p, char* base, Layout* lo) {
  size_t off = 0;
  auto take = [&](size_t bytes) -> char* {
    off = align_up(off, 256);
    char* ptr = base ? base + off : nullptr;
    off += bytes;
    return ptr;
  };
  const size_t U = (size_t)p.L * p.S;
  lo->state_begin = 0;
  lo->st.Kc = (bf16*)take(U * p.Hkv * p.cap * p.d * 2);
  lo->st.Vc = (bf16*)take(U * p.Hkv * p.cap * p.d * 2);
  lo->st.kidx = (bf16*)take(U * p.cap * p.dI * 2);
  lo->st.pos = (int32_t*)take(U * p.cap * 4);
  lo->st.imp = (float*)take(U * p.cap * 4);
  lo->st.keep = (uint8_t*)take(U * p.cap);
  lo->st.sel_pos = (int32_t*)take(U * p.cap * 4);
  lo->st.sel_imp = (float*)take(U * p.cap * 4);
  lo->st.ev_slot = (int32_t*)take(U * p.tail * 4);
  lo->st.ev_pos = (int32_t*)take(U * p.tail * 4);
  lo->st.Mhat = (float*)take(U * p.dM * p.Dkv * 4);
  lo->st.bvec = (float*)take(U * p.dM * 4);
  lo->st.cscale = (float*)take(U * 4);
  lo->st.pend_phi = (float*)take(U * p.F * p.dM * 4);
  lo->st.pend_v = (bf16*)take(U * p.F * p.Dkv * 2);
  lo->st.pend_w = (float*)take(U * p.F * 4);
  lo->st.ctr = (int32_t*)take(U * CTR_STRIDE * 4);
  lo->st.status = (int32_t*)take(256);
  lo->st.hpos = lo->st.hsel_pos = lo->st.hev_slot = lo->st.hev_pos = nullptr;
  lo->st.hscore = lo->st.hsel_score = nullptr;
  lo->st.hkeep = nullptr;
  if (p.scorer) {  // a retained set per KV head: position / score / selection bookkeeping per (unit, head) row
    const size_t R = U * p.Hkv;
    lo->st.hpos = (int32_t*)take(R * p.cap * 4);
    lo->st.hscore = (float*)take(R * p.cap * 4);
    lo->st.hsel_pos = (int32_t*)take(R * p.cap * 4);
    lo->st.hsel_score = (float*)take(R * p.cap * 4);
    lo->st.hev_slot = (int32_t*)take(R * p.tail * 4);
    lo->st.hev_pos = (int32_t*)take(R * p.tail * 4);
    lo->st.hkeep = (uint8_t*)take(R * p.cap);
  }
  lo->state_end = off;
  lo->w.resize(p.L);
  for (int l = 0; l < p.L; ++l) {
    ImWeights& w = lo->w[l];
    w.Uq = (bf16*)take((size_t)p.HI * p.dI * p.D * 2);
    w.Uk = (bf16*)take((size_t)p.dI * p.D * 2);
    w.G = (bf16*)take((size_t)p.HI * p.D * 2);
    w.Wt = (bf16*)take((size_t)p.dM * p.D * 2);
    w.wg = (bf16*)take((size_t)p.D * 2);
    w.bg = (float*)take(256);
    w.Wfh = (bf16*)take((size_t)p.dM * p.Dkv * 2);
    w.Wfl = (bf16*)take((size_t)p.dM * p.Dkv * 2);
  }
  lo->sc.raw = (float*)take((size_t)p.S * std::max(p.max_chunk, IM_KSPLIT) * p.R5 * 4);
  lo->sc.keyp = (double*)take((size_t)p.S * std::max(p.max_chunk, IM_KSPLIT_KEY) * p.dI * 8);
  lo->sc.evK = (bf16*)take((size_t)p.S * p.evr * p.Dkv * 2);
  lo->sc.evV = (bf16*)take((size_t)p.S * p.evr * p.Dkv * 2);
  lo->sc.phi = (float*)take((size_t)p.S * p.evr * p.dM * 4);
  lo->sc.hsurv = lo->sc.hnhole = lo->sc.hrowmap = lo->sc.hntok = nullptr;
  if (p.scorer) {
    lo->sc.hsurv = (int32_t*)take((size_t)p.S * p.Hkv * p.tail * 4);
    lo->sc.hnhole = (int32_t*)take((size_t)p.S * p.Hkv * 4);
    lo->sc.hrowmap = (int32_t*)take((size_t)p.S * p.Hkv * p.tail * 4);
    lo->sc.hntok = (int32_t*)take((size_t)p.S * 4);
  }
  lo->sc.phip = (float*)take((size_t)IM_KSPLIT * p.S * p.F * p.dM * 4);
  lo->sc.surv = (int32_t*)take((size_t)p.S * p.tail * 4);
  lo->sc.nhole = (int32_t*)take((size_t)p.S * 4);
  {
    const size_t generic = (size_t)p.S * p.H * p.max_splits * (p.d + 2);
    const size_t stream = ((size_t)IM_ATTN_MAX_CTAS * IM_ATTN_WARPS + (size_t)p.S * p.Hkv) * p.Gq * (p.d + 2);
    lo->sc.part = (float*)take(std::max(generic, stream) * 4);
  }
  lo->sc.mres = (float*)take((size_t)p.S * IM_MRES_ROW(p) * 4);
  lo->sc.phiq = (float*)take((size_t)p.S * p.dM * 4);
  lo->sc.n_att = (int32_t*)take((size_t)p.S * 4);
  lo->sc.rpart = (float*)take((size_t)(IM_ATTN_MAX_CTAS + p.S) * p.Dkv * 4);
  lo->sc.phiT = nullptr;
  lo->sc.vT = nullptr;
  lo->sc.gpart_vecs = std::min<long long>((long long)p.S * p.max_chunk, 8192);
  lo->sc.gpart = (float*)take((size_t)IM_TC_KSPLIT * lo->sc.gpart_vecs * p.R3 * 4);
  lo->sc.pack_k = 0;
  lo->sc.bpart = nullptr;
  if (p.tail > p.F) {
    // one sequence's largest evicted set at least; 4096 entries so that the sequences of a decode call with a long
    // compression interval go through one batched launch
    const size_t KE = std::max<size_t>(((size_t)p.tail + 63) / 64 * 64, 4096);
    lo->sc.phiT = (bf16*)take(2 * (size_t)p.dM * KE * 2);
    lo->sc.vT = (bf16*)take((size_t)p.Dkv * KE * 2);
    lo->sc.pack_k = (long long)KE;
    lo->sc.bpart = (float*)take((KE / 32) * (size_t)p.dM * 4);
  }
  lo->sc.mch = nullptr;
  if (p.chunk_out) lo->sc.mch = (float*)take((size_t)p.S * p.max_chunk * p.Dkv * 4);
  lo->sc.qpack = nullptr;
  if (im_score_tc_supported(p))
    lo->sc.qpack = (uint8_t*)take((size_t)p.S * ((p.max_chunk + IM_TC_QT - 1) / IM_TC_QT) * IM_TC_TILE_BYTES);
  // Pipelined stack calls keep IM_STACK_LANES layers in flight, each with the scratch a deferred-compaction decode
  // call writes: projection partials, gathered evicted pairs, phi partials, moves, attention / readout partials, the
  // readout's small vectors, entry counts, claim counters.  A lane's gathered evicted pairs are at most
  // IM_FRONT_MAX_NE rows per sequence; where a sequence's region of evK / evV has room (row stride `tail`), lane k
  // uses rows [k, k + 1) * IM_FRONT_MAX_NE of the shared arrays, else arrays of its own.
  lo->sc.claim = (int32_t*)take(256);
  lo->claims = (int32_t*)take((size_t)IM_STACK_LANES * 8 * 4);
  for (int k = 0; k < IM_STACK_LANES; ++k) {
    ImScratch& ln = lo->lane[k];
    ln = lo->sc;
    if (p.scorer) continue;
    ln.raw = (float*)take((size_t)p.S * IM_KSPLIT * p.R5 * 4);
    ln.keyp = (double*)take((size_t)p.S * IM_KSPLIT_KEY * p.dI * 8);
    if (p.tail >= IM_FRONT_MAX_NE * IM_STACK_LANES) {
      ln.evK = base ? lo->sc.evK + (size_t)k * IM_FRONT_MAX_NE * p.Dkv : nullptr;
      ln.evV = base ? lo->sc.evV + (size_t)k * IM_FRONT_MAX_NE * p.Dkv : nullptr;
    } else {
      ln.evK = (bf16*)take((size_t)p.S * p.evr * p.Dkv * 2);
      ln.evV = (bf16*)take((size_t)p.S * p.evr * p.Dkv * 2);
    }
    ln.phip = (float*)take((size_t)IM_KSPLIT * p.S * p.F * p.dM * 4);
    ln.surv = (int32_t*)take((size_t)p.S * p.tail * 4);
    ln.nhole = (int32_t*)take((size_t)p.S * 4);
    ln.part = (float*)take(((size_t)IM_ATTN_MAX_CTAS * IM_ATTN_WARPS + (size_t)p.S * p.Hkv) * p.Gq * (p.d + 2) * 4);
    ln.mres = (float*)take((size_t)p.S * IM_MRES_ROW(p) * 4);
    ln.phiq = (float*)take((size_t)p.S * p.dM * 4);
    ln.n_att = (int32_t*)take((size_t)p.S * 4);
    ln.rpart = (float*)take((size_t)(IM_ATTN_MAX_CTAS + p.S) * p.Dkv * 4);
    ln.claim = base ? lo->claims + k * 8 : nullptr;
  }
  lo->total = align_up(off, 256);
}

struct HostUnit {
  int n = 0;       // cached entries
  long long T = 0; // tokens seen
  int since = 0;   // decode tokens since the last compression
};

}  // namespace

struct im_ctx {
  im_config cfg;
  ImDims p;
  Layout lo;
  std::vector<HostUnit> hu;
  int64_t launches = 0;
  int device = 0;
  alignas(64) unsigned char mapK[128];  // TMA descriptors of the K / V caches
  alignas(64) unsigned char mapV[128];
  alignas(64) unsigned char mapKs[128];    // the same caches with the boxes of the mma.sync streaming attention kernel
  alignas(64) unsigned char mapVs[128];
  alignas(64) unsigned char mapK128[128];  // the same caches with 128-row boxes (full tiles of the tensor-core attention)
  alignas(64) unsigned char mapV128[128];
  struct ExtScores { const float* ptr = nullptr; long long n_pos = 0; int n_seq = 0; };
  std::vector<ExtScores> ext;        // per layer: scores handed in by the caller for the next compressing call (scorer = 2)
  bool ro_stream = false;            // phi(q)^T Mhat by the bulk-copy streaming kernel where it runs next to the attention kernel (IM_OPT_READOUT_STAGES)
  int ro_stages = 2;                 // ... with this many 32 KB stages per CTA
  bool ro_explicit = false;          // IM_OPT_READOUT_STAGES has been set: it rules stack calls too (which otherwise take
                                     // the bulk-copy kernel with two stages where it serves the shape)
  bool attn_tc_ready = false;        // the tensor-core streaming attention kernel takes this shape and is set up
  bool attn_tc = false;              // ... and im_decode_step uses it (IM_OPT_DECODE_TENSOR)
  bool fast_attn = false;
  // Independent pieces of one decode call run on three side streams that fork from and join back into
  // the caller's stream (plain event dependencies, so the pattern can be captured into a CUDA graph).
  cudaStream_t side[4] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t ev[14] = {};
  bool concurrent = false;
  bool prefetch_next = true;         // warm L2 with the next layer's weights / index state during attention
  int n_ctas = 1;                    // grid of the streaming attention kernel (SM count)
  int n_sm = 1;                      // SMs of the device
  // The last kernel this context put on a caller's stream, if that was the merge kernel of a concurrent decode
  // call (which writes the call's output and fills the holes of layer `tail_layer`'s cache): only then, and only for
  // another layer, may the next call's attention kernel be launched as its programmatic dependent and fetch cache
  // tiles before that kernel has ended.  After a prefill call, an in-order decode call or a state import the stream's
  // last kernel may have written any layer's cache.
  cudaStream_t tail_stream = nullptr;
  bool tail_is_merge = false;
  int tail_layer = -1;
  bool layer_overlap = true;         // IM_OPT_LAYER_OVERLAP
  // A prefill call that evicts more than the pending list holds leaves the state update of its memory write (Eq. 6-7:
  // pack, sums, Phi^T V) running on `late` when it returns: it needs nothing of the next chunk's projections, append
  // and scoring and runs next to them.  The next call of the context, whatever it is, first makes its stream wait
  // for `ev_late` (a prefill call: just before its own commit kernel, the first that writes a word the update reads).
  cudaStream_t late = nullptr;
  cudaEvent_t ev_late = nullptr, ev_phi = nullptr;
  bool late_pending = false;
  // Such a call also leaves everything behind its append kernel (scoring, commit, selection, gather, hole filling, phi
  // of the evicted keys) running on `pf_tail` when it returns, so that the NEXT chunk's projections, which read the
  // caller's inputs and write scratch that only the append kernel reads, run next to it.  The next prefill call waits
  // for `ev_cache` (cache and counters final) before its fold and append kernels and for `ev_late` before its commit
  // kernel; every other call waits for `ev_late`, which is recorded behind all of it.  (IM_OPT_PREFILL_PIPELINE.)
  cudaStream_t pf_tail = nullptr;
  cudaEvent_t ev_cache = nullptr, ev_app = nullptr;
  bool cache_pending = false;
  bool prefill_pipeline = true;
  // Pipelined stack calls (im_decode_stack): the attention kernels of the call's layers follow one another on
  // `st_attn`, the readout kernels on `st_ro`; everything else of layer j runs on the streams of lane j %
  // IM_STACK_LANES (main: merge; side: the four chains of a decode call), with the lane's events and scratch set.
  struct Lane {
    cudaStream_t main = nullptr, side[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ev[16] = {};
    cudaEvent_t done = nullptr;  // everything of the lane's latest layer has been enqueued behind this
    bool used = false;           // (within the current call)
  } lane[IM_STACK_LANES];
  cudaStream_t st_attn = nullptr, st_ro = nullptr;
  cudaEvent_t st_fork = nullptr, st_attn_done = nullptr, st_ro_done = nullptr;
  std::vector<int> sm_ids;           // ids of the device's SMs (ascending) as a probe kernel saw them; empty: unknown
  bool stack_pipeline = true;        // IM_OPT_STACK_PIPELINE
  int stack_reserved = 0;            // IM_OPT_STACK_RESERVED: SMs kept free of streaming blocks (0: one per sequence, at most 24 / 8)
  bool fold_tensor = true;           // IM_OPT_FOLD_TENSOR
  int stack_chunks = 2;              // IM_OPT_STACK_CHUNKS: runs per warp the attention kernel's tiles are cut into
#ifdef IM_TRACE
  int tune[8] = {0, -1, -1, 0, 0, 0, 0, 0};  // development builds: knobs set through options 100 + k
#endif
  bool score_tc = false;             // prefill scoring runs on the tensor cores (tcgen05)
  bool attend_tc = true;             // chunk attention of im_prefill_chunk_attend on tcgen05 where head_dim is 128
  int prof_target = 0;               // kernel timed by im_profile_*: 0 attention (decode), 1 prefill scoring
  std::vector<cudaEvent_t> prof_ev;  // pairs (start, stop)
  size_t prof_used = 0;              // events recorded so far
};

namespace {

ImLaunch make_launch(im_ctx* ctx, int layer, cudaStream_t s) {
  ImLaunch L;
  L.p = ctx->p;
  L.st = ctx->lo.st;
  L.w = ctx->lo.w[layer];
  L.sc = ctx->lo.sc;
  L.stream = s;
  L.launches = &ctx->launches;
  return L;
}

// makes `s` wait for a state update that an earlier prefill call left running (see im_ctx::late)
cudaError_t join_late(im_ctx* ctx, cudaStream_t s) {
  ctx->cache_pending = false;  // (ev_late is recorded behind everything ev_cache covers)
  if (!ctx->late_pending) return cudaSuccess;
  ctx->late_pending = false;
  return cudaStreamWaitEvent(s, ctx->ev_late, 0);
}

void destroy_lanes(im_ctx* ctx) {
  for (int k = 0; k < IM_STACK_LANES; ++k) {
    im_ctx::Lane& ln = ctx->lane[k];
    if (ln.main) cudaStreamDestroy(ln.main);
    for (int j = 0; j < 4; ++j) if (ln.side[j]) cudaStreamDestroy(ln.side[j]);
    for (int j = 0; j < 16; ++j) if (ln.ev[j]) cudaEventDestroy(ln.ev[j]);
    if (ln.done) cudaEventDestroy(ln.done);
  }
  if (ctx->st_attn) cudaStreamDestroy(ctx->st_attn);
  if (ctx->st_ro) cudaStreamDestroy(ctx->st_ro);
  if (ctx->st_fork) cudaEventDestroy(ctx->st_fork);
  if (ctx->st_attn_done) cudaEventDestroy(ctx->st_attn_done);
  if (ctx->st_ro_done) cudaEventDestroy(ctx->st_ro_done);
}

int check_call(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, ImCall* call) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  if (layer < 0 || layer >= ctx->p.L) return fail(IM_ERR_ARG, "layer %d out of range [0,%d)", layer, ctx->p.L);
  if (n_seq < 1 || n_seq > ctx->p.S || n_seq > IM_MAX_CALL_SEQS)
    return fail(IM_ERR_ARG, "n_seq %d out of range [1,%d]", n_seq, std::min(ctx->p.S, IM_MAX_CALL_SEQS));
  if (!seq_ids) return fail(IM_ERR_ARG, "null seq_ids");
  std::vector<char> seen(ctx->p.S, 0);
  for (int i = 0; i < n_seq; ++i) {
    int s = seq_ids[i];
    if (s < 0 || s >= ctx->p.S) return fail(IM_ERR_ARG, "seq id %d out of range [0,%d)", s, ctx->p.S);
    if (seen[s]) return fail(IM_ERR_ARG, "seq id %d repeated in one call", s);
    seen[s] = 1;
    call->seq[i] = s;
  }
  call->layer = layer;
  call->n_seq = n_seq;
  call->lead = (ctx->p.share >= 2 && layer % ctx->p.share) ? layer - layer % ctx->p.share : -1;
  call->C = 1;
  call->pack = 0;
  call->defer = 0;
  call->fold_all = 0;
  for (int k = 0; k < 5; ++k) { call->warm[k] = nullptr; call->warm_bytes[k] = 0; }
  call->early_cache = 0;
  call->stack = 0;
  call->att_workers = call->ro_claim = call->att_chunks = 0;
  call->fold_ffma = ctx->fold_tensor ? 0 : 1;
  for (int k = 0; k < 4; ++k) call->sm_stream[k] = 0;
  return IM_OK;
}

#define CKL(call)                                                                                 \
  do {                                                                                            \
    cudaError_t e_ = (call);                                                                      \
    if (e_ != cudaSuccess) return fail(IM_ERR_CUDA, "launch %s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

int pick_ksplit(int K, int want) {
  for (int s = want; s > 1; --s)
    if (K % (16 * s) == 0) return s;
  return 1;
}

// the state update of Eq. 6-7 with the per-sequence evicted counts of this call from the host mirror (must be
// called before the mirror is advanced)
cudaError_t launch_mem_update(im_ctx* ctx, const ImLaunch& L, const ImCall& call, int ne_max) {
  const ImDims& p = ctx->p;
  int ne_host[IM_MAX_CALL_SEQS];
  for (int i = 0; i < call.n_seq; ++i) {
    const HostUnit& u = ctx->hu[(size_t)call.layer * p.S + call.seq[i]];
    const bool due = call.prefill || (u.since + 1 == p.tau);
    ne_host[i] = due ? std::max(0, u.n + call.C - p.B) : 0;
  }
  return im_launch_mem_update(L, call, ne_max, ne_host);
}

// phi of the gathered evicted keys (skinny GEMM against the folded Linear_theta), then Eq. 6-7.
// With `update` = false only the GEMM is launched (the caller launches im_launch_mem_update later).
// `before_update`: an event that the kernels changing the memory state wait for (a reader of the state of before)
int run_memory_write(im_ctx* ctx, const ImLaunch& L, ImCall& call, int ne_max, bool update = true, int smem_floor = 0,
                     cudaEvent_t before_update = nullptr, int programmatic = 0, bool own_partials = true) {
  const ImDims& p = ctx->p;
  ImGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.job[0] = {L.w.Wfh, L.w.Wfl, p.dM, 0, 0};
  g.n_jobs = 1;
  g.in[0] = L.sc.evK;
  g.in_cnt[0] = ne_max;
  g.in_outer[0] = (long long)p.tail * p.Dkv;
  g.in_inner[0] = p.Dkv;
  g.NV = call.n_seq * ne_max;
  g.K = p.Dkv;
  g.out_cnt = ne_max;
  g.out_inner = p.dM;
  g.tensor = (call.prefill || g.NV >= 1024) ? 1 : 0;  // thousands of evicted keys: the tensor-core variant
  IM_TRACE_GEMM(g, L, call.layer, 2);
  if (ne_max > p.F) {
    call.phi_large = 1;
    g.out = L.sc.phi;
    g.out_outer = (long long)p.tail * p.dM;
    g.ksplit = 1;
    g.ks_stride = 0;
    // a prefill chunk's few output tiles: two CTAs per tile over the K range, where the partial buffers have room
    const long long extent = (long long)call.n_seq * p.tail * p.dM;
    // (not while the next chunk's projections may be writing those buffers)
    if (own_partials && call.prefill && (p.Dkv / 64) % 2 == 0 && 2 * extent <= (long long)IM_TC_KSPLIT * L.sc.gpart_vecs * p.R3) {
      g.tc_ksplit = 2;
      g.part = L.sc.gpart;
      g.part_stride = extent;
    }
  } else {
    call.phi_large = 0;
    g.out = L.sc.phip;
    g.out_outer = (long long)p.F * p.dM;
    g.ksplit = call.ksplit_phi;
    g.ks_stride = (long long)call.n_seq * p.F * p.dM;
    g.kc = 64;  // 18 KB of shared memory: fits next to the resident attention blocks
    g.direct = call.prefill ? 0 : 1;
    g.smem_floor = smem_floor;
    g.programmatic = programmatic;
  }
  CKL(im_launch_gemm(L, g));
  if (update && before_update) CK(cudaStreamWaitEvent(L.stream, before_update, 0));
  if (update) CKL(launch_mem_update(ctx, L, call, ne_max));
  return IM_OK;
}

// ---- a retained set per KV head (scorer = 1 Knorm, 2 the caller's scores): both calls in order on the caller's stream.
// Append; if due: scores in, selection per head, the evict step's memory write (rows assembled per token, phi by the
// skinny / tensor-core GEMM against the folded Linear_theta, accumulation straight into Mhat), hole filling; decode
// then attends per head slab and adds the readout (Eq. 4-5).
int perhead_compress(im_ctx* ctx, const ImLaunch& L, ImCall& call, int layer, int ne_max, long long T_after) {
  const ImDims& p = ctx->p;
  const float* ext = nullptr;
  long long n_pos = 0;
  if (p.scorer == 2) {
    im_ctx::ExtScores& x = ctx->ext[layer];
    if (!x.ptr) return fail(IM_ERR_STATE, "layer %d compresses with the caller's scores: call im_set_scores first", layer);
    if (x.n_seq != call.n_seq) return fail(IM_ERR_ARG, "im_set_scores named %d sequences, this call %d", x.n_seq, call.n_seq);
    if (x.n_pos < T_after) return fail(IM_ERR_ARG, "the caller's scores cover %lld positions, %lld are cached", x.n_pos, T_after);
    ext = x.ptr;
    n_pos = x.n_pos;
    x = im_ctx::ExtScores();  // consumed
  }
  CKL(im_ph_launch_select(L, call, ext, n_pos));
  if (ne_max > 0) {
    if (p.mem) {
      CKL(im_ph_launch_assemble(L, call, ne_max));
      ImGemmArgs g;
      memset(&g, 0, sizeof(g));
      g.job[0] = {L.w.Wfh, L.w.Wfl, p.dM, 0, 0};
      g.n_jobs = 1;
      g.in[0] = L.sc.evK;
      g.in_cnt[0] = ne_max * p.Hkv;
      g.in_outer[0] = (long long)p.evr * p.Dkv;
      g.in_inner[0] = p.Dkv;
      g.NV = call.n_seq * ne_max * p.Hkv;
      g.K = p.Dkv;
      g.out = L.sc.phi;
      g.out_cnt = ne_max * p.Hkv;
      g.out_outer = (long long)p.evr * p.dM;
      g.out_inner = p.dM;
      g.ksplit = 1;
      g.tensor = g.NV >= 1024 ? 1 : 0;
      CKL(im_launch_gemm(L, g));
      CKL(im_ph_launch_mem_write(L, call));
    }
    CKL(im_ph_launch_move(L, call));
  }
  return IM_OK;
}

int perhead_prefill(im_ctx* ctx, ImCall& call, int layer, int chunk_len, const void* k, const void* v, void* cuda_stream) {
  const ImDims& p = ctx->p;
  int ne_max = 0;
  long long T_after = 0;
  for (int i = 0; i < call.n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    if (u.n + chunk_len > p.cap)
      return fail(IM_ERR_CAPACITY, "sequence %d: %d cached + chunk %d exceeds capacity %d", call.seq[i], u.n, chunk_len, p.cap);
    ne_max = std::max(ne_max, u.n + chunk_len - p.B);
    T_after = std::max(T_after, u.T + chunk_len);
  }
  if ((long long)ne_max * p.Hkv > IM_PH_MAX_PAIRS)
    return fail(IM_ERR_CAPACITY, "per-head sets: %d evicted entries x %d heads exceed %d pairs per evict step", ne_max, p.Hkv, IM_PH_MAX_PAIRS);
  call.C = chunk_len;
  call.prefill = 1;
  call.due = 1;
  ImLaunch L = make_launch(ctx, layer, (cudaStream_t)cuda_stream);
  CKL(im_ph_launch_append(L, call, k, v));
  int rc = perhead_compress(ctx, L, call, layer, ne_max, T_after);
  if (rc) return rc;
  for (int i = 0; i < call.n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    const int ne = std::max(0, u.n + chunk_len - p.B);
    u.n = u.n + chunk_len - ne;
    u.T += chunk_len;
    u.since = 0;
  }
  return IM_OK;
}

int perhead_decode(im_ctx* ctx, ImCall& call, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                   void* cuda_stream) {
  const ImDims& p = ctx->p;
  bool due_any = false, due_all = true;
  int ne_max = 0, n_att = 0;
  long long T_after = 0;
  for (int i = 0; i < call.n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    if (u.n + 1 > p.cap) return fail(IM_ERR_CAPACITY, "sequence %d has no free slot (capacity %d)", call.seq[i], p.cap);
    const bool due = (u.since + 1 == p.tau);
    due_any |= due;
    due_all &= due;
    ne_max = std::max(ne_max, u.n + 1 - p.B);
    T_after = std::max(T_after, u.T + 1);
  }
  if (due_any != due_all)
    return fail(IM_ERR_ARG, "sequences of one decode call must be at the same phase of the compression interval");
  const bool due = due_all;
  if (!due) ne_max = 0;
  if ((long long)ne_max * p.Hkv > IM_PH_MAX_PAIRS)
    return fail(IM_ERR_CAPACITY, "per-head sets: %d evicted entries x %d heads exceed %d pairs per evict step", ne_max, p.Hkv, IM_PH_MAX_PAIRS);
  call.due = due ? 1 : 0;
  call.C = 1;
  call.prefill = 0;
  call.ksplit = pick_ksplit(p.D, IM_KSPLIT);
  call.ksplit_key = 1;
  call.ksplit_phi = 1;
  ImLaunch L = make_launch(ctx, layer, (cudaStream_t)cuda_stream);
  CKL(im_ph_launch_append(L, call, k_new, v_new));
  if (p.mem) {  // phi(q) of Eq. 5 and the gate logit of Eq. 4 (K-split partials, summed by their consumers)
    ImRows r = im_rows(p);
    ImGemmArgs g;
    memset(&g, 0, sizeof(g));
    g.in[2] = (const bf16*)q;
    g.in_cnt[2] = 1;
    g.in_outer[2] = p.D;
    g.out = L.sc.raw;
    g.out_cnt = 1;
    g.out_outer = p.R5;
    g.ks_stride = (long long)call.n_seq * p.R5;
    g.NV = call.n_seq;
    g.K = p.D;
    g.ksplit = call.ksplit;
    g.direct = 1;
    g.job[0] = {L.w.Wt, nullptr, p.dM, r.theta, 2};
    g.job[1] = {L.w.wg, nullptr, 1, r.wg, 2};
    g.n_jobs = 2;
    CKL(im_launch_gemm(L, g));
  }
  if (due) {
    int rc = perhead_compress(ctx, L, call, layer, ne_max, T_after);
    if (rc) return rc;
  }
  for (int i = 0; i < call.n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    const int ne = due ? std::max(0, u.n + 1 - p.B) : 0;
    u.n = u.n + 1 - ne;
    u.T += 1;
    u.since = due ? 0 : u.since + 1;
    n_att = std::max(n_att, u.n);
  }
  // a5 / a6 over the heads' own slabs (all heads of a sequence hold the same number of entries)
  if (ctx->fast_attn) {
    CKL(im_launch_attention_fast(L, call, ctx->mapKs, ctx->mapVs, q, ctx->n_ctas, 0));
    if (p.mem) {
      CKL(im_launch_readout(L, call, ctx->n_sm, 0));
      CKL(im_launch_readout_finish(L, call));
    }
    CKL(im_launch_attention_merge(L, call, out, ctx->n_ctas * IM_ATTN_WARPS, IM_ATTN_STREAM_TILE, 0, q, k_new, v_new, 0));
  } else {
    CKL(im_launch_attention(L, call, q, out, n_att));
  }
  ctx->tail_stream = L.stream;
  return IM_OK;
}

}  // namespace

extern "C" {

const char* im_last_error(void) { return g_err; }

size_t im_workspace_bytes(const im_config* cfg) {
  im_config c;
  ImDims p;
  if (!resolve(cfg, &c, &p)) return 0;
  Layout lo;
  carve(p, nullptr, &lo);
  return lo.total;
}

int im_create(const im_config* cfg, void* dev_workspace, size_t workspace_bytes, im_ctx** out) {
  if (!out) return fail(IM_ERR_ARG, "null out");
  *out = nullptr;
  im_config c;
  ImDims p;
  if (!resolve(cfg, &c, &p)) return fail(IM_ERR_ARG, "invalid configuration");
  if (!dev_workspace || ((uintptr_t)dev_workspace & 255)) return fail(IM_ERR_ARG, "workspace null or not 256-byte aligned");
  im_ctx* ctx = new (std::nothrow) im_ctx();
  if (!ctx) return fail(IM_ERR_ARG, "out of host memory");
  ctx->cfg = c;
  ctx->p = p;
  carve(p, (char*)dev_workspace, &ctx->lo);
#ifdef IM_TRACE
  {
    void* tr = nullptr;
    const size_t bytes = (size_t)p.L * IM_TRACE_KERNELS * IM_TRACE_MARKS * 8;
    if (cudaMalloc(&tr, bytes) == cudaSuccess) cudaMemset(tr, 0, bytes);
    ctx->lo.sc.trace = (unsigned long long*)tr;
  }
#endif
  if (ctx->lo.total > workspace_bytes) {
    size_t need = ctx->lo.total;
    delete ctx;
    return fail(IM_ERR_CAPACITY, "workspace too small: need %zu bytes, got %zu", need, workspace_bytes);
  }
  ctx->hu.assign((size_t)p.L * p.S, HostUnit());
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess)
    e = cudaMemsetAsync((char*)dev_workspace + ctx->lo.state_begin, 0, ctx->lo.state_end - ctx->lo.state_begin, 0);
  // cscale = 1 for every unit
  if (e == cudaSuccess) {
    std::vector<float> ones((size_t)p.L * p.S, 1.0f);
    e = cudaMemcpy(ctx->lo.st.cscale, ones.data(), ones.size() * 4, cudaMemcpyHostToDevice);
  }
  for (int l = 0; l < p.L && e == cudaSuccess; ++l) {
    e = im_launch_init_weights(p, ctx->lo.w[l], l, c.seed, c.init_std, 0);
    if (e == cudaSuccess) e = im_launch_fold_theta(p, ctx->lo.w[l], 0);
  }
  if (e == cudaSuccess && im_attn_fast_supported(p)) {
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e == cudaSuccess) e = im_attn_make_maps(p, ctx->lo.st, ctx->mapK, ctx->mapV, IM_ATTN_TILE);
    if (e == cudaSuccess) e = im_attn_make_maps(p, ctx->lo.st, ctx->mapKs, ctx->mapVs, IM_ATTN_STREAM_TILE, p.d == 128 ? 1 : 0);
    if (e == cudaSuccess) e = im_attn_prepare(p);
    if (e == cudaSuccess && im_attn_tc_supported(p)) {
      e = im_attn_make_maps(p, ctx->lo.st, ctx->mapK128, ctx->mapV128, IM_ATTN_TC_TILE);
      if (e == cudaSuccess) e = im_attn_tc_prepare();
      ctx->attn_tc_ready = (e == cudaSuccess);
    }
    if (e == cudaSuccess && p.mem && im_readout_stream_supported(p)) e = im_readout_stream_prepare(p);
    if (e == cudaSuccess) e = im_gemm_prepare_decode();
    if (e == cudaSuccess) e = im_memory_prepare_decode();
    if (e == cudaSuccess) e = im_front_prepare_decode();
    if (e == cudaSuccess) e = im_prefetch_prepare_decode();
    if (e == cudaSuccess) e = im_chunk_attn_prepare(p);
    if (e == cudaSuccess && im_chunk_attn_tc_supported(p)) e = im_chunk_attn_tc_prepare();
    ctx->n_ctas = std::max(1, std::min(sms, IM_ATTN_MAX_CTAS));
    ctx->fast_attn = (e == cudaSuccess);
  }
  ctx->ext.resize(p.L);
  if (e == cudaSuccess && p.scorer) e = im_perhead_prepare(p);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, ctx->device);
  if (e == cudaSuccess && im_score_tc_supported(p)) {
    e = im_score_tc_prepare();
    ctx->score_tc = (e == cudaSuccess);
  }
  {
    // the short side kernels should be dispatched ahead of the long attention grid when both are ready
    int prio_lo = 0, prio_hi = 0;
    if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    // (numerically lower = higher priority).  The readout stream (side[1]) one step below the others: its
    // kernel has hundreds of blocks, and when it gets onto the SMs first the front kernel (one fat block per
    // sequence, on the critical path) waits until those have drained.
    for (int k = 0; k < 4 && e == cudaSuccess; ++k)
      e = cudaStreamCreateWithPriority(&ctx->side[k], cudaStreamNonBlocking,
                                       (k == 1 && prio_hi + 1 <= prio_lo) ? prio_hi + 1 : prio_hi);
  }
  for (int k = 0; k < 14 && e == cudaSuccess; ++k) e = cudaEventCreateWithFlags(&ctx->ev[k], cudaEventDisableTiming);
  {
    // (highest priority for the state update, one below for the rest of a chunk's tail: with the tail left running
    // the cycle selection -> gather -> phi -> state update -> the next chunk's commit kernel bounds a chunk, and the
    // next chunk's projections, whose blocks are ready at the same time, have the whole of that cycle to finish in:
    // 1.93 against 2.20 ms per 32,768-token prompt with all streams at one priority)
    int prio_lo = 0, prio_hi = 0;
    if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->late, cudaStreamNonBlocking, prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->pf_tail, cudaStreamNonBlocking, std::min(prio_lo, prio_hi + 1));
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_late, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_phi, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_cache, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_app, cudaEventDisableTiming);
  ctx->concurrent = ctx->fast_attn;
  if (e == cudaSuccess && ctx->fast_attn && !p.scorer) {
    // streams, events and the SM ids of pipelined stack calls
    int prio_lo = 0, prio_hi = 0;
    e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
    for (int k = 0; k < IM_STACK_LANES && e == cudaSuccess; ++k) {
      im_ctx::Lane& ln = ctx->lane[k];
      e = cudaStreamCreateWithPriority(&ln.main, cudaStreamNonBlocking, prio_lo);
      for (int j = 0; j < 4 && e == cudaSuccess; ++j) e = cudaStreamCreateWithPriority(&ln.side[j], cudaStreamNonBlocking, prio_lo);
      for (int j = 0; j < 16 && e == cudaSuccess; ++j) e = cudaEventCreateWithFlags(&ln.ev[j], cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ln.done, cudaEventDisableTiming);
    }
    // (the attention kernels above the lanes' small kernels: where a block of either kind could take the registers
    // or the shared memory that an attention block of the previous layer has just released, the next layer's
    // attention block, which is already waiting, gets them; the small kernels run on the SMs set aside and in what is
    // left.  The readout kernels at the lanes' priority: they have half a layer of slack, and with the attention
    // stream's priority their blocks were placed ahead of the chain's; measured over alternated runs 1.940-1.943
    // against 1.949-1.954 ms per step)
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->st_attn, cudaStreamNonBlocking, prio_hi);
    if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&ctx->st_ro, cudaStreamNonBlocking, prio_lo);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->st_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->st_attn_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->st_ro_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->lo.claims, 0, (size_t)IM_STACK_LANES * 8 * 4, 0);
    if (e == cudaSuccess && ctx->n_sm <= 256) {
      std::vector<int> ids(ctx->n_sm);
      int n = 0;
      e = im_probe_sm_ids(ctx->lo.sc.raw, ctx->n_sm, ids.data(), &n, 0);
      if (e == cudaSuccess && n == ctx->n_sm) ctx->sm_ids = ids;
    }
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    destroy_lanes(ctx);
    for (int k = 0; k < 4; ++k) if (ctx->side[k]) cudaStreamDestroy(ctx->side[k]);
    for (int k = 0; k < 14; ++k) if (ctx->ev[k]) cudaEventDestroy(ctx->ev[k]);
    if (ctx->late) cudaStreamDestroy(ctx->late);
    if (ctx->ev_late) cudaEventDestroy(ctx->ev_late);
    if (ctx->ev_phi) cudaEventDestroy(ctx->ev_phi);
    if (ctx->pf_tail) cudaStreamDestroy(ctx->pf_tail);
    if (ctx->ev_cache) cudaEventDestroy(ctx->ev_cache);
    if (ctx->ev_app) cudaEventDestroy(ctx->ev_app);
    delete ctx;
    return fail(IM_ERR_CUDA, "im_create: %s", cudaGetErrorString(e));
  }
  *out = ctx;
  return IM_OK;
}

int im_destroy(im_ctx* ctx) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  cudaError_t e = cudaDeviceSynchronize();
  destroy_lanes(ctx);
  for (int k = 0; k < 4; ++k) if (ctx->side[k]) cudaStreamDestroy(ctx->side[k]);
  for (int k = 0; k < 14; ++k) if (ctx->ev[k]) cudaEventDestroy(ctx->ev[k]);
  if (ctx->late) cudaStreamDestroy(ctx->late);
  if (ctx->ev_late) cudaEventDestroy(ctx->ev_late);
  if (ctx->ev_phi) cudaEventDestroy(ctx->ev_phi);
  if (ctx->pf_tail) cudaStreamDestroy(ctx->pf_tail);
  if (ctx->ev_cache) cudaEventDestroy(ctx->ev_cache);
  if (ctx->ev_app) cudaEventDestroy(ctx->ev_app);
  delete ctx;
  if (e != cudaSuccess) return fail(IM_ERR_CUDA, "im_destroy: %s", cudaGetErrorString(e));
  return IM_OK;
}

int im_get_config(im_ctx* ctx, im_config* out, int32_t* capacity) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  if (out) *out = ctx->cfg;
  if (capacity) *capacity = ctx->p.cap;
  return IM_OK;
}

int64_t im_launch_count(im_ctx* ctx) { return ctx ? ctx->launches : 0; }

int im_reset(im_ctx* ctx, int layer, int seq, void* cuda_stream) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  const ImDims& p = ctx->p;
  if (layer < -1 || layer >= p.L || seq < -1 || seq >= p.S) return fail(IM_ERR_ARG, "layer/seq out of range");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  CK(join_late(ctx, s));
  for (int l = 0; l < p.L; ++l) {
    if (layer >= 0 && l != layer) continue;
    for (int q = 0; q < p.S; ++q) {
      if (seq >= 0 && q != seq) continue;
      size_t u = (size_t)l * p.S + q;
      ImState& st = ctx->lo.st;
      CK(cudaMemsetAsync(st.ctr + u * CTR_STRIDE, 0, CTR_STRIDE * 4, s));
      CK(cudaMemsetAsync(st.Mhat + u * p.dM * p.Dkv, 0, (size_t)p.dM * p.Dkv * 4, s));
      CK(cudaMemsetAsync(st.bvec + u * p.dM, 0, (size_t)p.dM * 4, s));
      // 1.0f as a byte pattern cannot be produced by memset: use a 4-byte copy from a static
      static const float one = 1.0f;
      CK(cudaMemcpyAsync(st.cscale + u, &one, 4, cudaMemcpyHostToDevice, s));
      ctx->hu[u] = HostUnit();
    }
  }
  // a reset of everything also clears the sticky device status word
  if (layer < 0 && seq < 0) CK(cudaMemsetAsync(ctx->lo.st.status, 0, 4, s));
  return IM_OK;
}

// im_prefill_chunk (q = out = null) and im_prefill_chunk_attend
static int prefill_impl(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, int chunk_len, const void* x,
                        const void* q_pre, const void* q, const void* k, const void* v, void* out, bool attend,
                        void* cuda_stream) {
  ImCall call;
  int rc = check_call(ctx, layer, n_seq, seq_ids, &call);
  if (rc) return rc;
  ctx->tail_is_merge = false;
  const ImDims& p = ctx->p;
  if (chunk_len < 1 || chunk_len > p.max_chunk)
    return fail(IM_ERR_ARG, "chunk_len %d out of range [1,%d]", chunk_len, p.max_chunk);
  if (p.scorer) {  // a retained set per KV head: no indexer inputs
    if (attend) return fail(IM_ERR_ARG, "im_prefill_chunk_attend is not available with a retained set per KV head");
    if (!k || !v) return fail(IM_ERR_ARG, "null tensor");
    CK(join_late(ctx, (cudaStream_t)cuda_stream));
    return perhead_prefill(ctx, call, layer, chunk_len, k, v, cuda_stream);
  }
  if (!x || !q_pre || !k || !v) return fail(IM_ERR_ARG, "null tensor");
  if (attend) {
    if (!q || !out) return fail(IM_ERR_ARG, "null tensor");
    if (!p.chunk_out) return fail(IM_ERR_ARG, "im_prefill_chunk_attend needs chunk_outputs = 1 in the configuration");
    if (!ctx->fast_attn)
      return fail(IM_ERR_ARG, "im_prefill_chunk_attend needs head_dim 64 or 128 and at most 8 query heads per KV head");
  }
  int n_max = 0, ne_max = 0;
  for (int i = 0; i < n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    if (u.n + chunk_len > p.cap)
      return fail(IM_ERR_CAPACITY, "sequence %d: %d cached + chunk %d exceeds capacity %d", call.seq[i], u.n, chunk_len, p.cap);
    n_max = std::max(n_max, u.n + chunk_len);
    ne_max = std::max(ne_max, u.n + chunk_len - p.B);
  }
  const bool follow = call.lead >= 0;
  if (follow)  // the leading layer of the group must already have ingested this chunk
    for (int i = 0; i < n_seq; ++i) {
      const HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
      const HostUnit& ul = ctx->hu[(size_t)call.lead * p.S + call.seq[i]];
      if (ul.T != u.T + chunk_len || ul.n != std::min(u.n + chunk_len, p.B))
        return fail(IM_ERR_STATE, "layer %d reuses the scores of layer %d, which has to make this call first (sequence %d)",
                    layer, call.lead, call.seq[i]);
    }
  call.C = chunk_len;
  call.prefill = 1;
  call.due = 1;
  call.ksplit = 1;
  call.ksplit_key = 1;
  call.ksplit_phi = pick_ksplit(p.Dkv, IM_KSPLIT);
  call.pack = (ctx->score_tc && !follow) ? 1 : 0;
  call.fold_all = attend && p.mem ? 1 : 0;
  ImLaunch L = make_launch(ctx, layer, (cudaStream_t)cuda_stream);
  // A state update that the previous prefill call left running (im_ctx::late): the projections, the append and the
  // scoring of this chunk touch nothing that it reads or writes (after a write of that size the pending list of its
  // sequences is empty, so the fold kernel below only looks at their counters), and this call waits for it just before
  // its commit kernel.  A call with outputs reads the memory early: it waits at once.
  if (attend || !ctx->concurrent) CK(join_late(ctx, L.stream));
  const int NV = n_seq * chunk_len;
  // Is everything behind the append kernel left running when the call returns (im_ctx::pf_tail)?  Calls whose every
  // sequence evicts more than the pending list holds (their state update is left running anyway), with the scoring on
  // the tensor cores (the other scoring kernel reads the projections' scratch), not under stream capture.
  bool pipe_tail = ctx->prefill_pipeline && ctx->concurrent && !attend && !follow && p.mem && call.pack && ne_max > p.F;
  for (int i = 0; i < n_seq && pipe_tail; ++i)
    pipe_tail = ctx->hu[(size_t)layer * p.S + call.seq[i]].n + chunk_len - p.B > p.F;
  if (pipe_tail) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(L.stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) pipe_tail = false;
  }
  // pending rank-one terms are folded into M before a compression that cannot append to the list (behind the previous
  // call's tail where that is still running: the fold kernels read the counters it leaves)
  const bool fold_behind = ctx->cache_pending;
  if (!fold_behind && p.mem && (ne_max > 0 || attend)) CKL(im_launch_mem_fold(L, call));
  // a0: indexer projections of every chunk token (Sec. 3.1)
  ImRows r = im_rows(p);
  ImGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.n_jobs = 1;
  g.in[0] = (const bf16*)q_pre;
  g.in[1] = (const bf16*)x;
  for (int k = 0; k < 2; ++k) { g.in_cnt[k] = 1; g.in_outer[k] = p.D; g.in_inner[k] = 0; }
  g.out = L.sc.raw;
  g.out_cnt = 1;
  g.out_outer = p.R3;
  g.NV = NV;
  g.K = p.D;
  g.ksplit = 1;
  g.tensor = 1;
  // few output tiles: cut the K range over more CTAs (not next to the memory-side projections of a call with
  // outputs, whose 80 CTAs already fill the SMs that the two indexer-side launches leave)
  if (!(attend && p.mem) && NV <= L.sc.gpart_vecs && (p.D / 64) % IM_TC_KSPLIT == 0) {
    g.tc_ksplit = IM_TC_KSPLIT;
    g.part = L.sc.gpart;
    g.part_stride = L.sc.gpart_vecs * p.R3;
  }
  // The projections of a chunk are independent of one another and each fills a fraction of the SMs (a launch is
  // bound by the K loop of one CTA): with IM_OPT_CONCURRENCY they run next to one another on the side streams,
  // forked from and joined back into the caller's stream with events.
  const bool fork = ctx->concurrent;
  const bool memside = attend && p.mem;
  ImLaunch Lg = L, Lk = L, Lt = L, Lw = L;
  if (fork) {
    Lg.stream = ctx->side[0];
    Lk.stream = ctx->side[1];
    CK(cudaEventRecord(ctx->ev[0], L.stream));
    CK(cudaStreamWaitEvent(Lg.stream, ctx->ev[0], 0));
    CK(cudaStreamWaitEvent(Lk.stream, ctx->ev[0], 0));
    if (memside) {
      Lt.stream = ctx->side[2];
      Lw.stream = ctx->side[3];
      CK(cudaStreamWaitEvent(Lt.stream, ctx->ev[0], 0));
      CK(cudaStreamWaitEvent(Lw.stream, ctx->ev[0], 0));
    }
  }
  if (!follow) {  // (a layer that reuses another layer's scores has no indexer work)
    g.job[0] = {L.w.Uq, nullptr, p.HI * p.dI, r.uq, 0};
    CKL(im_launch_gemm(L, g));
    g.job[0] = {L.w.G, nullptr, p.HI, r.g, 1};
    CKL(im_launch_gemm(Lg, g));
    CKL(im_launch_proj_key_split(Lk, x, NV, 1));
  }
  if (memside) {
    // phi(q) and the gate logit of every chunk token (behind the indexer-side block of the projection scratch)
    ImGemmArgs g2;
    memset(&g2, 0, sizeof(g2));
    g2.n_jobs = 1;
    g2.in[0] = (const bf16*)q;
    g2.in_cnt[0] = 1;
    g2.in_outer[0] = p.D;
    g2.out = L.sc.raw + (size_t)p.S * p.max_chunk * p.R3;
    g2.out_cnt = 1;
    g2.out_outer = p.dM + 1;
    g2.NV = NV;
    g2.K = p.D;
    g2.ksplit = 1;
    g2.tensor = 1;
    g2.job[0] = {L.w.Wt, nullptr, p.dM, 0, 0};
    CKL(im_launch_gemm(Lt, g2));
    g2.job[0] = {L.w.wg, nullptr, 1, p.dM, 0};
    CKL(im_launch_gemm(Lw, g2));
  }
  if (fork) {
    CK(cudaEventRecord(ctx->ev[1], Lg.stream));
    CK(cudaEventRecord(ctx->ev[2], Lk.stream));
    CK(cudaStreamWaitEvent(L.stream, ctx->ev[1], 0));
    CK(cudaStreamWaitEvent(L.stream, ctx->ev[2], 0));
  }
  if (ctx->cache_pending) {  // the previous call's tail: cache compacted, counters final
    CK(cudaStreamWaitEvent(L.stream, ctx->ev_cache, 0));
    ctx->cache_pending = false;
  }
  if (fold_behind && p.mem && (ne_max > 0 || attend)) CKL(im_launch_mem_fold(L, call));
  CKL(im_launch_prefill_append(L, call, k, v));
  // the rest of the call: on the caller's stream, or on a stream of the library's own that the call leaves running
  ImLaunch T = L;
  if (pipe_tail) {
    CK(cudaEventRecord(ctx->ev_app, L.stream));
    T.stream = ctx->pf_tail;
    CK(cudaStreamWaitEvent(T.stream, ctx->ev_app, 0));
  }
  if (attend) {
    // Layer outputs of the chunk's own queries, before the chunk is compressed: Eq. 5 over the memory of before
    // this chunk, then attention over (cached entries + causal chunk) with the readout added (Eq. 4).  They read the
    // cache and the memory as the append kernel left them (the entry count of before the chunk from CTR_NNEXT, which
    // that kernel sets), so with IM_OPT_CONCURRENCY they run on a side stream NEXT TO the scoring, the selection,
    // the gather and the GEMMs of the memory write; only the kernels that overwrite what they read wait for them:
    // the filling of the holes for the attention kernel (ev[9]), the memory update for the readout (ev[8]).
    ImLaunch La = L;
    if (fork) La.stream = ctx->side[2];  // (the phi(q) projection runs there when there is a memory)
    if (memside) {
      // the readout needs the two memory-side projections only, not the appended chunk
      if (fork) {
        CK(cudaEventRecord(ctx->ev[4], Lw.stream));
        CK(cudaStreamWaitEvent(La.stream, ctx->ev[4], 0));
      }
      CKL(im_launch_chunk_readout(La, call));
      if (fork) CK(cudaEventRecord(ctx->ev[8], La.stream));
    }
    if (fork) {
      CK(cudaEventRecord(ctx->ev[7], L.stream));  // the chunk is appended
      CK(cudaStreamWaitEvent(La.stream, ctx->ev[7], 0));
    }
    if (ctx->attend_tc && im_chunk_attn_tc_supported(p)) CKL(im_launch_chunk_attention_tc(La, call, ctx->mapK, ctx->mapV, q, out));
    else CKL(im_launch_chunk_attention(La, call, ctx->mapK, ctx->mapV, q, out));
    if (fork) CK(cudaEventRecord(ctx->ev[9], La.stream));
  }
  // a1: pooled importance under the causal mask
  {
    const bool prof = ctx->prof_target == 1 && ctx->prof_used + 2 <= ctx->prof_ev.size();
    if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used], T.stream));
    if (follow) {}  // the scores come from the leading layer, after the commit below
    else if (call.pack) CKL(im_launch_prefill_score_tc(T, call, n_max, ctx->n_sm));
    else CKL(im_launch_prefill_score(T, call, n_max));
    if (prof) {
      CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], T.stream));
      ctx->prof_used += 2;
    }
  }
  CK(join_late(ctx, T.stream));
  CKL(im_launch_prefill_commit(T, call));
  if (follow) CKL(im_launch_follow_scores(T, call));
  // a2: selection (also restarts the pooling); a4: gather the evicted pairs, fill the holes
  CKL(im_launch_select(T, call));
  if (ne_max > 0) {
    if (fork && p.mem) {
      // the holes are filled next to the memory write, which works from the gathered copies
      ImLaunch Lm = T;
      Lm.stream = pipe_tail ? ctx->side[2] : ctx->side[0];  // (side[0] may already run the next call's projections)
      CKL(im_launch_gather(T, call, ne_max));
      CK(cudaEventRecord(ctx->ev[5], T.stream));
      CK(cudaStreamWaitEvent(Lm.stream, ctx->ev[5], 0));
      if (attend) CK(cudaStreamWaitEvent(Lm.stream, ctx->ev[9], 0));  // the chunk attention reads the slots that are filled
      CKL(im_launch_move(Lm, call, ne_max));
      CK(cudaEventRecord(ctx->ev[6], Lm.stream));
      if (pipe_tail) {
        CK(cudaEventRecord(ctx->ev_cache, Lm.stream));
        ctx->cache_pending = true;
      }
      // a3.  When every sequence of the call evicts more than the pending list holds, the state update runs on a
      // stream of its own behind phi of the evicted keys and is left running (im_ctx::late); not under stream capture,
      // which every stream that was forked has to rejoin
      bool late = !attend && ne_max > p.F;
      for (int i = 0; i < n_seq && late; ++i)
        late = ctx->hu[(size_t)layer * p.S + call.seq[i]].n + chunk_len - p.B > p.F;
      if (late) {
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(L.stream, &cs) != cudaSuccess || cs != cudaStreamCaptureStatusNone) late = false;
      }
      if (late) {
        if ((rc = run_memory_write(ctx, T, call, ne_max, false, 0, nullptr, 0, !pipe_tail))) return rc;  // phi of the evicted keys
        CK(cudaEventRecord(ctx->ev_phi, T.stream));
        ImLaunch Ll = T;
        Ll.stream = ctx->late;
        CK(cudaStreamWaitEvent(Ll.stream, ctx->ev_phi, 0));
        if (pipe_tail) CK(cudaStreamWaitEvent(Ll.stream, ctx->ev[6], 0));  // ev_late stands for all the call has left running
        CKL(launch_mem_update(ctx, Ll, call, ne_max));
        CK(cudaEventRecord(ctx->ev_late, Ll.stream));
        ctx->late_pending = true;
      } else if ((rc = run_memory_write(ctx, T, call, ne_max, true, 0, memside ? ctx->ev[8] : nullptr))) {
        return rc;
      }
      CK(cudaStreamWaitEvent(T.stream, ctx->ev[6], 0));
    } else {
      if (attend && fork) CK(cudaStreamWaitEvent(T.stream, ctx->ev[9], 0));  // the chunk attention reads the cache
      CKL(im_launch_gather_move(T, call, ne_max));
      // a3: memory write
      if (p.mem && (rc = run_memory_write(ctx, T, call, ne_max))) return rc;
    }
  }
  if (attend && fork) CK(cudaStreamWaitEvent(L.stream, ctx->ev[9], 0));  // join (also when nothing was evicted)
  for (int i = 0; i < n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    const int ne = std::max(0, u.n + chunk_len - p.B);
    u.n = u.n + chunk_len - ne;
    u.T += chunk_len;
    u.since = 0;
  }
  return IM_OK;
}

int im_prefill_chunk(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, int chunk_len, const void* x,
                     const void* q_pre, const void* k, const void* v, void* cuda_stream) {
  return prefill_impl(ctx, layer, n_seq, seq_ids, chunk_len, x, q_pre, nullptr, k, v, nullptr, false, cuda_stream);
}

int im_prefill_chunk_attend(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, int chunk_len, const void* x,
                            const void* q_pre, const void* q, const void* k, const void* v, void* out,
                            void* cuda_stream) {
  return prefill_impl(ctx, layer, n_seq, seq_ids, chunk_len, x, q_pre, q, k, v, out, true, cuda_stream);
}

int im_decode_step(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, const void* x, const void* q_pre,
                   const void* q, const void* k_new, const void* v_new, void* out, void* cuda_stream) {
  ImCall call;
  int rc = check_call(ctx, layer, n_seq, seq_ids, &call);
  if (rc) return rc;
  const ImDims& p = ctx->p;
  CK(join_late(ctx, (cudaStream_t)cuda_stream));
  if (p.scorer) {  // a retained set per KV head: no indexer inputs
    if (!q || !k_new || !v_new || !out) return fail(IM_ERR_ARG, "null tensor");
    ctx->tail_is_merge = false;
    return perhead_decode(ctx, call, layer, q, k_new, v_new, out, cuda_stream);
  }
  if (!x || !q_pre || !q || !k_new || !v_new || !out) return fail(IM_ERR_ARG, "null tensor");
  bool due_any = false, due_all = true;
  int n_max = 0, ne_max = 0;
  for (int i = 0; i < n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    if (u.n + 1 > p.cap) return fail(IM_ERR_CAPACITY, "sequence %d has no free slot (capacity %d)", call.seq[i], p.cap);
    bool due = (u.since + 1 == p.tau);
    due_any |= due;
    due_all &= due;
    n_max = std::max(n_max, u.n + 1);
    ne_max = std::max(ne_max, u.n + 1 - p.B);
  }
  if (due_any != due_all)
    return fail(IM_ERR_ARG, "sequences of one decode call must be at the same phase of the compression interval");
  const bool due = due_all;
  if (!due) ne_max = 0;
  const bool follow = call.lead >= 0;
  if (follow)  // the leading layer of the group must already have taken this token
    for (int i = 0; i < n_seq; ++i) {
      const HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
      const HostUnit& ul = ctx->hu[(size_t)call.lead * p.S + call.seq[i]];
      const int n_after = due ? std::min(u.n + 1, p.B) : u.n + 1;
      if (ul.T != u.T + 1 || ul.n != n_after)
        return fail(IM_ERR_STATE, "layer %d reuses the scores of layer %d, which has to make this call first (sequence %d)",
                    layer, call.lead, call.seq[i]);
    }
  call.due = due ? 1 : 0;
  call.C = 1;
  call.prefill = 0;
  call.ksplit = pick_ksplit(p.D, IM_KSPLIT);
  call.ksplit_key = (p.D % (8 * IM_KSPLIT_KEY) == 0) ? IM_KSPLIT_KEY : 1;
  call.ksplit_phi = pick_ksplit(p.Dkv, IM_KSPLIT);
#ifdef IM_TRACE
  if (ctx->tune[0] > 0) call.ksplit_phi = pick_ksplit(p.Dkv, ctx->tune[0]);
#endif
  // Two schedules.
  //  (A) deferred compaction - the streaming attention kernel is available and the selection, if one is
  //      due, fits the fused front kernel: attention needs nothing of this call but q, so it starts at
  //      once over the entries cached before the call.  The merge adds the new token, removes the evicted
  //      entries again (exactly, see k_attn_merge_rows), adds the terms of this call's memory write to the
  //      readout, and fills the holes.
  //        s0: attention (with SMs set aside for the front kernel: from the start of the call, else after the three
  //            projections) ---------------------------------------------------------> merge
  //        s1: indexer projections -> front (append, score, select, gather) -> phi of the evicted keys
  //            [-> memory write: not needed by the merge, it only has to end with the call]
  //        s2: phi(q) / gate projections -> (front kernel's blocks resident) -> phi(q)^T Mhat next to the attention kernel
  //        s3: float64 key projection (needed by front) -> L2 prefetch for the next layer
  //      The holes of the cache are filled by the merge kernel (the front kernel has listed the moves; the attention
  //      kernel has read the cache by then).
  //        s4: fold of the pending list (before front, which changes the counters, and before the readout) ->
  //            the readout terms that do not go through Mhat, over the memory as it is before the write
  //      With IM_OPT_CONCURRENCY off the same kernels run on s0 in an order that respects these arrows.
  //  (B) in order on s0, attention after the compaction: everything else (large evicted sets, budgets
  //      beyond the fused front kernel, head shapes without the streaming attention kernel).
  {
    const void* in[5] = {x, q_pre, q, k_new, v_new};
    const size_t by[5] = {(size_t)p.D * 2, (size_t)p.D * 2, (size_t)p.D * 2, (size_t)p.Dkv * 2, (size_t)p.Dkv * 2};
    for (int k = 0; k < 5; ++k) { call.warm[k] = in[k]; call.warm_bytes[k] = (unsigned)(by[k] * n_seq); }
  }
  cudaStream_t s0 = (cudaStream_t)cuda_stream;
  // (the merge kernel also fills the holes of ITS layer's cache, after its own wait: a programmatic dependent on the
  // same layer waits for it before it reads anything, see ImCall::early_cache)
  const bool after_merge = ctx->layer_overlap && ctx->tail_is_merge && ctx->tail_stream == s0;
  call.early_cache = (after_merge && ctx->tail_layer != layer) ? 1 : 0;
  ctx->tail_is_merge = false;
  const bool fused = due && n_max <= IM_FRONT_MAX_N && ne_max <= IM_FRONT_MAX_NE;
  const bool defer = ctx->fast_attn && (!due || fused) && ne_max <= p.F;
  const bool conc = defer && ctx->concurrent;
  call.defer = defer ? 1 : 0;
  ImLaunch L = make_launch(ctx, layer, s0);
  ImLaunch L1 = L, L2 = L, L3 = L, L4 = L;
  const bool mem_write = due && ne_max > 0 && p.mem;
  // concurrent schedule: the SMs left to the latency-bound chain (see IM_SMEM_FRONT)
  const int n_res = conc ? im_reserved_sms(ctx->n_sm, n_seq) : 0;
  const int n_ctas_max = n_res > 0 ? std::max(1, std::min(ctx->n_ctas, ctx->n_sm - n_res)) : ctx->n_ctas;
  // the attention grid: no more CTAs than give every warp a run of IM_ATTN_MIN_RUN tiles (a small call cut into
  // one-tile runs leaves the merge kernel a long row of partial results to add per head)
  int n_ctas = n_ctas_max;
  if (!ctx->attn_tc) {
    long long tiles = 0;
    for (int i = 0; i < n_seq; ++i)
      tiles += (long long)((ctx->hu[(size_t)layer * p.S + call.seq[i]].n + IM_ATTN_STREAM_TILE - 1) / IM_ATTN_STREAM_TILE) * p.Hkv;
    const long long want = (tiles + IM_ATTN_WARPS * IM_ATTN_MIN_RUN - 1) / (IM_ATTN_WARPS * IM_ATTN_MIN_RUN);
    n_ctas = (int)std::max<long long>(1, std::min<long long>(n_ctas_max, want));
  }
  if (conc) {
    L1.stream = ctx->side[0];
    L2.stream = ctx->side[1];
    L3.stream = ctx->side[2];
    L4.stream = ctx->side[3];
    CK(cudaEventRecord(ctx->ev[0], s0));
    CK(cudaStreamWaitEvent(L1.stream, ctx->ev[0], 0));
    CK(cudaStreamWaitEvent(L2.stream, ctx->ev[0], 0));
    CK(cudaStreamWaitEvent(L3.stream, ctx->ev[0], 0));
    CK(cudaStreamWaitEvent(L4.stream, ctx->ev[0], 0));
  }
  const bool prof = ctx->prof_target == 0 && ctx->prof_used + 2 <= ctx->prof_ev.size();
  // a0: projections as K-split partial sums: indexer part (Sec. 3.1 features) on s1, launched first: it heads the
  // longest chain of the call ...
  ImRows r = im_rows(p);
  ImGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.in[0] = (const bf16*)q_pre;
  g.in[1] = (const bf16*)x;
  g.in[2] = (const bf16*)q;
  for (int k = 0; k < 3; ++k) { g.in_cnt[k] = 1; g.in_outer[k] = p.D; g.in_inner[k] = 0; }
  g.out = L.sc.raw;
  g.out_cnt = 1;
  g.out_outer = p.R5;
  g.ks_stride = (long long)n_seq * p.R5;
  g.NV = n_seq;
  g.K = p.D;
  g.ksplit = call.ksplit;
  g.kc = conc ? 64 : 0;  // next to the attention CTAs only a small staging buffer fits into an SM's shared memory
  g.direct = 1;          // (used only where the direct variant cannot be: K splits that are not multiples of 32)
  g.job[0] = {L.w.Uq, nullptr, p.HI * p.dI, r.uq, 0};
  g.job[1] = {L.w.G, nullptr, p.HI, r.g, 1};
  g.n_jobs = 2;
  // (the float64 key projection rides along in the same launch where its K range divides: the front kernel then
  // depends on one kernel only and starts behind it as its programmatic dependent)
  // (small calls only: in a large one the projection's blocks share the SMs set aside for the chain with the front
  // blocks, which then find no room to start early)
  int key_ride = 0;
  if (conc && !follow && (p.dI == 8 || p.dI == 16) && (n_res == 0 || (long long)n_seq * (p.Dkv / 64) < ctx->n_sm - n_res))
    for (int ks = 8; ks >= 1 && !key_ride; --ks)
      if (p.D % (256 * ks) == 0) key_ride = ks;
  if (key_ride) {
    g.key_W = L.w.Uk;
    g.key_x = (const bf16*)x;
    g.key_out = L.sc.keyp;
    g.key_nv = n_seq;
    g.key_ksplit = key_ride;
    g.key_dI = p.dI;
    call.ksplit_key = key_ride;
  }
  IM_TRACE_GEMM(g, L, layer, 3);
  g.smem_floor = n_res > 0 ? IM_SMEM_HEAD : 0;  // on the SMs without an attention CTA: its loads are not queued behind a stream's
#ifdef IM_TRACE
  if (ctx->tune[1] >= 0) g.smem_floor = ctx->tune[1] * 1024;
  g.trace_skip = ctx->tune[3];
#endif
  if (!follow) CKL(im_launch_gemm(L1, g));  // (a layer that reuses another layer's scores has no indexer work)
  g.smem_floor = 0;
  g.key_W = nullptr;
  IM_TRACE_GEMM_OFF(g);
  // s3: key projection; s4: fold (reads the counters of before the call; the readout reads the folded state)
  if (!follow && !key_ride) CKL(im_launch_proj_key_split(L3, x, n_seq, call.ksplit_key));
  if (conc) CK(cudaEventRecord(ctx->ev[2], L3.stream));  // key projection done
  if (mem_write) {
    CKL(im_launch_mem_fold(L4, call));
    if (conc) CK(cudaEventRecord(ctx->ev[7], L4.stream));
  }
  // ... memory part (phi(q) of Eq. 5, gate logit of Eq. 4) on s2, followed by the readout
  if (p.mem) {
    g.job[0] = {L.w.Wt, nullptr, p.dM, r.theta, 2};
    g.job[1] = {L.w.wg, nullptr, 1, r.wg, 2};
    CKL(im_launch_gemm(L2, g));
  }
  if (conc) {
    // a5.  The attention kernel needs nothing of the call but q.  Where the front kernel has SMs of its own
    // (n_res > 0) it starts at once and streams the cache while the projections run.  Otherwise the three
    // projections, which head every side chain and are latency bound (one memory round trip each), get the first
    // microseconds of the call to themselves: a memory access issued on an SM that an attention CTA keeps busy
    // takes several times longer, and every kernel of the chain would pay for it.
    CK(cudaEventRecord(ctx->ev[1], L1.stream));
    CK(cudaEventRecord(ctx->ev[6], L2.stream));
    if (n_res == 0) {
      CK(cudaStreamWaitEvent(s0, ctx->ev[1], 0));
      CK(cudaStreamWaitEvent(s0, ctx->ev[6], 0));
      CK(cudaStreamWaitEvent(s0, ctx->ev[2], 0));
    }
    if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used], s0));
    if (ctx->attn_tc) CKL(im_launch_attention_tc(L, call, ctx->mapK, ctx->mapV, ctx->mapK128, ctx->mapV128, q, n_ctas, n_res > 0 && after_merge ? 1 : 0));
    else CKL(im_launch_attention_fast(L, call, ctx->mapKs, ctx->mapVs, q, n_ctas, n_res > 0 && after_merge ? 1 : 0));
    if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], s0));
    CK(cudaEventRecord(ctx->ev[9], s0));  // the attention kernel has ended
  }
  // an evicted set larger than the pending list is accumulated into Mhat itself, which the readout reads
  const bool readout_early = !(mem_write && ne_max > p.F);
  if (conc && mem_write) CK(cudaStreamWaitEvent(L2.stream, ctx->ev[7], 0));
  // s4 again: the part of the readout that does not go through Mhat, over the memory as it is before this call's write
  if (conc) CK(cudaStreamWaitEvent(L4.stream, ctx->ev[6], 0));
  if (defer && p.mem) CKL(im_launch_readout_finish(L4, call));
  if (conc) CK(cudaEventRecord(ctx->ev[4], L4.stream));
  if (conc) {
    CK(cudaStreamWaitEvent(L1.stream, ctx->ev[2], 0));
  }
  // append + a1 (+ a2 and the gather of the evicted pairs when the evicted set is small enough for one
  // block per sequence; a4 in the same kernel unless the compaction is deferred)
  // (with SMs set aside: ev[13] triggers when all blocks of the front kernel have begun to run)
  const bool front_started_ev = conc && n_res > 0;
  int front_pdl = conc && !follow ? 1 : 0;
#ifdef IM_TRACE
  if (ctx->tune[5]) front_pdl = 0;
#endif
  CKL(im_launch_decode_front(L1, call, k_new, v_new, fused ? 1 : 0, n_max, n_res > 0 ? IM_SMEM_FRONT : 0,
                             front_started_ev ? ctx->ev[13] : nullptr, front_pdl));
  if (due && !fused) {
    CKL(im_launch_select(L1, call));
    if (ne_max > 0) CKL(im_launch_gather_move(L1, call, ne_max));
  }
  if (conc) {
    CK(cudaEventRecord(ctx->ev[11], L1.stream));
    CK(cudaStreamWaitEvent(L3.stream, ctx->ev[11], 0));
  }
  // phi(q)^T Mhat on s2.  Where SMs are set aside for the front kernel it starts when every block of that kernel has
  // BEGUN to run (a programmatic event that triggers at block start): launched earlier, its blocks would settle on
  // just those SMs (the emptiest ones) and keep the front blocks out; once the front blocks are resident their
  // registers leave no room for a readout block, so the readout runs beside the attention CTAs and the two streaming
  // kernels end together.
  if (conc) {
    // (a readout with fewer blocks than there are other SMs cannot keep the front blocks out: no need to hold it back)
    const bool few_blocks = (long long)n_seq * (p.Dkv / 64) < ctx->n_sm - n_res;
    if (n_res > 0 && few_blocks) {
    } else if (n_res > 0) {
      CK(cudaStreamWaitEvent(L2.stream, front_started_ev ? ctx->ev[13] : ctx->ev[11], 0));
    } else {
      CK(cudaStreamWaitEvent(L2.stream, ctx->ev[1], 0));
      CK(cudaStreamWaitEvent(L2.stream, ctx->ev[2], 0));
    }
  }
  // (with SMs set aside and the bulk-copy kernel: one CTA beside each attention CTA, its ring next to that CTA's)
  int ro_workers = 0;
  if (ctx->fast_attn && p.mem && readout_early) {
    if (conc && n_res > 0 && ctx->ro_stream) {
      ro_workers = (int)std::min<long long>(n_ctas_max, (long long)n_seq * im_readout_stream_chunks(p));
      CKL(im_launch_readout_stream(L2, call, ro_workers, ctx->ro_stages));
    } else {
      CKL(im_launch_readout(L2, call, n_res > 0 ? n_ctas_max : ctx->n_sm, conc && n_res == 0));
    }
  }
  if (conc) CK(cudaEventRecord(ctx->ev[12], L2.stream));  // s2 finished: the merge needs phi(q)^T Mhat
  // (a context of one layer has no next layer to warm L2 for: what the next call reads is what this one has just read,
  // and the two kernels, which end after the merge, would only hold the next call back: 7 us of a 31 us step)
  const bool warm_next = ctx->prefetch_next && p.L > 1;
  if (warm_next && ctx->fast_attn) {
    // warm L2 for the next layer's small kernels while this layer's attention streams K/V; after the front kernel,
    // which should find its SMs free of other kernels' blocks
    ImLaunch Lp = L3;
    ImCall nxt = call;
    nxt.layer = (layer + 1) % p.L;
    Lp.w = ctx->lo.w[nxt.layer];
    CKL(im_launch_prefetch_layer(Lp, nxt));
  }
  if (conc && warm_next && p.mem && n_res > 0) {
    // Half of the next layer's memory matrices go into L2 while this call's merge runs: the streaming kernels have
    // ended, nothing else asks for HBM, and the next call's readout then finds these rows in L2 while its attention
    // kernel has the DRAM channels (measured: a step of the 32-layer benchmark takes 2.26 ms with half of each
    // matrix, 2.30 ms with a quarter, 2.37 ms with none, 2.40 ms with all of it, which the streams evict again)
    int eighths = IM_PREFETCH_MEM_EIGHTHS;
#ifdef IM_TRACE
    if (ctx->tune[2] >= 0) eighths = ctx->tune[2];
#endif
    ImCall nxt = call;
    nxt.layer = (layer + 1) % p.L;
    CK(cudaStreamWaitEvent(L3.stream, ctx->ev[9], 0));
    int pm_blocks = 1;
#ifdef IM_TRACE
    if (ctx->tune[4] > 0) pm_blocks = ctx->tune[4];
#endif
    CKL(im_launch_prefetch_memory(L3, nxt, eighths, pm_blocks));
  }
  if (conc) CK(cudaEventRecord(ctx->ev[10], L3.stream));  // s3 has to end with the call
  // a3: memory write (needs the gathered evicted pairs and the fold).  With deferred compaction the merge kernel
  // forms the readout of the state after the write from phi of the evicted keys, and the state update itself
  // follows off the critical path, after the readout kernels that want the state from before it.
  // (a small call on an idle device: the phi GEMM starts behind the front kernel as its programmatic dependent; in a
  // large one its blocks would wait on SMs that a streaming kernel keeps busy)
  const bool phi_pdl = conc && fused && n_res > 0 && (long long)n_seq * (p.Dkv / 64) < ctx->n_sm - n_res;
  if (mem_write && (rc = run_memory_write(ctx, L1, call, ne_max, !defer, n_res > 0 ? IM_SMEM_SIDE : 0, nullptr, phi_pdl ? 1 : 0))) return rc;
  if (conc) CK(cudaEventRecord(ctx->ev[3], L1.stream));  // everything the merge needs from s1
  if (conc) CK(cudaStreamWaitEvent(L1.stream, ctx->ev[4], 0));  // k_readout_finish reads what the update changes
  if (defer && mem_write) CKL(launch_mem_update(ctx, L1, call, ne_max));
  if (mem_write && ctx->fast_attn && !readout_early) CKL(im_launch_readout(L1, call, ctx->n_sm, 0));
  int n_att = 0;
  for (int i = 0; i < n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    const int ne = due ? std::max(0, u.n + 1 - p.B) : 0;
    u.n = u.n + 1 - ne;
    u.T += 1;
    u.since = due ? 0 : u.since + 1;
    n_att = std::max(n_att, u.n);
  }
  // a5: attention; a6: merge, gate, fuse (Eq. 4)
  if (ctx->fast_attn) {
    if (!conc) {
      if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used], s0));
      if (ctx->attn_tc) CKL(im_launch_attention_tc(L, call, ctx->mapK, ctx->mapV, ctx->mapK128, ctx->mapV128, q, n_ctas, 0));
      else CKL(im_launch_attention_fast(L, call, ctx->mapKs, ctx->mapVs, q, n_ctas, 0));
      if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], s0));
    }
    if (!defer && p.mem) CKL(im_launch_readout_finish(L, call));  // after the memory write
    if (conc) {
      CK(cudaStreamWaitEvent(s0, ctx->ev[3], 0));  // s1 (which waited for s2)
      CK(cudaStreamWaitEvent(s0, ctx->ev[12], 0));  // s2
      CK(cudaStreamWaitEvent(s0, ctx->ev[4], 0));   // s4
    }
    CKL(im_launch_attention_merge(L, call, out, ctx->attn_tc ? n_ctas : n_ctas * IM_ATTN_WARPS,
                                  ctx->attn_tc ? IM_ATTN_TC_TILE : IM_ATTN_STREAM_TILE, ro_workers, q, k_new, v_new, conc ? 1 : 0));
    if (conc) CK(cudaStreamWaitEvent(s0, ctx->ev[10], 0));
    if (conc) {  // the memory write only has to end with the call
      CK(cudaEventRecord(ctx->ev[5], L1.stream));
      CK(cudaStreamWaitEvent(s0, ctx->ev[5], 0));
    }
  } else {
    if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used], s0));
    CKL(im_launch_attention(L, call, q, out, n_att));
    if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], s0));
  }
  if (prof) ctx->prof_used += 2;
  ctx->tail_is_merge = conc;
  ctx->tail_stream = s0;
  ctx->tail_layer = layer;
  return IM_OK;
}

namespace {

// What a decode call on `layer` would do, from the host mirror: phase of the interval, largest entry count after the
// append and largest evicted set among the call's sequences.  Returns false where im_decode_step would refuse the call.
bool decode_plan(im_ctx* ctx, int layer, const ImCall& call, bool* due, int* n_max, int* ne_max) {
  const ImDims& p = ctx->p;
  bool due_any = false, due_all = true;
  *n_max = 0;
  *ne_max = 0;
  for (int i = 0; i < call.n_seq; ++i) {
    const HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    if (u.n + 1 > p.cap) return false;
    const bool d = (u.since + 1 == p.tau);
    due_any |= d;
    due_all &= d;
    *n_max = std::max(*n_max, u.n + 1);
    *ne_max = std::max(*ne_max, u.n + 1 - p.B);
  }
  if (due_any != due_all) return false;
  *due = due_all;
  if (!*due) *ne_max = 0;
  return true;
}

// does a pipelined stack call form phi(q)^T Mhat with the bulk-copy kernel?
bool stack_bulk_readout(const im_ctx* ctx) {
  return (ctx->ro_explicit ? ctx->ro_stream : true) && ctx->p.mem && im_readout_stream_supported(ctx->p);
}

// One layer of a pipelined stack call (see im_decode_stack): the kernels of im_decode_step's concurrent schedule with
// deferred compaction, enqueued on the lane's streams, the call's attention stream and its readout stream.
int stack_layer(im_ctx* ctx, int j, int layer, int n_seq, const int32_t* seq_ids, int n_res, const unsigned long long* sm_stream,
                const void* x, const void* q_pre, const void* q, const void* k_new, const void* v_new, void* out,
                cudaEvent_t ready, cudaEvent_t done) {
  const ImDims& p = ctx->p;
  ImCall call;
  int rc = check_call(ctx, layer, n_seq, seq_ids, &call);
  if (rc) return rc;
  bool due = false;
  int n_max = 0, ne_max = 0;
  if (!decode_plan(ctx, layer, call, &due, &n_max, &ne_max)) return fail(IM_ERR_STATE, "layer %d: the call's plan changed under it", layer);
  const int k = j % IM_STACK_LANES;
  im_ctx::Lane& ln = ctx->lane[k];
  call.due = due ? 1 : 0;
  call.C = 1;
  call.prefill = 0;
  call.ksplit = pick_ksplit(p.D, IM_KSPLIT);
  call.ksplit_key = (p.D % (8 * IM_KSPLIT_KEY) == 0) ? IM_KSPLIT_KEY : 1;
  call.ksplit_phi = pick_ksplit(p.Dkv, IM_KSPLIT);
  call.defer = 1;
  call.early_cache = 1;
  call.stack = 1;
  for (int w = 0; w < 4; ++w) call.sm_stream[w] = sm_stream[w];
  const bool fused = due;
  const bool mem_write = due && ne_max > 0;
  // workers of the two streaming kernels
  const int n_wk_max = std::max(1, std::min(ctx->n_ctas, ctx->n_sm - n_res));
  long long tiles = 0;
  for (int i = 0; i < n_seq; ++i)
    tiles += (long long)((ctx->hu[(size_t)layer * p.S + call.seq[i]].n + IM_ATTN_STREAM_TILE - 1) / IM_ATTN_STREAM_TILE) * p.Hkv;
  const long long want = (tiles + IM_ATTN_WARPS * IM_ATTN_MIN_RUN - 1) / (IM_ATTN_WARPS * IM_ATTN_MIN_RUN);
  call.att_workers = (int)std::max<long long>(1, std::min<long long>(n_wk_max, want));
  call.ro_claim = (int)std::max<long long>(1, std::min<long long>(n_wk_max, (long long)n_seq * (p.Dkv / 64)));
  // runs the attention kernel's tiles are cut into: a few per warp, so that a block that starts late takes fewer
  call.att_chunks = std::min(call.att_workers * IM_ATTN_WARPS * ctx->stack_chunks, IM_ATTN_MAX_CTAS * IM_ATTN_WARPS);
  // streams: the lane's own wait for the lane's previous layer (its scratch set), or for the start of the call
  ImLaunch L = make_launch(ctx, layer, ln.main);
  L.sc = ctx->lo.lane[k];
  ImLaunch L1 = L, L2 = L, L3 = L, L4 = L, LA = L, LR = L;
  L1.stream = ln.side[0];
  L2.stream = ln.side[1];
  L3.stream = ln.side[2];
  L4.stream = ln.side[3];
  LA.stream = ctx->st_attn;
  LR.stream = ctx->st_ro;
  if (!ln.used) {
    CK(cudaStreamWaitEvent(ln.main, ctx->st_fork, 0));
    for (int w = 0; w < 4; ++w) CK(cudaStreamWaitEvent(ln.side[w], ctx->st_fork, 0));
  } else {
    for (int w = 0; w < 4; ++w) CK(cudaStreamWaitEvent(ln.side[w], ln.done, 0));
    CK(cudaStreamWaitEvent(LA.stream, ln.done, 0));
    CK(cudaStreamWaitEvent(LR.stream, ln.done, 0));
  }
  // The caller's event for this layer's inputs: every stream of the lane that reads them waits for it.  The attention
  // kernel (launched as a programmatic dependent, and reading q before it waits for anything) is held behind the
  // lane's first projection instead, an ordinary launch that has waited for the event in full.
  if (ready) {
    for (int w = 0; w < 4; ++w) CK(cudaStreamWaitEvent(ln.side[w], ready, 0));
    CK(cudaStreamWaitEvent(ln.main, ready, 0));
  }
  // a0: projections.  s1: indexer part (heads the chain that decides the eviction)
  ImRows r = im_rows(p);
  ImGemmArgs g;
  memset(&g, 0, sizeof(g));
  g.in[0] = (const bf16*)q_pre;
  g.in[1] = (const bf16*)x;
  g.in[2] = (const bf16*)q;
  for (int w = 0; w < 3; ++w) { g.in_cnt[w] = 1; g.in_outer[w] = p.D; g.in_inner[w] = 0; }
  g.out = L.sc.raw;
  g.out_cnt = 1;
  g.out_outer = p.R5;
  g.ks_stride = (long long)n_seq * p.R5;
  g.NV = n_seq;
  g.K = p.D;
  g.ksplit = call.ksplit;
  g.kc = 64;
  g.direct = 1;
  g.job[0] = {L.w.Uq, nullptr, p.HI * p.dI, r.uq, 0};
  g.job[1] = {L.w.G, nullptr, p.HI, r.g, 1};
  g.n_jobs = 2;
  int key_ride = 0;
  if ((p.dI == 8 || p.dI == 16) && (long long)n_seq * (p.Dkv / 64) < ctx->n_sm - n_res)
    for (int ks = 8; ks >= 1 && !key_ride; --ks)
      if (p.D % (256 * ks) == 0) key_ride = ks;
  if (key_ride) {
    g.key_W = L.w.Uk;
    g.key_x = (const bf16*)x;
    g.key_out = L.sc.keyp;
    g.key_nv = n_seq;
    g.key_ksplit = key_ride;
    g.key_dI = p.dI;
    call.ksplit_key = key_ride;
  }
  // (no shared-memory floors here: in im_decode_step they keep the small kernels' blocks off the SMs of the attention
  // blocks, in a stack call they would keep an attention block off an SM it finds free between two layers)
  CKL(im_launch_gemm(L1, g));
  if (ready) {
    CK(cudaEventRecord(ln.ev[10], L1.stream));
    CK(cudaStreamWaitEvent(LA.stream, ln.ev[10], 0));
  }
  g.key_W = nullptr;
  // s3: key projection; s4: fold of the pending list
  if (!key_ride) CKL(im_launch_proj_key_split(L3, x, n_seq, call.ksplit_key));
  CK(cudaEventRecord(ln.ev[2], L3.stream));
  if (mem_write) {
    CKL(im_launch_mem_fold(L4, call));
    CK(cudaEventRecord(ln.ev[7], L4.stream));
  }
  // s2: phi(q) and the gate logit
  g.job[0] = {L.w.Wt, nullptr, p.dM, r.theta, 2};
  g.job[1] = {L.w.wg, nullptr, 1, r.wg, 2};
  CKL(im_launch_gemm(L2, g));
  CK(cudaEventRecord(ln.ev[6], L2.stream));
  // a5 on the call's attention stream: behind the previous layer's attention kernel as its programmatic dependent
  // (it becomes resident as that kernel's blocks end, and waits for nothing)
  const bool prof = ctx->prof_target == 0 && ctx->prof_used + 2 <= ctx->prof_ev.size();
  if (prof) CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used], LA.stream));
  CKL(im_launch_attention_fast(LA, call, ctx->mapKs, ctx->mapVs, q, std::max(ctx->n_sm, call.att_workers), j > 0 ? 1 : 0));
  if (prof) {
    CK(cudaEventRecord(ctx->prof_ev[ctx->prof_used + 1], LA.stream));
    ctx->prof_used += 2;
  }
  CK(cudaEventRecord(ln.ev[9], LA.stream));
  // s4: the part of the readout that does not go through Mhat, over the memory as it is before this call's write
  CK(cudaStreamWaitEvent(L4.stream, ln.ev[6], 0));
  CKL(im_launch_readout_finish(L4, call));
  CK(cudaEventRecord(ln.ev[4], L4.stream));
  // s1: append, score, select, gather, list the moves
  CK(cudaStreamWaitEvent(L1.stream, ln.ev[2], 0));
  CKL(im_launch_decode_front(L1, call, k_new, v_new, fused ? 1 : 0, n_max, 0, nullptr, 1));
  // phi(q)^T Mhat on the call's readout stream
  CK(cudaStreamWaitEvent(LR.stream, ln.ev[6], 0));
  if (mem_write) CK(cudaStreamWaitEvent(LR.stream, ln.ev[7], 0));
  // The bulk-copy kernel by default (fixed runs of 32 KB chunks, a partial vector per block, two stages per block): it
  // needs a few registers where the plain-load kernel fills the SM's register file next to an attention block, so the
  // small kernels of the layers in flight find room on the streaming SMs at all times, and the memory system serves
  // its few large copies better than the other's many small loads (1.87 against 1.96 ms per step of the 32-layer
  // benchmark, with 24 against 8 SMs set aside).
  int ro_workers = 0;
  if (stack_bulk_readout(ctx)) {
    ro_workers = (int)std::min<long long>(n_wk_max, (long long)n_seq * im_readout_stream_chunks(p));
    CKL(im_launch_readout_stream(LR, call, ro_workers, ctx->ro_explicit ? ctx->ro_stages : 2));
  } else {
    CKL(im_launch_readout(LR, call, std::max(ctx->n_sm, call.ro_claim), 0));
  }
  CK(cudaEventRecord(ln.ev[12], LR.stream));
  // a3: phi of the evicted keys, then (off the path to the merge) the state update
  if (mem_write && (rc = run_memory_write(ctx, L1, call, ne_max, false, 0, nullptr, 0))) return rc;
  CK(cudaEventRecord(ln.ev[3], L1.stream));
  CK(cudaStreamWaitEvent(L1.stream, ln.ev[4], 0));
  if (mem_write) CKL(launch_mem_update(ctx, L1, call, ne_max));
  CK(cudaEventRecord(ln.ev[5], L1.stream));
  for (int i = 0; i < n_seq; ++i) {
    HostUnit& u = ctx->hu[(size_t)layer * p.S + call.seq[i]];
    const int ne = due ? std::max(0, u.n + 1 - p.B) : 0;
    u.n = u.n + 1 - ne;
    u.T += 1;
    u.since = due ? 0 : u.since + 1;
  }
  // a6: merge, gate, fuse; a4: the merge fills the holes
  CK(cudaStreamWaitEvent(ln.main, ln.ev[9], 0));
  CK(cudaStreamWaitEvent(ln.main, ln.ev[3], 0));
  CK(cudaStreamWaitEvent(ln.main, ln.ev[12], 0));
  CK(cudaStreamWaitEvent(ln.main, ln.ev[4], 0));
  CKL(im_launch_attention_merge(L, call, out, call.att_chunks, IM_ATTN_STREAM_TILE, ro_workers, q, k_new, v_new, 0));
  if (done) CK(cudaEventRecord(done, ln.main));  // the layer's output is complete
  CK(cudaStreamWaitEvent(ln.main, ln.ev[5], 0));
  CK(cudaStreamWaitEvent(ln.main, ln.ev[2], 0));
  CK(cudaEventRecord(ln.done, ln.main));
  ln.used = true;
  return IM_OK;
}

}  // namespace

extern "C" int im_decode_stack(im_ctx* ctx, int n_layers, const int32_t* layers, int n_seq, const int32_t* seq_ids,
                               const void* const* x, const void* const* q_pre, const void* const* q, const void* const* k_new,
                               const void* const* v_new, void* const* out, void* cuda_stream) {
  return im_decode_stack_events(ctx, n_layers, layers, n_seq, seq_ids, x, q_pre, q, k_new, v_new, out, nullptr, nullptr, cuda_stream);
}

extern "C" int im_decode_stack_events(im_ctx* ctx, int n_layers, const int32_t* layers, int n_seq, const int32_t* seq_ids,
                                      const void* const* x, const void* const* q_pre, const void* const* q,
                                      const void* const* k_new, const void* const* v_new, void* const* out,
                                      void* const* ready_events, void* const* done_events, void* cuda_stream) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  const ImDims& p = ctx->p;
  if (n_layers < 1 || n_layers > p.L) return fail(IM_ERR_ARG, "n_layers %d out of range [1,%d]", n_layers, p.L);
  if (!layers || !q || !k_new || !v_new || !out || (!p.scorer && (!x || !q_pre))) return fail(IM_ERR_ARG, "null pointer list");
  {
    std::vector<char> seen(p.L, 0);
    for (int j = 0; j < n_layers; ++j) {
      if (layers[j] < 0 || layers[j] >= p.L) return fail(IM_ERR_ARG, "layer %d out of range [0,%d)", layers[j], p.L);
      if (seen[layers[j]]) return fail(IM_ERR_ARG, "layer %d repeated in one call", layers[j]);
      seen[layers[j]] = 1;
    }
  }
  // The pipelined schedule takes calls whose every layer runs im_decode_step's concurrent schedule with deferred
  // compaction and SMs set aside for the chain of small kernels; anything else goes layer by layer.
  bool pipe = ctx->stack_pipeline && n_layers >= 2 && ctx->fast_attn && ctx->concurrent && !ctx->attn_tc &&
              !p.scorer && !p.share && p.mem && !ctx->sm_ids.empty() && ctx->st_attn != nullptr;
  int n_res = 0;
  if (pipe) {
    // (far fewer than im_decode_step sets aside: the small kernels are off the path that bounds the call, and while
    // a layer's readout block is absent from a streaming SM they find registers there as well)
    // (with the bulk-copy readout kernel, whose shared-memory ring leaves little room for the small kernels' blocks next
    // to an attention block, a few more: 24 measured best on the 32-layer benchmark, 16: +2 %, 32: +4 %; with the
    // plain-load kernel 8)
    n_res = ctx->stack_reserved > 0 ? ctx->stack_reserved
                                    : std::min(im_reserved_sms(ctx->n_sm, n_seq), stack_bulk_readout(ctx) ? 24 : 8);
    pipe = n_res > 0 && n_res < ctx->n_sm;
  }
  for (int j = 0; j < n_layers && pipe; ++j) {
    ImCall call;
    if (check_call(ctx, layers[j], n_seq, seq_ids, &call)) { pipe = false; break; }
    bool due = false;
    int n_max = 0, ne_max = 0;
    if (!decode_plan(ctx, layers[j], call, &due, &n_max, &ne_max)) { pipe = false; break; }
    if (due && !(n_max <= IM_FRONT_MAX_N && ne_max <= IM_FRONT_MAX_NE)) pipe = false;
    if (ne_max > p.F) pipe = false;
  }
  if (!pipe) {
    for (int j = 0; j < n_layers; ++j) {
      if (ready_events && ready_events[j]) CK(cudaStreamWaitEvent((cudaStream_t)cuda_stream, (cudaEvent_t)ready_events[j], 0));
      const int rc = im_decode_step(ctx, layers[j], n_seq, seq_ids, x ? x[j] : nullptr, q_pre ? q_pre[j] : nullptr, q[j], k_new[j],
                                    v_new[j], out[j], cuda_stream);
      if (rc) return rc;
      if (done_events && done_events[j]) CK(cudaEventRecord((cudaEvent_t)done_events[j], (cudaStream_t)cuda_stream));
    }
    return IM_OK;
  }
  for (int j = 0; j < n_layers; ++j)
    if (!x[j] || !q_pre[j] || !q[j] || !k_new[j] || !v_new[j] || !out[j]) return fail(IM_ERR_ARG, "null tensor (layer %d)", layers[j]);
  cudaStream_t s0 = (cudaStream_t)cuda_stream;
  CK(join_late(ctx, s0));
  ctx->tail_is_merge = false;
  // SMs for the streaming kernels: all but n_res, taken as pairs of neighbouring ids at even distances over the id
  // range, so that every part of the chip keeps both kinds of SMs
  unsigned long long sm_stream[4] = {0, 0, 0, 0};
  {
    const int n = ctx->n_sm;
    std::vector<char> res(n, 0);
    const int pairs = n / 2, want = n_res / 2;
    for (int k = 0; k < want; ++k) {
      const int t = (int)(((long long)(2 * k + 1) * pairs) / (2 * want));
      res[2 * t] = res[2 * t + 1] = 1;
    }
    if (n_res & 1)  // one more: the first SM that is still free
      for (int w = 0; w < n; ++w)
        if (!res[w]) { res[w] = 1; break; }
    for (int w = 0; w < n; ++w)
      if (!res[w]) sm_stream[ctx->sm_ids[w] >> 6] |= 1ull << (ctx->sm_ids[w] & 63);
  }
  CK(cudaEventRecord(ctx->st_fork, s0));
  CK(cudaStreamWaitEvent(ctx->st_attn, ctx->st_fork, 0));
  CK(cudaStreamWaitEvent(ctx->st_ro, ctx->st_fork, 0));
  for (int k = 0; k < IM_STACK_LANES; ++k) ctx->lane[k].used = false;
  for (int j = 0; j < n_layers; ++j) {
    const int rc = stack_layer(ctx, j, layers[j], n_seq, seq_ids, n_res, sm_stream, x[j], q_pre[j], q[j], k_new[j], v_new[j], out[j],
                               ready_events ? (cudaEvent_t)ready_events[j] : nullptr, done_events ? (cudaEvent_t)done_events[j] : nullptr);
    if (rc) return rc;  // (streams forked so far are rejoined by the caller's next synchronisation only: the call has failed)
  }
  CK(cudaEventRecord(ctx->st_attn_done, ctx->st_attn));
  CK(cudaEventRecord(ctx->st_ro_done, ctx->st_ro));
  CK(cudaStreamWaitEvent(s0, ctx->st_attn_done, 0));
  CK(cudaStreamWaitEvent(s0, ctx->st_ro_done, 0));
  for (int k = 0; k < IM_STACK_LANES; ++k)
    if (ctx->lane[k].used) CK(cudaStreamWaitEvent(s0, ctx->lane[k].done, 0));
  return IM_OK;
}

#ifdef IM_TRACE
extern "C" int im_trace_read(im_ctx* ctx, unsigned long long* host, long long n) {
  cudaDeviceSynchronize();
  const long long have = (long long)ctx->p.L * IM_TRACE_KERNELS * IM_TRACE_MARKS;
  return cudaMemcpy(host, ctx->lo.sc.trace, (size_t)std::min(n, have) * 8, cudaMemcpyDeviceToHost) == cudaSuccess ? 0 : -1;
}
#endif

int im_set_option(im_ctx* ctx, int option, int value) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  switch (option) {
    case IM_OPT_CONCURRENCY: ctx->concurrent = value != 0; return IM_OK;
    case IM_OPT_PREFETCH_NEXT: ctx->prefetch_next = value != 0; return IM_OK;
    case IM_OPT_PREFILL_TENSOR:
      if (value && !im_score_tc_supported(ctx->p) && !im_chunk_attn_tc_supported(ctx->p))
        return fail(IM_ERR_ARG, "no tensor-core prefill kernel takes this shape (scoring: at most %d indexer heads of width 8 or 16; chunk attention: head_dim 128)", IM_TC_HP);
      ctx->score_tc = value != 0 && im_score_tc_supported(ctx->p);
      ctx->attend_tc = value != 0;
      return IM_OK;
    case IM_OPT_PROFILE_TARGET:
      if (value != 0 && value != 1) return fail(IM_ERR_ARG, "profile target %d: 0 = attention, 1 = prefill scoring", value);
      if (!ctx->prof_ev.empty()) return fail(IM_ERR_STATE, "profiling is active");
      ctx->prof_target = value;
      return IM_OK;
    case IM_OPT_DECODE_TENSOR:
      if (value && !(ctx->fast_attn && ctx->attn_tc_ready))
        return fail(IM_ERR_ARG, "the tensor-core decode attention kernel needs head_dim 128 and at most 8 query heads per KV head");
      ctx->attn_tc = value != 0;
      ctx->tail_is_merge = false;
      return IM_OK;
    case IM_OPT_LAYER_OVERLAP: ctx->layer_overlap = value != 0; return IM_OK;
    case IM_OPT_STACK_PIPELINE: ctx->stack_pipeline = value != 0; return IM_OK;
    case IM_OPT_FOLD_TENSOR: ctx->fold_tensor = value != 0; return IM_OK;
    case IM_OPT_PREFILL_PIPELINE: ctx->prefill_pipeline = value != 0; return IM_OK;
    case IM_OPT_STACK_CHUNKS:
      if (value < 1 || value > 16) return fail(IM_ERR_ARG, "runs per warp %d out of range [1,16]", value);
      ctx->stack_chunks = value;
      return IM_OK;
    case IM_OPT_STACK_RESERVED:
      if (value < 0 || value >= ctx->n_sm) return fail(IM_ERR_ARG, "reserved SMs %d out of range [0,%d)", value, ctx->n_sm);
      ctx->stack_reserved = value;
      return IM_OK;
#ifdef IM_TRACE
    case 100: case 101: case 102: case 103: case 104: case 105: case 106: case 107: ctx->tune[option - 100] = value; return IM_OK;
#endif
    case IM_OPT_WAIT_LIMIT:
      if (value < 0) return fail(IM_ERR_ARG, "wait limit %d: 0 = default, k >= 1 = k - 1 attempts", value);
      ctx->p.wait_limit = value == 0 ? IM_WAIT_LIMIT : (uint32_t)(value - 1);
      return IM_OK;
    case IM_OPT_READOUT_STAGES:
      if (value < 0 || value > 6) return fail(IM_ERR_ARG, "readout stages %d out of range [0,6]", value);
      if (value > 0 && !(ctx->fast_attn && ctx->p.mem && im_readout_stream_supported(ctx->p)))
        return fail(IM_ERR_ARG, "the bulk-copy readout kernel does not take this shape (D_kv a power of two of at most 1024, d_M a multiple of 8192 / D_kv)");
      ctx->ro_stream = value > 0;
      ctx->ro_explicit = true;
      if (value > 0) ctx->ro_stages = value;
      return IM_OK;
    default: return fail(IM_ERR_ARG, "unknown option %d", option);
  }
}

int im_profile_begin(im_ctx* ctx, int max_records) {
  if (!ctx || max_records < 1 || max_records > (1 << 20)) return fail(IM_ERR_ARG, "bad profile request");
  if (!ctx->prof_ev.empty()) return fail(IM_ERR_STATE, "profiling already active");
  ctx->prof_ev.resize((size_t)max_records * 2);
  ctx->prof_used = 0;
  for (auto& e : ctx->prof_ev) {
    cudaError_t rc = cudaEventCreate(&e);
    if (rc != cudaSuccess) {
      ctx->prof_ev.clear();
      return fail(IM_ERR_CUDA, "cudaEventCreate: %s", cudaGetErrorString(rc));
    }
  }
  return IM_OK;
}

int im_profile_end(im_ctx* ctx, double* total_ms, int64_t* n_records) {
  if (!ctx || !total_ms || !n_records) return fail(IM_ERR_ARG, "null argument");
  *total_ms = 0.0;
  *n_records = 0;
  if (ctx->prof_ev.empty()) return fail(IM_ERR_STATE, "profiling not active");
  cudaError_t rc = cudaDeviceSynchronize();
  for (size_t i = 0; i + 1 < ctx->prof_used && rc == cudaSuccess; i += 2) {
    float ms = 0.f;
    rc = cudaEventElapsedTime(&ms, ctx->prof_ev[i], ctx->prof_ev[i + 1]);
    *total_ms += ms;
    *n_records += 1;
  }
  for (auto& e : ctx->prof_ev) cudaEventDestroy(e);
  ctx->prof_ev.clear();
  ctx->prof_used = 0;
  if (rc != cudaSuccess) return fail(IM_ERR_CUDA, "im_profile_end: %s", cudaGetErrorString(rc));
  return IM_OK;
}

static size_t weight_bytes(const ImDims& p, int which) {
  switch (which) {
    case IM_W_UQ: return (size_t)p.HI * p.dI * p.D * 2;
    case IM_W_UK: return (size_t)p.dI * p.D * 2;
    case IM_W_G: return (size_t)p.HI * p.D * 2;
    case IM_W_THETA: return (size_t)p.dM * p.D * 2;
    case IM_W_WG: return (size_t)p.D * 2;
    case IM_W_BG: return 4;
    default: return 0;
  }
}
static void* weight_ptr(const ImWeights& w, int which) {
  switch (which) {
    case IM_W_UQ: return w.Uq;
    case IM_W_UK: return w.Uk;
    case IM_W_G: return w.G;
    case IM_W_THETA: return w.Wt;
    case IM_W_WG: return w.wg;
    case IM_W_BG: return w.bg;
    default: return nullptr;
  }
}

int im_set_weights(im_ctx* ctx, int layer, int which, const void* host_buf, size_t bytes) {
  if (!ctx || !host_buf) return fail(IM_ERR_ARG, "null argument");
  if (layer < 0 || layer >= ctx->p.L) return fail(IM_ERR_ARG, "layer out of range");
  size_t want = weight_bytes(ctx->p, which);
  if (want == 0 || want != bytes) return fail(IM_ERR_ARG, "weight %d: expected %zu bytes, got %zu", which, want, bytes);
  ctx->tail_is_merge = false;
  CK(cudaDeviceSynchronize());
  CK(cudaMemcpy(weight_ptr(ctx->lo.w[layer], which), host_buf, bytes, cudaMemcpyHostToDevice));
  if (which == IM_W_THETA) {
    CKL(im_launch_fold_theta(ctx->p, ctx->lo.w[layer], 0));
    CK(cudaDeviceSynchronize());
  }
  return IM_OK;
}

int im_get_weights(im_ctx* ctx, int layer, int which, void* host_buf, size_t bytes) {
  if (!ctx || !host_buf) return fail(IM_ERR_ARG, "null argument");
  if (layer < 0 || layer >= ctx->p.L) return fail(IM_ERR_ARG, "layer out of range");
  size_t want = weight_bytes(ctx->p, which);
  if (want == 0 || want != bytes) return fail(IM_ERR_ARG, "weight %d: expected %zu bytes, got %zu", which, want, bytes);
  CK(cudaDeviceSynchronize());
  CK(cudaMemcpy(host_buf, weight_ptr(ctx->lo.w[layer], which), bytes, cudaMemcpyDeviceToHost));
  return IM_OK;
}

int im_state_export(im_ctx* ctx, int layer, int seq, int which, void* host_buf, size_t bytes) {
  if (!ctx || !host_buf) return fail(IM_ERR_ARG, "null argument");
  const ImDims& p = ctx->p;
  if (layer < 0 || layer >= p.L || seq < 0 || seq >= p.S) return fail(IM_ERR_ARG, "layer/seq out of range");
  ctx->tail_is_merge = false;
  CK(cudaDeviceSynchronize());
  const size_t u = (size_t)layer * p.S + seq;
  const ImState& st = ctx->lo.st;
  int32_t ctr[CTR_STRIDE];
  CK(cudaMemcpy(ctr, st.ctr + u * CTR_STRIDE, sizeof(ctr), cudaMemcpyDeviceToHost));
  const int n = ctr[CTR_N];
  if (n < 0 || n > p.cap) return fail(IM_ERR_STATE, "device entry count %d outside [0,%d]", n, p.cap);
  auto need = [&](size_t want) -> int {
    if (bytes < want) return fail(IM_ERR_ARG, "state %d: buffer of %zu bytes, need %zu", which, bytes, want);
    return IM_OK;
  };
  int rc;
  if (p.scorer && which != IM_S_COUNTS && which != IM_S_M && which != IM_S_B)
    return fail(IM_ERR_ARG, "state piece %d is kept per KV head in this configuration: use im_state_export_head", which);
  switch (which) {
    case IM_S_COUNTS:
      if ((rc = need(sizeof(ctr)))) return rc;
      memcpy(host_buf, ctr, sizeof(ctr));
      return IM_OK;
    case IM_S_POS:
      if ((rc = need((size_t)n * 4))) return rc;
      CK(cudaMemcpy(host_buf, st.pos + u * p.cap, (size_t)n * 4, cudaMemcpyDeviceToHost));
      return IM_OK;
    case IM_S_IMP:
      if ((rc = need((size_t)n * 4))) return rc;
      CK(cudaMemcpy(host_buf, st.imp + u * p.cap, (size_t)n * 4, cudaMemcpyDeviceToHost));
      return IM_OK;
    case IM_S_KIDX:
      if ((rc = need((size_t)n * p.dI * 2))) return rc;
      CK(cudaMemcpy(host_buf, st.kidx + u * p.cap * p.dI, (size_t)n * p.dI * 2, cudaMemcpyDeviceToHost));
      return IM_OK;
    case IM_S_K:
    case IM_S_V: {
      if ((rc = need((size_t)n * p.Dkv * 2))) return rc;
      const bf16* src = (which == IM_S_K ? st.Kc : st.Vc) + u * p.Hkv * p.cap * p.d;
      // device layout [Hkv][cap][d] -> host layout [n][Hkv][d]
      for (int h = 0; h < p.Hkv; ++h)
        CK(cudaMemcpy2D((char*)host_buf + (size_t)h * p.d * 2, (size_t)p.Dkv * 2, src + (size_t)h * p.cap * p.d,
                        (size_t)p.d * 2, (size_t)p.d * 2, n, cudaMemcpyDeviceToHost));
      return IM_OK;
    }
    case IM_S_M: {
      const size_t cnt = (size_t)p.dM * p.Dkv;
      if ((rc = need(cnt * 4))) return rc;
      std::vector<float> M(cnt), phi((size_t)p.F * p.dM), w(p.F);
      std::vector<uint16_t> pv((size_t)p.F * p.Dkv);
      float c = 1.f;
      CK(cudaMemcpy(M.data(), st.Mhat + u * cnt, cnt * 4, cudaMemcpyDeviceToHost));
      CK(cudaMemcpy(phi.data(), st.pend_phi + u * p.F * p.dM, phi.size() * 4, cudaMemcpyDeviceToHost));
      CK(cudaMemcpy(pv.data(), st.pend_v + u * p.F * p.Dkv, pv.size() * 2, cudaMemcpyDeviceToHost));
      CK(cudaMemcpy(w.data(), st.pend_w + u * p.F, w.size() * 4, cudaMemcpyDeviceToHost));
      CK(cudaMemcpy(&c, st.cscale + u, 4, cudaMemcpyDeviceToHost));
      const int np = ctr[CTR_NPEND];
      float* outp = (float*)host_buf;
      for (int m = 0; m < p.dM; ++m)
        for (int col = 0; col < p.Dkv; ++col) {
          double acc = M[(size_t)m * p.Dkv + col];
          for (int q = 0; q < np; ++q) {
            uint32_t bits = ((uint32_t)pv[(size_t)q * p.Dkv + col]) << 16;
            float vv;
            memcpy(&vv, &bits, 4);
            acc += (double)w[q] * (double)phi[(size_t)q * p.dM + m] * (double)vv;
          }
          outp[(size_t)m * p.Dkv + col] = (float)((double)c * acc);
        }
      return IM_OK;
    }
    case IM_S_B:
      if ((rc = need((size_t)p.dM * 4))) return rc;
      CK(cudaMemcpy(host_buf, st.bvec + u * p.dM, (size_t)p.dM * 4, cudaMemcpyDeviceToHost));
      return IM_OK;
    case IM_S_EVICTED: {
      const int ne = ctr[CTR_NEVICT];
      if (ne < 0 || ne > p.tail) return fail(IM_ERR_STATE, "device evicted count %d outside [0,%d]", ne, p.tail);
      if ((rc = need((size_t)ne * 4))) return rc;
      CK(cudaMemcpy(host_buf, st.ev_pos + u * p.tail, (size_t)ne * 4, cudaMemcpyDeviceToHost));
      std::sort((int32_t*)host_buf, (int32_t*)host_buf + ne);
      return IM_OK;
    }
    case IM_S_SEL_POS:
    case IM_S_SEL_IMP: {
      const int ns = ctr[CTR_NSEL];
      if (ns < 0 || ns > p.cap) return fail(IM_ERR_STATE, "device selection count %d outside [0,%d]", ns, p.cap);
      if ((rc = need((size_t)ns * 4))) return rc;
      const void* src = which == IM_S_SEL_POS ? (const void*)(st.sel_pos + u * p.cap) : (const void*)(st.sel_imp + u * p.cap);
      CK(cudaMemcpy(host_buf, src, (size_t)ns * 4, cudaMemcpyDeviceToHost));
      return IM_OK;
    }
    default:
      return fail(IM_ERR_ARG, "unknown state piece %d", which);
  }
}

int im_state_import(im_ctx* ctx, int layer, int seq, int which, const void* host_buf, size_t bytes) {
  if (!ctx || !host_buf) return fail(IM_ERR_ARG, "null argument");
  const ImDims& p = ctx->p;
  if (layer < 0 || layer >= p.L || seq < 0 || seq >= p.S) return fail(IM_ERR_ARG, "layer/seq out of range");
  CK(cudaDeviceSynchronize());
  const size_t u = (size_t)layer * p.S + seq;
  const ImState& st = ctx->lo.st;
  HostUnit& hu = ctx->hu[u];
  auto exact = [&](size_t want) -> int {
    if (bytes != want) return fail(IM_ERR_ARG, "state %d: got %zu bytes, expected %zu", which, bytes, want);
    return IM_OK;
  };
  int rc;
  const int n = hu.n;
  if (p.scorer && which != IM_S_COUNTS && which != IM_S_M && which != IM_S_B)
    return fail(IM_ERR_ARG, "state piece %d is kept per KV head in this configuration: use im_state_import_head", which);
  switch (which) {
    case IM_S_COUNTS: {
      if ((rc = exact(CTR_STRIDE * 4))) return rc;
      int32_t ctr[CTR_STRIDE];
      memcpy(ctr, host_buf, sizeof(ctr));
      if (ctr[CTR_N] < 0 || ctr[CTR_N] > p.cap || ctr[CTR_SINCE] < 0 || ctr[CTR_SINCE] >= p.tau || ctr[CTR_T] < ctr[CTR_N])
        return fail(IM_ERR_ARG, "inconsistent counters");
      ctr[CTR_NPEND] = 0;  // pending writes cannot be imported; IM_S_M carries the folded state
      ctr[CTR_NEVICT] = 0;
      ctr[CTR_NNEXT] = ctr[CTR_N];
      ctr[CTR_NSEL] = 0;
      int32_t old[CTR_STRIDE];
      CK(cudaMemcpy(old, st.ctr + u * CTR_STRIDE, sizeof(old), cudaMemcpyDeviceToHost));
      if (old[CTR_NPEND] != 0) return fail(IM_ERR_STATE, "import IM_S_M before IM_S_COUNTS when writes are pending");
      CK(cudaMemcpy(st.ctr + u * CTR_STRIDE, ctr, sizeof(ctr), cudaMemcpyHostToDevice));
      hu.n = ctr[CTR_N];
      hu.T = ctr[CTR_T];
      hu.since = ctr[CTR_SINCE];
      return IM_OK;
    }
    case IM_S_POS:
      if ((rc = exact((size_t)n * 4))) return rc;
      CK(cudaMemcpy(st.pos + u * p.cap, host_buf, bytes, cudaMemcpyHostToDevice));
      return IM_OK;
    case IM_S_IMP:
      if ((rc = exact((size_t)n * 4))) return rc;
      CK(cudaMemcpy(st.imp + u * p.cap, host_buf, bytes, cudaMemcpyHostToDevice));
      return IM_OK;
    case IM_S_KIDX:
      if ((rc = exact((size_t)n * p.dI * 2))) return rc;
      CK(cudaMemcpy(st.kidx + u * p.cap * p.dI, host_buf, bytes, cudaMemcpyHostToDevice));
      return IM_OK;
    case IM_S_K:
    case IM_S_V: {
      if ((rc = exact((size_t)n * p.Dkv * 2))) return rc;
      bf16* dst = (which == IM_S_K ? st.Kc : st.Vc) + u * p.Hkv * p.cap * p.d;
      for (int h = 0; h < p.Hkv; ++h)
        CK(cudaMemcpy2D(dst + (size_t)h * p.cap * p.d, (size_t)p.d * 2, (const char*)host_buf + (size_t)h * p.d * 2,
                        (size_t)p.Dkv * 2, (size_t)p.d * 2, n, cudaMemcpyHostToDevice));
      return IM_OK;
    }
    case IM_S_M: {
      if ((rc = exact((size_t)p.dM * p.Dkv * 4))) return rc;
      CK(cudaMemcpy(st.Mhat + u * p.dM * p.Dkv, host_buf, bytes, cudaMemcpyHostToDevice));
      const float one = 1.f;
      const int32_t zero = 0;
      CK(cudaMemcpy(st.cscale + u, &one, 4, cudaMemcpyHostToDevice));
      CK(cudaMemcpy(st.ctr + u * CTR_STRIDE + CTR_NPEND, &zero, 4, cudaMemcpyHostToDevice));
      return IM_OK;
    }
    case IM_S_B:
      if ((rc = exact((size_t)p.dM * 4))) return rc;
      CK(cudaMemcpy(st.bvec + u * p.dM, host_buf, bytes, cudaMemcpyHostToDevice));
      return IM_OK;
    default:
      return fail(IM_ERR_ARG, "state piece %d cannot be imported", which);
  }
}

int im_set_scores(im_ctx* ctx, int layer, int n_seq, const float* scores, int64_t n_positions) {
  if (!ctx) return fail(IM_ERR_ARG, "null context");
  const ImDims& p = ctx->p;
  if (p.scorer != 2) return fail(IM_ERR_ARG, "im_set_scores needs scorer = 2 in the configuration");
  if (layer < 0 || layer >= p.L) return fail(IM_ERR_ARG, "layer %d out of range [0,%d)", layer, p.L);
  if (!scores || n_seq < 1 || n_seq > p.S || n_positions < 1) return fail(IM_ERR_ARG, "bad scores");
  ctx->ext[layer].ptr = scores;
  ctx->ext[layer].n_pos = n_positions;
  ctx->ext[layer].n_seq = n_seq;
  return IM_OK;
}

static int head_piece(im_ctx* ctx, int layer, int seq, int head, int which, void* host_buf, size_t bytes, bool import) {
  if (!ctx || !host_buf) return fail(IM_ERR_ARG, "null argument");
  const ImDims& p = ctx->p;
  if (!p.scorer) return fail(IM_ERR_ARG, "per-head state pieces need scorer = 1 or 2 in the configuration");
  if (layer < 0 || layer >= p.L || seq < 0 || seq >= p.S || head < 0 || head >= p.Hkv) return fail(IM_ERR_ARG, "layer/seq/head out of range");
  ctx->tail_is_merge = false;
  CK(cudaDeviceSynchronize());
  const size_t u = (size_t)layer * p.S + seq;
  const ImState& st = ctx->lo.st;
  int32_t ctr[CTR_STRIDE];
  CK(cudaMemcpy(ctr, st.ctr + u * CTR_STRIDE, sizeof(ctr), cudaMemcpyDeviceToHost));
  const int n = import ? ctx->hu[u].n : ctr[CTR_N];
  if (n < 0 || n > p.cap) return fail(IM_ERR_STATE, "entry count %d outside [0,%d]", n, p.cap);
  const size_t row = (u * p.Hkv + head) * (size_t)p.cap, erow = (u * p.Hkv + head) * (size_t)p.tail;
  void* dev = nullptr;
  size_t want = 0;
  switch (which) {
    case IM_S_POS: dev = st.hpos + row; want = (size_t)n * 4; break;
    case IM_S_IMP: dev = st.hscore + row; want = (size_t)n * 4; break;
    case IM_S_K: dev = st.Kc + row * p.d; want = (size_t)n * p.d * 2; break;
    case IM_S_V: dev = st.Vc + row * p.d; want = (size_t)n * p.d * 2; break;
    case IM_S_EVICTED: {
      if (import) return fail(IM_ERR_ARG, "state piece %d cannot be imported", which);
      const int ne = ctr[CTR_NEVICT];
      if (ne < 0 || ne > p.tail) return fail(IM_ERR_STATE, "device evicted count %d outside [0,%d]", ne, p.tail);
      dev = st.hev_pos + erow;
      want = (size_t)ne * 4;
      break;
    }
    case IM_S_SEL_POS:
    case IM_S_SEL_IMP: {
      if (import) return fail(IM_ERR_ARG, "state piece %d cannot be imported", which);
      const int ns = ctr[CTR_NSEL];
      if (ns < 0 || ns > p.cap) return fail(IM_ERR_STATE, "device selection count %d outside [0,%d]", ns, p.cap);
      dev = which == IM_S_SEL_POS ? (void*)(st.hsel_pos + row) : (void*)(st.hsel_score + row);
      want = (size_t)ns * 4;
      break;
    }
    default: return fail(IM_ERR_ARG, "state piece %d has no per-head form", which);
  }
  if (import ? bytes != want : bytes < want) return fail(IM_ERR_ARG, "state %d: buffer of %zu bytes, need %zu", which, bytes, want);
  if (import) CK(cudaMemcpy(dev, host_buf, want, cudaMemcpyHostToDevice));
  else CK(cudaMemcpy(host_buf, dev, want, cudaMemcpyDeviceToHost));
  if (!import && which == IM_S_EVICTED) std::sort((int32_t*)host_buf, (int32_t*)host_buf + want / 4);
  return IM_OK;
}
int im_state_export_head(im_ctx* ctx, int layer, int seq, int head, int which, void* host_buf, size_t bytes) {
  return head_piece(ctx, layer, seq, head, which, host_buf, bytes, false);
}
int im_state_import_head(im_ctx* ctx, int layer, int seq, int head, int which, const void* host_buf, size_t bytes) {
  return head_piece(ctx, layer, seq, head, which, const_cast<void*>(host_buf), bytes, true);
}

int im_topb_select(const float* scores, const int32_t* pos, int rows, int n, int budget, int n_sink, uint8_t* keep,
                   int32_t* n_evict, void* cuda_stream) {
  if (!scores || !pos || !keep || !n_evict) return fail(IM_ERR_ARG, "null tensor");
  if (rows < 0 || n < 0 || budget < 0 || n_sink < 0) return fail(IM_ERR_ARG, "negative size");
  if (rows == 0) return IM_OK;
  CKL(im_launch_topb(scores, pos, rows, n, budget, n_sink, keep, n_evict, (cudaStream_t)cuda_stream));
  return IM_OK;
}

int im_event_count(im_ctx* ctx, int counter, int64_t* value) {
  if (!ctx || !value) return fail(IM_ERR_ARG, "null argument");
  if (counter != IM_COUNT_MERGE_RECOMPUTE) return fail(IM_ERR_ARG, "unknown counter %d", counter);
  CK(cudaDeviceSynchronize());
  int32_t v = 0;
  CK(cudaMemcpy(&v, ctx->lo.st.status + 1, 4, cudaMemcpyDeviceToHost));
  *value = v;
  return IM_OK;
}

int im_status(im_ctx* ctx, void* cuda_stream, int32_t* device_status) {
  if (!ctx || !device_status) return fail(IM_ERR_ARG, "null argument");
  CK(join_late(ctx, (cudaStream_t)cuda_stream));
  CK(cudaStreamSynchronize((cudaStream_t)cuda_stream));
  CK(cudaMemcpy(device_status, ctx->lo.st.status, 4, cudaMemcpyDeviceToHost));
  if (*device_status & ST_TIMEOUT) return fail(IM_ERR_TIMEOUT, "a bounded device wait gave up (status %d)", *device_status);
  if (*device_status)
    return fail(IM_ERR_STATE, "device status %d (1: non-finite score, 2: count mismatch, 8: a layer that reuses another layer's scores holds other positions than that layer)",
                *device_status);
  return IM_OK;
}

}  // extern "C"

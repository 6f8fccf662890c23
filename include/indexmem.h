/*
 * indexmem.h — C ABI of the IndexMem per-layer decode / chunked-prefill hot path for NVIDIA B200.
 *
 * The library keeps, for every (layer, sequence) pair, a budgeted KV cache, the indexer key cache,
 * the pooled importance scores and the latent memory state (M, b), and advances them with two hot
 * calls: im_prefill_chunk and im_decode_step.  Symbols follow the paper: H query heads, H_kv KV
 * heads, d = d_head, D = d_model = H*d, D_kv = H_kv*d, G_q = H/H_kv, H_I = H_index, d_I = d_index,
 * d_M = d_mem, B = KV budget B_max, tau = compression interval.
 *
 * Conventions for every entry point
 *   - "dev" pointers are device (HBM) addresses owned by the caller; "host" pointers are ordinary
 *     host memory.  Tensors are dense, row-major, innermost dimension last, 16-byte aligned.
 *   - bf16 means the 16-bit brain-float bit pattern (upper half of an IEEE float32).
 *   - The two hot calls only enqueue kernels on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and return without synchronising; they allocate nothing.  All calls
 *     on one context must be issued in stream order on one stream at a time.  A prefill call may leave the last
 *     part of its work (everything behind the kernel that appends the chunk, or the state update of its memory
 *     write alone: IM_OPT_PREFILL_PIPELINE) running on streams of the context's own when it
 *     returns; every later call on the context orders itself behind that work, and im_destroy synchronises the
 *     device, so the caller sees no difference as long as the workspace is touched through this interface only
 *     (under stream capture nothing is left running: a capture has to end with every stream rejoined).
 *   - Return value: IM_OK (0) or a negative im_error.  No exception, abort or device trap crosses the
 *     boundary.  im_last_error() describes the most recent failure on the calling thread.  Problems
 *     that only the device can see (for example a non-finite score) set a sticky device status word
 *     that im_status() reads back.
 *   - There is no CPU fallback: without a CUDA device every call that needs one fails with
 *     IM_ERR_CUDA.
 */
#ifndef INDEXMEM_H_
#define INDEXMEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct im_ctx im_ctx; /* opaque host object; device state lives in the caller's workspace */

typedef enum im_error {
  IM_OK = 0,
  IM_ERR_ARG = -1,      /* invalid argument or configuration                                  */
  IM_ERR_CAPACITY = -2, /* a sequence would exceed its slot capacity, or workspace too small  */
  IM_ERR_STATE = -3,    /* device status word is set (non-finite score, inconsistent count)   */
  IM_ERR_CUDA = -4,     /* a CUDA runtime/driver call failed                                   */
  IM_ERR_TIMEOUT = -5   /* a bounded device-side wait gave up                                  */
} im_error;

/* Hyper-parameters of the method.  Zero in a field marked "0 =>" selects the paper's value. */
typedef struct im_config {
  int32_t n_layers;          /* independent layers held by the context                              */
  int32_t max_seqs;          /* sequence states per layer                                           */
  int32_t n_q_heads;         /* H                                              (App. Notation)      */
  int32_t n_kv_heads;        /* H_kv, divides H                                (App. Notation)      */
  int32_t head_dim;          /* d, a multiple of 16, <= 256                    (App. Notation)      */
  int32_t n_index_heads;     /* H_I ; 0 => max(1, H/4)                         (Sec. 4, hyperparameters) */
  int32_t index_dim;         /* d_I ; 0 => max(1, d/8); <= 64                  (Sec. 4, hyperparameters) */
  int32_t mem_dim;           /* d_M ; 0 => max(1, D/8)                         (Sec. 4, hyperparameters) */
  int32_t budget;            /* B: entries kept by a compression, sinks included (Sec. 4, schedule) */
  int32_t compress_interval; /* tau >= 1: decode tokens between compressions   (Sec. 4, schedule)   */
  int32_t max_chunk;         /* longest prefill chunk; slot capacity is B + max(tau, max_chunk)     */
  int32_t n_sink;            /* first tokens that are never evicted; < B       (Sec. 4, setup)      */
  int32_t act;               /* indexer activation: 0 ReLU, 1 identity         (Sec. 3.1, z = act(q.k)) */
  int32_t enable_memory;     /* 0: no memory write and no readout term         (Eq. 4 with g = 0)   */
  int32_t out_f32;           /* 0: `out` of im_decode_step is bf16; 1: float32                       */
  int32_t pending_slots;     /* rank-one writes folded lazily into M (0 => 32); see im_decode_step  */
  int32_t chunk_outputs;     /* 1: reserve workspace for im_prefill_chunk_attend (max_seqs * max_chunk * D_kv floats) */
  int32_t score_share;       /* g >= 2: layers l with l % g != 0 reuse the indexer scores of layer l - l % g (App. B,
                                IndexCache-style reuse; the paper uses 4); 0 or 1: every layer scores for itself      */
  int32_t scorer;            /* 0: the learnable indexer, one score row per sequence (Sec. 3.1).  A retained set per KV head
                                (Sec. 2.2, S in R^{B x H_kv x L}): 1 Knorm, S_t = ||K_t||_2 (Sec. 2.2); 2 scores handed in
                                by the caller with im_set_scores (Sec. 5 ablation: the memory on another eviction policy) */
  float softmax_scale;       /* 0 => 1/sqrt(d)                                 (Sec. 2.1)           */
  float lambda;              /* decay of Eq. 6-7, (0,1]; 0 => 1                                      */
  float eta;                 /* write strength of Eq. 6-7, > 0; 0 => 1                               */
  float eps;                 /* epsilon of Eq. 5; 0 => 1e-6                                          */
  float norm_eps;            /* epsilon of the indexer RMSNorm; 0 => 1e-6     (Sec. 3.1)            */
  float init_std;            /* std of the seeded weight init; 0 => 0.02                             */
  uint64_t seed;             /* seed of the weight init done by im_create                            */
} im_config;

/* Weight tensors of one layer (Sec. 3.1 and 3.2), all bf16 except IM_W_BG (one float32). */
typedef enum im_weight {
  IM_W_UQ = 0,    /* U_q      [H_I*d_I, D]   indexer query down-projection           */
  IM_W_UK = 1,    /* U_k      [d_I, D]       indexer key projection                  */
  IM_W_G = 2,     /* G        [H_I, D]       head gate                               */
  IM_W_THETA = 3, /* Linear_theta [d_M, D]   memory feature map phi                  */
  IM_W_WG = 4,    /* w_g      [D]            weight of the scalar readout gate g(q)  */
  IM_W_BG = 5     /* b_g      [1] float32    bias of g(q)                            */
} im_weight;

/* Per-(layer, sequence) state pieces for im_state_export / im_state_import. */
typedef enum im_state {
  IM_S_COUNTS = 0, /* int32[8]: n entries, tokens seen T, since, evict steps, n evicted by last compression, pending writes, 0, n_sel */
  IM_S_POS = 1,    /* int32[n]          original position of the entry in each slot                   */
  IM_S_IMP = 2,    /* float32[n]        pooled importance since the last compression (-inf = unscored) */
  IM_S_KIDX = 3,   /* bf16[n, d_I]      cached indexer keys                                            */
  IM_S_K = 4,      /* bf16[n, H_kv, d]  cached keys                                                    */
  IM_S_V = 5,      /* bf16[n, H_kv, d]  cached values                                                  */
  IM_S_M = 6,      /* float32[d_M, D_kv] latent state in KV space (export folds pending writes and decay in) */
  IM_S_B = 7,      /* float32[d_M]      stabiliser vector b                                            */
  IM_S_EVICTED = 8, /* int32[n_evicted] positions evicted by the last compression, ascending (export only) */
  IM_S_SEL_POS = 9, /* int32[n_sel]     positions of the entries the last compression chose among (export only) */
  IM_S_SEL_IMP = 10 /* float32[n_sel]   their pooled importance at that moment, same order (export only)        */
} im_state;

/* Bytes of device workspace im_create needs for `cfg`; 0 if the configuration is invalid. */
size_t im_workspace_bytes(const im_config* cfg);

/*
 * Creates a context over `dev_workspace` (device memory of at least im_workspace_bytes(cfg) bytes,
 * 256-byte aligned, owned by the caller, must outlive the context and the current CUDA device must
 * be the one that owns it).  Zeroes the state, draws seeded N(0, init_std^2) bf16 weights for every
 * layer (b_g = 0) and synchronises the device once.  On success *out receives the context.
 */
int im_create(const im_config* cfg, void* dev_workspace, size_t workspace_bytes, im_ctx** out);

/* Releases the host object.  The workspace stays with the caller.  Synchronises the device. */
int im_destroy(im_ctx* ctx);

/* Clears the state of one sequence in one layer (layer = -1: all layers; seq = -1: all sequences); with both -1 also the
 * sticky device status word that im_status reports.  Enqueued on the stream. */
int im_reset(im_ctx* ctx, int layer, int seq, void* cuda_stream);

/*
 * Chunked prefill of one layer for n_seq sequences (Sec. 4 schedule: ingest, score with every query
 * of the chunk, compress to the budget, write the evicted pairs to memory; Sec. 3.1; Eq. 6-7).
 *   seq_ids  host int32[n_seq], distinct, each in [0, max_seqs)
 *   chunk_len C, 1 <= C <= max_chunk; the same for all sequences of the call
 *   x        dev bf16 [n_seq, C, D]       hidden states X
 *   q_pre    dev bf16 [n_seq, C, H, d]    pre-RoPE queries Q (indexer input)
 *   k, v     dev bf16 [n_seq, C, H_kv, d] keys / values to cache
 * Appends the C tokens, pools A_{s,t} (Sec. 3.1) over the chunk's queries under the causal mask into
 * the importance of every cached entry, then compresses: if more than B entries are cached the B
 * best (importance descending, position ascending, sinks first) stay, the rest are written to the
 * latent memory (Eq. 6-7, one evict step) and the cache is compacted.  Attention outputs for the
 * chunk's own queries are not produced (see im_prefill_chunk_attend).
 * Errors: IM_ERR_ARG (bad ids, sizes, null pointers), IM_ERR_CAPACITY (n + C > capacity).
 */
int im_prefill_chunk(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, int chunk_len,
                     const void* x, const void* q_pre, const void* k, const void* v, void* cuda_stream);

/*
 * im_prefill_chunk that also returns the layer outputs of the chunk's own queries (Eq. 4-5 during chunked
 * prefill; the chunk is processed before it is compressed, Sec. 4 schedule).
 *   q    dev bf16 [n_seq, C, H, d]  queries as the attention sees them (may alias q_pre)
 *   out  dev [n_seq, C, H, d] bf16 (float32 when out_f32 = 1)
 * Query s of the chunk attends to every entry cached when the call starts and to the chunk's tokens up to
 * and including itself (Sec. 2.1, causal), and adds g(q_s) m(q_s) read from the memory as the evict steps of
 * earlier calls left it (Eq. 5); the evict step of this chunk does not enter its own outputs.  The state
 * after the call is the one im_prefill_chunk leaves.
 * Needs chunk_outputs = 1 in the configuration (workspace) and head_dim 64 or 128 with at most 8 query heads
 * per KV head; otherwise IM_ERR_ARG.  Other errors as for im_prefill_chunk; IM_ERR_TIMEOUT is reported through
 * im_status if a bounded wait on a tile copy gave up.
 */
int im_prefill_chunk_attend(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, int chunk_len,
                            const void* x, const void* q_pre, const void* q, const void* k, const void* v,
                            void* out, void* cuda_stream);

/*
 * One decode token per sequence for one layer (Sec. 4 schedule, decode side; Eq. 4-7).
 *   x      dev bf16 [n_seq, D]        hidden state of the new token
 *   q_pre  dev bf16 [n_seq, H, d]     pre-RoPE query (indexer input); may alias q
 *   q      dev bf16 [n_seq, H, d]     attention query; also the input of Linear_theta and g
 *   k_new, v_new dev bf16 [n_seq, H_kv, d]
 *   out    dev [n_seq, H, d] bf16 (float32 when out_f32 = 1): o = o_attn + g(q) m(q)   (Eq. 4)
 * Steps: append the token; score every cached entry with the new query and pool by max into its
 * importance; every tau-th token of a sequence compress to the budget as in im_prefill_chunk; then
 * attention over the retained entries plus the gated memory readout (Eq. 5).  The evict step happens
 * before the attention of the same call.
 * A compression that evicts at most `pending_slots` entries keeps them as rank-one terms next to M
 * and the readout adds them exactly; they are folded into M when the list fills.  This is Eq. 6-7
 * re-associated, not an approximation.
 * CUDA graphs: the kernels of a call take entry counts, positions and pending writes from device memory, so a
 * captured call can be replayed on later tokens; which kernels a call launches, however, is decided on the host
 * (compression due or not, evicted set small or large).  With tau = 1 every call is alike and one captured
 * step replays indefinitely (from the moment every sequence holds B entries); with tau > 1 capture one graph
 * per phase of the interval or call eagerly.  A replay in the wrong phase leaves the cache uncompressed and is
 * reported through im_status (count mismatch) once a sequence runs out of slots.
 * Errors: IM_ERR_ARG, IM_ERR_CAPACITY (a sequence has no free slot).
 */
int im_decode_step(im_ctx* ctx, int layer, int n_seq, const int32_t* seq_ids, const void* x,
                   const void* q_pre, const void* q, const void* k_new, const void* v_new, void* out,
                   void* cuda_stream);

/*
 * One decode token per sequence for several layers in one call: the same computation, layer by layer, as
 * im_decode_step(layers[j], ..., x[j], q_pre[j], q[j], k_new[j], v_new[j], out[j]) for j = 0 .. n_layers - 1 (Sec. 4
 * schedule, decode side; Eq. 4-7), for callers that hold the inputs of all those layers when they make the call: a
 * stack of per-layer states driven from recorded or synthetic activations, layers of independent models that share a
 * context.  Inside a transformer the query of layer l + 1 depends on the output of layer l, and the layers are then
 * called one by one with im_decode_step.
 *   layers           host int32 [n_layers], distinct
 *   x, q_pre, q, k_new, v_new, out   host arrays of n_layers device pointers, shapes as for im_decode_step
 * No input of the call may be written by the call (no out[j] overlaps an input of any layer): the layers overlap in
 * time.  The (layer, sequence) states of different layers are independent, so the call keeps several layers in
 * flight: the attention kernels of consecutive layers follow one another without a gap on one internal stream, the
 * readout kernels on a second one, and each layer's projections, front kernel, phi of the evicted keys and merge
 * run on the streams of one of three lanes with a scratch set per lane, next to the streams of the layers ahead of
 * it.  All internal streams fork from `cuda_stream` when the call starts and join it when it ends: every output is
 * complete in stream order after the call, and the call can be captured into a CUDA graph like im_decode_step.
 * The streaming kernels are kept to a fixed subset of the SMs by SM id (a block that finds itself on an SM set
 * aside for the small kernels hands its work to a block that is still to come), since with layers overlapping the
 * occupancy rules that make this split in im_decode_step no longer hold.  phi(q)^T Mhat is formed by the bulk-copy
 * readout kernel where it serves the shape (see IM_OPT_READOUT_STAGES).
 * The pipelined schedule needs every layer of the call to qualify for im_decode_step's concurrent schedule with
 * SMs set aside (at most n_SM / 4 sequences, evicted sets of at most min(16, pending_slots) entries, budgets of at
 * most 6144 entries, the indexer as scorer, no score reuse, memory enabled); otherwise, and with
 * IM_OPT_STACK_PIPELINE = 0, the layers are simply called in order.  Results are those of im_decode_step either way.
 * Errors: as for im_decode_step; IM_ERR_ARG also for a repeated layer or a null entry.
 */
int im_decode_stack(im_ctx* ctx, int n_layers, const int32_t* layers, int n_seq, const int32_t* seq_ids,
                    const void* const* x, const void* const* q_pre, const void* const* q, const void* const* k_new,
                    const void* const* v_new, void* const* out, void* cuda_stream);

/*
 * im_decode_stack for a caller whose per-layer inputs arrive, and whose per-layer outputs leave, while the call runs
 * (copies from and to host memory on streams of the caller's, say): the same computation (Sec. 4 schedule, decode side;
 * Eq. 4-7) with one event per layer on either side.
 *   ready_events     host array of n_layers CUDA events (cudaEvent_t), or NULL; entries may be NULL.  The inputs of
 *                    layers[j] (x[j], q_pre[j], q[j], k_new[j], v_new[j]) need only be complete once ready_events[j] has
 *                    occurred: no kernel of the call reads them before.  The caller has recorded the event before
 *                    the call (with a NULL entry, or a NULL array, the inputs are complete in `cuda_stream` order when
 *                    the call is made, as for im_decode_stack).
 *   done_events      host array of n_layers CUDA events, or NULL; entries may be NULL.  The call records
 *                    done_events[j] on an internal stream once out[j] is complete; a stream of the caller's that waits
 *                    for it may read out[j] while later layers of the call still run.
 * The events are the caller's (created, and destroyed after the work has ended, by the caller).  Under stream
 * capture the ready events must have been recorded on streams of the same capture, and the streams that wait for the
 * done events must be joined back into the capturing stream by the caller.  Everything else as for im_decode_stack,
 * which is this call with both arrays NULL.
 */
int im_decode_stack_events(im_ctx* ctx, int n_layers, const int32_t* layers, int n_seq, const int32_t* seq_ids,
                           const void* const* x, const void* const* q_pre, const void* const* q, const void* const* k_new,
                           const void* const* v_new, void* const* out, void* const* ready_events,
                           void* const* done_events, void* cuda_stream);

/* Copies one weight tensor of a layer from / to host memory (bytes must equal the tensor size). Synchronous. */
int im_set_weights(im_ctx* ctx, int layer, int which, const void* host_buf, size_t bytes);
int im_get_weights(im_ctx* ctx, int layer, int which, void* host_buf, size_t bytes);

/*
 * Copies one piece of a sequence's state to / from host memory.  Synchronous (device-wide).
 * Export: `bytes` is the buffer capacity; the piece is sized by the current entry count n.
 * Import: IM_S_COUNTS first fixes n, then the other pieces must have exactly the matching size;
 * importing IM_S_M replaces the latent state (pending writes are dropped, decay scale reset).
 * Slot order is free: entries are identified by their position.
 */
int im_state_export(im_ctx* ctx, int layer, int seq, int which, void* host_buf, size_t bytes);
int im_state_import(im_ctx* ctx, int layer, int seq, int which, const void* host_buf, size_t bytes);

/*
 * Row-generic budgeted selection (Sec. 2.2: I = TopK(S, L')), usable without a context.
 *   scores dev float32 [rows, n], pos dev int32 [rows, n] (distinct within a row)
 *   keep   dev uint8  [rows, n]  receives 1 for the min(B, n) retained entries of each row
 *   n_evict dev int32 [rows]     receives n - min(B, n)
 * Order: key descending, position ascending, where key = +inf for pos < n_sink and -0.0 == +0.0.
 * Bit-exact and deterministic.  Scores must not be NaN.
 */
int im_topb_select(const float* scores, const int32_t* pos, int rows, int n, int budget, int n_sink,
                   uint8_t* keep, int32_t* n_evict, void* cuda_stream);

/* Synchronises the stream and returns the sticky device status word (0 = clean) in *device_status. */
int im_status(im_ctx* ctx, void* cuda_stream, int32_t* device_status);

/*
 * Measurement hook (no counterpart in the paper): between im_profile_begin and im_profile_end every
 * im_decode_step records a pair of CUDA events on its stream around the attention + readout kernel
 * (the kernel that streams the retained K/V and M).  im_profile_end synchronises, returns the summed
 * device time of the recorded launches in *total_ms and their number in *n_records, and releases the
 * events.  At most max_records launches are recorded.  Must not be used while the stream is being
 * captured into a CUDA graph.
 */
int im_profile_begin(im_ctx* ctx, int max_records);
int im_profile_end(im_ctx* ctx, double* total_ms, int64_t* n_records);

/*
 * Execution options (no counterpart in the paper).  Results are identical for every setting unless stated.
 *   IM_OPT_CONCURRENCY   1 (default where the streaming attention kernel is available): im_decode_step
 *                        starts the attention kernel at once over the entries cached before the call and
 *                        runs the rest of the call (projections, append / score / select, memory write,
 *                        readout) next to it on four internal side streams that fork from and join back
 *                        into `cuda_stream` inside the call (events only, so the pattern can be captured
 *                        into a CUDA graph); the merge adds the new token and removes the evicted entries
 *                        from the softmax sums again, so the result is the attention over the retained set.
 *                        Behind another concurrent im_decode_step on the same stream the attention kernel is
 *                        launched as a programmatic dependent: it may request tiles of its own layer's cache
 *                        while that call's last kernel is still running, and waits for it before it reads `q`.
 *                        The prefill calls run the chunk's independent projections next to one another on the
 *                        same side streams, and im_prefill_chunk_attend forms the layer outputs (readout and
 *                        attention of the chunk's queries) next to the scoring, the selection and the memory
 *                        write of the chunk.  0: everything is enqueued on `cuda_stream` in order.
 *   IM_OPT_PREFETCH_NEXT 1 (default): while the attention kernel of layer l streams the K/V cache,
 *                        im_decode_step prefetches into L2 what the small latency-bound kernels of layer
 *                        (l + 1) mod n_layers will read for the same sequences (weights, indexer key cache,
 *                        counters, pending memory terms), and, once the attention kernel has ended, the first half
 *                        of that layer's memory matrices (HBM has little else to do while the merge kernel runs);
 *                        none of it depends on the output of layer l.
 *   IM_OPT_PREFILL_TENSOR 1 (default): the tcgen05 kernels of the prefill calls are used where they apply - the
 *                        indexer scoring of the chunk (Sec. 3.1, a dense [keys x d_I] x [d_I x queries * heads]
 *                        contraction; n_index_heads <= 8, index_dim 8 or 16; float32 features split into three
 *                        bf16 terms) and the chunk attention of im_prefill_chunk_attend (head_dim 128); 0: the
 *                        CUDA-core scoring kernel and the mma.sync attention kernel.  Both settings are within
 *                        the stated tolerances of a float32 evaluation; they need not agree to the last bit.
 *                        Setting 1 where neither kernel applies returns IM_ERR_ARG.
 *   IM_OPT_PROFILE_TARGET which kernel im_profile_begin / im_profile_end time: 0 (default) the attention
 *                        kernel of im_decode_step, 1 the scoring kernel of im_prefill_chunk.  Cannot be
 *                        changed while profiling is active (IM_ERR_STATE).
 *   IM_OPT_DECODE_TENSOR 1: the attention over the retained entries of im_decode_step (Sec. 2.1, Eq. 4) runs as the
 *                        warp-specialised tcgen05 kernel (head_dim 128, G_q <= 8: tiles of 128 keys on the M axis, the
 *                        G_q query heads on N, accumulators in tensor memory, K and V tiles through TMA rings of their
 *                        own); 0 (default): the mma.sync kernel with a TMA ring per warp, which also serves head_dim
 *                        64.  Both are within the stated tolerances of a float32 evaluation; they need not agree to
 *                        the last bit.  Setting 1 for a shape the tensor-core kernel does not take returns IM_ERR_ARG.
 *   IM_OPT_READOUT_STAGES k >= 1: in concurrent decode calls with SMs set aside for
 *                        the front kernel, phi(q)^T Mhat of Eq. 5 is formed by a persistent kernel that brings the rows of
 *                        Mhat in through a ring of k 32 KB bulk copies per CTA, one CTA beside each attention CTA
 *                        (k <= 6; D_kv a power of two of at most 1024 and d_M a multiple of 8192 / D_kv); 0 (default): by the
 *                        kernel built on plain loads, which serves every shape and schedule.  The two add the rows in different
 *                        orders (float32); both are within the stated tolerances.  While the option has not been set, a
 *                        pipelined im_decode_stack uses the bulk-copy kernel with two stages where it serves the shape
 *                        and im_decode_step the plain-load kernel; once set, the value holds for both.
 *   IM_OPT_LAYER_OVERLAP 1 (default): in the concurrent schedule the attention kernel of a decode call on ANOTHER layer than
 *                        the call before it on the same stream is launched as programmatic dependent of that call's last
 *                        kernel: it requests its first cache tiles while that kernel still runs and waits for it before it
 *                        touches anything else.  0: it is launched in plain stream order.
 *   IM_OPT_STACK_PIPELINE 1 (default): im_decode_stack overlaps the layers of a call where they qualify; 0: it calls
 *                        im_decode_step layer by layer.
 *   IM_OPT_STACK_RESERVED k >= 1: SMs that a pipelined im_decode_stack keeps free of streaming blocks, for the small
 *                        kernels of the layers in flight; 0 (default): one per sequence of the call, at most 24 with
 *                        the bulk-copy readout kernel and 8 with the plain-load one.
 *   IM_OPT_STACK_CHUNKS  k in [1, 16] (default 2): a pipelined im_decode_stack cuts the tiles of a layer's attention into k
 *                        runs per warp, which the warps take from a counter.  With k = 1 the runs, and with them the
 *                        order of every float32 sum, are those of im_decode_step: the two then agree bit for bit.
 *   IM_OPT_FOLD_TENSOR   1 (default): where d_M and D_kv are multiples of 64, the listed rank-one terms are folded into M on
 *                        the tensor cores (w_p phi_p as three bf16 terms, v_p as stored: exact products, float32 sums); 0:
 *                        by float32 multiply-adds in list order, as for every other shape.  The two differ by rounding
 *                        order only.
 *   IM_OPT_PREFILL_PIPELINE 1 (default): an im_prefill_chunk call whose every sequence evicts more than pending_slots entries
 *                        (tensor-core scoring, not under stream capture) returns with everything behind its append kernel
 *                        still running on a stream of the library's own, so that the next chunk's projections run next to
 *                        this chunk's scoring, selection and memory write; the next call of the context, whatever it is,
 *                        orders itself behind that work (a stream of the caller's that reads the state by other means has
 *                        to make a library call first, im_status for instance).  0: only the state update of the memory
 *                        write is left running.  Results are the same.
 *   IM_OPT_WAIT_LIMIT    (test aid) attempts of the bounded device-side waits in which a consumer waits for its copies to
 *                        arrive (TMA / bulk-copy rings of the decode attention kernels, the bulk-copy readout kernel and
 *                        the tcgen05 chunk attention kernel): 0 restores the default (2^22), k >= 1 allows k - 1 attempts,
 *                        so 1 makes every such wait give up at once.  A wait that gives up sets the sticky status word
 *                        (im_status then returns IM_ERR_TIMEOUT), the CTA still waits, with the full default limit, for
 *                        the copies it has in flight, frees its tensor memory and returns; the outputs of that call are
 *                        undefined, the context stays usable.
 */
typedef enum im_option {
  IM_OPT_CONCURRENCY = 0,
  IM_OPT_PREFETCH_NEXT = 1,
  IM_OPT_PREFILL_TENSOR = 2,
  IM_OPT_PROFILE_TARGET = 3,
  IM_OPT_DECODE_TENSOR = 4,
  IM_OPT_READOUT_STAGES = 5,
  IM_OPT_WAIT_LIMIT = 6,
  IM_OPT_LAYER_OVERLAP = 7,
  IM_OPT_STACK_PIPELINE = 8,
  IM_OPT_STACK_RESERVED = 9,
  IM_OPT_STACK_CHUNKS = 10,
  IM_OPT_FOLD_TENSOR = 11,
  IM_OPT_PREFILL_PIPELINE = 12
} im_option;
int im_set_option(im_ctx* ctx, int option, int value);

/*
 * Event counters kept on the device (no counterpart in the paper).  Synchronises the device.
 *   IM_COUNT_MERGE_RECOMPUTE  query heads for which the merge of a decode call with concurrency found more
 *                             than 90 % of the softmax mass on entries evicted in the same call and recomputed
 *                             the head over the retained entries instead of removing those terms from the sums.
 */
typedef enum im_counter { IM_COUNT_MERGE_RECOMPUTE = 0 } im_counter;
int im_event_count(im_ctx* ctx, int counter, int64_t* value);

/* Number of kernels this library has launched on behalf of `ctx` since im_create. */
int64_t im_launch_count(im_ctx* ctx);

/* Resolved configuration (defaults filled in) and slot capacity per sequence. */
int im_get_config(im_ctx* ctx, im_config* out, int32_t* capacity);

/*
 * Softmax attention of one query token over a given K/V set, for callers that cannot allocate.
 * (The paper has no counterpart: this is a service entry point, not a step of the method.)
 *
 * Some hosts of this library may not call cudaMalloc while they run: code inside a captured or
 * latency-critical serving loop, plug-ins that are handed a fixed memory arena, processes whose
 * device memory is fully committed to a KV pool.  Every other attention path here needs scratch
 * (the per-split partial results) carved out of a caller-provided workspace.  This variant keeps that
 * scratch in a fixed array inside the library image instead: 4 MiB of device memory that every GPU
 * loading the library holds until the process exits.  The call makes no allocation of any kind.
 *
 *   q    dev bf16 [n_q_heads, head_dim]
 *   k, v dev bf16 [n_kv_heads, n, head_dim]   (one contiguous slab per KV head)
 *   out  dev bf16 [n_q_heads, head_dim]       out_j = sum_t softmax_t(scale * q_j . k_t) v_t, KV head j / G_q
 *   softmax_scale 0 => 1/sqrt(head_dim);  head_dim <= 256;  n_q_heads a multiple of n_kv_heads, at most 65535
 * Limit: n_q_heads * ceil(n / 256) * (head_dim + 2) <= 1,048,576 (the array's float count); larger
 * problems are rejected with IM_ERR_CAPACITY and a message naming both numbers.
 * The first call on a device looks up the array's device address (a host-side set-up step); make
 * that first call before any stream capture.  All calls share the one array and nothing in it
 * needs to start at zero (every partial that is read was written by the same call), but two calls
 * that overlap on the GPU - different streams, or different host threads - race on it: serialise
 * them.  Kernels are enqueued on `cuda_stream`; the call does not synchronise.
 */
int im_attention_noalloc(const void* q, const void* k, const void* v, int n_q_heads, int n_kv_heads, int head_dim,
                         int n, float softmax_scale, void* out, void* cuda_stream);

/*
 * Retained sets per KV head (configuration scorer = 1 or 2; Sec. 2.2 frames eviction as S = f(.) in R^{B x H_kv x L},
 * I = TopK(S, L'), [K', V'] = Gather(K, V, I)).  im_prefill_chunk and im_decode_step then keep, for every KV head of a
 * sequence, the B entries with the largest score of THAT head (score descending, position ascending, the first n_sink
 * positions first); x and q_pre are ignored (there is no indexer), im_prefill_chunk_attend and score_share are not
 * available.  All heads hold the same number of entries; which positions they are differs per head.
 * The memory write of an evict step (Eq. 6-7; Alg. 1: "evicted_v is summed across heads per token"): every token that
 * loses at least one head slice in the step contributes ONE pair (k~, v~) in model space, the evicted slices at the
 * places of their query heads and zeros at the heads that keep the token.  With the same scores for every head this
 * is the shared-row path.
 *
 * im_set_scores (scorer = 2): `scores` is dev float32 [n_seq][H_kv][n_positions]; scores[i][h][t] is the importance of
 * token position t of the i-th sequence of the NEXT compressing call on `layer` for KV head h.  n_positions must cover
 * every position cached after that call's append, the call must name the same number of sequences, and the array must
 * stay valid until that call's kernels have run.  The scores are consumed by that call; a compressing call without
 * scores returns IM_ERR_STATE.  Non-finite scores set the status word.
 */
int im_set_scores(im_ctx* ctx, int layer, int n_seq, const float* scores, int64_t n_positions);

/*
 * Per-head pieces of the state in per-head mode (head in [0, H_kv)): IM_S_POS int32[n], IM_S_IMP float32[n] (the head's
 * scores), IM_S_K / IM_S_V bf16 [n][d] (the head's slab, slot order), IM_S_EVICTED int32[n_evicted] (ascending),
 * IM_S_SEL_POS / IM_S_SEL_IMP (what the head's latest selection chose among).  Import: IM_S_POS, IM_S_IMP, IM_S_K,
 * IM_S_V.  IM_S_COUNTS, IM_S_M and IM_S_B go through im_state_export / im_state_import in either mode; the pieces
 * above are refused there in per-head mode (and here otherwise).  Both synchronise the device.
 */
int im_state_export_head(im_ctx* ctx, int layer, int seq, int head, int which, void* host_buf, size_t bytes);
int im_state_import_head(im_ctx* ctx, int layer, int seq, int head, int which, const void* host_buf, size_t bytes);

/* Thread-local description of the last error returned on this thread ("" if none). */
const char* im_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* INDEXMEM_H_ */

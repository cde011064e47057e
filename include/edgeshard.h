/*
 * edgeshard.h — C ABI of the shard-execution library (sm_100a).
 *
 * EdgeShard cuts an LLM of N layers into contiguous shards and places each on one device
 * (paper, Sec. "System Model" and Sec. "Optimize LLM Inference"): a shard runs layers i..m,
 * takes the previous shard's activation (or the prompt's token ids if it holds the embedding
 * layer) and emits the activation of its last layer (or, if it holds the output layer, the
 * logits and the generated token).  Inference is a prefill over the prompt followed by
 * one-token-at-a-time generation against a KV cache that is reserved on the device beforehand
 * (Sec. "Generative LLM Inference", Sec. "Collaborative inference").  The partition algorithms
 * consume a per-layer profile: execution time, activation size and memory (Sec. "Profiling").
 *
 * This library is the execution of ONE shard on ONE GPU.  The decoder is Llama-2 (RMSNorm,
 * rotary position embedding on adjacent pairs (2i,2i+1), causal attention with grouped KV
 * heads, SwiGLU feed-forward), fp16 weights / KV / intermediate activations, fp32 accumulation,
 * fp32 residual stream (the activation that is handed off is fp32).
 *
 * Conventions
 *  - Every function returns a status and never throws or aborts.  On error nothing has been
 *    launched unless stated otherwise, out-parameters are untouched, and es_last_error()
 *    returns a thread-local message.
 *  - "dev" pointers are CUDA device pointers on the current device; "host" pointers are
 *    ordinary host memory.  The library allocates no device memory: weights, KV pages and
 *    scratch all belong to the caller and must outlive the shard.
 *  - Work is enqueued on the stream given at creation; calls do not synchronise unless stated.
 *  - Layer indices are decoder-layer indices in [0, n_layers_total).  The paper's layer 0
 *    (embedding) belongs to the shard with layer_begin == 0 and its layer N-1 (output layer)
 *    to the shard with layer_end == n_layers_total.
 */
#ifndef EDGESHARD_H_
#define EDGESHARD_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ES_API __attribute__((visibility("default")))
#else
#define ES_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct es_shard es_shard_t; /* opaque, library-owned host object */

typedef enum {
  ES_OK = 0,
  ES_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, both/neither of ids and hidden_in */
  ES_ERR_SHAPE = 2,          /* model dimensions the kernels do not support */
  ES_ERR_RANGE = 3,          /* layer range outside [0, n_layers_total], slot or length out of range */
  ES_ERR_STATE = 4,          /* decode on a slot that was never prefilled, handoff before any pass */
  ES_ERR_KV_FULL = 5,        /* the slot's context would exceed max_seq */
  ES_ERR_WORKSPACE = 6,      /* a caller buffer is smaller than es_shard_workspace_bytes says */
  ES_ERR_CUDA = 7,           /* a CUDA runtime call failed; message holds cudaGetErrorString */
  ES_ERR_DEVICE_TIMEOUT = 8, /* a bounded device-side wait gave up (see es_shard_device_status) */
  ES_ERR_UNSUPPORTED = 9
} es_status_t;

typedef enum { ES_DTYPE_F16 = 0, ES_DTYPE_F32 = 1, ES_DTYPE_I32 = 2 } es_dtype_t;

/* Model and capacity description.  max_slots = number of sequences whose KV is kept at once;
 * max_seq = longest context (prompt + generated) per slot; max_tokens = largest B*T of one
 * prefill call; kv_page_tokens = tokens per KV page (power of two, >= 16; 64 is the default
 * choice).  max_batch = largest B of one call (<= max_slots). */
typedef struct {
  int32_t n_layers_total, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rms_eps, rope_theta;
  int32_t max_slots, max_seq, max_tokens, max_batch, kv_page_tokens;
} es_model_desc_t;

/* One decoder layer: dev pointers, fp16, matrices row-major [out, in].
 *   attn_norm, ffn_norm [d_model]; wq [n_heads*head_dim, d_model]; wk, wv [n_kv_heads*head_dim, d_model];
 *   wo [d_model, n_heads*head_dim]; w_gate, w_up [d_ffn, d_model]; w_down [d_model, d_ffn].
 * All matrix pointers must be 16-byte aligned.  Borrowed for the shard's life. */
typedef struct {
  const void *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
} es_layer_weights_t;

typedef struct {
  const void *tok_embedding;         /* dev fp16 [vocab, d_model]; required iff layer_begin == 0 */
  const void *final_norm, *lm_head;  /* dev fp16 [d_model], [vocab, d_model]; required iff layer_end == n_layers_total */
  const es_layer_weights_t *layers;  /* host array of layer_end - layer_begin entries */
} es_weights_t;

/* A borrowed view of a device tensor, row-major, contiguous. */
typedef struct {
  void *data;
  int32_t dtype; /* es_dtype_t */
  int32_t rank;
  int64_t shape[4];
} es_tensor_t;

/* One entry of the per-layer profile (the t_comp / O_i / Req_i traces of Sec. "Profiling").
 * layer: -1 = embedding, n_layers_total = final norm + LM head, otherwise the decoder layer.
 * avg_ms_per_token = (sum of prefill ms + sum of decode ms) / (n_prefill + n_decode): each
 * prefill call and each decode step generates one token per sequence. */
typedef struct {
  int32_t layer;
  int32_t n_prefill, n_decode;
  float prefill_ms_mean, decode_ms_mean, avg_ms_per_token;
  int64_t activation_bytes; /* output of this layer for one token: d_model * 4 (or vocab * 4 for the head) */
  int64_t weight_bytes;     /* Req_i, parameters */
  int64_t kv_bytes;         /* Req_i, reserved KV cache of this layer (all slots) */
} es_layer_profile_t;

/* Sizes of the two caller-owned device buffers a shard [layer_begin, layer_end) needs.
 * Host-only; validates the description exactly as es_shard_create does. */
ES_API es_status_t es_shard_workspace_bytes(const es_model_desc_t *desc, int32_t layer_begin, int32_t layer_end,
                                     size_t *kv_bytes, size_t *scratch_bytes);

/* Creates the shard for decoder layers [layer_begin, layer_end) (paper: layers i..m on device j).
 * kv_buffer / scratch_buffer: dev, 256-byte aligned, at least the sizes reported above; the
 * library initialises them (enqueued on `cuda_stream`, a cudaStream_t cast to void*, may be 0).
 * KV pages of every slot are reserved here, before any inference call. */
ES_API es_status_t es_shard_create(const es_model_desc_t *desc, int32_t layer_begin, int32_t layer_end,
                            const es_weights_t *weights, void *kv_buffer, size_t kv_bytes,
                            void *scratch_buffer, size_t scratch_bytes, void *cuda_stream, es_shard_t **out);

/* Prefill: runs the shard over B prompts of T tokens each, filling the KV cache of the given slots
 * from position 0 (earlier content of those slots is discarded).
 *   ids        dev int32 [B, T]   — required iff the shard holds the embedding, else NULL
 *   hidden_in  fp32 [B, T, d_model] view of the previous shard's handoff — required iff it does not
 *   slots      host int32 [B], distinct, each in [0, max_slots)
 * Result: es_shard_handoff() gives hidden [B, T, d_model]; with the output layer also logits of the
 * LAST prompt position [B, vocab] and the greedy token [B] (lowest index wins ties). */
ES_API es_status_t es_shard_prefill(es_shard_t *shard, const int32_t *ids, const es_tensor_t *hidden_in,
                             int32_t B, int32_t T, const int32_t *slots);

/* Prefill of prompts of different lengths in one batch (Sec. "Generative LLM Inference": requests are
 * padded to a common length).  Arguments as for es_shard_prefill; the B prompts are RIGHT-padded to T
 * rows each, and
 *   lens       host int32 [B], 1 <= lens[b] <= T: the real tokens of sequence b are its first lens[b] rows.
 * Padding ids must be valid token ids (their values do not matter).  All B * T rows are computed; causal
 * attention keeps padding out of every real row.  Slot b then holds lens[b] positions, so the next
 * es_shard_decode_step continues each sequence at its own position (the padded rows' K/V beyond it are
 * overwritten as the sequence grows and are never read).  With the output layer, logits and the greedy
 * token are those of row lens[b] - 1 of each sequence.  es_shard_handoff() gives hidden [B, T, d_model];
 * rows at or beyond lens[b] are padding, and the next shard must be given the same lens.
 * ES_ERR_RANGE if a length is outside [1, T]. */
ES_API es_status_t es_shard_prefill_ragged(es_shard_t *shard, const int32_t *ids, const es_tensor_t *hidden_in,
                                    int32_t B, int32_t T, const int32_t *slots, const int32_t *lens);

/* The same prompts without the padding (Sec. "Generative LLM Inference" pads a batch to one length; this form
 * computes only the real tokens): the B prompts are PACKED one after the other,
 *   ids        dev int32 [sum(lens)]            (shard with the embedding), or
 *   hidden_in  dev fp32 [sum(lens), d_model]    (other shards: the previous shard's packed handoff),
 *   lens       host int32 [B], 1 <= lens[b] <= max_seq; sum(lens) <= max_tokens.
 * Sequence b owns rows sum(lens[0..b-1]) .. + lens[b] - 1; every product runs over sum(lens) rows, attention runs
 * per sequence over its own rows, K/V go to the sequence's slot, and slot b then holds lens[b] positions exactly
 * as after es_shard_prefill_ragged.  With the output layer, logits and greedy tokens are [B, ...], those of each
 * sequence's last token.  es_shard_handoff() gives hidden as [1, sum(lens), d_model] (packed the same way): the
 * next shard takes it with the same lens.  Results equal the padded form's up to fp32 summation order (the
 * products see a different number of rows).  ES_ERR_RANGE / ES_ERR_KV_FULL as for the other prefill calls. */
ES_API es_status_t es_shard_prefill_packed(es_shard_t *shard, const int32_t *ids, const es_tensor_t *hidden_in,
                                           int32_t B, const int32_t *slots, const int32_t *lens);

/* One autoregressive step for B sequences: each consumes one token (ids dev int32 [B]) or one
 * activation row (hidden_in fp32 [B, d_model]) at its slot's next position and attends to the
 * slot's cached keys/values.  ES_ERR_STATE if a slot has no prefilled context, ES_ERR_KV_FULL if
 * it is at max_seq.  `ids` may be the next_ids pointer returned by es_shard_handoff (greedy
 * feedback without leaving the device). */
ES_API es_status_t es_shard_decode_step(es_shard_t *shard, const int32_t *ids, const es_tensor_t *hidden_in,
                                 int32_t B, const int32_t *slots);

/* The inter-shard activation of the most recent prefill/decode call: the residual stream after
 * layer layer_end-1, fp32, [B, T, d_model] after a prefill and [B, 1, d_model] after a decode step
 * (size O_i of the paper; on the same device the hand-over is this pointer, zero copy).  With the
 * output layer, `logits` (fp32 [B, vocab]) and `next_ids` (int32 [B]) are filled as well, otherwise
 * their data is NULL.  Any of the three out-pointers may be NULL.  Views stay valid, and their
 * contents unchanged, until the next prefill/decode call on this shard. */
ES_API es_status_t es_shard_handoff(es_shard_t *shard, es_tensor_t *hidden_out, es_tensor_t *logits,
                             es_tensor_t *next_ids);

/* Per-layer device time, activation size and memory.  Timing is collected only while profiling is
 * switched on (es_shard_set_profiling), with one CUDA event pair per layer per call; this call
 * synchronises the stream.  Writes min(capacity, entries) items to `out` and the number of entries
 * (layers in the shard, plus embedding and/or head when present) to *n. */
ES_API es_status_t es_layer_profile(es_shard_t *shard, es_layer_profile_t *out, int32_t capacity, int32_t *n);
ES_API es_status_t es_shard_set_profiling(es_shard_t *shard, int32_t enabled);

/* Forget the context of the given slots (host int32 [n]); NULL / n == 0 resets every slot. */
ES_API es_status_t es_shard_reset_slots(es_shard_t *shard, const int32_t *slots, int32_t n);

/* Replace the logical->physical KV page map: host int32 [max_slots * pages_per_slot], a permutation
 * of 0..max_slots*pages_per_slot-1 (pages_per_slot = ceil(max_seq / kv_page_tokens)).  Resets all
 * slots.  Results never depend on the map. */
ES_API es_status_t es_shard_set_page_table(es_shard_t *shard, const int32_t *table);

/* Run decode steps as replayed CUDA graphs (default on; needs a shard created on a stream other than
 * the default stream, which cannot be captured, and profiling off).  With graphs off every kernel
 * is launched individually; results are identical. */
ES_API es_status_t es_shard_set_graphs(es_shard_t *shard, int32_t enabled);

/* Reads the device status word (synchronises): ES_OK, or ES_ERR_DEVICE_TIMEOUT if a bounded wait
 * inside a kernel ran out since the last call.
 * Checking mode: with ES_DEBUG=1 in the environment of the process (read once), the call also verifies
 * that the 256 guard bytes the library keeps behind every region it carves out of the scratch buffer are
 * intact (a kernel that wrote past its region lands there first) and that the tables the kernels index
 * with hold values inside their ranges (page numbers, context lengths against the host's own count, the
 * uploaded slot list); a violation is ES_ERR_STATE with the region or entry named in es_last_error.  In
 * this mode every prefill / decode call first synchronises and runs the same checks on what the previous
 * pass left behind (so it is for testing, not for timing). */
ES_API es_status_t es_shard_device_status(es_shard_t *shard);

/* Exercises the time-out path above without any kernel misbehaving: enqueues a one-CTA kernel built like the
 * tensor-core kernels (barrier, TMEM allocation, bounded wait, common teardown) whose barrier is never arrived
 * on.  Its wait gives up after limit_us microseconds (1 .. 100000), records its code in the status word, frees
 * its TMEM and returns; the next es_shard_device_status reports ES_ERR_DEVICE_TIMEOUT and clears the word, and
 * the shard stays usable.  For tests of a caller's error handling; the paper has no counterpart. */
ES_API es_status_t es_shard_wait_probe(es_shard_t *shard, int32_t limit_us);

/* Launch-by-launch timing of the linear-layer kernels (the weight-streaming and tensor-core
 * products that dominate a pass): while on, every such launch is bracketed by a CUDA event pair on
 * the shard's stream (every launch of a pass, by category) and decode steps are not replayed as graphs.  Switching it on or off clears
 * the record.  es_shard_kernel_timing synchronises and reports the summed event time, the weight
 * bytes those launches had to read (N*K*2 each) and their number. */
typedef enum {
  ES_KT_EMBED = 0, ES_KT_RMSNORM = 1, ES_KT_QKV = 2, ES_KT_ATTENTION = 3, ES_KT_O = 4, ES_KT_GATE_UP = 5,
  ES_KT_DOWN = 6, ES_KT_LM_HEAD = 7, ES_KT_ARGMAX = 8, ES_KT_SET_CTX = 9,
  ES_KT_FINISH = 10,  /* epilogue kernel of a K-sliced product (SwiGLU / QKV forms) */
  ES_KT_REDUCE = 11,  /* slice reduction + residual (+ RMSNorm for the next product) of a K-sliced product */
  ES_KT_COUNT = 12
} es_kernel_category_t;
ES_API es_status_t es_shard_set_kernel_timing(es_shard_t *shard, int32_t enabled);
/* The same record split by kernel category: three arrays of ES_KT_COUNT entries (any may be NULL):
 * summed event milliseconds, algorithmic bytes (weights for the linear kernels, rows for the
 * element-wise ones, 0 where not modelled) and launches (an attention entry may be two kernels). */
ES_API es_status_t es_shard_kernel_timing_detail(es_shard_t *shard, double *ms, double *bytes, int64_t *launches);
ES_API es_status_t es_shard_kernel_timing(es_shard_t *shard, double *total_ms, double *weight_bytes,
                                          int64_t *launches);

/* Timing from inside a step (Sec. "Profiling" asks what each layer costs on the device; this is the same
 * question one level down, per kernel of a replayed step).  While on, every kernel of a pass records the
 * earliest time any of its CTAs started and the latest time the first thread of any of its CTAs finished
 * (%globaltimer, two atomics per CTA) into a slot of the scratch buffer; decode steps are still replayed as graphs
 * with programmatic dependent launch, so the overlap between consecutive kernels is what it is in a normal
 * step (measured: a step takes the same time with and without the stamps).  Switching it on or off drops the captured
 * graphs.  es_shard_step_timing synchronises and returns, for each launch of the most recently enqueued
 * pass in launch order (up to `capacity`; *n = how many there were): its category, its start and end in
 * microseconds relative to the first start of the pass, and its algorithmic bytes (as in
 * es_shard_kernel_timing_detail).  A decode-attention entry covers the split and the merge kernel.
 * At most 2048 launches per pass are stamped; later ones are left out. */
ES_API es_status_t es_shard_set_step_timing(es_shard_t *shard, int32_t enabled);
ES_API es_status_t es_shard_step_timing(es_shard_t *shard, int32_t capacity, int32_t *n, int32_t *category,
                                        double *start_us, double *end_us, double *bytes);

/* Number of kernels this shard has launched (graph replays count their nodes). */
ES_API int64_t es_shard_launch_count(const es_shard_t *shard);

ES_API void es_shard_destroy(es_shard_t *shard);

ES_API const char *es_last_error(void);
ES_API const char *es_version(void);

/* ---- partition planners (host only) ------------------------------------------------------------
 * The paper's two dynamic programs over the profiled traces.  N layers (layer 0 = embedding, pinned to
 * device 0 by the privacy constraint), M devices; all arrays host, double:
 *   t_comp [N, M]  time of layer i on device j          O   [N]  activation size of layer i
 *   Req    [N]     memory of layer i                     Mem [M]  memory budget of device j
 *   Bw     [M, M]  bandwidth from device k to device j (same unit as O per unit of time; diagonal unused)
 *   assign [N]     out: device of every layer
 * ES_ERR_RANGE if no placement fits the memory budgets.
 *
 * es_partition_latency — Algorithm 1 / Eq. 4: DP(i, j) = min_k DP(i-1, k) + t_comp(i, j) + O(i-1)/Bw(k, j),
 * plus the return of the token O(N-1)/Bw(j, 0) at the last layer; DP(0, 0) = t_comp(0, 0).  Memory is
 * tracked along each cell's own best path (the algorithm's "update memory" step): the result is always
 * feasible, and optimal whenever the budgets do not bind on that path.  *latency = total time T_tol (Eq. 2).
 *
 * es_partition_throughput — Algorithm 2: every chosen device holds one contiguous range of layers;
 * g(m, S + {j}, j) = min over (i, k) of max(g(i, S, k), O(i-1)/Bw(k, j), t_comp(i..m-1, j)), memory
 * Req(i..m-1) <= Mem(j) per device; the source device holds the first range, which contains layer 0 and
 * may contain more.  *bottleneck = the slowest stage's time (its reciprocal is the pipeline throughput).
 * Exact; cost O(N^2 2^M M^2), M <= 20.
 *
 * Both planners refuse (ES_ERR_UNSUPPORTED, nothing computed) a problem whose table would exceed 4 GiB of host
 * memory — (N + 1) * 2^M * M cells of 12 bytes for es_partition_throughput (N = 82 layers: M <= 17), N * M cells
 * of 12 + 8 M bytes for es_partition_latency — and report an allocation failure the same way. */
ES_API es_status_t es_partition_latency(int32_t N, int32_t M, const double *t_comp, const double *O, const double *Req,
                                        const double *Mem, const double *Bw, int32_t *assign, double *latency);
ES_API es_status_t es_partition_throughput(int32_t N, int32_t M, const double *t_comp, const double *O,
                                           const double *Req, const double *Mem, const double *Bw, int32_t *assign,
                                           double *bottleneck);

/* ---- single operations (the steps of the path, exposed for unit parity tests) -----------------
 * All pointers dev unless marked host; `stream` is a cudaStream_t cast to void*.              */

/* y[m,:] = x[m,:] * gain / sqrt(mean(x[m,:]^2) + eps);  x fp32 [M, d], gain fp16 [d], y fp16 [M, d]. */
ES_API es_status_t es_op_rmsnorm(const float *x, const void *gain, void *y, int32_t M, int32_t d, float eps,
                          void *stream);

/* C = A * W^T (+ R):  A fp16 [M, K], W fp16 [N, K], C fp32 [M, N], R fp32 [M, N] or NULL.
 * path: 0 = automatic, 1 = tensor-core (tcgen05) kernel, 2 = weight-streaming kernel (M <= 16),
 * 3 = plain reference kernel, 4 = weight-streaming kernel on tensor cores (M <= 16, K % 256 == 0),
 * 5 = tensor-core kernel on CTA pairs (needs M >= 256 and at least 40 tiles of 256 x 256),
 * 6 = the same with 256 x 512 tiles per pair. */
ES_API es_status_t es_op_linear(const void *A, const void *W, const float *R, float *C, int32_t M, int32_t N,
                         int32_t K, int32_t path, void *stream);

/* The tensor-core product with its K range cut into k_splits slices (Sec. "Experimental Setup" runs
 * short prompts, for which a d_model-wide product has too few output tiles to fill the machine):
 * C[M, N] = A[M, K] * W[N, K]^T (+ R), fp16 in, fp32 out, all device pointers, row-major, dense.
 * Every (tile, slice) pair is computed by its own CTA into `workspace` ([k_splits, M, N] fp32,
 * device, 16-byte aligned, at least es_op_linear_splitk_workspace_bytes bytes); a second kernel adds
 * the slices in ascending order and the residual, so the result does not depend on scheduling.
 * With 256 or more rows the slices are computed by CTA pairs (256 x 256 tiles), below that by single CTAs.
 * k_splits = 0 lets the library choose (1 = no split, no workspace needed).  Slices must not be
 * empty: (k_splits - 1) * ceil(ceil(K / 64) / k_splits) < ceil(K / 64), else ES_ERR_INVALID_ARG.
 * N must be a multiple of 4, K of 8.  R may be NULL and may alias C.
 * With 3 <= M <= 16 (a decode step of several sequences) the weight-streaming kernel is used instead:
 * every CTA keeps one K slice of the activations in shared memory and streams 16-row groups of W over
 * it; K must be a multiple of 256 and K / 32 divisible by k_splits, a slice of 8 (M <= 8) or 16 rows
 * must fit 100 KB.  M <= 2 is ES_ERR_UNSUPPORTED (such products never need slicing). */
ES_API size_t es_op_linear_splitk_workspace_bytes(int32_t M, int32_t N, int32_t k_splits);
ES_API es_status_t es_op_linear_splitk(const void *A, const void *W, const float *R, float *C, int32_t M, int32_t N,
                                       int32_t K, int32_t k_splits, void *workspace, size_t workspace_bytes,
                                       void *stream);

/* Causal self-attention over a prompt.  q fp16 [B, T, Hq, hd] (already rotated); k, v fp16
 * [B, T, Hkv, hd]; out fp16 [B, T, Hq*hd].  Query t sees keys 0..t; scale 1/sqrt(hd).
 * path: 0 = automatic, 1 = tensor-core (tcgen05) kernel, 2 = CUDA-core kernel. */
ES_API es_status_t es_op_prefill_attention(const void *q, const void *k, const void *v, void *out, int32_t B,
                                    int32_t T, int32_t Hq, int32_t Hkv, int32_t hd, int32_t path, void *stream);

/* Bytes of scratch es_op_decode_attention needs. */
ES_API size_t es_op_decode_attention_scratch_bytes(int32_t B, int32_t Hq, int32_t hd, int32_t max_ctx,
                                            int32_t page_tokens);

/* Split-KV attention of one query row per (sequence, head) over a paged cache.
 *   q fp16 [B, Hq, hd]; k_pages, v_pages fp16 [n_pages, Hkv, P, hd];
 *   block_table int32 [B, pages_per_seq] (physical page of each logical page);
 *   ctx_len int32 [B] (keys visible to the query, >= 1); out fp16 [B, Hq*hd];
 *   scratch: dev, es_op_decode_attention_scratch_bytes(...) bytes. */
ES_API es_status_t es_op_decode_attention(const void *q, const void *k_pages, const void *v_pages,
                                   const int32_t *block_table, const int32_t *ctx_len, void *out,
                                   int32_t B, int32_t Hq, int32_t Hkv, int32_t hd, int32_t page_tokens,
                                   int32_t pages_per_seq, int32_t max_ctx, void *scratch, size_t scratch_bytes,
                                   void *stream);

/* The same operation as es_op_decode_attention for callers that must not allocate device memory
 * and have no buffer to lend — for instance code running under a memory pool that forbids
 * cudaMalloc, inside a region where allocation would synchronise the device, or a plug-in that
 * is only ever given its inputs and outputs.  (The paper has no counterpart; this is a
 * convenience of the library.)  The split-KV partials go to an array built into the library
 * image, es_op_decode_attention_static_capacity() bytes (8 MiB) on every GPU that loads the
 * library, held until the process exits.  The call performs no allocation of any kind.
 *   - A call whose partials do not fit returns ES_ERR_WORKSPACE and launches nothing; use
 *     es_op_decode_attention with your own buffer for such sizes.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture.
 *   - All calls share the one array.  Each call overwrites what it later reads, so stale contents
 *     are harmless, but two calls that overlap on the GPU (different streams) race: order them.
 * Arguments and result are those of es_op_decode_attention, without scratch / scratch_bytes. */
ES_API size_t es_op_decode_attention_static_capacity(void);
ES_API es_status_t es_op_decode_attention_static(const void *q, const void *k_pages, const void *v_pages,
                                                 const int32_t *block_table, const int32_t *ctx_len, void *out,
                                                 int32_t B, int32_t Hq, int32_t Hkv, int32_t hd,
                                                 int32_t page_tokens, int32_t pages_per_seq, int32_t max_ctx,
                                                 void *stream);

#ifdef __cplusplus
}
#endif
#endif /* EDGESHARD_H_ */

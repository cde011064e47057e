// Internal declarations shared by the kernels and the host side of the shard library.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "edgeshard.h"

namespace es {

// ---- error plumbing -----------------------------------------------------------------------
void set_error(const char* fmt, ...);
es_status_t fail(es_status_t st, const char* fmt, ...);

#define ES_CUDA_CHECK(expr)                                                                   \
  do {                                                                                        \
    cudaError_t _e = (expr);                                                                  \
    if (_e != cudaSuccess)                                                                    \
      return ::es::fail(ES_ERR_CUDA, "%s failed: %s (%s:%d)", #expr, cudaGetErrorString(_e), \
                        __FILE__, __LINE__);                                                  \
  } while (0)

#define ES_TRY(expr)                 \
  do {                               \
    es_status_t _s = (expr);         \
    if (_s != ES_OK) return _s;      \
  } while (0)

// ---- tuning knobs (read once from the environment; defaults are the measured best) -----------
struct Tunables {
  int stream_deep;   // ES_STREAM_DEEP: weight-streaming kernel chunk depth, 1 = 4 KB per warp per buffer (default), 0 = 2 KB
  int tc_pair;       // ES_TC_PAIR: CTA-pair tensor-core kernel for large prefill products (1, default) or never (0)
  int tc_pair_wide;  // ES_TC_PAIR_WIDE: 256 x 512 pair tiles: chosen per shape (1, default), never (0), always (2)
  int split_pairs;   // ES_SPLIT_PAIRS: split-K products with 256 or more rows run on CTA pairs (1, default) or on single CTAs (0)
  int pdl;           // ES_PDL: programmatic dependent launch in decode steps (1, default) or plain stream order (0)
  int attn_mma;      // ES_ATTN_MMA: tensor-core decode attention for launches with many items (1, default) or never (0)
  int split_k;       // ES_SPLIT_K: split-K for the O and down projections of short prefills (1, default) or never (0)
  int ks_min_slice;        // ES_KS_MIN_SLICE: smallest K slice of the K-sliced streaming kernel (elements, default 512)
  int ks_splits;           // ES_KS_SPLITS: K slices of the K-sliced streaming kernel (0 = chosen per shape; a value that does not fit is ignored)
  int ks_cols;             // ES_KS_COLS: column ranges per K slice of that kernel (0 = chosen per shape)
  int attn_split_tokens;   // ES_ATTN_SPLIT_TOKENS: smallest split of a decode-attention context (tokens; 0 = 256, or 384 for groups of 4-8 query heads)
  int debug_checks;        // ES_DEBUG: es_shard_device_status also verifies the guard bytes behind every scratch region and the ranges of the page table, context lengths and slot list (1) or not (0, default)
  int even_grid;           // ES_EVEN_GRID: weight-streaming kernels shrink their grid so that every CTA (warp) gets the same number of units (1) or fill the machine (0)
};
const Tunables& tunables();

// Number of SMs of the current device (148 on a B200; 0 if the query fails, which callers treat as 1).  Every
// grid size, wave count and split rule below is written in terms of it.
int sm_count();

// ---- the linear layer family ----------------------------------------------------------------
// C[m, n] = sum_k A[m, k] * W[n, k], A fp16 [M, K] row-major (row stride lda), W fp16 row-major
// [*, K].  The N output columns are a concatenation of up to three weight matrices ("segments",
// used for Wq|Wk|Wv); with EPI_SWIGLU the kernel contracts against w[0] (gate) and w[1] (up) for
// the same n and emits one column.

enum Epilogue : int {
  EPI_F32 = 0,     // out_f32[m, n] = acc (+ res[m, n])
  EPI_SWIGLU = 1,  // out_f16[m, n] = silu(acc_gate) * acc_up
  EPI_QKV = 2      // rotate q and k, q -> out_f16 [M, Nq], k/v -> paged cache
};

// Four TMA tensor maps (A and up to three weight segments) of one tensor-core launch; opaque here.
struct alignas(64) TcMaps { unsigned char bytes[512]; };

struct LinearParams {
  const TcMaps* tc_maps;   // host pointer to pre-encoded maps (rows of A >= M), or nullptr: encode per launch
  const __half* A;
  int64_t lda;
  // optional fused RMSNorm (weight-streaming kernel, M <= 2): A = rmsnorm(norm_x rows; norm_gain)
  const float* norm_x;     // fp32 [M, K], row stride norm_ldx; nullptr = read A
  int64_t norm_ldx;
  const __half* norm_gain;
  float norm_eps;
  const __half* w[3];
  int seg_rows[3];
  int M, N, K;
  // EPI_F32
  float* out_f32;
  const float* res;   // may alias out_f32 (same element read then written by one thread)
  int64_t ldo;
  // EPI_SWIGLU / EPI_QKV (q)
  __half* out_f16;
  // EPI_QKV
  __half* k_cache;    // this layer's K pages [n_pages, Hkv, P, hd]
  __half* v_cache;
  const int* block_table;  // [max_slots, pages_per_slot]
  const int* ctx_len;      // [max_slots], device-side context length of each slot
  const int* slots;        // [B]
  const float* rope_cos;   // [max_seq, hd/2]
  const float* rope_sin;
  int T;                   // rows per sequence: row m belongs to sequence m / T at prompt offset m % T
  int is_decode;           // position = ctx_len[slot] instead of m % T
  const int* cu_rows;      // packed prompts: [n_seq + 1] first row of every sequence (device); row m then belongs to the
  int n_seq;               // sequence b with cu_rows[b] <= m < cu_rows[b + 1], at offset m - cu_rows[b].  nullptr = m / T
  int Hq, Hkv, hd, P, pages_per_slot, max_seq;
  // split-K (tensor-core kernel with EPI_F32; K-sliced streaming kernel with any epilogue): > 1 = raw partial
  // sums go to part[k_splits, M, columns] and a second kernel finishes the product
  int k_splits;
  float* part;
  // CTA-pair tensor-core kernel: accumulators per tile, 1 = 256 x 256 tiles, 2 = 256 x 512 tiles, 0 = chosen per shape
  int pair_nacc;
  // k_splits > 1 on the tensor-core path: the CTA-pair kernel computes the slices (else the single-CTA kernel)
  int split_on_pairs;
  // optional time stamps of this launch (see launch.cuh), nullptr = none
  unsigned long long* stamp;
};

// Kernel families.  Each returns after enqueuing; `launches` is incremented per kernel launched.
es_status_t launch_linear_reference(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches);
es_status_t launch_linear_stream(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl = false);   // M <= 16
bool linear_stream_can_fuse_norm(int M);
// tensor-core (mma.sync) variant of the weight-streaming kernel for 3..16 rows
bool linear_stream_mma_supported(const LinearParams& p, int epi);
es_status_t launch_linear_stream_mma(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl = false);
// K slices across CTAs for this product (1 = the activations fit in shared memory whole); with p.k_splits > 1
// the kernel writes partial sums to p.part ([k_splits, M, N], SwiGLU: [k_splits, M, 2N] gate | up) and the
// product is finished by launch_splitk_reduce (plain epilogue) or launch_splitk_finish (SwiGLU, QKV)
int linear_stream_mma_splits(const LinearParams& p, int epi, size_t workspace_bytes);
es_status_t launch_splitk_finish(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl = false);
es_status_t launch_linear_tc(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, int* status_word, bool pdl = false);
bool linear_tc_supported(const LinearParams& p, int epi);
// number of K slices the tensor-core kernel should use for this product (1 = do not split), and the
// workspace that covers any product for which the answer is > 1
int linear_tc_splits(const LinearParams& p, int epi);
size_t linear_tc_split_workspace_bytes();
// out[m, :] = (res ? res[m, :] : 0) + sum over slices (ascending) of part[s, m, :]; with gain != nullptr also
// y[m, :] = rmsnorm(out[m, :]) * gain in fp16.  N % 4 == 0.  res may alias out.
es_status_t launch_splitk_reduce(const float* part, int k_splits, const float* res, float* out, int M, int N, int64_t ldo,
                                 const __half* gain, __half* y, float eps, cudaStream_t s, int64_t* launches, bool pdl = false,
                                 unsigned long long* stamp = nullptr);
// CTA-pair (cta_group::2) variant for large M; uses the same tensor maps
bool linear_tc2_supported(const LinearParams& p, int epi);
int linear_tc2_splits(const LinearParams& p, int epi);   // K slices for a plain product on CTA pairs (1 = not this way)
es_status_t launch_linear_tc2(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, int* status_word, bool pdl = false);
// Encodes the tensor maps for p's operands; the A map covers a_rows rows (the buffer's capacity).
es_status_t tc_build_maps(const LinearParams& p, int epi, int64_t a_rows, TcMaps* out);

// TMA tensor map (128 bytes, 64-byte aligned) of an fp16 row-major matrix [rows, cols] with row stride
// ld elements: boxes of 64 columns x box_rows rows, 128-byte swizzle, zero fill outside.
es_status_t tma_encode_2d_f16(void* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows);
bool tma_available();

// ---- element-wise / reductions ---------------------------------------------------------------
es_status_t launch_embed(const int* ids, const __half* table, float* x, int M, int d, int vocab,
                         cudaStream_t s, int64_t* launches, bool pdl = false, unsigned long long* stamp = nullptr);
// row r of y = rmsnorm(row (r * row_stride + row_offset) of x); with last_of (device, [M]) the source row is
// r * row_stride + last_of[r] - 1 instead (the last of the first last_of[r] rows of block r)
es_status_t launch_rmsnorm(const float* x, const __half* gain, __half* y, int M, int d, float eps,
                           int64_t row_stride, int64_t row_offset, cudaStream_t s, int64_t* launches,
                           bool pdl = false, const int* last_of = nullptr, unsigned long long* stamp = nullptr);
es_status_t launch_argmax(const float* logits, int* out, int B, int V, cudaStream_t s, int64_t* launches,
                          bool pdl = false, unsigned long long* stamp = nullptr);
// ctx_len[slots[b]] = (add ? ctx_len[slots[b]] : 0) + (values ? values[b] : value)
es_status_t launch_set_ctx(int* ctx_len, const int* slots, int B, int value, int add, cudaStream_t s,
                           int64_t* launches, bool pdl = false, const int* values = nullptr,
                           unsigned long long* stamp = nullptr);

// A one-CTA kernel whose only barrier is never arrived on: its bounded wait runs out after limit_ns and writes
// its code to `status` (two ints), then the CTA leaves through the usual teardown.  Test support.
es_status_t launch_wait_probe(int* status, unsigned long long limit_ns, cudaStream_t s, int64_t* launches);

// ---- attention -------------------------------------------------------------------------------
// K/V addressing shared by both attention kernels: token t of sequence b, kv head g lives at
//   base + page * page_stride + g * head_stride + (t % P) * tok_stride,
//   page = block_table ? block_table[slot(b) * pages_per_slot + t / P] : b * pages_per_slot + t / P
struct KvView {
  const __half* k;
  const __half* v;
  const int* block_table;
  const int* slots;       // [B] or nullptr (slot = b)
  int64_t page_stride, head_stride, tok_stride;
  int P, pages_per_slot;
};

__device__ __forceinline__ const __half* kv_addr(const KvView& kv, const __half* base, int slot, int t, int g) {
  const int lp = t / kv.P;
  const int page = kv.block_table ? kv.block_table[(int64_t)slot * kv.pages_per_slot + lp]
                                  : slot * kv.pages_per_slot + lp;
  return base + (int64_t)page * kv.page_stride + (int64_t)g * kv.head_stride + (int64_t)(t - lp * kv.P) * kv.tok_stride;
}

struct PrefillAttnParams {
  const __half* q;   // [B, T, Hq, hd]
  __half* out;       // [B, T, Hq*hd]
  KvView kv;
  int B, T, Hq, Hkv, hd;
  int64_t kv_rows;          // rows of the K / V matrices as 2-D [rows, row width] views (tensor-core kernel)
  const int* cu_rows;       // packed prompts: [B + 1] first query row of every sequence (T = the longest prompt), or nullptr
  const TcMaps* tc_maps;    // pre-encoded maps {q, k, v} or nullptr: encode per launch
  int* status;
  unsigned long long* stamp;   // optional time stamps of this launch, nullptr = none
};
// path: 0 = automatic, 1 = tensor-core (tcgen05) kernel, 2 = CUDA-core kernel
es_status_t launch_prefill_attention(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches, int path = 0, bool pdl = false);
es_status_t launch_prefill_attention_simt(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches);
bool prefill_attention_tc_supported(const PrefillAttnParams& p);
es_status_t prefill_attention_tc_build_maps(const PrefillAttnParams& p, int64_t q_rows, TcMaps* out);
es_status_t launch_prefill_attention_tc(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches, bool pdl = false);

struct DecodeAttnParams {
  const __half* q;   // [B, Hq, hd]
  __half* out;       // [B, Hq*hd]
  KvView kv;
  const int* ctx_len;     // indexed by slot (or by b when kv.slots == nullptr)
  int ctx_add;            // keys visible = ctx_len[.] + ctx_add
  float* part;            // scratch [B, Hq, n_splits, hd + 2]
  int* split_cnt;         // one arrival counter per (sequence, KV head), zero before the launch and zero again after
                          // it (needed when n_splits > 1 and the launch is small enough to merge in the kernel)
  int B, Hq, Hkv, hd;
  int n_splits, pages_per_split;
  int merge_in_kernel;    // set by launch_decode_attention: the last split CTA to arrive merges (else a merge launch)
  unsigned long long* stamp;   // optional time stamps of the launch (split and merge kernels share them), nullptr = none
};
size_t decode_attention_scratch_bytes(int B, int Hq, int hd, int n_splits);
// byte offset of the arrival counters inside the scratch, and their size
size_t decode_attention_counter_offset(int B, int Hq, int hd, int n_splits);
size_t decode_attention_counter_bytes(int B, int Hq);

// The end of both split kernels when the context was cut into several splits: the CTA has written its
// unnormalised partial (o, max, sum) of the G heads of (sequence b, KV head kvh); the CTA that arrives last
// (a counter per (b, kvh); CTAs of splits beyond the context never arrive) merges the splits in ascending order,
// writes the final rows and puts the counter back to zero.  Nobody waits.  All threads of the CTA call.
template <int HD, int G>
__device__ __forceinline__ void merge_splits_if_last(const DecodeAttnParams& p, int b, int kvh, int ctx, int* s_flag) {
  int* cnt = p.split_cnt + (b * p.Hkv + kvh);
  const int tokens_per_split = p.pages_per_split * p.kv.P;
  int active = (ctx + tokens_per_split - 1) / tokens_per_split;
  active = active < p.n_splits ? active : p.n_splits;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *s_flag = (atomicAdd(cnt, 1) == active - 1) ? 1 : 0;
  __syncthreads();
  if (*s_flag == 0) return;
  __threadfence();
  for (int i = threadIdx.x; i < G * HD; i += blockDim.x) {
    const int j = i / HD, c = i - j * HD;
    const int64_t row = (int64_t)b * p.Hq + ((int64_t)kvh * G + j);
    const float* src = p.part + row * p.n_splits * (HD + 2);
    float mm = -INFINITY;
    for (int s = 0; s < active; ++s) mm = fmaxf(mm, __ldcg(src + (int64_t)s * (HD + 2) + HD));
    float o = 0.f, ll = 0.f;
    for (int s = 0; s < active; ++s) {
      const float f = __expf(__ldcg(src + (int64_t)s * (HD + 2) + HD) - mm);
      o += __ldcg(src + (int64_t)s * (HD + 2) + c) * f;
      ll += __ldcg(src + (int64_t)s * (HD + 2) + HD + 1) * f;
    }
    p.out[row * HD + c] = __float2half_rn(o / ll);
  }
  if (threadIdx.x == 0) *cnt = 0;
}
void choose_splits(int max_ctx, int P, int B, int Hkv, int group, int* n_splits, int* pages_per_split);
es_status_t launch_decode_attention(const DecodeAttnParams& p, cudaStream_t s, int64_t* launches, bool pdl = false);
// tensor-core (mma.sync) split kernel for head_dim 128; same partial layout, merged by the same merge kernel
bool decode_attention_mma_supported(const DecodeAttnParams& p);
es_status_t launch_decode_attention_mma(const DecodeAttnParams& p, cudaStream_t s, bool pdl = false);

}  // namespace es

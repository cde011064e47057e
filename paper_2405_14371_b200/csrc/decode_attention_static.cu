// Decode attention for callers that cannot hand over scratch memory: the split-KV partials live in
// a fixed array that is part of the library image instead of a caller buffer.
#include <mutex>

#include "es_internal.cuh"

namespace {

// Room for the per-split partial results (o, max, sum) of one call.  It is reserved on every GPU
// that loads the library, for as long as the process lives, so it is kept modest: 8 MiB covers
// e.g. 16 sequences x 64 heads x 128 dims cut into up to 15 splits.
constexpr size_t STATIC_SCRATCH_BYTES = 8u << 20;
static __device__ __align__(256) unsigned char g_decode_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
void* g_scratch_ptr[MAX_DEVICES] = {};

// In host code `g_decode_scratch` is only a handle for the symbol, not a device address; the real
// address is looked up once per device, with that device current.
es_status_t scratch_address(void** out, cudaStream_t stream) {
  int dev = -1;
  ES_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= MAX_DEVICES) return es::fail(ES_ERR_UNSUPPORTED, "device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    // the look-up may load the module, which a stream capture in progress does not survive
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap != cudaStreamCaptureStatusNone)
      return es::fail(ES_ERR_STATE, "the first call on a device must come before any stream capture");
    void* p = nullptr;
    ES_CUDA_CHECK(cudaGetSymbolAddress(&p, g_decode_scratch));
    if (!p) return es::fail(ES_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return ES_OK;
}

}  // namespace

extern "C" {

size_t es_op_decode_attention_static_capacity(void) { return STATIC_SCRATCH_BYTES; }

es_status_t es_op_decode_attention_static(const void* q, const void* k_pages, const void* v_pages,
                                          const int32_t* block_table, const int32_t* ctx_len, void* out, int32_t B,
                                          int32_t Hq, int32_t Hkv, int32_t hd, int32_t page_tokens,
                                          int32_t pages_per_seq, int32_t max_ctx, void* stream) {
  using namespace es;
  if (!q || !k_pages || !v_pages || !block_table || !ctx_len || !out) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || page_tokens <= 0 || pages_per_seq <= 0 || max_ctx <= 0)
    return fail(ES_ERR_INVALID_ARG, "bad sizes");
  if (max_ctx > page_tokens * pages_per_seq) return fail(ES_ERR_RANGE, "max_ctx exceeds the block table");
  // shapes first: the capacity test below computes with them
  if (hd != 64 && hd != 128) return fail(ES_ERR_SHAPE, "head_dim must be 64 or 128");
  if (Hq % Hkv != 0) return fail(ES_ERR_SHAPE, "Hq must be a multiple of Hkv");
  const int group = Hq / Hkv;
  if (group != 1 && group != 2 && group != 4 && group != 8) return fail(ES_ERR_SHAPE, "Hq / Hkv must be 1, 2, 4 or 8");
  DecodeAttnParams p{};
  p.q = (const __half*)q; p.out = (__half*)out; p.ctx_len = ctx_len; p.ctx_add = 0;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.hd = hd;
  p.kv.k = (const __half*)k_pages; p.kv.v = (const __half*)v_pages; p.kv.block_table = block_table; p.kv.slots = nullptr;
  p.kv.page_stride = (int64_t)Hkv * page_tokens * hd; p.kv.head_stride = (int64_t)page_tokens * hd; p.kv.tok_stride = hd;
  p.kv.P = page_tokens; p.kv.pages_per_slot = pages_per_seq;
  choose_splits(max_ctx, page_tokens, B, Hkv, Hq / Hkv, &p.n_splits, &p.pages_per_split);
  const size_t need = decode_attention_scratch_bytes(B, Hq, hd, p.n_splits);
  if (need > STATIC_SCRATCH_BYTES)
    return fail(ES_ERR_WORKSPACE, "this call needs %zu bytes of split-KV scratch but the built-in array holds %zu; "
                "use es_op_decode_attention with a caller buffer", need, STATIC_SCRATCH_BYTES);
  void* scratch = nullptr;
  ES_TRY(scratch_address(&scratch, (cudaStream_t)stream));
  // The partials need no clearing (every split that the merge reads is written earlier in this same call); the
  // arrival counters that follow them must start at zero.  A fill is not an allocation.
  p.part = (float*)scratch;
  p.split_cnt = (int*)((unsigned char*)scratch + decode_attention_counter_offset(B, Hq, hd, p.n_splits));
  if (p.n_splits > 1)
    ES_CUDA_CHECK(cudaMemsetAsync(p.split_cnt, 0, decode_attention_counter_bytes(B, Hq), (cudaStream_t)stream));
  return launch_decode_attention(p, (cudaStream_t)stream, nullptr);
}

}  // extern "C"

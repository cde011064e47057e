// Host side of the shard library: validation, buffer carving, KV page tables, the per-layer
// launch sequence for prefill and decode, CUDA-graph replay of decode steps, per-layer event
// timing, and the C ABI.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <map>
#include <new>
#include <string>
#include <vector>

#include "es_internal.cuh"
#include "launch.cuh"

namespace es {

// ---- thread-local error text ---------------------------------------------------------------
static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

es_status_t fail(es_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return st;
}

static int env_int(const char* name, int dflt) {
  const char* v = getenv(name);
  return (v && *v) ? atoi(v) : dflt;
}

const Tunables& tunables() {
  static const Tunables t = [] {
    Tunables v;
    v.stream_deep = env_int("ES_STREAM_DEEP", 1);
    v.tc_pair = env_int("ES_TC_PAIR", 1);
    v.tc_pair_wide = env_int("ES_TC_PAIR_WIDE", 1);
    v.split_pairs = env_int("ES_SPLIT_PAIRS", 1);
    v.pdl = env_int("ES_PDL", 1);
    v.attn_mma = env_int("ES_ATTN_MMA", 1);
    v.split_k = env_int("ES_SPLIT_K", 1);
    v.ks_min_slice = env_int("ES_KS_MIN_SLICE", 512);
    v.ks_splits = env_int("ES_KS_SPLITS", 0);
    v.ks_cols = env_int("ES_KS_COLS", 0);
    v.attn_split_tokens = env_int("ES_ATTN_SPLIT_TOKENS", 0);
    v.even_grid = env_int("ES_EVEN_GRID", 0);
    v.debug_checks = env_int("ES_DEBUG", 0);
    return v;
  }();
  return t;
}

int sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 1;
  return n;
}

// How the context of a decode-attention call is cut into splits: enough CTAs to fill the machine,
// never less than one KV page per split.
void choose_splits(int max_ctx, int P, int B, int Hkv, int group, int* n_splits, int* pages_per_split) {
  const int pages = (max_ctx + P - 1) / P;
  // about one CTA per SM when every KV head serves one or two query heads (the kernel then lives on
  // bytes in flight); four times as many for larger groups, whose CTAs are arithmetic heavy
  const int ctas = (group >= 4 ? 4 : 1) * sm_count();
  long long pps = (long long)pages * B * Hkv / ctas;
  // at least 256 tokens per split (384 for large groups, whose CTAs carry more fixed work per split)
  // ... except for one or two sequences with a context beyond 256 tokens: those launches are latency bound, their
  // splits are merged inside the kernel, and 128-token splits measured faster (one sequence of 512..768 keys:
  // 8.3 -> 6.9 us per layer; a context of at most 256 tokens stays one split: 4.9 us against 7.1 with two)
  const bool few = (long long)B * Hkv <= 64 && max_ctx > 256;
  const int min_tokens = tunables().attn_split_tokens > 0 ? tunables().attn_split_tokens : (group >= 4 ? 384 : few ? 128 : 256);
  const int min_pps = min_tokens / P > 1 ? min_tokens / P : 1;
  if (pps < min_pps) pps = min_pps;
  if (pps > pages) pps = pages;
  *pages_per_split = (int)pps;
  *n_splits = (pages + (int)pps - 1) / (int)pps;
}

namespace {

constexpr size_t ALIGN = 256;
constexpr size_t CANARY_BYTES = 256;
constexpr unsigned char CANARY = 0xC5;
inline size_t align_up(size_t v) { return (v + ALIGN - 1) / ALIGN * ALIGN; }

struct Layout {
  int pages_per_slot, n_pages, n_splits, pages_per_split;
  size_t page_elems;   // halves in one page of one of K / V
  size_t kv_bytes;
  size_t off_x, off_h, off_q, off_ao, off_act, off_logits, off_next, off_hlast, off_part, off_cos, off_sin,
      off_table, off_ctx, off_slots, off_status, off_splitk, off_stamps;
  size_t scratch_bytes;
  // every carved region is followed by CANARY_BYTES that no kernel may touch: (offset of the guard, region name)
  std::vector<std::pair<size_t, const char*>> guards;
};

es_status_t validate_desc(const es_model_desc_t* d, int begin, int end) {
  if (!d) return fail(ES_ERR_INVALID_ARG, "desc is null");
  if (d->n_layers_total <= 0 || d->d_model <= 0 || d->n_heads <= 0 || d->n_kv_heads <= 0 || d->head_dim <= 0 ||
      d->d_ffn <= 0 || d->vocab <= 0 || d->max_slots <= 0 || d->max_seq <= 0 || d->max_tokens <= 0 ||
      d->max_batch <= 0 || d->kv_page_tokens <= 0)
    return fail(ES_ERR_INVALID_ARG, "model description has a non-positive field");
  if (begin < 0 || end > d->n_layers_total || begin >= end)
    return fail(ES_ERR_RANGE, "layer range [%d, %d) is not inside [0, %d] or is empty", begin, end, d->n_layers_total);
  if (d->head_dim != 64 && d->head_dim != 128) return fail(ES_ERR_SHAPE, "head_dim must be 64 or 128");
  if (d->n_heads % d->n_kv_heads != 0) return fail(ES_ERR_SHAPE, "n_heads must be a multiple of n_kv_heads");
  const int grp = d->n_heads / d->n_kv_heads;
  if (grp != 1 && grp != 2 && grp != 4 && grp != 8) return fail(ES_ERR_SHAPE, "n_heads / n_kv_heads must be 1, 2, 4 or 8");
  if (d->d_model % 8 != 0 || d->d_ffn % 8 != 0) return fail(ES_ERR_SHAPE, "d_model and d_ffn must be multiples of 8");
  if (d->kv_page_tokens < 16 || (d->kv_page_tokens & (d->kv_page_tokens - 1)))
    return fail(ES_ERR_SHAPE, "kv_page_tokens must be a power of two >= 16");
  if (d->max_batch > d->max_slots) return fail(ES_ERR_INVALID_ARG, "max_batch exceeds max_slots");
  if (d->max_tokens < d->max_batch) return fail(ES_ERR_INVALID_ARG, "max_tokens is smaller than max_batch");
  if (!(d->rms_eps >= 0.f) || !(d->rope_theta > 0.f)) return fail(ES_ERR_INVALID_ARG, "rms_eps / rope_theta out of range");
  return ES_OK;
}

Layout make_layout(const es_model_desc_t& d, int begin, int end) {
  Layout L{};
  const int nl = end - begin;
  const int P = d.kv_page_tokens;
  L.pages_per_slot = (d.max_seq + P - 1) / P;
  L.n_pages = L.pages_per_slot * d.max_slots;
  L.page_elems = (size_t)d.n_kv_heads * P * d.head_dim;
  L.kv_bytes = align_up((size_t)nl * 2 * L.n_pages * L.page_elems * sizeof(__half));
  choose_splits(d.max_seq, P, d.max_batch, d.n_kv_heads, d.n_heads / d.n_kv_heads, &L.n_splits, &L.pages_per_split);
  const size_t M = d.max_tokens, B = d.max_batch, nq = (size_t)d.n_heads * d.head_dim;
  const bool head = end == d.n_layers_total;
  size_t o = 0;
  auto take = [&](size_t bytes, const char* name) {
    size_t at = o;
    o += align_up(bytes);
    L.guards.emplace_back(o, name);
    o += CANARY_BYTES;
    return at;
  };
  L.off_x = take(M * d.d_model * 4, "residual stream");
  L.off_h = take(M * d.d_model * 2, "normalised activations");
  L.off_q = take(M * nq * 2, "q");
  L.off_ao = take(M * nq * 2, "attention output");
  L.off_act = take(M * (size_t)d.d_ffn * 2, "ffn activations");
  L.off_logits = take(head ? B * (size_t)d.vocab * 4 : 0, "logits");
  L.off_next = take(B * 4, "next ids");
  L.off_hlast = take(B * (size_t)d.d_model * 2, "last-row norm");
  L.off_part = take(decode_attention_scratch_bytes((int)B, d.n_heads, d.head_dim, L.n_splits), "attention partials");
  L.off_cos = take((size_t)d.max_seq * (d.head_dim / 2) * 4, "rope cos");
  L.off_sin = take((size_t)d.max_seq * (d.head_dim / 2) * 4, "rope sin");
  L.off_table = take((size_t)L.n_pages * 4, "page table");
  L.off_ctx = take((size_t)d.max_slots * 4, "context lengths");
  L.off_slots = take((3 * B + 1) * 4, "slots");  // slots, the prompt lengths of a ragged prefill, the first rows of packed prompts
  L.off_status = take(256, "status words");
  L.off_splitk = take(d.max_tokens > 2 ? linear_tc_split_workspace_bytes() : 0, "split-K workspace");   // split-K partial sums of short prefills
  L.off_stamps = take((size_t)2 * STAMP_SLOTS * sizeof(unsigned long long), "time stamps");
  L.scratch_bytes = o;
  return L;
}

struct ProfileEntry {
  int layer;
  cudaEvent_t ev[2];
  double prefill_ms = 0, decode_ms = 0;
  int n_prefill = 0, n_decode = 0;
};

// A captured decode step is valid for one batch size and one pair of input pointers; slots and
// positions are read from device memory at run time.
struct GraphKey {
  int B;
  const void* ids;
  const void* hidden;
  bool operator<(const GraphKey& o) const {
    if (B != o.B) return B < o.B;
    if (ids != o.ids) return ids < o.ids;
    return hidden < o.hidden;
  }
};

struct GraphEntry {
  cudaGraphExec_t exec = nullptr;
  int64_t nodes = 0;
};

}  // namespace
}  // namespace es

using namespace es;

struct es_shard {
  es_model_desc_t d;
  int begin, end, nl;
  bool has_emb, has_head;
  std::vector<es_layer_weights_t> lw;
  const __half *emb = nullptr, *fnorm = nullptr, *lmh = nullptr;
  cudaStream_t stream = nullptr;
  Layout lay;
  __half* kv = nullptr;
  unsigned char* scratch = nullptr;
  float* x;
  __half *h, *q, *ao, *act, *h_last;
  float *logits, *part, *rope_cos, *rope_sin;
  int *next_ids, *block_table, *ctx_len, *slots_dev, *lens_dev, *cu_dev, *status;
  float* splitk = nullptr;      // split-K workspace (nullptr when the shard never runs more than 2 rows)
  std::vector<int> ctx;         // host mirror of ctx_len, -1 = never prefilled
  std::vector<int> slots_host;  // slots currently uploaded to slots_dev
  std::vector<int> lens_host;   // prompt lengths of the last ragged prefill (source of the upload)
  std::vector<int> cu_host;     // first rows of the last packed prefill (source of the upload)
  int last_B = 0, last_T = 0;
  int last_head_rows = 0;      // rows of logits / next ids of the last pass (sequences, also when the hidden rows are packed)
  bool last_valid = false;
  int64_t launches = 0;
  bool profiling = false;
  bool pending = false, pending_prefill = false;
  std::vector<ProfileEntry> prof;
  bool graphs = true;
  bool pdl_now = false;   // the pass being enqueued uses programmatic dependent launch (decode steps)
  const int* pass_cu = nullptr;   // the pass being enqueued is a prefill of packed prompts: their first-row table (device)
  int pass_n_seq = 0;
  std::map<GraphKey, GraphEntry> graph_cache;
  // tensor maps of the prefill GEMMs, encoded once: [layer][qkv, o, gate/up, down]
  std::vector<TcMaps> tmaps;
  bool tmaps_valid = false;
  std::vector<TcMaps> attn_maps;        // per layer {q, k pages, v pages}
  bool attn_maps_valid = false;
  // launch-by-launch timing of the linear-layer kernels (off by default)
  bool kernel_timing = false;
  std::vector<cudaEvent_t> kt_events;   // pairs
  std::vector<int> kt_cat;              // category of each pair
  std::vector<double> kt_pair_bytes;    // algorithmic bytes of each pair
  size_t kt_used = 0;
  int kt_next_cat = 0;
  // time stamps written by the kernels of the last enqueued (or captured) pass: see es_shard_set_step_timing
  unsigned long long* stamps = nullptr;   // device: STAMP_SLOTS earliest starts, then STAMP_SLOTS latest ends
  bool step_timing = false;
  int st_used = 0;
  std::vector<int> st_cat;
  std::vector<double> st_bytes;

  __half* k_pages(int li) const { return kv + (size_t)(2 * li) * lay.n_pages * lay.page_elems; }
  __half* v_pages(int li) const { return kv + (size_t)(2 * li + 1) * lay.n_pages * lay.page_elems; }
};

namespace es {
namespace {

es_status_t harvest_profile(es_shard* s) {
  if (!s->pending) return ES_OK;
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  for (auto& e : s->prof) {
    float ms = 0.f;
    ES_CUDA_CHECK(cudaEventElapsedTime(&ms, e.ev[0], e.ev[1]));
    if (s->pending_prefill) { e.prefill_ms += ms; e.n_prefill++; }
    else { e.decode_ms += ms; e.n_decode++; }
  }
  s->pending = false;
  return ES_OK;
}

es_status_t upload_slots(es_shard* s, const int32_t* slots, int B) {
  if ((int)s->slots_host.size() == B && memcmp(s->slots_host.data(), slots, B * sizeof(int)) == 0) return ES_OK;
  s->slots_host.assign(slots, slots + B);
  ES_CUDA_CHECK(cudaMemcpyAsync(s->slots_dev, s->slots_host.data(), B * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  return ES_OK;
}

es_status_t check_tensor(const es_tensor_t* t, int64_t rows, int64_t d, const char* what) {
  if (!t->data) return fail(ES_ERR_INVALID_ARG, "%s: data is null", what);
  if (t->dtype != ES_DTYPE_F32) return fail(ES_ERR_INVALID_ARG, "%s: must be fp32", what);
  int64_t n = 1;
  if (t->rank < 1 || t->rank > 4) return fail(ES_ERR_INVALID_ARG, "%s: bad rank", what);
  for (int i = 0; i < t->rank; ++i) n *= t->shape[i];
  if (n != rows * d || t->shape[t->rank - 1] != d)
    return fail(ES_ERR_SHAPE, "%s: expected %lld x %lld elements", what, (long long)rows, (long long)d);
  return ES_OK;
}

es_status_t dispatch_linear(es_shard* s, const LinearParams& p, int epi) {
  if (p.M > 2 && p.M <= 16 && linear_stream_mma_supported(p, epi))
    return launch_linear_stream_mma(p, epi, s->stream, &s->launches, s->pdl_now);
  if (p.M <= 16) return launch_linear_stream(p, epi, s->stream, &s->launches, s->pdl_now);
  if (p.k_splits > 1)
    return p.split_on_pairs ? launch_linear_tc2(p, epi, s->stream, &s->launches, s->status, s->pdl_now)
                            : launch_linear_tc(p, epi, s->stream, &s->launches, s->status, s->pdl_now);
  if (tunables().tc_pair && linear_tc2_supported(p, epi)) return launch_linear_tc2(p, epi, s->stream, &s->launches, s->status, s->pdl_now);
  if (linear_tc_supported(p, epi)) return launch_linear_tc(p, epi, s->stream, &s->launches, s->status, s->pdl_now);
  return launch_linear_reference(p, epi, s->stream, &s->launches);
}

// Launch-by-launch timing: an event pair around one launch, tagged with a category.
es_status_t kt_begin(es_shard* s) {
  if (!s->kernel_timing) return ES_OK;
  if (s->kt_used + 2 > s->kt_events.size()) {
    cudaEvent_t a, b;
    ES_CUDA_CHECK(cudaEventCreate(&a));
    ES_CUDA_CHECK(cudaEventCreate(&b));
    s->kt_events.push_back(a);
    s->kt_events.push_back(b);
  }
  ES_CUDA_CHECK(cudaEventRecord(s->kt_events[s->kt_used], s->stream));
  return ES_OK;
}

// Time-stamp slot for the next launch (nullptr unless step timing is on), tagged like an event pair.
unsigned long long* next_stamp(es_shard* s, int cat, double bytes) {
  if (!s->step_timing || s->st_used >= STAMP_SLOTS) return nullptr;
  s->st_cat.push_back(cat);
  s->st_bytes.push_back(bytes);
  return s->stamps + s->st_used++;
}

es_status_t kt_end(es_shard* s, int cat, double bytes) {
  if (!s->kernel_timing) return ES_OK;
  ES_CUDA_CHECK(cudaEventRecord(s->kt_events[s->kt_used + 1], s->stream));
  s->kt_used += 2;
  s->kt_cat.push_back(cat);
  s->kt_pair_bytes.push_back(bytes);
  return ES_OK;
}

es_status_t run_linear(es_shard* s, const LinearParams& p0, int epi) {
  LinearParams p = p0;
  const double bytes = (double)p.N * p.K * 2.0 * (epi == EPI_SWIGLU ? 2.0 : 1.0);
  p.stamp = next_stamp(s, s->kt_next_cat, bytes);
  ES_TRY(kt_begin(s));
  ES_TRY(dispatch_linear(s, p, epi));
  return kt_end(s, s->kt_next_cat, bytes);
}

LinearParams base_params(const es_shard* s, int M, int T, bool decode) {
  LinearParams p{};
  p.M = M;
  p.T = T;
  p.is_decode = decode ? 1 : 0;
  p.block_table = s->block_table;
  p.ctx_len = s->ctx_len;
  p.slots = s->slots_dev;
  p.rope_cos = s->rope_cos;
  p.rope_sin = s->rope_sin;
  p.Hq = s->d.n_heads;
  p.Hkv = s->d.n_kv_heads;
  p.hd = s->d.head_dim;
  p.P = s->d.kv_page_tokens;
  p.pages_per_slot = s->lay.pages_per_slot;
  p.max_seq = s->d.max_seq;
  p.cu_rows = s->pass_cu;
  p.n_seq = s->pass_n_seq;
  return p;
}

// K slices for a product on the tensor-core path (1 = whole K range per tile).
int split_k_for(const es_shard* s, LinearParams& p, int epi) {
  p.split_on_pairs = 0;
  if (s->splitk == nullptr || p.M <= 2 || tunables().split_k == 0) return 1;
  if (p.M <= 16) return linear_stream_mma_splits(p, epi, linear_tc_split_workspace_bytes());   // decode with several sequences
  if (!linear_tc_supported(p, epi)) return 1;
  if (tunables().tc_pair && tunables().split_pairs) {
    const int ps = linear_tc2_splits(p, epi);        // 256 or more rows: slices on CTA pairs
    if (ps > 1) { p.split_on_pairs = 1; return ps; }
  }
  return linear_tc_splits(p, epi);
}

// A product whose K range may be sliced (QKV and gate / up forms): the kernel, then the finishing kernel.
es_status_t run_linear_sliced(es_shard* s, LinearParams& p, int epi, bool pdl) {
  const int splits = split_k_for(s, p, epi);
  if (splits <= 1 || p.M > 16) return run_linear(s, p, epi);
  p.k_splits = splits;
  p.part = s->splitk;
  ES_TRY(run_linear(s, p, epi));
  p.stamp = next_stamp(s, ES_KT_FINISH, 0.0);
  ES_TRY(kt_begin(s));
  ES_TRY(launch_splitk_finish(p, epi, s->stream, &s->launches, pdl));
  return kt_end(s, ES_KT_FINISH, 0.0);
}

// Parameters of the four linear layers of decoder layer li (kind: 0 qkv, 1 o, 2 gate/up, 3 down).
LinearParams layer_linear(const es_shard* s, int li, int kind, int M, int T, bool decode, const float* xin, int* epi) {
  const es_model_desc_t& d = s->d;
  const es_layer_weights_t& w = s->lw[li];
  const int nq = d.n_heads * d.head_dim, nkv = d.n_kv_heads * d.head_dim;
  LinearParams p = base_params(s, M, T, decode);
  switch (kind) {
    case 0:
      p.A = s->h; p.lda = d.d_model; p.K = d.d_model; p.N = nq + 2 * nkv;
      p.w[0] = (const __half*)w.wq; p.w[1] = (const __half*)w.wk; p.w[2] = (const __half*)w.wv;
      p.seg_rows[0] = nq; p.seg_rows[1] = nkv; p.seg_rows[2] = nkv;
      p.out_f16 = s->q; p.k_cache = s->k_pages(li); p.v_cache = s->v_pages(li);
      *epi = EPI_QKV;
      break;
    case 1:
      p.A = s->ao; p.lda = nq; p.K = nq; p.N = d.d_model;
      p.w[0] = (const __half*)w.wo; p.seg_rows[0] = d.d_model;
      p.out_f32 = s->x; p.res = xin; p.ldo = d.d_model;
      *epi = EPI_F32;
      break;
    case 2:
      p.A = s->h; p.lda = d.d_model; p.K = d.d_model; p.N = d.d_ffn;
      p.w[0] = (const __half*)w.w_gate; p.w[1] = (const __half*)w.w_up; p.seg_rows[0] = d.d_ffn;
      p.out_f16 = s->act; p.ldo = d.d_ffn;
      *epi = EPI_SWIGLU;
      break;
    default:
      p.A = s->act; p.lda = d.d_ffn; p.K = d.d_ffn; p.N = d.d_model;
      p.w[0] = (const __half*)w.w_down; p.seg_rows[0] = d.d_model;
      p.out_f32 = s->x; p.res = s->x; p.ldo = d.d_model;
      *epi = EPI_F32;
      break;
  }
  if (s->tmaps_valid && M > 16) p.tc_maps = &s->tmaps[(size_t)li * 4 + kind];
  return p;
}

inline void prof_mark(es_shard* s, int idx, int which) {
  if (s->profiling) cudaEventRecord(s->prof[idx].ev[which], s->stream);
}

// The launch sequence of one pass (prefill: T tokens per sequence; decode: T == 1 at each slot's
// next position).  Everything is enqueued on s->stream.
// lens (device, [B]) != nullptr: a prefill of right-padded prompts; sequence b has lens[b] <= T real tokens
// cu (device, [B + 1]) != nullptr: a prefill of PACKED prompts; sequence b owns rows cu[b] .. cu[b + 1] - 1 of the
// total_rows rows, T is the longest prompt, lens its lengths
es_status_t enqueue_pass(es_shard* s, const int32_t* ids, const float* hidden_in, int B, int T, bool decode,
                         const int* lens = nullptr, const int* cu = nullptr, int total_rows = 0) {
  const es_model_desc_t& d = s->d;
  const int M = cu ? total_rows : B * T;
  s->pass_cu = cu;
  s->pass_n_seq = cu ? B : 0;
  int pi = 0;
  const float* xin = s->x;
  const bool pdl = tunables().pdl != 0;
  s->pdl_now = pdl;
  const bool fuse_norm = M <= 16 && linear_stream_can_fuse_norm(M);
  bool h_ready = false;   // s->h already holds the normalised input of the coming layer
  if (s->step_timing) {
    s->st_used = 0;
    s->st_cat.clear();
    s->st_bytes.clear();
    ES_CUDA_CHECK(cudaMemsetAsync(s->stamps, 0xFF, STAMP_SLOTS * sizeof(unsigned long long), s->stream));
    ES_CUDA_CHECK(cudaMemsetAsync(s->stamps + STAMP_SLOTS, 0, STAMP_SLOTS * sizeof(unsigned long long), s->stream));
  }
  if (s->has_emb) {
    prof_mark(s, pi, 0);
    ES_TRY(kt_begin(s));
    // the first kernel of a pass is launched with a full dependency: everything from earlier passes
    // has completed before any kernel of this pass begins
    ES_TRY(launch_embed(ids, s->emb, s->x, M, d.d_model, d.vocab, s->stream, &s->launches, false,
                        next_stamp(s, ES_KT_EMBED, (double)M * d.d_model * 6.0)));
    ES_TRY(kt_end(s, ES_KT_EMBED, (double)M * d.d_model * 6.0));
    prof_mark(s, pi, 1);
    ++pi;
  } else {
    xin = hidden_in;
  }
  for (int li = 0; li < s->nl; ++li, ++pi) {
    const es_layer_weights_t& w = s->lw[li];
    prof_mark(s, pi, 0);
    const bool pdl0 = (li == 0 && !s->has_emb) ? false : pdl;     // first kernel of the pass: full dependency
    if (!fuse_norm && !h_ready) {
      ES_TRY(kt_begin(s));
      ES_TRY(launch_rmsnorm(xin, (const __half*)w.attn_norm, s->h, M, d.d_model, d.rms_eps, 1, 0, s->stream, &s->launches, pdl0,
                            nullptr, next_stamp(s, ES_KT_RMSNORM, (double)M * d.d_model * 6.0)));
      ES_TRY(kt_end(s, ES_KT_RMSNORM, (double)M * d.d_model * 6.0));
    }
    h_ready = false;
    int epi = 0;
    {
      LinearParams p = layer_linear(s, li, 0, M, T, decode, xin, &epi);
      if (fuse_norm) { p.norm_x = xin; p.norm_ldx = d.d_model; p.norm_gain = (const __half*)w.attn_norm; p.norm_eps = d.rms_eps; }
      s->kt_next_cat = ES_KT_QKV;
      s->pdl_now = fuse_norm ? pdl0 : pdl;
      ES_TRY(run_linear_sliced(s, p, epi, pdl));
      s->pdl_now = pdl;
    }
    KvView kvv{};
    kvv.k = s->k_pages(li); kvv.v = s->v_pages(li);
    kvv.block_table = s->block_table; kvv.slots = s->slots_dev;
    kvv.page_stride = (int64_t)s->lay.page_elems; kvv.head_stride = (int64_t)d.kv_page_tokens * d.head_dim;
    kvv.tok_stride = d.head_dim; kvv.P = d.kv_page_tokens; kvv.pages_per_slot = s->lay.pages_per_slot;
    ES_TRY(kt_begin(s));
    if (decode) {
      DecodeAttnParams a{};
      a.q = s->q; a.out = s->ao; a.kv = kvv; a.ctx_len = s->ctx_len; a.ctx_add = 1; a.part = s->part;
      // the counters sit behind the partials of the LARGEST batch, so that no batch's partials ever cover them
      a.split_cnt = (int*)((unsigned char*)s->part + decode_attention_counter_offset(d.max_batch, d.n_heads, d.head_dim, s->lay.n_splits));
      a.B = B; a.Hq = d.n_heads; a.Hkv = d.n_kv_heads; a.hd = d.head_dim;
      a.n_splits = s->lay.n_splits; a.pages_per_split = s->lay.pages_per_split;
      a.stamp = next_stamp(s, ES_KT_ATTENTION, 0.0);
      ES_TRY(launch_decode_attention(a, s->stream, &s->launches, pdl));
    } else {
      PrefillAttnParams a{};
      a.q = s->q; a.out = s->ao; a.kv = kvv; a.B = B; a.T = T; a.Hq = d.n_heads; a.Hkv = d.n_kv_heads; a.hd = d.head_dim;
      a.kv_rows = (int64_t)s->lay.n_pages * d.n_kv_heads * d.kv_page_tokens;
      a.status = s->status;
      a.tc_maps = s->attn_maps_valid ? &s->attn_maps[li] : nullptr;
      a.cu_rows = cu;
      a.stamp = next_stamp(s, ES_KT_ATTENTION, 0.0);
      ES_TRY(launch_prefill_attention(a, s->stream, &s->launches, 0, pdl));
    }
    ES_TRY(kt_end(s, ES_KT_ATTENTION, 0.0));
    bool o_split = false;
    {
      LinearParams p = layer_linear(s, li, 1, M, T, decode, xin, &epi);
      s->kt_next_cat = ES_KT_O;
      const int splits = split_k_for(s, p, epi);
      if (splits > 1) {
        // short prompt: K slices into the workspace, then residual + RMSNorm for gate / up in the reduction
        p.k_splits = splits; p.part = s->splitk;
        ES_TRY(run_linear(s, p, epi));
        ES_TRY(kt_begin(s));
        ES_TRY(launch_splitk_reduce(s->splitk, splits, p.res, p.out_f32, M, p.N, p.ldo, (const __half*)w.ffn_norm, s->h,
                                    d.rms_eps, s->stream, &s->launches, pdl,
                                    next_stamp(s, ES_KT_REDUCE, (double)M * d.d_model * (8.0 + 4.0 * splits + 2.0))));
        ES_TRY(kt_end(s, ES_KT_REDUCE, (double)M * d.d_model * (8.0 + 4.0 * splits + 2.0)));
        o_split = true;
      } else {
        ES_TRY(run_linear(s, p, epi));
      }
    }
    xin = s->x;
    if (!fuse_norm && !o_split) {
      ES_TRY(kt_begin(s));
      ES_TRY(launch_rmsnorm(s->x, (const __half*)w.ffn_norm, s->h, M, d.d_model, d.rms_eps, 1, 0, s->stream, &s->launches, pdl,
                            nullptr, next_stamp(s, ES_KT_RMSNORM, (double)M * d.d_model * 6.0)));
      ES_TRY(kt_end(s, ES_KT_RMSNORM, (double)M * d.d_model * 6.0));
    }
    {
      LinearParams p = layer_linear(s, li, 2, M, T, decode, xin, &epi);
      if (fuse_norm) { p.norm_x = s->x; p.norm_ldx = d.d_model; p.norm_gain = (const __half*)w.ffn_norm; p.norm_eps = d.rms_eps; }
      s->kt_next_cat = ES_KT_GATE_UP;
      ES_TRY(run_linear_sliced(s, p, epi, pdl));
    }
    {
      LinearParams p = layer_linear(s, li, 3, M, T, decode, xin, &epi);
      s->kt_next_cat = ES_KT_DOWN;
      const int splits = split_k_for(s, p, epi);
      if (splits > 1) {
        // the reduction also normalises the finished rows for the next layer's QKV projection
        p.k_splits = splits; p.part = s->splitk;
        ES_TRY(run_linear(s, p, epi));
        const bool more = li + 1 < s->nl;
        ES_TRY(kt_begin(s));
        ES_TRY(launch_splitk_reduce(s->splitk, splits, p.res, p.out_f32, M, p.N, p.ldo,
                                    more ? (const __half*)s->lw[li + 1].attn_norm : nullptr, s->h, d.rms_eps, s->stream,
                                    &s->launches, pdl,
                                    next_stamp(s, ES_KT_REDUCE, (double)M * d.d_model * (8.0 + 4.0 * splits + (more ? 2.0 : 0.0)))));
        ES_TRY(kt_end(s, ES_KT_REDUCE, (double)M * d.d_model * (8.0 + 4.0 * splits + (more ? 2.0 : 0.0))));
        h_ready = more;
      } else {
        ES_TRY(run_linear(s, p, epi));
      }
    }
    prof_mark(s, pi, 1);
  }
  if (s->has_head) {
    prof_mark(s, pi, 0);
    // last position of every sequence only
    const bool fuse_head = lens == nullptr && linear_stream_can_fuse_norm(B);
    if (!fuse_head) {
      ES_TRY(kt_begin(s));
      // last row of every sequence: row b * T + lens[b] - 1, or with packed prompts row cu[b + 1] - 1
      ES_TRY(launch_rmsnorm(s->x, s->fnorm, s->h_last, B, d.d_model, d.rms_eps, cu ? 0 : T, T - 1, s->stream, &s->launches, pdl,
                            cu ? cu + 1 : lens,
                            next_stamp(s, ES_KT_RMSNORM, (double)B * d.d_model * 6.0)));
      ES_TRY(kt_end(s, ES_KT_RMSNORM, (double)B * d.d_model * 6.0));
    }
    for (int b0 = 0; b0 < B; b0 += 16) {
      LinearParams p = base_params(s, (B - b0 < 16 ? B - b0 : 16), 1, decode);
      p.A = s->h_last + (size_t)b0 * d.d_model; p.lda = d.d_model; p.K = d.d_model; p.N = d.vocab;
      p.w[0] = s->lmh; p.seg_rows[0] = d.vocab;
      p.out_f32 = s->logits + (size_t)b0 * d.vocab; p.res = nullptr; p.ldo = d.vocab;
      if (fuse_head) {
        p.norm_x = s->x + (size_t)(T - 1) * d.d_model; p.norm_ldx = (int64_t)T * d.d_model;
        p.norm_gain = s->fnorm; p.norm_eps = d.rms_eps;
      }
      s->kt_next_cat = ES_KT_LM_HEAD;
      ES_TRY(run_linear(s, p, EPI_F32));
    }
    ES_TRY(kt_begin(s));
    ES_TRY(launch_argmax(s->logits, s->next_ids, B, d.vocab, s->stream, &s->launches, pdl,
                         next_stamp(s, ES_KT_ARGMAX, (double)B * d.vocab * 4.0)));
    ES_TRY(kt_end(s, ES_KT_ARGMAX, (double)B * d.vocab * 4.0));
    prof_mark(s, pi, 1);
  }
  // the slots' contexts now hold T (prefill) or one more (decode) position
  ES_TRY(kt_begin(s));
  ES_TRY(launch_set_ctx(s->ctx_len, s->slots_dev, B, decode ? 1 : T, decode ? 1 : 0, s->stream, &s->launches, pdl, lens,
                        next_stamp(s, ES_KT_SET_CTX, 0.0)));
  ES_TRY(kt_end(s, ES_KT_SET_CTX, 0.0));
  s->pdl_now = false;
  s->pass_cu = nullptr;
  s->pass_n_seq = 0;
  return ES_OK;
}

es_status_t check_slots(const es_shard* s, const int32_t* slots, int B) {
  if (!slots) return fail(ES_ERR_INVALID_ARG, "slots is null");
  for (int b = 0; b < B; ++b) {
    if (slots[b] < 0 || slots[b] >= s->d.max_slots)
      return fail(ES_ERR_RANGE, "slot %d (batch row %d) outside [0, %d)", slots[b], b, s->d.max_slots);
    for (int c = 0; c < b; ++c)
      if (slots[c] == slots[b]) return fail(ES_ERR_INVALID_ARG, "slot %d appears twice in the batch", slots[b]);
  }
  return ES_OK;
}

es_status_t check_inputs(const es_shard* s, const int32_t* ids, const es_tensor_t* hidden_in, int64_t rows,
                         const float** hin) {
  *hin = nullptr;
  if (s->has_emb) {
    if (!ids || hidden_in) return fail(ES_ERR_INVALID_ARG, "this shard holds the embedding: pass ids, not hidden_in");
  } else {
    if (ids || !hidden_in) return fail(ES_ERR_INVALID_ARG, "this shard starts at layer %d: pass hidden_in, not ids", s->begin);
    ES_TRY(check_tensor(hidden_in, rows, s->d.d_model, "hidden_in"));
    *hin = (const float*)hidden_in->data;
  }
  return ES_OK;
}

// The checking mode (ES_DEBUG=1): the guard bytes behind every carved region of the scratch buffer must be intact
// (a kernel that wrote past its region lands there first), and the tables the kernels index with must hold values
// inside their ranges: page numbers, context lengths, the uploaded slot list.  Reads device memory; synchronises.
es_status_t debug_checks(es_shard* s) {
  std::vector<unsigned char> g(CANARY_BYTES);
  for (const auto& gd : s->lay.guards) {
    ES_CUDA_CHECK(cudaMemcpy(g.data(), s->scratch + gd.first, CANARY_BYTES, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < CANARY_BYTES; ++i)
      if (g[i] != CANARY) return fail(ES_ERR_STATE, "debug check: the guard behind '%s' was overwritten at byte %zu", gd.second, i);
  }
  std::vector<int> table(s->lay.n_pages), ctx(s->d.max_slots);
  ES_CUDA_CHECK(cudaMemcpy(table.data(), s->block_table, table.size() * 4, cudaMemcpyDeviceToHost));
  ES_CUDA_CHECK(cudaMemcpy(ctx.data(), s->ctx_len, ctx.size() * 4, cudaMemcpyDeviceToHost));
  for (int i = 0; i < s->lay.n_pages; ++i)
    if (table[i] < 0 || table[i] >= s->lay.n_pages) return fail(ES_ERR_STATE, "debug check: page table entry %d = %d", i, table[i]);
  for (int i = 0; i < s->d.max_slots; ++i) {
    if (ctx[i] < 0 || ctx[i] > s->d.max_seq) return fail(ES_ERR_STATE, "debug check: context length of slot %d = %d", i, ctx[i]);
    if (s->ctx[i] >= 0 && ctx[i] != s->ctx[i])
      return fail(ES_ERR_STATE, "debug check: slot %d holds %d positions on the device, %d on the host", i, ctx[i], s->ctx[i]);
  }
  if (!s->slots_host.empty()) {
    std::vector<int> sl(s->slots_host.size());
    ES_CUDA_CHECK(cudaMemcpy(sl.data(), s->slots_dev, sl.size() * 4, cudaMemcpyDeviceToHost));
    for (size_t i = 0; i < sl.size(); ++i)
      if (sl[i] != s->slots_host[i]) return fail(ES_ERR_STATE, "debug check: uploaded slot %zu = %d, expected %d", i, sl[i], s->slots_host[i]);
  }
  return ES_OK;
}

es_status_t debug_checks_now(es_shard* s) {
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  return debug_checks(s);
}

}  // namespace
}  // namespace es

// =============================================================================================
// C ABI

extern "C" {

const char* es_last_error(void) { return es::g_err; }
const char* es_version(void) { return "edgeshard-b200 0.1 (sm_100a)"; }

es_status_t es_shard_workspace_bytes(const es_model_desc_t* desc, int32_t layer_begin, int32_t layer_end,
                                     size_t* kv_bytes, size_t* scratch_bytes) {
  ES_TRY(validate_desc(desc, layer_begin, layer_end));
  const Layout L = make_layout(*desc, layer_begin, layer_end);
  if (kv_bytes) *kv_bytes = L.kv_bytes;
  if (scratch_bytes) *scratch_bytes = L.scratch_bytes;
  return ES_OK;
}

es_status_t es_shard_create(const es_model_desc_t* desc, int32_t layer_begin, int32_t layer_end,
                            const es_weights_t* weights, void* kv_buffer, size_t kv_bytes, void* scratch_buffer,
                            size_t scratch_bytes, void* cuda_stream, es_shard_t** out) {
  ES_TRY(validate_desc(desc, layer_begin, layer_end));
  if (!weights || !weights->layers || !kv_buffer || !scratch_buffer || !out)
    return fail(ES_ERR_INVALID_ARG, "null argument");
  const Layout L = make_layout(*desc, layer_begin, layer_end);
  if (kv_bytes < L.kv_bytes) return fail(ES_ERR_WORKSPACE, "kv buffer: %zu bytes given, %zu needed", kv_bytes, L.kv_bytes);
  if (scratch_bytes < L.scratch_bytes)
    return fail(ES_ERR_WORKSPACE, "scratch buffer: %zu bytes given, %zu needed", scratch_bytes, L.scratch_bytes);
  if (((uintptr_t)kv_buffer | (uintptr_t)scratch_buffer) % ALIGN)
    return fail(ES_ERR_INVALID_ARG, "kv / scratch buffers must be %zu-byte aligned", ALIGN);
  const bool has_emb = layer_begin == 0, has_head = layer_end == desc->n_layers_total;
  if (has_emb && !weights->tok_embedding) return fail(ES_ERR_INVALID_ARG, "tok_embedding is required when layer_begin == 0");
  if (has_head && (!weights->final_norm || !weights->lm_head))
    return fail(ES_ERR_INVALID_ARG, "final_norm and lm_head are required when layer_end == n_layers_total");
  const int nl = layer_end - layer_begin;
  for (int i = 0; i < nl; ++i) {
    const es_layer_weights_t& w = weights->layers[i];
    const void* ptrs[9] = {w.attn_norm, w.wq, w.wk, w.wv, w.wo, w.ffn_norm, w.w_gate, w.w_up, w.w_down};
    for (int j = 0; j < 9; ++j) {
      if (!ptrs[j]) return fail(ES_ERR_INVALID_ARG, "layer %d: weight pointer %d is null", layer_begin + i, j);
      if ((uintptr_t)ptrs[j] % 16) return fail(ES_ERR_INVALID_ARG, "layer %d: weight pointer %d is not 16-byte aligned", layer_begin + i, j);
    }
  }
  es_shard* s = new (std::nothrow) es_shard();
  if (!s) return fail(ES_ERR_INVALID_ARG, "out of host memory");
  s->d = *desc;
  s->begin = layer_begin; s->end = layer_end; s->nl = nl;
  s->has_emb = has_emb; s->has_head = has_head;
  s->lw.assign(weights->layers, weights->layers + nl);
  s->emb = (const __half*)weights->tok_embedding;
  s->fnorm = (const __half*)weights->final_norm;
  s->lmh = (const __half*)weights->lm_head;
  s->stream = (cudaStream_t)cuda_stream;
  s->lay = L;
  s->kv = (__half*)kv_buffer;
  unsigned char* sb = (unsigned char*)scratch_buffer;
  s->scratch = sb;
  s->x = (float*)(sb + L.off_x);
  s->h = (__half*)(sb + L.off_h);
  s->q = (__half*)(sb + L.off_q);
  s->ao = (__half*)(sb + L.off_ao);
  s->act = (__half*)(sb + L.off_act);
  s->logits = (float*)(sb + L.off_logits);
  s->next_ids = (int*)(sb + L.off_next);
  s->h_last = (__half*)(sb + L.off_hlast);
  s->part = (float*)(sb + L.off_part);
  s->rope_cos = (float*)(sb + L.off_cos);
  s->rope_sin = (float*)(sb + L.off_sin);
  s->block_table = (int*)(sb + L.off_table);
  s->ctx_len = (int*)(sb + L.off_ctx);
  s->slots_dev = (int*)(sb + L.off_slots);
  s->lens_dev = s->slots_dev + desc->max_batch;
  s->cu_dev = s->lens_dev + desc->max_batch;
  s->status = (int*)(sb + L.off_status);
  s->splitk = desc->max_tokens > 2 ? (float*)(sb + L.off_splitk) : nullptr;
  s->stamps = (unsigned long long*)(sb + L.off_stamps);
  s->ctx.assign(desc->max_slots, -1);

  auto bail = [&](es_status_t st) { delete s; return st; };
  // rotary table: angle = pos * theta^(-2i/hd), evaluated in double, stored as fp32
  {
    const int half_hd = desc->head_dim / 2;
    std::vector<float> c((size_t)desc->max_seq * half_hd), sn(c.size());
    for (int i = 0; i < half_hd; ++i) {
      const double inv = pow((double)desc->rope_theta, -2.0 * i / desc->head_dim);
      for (int p = 0; p < desc->max_seq; ++p) {
        c[(size_t)p * half_hd + i] = (float)cos(p * inv);
        sn[(size_t)p * half_hd + i] = (float)sin(p * inv);
      }
    }
    std::vector<int> table(L.n_pages);
    for (int i = 0; i < L.n_pages; ++i) table[i] = i;
    cudaError_t e = cudaMemcpyAsync(s->rope_cos, c.data(), c.size() * 4, cudaMemcpyHostToDevice, s->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s->rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice, s->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s->block_table, table.data(), table.size() * 4, cudaMemcpyHostToDevice, s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->ctx_len, 0, (size_t)desc->max_slots * 4, s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->status, 0, 256, s->stream);
    for (const auto& g : L.guards)
      if (e == cudaSuccess) e = cudaMemsetAsync(sb + g.first, CANARY, CANARY_BYTES, s->stream);
    if (e == cudaSuccess)       // arrival counters of the decode-attention splits (they follow the partials)
      e = cudaMemsetAsync(s->part, 0, decode_attention_scratch_bytes((int)desc->max_batch, desc->n_heads, desc->head_dim, L.n_splits), s->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(s->kv, 0, L.kv_bytes, s->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);
    if (e != cudaSuccess) return bail(fail(ES_ERR_CUDA, "shard initialisation failed: %s", cudaGetErrorString(e)));
  }
  // tensor maps of the prefill GEMMs (A buffers are fixed, so one encoding serves every call)
  if (desc->max_tokens > 16) {
    s->tmaps.resize((size_t)nl * 4);
    bool ok = true;
    for (int li = 0; li < nl && ok; ++li)
      for (int kind = 0; kind < 4 && ok; ++kind) {
        int epi = 0;
        LinearParams p = layer_linear(s, li, kind, desc->max_tokens, 1, false, s->x, &epi);
        ok = linear_tc_supported(p, epi) && tc_build_maps(p, epi, desc->max_tokens, &s->tmaps[(size_t)li * 4 + kind]) == ES_OK;
      }
    s->tmaps_valid = ok;
  }
  // tensor maps of the prefill attention (q buffer and this layer's K / V pages)
  {
    s->attn_maps.resize(nl);
    bool ok = true;
    for (int li = 0; li < nl && ok; ++li) {
      PrefillAttnParams a{};
      a.q = s->q; a.out = s->ao; a.B = 1; a.T = 1; a.Hq = desc->n_heads; a.Hkv = desc->n_kv_heads; a.hd = desc->head_dim;
      a.kv.k = s->k_pages(li); a.kv.v = s->v_pages(li); a.kv.block_table = s->block_table; a.kv.slots = s->slots_dev;
      a.kv.page_stride = (int64_t)L.page_elems; a.kv.head_stride = (int64_t)desc->kv_page_tokens * desc->head_dim;
      a.kv.tok_stride = desc->head_dim; a.kv.P = desc->kv_page_tokens; a.kv.pages_per_slot = L.pages_per_slot;
      a.kv_rows = (int64_t)L.n_pages * desc->n_kv_heads * desc->kv_page_tokens;
      ok = prefill_attention_tc_supported(a) &&
           prefill_attention_tc_build_maps(a, desc->max_tokens, &s->attn_maps[li]) == ES_OK;
    }
    s->attn_maps_valid = ok;
  }
  // profile entries: [embedding] layers... [head]
  auto add_entry = [&](int layer) {
    ProfileEntry pe;
    pe.layer = layer;
    cudaEventCreate(&pe.ev[0]);
    cudaEventCreate(&pe.ev[1]);
    s->prof.push_back(pe);
  };
  if (has_emb) add_entry(-1);
  for (int i = layer_begin; i < layer_end; ++i) add_entry(i);
  if (has_head) add_entry(desc->n_layers_total);
  if (cudaGetLastError() != cudaSuccess) return bail(fail(ES_ERR_CUDA, "event creation failed"));
  *out = s;
  return ES_OK;
}

void es_shard_destroy(es_shard_t* s) {
  if (!s) return;
  cudaStreamSynchronize(s->stream);
  for (auto& e : s->prof) { cudaEventDestroy(e.ev[0]); cudaEventDestroy(e.ev[1]); }
  for (auto& g : s->graph_cache) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
  for (auto& e : s->kt_events) cudaEventDestroy(e);
  delete s;
}

es_status_t es_shard_prefill(es_shard_t* s, const int32_t* ids, const es_tensor_t* hidden_in, int32_t B, int32_t T,
                             const int32_t* slots) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (B <= 0 || T <= 0) return fail(ES_ERR_INVALID_ARG, "B and T must be positive");
  if (B > s->d.max_batch) return fail(ES_ERR_RANGE, "B = %d exceeds max_batch = %d", B, s->d.max_batch);
  if ((int64_t)B * T > s->d.max_tokens) return fail(ES_ERR_RANGE, "B*T = %lld exceeds max_tokens = %d", (long long)B * T, s->d.max_tokens);
  if (T > s->d.max_seq) return fail(ES_ERR_KV_FULL, "prompt of %d tokens exceeds max_seq = %d", T, s->d.max_seq);
  ES_TRY(check_slots(s, slots, B));
  const float* hin;
  ES_TRY(check_inputs(s, ids, hidden_in, (int64_t)B * T, &hin));
  if (s->profiling) ES_TRY(harvest_profile(s));
  if (tunables().debug_checks) ES_TRY(debug_checks_now(s));    // checking mode: what the previous pass left behind
  ES_TRY(upload_slots(s, slots, B));
  s->last_valid = false;
  ES_TRY(enqueue_pass(s, ids, hin, B, T, false));
  for (int b = 0; b < B; ++b) s->ctx[slots[b]] = T;
  s->last_B = B; s->last_T = T; s->last_head_rows = B; s->last_valid = true;
  if (s->profiling) { s->pending = true; s->pending_prefill = true; }
  return ES_OK;
}

es_status_t es_shard_prefill_ragged(es_shard_t* s, const int32_t* ids, const es_tensor_t* hidden_in, int32_t B, int32_t T,
                                    const int32_t* slots, const int32_t* lens) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (!lens) return fail(ES_ERR_INVALID_ARG, "lens is null");
  if (B <= 0 || T <= 0) return fail(ES_ERR_INVALID_ARG, "B and T must be positive");
  if (B > s->d.max_batch) return fail(ES_ERR_RANGE, "B = %d exceeds max_batch = %d", B, s->d.max_batch);
  if ((int64_t)B * T > s->d.max_tokens) return fail(ES_ERR_RANGE, "B*T = %lld exceeds max_tokens = %d", (long long)B * T, s->d.max_tokens);
  if (T > s->d.max_seq) return fail(ES_ERR_KV_FULL, "prompt of %d tokens exceeds max_seq = %d", T, s->d.max_seq);
  for (int b = 0; b < B; ++b)
    if (lens[b] < 1 || lens[b] > T) return fail(ES_ERR_RANGE, "lens[%d] = %d outside [1, %d]", b, lens[b], T);
  ES_TRY(check_slots(s, slots, B));
  const float* hin;
  ES_TRY(check_inputs(s, ids, hidden_in, (int64_t)B * T, &hin));
  if (s->profiling) ES_TRY(harvest_profile(s));
  if (tunables().debug_checks) ES_TRY(debug_checks_now(s));    // checking mode: what the previous pass left behind
  ES_TRY(upload_slots(s, slots, B));
  s->lens_host.assign(lens, lens + B);
  ES_CUDA_CHECK(cudaMemcpyAsync(s->lens_dev, s->lens_host.data(), B * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  s->last_valid = false;
  ES_TRY(enqueue_pass(s, ids, hin, B, T, false, s->lens_dev));
  for (int b = 0; b < B; ++b) s->ctx[slots[b]] = lens[b];
  s->last_B = B; s->last_T = T; s->last_head_rows = B; s->last_valid = true;
  if (s->profiling) { s->pending = true; s->pending_prefill = true; }
  return ES_OK;
}

es_status_t es_shard_prefill_packed(es_shard_t* s, const int32_t* ids, const es_tensor_t* hidden_in, int32_t B,
                                    const int32_t* slots, const int32_t* lens) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (!lens) return fail(ES_ERR_INVALID_ARG, "lens is null");
  if (B <= 0) return fail(ES_ERR_INVALID_ARG, "B must be positive");
  if (B > s->d.max_batch) return fail(ES_ERR_RANGE, "B = %d exceeds max_batch = %d", B, s->d.max_batch);
  int64_t total = 0;
  int longest = 0;
  for (int b = 0; b < B; ++b) {
    if (lens[b] < 1) return fail(ES_ERR_RANGE, "lens[%d] = %d must be at least 1", b, lens[b]);
    if (lens[b] > s->d.max_seq) return fail(ES_ERR_KV_FULL, "prompt %d of %d tokens exceeds max_seq = %d", b, lens[b], s->d.max_seq);
    total += lens[b];
    if (lens[b] > longest) longest = lens[b];
  }
  if (total > s->d.max_tokens) return fail(ES_ERR_RANGE, "%lld packed rows exceed max_tokens = %d", (long long)total, s->d.max_tokens);
  ES_TRY(check_slots(s, slots, B));
  const float* hin;
  ES_TRY(check_inputs(s, ids, hidden_in, total, &hin));
  if (s->profiling) ES_TRY(harvest_profile(s));
  if (tunables().debug_checks) ES_TRY(debug_checks_now(s));    // checking mode: what the previous pass left behind
  ES_TRY(upload_slots(s, slots, B));
  s->lens_host.assign(lens, lens + B);
  s->cu_host.assign(B + 1, 0);
  for (int b = 0; b < B; ++b) s->cu_host[b + 1] = s->cu_host[b] + lens[b];
  ES_CUDA_CHECK(cudaMemcpyAsync(s->lens_dev, s->lens_host.data(), B * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  ES_CUDA_CHECK(cudaMemcpyAsync(s->cu_dev, s->cu_host.data(), (B + 1) * sizeof(int), cudaMemcpyHostToDevice, s->stream));
  s->last_valid = false;
  ES_TRY(enqueue_pass(s, ids, hin, B, longest, false, s->lens_dev, s->cu_dev, (int)total));
  for (int b = 0; b < B; ++b) s->ctx[slots[b]] = lens[b];
  s->last_B = 1; s->last_T = (int)total; s->last_valid = true;     // the handoff is the packed [1, total rows, d_model]
  s->last_head_rows = B;
  if (s->profiling) { s->pending = true; s->pending_prefill = true; }
  return ES_OK;
}

es_status_t es_shard_decode_step(es_shard_t* s, const int32_t* ids, const es_tensor_t* hidden_in, int32_t B,
                                 const int32_t* slots) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (B <= 0) return fail(ES_ERR_INVALID_ARG, "B must be positive");
  if (B > s->d.max_batch) return fail(ES_ERR_RANGE, "B = %d exceeds max_batch = %d", B, s->d.max_batch);
  ES_TRY(check_slots(s, slots, B));
  for (int b = 0; b < B; ++b) {
    const int c = s->ctx[slots[b]];
    if (c <= 0) return fail(ES_ERR_STATE, "slot %d has no prefilled context", slots[b]);
    if (c + 1 > s->d.max_seq) return fail(ES_ERR_KV_FULL, "slot %d is full (%d of %d positions)", slots[b], c, s->d.max_seq);
  }
  const float* hin;
  ES_TRY(check_inputs(s, ids, hidden_in, B, &hin));
  if (s->profiling) ES_TRY(harvest_profile(s));
  if (tunables().debug_checks) ES_TRY(debug_checks_now(s));    // checking mode: what the previous pass left behind
  ES_TRY(upload_slots(s, slots, B));
  s->last_valid = false;

  // the legacy default stream cannot be captured: steps on it are launched kernel by kernel
  const bool capturable = s->stream != nullptr && s->stream != cudaStreamLegacy && s->stream != cudaStreamPerThread;
  const bool use_graph = s->graphs && !s->profiling && !s->kernel_timing && capturable;
  if (!use_graph) {
    ES_TRY(enqueue_pass(s, ids, hin, B, 1, true));
  } else {
    GraphKey key{B, ids, hin};
    auto it = s->graph_cache.find(key);
    if (it == s->graph_cache.end()) {
      // capture the step once; positions live in device memory, so the same graph serves every step
      if (s->graph_cache.size() >= 64) {
        for (auto& g : s->graph_cache) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
        s->graph_cache.clear();
      }
      ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
      const int64_t before = s->launches;
      ES_CUDA_CHECK(cudaStreamBeginCapture(s->stream, cudaStreamCaptureModeThreadLocal));
      es_status_t st = enqueue_pass(s, ids, hin, B, 1, true);
      cudaGraph_t graph = nullptr;
      cudaError_t e = cudaStreamEndCapture(s->stream, &graph);
      const int64_t nodes = s->launches - before;
      s->launches = before;
      if (st != ES_OK) { if (graph) cudaGraphDestroy(graph); return st; }
      if (e != cudaSuccess) return fail(ES_ERR_CUDA, "graph capture failed: %s", cudaGetErrorString(e));
      GraphEntry ge;
      e = cudaGraphInstantiate(&ge.exec, graph, 0);
      cudaGraphDestroy(graph);
      if (e != cudaSuccess) return fail(ES_ERR_CUDA, "graph instantiation failed: %s", cudaGetErrorString(e));
      ge.nodes = nodes;
      it = s->graph_cache.emplace(key, ge).first;
    }
    ES_CUDA_CHECK(cudaGraphLaunch(it->second.exec, s->stream));
    s->launches += it->second.nodes;
  }
  for (int b = 0; b < B; ++b) s->ctx[slots[b]] += 1;
  s->last_B = B; s->last_T = 1; s->last_head_rows = B; s->last_valid = true;
  if (s->profiling) { s->pending = true; s->pending_prefill = false; }
  return ES_OK;
}

es_status_t es_shard_handoff(es_shard_t* s, es_tensor_t* hidden_out, es_tensor_t* logits, es_tensor_t* next_ids) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (!s->last_valid) return fail(ES_ERR_STATE, "no completed prefill/decode call to hand off");
  if (hidden_out) {
    hidden_out->data = s->x; hidden_out->dtype = ES_DTYPE_F32; hidden_out->rank = 3;
    hidden_out->shape[0] = s->last_B; hidden_out->shape[1] = s->last_T; hidden_out->shape[2] = s->d.d_model; hidden_out->shape[3] = 1;
  }
  if (logits) {
    logits->data = s->has_head ? s->logits : nullptr; logits->dtype = ES_DTYPE_F32; logits->rank = 2;
    logits->shape[0] = s->last_head_rows; logits->shape[1] = s->d.vocab; logits->shape[2] = logits->shape[3] = 1;
  }
  if (next_ids) {
    next_ids->data = s->has_head ? s->next_ids : nullptr; next_ids->dtype = ES_DTYPE_I32; next_ids->rank = 1;
    next_ids->shape[0] = s->last_head_rows; next_ids->shape[1] = next_ids->shape[2] = next_ids->shape[3] = 1;
  }
  return ES_OK;
}

es_status_t es_shard_set_profiling(es_shard_t* s, int32_t enabled) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (!enabled && s->profiling) ES_TRY(harvest_profile(s));
  s->profiling = enabled != 0;
  return ES_OK;
}

es_status_t es_layer_profile(es_shard_t* s, es_layer_profile_t* out, int32_t capacity, int32_t* n) {
  if (!s || !n) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (capacity > 0 && !out) return fail(ES_ERR_INVALID_ARG, "out is null");
  ES_TRY(harvest_profile(s));
  const es_model_desc_t& d = s->d;
  const int64_t nq = (int64_t)d.n_heads * d.head_dim, nkv = (int64_t)d.n_kv_heads * d.head_dim;
  const int64_t layer_w = 2 * (2 * (int64_t)d.d_model + nq * d.d_model + 2 * nkv * d.d_model + d.d_model * nq + 3 * (int64_t)d.d_model * d.d_ffn);
  const int64_t layer_kv = 2 * (int64_t)s->lay.n_pages * s->lay.page_elems * 2;
  int i = 0;
  for (const auto& e : s->prof) {
    if (i < capacity) {
      es_layer_profile_t& o = out[i];
      o.layer = e.layer;
      o.n_prefill = e.n_prefill; o.n_decode = e.n_decode;
      o.prefill_ms_mean = e.n_prefill ? (float)(e.prefill_ms / e.n_prefill) : 0.f;
      o.decode_ms_mean = e.n_decode ? (float)(e.decode_ms / e.n_decode) : 0.f;
      const int tok = e.n_prefill + e.n_decode;
      o.avg_ms_per_token = tok ? (float)((e.prefill_ms + e.decode_ms) / tok) : 0.f;
      if (e.layer == -1) { o.activation_bytes = (int64_t)d.d_model * 4; o.weight_bytes = 2 * (int64_t)d.vocab * d.d_model; o.kv_bytes = 0; }
      else if (e.layer == d.n_layers_total) { o.activation_bytes = (int64_t)d.vocab * 4; o.weight_bytes = 2 * ((int64_t)d.vocab * d.d_model + d.d_model); o.kv_bytes = 0; }
      else { o.activation_bytes = (int64_t)d.d_model * 4; o.weight_bytes = layer_w; o.kv_bytes = layer_kv; }
    }
    ++i;
  }
  *n = i;
  return ES_OK;
}

es_status_t es_shard_reset_slots(es_shard_t* s, const int32_t* slots, int32_t n) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (!slots || n <= 0) {
    std::fill(s->ctx.begin(), s->ctx.end(), -1);
    ES_CUDA_CHECK(cudaMemsetAsync(s->ctx_len, 0, (size_t)s->d.max_slots * 4, s->stream));
    return ES_OK;
  }
  for (int i = 0; i < n; ++i)
    if (slots[i] < 0 || slots[i] >= s->d.max_slots) return fail(ES_ERR_RANGE, "slot %d out of range", slots[i]);
  for (int i = 0; i < n; ++i) {
    s->ctx[slots[i]] = -1;
    ES_CUDA_CHECK(cudaMemsetAsync(s->ctx_len + slots[i], 0, 4, s->stream));
  }
  return ES_OK;
}

es_status_t es_shard_set_page_table(es_shard_t* s, const int32_t* table) {
  if (!s || !table) return fail(ES_ERR_INVALID_ARG, "null argument");
  const int n = s->lay.n_pages;
  std::vector<char> seen(n, 0);
  for (int i = 0; i < n; ++i) {
    if (table[i] < 0 || table[i] >= n || seen[table[i]]) return fail(ES_ERR_INVALID_ARG, "page table is not a permutation of 0..%d", n - 1);
    seen[table[i]] = 1;
  }
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  ES_CUDA_CHECK(cudaMemcpy(s->block_table, table, (size_t)n * 4, cudaMemcpyHostToDevice));
  return es_shard_reset_slots(s, nullptr, 0);
}

es_status_t es_shard_set_graphs(es_shard_t* s, int32_t enabled) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  s->graphs = enabled != 0;
  return ES_OK;
}

es_status_t es_shard_device_status(es_shard_t* s) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  int host[2] = {0, 0};
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  ES_CUDA_CHECK(cudaMemcpy(host, s->status, sizeof(host), cudaMemcpyDeviceToHost));
  if (host[0] != 0) {
    cudaMemset(s->status, 0, 256);
    return fail(ES_ERR_DEVICE_TIMEOUT, "a device-side wait ran out (code %d, detail %d)", host[0], host[1]);
  }
  if (tunables().debug_checks) ES_TRY(debug_checks(s));
  return ES_OK;
}

es_status_t es_shard_wait_probe(es_shard_t* s, int32_t limit_us) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if (limit_us < 1 || limit_us > 100000) return fail(ES_ERR_RANGE, "limit_us must be in [1, 100000]");
  return launch_wait_probe(s->status, (unsigned long long)limit_us * 1000ull, s->stream, &s->launches);
}

int64_t es_shard_launch_count(const es_shard_t* s) { return s ? s->launches : 0; }

es_status_t es_shard_set_kernel_timing(es_shard_t* s, int32_t enabled) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  s->kernel_timing = enabled != 0;
  s->kt_used = 0;
  s->kt_cat.clear();
  s->kt_pair_bytes.clear();
  return ES_OK;
}

es_status_t es_shard_set_step_timing(es_shard_t* s, int32_t enabled) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  if ((enabled != 0) == s->step_timing) return ES_OK;
  // captured steps carry (or lack) the stamp slots of their launches: capture afresh
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  for (auto& g : s->graph_cache) if (g.second.exec) cudaGraphExecDestroy(g.second.exec);
  s->graph_cache.clear();
  s->step_timing = enabled != 0;
  s->st_used = 0;
  s->st_cat.clear();
  s->st_bytes.clear();
  return ES_OK;
}

es_status_t es_shard_step_timing(es_shard_t* s, int32_t capacity, int32_t* n, int32_t* category, double* start_us,
                                 double* end_us, double* bytes) {
  if (!s || !n) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (capacity > 0 && (!category || !start_us || !end_us || !bytes)) return fail(ES_ERR_INVALID_ARG, "null output array");
  *n = s->st_used;
  if (s->st_used == 0 || capacity <= 0) return ES_OK;
  std::vector<unsigned long long> host(2 * (size_t)STAMP_SLOTS);
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  ES_CUDA_CHECK(cudaMemcpy(host.data(), s->stamps, host.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  unsigned long long t0 = ~0ull;
  for (int i = 0; i < s->st_used; ++i) if (host[i] < t0) t0 = host[i];
  for (int i = 0; i < s->st_used && i < capacity; ++i) {
    const unsigned long long a = host[i], b = host[STAMP_SLOTS + i];
    category[i] = s->st_cat[i];
    bytes[i] = s->st_bytes[i];
    // a launch that never ran (or whose stamps were lost) reports a negative start
    start_us[i] = (a == ~0ull) ? -1.0 : (double)(a - t0) * 1e-3;
    end_us[i] = (a == ~0ull || b < t0) ? -1.0 : (double)(b - t0) * 1e-3;
  }
  return ES_OK;
}

es_status_t es_shard_kernel_timing_detail(es_shard_t* s, double* ms, double* bytes, int64_t* launches) {
  if (!s) return fail(ES_ERR_INVALID_ARG, "shard is null");
  ES_CUDA_CHECK(cudaStreamSynchronize(s->stream));
  double m[ES_KT_COUNT] = {}, b[ES_KT_COUNT] = {};
  int64_t n[ES_KT_COUNT] = {};
  for (size_t i = 0; i + 1 < s->kt_used; i += 2) {
    float t = 0.f;
    ES_CUDA_CHECK(cudaEventElapsedTime(&t, s->kt_events[i], s->kt_events[i + 1]));
    const int c = s->kt_cat[i / 2];
    m[c] += t;
    b[c] += s->kt_pair_bytes[i / 2];
    n[c] += 1;
  }
  for (int c = 0; c < ES_KT_COUNT; ++c) {
    if (ms) ms[c] = m[c];
    if (bytes) bytes[c] = b[c];
    if (launches) launches[c] = n[c];
  }
  return ES_OK;
}

es_status_t es_shard_kernel_timing(es_shard_t* s, double* total_ms, double* weight_bytes, int64_t* launches) {
  double m[ES_KT_COUNT], b[ES_KT_COUNT];
  int64_t n[ES_KT_COUNT];
  ES_TRY(es_shard_kernel_timing_detail(s, m, b, n));
  const int lin[5] = {ES_KT_QKV, ES_KT_O, ES_KT_GATE_UP, ES_KT_DOWN, ES_KT_LM_HEAD};
  double tm = 0, tb = 0;
  int64_t tn = 0;
  for (int c : lin) { tm += m[c]; tb += b[c]; tn += n[c]; }
  if (total_ms) *total_ms = tm;
  if (weight_bytes) *weight_bytes = tb;
  if (launches) *launches = tn;
  return ES_OK;
}

}  // extern "C"

extern "C" {

// ---- single operations -----------------------------------------------------------------------

es_status_t es_op_rmsnorm(const float* x, const void* gain, void* y, int32_t M, int32_t d, float eps, void* stream) {
  if (M < 0 || d <= 0 || d % 8) return fail(ES_ERR_SHAPE, "d must be a positive multiple of 8");
  if (M == 0) return ES_OK;
  if (!x || !gain || !y) return fail(ES_ERR_INVALID_ARG, "null argument");
  return launch_rmsnorm(x, (const __half*)gain, (__half*)y, M, d, eps, 1, 0, (cudaStream_t)stream, nullptr);
}

es_status_t es_op_linear(const void* A, const void* W, const float* R, float* C, int32_t M, int32_t N, int32_t K,
                         int32_t path, void* stream) {
  if (!A || !W || !C) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (M < 0 || N <= 0 || K <= 0 || K % 8) return fail(ES_ERR_SHAPE, "N, K must be positive and K a multiple of 8");
  LinearParams p{};
  p.A = (const __half*)A; p.lda = K; p.w[0] = (const __half*)W; p.seg_rows[0] = N;
  p.M = M; p.N = N; p.K = K; p.out_f32 = C; p.res = R; p.ldo = N; p.T = 1;
  cudaStream_t st = (cudaStream_t)stream;
  if (path == 0) path = (M > 2 && M <= 16 && linear_stream_mma_supported(p, EPI_F32)) ? 4 : (M <= 16) ? 2 : (linear_tc_supported(p, EPI_F32) ? 1 : 3);
  switch (path) {
    case 1:
      if (!linear_tc_supported(p, EPI_F32)) return fail(ES_ERR_UNSUPPORTED, "tensor-core kernel does not take this shape");
      return launch_linear_tc(p, EPI_F32, st, nullptr, nullptr);
    case 2: return launch_linear_stream(p, EPI_F32, st, nullptr);
    case 3: return launch_linear_reference(p, EPI_F32, st, nullptr);
    case 5:
    case 6:
      if (!linear_tc2_supported(p, EPI_F32)) return fail(ES_ERR_UNSUPPORTED, "pair kernel does not take this shape");
      p.pair_nacc = path == 5 ? 1 : 2;
      return launch_linear_tc2(p, EPI_F32, st, nullptr, nullptr);
    case 4:
      if (!linear_stream_mma_supported(p, EPI_F32)) return fail(ES_ERR_UNSUPPORTED, "tensor-core streaming kernel does not take this shape");
      return launch_linear_stream_mma(p, EPI_F32, st, nullptr);
    default: return fail(ES_ERR_INVALID_ARG, "unknown path %d", path);
  }
}

size_t es_op_linear_splitk_workspace_bytes(int32_t M, int32_t N, int32_t k_splits) {
  if (M <= 0 || N <= 0 || k_splits <= 0) return 0;
  return (size_t)k_splits * M * N * sizeof(float);
}

es_status_t es_op_linear_splitk(const void* A, const void* W, const float* R, float* C, int32_t M, int32_t N, int32_t K,
                                int32_t k_splits, void* workspace, size_t workspace_bytes, void* stream) {
  if (!A || !W || !C) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (M <= 0 || N <= 0 || K <= 0 || K % 8 || N % 4) return fail(ES_ERR_SHAPE, "M, N, K must be positive, K a multiple of 8 and N of 4");
  LinearParams p{};
  p.A = (const __half*)A; p.lda = K; p.w[0] = (const __half*)W; p.seg_rows[0] = N;
  p.M = M; p.N = N; p.K = K; p.out_f32 = C; p.res = R; p.ldo = N; p.T = 1;
  cudaStream_t st = (cudaStream_t)stream;
  const bool skinny = M <= 16;            // decode-sized: the K-sliced weight-streaming kernel
  if (skinny) {
    if (M < 3 || !linear_stream_mma_supported(p, EPI_F32))
      return fail(ES_ERR_UNSUPPORTED, "K-sliced streaming kernel takes 3..16 rows and K a multiple of 256");
    if (k_splits == 0) k_splits = linear_stream_mma_splits(p, EPI_F32, workspace ? workspace_bytes : 0);
  } else {
    if (!linear_tc_supported(p, EPI_F32)) return fail(ES_ERR_UNSUPPORTED, "tensor-core kernel does not take this shape");
    p.split_on_pairs = (M >= 256 && tunables().tc_pair && tunables().split_pairs) ? 1 : 0;   // 256 or more rows: slices on CTA pairs
    if (k_splits == 0) {
      k_splits = p.split_on_pairs ? linear_tc2_splits(p, EPI_F32) : 1;
      if (k_splits <= 1) { p.split_on_pairs = 0; k_splits = linear_tc_splits(p, EPI_F32); }
    }
  }
  if (k_splits < 1 || k_splits > 64) return fail(ES_ERR_INVALID_ARG, "k_splits must be 0 (automatic) or 1..64");
  if (k_splits == 1)
    return skinny ? launch_linear_stream_mma(p, EPI_F32, st, nullptr) : launch_linear_tc(p, EPI_F32, st, nullptr, nullptr);
  if (!workspace || workspace_bytes < es_op_linear_splitk_workspace_bytes(M, N, k_splits))
    return fail(ES_ERR_WORKSPACE, "split-K workspace: %zu bytes given, %zu needed", workspace_bytes,
                es_op_linear_splitk_workspace_bytes(M, N, k_splits));
  if ((uintptr_t)workspace % 16) return fail(ES_ERR_INVALID_ARG, "workspace must be 16-byte aligned");
  p.k_splits = k_splits; p.part = (float*)workspace;
  if (skinny) {
    ES_TRY(launch_linear_stream_mma(p, EPI_F32, st, nullptr));
    return launch_splitk_reduce(p.part, k_splits, R, C, M, N, N, nullptr, nullptr, 0.f, st, nullptr);
  }
  p.k_splits = k_splits; p.part = (float*)workspace;
  if (p.split_on_pairs) ES_TRY(launch_linear_tc2(p, EPI_F32, st, nullptr, nullptr));
  else ES_TRY(launch_linear_tc(p, EPI_F32, st, nullptr, nullptr));
  return launch_splitk_reduce(p.part, k_splits, R, C, M, N, N, nullptr, nullptr, 0.f, st, nullptr);
}

es_status_t es_op_prefill_attention(const void* q, const void* k, const void* v, void* out, int32_t B, int32_t T,
                                    int32_t Hq, int32_t Hkv, int32_t hd, int32_t path, void* stream) {
  if (!q || !k || !v || !out) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (B < 0 || T < 0 || Hq <= 0 || Hkv <= 0) return fail(ES_ERR_INVALID_ARG, "bad sizes");
  PrefillAttnParams p{};
  p.q = (const __half*)q; p.out = (__half*)out; p.B = B; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.hd = hd;
  p.kv.k = (const __half*)k; p.kv.v = (const __half*)v; p.kv.block_table = nullptr; p.kv.slots = nullptr;
  p.kv.page_stride = (int64_t)T * Hkv * hd; p.kv.head_stride = hd; p.kv.tok_stride = (int64_t)Hkv * hd;
  p.kv.P = T > 0 ? T : 1; p.kv.pages_per_slot = 1;
  p.kv_rows = (int64_t)B * T;
  if (path == 1 && !prefill_attention_tc_supported(p)) return fail(ES_ERR_UNSUPPORTED, "tensor-core attention does not take this shape");
  return launch_prefill_attention(p, (cudaStream_t)stream, nullptr, path);
}

size_t es_op_decode_attention_scratch_bytes(int32_t B, int32_t Hq, int32_t hd, int32_t max_ctx, int32_t page_tokens) {
  if (B <= 0 || Hq <= 0 || hd <= 0 || max_ctx <= 0 || page_tokens <= 0) return 0;
  // worst case over the KV-head count: one page per split
  return decode_attention_scratch_bytes(B, Hq, hd, (max_ctx + page_tokens - 1) / page_tokens);
}

es_status_t es_op_decode_attention(const void* q, const void* k_pages, const void* v_pages, const int32_t* block_table,
                                   const int32_t* ctx_len, void* out, int32_t B, int32_t Hq, int32_t Hkv, int32_t hd,
                                   int32_t page_tokens, int32_t pages_per_seq, int32_t max_ctx, void* scratch,
                                   size_t scratch_bytes, void* stream) {
  if (!q || !k_pages || !v_pages || !block_table || !ctx_len || !out || !scratch) return fail(ES_ERR_INVALID_ARG, "null argument");
  if (B <= 0 || Hq <= 0 || Hkv <= 0 || page_tokens <= 0 || pages_per_seq <= 0 || max_ctx <= 0)
    return fail(ES_ERR_INVALID_ARG, "bad sizes");
  if (max_ctx > page_tokens * pages_per_seq) return fail(ES_ERR_RANGE, "max_ctx exceeds the block table");
  DecodeAttnParams p{};
  p.q = (const __half*)q; p.out = (__half*)out; p.ctx_len = ctx_len; p.ctx_add = 0; p.part = (float*)scratch;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.hd = hd;
  p.kv.k = (const __half*)k_pages; p.kv.v = (const __half*)v_pages; p.kv.block_table = block_table; p.kv.slots = nullptr;
  p.kv.page_stride = (int64_t)Hkv * page_tokens * hd; p.kv.head_stride = (int64_t)page_tokens * hd; p.kv.tok_stride = hd;
  p.kv.P = page_tokens; p.kv.pages_per_slot = pages_per_seq;
  choose_splits(max_ctx, page_tokens, B, Hkv, Hq / Hkv, &p.n_splits, &p.pages_per_split);
  if (scratch_bytes < decode_attention_scratch_bytes(B, Hq, hd, p.n_splits))
    return fail(ES_ERR_WORKSPACE, "scratch: %zu bytes given, %zu needed", scratch_bytes,
                decode_attention_scratch_bytes(B, Hq, hd, p.n_splits));
  p.split_cnt = (int*)((unsigned char*)scratch + decode_attention_counter_offset(B, Hq, hd, p.n_splits));
  if (p.n_splits > 1)         // the splits' arrival counters start at zero
    ES_CUDA_CHECK(cudaMemsetAsync(p.split_cnt, 0, decode_attention_counter_bytes(B, Hq), (cudaStream_t)stream));
  return launch_decode_attention(p, (cudaStream_t)stream, nullptr);
}

}  // extern "C"

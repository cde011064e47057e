// Split-KV decode attention over the paged cache: one query row per (sequence, head).
// A CTA takes one split (a run of KV pages) of one KV head and serves all query heads of that
// group, so K and V are read from HBM once per group.  Inside a warp the head dimension is spread
// over the lanes; scores are reduced with warp shuffles, the softmax is the running (max, sum)
// form.  Each split writes an unnormalised partial (o, max, sum); a second kernel merges the
// partials of a row in split order, so the result does not depend on scheduling.
#include "es_internal.cuh"

namespace es {

namespace {

constexpr int DWARPS = 4;

template <int E>
__device__ __forceinline__ void load_vec(const __half* p, float (&f)[E]) {
  if (E == 4) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    const __half2* h = reinterpret_cast<const __half2*>(&u);
    const float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
  } else {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(p));
    f[0] = a.x; f[1] = a.y;
  }
}

template <int HD, int G>
__global__ void __launch_bounds__(DWARPS * 32) decode_attn_split_kernel(const DecodeAttnParams p) {
  constexpr int E = HD / 32;
  __shared__ float sm_o[DWARPS][G][HD];
  __shared__ float sm_m[DWARPS][G];
  __shared__ float sm_l[DWARPS][G];

  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int slot = p.kv.slots ? p.kv.slots[b] : b;
  const int ctx = p.ctx_len[slot] + p.ctx_add;
  const int tokens_per_split = p.pages_per_split * p.kv.P;
  const int t_begin = split * tokens_per_split;
  if (t_begin >= ctx) return;
  const int t_end = min(ctx, t_begin + tokens_per_split);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float scale = rsqrtf((float)HD);

  float q[G][E], acc[G][E], m[G], l[G];
#pragma unroll
  for (int j = 0; j < G; ++j) {
    load_vec<E>(p.q + ((int64_t)b * p.Hq + (g * G + j)) * HD + lane * E, q[j]);
#pragma unroll
    for (int e = 0; e < E; ++e) { q[j][e] *= scale; acc[j][e] = 0.f; }
    m[j] = -INFINITY;
    l[j] = 0.f;
  }

  for (int t = t_begin + warp; t < t_end; t += DWARPS) {
    float kf[E], vf[E];
    load_vec<E>(kv_addr(p.kv, p.kv.k, slot, t, g) + lane * E, kf);
    load_vec<E>(kv_addr(p.kv, p.kv.v, slot, t, g) + lane * E, vf);
#pragma unroll
    for (int j = 0; j < G; ++j) {
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < E; ++e) s = fmaf(q[j][e], kf[e], s);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float mn = fmaxf(m[j], s);
      const float alpha = __expf(m[j] - mn);
      const float pj = __expf(s - mn);
      l[j] = l[j] * alpha + pj;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[j][e] = acc[j][e] * alpha + pj * vf[e];
      m[j] = mn;
    }
  }

#pragma unroll
  for (int j = 0; j < G; ++j) {
#pragma unroll
    for (int e = 0; e < E; ++e) sm_o[warp][j][lane * E + e] = acc[j][e];
    if (lane == 0) { sm_m[warp][j] = m[j]; sm_l[warp][j] = l[j]; }
  }
  __syncthreads();
  // merge the warps in warp order; thread -> (head j, column c)
  for (int i = threadIdx.x; i < G * HD; i += DWARPS * 32) {
    const int j = i / HD, c = i - j * HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < DWARPS; ++w) mm = fmaxf(mm, sm_m[w][j]);
    float o = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < DWARPS; ++w) {
      const float f = (sm_m[w][j] == -INFINITY) ? 0.f : __expf(sm_m[w][j] - mm);
      o += sm_o[w][j][c] * f;
      ll += sm_l[w][j] * f;
    }
    float* dst = p.part + (((int64_t)b * p.Hq + (g * G + j)) * p.n_splits + split) * (HD + 2);
    dst[c] = o;
    if (c == 0) { dst[HD] = mm; dst[HD + 1] = ll; }
  }
}

template <int HD>
__global__ void __launch_bounds__(HD) decode_attn_merge_kernel(const DecodeAttnParams p) {
  const int h = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  const int slot = p.kv.slots ? p.kv.slots[b] : b;
  const int ctx = p.ctx_len[slot] + p.ctx_add;
  const int tokens_per_split = p.pages_per_split * p.kv.P;
  int active = (ctx + tokens_per_split - 1) / tokens_per_split;
  active = active < p.n_splits ? active : p.n_splits;
  const float* src = p.part + ((int64_t)b * p.Hq + h) * p.n_splits * (HD + 2);
  float mm = -INFINITY;
  for (int s = 0; s < active; ++s) mm = fmaxf(mm, src[(int64_t)s * (HD + 2) + HD]);
  float o = 0.f, ll = 0.f;
  for (int s = 0; s < active; ++s) {
    const float f = __expf(src[(int64_t)s * (HD + 2) + HD] - mm);
    o += src[(int64_t)s * (HD + 2) + c] * f;
    ll += src[(int64_t)s * (HD + 2) + HD + 1] * f;
  }
  p.out[((int64_t)b * p.Hq + h) * HD + c] = __float2half_rn(active > 0 ? o / ll : 0.f);
}

template <int HD>
es_status_t launch_hd(const DecodeAttnParams& p, cudaStream_t s) {
  const dim3 grid(p.n_splits, p.Hkv, p.B);
  switch (p.Hq / p.Hkv) {
    case 1: decode_attn_split_kernel<HD, 1><<<grid, DWARPS * 32, 0, s>>>(p); break;
    case 2: decode_attn_split_kernel<HD, 2><<<grid, DWARPS * 32, 0, s>>>(p); break;
    case 4: decode_attn_split_kernel<HD, 4><<<grid, DWARPS * 32, 0, s>>>(p); break;
    case 8: decode_attn_split_kernel<HD, 8><<<grid, DWARPS * 32, 0, s>>>(p); break;
    default: return fail(ES_ERR_SHAPE, "query heads per KV head must be 1, 2, 4 or 8");
  }
  ES_CUDA_CHECK(cudaGetLastError());
  decode_attn_merge_kernel<HD><<<dim3(p.Hq, p.B), HD, 0, s>>>(p);
  ES_CUDA_CHECK(cudaGetLastError());
  return ES_OK;
}

}  // namespace

size_t decode_attention_scratch_bytes(int B, int Hq, int hd, int n_splits) {
  return (size_t)B * Hq * n_splits * (hd + 2) * sizeof(float);
}

es_status_t launch_decode_attention(const DecodeAttnParams& p, cudaStream_t s, int64_t* launches) {
  if (p.B <= 0) return ES_OK;
  if (p.Hq % p.Hkv != 0) return fail(ES_ERR_SHAPE, "n_heads %% n_kv_heads != 0");
  es_status_t st;
  if (p.hd == 128) st = launch_hd<128>(p, s);
  else if (p.hd == 64) st = launch_hd<64>(p, s);
  else return fail(ES_ERR_SHAPE, "head_dim must be 64 or 128, got %d", p.hd);
  if (st == ES_OK && launches) *launches += 2;
  return st;
}

}  // namespace es

// Causal prefill attention.
//
// prefill_attn_simt_kernel: one warp per query row.  Keys are taken 32 at a time, one per lane
// (each lane forms the whole dot product of its key with the query row held in shared memory);
// the running-softmax statistics are reduced with warp shuffles; for the value product the head
// dimension is spread over the lanes and the 32 probabilities are broadcast lane by lane.
#include "es_internal.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int PWARPS = 4;

template <int HD>
__global__ void __launch_bounds__(PWARPS * 32) prefill_attn_simt_kernel(const PrefillAttnParams p) {
  constexpr int E = HD / 32;
  __shared__ float q_s[PWARPS][HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * PWARPS + warp;
  const int h = blockIdx.y, b = blockIdx.z;
  const int g = h / (p.Hq / p.Hkv);
  const int slot = p.kv.slots ? p.kv.slots[b] : b;
  // packed prompts: the sequence's first row and length come from the first-row table (p.T = the longest prompt)
  const int row0 = p.cu_rows ? p.cu_rows[b] : b * p.T;
  const int Tb = p.cu_rows ? p.cu_rows[b + 1] - row0 : p.T;
  const bool active = t < Tb;
  const float scale = rsqrtf((float)HD);
  stamp_begin(p.stamp);
  if (active) {
    const __half* qrow = p.q + (((int64_t)row0 + t) * p.Hq + h) * HD;
#pragma unroll
    for (int e = 0; e < E; ++e) q_s[warp][lane * E + e] = __half2float(qrow[lane * E + e]) * scale;
  }
  __syncwarp();
  if (!active) { stamp_end(p.stamp); return; }

  float acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  float m = -INFINITY, l = 0.f;

  for (int j0 = 0; j0 <= t; j0 += 32) {
    const int j = j0 + lane;
    float s = -INFINITY;
    if (j <= t) {
      const uint4* kr = reinterpret_cast<const uint4*>(kv_addr(p.kv, p.kv.k, slot, j, g));
      float d = 0.f;
#pragma unroll
      for (int c = 0; c < HD / 8; ++c) {
        const uint4 u = kr[c];
        const __half2* h2 = reinterpret_cast<const __half2*>(&u);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 kf = __half22float2(h2[i]);
          d = fmaf(q_s[warp][c * 8 + 2 * i], kf.x, d);
          d = fmaf(q_s[warp][c * 8 + 2 * i + 1], kf.y, d);
        }
      }
      s = d;
    }
    float cm = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
    const float mn = fmaxf(m, cm);
    const float alpha = __expf(m - mn);          // m = -inf on the first chunk -> 0
    const float pj = (j <= t) ? __expf(s - mn) : 0.f;
    float ps = pj;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    l = l * alpha + ps;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] *= alpha;
    m = mn;
    const int cnt = min(32, t - j0 + 1);
    for (int jj = 0; jj < cnt; ++jj) {
      const float pv = __shfl_sync(0xffffffffu, pj, jj);
      const __half* vr = kv_addr(p.kv, p.kv.v, slot, j0 + jj, g) + lane * E;
      if (E == 4) {
        const uint2 u = *reinterpret_cast<const uint2*>(vr);
        const __half2* h2 = reinterpret_cast<const __half2*>(&u);
        const float2 a = __half22float2(h2[0]), c2 = __half22float2(h2[1]);
        acc[0] = fmaf(pv, a.x, acc[0]); acc[1] = fmaf(pv, a.y, acc[1]);
        acc[E - 2] = fmaf(pv, c2.x, acc[E - 2]); acc[E - 1] = fmaf(pv, c2.y, acc[E - 1]);
      } else {
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(vr));
        acc[0] = fmaf(pv, a.x, acc[0]); acc[1] = fmaf(pv, a.y, acc[1]);
      }
    }
  }
  __half* orow = p.out + (((int64_t)row0 + t) * p.Hq + h) * HD + lane * E;
  const float inv = 1.0f / l;
#pragma unroll
  for (int e = 0; e < E; ++e) orow[e] = __float2half_rn(acc[e] * inv);
  stamp_end(p.stamp);
}

}  // namespace

es_status_t launch_prefill_attention(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches, int path, bool pdl) {
  if (p.B <= 0 || p.T <= 0) return ES_OK;
  if (path == 0) path = prefill_attention_tc_supported(p) ? 1 : 2;
  if (path == 1) return launch_prefill_attention_tc(p, s, launches, pdl);
  if (path == 2) return launch_prefill_attention_simt(p, s, launches);
  return fail(ES_ERR_INVALID_ARG, "unknown attention path %d", path);
}

es_status_t launch_prefill_attention_simt(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches) {
  if (p.B <= 0 || p.T <= 0) return ES_OK;
  if (p.Hq % p.Hkv != 0) return fail(ES_ERR_SHAPE, "n_heads %% n_kv_heads != 0");
  const dim3 grid((p.T + PWARPS - 1) / PWARPS, p.Hq, p.B);
  if (p.hd == 128) prefill_attn_simt_kernel<128><<<grid, PWARPS * 32, 0, s>>>(p);
  else if (p.hd == 64) prefill_attn_simt_kernel<64><<<grid, PWARPS * 32, 0, s>>>(p);
  else return fail(ES_ERR_SHAPE, "head_dim must be 64 or 128, got %d", p.hd);
  if (launches) ++*launches;
  ES_CUDA_CHECK(cudaGetLastError());
  return ES_OK;
}

}  // namespace es

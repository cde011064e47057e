// Epilogues of the linear-layer kernels: what happens to a finished fp32 accumulator.
// Every kernel of the family (reference, weight-streaming, tensor-core) funnels its results
// through these functions, two adjacent output columns at a time, so that they all round and
// store identically.
#pragma once

#include "es_internal.cuh"

namespace es {

__device__ __forceinline__ float silu_f(float z) { return z / (1.0f + __expf(-z)); }

// Residual / plain store of columns n and n+1 of row m.
__device__ __forceinline__ void epi_f32_pair(const LinearParams& p, int m, int n, float v0, float v1) {
  if (m >= p.M || n >= p.N) return;
  const int64_t o = (int64_t)m * p.ldo + n;
  const bool two = (n + 1 < p.N);
  if (p.res != nullptr) {
    v0 += p.res[o];
    if (two) v1 += p.res[o + 1];
  }
  p.out_f32[o] = v0;
  if (two) p.out_f32[o + 1] = v1;
}

// SwiGLU: one output column from the gate and up accumulators of the same n.
__device__ __forceinline__ void epi_swiglu(const LinearParams& p, int m, int n, float gate, float up) {
  if (m >= p.M || n >= p.N) return;
  p.out_f16[(int64_t)m * p.ldo + n] = __float2half_rn(silu_f(gate) * up);
}

// Fused QKV: columns (n, n+1) of the concatenated [q | k | v] projection of row m, n even.
// q and k are rotated by the row's position (adjacent-pair convention) in fp32 and rounded to
// fp16 once; k and v go straight to the slot's KV page.
__device__ __forceinline__ void epi_qkv_pair(const LinearParams& p, int m, int n, float v0, float v1) {
  if (m >= p.M || n >= p.N) return;
  const int b = m / p.T;
  const int slot = p.slots[b];
  const int pos = p.is_decode ? p.ctx_len[slot] : (m - b * p.T);
  if (pos < 0 || pos >= p.max_seq) return;   // host validates; never index outside the tables
  const int nq = p.Hq * p.hd, nkv = p.Hkv * p.hd;
  int c;          // column inside its head
  if (n < nq + nkv) {
    c = (n < nq ? n : n - nq) % p.hd;
    const int i = c >> 1;
    const float cs = p.rope_cos[(int64_t)pos * (p.hd / 2) + i];
    const float sn = p.rope_sin[(int64_t)pos * (p.hd / 2) + i];
    const float r0 = v0 * cs - v1 * sn;
    const float r1 = v0 * sn + v1 * cs;
    v0 = r0;
    v1 = r1;
  }
  const __half2 hv = __floats2half2_rn(v0, v1);
  if (n < nq) {
    *reinterpret_cast<__half2*>(p.out_f16 + (int64_t)m * nq + n) = hv;
    return;
  }
  const bool is_k = n < nq + nkv;
  const int kn = is_k ? n - nq : n - nq - nkv;
  const int g = kn / p.hd;
  c = kn - g * p.hd;
  const int page = p.block_table[(int64_t)slot * p.pages_per_slot + pos / p.P];
  const int64_t off = (((int64_t)page * p.Hkv + g) * p.P + (pos % p.P)) * p.hd + c;
  *reinterpret_cast<__half2*>((is_k ? p.k_cache : p.v_cache) + off) = hv;
}

template <int EPI>
__device__ __forceinline__ void epi_pair(const LinearParams& p, int m, int n, float v0, float v1) {
  if (EPI == EPI_F32) epi_f32_pair(p, m, n, v0, v1);
  else if (EPI == EPI_SWIGLU) epi_swiglu(p, m, n, v0, v1);
  else epi_qkv_pair(p, m, n, v0, v1);
}

// Pointer to row n (virtual, over the concatenated segments) of the weight; nullptr past N.
__device__ __forceinline__ const __half* weight_row(const LinearParams& p, int n) {
  if (n < p.seg_rows[0]) return p.w[0] + (int64_t)n * p.K;
  n -= p.seg_rows[0];
  if (n < p.seg_rows[1]) return p.w[1] + (int64_t)n * p.K;
  n -= p.seg_rows[1];
  if (n < p.seg_rows[2]) return p.w[2] + (int64_t)n * p.K;
  return nullptr;
}

}  // namespace es

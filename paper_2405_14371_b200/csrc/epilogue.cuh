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

// ---- 32-column row chunks (tensor-core kernel: a thread owns 32 adjacent accumulator columns of
// one row).  Same arithmetic as the pair functions above, with 16-byte loads and stores wherever
// the chunk is whole and aligned; ragged edges fall back to the pair functions. -------------------

__device__ __forceinline__ void epi_f32_chunk32(const LinearParams& p, int m, int n, const float (&v)[32]) {
  if (m >= p.M || n >= p.N) return;
  const int64_t o = (int64_t)m * p.ldo + n;
  const bool fast = (n + 32 <= p.N) && ((p.ldo & 3) == 0) && ((n & 3) == 0) &&
                    (((uintptr_t)p.out_f32 & 15) == 0) && (p.res == nullptr || ((uintptr_t)p.res & 15) == 0);
  if (!fast) {
#pragma unroll
    for (int j = 0; j < 32; j += 2) epi_f32_pair(p, m, n + j, v[j], v[j + 1]);
    return;
  }
  float4* dst = reinterpret_cast<float4*>(p.out_f32 + o);
  if (p.res != nullptr) {
    const float4* r = reinterpret_cast<const float4*>(p.res + o);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 rv = r[q];
      dst[q] = make_float4(v[4 * q] + rv.x, v[4 * q + 1] + rv.y, v[4 * q + 2] + rv.z, v[4 * q + 3] + rv.w);
    }
  } else {
#pragma unroll
    for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  }
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

__device__ __forceinline__ void epi_swiglu_chunk32(const LinearParams& p, int m, int n, const float (&g)[32],
                                                   const float (&u)[32]) {
  if (m >= p.M || n >= p.N) return;
  const bool fast = (n + 32 <= p.N) && ((p.ldo & 7) == 0) && ((n & 7) == 0) && (((uintptr_t)p.out_f16 & 15) == 0);
  if (!fast) {
#pragma unroll
    for (int j = 0; j < 32; ++j) epi_swiglu(p, m, n + j, g[j], u[j]);
    return;
  }
  uint4* dst = reinterpret_cast<uint4*>(p.out_f16 + (int64_t)m * p.ldo + n);
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    uint4 o;
    o.x = pack_half2(silu_f(g[8 * q]) * u[8 * q], silu_f(g[8 * q + 1]) * u[8 * q + 1]);
    o.y = pack_half2(silu_f(g[8 * q + 2]) * u[8 * q + 2], silu_f(g[8 * q + 3]) * u[8 * q + 3]);
    o.z = pack_half2(silu_f(g[8 * q + 4]) * u[8 * q + 4], silu_f(g[8 * q + 5]) * u[8 * q + 5]);
    o.w = pack_half2(silu_f(g[8 * q + 6]) * u[8 * q + 6], silu_f(g[8 * q + 7]) * u[8 * q + 7]);
    dst[q] = o;
  }
}

// 32 columns of the fused [q | k | v] projection; n is a multiple of 32, so the chunk lies inside one
// head of one segment (head_dim is 64 or 128).
__device__ __forceinline__ void epi_qkv_chunk32(const LinearParams& p, int m, int n, const float (&v)[32]) {
  if (m >= p.M || n >= p.N) return;
  const int nq = p.Hq * p.hd, nkv = p.Hkv * p.hd;
  const bool fast = (n + 32 <= p.N) && ((n & 31) == 0) && ((p.hd & 31) == 0);
  if (!fast) {
#pragma unroll
    for (int j = 0; j < 32; j += 2) epi_qkv_pair(p, m, n + j, v[j], v[j + 1]);
    return;
  }
  const int b = m / p.T;
  const int slot = p.slots[b];
  const int pos = p.is_decode ? p.ctx_len[slot] : (m - b * p.T);
  if (pos < 0 || pos >= p.max_seq) return;
  const bool is_q = n < nq, is_k = !is_q && n < nq + nkv;
  const int local = is_q ? n : (is_k ? n - nq : n - nq - nkv);
  const int head = local / p.hd, c0 = local - head * p.hd;
  __half* dst;
  if (is_q) {
    dst = p.out_f16 + (int64_t)m * nq + n;
  } else {
    const int page = p.block_table[(int64_t)slot * p.pages_per_slot + pos / p.P];
    dst = (is_k ? p.k_cache : p.v_cache) + (((int64_t)page * p.Hkv + head) * p.P + (pos % p.P)) * p.hd + c0;
  }
  uint4* d4 = reinterpret_cast<uint4*>(dst);
  if (is_q || is_k) {
    const float4* cs4 = reinterpret_cast<const float4*>(p.rope_cos + (int64_t)pos * (p.hd / 2) + c0 / 2);
    const float4* sn4 = reinterpret_cast<const float4*>(p.rope_sin + (int64_t)pos * (p.hd / 2) + c0 / 2);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 cs = cs4[q], sn = sn4[q];
      uint4 o;
      o.x = pack_half2(v[8 * q] * cs.x - v[8 * q + 1] * sn.x, v[8 * q] * sn.x + v[8 * q + 1] * cs.x);
      o.y = pack_half2(v[8 * q + 2] * cs.y - v[8 * q + 3] * sn.y, v[8 * q + 2] * sn.y + v[8 * q + 3] * cs.y);
      o.z = pack_half2(v[8 * q + 4] * cs.z - v[8 * q + 5] * sn.z, v[8 * q + 4] * sn.z + v[8 * q + 5] * cs.z);
      o.w = pack_half2(v[8 * q + 6] * cs.w - v[8 * q + 7] * sn.w, v[8 * q + 6] * sn.w + v[8 * q + 7] * cs.w);
      d4[q] = o;
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 o;
      o.x = pack_half2(v[8 * q], v[8 * q + 1]);
      o.y = pack_half2(v[8 * q + 2], v[8 * q + 3]);
      o.z = pack_half2(v[8 * q + 4], v[8 * q + 5]);
      o.w = pack_half2(v[8 * q + 6], v[8 * q + 7]);
      d4[q] = o;
    }
  }
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

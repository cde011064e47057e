// Epilogues of the linear-layer kernels: what happens to a finished fp32 accumulator.
// Every kernel of the family (reference, weight-streaming, tensor-core) funnels its results
// through these functions, two adjacent output columns at a time, so that they all round and
// store identically.
#pragma once

#include "es_internal.cuh"

namespace es {

// silu(z) = z / (1 + e^-z) with the fast exponential and the fast division (2 ulp; a denominator beyond 2^126, i.e.
// z below about -87, gives 0 where the exact value is below 1e-36 in magnitude).  Every kernel path uses this one.
__device__ __forceinline__ float silu_f(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

// Sequence and prompt offset of row m of a prefill: m / T and m % T, or with packed prompts the sequence whose row
// range holds m (binary search over the first-row table) and the offset inside it.
__device__ __forceinline__ void row_to_seq(const LinearParams& p, int m, int& b, int& off) {
  if (p.cu_rows == nullptr) {
    b = m / p.T;
    off = m - b * p.T;
    return;
  }
  int lo = 0, hi = p.n_seq;                  // invariant: cu_rows[lo] <= m < cu_rows[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.cu_rows[mid] <= m) lo = mid; else hi = mid;
  }
  b = lo;
  off = m - p.cu_rows[lo];
}

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
  int b, row_off;
  row_to_seq(p, m, b, row_off);
  const int slot = p.slots[b];
  const int pos = p.is_decode ? p.ctx_len[slot] : row_off;
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

// SwiGLU of 32 adjacent columns of row m, packed as 32 fp16 values; dst = where they go (nullptr: row past M).
// False when the chunk is ragged or unaligned and must take the element-wise path (same for every row).
__device__ __forceinline__ bool swiglu_chunk32_fast(const LinearParams& p, int n) {
  return (n + 32 <= p.N) && ((p.ldo & 7) == 0) && ((n & 7) == 0) && (((uintptr_t)p.out_f16 & 15) == 0);
}
__device__ __forceinline__ void swiglu_pack32(const LinearParams& p, int m, int n, const float (&g)[32], const float (&u)[32],
                                              uint4 (&o)[4], __half*& dst) {
  dst = (m < p.M) ? p.out_f16 + (int64_t)m * p.ldo + n : nullptr;
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    o[q].x = pack_half2(silu_f(g[8 * q]) * u[8 * q], silu_f(g[8 * q + 1]) * u[8 * q + 1]);
    o[q].y = pack_half2(silu_f(g[8 * q + 2]) * u[8 * q + 2], silu_f(g[8 * q + 3]) * u[8 * q + 3]);
    o[q].z = pack_half2(silu_f(g[8 * q + 4]) * u[8 * q + 4], silu_f(g[8 * q + 5]) * u[8 * q + 5]);
    o[q].w = pack_half2(silu_f(g[8 * q + 6]) * u[8 * q + 6], silu_f(g[8 * q + 7]) * u[8 * q + 7]);
  }
}

__device__ __forceinline__ void epi_swiglu_chunk32(const LinearParams& p, int m, int n, const float (&g)[32],
                                                   const float (&u)[32]) {
  if (m >= p.M || n >= p.N) return;
  if (!swiglu_chunk32_fast(p, n)) {
#pragma unroll
    for (int j = 0; j < 32; ++j) epi_swiglu(p, m, n + j, g[j], u[j]);
    return;
  }
  uint4 o[4];
  __half* dst;
  swiglu_pack32(p, m, n, g, u, o, dst);
#pragma unroll
  for (int q = 0; q < 4; ++q) reinterpret_cast<uint4*>(dst)[q] = o[q];
}

// 32 columns of the fused [q | k | v] projection; n is a multiple of 32, so the chunk lies inside one
// head of one segment (head_dim is 64 or 128).
__device__ __forceinline__ bool qkv_chunk32_fast(const LinearParams& p, int n) {
  return (n + 32 <= p.N) && ((n & 31) == 0) && ((p.hd & 31) == 0);
}
// What a row of the fused QKV product needs from memory, the same for every column chunk of the row: its
// position (for the rotation table), its row of the q output and its token's place in the KV pages.
struct QkvRow {
  bool valid;            // row < M and position inside the tables
  int rope_off;          // pos * (hd / 2): offset of the row's cos / sin entries
  int64_t q_off;         // m * Hq * hd
  int64_t kv_off;        // (page * Hkv * P + pos % P) * hd: head 0, column 0 of the token in a K or V page
};
__device__ __forceinline__ QkvRow qkv_row(const LinearParams& p, int m) {
  QkvRow r;
  r.valid = false;
  r.rope_off = 0; r.q_off = 0; r.kv_off = 0;
  if (m >= p.M) return r;
  int b, off;
  row_to_seq(p, m, b, off);
  const int slot = p.slots[b];
  const int pos = p.is_decode ? p.ctx_len[slot] : off;
  if (pos < 0 || pos >= p.max_seq) return r;
  const int page = p.block_table[(int64_t)slot * p.pages_per_slot + pos / p.P];
  r.valid = true;
  r.rope_off = pos * (p.hd / 2);
  r.q_off = (int64_t)m * p.Hq * p.hd;
  r.kv_off = ((int64_t)page * p.Hkv * p.P + (pos % p.P)) * p.hd;
  return r;
}
// Rotated / rounded values of the chunk as 32 fp16 and their destination (nullptr: nothing to store for this row).
__device__ __forceinline__ void qkv_pack32_row(const LinearParams& p, const QkvRow& row, int n, const float (&v)[32],
                                               uint4 (&o)[4], __half*& dst) {
  dst = nullptr;
  if (!row.valid) return;
  const int nq = p.Hq * p.hd, nkv = p.Hkv * p.hd;
  const bool is_q = n < nq, is_k = !is_q && n < nq + nkv;
  const int local = is_q ? n : (is_k ? n - nq : n - nq - nkv);
  const int head = local / p.hd, c0 = local - head * p.hd;
  if (is_q) dst = p.out_f16 + row.q_off + n;
  else dst = (is_k ? p.k_cache : p.v_cache) + row.kv_off + (int64_t)head * p.P * p.hd + c0;
  if (is_q || is_k) {
    const float4* cs4 = reinterpret_cast<const float4*>(p.rope_cos + row.rope_off + c0 / 2);
    const float4* sn4 = reinterpret_cast<const float4*>(p.rope_sin + row.rope_off + c0 / 2);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 cs = cs4[q], sn = sn4[q];
      o[q].x = pack_half2(v[8 * q] * cs.x - v[8 * q + 1] * sn.x, v[8 * q] * sn.x + v[8 * q + 1] * cs.x);
      o[q].y = pack_half2(v[8 * q + 2] * cs.y - v[8 * q + 3] * sn.y, v[8 * q + 2] * sn.y + v[8 * q + 3] * cs.y);
      o[q].z = pack_half2(v[8 * q + 4] * cs.z - v[8 * q + 5] * sn.z, v[8 * q + 4] * sn.z + v[8 * q + 5] * cs.z);
      o[q].w = pack_half2(v[8 * q + 6] * cs.w - v[8 * q + 7] * sn.w, v[8 * q + 6] * sn.w + v[8 * q + 7] * cs.w);
    }
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      o[q].x = pack_half2(v[8 * q], v[8 * q + 1]);
      o[q].y = pack_half2(v[8 * q + 2], v[8 * q + 3]);
      o[q].z = pack_half2(v[8 * q + 4], v[8 * q + 5]);
      o[q].w = pack_half2(v[8 * q + 6], v[8 * q + 7]);
    }
  }
}
__device__ __forceinline__ void qkv_pack32(const LinearParams& p, int m, int n, const float (&v)[32], uint4 (&o)[4], __half*& dst) {
  qkv_pack32_row(p, qkv_row(p, m), n, v, o, dst);
}

__device__ __forceinline__ void epi_qkv_chunk32(const LinearParams& p, int m, int n, const float (&v)[32]) {
  if (m >= p.M || n >= p.N) return;
  if (!qkv_chunk32_fast(p, n)) {
#pragma unroll
    for (int j = 0; j < 32; j += 2) epi_qkv_pair(p, m, n + j, v[j], v[j + 1]);
    return;
  }
  uint4 o[4];
  __half* dst;
  qkv_pack32(p, m, n, v, o, dst);
  if (dst == nullptr) return;
#pragma unroll
  for (int q = 0; q < 4; ++q) reinterpret_cast<uint4*>(dst)[q] = o[q];
}

// epi_qkv_pair with the row's lookups (slot, position, page) done once by the caller: row = qkv_row(p, m).
__device__ __forceinline__ void epi_qkv_pair_row(const LinearParams& p, const QkvRow& row, int n, float v0, float v1) {
  if (!row.valid || n >= p.N) return;
  const int nq = p.Hq * p.hd, nkv = p.Hkv * p.hd;
  if (n < nq + nkv) {
    const int c = (n < nq ? n : n - nq) % p.hd;
    const int i = c >> 1;
    const float cs = p.rope_cos[row.rope_off + i];
    const float sn = p.rope_sin[row.rope_off + i];
    const float r0 = v0 * cs - v1 * sn;
    const float r1 = v0 * sn + v1 * cs;
    v0 = r0;
    v1 = r1;
  }
  const __half2 hv = __floats2half2_rn(v0, v1);
  if (n < nq) {
    *reinterpret_cast<__half2*>(p.out_f16 + row.q_off + n) = hv;
    return;
  }
  const bool is_k = n < nq + nkv;
  const int kn = is_k ? n - nq : n - nq - nkv;
  const int g = kn / p.hd;
  const int c = kn - g * p.hd;
  *reinterpret_cast<__half2*>((is_k ? p.k_cache : p.v_cache) + row.kv_off + (int64_t)g * p.P * p.hd + c) = hv;
}

// epi_pair for a caller that finishes many pairs of the same row m: row = qkv_row(p, m) (used by the QKV form only)
template <int EPI>
__device__ __forceinline__ void epi_pair_row(const LinearParams& p, const QkvRow& row, int m, int n, float v0, float v1) {
  if (EPI == EPI_QKV) epi_qkv_pair_row(p, row, n, v0, v1);
  else epi_pair<EPI>(p, m, n, v0, v1);
}

// ---- the same chunks stored through a per-warp shared-memory tile -------------------------------
// A thread that owns 32 adjacent columns of ONE row would store 16 bytes into a row of its own: 32 rows per
// instruction, half a 32-byte sector each.  The variants below are called by a whole warp whose lane l owns
// row m0 + l; they pass the chunk through `stage` (shared memory private to the warp) and then store it with
// several lanes per row, so that every instruction writes (and, for the residual, reads) whole row segments.
// The arithmetic is that of the functions above.
constexpr int EPI_STAGE_BYTES = 32 * 80 + 32 * 8;   // fp16 chunks: 32 rows of 64 bytes in 80-byte rows, then one pointer per row

// After the turn-around lane l holds, for i = 0..3, piece (l >> 3) of row i * 8 + (l & 7).
__device__ __forceinline__ int staged_row(int i, int lane) { return i * 8 + (lane & 7); }
__device__ __forceinline__ int staged_piece(int lane) { return lane >> 3; }

// in: o = this lane's row, 64 bytes.  out: t[i] = piece staged_piece(lane) of row staged_row(i, lane).
__device__ __forceinline__ void stage_turn(const uint4 (&o)[4], uint4 (&t)[4], unsigned char* stage, int lane) {
  uint4* tile = reinterpret_cast<uint4*>(stage);                      // rows of 5 x 16 bytes (4 used): conflict-free both ways
#pragma unroll
  for (int q = 0; q < 4; ++q) tile[lane * 5 + q] = o[q];
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) t[i] = tile[staged_row(i, lane) * 5 + staged_piece(lane)];
  __syncwarp();
}

// 32 fp16 values per row (o) to dst (nullptr = skip the row)
__device__ __forceinline__ void rows16_store_staged(__half* dst, const uint4 (&o)[4], unsigned char* stage, int lane) {
  unsigned long long* rowptr = reinterpret_cast<unsigned long long*>(stage + 32 * 80);
  rowptr[lane] = reinterpret_cast<unsigned long long>(dst);
  uint4 t[4];
  stage_turn(o, t, stage, lane);                 // its first __syncwarp also publishes rowptr
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __half* d = reinterpret_cast<__half*>(rowptr[staged_row(i, lane)]);
    if (d != nullptr) reinterpret_cast<uint4*>(d)[staged_piece(lane)] = t[i];
  }
  __syncwarp();                                  // rowptr is rewritten by the next call
}

// fp32 chunks turn around as a whole 32 x 32 tile (rows of 36 words: conflict-free both ways), so that eight
// lanes cover the 128 bytes of a row and every store writes whole lines.
constexpr int EPI_STAGE_F32_BYTES = 32 * 36 * 4;

__device__ __forceinline__ bool f32_chunk32_fast(const float* out, const float* res, int64_t ldo, int N, int n) {
  return (n + 32 <= N) && ((ldo & 3) == 0) && ((n & 3) == 0) && (((uintptr_t)out & 15) == 0) &&
         (res == nullptr || ((uintptr_t)res & 15) == 0);
}
// The residual values this lane will add for the chunk at column n (row i * 4 + lane / 8, columns (lane % 8) * 4 ..),
// fetched ahead of time.  Nothing is loaded (and rv is left alone) when there is no residual or the chunk takes
// the element-wise path.
__device__ __forceinline__ void f32_chunk32_load_res(const float* out, const float* res, int64_t ldo, int M, int N, int m0,
                                                     int n, int lane, float4 (&rv)[8]) {
  if (res == nullptr || n >= N || !f32_chunk32_fast(out, res, ldo, N, n)) return;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int m = m0 + i * 4 + (lane >> 3);
    rv[i] = (m < M) ? __ldcs(reinterpret_cast<const float4*>(res + (int64_t)m * ldo + n + (lane & 7) * 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

// out[m, n .. n+31] = v (+ res[m, n .. n+31]) for the 32 rows m0 + lane; out / res row stride ldo; rows >= M and
// columns >= N are skipped.  res may alias out (a thread reads and writes exactly the same elements, so its loads
// may be hoisted above its stores).  PRELOADED: rv already holds what f32_chunk32_load_res fetched for this chunk.
// stage: EPI_STAGE_F32_BYTES of shared memory private to the warp.
template <bool PRELOADED>
__device__ __forceinline__ void f32_chunk32_staged(float* out, const float* res, int64_t ldo, int M, int N, int m0, int n,
                                                   const float (&v)[32], float4 (&rv)[8], unsigned char* stage, int lane) {
  if (n >= N) return;
  if (!f32_chunk32_fast(out, res, ldo, N, n)) {   // same decision in every lane: element-wise, one row per thread
    const int m = m0 + lane;
    if (m < M) {
      const int64_t o = (int64_t)m * ldo + n;
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (n + j < N) out[o + j] = (res != nullptr) ? v[j] + res[o + j] : v[j];
    }
    return;
  }
  if (!PRELOADED) f32_chunk32_load_res(out, res, ldo, M, N, m0, n, lane, rv);
  float* tile = reinterpret_cast<float*>(stage);
#pragma unroll
  for (int q = 0; q < 8; ++q)
    *reinterpret_cast<float4*>(tile + lane * 36 + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
  __syncwarp();
  const int cq = (lane & 7) * 4;                  // eight lanes cover the 128 bytes of one row
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int rr = i * 4 + (lane >> 3);
    const int m = m0 + rr;
    if (m < M) {
      float4 x = *reinterpret_cast<const float4*>(tile + rr * 36 + cq);
      if (res != nullptr) x = make_float4(x.x + rv[i].x, x.y + rv[i].y, x.z + rv[i].z, x.w + rv[i].w);
      *reinterpret_cast<float4*>(out + (int64_t)m * ldo + n + cq) = x;
    }
  }
  __syncwarp();
}

__device__ __forceinline__ void epi_f32_chunk32_staged(const LinearParams& p, int m0, int n, const float (&v)[32],
                                                       unsigned char* stage, int lane) {
  float4 rv[8];
  f32_chunk32_staged<false>(p.out_f32, p.res, p.ldo, p.M, p.N, m0, n, v, rv, stage, lane);
}

__device__ __forceinline__ void epi_swiglu_chunk32_staged(const LinearParams& p, int m0, int n, const float (&g)[32],
                                                          const float (&u)[32], unsigned char* stage, int lane) {
  if (n >= p.N) return;
  if (!swiglu_chunk32_fast(p, n)) {
    epi_swiglu_chunk32(p, m0 + lane, n, g, u);
    return;
  }
  uint4 o[4];
  __half* dst;
  swiglu_pack32(p, m0 + lane, n, g, u, o, dst);
  rows16_store_staged(dst, o, stage, lane);
}

// row = qkv_row(p, m0 + lane), computed once per tile
__device__ __forceinline__ void epi_qkv_chunk32_staged(const LinearParams& p, const QkvRow& row, int m0, int n,
                                                       const float (&v)[32], unsigned char* stage, int lane) {
  if (n >= p.N) return;
  if (!qkv_chunk32_fast(p, n)) {
    epi_qkv_chunk32(p, m0 + lane, n, v);
    return;
  }
  uint4 o[4];
  __half* dst;
  qkv_pack32_row(p, row, n, v, o, dst);
  rows16_store_staged(dst, o, stage, lane);
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

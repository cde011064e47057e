// Memory-bound helpers of the path: embedding gather, RMSNorm, greedy argmax, context counters.
#include <cooperative_groups.h>

#include "es_internal.cuh"
#include "launch.cuh"

namespace es {

namespace {

// x[m, :] = table[ids[m], :] widened to fp32.  One CTA per row.
__global__ void embed_kernel(const int* __restrict__ ids, const __half* __restrict__ table,
                             float* __restrict__ x, int d, int vocab, unsigned long long* stamp) {
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int m = blockIdx.x;
  int id = ids[m];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);   // out-of-range ids are clamped, never dereferenced
  const uint4* src = reinterpret_cast<const uint4*>(table + (int64_t)id * d);
  float4* dst = reinterpret_cast<float4*>(x + (int64_t)m * d);
  for (int c = threadIdx.x; c < d / 8; c += blockDim.x) {
    const uint4 v = __ldg(src + c);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
    const float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
    const float2 e = __half22float2(h[2]), f = __half22float2(h[3]);
    dst[2 * c] = make_float4(a.x, a.y, b.x, b.y);
    dst[2 * c + 1] = make_float4(e.x, e.y, f.x, f.y);
  }
  stamp_end(stamp);
}

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) red[warp] = v;
  __syncthreads();
  const int nw = blockDim.x >> 5;
  float t = (lane < nw) ? red[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  __syncthreads();
  return t;
}

// One CTA per row; the row stays in registers between the two passes (THREADS x REGS float4, i.e.
// d <= 8192); longer rows are re-read.  Two shapes: 256 threads x 8 when there are many rows,
// 1024 x 2 for decode steps and short prompts (a row then has four times the threads).  The
// split-K reduction below uses the same two shapes and the same order of additions, so a row
// normalised there and a row normalised here agree bit for bit.
constexpr int RMS_THREADS = 256;
constexpr int RMS_REGS = 8;
constexpr int WIDE_ROWS_MAX = 256;     // up to this many rows: 1024 threads per row (too few rows to fill the machine otherwise)

template <int THREADS, int REGS>
__global__ void __launch_bounds__(THREADS) rmsnorm_kernel(const float* __restrict__ x,
                                                              const __half* __restrict__ gain,
                                                              __half* __restrict__ y, int d, float eps,
                                                              int64_t row_stride, int64_t row_offset,
                                                              const int* __restrict__ last_of, unsigned long long* stamp) {
  __shared__ float red[32];
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int r = blockIdx.x;
  // source row: r * row_stride + row_offset, or with last_of the last of the first last_of[r] rows of block r
  const int64_t off = last_of ? (int64_t)last_of[r] - 1 : row_offset;
  const float4* src = reinterpret_cast<const float4*>(x + ((int64_t)r * row_stride + off) * d);
  const int n4 = d / 4;
  float4 v[REGS];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < REGS; ++i) {
    const int c = threadIdx.x + i * THREADS;
    if (c < n4) {
      v[i] = src[c];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  for (int c = threadIdx.x + REGS * THREADS; c < n4; c += THREADS) {
    const float4 t = src[c];
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  const float total = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(total / (float)d + eps);
  __half2* dst = reinterpret_cast<__half2*>(y + (int64_t)r * d);
  const __half2* g2 = reinterpret_cast<const __half2*>(gain);
#pragma unroll
  for (int i = 0; i < REGS; ++i) {
    const int c = threadIdx.x + i * THREADS;
    if (c < n4) {
      const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
      dst[2 * c] = __floats2half2_rn(v[i].x * inv * ga.x, v[i].y * inv * ga.y);
      dst[2 * c + 1] = __floats2half2_rn(v[i].z * inv * gb.x, v[i].w * inv * gb.y);
    }
  }
  for (int c = threadIdx.x + REGS * THREADS; c < n4; c += THREADS) {
    const float4 t = src[c];
    const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
    dst[2 * c] = __floats2half2_rn(t.x * inv * ga.x, t.y * inv * ga.y);
    dst[2 * c + 1] = __floats2half2_rn(t.z * inv * gb.x, t.w * inv * gb.y);
  }
  stamp_end(stamp);
}

// Finishes a split-K product: out[r, :] = (res ? res[r, :] : 0) + part[0, r, :] + part[1, r, :] + ...
// (slices in ascending order, so the sum does not depend on scheduling) and, with a gain vector, the
// RMSNorm of the finished row in fp16 for the next product — one CTA per row, the row kept in
// registers between the two passes like rmsnorm_kernel does.  THREADS x REGS float4 columns stay in
// registers (prefill: many rows, 256 threads; decode: up to 16 rows, 1024 threads each).
template <int THREADS, int REGS>
__global__ void __launch_bounds__(THREADS) splitk_reduce_kernel(const float* __restrict__ part, int k_splits,
                                                                const float* res, float* out, int M, int N,
                                                                int64_t ldo, const __half* __restrict__ gain,
                                                                __half* __restrict__ y, float eps, unsigned long long* stamp) {
  __shared__ float red[32];
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int r = blockIdx.x;
  const int n4 = N / 4;
  const int64_t slice4 = (int64_t)M * N / 4;
  const float4* src = reinterpret_cast<const float4*>(part + (int64_t)r * N);
  const float4* rs = res ? reinterpret_cast<const float4*>(res + (int64_t)r * ldo) : nullptr;
  float4* dst = reinterpret_cast<float4*>(out + (int64_t)r * ldo);
  // a = the residual element; then the slices, eight requested at a time and added in slice order
  auto finish = [&](int c, float4 a) {
    for (int s0 = 0; s0 < k_splits; s0 += 8) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        v[j] = (s0 + j < k_splits) ? __ldcs(src + (s0 + j) * slice4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (s0 + j < k_splits) { a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w; }
    }
    dst[c] = a;
    return a;
  };
  float4 v[REGS];
  float ss = 0.f;
  // The residual may alias the output, so the compiler cannot move a column's residual load above the previous
  // column's store and a thread would wait out one memory round trip per column; a thread reads and writes only
  // its own elements, so all its residual elements are requested up front.
#pragma unroll
  for (int i = 0; i < REGS; ++i) {
    const int c = threadIdx.x + i * THREADS;
    v[i] = (rs && c < n4) ? rs[c] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  // The slices of ALL of a thread's register-resident columns are requested four slices at a time before anything
  // is added or stored (one memory round trip per four slices instead of one per column); every element is still
  // residual + slice 0 + slice 1 + ... in that order.
  constexpr int SB = 4;
  for (int s0 = 0; s0 < k_splits; s0 += SB) {
    float4 t[REGS][SB];
#pragma unroll
    for (int i = 0; i < REGS; ++i) {
      const int c = threadIdx.x + i * THREADS;
#pragma unroll
      for (int j = 0; j < SB; ++j)
        t[i][j] = (c < n4 && s0 + j < k_splits) ? __ldcs(src + (s0 + j) * slice4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < REGS; ++i)
#pragma unroll
      for (int j = 0; j < SB; ++j)
        if (s0 + j < k_splits) { v[i].x += t[i][j].x; v[i].y += t[i][j].y; v[i].z += t[i][j].z; v[i].w += t[i][j].w; }
  }
#pragma unroll
  for (int i = 0; i < REGS; ++i) {
    const int c = threadIdx.x + i * THREADS;
    if (c < n4) {
      dst[c] = v[i];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  for (int c = threadIdx.x + REGS * THREADS; c < n4; c += THREADS) {
    const float4 t = finish(c, rs ? rs[c] : make_float4(0.f, 0.f, 0.f, 0.f));
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  if (gain == nullptr) { stamp_end(stamp); return; }   // uniform over the CTA
  const float total = block_sum(ss, red);
  const float inv = 1.0f / sqrtf(total / (float)N + eps);
  __half2* yd = reinterpret_cast<__half2*>(y + (int64_t)r * N);
  const __half2* g2 = reinterpret_cast<const __half2*>(gain);
#pragma unroll
  for (int i = 0; i < REGS; ++i) {
    const int c = threadIdx.x + i * THREADS;
    if (c < n4) {
      const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
      yd[2 * c] = __floats2half2_rn(v[i].x * inv * ga.x, v[i].y * inv * ga.y);
      yd[2 * c + 1] = __floats2half2_rn(v[i].z * inv * gb.x, v[i].w * inv * gb.y);
    }
  }
  for (int c = threadIdx.x + REGS * THREADS; c < n4; c += THREADS) {
    const float4 t = dst[c];                         // written by this thread above
    const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
    yd[2 * c] = __floats2half2_rn(t.x * inv * ga.x, t.y * inv * ga.y);
    yd[2 * c + 1] = __floats2half2_rn(t.z * inv * gb.x, t.w * inv * gb.y);
  }
  stamp_end(stamp);
}

// ---- up to 16 rows (decode steps of several sequences): a cluster of ROW_CTAS CTAs per row ------------------
// With one CTA per row a 16-row launch runs on 16 SMs, and what one SM can pull in per microsecond bounds it: the
// reduction of a product cut into 16 K slices reads 0.5 MB per row.  Here the columns of a row are cut into
// ROW_CTAS contiguous parts, one per CTA of a thread-block cluster; each CTA adds up the squares of its part, the
// parts' sums are exchanged through the cluster's shared memory and added in part order by every CTA, and each CTA
// then normalises its own part.  Both kernels below use this one order of additions, so a row normalised in the
// reduction and the same row normalised by the stand-alone kernel agree bit for bit.
constexpr int ROW_CTAS = 8;
constexpr int ROW_THREADS = 256;
constexpr int ROW_REGS = 2;            // float4 columns per thread kept in registers (covers N <= 16384)

// Sum of the ROW_CTAS per-CTA values, the same in every CTA of the cluster.  All threads of all CTAs call.
__device__ __forceinline__ float cluster_row_total(float mine, float* parts /* [ROW_CTAS] shared */) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster.block_rank();
  if (threadIdx.x < ROW_CTAS) *cluster.map_shared_rank(parts + rank, threadIdx.x) = mine;   // my value into everybody's slot
  cluster.sync();
  float total = 0.f;
#pragma unroll
  for (int r = 0; r < ROW_CTAS; ++r) total += parts[r];
  return total;
}

// y[r, :] = rmsnorm(x[row r]) for M <= 16 rows; grid = M clusters of ROW_CTAS CTAs; N % (4 * ROW_CTAS) == 0.
__global__ void __launch_bounds__(ROW_THREADS) rmsnorm_rows_kernel(const float* __restrict__ x, const __half* __restrict__ gain,
                                                                   __half* __restrict__ y, int d, float eps, int64_t row_stride,
                                                                   int64_t row_offset, const int* __restrict__ last_of,
                                                                   unsigned long long* stamp) {
  __shared__ float red[32];
  __shared__ float parts[ROW_CTAS];
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int r = blockIdx.x / ROW_CTAS, part = blockIdx.x % ROW_CTAS;
  const int64_t off = last_of ? (int64_t)last_of[r] - 1 : row_offset;
  const int n4 = d / 4 / ROW_CTAS, lo = part * n4;                  // this CTA's float4 columns [lo, lo + n4)
  const float4* src = reinterpret_cast<const float4*>(x + ((int64_t)r * row_stride + off) * d) + lo;
  float4 v[ROW_REGS];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < ROW_REGS; ++i) {
    const int c = threadIdx.x + i * ROW_THREADS;
    if (c < n4) {
      v[i] = src[c];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  for (int c = threadIdx.x + ROW_REGS * ROW_THREADS; c < n4; c += ROW_THREADS) {
    const float4 t = src[c];
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  const float total = cluster_row_total(block_sum(ss, red), parts);
  const float inv = 1.0f / sqrtf(total / (float)d + eps);
  __half2* dst = reinterpret_cast<__half2*>(y + (int64_t)r * d) + 2 * lo;
  const __half2* g2 = reinterpret_cast<const __half2*>(gain) + 2 * lo;
#pragma unroll
  for (int i = 0; i < ROW_REGS; ++i) {
    const int c = threadIdx.x + i * ROW_THREADS;
    if (c < n4) {
      const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
      dst[2 * c] = __floats2half2_rn(v[i].x * inv * ga.x, v[i].y * inv * ga.y);
      dst[2 * c + 1] = __floats2half2_rn(v[i].z * inv * gb.x, v[i].w * inv * gb.y);
    }
  }
  for (int c = threadIdx.x + ROW_REGS * ROW_THREADS; c < n4; c += ROW_THREADS) {
    const float4 t = src[c];
    const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
    dst[2 * c] = __floats2half2_rn(t.x * inv * ga.x, t.y * inv * ga.y);
    dst[2 * c + 1] = __floats2half2_rn(t.z * inv * gb.x, t.w * inv * gb.y);
  }
  stamp_end(stamp);
}

// The split-K reduction for M <= 16 rows, same cluster shape: out[r, :] = res[r, :] + slices in ascending order,
// then (with gain) y[r, :] = rmsnorm(out[r, :]).
__global__ void __launch_bounds__(ROW_THREADS) splitk_reduce_rows_kernel(const float* __restrict__ part, int k_splits, const float* res,
                                                                         float* out, int M, int N, int64_t ldo,
                                                                         const __half* __restrict__ gain, __half* __restrict__ y,
                                                                         float eps, unsigned long long* stamp) {
  __shared__ float red[32];
  __shared__ float parts[ROW_CTAS];
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int r = blockIdx.x / ROW_CTAS, pt = blockIdx.x % ROW_CTAS;
  const int n4 = N / 4 / ROW_CTAS, lo = pt * n4;
  const int64_t slice4 = (int64_t)M * N / 4;
  const float4* src = reinterpret_cast<const float4*>(part + (int64_t)r * N) + lo;
  const float4* rs = res ? reinterpret_cast<const float4*>(res + (int64_t)r * ldo) + lo : nullptr;
  float4* dst = reinterpret_cast<float4*>(out + (int64_t)r * ldo) + lo;
  auto finish = [&](int c, float4 a) {
    for (int s0 = 0; s0 < k_splits; s0 += 8) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j)
        v[j] = (s0 + j < k_splits) ? __ldcs(src + (s0 + j) * slice4 + c) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (s0 + j < k_splits) { a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w; }
    }
    dst[c] = a;
    return a;
  };
  float4 v[ROW_REGS];
  float ss = 0.f;
  // the residual may alias the output: all of a thread's residual elements are requested before it stores anything
#pragma unroll
  for (int i = 0; i < ROW_REGS; ++i) {
    const int c = threadIdx.x + i * ROW_THREADS;
    v[i] = (rs && c < n4) ? rs[c] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int i = 0; i < ROW_REGS; ++i) {
    const int c = threadIdx.x + i * ROW_THREADS;
    if (c < n4) {
      v[i] = finish(c, v[i]);
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  for (int c = threadIdx.x + ROW_REGS * ROW_THREADS; c < n4; c += ROW_THREADS) {
    const float4 t = finish(c, rs ? rs[c] : make_float4(0.f, 0.f, 0.f, 0.f));
    ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
  }
  if (gain == nullptr) { stamp_end(stamp); return; }   // uniform over the cluster
  const float total = cluster_row_total(block_sum(ss, red), parts);
  const float inv = 1.0f / sqrtf(total / (float)N + eps);
  __half2* yd = reinterpret_cast<__half2*>(y + (int64_t)r * N) + 2 * lo;
  const __half2* g2 = reinterpret_cast<const __half2*>(gain) + 2 * lo;
#pragma unroll
  for (int i = 0; i < ROW_REGS; ++i) {
    const int c = threadIdx.x + i * ROW_THREADS;
    if (c < n4) {
      const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
      yd[2 * c] = __floats2half2_rn(v[i].x * inv * ga.x, v[i].y * inv * ga.y);
      yd[2 * c + 1] = __floats2half2_rn(v[i].z * inv * gb.x, v[i].w * inv * gb.y);
    }
  }
  for (int c = threadIdx.x + ROW_REGS * ROW_THREADS; c < n4; c += ROW_THREADS) {
    const float4 t = dst[c];                         // written by this thread above
    const float2 ga = __half22float2(g2[2 * c]), gb = __half22float2(g2[2 * c + 1]);
    yd[2 * c] = __floats2half2_rn(t.x * inv * ga.x, t.y * inv * ga.y);
    yd[2 * c + 1] = __floats2half2_rn(t.z * inv * gb.x, t.w * inv * gb.y);
  }
  stamp_end(stamp);
}

// Launch of the cluster kernels: M clusters of ROW_CTAS CTAs.
template <typename... KArgs, typename... Args>
cudaError_t launch_row_clusters(void (*kernel)(KArgs...), int M, cudaStream_t stream, bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(M * ROW_CTAS);
  cfg.blockDim = dim3(ROW_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = ROW_CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Where the cluster kernels are used: few rows (one CTA per row would leave most SMs idle) that are long (the
// slices of a wide product are what one SM cannot pull in fast enough).  Measured per layer, in a replayed step:
// 16 rows of 8192 columns, 16 slices: 17.3 -> 12.8 us for the two reductions; 8 rows of 4096 columns: 7.1 -> 8.5 us
// (the cluster launch costs more than it saves), hence the width threshold.  The rule depends on the shape only,
// never on the slice count, so the reduction and the stand-alone kernel always agree on it.
constexpr int ROW_CLUSTER_MAX_ROWS = 16;
constexpr int ROW_CLUSTER_MIN_COLS = 8192;
inline bool use_row_clusters(int M, int N) { return M <= ROW_CLUSTER_MAX_ROWS && N >= ROW_CLUSTER_MIN_COLS && N % (4 * ROW_CTAS) == 0; }

// Greedy token: index of the largest logit, the lowest index on ties.  One CTA of 1024 threads per sequence; a
// thread requests up to eight 16-byte pieces of the row at a time (a 256-thread CTA reading one float per
// iteration took 35 us per step for 32000 logits, latency bound).
constexpr int ARGMAX_THREADS = 1024;
__device__ __forceinline__ void argmax_take(float v, int i, float& best, int& idx) {
  if (v > best || (v == best && i < idx)) { best = v; idx = i; }
}
__global__ void __launch_bounds__(ARGMAX_THREADS) argmax_kernel(const float* __restrict__ logits, int* __restrict__ out, int V,
                                                                 unsigned long long* stamp) {
  __shared__ float bv[32];
  __shared__ int bi[32];
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const float* row = logits + (int64_t)blockIdx.x * V;
  float best = -INFINITY;
  int idx = 0x7fffffff;
  if ((V & 3) == 0 && ((uintptr_t)row & 15) == 0) {
    const float4* row4 = reinterpret_cast<const float4*>(row);
    const int n4 = V / 4;
    for (int c0 = threadIdx.x; c0 < n4; c0 += 8 * ARGMAX_THREADS) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int c = c0 + j * ARGMAX_THREADS;
        v[j] = (c < n4) ? row4[c] : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int i = 4 * (c0 + j * ARGMAX_THREADS);
        if (i >= V) continue;                          // a piece past the end of the row
        argmax_take(v[j].x, i, best, idx);
        argmax_take(v[j].y, i + 1, best, idx);
        argmax_take(v[j].z, i + 2, best, idx);
        argmax_take(v[j].w, i + 3, best, idx);
      }
    }
  } else {
    for (int i = threadIdx.x; i < V; i += ARGMAX_THREADS) argmax_take(row[i], i, best, idx);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    argmax_take(ov, oi, best, idx);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { bv[warp] = best; bi[warp] = idx; }
  __syncthreads();
  if (warp == 0) {
    best = bv[lane];
    idx = bi[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
      argmax_take(ov, oi, best, idx);
    }
    if (lane == 0) out[blockIdx.x] = (idx == 0x7fffffff) ? 0 : idx;
  }
  stamp_end(stamp);
}

// ctx_len[slots[b]] = add ? ctx_len[..] + value : value; with `values` the value of row b is values[b]
__global__ void set_ctx_kernel(int* ctx_len, const int* slots, int B, int value, int add, const int* values,
                               unsigned long long* stamp) {
  pdl_launch_dependents();
  stamp_begin(stamp);
  pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) {
    const int s = slots[b];
    const int v = values ? values[b] : value;
    ctx_len[s] = add ? ctx_len[s] + v : v;
  }
  stamp_end(stamp);
}

}  // namespace

es_status_t launch_embed(const int* ids, const __half* table, float* x, int M, int d, int vocab,
                         cudaStream_t s, int64_t* launches, bool pdl, unsigned long long* stamp) {
  if (M <= 0) return ES_OK;
  ES_CUDA_CHECK(launch_kernel(embed_kernel, dim3(M), dim3(128), 0, s, pdl, ids, table, x, d, vocab, stamp));
  if (launches) ++*launches;
  return ES_OK;
}

es_status_t launch_rmsnorm(const float* x, const __half* gain, __half* y, int M, int d, float eps,
                           int64_t row_stride, int64_t row_offset, cudaStream_t s, int64_t* launches, bool pdl,
                           const int* last_of, unsigned long long* stamp) {
  if (M <= 0) return ES_OK;
  if (use_row_clusters(M, d))
    ES_CUDA_CHECK(launch_row_clusters(rmsnorm_rows_kernel, M, s, pdl, x, gain, y, d, eps, row_stride, row_offset, last_of, stamp));
  else if (M <= WIDE_ROWS_MAX)
    ES_CUDA_CHECK(launch_kernel(rmsnorm_kernel<1024, 2>, dim3(M), dim3(1024), 0, s, pdl, x, gain, y, d, eps, row_stride, row_offset, last_of, stamp));
  else
    ES_CUDA_CHECK(launch_kernel(rmsnorm_kernel<RMS_THREADS, RMS_REGS>, dim3(M), dim3(RMS_THREADS), 0, s, pdl, x, gain, y, d, eps, row_stride, row_offset, last_of, stamp));
  if (launches) ++*launches;
  return ES_OK;
}

es_status_t launch_argmax(const float* logits, int* out, int B, int V, cudaStream_t s, int64_t* launches, bool pdl,
                          unsigned long long* stamp) {
  if (B <= 0) return ES_OK;
  ES_CUDA_CHECK(launch_kernel(argmax_kernel, dim3(B), dim3(ARGMAX_THREADS), 0, s, pdl, logits, out, V, stamp));
  if (launches) ++*launches;
  return ES_OK;
}

es_status_t launch_splitk_reduce(const float* part, int k_splits, const float* res, float* out, int M, int N, int64_t ldo,
                                 const __half* gain, __half* y, float eps, cudaStream_t s, int64_t* launches, bool pdl,
                                 unsigned long long* stamp) {
  if (M <= 0 || N <= 0) return ES_OK;
  if (N % 4 != 0 || ldo % 4 != 0) return fail(ES_ERR_SHAPE, "split-K reduction needs N and the row stride to be multiples of 4");
  if (use_row_clusters(M, N))
    ES_CUDA_CHECK(launch_row_clusters(splitk_reduce_rows_kernel, M, s, pdl, part, k_splits, res, out, M, N, ldo, gain, y, eps, stamp));
  else if (M <= WIDE_ROWS_MAX)
    ES_CUDA_CHECK(launch_kernel(splitk_reduce_kernel<1024, 2>, dim3(M), dim3(1024), 0, s, pdl, part, k_splits, res, out, M, N, ldo, gain, y, eps, stamp));
  else
    ES_CUDA_CHECK(launch_kernel(splitk_reduce_kernel<RMS_THREADS, RMS_REGS>, dim3(M), dim3(RMS_THREADS), 0, s, pdl, part, k_splits, res, out, M, N, ldo, gain, y, eps, stamp));
  if (launches) ++*launches;
  return ES_OK;
}

es_status_t launch_set_ctx(int* ctx_len, const int* slots, int B, int value, int add, cudaStream_t s,
                           int64_t* launches, bool pdl, const int* values, unsigned long long* stamp) {
  if (B <= 0) return ES_OK;
  ES_CUDA_CHECK(launch_kernel(set_ctx_kernel, dim3((B + 63) / 64), dim3(64), 0, s, pdl, ctx_len, slots, B, value, add, values, stamp));
  if (launches) ++*launches;
  return ES_OK;
}

}  // namespace es

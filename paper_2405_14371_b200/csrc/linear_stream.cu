// Weight-streaming kernel of the linear-layer family for skinny products (M <= 16 activation
// rows, i.e. decode steps and the LM head).  The product is bound by reading every weight byte
// from HBM exactly once: each warp owns two weight rows at a time, every lane streams 16-byte
// pieces of both rows (coalesced 512-byte warp requests, several in flight per lane, no L1
// allocation), multiplies them against the activation rows held in shared memory and reduces
// with warp shuffles.  Accumulation is fp32 in a fixed order, so results are deterministic.
#include "epilogue.cuh"

namespace es {

namespace {

constexpr int WARPS = 8;
constexpr int UNROLL = 4;

__device__ __forceinline__ uint4 ld_stream(const void* ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

__device__ __forceinline__ void fma8(float& acc, const uint4& w, const uint4& a) {
  const __half2* wh = reinterpret_cast<const __half2*>(&w);
  const __half2* ah = reinterpret_cast<const __half2*>(&a);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 wf = __half22float2(wh[i]);
    const float2 af = __half22float2(ah[i]);
    acc = fmaf(wf.x, af.x, acc);
    acc = fmaf(wf.y, af.y, acc);
  }
}

// A_SMEM: activation rows are copied to shared memory once per CTA; otherwise they are read
// through L1 from global memory (large M*K).
template <int MB, int EPI, bool A_SMEM>
__global__ void __launch_bounds__(WARPS * 32) linear_stream_kernel(const LinearParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* a_s = reinterpret_cast<__half*>(smem_raw);
  const int K = p.K;
  if (A_SMEM) {
    const int chunks = K / 8;
    for (int i = threadIdx.x; i < MB * chunks; i += blockDim.x) {
      const int m = i / chunks, c = i - m * chunks;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (m < p.M) v = *reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + c * 8);
      *reinterpret_cast<uint4*>(a_s + (int64_t)m * K + c * 8) = v;
    }
    __syncthreads();
  }
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n_units = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  const int total_warps = gridDim.x * WARPS;

  for (int unit = blockIdx.x * WARPS + warp; unit < n_units; unit += total_warps) {
    const __half* r0;
    const __half* r1;
    int n;
    if (EPI == EPI_SWIGLU) {
      n = unit;
      r0 = p.w[0] + (int64_t)n * K;
      r1 = p.w[1] + (int64_t)n * K;
    } else {
      n = unit * 2;
      r0 = weight_row(p, n);
      r1 = weight_row(p, n + 1);
      if (r1 == nullptr) r1 = r0;   // odd N: second row is a duplicate that is never stored
    }
    float acc0[MB], acc1[MB];
#pragma unroll
    for (int m = 0; m < MB; ++m) acc0[m] = acc1[m] = 0.f;

    int k = lane * 8;
    for (; k + (UNROLL - 1) * 256 < K; k += UNROLL * 256) {
      uint4 w0[UNROLL], w1[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        w0[u] = ld_stream(r0 + k + u * 256);
        w1[u] = ld_stream(r1 + k + u * 256);
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
#pragma unroll
        for (int m = 0; m < MB; ++m) {
          uint4 a;
          if (A_SMEM) a = *reinterpret_cast<const uint4*>(a_s + (int64_t)m * K + k + u * 256);
          else a = (m < p.M) ? __ldg(reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + k + u * 256))
                             : make_uint4(0, 0, 0, 0);
          fma8(acc0[m], w0[u], a);
          fma8(acc1[m], w1[u], a);
        }
      }
    }
    for (; k < K; k += 256) {
      const uint4 w0 = ld_stream(r0 + k);
      const uint4 w1 = ld_stream(r1 + k);
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        uint4 a;
        if (A_SMEM) a = *reinterpret_cast<const uint4*>(a_s + (int64_t)m * K + k);
        else a = (m < p.M) ? __ldg(reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + k))
                           : make_uint4(0, 0, 0, 0);
        fma8(acc0[m], w0, a);
        fma8(acc1[m], w1, a);
      }
    }
#pragma unroll
    for (int m = 0; m < MB; ++m) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        acc0[m] += __shfl_xor_sync(0xffffffffu, acc0[m], o);
        acc1[m] += __shfl_xor_sync(0xffffffffu, acc1[m], o);
      }
    }
    // lane m finishes activation row m
    float v0 = 0.f, v1 = 0.f;
#pragma unroll
    for (int m = 0; m < MB; ++m)
      if (lane == m) { v0 = acc0[m]; v1 = acc1[m]; }
    if (lane < MB) epi_pair<EPI>(p, lane, n, v0, v1);
  }
}

template <int MB, int EPI>
es_status_t launch_mb(const LinearParams& p, cudaStream_t s) {
  const size_t a_bytes = (size_t)MB * p.K * sizeof(__half);
  const bool a_smem = a_bytes <= 96 * 1024;
  const int n_units = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int ctas_per_sm = a_smem ? (a_bytes > 48 * 1024 ? 2 : (a_bytes > 24 * 1024 ? 4 : 8)) : 8;
  int grid = (n_units + WARPS - 1) / WARPS;
  if (grid > sms * ctas_per_sm) grid = sms * ctas_per_sm;
  if (a_smem) {
    auto kern = linear_stream_kernel<MB, EPI, true>;
    if (a_bytes > 48 * 1024)
      ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)a_bytes));
    kern<<<grid, WARPS * 32, a_bytes, s>>>(p);
  } else {
    linear_stream_kernel<MB, EPI, false><<<grid, WARPS * 32, 0, s>>>(p);
  }
  ES_CUDA_CHECK(cudaGetLastError());
  return ES_OK;
}

template <int EPI>
es_status_t launch_epi(const LinearParams& p, cudaStream_t s) {
  if (p.M <= 1) return launch_mb<1, EPI>(p, s);
  if (p.M <= 2) return launch_mb<2, EPI>(p, s);
  if (p.M <= 4) return launch_mb<4, EPI>(p, s);
  if (p.M <= 8) return launch_mb<8, EPI>(p, s);
  return launch_mb<16, EPI>(p, s);
}

}  // namespace

es_status_t launch_linear_stream(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches) {
  if (p.M <= 0 || p.N <= 0) return ES_OK;
  if (p.M > 16) return fail(ES_ERR_UNSUPPORTED, "weight-streaming kernel takes at most 16 rows, got %d", p.M);
  if (p.K % 8 != 0) return fail(ES_ERR_SHAPE, "K = %d is not a multiple of 8", p.K);
  es_status_t st;
  switch (epi) {
    case EPI_F32: st = launch_epi<EPI_F32>(p, s); break;
    case EPI_SWIGLU: st = launch_epi<EPI_SWIGLU>(p, s); break;
    case EPI_QKV: st = launch_epi<EPI_QKV>(p, s); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

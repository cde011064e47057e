// Plain tiled CUDA-core kernel of the linear-layer family.  It handles every shape (ragged M, N,
// K) and every epilogue, and serves as the on-device cross-check of the tensor-core kernel and
// as the path for shapes the tensor-core kernel does not take.  64x64 output tile, 16-deep K
// slices staged through shared memory as fp32, 4x4 outputs per thread.
#include "epilogue.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <int EPI>
__global__ void __launch_bounds__(256) linear_reference_kernel(const LinearParams p) {
  constexpr bool DUAL = (EPI == EPI_SWIGLU);
  __shared__ float As[TK][TM + 1];
  __shared__ float Bs[DUAL ? 2 : 1][TK][TN + 1];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  stamp_begin(p.stamp);

  float acc[DUAL ? 2 : 1][4][4];
#pragma unroll
  for (int z = 0; z < (DUAL ? 2 : 1); ++z)
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[z][i][j] = 0.f;

  // each thread stages 4 elements of A and 4 of (each) B per K slice
  const int lr = tid >> 2;          // 0..63: tile row (A) / tile column (B)
  const int lk = (tid & 3) * 4;     // 0,4,8,12
  const int am = m0 + lr;
  const __half* arow = (am < p.M) ? p.A + (int64_t)am * p.lda : nullptr;
  const int bn = n0 + lr;
  const __half* brow0;
  const __half* brow1 = nullptr;
  if (DUAL) {
    brow0 = (bn < p.N) ? p.w[0] + (int64_t)bn * p.K : nullptr;
    brow1 = (bn < p.N) ? p.w[1] + (int64_t)bn * p.K : nullptr;
  } else {
    brow0 = (bn < p.N) ? weight_row(p, bn) : nullptr;
  }

  for (int k0 = 0; k0 < p.K; k0 += TK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int k = k0 + lk + e;
      const bool kin = k < p.K;
      As[lk + e][lr] = (arow && kin) ? __half2float(arow[k]) : 0.f;
      Bs[0][lk + e][lr] = (brow0 && kin) ? __half2float(brow0[k]) : 0.f;
      if (DUAL) Bs[DUAL ? 1 : 0][lk + e][lr] = (brow1 && kin) ? __half2float(brow1[k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int z = 0; z < (DUAL ? 2 : 1); ++z) {
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[z][kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[z][i][j] = fmaf(a[i], b[j], acc[z][i][j]);
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    const int n = n0 + tx * 4;
    if (DUAL) {
#pragma unroll
      for (int j = 0; j < 4; ++j) epi_pair<EPI>(p, m, n + j, acc[0][i][j], acc[DUAL ? 1 : 0][i][j]);
    } else {
      epi_pair<EPI>(p, m, n, acc[0][i][0], acc[0][i][1]);
      epi_pair<EPI>(p, m, n + 2, acc[0][i][2], acc[0][i][3]);
    }
  }
  stamp_end(p.stamp);
}

}  // namespace

es_status_t launch_linear_reference(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches) {
  if (p.M <= 0 || p.N <= 0 || p.K <= 0) return ES_OK;
  dim3 grid((p.N + TN - 1) / TN, (p.M + TM - 1) / TM);
  switch (epi) {
    case EPI_F32: linear_reference_kernel<EPI_F32><<<grid, 256, 0, s>>>(p); break;
    case EPI_SWIGLU: linear_reference_kernel<EPI_SWIGLU><<<grid, 256, 0, s>>>(p); break;
    case EPI_QKV: linear_reference_kernel<EPI_QKV><<<grid, 256, 0, s>>>(p); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (launches) ++*launches;
  ES_CUDA_CHECK(cudaGetLastError());
  return ES_OK;
}

}  // namespace es

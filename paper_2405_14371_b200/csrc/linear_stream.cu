// Weight-streaming kernel of the linear-layer family for skinny products (M <= 16 activation
// rows: decode steps and the LM head).  The product is bound by reading every weight byte from
// HBM exactly once, so the kernel is organised around keeping loads in flight:
//
//  * a work unit is a pair of weight rows (adjacent output columns, or the gate row and the up
//    row of one SwiGLU column); the grid is sized to the machine, every CTA owns a contiguous,
//    balanced range of units and its warps take them round-robin;
//  * a warp walks its units as one flat sequence of chunks (2 rows x U x 512 bytes), double
//    buffered in registers: the loads of chunk c+1 are issued before chunk c is consumed, across
//    unit boundaries too; loads are 16-byte, coalesced, and bypass L1;
//  * the first chunk is requested before the programmatic-dependency wait, so the ramp-up of this
//    kernel overlaps the tail of the previous one (weights are never written by a kernel);
//  * the activation rows sit in shared memory; with NORM the CTA builds them itself from the fp32
//    residual stream (fused RMSNorm), saving a launch and a round trip through HBM;
//  * accumulation is fp32, reduced with warp shuffles in a fixed order: results are deterministic.
#include "epilogue.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int WARPS = 8;
constexpr int THREADS = WARPS * 32;

__device__ __forceinline__ uint4 ld_stream(const void* ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

// acc += w * a over 8 fp16 pairs, each product formed exactly and added in fp32 by the
// mixed-precision FMA (fp16 x fp16 + fp32), so no conversion instructions are spent.
__device__ __forceinline__ void fma8(float& acc, const uint4& w, const uint4& a) {
  const uint32_t* wr = reinterpret_cast<const uint32_t*>(&w);
  const uint32_t* ar = reinterpret_cast<const uint32_t*>(&a);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    asm("{\n.reg .b16 wl, wh, al, ah;\n"
        "mov.b32 {wl, wh}, %1;\n"
        "mov.b32 {al, ah}, %2;\n"
        "fma.rn.f32.f16 %0, wl, al, %0;\n"
        "fma.rn.f32.f16 %0, wh, ah, %0;\n}"
        : "+f"(acc)
        : "r"(wr[i]), "r"(ar[i]));
  }
}

template <int MB, int EPI, bool NORM, int U, bool A_SMEM>
__global__ void __launch_bounds__(THREADS, (U == 2 && MB <= 2) ? 4 : 2) linear_stream_kernel(const LinearParams p) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* a_s = reinterpret_cast<__half*>(smem_raw);
  __shared__ float red[WARPS];

  const int K = p.K;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n_units = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  const int u0 = (int)((int64_t)blockIdx.x * n_units / gridDim.x);
  const int u1 = (int)((int64_t)(blockIdx.x + 1) * n_units / gridDim.x);
  const int n_my = (u1 - u0 - warp + WARPS - 1) / WARPS;          // units of this warp (may be <= 0)
  constexpr int CHUNK_K = U * 256;
  const int chunks_per_unit = (K + CHUNK_K - 1) / CHUNK_K;
  const int total = n_my > 0 ? n_my * chunks_per_unit : 0;

  auto unit_rows = [&](int i, const __half*& r0, const __half*& r1) -> int {
    const int u = u0 + warp + i * WARPS;
    if (EPI == EPI_SWIGLU) {
      r0 = p.w[0] + (int64_t)u * K;
      r1 = p.w[1] + (int64_t)u * K;
      return u;
    }
    const int n = u * 2;
    r0 = weight_row(p, n);
    r1 = weight_row(p, n + 1);
    if (r1 == nullptr) r1 = r0;      // odd N: the duplicate row is never stored
    return n;
  };

  // ---- "next chunk to request" cursor ----
  int nxt_i = 0, nxt_cc = 0;
  const __half* nr0 = nullptr;
  const __half* nr1 = nullptr;
  if (total > 0) unit_rows(0, nr0, nr1);
  auto issue = [&](uint4 (&w0)[U], uint4 (&w1)[U]) {
    const int kb = nxt_cc * CHUNK_K + lane * 8;
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int k = kb + j * 256;
      if (k < K) {
        w0[j] = ld_stream(nr0 + k);
        w1[j] = ld_stream(nr1 + k);
      } else {
        w0[j] = make_uint4(0, 0, 0, 0);
        w1[j] = make_uint4(0, 0, 0, 0);
      }
    }
    if (++nxt_cc == chunks_per_unit) {
      nxt_cc = 0;
      if (++nxt_i < n_my) unit_rows(nxt_i, nr0, nr1);
    }
  };

  uint4 b0w0[U], b0w1[U], b1w0[U], b1w1[U];
  if (total > 0) {
    // requested while the previous kernel drains
    issue(b0w0, b0w1);
    if (total > 1) issue(b1w0, b1w1);        // both buffers on their way: HBM stays busy while activations are staged
  }

  // RMSNorm gains are weights too: the first XV float4-columns of every thread are fetched before the wait
  constexpr int XV = 4;                            // covers K <= 4096 with 256 threads; further columns are re-read
  uint2 gpre[XV];
  if (NORM) {
#pragma unroll
    for (int j = 0; j < XV; ++j) {
      const int i = threadIdx.x + j * THREADS;
      gpre[j] = (i < K / 4) ? __ldg(reinterpret_cast<const uint2*>(p.norm_gain) + i) : make_uint2(0, 0);
    }
  }

  pdl_wait();

  // ---- activation rows -> shared memory ----
  if (A_SMEM) {
    if (NORM) {
      // fused RMSNorm of the fp32 residual rows (K == d_model)
      for (int m = 0; m < MB; ++m) {
        if (m >= p.M) {
          for (int i = threadIdx.x; i < K / 8; i += THREADS) *reinterpret_cast<uint4*>(a_s + (int64_t)m * K + i * 8) = make_uint4(0, 0, 0, 0);
          continue;
        }
        const float4* xr = reinterpret_cast<const float4*>(p.norm_x + (int64_t)m * p.norm_ldx);
        float4 xv[XV];                             // this thread's first XV float4-columns stay in registers
#pragma unroll
        for (int j = 0; j < XV; ++j) {
          const int i = threadIdx.x + j * THREADS;
          xv[j] = (i < K / 4) ? xr[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < XV; ++j) {
          const float4 v = xv[j];
          if (threadIdx.x + j * THREADS < K / 4) ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        for (int i = threadIdx.x + XV * THREADS; i < K / 4; i += THREADS) {
          const float4 v = xr[i];
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if (lane == 0) red[warp] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) tot += red[w];
        __syncthreads();
        const float inv = 1.0f / sqrtf(tot / (float)K + p.norm_eps);
        const __half2* g2 = reinterpret_cast<const __half2*>(p.norm_gain);
        __half2* dst = reinterpret_cast<__half2*>(a_s + (int64_t)m * K);
#pragma unroll
        for (int j = 0; j < XV; ++j) {
          const int i = threadIdx.x + j * THREADS;
          if (i < K / 4) {
            const float4 v = xv[j];
            const float2 ga = __half22float2(*reinterpret_cast<const __half2*>(&gpre[j].x));
            const float2 gb = __half22float2(*reinterpret_cast<const __half2*>(&gpre[j].y));
            uint2 o;
            *reinterpret_cast<__half2*>(&o.x) = __floats2half2_rn(v.x * inv * ga.x, v.y * inv * ga.y);
            *reinterpret_cast<__half2*>(&o.y) = __floats2half2_rn(v.z * inv * gb.x, v.w * inv * gb.y);
            *reinterpret_cast<uint2*>(dst + 2 * i) = o;
          }
        }
        for (int i = threadIdx.x + XV * THREADS; i < K / 4; i += THREADS) {
          const float4 v = xr[i];
          const float2 ga = __half22float2(g2[2 * i]), gb = __half22float2(g2[2 * i + 1]);
          dst[2 * i] = __floats2half2_rn(v.x * inv * ga.x, v.y * inv * ga.y);
          dst[2 * i + 1] = __floats2half2_rn(v.z * inv * gb.x, v.w * inv * gb.y);
        }
      }
    } else {
      const int chunks = K / 8;
      for (int i = threadIdx.x; i < MB * chunks; i += THREADS) {
        const int m = i / chunks, c = i - m * chunks;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m < p.M) v = *reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + c * 8);
        *reinterpret_cast<uint4*>(a_s + (int64_t)m * K + c * 8) = v;
      }
    }
    __syncthreads();
  }

  // lane m finishes activation row m: its slot, position and KV page are looked up once, not per pair of columns
  QkvRow qrow;
  if (EPI == EPI_QKV) qrow = qkv_row(p, lane < MB ? lane : p.M);

  // ---- "chunk being consumed" cursor ----
  int cur_i = 0, cur_cc = 0;
  float acc0[MB], acc1[MB];
#pragma unroll
  for (int m = 0; m < MB; ++m) acc0[m] = acc1[m] = 0.f;

  // plain epilogue: the two residual elements lane m will add at the end of a unit are requested when the unit
  // begins (the same lane reads and later writes them, so this is safe when the residual aliases the output)
  float rpre0 = 0.f, rpre1 = 0.f;
  auto consume = [&](const uint4 (&w0)[U], const uint4 (&w1)[U]) {
    const int kb = cur_cc * CHUNK_K + lane * 8;
    if (EPI == EPI_F32 && cur_cc == 0 && p.res != nullptr && lane < MB && lane < p.M) {
      const int n = (u0 + warp + cur_i * WARPS) * 2;
      const int64_t o = (int64_t)lane * p.ldo + n;
      if (n < p.N) rpre0 = p.res[o];
      if (n + 1 < p.N) rpre1 = p.res[o + 1];
    }
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const int k = kb + j * 256;
      if (k < K) {
#pragma unroll
        for (int m = 0; m < MB; ++m) {
          uint4 a;
          if (A_SMEM) a = *reinterpret_cast<const uint4*>(a_s + (int64_t)m * K + k);
          else a = (m < p.M) ? __ldg(reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + k)) : make_uint4(0, 0, 0, 0);
          fma8(acc0[m], w0[j], a);
          fma8(acc1[m], w1[j], a);
        }
      }
    }
    if (++cur_cc == chunks_per_unit) {
      // unit finished: reduce over the lanes, lane m finishes activation row m
#pragma unroll
      for (int m = 0; m < MB; ++m) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          acc0[m] += __shfl_xor_sync(0xffffffffu, acc0[m], o);
          acc1[m] += __shfl_xor_sync(0xffffffffu, acc1[m], o);
        }
      }
      float v0 = 0.f, v1 = 0.f;
#pragma unroll
      for (int m = 0; m < MB; ++m)
        if (lane == m) { v0 = acc0[m]; v1 = acc1[m]; }
      const int u = u0 + warp + cur_i * WARPS;
      const int n = (EPI == EPI_SWIGLU) ? u : u * 2;
      if (lane < MB) {
        if (EPI == EPI_F32) {
          // epi_f32_pair with the residual already in registers
          if (lane < p.M && n < p.N) {
            const int64_t o = (int64_t)lane * p.ldo + n;
            const bool two = (n + 1 < p.N);
            if (p.res != nullptr) { v0 += rpre0; if (two) v1 += rpre1; }
            p.out_f32[o] = v0;
            if (two) p.out_f32[o + 1] = v1;
          }
        } else {
          epi_pair_row<EPI>(p, qrow, lane, n, v0, v1);
        }
      }
#pragma unroll
      for (int m = 0; m < MB; ++m) acc0[m] = acc1[m] = 0.f;
      cur_cc = 0;
      ++cur_i;
    }
  };

  // chunks c and c+1 are in flight in buffers 0 and 1; each buffer is refilled (chunk c+2, c+3) as soon
  // as it has been consumed
  for (int c = 0; c < total; c += 2) {
    consume(b0w0, b0w1);
    if (c + 2 < total) issue(b0w0, b0w1);
    if (c + 1 < total) {
      consume(b1w0, b1w1);
      if (c + 3 < total) issue(b1w0, b1w1);
    }
  }
  stamp_end(p.stamp);
}

template <int MB, int EPI, bool NORM, int U, bool A_SMEM>
es_status_t launch_inst(const LinearParams& p, cudaStream_t s, bool pdl) {
  auto kern = linear_stream_kernel<MB, EPI, NORM, U, A_SMEM>;
  const size_t smem = A_SMEM ? (size_t)MB * p.K * sizeof(__half) : 0;
  static size_t configured_smem = 0;
  if (smem > 48 * 1024 && smem > configured_smem) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured_smem = smem;
  }
  const int sms = sm_count();          // of the current device: a process may drive GPUs of different sizes
  int per_sm = 0;
  ES_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, THREADS, smem));
  if (per_sm < 1) return fail(ES_ERR_SHAPE, "weight-streaming kernel does not fit (K = %d, %d rows)", p.K, p.M);
  const int n_units = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  int grid = sms * per_sm;
  const int max_useful = (n_units + WARPS - 1) / WARPS;
  if (grid > max_useful) grid = max_useful;
  // When the units do not nearly fill a whole number of rounds over the warps (13B O / down at one row: 2560
  // units on 2368 warps, i.e. 192 warps with two units and the rest with one), a smaller grid in which every warp
  // gets the same number evens the finish: 33.2 -> 30.7 us for that product.  With three or more units per warp the
  // full grid measured faster (7B QKV 17.5 against 18.1 us), so the rule looks at the imbalance.
  {
    const int per_warp = (n_units + grid * WARPS - 1) / (grid * WARPS);   // units of the busiest warp
    const bool uneven = (long long)per_warp * grid * WARPS * 10 > (long long)n_units * 14;      // busiest > 1.4 x average
    if (tunables().even_grid || uneven) grid = (n_units + per_warp * WARPS - 1) / (per_warp * WARPS);
  }
  ES_CUDA_CHECK(launch_kernel(kern, dim3(grid), dim3(THREADS), smem, s, pdl, p));
  return ES_OK;
}

template <int MB, int EPI>
es_status_t launch_mb(const LinearParams& p, cudaStream_t s, bool pdl) {
  const size_t a_bytes = (size_t)MB * p.K * sizeof(__half);
  const int n_units = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  if (MB <= 2) {
    if (a_bytes > 200 * 1024) return fail(ES_ERR_SHAPE, "K = %d too large for the weight-streaming kernel", p.K);
    // 4 KB per warp per buffer (U = 4) beat 2 KB at every layer shape measured; U = 2 is kept for ES_STREAM_DEEP=0
    const bool deep = tunables().stream_deep != 0;
    if (p.norm_x) return deep ? launch_inst<MB, EPI, true, 4, true>(p, s, pdl) : launch_inst<MB, EPI, true, 2, true>(p, s, pdl);
    return deep ? launch_inst<MB, EPI, false, 4, true>(p, s, pdl) : launch_inst<MB, EPI, false, 2, true>(p, s, pdl);
  }
  if (p.norm_x) return fail(ES_ERR_UNSUPPORTED, "fused RMSNorm is limited to 2 activation rows");
  if (a_bytes <= 96 * 1024) return launch_inst<MB, EPI, false, 2, true>(p, s, pdl);
  return launch_inst<MB, EPI, false, 2, false>(p, s, pdl);
}

template <int EPI>
es_status_t launch_epi(const LinearParams& p, cudaStream_t s, bool pdl) {
  if (p.M <= 1) return launch_mb<1, EPI>(p, s, pdl);
  if (p.M <= 2) return launch_mb<2, EPI>(p, s, pdl);
  if (p.M <= 4) return launch_mb<4, EPI>(p, s, pdl);
  if (p.M <= 8) return launch_mb<8, EPI>(p, s, pdl);
  return launch_mb<16, EPI>(p, s, pdl);
}

}  // namespace

bool linear_stream_can_fuse_norm(int M) { return M <= 2; }

es_status_t launch_linear_stream(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl) {
  if (p.M <= 0 || p.N <= 0) return ES_OK;
  if (p.M > 16) return fail(ES_ERR_UNSUPPORTED, "weight-streaming kernel takes at most 16 rows, got %d", p.M);
  if (p.K % 8 != 0) return fail(ES_ERR_SHAPE, "K = %d is not a multiple of 8", p.K);
  es_status_t st;
  switch (epi) {
    case EPI_F32: st = launch_epi<EPI_F32>(p, s, pdl); break;
    case EPI_SWIGLU: st = launch_epi<EPI_SWIGLU>(p, s, pdl); break;
    case EPI_QKV: st = launch_epi<EPI_QKV>(p, s, pdl); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

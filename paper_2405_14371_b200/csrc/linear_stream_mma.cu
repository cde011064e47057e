// Weight-streaming kernel for decode steps with several sequences (3 <= M <= 16 activation rows).
// Like the single-row kernel it reads every weight byte once, straight from global memory into
// registers (16-byte loads, double buffered across work units, first chunks requested before the
// programmatic-dependency wait), but the arithmetic runs on the tensor cores: at 8 or 16 rows the
// plain ALUs cannot keep up with HBM.
//
//  * a work unit is 16 weight rows (or 8 gate rows + 8 up rows for SwiGLU).  A CTA owns a contiguous,
//    balanced range of units; its 8 warps all work on the same unit, each on one eighth of K, and
//    their partial sums are added in warp order through shared memory (deterministic);
//  * per 32 K-elements a lane loads 16 bytes of row g and of row g+8 (g = lane / 4) and issues two
//    mma.sync.m16n8k16 per group of 8 sequences.  The 8 consecutive elements a lane holds are fed to
//    the MMAs under a fixed permutation of the K index; the activation operand is read with the
//    same permutation (one 16-byte load per lane), so the products pair up correctly;
//  * activations sit in shared memory when they fit.  When they do not (long K, 8-16 rows), a second
//    kernel cuts K into slices ACROSS CTAs instead: a CTA keeps only its slice of the activations in
//    shared memory and its warps stream different 16-row groups over that slice, so activations are
//    read once per CTA rather than once per row group (on this machine what the SMs can take in
//    is about what HBM delivers, so re-read activations cost as much as weights).  The slices' partial
//    sums go to a workspace [slices, M, columns] and a finishing kernel adds them in slice order and
//    applies the epilogue.
#include "epilogue.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int MW = 8;                 // warps per CTA
constexpr int MTHREADS = MW * 32;
constexpr int KSTEP = 32;             // K elements per lane-load step
constexpr int UM_TOTAL = 4;           // lane-load steps per chunk over all row groups of a warp
inline int ks_grid() { return 2 * sm_count(); }   // CTAs of the K-sliced kernel: two per SM
constexpr size_t KS_SMEM_MAX = 100 * 1024;   // activation slice per CTA (two CTAs per SM)

__device__ __forceinline__ uint4 ld_stream16(const void* ptr) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(ptr));
  return v;
}

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// NT: groups of 8 activation rows (1 or 2).  RG: 16-row groups of weights a warp carries at once (1 or
// 2); with two, every activation fragment is used twice, which halves the activation traffic when
// the activations do not fit in shared memory and come through L1 / L2.
template <int NT, int EPI, bool A_SMEM, int RG>
__global__ void __launch_bounds__(MTHREADS, 2) linear_stream_mma_kernel(const LinearParams p, int a_stride) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* a_s = reinterpret_cast<__half*>(smem_raw);                 // [NT*8][a_stride], padded rows
  __shared__ float red[2][MW][RG][NT][32][4];

  const int K = p.K;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, q = lane & 3;
  constexpr int COLS = RG * ((EPI == EPI_SWIGLU) ? 8 : 16);           // output columns per unit
  const int n_units = (p.N + COLS - 1) / COLS;
  const int u0 = (int)((int64_t)blockIdx.x * n_units / gridDim.x);
  const int u1 = (int)((int64_t)(blockIdx.x + 1) * n_units / gridDim.x);
  const int n_my = u1 - u0;
  const int kslice = K / MW;                                         // multiple of KSTEP (checked on the host)
  const int k_lo = warp * kslice, k_hi = k_lo + kslice;
  constexpr int UM = UM_TOTAL / RG;                                    // steps per chunk: same registers for either RG
  constexpr int CHUNK_K = KSTEP * UM;
  const int chunks_per_unit = (kslice + CHUNK_K - 1) / CHUNK_K;
  const int total = n_my * chunks_per_unit;

  auto unit_rows = [&](int i, const __half* (&r0)[RG], const __half* (&r1)[RG]) {
    const int u = u0 + i;
#pragma unroll
    for (int rg = 0; rg < RG; ++rg) {
      if (EPI == EPI_SWIGLU) {
        const int n = u * COLS + rg * 8 + g;
        r0[rg] = (n < p.N) ? p.w[0] + (int64_t)n * K : nullptr;
        r1[rg] = (n < p.N) ? p.w[1] + (int64_t)n * K : nullptr;
      } else {
        const int n = u * COLS + rg * 16 + g;
        r0[rg] = (n < p.N) ? weight_row(p, n) : nullptr;
        r1[rg] = (n + 8 < p.N) ? weight_row(p, n + 8) : nullptr;
      }
    }
  };

  int nxt_i = 0, nxt_cc = 0;
  const __half* nr0[RG];
  const __half* nr1[RG];
#pragma unroll
  for (int rg = 0; rg < RG; ++rg) nr0[rg] = nr1[rg] = nullptr;
  if (total > 0) unit_rows(0, nr0, nr1);
  auto issue = [&](uint4 (&w0)[RG][UM], uint4 (&w1)[RG][UM]) {
    const int kb = k_lo + nxt_cc * CHUNK_K + q * 8;
#pragma unroll
    for (int j = 0; j < UM; ++j) {
      const int k = kb + j * KSTEP;
      const bool in = k < k_hi;
#pragma unroll
      for (int rg = 0; rg < RG; ++rg) {
        w0[rg][j] = (in && nr0[rg]) ? ld_stream16(nr0[rg] + k) : make_uint4(0, 0, 0, 0);
        w1[rg][j] = (in && nr1[rg]) ? ld_stream16(nr1[rg] + k) : make_uint4(0, 0, 0, 0);
      }
    }
    if (++nxt_cc == chunks_per_unit) {
      nxt_cc = 0;
      if (++nxt_i < n_my) unit_rows(nxt_i, nr0, nr1);
    }
  };

  uint4 b0w0[RG][UM], b0w1[RG][UM], b1w0[RG][UM], b1w1[RG][UM];
  if (total > 0) {
    issue(b0w0, b0w1);
    if (total > 1) issue(b1w0, b1w1);
  }

  pdl_wait();

  if (A_SMEM) {
    const int chunks = K / 8;
    for (int i = threadIdx.x; i < NT * 8 * chunks; i += MTHREADS) {
      const int m = i / chunks, c = i - m * chunks;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (m < p.M) v = *reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + c * 8);
      *reinterpret_cast<uint4*>(a_s + (int64_t)m * a_stride + c * 8) = v;
    }
    __syncthreads();
  }

  // In the unit epilogue below thread i always finishes activation row (i / 8) % (NT * 8) (the loop over idx runs
  // at most once: RG * 8 * NT * 8 <= MTHREADS): its slot, position and KV page are looked up once.
  static_assert(RG * 8 * NT * 8 <= MTHREADS, "one epilogue element per thread");
  QkvRow qrow;
  if (EPI == EPI_QKV) qrow = qkv_row(p, (threadIdx.x >> 3) % (NT * 8));

  float acc[RG][NT][4];
#pragma unroll
  for (int rg = 0; rg < RG; ++rg)
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[rg][t][i] = 0.f;
  int cur_i = 0, cur_cc = 0;

  auto consume = [&](const uint4 (&w0)[RG][UM], const uint4 (&w1)[RG][UM]) {
    const int kb = k_lo + cur_cc * CHUNK_K + q * 8;
#pragma unroll
    for (int j = 0; j < UM; ++j) {
      const int k = kb + j * KSTEP;
      if (k < k_hi) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          const int m = t * 8 + g;
          uint4 a;
          if (A_SMEM) a = *reinterpret_cast<const uint4*>(a_s + (int64_t)m * a_stride + k);
          else a = (m < p.M) ? __ldg(reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + k)) : make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int rg = 0; rg < RG; ++rg) {
            mma16816(acc[rg][t], w0[rg][j].x, w1[rg][j].x, w0[rg][j].y, w1[rg][j].y, a.x, a.y);
            mma16816(acc[rg][t], w0[rg][j].z, w1[rg][j].z, w0[rg][j].w, w1[rg][j].w, a.z, a.w);
          }
        }
      }
    }
    if (++cur_cc == chunks_per_unit) {
      // unit finished in this warp's K slice: add the 8 slices in warp order
      const int buf = cur_i & 1;
#pragma unroll
      for (int rg = 0; rg < RG; ++rg)
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          *reinterpret_cast<float4*>(&red[buf][warp][rg][t][lane][0]) =
              make_float4(acc[rg][t][0], acc[rg][t][1], acc[rg][t][2], acc[rg][t][3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[rg][t][i] = 0.f;
        }
      __syncthreads();
      // thread -> (row group rg, output pair pr, activation row m).  Accumulator element (row r, column m)
      // of group t lives in lane (r % 8) * 4 + (m % 8) / 2, register (r / 8) * 2 + (m % 2).
      for (int idx = threadIdx.x; idx < RG * 8 * NT * 8; idx += MTHREADS) {
        const int pr = idx & 7, m = (idx >> 3) % (NT * 8), rg = idx / (8 * NT * 8);
        const int t = m >> 3, mc = m & 7;
        int ra, rb;                                  // the two accumulator rows this thread combines
        if (EPI == EPI_SWIGLU) { ra = pr; rb = pr + 8; }
        else { ra = 2 * pr; rb = 2 * pr + 1; }
        const int la = (ra & 7) * 4 + (mc >> 1), ia = (ra >> 3) * 2 + (mc & 1);
        const int lb = (rb & 7) * 4 + (mc >> 1), ib = (rb >> 3) * 2 + (mc & 1);
        float v0 = 0.f, v1 = 0.f;
#pragma unroll
        for (int w = 0; w < MW; ++w) {
          v0 += red[buf][w][rg][t][la][ia];
          v1 += red[buf][w][rg][t][lb][ib];
        }
        const int u = u0 + cur_i;
        const int n = (EPI == EPI_SWIGLU) ? u * COLS + rg * 8 + pr : u * COLS + rg * 16 + 2 * pr;
        epi_pair_row<EPI>(p, qrow, m, n, v0, v1);       // idx == threadIdx.x: the row is the one looked up before the loop
      }
      cur_cc = 0;
      ++cur_i;
    }
  };

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

// ---- K sliced across CTAs (activations too large for shared memory) ---------------------------------
// CTA blockIdx.x works on K slice blockIdx.x / n_col_ctas and on the (blockIdx.x % n_col_ctas)-th balanced
// range of 16-row units; warp w takes units w, w + 8, ... of that range over the CTA's whole slice.
// Raw accumulators are stored to part[slice][m][column]; with SwiGLU the gate rows land in columns
// [0, N) and the up rows in [N, 2N).
template <int NT, int EPI>
__global__ void __launch_bounds__(MTHREADS, 2) linear_stream_mma_ks_kernel(const LinearParams p, int a_stride, int n_col_ctas) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* a_s = reinterpret_cast<__half*>(smem_raw);                 // [NT*8][a_stride]: this CTA's K slice of the activations

  const int K = p.K;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, q = lane & 3;
  constexpr int COLS = (EPI == EPI_SWIGLU) ? 8 : 16;
  constexpr int UM = UM_TOTAL;
  constexpr int CHUNK_K = KSTEP * UM;
  const int ks = blockIdx.x / n_col_ctas, nc = blockIdx.x - ks * n_col_ctas;
  const int kslice = K / p.k_splits;                                  // multiple of KSTEP (host)
  const int k_lo = ks * kslice, k_hi = k_lo + kslice;
  const int n_units = (p.N + COLS - 1) / COLS;
  const int u0 = (int)((int64_t)nc * n_units / n_col_ctas);
  const int u1 = (int)((int64_t)(nc + 1) * n_units / n_col_ctas);
  const int n_my = (u1 - u0 - warp + MW - 1) / MW;
  const int chunks_per_unit = (kslice + CHUNK_K - 1) / CHUNK_K;
  const int total = n_my > 0 ? n_my * chunks_per_unit : 0;

  auto unit_rows = [&](int i, const __half*& r0, const __half*& r1) {
    const int u = u0 + warp + i * MW;
    if (EPI == EPI_SWIGLU) {
      const int n = u * COLS + g;
      r0 = (n < p.N) ? p.w[0] + (int64_t)n * K : nullptr;
      r1 = (n < p.N) ? p.w[1] + (int64_t)n * K : nullptr;
    } else {
      const int n = u * COLS + g;
      r0 = (n < p.N) ? weight_row(p, n) : nullptr;
      r1 = (n + 8 < p.N) ? weight_row(p, n + 8) : nullptr;
    }
  };

  int nxt_i = 0, nxt_cc = 0;
  const __half* nr0 = nullptr;
  const __half* nr1 = nullptr;
  if (total > 0) unit_rows(0, nr0, nr1);
  auto issue = [&](uint4 (&w0)[UM], uint4 (&w1)[UM]) {
    const int kb = k_lo + nxt_cc * CHUNK_K + q * 8;
#pragma unroll
    for (int j = 0; j < UM; ++j) {
      const int k = kb + j * KSTEP;
      const bool in = k < k_hi;
      w0[j] = (in && nr0) ? ld_stream16(nr0 + k) : make_uint4(0, 0, 0, 0);
      w1[j] = (in && nr1) ? ld_stream16(nr1 + k) : make_uint4(0, 0, 0, 0);
    }
    if (++nxt_cc == chunks_per_unit) {
      nxt_cc = 0;
      if (++nxt_i < n_my) unit_rows(nxt_i, nr0, nr1);
    }
  };

  uint4 b0w0[UM], b0w1[UM], b1w0[UM], b1w1[UM];
  if (total > 0) {
    issue(b0w0, b0w1);
    if (total > 1) issue(b1w0, b1w1);
  }

  pdl_wait();

  {
    const int chunks = kslice / 8;
    for (int i = threadIdx.x; i < NT * 8 * chunks; i += MTHREADS) {
      const int m = i / chunks, c = i - m * chunks;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (m < p.M) v = *reinterpret_cast<const uint4*>(p.A + (int64_t)m * p.lda + k_lo + c * 8);
      *reinterpret_cast<uint4*>(a_s + (int64_t)m * a_stride + c * 8) = v;
    }
    __syncthreads();
  }

  float acc[NT][4];
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;
  int cur_i = 0, cur_cc = 0;
  const int64_t part_cols = (EPI == EPI_SWIGLU) ? 2 * (int64_t)p.N : p.N;
  float* part = p.part + (int64_t)ks * p.M * part_cols;

  auto consume = [&](const uint4 (&w0)[UM], const uint4 (&w1)[UM]) {
    const int kb = cur_cc * CHUNK_K + q * 8;                          // offset inside the slice
#pragma unroll
    for (int j = 0; j < UM; ++j) {
      const int k = kb + j * KSTEP;
      if (k < kslice) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          const uint4 a = *reinterpret_cast<const uint4*>(a_s + (int64_t)(t * 8 + g) * a_stride + k);
          mma16816(acc[t], w0[j].x, w1[j].x, w0[j].y, w1[j].y, a.x, a.y);
          mma16816(acc[t], w0[j].z, w1[j].z, w0[j].w, w1[j].w, a.z, a.w);
        }
      }
    }
    if (++cur_cc == chunks_per_unit) {
      // accumulator element (weight row r, activation row m) of group t: lane (r % 8) * 4 + (m % 8) / 2,
      // register (r / 8) * 2 + (m % 2)
      const int u = u0 + warp + cur_i * MW;
      const int na = u * COLS + g;                                     // rows 0..7 of the unit
      const int64_t ca = na;
      const int64_t cb = (EPI == EPI_SWIGLU) ? (int64_t)p.N + na : (int64_t)na + 8;
      const bool va = na < p.N, vb = (EPI == EPI_SWIGLU) ? va : (na + 8 < p.N);
#pragma unroll
      for (int t = 0; t < NT; ++t) {
        const int m0 = t * 8 + 2 * q;
        if (m0 < p.M) {
          if (va) part[(int64_t)m0 * part_cols + ca] = acc[t][0];
          if (vb) part[(int64_t)m0 * part_cols + cb] = acc[t][2];
        }
        if (m0 + 1 < p.M) {
          if (va) part[(int64_t)(m0 + 1) * part_cols + ca] = acc[t][1];
          if (vb) part[(int64_t)(m0 + 1) * part_cols + cb] = acc[t][3];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[t][i] = 0.f;
      }
      cur_cc = 0;
      ++cur_i;
    }
  };

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

// Adds the K slices of one output pair in slice order and applies the epilogue (SwiGLU / QKV forms;
// the plain form is finished by the reduction kernel that also fuses the following RMSNorm).
template <int EPI>
__global__ void __launch_bounds__(256) splitk_finish_kernel(const LinearParams p) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  pdl_wait();
  const int pairs = (EPI == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  const int64_t part_cols = (EPI == EPI_SWIGLU) ? 2 * (int64_t)p.N : p.N;
  const int64_t slice = (int64_t)p.M * part_cols;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < (int64_t)p.M * pairs; idx += (int64_t)gridDim.x * blockDim.x) {
    const int m = (int)(idx / pairs), pr = (int)(idx - (int64_t)m * pairs);
    const int n = (EPI == EPI_SWIGLU) ? pr : 2 * pr;
    const int64_t c0 = n, c1 = (EPI == EPI_SWIGLU) ? (int64_t)p.N + n : (int64_t)n + 1;
    const bool has1 = (EPI == EPI_SWIGLU) || (n + 1 < p.N);
    const float* src = p.part + (int64_t)m * part_cols;
    // the row's slot, position and KV page do not depend on the sums: looked up while the slices are on their way
    QkvRow row;
    if (EPI == EPI_QKV) row = qkv_row(p, m);
    float v0 = 0.f, v1 = 0.f;
    // eight slices are requested at a time and then added in slice order; adjacent columns (n even, N even) come
    // as one 8-byte load
    const bool pair8 = (EPI != EPI_SWIGLU) && has1 && ((part_cols & 1) == 0);
    for (int s0 = 0; s0 < p.k_splits; s0 += 8) {
      float a[8], b[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const bool in = s0 + j < p.k_splits;
        if (pair8) {
          const float2 t = in ? __ldcs(reinterpret_cast<const float2*>(src + (s0 + j) * slice + c0)) : make_float2(0.f, 0.f);
          a[j] = t.x;
          b[j] = t.y;
        } else {
          a[j] = in ? __ldcs(src + (s0 + j) * slice + c0) : 0.f;
          b[j] = (in && has1) ? __ldcs(src + (s0 + j) * slice + c1) : 0.f;
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (s0 + j < p.k_splits) { v0 += a[j]; v1 += b[j]; }
    }
    if (EPI == EPI_QKV) epi_qkv_pair_row(p, row, n, v0, v1);
    else epi_pair<EPI>(p, m, n, v0, v1);
  }
  stamp_end(p.stamp);
}

int ks_col_ctas(int ks);   // defined with the host-side planning below

template <int NT, int EPI>
es_status_t launch_ks(const LinearParams& p, cudaStream_t s, bool pdl) {
  auto kern = linear_stream_mma_ks_kernel<NT, EPI>;
  const int kslice = p.K / p.k_splits;
  const int a_stride = kslice + 8;
  const size_t smem = (size_t)NT * 8 * a_stride * sizeof(__half);
  static size_t configured = 0;
  if (smem > 32 * 1024 && smem > configured) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = smem;
  }
  const int n_col_ctas = ks_col_ctas(p.k_splits);
  ES_CUDA_CHECK(launch_kernel(kern, dim3(n_col_ctas * p.k_splits), dim3(MTHREADS), smem, s, pdl, p, a_stride, n_col_ctas));
  return ES_OK;
}

template <int NT, int EPI, bool A_SMEM, int RG>
es_status_t launch_inst(const LinearParams& p, cudaStream_t s, bool pdl) {
  auto kern = linear_stream_mma_kernel<NT, EPI, A_SMEM, RG>;
  const int a_stride = p.K + 8;                       // 16 bytes of padding: the 8 rows fall into different banks
  const size_t smem = A_SMEM ? (size_t)NT * 8 * a_stride * sizeof(__half) : 0;
  static size_t configured = 0;
  if (smem > 16 * 1024 && smem > configured) {      // static shared memory counts against the 48 KB default too
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    configured = smem;
  }
  const int sms = sm_count();          // of the current device: a process may drive GPUs of different sizes
  int per_sm = 0;
  ES_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, MTHREADS, smem));
  if (per_sm < 1) return fail(ES_ERR_SHAPE, "tensor-core streaming kernel does not fit (K = %d)", p.K);
  constexpr int COLS = RG * ((EPI == EPI_SWIGLU) ? 8 : 16);
  const int n_units = (p.N + COLS - 1) / COLS;
  int grid = sms * per_sm;
  if (grid > n_units) grid = n_units;
  if (tunables().even_grid) {
    const int per_cta = (n_units + grid - 1) / grid;       // the same number of units for every CTA
    grid = (n_units + per_cta - 1) / per_cta;
  }
  ES_CUDA_CHECK(launch_kernel(kern, dim3(grid), dim3(MTHREADS), smem, s, pdl, p, a_stride));
  return ES_OK;
}

template <int NT, int EPI>
es_status_t launch_nt(const LinearParams& p, cudaStream_t s, bool pdl) {
  const size_t a_bytes = (size_t)NT * 8 * (p.K + 8) * sizeof(__half);
  if (a_bytes <= 100 * 1024) return launch_inst<NT, EPI, true, 1>(p, s, pdl);
  // through L1 / L2: with 16 activation rows their traffic equals the weights', so a warp carries two
  // weight row groups per activation fragment; with 8 rows the longer contiguous runs per row win
  return launch_inst<NT, EPI, false, (NT == 2 ? 2 : 1)>(p, s, pdl);
}

template <int EPI>
es_status_t launch_epi(const LinearParams& p, cudaStream_t s, bool pdl) {
  if (p.k_splits > 1) return p.M <= 8 ? launch_ks<1, EPI>(p, s, pdl) : launch_ks<2, EPI>(p, s, pdl);
  if (p.M <= 8) return launch_nt<1, EPI>(p, s, pdl);
  return launch_nt<2, EPI>(p, s, pdl);
}

}  // namespace

bool linear_stream_mma_supported(const LinearParams& p, int epi) {
  if (p.M < 1 || p.M > 16 || p.N <= 0 || p.norm_x != nullptr) return false;
  if (p.K % (MW * KSTEP) != 0) return false;            // every warp gets a whole number of 32-element steps
  if (p.lda % 8 != 0 || ((uintptr_t)p.A % 16)) return false;
  for (int i = 0; i < 3; ++i)
    if (p.w[i] && ((uintptr_t)p.w[i] % 16)) return false;
  if (epi == EPI_QKV && (p.N % 2)) return false;
  return true;
}

namespace {

// Column ranges per K slice: as many as fill the machine (two CTAs per SM).  Fewer, evenly loaded CTAs were
// measured and lost at every shape of the 70B layer (e.g. gate / up 163 -> 175 us with 64 instead of 74 ranges).
int ks_col_ctas(int ks) {
  const int hi = ks_grid() / ks;
  return (tunables().ks_cols > 0 && tunables().ks_cols <= hi) ? tunables().ks_cols : hi;
}

}  // namespace

int linear_stream_mma_splits(const LinearParams& p, int epi, size_t workspace_bytes) {
  if (!linear_stream_mma_supported(p, epi) || p.M < 3) return 1;
  const int nt = p.M <= 8 ? 1 : 2;
  if ((size_t)nt * 8 * (p.K + 8) * sizeof(__half) <= KS_SMEM_MAX) return 1;     // the whole K range fits: no slicing
  const int steps = p.K / KSTEP;
  const int cols = (epi == EPI_SWIGLU) ? 8 : 16;
  const int n_units = (p.N + cols - 1) / cols;
  const size_t part_cols = (epi == EPI_SWIGLU) ? 2 * (size_t)p.N : (size_t)p.N;
  // The slice count that minimises the K elements the busiest warp walks.  Measured on the 70B layer at 16 rows
  // (in-step, normalised): QKV 16 slices 32 us, 8 slices 35, 4 slices 40; down 16 slices 83 us, 14 slices 86.
  int best = 1;
  long long best_cost = 0;
  const int grid_max = ks_grid();
  for (int ks = 2; ks <= 64 && ks <= grid_max; ++ks) {
    if (steps % ks) continue;
    const int kslice = p.K / ks;
    if (kslice < tunables().ks_min_slice) break;
    if ((size_t)nt * 8 * (kslice + 8) * sizeof(__half) > KS_SMEM_MAX) continue;
    if ((size_t)ks * p.M * part_cols * sizeof(float) > workspace_bytes) continue;
    if (tunables().ks_splits == ks) return ks;
    const int ncol = grid_max / ks;
    const int units_per_cta = (n_units + ncol - 1) / ncol;
    const long long cost = (long long)((units_per_cta + MW - 1) / MW) * kslice;   // K elements the busiest warp walks
    if (best == 1 || cost < best_cost) { best = ks; best_cost = cost; }
  }
  return best;
}

es_status_t launch_splitk_finish(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl) {
  if (p.k_splits < 2 || p.part == nullptr) return fail(ES_ERR_INVALID_ARG, "nothing to finish");
  const int pairs = (epi == EPI_SWIGLU) ? p.N : (p.N + 1) / 2;
  const long long work = (long long)p.M * pairs;
  int grid = (int)((work + 255) / 256);
  if (grid > 4 * sm_count()) grid = 4 * sm_count();
  switch (epi) {
    case EPI_SWIGLU: ES_CUDA_CHECK(launch_kernel(splitk_finish_kernel<EPI_SWIGLU>, dim3(grid), dim3(256), 0, s, pdl, p)); break;
    case EPI_QKV: ES_CUDA_CHECK(launch_kernel(splitk_finish_kernel<EPI_QKV>, dim3(grid), dim3(256), 0, s, pdl, p)); break;
    default: return fail(ES_ERR_INVALID_ARG, "the plain epilogue is finished by the reduction kernel");
  }
  if (launches) ++*launches;
  return ES_OK;
}

es_status_t launch_linear_stream_mma(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, bool pdl) {
  if (!linear_stream_mma_supported(p, epi)) return fail(ES_ERR_UNSUPPORTED, "tensor-core streaming kernel does not take this shape");
  if (p.k_splits > 1) {
    const int nt = p.M <= 8 ? 1 : 2;
    if (p.part == nullptr || (p.K / KSTEP) % p.k_splits != 0 || p.k_splits > ks_grid() ||
        (size_t)nt * 8 * (p.K / p.k_splits + 8) * sizeof(__half) > KS_SMEM_MAX)
      return fail(ES_ERR_INVALID_ARG, "K-sliced streaming kernel: %d slices do not fit K = %d", p.k_splits, p.K);
  }
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

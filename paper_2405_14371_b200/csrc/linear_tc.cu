// Tensor-core kernel of the linear-layer family for sm_100a: C[M,N] = A[M,K] * W[N,K]^T with the
// fused epilogues, for M > 16 (prefill).
//
// One CTA computes a 128 x BN output tile.  A single elected thread feeds a ring of shared-memory
// stages with TMA (128-byte-swizzled K-major tiles of A and W, 64 K-elements deep); a second
// elected thread issues tcgen05.mma (M=128, N=BN, K=16, fp16 in, fp32 accumulate) into a TMEM
// accumulator and releases each stage with tcgen05.commit; four epilogue warps read the
// accumulator back with tcgen05.ld (each warp its own 32-lane quarter) and run the epilogue, passing
// each 32-column chunk through a shared-memory tile so that global accesses cover whole row segments.
// Ragged M, N and K are handled by TMA zero fill on the way in and by guards on the way out.
// Split-K (plain / residual epilogue only): when a product has too few output tiles for the machine
// (short prompts: M = 128..512 against N = d_model), the K range is cut into k_splits slices, every
// (tile, slice) pair is a work item, and the raw fp32 accumulators go to a workspace
// [k_splits, M, N]; a reduction kernel adds the slices in slice order (and the residual) afterwards.
// That cuts what a CTA must pull through L2 for its tile from 128 + BN rows of K elements to
// (128 + BN) / k_splits, which is what bounds these launches.
// Every wait is bounded: if a barrier does not flip within about a second the CTA records an
// error code in the status word and leaves through the normal teardown (TMEM freed).
#include <cuda.h>
#include <string.h>

#include "epilogue.cuh"
#include "launch.cuh"
#include "sm100.cuh"

namespace es {

namespace {

constexpr int BM = 128, BK = 64, UMMA_K = 16;
constexpr int W_BOX_ROWS = 32;
constexpr int TC_THREADS = 192;
constexpr int A_STAGE_BYTES = BM * BK * 2;

template <int BN> struct TileCfg {
  static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "tile width: a multiple of the 32-row weight box, at most one MMA wide");
  static constexpr int B_STAGE_BYTES = BN * BK * 2;
  static constexpr int STAGES = (200 * 1024) / (A_STAGE_BYTES + B_STAGE_BYTES) > 8 ? 8 : (200 * 1024) / (A_STAGE_BYTES + B_STAGE_BYTES);
  static constexpr int TMEM_COLS = BN;                                       // one accumulator buffer
  static constexpr int TMEM_ALLOC = 2 * BN <= 64 ? 64 : 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512;   // two buffers, power of two
  static constexpr size_t SMEM = 1024 + (size_t)STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 4 * EPI_STAGE_F32_BYTES + 256;
};

struct TmapSet {
  CUtensorMap a;
  CUtensorMap w[3];
};
static_assert(sizeof(TmapSet) == sizeof(TcMaps), "TcMaps must hold four tensor maps");

// ---- the kernel --------------------------------------------------------------------------------
// Persistent: a CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The accumulator is double
// buffered in TMEM, so the epilogue of one tile runs while the tensor cores work on the next.
template <int EPI, int BN>
__global__ void __launch_bounds__(TC_THREADS, 1)
linear_tc_kernel(const __grid_constant__ TmapSet maps, const LinearParams p, int* status, int m_tiles, int n_tiles) {
  using Cfg = TileCfg<BN>;
  constexpr int STAGES = Cfg::STAGES;
  constexpr int BN_OUT = (EPI == EPI_SWIGLU) ? BN / 2 : BN;   // output columns per tile
  constexpr int ACC_COLS = Cfg::TMEM_COLS;                    // TMEM columns of one accumulator buffer

  pdl_launch_dependents();
  stamp_begin(p.stamp);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* a_tiles = smem;
  unsigned char* b_tiles = smem + (size_t)STAGES * A_STAGE_BYTES;
  unsigned char* epi_stage = b_tiles + (size_t)STAGES * Cfg::B_STAGE_BYTES;   // one store-staging tile per epilogue warp
  uint64_t* bars = (uint64_t*)(epi_stage + 4 * EPI_STAGE_F32_BYTES);
  uint64_t* full_bar = bars;
  uint64_t* empty_bar = bars + STAGES;
  uint64_t* acc_full = bars + 2 * STAGES;        // [2]
  uint64_t* acc_empty = bars + 2 * STAGES + 2;   // [2]
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * STAGES + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int k_splits = (EPI == EPI_F32 && p.k_splits > 1) ? p.k_splits : 1;
  const int mn_tiles = m_tiles * n_tiles;
  const int num_tiles = mn_tiles * k_splits;        // work items: slice-major, so concurrent CTAs share a K slice of A
  const int num_kb = (p.K + BK - 1) / BK;
  const int kb_per = (num_kb + k_splits - 1) / k_splits;

  // tile order: groups of up to 16 row tiles share each column tile while it is hot in L2
  auto tile_origin = [&](int tile, int& m0, int& n0) {
    constexpr int GM = 16;
    const int per_group = GM * n_tiles;
    const int first_m = (tile / per_group) * GM;
    const int gsz = min(GM, m_tiles - first_m);
    m0 = (first_m + (tile % per_group) % gsz) * BM;
    n0 = ((tile % per_group) / gsz) * BN_OUT;
  };

  if (threadIdx.x == 0) {
    prefetch_tmap(&maps.a);
    prefetch_tmap(&maps.w[0]);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 4);     // one arrival per epilogue warp
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::TMEM_ALLOC);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // barriers, tensor-map prefetch and the TMEM allocation above overlap the previous kernel's tail;
  // nothing below reads or writes global memory before the previous kernel has completed
  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer ----
      // the B stage is BN rows of W, fetched 32 rows per copy; with SwiGLU the first half of the
      // rows comes from the gate matrix and the second half from the up matrix (same row range)
      constexpr int N_LOADS = BN / W_BOX_ROWS;
      int it = 0;                                  // k-block counter across tiles
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int m0, n0;
        const int ks = tile / mn_tiles;
        tile_origin(tile - ks * mn_tiles, m0, n0);
        const int kb0 = ks * kb_per, kb1 = min(num_kb, kb0 + kb_per);
        const CUtensorMap* wmap[N_LOADS];
        int wrow[N_LOADS];
        if (EPI == EPI_SWIGLU) {
#pragma unroll
          for (int i = 0; i < N_LOADS; ++i) {
            const bool up = i >= N_LOADS / 2;
            wmap[i] = up ? &maps.w[1] : &maps.w[0];
            wrow[i] = n0 + (up ? i - N_LOADS / 2 : i) * W_BOX_ROWS;
          }
        } else {
          int n = n0, seg = 0;
          while (seg < 2 && n >= p.seg_rows[seg]) { n -= p.seg_rows[seg]; ++seg; }
#pragma unroll
          for (int i = 0; i < N_LOADS; ++i) { wmap[i] = &maps.w[seg]; wrow[i] = n + i * W_BOX_ROWS; }
        }
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, abort_flag, status, 1)) { ok = false; break; }
          const uint32_t fb = smem_u32(&full_bar[s]);
          mbar_expect_tx(fb, A_STAGE_BYTES + Cfg::B_STAGE_BYTES);
          tma_load_2d(smem_u32(a_tiles + (size_t)s * A_STAGE_BYTES), &maps.a, kb * BK, m0, fb);
          const uint32_t bdst = smem_u32(b_tiles + (size_t)s * Cfg::B_STAGE_BYTES);
#pragma unroll
          for (int i = 0; i < N_LOADS; ++i)
            tma_load_2d(bdst + i * W_BOX_ROWS * (BK * 2), wmap[i], kb * BK, wrow[i], fb);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      constexpr uint32_t idesc = umma_idesc_f16(BM, BN);
      int it = 0, local = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++local) {
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        ok = mbar_wait(smem_u32(&acc_empty[buf]), (use & 1) ^ 1, abort_flag, status, 5);   // epilogue drained it
        if (!ok) break;
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * ACC_COLS);
        const int ks = tile / mn_tiles;
        const int kb0 = ks * kb_per, kb1 = min(num_kb, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1;
          ok = mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag, status, 2);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(a_tiles + (size_t)s * A_STAGE_BYTES);
          const uint32_t b0 = smem_u32(b_tiles + (size_t)s * Cfg::B_STAGE_BYTES);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k)
            umma_f16(tacc, umma_desc_sw128(a0 + k * UMMA_K * 2), umma_desc_sw128(b0 + k * UMMA_K * 2), idesc,
                     (kb > kb0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&empty_bar[s]));      // frees the stage once these MMAs have read it
        }
        if (ok) umma_commit(smem_u32(&acc_full[buf]));   // accumulator complete
      }
    }
  } else {
    // ---- epilogue warps: TMEM lane quarter = warp % 4 ----
    const int quarter = warp & 3;
    int local = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++local) {
      const int buf = local & 1;
      const uint32_t use = (uint32_t)(local >> 1);
      if (!mbar_wait(smem_u32(&acc_full[buf]), use & 1, abort_flag, status, 3)) break;
      tc_fence_after();
      int m0, n0;
      const int ks = tile / mn_tiles;
      tile_origin(tile - ks * mn_tiles, m0, n0);
      const int mw = m0 + quarter * 32;              // row of lane 0
      const uint32_t trow = tmem_base + (uint32_t)(buf * ACC_COLS) + ((uint32_t)(quarter * 32) << 16);
      unsigned char* stage = epi_stage + (size_t)(warp - 2) * EPI_STAGE_F32_BYTES;   // large enough for either kind of chunk
      if (EPI == EPI_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < BN_OUT; c += 32) {
          float g[32], u[32];
          tmem_ld32(trow + c, g);
          tmem_ld32(trow + BN_OUT + c, u);
          epi_swiglu_chunk32_staged(p, mw, n0 + c, g, u, stage, lane);
        }
      } else if (EPI == EPI_QKV) {
        const QkvRow row = qkv_row(p, mw + lane);      // the row's place in the q output and the KV pages, once per tile
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          float v[32];
          tmem_ld32(trow + c, v);
          epi_qkv_chunk32_staged(p, row, mw, n0 + c, v, stage, lane);
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < BN; c += 32) {
          float v[32];
          float4 rv[8];
          tmem_ld32(trow + c, v);
          // split-K: the raw accumulator goes to slice ks of the workspace [k_splits, M, N]
          if (k_splits > 1) f32_chunk32_staged<false>(p.part + (int64_t)ks * p.M * p.N, nullptr, p.N, p.M, p.N, mw, n0 + c, v, rv, stage, lane);
          else f32_chunk32_staged<false>(p.out_f32, p.res, p.ldo, p.M, p.N, mw, n0 + c, v, rv, stage, lane);
        }
      }
      // this warp has read its quarter of the buffer: hand it back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (*abort_flag) __nanosleep(100000);     // let copies still in flight land before the CTA's memory is released
    tmem_dealloc(tmem_base, Cfg::TMEM_ALLOC);
  }
  stamp_end(p.stamp);
}

// ---- host side -----------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)f;
  }
  return fn;
}

// fp16 row-major [rows, K] matrix, box = 64 K-elements x box_rows rows, 128-byte swizzle, zero fill
es_status_t encode_2d(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int64_t ld, int box_rows) {
  return tma_encode_2d_f16(map, base, rows, K, ld, box_rows);
}

int pick_bn(const LinearParams& p, int epi) {
  if (epi == EPI_F32 && p.k_splits > 1) return 256;
  // Every CTA pulls a 128-row slice of A and a bn-row slice of W through L2 for the whole K range,
  // one CTA per SM at a time, so the time goes as (waves of CTAs) x (128 + bn).  Take the width
  // that minimises it (the wider one on ties); QKV segments must be whole tiles.
  const int m_tiles = (p.M + BM - 1) / BM;
  const int cands[8] = {256, 224, 192, 160, 128, 96, 64, 32};
  const int sms = sm_count();
  int best = 0;
  long long best_cost = 0;
  for (int bn : cands) {
    const int out = (epi == EPI_SWIGLU) ? bn / 2 : bn;
    bool fits = !(epi == EPI_SWIGLU && bn % (2 * W_BOX_ROWS) != 0);      // gate half and up half are whole weight boxes
    if (epi == EPI_QKV)
      for (int s = 0; s < 3; ++s) if (p.seg_rows[s] % out) fits = false;
    if (!fits) continue;
    const long long tiles = (long long)m_tiles * ((p.N + out - 1) / out);
    const long long waves = (tiles + sms - 1) / sms;
    const long long cost = waves * (BM + bn);
    if (best == 0 || cost < best_cost) { best = bn; best_cost = cost; }
  }
  return best;
}

template <int EPI, int BN>
es_status_t launch_bn(const TmapSet& maps, const LinearParams& p, int* status, cudaStream_t s, bool pdl) {
  constexpr int out = (EPI == EPI_SWIGLU) ? BN / 2 : BN;
  const int m_tiles = (p.M + BM - 1) / BM, n_tiles = (p.N + out - 1) / out;
  auto kern = linear_tc_kernel<EPI, BN>;
  static bool configured = false;
  if (!configured) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TileCfg<BN>::SMEM));
    configured = true;
  }
  const int sms = sm_count();          // of the current device: a process may drive GPUs of different sizes
  const int tiles = m_tiles * n_tiles * ((EPI == EPI_F32 && p.k_splits > 1) ? p.k_splits : 1);
  ES_CUDA_CHECK(launch_kernel(kern, dim3(tiles < sms ? tiles : sms), dim3(TC_THREADS), TileCfg<BN>::SMEM, s, pdl, maps, p, status,
                              m_tiles, n_tiles));
  return ES_OK;
}

template <int EPI>
es_status_t launch_epi(const TmapSet& maps, const LinearParams& p, int bn, int* status, cudaStream_t s, bool pdl) {
  switch (bn) {
    case 256: return launch_bn<EPI, 256>(maps, p, status, s, pdl);
    case 192: return launch_bn<EPI, 192>(maps, p, status, s, pdl);
    case 128: return launch_bn<EPI, 128>(maps, p, status, s, pdl);
    case 64: return launch_bn<EPI, 64>(maps, p, status, s, pdl);
  }
  if constexpr (EPI != EPI_SWIGLU) {      // widths whose halves are not whole weight boxes
    switch (bn) {
      case 224: return launch_bn<EPI, 224>(maps, p, status, s, pdl);
      case 160: return launch_bn<EPI, 160>(maps, p, status, s, pdl);
      case 96: return launch_bn<EPI, 96>(maps, p, status, s, pdl);
      case 32: return launch_bn<EPI, 32>(maps, p, status, s, pdl);
    }
  }
  return fail(ES_ERR_UNSUPPORTED, "no tile width for this shape");
}

}  // namespace

bool tma_available() { return encode_fn() != nullptr; }

es_status_t tma_encode_2d_f16(void* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return fail(ES_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(reinterpret_cast<CUtensorMap*>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims,
                  strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ES_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return ES_OK;
}

int linear_tc_splits(const LinearParams& p, int epi) {
  // Worth it when 256-wide tiles over the whole K range would leave at least half of the SMs idle;
  // every slice keeps at least four 64-element K blocks.
  if (epi != EPI_F32 || p.M <= 16 || p.N % 4 != 0) return 1;
  const int tiles = ((p.M + BM - 1) / BM) * ((p.N + 255) / 256);
  const int num_kb = (p.K + BK - 1) / BK;
  int s = sm_count() / tiles;
  if (s > 8) s = 8;
  if (s > num_kb / 4) s = num_kb / 4;
  if (s < 2) return 1;
  const int kb_per = (num_kb + s - 1) / s;
  return (num_kb + kb_per - 1) / kb_per;       // no empty slice
}

size_t linear_tc_split_workspace_bytes() { return (size_t)sm_count() * BM * 256 * sizeof(float); }

bool linear_tc_supported(const LinearParams& p, int epi) {
  if (p.M <= 0 || p.N <= 0 || p.K <= 0) return false;
  if (p.K % 8 != 0 || p.lda % 8 != 0) return false;                 // TMA strides are multiples of 16 bytes
  if (((uintptr_t)p.A | (uintptr_t)p.w[0]) % 16) return false;
  if (epi == EPI_QKV && (((uintptr_t)p.w[1] | (uintptr_t)p.w[2]) % 16)) return false;
  if (epi == EPI_SWIGLU && ((uintptr_t)p.w[1] % 16)) return false;
  return pick_bn(p, epi) != 0 && encode_fn() != nullptr;
}

es_status_t tc_build_maps(const LinearParams& p, int epi, int64_t a_rows, TcMaps* out) {
  TmapSet* t = reinterpret_cast<TmapSet*>(out);
  memset(t, 0, sizeof(*t));
  ES_TRY(encode_2d(&t->a, p.A, a_rows, p.K, p.lda, BM));
  const int nseg = (epi == EPI_QKV) ? 3 : (epi == EPI_SWIGLU ? 2 : 1);
  for (int s = 0; s < nseg; ++s) {
    const int64_t rows = (epi == EPI_SWIGLU) ? p.N : p.seg_rows[s];
    ES_TRY(encode_2d(&t->w[s], p.w[s], rows, p.K, p.K, W_BOX_ROWS));
  }
  return ES_OK;
}

es_status_t launch_linear_tc(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, int* status_word, bool pdl) {
  if (!linear_tc_supported(p, epi)) return fail(ES_ERR_UNSUPPORTED, "tensor-core kernel does not take this shape");
  if (p.k_splits > 1) {
    if (epi != EPI_F32 || p.part == nullptr || p.N % 4 != 0)
      return fail(ES_ERR_INVALID_ARG, "split-K needs the plain epilogue, a workspace and N %% 4 == 0");
    const int num_kb = (p.K + BK - 1) / BK;
    const int kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
    if ((p.k_splits - 1) * kb_per >= num_kb) return fail(ES_ERR_INVALID_ARG, "split-K: %d slices leave one empty (K = %d)", p.k_splits, p.K);
  }
  TcMaps local;
  const TcMaps* maps = p.tc_maps;
  if (!maps) {
    ES_TRY(tc_build_maps(p, epi, p.M, &local));
    maps = &local;
  }
  const TmapSet& t = *reinterpret_cast<const TmapSet*>(maps);
  const int bn = pick_bn(p, epi);
  es_status_t st;
  switch (epi) {
    case EPI_F32: st = launch_epi<EPI_F32>(t, p, bn, status_word, s, pdl); break;
    case EPI_SWIGLU: st = launch_epi<EPI_SWIGLU>(t, p, bn, status_word, s, pdl); break;
    case EPI_QKV: st = launch_epi<EPI_QKV>(t, p, bn, status_word, s, pdl); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

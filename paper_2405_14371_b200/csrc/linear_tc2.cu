// Tensor-core kernel of the linear-layer family on CTA pairs (tcgen05 cta_group::2), for large M.
//
// A cluster of two CTAs computes a 256 x 256 output tile: each CTA stages its own 128 rows of A and
// one half (128 rows) of the W tile per 64-deep K block, and one thread of the pair's first CTA
// issues MMAs (M=256, N=256, K=16) that read both CTAs' shared memory and write both CTAs' TMEM
// (each CTA ends up with its 128 rows x 256 columns).  Per CTA that is half the shared-memory
// operand traffic per flop of the single-CTA 128 x 256 tile and a third less staging per K block,
// so the ring is deeper in time and the tensor pipe stalls less.  Persistent pairs walk the tiles;
// the accumulator is double buffered in TMEM (2 x 256 columns) so epilogues overlap the next tile.
// Barrier traffic: both CTAs' TMA bytes are counted on the first CTA's "full" barrier; the MMA
// issuer's commits arrive on the "empty" / "accumulator ready" barriers of both CTAs; both CTAs'
// epilogue warps arrive on the first CTA's "accumulator free" barrier.  Waits are bounded.
#include <cuda.h>
#include <string.h>

#include "epilogue.cuh"
#include "launch.cuh"
#include "sm100.cuh"

namespace es {

namespace {

constexpr int BM2 = 128;          // rows per CTA (256 per pair)
constexpr int BN2 = 256;
constexpr int BK2 = 64, UK2 = 16;
constexpr int W_BOX = 32;
constexpr int T2_THREADS = 192;
constexpr int STAGES2 = 6;
constexpr int A_BYTES2 = BM2 * BK2 * 2;          // 16 KB
constexpr int B_BYTES2 = (BN2 / 2) * BK2 * 2;    // this CTA's half of the W tile, 16 KB
constexpr size_t SMEM2 = 1024 + (size_t)STAGES2 * (A_BYTES2 + B_BYTES2) + 256;

struct TmapSet2 {
  CUtensorMap a;
  CUtensorMap w[3];
};
static_assert(sizeof(TmapSet2) == sizeof(TcMaps), "TcMaps must hold four tensor maps");

template <int EPI>
__global__ void __launch_bounds__(T2_THREADS, 1)
linear_tc2_kernel(const __grid_constant__ TmapSet2 maps, const LinearParams p, int* status, int m_tiles, int n_tiles) {
  constexpr int BN_OUT = (EPI == EPI_SWIGLU) ? BN2 / 2 : BN2;
  pdl_launch_dependents();

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* a_tiles = smem;
  unsigned char* b_tiles = smem + (size_t)STAGES2 * A_BYTES2;
  uint64_t* bars = (uint64_t*)(b_tiles + (size_t)STAGES2 * B_BYTES2);
  uint64_t* full_bar = bars;                     // used in rank 0 only
  uint64_t* empty_bar = bars + STAGES2;          // one copy per CTA
  uint64_t* acc_full = bars + 2 * STAGES2;       // [2], one copy per CTA
  uint64_t* acc_empty = bars + 2 * STAGES2 + 2;  // [2], used in rank 0 only (8 arrivals)
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * STAGES2 + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int num_tiles = m_tiles * n_tiles;
  const int num_kb = (p.K + BK2 - 1) / BK2;

  auto tile_origin = [&](int tile, int& m0, int& n0) {
    constexpr int GM = 8;                          // 8 row tiles of 256 share a column tile in L2
    const int per_group = GM * n_tiles;
    const int first_m = (tile / per_group) * GM;
    const int gsz = min(GM, m_tiles - first_m);
    m0 = (first_m + (tile % per_group) % gsz) * (2 * BM2);
    n0 = ((tile % per_group) / gsz) * BN_OUT;
  };

  if (threadIdx.x == 0) {
    prefetch_tmap(&maps.a);
    prefetch_tmap(&maps.w[0]);
    for (int s = 0; s < STAGES2; ++s) {
      mbar_init(smem_u32(&full_bar[s]), 1);
      mbar_init(smem_u32(&empty_bar[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), 8);       // four epilogue warps in each CTA of the pair
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), 512);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                              // both CTAs' barriers exist before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                      // set-up above overlaps the previous kernel's tail

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer (both CTAs): own 128 rows of A, own half of the W tile ----
      constexpr int N_LOADS = (BN2 / 2) / W_BOX;
      int it = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += n_pairs) {
        int m0, n0;
        tile_origin(tile, m0, n0);
        const CUtensorMap* wmap;
        int wrow;
        if (EPI == EPI_SWIGLU) {
          wmap = rank ? &maps.w[1] : &maps.w[0];   // rank 0 stages gate rows, rank 1 the up rows of the same columns
          wrow = n0;
        } else {
          int n = n0, seg = 0;
          while (seg < 2 && n >= p.seg_rows[seg]) { n -= p.seg_rows[seg]; ++seg; }
          wmap = &maps.w[seg];
          wrow = n + (int)rank * (BN2 / 2);
        }
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES2;
          const uint32_t ph = (it / STAGES2) & 1;
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, abort_flag, status, 31)) { ok = false; break; }
          const uint32_t fb = smem_u32(&full_bar[s]);
          if (rank == 0) mbar_expect_tx(fb, 2 * (A_BYTES2 + B_BYTES2));     // both CTAs' bytes land on this barrier
          tma_load_2d_pair(smem_u32(a_tiles + (size_t)s * A_BYTES2), &maps.a, kb * BK2, m0 + (int)rank * BM2, fb);
          const uint32_t bdst = smem_u32(b_tiles + (size_t)s * B_BYTES2);
#pragma unroll
          for (int i = 0; i < N_LOADS; ++i)
            tma_load_2d_pair(bdst + i * W_BOX * (BK2 * 2), wmap, kb * BK2, wrow + i * W_BOX, fb);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---- MMA issuer (first CTA of the pair only) ----
      constexpr uint32_t idesc = umma_idesc_f16(2 * BM2, BN2);
      int it = 0, local = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += n_pairs, ++local) {
        const int buf = local & 1;
        const uint32_t use = (uint32_t)(local >> 1);
        ok = mbar_wait(smem_u32(&acc_empty[buf]), (use & 1) ^ 1, abort_flag, status, 35);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * BN2);
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % STAGES2;
          const uint32_t ph = (it / STAGES2) & 1;
          ok = mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag, status, 32);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(a_tiles + (size_t)s * A_BYTES2);
          const uint32_t b0 = smem_u32(b_tiles + (size_t)s * B_BYTES2);
#pragma unroll
          for (int k = 0; k < BK2 / UK2; ++k)
            umma_f16_pair(tacc, umma_desc_sw128(a0 + k * UK2 * 2), umma_desc_sw128(b0 + k * UK2 * 2), idesc,
                          (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit_pair(smem_u32(&empty_bar[s]));
        }
        if (ok) umma_commit_pair(smem_u32(&acc_full[buf]));
      }
    }
  } else {
    // ---- epilogue warps (both CTAs): own 128 rows x 256 columns ----
    const int quarter = warp & 3;
    int local = 0;
    for (int tile = pair; tile < num_tiles; tile += n_pairs, ++local) {
      const int buf = local & 1;
      const uint32_t use = (uint32_t)(local >> 1);
      if (!mbar_wait(smem_u32(&acc_full[buf]), use & 1, abort_flag, status, 33)) break;
      tc_fence_after();
      int m0, n0;
      tile_origin(tile, m0, n0);
      const int m = m0 + (int)rank * BM2 + quarter * 32 + lane;
      const uint32_t trow = tmem_base + (uint32_t)(buf * BN2) + ((uint32_t)(quarter * 32) << 16);
      if (EPI == EPI_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < BN_OUT; c += 32) {
          float g[32], u[32];
          tmem_ld32(trow + c, g);
          tmem_ld32(trow + BN_OUT + c, u);
          epi_swiglu_chunk32(p, m, n0 + c, g, u);
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < BN2; c += 32) {
          float v[32];
          tmem_ld32(trow + c, v);
          if (EPI == EPI_F32) epi_f32_chunk32(p, m, n0 + c, v);
          else epi_qkv_chunk32(p, m, n0 + c, v);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_rank0(smem_u32(&acc_empty[buf]));
    }
  }

  // ---- teardown: neither CTA leaves while its partner may still signal or read it ----
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    if (*abort_flag) __nanosleep(100000);
    tmem_dealloc_pair(tmem_base, 512);
  }
}

template <int EPI>
es_status_t launch_pair(const TmapSet2& maps, const LinearParams& p, int* status, cudaStream_t s, bool pdl) {
  constexpr int out = (EPI == EPI_SWIGLU) ? BN2 / 2 : BN2;
  const int m_tiles = (p.M + 2 * BM2 - 1) / (2 * BM2), n_tiles = (p.N + out - 1) / out;
  auto kern = linear_tc2_kernel<EPI>;
  static bool configured = false;
  if (!configured) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM2));
    configured = true;
  }
  static int sms = 0;
  if (sms == 0) {
    int dev = 0;
    ES_CUDA_CHECK(cudaGetDevice(&dev));
    ES_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  }
  const int tiles = m_tiles * n_tiles;
  int pairs = sms / 2;
  if (pairs > tiles) pairs = tiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(T2_THREADS);
  cfg.dynamicSmemBytes = SMEM2;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  ES_CUDA_CHECK(cudaLaunchKernelEx(&cfg, kern, maps, p, status, m_tiles, n_tiles));
  return ES_OK;
}

}  // namespace

// The pair kernel pays off when there are enough 256 x 256 tiles to keep every pair busy.
bool linear_tc2_supported(const LinearParams& p, int epi) {
  if (!linear_tc_supported(p, epi)) return false;
  const int out = (epi == EPI_SWIGLU) ? BN2 / 2 : BN2;
  if (epi == EPI_QKV)
    for (int s = 0; s < 3; ++s) if (p.seg_rows[s] % out) return false;
  const long long tiles = (long long)((p.M + 2 * BM2 - 1) / (2 * BM2)) * ((p.N + out - 1) / out);
  return p.M >= 2 * BM2 && tiles >= 74;
}

es_status_t launch_linear_tc2(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, int* status_word, bool pdl) {
  if (!linear_tc2_supported(p, epi)) return fail(ES_ERR_UNSUPPORTED, "pair kernel does not take this shape");
  TcMaps local;
  const TcMaps* maps = p.tc_maps;
  if (!maps) {
    ES_TRY(tc_build_maps(p, epi, p.M, &local));
    maps = &local;
  }
  const TmapSet2& t = *reinterpret_cast<const TmapSet2*>(maps);
  es_status_t st;
  switch (epi) {
    case EPI_F32: st = launch_pair<EPI_F32>(t, p, status_word, s, pdl); break;
    case EPI_SWIGLU: st = launch_pair<EPI_SWIGLU>(t, p, status_word, s, pdl); break;
    case EPI_QKV: st = launch_pair<EPI_QKV>(t, p, status_word, s, pdl); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

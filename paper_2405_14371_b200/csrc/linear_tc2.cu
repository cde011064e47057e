// Tensor-core kernel of the linear-layer family on CTA pairs (tcgen05 cta_group::2), for large M.
//
// A cluster of two CTAs computes a 256 x 256 output tile: each CTA stages its own 128 rows of A and
// one half (128 rows) of the W tile per 64-deep K block, and one thread of the pair's first CTA
// issues MMAs (M=256, N=256, K=16) that read both CTAs' shared memory and write both CTAs' TMEM
// (each CTA ends up with its 128 rows x 256 columns).  Per CTA that is half the shared-memory
// operand traffic per flop of the single-CTA 128 x 256 tile and a third less staging per K block,
// so the ring is deeper in time and the tensor pipe stalls less.  Persistent pairs walk the tiles;
// the accumulator is double buffered in TMEM (2 x 256 columns) so epilogues overlap the next tile.
// With NACC = 2 a pair computes a 256 x 512 tile instead (two 256-column accumulators that share the A
// rows; each CTA stages 128 rows of A and 256 rows of W per K block): a quarter fewer operand bytes per
// flop pulled through L2 — on a power-capped part those transfers cost about as much energy as the MMAs
// themselves — at the price of an epilogue that no longer overlaps the MMAs (all 512 TMEM columns hold
// one tile), so the loads of the next tile are all that runs beside it.
// Epilogue warps pass every 32-column chunk through a small shared-memory tile so that global stores
// (and residual loads) cover whole row segments instead of 16 bytes in each of 32 rows.
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
constexpr int A_BYTES2 = BM2 * BK2 * 2;          // 16 KB
constexpr int B_BYTES2 = (BN2 / 2) * BK2 * 2;    // this CTA's half of one 256-row W tile, 16 KB
constexpr int RING_BYTES2 = 192 * 1024;          // 6 stages of 32 KB (NACC = 1) or 4 of 48 KB (NACC = 2)
constexpr int MAX_STAGES2 = 6;
constexpr int EPI_AREA2 = 8 * EPI_STAGE_BYTES > 4 * EPI_STAGE_F32_BYTES ? 8 * EPI_STAGE_BYTES : 4 * EPI_STAGE_F32_BYTES;
constexpr size_t SMEM2 = 1024 + (size_t)RING_BYTES2 + EPI_AREA2 + 256;   // eight small or four large store-staging tiles

struct TmapSet2 {
  CUtensorMap a;
  CUtensorMap w[3];
};
static_assert(sizeof(TmapSet2) == sizeof(TcMaps), "TcMaps must hold four tensor maps");

// Threads: warp 0 = TMA producer, warp 1 = MMA issuer / TMEM owner, then the epilogue warps (TMEM lane quarter =
// warp % 4): four per accumulator for the fp16 epilogues; four in all for the fp32 one, whose store-staging tiles
// are larger (each warp then drains both accumulators of its quarter).
template <int EPI, int NACC> struct PairCfg {
  static constexpr int EPI_WARPS = (EPI == EPI_F32) ? 4 : 4 * NACC;
  static constexpr int THREADS = 64 + 32 * EPI_WARPS;
  static constexpr int STAGE = (EPI == EPI_F32) ? EPI_STAGE_F32_BYTES : EPI_STAGE_BYTES;
};

template <int EPI, int NACC>
__global__ void __launch_bounds__(PairCfg<EPI, NACC>::THREADS, 1)
linear_tc2_kernel(const __grid_constant__ TmapSet2 maps, const LinearParams p, int* status, int m_tiles, int n_tiles) {
  constexpr int ACC_OUT = (EPI == EPI_SWIGLU) ? BN2 / 2 : BN2;   // output columns of one accumulator
  constexpr int BN_OUT = NACC * ACC_OUT;                           // output columns of a tile
  constexpr int STAGE_BYTES = A_BYTES2 + NACC * B_BYTES2;
  constexpr int STAGES2 = RING_BYTES2 / STAGE_BYTES;
  constexpr int NBUF = 2 / NACC;                                   // accumulator buffers in the 512 TMEM columns
  static_assert(STAGES2 <= MAX_STAGES2 && STAGES2 * STAGE_BYTES == RING_BYTES2, "ring layout");
  pdl_launch_dependents();
  stamp_begin(p.stamp);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = smem;                    // stage s: A tile, then NACC half W tiles
  unsigned char* epi_stage = smem + RING_BYTES2;
  uint64_t* bars = (uint64_t*)(epi_stage + EPI_AREA2);
  uint64_t* full_bar = bars;                         // used in rank 0 only
  uint64_t* empty_bar = bars + MAX_STAGES2;          // one copy per CTA
  uint64_t* acc_full = bars + 2 * MAX_STAGES2;       // [2], one copy per CTA
  uint64_t* acc_empty = bars + 2 * MAX_STAGES2 + 2;  // [2], used in rank 0 only (every epilogue warp of both CTAs arrives)
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * MAX_STAGES2 + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  // split-K (plain epilogue only): every (tile, K slice) pair is a work item, slice-major, and the raw accumulator
  // goes to slice ks of the workspace [k_splits, M, N]
  const int k_splits = (EPI == EPI_F32 && p.k_splits > 1) ? p.k_splits : 1;
  const int mn_tiles = m_tiles * n_tiles;
  const int num_tiles = mn_tiles * k_splits;
  const int num_kb = (p.K + BK2 - 1) / BK2;
  const int kb_per = (num_kb + k_splits - 1) / k_splits;

  auto tile_origin = [&](int tile, int& m0, int& n0) {
    constexpr int GM = 16;                         // 16 row tiles of 256 share a column tile in L2 (8 measured 2-3 % slower, 32 the same)
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
      mbar_init(smem_u32(&acc_empty[b]), 2 * PairCfg<EPI, NACC>::EPI_WARPS);   // the epilogue warps of both CTAs
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
        const int ks = tile / mn_tiles;
        tile_origin(tile - ks * mn_tiles, m0, n0);
        const int kb0 = ks * kb_per, kb1 = min(num_kb, kb0 + kb_per);
        // W rows this CTA stages for accumulator a: SwiGLU - rank 0 the gate rows, rank 1 the up rows of the same
        // 128 columns; otherwise rows [r * 128, r * 128 + 128) of the accumulator's 256 columns, inside one segment
        const CUtensorMap* wmap[NACC];
        int wrow[NACC];
#pragma unroll
        for (int a = 0; a < NACC; ++a) {
          if (EPI == EPI_SWIGLU) {
            wmap[a] = rank ? &maps.w[1] : &maps.w[0];
            wrow[a] = n0 + a * ACC_OUT;
          } else {
            int n = n0 + a * ACC_OUT, seg = 0;
            while (seg < 2 && n >= p.seg_rows[seg]) { n -= p.seg_rows[seg]; ++seg; }
            wmap[a] = &maps.w[seg];
            wrow[a] = n + (int)rank * (BN2 / 2);
          }
        }
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES2;
          const uint32_t ph = (it / STAGES2) & 1;
          if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1, abort_flag, status, 31)) { ok = false; break; }
          const uint32_t fb = smem_u32(&full_bar[s]);
          if (rank == 0) mbar_expect_tx(fb, 2 * STAGE_BYTES);                 // both CTAs' bytes land on this barrier
          const uint32_t sdst = smem_u32(ring + (size_t)s * STAGE_BYTES);
          tma_load_2d_pair(sdst, &maps.a, kb * BK2, m0 + (int)rank * BM2, fb);
#pragma unroll
          for (int a = 0; a < NACC; ++a) {
            const uint32_t bdst = sdst + A_BYTES2 + a * B_BYTES2;
#pragma unroll
            for (int i = 0; i < N_LOADS; ++i)
              tma_load_2d_pair(bdst + i * W_BOX * (BK2 * 2), wmap[a], kb * BK2, wrow[a] + i * W_BOX, fb);
          }
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
        const int buf = local % NBUF;
        const uint32_t use = (uint32_t)(local / NBUF);
        ok = mbar_wait(smem_u32(&acc_empty[buf]), (use & 1) ^ 1, abort_flag, status, 35);
        if (!ok) break;
        tc_fence_after();
        const uint32_t tacc = tmem_base + (uint32_t)(buf * BN2);
        const int ks = tile / mn_tiles;
        const int kb0 = ks * kb_per, kb1 = min(num_kb, kb0 + kb_per);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % STAGES2;
          const uint32_t ph = (it / STAGES2) & 1;
          ok = mbar_wait(smem_u32(&full_bar[s]), ph, abort_flag, status, 32);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a0 = smem_u32(ring + (size_t)s * STAGE_BYTES);
          const uint32_t b0 = a0 + A_BYTES2;
#pragma unroll
          for (int k = 0; k < BK2 / UK2; ++k) {
            const uint64_t adesc = umma_desc_sw128(a0 + k * UK2 * 2);
#pragma unroll
            for (int a = 0; a < NACC; ++a)
              umma_f16_pair(tacc + (uint32_t)(a * BN2), adesc, umma_desc_sw128(b0 + a * B_BYTES2 + k * UK2 * 2), idesc,
                            (kb > kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(smem_u32(&empty_bar[s]));
        }
        if (ok) umma_commit_pair(smem_u32(&acc_full[buf]));
      }
    }
  } else {
    // ---- epilogue warps (both CTAs): own 128 rows x 256 columns ----
    using PC = PairCfg<EPI, NACC>;
    const int quarter = warp & 3;
    const int a0 = (EPI == EPI_F32) ? 0 : (warp - 2) >> 2;       // first accumulator of this warp
    constexpr int N_MY = (EPI == EPI_F32) ? NACC : 1;            // accumulators this warp drains
    unsigned char* stage = epi_stage + (size_t)(warp - 2) * PC::STAGE;
    int local = 0;
    for (int tile = pair; tile < num_tiles; tile += n_pairs, ++local) {
      const int buf = local % NBUF;
      const uint32_t use = (uint32_t)(local / NBUF);
      int m0, n0;
      const int ks = tile / mn_tiles;
      tile_origin(tile - ks * mn_tiles, m0, n0);
      const int mw = m0 + (int)rank * BM2 + quarter * 32;          // row of lane 0
      const int na = n0 + a0 * ACC_OUT;                            // first output column of this warp
      // plain epilogue: where the rows go and what is added to them (split-K: raw sums to the workspace slice)
      float* f_out = p.out_f32;
      const float* f_res = p.res;
      int64_t f_ld = p.ldo;
      if (k_splits > 1) { f_out = p.part + (int64_t)ks * p.M * p.N; f_res = nullptr; f_ld = p.N; }
      // what does not depend on the accumulator is fetched before it is complete: the row's place in the q output
      // and the KV pages, or the first chunk of the residual
      QkvRow row;
      float4 rv[2][8];
      if (EPI == EPI_QKV) row = qkv_row(p, mw + lane);
      if (EPI == EPI_F32) {
        f32_chunk32_load_res(f_out, f_res, f_ld, p.M, p.N, mw, na, lane, rv[0]);
      }
      if (!mbar_wait(smem_u32(&acc_full[buf]), use & 1, abort_flag, status, 33)) break;
      tc_fence_after();
      const uint32_t tacc = tmem_base + (uint32_t)(buf * BN2 + a0 * BN2) + ((uint32_t)(quarter * 32) << 16);
      if (EPI == EPI_SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < ACC_OUT; c += 32) {
          float g[32], u[32];
          tmem_ld32(tacc + c, g);
          tmem_ld32(tacc + ACC_OUT + c, u);
          epi_swiglu_chunk32_staged(p, mw, na + c, g, u, stage, lane);
        }
      } else if (EPI == EPI_QKV) {
#pragma unroll 1
        for (int c = 0; c < BN2; c += 32) {
          float v[32];
          tmem_ld32(tacc + c, v);
          epi_qkv_chunk32_staged(p, row, mw, na + c, v, stage, lane);
        }
      } else {
        // accumulator columns and output columns coincide (ACC_OUT == BN2); the residual of the next chunk is
        // requested before the current one is stored (two register sets, two chunks per trip of a rolled loop)
        constexpr int NCH = N_MY * (BN2 / 32);
#pragma unroll 1
        for (int c = 0; c < NCH; c += 2) {
          float v[32];
          f32_chunk32_load_res(f_out, f_res, f_ld, p.M, p.N, mw, na + (c + 1) * 32, lane, rv[1]);
          tmem_ld32(tacc + c * 32, v);
          f32_chunk32_staged<true>(f_out, f_res, f_ld, p.M, p.N, mw, na + c * 32, v, rv[0], stage, lane);
          if (c + 2 < NCH) f32_chunk32_load_res(f_out, f_res, f_ld, p.M, p.N, mw, na + (c + 2) * 32, lane, rv[0]);
          tmem_ld32(tacc + (c + 1) * 32, v);
          f32_chunk32_staged<true>(f_out, f_res, f_ld, p.M, p.N, mw, na + (c + 1) * 32, v, rv[1], stage, lane);
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
  stamp_end(p.stamp);
}

template <int EPI, int NACC>
es_status_t launch_pair(const TmapSet2& maps, const LinearParams& p, int* status, cudaStream_t s, bool pdl) {
  constexpr int out = NACC * ((EPI == EPI_SWIGLU) ? BN2 / 2 : BN2);
  const int m_tiles = (p.M + 2 * BM2 - 1) / (2 * BM2), n_tiles = (p.N + out - 1) / out;
  auto kern = linear_tc2_kernel<EPI, NACC>;
  static bool configured = false;
  if (!configured) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM2));
    configured = true;
  }
  const int sms = sm_count();          // of the current device: a process may drive GPUs of different sizes
  const int tiles = m_tiles * n_tiles * ((EPI == EPI_F32 && p.k_splits > 1) ? p.k_splits : 1);
  int pairs = sms / 2;
  if (pairs > tiles) pairs = tiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(PairCfg<EPI, NACC>::THREADS);
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

// Accumulators per tile: the 256 x 512 tile moves a quarter fewer operand bytes per flop but cannot hide its
// epilogue and quantises into coarser waves.  Measured against the 256 x 256 tile (same launch, 16384 or 8192
// rows): K = 4096 +-2 %, K = 8192 +7 % (+1 % with a residual to read), K = 28672 +13 % (+10 %).  It is taken
// for K >= 8192 when its waves, discounted for the traffic saved, come out shorter.
int pair_nacc(const LinearParams& p, int epi) {
  if (p.k_splits > 1) return 1;
  if (p.pair_nacc == 1 || p.pair_nacc == 2) return p.pair_nacc;
  const int force = tunables().tc_pair_wide;
  if (force == 0) return 1;
  if (force == 2) return 2;
  if (p.K < 8192) return 1;
  const int out = (epi == EPI_SWIGLU) ? BN2 / 2 : BN2;
  const long long mt = (p.M + 2 * BM2 - 1) / (2 * BM2);
  const long long t1 = mt * ((p.N + out - 1) / out), t2 = mt * ((p.N + 2 * out - 1) / (2 * out));
  const long long pairs = sm_count() / 2 > 0 ? sm_count() / 2 : 1;
  const long long w1 = (t1 + pairs - 1) / pairs, w2 = 2 * ((t2 + pairs - 1) / pairs);
  return (w2 * 92 < w1 * 100) ? 2 : 1;
}

template <int EPI>
es_status_t launch_pair_epi(const TmapSet2& maps, const LinearParams& p, int* status, cudaStream_t s, bool pdl) {
  return pair_nacc(p, EPI) == 2 ? launch_pair<EPI, 2>(maps, p, status, s, pdl) : launch_pair<EPI, 1>(maps, p, status, s, pdl);
}

}  // namespace

// The pair kernel pays off from about 40 tiles of 256 x 256 on: with fewer than the machine's 74 pairs' worth some
// SMs idle, but a CTA of a pair stages 128 + 128 rows per K block where a single CTA stages 128 + 256, and these
// launches are bound by what a CTA pulls through L2 (measured: 7B layers at 256 / 768 / 1024 tokens +3 / +3.5 / +6.5 %,
// 13B layers at 256 tokens +3 %, against a threshold of 74).
bool linear_tc2_supported(const LinearParams& p, int epi) {
  if (!linear_tc_supported(p, epi)) return false;
  const int out = (epi == EPI_SWIGLU) ? BN2 / 2 : BN2;
  if (epi == EPI_QKV)
    for (int s = 0; s < 3; ++s) if (p.seg_rows[s] % out) return false;
  const long long tiles = (long long)((p.M + 2 * BM2 - 1) / (2 * BM2)) * ((p.N + out - 1) / out);
  return p.M >= 2 * BM2 && tiles >= 40;
}

// K slices for a plain product with too few 256 x 256 tiles for the machine's 74 pairs (1 = do not use the pair
// kernel this way): as many slices as keep every (tile, slice) item in one wave, at least four K blocks each, and a
// workspace of linear_tc_split_workspace_bytes() must hold the partial sums.  Against the single-CTA split kernel
// a CTA pulls a third fewer operand bytes through L2 for the same output.
int linear_tc2_splits(const LinearParams& p, int epi) {
  if (epi != EPI_F32 || p.M < 2 * BM2 || p.N % 4 != 0 || !linear_tc_supported(p, epi)) return 1;
  const int tiles = ((p.M + 2 * BM2 - 1) / (2 * BM2)) * ((p.N + BN2 - 1) / BN2);
  const int pairs = sm_count() / 2;
  if (tiles >= pairs) return 1;
  const int num_kb = (p.K + BK2 - 1) / BK2;
  int s = pairs / tiles;
  if (s > 8) s = 8;
  if (s > num_kb / 4) s = num_kb / 4;
  while (s > 1 && (size_t)s * p.M * p.N * sizeof(float) > linear_tc_split_workspace_bytes()) --s;
  if (s < 2) return 1;
  const int kb_per = (num_kb + s - 1) / s;
  return (num_kb + kb_per - 1) / kb_per;       // no empty slice
}

es_status_t launch_linear_tc2(const LinearParams& p, int epi, cudaStream_t s, int64_t* launches, int* status_word, bool pdl) {
  if (p.k_splits > 1) {
    if (epi != EPI_F32 || p.part == nullptr || p.N % 4 != 0 || p.M < 2 * BM2 || !linear_tc_supported(p, epi))
      return fail(ES_ERR_INVALID_ARG, "split-K on CTA pairs needs the plain epilogue, a workspace, N %% 4 == 0 and M >= 256");
    const int num_kb = (p.K + BK2 - 1) / BK2;
    const int kb_per = (num_kb + p.k_splits - 1) / p.k_splits;
    if ((p.k_splits - 1) * kb_per >= num_kb) return fail(ES_ERR_INVALID_ARG, "split-K: %d slices leave one empty (K = %d)", p.k_splits, p.K);
  } else if (!linear_tc2_supported(p, epi)) {
    return fail(ES_ERR_UNSUPPORTED, "pair kernel does not take this shape");
  }
  TcMaps local;
  const TcMaps* maps = p.tc_maps;
  if (!maps) {
    ES_TRY(tc_build_maps(p, epi, p.M, &local));
    maps = &local;
  }
  const TmapSet2& t = *reinterpret_cast<const TmapSet2*>(maps);
  es_status_t st;
  switch (epi) {
    case EPI_F32: st = launch_pair_epi<EPI_F32>(t, p, status_word, s, pdl); break;
    case EPI_SWIGLU: st = launch_pair_epi<EPI_SWIGLU>(t, p, status_word, s, pdl); break;
    case EPI_QKV: st = launch_pair_epi<EPI_QKV>(t, p, status_word, s, pdl); break;
    default: return fail(ES_ERR_INVALID_ARG, "unknown epilogue %d", epi);
  }
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

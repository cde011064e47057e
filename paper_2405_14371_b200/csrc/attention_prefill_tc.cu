// Causal prefill attention on the tensor cores of sm_100a (tcgen05 / TMEM / TMA).
//
// One CTA handles 128 query rows of one (sequence, head); two CTAs share an SM, so that one's softmax
// runs beside the other's MMAs.  Q stays resident in shared memory; K and V arrive 64 keys at a time
// through a two-stage TMA ring (a 64-key tile is one KV page, or 64 rows of a contiguous K / V matrix).
// Per KV tile j:
//   S = Q K^T      tcgen05.mma, M=128 queries, N=64 keys, K=head_dim, fp32 in TMEM; S has two buffers
//                  (columns [0,64) and [64,128)) and S(j+1) is issued before the softmax of tile j has
//                  finished, so the softmax warps never wait for the tensor cores in steady state
//   softmax        four warps, one query row per thread (the thread holds its whole score row, so
//                  the row maximum and sum need no cross-lane traffic): running max / sum, P in fp16
//                  written to shared memory in the 128-byte-swizzled K-major layout.  With head_dim 128
//                  P(j) takes the place of K(j) in its ring stage (same size; K(j) is dead once S(j)
//                  is complete), which is what lets two CTAs fit in an SM.
//   O += P V       the accumulator lives in TMEM columns [128, 128+head_dim).  The running maximum is
//                  moved lazily: a row keeps its old reference maximum until the new one exceeds it by
//                  more than 8 (in log2 units: probabilities then stay below 256, exact enough in fp16
//                  and harmless in the fp32 sum), so the in-place rescale of O (tcgen05.ld / tcgen05.st,
//                  which must wait for the previous P V) is rare; the final division by the row sum makes
//                  the result independent of the reference used.
//                  V is consumed as an MN-major operand straight from its row-major tile
// Tiles entirely above the diagonal are skipped; the diagonal tile is masked in registers.
// Every wait is bounded; on a timeout the CTA records a code in the status word and leaves through
// the normal teardown (TMEM freed).
#include <string.h>

#include "es_internal.cuh"
#include "launch.cuh"
#include "sm100.cuh"

namespace es {

namespace {

constexpr int QT = 128;          // query rows per CTA
constexpr int KT = 64;           // keys per tile
constexpr int ATT_THREADS = 192;
constexpr int TMEM_ALLOC = 256;  // S: two buffers of 64 columns, O: up to 128
constexpr float RESCALE_GAP = 8.0f;   // a row's reference maximum moves only when the new maximum exceeds it by this (log2 units)

struct AttnMaps {
  CUtensorMap q, k, v, unused;
};
static_assert(sizeof(AttnMaps) == sizeof(TcMaps), "TcMaps must hold the attention maps");

struct AttnArgs {
  __half* out;               // [B, T, Hq*hd]
  const int* block_table;    // paged mode
  const int* slots;          // paged mode: [B] or nullptr
  int* status;
  int B, T, Hq, Hkv;
  int paged, P, pages_per_slot;
  const int* cu_rows;        // packed prompts: first query row of every sequence [B + 1], or nullptr (row b * T)
  float scale_log2e;         // log2(e) / sqrt(hd)
  unsigned long long* stamp; // optional time stamps of the launch, nullptr = none
};

template <int HD>
struct AttnSmem {
  static constexpr int HALVES = HD / 64;                 // 64-column pieces of a row
  static constexpr int Q_BYTES = QT * HD * 2;
  static constexpr int KV_TILE_BYTES = KT * HD * 2;      // one of K / V, one stage
  static constexpr int P_BYTES = QT * KT * 2;
  static constexpr bool P_IN_K = (KV_TILE_BYTES >= P_BYTES);   // P(j) overwrites K(j) in its ring stage
  static constexpr size_t TOTAL = 1024 + Q_BYTES + 4 * KV_TILE_BYTES + (P_IN_K ? 0 : 2 * P_BYTES) + 128;
};

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS, 2)
prefill_attn_tc_kernel(const __grid_constant__ AttnMaps maps, const AttnArgs a) {
  using L = AttnSmem<HD>;
  constexpr int HALVES = L::HALVES;
  pdl_launch_dependents();
  stamp_begin(a.stamp);
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* q_s = smem;                                   // [HALVES][128 rows][128 B]
  unsigned char* k_s = q_s + L::Q_BYTES;                       // [2 stages][HALVES][64 rows][128 B]
  unsigned char* v_s = k_s + 2 * L::KV_TILE_BYTES;
  unsigned char* p_own = v_s + 2 * L::KV_TILE_BYTES;           // [2][128 rows][128 B] when P does not fit a K stage
  uint64_t* bars = (uint64_t*)(p_own + (L::P_IN_K ? 0 : 2 * L::P_BYTES));
  uint64_t* q_full = bars;           // 1
  uint64_t* kv_full = bars + 1;      // [2]
  uint64_t* kv_empty = bars + 3;     // [2]
  uint64_t* s_full = bars + 5;       // [2] S buffer ready in TMEM
  uint64_t* p_full = bars + 7;       // [2] P of tile j in smem, O rescaled if it had to be (4 arrivals); one barrier per
                                     // tile parity: a warp may be one tile ahead of another, never two
  uint64_t* pv_done = bars + 9;      // P V accumulated
  uint32_t* tmem_slot = (uint32_t*)(bars + 10);
  // P of tile j (ring stage j & 1)
  auto p_tile = [&](int stage) -> unsigned char* {
    return L::P_IN_K ? k_s + stage * L::KV_TILE_BYTES : p_own + stage * L::P_BYTES;
  };
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q0 = blockIdx.x * QT, h = blockIdx.y, b = blockIdx.z;
  const int g = h / (a.Hq / a.Hkv);
  // rows of this sequence in the q / output matrices and its prompt length (packed prompts: from the first-row
  // table, which the host uploaded before the pass began; a.T is then the longest prompt and sizes the grid)
  const int row0 = a.cu_rows ? a.cu_rows[b] : b * a.T;
  const int Tb = a.cu_rows ? a.cu_rows[b + 1] - row0 : a.T;
  if (q0 >= Tb) {                                        // a tile past the end of a shorter prompt: nothing set up yet
    stamp_end(a.stamp);
    return;
  }
  const int q_hi = min(Tb, q0 + QT);                     // one past the last query row of this tile
  const int n_kv = (q_hi + KT - 1) / KT;                 // causal: keys 0 .. q_hi-1

  if (threadIdx.x == 0) {
    prefetch_tmap(&maps.q);
    prefetch_tmap(&maps.k);
    prefetch_tmap(&maps.v);
    mbar_init(smem_u32(q_full), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(smem_u32(&kv_full[s]), 1);
      mbar_init(smem_u32(&kv_empty[s]), 1);
    }
    mbar_init(smem_u32(&s_full[0]), 1);
    mbar_init(smem_u32(&s_full[1]), 1);
    mbar_init(smem_u32(&p_full[0]), 4);
    mbar_init(smem_u32(&p_full[1]), 4);
    mbar_init(smem_u32(pv_done), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(tmem_slot), TMEM_ALLOC);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();                                   // set-up above overlaps the previous kernel's tail
  const uint32_t tmem_s = tmem_base;            // two S buffers: columns [0, 64) and [64, 128)
  const uint32_t tmem_o = tmem_base + 128;      // columns [128, 128 + HD)

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer ----
      const uint32_t qb = smem_u32(q_full);
      mbar_expect_tx(qb, L::Q_BYTES);
#pragma unroll
      for (int hf = 0; hf < HALVES; ++hf)
        tma_load_2d(smem_u32(q_s + hf * (QT * 128)), &maps.q, h * HD + hf * 64, row0 + q0, qb);
      const int slot = a.paged ? (a.slots ? a.slots[b] : b) : 0;
      for (int j = 0; j < n_kv; ++j) {
        const int s = j & 1;
        const uint32_t ph = (uint32_t)((j >> 1) & 1);
        if (!mbar_wait(smem_u32(&kv_empty[s]), ph ^ 1, abort_flag, a.status, 11)) break;
        int row, col;
        if (a.paged) {
          const int t0 = j * KT;
          const int page = a.block_table[(int64_t)slot * a.pages_per_slot + t0 / a.P];
          row = (page * a.Hkv + g) * a.P + (t0 % a.P);
          col = 0;
        } else {
          row = row0 + j * KT;
          col = g * HD;
        }
        const uint32_t fb = smem_u32(&kv_full[s]);
        mbar_expect_tx(fb, 2 * L::KV_TILE_BYTES);
#pragma unroll
        for (int hf = 0; hf < HALVES; ++hf) {
          tma_load_2d(smem_u32(k_s + s * L::KV_TILE_BYTES + hf * (KT * 128)), &maps.k, col + hf * 64, row, fb);
          tma_load_2d(smem_u32(v_s + s * L::KV_TILE_BYTES + hf * (KT * 128)), &maps.v, col + hf * 64, row, fb);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issuer ----
      constexpr uint32_t idesc_s = umma_idesc_f16(QT, KT);                      // Q, K both K-major
      constexpr uint32_t idesc_o = umma_idesc_f16(QT, HD) | (1u << 16);          // V is MN-major
      bool ok = mbar_wait(smem_u32(q_full), 0, abort_flag, a.status, 12);
      // S(t) = Q K(t)^T into S buffer t & 1 (its previous reader, the softmax of tile t - 2, has signalled p_full)
      auto issue_s = [&](int t) {
        const uint32_t kb = smem_u32(k_s + (t & 1) * L::KV_TILE_BYTES);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const int hf = k / 4, kk = k % 4;
          umma_f16(tmem_s + (uint32_t)((t & 1) * KT), umma_desc_sw128(smem_u32(q_s + hf * (QT * 128)) + kk * 32),
                   umma_desc_sw128(kb + hf * (KT * 128) + kk * 32), idesc_s, k > 0 ? 1u : 0u);
        }
        umma_commit(smem_u32(&s_full[t & 1]));
      };
      int s_next = 0;                              // next S product to issue; runs at most one tile ahead of P V
      const uint64_t t_start = global_timer_ns();
      for (int j = 0; j < n_kv && ok;) {
        bool progressed = false;
        if (s_next < n_kv && s_next <= j + 1 && mbar_try_wait(smem_u32(&kv_full[s_next & 1]), (uint32_t)((s_next >> 1) & 1))) {
          tc_fence_after();
          issue_s(s_next);
          ++s_next;
          progressed = true;
        }
        // O += P V once the softmax threads have written P (and rescaled O if they had to)
        if (s_next > j && mbar_try_wait(smem_u32(&p_full[j & 1]), (uint32_t)((j >> 1) & 1))) {
          tc_fence_after();
          const int s = j & 1;
          const uint32_t vb = smem_u32(v_s + s * L::KV_TILE_BYTES);
          const uint32_t pb = smem_u32(p_tile(s));
#pragma unroll
          for (int k = 0; k < KT / 16; ++k)
            umma_f16(tmem_o, umma_desc_sw128(pb + k * 32),
                     umma_desc_sw128_mn(vb + k * (16 * 128), KT * 128, 1024), idesc_o, (j > 0 || k > 0) ? 1u : 0u);
          umma_commit(smem_u32(&kv_empty[s]));
          umma_commit(smem_u32(pv_done));
          ++j;
          progressed = true;
        }
        if (!progressed) {
          if (*abort_flag) { ok = false; break; }
          if (global_timer_ns() - t_start > 2000000000ull) {      // bounded: the whole tile loop gets two seconds
            *abort_flag = 1;
            if (a.status) { atomicCAS(a.status, 0, 13); a.status[1] = (int)blockIdx.x; }
            ok = false;
          }
        }
      }
    }
  } else {
    // ---- softmax / epilogue warps: thread = query row, TMEM lane quarter = warp % 4 ----
    const int quarter = warp & 3;
    const int r = quarter * 32 + lane;                 // row inside the tile
    const int qi = q0 + r;                             // absolute query position
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    float m_ref = -INFINITY, l_run = 0.f;              // reference maximum of the row (log2 units), running sum
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(smem_u32(&s_full[j & 1]), (uint32_t)((j >> 1) & 1), abort_flag, a.status, 15);
      if (!ok) break;
      tc_fence_after();
      float sc[KT];
      {
        float t0[32], t1[32];
        tmem_ld32(tmem_s + (uint32_t)((j & 1) * KT) + lane_off, t0);
        tmem_ld32(tmem_s + (uint32_t)((j & 1) * KT) + lane_off + 32, t1);
#pragma unroll
        for (int c = 0; c < 32; ++c) { sc[c] = t0[c]; sc[32 + c] = t1[c]; }
      }
      const int k0 = j * KT;
      float mx = -INFINITY;
      const bool diag = (k0 + KT - 1 > qi);            // some keys of this tile lie after the query
#pragma unroll
      for (int c = 0; c < KT; ++c) {
        float v = sc[c] * a.scale_log2e;
        if (diag && (k0 + c > qi)) v = -INFINITY;
        sc[c] = v;
        mx = fmaxf(mx, v);
      }
      // move the reference only on the first tile or when the new maximum is far above it
      const bool move = (mx > m_ref + RESCALE_GAP) || (m_ref == -INFINITY && mx > -INFINITY);
      const float m_new = move ? mx : m_ref;
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;      // a fully masked row (only rows past T) stays at 0
      const float alpha = move ? exp2f(m_ref - m_use) : 1.0f;       // m_ref = -inf on the first tile -> 0
      float psum = 0.f;
      uint32_t packed[KT / 2];
#pragma unroll
      for (int c = 0; c < KT; c += 2) {
        const float p0 = exp2f(sc[c] - m_use), p1 = exp2f(sc[c + 1] - m_use);
        const __half2 hh = __floats2half2_rn(p0, p1);
        // the sum uses the rounded probabilities, the same values the tensor cores multiply with V
        const float2 back = __half22float2(hh);
        psum += back.x + back.y;
        packed[c / 2] = *reinterpret_cast<const uint32_t*>(&hh);
      }
      l_run = l_run * alpha + psum;
      m_ref = m_new;
      // P row -> shared memory, 16-byte pieces at their swizzled places
      unsigned char* prow = p_tile(j & 1) + r * 128;
#pragma unroll
      for (int c8 = 0; c8 < 8; ++c8) {
        const uint4 val = make_uint4(packed[4 * c8], packed[4 * c8 + 1], packed[4 * c8 + 2], packed[4 * c8 + 3]);
        *reinterpret_cast<uint4*>(prow + ((c8 ^ (r & 7)) << 4)) = val;
      }
      // The previous P V must have landed before this warp signals tile j: every warp then follows pv_done phase by
      // phase (the parity test can only tell "this phase" from "the next", so a phase must never be skipped; waiting
      // for two phases at the end instead deadlocked whenever both had already completed).  P V(j - 1) was issued
      // before this tile's softmax began, so the wait is normally over at once.
      if (j > 0) {
        ok = mbar_wait(smem_u32(pv_done), (uint32_t)((j - 1) & 1), abort_flag, a.status, 16);
        if (!ok) break;
        tc_fence_after();
        // rescale the accumulator rows of this warp if any of them moved its reference; on the first tile there is
        // nothing to rescale: P V(0) overwrites O
        if (__any_sync(0xffffffffu, move)) {
#pragma unroll 1
          for (int c = 0; c < HD; c += 32) {
            float o[32];
            tmem_ld32(tmem_o + lane_off + c, o);
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= alpha;
            tmem_st32(tmem_o + lane_off + c, o);
          }
        }
      }
      fence_proxy_async_smem();      // P (generic stores) must be visible to the tensor cores' reads
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&p_full[j & 1]));
    }
    // every earlier phase of pv_done has been waited for inside the loop; the last one remains
    if (ok) ok = mbar_wait(smem_u32(pv_done), (uint32_t)((n_kv - 1) & 1), abort_flag, a.status, 17);
    if (ok) {
      tc_fence_after();
      const float inv = (l_run > 0.f) ? 1.0f / l_run : 0.f;
      __half* orow = a.out + ((int64_t)row0 + qi) * ((int64_t)a.Hq * HD) + (int64_t)h * HD;
#pragma unroll 1
      for (int c = 0; c < HD; c += 32) {
        float o[32];
        tmem_ld32(tmem_o + lane_off + c, o);
        if (qi < Tb) {
#pragma unroll
          for (int q8 = 0; q8 < 4; ++q8) {
            uint4 val;
            __half2 h0 = __floats2half2_rn(o[8 * q8] * inv, o[8 * q8 + 1] * inv);
            __half2 h1 = __floats2half2_rn(o[8 * q8 + 2] * inv, o[8 * q8 + 3] * inv);
            __half2 h2 = __floats2half2_rn(o[8 * q8 + 4] * inv, o[8 * q8 + 5] * inv);
            __half2 h3 = __floats2half2_rn(o[8 * q8 + 6] * inv, o[8 * q8 + 7] * inv);
            val.x = *reinterpret_cast<uint32_t*>(&h0); val.y = *reinterpret_cast<uint32_t*>(&h1);
            val.z = *reinterpret_cast<uint32_t*>(&h2); val.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(orow + c + 8 * q8) = val;
          }
        }
      }
    }
  }

  // ---- teardown ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (*abort_flag) __nanosleep(100000);
    tmem_dealloc(tmem_base, TMEM_ALLOC);
  }
  stamp_end(a.stamp);
}

bool is_paged(const PrefillAttnParams& p) { return p.kv.block_table != nullptr; }

template <int HD>
es_status_t launch_hd(const AttnMaps& maps, const PrefillAttnParams& p, cudaStream_t s, bool pdl) {
  auto kern = prefill_attn_tc_kernel<HD>;
  static bool configured = false;
  if (!configured) {
    ES_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)AttnSmem<HD>::TOTAL));
    configured = true;
  }
  AttnArgs a{};
  a.stamp = p.stamp;
  a.out = p.out;
  a.block_table = p.kv.block_table;
  a.slots = p.kv.slots;
  a.status = p.status;
  a.B = p.B; a.T = p.T; a.Hq = p.Hq; a.Hkv = p.Hkv;
  a.cu_rows = p.cu_rows;
  a.paged = is_paged(p) ? 1 : 0;
  a.P = p.kv.P;
  a.pages_per_slot = p.kv.pages_per_slot;
  a.scale_log2e = 1.4426950408889634f / sqrtf((float)HD);
  const dim3 grid((p.T + QT - 1) / QT, p.Hq, p.B);
  ES_CUDA_CHECK(launch_kernel(kern, grid, dim3(ATT_THREADS), AttnSmem<HD>::TOTAL, s, pdl, maps, a));
  return ES_OK;
}

}  // namespace

bool prefill_attention_tc_supported(const PrefillAttnParams& p) {
  if (!tma_available()) return false;
  if (p.hd != 64 && p.hd != 128) return false;
  if (p.Hq % p.Hkv) return false;
  if (((uintptr_t)p.q | (uintptr_t)p.kv.k | (uintptr_t)p.kv.v | (uintptr_t)p.out) % 16) return false;
  if (is_paged(p)) {
    // a 64-key tile must be one run of rows of the [pages * heads * page_tokens, head_dim] matrix
    if (p.kv.P % KT != 0) return false;
    if (p.kv.tok_stride != p.hd || p.kv.head_stride != (int64_t)p.kv.P * p.hd) return false;
  } else {
    if (p.kv.tok_stride != (int64_t)p.Hkv * p.hd || p.kv.head_stride != p.hd) return false;
  }
  return true;
}

es_status_t prefill_attention_tc_build_maps(const PrefillAttnParams& p, int64_t q_rows, TcMaps* out) {
  AttnMaps* m = reinterpret_cast<AttnMaps*>(out);
  memset(m, 0, sizeof(*m));
  const int64_t qw = (int64_t)p.Hq * p.hd;
  ES_TRY(tma_encode_2d_f16(&m->q, p.q, q_rows, qw, qw, QT));
  const int64_t kw = is_paged(p) ? p.hd : (int64_t)p.Hkv * p.hd;
  ES_TRY(tma_encode_2d_f16(&m->k, p.kv.k, p.kv_rows, kw, kw, KT));
  ES_TRY(tma_encode_2d_f16(&m->v, p.kv.v, p.kv_rows, kw, kw, KT));
  return ES_OK;
}

es_status_t launch_prefill_attention_tc(const PrefillAttnParams& p, cudaStream_t s, int64_t* launches, bool pdl) {
  if (p.B <= 0 || p.T <= 0) return ES_OK;
  if (!prefill_attention_tc_supported(p)) return fail(ES_ERR_UNSUPPORTED, "tensor-core attention does not take this layout");
  TcMaps local;
  const TcMaps* maps = p.tc_maps;
  if (!maps) {
    ES_TRY(prefill_attention_tc_build_maps(p, (int64_t)p.B * p.T, &local));
    maps = &local;
  }
  const AttnMaps& m = *reinterpret_cast<const AttnMaps*>(maps);
  es_status_t st = (p.hd == 128) ? launch_hd<128>(m, p, s, pdl) : launch_hd<64>(m, p, s, pdl);
  if (st == ES_OK && launches) ++*launches;
  return st;
}

}  // namespace es

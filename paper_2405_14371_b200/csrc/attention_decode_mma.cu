// Split-KV decode attention on the tensor cores (mma.sync m16n8k16), for launches with many
// (sequence, KV head, split) items: several sequences, long contexts, grouped-query heads.
//
// The kernel is bound by reading K and V once from HBM, so it is organised around what a warp has
// in flight: a warp owns 16 tokens at a time and fetches their K and V rows straight from global
// memory into registers with 16-byte loads, already in the layout the MMAs consume — no shared
// memory staging, no transposes:
//
//   * scores S[head, token] = q K^T: A = the group's query rows (up to 8 heads, padded to 16 rows),
//     B = K.  The contraction over the head dimension does not care in which order the dimensions
//     are visited, so thread (g, t) of a warp takes 16-byte pieces 4j + t of token g's row: its
//     eight halves are exactly the B fragments of two k-steps, and a warp-wide load touches 64
//     contiguous bytes of 8 rows.  The query fragments are gathered once with the same permutation.
//   * softmax: online (running max / sum per head), in fp32, on the accumulator fragments; the
//     probabilities, rounded to fp16, already sit where the next MMA wants its B operand.
//   * output O^T[dim, head] = V^T P^T: A = V^T.  A register of that fragment pairs one dimension of
//     two different tokens, so thread (g, t) loads the 16-byte pieces g and g + 8 of its four
//     tokens' rows (a warp-wide load touches 128 contiguous bytes of 4 rows) and builds the pairs
//     with one byte-permute each; MMA number i then produces dimensions 8g + i and 64 + 8g + i.
//
// A register set is refilled with a later block as soon as it has been consumed (K after the score MMAs, V
// after the output MMAs), so loads and arithmetic overlap.  With one or two query heads per KV head (DB) a
// warp keeps two 16-token blocks in registers — while it works on one, the other is on its way — at two CTAs
// per SM; with larger groups, whose blocks carry more arithmetic, one block per warp at three CTAs per SM
// measured faster (config 4 shape 30.5 against 33.7 us; 8 sequences x 32 heads x 680 keys 27.1 -> 25.0 us
// with two).  The four
// warps of a CTA are merged through shared memory in warp order and the result is written as the
// final row (one split) or as an unnormalised partial (o, max, sum) that the last CTA to arrive for the
// (sequence, KV head) merges in split order, exactly like the CUDA-core kernel, so results do not depend
// on scheduling.
#include "es_internal.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int MW = 4;          // warps per CTA
constexpr int MHD = 128;       // head dimension served by this kernel

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ld_kv(const __half* ptr) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr));
  return v;
}

__device__ __forceinline__ uint32_t word_of(const uint4& v, int w) { return w == 0 ? v.x : w == 1 ? v.y : w == 2 ? v.z : v.w; }

// halves number `i` (0..7) of two 16-byte pieces, packed {lo: from a, hi: from b}
__device__ __forceinline__ uint32_t pair_of(const uint4& a, const uint4& b, int i) {
  return __byte_perm(word_of(a, i >> 1), word_of(b, i >> 1), (i & 1) ? 0x7632 : 0x5410);
}

__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

template <int G, bool DB>
__global__ void __launch_bounds__(MW * 32, DB ? 2 : 3) decode_attn_mma_kernel(const DecodeAttnParams p) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  constexpr int HD = MHD;
  __shared__ float sm_o[MW][G][HD];
  __shared__ float sm_m[MW][G];
  __shared__ float sm_l[MW][G];
  __shared__ int s_last;

  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  // read-only state of earlier passes (slot list, page map, context length) may be read before the wait
  const int slot = p.kv.slots ? p.kv.slots[b] : b;
  // a context length beyond the sequence's page list is clamped to it: no page index is ever read past the row
  const int ctx_old = min(p.ctx_len[slot], p.kv.pages_per_slot * p.kv.P - p.ctx_add);
  const int ctx = ctx_old + p.ctx_add;
  const int tokens_per_split = p.pages_per_split * p.kv.P;
  const int t_begin = split * tokens_per_split;
  if (t_begin >= ctx) {
    pdl_wait();
    // an empty context: nobody will arrive to merge, the CTA of split 0 writes the zero rows
    if (split == 0 && ctx <= 0)
      for (int i = threadIdx.x; i < G * HD; i += MW * 32)
        p.out[((int64_t)b * p.Hq + ((int64_t)kvh * G + i / HD)) * HD + (i % HD)] = __float2half_rn(0.f);
    stamp_end(p.stamp);
    return;
  }
  const int t_end = min(ctx, t_begin + tokens_per_split);
  const float scale = rsqrtf((float)HD);
  const int64_t kv_head_off = (int64_t)kvh * p.kv.head_stride;
  const int* table = p.kv.block_table ? p.kv.block_table + (int64_t)slot * p.kv.pages_per_slot : nullptr;

  // base address of the 16-token block starting at token T (inside one page: P >= 16, T % 16 == 0)
  auto block_base = [&](int T) -> int64_t {
    const int lp = T / p.kv.P;
    const int page = table ? table[lp] : slot * p.kv.pages_per_slot + lp;
    return (int64_t)page * p.kv.page_stride + kv_head_off + (int64_t)(T - lp * p.kv.P) * p.kv.tok_stride;
  };
  auto load_k = [&](int T, uint4 (&kreg)[2][4]) {
    const int64_t base = block_base(T);
    const int last = t_end - 1 - T;                      // tokens past the end re-read the last valid row (masked below)
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int r = min(8 * nt + g, last);
      const __half* row = p.kv.k + base + (int64_t)r * p.kv.tok_stride;
#pragma unroll
      for (int j = 0; j < 4; ++j) kreg[nt][j] = ld_kv(row + (4 * j + t) * 8);
    }
  };
  auto load_v = [&](int T, uint4 (&vreg)[4][2]) {
    const int64_t base = block_base(T);
    const int last = t_end - 1 - T;
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
      const int r = min(2 * t + (q4 & 1) + 8 * (q4 >> 1), last);
      const __half* row = p.kv.v + base + (int64_t)r * p.kv.tok_stride;
      vreg[q4][0] = ld_kv(row + g * 8);
      vreg[q4][1] = ld_kv(row + (g + 8) * 8);
    }
  };

  float oacc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;      // head g (replicated in the 4 threads of the group)

  // A block's K and V rows are requested before the dependency wait when every one of its tokens was cached
  // by an earlier pass (the newest token's rows come from the kernel just before).
  constexpr int STEP = MW * 16;              // tokens between consecutive blocks of one warp
  uint4 kA[2][4], vA[4][2], kB[2][4], vB[4][2];
  const int T0 = t_begin + warp * 16;
  const bool earlyA = T0 < t_end && T0 + 16 <= ctx_old;
  const bool earlyB = DB && T0 + STEP < t_end && T0 + STEP + 16 <= ctx_old;
  if (earlyA) { load_k(T0, kA); load_v(T0, vA); }
  if (earlyB) { load_k(T0 + STEP, kB); load_v(T0 + STEP, vB); }

  pdl_wait();

  // query fragments: row g of the A operand = head g of the group (rows >= G and rows 8..15 are zero)
  uint4 qa[4];
  {
    const __half* qrow = p.q + ((int64_t)b * p.Hq + (int64_t)kvh * G + (g < G ? g : 0)) * HD;
#pragma unroll
    for (int j = 0; j < 4; ++j) qa[j] = (g < G) ? *reinterpret_cast<const uint4*>(qrow + (4 * j + t) * 8) : make_uint4(0, 0, 0, 0);
  }
  if (T0 < t_end && !earlyA) { load_k(T0, kA); load_v(T0, vA); }
  if (DB && T0 + STEP < t_end && !earlyB) { load_k(T0 + STEP, kB); load_v(T0 + STEP, vB); }

  // one block of 16 tokens at T out of (kreg, vreg); the registers are refilled with the block at Tn
  auto block = [&](int T, int Tn, uint4 (&kreg)[2][4], uint4 (&vreg)[4][2]) {
    // ---- scores of 16 tokens ----
    float s[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mma_f16(s[nt], qa[j].x, 0u, qa[j].y, 0u, kreg[nt][j].x, kreg[nt][j].y);
        mma_f16(s[nt], qa[j].z, 0u, qa[j].w, 0u, kreg[nt][j].z, kreg[nt][j].w);
      }
    }
    if (Tn < t_end) load_k(Tn, kreg);
    // ---- online softmax: this thread holds head g, tokens T + 2t, T + 2t + 1, T + 8 + 2t, T + 9 + 2t ----
    float sv[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int tok = T + 2 * t + (e & 1) + 8 * (e >> 1);
      sv[e] = (tok < t_end) ? s[e >> 1][e & 1] * scale : -INFINITY;
    }
    float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float mn = fmaxf(m_run, mx);              // finite: token T is valid
    const float alpha = __expf(m_run - mn);
    float pr[4], ps = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) { pr[e] = __expf(sv[e] - mn); ps += pr[e]; }
    ps += __shfl_xor_sync(0xffffffffu, ps, 1);
    ps += __shfl_xor_sync(0xffffffffu, ps, 2);
    l_run = l_run * alpha + ps;
    m_run = mn;
    // the output fragments hold heads 2t and 2t + 1: fetch their rescale factors from groups 2t, 2t + 1
    const float a_lo = __shfl_sync(0xffffffffu, alpha, (2 * t) * 4);
    const float a_hi = __shfl_sync(0xffffffffu, alpha, (2 * t + 1) * 4);
    const uint32_t pb0 = pack_h2(pr[0], pr[1]), pb1 = pack_h2(pr[2], pr[3]);
    // ---- output: 8 MMAs, number i yields dimensions 8g + i (rows 0..7) and 64 + 8g + i (rows 8..15) ----
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      oacc[i][0] *= a_lo; oacc[i][1] *= a_hi; oacc[i][2] *= a_lo; oacc[i][3] *= a_hi;
      mma_f16(oacc[i], pair_of(vreg[0][0], vreg[1][0], i), pair_of(vreg[0][1], vreg[1][1], i),
              pair_of(vreg[2][0], vreg[3][0], i), pair_of(vreg[2][1], vreg[3][1], i), pb0, pb1);
    }
    if (Tn < t_end) load_v(Tn, vreg);
  };
  if (DB) {
    for (int T = T0; T < t_end; T += 2 * STEP) {
      block(T, T + 2 * STEP, kA, vA);
      if (T + STEP < t_end) block(T + STEP, T + 3 * STEP, kB, vB);
    }
  } else {
    for (int T = T0; T < t_end; T += STEP) block(T, T + STEP, kA, vA);
  }

  // ---- merge the warps in warp order ----
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (2 * t < G) { sm_o[warp][2 * t][8 * g + i] = oacc[i][0]; sm_o[warp][2 * t][64 + 8 * g + i] = oacc[i][2]; }
    if (2 * t + 1 < G) { sm_o[warp][2 * t + 1][8 * g + i] = oacc[i][1]; sm_o[warp][2 * t + 1][64 + 8 * g + i] = oacc[i][3]; }
  }
  if (t == 0 && g < G) { sm_m[warp][g] = m_run; sm_l[warp][g] = l_run; }
  __syncthreads();
  for (int i = threadIdx.x; i < G * HD; i += MW * 32) {
    const int j = i / HD, c = i - j * HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < MW; ++w) mm = fmaxf(mm, sm_m[w][j]);
    float o = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < MW; ++w) {
      const float f = (sm_m[w][j] == -INFINITY) ? 0.f : __expf(sm_m[w][j] - mm);
      o += sm_o[w][j][c] * f;
      ll += sm_l[w][j] * f;
    }
    const int64_t row = (int64_t)b * p.Hq + ((int64_t)kvh * G + j);
    if (p.n_splits == 1) {
      p.out[row * HD + c] = __float2half_rn(o / ll);
    } else {
      float* dst = p.part + (row * p.n_splits + split) * (HD + 2);
      dst[c] = o;
      if (c == 0) { dst[HD] = mm; dst[HD + 1] = ll; }
    }
  }
  if (p.n_splits > 1 && p.merge_in_kernel) merge_splits_if_last<HD, G>(p, b, kvh, ctx, &s_last);
  stamp_end(p.stamp);
}

template <int G>
es_status_t launch_g(const DecodeAttnParams& p, cudaStream_t s, bool pdl) {
  ES_CUDA_CHECK(launch_kernel(decode_attn_mma_kernel<G, (G <= 2)>, dim3(p.n_splits, p.Hkv, p.B), dim3(MW * 32), 0, s, pdl, p));
  return ES_OK;
}

}  // namespace

bool decode_attention_mma_supported(const DecodeAttnParams& p) {
  if (p.hd != MHD || p.Hq % p.Hkv != 0) return false;
  const int G = p.Hq / p.Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8) return false;
  if (p.kv.P < 16 || p.kv.P % 16 != 0) return false;                      // a 16-token block never straddles pages
  if (p.kv.tok_stride % 8 != 0 || p.kv.head_stride % 8 != 0 || p.kv.page_stride % 8 != 0) return false;   // 16-byte loads
  if (((uintptr_t)p.kv.k | (uintptr_t)p.kv.v | (uintptr_t)p.q) % 16) return false;
  return true;
}

// The split kernel only; with p.merge_in_kernel the last CTA to arrive for a (sequence, KV head) merges the splits,
// otherwise the caller launches the merge kernel.
es_status_t launch_decode_attention_mma(const DecodeAttnParams& p, cudaStream_t s, bool pdl) {
  if (!decode_attention_mma_supported(p)) return fail(ES_ERR_UNSUPPORTED, "tensor-core decode attention does not take this layout");
  switch (p.Hq / p.Hkv) {
    case 1: return launch_g<1>(p, s, pdl);
    case 2: return launch_g<2>(p, s, pdl);
    case 4: return launch_g<4>(p, s, pdl);
    default: return launch_g<8>(p, s, pdl);
  }
}

}  // namespace es

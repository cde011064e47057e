// Split-KV decode attention over the paged cache: one query row per (sequence, head).
//
// A CTA takes one split (a run of KV pages) of one KV head and serves all query heads of that
// group, so K and V are read from HBM once per group.  Its warps take 32 tokens at a time:
//   * scores: one token per lane — the lane reads its token's whole K row with 16-byte loads and
//     forms the dot products with the query rows held in shared memory (no cross-lane traffic);
//   * softmax: running (max, sum) per head, updated once per 32 tokens with warp shuffles;
//   * values: the head dimension is spread over the lanes (coalesced V rows), the 32
//     probabilities are broadcast lane by lane with shuffles.
// The warps of a CTA are merged through shared memory in warp order.  With a single split the
// CTA writes the final output; otherwise it writes an unnormalised partial (o, max, sum) and bumps an
// arrival counter of its (sequence, KV head): the CTA that arrives last merges the partials of the
// group's rows in split order (no second launch, nobody waits, and the order of the merge is fixed,
// so results never depend on scheduling).
#include "es_internal.cuh"
#include "launch.cuh"

namespace es {

namespace {

constexpr int DWARPS = 8;

// PRE: keep the first block's K rows in registers across the dependency wait.  That shortens the
// critical path of small, latency-bound launches but costs registers, so launches with many CTAs
// (several sequences, long contexts), which live on occupancy, are built without it.
template <int HD, int G, bool PRE>
__global__ void __launch_bounds__(DWARPS * 32, PRE ? 1 : 2) decode_attn_split_kernel(const DecodeAttnParams p) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  constexpr int E = HD / 32;
  __shared__ __align__(16) float q_s[G][HD];
  __shared__ float sm_o[DWARPS][G][HD];
  __shared__ float sm_m[DWARPS][G];
  __shared__ float sm_l[DWARPS][G];
  __shared__ int s_last;

  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Everything up to pdl_wait() reads only state that no kernel of the current pass has written:
  // the slot list and page map (fixed), the slot's context length (last written when the previous
  // pass ended; the first kernel of a pass is launched with a full dependency) and the K / V rows of
  // tokens cached by earlier passes.  The newest token's K / V and the query come from the kernel
  // just before this one and are read after the wait.
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
      for (int i = threadIdx.x; i < G * HD; i += DWARPS * 32)
        p.out[((int64_t)b * p.Hq + (g * G + i / HD)) * HD + (i % HD)] = __float2half_rn(0.f);
    stamp_end(p.stamp);
    return;
  }
  const int t_end = min(ctx, t_begin + tokens_per_split);
  const float scale = rsqrtf((float)HD);
  constexpr bool PRELOAD = PRE && (G <= 2);     // K row of the first block kept in registers across the wait

  const int t_first = t_begin + warp * 32 + lane;
  const bool first_valid = t_first < t_end;
  const bool first_old = first_valid && t_first < ctx_old;
  uint32_t off16_first = 0;
  uint4 kpre[PRELOAD ? HD / 8 : 1];
  if (first_valid) {
    const __half* kr = kv_addr(p.kv, p.kv.k, slot, t_first, g);
    off16_first = (uint32_t)((kr - p.kv.k) >> 3);
    if (first_old) {
      if (PRELOAD) {
#pragma unroll
        for (int c = 0; c < (PRELOAD ? HD / 8 : 1); ++c) kpre[c] = reinterpret_cast<const uint4*>(kr)[c];
      } else {
#pragma unroll
        for (int c = 0; c < HD * 2; c += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(kr) + c));
      }
      const char* vr = reinterpret_cast<const char*>(p.kv.v + ((int64_t)off16_first << 3));
#pragma unroll
      for (int c = 0; c < HD * 2; c += 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(vr + c));
    }
  }

  pdl_wait();

  for (int i = threadIdx.x; i < G * HD; i += DWARPS * 32) {
    const int j = i / HD, c = i - j * HD;
    q_s[j][c] = __half2float(p.q[((int64_t)b * p.Hq + (g * G + j)) * HD + c]) * scale;
  }
  __syncthreads();

  float acc[G][E], m[G], l[G];
#pragma unroll
  for (int j = 0; j < G; ++j) {
#pragma unroll
    for (int e = 0; e < E; ++e) acc[j][e] = 0.f;
    m[j] = -INFINITY;
    l[j] = 0.f;
  }

  for (int t0 = t_begin + warp * 32; t0 < t_end; t0 += DWARPS * 32) {
    const int t = t0 + lane;
    const bool valid = t < t_end;
    const bool first = (t0 == t_begin + warp * 32);
    // offset of this lane's token row (same for K and V), in 16-byte units
    uint32_t off16 = 0;
    float s[G];
#pragma unroll
    for (int j = 0; j < G; ++j) s[j] = 0.f;
    if (valid) {
      const __half* kr;
      if (first) { off16 = off16_first; kr = p.kv.k + ((int64_t)off16 << 3); }
      else { kr = kv_addr(p.kv, p.kv.k, slot, t, g); off16 = (uint32_t)((kr - p.kv.k) >> 3); }
      const uint4* k4 = reinterpret_cast<const uint4*>(kr);
      const bool use_pre = PRELOAD && first && first_old;
      // all 16-byte pieces of the row are requested up front when registers allow (small groups)
      constexpr int KU = PRE ? ((G <= 2) ? HD / 8 : 4) : 8;
#pragma unroll KU
      for (int c = 0; c < HD / 8; ++c) {
        const uint4 u = use_pre ? kpre[PRELOAD ? c : 0] : k4[c];
        const __half2* h2 = reinterpret_cast<const __half2*>(&u);
        float kf[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __half22float2(h2[i]);
          kf[2 * i] = f.x;
          kf[2 * i + 1] = f.y;
        }
#pragma unroll
        for (int j = 0; j < G; ++j) {
          const float4 qa = *reinterpret_cast<const float4*>(&q_s[j][c * 8]);
          const float4 qb = *reinterpret_cast<const float4*>(&q_s[j][c * 8 + 4]);
          s[j] = fmaf(qa.x, kf[0], s[j]); s[j] = fmaf(qa.y, kf[1], s[j]);
          s[j] = fmaf(qa.z, kf[2], s[j]); s[j] = fmaf(qa.w, kf[3], s[j]);
          s[j] = fmaf(qb.x, kf[4], s[j]); s[j] = fmaf(qb.y, kf[5], s[j]);
          s[j] = fmaf(qb.z, kf[6], s[j]); s[j] = fmaf(qb.w, kf[7], s[j]);
        }
      }
    }
    float pr[G];
#pragma unroll
    for (int j = 0; j < G; ++j) {
      float cm = valid ? s[j] : -INFINITY;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(0xffffffffu, cm, o));
      const float mn = fmaxf(m[j], cm);          // finite: lane 0 of every block is valid
      const float alpha = __expf(m[j] - mn);
      pr[j] = valid ? __expf(s[j] - mn) : 0.f;
      float ps = pr[j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      l[j] = l[j] * alpha + ps;
#pragma unroll
      for (int e = 0; e < E; ++e) acc[j][e] *= alpha;
      m[j] = mn;
    }
    // value rows of the 32 tokens; lanes past the end carry probability 0 and a valid (repeated) offset
    const int cnt = min(32, t_end - t0);
    constexpr int VU = (PRE && G <= 2) ? 16 : 8;
#pragma unroll VU
    for (int jj = 0; jj < 32; ++jj) {
      const uint32_t o16 = __shfl_sync(0xffffffffu, off16, jj < cnt ? jj : 0);
      const __half* vr = p.kv.v + ((int64_t)o16 << 3) + lane * E;
      float vf[E];
      if (E == 4) {
        const uint2 u = *reinterpret_cast<const uint2*>(vr);
        const __half2* h2 = reinterpret_cast<const __half2*>(&u);
        const float2 a = __half22float2(h2[0]), c2 = __half22float2(h2[1]);
        vf[0] = a.x; vf[1] = a.y; vf[E - 2] = c2.x; vf[E - 1] = c2.y;
      } else {
        const float2 a = __half22float2(*reinterpret_cast<const __half2*>(vr));
        vf[0] = a.x; vf[1] = a.y;
      }
#pragma unroll
      for (int j = 0; j < G; ++j) {
        const float pv = __shfl_sync(0xffffffffu, pr[j], jj);
#pragma unroll
        for (int e = 0; e < E; ++e) acc[j][e] = fmaf(pv, vf[e], acc[j][e]);
      }
    }
  }

#pragma unroll
  for (int j = 0; j < G; ++j) {
#pragma unroll
    for (int e = 0; e < E; ++e) sm_o[warp][j][lane * E + e] = acc[j][e];
    if (lane == 0) { sm_m[warp][j] = m[j]; sm_l[warp][j] = l[j]; }
  }
  __syncthreads();
  // merge the warps in warp order; thread -> (head j, column c)
  for (int i = threadIdx.x; i < G * HD; i += DWARPS * 32) {
    const int j = i / HD, c = i - j * HD;
    float mm = -INFINITY;
#pragma unroll
    for (int w = 0; w < DWARPS; ++w) mm = fmaxf(mm, sm_m[w][j]);
    float o = 0.f, ll = 0.f;
#pragma unroll
    for (int w = 0; w < DWARPS; ++w) {
      const float f = (sm_m[w][j] == -INFINITY) ? 0.f : __expf(sm_m[w][j] - mm);
      o += sm_o[w][j][c] * f;
      ll += sm_l[w][j] * f;
    }
    const int64_t row = (int64_t)b * p.Hq + (g * G + j);
    if (p.n_splits == 1) {
      p.out[row * HD + c] = __float2half_rn(o / ll);
    } else {
      float* dst = p.part + (row * p.n_splits + split) * (HD + 2);
      dst[c] = o;
      if (c == 0) { dst[HD] = mm; dst[HD + 1] = ll; }
    }
  }
  if (p.n_splits > 1 && p.merge_in_kernel) merge_splits_if_last<HD, G>(p, b, g, ctx, &s_last);
  stamp_end(p.stamp);
}

// Merge of the splits as a launch of its own, for launches with many CTAs (see merge_in_kernel below): one CTA
// per (sequence, head), the same arithmetic in the same order as merge_splits_if_last.
template <int HD>
__global__ void __launch_bounds__(HD) decode_attn_merge_kernel(const DecodeAttnParams p) {
  pdl_launch_dependents();
  stamp_begin(p.stamp);
  const int h = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
  pdl_wait();
  const int slot = p.kv.slots ? p.kv.slots[b] : b;
  const int ctx = min(p.ctx_len[slot] + p.ctx_add, p.kv.pages_per_slot * p.kv.P);
  const int tokens_per_split = p.pages_per_split * p.kv.P;
  int active = (ctx + tokens_per_split - 1) / tokens_per_split;
  active = active < p.n_splits ? active : p.n_splits;
  const float* src = p.part + ((int64_t)b * p.Hq + h) * p.n_splits * (HD + 2);
  float mm = -INFINITY;
  for (int s = 0; s < active; ++s) mm = fmaxf(mm, src[(int64_t)s * (HD + 2) + HD]);
  float o = 0.f, ll = 0.f;
  for (int s = 0; s < active; ++s) {
    const float f = __expf(src[(int64_t)s * (HD + 2) + HD] - mm);
    o += src[(int64_t)s * (HD + 2) + c] * f;
    ll += src[(int64_t)s * (HD + 2) + HD + 1] * f;
  }
  p.out[((int64_t)b * p.Hq + h) * HD + c] = __float2half_rn(active > 0 ? o / ll : 0.f);
  stamp_end(p.stamp);
}

template <int HD, int G>
es_status_t launch_g(const DecodeAttnParams& p, cudaStream_t s, bool pdl) {
  const bool small = (long long)p.n_splits * p.Hkv * p.B <= 2 * sm_count();
  if (small)
    ES_CUDA_CHECK(launch_kernel(decode_attn_split_kernel<HD, G, true>, dim3(p.n_splits, p.Hkv, p.B), dim3(DWARPS * 32), 0, s, pdl, p));
  else
    ES_CUDA_CHECK(launch_kernel(decode_attn_split_kernel<HD, G, false>, dim3(p.n_splits, p.Hkv, p.B), dim3(DWARPS * 32), 0, s, pdl, p));
  return ES_OK;
}

template <int HD>
es_status_t launch_hd(const DecodeAttnParams& p, cudaStream_t s, bool pdl, int64_t* launches) {
  es_status_t st;
  // many items (several sequences, long contexts): the tensor-core kernel, which keeps more bytes in flight
  const bool many = (long long)p.n_splits * p.Hkv * p.B >= 128;
  if (many && tunables().attn_mma != 0 && decode_attention_mma_supported(p)) {
    ES_TRY(launch_decode_attention_mma(p, s, pdl));
    if (launches) ++*launches;
    if (p.n_splits > 1 && !p.merge_in_kernel) {
      ES_CUDA_CHECK(launch_kernel(decode_attn_merge_kernel<HD>, dim3(p.Hq, p.B), dim3(HD), 0, s, pdl, p));
      if (launches) ++*launches;
    }
    return ES_OK;
  }
  switch (p.Hq / p.Hkv) {
    case 1: st = launch_g<HD, 1>(p, s, pdl); break;
    case 2: st = launch_g<HD, 2>(p, s, pdl); break;
    case 4: st = launch_g<HD, 4>(p, s, pdl); break;
    case 8: st = launch_g<HD, 8>(p, s, pdl); break;
    default: return fail(ES_ERR_SHAPE, "query heads per KV head must be 1, 2, 4 or 8");
  }
  ES_TRY(st);
  if (launches) ++*launches;
  if (p.n_splits > 1 && !p.merge_in_kernel) {
    ES_CUDA_CHECK(launch_kernel(decode_attn_merge_kernel<HD>, dim3(p.Hq, p.B), dim3(HD), 0, s, pdl, p));
    if (launches) ++*launches;
  }
  return ES_OK;
}

}  // namespace

size_t decode_attention_counter_offset(int B, int Hq, int hd, int n_splits) {
  return ((size_t)B * Hq * n_splits * (hd + 2) * sizeof(float) + 255) / 256 * 256;
}
size_t decode_attention_counter_bytes(int B, int Hq) { return ((size_t)B * Hq * sizeof(int) + 255) / 256 * 256; }
size_t decode_attention_scratch_bytes(int B, int Hq, int hd, int n_splits) {
  return decode_attention_counter_offset(B, Hq, hd, n_splits) + decode_attention_counter_bytes(B, Hq);
}

es_status_t launch_decode_attention(const DecodeAttnParams& p0, cudaStream_t s, int64_t* launches, bool pdl) {
  if (p0.B <= 0) return ES_OK;
  if (p0.Hq % p0.Hkv != 0) return fail(ES_ERR_SHAPE, "n_heads %% n_kv_heads != 0");
  // Who merges the splits.  A small launch (about one wave of CTAs: one sequence) is bound by latency, and the
  // last CTA to arrive merges in place of a second launch (measured: 8.8 -> 8.0 us per layer at one sequence of
  // 512..768 keys).  A large launch merges faster with a kernel of its own, one CTA per head (16 sequences x 8 KV
  // heads x 3 splits: 30 us against 40 us per layer with the merge in the split kernel's tail).
  DecodeAttnParams p = p0;
  p.merge_in_kernel = (long long)p.n_splits * p.Hkv * p.B <= 2 * sm_count() ? 1 : 0;
  if (p.hd == 128) return launch_hd<128>(p, s, pdl, launches);
  if (p.hd == 64) return launch_hd<64>(p, s, pdl, launches);
  return fail(ES_ERR_SHAPE, "head_dim must be 64 or 128, got %d", p.hd);
}

}  // namespace es

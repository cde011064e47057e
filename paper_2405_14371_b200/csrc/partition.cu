// Host-side partition planners of the paper: joint device selection and layer-wise partition for
// minimum latency (Algorithm 1, Eq. 4) and for maximum pipeline throughput (Algorithm 2 and its
// state-transition equation).  Plain C++; nothing here touches the GPU.  The traces they consume
// (per-layer time, activation size, memory) are what es_layer_profile exports.
#include <math.h>

#include <limits>
#include <new>
#include <vector>

#include "es_internal.cuh"

namespace {

const double INF = std::numeric_limits<double>::infinity();

inline double comm(const double* O, const double* Bw, int M, int layer, int k, int j) {
  // Eq. 1: activation of `layer` sent from device k to device j; free on the same device
  if (k == j) return 0.0;
  const double b = Bw[(size_t)k * M + j];
  return b > 0.0 ? O[layer] / b : INF;
}

es_status_t check_common(int N, int M, const double* t_comp, const double* O, const double* Req, const double* Mem,
                         const double* Bw, int32_t* assign, double* value) {
  if (N <= 0 || M <= 0) return es::fail(ES_ERR_INVALID_ARG, "N and M must be positive");
  if (!t_comp || !O || !Req || !Mem || !Bw || !assign || !value) return es::fail(ES_ERR_INVALID_ARG, "null argument");
  return ES_OK;
}

// Largest dynamic-programming table either planner will allocate; beyond it the call is refused with
// ES_ERR_UNSUPPORTED instead of exhausting host memory.
constexpr double TABLE_BYTES_MAX = 4.0 * 1024 * 1024 * 1024;

es_status_t latency_impl(int32_t N, int32_t M, const double* t_comp, const double* O, const double* Req,
                         const double* Mem, const double* Bw, int32_t* assign, double* latency) {
  ES_TRY(check_common(N, M, t_comp, O, Req, Mem, Bw, assign, latency));
  if ((double)N * M * (12.0 + 8.0 * M) > TABLE_BYTES_MAX)
    return es::fail(ES_ERR_UNSUPPORTED, "N x M cells with M memory budgets each would exceed 4 GiB (N = %d, M = %d)", N, M);
  // DP(i, j): least time of layers 0..i with layer i on device j (Eq. 4); choice(i, j): device of layer i-1.
  // Each cell also carries the memory its own best path has placed on every device, which is how the
  // algorithm's "update memory" step is read: a move to device j is allowed only if that path still has room.
  std::vector<double> dp((size_t)N * M, INF);
  std::vector<int> choice((size_t)N * M, -1);
  std::vector<std::vector<double>> used((size_t)N * M);
  if (Req[0] > Mem[0]) return es::fail(ES_ERR_RANGE, "layer 0 does not fit on the source device");
  dp[0] = t_comp[0];                                   // privacy constraint: layer 0 on device 0
  used[0].assign(M, 0.0);
  used[0][0] = Req[0];
  for (int i = 1; i < N; ++i) {
    for (int j = 0; j < M; ++j) {
      double best = INF;
      int bk = -1;
      for (int k = 0; k < M; ++k) {
        const size_t prev = (size_t)(i - 1) * M + k;
        if (dp[prev] == INF) continue;
        if (used[prev][j] + Req[i] > Mem[j]) continue;
        double t = dp[prev] + t_comp[(size_t)i * M + j] + comm(O, Bw, M, i - 1, k, j);
        if (i == N - 1) t += comm(O, Bw, M, i, j, 0);  // the generated token returns to the source
        if (t < best) { best = t; bk = k; }
      }
      if (bk >= 0) {
        const size_t cur = (size_t)i * M + j;
        dp[cur] = best;
        choice[cur] = bk;
        used[cur] = used[(size_t)(i - 1) * M + bk];
        used[cur][j] += Req[i];
      }
    }
  }
  if (N == 1) {
    assign[0] = 0;
    *latency = dp[0] + comm(O, Bw, M, 0, 0, 0);
    return ES_OK;
  }
  int last = -1;
  double best = INF;
  for (int j = 0; j < M; ++j)
    if (dp[(size_t)(N - 1) * M + j] < best) { best = dp[(size_t)(N - 1) * M + j]; last = j; }
  if (last < 0) return es::fail(ES_ERR_RANGE, "no placement satisfies the memory budgets");
  for (int i = N - 1; i >= 0; --i) {
    assign[i] = last;
    last = choice[(size_t)i * M + last];
  }
  *latency = best;
  return ES_OK;
}

es_status_t throughput_impl(int32_t N, int32_t M, const double* t_comp, const double* O, const double* Req,
                            const double* Mem, const double* Bw, int32_t* assign, double* bottleneck) {
  ES_TRY(check_common(N, M, t_comp, O, Req, Mem, Bw, assign, bottleneck));
  if (M > 20) return es::fail(ES_ERR_UNSUPPORTED, "the subset table is 2^M: at most 20 devices");
  if (N >= (1 << 24)) return es::fail(ES_ERR_UNSUPPORTED, "at most 2^24 layers");
  const int S_ALL = 1 << M;
  // (N + 1) x 2^M x M cells of one double and one packed back-pointer
  if ((double)(N + 1) * S_ALL * M * 12.0 > TABLE_BYTES_MAX)
    return es::fail(ES_ERR_UNSUPPORTED, "the table of (N + 1) x 2^M x M cells would exceed 4 GiB (N = %d, M = %d)", N, M);
  // prefix sums of time per device and of memory: t_comp^{i->m, j} and Req_{i->m}
  std::vector<double> tp((size_t)(N + 1) * M, 0.0), rp(N + 1, 0.0);
  for (int i = 0; i < N; ++i) {
    rp[i + 1] = rp[i] + Req[i];
    for (int j = 0; j < M; ++j) tp[(size_t)(i + 1) * M + j] = tp[(size_t)i * M + j] + t_comp[(size_t)i * M + j];
  }
  auto seg_t = [&](int a, int b, int j) { return tp[(size_t)b * M + j] - tp[(size_t)a * M + j]; };   // layers a..b-1
  // g(c, S, k): least bottleneck stage time for the first c layers on the device set S (every device one
  // contiguous range, in the order used) with k last.  c counts layers, 1 <= c <= N.
  auto idx = [&](int c, int S, int k) { return ((size_t)c * S_ALL + S) * M + k; };
  std::vector<double> g((size_t)(N + 1) * S_ALL * M, INF);
  std::vector<int> from((size_t)(N + 1) * S_ALL * M, -1);      // previous (layer count, last device) as count * 32 + device
  // the source device holds the first shard: layer 0 is pinned to it, and it may keep more layers
  for (int c = 1; c <= N; ++c)
    if (rp[c] - rp[0] <= Mem[0]) g[idx(c, 1, 0)] = seg_t(0, c, 0);
  for (int c = 1; c < N; ++c) {
    for (int S = 1; S < S_ALL; ++S) {
      if (!(S & 1)) continue;
      for (int k = 0; k < M; ++k) {
        if (!((S >> k) & 1)) continue;
        const double cur = g[idx(c, S, k)];
        if (cur == INF) continue;
        for (int j = 0; j < M; ++j) {
          if ((S >> j) & 1) continue;
          const int S2 = S | (1 << j);
          const double tc = comm(O, Bw, M, c - 1, k, j);          // activation of the previous shard's last layer
          for (int m = c + 1; m <= N; ++m) {                       // device j takes layers c..m-1
            if (rp[m] - rp[c] > Mem[j]) break;
            const double t = fmax(cur, fmax(tc, seg_t(c, m, j)));
            const size_t at = idx(m, S2, j);
            if (t < g[at]) { g[at] = t; from[at] = c * 32 + k; }
          }
        }
      }
    }
  }
  double best = INF;
  int bS = -1, bk = -1;
  for (int S = 1; S < S_ALL; ++S)
    for (int k = 0; k < M; ++k)
      if (g[idx(N, S, k)] < best) { best = g[idx(N, S, k)]; bS = S; bk = k; }
  if (bS < 0) return es::fail(ES_ERR_RANGE, "no placement satisfies the memory budgets");
  int c = N, S = bS, k = bk;
  while (c > 0) {
    const size_t at = idx(c, S, k);
    const int pc = from[at] < 0 ? 0 : from[at] / 32;
    for (int i = pc; i < c; ++i) assign[i] = k;
    if (from[at] < 0) break;
    const int pk = from[at] % 32;
    S &= ~(1 << k);
    k = pk;
    c = pc;
  }
  *bottleneck = best;
  return ES_OK;
}

}  // namespace

extern "C" {

// Nothing is thrown across the C boundary: running out of host memory is reported as a status.
es_status_t es_partition_latency(int32_t N, int32_t M, const double* t_comp, const double* O, const double* Req,
                                 const double* Mem, const double* Bw, int32_t* assign, double* latency) {
  try {
    return latency_impl(N, M, t_comp, O, Req, Mem, Bw, assign, latency);
  } catch (const std::bad_alloc&) {
    return es::fail(ES_ERR_UNSUPPORTED, "out of host memory for the planner's table (N = %d, M = %d)", N, M);
  }
}

es_status_t es_partition_throughput(int32_t N, int32_t M, const double* t_comp, const double* O, const double* Req,
                                    const double* Mem, const double* Bw, int32_t* assign, double* bottleneck) {
  try {
    return throughput_impl(N, M, t_comp, O, Req, Mem, Bw, assign, bottleneck);
  } catch (const std::bad_alloc&) {
    return es::fail(ES_ERR_UNSUPPORTED, "out of host memory for the planner's table (N = %d, M = %d)", N, M);
  }
}

}  // extern "C"

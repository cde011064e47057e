"""Brute-force judges for the paper's two partition problems.  TEST INFRASTRUCTURE ONLY.

Plain enumeration straight from the problem statements (Sec. "Optimize LLM inference latency", Eq. 1-2 with
the privacy and memory constraints; Sec. "Optimize LLM inference throughput"): no dynamic programming, no
pruning, so that the planners in the library can be checked against something obviously correct on tiny
instances.  Shares no code with the library.
"""
from __future__ import annotations

import itertools
import math


def _comm(O, Bw, layer, k, j):
    if k == j:
        return 0.0
    return O[layer] / Bw[k][j] if Bw[k][j] > 0 else math.inf


def latency_bruteforce(t_comp, O, Req, Mem, Bw):
    """min over ALL layer->device maps with X[0,0] = 1 and per-device memory sums within budget of
    T_tol (Eq. 2) plus the token's return from the last layer's device to device 0."""
    N, M = len(t_comp), len(t_comp[0])
    best, arg = math.inf, None
    for tail in itertools.product(range(M), repeat=N - 1):
        a = (0,) + tail
        use = [0.0] * M
        for i, j in enumerate(a):
            use[j] += Req[i]
        if any(use[j] > Mem[j] for j in range(M)):
            continue
        t = sum(t_comp[i][a[i]] for i in range(N))
        t += sum(_comm(O, Bw, i - 1, a[i - 1], a[i]) for i in range(1, N))
        t += _comm(O, Bw, N - 1, a[N - 1], 0)
        if t < best:
            best, arg = t, list(a)
    return arg, best


def throughput_bruteforce(t_comp, O, Req, Mem, Bw):
    """min over ordered device sequences starting at device 0 (each device used once, one contiguous layer
    range each, in order) and over all cut points, of the slowest stage: max over stages of
    max(stage compute time, time to receive the previous stage's last activation)."""
    N, M = len(t_comp), len(t_comp[0])
    best, arg = math.inf, None
    others = list(range(1, M))
    for r in range(0, M):
        for perm in itertools.permutations(others, r):
            devs = (0,) + perm
            s = len(devs)
            if s > N:
                continue
            for cuts in itertools.combinations(range(1, N), s - 1):
                bounds = (0,) + cuts + (N,)
                worst, ok = 0.0, True
                for q in range(s):
                    a, b, j = bounds[q], bounds[q + 1], devs[q]
                    if sum(Req[a:b]) > Mem[j]:
                        ok = False
                        break
                    stage = sum(t_comp[i][j] for i in range(a, b))
                    if q > 0:
                        stage = max(stage, _comm(O, Bw, a - 1, devs[q - 1], j))
                    worst = max(worst, stage)
                if ok and worst < best:
                    best = worst
                    arg = [devs[q] for q in range(s) for _ in range(bounds[q], bounds[q + 1])]
    return arg, best

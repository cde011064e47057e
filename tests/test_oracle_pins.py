"""Pins for the CPU oracle: checks against things the mathematics fixes, not against itself."""
import math
import os

import pytest
import torch

from oracle import decoder as O
from workload import TINY, LLAMA2_7B, LLAMA2_13B, LLAMA2_70B, ModelShape, shard_weights, prompt_ids

torch.manual_seed(0)
SMALL = ModelShape("small", 3, 32, 4, 2, 8, 48, 50)


def _rand_weights(model, n_layers, scale=0.3, seed=1):
    g = torch.Generator().manual_seed(seed)
    d, f = model.d_model, model.d_ffn

    def r(*s):
        return (torch.randn(*s, generator=g) * scale).half()

    layers = []
    for _ in range(n_layers):
        layers.append({
            "attn_norm": (1 + 0.1 * torch.randn(d, generator=g)).half(),
            "wq": r(model.q_dim, d), "wk": r(model.kv_dim, d), "wv": r(model.kv_dim, d),
            "wo": r(d, model.q_dim),
            "ffn_norm": (1 + 0.1 * torch.randn(d, generator=g)).half(),
            "w_gate": r(f, d), "w_up": r(f, d), "w_down": r(d, f),
        })
    return {"layers": layers, "tok_embedding": r(model.vocab, d),
            "final_norm": (1 + 0.1 * torch.randn(d, generator=g)).half(), "lm_head": r(model.vocab, d)}


# ---- attention -------------------------------------------------------------------------

def _bruteforce_attention(q, k, v, q_pos0=0):
    """Scalar loops straight from the definition."""
    Tq, Hq, hd = q.shape
    Tk, Hkv, _ = k.shape
    grp = Hq // Hkv
    out = [[[0.0] * hd for _ in range(Hq)] for _ in range(Tq)]
    for i in range(Tq):
        for h in range(Hq):
            g = h // grp
            scores = []
            for j in range(Tk):
                if j <= i + q_pos0:
                    scores.append(sum(float(q[i, h, c]) * float(k[j, g, c]) for c in range(hd)) / math.sqrt(hd))
            mx = max(scores)
            e = [math.exp(s - mx) for s in scores]
            z = sum(e)
            for c in range(hd):
                out[i][h][c] = sum(e[j] / z * float(v[j, g, c]) for j in range(len(scores)))
    return torch.tensor(out, dtype=torch.float64)


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (4, 2), (4, 1)])
def test_attention_matches_bruteforce(Hq, Hkv):
    q = torch.randn(6, Hq, 8, dtype=torch.float64)
    k = torch.randn(6, Hkv, 8, dtype=torch.float64)
    v = torch.randn(6, Hkv, 8, dtype=torch.float64)
    got = O.causal_attention_matrix(q, k, v)
    assert torch.allclose(got, _bruteforce_attention(q, k, v), atol=1e-12)


def test_attention_with_query_offset_matches_bruteforce():
    q = torch.randn(2, 2, 4, dtype=torch.float64)
    k = torch.randn(5, 1, 4, dtype=torch.float64)
    v = torch.randn(5, 1, 4, dtype=torch.float64)
    got = O.causal_attention_matrix(q, k, v, q_pos0=3)
    assert torch.allclose(got, _bruteforce_attention(q, k, v, 3), atol=1e-12)


def test_softmax_rows_sum_to_one_via_ones_values():
    # with v == 1 everywhere the output is the row sum of the softmax
    q = torch.randn(7, 2, 4, dtype=torch.float64)
    k = torch.randn(7, 2, 4, dtype=torch.float64)
    v = torch.ones(7, 2, 4, dtype=torch.float64)
    assert torch.allclose(O.causal_attention_matrix(q, k, v), torch.ones(7, 2, 4, dtype=torch.float64), atol=1e-14)


def test_zero_queries_give_running_mean_of_values():
    T = 9
    q = torch.zeros(T, 2, 4, dtype=torch.float64)
    k = torch.randn(T, 2, 4, dtype=torch.float64)
    v = torch.randn(T, 2, 4, dtype=torch.float64)
    want = torch.cumsum(v, 0) / torch.arange(1, T + 1, dtype=torch.float64)[:, None, None]
    assert torch.allclose(O.causal_attention_matrix(q, k, v), want, atol=1e-13)


def test_first_position_returns_its_own_value():
    q = torch.randn(4, 2, 4); k = torch.randn(4, 2, 4); v = torch.randn(4, 2, 4)
    assert torch.allclose(O.causal_attention_matrix(q, k, v)[0], v[0], atol=1e-6)


def test_gqa_equals_mha_with_repeated_kv():
    q = torch.randn(5, 4, 8, dtype=torch.float64)
    k = torch.randn(5, 2, 8, dtype=torch.float64)
    v = torch.randn(5, 2, 8, dtype=torch.float64)
    a = O.causal_attention_matrix(q, k, v)
    b = O.causal_attention_matrix(q, k.repeat_interleave(2, dim=1), v.repeat_interleave(2, dim=1))
    assert torch.equal(a, b)


# ---- RoPE ------------------------------------------------------------------------------

def test_rope_identity_at_position_zero():
    x = torch.randn(1, 3, 16, dtype=torch.float64)
    assert torch.equal(O.apply_rope(x, torch.tensor([0]), 10000.0), x)


def test_rope_hand_computed_rotation():
    # head_dim 4: pair 0 turns by p*1, pair 1 by p*theta^(-1/2)
    x = torch.tensor([[[1.0, 0.0, 0.0, 2.0]]], dtype=torch.float64)
    p, theta = 3, 100.0
    y = O.apply_rope(x, torch.tensor([p]), theta)[0, 0]
    a1 = p * theta ** -0.5
    want = [math.cos(p), math.sin(p), -2.0 * math.sin(a1), 2.0 * math.cos(a1)]
    assert torch.allclose(y, torch.tensor(want, dtype=torch.float64), atol=1e-15)


def test_rope_preserves_norm_and_is_relative():
    q = torch.randn(6, 2, 16, dtype=torch.float64)
    k = torch.randn(6, 2, 16, dtype=torch.float64)
    pos = torch.arange(6)
    qa, ka = O.apply_rope(q, pos, 10000.0), O.apply_rope(k, pos, 10000.0)
    assert torch.allclose(qa.norm(dim=-1), q.norm(dim=-1), atol=1e-12)
    qb, kb = O.apply_rope(q, pos + 37, 10000.0), O.apply_rope(k, pos + 37, 10000.0)
    sa = torch.einsum("ihc,jhc->hij", qa, ka)
    sb = torch.einsum("ihc,jhc->hij", qb, kb)
    assert torch.allclose(sa, sb, atol=1e-10)


def test_rope_frequency_of_last_pair():
    # the last pair turns by pos * theta^(-(hd-2)/hd)
    hd, theta, p = 8, 10000.0, 5
    x = torch.zeros(1, 1, hd, dtype=torch.float64); x[0, 0, hd - 2] = 1.0
    y = O.apply_rope(x, torch.tensor([p]), theta)[0, 0]
    ang = p * theta ** (-(hd - 2) / hd)
    assert abs(float(y[hd - 2]) - math.cos(ang)) < 1e-15 and abs(float(y[hd - 1]) - math.sin(ang)) < 1e-15


# ---- RMSNorm, SwiGLU -------------------------------------------------------------------

def test_rmsnorm_constant_vector_closed_form():
    c, eps = 3.0, 1e-5
    y = O.rmsnorm(torch.full((2, 64), c, dtype=torch.float64), torch.ones(64, dtype=torch.float64), eps)
    assert torch.allclose(y, torch.full((2, 64), c / math.sqrt(c * c + eps), dtype=torch.float64), atol=1e-15)


def test_rmsnorm_unit_rms_scale_invariance_and_gain():
    x = torch.randn(3, 128, dtype=torch.float64)
    g = torch.rand(128, dtype=torch.float64) + 0.5
    y = O.rmsnorm(x, torch.ones(128, dtype=torch.float64), 0.0)
    assert torch.allclose((y * y).mean(-1), torch.ones(3, dtype=torch.float64), atol=1e-12)
    assert torch.allclose(O.rmsnorm(7.5 * x, g, 0.0), O.rmsnorm(x, g, 0.0), atol=1e-12)
    assert torch.allclose(O.rmsnorm(x, g, 0.0), y * g, atol=1e-12)


def test_rmsnorm_eps_inside_sqrt():
    # x = 0 except one element: mean of squares = a^2/n; eps must add to that, under the root
    n, a, eps = 4, 2.0, 0.5
    x = torch.zeros(1, n, dtype=torch.float64); x[0, 1] = a
    y = O.rmsnorm(x, torch.ones(n, dtype=torch.float64), eps)
    assert abs(float(y[0, 1]) - a / math.sqrt(a * a / n + eps)) < 1e-15


def test_silu_special_values():
    z = torch.tensor([0.0, 40.0, -40.0, 1.0], dtype=torch.float64)
    y = O.silu(z)
    assert float(y[0]) == 0.0
    assert abs(float(y[1]) - 40.0) < 1e-12 and abs(float(y[2])) < 1e-12
    assert abs(float(y[3]) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15


# ---- layer plumbing --------------------------------------------------------------------

def test_zero_output_projections_make_layers_identity():
    w = _rand_weights(SMALL, 3)
    for lw in w["layers"]:
        lw["wo"].zero_(); lw["w_down"].zero_()
    ids = torch.tensor([3, 1, 4, 1, 5])
    x, _ = O.shard_forward_full(SMALL, w, 0, 3, ids=ids)
    assert torch.equal(x, w["tok_embedding"][ids].float())


def test_zero_gate_removes_ffn():
    w = _rand_weights(SMALL, 1)
    w2 = {k: v for k, v in w.items()}
    lw = dict(w["layers"][0]); lw["w_gate"] = torch.zeros_like(lw["w_gate"])
    lw_noffn = dict(lw); lw_noffn["w_down"] = torch.zeros_like(lw["w_down"])
    x = torch.randn(4, SMALL.d_model, dtype=torch.float64)
    a = O.layer_forward_full(x, lw, SMALL, dtype=torch.float64)
    b = O.layer_forward_full(x, lw_noffn, SMALL, dtype=torch.float64)
    assert torch.equal(a, b)


def test_layer_against_handwritten_single_token():
    # T = 1: attention returns v, RoPE at position 0 is the identity -> closed form
    w = _rand_weights(SMALL, 1)["layers"][0]
    d = SMALL.d_model
    x = torch.randn(1, d, dtype=torch.float64)
    W = {k: v.double() for k, v in w.items()}
    h = x / torch.sqrt((x * x).mean() + SMALL.rms_eps) * W["attn_norm"]
    v = h @ W["wv"].T                                                # [1, Hkv*hd]
    o = v.reshape(SMALL.n_kv_heads, 1, SMALL.head_dim).expand(-1, 2, -1).reshape(1, -1)  # kv head g serves q heads 2g, 2g+1
    y = x + o @ W["wo"].T
    h2 = y / torch.sqrt((y * y).mean() + SMALL.rms_eps) * W["ffn_norm"]
    gte = h2 @ W["w_gate"].T
    y = y + ((gte / (1 + torch.exp(-gte))) * (h2 @ W["w_up"].T)) @ W["w_down"].T
    got = O.layer_forward_full(x, w, SMALL, dtype=torch.float64)
    assert torch.allclose(got, y, atol=1e-12)


# ---- whole decoder ---------------------------------------------------------------------

@pytest.mark.parametrize("dtype,tol", [(torch.float64, 1e-11), (torch.float32, 2e-5)])
def test_incremental_equals_full(dtype, tol):
    w = _rand_weights(SMALL, 3)
    ids = torch.tensor([7, 3, 9, 11, 2, 40, 8])
    xa, la = O.shard_forward_full(SMALL, w, 0, 3, ids=ids, dtype=dtype)
    sh = O.IncrementalShard(SMALL, w, 0, 3, dtype)
    xs = []
    for t in ids.tolist():
        x, lb = sh.step(token=t)
        xs.append(x)
    xb = torch.stack(xs)
    scale = float(xa.abs().max())
    assert float((xa - xb).abs().max()) / scale < tol
    assert float((la - lb).abs().max()) / float(la.abs().max()) < tol


def test_decode_step_equals_prefill_of_extended_sequence():
    w = _rand_weights(SMALL, 3)
    ids = torch.tensor([5, 6, 7, 8])
    toks, logits, hidden = O.generate_greedy(SMALL, w, ids, 3, torch.float64)
    ext = torch.cat([ids, toks[:3]])
    xa, la = O.shard_forward_full(SMALL, w, 0, 3, ids=ext, dtype=torch.float64)
    assert torch.allclose(hidden, xa, atol=1e-10)
    assert torch.allclose(logits[-1], la, atol=1e-10)
    # and every earlier logit row is the full-form head at that prefix
    for s in range(3):
        _, l = O.shard_forward_full(SMALL, w, 0, 3, ids=ext[:4 + s], dtype=torch.float64)
        assert torch.allclose(logits[s], l, atol=1e-10)
        assert int(toks[s]) == int(torch.argmax(l))


@pytest.mark.parametrize("k", [0, 1, 2, 3])
def test_split_invariance_bitwise(k):
    L = 3
    w = _rand_weights(SMALL, L)
    ids = torch.tensor([1, 2, 3, 4, 5, 6])
    full, lf = O.shard_forward_full(SMALL, w, 0, L, ids=ids)
    if k == 0:
        x = O.embed(ids, w["tok_embedding"])
        a = x
    else:
        wa = dict(w); wa["layers"] = w["layers"][:k]
        a, _ = O.shard_forward_full(SMALL, wa, 0, k, ids=ids)
    wb = dict(w); wb["layers"] = w["layers"][k:]
    b, lb = O.shard_forward_full(SMALL, wb, k, L, hidden_in=a)
    assert torch.equal(b, full) and torch.equal(lb, lf)


def test_batch_rows_are_independent():
    w = _rand_weights(SMALL, 2)
    wl = dict(w); wl["layers"] = w["layers"][:2]
    ids = torch.tensor([[1, 2, 3, 4], [9, 8, 7, 6]])
    sm = ModelShape("s2", 2, 32, 4, 2, 8, 48, 50)
    outs = [O.shard_forward_full(sm, wl, 0, 2, ids=ids[b])[0] for b in range(2)]
    swapped = [O.shard_forward_full(sm, wl, 0, 2, ids=ids[b])[0] for b in (1, 0)]
    assert torch.equal(outs[0], swapped[1]) and torch.equal(outs[1], swapped[0])
    assert not torch.equal(outs[0], outs[1])


def test_causality_future_tokens_do_not_matter():
    w = _rand_weights(SMALL, 3)
    a, _ = O.shard_forward_full(SMALL, w, 0, 3, ids=torch.tensor([4, 5, 6, 7, 8]))
    b, _ = O.shard_forward_full(SMALL, w, 0, 3, ids=torch.tensor([4, 5, 6, 30, 31]))
    assert torch.equal(a[:3], b[:3]) and not torch.equal(a[3], b[3])


def test_greedy_lowest_index_on_tie():
    l = torch.tensor([[0.0, 2.0, 1.0, 2.0], [5.0, 5.0, 5.0, 5.0], [-1.0, -3.0, -1.0, -2.0]])
    assert O.greedy(l).tolist() == [1, 0, 0]


# ---- output layer ------------------------------------------------------------------------

def test_lm_head_constant_vector_closed_form():
    # x = c*1: mean of squares is c^2, so logit v = c / sqrt(c^2 + eps) * sum_j g_j W[v, j]
    c, eps, d = 1.5, 1e-5, 6
    g = [0.5, 1.0, 1.5, 2.0, 0.25, 3.0]
    W = [[1, 0, 0, 0, 0, 0], [0, 2, 0, 0, 0, -1], [1, 1, 1, 1, 1, 1], [0.5, -0.5, 0.25, -0.25, 2.0, 0.0]]
    x = torch.full((1, d), c, dtype=torch.float64)
    got = O.lm_head(x, torch.tensor(g, dtype=torch.float64), torch.tensor(W, dtype=torch.float64), eps, torch.float64)
    assert got.shape == (1, 4)
    for v in range(4):
        want = c / math.sqrt(c * c + eps) * sum(g[j] * W[v][j] for j in range(d))
        assert abs(float(got[0, v]) - want) < 1e-12


def test_lm_head_hand_computed_two_by_three():
    # d = 3, V = 2, non-constant x, two rows; every number below is written out by hand with scalar arithmetic
    eps = 0.25
    xs = [[1.0, -2.0, 3.0], [0.5, 0.0, -1.5]]
    g = [2.0, 0.5, -1.0]
    W = [[1.0, 2.0, 3.0], [-1.0, 0.5, 4.0]]
    got = O.lm_head(torch.tensor(xs, dtype=torch.float64), torch.tensor(g, dtype=torch.float64),
                    torch.tensor(W, dtype=torch.float64), eps, torch.float64)
    assert got.shape == (2, 2)
    for b, x in enumerate(xs):
        r = math.sqrt((x[0] * x[0] + x[1] * x[1] + x[2] * x[2]) / 3.0 + eps)
        n = [x[0] / r * g[0], x[1] / r * g[1], x[2] / r * g[2]]
        for v in range(2):
            want = n[0] * W[v][0] + n[1] * W[v][1] + n[2] * W[v][2]
            assert abs(float(got[b, v]) - want) < 1e-12
    # row 0 spelled out once more as plain numbers: mean of squares 14/3, r = sqrt(14/3 + 1/4)
    r0 = math.sqrt(14.0 / 3.0 + 0.25)
    assert abs(float(got[0, 0]) - (2.0 - 2.0 - 9.0) / r0) < 1e-12
    assert abs(float(got[0, 1]) - (-2.0 - 0.5 - 12.0) / r0) < 1e-12


def test_lm_head_square_matrix_is_used_row_by_row():
    # V == d: logit v is the product with ROW v of the matrix (a transposed operand changes the result)
    eps, d = 1e-5, 4
    W = torch.tensor([[1.0, 2.0, 3.0, 4.0], [0.0, 1.0, 0.0, 0.0], [5.0, 0.0, 0.0, 0.0], [0.0, 0.0, 0.0, 7.0]], dtype=torch.float64)
    x = torch.tensor([[1.0, 1.0, -1.0, 2.0]], dtype=torch.float64)
    r = math.sqrt((1.0 + 1.0 + 1.0 + 4.0) / 4.0 + eps)
    got = O.lm_head(x, torch.ones(d, dtype=torch.float64), W, eps, torch.float64)[0]
    want = [(1.0 + 2.0 - 3.0 + 8.0) / r, 1.0 / r, 5.0 / r, 14.0 / r]
    for v in range(4):
        assert abs(float(got[v]) - want[v]) < 1e-12


def test_shard_logits_are_the_output_layer_of_the_last_position():
    # Wo = Wd = 0 makes every decoder layer the identity, so the logits of both forms must be the output
    # layer (final-norm gains, not a decoder layer's) applied to the LAST prompt token's embedding row
    w = _rand_weights(SMALL, 3)
    for lw in w["layers"]:
        lw["wo"].zero_(); lw["w_down"].zero_()
    ids = torch.tensor([3, 1, 4, 1, 5])
    d, V, eps = SMALL.d_model, SMALL.vocab, SMALL.rms_eps
    e = w["tok_embedding"][5].double().tolist()
    g = w["final_norm"].double().tolist()
    Wl = w["lm_head"].double().tolist()
    r = math.sqrt(sum(t * t for t in e) / d + eps)
    want = torch.tensor([sum(e[j] / r * g[j] * Wl[v][j] for j in range(d)) for v in range(V)], dtype=torch.float64)
    _, la = O.shard_forward_full(SMALL, w, 0, 3, ids=ids, dtype=torch.float64)
    assert la.shape == (V,) and torch.allclose(la, want, atol=1e-12)
    sh = O.IncrementalShard(SMALL, w, 0, 3, torch.float64)
    for t in ids.tolist():
        _, lb = sh.step(token=t)
    assert torch.allclose(lb, want, atol=1e-12)
    # a shard that does not end at the last layer has no output layer
    wa = dict(w); wa["layers"] = w["layers"][:2]
    assert O.shard_forward_full(SMALL, wa, 0, 2, ids=ids)[1] is None


# ---- shapes: the paper's memory table ------------------------------------------------------

def test_parameter_counts_match_paper_memory_table():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_memory_table.txt")
    table = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            name, gb = line.split()
            table[name] = float(gb)
    assert LLAMA2_7B.total_params() == 6_738_415_616
    assert LLAMA2_13B.total_params() == 13_015_864_320
    for m in (LLAMA2_7B, LLAMA2_13B, LLAMA2_70B):
        gb = 4.0 * m.total_params() / 1e9
        assert abs(gb - table[m.name]) / table[m.name] < 0.05, (m.name, gb)
    # the oracle's weight dict has exactly that many elements (tiny model, all tensors)
    w = shard_weights(0, TINY, 0, TINY.n_layers)
    n = sum(t.numel() for lw in w["layers"] for t in lw.values())
    n += w["tok_embedding"].numel() + w["final_norm"].numel() + w["lm_head"].numel()
    assert n == TINY.total_params()


def test_tiny_config_runs_and_margin_rule():
    w = shard_weights(0, TINY, 0, 2)
    ids = prompt_ids(0, 1, 16, TINY.vocab)[0]
    toks, logits, hidden = O.generate_greedy(TINY, w, ids, 8)
    assert toks.shape == (9,) and logits.shape == (9, 1000) and hidden.shape == (24, 256)
    assert torch.isfinite(logits).all()

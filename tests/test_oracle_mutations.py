"""Plants plausible mistakes in the oracle (on the CPU, one at a time) and checks that the pins notice:
a dropped term, a wrong sign or index, a transposed operand must each fail at least one pin."""
import math

import pytest
import torch

from oracle import decoder as O
from tests import test_oracle_pins as pins


def _all_pins():
    """A subset of the pin tests that needs no fixtures, run as plain functions."""
    names = ["test_softmax_rows_sum_to_one_via_ones_values", "test_zero_queries_give_running_mean_of_values",
             "test_first_position_returns_its_own_value", "test_gqa_equals_mha_with_repeated_kv",
             "test_rope_identity_at_position_zero", "test_rope_hand_computed_rotation",
             "test_rope_preserves_norm_and_is_relative", "test_rope_frequency_of_last_pair",
             "test_rmsnorm_constant_vector_closed_form", "test_rmsnorm_unit_rms_scale_invariance_and_gain",
             "test_rmsnorm_eps_inside_sqrt", "test_silu_special_values", "test_zero_output_projections_make_layers_identity",
             "test_layer_against_handwritten_single_token", "test_decode_step_equals_prefill_of_extended_sequence",
             "test_causality_future_tokens_do_not_matter", "test_greedy_lowest_index_on_tie",
             "test_lm_head_constant_vector_closed_form", "test_lm_head_hand_computed_two_by_three",
             "test_lm_head_square_matrix_is_used_row_by_row", "test_shard_logits_are_the_output_layer_of_the_last_position"]
    fns = [getattr(pins, n) for n in names]
    fns += [lambda hq=hq, hkv=hkv: pins.test_attention_matches_bruteforce(hq, hkv) for hq, hkv in ((4, 4), (4, 2), (4, 1))]
    fns += [pins.test_attention_with_query_offset_matches_bruteforce]
    fns += [lambda: pins.test_incremental_equals_full(torch.float64, 1e-11)]
    return fns


def _pins_fail() -> bool:
    for fn in _all_pins():
        try:
            fn()
        except AssertionError:
            return True
        except Exception:
            return True
    return False


def test_unmutated_oracle_passes():
    assert not _pins_fail()


def _rms_eps_outside(x, gain, eps):
    return x / (torch.sqrt((x * x).mean(dim=-1, keepdim=True)) + eps) * gain.to(x.dtype)


def _rms_no_gain(x, gain, eps):
    return x / torch.sqrt((x * x).mean(dim=-1, keepdim=True) + eps)


def _rms_sum_not_mean(x, gain, eps):
    return x / torch.sqrt((x * x).sum(dim=-1, keepdim=True) + eps) * gain.to(x.dtype)


def _rope_wrong_sign(x, positions, theta):
    T, H, hd = x.shape
    cos, sin = O.rope_cos_sin(positions, hd, theta)
    cos, sin = cos.to(x.dtype)[:, None, :], sin.to(x.dtype)[:, None, :]
    out = torch.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * cos + x[..., 1::2] * sin
    out[..., 1::2] = -x[..., 0::2] * sin + x[..., 1::2] * cos
    return out


def _rope_split_half(x, positions, theta):
    T, H, hd = x.shape
    cos, sin = O.rope_cos_sin(positions, hd, theta)
    cos, sin = cos.to(x.dtype)[:, None, :], sin.to(x.dtype)[:, None, :]
    a, b = x[..., : hd // 2], x[..., hd // 2:]
    return torch.cat([a * cos - b * sin, a * sin + b * cos], dim=-1)


def _rope_wrong_frequency(positions, head_dim, theta):
    i = torch.arange(head_dim // 2, dtype=torch.float64)
    inv = torch.pow(torch.tensor(float(theta), dtype=torch.float64), -i / head_dim)       # exponent halved
    ang = positions.to(torch.float64)[:, None] * inv[None, :]
    return torch.cos(ang), torch.sin(ang)


def _attn_variant(scale_pow=0.5, mask="causal", head_map="div"):
    def f(q, k, v, q_pos0=0):
        Tq, Hq, hd = q.shape
        Tk, Hkv, _ = k.shape
        group = Hq // Hkv
        out = torch.empty_like(q)
        qi = torch.arange(Tq)[:, None] + q_pos0
        kj = torch.arange(Tk)[None, :]
        visible = {"causal": kj <= qi, "strict": kj < qi, "none": kj >= 0}[mask]
        visible = visible | (kj == 0)
        for h in range(Hq):
            g = h // group if head_map == "div" else h % Hkv
            s = (q[:, h, :] @ k[:, g, :].T) / (hd ** scale_pow)
            s = s.masked_fill(~visible, float("-inf"))
            p = torch.softmax(s, dim=-1)
            out[:, h, :] = p @ v[:, g, :]
        return out
    return f


def _silu_wrong(z):
    return z / (1.0 + torch.exp(z))


def _greedy_last(logits):
    m = logits.max(dim=-1, keepdim=True).values
    idx = torch.arange(logits.shape[-1]).expand_as(logits)
    return torch.where(logits == m, idx, torch.full_like(idx, -1)).max(dim=-1).values


def _lm_head_no_norm(x_last, final_norm, w_lm, eps, dtype=torch.float32):
    return x_last.to(dtype) @ w_lm.to(dtype).T


def _lm_head_gain_before_division(x_last, final_norm, w_lm, eps, dtype=torch.float32):
    y = x_last * final_norm.to(dtype)
    return (y / torch.sqrt((y * y).mean(dim=-1, keepdim=True) + eps)) @ w_lm.to(dtype).T


def _lm_head_untransposed(x_last, final_norm, w_lm, eps, dtype=torch.float32):
    w = w_lm.to(dtype)
    return O.rmsnorm(x_last, final_norm.to(dtype), eps) @ (w if w.shape[0] == w.shape[1] else w.T)


def _lm_head_no_gain(x_last, final_norm, w_lm, eps, dtype=torch.float32):
    return O.rmsnorm(x_last, torch.ones_like(final_norm, dtype=dtype), eps) @ w_lm.to(dtype).T


MUTANTS = [
    ("lm_head", _lm_head_no_norm), ("lm_head", _lm_head_gain_before_division), ("lm_head", _lm_head_untransposed),
    ("lm_head", _lm_head_no_gain),
    ("rmsnorm", _rms_eps_outside), ("rmsnorm", _rms_no_gain), ("rmsnorm", _rms_sum_not_mean),
    ("apply_rope", _rope_wrong_sign), ("apply_rope", _rope_split_half), ("rope_cos_sin", _rope_wrong_frequency),
    ("causal_attention_matrix", _attn_variant(scale_pow=1.0)), ("causal_attention_matrix", _attn_variant(scale_pow=0.0)),
    ("causal_attention_matrix", _attn_variant(mask="strict")), ("causal_attention_matrix", _attn_variant(mask="none")),
    ("causal_attention_matrix", _attn_variant(head_map="mod")),
    ("silu", _silu_wrong), ("greedy", _greedy_last),
]


@pytest.mark.parametrize("name,mutant", MUTANTS, ids=[f"{n}-{i}" for i, (n, _) in enumerate(MUTANTS)])
def test_each_planted_mistake_is_caught(monkeypatch, name, mutant):
    monkeypatch.setattr(O, name, mutant)
    assert _pins_fail(), f"no pin noticed the planted mistake in {name}"


def _layer_mutant(kind):
    orig = O.layer_forward_full

    def f(x, w, model, pos0=0, dtype=torch.float32, return_kv=False):
        w = dict(w)
        if kind == "swap_gate_up":
            w["w_gate"], w["w_up"] = w["w_up"], w["w_gate"]
        elif kind == "no_residual":
            y = orig(x, w, model, pos0, dtype)
            return y - x
        elif kind == "shared_norm":
            w["ffn_norm"] = w["attn_norm"]
        return orig(x, w, model, pos0, dtype, return_kv)
    return f


@pytest.mark.parametrize("kind", ["swap_gate_up", "no_residual", "shared_norm"])
def test_layer_level_mistakes_are_caught(monkeypatch, kind):
    monkeypatch.setattr(O, "layer_forward_full", _layer_mutant(kind))
    assert _pins_fail(), kind


def _wrong_gain_vector(form):
    """The output layer normalised with the last decoder layer's attention-norm gains instead of its own."""
    if form == "A":
        orig = O.shard_forward_full

        def f(model, weights, layer_begin, layer_end, **kw):
            w = dict(weights)
            if "final_norm" in w:
                w["final_norm"] = w["layers"][-1]["attn_norm"]
            return orig(model, w, layer_begin, layer_end, **kw)
        return "shard_forward_full", f
    orig_cls = O.IncrementalShard

    class Wrong(orig_cls):
        def __init__(self, model, weights, layer_begin, layer_end, dtype=torch.float32):
            w = dict(weights)
            if "final_norm" in w:
                w["final_norm"] = w["layers"][-1]["attn_norm"]
            super().__init__(model, w, layer_begin, layer_end, dtype)
    return "IncrementalShard", Wrong


@pytest.mark.parametrize("form", ["A", "B"])
def test_output_layer_with_the_wrong_gain_vector_is_caught(monkeypatch, form):
    name, mutant = _wrong_gain_vector(form)
    monkeypatch.setattr(O, name, mutant)
    assert _pins_fail(), form


def test_last_position_rule_of_the_logits_is_pinned(monkeypatch):
    """Logits taken from the first position instead of the last must fail a pin."""
    orig = O.lm_head
    orig_full = O.shard_forward_full

    def f(model, weights, layer_begin, layer_end, **kw):
        x, logits = orig_full(model, weights, layer_begin, layer_end, **kw)
        if logits is not None:
            logits = orig(x[:1, :], weights["final_norm"], weights["lm_head"], model.rms_eps, kw.get("dtype", torch.float32))[0]
        return x, logits
    monkeypatch.setattr(O, "shard_forward_full", f)
    assert _pins_fail()

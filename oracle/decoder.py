"""CPU oracle for the shard forward pass.  TEST INFRASTRUCTURE ONLY.

This file is the checker, not the product: only tests, the smoke entry and the benchmark's
CPU-baseline leg may import it, and it shares no code with the CUDA library.

What it computes.  EdgeShard (Sec. "System Model") treats the LLM as an embedding layer, a
stack of decoder layers and an output layer, cut into contiguous shards; a shard takes token
ids (if it holds the embedding) or the previous shard's activation, and emits the activation
of its last layer (or logits and the next token if it holds the output layer).  Inference is
a prefill over the whole prompt followed by one-token-at-a-time generation with a KV cache
(Sec. "Generative LLM Inference").  The paper does not spell out the decoder's equations; it
names Llama-2 (Sec. "Experimental Setup"), so the functions below are the public Llama-2
decoder written out plainly:

    h   = x * g / sqrt(mean(x^2) + eps)                              (RMSNorm)
    q,k,v = h Wq^T, h Wk^T, h Wv^T, split into heads of head_dim
    RoPE on q and k: pair (2i, 2i+1) rotated by angle pos * theta^(-2i/head_dim)
    o_i = sum_j softmax_j(q_i.k_j / sqrt(head_dim), j <= i) v_j      (causal; GQA: kv head = h // group)
    x  += o Wo^T
    x  += (silu(h2 Wg^T) * (h2 Wu^T)) Wd^T,  h2 = RMSNorm(x)
    logits = RMSNorm(x_last) Wlm^T, greedy token = lowest index of the maximum

Two independently written forms exist on purpose:

* form A (`shard_forward_full`): whole sequence at once, an explicit T x T masked score matrix;
* form B (`IncrementalShard`): one position at a time against a growing K/V list.

They must agree ("a decode step equals prefill of the extended sequence").  Arithmetic is fp32
by default (the paper runs full precision); pass dtype=torch.float64 to check that fp32
rounding is immaterial.  Weights arrive as fp16 tensors and are widened exactly.

Pins (tests/test_oracle_pins.py): brute-force scalar-loop attention on tiny inputs, softmax
rows sum to 1, RoPE identity at position 0 / norm preservation / relative-position property /
hand-computed rotation, RMSNorm closed form on constant vectors, silu special values, zeroed
Wo/Wd make a layer the identity, zero Wq gives running means of v, GQA == MHA with repeated kv
weights, form A == form B, split invariance at every cut, batch-row independence, the output
layer against closed forms and hand-computed numbers (constant vector, a 2 x 3 case, a square
matrix, identity layers so the logits are the output layer of the last token's embedding), the
parameter counts behind the paper's memory table, and greedy tie-breaking on a hand-made tie.
Absolute logits of random-weight models have no printed reference value in the paper: for
those the parity is unpinned beyond the invariants above.
"""
from __future__ import annotations

import math

import torch


def _w(t: torch.Tensor, dtype) -> torch.Tensor:
    return t.to(dtype)


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    """x: [..., d]; eps is added to the mean of squares, inside the square root."""
    ms = (x * x).mean(dim=-1, keepdim=True)
    return x / torch.sqrt(ms + eps) * gain.to(x.dtype)


def rope_cos_sin(positions: torch.Tensor, head_dim: int, theta: float):
    """cos/sin of pos * theta^(-2i/head_dim), i in [0, head_dim/2); computed in fp64."""
    i = torch.arange(head_dim // 2, dtype=torch.float64)
    inv_freq = torch.pow(torch.tensor(float(theta), dtype=torch.float64), -2.0 * i / head_dim)
    ang = positions.to(torch.float64)[:, None] * inv_freq[None, :]
    return torch.cos(ang), torch.sin(ang)


def apply_rope(x: torch.Tensor, positions: torch.Tensor, theta: float) -> torch.Tensor:
    """x: [T, H, head_dim]; rotates adjacent pairs (2i, 2i+1) of every head."""
    T, H, hd = x.shape
    cos, sin = rope_cos_sin(positions, hd, theta)
    cos = cos.to(x.dtype)[:, None, :]
    sin = sin.to(x.dtype)[:, None, :]
    a = x[..., 0::2]
    b = x[..., 1::2]
    out = torch.empty_like(x)
    out[..., 0::2] = a * cos - b * sin
    out[..., 1::2] = a * sin + b * cos
    return out


def silu(z: torch.Tensor) -> torch.Tensor:
    return z / (1.0 + torch.exp(-z))


def causal_attention_matrix(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                            q_pos0: int = 0) -> torch.Tensor:
    """Form A attention.  q: [Tq, Hq, hd]; k, v: [Tk, Hkv, hd]; query i sits at absolute position
    q_pos0 + i and sees keys 0..q_pos0+i.  Returns [Tq, Hq, hd]."""
    Tq, Hq, hd = q.shape
    Tk, Hkv, _ = k.shape
    group = Hq // Hkv
    out = torch.empty_like(q)
    qi = torch.arange(Tq)[:, None] + q_pos0
    kj = torch.arange(Tk)[None, :]
    visible = kj <= qi                                    # [Tq, Tk]
    for h in range(Hq):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) / math.sqrt(hd)   # [Tq, Tk]
        s = s.masked_fill(~visible, float("-inf"))
        s = s - s.max(dim=-1, keepdim=True).values
        p = torch.exp(s)
        p = p / p.sum(dim=-1, keepdim=True)
        out[:, h, :] = p @ v[:, g, :]
    return out


def layer_forward_full(x: torch.Tensor, w: dict, model, pos0: int = 0, dtype=torch.float32,
                       return_kv: bool = False):
    """One decoder layer over a whole sequence x: [T, d] (form A)."""
    T, d = x.shape
    Hq, Hkv, hd = model.n_heads, model.n_kv_heads, model.head_dim
    pos = torch.arange(pos0, pos0 + T)
    h = rmsnorm(x, _w(w["attn_norm"], dtype), model.rms_eps)
    q = (h @ _w(w["wq"], dtype).T).reshape(T, Hq, hd)
    k = (h @ _w(w["wk"], dtype).T).reshape(T, Hkv, hd)
    v = (h @ _w(w["wv"], dtype).T).reshape(T, Hkv, hd)
    q = apply_rope(q, pos, model.rope_theta)
    k = apply_rope(k, pos, model.rope_theta)
    o = causal_attention_matrix(q, k, v, 0).reshape(T, Hq * hd)
    x = x + o @ _w(w["wo"], dtype).T
    h2 = rmsnorm(x, _w(w["ffn_norm"], dtype), model.rms_eps)
    a = silu(h2 @ _w(w["w_gate"], dtype).T) * (h2 @ _w(w["w_up"], dtype).T)
    x = x + a @ _w(w["w_down"], dtype).T
    if return_kv:
        return x, k, v
    return x


def embed(ids: torch.Tensor, table: torch.Tensor, dtype=torch.float32) -> torch.Tensor:
    return table[ids.long()].to(dtype)


def lm_head(x_last: torch.Tensor, final_norm: torch.Tensor, w_lm: torch.Tensor, eps: float,
            dtype=torch.float32) -> torch.Tensor:
    """x_last: [B, d] -> logits [B, V]."""
    return rmsnorm(x_last, _w(final_norm, dtype), eps) @ _w(w_lm, dtype).T


def greedy(logits: torch.Tensor) -> torch.Tensor:
    """Index of the maximum; the lowest index wins a tie.  logits: [B, V] -> int64 [B]."""
    m = logits.max(dim=-1, keepdim=True).values
    V = logits.shape[-1]
    idx = torch.arange(V).expand_as(logits)
    return torch.where(logits == m, idx, torch.full_like(idx, V)).min(dim=-1).values


def shard_forward_full(model, weights: dict, layer_begin: int, layer_end: int, *,
                       ids: torch.Tensor | None = None, hidden_in: torch.Tensor | None = None,
                       dtype=torch.float32):
    """Form A over one sequence.  ids: [T] (shard holds the embedding) or hidden_in: [T, d].

    Returns (hidden [T, d], logits_last [V] or None).  `weights["layers"][i]` is decoder layer
    layer_begin + i.
    """
    if (ids is None) == (hidden_in is None):
        raise ValueError("exactly one of ids / hidden_in")
    if ids is not None:
        if layer_begin != 0:
            raise ValueError("ids only for the shard that holds the embedding")
        x = embed(ids, weights["tok_embedding"], dtype)
    else:
        x = hidden_in.to(dtype)
    for li in range(layer_end - layer_begin):
        x = layer_forward_full(x, weights["layers"][li], model, 0, dtype)
    logits = None
    if layer_end == model.n_layers:
        logits = lm_head(x[-1:, :], weights["final_norm"], weights["lm_head"], model.rms_eps, dtype)[0]
    return x, logits


class IncrementalShard:
    """Form B: KV-cached, one position at a time, for one sequence."""

    def __init__(self, model, weights: dict, layer_begin: int, layer_end: int, dtype=torch.float32):
        self.model, self.weights = model, weights
        self.begin, self.end, self.dtype = layer_begin, layer_end, dtype
        n = layer_end - layer_begin
        self.k_cache = [[] for _ in range(n)]      # per layer: list over positions of [Hkv, hd]
        self.v_cache = [[] for _ in range(n)]
        self.pos = 0

    def _attend(self, q: torch.Tensor, keys, values) -> torch.Tensor:
        """q: [Hq, hd]; keys/values: lists of [Hkv, hd] for positions 0..pos."""
        m = self.model
        group = m.n_heads // m.n_kv_heads
        K = torch.stack(keys)                      # [ctx, Hkv, hd]
        V = torch.stack(values)
        out = torch.empty_like(q)
        for h in range(m.n_heads):
            g = h // group
            s = (K[:, g, :] @ q[h]) / math.sqrt(m.head_dim)     # [ctx]
            p = torch.exp(s - s.max())
            p = p / p.sum()
            out[h] = p @ V[:, g, :]
        return out

    def step(self, *, token: int | None = None, hidden_in: torch.Tensor | None = None):
        """Advance one position.  Returns (hidden [d], logits [V] or None)."""
        m, dt = self.model, self.dtype
        if token is not None:
            x = self.weights["tok_embedding"][int(token)].to(dt)
        else:
            x = hidden_in.to(dt)
        pos = torch.tensor([self.pos])
        for li in range(self.end - self.begin):
            w = self.weights["layers"][li]
            h = rmsnorm(x, _w(w["attn_norm"], dt), m.rms_eps)
            q = (_w(w["wq"], dt) @ h).reshape(1, m.n_heads, m.head_dim)
            k = (_w(w["wk"], dt) @ h).reshape(1, m.n_kv_heads, m.head_dim)
            v = (_w(w["wv"], dt) @ h).reshape(m.n_kv_heads, m.head_dim)
            q = apply_rope(q, pos, m.rope_theta)[0]
            k = apply_rope(k, pos, m.rope_theta)[0]
            self.k_cache[li].append(k)
            self.v_cache[li].append(v)
            o = self._attend(q, self.k_cache[li], self.v_cache[li]).reshape(-1)
            x = x + _w(w["wo"], dt) @ o
            h2 = rmsnorm(x, _w(w["ffn_norm"], dt), m.rms_eps)
            a = silu(_w(w["w_gate"], dt) @ h2) * (_w(w["w_up"], dt) @ h2)
            x = x + _w(w["w_down"], dt) @ a
        self.pos += 1
        logits = None
        if self.end == m.n_layers:
            logits = lm_head(x[None, :], self.weights["final_norm"], self.weights["lm_head"],
                             m.rms_eps, dt)[0]
        return x, logits


def generate_greedy(model, weights: dict, prompt: torch.Tensor, steps: int, dtype=torch.float32):
    """Prefill + greedy decoding of one sequence with the full model (form B).

    Returns (tokens [steps+1] — the token produced by the prefill and by each decode step,
    logits [steps+1, V], hidden [T+steps, d]).
    """
    sh = IncrementalShard(model, weights, 0, model.n_layers, dtype)
    hidden, all_logits, toks = [], [], []
    logits = None
    for t in prompt.tolist():
        x, logits = sh.step(token=t)
        hidden.append(x)
    all_logits.append(logits)
    toks.append(int(greedy(logits[None, :])[0]))
    for _ in range(steps):
        x, logits = sh.step(token=toks[-1])
        hidden.append(x)
        all_logits.append(logits)
        toks.append(int(greedy(logits[None, :])[0]))
    return torch.tensor(toks), torch.stack(all_logits), torch.stack(hidden)

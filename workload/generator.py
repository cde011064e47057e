"""Seeded synthetic inputs: model shapes, random-init fp16 weights and token ids.

This module serves both the CPU oracle and the CUDA path and contains none of the
decoder's arithmetic.  Every value is a pure function of (seed, tensor id, element index),
so any row range of any tensor can be regenerated on its own, on the CPU or on a CUDA
device, with bit-identical results:

* a 64-bit counter hash (the splitmix64 finaliser) done in wrapping int64 arithmetic,
* a piecewise-linear inverse normal CDF over a 65537-entry fp32 quantile table that is
  computed once on the host (so CPU and GPU interpolate the same table),
* only individually rounded fp32 operations (one multiply, one add at a time) before the
  final round-to-nearest-even conversion to fp16.

The workloads stand in for the paper's text-generation runs on trained Llama-2 weights
(Sec. "Experimental Setup"): random-init weights of the same shapes and uniform random
token ids; with random weights the text content cannot influence timing.
"""
from __future__ import annotations

import dataclasses
import functools

import numpy as np
import torch

_M64 = (1 << 64) - 1
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB
_GOLDEN = 0x9E3779B97F4A7C15
_CHUNK = 1 << 22


def _signed(c: int) -> int:
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def _mix_int(x: int) -> int:
    x &= _M64
    x ^= x >> 30
    x = (x * _C1) & _M64
    x ^= x >> 27
    x = (x * _C2) & _M64
    x ^= x >> 31
    return x


def _srl(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix_t(x: torch.Tensor) -> torch.Tensor:
    x = x ^ _srl(x, 30)
    x = x * _signed(_C1)
    x = x ^ _srl(x, 27)
    x = x * _signed(_C2)
    x = x ^ _srl(x, 31)
    return x


def stream_key(seed: int, tensor_id: int) -> int:
    """Key of one tensor's random stream."""
    return _mix_int(_mix_int(seed & _M64) ^ ((tensor_id * _GOLDEN) & _M64))


def _hash_range(key: int, start: int, n: int, device) -> torch.Tensor:
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    return _mix_t(idx * _signed(_GOLDEN) + _signed(key))


@functools.lru_cache(maxsize=1)
def _quantile_table_host() -> torch.Tensor:
    from scipy.special import ndtri

    n = 65536
    p = np.arange(n + 1, dtype=np.float64) / n
    p[0] = 2.0 ** -18
    p[n] = 1.0 - 2.0 ** -18
    return torch.from_numpy(ndtri(p).astype(np.float32))


@functools.lru_cache(maxsize=8)
def _quantile_table(device_str: str) -> torch.Tensor:
    return _quantile_table_host().to(device_str)


def standard_normal_f32(seed: int, tensor_id: int, start: int, n: int, device="cpu") -> torch.Tensor:
    """n draws (element indices start..start+n) of an (almost exactly) N(0,1) variate, fp32."""
    device = torch.device(device)
    table = _quantile_table(str(device))
    key = stream_key(seed, tensor_id)
    out = torch.empty(n, dtype=torch.float32, device=device)
    chunk = _CHUNK * 8 if device.type == "cuda" else _CHUNK      # fewer, larger launches on a GPU
    for o in range(0, n, chunk):
        m = min(chunk, n - o)
        h = _hash_range(key, start + o, m, device)
        i = _srl(h, 48)
        f = (_srl(h, 24) & 0xFFFFFF).to(torch.float32) * (2.0 ** -24)
        t0 = table[i]
        d = table[i + 1] - t0
        out[o:o + m] = t0 + f * d          # two separately rounded fp32 ops
    return out


def normal_fp16(seed: int, tensor_id: int, shape, std: float = 0.02, mean: float = 0.0,
                device="cpu", row_begin: int = 0) -> torch.Tensor:
    """fp16 tensor of the given shape, elements mean + std * N(0,1).

    `row_begin` offsets the element index by row_begin * prod(shape[1:]), so that
    normal_fp16(.., (r, c), row_begin=k) equals rows k..k+r of the full tensor.
    """
    shape = tuple(int(s) for s in shape)
    n = int(np.prod(shape)) if shape else 1
    inner = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    z = standard_normal_f32(seed, tensor_id, row_begin * inner, n, device)
    z = z * float(np.float32(std))
    if mean != 0.0:
        z = z + float(np.float32(mean))
    return z.to(torch.float16).reshape(shape)


def token_ids(seed: int, stream_id: int, shape, vocab: int, device="cpu") -> torch.Tensor:
    """int32 ids, uniform on [0, vocab)."""
    shape = tuple(int(s) for s in shape)
    n = int(np.prod(shape))
    key = stream_key(seed, (1 << 40) + stream_id)
    h = _hash_range(key, 0, n, torch.device(device))
    return ((_srl(h, 33) * vocab) >> 31).to(torch.int32).reshape(shape)


# ----------------------------------------------------------------------------------------
# Model shapes and workloads


@dataclasses.dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def q_dim(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def layer_params(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 2 * d + self.q_dim * d + 2 * self.kv_dim * d + d * self.q_dim + 3 * d * f

    def total_params(self) -> int:
        return self.n_layers * self.layer_params() + 2 * self.vocab * self.d_model + self.d_model


@dataclasses.dataclass(frozen=True)
class Workload:
    cfg: int
    model: ModelShape
    layer_begin: int
    layer_end: int
    batch: int
    prompt_len: int
    decode_steps: int
    n_shards: int = 1
    micro_batches: int = 1

    @property
    def has_embedding(self) -> bool:
        return self.layer_begin == 0

    @property
    def has_head(self) -> bool:
        return self.layer_end == self.model.n_layers


TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 688, 1000)
LLAMA2_7B = ModelShape("llama2-7b", 32, 4096, 32, 32, 128, 11008, 32000)
LLAMA2_13B = ModelShape("llama2-13b", 40, 5120, 40, 40, 128, 13824, 32000)
LLAMA2_70B = ModelShape("llama2-70b", 80, 8192, 64, 8, 128, 28672, 32000)

WORKLOADS = {
    "cfg0": Workload(0, TINY, 0, 2, 1, 16, 8),
    "cfg1": Workload(1, LLAMA2_7B, 0, 8, 1, 128, 128),
    "cfg2_b1": Workload(2, LLAMA2_7B, 0, 32, 1, 512, 256),
    "cfg2_b8": Workload(2, LLAMA2_7B, 0, 32, 8, 512, 256),
    "cfg3": Workload(3, LLAMA2_13B, 0, 40, 1, 256, 128, n_shards=4, micro_batches=8),
    "cfg4": Workload(4, LLAMA2_70B, 0, 40, 16, 1024, 128),
    # the shape the paper measures on (Sec. "Experimental Setup": 32 prompt tokens, 96 generated, batch 8):
    # a context run next to the paper's own figures, not one of the parity configurations
    "paper_7b_b8": Workload(2, LLAMA2_7B, 0, 32, 8, 32, 96),
    "paper_13b_b8": Workload(3, LLAMA2_13B, 0, 40, 8, 32, 96),
}

_KINDS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")
_GLOBAL_BASE = 1 << 20
_GLOBAL = {"tok_embedding": 0, "final_norm": 1, "lm_head": 2}


def weight_seed(cfg: int) -> int:
    return 1000 * cfg + 7


def tensor_shape(model: ModelShape, kind: str):
    d, f = model.d_model, model.d_ffn
    return {
        "attn_norm": (d,), "ffn_norm": (d,), "final_norm": (d,),
        "wq": (model.q_dim, d), "wk": (model.kv_dim, d), "wv": (model.kv_dim, d),
        "wo": (d, model.q_dim), "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
        "tok_embedding": (model.vocab, d), "lm_head": (model.vocab, d),
    }[kind]


def weight_tensor(cfg: int, model: ModelShape, kind: str, layer: int = -1, device="cpu",
                  row_begin: int = 0, rows: int | None = None) -> torch.Tensor:
    """One weight tensor (or a row range of it): fp16, row-major [out, in].

    Matrices are N(0, 0.02^2); RMSNorm gains are 1 + N(0, 0.02^2) so that the gain multiply is
    exercised and attention scores stay O(1).
    """
    shape = tensor_shape(model, kind)
    if kind in _GLOBAL:
        tid = _GLOBAL_BASE + _GLOBAL[kind]
    else:
        tid = layer * 16 + _KINDS.index(kind)
    if rows is not None:
        shape = (rows,) + tuple(shape[1:])
    mean = 1.0 if kind.endswith("norm") else 0.0
    return normal_fp16(weight_seed(cfg), tid, shape, 0.02, mean, device, row_begin)


def layer_weights(cfg: int, model: ModelShape, layer: int, device="cpu") -> dict:
    return {k: weight_tensor(cfg, model, k, layer, device) for k in _KINDS}


def shard_weights(cfg: int, model: ModelShape, layer_begin: int, layer_end: int, device="cpu") -> dict:
    """All tensors a shard [layer_begin, layer_end) owns."""
    w = {"layers": [layer_weights(cfg, model, l, device) for l in range(layer_begin, layer_end)]}
    if layer_begin == 0:
        w["tok_embedding"] = weight_tensor(cfg, model, "tok_embedding", device=device)
    if layer_end == model.n_layers:
        w["final_norm"] = weight_tensor(cfg, model, "final_norm", device=device)
        w["lm_head"] = weight_tensor(cfg, model, "lm_head", device=device)
    return w


def prompt_ids(cfg: int, batch: int, prompt_len: int, vocab: int, device="cpu", seed: int | None = None):
    return token_ids(cfg if seed is None else seed, 0, (batch, prompt_len), vocab, device)


def forced_decode_ids(cfg: int, batch: int, steps: int, vocab: int, device="cpu", seed: int | None = None):
    """Decode-time input ids for shards without an LM head (teacher-forced), [steps, batch]."""
    return token_ids(cfg if seed is None else seed, 1, (steps, batch), vocab, device)

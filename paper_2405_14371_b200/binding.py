"""ctypes binding of libedgeshard.so: the same entry points as include/edgeshard.h.

Argument marshalling only — every step of the path runs inside the library's CUDA kernels.
torch supplies device memory and streams.  Importing this module loads the shared library and
raises if it is missing: there is no CPU or eager fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libedgeshard.so")

ES_OK = 0
STATUS_NAMES = {
    0: "ES_OK", 1: "ES_ERR_INVALID_ARG", 2: "ES_ERR_SHAPE", 3: "ES_ERR_RANGE", 4: "ES_ERR_STATE",
    5: "ES_ERR_KV_FULL", 6: "ES_ERR_WORKSPACE", 7: "ES_ERR_CUDA", 8: "ES_ERR_DEVICE_TIMEOUT",
    9: "ES_ERR_UNSUPPORTED",
}
ES_DTYPE_F16, ES_DTYPE_F32, ES_DTYPE_I32 = 0, 1, 2
KERNEL_CATEGORIES = ("embed", "rmsnorm", "qkv", "attention", "o", "gate_up", "down", "lm_head", "argmax", "set_ctx",
                     "splitk_finish", "splitk_reduce")
LAYER_KEYS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


class EsError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status
        self.message = message


class es_model_desc_t(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers_total", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_slots", "max_seq", "max_tokens", "max_batch", "kv_page_tokens")]


class es_layer_weights_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in LAYER_KEYS]


class es_weights_t(C.Structure):
    _fields_ = [("tok_embedding", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("layers", C.POINTER(es_layer_weights_t))]


class es_tensor_t(C.Structure):
    _fields_ = [("data", C.c_void_p), ("dtype", C.c_int32), ("rank", C.c_int32), ("shape", C.c_int64 * 4)]


class es_layer_profile_t(C.Structure):
    _fields_ = [("layer", C.c_int32), ("n_prefill", C.c_int32), ("n_decode", C.c_int32),
                ("prefill_ms_mean", C.c_float), ("decode_ms_mean", C.c_float), ("avg_ms_per_token", C.c_float),
                ("activation_bytes", C.c_int64), ("weight_bytes", C.c_int64), ("kv_bytes", C.c_int64)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2405_14371_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    P = C.POINTER
    sig = {
        "es_shard_workspace_bytes": (i32, [P(es_model_desc_t), i32, i32, P(sz), P(sz)]),
        "es_shard_create": (i32, [P(es_model_desc_t), i32, i32, P(es_weights_t), vp, sz, vp, sz, vp, P(vp)]),
        "es_shard_prefill": (i32, [vp, vp, P(es_tensor_t), i32, i32, P(i32)]),
        "es_shard_prefill_ragged": (i32, [vp, vp, P(es_tensor_t), i32, i32, P(i32), P(i32)]),
        "es_shard_prefill_packed": (i32, [vp, vp, P(es_tensor_t), i32, P(i32), P(i32)]),
        "es_shard_decode_step": (i32, [vp, vp, P(es_tensor_t), i32, P(i32)]),
        "es_shard_handoff": (i32, [vp, P(es_tensor_t), P(es_tensor_t), P(es_tensor_t)]),
        "es_layer_profile": (i32, [vp, P(es_layer_profile_t), i32, P(i32)]),
        "es_shard_set_profiling": (i32, [vp, i32]),
        "es_shard_reset_slots": (i32, [vp, P(i32), i32]),
        "es_shard_set_page_table": (i32, [vp, P(i32)]),
        "es_shard_set_graphs": (i32, [vp, i32]),
        "es_shard_device_status": (i32, [vp]),
        "es_shard_launch_count": (C.c_int64, [vp]),
        "es_shard_wait_probe": (i32, [vp, i32]),
        "es_shard_set_kernel_timing": (i32, [vp, i32]),
        "es_shard_kernel_timing": (i32, [vp, P(C.c_double), P(C.c_double), P(C.c_int64)]),
        "es_shard_kernel_timing_detail": (i32, [vp, P(C.c_double), P(C.c_double), P(C.c_int64)]),
        "es_shard_set_step_timing": (i32, [vp, i32]),
        "es_shard_step_timing": (i32, [vp, i32, P(i32), P(i32), P(C.c_double), P(C.c_double), P(C.c_double)]),
        "es_shard_destroy": (None, [vp]),
        "es_last_error": (C.c_char_p, []),
        "es_version": (C.c_char_p, []),
        "es_partition_latency": (i32, [i32, i32] + [P(C.c_double)] * 5 + [P(i32), P(C.c_double)]),
        "es_partition_throughput": (i32, [i32, i32] + [P(C.c_double)] * 5 + [P(i32), P(C.c_double)]),
        "es_op_rmsnorm": (i32, [vp, vp, vp, i32, i32, C.c_float, vp]),
        "es_op_linear": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, vp]),
        "es_op_linear_splitk_workspace_bytes": (sz, [i32, i32, i32]),
        "es_op_linear_splitk": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp]),
        "es_op_prefill_attention": (i32, [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]),
        "es_op_decode_attention_scratch_bytes": (sz, [i32, i32, i32, i32, i32]),
        "es_op_decode_attention": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, sz, vp]),
        "es_op_decode_attention_static_capacity": (sz, []),
        "es_op_decode_attention_static": (i32, [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


lib = _load()
EXPORTS = ("es_shard_workspace_bytes es_shard_create es_shard_prefill es_shard_prefill_ragged es_shard_prefill_packed es_shard_decode_step es_shard_handoff "
           "es_layer_profile es_shard_set_profiling es_shard_reset_slots es_shard_set_page_table es_shard_set_graphs "
           "es_partition_latency es_partition_throughput es_shard_device_status es_shard_wait_probe es_shard_launch_count es_shard_set_kernel_timing es_shard_kernel_timing es_shard_kernel_timing_detail es_shard_set_step_timing es_shard_step_timing es_shard_destroy es_last_error es_version es_op_rmsnorm "
           "es_op_linear es_op_linear_splitk_workspace_bytes es_op_linear_splitk es_op_prefill_attention es_op_decode_attention_scratch_bytes es_op_decode_attention "
           "es_op_decode_attention_static_capacity es_op_decode_attention_static").split()


def es_last_error() -> str:
    return lib.es_last_error().decode()


def es_version() -> str:
    return lib.es_version().decode()


def _check(status: int) -> None:
    if status != ES_OK:
        raise EsError(status, es_last_error())


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _i32_array(values: Sequence[int]):
    return (C.c_int32 * len(values))(*[int(v) for v in values])


def make_desc(model, max_slots: int, max_seq: int, max_tokens: int, max_batch: int,
              kv_page_tokens: int = 64) -> es_model_desc_t:
    """`model` needs n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, rms_eps, rope_theta."""
    return es_model_desc_t(model.n_layers, model.d_model, model.n_heads, model.n_kv_heads, model.head_dim,
                           model.d_ffn, model.vocab, model.rms_eps, model.rope_theta,
                           max_slots, max_seq, max_tokens, max_batch, kv_page_tokens)


def es_shard_workspace_bytes(desc: es_model_desc_t, layer_begin: int, layer_end: int):
    kv, sc = C.c_size_t(0), C.c_size_t(0)
    _check(lib.es_shard_workspace_bytes(C.byref(desc), layer_begin, layer_end, C.byref(kv), C.byref(sc)))
    return kv.value, sc.value


def _as_tensor_struct(t: torch.Tensor) -> es_tensor_t:
    if not t.is_cuda or not t.is_contiguous():
        raise EsError(1, "hidden_in must be a contiguous CUDA tensor")
    dt = {torch.float32: ES_DTYPE_F32, torch.float16: ES_DTYPE_F16, torch.int32: ES_DTYPE_I32}[t.dtype]
    shape = list(t.shape) + [1] * (4 - t.dim())
    return es_tensor_t(int(t.data_ptr()), dt, t.dim(), (C.c_int64 * 4)(*shape))


class Shard:
    """One shard [layer_begin, layer_end) on the current CUDA device.

    weights: {"layers": [ {attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down}, ... ],
              "tok_embedding"?, "final_norm"?, "lm_head"?} — contiguous fp16 CUDA tensors, borrowed.
    """

    def __init__(self, model, layer_begin: int, layer_end: int, weights: dict, *, max_slots: int, max_seq: int,
                 max_tokens: int, max_batch: Optional[int] = None, kv_page_tokens: int = 64, stream=None):
        self.model = model
        self.layer_begin, self.layer_end = layer_begin, layer_end
        self.desc = make_desc(model, max_slots, max_seq, max_tokens, max_batch or max_slots, kv_page_tokens)
        self._handle = C.c_void_p(None)
        kv_bytes, scratch_bytes = es_shard_workspace_bytes(self.desc, layer_begin, layer_end)
        self.kv_bytes, self.scratch_bytes = kv_bytes, scratch_bytes
        self.stream = stream if stream is not None else torch.cuda.current_stream()
        with torch.cuda.stream(self.stream):
            self.kv_buffer = torch.empty(kv_bytes, dtype=torch.uint8, device="cuda")
            self.scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device="cuda")
        self._weights = weights  # keep the tensors alive: the library borrows them
        layers = weights["layers"]
        if len(layers) != layer_end - layer_begin:
            raise EsError(1, f"expected {layer_end - layer_begin} layer weight dicts, got {len(layers)}")
        arr = (es_layer_weights_t * len(layers))()
        for i, lw in enumerate(layers):
            for k in LAYER_KEYS:
                t = lw[k]
                if not (t.is_cuda and t.dtype == torch.float16 and t.is_contiguous()):
                    raise EsError(1, f"layer {i} {k}: need a contiguous fp16 CUDA tensor")
                setattr(arr[i], k, int(t.data_ptr()))
        w = es_weights_t(_ptr(weights.get("tok_embedding")), _ptr(weights.get("final_norm")),
                         _ptr(weights.get("lm_head")), arr)
        self._layer_array = arr
        _check(lib.es_shard_create(C.byref(self.desc), layer_begin, layer_end, C.byref(w),
                                   int(self.kv_buffer.data_ptr()), kv_bytes, int(self.scratch.data_ptr()),
                                   scratch_bytes, _stream_ptr(self.stream), C.byref(self._handle)))

    # -- the five calls ---------------------------------------------------------------------
    def es_shard_prefill(self, ids: Optional[torch.Tensor], hidden_in: Optional[torch.Tensor], B: int, T: int,
                         slots: Sequence[int]) -> None:
        hin = C.byref(_as_tensor_struct(hidden_in)) if hidden_in is not None else None
        if ids is not None and not (ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()):
            raise EsError(1, "ids must be a contiguous int32 CUDA tensor")
        _check(lib.es_shard_prefill(self._handle, _ptr(ids), hin, B, T, _i32_array(slots)))

    def es_shard_prefill_ragged(self, ids: Optional[torch.Tensor], hidden_in: Optional[torch.Tensor], B: int, T: int,
                                slots: Sequence[int], lens: Sequence[int]) -> None:
        hin = C.byref(_as_tensor_struct(hidden_in)) if hidden_in is not None else None
        if ids is not None and not (ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()):
            raise EsError(1, "ids must be a contiguous int32 CUDA tensor")
        if len(lens) != B:
            raise EsError(1, "lens must have one entry per sequence")
        _check(lib.es_shard_prefill_ragged(self._handle, _ptr(ids), hin, B, T, _i32_array(slots), _i32_array(lens)))

    def es_shard_prefill_packed(self, ids: Optional[torch.Tensor], hidden_in: Optional[torch.Tensor], B: int,
                                slots: Sequence[int], lens: Sequence[int]) -> None:
        """Prompts of different lengths packed one after the other: ids [sum(lens)] or hidden_in [sum(lens), d]."""
        hin = C.byref(_as_tensor_struct(hidden_in)) if hidden_in is not None else None
        if ids is not None and not (ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()):
            raise EsError(1, "ids must be a contiguous int32 CUDA tensor")
        if len(lens) != B:
            raise EsError(1, "lens must have one entry per sequence")
        _check(lib.es_shard_prefill_packed(self._handle, _ptr(ids), hin, B, _i32_array(slots), _i32_array(lens)))

    def es_shard_decode_step(self, ids: Optional[torch.Tensor], hidden_in: Optional[torch.Tensor], B: int,
                             slots: Sequence[int]) -> None:
        hin = C.byref(_as_tensor_struct(hidden_in)) if hidden_in is not None else None
        if ids is not None and not (ids.is_cuda and ids.dtype == torch.int32 and ids.is_contiguous()):
            raise EsError(1, "ids must be a contiguous int32 CUDA tensor")
        _check(lib.es_shard_decode_step(self._handle, _ptr(ids), hin, B, _i32_array(slots)))

    def es_shard_handoff(self):
        """(hidden [B, T, d] fp32, logits [B, V] fp32 or None, next_ids [B] int32 or None): views of
        the shard's device buffers, valid until its next prefill/decode call."""
        h, l, n = es_tensor_t(), es_tensor_t(), es_tensor_t()
        _check(lib.es_shard_handoff(self._handle, C.byref(h), C.byref(l), C.byref(n)))
        return self._view(h), self._view(l), self._view(n)

    def es_layer_profile(self):
        n = C.c_int32(0)
        cap = self.layer_end - self.layer_begin + 2
        out = (es_layer_profile_t * cap)()
        _check(lib.es_layer_profile(self._handle, out, cap, C.byref(n)))
        return [{f: getattr(out[i], f) for f, _ in es_layer_profile_t._fields_} for i in range(n.value)]

    # -- auxiliaries --------------------------------------------------------------------------
    def es_shard_set_profiling(self, enabled: bool) -> None:
        _check(lib.es_shard_set_profiling(self._handle, int(enabled)))

    def es_shard_reset_slots(self, slots: Optional[Sequence[int]] = None) -> None:
        if slots is None:
            _check(lib.es_shard_reset_slots(self._handle, None, 0))
        else:
            _check(lib.es_shard_reset_slots(self._handle, _i32_array(slots), len(slots)))

    def es_shard_set_page_table(self, table: Sequence[int]) -> None:
        _check(lib.es_shard_set_page_table(self._handle, _i32_array(table)))

    def es_shard_set_graphs(self, enabled: bool) -> None:
        _check(lib.es_shard_set_graphs(self._handle, int(enabled)))

    def es_shard_device_status(self) -> None:
        _check(lib.es_shard_device_status(self._handle))

    def es_shard_wait_probe(self, limit_us: int) -> None:
        _check(lib.es_shard_wait_probe(self._handle, int(limit_us)))

    def es_shard_launch_count(self) -> int:
        return int(lib.es_shard_launch_count(self._handle))

    def es_shard_set_kernel_timing(self, enabled: bool) -> None:
        _check(lib.es_shard_set_kernel_timing(self._handle, int(enabled)))

    def es_shard_kernel_timing(self) -> dict:
        ms, by, n = C.c_double(0), C.c_double(0), C.c_int64(0)
        _check(lib.es_shard_kernel_timing(self._handle, C.byref(ms), C.byref(by), C.byref(n)))
        return {"ms": ms.value, "bytes": by.value, "launches": n.value}

    def es_shard_kernel_timing_detail(self) -> dict:
        n = len(KERNEL_CATEGORIES)
        ms, by, cnt = (C.c_double * n)(), (C.c_double * n)(), (C.c_int64 * n)()
        _check(lib.es_shard_kernel_timing_detail(self._handle, ms, by, cnt))
        return {name: {"ms": ms[i], "bytes": by[i], "launches": cnt[i]} for i, name in enumerate(KERNEL_CATEGORIES)}

    def es_shard_set_step_timing(self, enabled: bool) -> None:
        _check(lib.es_shard_set_step_timing(self._handle, int(enabled)))

    def es_shard_step_timing(self) -> list:
        """One dict per launch of the last enqueued pass, in launch order: category name, start / end in
        microseconds from the first start of the pass, algorithmic bytes."""
        cap = 2048
        n = C.c_int32(0)
        cat, t0, t1, by = (C.c_int32 * cap)(), (C.c_double * cap)(), (C.c_double * cap)(), (C.c_double * cap)()
        _check(lib.es_shard_step_timing(self._handle, cap, C.byref(n), cat, t0, t1, by))
        return [{"category": KERNEL_CATEGORIES[cat[i]], "start_us": t0[i], "end_us": t1[i], "bytes": by[i]}
                for i in range(min(n.value, cap))]

    @property
    def n_pages(self) -> int:
        p = self.desc.kv_page_tokens
        return self.desc.max_slots * ((self.desc.max_seq + p - 1) // p)

    def _view(self, t: es_tensor_t) -> Optional[torch.Tensor]:
        if not t.data:
            return None
        dtype = {ES_DTYPE_F32: torch.float32, ES_DTYPE_F16: torch.float16, ES_DTYPE_I32: torch.int32}[t.dtype]
        shape = [int(t.shape[i]) for i in range(t.rank)]
        n = 1
        for s_ in shape:
            n *= s_
        off = int(t.data) - int(self.scratch.data_ptr())
        nbytes = n * torch.empty((), dtype=dtype).element_size()
        if off < 0 or off + nbytes > self.scratch.numel():
            raise EsError(7, "handoff view lies outside the scratch buffer")
        return self.scratch[off:off + nbytes].view(dtype).view(shape)

    def close(self) -> None:
        if self._handle:
            lib.es_shard_destroy(self._handle)
            self._handle = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- single operations ---------------------------------------------------------------------

def es_op_rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float, stream=None) -> torch.Tensor:
    M, d = x.shape
    y = torch.empty(M, d, dtype=torch.float16, device=x.device)
    _check(lib.es_op_rmsnorm(_ptr(x), _ptr(gain), _ptr(y), M, d, eps, _stream_ptr(stream)))
    return y


def es_op_linear(A: torch.Tensor, W: torch.Tensor, R: Optional[torch.Tensor] = None, path: int = 0,
                 stream=None) -> torch.Tensor:
    M, K = A.shape
    N = W.shape[0]
    Cout = torch.empty(M, N, dtype=torch.float32, device=A.device)
    _check(lib.es_op_linear(_ptr(A), _ptr(W), _ptr(R), _ptr(Cout), M, N, K, path, _stream_ptr(stream)))
    return Cout


def es_op_linear_splitk_workspace_bytes(M: int, N: int, k_splits: int) -> int:
    return int(lib.es_op_linear_splitk_workspace_bytes(M, N, k_splits))


def es_op_linear_splitk(A: torch.Tensor, W: torch.Tensor, R: Optional[torch.Tensor] = None, k_splits: int = 0,
                        workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    M, K = A.shape
    N = W.shape[0]
    Cout = torch.empty(M, N, dtype=torch.float32, device=A.device)
    if workspace is None:
        workspace = torch.empty(max(1, es_op_linear_splitk_workspace_bytes(M, N, max(k_splits, 8 if M > 16 else 32))), dtype=torch.uint8,
                                device=A.device)
    _check(lib.es_op_linear_splitk(_ptr(A), _ptr(W), _ptr(R), _ptr(Cout), M, N, K, k_splits, _ptr(workspace),
                                   workspace.numel() * workspace.element_size(), _stream_ptr(stream)))
    return Cout


def es_op_prefill_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, path: int = 0, stream=None) -> torch.Tensor:
    B, T, Hq, hd = q.shape
    Hkv = k.shape[2]
    out = torch.empty(B, T, Hq * hd, dtype=torch.float16, device=q.device)
    _check(lib.es_op_prefill_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, T, Hq, Hkv, hd, path, _stream_ptr(stream)))
    return out


def es_op_decode_attention_scratch_bytes(B: int, Hq: int, hd: int, max_ctx: int, page_tokens: int) -> int:
    return int(lib.es_op_decode_attention_scratch_bytes(B, Hq, hd, max_ctx, page_tokens))


def es_op_decode_attention(q: torch.Tensor, k_pages: torch.Tensor, v_pages: torch.Tensor, block_table: torch.Tensor,
                           ctx_len: torch.Tensor, max_ctx: int, scratch: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    B, Hq, hd = q.shape
    _, Hkv, P, _ = k_pages.shape
    pages_per_seq = block_table.shape[1]
    if scratch is None:
        scratch = torch.empty(es_op_decode_attention_scratch_bytes(B, Hq, hd, max_ctx, P), dtype=torch.uint8,
                              device=q.device)
    out = torch.empty(B, Hq * hd, dtype=torch.float16, device=q.device)
    _check(lib.es_op_decode_attention(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(ctx_len),
                                      _ptr(out), B, Hq, Hkv, hd, P, pages_per_seq, max_ctx, _ptr(scratch),
                                      scratch.numel(), _stream_ptr(stream)))
    return out


def es_op_decode_attention_static_capacity() -> int:
    return int(lib.es_op_decode_attention_static_capacity())


def es_op_decode_attention_static(q: torch.Tensor, k_pages: torch.Tensor, v_pages: torch.Tensor,
                                  block_table: torch.Tensor, ctx_len: torch.Tensor, max_ctx: int,
                                  out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Decode attention whose split-KV partials live in the library's built-in array: the call itself
    allocates nothing (pass `out` to keep the binding from allocating the result either).  Calls that
    overlap on the GPU race on that array; sizes beyond its capacity raise ES_ERR_WORKSPACE."""
    B, Hq, hd = q.shape
    _, Hkv, P, _ = k_pages.shape
    if out is None:
        out = torch.empty(B, Hq * hd, dtype=torch.float16, device=q.device)
    _check(lib.es_op_decode_attention_static(_ptr(q), _ptr(k_pages), _ptr(v_pages), _ptr(block_table), _ptr(ctx_len),
                                             _ptr(out), B, Hq, Hkv, hd, P, block_table.shape[1], max_ctx,
                                             _stream_ptr(stream)))
    return out


def _partition(fn, t_comp, O, Req, Mem, Bw):
    import numpy as np
    t_comp = np.ascontiguousarray(t_comp, dtype=np.float64)
    N, M = t_comp.shape
    arrs = [t_comp] + [np.ascontiguousarray(a, dtype=np.float64) for a in (O, Req, Mem, Bw)]
    if arrs[1].shape != (N,) or arrs[2].shape != (N,) or arrs[3].shape != (M,) or arrs[4].shape != (M, M):
        raise EsError(2, "partition planner: array shapes do not match [N, M] / [N] / [N] / [M] / [M, M]")
    assign = (C.c_int32 * N)()
    value = C.c_double(0)
    ptrs = [a.ctypes.data_as(C.POINTER(C.c_double)) for a in arrs]
    _check(fn(N, M, *ptrs, assign, C.byref(value)))
    return list(assign), value.value


def es_partition_latency(t_comp, O, Req, Mem, Bw):
    """(device of every layer, total latency): the paper's Algorithm 1 over profiled traces."""
    return _partition(lib.es_partition_latency, t_comp, O, Req, Mem, Bw)


def es_partition_throughput(t_comp, O, Req, Mem, Bw):
    """(device of every layer, slowest stage time): the paper's Algorithm 2 over profiled traces."""
    return _partition(lib.es_partition_throughput, t_comp, O, Req, Mem, Bw)

"""B200-native execution of one EdgeShard model shard (prefill, KV-cached decode, handoff, per-layer
profile) as a C-ABI CUDA library for sm_100a, with a thin ctypes binding.

    from paper_2405_14371_b200 import Shard

The binding loads `libedgeshard.so` from this directory and raises ImportError if it has not been
built (`python -m paper_2405_14371_b200.build`); nothing falls back to the CPU.
"""
import importlib

__all__ = ["binding", "build", "Shard", "EsError"]


def __getattr__(name):
    if name in ("binding", "build"):
        return importlib.import_module(f"{__name__}.{name}")
    if name in ("Shard", "EsError", "make_desc", "es_shard_workspace_bytes", "es_op_rmsnorm", "es_op_linear",
                "es_op_prefill_attention", "es_op_decode_attention", "es_op_decode_attention_scratch_bytes",
                "es_last_error", "es_version"):
        return getattr(importlib.import_module(f"{__name__}.binding"), name)
    raise AttributeError(name)

"""CPU-only checks of the boundary: the library loads, exports every declared symbol, and its
host-side validation returns the documented error codes before anything touches a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2405_14371_b200 import build
    build.build()
    from paper_2405_14371_b200 import binding as b
    return b


def _declared():
    text = open(os.path.join(ROOT, "include", "edgeshard.h")).read()
    return sorted(set(re.findall(r"ES_API[^;(]*?\b(es_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared()
    assert len(names) >= 20 and "es_shard_create" in names and "es_layer_profile" in names
    raw = C.CDLL(binding.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
    assert sorted(binding.EXPORTS) == names


def test_version_and_error_string(binding):
    assert "sm_100a" in binding.es_version()


def _desc(binding, **kw):
    from workload import TINY
    d = binding.make_desc(TINY, 2, 64, 32, 2, 16)
    for k, v in kw.items():
        setattr(d, k, v)
    return d


def test_workspace_sizes_scale(binding):
    kv, sc = binding.es_shard_workspace_bytes(_desc(binding), 0, 2)
    # K and V, 2 layers, 2 slots x 4 pages of 16 tokens, 4 heads x 64, fp16
    assert kv == 2 * 2 * (2 * 4) * (4 * 16 * 64) * 2
    kv1, _ = binding.es_shard_workspace_bytes(_desc(binding), 0, 1)
    assert kv1 * 2 == kv
    _, sc2 = binding.es_shard_workspace_bytes(_desc(binding, max_tokens=64), 0, 2)
    assert sc2 > sc and sc % 256 == 0


@pytest.mark.parametrize("kw,begin,end,status", [
    ({}, 0, 3, 3), ({}, 1, 1, 3), ({}, -1, 1, 3),
    ({"head_dim": 48}, 0, 2, 2), ({"n_kv_heads": 3}, 0, 2, 2), ({"d_ffn": 100}, 0, 2, 2),
    ({"kv_page_tokens": 24}, 0, 2, 2), ({"max_batch": 3}, 0, 2, 1), ({"max_seq": 0}, 0, 2, 1),
    ({"max_tokens": 1}, 0, 2, 1),
])
def test_description_validation(binding, kw, begin, end, status):
    with pytest.raises(binding.EsError) as e:
        binding.es_shard_workspace_bytes(_desc(binding, **kw), begin, end)
    assert e.value.status == status and e.value.message


def test_null_arguments_are_rejected_without_a_gpu(binding):
    lib = binding.lib
    assert lib.es_shard_prefill(None, None, None, 1, 1, None) == 1
    assert lib.es_shard_prefill_ragged(None, None, None, 1, 1, None, None) == 1
    assert lib.es_shard_decode_step(None, None, None, 1, None) == 1
    assert lib.es_shard_handoff(None, None, None, None) == 1
    assert lib.es_layer_profile(None, None, 0, None) == 1
    assert lib.es_op_linear(None, None, None, None, 1, 1, 8, 0, None) == 1
    d = _desc(binding)
    out = C.c_void_p()
    assert lib.es_shard_create(C.byref(d), 0, 2, None, None, 0, None, 0, None, C.byref(out)) == 1
    assert "null" in binding.es_last_error()
    lib.es_shard_destroy(None)
    assert lib.es_shard_launch_count(None) == 0
    assert lib.es_op_decode_attention_scratch_bytes(0, 4, 64, 16, 16) == 0

"""The seeded input generator: deterministic, sliceable, right distribution, same bits on GPU."""
import hashlib

import pytest
import torch

from workload import (TINY, LLAMA2_7B, normal_fp16, token_ids, weight_tensor, standard_normal_f32,
                      WORKLOADS, prompt_ids)


def test_deterministic_and_sliceable():
    a = normal_fp16(3, 5, (10, 7))
    assert torch.equal(a, normal_fp16(3, 5, (10, 7)))
    assert torch.equal(a[3:7], normal_fp16(3, 5, (4, 7), row_begin=3))
    assert not torch.equal(a, normal_fp16(3, 6, (10, 7)))
    assert not torch.equal(a, normal_fp16(4, 5, (10, 7)))


def test_normal_moments():
    z = standard_normal_f32(11, 2, 0, 1 << 21).double()
    assert abs(float(z.mean())) < 3e-3
    assert abs(float(z.std()) - 1.0) < 3e-3
    assert abs(float((z ** 3).mean())) < 2e-2
    assert abs(float((z ** 4).mean()) - 3.0) < 5e-2
    # tail mass beyond 2 sigma: 4.55 %
    assert abs(float((z.abs() > 2).double().mean()) - 0.0455) < 1e-3


def test_weight_scale_and_gain_mean():
    w = weight_tensor(1, LLAMA2_7B, "wq", 0, rows=64).float()
    assert abs(float(w.std()) - 0.02) < 5e-4 and abs(float(w.mean())) < 5e-4
    g = weight_tensor(1, LLAMA2_7B, "attn_norm", 3).float()
    assert abs(float(g.mean()) - 1.0) < 2e-3 and abs(float(g.std()) - 0.02) < 2e-3


def test_token_ids_uniform_in_range():
    ids = token_ids(0, 0, (64, 1000), 1000)
    assert ids.dtype == torch.int32 and int(ids.min()) == 0 and int(ids.max()) == 999
    counts = torch.bincount(ids.flatten().long(), minlength=1000).double()
    assert float(((counts - 64.0) ** 2 / 64.0).sum()) < 1200  # chi-square, 999 dof
    assert torch.equal(prompt_ids(2, 8, 512, 32000)[0, :16], token_ids(2, 0, (8, 512), 32000)[0, :16])


def test_stream_digest_is_stable():
    # guards against accidental changes of the hash or table; value written from this generator
    w = weight_tensor(0, TINY, "wq", 1)
    d = hashlib.sha256(w.numpy().tobytes()).hexdigest()
    assert w.shape == (256, 256)
    assert d[:16] == DIGEST_WQ1, d[:16]


def test_workload_table_matches_configs():
    w = WORKLOADS
    assert (w["cfg1"].layer_begin, w["cfg1"].layer_end, w["cfg1"].prompt_len, w["cfg1"].decode_steps) == (0, 8, 128, 128)
    assert w["cfg1"].has_embedding and not w["cfg1"].has_head
    assert w["cfg2_b8"].batch == 8 and w["cfg2_b8"].has_head
    assert w["cfg3"].n_shards == 4 and w["cfg3"].micro_batches == 8
    assert w["cfg4"].model.n_kv_heads == 8 and w["cfg4"].batch == 16 and not w["cfg4"].has_head


@pytest.mark.gpu
def test_gpu_generation_is_bit_identical():
    for kind in ("wq", "attn_norm", "w_down"):
        a = weight_tensor(0, TINY, kind, 1)
        b = weight_tensor(0, TINY, kind, 1, device="cuda")
        assert torch.equal(a, b.cpu())
    a = weight_tensor(1, LLAMA2_7B, "w_gate", 5, rows=300, row_begin=4000)
    b = weight_tensor(1, LLAMA2_7B, "w_gate", 5, rows=300, row_begin=4000, device="cuda")
    assert torch.equal(a, b.cpu())
    assert torch.equal(token_ids(4, 1, (128, 16), 32000), token_ids(4, 1, (128, 16), 32000, "cuda").cpu())


DIGEST_WQ1 = "3b3519d733ccbcbf"

"""The allocation-free decode-attention entry point (collected last on purpose).

Some callers may not allocate device memory at all — they run under a fixed memory pool, or in a
phase where cudaMalloc would stall the device — and have no spare buffer to lend either.  For them
es_op_decode_attention_static keeps the split-KV partials in an array that is part of the library.
It must give what es_op_decode_attention gives with a caller buffer, call after call, although the
array still holds the previous call's partials."""
import pytest
import torch

pytestmark = pytest.mark.gpu
TOL = 2e-3      # the tolerance of the decode-attention parity tests


def _case(Bn, Hq, Hkv, hd, P, ctxs, seed):
    g = torch.Generator().manual_seed(seed)
    max_ctx = max(ctxs)
    pps = (max_ctx + P - 1) // P
    n_pages = Bn * pps
    table = torch.randperm(n_pages, generator=g).to(torch.int32).reshape(Bn, pps)
    q = torch.randn(Bn, Hq, hd, generator=g).half()
    k = torch.randn(n_pages, Hkv, P, hd, generator=g).half()
    v = torch.randn(n_pages, Hkv, P, hd, generator=g).half()
    return [t.cuda() for t in (q, k, v, table, torch.tensor(ctxs, dtype=torch.int32))] + [max_ctx]


def _rel(a, b):
    return float((a.double() - b.double()).abs().max() / b.double().abs().max())


def test_static_scratch_matches_caller_scratch_on_consecutive_calls():
    from paper_2405_14371_b200 import binding as B
    assert B.es_op_decode_attention_static_capacity() == 8 << 20
    # a long-context call first, then a short one whose splits cover only the start of the array
    cases = [_case(4, 32, 8, 128, 64, [700, 513, 64, 1], seed=1), _case(2, 4, 4, 64, 16, [17, 40], seed=2),
             _case(4, 32, 8, 128, 64, [90, 700, 2, 300], seed=3)]
    for q, k, v, table, ctx, max_ctx in cases:
        want = B.es_op_decode_attention(q, k, v, table, ctx, max_ctx)
        out = torch.empty_like(want)
        n_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
        got = B.es_op_decode_attention_static(q, k, v, table, ctx, max_ctx, out=out)
        n_after = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
        assert n_after == n_before, (n_before, n_after)      # torch's allocator was not asked for anything
        torch.cuda.synchronize()
        assert _rel(got, want) < TOL
        assert torch.equal(got, want)       # same kernels, same order of operations


def test_static_scratch_rejects_oversized_calls():
    from paper_2405_14371_b200 import binding as B
    q, k, v, table, ctx, max_ctx = _case(1, 8, 8, 128, 16, [16], seed=4)
    # 64 sequences x 64 heads over a 6400-token context cut into 10 splits would need 21 MB of partials
    Bn, Hq, Hkv, hd, P, pps = 64, 64, 1, 128, 16, 400
    with pytest.raises(B.EsError) as e:
        B._check(B.lib.es_op_decode_attention_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), table.data_ptr(),
                                                     ctx.data_ptr(), q.data_ptr(), Bn, Hq, Hkv, hd, P, pps, P * pps, None))
    assert e.value.status == 6 and "8388608" in e.value.message

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
    # 256 sequences x 64 heads need 8.5 MB of partials even with a single split
    Bn, Hq, Hkv, hd, P, pps = 256, 64, 8, 128, 16, 4
    with pytest.raises(B.EsError) as e:
        B._check(B.lib.es_op_decode_attention_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), table.data_ptr(),
                                                     ctx.data_ptr(), q.data_ptr(), Bn, Hq, Hkv, hd, P, pps, P * pps, None))
    assert e.value.status == 6 and "8388608" in e.value.message
    # a shape the kernels do not take is reported as such, before any capacity arithmetic
    for bad in ((1, 8, 8, 96), (1, 8, 3, 128), (1, 64, 1, 128)):
        with pytest.raises(B.EsError) as e:
            B._check(B.lib.es_op_decode_attention_static(q.data_ptr(), k.data_ptr(), v.data_ptr(), table.data_ptr(),
                                                         ctx.data_ptr(), q.data_ptr(), bad[0], bad[1], bad[2], bad[3], 16, 1, 16, None))
        assert e.value.status == 2, bad


def test_static_scratch_takes_nothing_from_the_device_on_any_stream():
    """After a first call (which looks up the array's address), further calls must leave the driver's count of
    free device memory exactly where it was — a cudaMalloc inside the library would not show in torch's own
    allocator statistics — on the default stream and on a stream of the caller's."""
    from paper_2405_14371_b200 import binding as B
    q, k, v, table, ctx, max_ctx = _case(4, 32, 8, 128, 64, [700, 513, 64, 1], seed=5)
    want = B.es_op_decode_attention(q, k, v, table, ctx, max_ctx)
    out = torch.empty_like(want)
    side = torch.cuda.Stream()
    B.es_op_decode_attention_static(q, k, v, table, ctx, max_ctx, out=out)          # warm-up: address look-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for i in range(6):
        st = side if i % 2 else None
        out.zero_()
        if st is not None:
            st.wait_stream(torch.cuda.current_stream())
        n_before = torch.cuda.memory_stats().get("allocation.all.allocated", 0)
        got = B.es_op_decode_attention_static(q, k, v, table, ctx, max_ctx, out=out, stream=st)
        assert torch.cuda.memory_stats().get("allocation.all.allocated", 0) == n_before   # nor from torch's allocator
        torch.cuda.synchronize()                     # the calls share one array: never two in flight
        assert torch.cuda.mem_get_info()[0] == free_before
        assert torch.equal(got, want)

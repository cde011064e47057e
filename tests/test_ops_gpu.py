"""Per-kernel parity against the oracle's definitions, on small and ragged shapes (through the C ABI)."""
import math

import pytest
import torch

from oracle import decoder as O
from tests.helpers import rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2405_14371_b200 import binding
    return binding


def _randn(*shape, seed=0, scale=1.0, dtype=torch.float16):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(dtype)


@pytest.mark.parametrize("M,d", [(1, 256), (5, 4096), (3, 8192), (2, 16384), (7, 688), (0, 256), (256, 4096), (257, 688),
                                 (300, 8192), (260, 16384)])
def test_rmsnorm(B, M, d):
    x = _randn(M, d, seed=1, scale=3.0, dtype=torch.float32)
    g = (1 + 0.1 * _randn(d, seed=2, dtype=torch.float32)).half()
    y = B.es_op_rmsnorm(x.cuda(), g.cuda(), 1e-5)
    torch.cuda.synchronize()
    if M == 0:
        return
    want = O.rmsnorm(x.double(), g.double(), 1e-5)
    assert rel_err(y, want) < 2e-3


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("M,N,K", [(1, 256, 256), (1, 1000, 256), (3, 300, 688), (16, 768, 256), (8, 129, 1032),
                                   (13, 4096, 4096), (1, 11008, 4096)])
def test_linear_skinny_and_reference(B, path, M, N, K):
    A = _randn(M, K, seed=3)
    W = _randn(N, K, seed=4, scale=0.05)
    R = _randn(M, N, seed=5, dtype=torch.float32)
    want = A.double() @ W.double().T
    got = B.es_op_linear(A.cuda(), W.cuda(), None, path)
    assert rel_err(got, want) < 1e-5
    got = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), path)
    assert rel_err(got, want + R.double()) < 1e-5


@pytest.mark.parametrize("M,N,K", [(64, 128, 64), (100, 200, 136), (257, 1000, 688), (512, 4096, 4096)])
def test_linear_reference_large(B, M, N, K):
    A = _randn(M, K, seed=6)
    W = _randn(N, K, seed=7, scale=0.05)
    got = B.es_op_linear(A.cuda(), W.cuda(), None, 3)
    assert rel_err(got, A.double() @ W.double().T) < 1e-5


@pytest.mark.parametrize("M,N,K", [(17, 32, 64), (128, 128, 64), (100, 200, 136), (257, 1000, 688), (512, 4096, 4096),
                                   (300, 96, 4096), (128, 4096, 11008), (1024, 640, 256), (2100, 384, 1024),
                                   (128, 11008, 512), (128, 20000, 256), (100, 25000, 256), (128, 30000, 320)])
def test_linear_tensor_core(B, M, N, K):
    """tcgen05 path: every tile width (32 .. 256 in steps of 32 — the last four shapes select 96, 160, 192
    and 224), ragged M / N / K, long K, and agreement with the plain kernel."""
    A = _randn(M, K, seed=13)
    W = _randn(N, K, seed=14, scale=0.05)
    R = _randn(M, N, seed=15, dtype=torch.float32)
    want = A.double() @ W.double().T
    got = B.es_op_linear(A.cuda(), W.cuda(), None, 1)
    assert rel_err(got, want) < 5e-5   # fp32 tensor-core accumulation over K up to 11008
    got_r = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), 1)
    assert rel_err(got_r, want + R.double()) < 5e-5   # fp32 tensor-core accumulation over K up to 11008
    ref = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), 3)
    assert rel_err(got_r, ref) < 5e-5   # fp32 tensor-core accumulation over K up to 11008


@pytest.mark.parametrize("M,N,K", [(3, 64, 256), (8, 4096, 4096), (8, 1000, 512), (13, 136, 1024), (16, 8192, 8192),
                                   (16, 24, 28672), (5, 11008, 4096), (16, 4096, 11008)])
def test_linear_streaming_tensor_core(B, M, N, K):
    """mma.sync weight-streaming kernel (decode with several sequences): ragged N, long K, 1 and 2 row groups."""
    A = _randn(M, K, seed=16)
    W = _randn(N, K, seed=17, scale=0.05)
    R = _randn(M, N, seed=18, dtype=torch.float32)
    want = A.double() @ W.double().T
    got = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), 4)
    assert rel_err(got, want + R.double()) < 5e-5
    assert rel_err(B.es_op_linear(A.cuda(), W.cuda(), None, 4), want) < 5e-5


@pytest.mark.parametrize("M,N,K", [(2048, 4096, 1024), (1100, 5000, 520), (4096, 4096, 4096), (512, 12288, 4096)])
def test_linear_tensor_core_cta_pairs(B, M, N, K):
    """cta_group::2 kernel: 256 x 256 and 256 x 512 tiles on CTA pairs, ragged M / N / K, agreement with the single-CTA kernel."""
    A = _randn(M, K, seed=19)
    W = _randn(N, K, seed=20, scale=0.05)
    R = _randn(M, N, seed=21, dtype=torch.float32)
    ref = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), 1)
    want = A.double() @ W.double().T + R.double()
    for path in (5, 6):                          # 256 x 256 and 256 x 512 tiles
        got = B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), path)
        assert rel_err(got, want) < 5e-5
        assert rel_err(got, ref) < 1e-5
    assert rel_err(B.es_op_linear(A.cuda(), W.cuda(), None, 6), A.double() @ W.double().T) < 5e-5


@pytest.mark.parametrize("M,N,K,S", [(128, 4096, 4096, 0), (128, 4096, 11008, 0), (256, 5120, 5120, 0), (100, 260, 1096, 3),
                                     (17, 36, 512, 2), (300, 1000, 4096, 5), (128, 512, 256, 4), (512, 4096, 4096, 0),
                                     (128, 4096, 4096, 1), (512, 4096, 11008, 0), (700, 1000, 2080, 3), (256, 5120, 13824, 0)])
def test_linear_tensor_core_split_k(B, M, N, K, S):
    """K range cut into slices (automatic count and fixed counts), ragged M / N / K, residual aliasing the output."""
    A = _randn(M, K, seed=22)
    W = _randn(N, K, seed=23, scale=0.05)
    R = _randn(M, N, seed=24, dtype=torch.float32)
    want = A.double() @ W.double().T
    got = B.es_op_linear_splitk(A.cuda(), W.cuda(), None, S)
    assert rel_err(got, want) < 5e-5
    got_r = B.es_op_linear_splitk(A.cuda(), W.cuda(), R.cuda(), S)
    assert rel_err(got_r, want + R.double()) < 5e-5
    again = B.es_op_linear_splitk(A.cuda(), W.cuda(), R.cuda(), S)
    assert torch.equal(got_r, again)            # slices are added in a fixed order


@pytest.mark.parametrize("M,N,K,S", [(8, 4096, 11008, 0), (16, 2048, 28672, 0), (16, 1024, 8192, 0), (5, 1000, 2048, 2),
                                     (3, 36, 1024, 4), (13, 520, 4096, 8), (16, 8192, 8192, 4)])
def test_linear_streaming_k_sliced(B, M, N, K, S):
    """Decode-sized products with K sliced across CTAs (activation slice in shared memory), automatic and fixed slice
    counts, ragged N, 1 and 2 groups of 8 activation rows; must agree with the unsliced streaming kernel."""
    A = _randn(M, K, seed=25)
    W = _randn(N, K, seed=26, scale=0.05)
    R = _randn(M, N, seed=27, dtype=torch.float32)
    want = A.double() @ W.double().T + R.double()
    got = B.es_op_linear_splitk(A.cuda(), W.cuda(), R.cuda(), S)
    assert rel_err(got, want) < 5e-5
    assert rel_err(got, B.es_op_linear(A.cuda(), W.cuda(), R.cuda(), 4)) < 1e-5
    assert torch.equal(got, B.es_op_linear_splitk(A.cuda(), W.cuda(), R.cuda(), S))


def test_linear_split_k_rejects(B):
    A = _randn(128, 256, seed=1).cuda()
    W = _randn(64, 256, seed=2).cuda()
    with pytest.raises(B.EsError):               # 4 K blocks cannot make 3 non-empty slices of 2
        B.es_op_linear_splitk(A, W, None, 3)
    with pytest.raises(B.EsError):               # workspace too small
        B.es_op_linear_splitk(A, W, None, 2, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(B.EsError):               # N not a multiple of 4
        B.es_op_linear_splitk(A, _randn(62, 256, seed=3).cuda(), None, 2)


def test_linear_rejects_bad_shapes(B):
    A = _randn(17, 64).cuda()
    W = _randn(32, 64).cuda()
    with pytest.raises(B.EsError) as e:
        B.es_op_linear(A, W, None, 2)          # weight-streaming kernel takes <= 16 rows
    assert e.value.status == 9
    with pytest.raises(B.EsError) as e:
        B.es_op_linear(_randn(2, 12).cuda(), _randn(4, 12).cuda(), None, 0)   # K % 8
    assert e.value.status == 2


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("Bn,T,Hq,Hkv,hd", [(1, 1, 4, 4, 64), (2, 16, 4, 4, 64), (1, 37, 4, 2, 128), (2, 130, 8, 1, 128),
                                            (1, 200, 2, 2, 64), (2, 64, 2, 2, 128), (1, 128, 2, 1, 128), (3, 257, 4, 4, 64),
                                            (1, 512, 2, 2, 128),
                                            # enough CTAs for two to share every SM, many KV tiles per CTA
                                            (2, 576, 32, 8, 128), (3, 320, 40, 40, 64)])
def test_prefill_attention(B, path, Bn, T, Hq, Hkv, hd):
    """path 1 = tcgen05 kernel, 2 = CUDA-core kernel; N(0,1) q, k, v give peaked softmax rows."""
    q = _randn(Bn, T, Hq, hd, seed=8)
    k = _randn(Bn, T, Hkv, hd, seed=9)
    v = _randn(Bn, T, Hkv, hd, seed=10)
    got = B.es_op_prefill_attention(q.cuda(), k.cuda(), v.cuda(), path)
    for b in range(Bn):
        want = O.causal_attention_matrix(q[b].double(), k[b].double(), v[b].double()).reshape(T, Hq * hd)
        assert rel_err(got[b], want) < 2e-3


@pytest.mark.parametrize("Bn,Hq,Hkv,hd,P,ctxs", [
    (1, 4, 4, 64, 16, [1]), (2, 4, 4, 64, 16, [16, 17]), (3, 8, 2, 128, 64, [5, 64, 200]),
    (2, 8, 1, 128, 64, [300, 1]), (4, 32, 32, 128, 64, [128, 129, 255, 256]), (16, 64, 8, 128, 64, list(range(1000, 1016))),
    # many (sequence, head, split) items: the tensor-core kernel, all group sizes, ragged and tiny contexts, small pages
    (8, 32, 32, 128, 64, [640, 513, 300, 17, 1, 639, 256, 257]), (12, 16, 8, 128, 16, [100 + 27 * i for i in range(12)]),
    (10, 32, 8, 128, 32, [1, 15, 16, 17, 31, 33, 300, 299, 512, 700]), (40, 8, 8, 128, 64, [3 + 5 * i for i in range(40)]),
])
def test_decode_attention_paged(B, Bn, Hq, Hkv, hd, P, ctxs):
    max_ctx = max(ctxs)
    pps = (max_ctx + P - 1) // P + 1
    n_pages = Bn * pps
    g = torch.Generator().manual_seed(11)
    perm = torch.randperm(n_pages, generator=g).to(torch.int32).reshape(Bn, pps)   # scattered physical pages
    kp = torch.zeros(n_pages, Hkv, P, hd, dtype=torch.float16)
    vp = torch.zeros_like(kp)
    q = _randn(Bn, Hq, hd, seed=12)
    ks, vs = [], []
    for b in range(Bn):
        k = _randn(ctxs[b], Hkv, hd, seed=20 + b)
        v = _randn(ctxs[b], Hkv, hd, seed=40 + b)
        ks.append(k); vs.append(v)
        for t in range(ctxs[b]):
            pg = int(perm[b, t // P])
            kp[pg, :, t % P, :] = k[t]
            vp[pg, :, t % P, :] = v[t]
    got = B.es_op_decode_attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(),
                                   torch.tensor(ctxs, dtype=torch.int32).cuda(), max_ctx)
    for b in range(Bn):
        want = O.causal_attention_matrix(q[b:b + 1].double(), ks[b].double(), vs[b].double(), q_pos0=ctxs[b] - 1)
        assert rel_err(got[b], want.reshape(-1)) < 2e-3


@pytest.mark.parametrize("Bn,Hq,Hkv,hd,P,pps", [(2, 4, 4, 64, 16, 3), (9, 32, 8, 128, 64, 5)])
def test_decode_attention_clamps_context_lengths_to_the_page_list(B, Bn, Hq, Hkv, hd, P, pps):
    """A context length on the device that exceeds what the sequence's row of the page table can hold is read as
    "the whole row" (no page index past the row is ever followed), and an empty context gives zeros."""
    cap = P * pps
    n_pages = Bn * pps
    g = torch.Generator().manual_seed(5)
    perm = torch.randperm(n_pages, generator=g).to(torch.int32).reshape(Bn, pps)
    kp = torch.randn(n_pages, Hkv, P, hd, generator=g).half()
    vp = torch.randn(n_pages, Hkv, P, hd, generator=g).half()
    q = _randn(Bn, Hq, hd, seed=6)
    ctx_dev = [cap + 1000 * (b + 1) for b in range(Bn)]
    ctx_dev[-1] = 0                                                       # an empty sequence
    got = B.es_op_decode_attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(),
                                   torch.tensor(ctx_dev, dtype=torch.int32).cuda(), cap)
    for b in range(Bn - 1):
        k = torch.cat([kp[int(perm[b, i])] for i in range(pps)], dim=1).transpose(0, 1)      # [cap, Hkv, hd]
        v = torch.cat([vp[int(perm[b, i])] for i in range(pps)], dim=1).transpose(0, 1)
        want = O.causal_attention_matrix(q[b:b + 1].double(), k.double(), v.double(), q_pos0=cap - 1)
        assert rel_err(got[b], want.reshape(-1)) < 2e-3
    assert torch.count_nonzero(got[Bn - 1]) == 0

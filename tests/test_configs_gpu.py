"""Parity on the large configurations (through the C ABI, in the launch configuration bench.py times).

The oracle side is one causal pass (matrix form) over prompt + teacher-forced decode ids, so the
handoff activation can be checked at every position: after the prefill (all prompt positions) and
after every decode step."""
import pytest
import torch

from oracle import decoder as O
from tests.helpers import device_weights, rel_err
from workload import WORKLOADS, prompt_ids, forced_decode_ids

pytestmark = pytest.mark.gpu
TOL = 1e-2


@pytest.fixture(scope="module")
def B():
    from paper_2405_14371_b200 import binding
    return binding


def test_cfg1_prefill_and_every_decode_step(B):
    wl = WORKLOADS["cfg1"]
    m, T, S = wl.model, wl.prompt_len, wl.decode_steps
    wd, wh = device_weights(wl.cfg, m, wl.layer_begin, wl.layer_end)
    ids = prompt_ids(wl.cfg, 1, T, m.vocab)
    forced = forced_decode_ids(wl.cfg, 1, S, m.vocab)
    seq = torch.cat([ids[0], forced[:, 0]])
    want, _ = O.shard_forward_full(m, wh, wl.layer_begin, wl.layer_end, ids=seq)     # [T+S, d]
    del wh

    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        sh = B.Shard(m, wl.layer_begin, wl.layer_end, wd, max_slots=1, max_seq=T + S, max_tokens=T, stream=stream)
        sh.es_shard_prefill(ids.cuda(), None, 1, T, [0])
        h, lg, nx = sh.es_shard_handoff()
        assert lg is None and nx is None and h.shape == (1, T, m.d_model)
        got_prefill = h[0].clone()
        cur = torch.zeros(1, dtype=torch.int32, device="cuda")
        rows = []
        forced_d = forced.cuda()
        for s in range(S):
            cur.copy_(forced_d[s])
            sh.es_shard_decode_step(cur, None, 1, [0])
            rows.append(sh.es_shard_handoff()[0][0, 0].clone())
        sh.es_shard_device_status()
        sh.close()
    torch.cuda.synchronize()
    assert rel_err(got_prefill, want[:T]) < TOL
    got_dec = torch.stack(rows)
    assert rel_err(got_dec, want[T:]) < TOL
    worst = max(rel_err(got_dec[s], want[T + s]) for s in range(S))
    assert worst < TOL, worst

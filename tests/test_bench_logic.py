"""Host-side arithmetic of the benchmark: the byte / flop models the roofline fractions divide by, and the
attribution of a step's time to its kernels from their time stamps.  No GPU needed."""
import importlib.util
import os

import pytest

from workload import WORKLOADS

_spec = importlib.util.spec_from_file_location("bench", os.path.join(os.path.dirname(os.path.dirname(__file__)), "bench.py"))
bench = importlib.util.module_from_spec(_spec)
_spec.loader.exec_module(bench)


def test_decode_bytes_and_prefill_flops_match_the_hand_computed_figures():
    # config 1: 8 layers of Llama-2-7B, one sequence, average context 128 + 64.5
    wl = WORKLOADS["cfg1"]
    layer = 2 * (2 * 4096 + 4 * 4096 * 4096 + 3 * 4096 * 11008)
    kv = 8 * 1 * (128 + 129 / 2.0) * 2 * 32 * 128 * 2
    assert bench.algorithmic_decode_bytes(wl, 128 + 129 / 2.0) == pytest.approx(8 * layer + kv)
    assert bench.algorithmic_decode_bytes(wl, 192.5) / 1e9 == pytest.approx(3.263, abs=2e-3)
    gemm = 2.0 * 128 * 8 * (4 * 4096 * 4096 + 3 * 4096 * 11008)
    attn = 8 * 2.0 * 128 * 128 * 32 * 128
    assert bench.prefill_flops(wl) == pytest.approx(gemm + attn)
    # config 4: the step's bytes are dominated by 68.45 GB of weights
    wl4 = WORKLOADS["cfg4"]
    assert bench.linear_weight_bytes(wl4) / 1e9 == pytest.approx(68.45, abs=0.01)
    assert bench.algorithmic_decode_bytes(wl4, 1024 + 129 / 2.0) / 1e9 == pytest.approx(71.3, abs=0.1)
    assert bench.prefill_flops(wl4) / 1e12 == pytest.approx(1132, rel=5e-3)
    # a shard with the output layer adds the head's weights
    wl2 = WORKLOADS["cfg2_b1"]
    assert bench.linear_weight_bytes(wl2) - 32 * (layer - 2 * 2 * 4096) == pytest.approx(2 * 32000 * 4096)


def test_time_stamps_are_charged_so_that_the_shares_add_up_to_the_pass():
    # three launches that overlap (programmatic dependent launch): each is charged from the end of the one before it
    e = [{"category": "embed", "start_us": 0.0, "end_us": 2.0, "bytes": 1.0},
         {"category": "qkv", "start_us": 1.0, "end_us": 10.0, "bytes": 100.0},
         {"category": "attention", "start_us": 8.0, "end_us": 15.0, "bytes": 0.0},
         {"category": "qkv", "start_us": 14.0, "end_us": 21.0, "bytes": 100.0},
         {"category": "o", "start_us": -1.0, "end_us": -1.0, "bytes": 5.0}]            # stamps missing: left out
    b = bench.in_step_breakdown(e)
    assert b["span_us"] == 21.0
    assert b["categories"]["embed"]["us"] == 2.0
    assert b["categories"]["qkv"] == {"us": 8.0 + 6.0, "launches": 2, "bytes": 200.0}
    assert b["categories"]["attention"]["us"] == 5.0
    assert "o" not in b["categories"]
    assert sum(c["us"] for c in b["categories"].values()) == b["span_us"]
    # a launch that ends before its predecessor (it cannot, but clocks of different SMs may disagree by a tick) costs 0
    b = bench.in_step_breakdown([{"category": "a", "start_us": 0.0, "end_us": 5.0, "bytes": 0.0},
                                 {"category": "b", "start_us": 1.0, "end_us": 4.9, "bytes": 0.0}])
    assert b["categories"]["b"]["us"] == 0.0 and b["span_us"] == 5.0
    assert bench.in_step_breakdown([]) == {"span_us": 0.0, "categories": {}}

#!/usr/bin/env python
"""Benchmark of the shard forward pass: prefill latency and KV-cached decode throughput.

One "step" is one pass of the whole hot path over one batch: a prefill of the prompt followed by all decode
steps of the workload.  The default workload is the largest configuration that one GPU holds — the
Llama-2-70B-architecture shard of layers 0..39, batch 16, 1024-token prompts, 128 decode steps — and the other
configurations are measured after it with a few steps each and reported as sub-records of the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--also cfg1,cfg2_b1,...|none]
                    [--impl ours|reference]

With N > 1 every rank runs an independent replica of the workload on its own GPU ("replicas only": the path
has no cross-GPU exchange); the time is the maximum over ranks and the value the sum of all ranks' tokens over
that time.  Started as a plain `python bench.py --gpus N` it starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workload import WORKLOADS, forced_decode_ids, layer_weights, prompt_ids, shard_weights, weight_tensor  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
HBM_NOMINAL_GBS = 8000.0          # the figure the decode target is written against
TENSOR_NOMINAL_TFLOPS = 2250.0    # dense fp16, the figure the prefill target is written against
DEFAULT_ALSO = "cfg1,cfg2_b1,cfg2_b8,cfg3"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant decode kernel (average over the four
# products of a layer), from the ncu captures summarised under profiles/; an entry is None when that kernel
# has changed since its counters were taken.
TRAFFIC_PER_LAUNCH = {
    "cfg1": 103.7e6,      # profiles/linear_stream_kernel_cfg1_decode.md (same workload)
    "cfg4": 434.2e6,      # profiles/decode_kernels_cfg4_shapes_batch16_2layers.md: the four products of a layer, whose
                          # launches are the same in the 2-layer capture case and in the 40-layer workload
}


def _peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm": float(p["hbm_gbs"]), "tensor_burst": float(p["bf16_tflops"]),
                "tensor_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "kind": "measured"}
    return {"hbm": 6650.0, "tensor_burst": 1590.0, "tensor_sustained": 1400.0, "kind": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs (queries only)."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_decode_bytes(wl, ctx_avg: float) -> float:
    """Bytes one decode step must move: every weight of the shard once, the visible K/V, the head."""
    m = wl.model
    nl = wl.layer_end - wl.layer_begin
    wbytes = nl * 2 * m.layer_params()
    kv = nl * wl.batch * ctx_avg * 2 * m.n_kv_heads * m.head_dim * 2
    head = 2 * m.vocab * m.d_model if wl.has_head else 0
    return wbytes + kv + head


def linear_weight_bytes(wl) -> float:
    """Bytes the weight-streaming kernel family reads per decode step (matrices only)."""
    m = wl.model
    nl = wl.layer_end - wl.layer_begin
    per_layer = 2 * (m.q_dim * m.d_model + 2 * m.kv_dim * m.d_model + m.d_model * m.q_dim + 3 * m.d_model * m.d_ffn)
    return nl * per_layer + (2 * m.vocab * m.d_model if wl.has_head else 0)


def prefill_flops(wl) -> float:
    m = wl.model
    nl = wl.layer_end - wl.layer_begin
    M = wl.batch * wl.prompt_len
    gemm = 2.0 * M * nl * (m.q_dim * m.d_model + 2 * m.kv_dim * m.d_model + m.d_model * m.q_dim + 3 * m.d_model * m.d_ffn)
    attn = nl * wl.batch * 2.0 * wl.prompt_len ** 2 * m.n_heads * m.head_dim
    head = 2.0 * wl.batch * m.vocab * m.d_model if wl.has_head else 0.0
    return gemm + attn + head


LINEAR_CATS = ("qkv", "o", "gate_up", "down", "lm_head")


def in_step_breakdown(entries: list) -> dict:
    """Per-category time of one pass from the kernels' own time stamps.  A launch is charged the time from the
    end of the launch before it to its own end (the first one from its own start), so the shares add up to the
    span of the pass however much consecutive kernels overlap."""
    out, prev_end = {}, None
    for e in entries:
        if e["start_us"] < 0 or e["end_us"] < 0:
            continue                                   # a launch whose stamps are missing
        begin = e["start_us"] if prev_end is None else prev_end
        dur = max(0.0, e["end_us"] - begin)
        prev_end = e["end_us"] if prev_end is None else max(prev_end, e["end_us"])
        c = out.setdefault(e["category"], {"us": 0.0, "launches": 0, "bytes": 0.0})
        c["us"] += dur
        c["launches"] += 1
        c["bytes"] += e["bytes"]
    span = (prev_end or 0.0) - min((e["start_us"] for e in entries if e["start_us"] >= 0), default=0.0)
    return {"span_us": span, "categories": out}


def run_ours(args, name: str, steps: int, warmup: int, dist_ctx, with_clocks: bool):
    """Times one workload; returns the result dict on rank 0 (None elsewhere)."""
    from paper_2405_14371_b200 import binding as B
    from paper_2405_14371_b200 import replicas

    rank, local, world = dist_ctx
    wl = WORKLOADS[name]
    if args.layers:
        wl = dataclasses.replace(wl, layer_end=min(wl.layer_end, wl.layer_begin + args.layers * wl.n_shards))
    if args.model_layers:
        # a shallow model of the same layer shapes, so that a small capture case still ends with the output layer
        wl = dataclasses.replace(wl, model=dataclasses.replace(wl.model, n_layers=args.model_layers), layer_begin=0,
                                 layer_end=args.model_layers)
    m = wl.model
    Bn, T, S = (args.batch or wl.batch), (args.prompt_len or wl.prompt_len), (args.decode_steps or wl.decode_steps)
    if (Bn, T, S) != (wl.batch, wl.prompt_len, wl.decode_steps):
        wl = dataclasses.replace(wl, batch=Bn, prompt_len=T, decode_steps=S)
    dev = torch.device("cuda", local)
    stream = torch.cuda.Stream(device=dev)
    weights = shard_weights(wl.cfg, m, wl.layer_begin, wl.layer_end, device=dev)
    # a workload may run its layer range as several shards in sequence, with micro-batches of Bn
    # sequences each living in their own KV slots of every shard (the pipeline of config 3)
    n_sh, MB = wl.n_shards, wl.micro_batches
    per = (wl.layer_end - wl.layer_begin) // n_sh
    ids_host = prompt_ids(wl.cfg, MB * Bn, T, m.vocab).reshape(MB, Bn, T).pin_memory()
    forced_host = forced_decode_ids(wl.cfg, MB * Bn, S, m.vocab).reshape(S, MB, Bn).pin_memory()
    ids_dev = ids_host.to(dev)
    forced_dev = forced_host.to(dev)
    cur_ids = torch.zeros(MB, Bn, dtype=torch.int32, device=dev)
    slots = [list(range(mb * Bn, (mb + 1) * Bn)) for mb in range(MB)]
    hid_host = torch.empty(Bn, T, m.d_model, dtype=torch.float32).pin_memory()
    row_host = torch.empty(Bn, 1, m.d_model, dtype=torch.float32).pin_memory()
    tok_host = torch.empty(Bn, dtype=torch.int32).pin_memory()

    def shard_slice(i):
        b0, b1 = wl.layer_begin + i * per, wl.layer_begin + (i + 1) * per
        w = {"layers": weights["layers"][i * per:(i + 1) * per]}
        if b0 == 0:
            w["tok_embedding"] = weights["tok_embedding"]
        if b1 == m.n_layers:
            w["final_norm"], w["lm_head"] = weights["final_norm"], weights["lm_head"]
        return b0, b1, w

    pipelined = n_sh > 1 and args.schedule != "sequential"
    shard_streams = [torch.cuda.Stream(device=dev) if pipelined else stream for _ in range(n_sh)]
    with torch.cuda.stream(stream):
        shards = []
        for i in range(n_sh):
            b0, b1, w = shard_slice(i)
            shards.append(B.Shard(m, b0, b1, w, max_slots=MB * Bn, max_seq=T + S, max_tokens=Bn * T, max_batch=Bn,
                                  stream=shard_streams[i]))
        sh = shards[0]
        torch.cuda.synchronize(dev)

        def through(mb, first_ids, prefill):
            """one micro-batch through every shard; on one device the hand-over is the handoff view itself"""
            x = None
            for si, shd in enumerate(shards):
                if prefill:
                    shd.es_shard_prefill(first_ids if si == 0 else None, x, Bn, T, slots[mb])
                else:
                    shd.es_shard_decode_step(first_ids if si == 0 else None, x, Bn, slots[mb])
                x, lg, nx = shd.es_shard_handoff()
            return x, lg, nx

        def one_step(e2e: bool, events=None):
            """prefill + S decode steps.  e2e: inputs come from pinned host memory every call and the
            result (handoff activation, or the token when the last shard holds the head) goes back."""
            if events:
                events[0].record(stream)
            nx = None
            for mb in range(MB):
                if e2e:
                    ids_dev[mb].copy_(ids_host[mb], non_blocking=True)
                h, lg, nx = through(mb, ids_dev[mb], True)
                if wl.has_head and MB > 1:
                    cur_ids[mb].copy_(nx)
                if e2e:
                    (tok_host.copy_(nx, non_blocking=True) if wl.has_head else hid_host.copy_(h, non_blocking=True))
            if events:
                events[1].record(stream)
            for s in range(S):
                for mb in range(MB):
                    if wl.has_head:
                        src = nx if MB == 1 else cur_ids[mb]     # greedy feedback stays on the device
                    else:
                        cur_ids[mb].copy_(forced_host[s, mb] if e2e else forced_dev[s, mb], non_blocking=True)
                        src = cur_ids[mb]
                    h, lg, nx2 = through(mb, src, False)
                    if wl.has_head and MB > 1:
                        cur_ids[mb].copy_(nx2)
                    if e2e:
                        (tok_host.copy_(nx2, non_blocking=True) if wl.has_head else row_host.copy_(h, non_blocking=True))
            if events:
                events[2].record(stream)

        def one_step_pipelined(e2e: bool, events=None):
            """the same work under a pipelined schedule: one stream per shard, dependencies as events"""
            from paper_2405_14371_b200.pipeline import ShardPipeline

            pipe = ShardPipeline(shards, slots, Bn, args.schedule)
            if events:
                events[0].record(stream)
            if e2e:
                ids_dev.copy_(ids_host, non_blocking=True)

            def read_back(p, out):
                if e2e:
                    (tok_host.copy_(out[2], non_blocking=True) if wl.has_head else
                     (hid_host if p.iteration == 0 else row_host).copy_(out[0], non_blocking=True))

            pipe.fork(stream)
            pipe.prefill(ids_dev, T, on_output=read_back)
            pipe.join(stream)
            if events:
                events[1].record(stream)
            pipe.fork(stream)
            pipe.decode(S, forced=None if wl.has_head else (forced_host if e2e else forced_dev), on_output=read_back)
            pipe.join(stream)
            if events:
                events[2].record(stream)

        if pipelined:
            one_step = one_step_pipelined

        for _ in range(warmup):
            one_step(False)
        if not args.profile:
            one_step(True)
        stream.synchronize()

        def timed(e2e: bool):
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
            replicas.barrier(world)
            n0 = sum(x.es_shard_launch_count() for x in shards)
            for k in range(steps):
                one_step(e2e, evs[k])
            stream.synchronize()
            replicas.barrier(world)
            n1 = sum(x.es_shard_launch_count() for x in shards)
            pre = [e[0].elapsed_time(e[1]) for e in evs]
            dec = [e[1].elapsed_time(e[2]) for e in evs]
            return pre, dec, n1 - n0

        sampler = ClockSampler(local)
        if rank == 0 and with_clocks:
            sampler.start()
        pre, dec, launches = timed(False)
        if args.profile:
            # short run for a profiler capture: one timed pass, nothing else (not a bench value)
            if with_clocks:
                sampler.stop()
            stream.synchronize()
            if rank == 0:
                return {"profile_run": True, "workload": name, "batch": Bn, "prompt_len": T, "decode_steps": S,
                        "prefill_ms": sum(pre) / len(pre), "decode_ms_per_step": sum(dec) / (S * len(dec)),
                        "gpu_launches": int(launches)}
            return None
        pre_e, dec_e, _ = timed(True)
        clocks = sampler.stop() if (rank == 0 and with_clocks) else None

        # Where the time of a pass goes, from the kernels' own time stamps: one prefill and a few replayed decode
        # steps of the first shard after the timed region, graphs and programmatic dependent launch as in the
        # timed steps (the stamps are switched off again afterwards and are not part of the timed region).
        torch.cuda.synchronize(dev)
        with torch.cuda.stream(sh.stream):
            sh.es_shard_set_step_timing(True)
            sh.es_shard_prefill(ids_dev[0], None, Bn, T, slots[0])
            pre_stamps = in_step_breakdown(sh.es_shard_step_timing())
            src = sh.es_shard_handoff()[2] if (wl.has_head and n_sh == 1) else cur_ids[0]
            dec_breaks = []
            n_probe = min(40, S)
            for i in range(n_probe):
                sh.es_shard_decode_step(src, None, Bn, slots[0])
                # the first steps capture and upload the graph, and steps right behind a long prefill run at the low
                # clock the prefill left: the last few of a run of steps are read
                if i >= max(2, n_probe - 6):
                    dec_breaks.append(in_step_breakdown(sh.es_shard_step_timing()))
            sh.es_shard_set_step_timing(False)
        for x in shards:
            x.es_shard_device_status()

    dec_total = replicas.max_over_ranks(sum(dec), world)
    pre_mean = replicas.max_over_ranks(sum(pre) / len(pre), world)
    dec_total_e = replicas.max_over_ranks(sum(dec_e), world)
    pre_mean_e = replicas.max_over_ranks(sum(pre_e) / len(pre_e), world)
    total_ms = replicas.max_over_ranks(sum(pre) + sum(dec), world)
    for x in shards:
        x.close()
    del shards, weights
    torch.cuda.empty_cache()
    if rank != 0:
        return None

    peaks = _peaks()
    tokens = MB * Bn * S * steps * world
    value = tokens / (dec_total / 1e3)
    value_e = tokens / (dec_total_e / 1e3)
    ctx_avg = T + (S + 1) / 2.0
    step_bytes = MB * algorithmic_decode_bytes(wl, ctx_avg)     # every micro-batch pass re-streams the weights
    decode_ms = dec_total / (S * steps)
    step_gbs = step_bytes / (decode_ms / 1e3) / 1e9
    flops = MB * prefill_flops(wl)
    pre_tflops = flops / (pre_mean / 1e3) / 1e12

    # decode roofline: the weight-streaming linear kernels of the (first shard's) replayed step
    def merge(breaks):
        cats = {}
        for b in breaks:
            for c, v in b["categories"].items():
                t = cats.setdefault(c, {"us": 0.0, "launches": 0, "bytes": 0.0})
                for k in t:
                    t[k] += v[k] / len(breaks)
        return {"span_us": sum(b["span_us"] for b in breaks) / len(breaks), "categories": cats}

    dstep = merge(dec_breaks) if dec_breaks else {"span_us": 0.0, "categories": {}}
    lin_us = sum(v["us"] for c, v in dstep["categories"].items() if c in LINEAR_CATS)
    lin_bytes = sum(v["bytes"] for c, v in dstep["categories"].items() if c in LINEAR_CATS)
    lin_n = sum(v["launches"] for c, v in dstep["categories"].items() if c in LINEAR_CATS)
    lin_gbs = lin_bytes / (lin_us * 1e-6) / 1e9 if lin_us > 0 else 0.0
    dom = ("linear_stream_kernel" if Bn <= 2 else "linear_stream_mma_kernel / linear_stream_mma_ks_kernel")
    roofline = {"bound": "hbm", "kernel": dom, "achieved": lin_gbs, "peak": peaks["hbm"], "unit": "GB/s",
                "frac": lin_gbs / peaks["hbm"], "peak_source": peaks["kind"] + " copy bandwidth",
                "peak_nominal": HBM_NOMINAL_GBS, "frac_nominal": lin_gbs / HBM_NOMINAL_GBS,
                "how": "time stamps written by the kernels inside replayed decode steps; a launch is charged from the end "
                       "of the launch before it to its own end, so launches x avg_launch_us <= the step",
                "launches_per_step": lin_n, "avg_launch_us": lin_us / lin_n if lin_n else None,
                "bytes_per_launch": lin_bytes / lin_n if lin_n else None,
                "in_step_us": {c: round(v["us"], 2) for c, v in sorted(dstep["categories"].items())},
                "step_span_us": round(dstep["span_us"], 2),
                "traffic": TRAFFIC_PER_LAUNCH.get(name)}
    # prefill roofline: the whole prefill against the tensor peak, and the tensor-core products inside it
    pcat = pre_stamps["categories"]
    gemm_us = sum(v["us"] for c, v in pcat.items() if c in LINEAR_CATS[:4])
    gemm_flops = sum(v["bytes"] for c, v in pcat.items() if c in LINEAR_CATS[:4]) * Bn * T   # 2*M*N*K = M * weight bytes
    gemm_tflops = gemm_flops / (gemm_us * 1e-6) / 1e12 if gemm_us > 0 else 0.0
    M_rows = Bn * T
    weight_floor_ms = MB * linear_weight_bytes(wl) / (peaks["hbm"] * 1e9) * 1e3
    roofline_prefill = {"bound": "tensor" if M_rows >= 512 else "hbm (weight read: fewer than 512 rows per product)",
                        "kernel": "linear_tc2_kernel / linear_tc_kernel (tcgen05)", "achieved": pre_tflops,
                        "peak": peaks["tensor_sustained"], "unit": "TFLOP/s", "frac": pre_tflops / peaks["tensor_sustained"],
                        "peak_source": peaks["kind"] + " bf16 GEMM, sustained (the prefill is a seconds-long power-capped run)",
                        "peak_burst": peaks["tensor_burst"], "peak_nominal": TENSOR_NOMINAL_TFLOPS,
                        "frac_nominal": pre_tflops / TENSOR_NOMINAL_TFLOPS,
                        "what": "all prefill flops (products, causal attention, head) over the event-timed prefill",
                        "products_in_pass_tflops": gemm_tflops,
                        "weight_read_floor_ms": weight_floor_ms,
                        "in_pass_us": {c: round(v["us"], 1) for c, v in sorted(pcat.items())},
                        "pass_span_us": round(pre_stamps["span_us"], 1)}
    return {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": f"{name}: {m.name} layers {wl.layer_begin}-{wl.layer_end - 1}"
                               f"{' +embedding' if wl.has_embedding else ''}{' +head' if wl.has_head else ''}, "
                               f"batch {Bn}, prompt {T}, decode {S}"
                               + (f", {n_sh} shards in sequence, {MB} micro-batches, schedule {args.schedule}" if n_sh > 1 or MB > 1 else ""),
                   "parallelism": "replicas" if world > 1 else "single",
                   "l2": "no flush: each step streams %.2f GB of weights, far more than the 126 MB L2" % (linear_weight_bytes(wl) / 1e9)},
        "prefill_ms": pre_mean,
        "decode_ms_per_step": decode_ms,
        "decode_step_gbs": step_gbs,
        "decode_hbm_frac_of_step": step_gbs / peaks["hbm"],
        "decode_hbm_frac_of_step_nominal": step_gbs / HBM_NOMINAL_GBS,
        "prefill_tflops": pre_tflops,
        "prefill_frac_of_nominal": pre_tflops / TENSOR_NOMINAL_TFLOPS,
        "e2e": {"value": value_e, "unit": UNIT, "prefill_ms": pre_mean_e,
                "h2d_bytes_per_step": int(ids_host.numel() * 4 + (0 if wl.has_head else forced_host.numel() * 4)),
                "d2h_bytes_per_step": int(MB * ((tok_host.numel() * 4 * (S + 1)) if wl.has_head
                                                else (hid_host.numel() + S * row_host.numel()) * 4))},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roofline,
        "roofline_prefill": roofline_prefill,
    }


def cpu_oracle_sample(wl, threads=None, layers=None, decode_steps=2):
    """The oracle as it stands, timed on the host on a bounded sample of the workload: ONE sequence through the
    first `layers` layers of the shard — the full prompt in matrix form, then `decode_steps` KV-cached steps
    (incremental form) at the workload's real context (the cache is filled from the matrix-form pass).  The
    workload's rate is scaled from it: the oracle handles sequences one at a time and layers one after another,
    so a step of the whole batch through all layers costs batch x (all layers / sampled layers) sampled steps."""
    from oracle import decoder as O

    m = wl.model
    if threads:
        torch.set_num_threads(threads)
    nl_all = wl.layer_end - wl.layer_begin
    if layers is None:
        # about 10 TFLOP of matrix-form prefill per sample: ten to twenty seconds of host time with the decode steps
        per_layer = 2.0 * wl.prompt_len * m.layer_params()
        layers = max(1, min(nl_all, int(1.0e13 / per_layer)))
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    host = {"layers": [{k: v.cpu() for k, v in layer_weights(wl.cfg, m, wl.layer_begin + i, gen_dev).items()} for i in range(layers)]}
    if wl.has_embedding:
        host["tok_embedding"] = weight_tensor(wl.cfg, m, "tok_embedding", device=gen_dev).cpu()
    ids = prompt_ids(wl.cfg, 1, wl.prompt_len, m.vocab)[0]
    forced = forced_decode_ids(wl.cfg, 1, decode_steps, m.vocab)[:, 0]
    t0 = time.perf_counter()
    x = O.embed(ids, host["tok_embedding"]) if wl.has_embedding else torch.zeros(wl.prompt_len, m.d_model)
    inc = O.IncrementalShard(m, host, wl.layer_begin, wl.layer_begin + layers)
    for li in range(layers):
        x, k, v = O.layer_forward_full(x, host["layers"][li], m, return_kv=True)
        inc.k_cache[li] = list(k)                      # the prompt's keys / values become the step form's cache
        inc.v_cache[li] = list(v)
    inc.pos = wl.prompt_len
    t1 = time.perf_counter()
    step_in = (lambda t: {"token": int(t)}) if wl.has_embedding else (lambda t: {"hidden_in": torch.zeros(m.d_model)})
    for t in forced.tolist():
        inc.step(**step_in(t))
    t2 = time.perf_counter()
    scale = nl_all / layers
    step_s = (t2 - t1) / decode_steps                  # one sequence, `layers` layers, context >= prompt_len
    batch_all = wl.batch * wl.micro_batches
    return {"value": 1.0 / (step_s * scale), "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "prefill_ms": (t1 - t0) * 1e3 * scale * batch_all, "sample_seconds": t2 - t0,
            "measured": {"prefill_ms_one_sequence_sampled_layers": (t1 - t0) * 1e3, "decode_ms_per_step_one_sequence_sampled_layers": step_s * 1e3},
            "sample": f"one sequence of the workload through {layers} of its {nl_all} layers: the full {wl.prompt_len}-token prefill "
                      f"(matrix form) once, then {decode_steps} KV-cached decode steps (incremental form) at context "
                      f"{wl.prompt_len}+; tokens/s and prefill ms are scaled to all {nl_all} layers and {batch_all} sequences "
                      f"(x{scale:g} layers; the oracle runs sequences one at a time, so tokens/s does not grow with the batch)"}


def run_reference(args):
    """The CPU oracle timed on the host cores on the same workload (a bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    wl = WORKLOADS[args.workload]
    vals, pres, secs = [], [], []
    t_all = time.perf_counter()
    sample = None
    n_warm = min(args.warmup, 1)
    for i in range(n_warm + args.steps):
        if i > n_warm and time.perf_counter() - t_all > 150:
            break                                   # keep the whole run within a few minutes
        sample = cpu_oracle_sample(wl)
        if i >= n_warm:
            vals.append(sample["value"])
            pres.append(sample["prefill_ms"])
            secs.append(sample["sample_seconds"])
    v = statistics.mean(vals)
    m = wl.model
    return {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
        "warmup": n_warm, "ms_per_step": 1e3 * statistics.mean(secs),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {m.name} layers {wl.layer_begin}-{wl.layer_end - 1}, batch {wl.batch}, "
                               f"prompt {wl.prompt_len}, decode {wl.decode_steps}",
                   "step": "ms_per_step is the measured host time of one bounded sample (see cpu_baseline.sample), not of the whole workload"},
        "prefill_ms": statistics.mean(pres),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": sample["cores"], "kind": "oracle", "sample": sample["sample"],
                         "measured": sample["measured"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg4", choices=sorted(WORKLOADS))
    ap.add_argument("--also", default=None,
                    help="comma-separated workloads measured after the main one with a few steps each and reported as "
                         f"sub-records (default at one GPU with the default workload: {DEFAULT_ALSO}; 'none' = skip)")
    ap.add_argument("--also-steps", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--schedule", default="no_bubbles", choices=["sequential", "bubbles", "no_bubbles"],
                    help="micro-batch schedule of a multi-shard workload: one pass at a time, or the paper's two "
                         "pipelined schedules with one stream per shard")
    ap.add_argument("--profile", action="store_true",
                    help="short run for an ncu capture: 1 warm-up pass, 1 timed pass, no e2e / step-timing / CPU legs")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps (profile runs)")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt length (profile runs only)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profile runs only)")
    ap.add_argument("--layers", type=int, default=0, help="keep only the first LAYERS layers of every shard (profile runs only)")
    ap.add_argument("--model-layers", type=int, default=0,
                    help="run a model of only this many layers of the workload's shapes, output layer included (profile runs only)")
    args = ap.parse_args()
    if (args.prompt_len or args.batch or args.layers or args.model_layers) and not args.profile:
        ap.error("--prompt-len / --batch / --layers / --model-layers change the workload and are only accepted together with --profile")

    from paper_2405_14371_b200 import replicas
    relaunch = replicas.launch_plan(args.gpus, os.environ, sys.argv)
    if relaunch is not None and args.impl == "ours":
        os.execvp(relaunch[0], relaunch)          # N ranks under torch.distributed.run; does not return

    if args.profile:
        args.warmup, args.steps = 1, 1
    elif args.impl == "ours":
        args.warmup = max(args.warmup, 3)

    if args.impl == "reference":
        out = run_reference(args)
    else:
        dist_ctx = replicas.setup("nccl")
        out = run_ours(args, args.workload, args.steps, args.warmup, dist_ctx, with_clocks=True)
        single = out is not None and out.get("n_gpus") == 1 and not args.profile
        also = args.also if args.also is not None else (DEFAULT_ALSO if args.workload == "cfg4" else "none")
        if single and also != "none":
            out["other_workloads"] = {}
            for name in [a for a in also.split(",") if a and a != args.workload]:
                sub = run_ours(args, name, args.also_steps, 3, dist_ctx, with_clocks=True)
                for k in ("metric", "unit", "n_gpus", "higher_is_better", "scaling", "vs_baseline", "dtype", "data"):
                    sub.pop(k, None)
                out["other_workloads"][name] = sub
        if single and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_oracle_sample(WORKLOADS[args.workload])
    if out is not None:
        print(json.dumps(out))
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and args.impl == "ours":
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

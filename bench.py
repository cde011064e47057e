#!/usr/bin/env python
"""Benchmark of the shard forward pass: prefill latency and KV-cached decode throughput.

One "step" is one pass of the whole hot path over one batch: a prefill of the prompt followed by
all decode steps of the workload (default: the Llama-2-7B layers-0..7 shard, batch 1, 128-token
prompt, 128 decode steps).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg1] [--impl ours|reference]

With N > 1 (launched under torch.distributed.run) every rank runs an independent replica of the
workload on its own GPU ("replicas only": the path has no cross-GPU exchange); the time is the
maximum over ranks and the value the sum of all ranks' tokens over that time.
"""
from __future__ import annotations

import argparse
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

from workload import WORKLOADS, forced_decode_ids, prompt_ids, shard_weights  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
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
        # samples under load: the upper half of the observed clocks
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _dist_setup(n_gpus: int):
    from paper_2405_14371_b200 import replicas
    return replicas.setup("nccl")


def _barrier(world):
    from paper_2405_14371_b200 import replicas
    replicas.barrier(world)


def _max_over_ranks(x: float, world) -> float:
    from paper_2405_14371_b200 import replicas
    return replicas.max_over_ranks(x, world)


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


def run_ours(args):
    from paper_2405_14371_b200 import binding as B

    rank, local, world = _dist_setup(args.gpus)
    wl = WORKLOADS[args.workload]
    if args.layers:
        import dataclasses
        wl = dataclasses.replace(wl, layer_end=min(wl.layer_end, wl.layer_begin + args.layers * wl.n_shards))
    m = wl.model
    Bn, T, S = (args.batch or wl.batch), (args.prompt_len or wl.prompt_len), (args.decode_steps or wl.decode_steps)
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

        for _ in range(args.warmup):
            one_step(False)
            if not args.profile:
                one_step(True)
        stream.synchronize()

        def timed(e2e: bool):
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
            _barrier(world)
            n0 = sum(x.es_shard_launch_count() for x in shards)
            for k in range(args.steps):
                one_step(e2e, evs[k])
            stream.synchronize()
            _barrier(world)
            n1 = sum(x.es_shard_launch_count() for x in shards)
            pre = [e[0].elapsed_time(e[1]) for e in evs]
            dec = [e[1].elapsed_time(e[2]) for e in evs]
            return pre, dec, n1 - n0

        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        pre, dec, launches = timed(False)
        if args.profile:
            # short run for a profiler capture: one timed pass, nothing else (not a bench value)
            sampler.stop()
            stream.synchronize()
            if rank == 0:
                print(json.dumps({"profile_run": True, "workload": args.workload, "batch": Bn, "prompt_len": T, "decode_steps": S,
                                  "prefill_ms": sum(pre) / len(pre), "decode_ms_per_step": sum(dec) / (S * len(dec)),
                                  "gpu_launches": int(launches)}))
            return None
        pre_e, dec_e, _ = timed(True)
        clocks = sampler.stop() if rank == 0 else None

        # dominant kernel: the weight-streaming linear kernel, timed launch by launch with CUDA events
        torch.cuda.synchronize(dev)
        with torch.cuda.stream(sh.stream):
            sh.es_shard_prefill(ids_dev[0], None, Bn, T, slots[0])
            src = sh.es_shard_handoff()[2] if (wl.has_head and n_sh == 1) else cur_ids[0]
            sh.es_shard_set_kernel_timing(True)
            torch.cuda._sleep(4_000_000)           # let the host run ahead so the event pairs bracket only the kernels
            for _ in range(min(4, S)):
                sh.es_shard_decode_step(src, None, Bn, slots[0])
            t = sh.es_shard_kernel_timing()
            sh.es_shard_set_kernel_timing(False)
        kt = {"gbs": t["bytes"] / (t["ms"] / 1e3) / 1e9, "launches": t["launches"],
              "avg_us": 1e3 * t["ms"] / t["launches"], "bytes_per_launch": t["bytes"] / t["launches"]}
        for x in shards:
            x.es_shard_device_status()

    dec_total = _max_over_ranks(sum(dec), world)
    pre_mean = _max_over_ranks(sum(pre) / len(pre), world)
    dec_total_e = _max_over_ranks(sum(dec_e), world)
    pre_mean_e = _max_over_ranks(sum(pre_e) / len(pre_e), world)
    total_ms = _max_over_ranks(sum(pre) + sum(dec), world)
    if rank != 0:
        return None

    tokens = MB * Bn * S * args.steps * world
    value = tokens / (dec_total / 1e3)
    value_e = tokens / (dec_total_e / 1e3)
    ctx_avg = T + (S + 1) / 2.0
    step_bytes = MB * algorithmic_decode_bytes(wl, ctx_avg)     # every micro-batch pass re-streams the weights
    peak, peak_kind = _peaks()
    decode_ms = dec_total / (S * args.steps)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {m.name} layers {wl.layer_begin}-{wl.layer_end - 1}"
                               f"{' +embedding' if wl.has_embedding else ''}{' +head' if wl.has_head else ''}, "
                               f"batch {Bn}, prompt {T}, decode {S}"
                               + (f", {n_sh} shards in sequence, {MB} micro-batches, schedule {args.schedule}" if n_sh > 1 or MB > 1 else ""),
                   "parallelism": "replicas" if world > 1 else "single",
                   "l2": "no flush: each step streams %.2f GB of weights, far more than the 126 MB L2" % (linear_weight_bytes(wl) / 1e9)},
        "prefill_ms": pre_mean,
        "decode_ms_per_step": decode_ms,
        "decode_hbm_frac_of_step": step_bytes / (decode_ms / 1e3) / 1e9 / peak,
        "prefill_tflops": MB * prefill_flops(wl) / (pre_mean / 1e3) / 1e12,
        "e2e": {"value": value_e, "unit": UNIT, "prefill_ms": pre_mean_e,
                "h2d_bytes_per_step": int(ids_host.numel() * 4 + (0 if wl.has_head else forced_host.numel() * 4)),
                "d2h_bytes_per_step": int(MB * ((tok_host.numel() * 4 * (S + 1)) if wl.has_head
                                                else (hid_host.numel() + S * row_host.numel()) * 4))},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": ("linear_stream_kernel" if Bn <= 2 else "linear_stream_mma_kernel / linear_stream_mma_ks_kernel"), "achieved": kt["gbs"], "peak": peak,
                     "unit": "GB/s", "frac": kt["gbs"] / peak, "peak_source": peak_kind + " copy bandwidth",
                     "launches_timed": kt["launches"], "avg_launch_us": kt["avg_us"],
                     "bytes_per_launch": kt["bytes_per_launch"], "traffic": TRAFFIC_PER_LAUNCH.get(args.workload)},
    }
    return out


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel (average over the four
# products of a layer), from the ncu capture summarised in profiles/linear_stream_kernel_cfg1_decode.md;
# set a workload's entry to None when that kernel changes until the counters are taken again.
TRAFFIC_PER_LAUNCH = {"cfg1": 105.0e6}


def cpu_oracle_sample(wl, threads=None):
    """The oracle as it stands, timed on the host on a bounded sample of the workload."""
    from oracle import decoder as O

    m = wl.model
    if threads:
        torch.set_num_threads(threads)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = shard_weights(wl.cfg, m, wl.layer_begin, wl.layer_end, device=dev)
    host = {k: v.cpu() for k, v in w.items() if k != "layers"}
    host["layers"] = [{k: v.cpu() for k, v in lw.items()} for lw in w["layers"]]
    del w
    Tp, Sd = 8, 3
    ids = prompt_ids(wl.cfg, 1, wl.prompt_len, m.vocab)[0]
    forced = forced_decode_ids(wl.cfg, 1, Sd, m.vocab)[:, 0]
    t0 = time.perf_counter()
    if wl.has_embedding:
        x, _ = O.shard_forward_full(m, host, wl.layer_begin, wl.layer_end, ids=ids)
    else:
        x, _ = O.shard_forward_full(m, host, wl.layer_begin, wl.layer_end,
                                    hidden_in=torch.zeros(wl.prompt_len, m.d_model))
    t1 = time.perf_counter()
    inc = O.IncrementalShard(m, host, wl.layer_begin, wl.layer_end)
    step_in = (lambda t: {"token": int(t)}) if wl.has_embedding else (lambda t: {"hidden_in": torch.zeros(m.d_model)})
    for t in ids[:Tp].tolist():
        inc.step(**step_in(t))
    t2 = time.perf_counter()
    for t in forced.tolist():
        inc.step(**step_in(t))
    t3 = time.perf_counter()
    return {"value": Sd / (t3 - t2), "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "prefill_ms": (t1 - t0) * 1e3,
            "sample": f"one sequence of the workload: full {wl.prompt_len}-token prefill (matrix form) timed once; "
                      f"decode rate over {Sd} KV-cached steps after an {Tp}-token context (incremental form)"}


def run_reference(args):
    """The CPU oracle timed on the host cores on the same workload (bounded sample per step)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    wl = WORKLOADS[args.workload]
    vals, pres = [], []
    t_all = time.perf_counter()
    sample = None
    for i in range(args.warmup + args.steps):
        if i >= 1 and time.perf_counter() - t_all > 150:
            break                                   # keep the whole run within a few minutes
        sample = cpu_oracle_sample(wl)
        if i >= min(args.warmup, 1):
            vals.append(sample["value"])
            pres.append(sample["prefill_ms"])
    if not vals:
        vals, pres = [sample["value"]], [sample["prefill_ms"]]
    v = statistics.mean(vals)
    m = wl.model
    return {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
        "warmup": min(args.warmup, 1), "ms_per_step": statistics.mean(pres) + 1e3 * wl.decode_steps / v,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {m.name} layers {wl.layer_begin}-{wl.layer_end - 1}, batch {wl.batch}, "
                               f"prompt {wl.prompt_len}, decode {wl.decode_steps}"},
        "prefill_ms": statistics.mean(pres),
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": sample["cores"], "kind": "oracle", "sample": sample["sample"]},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg1", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--schedule", default="no_bubbles", choices=["sequential", "bubbles", "no_bubbles"],
                    help="micro-batch schedule of a multi-shard workload: one pass at a time, or the paper's two "
                         "pipelined schedules with one stream per shard")
    ap.add_argument("--profile", action="store_true",
                    help="short run for an ncu capture: 1 warm-up pass, 1 timed pass, no e2e / kernel-timing / CPU legs")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps (profile runs)")
    ap.add_argument("--prompt-len", type=int, default=0, help="override the workload's prompt length (profile runs only)")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profile runs only)")
    ap.add_argument("--layers", type=int, default=0, help="keep only the first LAYERS layers of every shard (profile runs only)")
    args = ap.parse_args()
    if (args.prompt_len or args.batch or args.layers) and not args.profile:
        ap.error("--prompt-len / --batch / --layers change the workload and are only accepted together with --profile")
    if args.profile:
        args.warmup, args.steps = 1, 1
    else:
        args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        out = run_reference(args)
    else:
        out = run_ours(args)
        if out is not None and out["n_gpus"] == 1 and not args.no_cpu_baseline:
            torch.cuda.empty_cache()
            out["cpu_baseline"] = cpu_oracle_sample(WORKLOADS[args.workload])
    if out is not None:
        print(json.dumps(out))
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and args.impl == "ours":
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

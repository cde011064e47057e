"""Micro-batched pipeline over several shards of one model (Sec. "Pipeline Execution Optimization").

The paper runs its shards on different devices and keeps them busy by cutting a batch into
micro-batches: while shard j works on micro-batch m, shard j-1 already works on micro-batch m+1.
It describes two schedules of the token iterations:

* "bubbles": iteration t+1 of any micro-batch starts only after every micro-batch has finished
  iteration t (the devices idle while the last micro-batch drains);
* "no_bubbles": a micro-batch starts its next iteration as soon as its own token has come back
  from the last shard.

Here all shards live on one GPU.  "sequential" enqueues every pass on one stream (one pass at a
time).  The two pipelined schedules give every shard its own stream and express exactly the paper's
dependencies as events, so passes of different micro-batches on different shards overlap on the
device (one fills the other's kernel ramps and tails).  This module only orders calls of the shard
library: every step of a pass still runs in its kernels, and all three schedules produce the same
bits.

`plan()` is pure host logic (no GPU needed): the passes in enqueue order, each with the passes it
must wait for.
"""
from __future__ import annotations

from typing import Iterator, List, NamedTuple, Optional, Sequence, Tuple

SCHEDULES = ("sequential", "bubbles", "no_bubbles")


class Pass(NamedTuple):
    shard: int
    micro_batch: int
    iteration: int          # 0 = prefill, 1.. = decode steps


def plan(n_shards: int, micro_batches: int, iterations: int, schedule: str) -> Iterator[Tuple[Pass, List[Pass]]]:
    """Passes in enqueue order with their dependencies on passes of OTHER streams.

    Passes on one shard run in enqueue order (a stream), which already orders the uses of its KV slots.
    Dependencies: the activation from the previous shard; for the first shard, the token the last
    shard produced for this micro-batch in the previous iteration; the consumer of this shard's
    previous output (the handoff tensor is a view of a buffer the next pass overwrites); and, under
    "bubbles", the end of the previous iteration.
    """
    if schedule not in SCHEDULES:
        raise ValueError(f"unknown schedule {schedule!r}")
    last = n_shards - 1
    previous: List[Optional[Pass]] = [None] * n_shards          # previous pass enqueued on each shard
    for it in range(iterations):
        for mb in range(micro_batches):
            for s in range(n_shards):
                p = Pass(s, mb, it)
                deps: List[Pass] = []
                if schedule != "sequential":
                    if s > 0:
                        deps.append(Pass(s - 1, mb, it))
                    elif it > 0 and last > 0:
                        deps.append(Pass(last, mb, it - 1))
                    prev = previous[s]
                    if prev is not None and s < last:
                        deps.append(Pass(s + 1, prev.micro_batch, prev.iteration))
                    if schedule == "bubbles" and it > 0 and s == 0 and last > 0:
                        deps.append(Pass(last, micro_batches - 1, it - 1))
                previous[s] = p
                yield p, [d for d in dict.fromkeys(deps) if d.shard != s]


class ShardPipeline:
    """Runs micro-batches through shards under one of the schedules.

    shards: binding.Shard objects covering consecutive layer ranges, the first holding the embedding.
    For the pipelined schedules each shard must have been created on its own stream.  Every
    micro-batch owns the KV slots `slots[mb]` in every shard.
    """

    def __init__(self, shards: Sequence, slots: Sequence[Sequence[int]], batch: int, schedule: str = "no_bubbles"):
        import torch

        if schedule not in SCHEDULES:
            raise ValueError(f"unknown schedule {schedule!r}")
        self.torch = torch
        self.shards = list(shards)
        self.slots = [list(s) for s in slots]
        self.batch = batch
        self.schedule = schedule
        self.streams = [s.stream for s in self.shards]
        if schedule != "sequential" and len({int(st.cuda_stream) for st in self.streams}) != len(self.streams):
            raise ValueError("pipelined schedules need one stream per shard")
        self.has_head = self.shards[-1].layer_end == self.shards[-1].desc.n_layers_total
        dev = self.streams[0].device
        self.tokens = torch.zeros(len(self.slots), batch, dtype=torch.int32, device=dev)   # token fed to the first shard
        self.events = {}
        self.iteration = 0
        self.outputs = [None] * len(self.slots)        # (hidden, logits, next_ids) views of the last shard, per micro-batch

    def _run(self, iterations: int, prompt_len: int, ids=None, forced=None, on_output=None):
        torch = self.torch
        n_sh, n_mb = len(self.shards), len(self.slots)
        first_it = self.iteration
        for p, deps in plan(n_sh, n_mb, first_it + iterations, self.schedule):
            if p.iteration < first_it:
                continue
            st = self.streams[p.shard]
            for d in deps:
                ev = self.events.get(d)
                if ev is not None:
                    st.wait_event(ev)
            shard = self.shards[p.shard]
            with torch.cuda.stream(st):
                hidden = None if p.shard == 0 else self.shards[p.shard - 1].es_shard_handoff()[0]
                if p.iteration == 0:
                    shard.es_shard_prefill(ids[p.micro_batch] if p.shard == 0 else None, hidden, self.batch, prompt_len,
                                           self.slots[p.micro_batch])
                else:
                    if p.shard == 0 and forced is not None:
                        self.tokens[p.micro_batch].copy_(forced[p.iteration - 1, p.micro_batch], non_blocking=True)
                    shard.es_shard_decode_step(self.tokens[p.micro_batch] if p.shard == 0 else None, hidden, self.batch,
                                               self.slots[p.micro_batch])
                if p.shard == n_sh - 1:
                    out = shard.es_shard_handoff()
                    if self.has_head:
                        self.tokens[p.micro_batch].copy_(out[2], non_blocking=True)      # greedy feedback stays on the device
                    self.outputs[p.micro_batch] = out
                    if on_output is not None:
                        on_output(p, out)
                if self.schedule != "sequential":
                    ev = torch.cuda.Event()
                    ev.record(st)
                    self.events[p] = ev
        self.iteration = first_it + iterations
        # events older than one iteration are never waited for again
        keep = self.iteration - 2
        self.events = {k: v for k, v in self.events.items() if k.iteration >= keep}

    def prefill(self, ids, prompt_len: int, on_output=None) -> None:
        """ids: [micro_batches, batch, prompt_len] int32 on the device."""
        if self.iteration != 0:
            raise RuntimeError("prefill must be the first call (create a new pipeline to start over)")
        self._run(1, prompt_len, ids=ids, on_output=on_output)

    def decode(self, steps: int, forced=None, on_output=None) -> None:
        """`steps` token iterations.  forced: [>= steps done so far, micro_batches, batch] int32 device tensor of
        teacher-forced inputs indexed by decode step, or None to feed the last shard's greedy token back."""
        if self.iteration == 0:
            raise RuntimeError("decode before prefill")
        if forced is None and not self.has_head:
            raise RuntimeError("the last shard has no LM head: pass forced token ids")
        self._run(steps, 0, forced=forced, on_output=on_output)

    def join(self, stream) -> None:
        """Makes `stream` wait for everything enqueued so far."""
        torch = self.torch
        for st in self.streams:
            if int(st.cuda_stream) != int(stream.cuda_stream):
                ev = torch.cuda.Event()
                ev.record(st)
                stream.wait_event(ev)

    def fork(self, stream) -> None:
        """Makes every shard stream wait for what `stream` holds now."""
        torch = self.torch
        ev = torch.cuda.Event()
        ev.record(stream)
        for st in self.streams:
            if int(st.cuda_stream) != int(stream.cuda_stream):
                st.wait_event(ev)

"""One shard per device: the deployment of Sec. "Collaborative inference" over torch.distributed.

Rank r of the group owns shard r (a contiguous layer range; rank 0 holds the embedding and is the paper's
source node, the last rank holds the output layer).  A pass of one micro-batch travels rank 0 -> 1 -> ... ->
last as point-to-point messages: the activation of a shard's last layer (fp32 [B, T, d_model] after a prefill,
[B, d_model] after a decode step) goes to the next rank, and the token ids the last rank produced go back to
rank 0, which feeds them into the next iteration (Eq. 4's return hop).  There is no collective on the data path.

Every message is received into a buffer the CONSUMER owns (preallocated per micro-batch), and the consumer's
shard then reads its own memory; nothing reads a peer's memory in place.  Sends are non-blocking, so a rank can
start on the next micro-batch while the previous one is still on the wire: with several micro-batches the ranks
work concurrently without any global step (the paper's "no bubbles" schedule falls out of the data dependencies;
its "bubbles" variant adds a barrier per iteration).

Ordering without tags.  NCCL matches point-to-point messages of a pair of ranks in issue order and runs a
communicator's operations one after the other, so two rules keep the flow free of deadlock there as well as over
gloo: both ends of every link walk the micro-batches in the same order, and the return hop (tokens, last rank ->
rank 0) has a communicator of its own.  With a single communicator rank 0 would queue the activations of all
micro-batches before its first token receive while the last rank queues each token send before its next
activation receive: each side's queue would wait for an operation the other side has not reached.

This module only moves tensors and orders calls: every step of a pass runs in the shard library's kernels.  The
`shard` argument is any object with the binding's `es_shard_prefill / es_shard_decode_step / es_shard_handoff`
methods.  Over NCCL the tensors live on the rank's GPU; over gloo on the CPU (the multi-process tests run there,
with a host stand-in for the shard object).
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch
import torch.distributed as dist

TAG_ACT = 1        # activation of a micro-batch, previous rank -> this rank
TAG_TOK = 2        # token ids of a micro-batch, last rank -> rank 0


class PipelineStage:
    """The part of a multi-device run that one rank executes."""

    def __init__(self, shard, d_model: int, micro_batches: int, batch: int, slots: Sequence[Sequence[int]],
                 device: torch.device, schedule: str = "no_bubbles", group=None):
        if schedule not in ("bubbles", "no_bubbles"):
            raise ValueError(f"unknown schedule {schedule!r}")
        if len(slots) != micro_batches or any(len(s) != batch for s in slots):
            raise ValueError("slots must hold one list of `batch` KV slots per micro-batch")
        self.shard, self.d, self.MB, self.B = shard, d_model, micro_batches, batch
        self.slots = [list(s) for s in slots]
        self.device, self.schedule, self.group = device, schedule, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.first, self.last = self.rank == 0, self.rank == self.world - 1
        # the return hop's own communicator (a collective call: every rank of the group constructs its stage)
        self.group_back = None
        if self.world > 1:
            ranks = list(range(dist.get_world_size())) if group is None else dist.get_process_group_ranks(group)
            self.group_back = dist.new_group(ranks=ranks)
        self._pending: List = []              # send requests in flight (their tensors are kept alive with them)
        self._tok_in = [torch.empty(batch, dtype=torch.int32, device=device) for _ in range(micro_batches)]
        self._row_in = [torch.empty(batch, 1, d_model, dtype=torch.float32, device=device) for _ in range(micro_batches)]
        self._act_in: List[Optional[torch.Tensor]] = [None] * micro_batches     # prefill activations, sized on first use

    # -- plumbing ----------------------------------------------------------------------------------
    def _link(self, tag: int):
        return self.group_back if tag == TAG_TOK else self.group

    def _send(self, t: torch.Tensor, dst: int, tag: int, mb: int) -> None:
        t = t.contiguous().clone()            # the handoff view is overwritten by this shard's next pass
        self._pending.append((dist.isend(t, dst, group=self._link(tag), tag=tag * 4096 + mb), t))

    def _recv(self, buf: torch.Tensor, src: int, tag: int, mb: int) -> torch.Tensor:
        dist.recv(buf, src, group=self._link(tag), tag=tag * 4096 + mb)
        return buf

    def _reap(self) -> None:
        keep = []
        for req, t in self._pending:
            if not req.is_completed():
                keep.append((req, t))
        self._pending = keep

    def flush(self) -> None:
        """Waits until every message this rank has sent is delivered."""
        for req, _ in self._pending:
            req.wait()
        self._pending = []

    def _forward(self, mb: int, out) -> Optional[torch.Tensor]:
        """What leaves this rank after a pass of micro-batch mb; returns the tokens on the last rank."""
        hidden, _logits, next_ids = out
        if not self.last:
            self._send(hidden, self.rank + 1, TAG_ACT, mb)
            return None
        if next_ids is None:                             # a last shard without the output layer returns no tokens
            return None
        # the handoff tensors are views of buffers the shard's next pass overwrites: copy before moving on
        if self.world > 1:
            self._send(next_ids, 0, TAG_TOK, mb)
        else:
            self._tok_in[mb].copy_(next_ids)             # single rank: the tokens are already where rank 0 reads them
        return next_ids.clone()

    # -- the two phases ----------------------------------------------------------------------------
    def prefill(self, ids: Optional[Sequence[torch.Tensor]], T: int) -> List[Optional[torch.Tensor]]:
        """One prefill pass per micro-batch.  ids: on rank 0 a list of int32 [B, T] tensors (one per micro-batch),
        elsewhere None.  Returns, per micro-batch, the first generated tokens on the last rank (None elsewhere)."""
        out: List[Optional[torch.Tensor]] = []
        for mb in range(self.MB):
            if self.first:
                self.shard.es_shard_prefill(ids[mb], None, self.B, T, self.slots[mb])
            else:
                if self._act_in[mb] is None or self._act_in[mb].shape[1] != T:
                    self._act_in[mb] = torch.empty(self.B, T, self.d, dtype=torch.float32, device=self.device)
                x = self._recv(self._act_in[mb], self.rank - 1, TAG_ACT, mb)
                self.shard.es_shard_prefill(None, x, self.B, T, self.slots[mb])
            out.append(self._forward(mb, self.shard.es_shard_handoff()))
            self._reap()
        if self.schedule == "bubbles":
            dist.barrier(group=self.group)
        return out

    def decode(self, steps: int, forced: Optional[torch.Tensor] = None) -> Optional[torch.Tensor]:
        """`steps` autoregressive iterations over every micro-batch.  Rank 0 feeds each micro-batch the tokens the
        last rank returned for it — the prefill's first, then each step's — and finally receives the last step's
        tokens too, so the source node ends up with everything that was generated: returns int32
        [steps + 1, micro_batches, B] on rank 0 (row 0 = the tokens of the prefill), None elsewhere.
        With `forced` (int32 [steps, micro_batches, B]: the last rank holds no output layer) rank 0 feeds those ids
        instead, no tokens travel, and nothing is returned."""
        gen = None
        if self.first and forced is None:
            gen = torch.empty(steps + 1, self.MB, self.B, dtype=torch.int32, device=self.device)

        def token_in(step: int, mb: int) -> torch.Tensor:
            # tokens produced by pass `step` (0 = prefill) of micro-batch mb, as they reach rank 0
            if self.world > 1:
                self._recv(self._tok_in[mb], self.world - 1, TAG_TOK, mb)
            gen[step, mb].copy_(self._tok_in[mb])
            return self._tok_in[mb]

        for s in range(steps):
            for mb in range(self.MB):
                if self.first:
                    tok = forced[s, mb].to(self.device) if forced is not None else token_in(s, mb)
                    self.shard.es_shard_decode_step(tok, None, self.B, self.slots[mb])
                else:
                    x = self._recv(self._row_in[mb], self.rank - 1, TAG_ACT, mb)
                    self.shard.es_shard_decode_step(None, x, self.B, self.slots[mb])
                out = self.shard.es_shard_handoff()
                if forced is not None and self.last:
                    continue                              # a headless last shard: its activation is the product
                self._forward(mb, out)
                self._reap()
            if self.schedule == "bubbles":
                dist.barrier(group=self.group)
        if gen is not None:
            for mb in range(self.MB):
                token_in(steps, mb)
        self.flush()
        return gen

    def prefill_and_decode(self, ids: Optional[Sequence[torch.Tensor]], T: int, steps: int) -> Optional[torch.Tensor]:
        """A whole greedy generation: prefill, then `steps` decode iterations.  Returns what decode() returns."""
        self.prefill(ids, T)
        return self.decode(steps)

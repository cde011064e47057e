"""One shard per rank over gloo on the CPU: the message flow of the multi-device pipeline (activations forward,
tokens back to rank 0, several micro-batches in flight, both schedules).  The shard object is a host stand-in built
on the oracle's incremental form, so what is tested here is the plumbing; the kernels are tested elsewhere."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _tiny3():
    """Three small layers (one per rank at most), two query heads on one KV head."""
    from workload import ModelShape
    return ModelShape("tiny3", 3, 64, 2, 1, 32, 96, 50)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


class HostShard:
    """The three calls of the shard binding, computed by the oracle one position at a time."""

    def __init__(self, model, weights, begin, end):
        from oracle import decoder as O
        self.O, self.m, self.w, self.begin, self.end = O, model, weights, begin, end
        self.seq = {}                                   # slot -> IncrementalShard
        self.out = None

    def _run(self, slots, rows_of):
        hs, ls = [], []
        for b, slot in enumerate(slots):
            sh = self.seq[slot]
            h_rows, logits = [], None
            for kw in rows_of(b):
                h, logits = sh.step(**kw)
                h_rows.append(h)
            hs.append(torch.stack(h_rows))
            ls.append(logits)
        hidden = torch.stack(hs).float()
        if self.end == self.m.n_layers:
            logits = torch.stack(ls).float()
            self.out = (hidden, logits, self.O.greedy(logits).to(torch.int32))
        else:
            self.out = (hidden, None, None)

    def es_shard_prefill(self, ids, hidden_in, B, T, slots):
        for slot in slots:
            self.seq[slot] = self.O.IncrementalShard(self.m, self.w, self.begin, self.end)
        if ids is not None:
            self._run(slots, lambda b: [{"token": int(t)} for t in ids[b].tolist()])
        else:
            self._run(slots, lambda b: [{"hidden_in": hidden_in[b, t]} for t in range(T)])

    def es_shard_decode_step(self, ids, hidden_in, B, slots):
        if ids is not None:
            self._run(slots, lambda b: [{"token": int(ids[b])}])
        else:
            self._run(slots, lambda b: [{"hidden_in": hidden_in[b, 0]}])

    def es_shard_handoff(self):
        return self.out


def _worker(rank, world, port, schedule, cuts, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2405_14371_b200.stage import PipelineStage
    from workload import prompt_ids, shard_weights

    torch.set_num_threads(1)
    dist.init_process_group("gloo")
    m = _tiny3()
    begin, end = cuts[rank], cuts[rank + 1]
    w = shard_weights(0, m, begin, end, device="cpu")
    MB, Bn, T, S = 3, 2, 5, 4
    slots = [[mb * Bn + b for b in range(Bn)] for mb in range(MB)]
    stage = PipelineStage(HostShard(m, w, begin, end), m.d_model, MB, Bn, slots, torch.device("cpu"), schedule)
    ids = prompt_ids(0, MB * Bn, T, m.vocab, seed=3).reshape(MB, Bn, T)
    gen = stage.prefill_and_decode([ids[mb] for mb in range(MB)] if rank == 0 else None, T, S)
    if rank == 0:
        out.put(gen.tolist())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,cuts,schedule", [(2, (0, 1, 3), "no_bubbles"), (3, (0, 1, 2, 3), "bubbles"), (2, (0, 2, 3), "bubbles")])
def test_ranks_pass_activations_forward_and_tokens_back(world, cuts, schedule):
    from oracle import decoder as O
    from workload import prompt_ids, shard_weights

    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, schedule, cuts, out)) for r in range(world)]
    for p in procs:
        p.start()
    gen = torch.tensor(out.get(timeout=300))            # [S + 1, MB, B] as received by rank 0
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    m = _tiny3()
    w = shard_weights(0, m, 0, m.n_layers, device="cpu")
    MB, Bn, T, S = 3, 2, 5, 4
    ids = prompt_ids(0, MB * Bn, T, m.vocab, seed=3).reshape(MB, Bn, T)
    for mb in range(MB):
        for b in range(Bn):
            want, _, _ = O.generate_greedy(m, w, ids[mb, b], S)
            assert gen[:, mb, b].tolist() == want.tolist()


def test_one_rank_is_the_whole_pipeline():
    """world_size 1: the same object runs prefill and decode with no message at all."""
    import torch.distributed as dist
    from oracle import decoder as O
    from paper_2405_14371_b200.stage import PipelineStage
    from workload import prompt_ids, shard_weights

    os.environ.update(RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    dist.init_process_group("gloo")
    try:
        m = _tiny3()
        w = shard_weights(0, m, 0, m.n_layers, device="cpu")
        ids = prompt_ids(0, 2, 4, m.vocab, seed=4).reshape(1, 2, 4)
        stage = PipelineStage(HostShard(m, w, 0, m.n_layers), m.d_model, 1, 2, [[0, 1]], torch.device("cpu"))
        gen = stage.prefill_and_decode([ids[0]], 4, 3)
        for b in range(2):
            want, _, _ = O.generate_greedy(m, w, ids[0, b], 3)
            assert gen[:, 0, b].tolist() == want.tolist()
    finally:
        dist.destroy_process_group()

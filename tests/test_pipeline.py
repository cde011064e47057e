"""The micro-batch pipeline schedules (Sec. "Pipeline Execution Optimization"): the dependency plan
on the CPU, and on the GPU that all schedules produce the same bits as running the micro-batches one
after the other."""
import itertools

import pytest
import torch

from paper_2405_14371_b200.pipeline import Pass, SCHEDULES, plan


@pytest.mark.parametrize("n_shards,mbs,iters", [(1, 1, 3), (2, 4, 3), (4, 8, 4), (3, 2, 5), (4, 1, 2)])
@pytest.mark.parametrize("schedule", SCHEDULES)
def test_plan_orders_every_pass_after_what_it_needs(n_shards, mbs, iters, schedule):
    seen = []
    for p, deps in plan(n_shards, mbs, iters, schedule):
        assert all(d in seen for d in deps), (p, deps)              # every awaited pass was enqueued before
        assert all(d.shard != p.shard for d in deps)                # same-shard order is the stream's
        seen.append(p)
        if schedule == "sequential":
            assert deps == []
            continue
        if p.shard > 0:
            assert Pass(p.shard - 1, p.micro_batch, p.iteration) in deps                     # the activation
        elif p.iteration > 0 and n_shards > 1:
            assert Pass(n_shards - 1, p.micro_batch, p.iteration - 1) in deps                # its own token
            if schedule == "bubbles":
                assert Pass(n_shards - 1, mbs - 1, p.iteration - 1) in deps                   # the whole previous iteration
    assert sorted(seen) == sorted(Pass(s, m, i) for i, m, s in itertools.product(range(iters), range(mbs), range(n_shards)))
    # per shard, passes appear in (iteration, micro-batch) order: the KV slots of a micro-batch are used in step order
    for s in range(n_shards):
        mine = [(p.iteration, p.micro_batch) for p in seen if p.shard == s]
        assert mine == sorted(mine)


def test_plan_protects_the_handoff_buffer():
    """A shard's next pass overwrites the buffer its previous output lives in, so it must wait for the
    consumer of that output."""
    for p, deps in plan(3, 4, 3, "no_bubbles"):
        if p.shard < 2 and (p.iteration, p.micro_batch) != (0, 0):
            prev_mb, prev_it = (p.micro_batch - 1, p.iteration) if p.micro_batch > 0 else (3, p.iteration - 1)
            assert Pass(p.shard + 1, prev_mb, prev_it) in deps


def test_plan_rejects_unknown_schedule():
    with pytest.raises(ValueError):
        list(plan(2, 2, 2, "zigzag"))


@pytest.mark.gpu
@pytest.mark.parametrize("with_head", [True, False])
def test_schedules_agree_bit_for_bit(with_head):
    from paper_2405_14371_b200 import binding as B
    from paper_2405_14371_b200.pipeline import ShardPipeline
    from tests.helpers import device_weights, slice_weights
    from workload import TINY, prompt_ids, forced_decode_ids

    wd, _ = device_weights(0, TINY, 0, TINY.n_layers)
    T, S, MB = 10, 5, 4
    ids = prompt_ids(0, MB, T, TINY.vocab, seed=17).cuda().reshape(MB, 1, T)
    forced = None if with_head else forced_decode_ids(0, MB, S, TINY.vocab, seed=17).cuda().reshape(S, MB, 1)
    n_layers = 2 if with_head else 1          # without head: a one-layer model prefix cut in ... two shards of one layer
    kw = dict(max_slots=MB, max_seq=T + S, max_tokens=T, max_batch=1, kv_page_tokens=16)

    def run(schedule):
        torch.cuda.synchronize()
        streams = [torch.cuda.Stream() for _ in range(2)]
        if schedule == "sequential":
            streams[1] = streams[0]
        if with_head:
            ranges = [(0, 1), (1, 2)]
            shards = [B.Shard(TINY, a, b, slice_weights(wd, TINY, a, b), stream=st, **kw) for (a, b), st in zip(ranges, streams)]
        else:
            big = TINY.__class__("tiny3", 3, TINY.d_model, TINY.n_heads, TINY.n_kv_heads, TINY.head_dim, TINY.d_ffn, TINY.vocab)
            w3 = {"layers": [wd["layers"][0], wd["layers"][1], wd["layers"][0]], "tok_embedding": wd["tok_embedding"]}
            ranges = [(0, 1), (1, 2)]
            shards = [B.Shard(big, a, b, {"layers": w3["layers"][a:b], **({"tok_embedding": w3["tok_embedding"]} if a == 0 else {})},
                              stream=st, **kw) for (a, b), st in zip(ranges, streams)]
        pipe = ShardPipeline(shards, [[m] for m in range(MB)], 1, schedule)
        got = []

        def keep(p, out):
            got.append((p, [t.clone() if t is not None else None for t in out]))

        pipe.prefill(ids, T, on_output=keep)
        pipe.decode(S, forced=forced, on_output=keep)
        main = torch.cuda.current_stream()
        pipe.join(main)
        torch.cuda.synchronize()
        for sh in shards:
            sh.es_shard_device_status()
            sh.close()
        return sorted(got, key=lambda x: x[0])

    ref = run("sequential")
    assert len(ref) == MB * (S + 1)
    for schedule in ("bubbles", "no_bubbles"):
        got = run(schedule)
        assert [p for p, _ in got] == [p for p, _ in ref]
        for (_, a), (_, b) in zip(ref, got):
            for x, y in zip(a, b):
                assert (x is None) == (y is None)
                if x is not None:
                    assert torch.equal(x, y), schedule


@pytest.mark.gpu
def test_schedules_at_the_13b_shapes_of_the_timed_pipeline():
    """The configuration the benchmark times for the 13B pipeline — four shards, eight micro-batches of one
    sequence, 256-token prompts, one stream per shard with event dependencies — at the 13B layer shapes with two
    layers per shard: both pipelined schedules must reproduce the one-stream order bit for bit, and micro-batches
    0 and 7 must match the oracle (greedy tokens fed back on the device, the oracle teacher-forced with them)."""
    from paper_2405_14371_b200 import binding as B
    from paper_2405_14371_b200.pipeline import ShardPipeline
    from tests.helpers import oracle_streamed, rel_err, report_err, slice_weights
    from workload import LLAMA2_13B, ModelShape, prompt_ids, shard_weights

    full = LLAMA2_13B
    m = ModelShape("llama2-13b-8layers", 8, full.d_model, full.n_heads, full.n_kv_heads, full.head_dim, full.d_ffn, full.vocab)
    n_sh, per, MB, T, S = 4, 2, 8, 256, 6
    wd = shard_weights(3, m, 0, m.n_layers, device="cuda")
    ids = prompt_ids(3, MB, T, m.vocab).cuda().reshape(MB, 1, T)
    kw = dict(max_slots=MB, max_seq=T + S, max_tokens=T, max_batch=1)

    def run(schedule):
        torch.cuda.synchronize()
        first = torch.cuda.Stream()
        streams = [first if schedule == "sequential" else torch.cuda.Stream() for _ in range(n_sh)]
        shards = [B.Shard(m, i * per, (i + 1) * per, slice_weights(wd, m, i * per, (i + 1) * per), stream=streams[i], **kw)
                  for i in range(n_sh)]
        pipe = ShardPipeline(shards, [[mb] for mb in range(MB)], 1, schedule)
        got = {}

        def keep(p, out):
            got[(p.iteration, p.micro_batch)] = [t.clone() for t in out]

        pipe.prefill(ids, T, on_output=keep)
        pipe.decode(S, on_output=keep)
        pipe.join(torch.cuda.current_stream())
        torch.cuda.synchronize()
        for sh in shards:
            sh.es_shard_device_status()
            sh.close()
        return got

    ref = run("sequential")
    assert len(ref) == MB * (S + 1)
    for schedule in ("bubbles", "no_bubbles"):
        got = run(schedule)
        assert got.keys() == ref.keys()
        for key in ref:
            for x, y in zip(ref[key], got[key]):
                assert torch.equal(x, y), (schedule, key)
    for mb in (0, MB - 1):
        fed = torch.stack([ref[(it, mb)][2][0] for it in range(S)]).cpu()              # token produced by iteration it
        seq = torch.cat([ids[mb, 0].cpu(), fed])
        xs, ls = oracle_streamed(m, wd, 0, m.n_layers, [seq], logits_from=T - 1)
        want_h, want_l = xs[0], ls[0]
        assert report_err(f"13B pipeline shapes micro-batch {mb} prefill hidden", rel_err(ref[(0, mb)][0][0], want_h[:T])) < 1e-2
        dec_h = torch.stack([ref[(it, mb)][0][0, 0] for it in range(1, S + 1)])
        assert report_err(f"13B pipeline shapes micro-batch {mb} decode hidden", rel_err(dec_h, want_h[T:])) < 1e-2
        logits = torch.stack([ref[(it, mb)][1][0] for it in range(S + 1)])
        assert report_err(f"13B pipeline shapes micro-batch {mb} logits", rel_err(logits, want_l)) < 1e-2

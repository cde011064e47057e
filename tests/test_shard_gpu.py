"""End-to-end parity of the CUDA shard against the CPU oracle on the tiny configuration, plus the
invariants of the path (split points, batch rows, page map, graphs) and the error paths."""
import os

import pytest
import torch

from oracle import decoder as O
from tests.helpers import device_weights, slice_weights, rel_err, report_err
from workload import TINY, WORKLOADS, prompt_ids, forced_decode_ids

pytestmark = pytest.mark.gpu
TOL = 1e-2          # max|gpu - oracle| / max|oracle| on hidden states and logits


@pytest.fixture(scope="module")
def B():
    from paper_2405_14371_b200 import binding
    return binding


@pytest.fixture(scope="module")
def tiny():
    return device_weights(0, TINY, 0, TINY.n_layers)


def _golden_cfg0():
    path = os.path.join(os.path.dirname(__file__), "golden", "cfg0_greedy.txt")
    out = {}
    for line in open(path):
        if not line.startswith("#"):
            k, *v = line.split()
            out[k] = v
    return int(out["seed"][0]), [int(t) for t in out["tokens"]]


def test_cfg0_greedy_generation_matches_oracle(B, tiny):
    wd, wh = tiny
    wl = WORKLOADS["cfg0"]
    seed, golden_tokens = _golden_cfg0()
    ids = prompt_ids(0, 1, wl.prompt_len, TINY.vocab, seed=seed)
    toks, logits, hidden = O.generate_greedy(TINY, wh, ids[0], wl.decode_steps)
    assert toks.tolist() == golden_tokens

    sh = B.Shard(TINY, 0, 2, wd, max_slots=1, max_seq=32, max_tokens=16)
    sh.es_shard_prefill(ids.cuda(), None, 1, wl.prompt_len, [0])
    h, l, n = sh.es_shard_handoff()
    assert h.shape == (1, 16, 256) and l.shape == (1, 1000) and n.shape == (1,)
    worst_h = rel_err(h[0], hidden[:16])
    worst_l = rel_err(l[0], logits[0])
    got = [int(n[0])]
    for s in range(wl.decode_steps):
        sh.es_shard_decode_step(n, None, 1, [0])       # greedy feedback stays on the device
        h, l, n = sh.es_shard_handoff()
        assert h.shape == (1, 1, 256)
        worst_h = max(worst_h, rel_err(h[0, 0], hidden[16 + s]))
        worst_l = max(worst_l, rel_err(l[0], logits[1 + s]))
        got.append(int(n[0]))
    assert report_err("cfg0 hidden states (prefill and every decode step)", worst_h) < TOL
    assert report_err("cfg0 logits (prefill and every decode step)", worst_l) < TOL
    assert got == golden_tokens
    sh.es_shard_device_status()
    assert sh.es_shard_launch_count() > 0
    sh.close()


@pytest.mark.parametrize("k", [1])
def test_split_point_equals_single_shard(B, tiny, k):
    """[0,k) then [k,L) on the GPU equals [0,L) bitwise (same kernels, same order of operations)."""
    wd, _ = tiny
    ids = prompt_ids(0, 2, 12, TINY.vocab).cuda()
    nxt = forced_decode_ids(0, 2, 3, TINY.vocab).cuda()
    full = B.Shard(TINY, 0, 2, wd, max_slots=2, max_seq=32, max_tokens=24)
    a = B.Shard(TINY, 0, k, slice_weights(wd, TINY, 0, k), max_slots=2, max_seq=32, max_tokens=24)
    b = B.Shard(TINY, k, 2, slice_weights(wd, TINY, k, 2), max_slots=2, max_seq=32, max_tokens=24)
    full.es_shard_prefill(ids, None, 2, 12, [0, 1])
    a.es_shard_prefill(ids, None, 2, 12, [0, 1])
    ha, la, _ = a.es_shard_handoff()
    assert la is None
    b.es_shard_prefill(None, ha, 2, 12, [0, 1])
    hf, lf, nf = full.es_shard_handoff()
    hb, lb, nb = b.es_shard_handoff()
    assert torch.equal(hf, hb) and torch.equal(lf, lb) and torch.equal(nf, nb)
    for s in range(3):
        full.es_shard_decode_step(nxt[s], None, 2, [0, 1])
        a.es_shard_decode_step(nxt[s], None, 2, [0, 1])
        ha, _, _ = a.es_shard_handoff()
        b.es_shard_decode_step(None, ha, 2, [0, 1])
        hf, lf, _ = full.es_shard_handoff()
        hb, lb, _ = b.es_shard_handoff()
        assert torch.equal(hf, hb) and torch.equal(lf, lb)
    for s_ in (full, a, b):
        s_.close()


@pytest.mark.parametrize("d,Hq,Hkv,F,Bn", [(512, 8, 4, 1536, 5), (512, 8, 4, 1536, 12), (4096, 32, 32, 11008, 8), (4096, 32, 32, 11008, 16),
                                            (8192, 64, 8, 4096, 16)])
def test_decode_of_several_sequences_on_tensor_core_streaming_shapes(B, d, Hq, Hkv, F, Bn):
    """Decode steps of 3..16 sequences on layer shapes where the tensor-core streaming kernels take every product:
    whole-K products with the activations in shared memory, and products whose activations do not fit, which are
    cut along K across CTAs and finished by a second kernel (slices added in slice order, RMSNorm for the next
    product fused into the reduction).  Checked against the oracle at every step, for the split
    [0,1) -> [1,3) == [0,3) bit for bit (a shard that receives its rows from another shard normalises them with
    the stand-alone kernel), and for repeatability."""
    from workload import ModelShape, shard_weights
    hd = 64 if d == 512 else 128
    m = ModelShape("mid", 3, d, Hq, Hkv, hd, F, 512)
    wd = shard_weights(11, m, 0, 3, device="cuda")
    wh = {k: v.cpu() for k, v in wd.items() if k != "layers"}
    wh["layers"] = [{k: v.cpu() for k, v in lw.items()} for lw in wd["layers"]]
    T, S = 5, 4
    ids = prompt_ids(11, Bn, T, m.vocab)
    nxt = forced_decode_ids(11, Bn, S, m.vocab)
    slots = list(range(Bn))
    kw = dict(max_slots=Bn, max_seq=T + S, max_tokens=Bn * T)
    full = B.Shard(m, 0, 3, wd, **kw)
    a = B.Shard(m, 0, 1, slice_weights(wd, m, 0, 1), **kw)
    b = B.Shard(m, 1, 3, slice_weights(wd, m, 1, 3), **kw)
    runs = []
    for rep in range(2):
        full.es_shard_reset_slots(None)
        full.es_shard_prefill(ids.cuda(), None, Bn, T, slots)
        hs, ls = [], []
        for s in range(S):
            full.es_shard_decode_step(nxt[s].cuda(), None, Bn, slots)
            h, l, _ = full.es_shard_handoff()
            hs.append(h[:, 0].clone()); ls.append(l.clone())
        runs.append((torch.stack(hs), torch.stack(ls)))
    assert torch.equal(runs[0][0], runs[1][0]) and torch.equal(runs[0][1], runs[1][1])
    a.es_shard_prefill(ids.cuda(), None, Bn, T, slots)
    b.es_shard_prefill(None, a.es_shard_handoff()[0], Bn, T, slots)
    for s in range(S):
        a.es_shard_decode_step(nxt[s].cuda(), None, Bn, slots)
        b.es_shard_decode_step(None, a.es_shard_handoff()[0], Bn, slots)
        hb, lb, _ = b.es_shard_handoff()
        assert torch.equal(hb[:, 0], runs[0][0][s]) and torch.equal(lb, runs[0][1][s]), s
    for r in (0, Bn - 1):
        seq = torch.cat([ids[r], nxt[:, r]])
        want_h, _ = O.shard_forward_full(m, wh, 0, 3, ids=seq)
        assert rel_err(runs[0][0][:, r], want_h[T:]) < TOL
        for s in (0, S - 1):
            _, want_l = O.shard_forward_full(m, wh, 0, 3, ids=seq[:T + s + 1])
            assert rel_err(runs[0][1][s, r], want_l) < TOL
    for sh in (full, a, b):
        sh.es_shard_device_status()
        sh.close()


def test_batch_rows_independent_and_match_oracle(B, tiny):
    wd, wh = tiny
    T, S, Bn = 9, 4, 3
    ids = prompt_ids(0, Bn, T, TINY.vocab, seed=5)
    nxt = forced_decode_ids(0, Bn, S, TINY.vocab, seed=5)
    sh = B.Shard(TINY, 0, 2, wd, max_slots=4, max_seq=16, max_tokens=Bn * T, kv_page_tokens=16)
    sh.es_shard_prefill(ids.cuda(), None, Bn, T, [2, 0, 3])
    h, l, _ = sh.es_shard_handoff()
    hs, ls = [h.clone()], [l.clone()]
    for s in range(S):
        sh.es_shard_decode_step(nxt[s].cuda(), None, Bn, [2, 0, 3])
        h, l, _ = sh.es_shard_handoff()
        hs.append(h.clone()); ls.append(l.clone())
    for b in range(Bn):
        seq = torch.cat([ids[b], nxt[:, b]])
        want_h, _ = O.shard_forward_full(TINY, wh, 0, 2, ids=seq)
        assert rel_err(hs[0][b], want_h[:T]) < TOL
        for s in range(S):
            assert rel_err(hs[1 + s][b, 0], want_h[T + s]) < TOL
            _, want_l = O.shard_forward_full(TINY, wh, 0, 2, ids=seq[:T + s + 1])
            assert rel_err(ls[1 + s][b], want_l) < TOL
    # the same sequence alone, in another slot, gives the same result as inside the batch (a different
    # kernel may serve the smaller row count, so equality is up to fp32 summation order)
    sh.es_shard_prefill(ids[1:2].cuda(), None, 1, T, [1])
    h1, l1, _ = sh.es_shard_handoff()
    assert rel_err(h1[0], hs[0][1]) < 2e-3 and rel_err(l1[0], ls[0][1]) < 2e-3
    sh.close()


def test_batch_size_changes_between_steps_with_split_contexts(B, tiny):
    """Contexts long enough to be cut into several splits (merged inside the kernel for so few sequences), decoded with a
    batch that shrinks and grows again between steps: what one batch size leaves in the scratch buffer (partials,
    arrival counters) must not disturb the next.  Every step is compared with the oracle, sequence by sequence."""
    wd, wh = tiny
    T, Bn = 300, 3
    ids = prompt_ids(0, Bn, T, TINY.vocab, seed=21)
    forced = forced_decode_ids(0, Bn, 6, TINY.vocab, seed=21)
    sh = B.Shard(TINY, 0, 2, wd, max_slots=Bn, max_seq=T + 8, max_tokens=Bn * T)
    sh.es_shard_prefill(ids.cuda(), None, Bn, T, [0, 1, 2])
    seqs = [ids[b].tolist() for b in range(Bn)]
    plan = [[0, 1, 2], [1], [0, 1, 2], [2, 0], [0, 1, 2], [1]]
    for step, rows in enumerate(plan):
        tok = torch.tensor([int(forced[step, b]) for b in rows], dtype=torch.int32)
        sh.es_shard_decode_step(tok.cuda(), None, len(rows), rows)
        h, l, _ = sh.es_shard_handoff()
        for i, b in enumerate(rows):
            seqs[b].append(int(tok[i]))
            want_h, want_l = O.shard_forward_full(TINY, wh, 0, 2, ids=torch.tensor(seqs[b]))
            assert rel_err(h[i, 0], want_h[-1]) < TOL, (step, b)
            assert rel_err(l[i], want_l) < TOL, (step, b)
    sh.es_shard_device_status()
    sh.close()


def test_page_map_and_graphs_do_not_change_results(B, tiny):
    wd, _ = tiny
    ids = prompt_ids(0, 2, 20, TINY.vocab, seed=9).cuda()
    nxt = forced_decode_ids(0, 2, 6, TINY.vocab, seed=9).cuda()

    stream = torch.cuda.Stream()

    def run(permute, graphs):
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            outs = _run(permute, graphs)
        torch.cuda.synchronize()
        return outs

    def _run(permute, graphs):
        sh = B.Shard(TINY, 0, 2, wd, max_slots=2, max_seq=48, max_tokens=40, kv_page_tokens=16, stream=stream)
        if permute:
            g = torch.Generator().manual_seed(3)
            sh.es_shard_set_page_table(torch.randperm(sh.n_pages, generator=g).tolist())
        sh.es_shard_set_graphs(graphs)
        sh.es_shard_prefill(ids, None, 2, 20, [0, 1])
        outs = [t.clone() for t in sh.es_shard_handoff()[:2]]
        for s in range(6):
            sh.es_shard_decode_step(nxt[s], None, 2, [0, 1])
            outs += [t.clone() for t in sh.es_shard_handoff()[:2]]
        n_launch = sh.es_shard_launch_count()
        sh.close()
        assert n_launch > 6 * 10
        return outs

    ref = run(False, False)
    for permute, graphs in ((True, False), (False, True), (True, True)):
        got = run(permute, graphs)
        assert all(torch.equal(a, b) for a, b in zip(ref, got)), (permute, graphs)


def test_micro_batch_pipeline_is_order_independent(B, tiny):
    """Two shards of one layer each, four micro-batches in four KV slots: walking micro-batch by
    micro-batch (hand-over by pointer) or shard by shard (hand-over through per-micro-batch copies)
    gives identical bits, and both equal the single two-layer shard."""
    wd, _ = tiny
    T, S, MB = 10, 3, 4
    ids = prompt_ids(0, MB, T, TINY.vocab, seed=11).cuda()
    nxt = forced_decode_ids(0, MB, S, TINY.vocab, seed=11).cuda()
    kw = dict(max_slots=MB, max_seq=16, max_tokens=T, max_batch=1, kv_page_tokens=16)

    def make():
        return [B.Shard(TINY, 0, 1, slice_weights(wd, TINY, 0, 1), **kw), B.Shard(TINY, 1, 2, slice_weights(wd, TINY, 1, 2), **kw)]

    def mb_major():
        s0, s1 = make()
        out = {}
        for mb in range(MB):
            s0.es_shard_prefill(ids[mb:mb + 1], None, 1, T, [mb])
            s1.es_shard_prefill(None, s0.es_shard_handoff()[0], 1, T, [mb])
            out[(mb, -1)] = [t.clone() for t in s1.es_shard_handoff()[:2]]
        for st in range(S):
            for mb in range(MB):
                s0.es_shard_decode_step(nxt[st, mb:mb + 1], None, 1, [mb])
                s1.es_shard_decode_step(None, s0.es_shard_handoff()[0], 1, [mb])
                out[(mb, st)] = [t.clone() for t in s1.es_shard_handoff()[:2]]
        s0.close(); s1.close()
        return out

    def shard_major():
        s0, s1 = make()
        out = {}
        acts = []
        for mb in reversed(range(MB)):                                     # another micro-batch order as well
            s0.es_shard_prefill(ids[mb:mb + 1], None, 1, T, [mb])
            acts.append((mb, s0.es_shard_handoff()[0].clone()))
        for mb, a in acts:
            s1.es_shard_prefill(None, a, 1, T, [mb])
            out[(mb, -1)] = [t.clone() for t in s1.es_shard_handoff()[:2]]
        for st in range(S):
            acts = []
            for mb in range(MB):
                s0.es_shard_decode_step(nxt[st, mb:mb + 1], None, 1, [mb])
                acts.append((mb, s0.es_shard_handoff()[0].clone()))
            for mb, a in reversed(acts):
                s1.es_shard_decode_step(None, a, 1, [mb])
                out[(mb, st)] = [t.clone() for t in s1.es_shard_handoff()[:2]]
        s0.close(); s1.close()
        return out

    x, y = mb_major(), shard_major()
    assert x.keys() == y.keys()
    for key in x:
        assert all(torch.equal(p, q) for p, q in zip(x[key], y[key])), key
    whole = B.Shard(TINY, 0, 2, wd, **kw)
    for mb in range(MB):
        whole.es_shard_prefill(ids[mb:mb + 1], None, 1, T, [mb])
        h, l, _ = whole.es_shard_handoff()
        assert torch.equal(h, x[(mb, -1)][0]) and torch.equal(l, x[(mb, -1)][1])
    whole.close()


def test_profile_reports_every_layer(B, tiny):
    wd, _ = tiny
    ids = prompt_ids(0, 1, 16, TINY.vocab).cuda()
    sh = B.Shard(TINY, 0, 2, wd, max_slots=1, max_seq=32, max_tokens=16)
    sh.es_shard_set_profiling(True)
    sh.es_shard_prefill(ids, None, 1, 16, [0])
    _, _, n = sh.es_shard_handoff()
    for _ in range(3):
        sh.es_shard_decode_step(n, None, 1, [0])
    prof = sh.es_layer_profile()
    assert [p["layer"] for p in prof] == [-1, 0, 1, 2]
    for p in prof:
        assert p["n_prefill"] == 1 and p["n_decode"] == 3
        assert p["prefill_ms_mean"] > 0 and p["decode_ms_mean"] > 0
        want = (p["prefill_ms_mean"] + 3 * p["decode_ms_mean"]) / 4
        assert abs(p["avg_ms_per_token"] - want) < 1e-3 * want + 1e-6
    layer = prof[1]
    assert layer["activation_bytes"] == 256 * 4
    assert layer["weight_bytes"] == 2 * TINY.layer_params()
    assert layer["kv_bytes"] == sh.kv_bytes // 2
    assert prof[0]["weight_bytes"] == 2 * 1000 * 256 and prof[3]["activation_bytes"] == 4000
    sh.close()


@pytest.mark.parametrize("Bn,T,P", [(1, 1, 64), (16, 3, 16), (5, 70, 64), (2, 129, 64), (16, 17, 64)])
def test_edge_shapes_match_oracle(B, tiny, Bn, T, P):
    """One-token prompts, the largest batch, prompts that straddle KV pages and attention tiles, both page
    sizes (64: tensor-core attention, 16: CUDA-core attention); decode runs until the slot is exactly full."""
    wd, wh = tiny
    S = 3
    ids = prompt_ids(0, Bn, T, TINY.vocab, seed=21)
    nxt = forced_decode_ids(0, Bn, S, TINY.vocab, seed=21)
    sh = B.Shard(TINY, 0, 2, wd, max_slots=Bn, max_seq=T + S, max_tokens=Bn * T, kv_page_tokens=P)
    slots = list(reversed(range(Bn)))
    sh.es_shard_prefill(ids.cuda(), None, Bn, T, slots)
    h, l, _ = sh.es_shard_handoff()
    hs, ls = [h.clone()], [l.clone()]
    for s_ in range(S):
        sh.es_shard_decode_step(nxt[s_].cuda(), None, Bn, slots)
        h, l, _ = sh.es_shard_handoff()
        hs.append(h.clone()); ls.append(l.clone())
    with pytest.raises(B.EsError) as e:
        sh.es_shard_decode_step(nxt[0].cuda(), None, Bn, slots)          # every slot is at max_seq now
    assert e.value.status == 5
    sh.es_shard_device_status()
    sh.close()
    for b in sorted({0, Bn // 2, Bn - 1}):
        seq = torch.cat([ids[b], nxt[:, b]])
        want_h, _ = O.shard_forward_full(TINY, wh, 0, 2, ids=seq)
        assert rel_err(hs[0][b], want_h[:T]) < TOL
        for s_ in range(S):
            assert rel_err(hs[1 + s_][b, 0], want_h[T + s_]) < TOL
        _, want_l = O.shard_forward_full(TINY, wh, 0, 2, ids=seq[:T + S])
        assert rel_err(ls[S][b], want_l) < TOL


@pytest.mark.parametrize("P,split", [(64, None), (16, 1)])
def test_ragged_prompts_and_sequences_that_stop_early(B, tiny, P, split):
    """Right-padded prompts of different lengths in one batch (one of them the full width, one a single token, one
    ending on a page boundary), then greedy decoding in which sequences leave the batch at different steps (the
    caller's EOS handling: a finished sequence's slot is simply no longer passed).  Every sequence must match the
    oracle run on that sequence alone; with `split` the model runs as two shards handing padded activations over."""
    wd, wh = tiny
    T, lens, stop_after = 40, [40, 1, 16, 23], [4, 1, 6, 3]        # decode steps each sequence stays for
    Bn = len(lens)
    ids = prompt_ids(0, Bn, T, TINY.vocab, seed=33)
    S = max(stop_after)
    slots = [2, 0, 3, 1]
    kw = dict(max_slots=Bn, max_seq=T + S, max_tokens=Bn * T, kv_page_tokens=P)
    if split is None:
        shards = [B.Shard(TINY, 0, 2, wd, **kw)]
    else:
        shards = [B.Shard(TINY, 0, split, slice_weights(wd, TINY, 0, split), **kw),
                  B.Shard(TINY, split, 2, slice_weights(wd, TINY, split, 2), **kw)]
    x = None
    for i, sh in enumerate(shards):
        sh.es_shard_prefill_ragged(ids.cuda() if i == 0 else None, x, Bn, T, slots, lens)
        x, logits, nxt = sh.es_shard_handoff()
    pre_h, step_logits = x.clone(), [logits.clone()]
    tokens = [nxt.clone().cpu()]                                   # tokens[s][row of the batch at step s]
    alive = list(range(Bn))
    rows_at = [list(alive)]
    for s_ in range(S):
        alive = [b for b in alive if stop_after[b] > s_]
        if not alive:
            break
        prev_rows = rows_at[-1]
        feed = torch.tensor([int(tokens[-1][prev_rows.index(b)]) for b in alive], dtype=torch.int32).cuda()
        x = None
        for i, sh in enumerate(shards):
            sh.es_shard_decode_step(feed if i == 0 else None, x, len(alive), [slots[b] for b in alive])
            x, logits, nxt = sh.es_shard_handoff()
        step_logits.append(logits.clone()); tokens.append(nxt.clone().cpu()); rows_at.append(list(alive))
    for sh in shards:
        sh.es_shard_device_status()
        sh.close()
    for b in range(Bn):
        fed = [int(tokens[s_][rows_at[s_].index(b)]) for s_ in range(len(rows_at) - 1) if b in rows_at[s_] and b in rows_at[s_ + 1]]
        seq = torch.cat([ids[b, :lens[b]], torch.tensor(fed, dtype=torch.int32)])
        want_h, _ = O.shard_forward_full(TINY, wh, 0, 2, ids=seq)
        assert rel_err(pre_h[b, :lens[b]], want_h[:lens[b]]) < TOL
        for s_ in range(len(fed) + 1):                            # logits after the prompt and after every fed token
            _, want_l = O.shard_forward_full(TINY, wh, 0, 2, ids=seq[:lens[b] + s_])
            got = step_logits[s_][rows_at[s_].index(b)]
            assert rel_err(got, want_l) < TOL


@pytest.mark.parametrize("lens,P,split", [([40, 1, 16, 23], 64, None), ([40, 1, 16, 23], 16, 1), ([3, 1, 5], 64, None),
                                          ([130, 64, 200, 7, 129], 64, 1)])
def test_packed_prompts_skip_the_padding(B, tiny, lens, P, split):
    """Prompts of different lengths packed one after the other (no padded rows are computed): the hidden rows, the
    logits of every sequence's last token and three greedy decode steps must match the oracle run on each
    sequence alone; with `split` the model runs as two shards handing the packed activation over.  The cases
    cover the tensor-core and the CUDA-core attention (64- and 16-token pages), prompts that end inside, on and
    just past a 128-row query tile, and a batch small enough (9 rows) for the weight-streaming kernels."""
    wd, wh = tiny
    Bn, total, S = len(lens), sum(lens), 3
    seqs = [prompt_ids(0, 1, L, TINY.vocab, seed=50 + b)[0] for b, L in enumerate(lens)]
    packed = torch.cat(seqs).cuda()
    slots = list(reversed(range(Bn)))
    kw = dict(max_slots=Bn, max_seq=max(lens) + S, max_tokens=total, max_batch=Bn, kv_page_tokens=P)
    if split is None:
        shards = [B.Shard(TINY, 0, 2, wd, **kw)]
    else:
        shards = [B.Shard(TINY, 0, split, slice_weights(wd, TINY, 0, split), **kw),
                  B.Shard(TINY, split, 2, slice_weights(wd, TINY, split, 2), **kw)]
    x = None
    for i, sh in enumerate(shards):
        sh.es_shard_prefill_packed(packed if i == 0 else None, x, Bn, slots, lens)
        x, logits, nxt = sh.es_shard_handoff()
    assert x.shape == (1, total, TINY.d_model) and logits.shape == (Bn, TINY.vocab) and nxt.shape == (Bn,)
    pre_h, all_logits, fed = x[0].clone(), [logits.clone()], []
    for _ in range(S):
        fed.append(nxt.clone().cpu())
        feed, x = nxt.clone(), None
        for i, sh in enumerate(shards):
            sh.es_shard_decode_step(feed if i == 0 else None, x, Bn, slots)
            x, logits, nxt = sh.es_shard_handoff()
        all_logits.append(logits.clone())
    for sh in shards:
        sh.es_shard_device_status()
        sh.close()
    row = 0
    for b, L in enumerate(lens):
        seq = torch.cat([seqs[b], torch.tensor([int(f[b]) for f in fed], dtype=torch.int32)])
        want_h, _ = O.shard_forward_full(TINY, wh, 0, 2, ids=seq)
        assert rel_err(pre_h[row:row + L], want_h[:L]) < TOL, b
        for s_ in range(S + 1):
            _, want_l = O.shard_forward_full(TINY, wh, 0, 2, ids=seq[:L + s_])
            assert rel_err(all_logits[s_][b], want_l) < TOL, (b, s_)
        row += L


def test_packed_prompts_on_7b_layer_shapes(B):
    """The packed prefill on layer shapes that take the CTA-pair tensor-core products and the tcgen05 attention
    (two Llama-2-7B-shaped layers, prompts of 300, 128 and 700 tokens = 1128 rows): hidden rows and last-token
    logits of every sequence against the oracle run on that sequence alone, and against the padded form."""
    from workload import ModelShape, shard_weights
    m = ModelShape("7b-2layers", 2, 4096, 32, 32, 128, 11008, 512)
    wd = shard_weights(12, m, 0, 2, device="cuda")
    wh = {k: v.cpu() for k, v in wd.items() if k != "layers"}
    wh["layers"] = [{k: v.cpu() for k, v in lw.items()} for lw in wd["layers"]]
    lens = [300, 128, 700]
    Bn, total, T = len(lens), sum(lens), max(lens)
    seqs = [prompt_ids(12, 1, L, m.vocab, seed=70 + b)[0] for b, L in enumerate(lens)]
    sh = B.Shard(m, 0, 2, wd, max_slots=Bn, max_seq=T + 2, max_tokens=Bn * T, max_batch=Bn)
    sh.es_shard_prefill_packed(torch.cat(seqs).cuda(), None, Bn, [0, 1, 2], lens)
    x, logits, nxt = sh.es_shard_handoff()
    packed_h, packed_l = x[0].clone(), logits.clone()
    padded = torch.zeros(Bn, T, dtype=torch.int32)
    for b, L in enumerate(lens):
        padded[b, :L] = seqs[b]
    sh.es_shard_reset_slots(None)
    sh.es_shard_prefill_ragged(padded.cuda(), None, Bn, T, [0, 1, 2], lens)
    xp, lp, _ = sh.es_shard_handoff()
    row = 0
    for b, L in enumerate(lens):
        want_h, want_l = O.shard_forward_full(m, wh, 0, 2, ids=seqs[b])
        assert report_err(f"packed prefill, 7B shapes, sequence of {L}: hidden", rel_err(packed_h[row:row + L], want_h)) < TOL
        assert report_err(f"packed prefill, 7B shapes, sequence of {L}: logits", rel_err(packed_l[b], want_l)) < TOL
        assert rel_err(packed_h[row:row + L], xp[b, :L]) < 2e-3 and rel_err(packed_l[b], lp[b]) < 2e-3
        row += L
    sh.es_shard_device_status()
    sh.close()


def test_pipeline_stage_drives_the_library_on_one_gpu(B, tiny):
    """The multi-device stage object with a single rank: it must drive the real shard (device tensors, greedy
    feedback, several micro-batches in their own KV slots) to the oracle's tokens.  The message flow between ranks
    is tested on the CPU (tests/test_stage.py); more than one GPU is not available to these tests."""
    import socket
    import torch.distributed as dist
    from paper_2405_14371_b200.stage import PipelineStage

    wd, wh = tiny
    sock = socket.socket(); sock.bind(("127.0.0.1", 0)); port = sock.getsockname()[1]; sock.close()
    os.environ.update(RANK="0", WORLD_SIZE="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo")
    try:
        MB, Bn, T, S = 2, 2, 16, 5
        seed, _ = _golden_cfg0()
        ids = prompt_ids(0, MB * Bn, T, TINY.vocab, seed=seed).reshape(MB, Bn, T)
        sh = B.Shard(TINY, 0, 2, wd, max_slots=MB * Bn, max_seq=T + S, max_tokens=Bn * T, max_batch=Bn)
        slots = [[mb * Bn + b for b in range(Bn)] for mb in range(MB)]
        stage = PipelineStage(sh, TINY.d_model, MB, Bn, slots, torch.device("cuda"))
        gen = stage.prefill_and_decode([ids[mb].cuda() for mb in range(MB)], T, S).cpu()
        sh.es_shard_device_status()
        sh.close()
    finally:
        dist.destroy_process_group()
    want, _, _ = O.generate_greedy(TINY, wh, ids[0, 0], S)          # the golden prompt: margins known to be wide
    assert gen[:, 0, 0].tolist() == want.tolist()
    for mb in range(MB):
        for b in range(Bn):
            w_t, w_l, _ = O.generate_greedy(TINY, wh, ids[mb, b], S)
            top2 = w_l.topk(2, dim=-1).values
            wide = bool(((top2[:, 0] - top2[:, 1]) > 1e-2 * w_l.abs().max()).all())
            if wide:                                                # near-ties may legitimately flip under fp16
                assert gen[:, mb, b].tolist() == w_t.tolist()


@pytest.mark.parametrize("Bn", [1, 8])
def test_step_timing_from_inside_a_replayed_step(B, tiny, Bn):
    """Time stamps written by the kernels of a decode step: every launch of the step is listed in launch order
    with a start and an end inside the step, the step's results are the same bits with and without the stamps,
    and the prefill pass is stamped too."""
    wd, _ = tiny
    T = 12
    ids = prompt_ids(0, Bn, T, TINY.vocab, seed=3).cuda()
    stream = torch.cuda.Stream()
    outs = {}
    with torch.cuda.stream(stream):
        for timing in (False, True):
            sh = B.Shard(TINY, 0, 2, wd, max_slots=Bn, max_seq=T + 6, max_tokens=Bn * T, stream=stream)
            sh.es_shard_set_step_timing(timing)
            sh.es_shard_prefill(ids, None, Bn, T, list(range(Bn)))
            if timing:
                pre = sh.es_shard_step_timing()
                assert {"embed", "qkv", "attention", "o", "gate_up", "down", "lm_head", "argmax", "set_ctx"} <= {e["category"] for e in pre}
            n = sh.es_shard_handoff()[2]
            rows = []
            for _ in range(4):
                sh.es_shard_decode_step(n, None, Bn, list(range(Bn)))
                h, l, n = sh.es_shard_handoff()
                rows.append((h.clone(), l.clone(), n.clone()))
            if timing:
                st = sh.es_shard_step_timing()
                assert len(st) >= 2 * 5 + 4                      # 5 kernels per layer, embedding, head, argmax, counter
                assert st[0]["category"] == "embed" and st[1]["category"] in ("rmsnorm", "qkv")
                assert st[-1]["category"] == "set_ctx"
                assert min(e["start_us"] for e in st) == 0.0
                for e in st:
                    assert 0.0 <= e["start_us"] <= e["end_us"] < 1e5, e
                ends = [e["end_us"] for e in st]
                # a kernel cannot finish before the one it depends on has finished
                assert all(b >= a for a, b in zip(ends, ends[1:])), ends
            sh.es_shard_device_status()
            sh.close()
            outs[timing] = rows
    stream.synchronize()
    for a, b in zip(outs[False], outs[True]):
        for x, y in zip(a, b):
            assert torch.equal(x, y)


def test_profile_feeds_the_partition_planners(B, tiny):
    """The per-layer profile is the planners' input: measured times for this GPU plus two synthetic slower
    devices (scaled times), activation and memory sizes from the profile."""
    wd, _ = tiny
    ids = prompt_ids(0, 1, 16, TINY.vocab).cuda()
    sh = B.Shard(TINY, 0, 2, wd, max_slots=1, max_seq=32, max_tokens=16)
    sh.es_shard_set_profiling(True)
    sh.es_shard_prefill(ids, None, 1, 16, [0])
    n = sh.es_shard_handoff()[2]
    for _ in range(4):
        sh.es_shard_decode_step(n, None, 1, [0])
    prof = sh.es_layer_profile()
    sh.close()
    scale = [1.0, 5.0, 20.0]                                   # device 0 is the source node (a slow one here)
    order = [2, 0, 1]                                          # so that the fast GPU is not the source
    t_comp = [[p["avg_ms_per_token"] * scale[order[j]] for j in range(3)] for p in prof]
    O = [p["activation_bytes"] for p in prof]
    Req = [p["weight_bytes"] + p["kv_bytes"] for p in prof]
    Mem = [sum(Req)] * 3
    Bw = [[0 if a == b else 1e9 for b in range(3)] for a in range(3)]
    a, t = B.es_partition_latency(t_comp, O, Req, Mem, Bw)
    assert a[0] == 0 and len(a) == len(prof) and t > 0
    assert a[1:] == [1] * (len(prof) - 1)                      # with fast links the work moves to the fast device
    a2, t2 = B.es_partition_throughput(t_comp, O, Req, Mem, Bw)
    assert a2[0] == 0 and t2 <= max(sum(r) for r in zip(*t_comp))


def test_a_device_wait_that_runs_out_is_reported_and_the_shard_stays_usable(B, tiny):
    """The bounded waits of the tensor-core kernels end with a code in the shard's status word instead of
    hanging.  A probe kernel with the same structure waits 2 ms on a barrier nobody arrives on: the status call
    must report ES_ERR_DEVICE_TIMEOUT with the probe's code, clear the word, and the shard must go on computing
    the same bits as before."""
    import time
    wd, _ = tiny
    ids = prompt_ids(0, 1, 16, TINY.vocab, seed=1).cuda()
    sh = B.Shard(TINY, 0, 2, wd, max_slots=1, max_seq=32, max_tokens=16)
    sh.es_shard_prefill(ids, None, 1, 16, [0])
    before = [t.clone() for t in sh.es_shard_handoff()]
    sh.es_shard_device_status()                          # clean so far
    t0 = time.perf_counter()
    sh.es_shard_wait_probe(2000)
    with pytest.raises(B.EsError) as e:
        sh.es_shard_device_status()
    assert time.perf_counter() - t0 < 5.0                # the wait ended by itself
    assert e.value.status == 8 and "code 90" in e.value.message
    sh.es_shard_device_status()                          # the word was cleared
    sh.es_shard_reset_slots(None)
    sh.es_shard_prefill(ids, None, 1, 16, [0])
    after = sh.es_shard_handoff()
    for x, y in zip(before, after):
        assert torch.equal(x, y)
    with pytest.raises(B.EsError):
        sh.es_shard_wait_probe(0)
    sh.close()


def test_checking_mode_passes_over_the_tiny_configuration():
    """ES_DEBUG=1 (read once per process, hence a child process): after every pass of the tiny-configuration
    tests the status call also verifies the guard bytes behind each scratch region and the ranges of the page
    table, context lengths and slot list.  All of those tests must still pass, i.e. no kernel writes outside its
    region and the device-side counters follow the host's."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, ES_DEBUG="1")
    sel = "cfg0_greedy or split_point or batch_rows or page_map or edge_shapes or ragged or micro_batch"
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_shard_gpu.py"), "-m", "gpu", "-q", "-x",
                        "-k", sel, "-p", "no:cacheprovider"], cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


def test_error_paths_launch_nothing(B, tiny):
    wd, _ = tiny
    ids = prompt_ids(0, 1, 8, TINY.vocab).cuda()
    sh = B.Shard(TINY, 0, 2, wd, max_slots=2, max_seq=10, max_tokens=8, max_batch=1)
    E = B.EsError
    with pytest.raises(E) as e:
        sh.es_shard_handoff()
    assert e.value.status == 4
    with pytest.raises(E) as e:
        sh.es_shard_decode_step(ids[0, :1], None, 1, [0])          # never prefilled
    assert e.value.status == 4
    with pytest.raises(E) as e:
        sh.es_shard_prefill(ids, None, 1, 8, [2])                   # slot out of range
    assert e.value.status == 3
    with pytest.raises(E) as e:
        sh.es_shard_prefill(None, torch.zeros(1, 8, 256, device="cuda"), 1, 8, [0])   # needs ids
    assert e.value.status == 1
    with pytest.raises(E) as e:
        sh.es_shard_prefill(ids.repeat(2, 1), None, 2, 8, [0, 1])   # B > max_batch
    assert e.value.status == 3
    n0 = sh.es_shard_launch_count()
    assert n0 == 0
    sh.es_shard_prefill(ids, None, 1, 8, [0])
    _, _, n = sh.es_shard_handoff()
    sh.es_shard_decode_step(n, None, 1, [0])
    sh.es_shard_decode_step(n, None, 1, [0])
    with pytest.raises(E) as e:
        sh.es_shard_decode_step(n, None, 1, [0])                    # context 10 == max_seq
    assert e.value.status == 5
    sh.es_shard_reset_slots([0])
    with pytest.raises(E) as e:
        sh.es_shard_decode_step(n, None, 1, [0])
    assert e.value.status == 4
    b = B.Shard(TINY, 1, 2, slice_weights(wd, TINY, 1, 2), max_slots=1, max_seq=10, max_tokens=8)
    with pytest.raises(E) as e:
        b.es_shard_prefill(ids, None, 1, 8, [0])                    # needs hidden_in
    assert e.value.status == 1
    with pytest.raises(E) as e:
        b.es_shard_prefill(None, torch.zeros(1, 8, 128, device="cuda"), 1, 8, [0])    # wrong width
    assert e.value.status == 2
    sh.es_shard_device_status()
    sh.close(); b.close()

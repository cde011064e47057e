"""Writes tests/golden/cfg4_handoff_digest.npz: the oracle's handoff activation of the 70B-architecture
shard (decoder layers 0-39, batch 16, 1024-token prompts, 128 teacher-forced decode ids) for batch
rows 0 and 15, through all 40 layers, at every one of the 1152 positions.  Calls only oracle/ and
workload/.

The full expected tensor (2 x 1152 x 8192 fp32, 75 MB) is too large to store, so the file keeps, per
row and position: the largest magnitude of the activation, the index where it occurs, and the values
at 64 fixed columns (every 128th, starting at 5).  The 68 GB of weights do not fit in host memory:
they are regenerated layer by layer (on a CUDA device if one is present — the seeded generator gives
the same bits on either — and copied to the host) and dropped after use; all arithmetic is the
oracle's, on the host.

Run from the repo root (about 160 TFLOP of fp32 host work):  python tests/golden/make_cfg4_golden.py
"""
import os
import sys
import time

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import decoder as O  # noqa: E402
from workload import WORKLOADS, forced_decode_ids, layer_weights, prompt_ids, weight_tensor  # noqa: E402

ROWS = (0, 15)
COLS = list(range(5, 8192, 128))


def main():
    wl = WORKLOADS["cfg4"]
    m, T, S, Bn = wl.model, wl.prompt_len, wl.decode_steps, wl.batch
    n_layers = int(os.environ.get("ES_GOLDEN_LAYERS", wl.layer_end))       # fewer layers only for a dry run
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    ids = prompt_ids(wl.cfg, Bn, T, m.vocab)
    forced = forced_decode_ids(wl.cfg, Bn, S, m.vocab)
    seqs = [torch.cat([ids[r], forced[:, r]]) for r in ROWS]
    emb = weight_tensor(wl.cfg, m, "tok_embedding", device=gen_dev).cpu()
    xs = [O.embed(s, emb) for s in seqs]
    del emb
    t0 = time.time()
    for li in range(n_layers):
        lw = {k: v.cpu() for k, v in layer_weights(wl.cfg, m, li, gen_dev).items()}
        xs = [O.layer_forward_full(x, lw, m) for x in xs]
        del lw
        print(f"layer {li}: {time.time() - t0:.0f} s, max |x| = {max(float(x.abs().max()) for x in xs):.4f}", flush=True)
    x = torch.stack(xs)                                                    # [2, T+S, d]
    amax = x.abs().max(dim=-1)
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)),
                       "cfg4_handoff_digest.npz" if n_layers == wl.layer_end else f"cfg4_handoff_digest_{n_layers}layers.npz")
    np.savez_compressed(out, rows=np.array(ROWS, dtype=np.int32), cols=np.array(COLS, dtype=np.int32),
                        n_layers=np.int32(n_layers), max_abs=amax.values.numpy().astype(np.float32),
                        argmax_abs=amax.indices.numpy().astype(np.int32),
                        values=x[:, :, COLS].numpy().astype(np.float32))
    print("wrote", out, os.path.getsize(out), "bytes")


if __name__ == "__main__":
    main()

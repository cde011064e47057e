"""Writes tests/golden/cfg0_greedy.txt: the prompt seed chosen for the tiny config and the
oracle's greedy tokens and top-1/top-2 margins for it.  Calls only oracle/ and workload/.

Rule (fixed before any CUDA code existed): the first prompt seed 0, 1, 2, ... for which the
smallest top-1/top-2 logit margin over the 9 generated tokens exceeds 1e-2 * max|logit|, so
that the greedy tokens are well defined under fp16 rounding differences.

Run from the repo root:  python tests/golden/make_cfg0_golden.py
"""
import os
import sys

import torch

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from oracle import decoder as O  # noqa: E402
from workload import TINY, shard_weights, prompt_ids  # noqa: E402


def main():
    w = shard_weights(0, TINY, 0, TINY.n_layers)
    for seed in range(64):
        ids = prompt_ids(0, 1, 16, TINY.vocab, seed=seed)[0]
        toks, logits, _ = O.generate_greedy(TINY, w, ids, 8, torch.float32)
        top2 = logits.topk(2, dim=-1).values
        margin = (top2[:, 0] - top2[:, 1]) / logits.abs().max()
        if float(margin.min()) > 1e-2:
            break
    else:
        raise SystemExit("no seed found")
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg0_greedy.txt")
    with open(out, "w") as f:
        f.write("# tiny config: prompt seed, oracle greedy tokens (prefill token first), relative margins\n")
        f.write("# written by tests/golden/make_cfg0_golden.py (oracle only)\n")
        f.write(f"seed {seed}\n")
        f.write("tokens " + " ".join(str(int(t)) for t in toks) + "\n")
        f.write("margins " + " ".join(f"{float(m):.6f}" for m in margin) + "\n")
    print(open(out).read())


if __name__ == "__main__":
    main()

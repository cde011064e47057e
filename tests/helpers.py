"""Shared test plumbing: device weights from the seeded generator, shard construction, and the
oracle run over the same inputs.  The oracle is only ever called from here and from the tests."""
from __future__ import annotations

import torch

from workload import shard_weights


def device_weights(cfg: int, model, layer_begin: int, layer_end: int):
    """(weights on cuda, the same weights on the host) — generated on the GPU, copied back."""
    w = shard_weights(cfg, model, layer_begin, layer_end, device="cuda")
    host = {k: v.cpu() for k, v in w.items() if k != "layers"}
    host["layers"] = [{k: v.cpu() for k, v in lw.items()} for lw in w["layers"]]
    return w, host


def slice_weights(w: dict, model, begin: int, end: int, base: int = 0) -> dict:
    """Weights of the sub-shard [begin, end) out of a dict that starts at layer `base`."""
    out = {"layers": w["layers"][begin - base:end - base]}
    if begin == 0:
        out["tok_embedding"] = w["tok_embedding"]
    if end == model.n_layers:
        out["final_norm"] = w["final_norm"]
        out["lm_head"] = w["lm_head"]
    return out


def rel_err(got: torch.Tensor, want: torch.Tensor) -> float:
    """max|got - want| / max|want| over the whole tensor (the stated parity metric)."""
    got = got.detach().double().cpu()
    want = want.detach().double().cpu()
    return float((got - want).abs().max() / want.abs().max())


def report_err(label: str, value: float) -> float:
    """Prints a measured parity error (pytest -s / -rP shows it) and, when ES_PARITY_LOG names a file,
    appends it there as one JSON line, so the worst error per configuration can be tabulated."""
    import json
    import os

    print(f"parity {label}: {value:.3e}")
    path = os.environ.get("ES_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps({"label": label, "rel_err": value}) + "\n")
    return value


def host_layer(lw: dict) -> dict:
    return {k: v.cpu() for k, v in lw.items()}


def oracle_streamed(model, wd: dict, layer_begin: int, layer_end: int, seqs, n_layers=None, logits_from=None):
    """Oracle (matrix form) over several independent sequences, layer by layer: each layer's weights are
    copied from the device to the host, used for every sequence and dropped, so models larger than host
    memory can be checked.  seqs: list of 1-D id tensors (the shard must hold the embedding).
    Returns (list of hidden [T, d], list of logits [T - logits_from, V] or None)."""
    from oracle import decoder as O

    emb = wd["tok_embedding"].cpu()
    xs = [O.embed(s, emb) for s in seqs]
    del emb
    n = (layer_end - layer_begin) if n_layers is None else n_layers
    for li in range(n):
        lw = host_layer(wd["layers"][li])
        xs = [O.layer_forward_full(x, lw, model) for x in xs]
        del lw
    logits = None
    if logits_from is not None:
        fn, lm = wd["final_norm"].cpu(), wd["lm_head"].cpu()
        logits = [O.lm_head(x[logits_from:], fn, lm, model.rms_eps) for x in xs]
    return xs, logits

"""Variant sweeps over the knobs the paper ablates, on synthetic inputs of the long-context shape:

* ``window``: the retained suffix window w (tokens) with and without the trailing position (the window-size
  study and the "no trailing position" ablation): time and bytes of the pruned attention call.
* ``alpha``: the adaptation strength of Eq. 10 (and the two readings of r_mask: block only / block plus the
  retained suffix rows): iterations per block of the whole decoding loop on seeded logits.

    python -m paper_2601_17917_b200.sweeps window
    python -m paper_2601_17917_b200.sweeps alpha

One JSON line per point; the functions also return the rows, which is how tests/test_gpu_sweeps.py checks a
small point of each sweep against the oracle.  The numbers describe the kernels and the loop mechanics, not model quality: the
logits are seeded noise with spikes, not a model's.
"""
from __future__ import annotations

import argparse
import json
import math

import torch

from . import AttnPlan, retained_indices
from . import workloads as wl
from .decode import BlockDecoder


def _time_us(fn, reps=30, warm=5):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / reps * 1e3


def sweep_window(device, base="long32-w64", windows=(0, 32, 64, 128, 256, 512, 1024, -1), cfg=None, reps=30,
                 keep_outputs=False, emit=print):
    """One row per (window, trailing position kept or not).  ``cfg`` replaces the named base configuration
    (its own w / keep_last are ignored).  With ``keep_outputs`` every row also carries the inputs, the index
    list and the attention output of its last launch (device tensors), so that a caller can check the point
    against a reference.  Rows are returned; ``emit`` (None to silence) gets each as one JSON line."""
    cfg0 = wl.CONFIGS[base] if cfg is None else cfg
    x = wl.attention_inputs(cfg0, device=device)
    scale = 1.0 / math.sqrt(cfg0.D)
    esz = 2 if cfg0.dtype == "bf16" else 4
    rows = []
    # both variants of a window back to back, the long-running whole-suffix point last: a point measured right
    # after seconds of dense work would see the power-capped clock, not its own
    for w in windows:
        for keep_last in (True, False):
            if w < 0 and not keep_last:
                continue
            idx = retained_indices(cfg0.gen, cfg0.K, 0, w, keep_last)
            idx_t = torch.tensor(idx, dtype=torch.int32, device=device)
            plan = AttnPlan(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"], idx_t, scale)
            us = _time_us(plan.launch, reps=reps)
            Lq = len(idx)
            nbytes = cfg0.B * (2 * cfg0.Hkv * (cfg0.P + Lq) + 2 * cfg0.Hq * Lq) * cfg0.D * esz
            flops = 4.0 * cfg0.B * cfg0.Hq * Lq * (cfg0.P + Lq) * cfg0.D
            row = {"sweep": "window", "workload": cfg0.name, "w_tokens": w, "keep_last": keep_last, "Lq": Lq,
                   "Lkv": cfg0.P + Lq, "attn_us": us, "GBps": nbytes / us / 1e3, "TFLOPs": flops / us / 1e6}
            if emit is not None:
                emit(json.dumps(row), flush=True) if emit is print else emit(json.dumps(row))
            if keep_outputs:
                row = dict(row, inputs=x, idx=idx, scale=scale, out=plan.out.clone())
            rows.append(row)
            del plan
    return rows


def alpha_sweep_config(B=8, K=32, n_blocks=8, V=32768):
    """The seeded configuration of the alpha sweep and the logits of (block n, iteration t) on it."""
    cfg = wl.shrink(wl.CONFIGS["llada8x32"], B=B, K=K, gen=K * n_blocks, V=V, spike_p=0.6, name="alpha-sweep")
    return cfg, (lambda n, t, device="cpu": wl.logits(cfg, device=device, step=64 * n + t, spike_range=(10.0, 24.0)))


def sweep_alpha(device, alphas=(0.0, 0.1, 0.2, 0.3, 0.4, 0.5, 0.6), B=8, K=32, n_blocks=8, V=32768, w=64,
                readings=(False, True), emit=print):
    """One row per (alpha, r_mask reading): iterations each block of the decoding loop needs.  ``readings``:
    False = r_mask over the block, True = the retained suffix rows counted as masked too."""
    cfg, table = alpha_sweep_config(B, K, n_blocks, V)
    pool = {}

    def logits(n, t):
        if (n, t) not in pool:
            pool[(n, t)] = table(n, t, device)
        return pool[(n, t)]
    rows = []
    for count_suffix in readings:
        for alpha in alphas:
            dec = BlockDecoder(B, cfg.gen, K, V, tau0=cfg.tau0, alpha=alpha, mask_id=V - 1, w_tokens=w, keep_last=True,
                               count_suffix=count_suffix, device=device, lookahead=2)
            got = dec.decode(lambda st: logits(st.n, st.t))
            torch.cuda.synchronize()
            row = {"sweep": "alpha", "alpha": alpha, "tau0": cfg.tau0, "ratio_counts_suffix": count_suffix,
                   "B": B, "K": K, "blocks": n_blocks, "iterations_per_block": sum(got["steps"]) / n_blocks,
                   "iterations": got["steps"]}
            if emit is not None:
                emit(json.dumps(row), flush=True) if emit is print else emit(json.dumps(row))
            rows.append(dict(row, x=got["x"].clone()))
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["window", "alpha"])
    args = ap.parse_args()
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    if args.what == "window":
        sweep_window(device)
    else:
        sweep_alpha(device)


if __name__ == "__main__":
    main()

"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and names shapes.  It holds none of the
method's arithmetic (no index-list construction, no softmax, no threshold), so
that the CUDA path and the CPU oracle can both be fed from it without sharing
any code of the method itself.  The retained-row list of Eq. 7 is built by each
side on its own.

Shapes follow the paper's settings: block size K = 32 and window sizes of
32-256 tokens (hyper-parameter table of the "Optimization and Schedule"
appendix), generation lengths 256-4096 (main tables and the generation-length
ablation), base threshold tau0 = 0.9.  Model dimensions (32 x 128 MHA with a
126464-entry vocabulary, 28/4 GQA with 152064 entries) are those of the 8B and
7B diffusion LLMs the paper evaluates.  The paper's real inputs (benchmark
prompts through trained weights) are replaced by N(0,1) Q/K/V and N(0,2^2)
logits with a +8 spike on a seeded fraction of rows.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class StepConfig:
    name: str
    B: int            # batch (sequences)
    Hq: int           # query heads
    Hkv: int          # key/value heads
    D: int            # head dimension
    P: int            # prefix (prompt + decoded blocks) length held in the KV cache
    gen: int          # generation length L; the tail (block + suffix) has T = gen rows at block 0
    K: int            # block size
    w: int            # retained window in tokens (suffix positions nearest the block); -1 = whole suffix
    keep_last: bool   # keep the trailing position of the sequence
    dtype: str        # "f32" | "bf16"
    V: int            # vocabulary size
    spike_p: float    # fraction of logit rows that get the +8 spike
    tau0: float = 0.9
    alpha: float = 0.3
    n_layers: int = 1  # independent KV caches resident (one attention call each per step)
    seed: int = 0
    spike: float = 8.0

    @property
    def T(self) -> int:
        return self.gen

    @property
    def rows(self) -> int:
        return self.B * self.K

    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    def with_window(self, w: int, keep_last: bool = True, tag: str | None = None) -> "StepConfig":
        return replace(self, w=w, keep_last=keep_last, name=tag or f"{self.name}-w{w}")


CONFIGS: dict[str, StepConfig] = {
    "tiny": StepConfig("tiny", B=1, Hq=4, Hkv=4, D=64, P=64, gen=256, K=32, w=16, keep_last=True,
                       dtype="f32", V=1024, spike_p=0.5, seed=0),
    "llada1": StepConfig("llada1", B=1, Hq=32, Hkv=32, D=128, P=512, gen=256, K=32, w=32, keep_last=True,
                         dtype="bf16", V=126464, spike_p=0.5, seed=2000),
    "llada8x32": StepConfig("llada8x32", B=8, Hq=32, Hkv=32, D=128, P=1024, gen=1024, K=32, w=64,
                            keep_last=True, dtype="bf16", V=126464, spike_p=0.5, n_layers=32, seed=3000),
    "dream16": StepConfig("dream16", B=16, Hq=28, Hkv=4, D=128, P=2048, gen=2048, K=32, w=64,
                          keep_last=True, dtype="bf16", V=152064, spike_p=0.3, seed=4000),
    "long32-w0": StepConfig("long32-w0", B=32, Hq=32, Hkv=32, D=128, P=4096, gen=4096, K=64, w=0,
                            keep_last=False, dtype="bf16", V=126464, spike_p=0.5, seed=5000),
    "long32-w64": StepConfig("long32-w64", B=32, Hq=32, Hkv=32, D=128, P=4096, gen=4096, K=64, w=64,
                             keep_last=True, dtype="bf16", V=126464, spike_p=0.5, seed=5000),
    "long32-w256": StepConfig("long32-w256", B=32, Hq=32, Hkv=32, D=128, P=4096, gen=4096, K=64, w=256,
                              keep_last=True, dtype="bf16", V=126464, spike_p=0.5, seed=5000),
    "long32-all": StepConfig("long32-all", B=32, Hq=32, Hkv=32, D=128, P=4096, gen=4096, K=64, w=-1,
                             keep_last=True, dtype="bf16", V=126464, spike_p=0.5, seed=5000),
    # the first step of a block ("cache refresh"): every position of the sequence is a query, nothing is cached yet;
    # prompt 1024 + generation 1024 rows, all retained -> dense bidirectional attention, bound by the tensor cores
    "refresh8": StepConfig("refresh8", B=8, Hq=32, Hkv=32, D=128, P=0, gen=2048, K=32, w=-1,
                           keep_last=True, dtype="bf16", V=126464, spike_p=0.5, seed=6000),
}


def shrink(cfg: StepConfig, **kw) -> StepConfig:
    """A smaller instance of the same shape family (for cases a CPU finishes in seconds)."""
    return replace(cfg, **kw)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, seed, device, dtype, std=1.0):
    """N(0, std^2) drawn in float32 on ``device``, rounded once to ``dtype``."""
    g = _gen(seed, device)
    x = torch.empty(shape, dtype=torch.float32, device=device)
    x.normal_(0.0, std, generator=g)
    return x.to(dtype)


def attention_inputs(cfg: StepConfig, device="cpu", layer: int = 0, q_scale: float = 1.0):
    """Q/K/V of one attention call: dict with q_tail [B,Hq,T,D], k_tail, v_tail
    [B,Hkv,T,D], k_pre, v_pre [B,Hkv,P,D], all N(0,1) (queries times q_scale)."""
    dt = cfg.torch_dtype()
    s = cfg.seed + 10 * layer
    out = {
        "q_tail": _normal((cfg.B, cfg.Hq, cfg.T, cfg.D), s + 1, device, torch.float32),
        "k_tail": _normal((cfg.B, cfg.Hkv, cfg.T, cfg.D), s + 2, device, dt),
        "v_tail": _normal((cfg.B, cfg.Hkv, cfg.T, cfg.D), s + 3, device, dt),
        "k_pre": _normal((cfg.B, cfg.Hkv, cfg.P, cfg.D), s + 4, device, dt),
        "v_pre": _normal((cfg.B, cfg.Hkv, cfg.P, cfg.D), s + 5, device, dt),
    }
    out["q_tail"] = (out["q_tail"] * q_scale).to(dt)
    return out


def logits(cfg: StepConfig, device="cpu", step: int = 0, spike_range=None, rows: int | None = None):
    """[rows, V] logits ~ N(0, 2^2); a seeded Bernoulli(spike_p) subset of rows
    gets ``spike`` added at a seeded column.  ``spike_range=(lo, hi)`` draws the
    spike height uniformly instead (supplementary inputs that spread the
    confidences over (0, 1))."""
    rows = cfg.rows if rows is None else rows
    dt = cfg.torch_dtype()
    s = cfg.seed + 100 + 7 * step
    z = _normal((rows, cfg.V), s, device, torch.float32, std=2.0)
    g = _gen(s + 1, "cpu")
    is_spiked = torch.rand(rows, generator=g) < cfg.spike_p
    col = torch.randint(0, cfg.V, (rows,), generator=g)
    if spike_range is None:
        height = torch.full((rows,), float(cfg.spike))
    else:
        height = spike_range[0] + (spike_range[1] - spike_range[0]) * torch.rand(rows, generator=g)
    r = torch.nonzero(is_spiked).flatten()
    if r.numel():
        z[r.to(z.device), col[r].to(z.device)] += height[r].to(z.device)
    return z.to(dt)


def block_state(cfg: StepConfig, mode: str = "all", mask_id: int | None = None):
    """Token ids and mask flags of the current block: (x_block int32 [B,K],
    masked uint8 [B,K]).  mode "all": every position masked; "half": a seeded
    random half; "few": 1..12 seeded positions per sequence."""
    g = _gen(cfg.seed + 200, "cpu")
    mask_id = cfg.V - 1 if mask_id is None else mask_id
    B, K = cfg.B, cfg.K
    masked = torch.zeros(B, K, dtype=torch.uint8)
    for b in range(B):
        perm = torch.randperm(K, generator=g)
        if mode == "all":
            n = K
        elif mode == "half":
            n = K // 2
        elif mode == "few":
            n = int(torch.randint(1, min(12, K) + 1, (1,), generator=g))
        else:
            raise ValueError(mode)
        masked[b, perm[:n]] = 1
    x = torch.randint(0, max(mask_id, 1), (B, K), generator=g, dtype=torch.int32)
    x[masked.bool()] = mask_id
    return x, masked


def uniform_confidences(cfg: StepConfig, eos_id: int, eos_p: float = 0.05, step: int = 0):
    """Supplementary selection inputs: conf ~ U(0,1), tok ~ U{0..V-1} with
    ``eos_id`` planted with probability eos_p.  Returns (conf f32 [B,K], tok i32 [B,K])."""
    g = _gen(cfg.seed + 300 + step, "cpu")
    conf = torch.rand(cfg.B, cfg.K, generator=g, dtype=torch.float32)
    tok = torch.randint(0, cfg.V, (cfg.B, cfg.K), generator=g, dtype=torch.int32)
    plant = torch.rand(cfg.B, cfg.K, generator=g) < eos_p
    tok[plant] = eos_id
    return conf, tok


def lmhead_inputs(cfg: StepConfig, hid: int, device="cpu", rows: int | None = None, V: int | None = None):
    """Inputs of the fused output projection: hidden [rows, hid] ~ N(0,1) and an output embedding
    weight [V, hid] ~ N(0, 4/hid), so that the logits hidden @ weight.T are ~ N(0, 2^2) like the stored
    logits of ``logits``.  A seeded Bernoulli(spike_p) subset of rows gets the spike: the embedding of a
    seeded token is moved along that row's hidden vector so that its logit rises by about ``spike``."""
    rows = cfg.rows if rows is None else rows
    V = cfg.V if V is None else V
    s = cfg.seed + 400
    h = _normal((rows, hid), s, device, torch.float32)
    w = _normal((V, hid), s + 1, device, torch.float32, std=2.0 / hid ** 0.5)
    g = _gen(s + 2, "cpu")
    is_spiked = torch.rand(rows, generator=g) < cfg.spike_p
    col = torch.randint(0, V, (rows,), generator=g)
    r = torch.nonzero(is_spiked).flatten().to(h.device)
    if r.numel():
        hr = h[r]
        w[col[r.cpu()].to(h.device)] += float(cfg.spike) * hr / (hr * hr).sum(1, keepdim=True)
    return h.to(torch.bfloat16), w.to(torch.bfloat16)

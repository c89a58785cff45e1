#!/usr/bin/env python
"""Benchmark of one suffix-pruned denoising step on B200.

A step = ds_attn_pruned (once per resident layer cache) + ds_confidence +
ds_unmask_select over one batch of seeded synthetic input.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

* ``value``: denoise steps/s with every input resident in HBM, timed with CUDA
  events on the launching stream (max over ranks; ranks are independent replicas,
  each with its own batch: weak scaling, no collective on the data path).
* ``roofline``: the attention kernel's algorithmic bytes / its mean launch time
  (CUDA events inside the timed region) against the measured HBM peak.
* ``e2e``: the same step through the public API starting from pinned HOST
  buffers: host->device copies of everything the step reads and device->host
  copies of its results are inside the timed region.
* ``cpu_baseline``: the CPU oracle, as it stands, timed on the machine's host
  cores on a bounded sample of the same workload and scaled to a full step.
* ``--impl reference`` times that oracle as the main line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "pruned-step attn+confidence: denoise steps/s"
DEFAULT_CONFIG = "long32-w64"
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (bytes; None until a capture of that kernel and workload exists)
NCU_TRAFFIC: dict = {
    # captured on the batch-4 instance of the workload (the committed ncu summaries) and scaled by the items one launch
    # processes (x8: traffic is proportional to the rows streamed); set back to None when a kernel changes
    "long32-w64": {"attn_bytes_per_launch": 8 * (281.25e6 + 4.71e6), "confidence_bytes_per_launch": 8 * (64.78e6 + 0.32e6)},
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def attn_algorithmic_bytes(cfg, Lq):
    e = 4 if cfg.dtype == "f32" else 2
    kv_prefix = 2 * cfg.B * cfg.Hkv * cfg.P * cfg.D * e
    kv_tail = 2 * cfg.B * cfg.Hkv * Lq * cfg.D * e
    q = cfg.B * cfg.Hq * Lq * cfg.D * e
    return kv_prefix + kv_tail + 2 * q          # + O, same size as Q


def attn_flops(cfg, Lq):
    return 4 * cfg.B * cfg.Hq * Lq * (cfg.P + Lq) * cfg.D


def conf_algorithmic_bytes(cfg):
    e = 4 if cfg.dtype == "f32" else 2
    return cfg.rows * cfg.V * e + 8 * cfg.rows


# --------------------------------------------------------------------------
# replicas: the path has no exchange step, so N GPUs run N independent batches
# --------------------------------------------------------------------------
def rank_config(cfg, rank):
    """The batch of one replica: same shapes, its own seeds."""
    from paper_2601_17917_b200 import workloads as wl
    return wl.shrink(cfg, seed=cfg.seed + 100000 * rank)


def max_over_ranks(value, world, device):
    """Slowest rank's time (the job's time).  The only collective of a multi-rank run, outside the timed region."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world, ms_per_step):
    """Whole-job steps/s: every replica completes one step of its own batch per ms_per_step."""
    return world * 1e3 / ms_per_step


def replica_command(n, argv, port=None):
    """The command that starts ``n`` ranks of this script on this node, one per GPU (the launch the multi-GPU
    contract describes: torch.distributed.run, rendezvous on 127.0.0.1)."""
    if port is None:
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *argv]


def spawn_replicas(n, argv):
    import subprocess
    return subprocess.call(replica_command(n, argv))


def dry_run(args, cfg):
    """What a multi-rank run adds to a single-GPU one, without a GPU: the ranks come up, each derives its own
    seeded batch, the slowest rank's (here: made-up) time becomes the job's time, rank 0 prints the line."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo")
    rcfg = rank_config(cfg, rank)
    seeds = [None] * world
    if world > 1:
        dist.all_gather_object(seeds, rcfg.seed)
    else:
        seeds = [rcfg.seed]
    ms = max_over_ranks(1.0 + rank, world, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"dry_run": True, "metric": METRIC, "n_gpus": world, "value": job_throughput(world, ms),
                          "unit": "steps/s", "ms_per_step": ms, "scaling": "weak", "rank_seeds": seeds,
                          "config": {"workload": cfg.name, "parallelism": f"replicas x{world}"}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------
# clock sampling (read-only NVML)
# --------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, torch_device_index: int, period_s: float = 0.004):
        self.samples = []      # (t, sm_mhz, reasons bitmask)
        self.period = period_s
        self._stop = threading.Event()
        self._thread = None
        self.h = None
        self.max_mhz = None
        try:
            import pynvml
            import torch
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as exc:  # NVML missing: report that, do not fail the run
            self.err = repr(exc)
            self.h = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    rs = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.perf_counter(), mhz, rs))
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, windows):
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        sel = [s for s in self.samples if any(a <= s[0] <= b for a, b in windows)]
        if not sel:
            sel = self.samples
        mhz = sorted(s[1] for s in sel)
        mask = 0
        for s in sel:
            mask |= s[2]
        reasons = [n for bit, n in self.REASONS.items() if mask & bit]
        return {"sm_mhz": mhz[len(mhz) // 2] if mhz else None, "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(sel)}


# --------------------------------------------------------------------------
# the GPU step
# --------------------------------------------------------------------------
class Step:
    """Device-resident inputs of one configuration and the three C-ABI calls of a step."""

    def __init__(self, cfg, device, compact_tail=False, stages=("attn", "confidence", "select"), fused_lmhead=False):
        import torch
        self.stages = tuple(stages)
        self.fused_lmhead = fused_lmhead
        import paper_2601_17917_b200 as ds
        from paper_2601_17917_b200 import workloads as wl
        self.torch, self.ds, self.cfg, self.device = torch, ds, cfg, device
        idx = ds.retained_indices(cfg.gen, cfg.K, 0, cfg.w, cfg.keep_last)
        self.Lq = len(idx)
        self.layers = []
        # a configuration whose per-step attention inputs would fit in L2 gets independent seeded copies,
        # rotated from step to step, so that every timed launch streams from HBM
        foot = attn_algorithmic_bytes(cfg, self.Lq) * cfg.n_layers
        self.copies = 1 if foot >= 256e6 else min(16, int(math.ceil(256e6 / foot)))
        self.tick = 0
        for layer in range(cfg.n_layers * self.copies):
            x = wl.attention_inputs(cfg, device=device, layer=layer)
            if compact_tail:
                sel = torch.tensor(idx, device=device)
                for k in ("q_tail", "k_tail", "v_tail"):
                    x[k] = x[k][:, :, sel].contiguous()
            self.layers.append(x)
        if compact_tail:
            idx = list(range(self.Lq))
        self.idx = torch.tensor(idx, dtype=torch.int32, device=device)
        self.scale = 1.0 / math.sqrt(cfg.D)
        if fused_lmhead:
            # the widened path: hidden states in, Eq. 4 out, the [rows x V] logits never stored
            self.hidden, self.weight = wl.lmhead_inputs(cfg, HIDDEN_SIZE.get(cfg.V, 4096), device=device)
            self.logits = None
            self.lm_ws = torch.empty(max(ds.ds_lmhead_confidence_workspace(cfg.rows, cfg.V), 256), dtype=torch.uint8,
                                     device=device)
        else:
            self.logits = wl.logits(cfg, device=device)
        x0, m0 = wl.block_state(cfg, "all")
        self.x0, self.m0 = x0.to(device), m0.to(device)
        self.x_block, self.masked = self.x0.clone(), self.m0.clone()
        self.no_exit = torch.zeros(cfg.B, dtype=torch.uint8, device=device)
        dt = cfg.torch_dtype()
        B, K = cfg.B, cfg.K
        self.out = torch.empty((B, cfg.Hq, self.Lq, cfg.D), dtype=dt, device=device)
        self.conf = torch.empty(cfg.rows, dtype=torch.float32, device=device)
        self.tok = torch.empty(cfg.rows, dtype=torch.int32, device=device)
        self.sel = dict(sel_idx=torch.empty((B, K), dtype=torch.int32, device=device),
                        sel_cnt=torch.zeros(B, dtype=torch.int32, device=device),
                        block_done=torch.zeros(B, dtype=torch.uint8, device=device),
                        eos_exit=torch.zeros(B, dtype=torch.uint8, device=device),
                        active_seq=torch.empty(B, dtype=torch.int32, device=device),
                        active_cnt=torch.zeros(1, dtype=torch.int32, device=device))
        x = self.layers[0]
        need = ds.ds_attn_pruned_workspace(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"],
                                           self.idx, self.scale, self.out)
        self.attn_ws = torch.empty(max(need, 256), dtype=torch.uint8, device=device)
        self.conf_ws = torch.empty(max(ds.ds_confidence_workspace(cfg.rows, cfg.V, dt), 256), dtype=torch.uint8,
                                   device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)

    def attn(self, layer=0):
        x = self.layers[(self.tick % self.copies) * self.cfg.n_layers + layer]
        self.ds.ds_attn_pruned(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"], self.idx, self.scale,
                               out=self.out, workspace=self.attn_ws, status=self.status)

    def confidence(self):
        if self.fused_lmhead:
            self.ds.ds_lmhead_confidence(self.hidden, self.weight, conf=self.conf, tok=self.tok, workspace=self.lm_ws,
                                         status=self.status)
        else:
            self.ds.ds_confidence(self.logits, conf=self.conf, tok=self.tok, workspace=self.conf_ws)

    def select(self):
        cfg = self.cfg
        # every timed step starts from the state a block begins with (every position masked)
        self.ds.ds_block_begin(self.no_exit, self.masked, self.x_block, cfg.V - 1, cfg.V - 2, self.sel["active_seq"],
                               self.sel["active_cnt"])
        self.ds.ds_unmask_select(self.conf.view(cfg.B, cfg.K), self.tok.view(cfg.B, cfg.K), self.masked, self.x_block,
                                 cfg.tau0, cfg.alpha, eos_id=cfg.V - 2, eos_tau=cfg.tau0, out=self.sel)

    def run(self, events=None):
        """One whole step.  ``events``: optional [4] CUDA events recorded between the stages."""
        if events:
            events[0].record()
        if "attn" in self.stages:
            for layer in range(self.cfg.n_layers):
                self.attn(layer)
        if events:
            events[1].record()
        if "confidence" in self.stages:
            self.confidence()
        if events:
            events[2].record()
        if "select" in self.stages:
            self.select()
        if events:
            events[3].record()
        self.tick += 1


def time_resident(step, steps, warmup, sampler, barrier):
    torch = step.torch
    for _ in range(warmup):
        step.run()
    torch.cuda.synchronize()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    barrier()
    torch.cuda.synchronize()
    launches0 = step.ds.ds_launch_count()
    t0 = time.perf_counter()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(steps):
        step.run(evs[i])
    end.record()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    barrier()
    total_ms = start.elapsed_time(end)
    launches = step.ds.ds_launch_count() - launches0
    stage_ms = [sum(e[k].elapsed_time(e[k + 1]) for e in evs) / steps for k in range(3)]
    windows = [(t0, t1)]
    # the sampler needs a few samples under this load: if the timed region was short, run identical
    # (untimed) steps for a moment longer
    extra = 0
    if sampler is not None and (t1 - t0) < 0.25:
        t2 = time.perf_counter()
        while time.perf_counter() - t2 < 0.3:
            for _ in range(8):
                step.run()
            torch.cuda.synchronize()
            extra += 8
        windows.append((t2, time.perf_counter()))
    return total_ms, stage_ms, launches, windows, extra


def time_attn_sustained(step, device_index, seconds=2.0, chunk=64):
    """The attention stage alone, back to back for at least ``seconds``: long enough for the power cap to settle
    the SM clock.  CUDA events every ``chunk`` launches; clocks sampled over the same window.  Returns the mean
    launch time of the whole region and of its second half, with the median SM clock of each."""
    torch = step.torch
    for _ in range(3):
        step.attn(0)
    torch.cuda.synchronize()
    sampler = ClockSampler(device_index)
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True)]
    evs[0].record()
    t0 = time.perf_counter()
    stamps = [t0]                            # host time at which chunk i - 1 had finished
    n = 0
    while True:
        for i in range(chunk):
            step.attn((n + i) % step.cfg.n_layers)
            if (n + i + 1) % step.cfg.n_layers == 0:
                step.tick += 1
        n += chunk
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        evs.append(e)
        evs[-2].synchronize()                # the chunk before this one is done; this one keeps the GPU busy
        stamps.append(time.perf_counter())
        if stamps[-1] - t0 >= seconds:
            break
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    sampler.stop()
    k = len(evs) - 1
    whole_ms = evs[0].elapsed_time(evs[k])
    half = k // 2
    tail_ms = evs[half].elapsed_time(evs[k])
    cl_all = sampler.summary([(t0, t1)])
    cl_tail = sampler.summary([(stamps[half], t1)])
    return {"launches": n, "seconds": whole_ms * 1e-3, "us_per_launch": whole_ms * 1e3 / n,
            "sm_mhz": cl_all["sm_mhz"], "reasons": cl_all["reasons"],
            "second_half": {"launches": n - half * chunk, "us_per_launch": tail_ms * 1e3 / max(1, n - half * chunk),
                            "sm_mhz": cl_tail["sm_mhz"]}}


def time_e2e(cfg, device, steps, warmup, cache_resident=False, fused_lmhead=False):
    """Same step from pinned host buffers: H2D of everything the step reads, the three calls,
    D2H of the results, all inside the timed region.  ``cache_resident``: the prefix KV cache stays on
    the device (the method computes it once per block and reuses it at every step); only what changes
    from step to step is copied.  ``fused_lmhead``: the step ends in ds_lmhead_confidence instead of
    ds_confidence, so the hidden states of the block's rows cross the link instead of their logits (the output
    embedding stays on the device like any weight)."""
    import torch
    dev_step = Step(cfg, device, compact_tail=True, fused_lmhead=fused_lmhead)
    host_in, dev_in = [], []
    for x in dev_step.layers:
        for k in ("q_tail", "k_tail", "v_tail") + (() if cache_resident else ("k_pre", "v_pre")):
            dev_in.append(x[k])
    dev_in += [dev_step.hidden if fused_lmhead else dev_step.logits, dev_step.x_block, dev_step.masked, dev_step.idx]
    for t in dev_in:
        h = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        h.copy_(t)
        host_in.append(h)
    dev_out = [dev_step.out, dev_step.x_block, dev_step.masked, dev_step.sel["sel_idx"], dev_step.sel["sel_cnt"],
               dev_step.sel["block_done"], dev_step.sel["eos_exit"], dev_step.sel["active_seq"],
               dev_step.sel["active_cnt"]]
    host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in dev_out]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    def one():
        for h, d in zip(host_in, dev_in):
            d.copy_(h, non_blocking=True)
        dev_step.run()
        for h, d in zip(host_out, dev_out):
            h.copy_(d, non_blocking=True)

    for _ in range(max(1, min(warmup, 3))):
        one()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        one()
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end) / steps, h2d, d2h


# --------------------------------------------------------------------------
# CPU oracle timing (baseline leg and --impl reference)
# --------------------------------------------------------------------------
class OracleSample:
    """A bounded sample of the workload for the CPU oracle: ``n_slices`` (batch, head) attention
    slices of one layer, ``n_rows`` logit rows, and the full selection.  ``time()`` runs the
    oracle on it and returns the seconds a whole step would take at that rate (linear scaling over
    slices, rows and layers)."""

    def __init__(self, cfg, n_slices, n_rows):
        import numpy as np
        import oracle
        from paper_2601_17917_b200 import workloads as wl
        self.np, self.oracle, self.cfg = np, oracle, cfg
        w = cfg.w if cfg.w >= 0 else cfg.gen
        self.idx = np.asarray(oracle.retained_indices(cfg.gen, cfg.K, 0, w, cfg.keep_last))
        n_slices = min(n_slices, cfg.B * cfg.Hq)
        hs = min(cfg.Hq, n_slices)
        bs = max(1, n_slices // hs)
        G = cfg.Hq // cfg.Hkv
        small = wl.shrink(cfg, B=bs, Hq=hs, Hkv=hs // G if hs % G == 0 else hs)
        self.small = small
        self.x = {k: v.float().numpy() for k, v in wl.attention_inputs(small, device="cpu").items()}
        self.n_rows = min(n_rows, cfg.rows)
        self.z = wl.logits(cfg, device="cpu", rows=self.n_rows).float().numpy()
        self.conf = np.random.default_rng(0).random((cfg.B, cfg.K)).astype(np.float32)
        self.tok = np.zeros((cfg.B, cfg.K), np.int32)
        xb, mk = wl.block_state(cfg, "all")
        self.xb, self.mk = xb.numpy(), mk.numpy()
        self.scale = 1.0 / math.sqrt(cfg.D)
        self.cores = oracle.num_threads()
        self.sample = (f"{small.B * small.Hq} of {cfg.B * cfg.Hq} (batch, head) attention slices of one layer, "
                       f"{self.n_rows} of {cfg.rows} logit rows, full selection; scaled linearly to one step"
                       + (f" x {cfg.n_layers} layers" if cfg.n_layers > 1 else ""))

    def time(self):
        cfg, x, o = self.cfg, self.x, self.oracle
        t0 = time.perf_counter()
        o.attn(x["q_tail"], x["k_tail"], x["v_tail"], x["k_pre"], x["v_pre"], self.idx, self.scale)
        t1 = time.perf_counter()
        o.confidence(self.z)
        t2 = time.perf_counter()
        o.select(self.conf, self.tok, self.mk, self.xb, cfg.tau0, cfg.alpha)
        t3 = time.perf_counter()
        full = ((t1 - t0) * (cfg.B * cfg.Hq) / (self.small.B * self.small.Hq) * cfg.n_layers
                + (t2 - t1) * cfg.rows / self.n_rows + (t3 - t2))
        return full, t3 - t0


HIDDEN_SIZE = {126464: 4096, 152064: 3584}   # hidden size of the model a vocabulary size belongs to


def time_lmhead(cfg, device, reps=10):
    """The widened path: output projection fused with Eq. 4 (ds_lmhead_confidence), timed alone with CUDA
    events, and the unfused alternative (library GEMM writing bf16 logits + ds_confidence) beside it."""
    import torch
    import paper_2601_17917_b200 as ds
    from paper_2601_17917_b200 import workloads as wl
    hid = HIDDEN_SIZE.get(cfg.V, 4096)
    h, w = wl.lmhead_inputs(cfg, hid, device=device)
    rows, V = cfg.rows, cfg.V
    ws = torch.empty(max(ds.ds_lmhead_confidence_workspace(rows, V), 256), dtype=torch.uint8, device=device)
    conf = torch.empty(rows, dtype=torch.float32, device=device)
    tok = torch.empty(rows, dtype=torch.int32, device=device)
    z = torch.empty(rows, V, dtype=torch.bfloat16, device=device)
    cws = torch.empty(max(ds.ds_confidence_workspace(rows, V, torch.bfloat16), 256), dtype=torch.uint8, device=device)

    def fused():
        ds.ds_lmhead_confidence(h, w, conf=conf, tok=tok, workspace=ws)

    def unfused():
        torch.matmul(h, w.T, out=z)
        ds.ds_confidence(z, conf=conf, tok=tok, workspace=cws)

    out = {}
    for name, fn in (("fused", fused), ("unfused", unfused)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        out[name] = a.elapsed_time(b) / reps
    flops = 2.0 * rows * hid * V
    return out, flops, hid, V * hid * 2 + rows * hid * 2


def time_decode_loop(device, n_blocks=8, batches=(8, 1)):
    """The whole block-wise procedure on the LLaDA-shaped configuration (32 layers, prompt 1024, n_blocks blocks
    of 32; 8 sequences, and 1 as in the paper's per-sample latency figures), driven by decode.BlockDecoder with
    the attention side of every layer done as the method does it.  Per layer the seeded buffers are un-rotated
    Q/K/V projections of every position and a prefix KV cache that starts with the prompt's rows:
      first iteration of block n   the finished block n-1 joins the cache (ds_rope_gather, n_append = K); dense
                                   attention over prefix + retained rows with nothing cached (rotary encoding +
                                   gather of all rows, then ds_attn_pruned with P = 0)
      later iterations             rotary encoding + gather of the retained tail rows, ds_attn_pruned over the
                                   cache rows 0 .. P + n K and the retained rows
    so block n + 1 attends over what block n appended.  The model's other layers are absent: the logits of an
    iteration are staged from a small pool of seeded buffers.  Three ways to drive the same device work: the
    synchronous loop (the host waits for every iteration), the host running two iterations ahead, and the latter
    with every iteration replayed as one CUDA graph."""
    import torch
    import paper_2601_17917_b200 as ds
    from paper_2601_17917_b200 import workloads as wl
    from paper_2601_17917_b200.decode import BlockDecoder
    base = wl.CONFIGS["llada8x32"]
    res = {"what": "whole block-wise decode (per layer: rotary encoding + gather, pruned attention over the growing "
                   "prefix cache, cache append at every block boundary; early exit off); not part of `value`",
           "blocks": n_blocks, "K": base.K, "n_layers": base.n_layers, "P": base.P, "batches": {}}
    status = torch.zeros(1, dtype=torch.int32, device=device)
    theta = 10000.0
    for nb in batches:
        cfg = wl.shrink(base, B=nb, gen=n_blocks * base.K, name=f"llada{nb}x32-decode")
        B, K, L, P, D, Hq, Hkv = cfg.B, cfg.K, cfg.gen, cfg.P, cfg.D, cfg.Hq, cfg.Hkv
        dt = cfg.torch_dtype()
        # per layer: raw projections of prompt + generation, and the cache (prompt rows filled below)
        raws, caches = [], []
        for l in range(cfg.n_layers):
            x = wl.attention_inputs(wl.shrink(cfg, P=0, gen=P + L, name="raw"), device=device, layer=l)
            raws.append((x["q_tail"], x["k_tail"], x["v_tail"]))
            caches.append((torch.zeros((B, Hkv, P + L, D), dtype=dt, device=device),
                           torch.zeros((B, Hkv, P + L, D), dtype=dt, device=device)))
        pool = [wl.logits(cfg, device=device, step=s, spike_range=(14.0, 26.0)) for s in range(4)]
        scale = 1.0 / math.sqrt(D)
        Lq_max = len(ds.retained_indices(L, K, 0, cfg.w, cfg.keep_last))
        n_max = P + L                                    # rows of a refresh iteration never exceed the sequence
        # compact rotated rows of the layer being processed (shared by the layers: they run one after another)
        qc = torch.empty((B, Hq, n_max, D), dtype=dt, device=device)
        kc = torch.empty((B, Hkv, n_max, D), dtype=dt, device=device)
        vc = torch.empty((B, Hkv, n_max, D), dtype=dt, device=device)
        out = torch.empty((B, Hq, n_max, D), dtype=dt, device=device)
        ar = torch.arange(n_max, dtype=torch.int32, device=device)
        rows_all = {}                                    # block -> rows of its refresh iteration (absolute positions)
        for n in range(n_blocks):
            keep = torch.tensor(ds.retained_indices(L, K, n, cfg.w, cfg.keep_last), dtype=torch.int32, device=device)
            rows_all[n] = torch.cat([ar[:P + n * K], keep + (P + n * K)])

        def prefill():
            for (q, k, v), (ck, cv) in zip(raws, caches):
                ds.ds_rope_gather(q, k, v, ar[:P], 0, theta, q_out=qc[:, :, :P], k_out=kc[:, :, :P], v_out=vc[:, :, :P],
                                  k_cache=ck, v_cache=cv, cache_row0=0, n_append=P, status=status)

        def forward_for(dec):
            # the attention calls of a block repeat with the same pointers: plan them once per block
            plans = {}

            def forward(st):
                n, b0 = st.n, P + st.n * K               # b0: rows of the cache in use = position of tail row 0
                key = (n, st.refresh)
                if st.refresh:
                    rows = rows_all[n]
                    nr = rows.numel()
                    if key not in plans:
                        plans[key] = ds.AttnPlan(qc[:, :, :nr], kc[:, :, :nr], vc[:, :, :nr], None, None, ar[:nr], scale,
                                                 out=out[:, :, :nr], status=status, seq_list=st.active_seq, n_seq=B,
                                                 n_seq_dev=st.active_cnt)
                    for (q, k, v), (ck, cv) in zip(raws, caches):
                        if n > 0:                        # the finished block joins the prefix
                            ds.ds_rope_gather(q[:, :, b0 - K:], k[:, :, b0 - K:], v[:, :, b0 - K:], ar[:K], b0 - K, theta,
                                              q_out=qc[:, :, :K], k_out=kc[:, :, :K], v_out=vc[:, :, :K], k_cache=ck,
                                              v_cache=cv, cache_row0=b0 - K, n_append=K, status=status)
                        ds.ds_rope_gather(q, k, v, rows, 0, theta, q_out=qc[:, :, :nr], k_out=kc[:, :, :nr],
                                          v_out=vc[:, :, :nr], status=status)
                        plans[key].launch()
                else:
                    lq = st.idx.numel()
                    if key not in plans:
                        plans[key] = [ds.AttnPlan(qc[:, :, :lq], kc[:, :, :lq], vc[:, :, :lq], ck[:, :, :b0], cv[:, :, :b0],
                                                  ar[:lq], scale, out=out[:, :, :lq], status=status, seq_list=st.active_seq,
                                                  n_seq=B, n_seq_dev=st.active_cnt) for ck, cv in caches]
                    for (q, k, v), pl in zip(raws, plans[key]):
                        ds.ds_rope_gather(q[:, :, b0:], k[:, :, b0:], v[:, :, b0:], st.idx, b0, theta, q_out=qc[:, :, :lq],
                                          k_out=kc[:, :, :lq], v_out=vc[:, :, :lq], status=status)
                        pl.launch()
            return forward

        runs = {}
        for name, la, graphs in (("sync", 0, False), ("lookahead2", 2, False), ("lookahead2_graphs", 2, True)):
            dec = BlockDecoder(B, L, K, cfg.V, tau0=cfg.tau0, alpha=cfg.alpha, mask_id=cfg.V - 1, w_tokens=cfg.w,
                               keep_last=cfg.keep_last, device=device, lookahead=la)
            forward = forward_for(dec)
            stage = lambda n, t: dec.logits.copy_(pool[(n + t) % len(pool)])
            prefill()
            dec.decode(forward, before_iteration=stage, graphs=graphs)      # warm-up: plans, graph capture
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            n0 = ds.ds_launch_count()
            a.record()
            got = dec.decode(forward, before_iteration=stage, graphs=graphs)
            b.record()
            torch.cuda.synchronize()
            ms = a.elapsed_time(b)
            runs[name] = {"ms": ms, "iterations": int(sum(got["steps"])),
                          "iterations_enqueued": int(sum(got["launched"])),
                          "ms_per_iteration": ms / max(1, sum(got["steps"])),
                          "host_launch_calls": int(ds.ds_launch_count() - n0)}
            del dec, forward
        res["batches"][f"B{nb}"] = runs
        del raws, caches, pool, qc, kc, vc, out
        torch.cuda.empty_cache()
    res["device_status"] = int(ds.ds_read_status(status))
    return res


def time_rope(cfg, device, reps=20):
    """The widened path: rotary encoding + gather of the retained rows (ds_rope_gather), timed alone."""
    import torch
    import paper_2601_17917_b200 as ds
    from paper_2601_17917_b200 import workloads as wl
    x = wl.attention_inputs(cfg, device=device)
    idx = torch.tensor(ds.retained_indices(cfg.gen, cfg.K, 0, cfg.w, cfg.keep_last), dtype=torch.int32, device=device)
    Lq = idx.numel()
    qo = torch.empty((cfg.B, cfg.Hq, Lq, cfg.D), dtype=torch.bfloat16, device=device)
    ko = torch.empty((cfg.B, cfg.Hkv, Lq, cfg.D), dtype=torch.bfloat16, device=device)
    vo = torch.empty_like(ko)

    def fn():
        ds.ds_rope_gather(x["q_tail"], x["k_tail"], x["v_tail"], idx, cfg.P, 10000.0, q_out=qo, k_out=ko, v_out=vo)

    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        fn()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    nbytes = 2 * cfg.B * (cfg.Hq + 2 * cfg.Hkv) * Lq * cfg.D * 2       # every retained row read once, written once
    return ms, nbytes


def run_reference(args, cfg):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    smp = OracleSample(cfg, 32, 256)
    for _ in range(min(args.warmup, 1)):
        smp.time()
    times = []
    t_all0 = time.perf_counter()
    for _ in range(max(args.steps, 1)):
        times.append(smp.time()[0])
        if time.perf_counter() - t_all0 > 150:       # bounded: a few minutes at most
            break
    sec = sum(times) / len(times)
    line = {
        "impl": "reference", "metric": METRIC, "value": 1.0 / sec, "unit": "steps/s", "n_gpus": args.gpus,
        "steps": len(times), "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "P": cfg.P,
                   "gen": cfg.gen, "K": cfg.K, "Lq": int(len(smp.idx)), "V": cfg.V, "n_layers": cfg.n_layers},
        "cpu_baseline": {"value": 1.0 / sec, "unit": "steps/s", "cores": smp.cores, "kind": "oracle",
                         "sample": smp.sample},
        "e2e": {"value": 1.0 / sec, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-lmhead", action="store_true", help="skip the extra timing of ds_lmhead_confidence")
    ap.add_argument("--no-decode-loop", action="store_true", help="skip the extra timing of the block-wise decode loop")
    ap.add_argument("--no-sustained", action="store_true",
                    help="skip the seconds-long attention-only region behind `roofline_sustained`")
    ap.add_argument("--sustained-seconds", type=float, default=2.0)
    ap.add_argument("--dry-run", action="store_true",
                    help="launch plumbing only: ranks, seeds and the max-over-ranks reduction on CPU (gloo), no GPU work")
    ap.add_argument("--stages", default="attn,confidence,select",
                    help="comma list of the stages a step runs (profiling a single kernel)")
    ap.add_argument("--vocab", type=int, default=0, help="override the vocabulary size (small profiler cases)")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the batch size of the configuration (small cases for profiler captures)")
    args = ap.parse_args()

    from paper_2601_17917_b200 import workloads as wl
    cfg = wl.CONFIGS[args.config]
    if args.batch > 0:
        cfg = wl.shrink(cfg, B=args.batch, name=f"{cfg.name}-B{args.batch}")
    if args.vocab > 0:
        cfg = wl.shrink(cfg, V=args.vocab, name=f"{cfg.name}-V{args.vocab}")
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started bare: become the launcher of N ranks (one per GPU) and pass their exit code on
        raise SystemExit(spawn_replicas(args.gpus, sys.argv[1:]))
    if args.dry_run:
        dry_run(args, cfg)
        return

    import torch
    import torch.distributed as dist
    import paper_2601_17917_b200 as ds
    ds.lib()                     # fail loudly if the CUDA library is not built: there is no fallback
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback exists)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()

    if args.stages == "lmhead":            # profiling run of the widened kernel alone
        t, flops, hid, in_bytes = time_lmhead(cfg, device, reps=max(1, args.steps))
        print(json.dumps({"stages": "lmhead", "config": {"workload": cfg.name, "rows": cfg.rows, "hidden": hid, "V": cfg.V},
                          "ms": t["fused"], "tflops": flops / (t["fused"] * 1e-3) / 1e12, "unfused_ms": t["unfused"]}),
              flush=True)
        return
    if args.stages == "rope":              # profiling run of the widened kernel alone
        ms, nbytes = time_rope(cfg, device, reps=max(1, args.steps))
        print(json.dumps({"stages": "rope", "config": {"workload": cfg.name}, "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9}),
              flush=True)
        return
    warmup = max(args.warmup, 3)
    # replicas: every rank draws its own batch (its rank offsets the seed); no data-path collective
    rcfg = rank_config(cfg, rank)
    step = Step(rcfg, device, stages=args.stages.split(","))
    sampler = ClockSampler(local)
    sampler.start()
    total_ms, stage_ms, launches, windows, extra = time_resident(step, args.steps, warmup, sampler, barrier)
    sampler.stop()
    clocks = sampler.summary(windows)
    if extra:
        clocks["note"] = f"timed region + {extra} further identical steps"
    sustained = None
    if not args.no_sustained and "attn" in step.stages and args.sustained_seconds > 0:
        sustained = time_attn_sustained(step, local, seconds=args.sustained_seconds)
        barrier()
    status = ds.ds_read_status(step.status)
    total_ms = max_over_ranks(total_ms, world, device)
    ms_per_step = total_ms / args.steps
    value = job_throughput(world, ms_per_step)

    e2e = None
    if not args.no_e2e and args.stages == "attn,confidence,select":
        e2e_steps = max(3, min(args.steps, 20))
        step.layers.clear()
        torch.cuda.empty_cache()
        e_ms, h2d, d2h = time_e2e(rcfg, device, e2e_steps, 3)
        e_ms = max_over_ranks(e_ms, world, device)
        e2e = {"value": job_throughput(world, e_ms), "unit": "steps/s", "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e_ms, "steps": e2e_steps,
               "layout": "tail rows shipped compact (T = Lq): only what the step reads crosses the link"}
        # second figure: the prefix KV cache resident, as it is between the steps of a block
        r_ms, r_h2d, r_d2h = time_e2e(rcfg, device, e2e_steps, 3, cache_resident=True)
        r_ms = max_over_ranks(r_ms, world, device)
        e2e["prefix_cache_resident"] = {"value": job_throughput(world, r_ms), "unit": "steps/s", "ms_per_step": r_ms,
                                        "h2d_bytes_per_step": int(r_h2d), "d2h_bytes_per_step": int(r_d2h)}
        # third figure: cache resident and the step ending in the fused output projection (hidden states in)
        if cfg.dtype == "bf16":
            f_ms, f_h2d, f_d2h = time_e2e(rcfg, device, e2e_steps, 3, cache_resident=True, fused_lmhead=True)
            f_ms = max_over_ranks(f_ms, world, device)
            e2e["fused_lmhead"] = {"value": job_throughput(world, f_ms), "unit": "steps/s", "ms_per_step": f_ms,
                                   "h2d_bytes_per_step": int(f_h2d), "d2h_bytes_per_step": int(f_d2h),
                                   "what": "prefix cache and output embedding resident; hidden states of the block's rows "
                                           "copied in; ds_lmhead_confidence in place of logits + ds_confidence"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    Lq = step.Lq
    a_bytes = attn_algorithmic_bytes(cfg, Lq)
    a_ms = stage_ms[0] / cfg.n_layers
    a_gbs = a_bytes / (a_ms * 1e-3) / 1e9
    c_bytes = conf_algorithmic_bytes(cfg)
    c_gbs = c_bytes / (stage_ms[1] * 1e-3) / 1e9
    fl = attn_flops(cfg, Lq)
    traffic = NCU_TRAFFIC.get(cfg.name, {})
    # the attention call is bound by whichever ideal time is longer: its bytes at the copy bandwidth or its
    # flops at the sustained GEMM rate (the pruned step: bytes; the dense first step of a block: flops)
    a_tf = fl / (a_ms * 1e-3) / 1e12
    if fl / (pk["bf16_tflops_sustained"] * 1e12) > a_bytes / (pk["hbm_gbs"] * 1e9) and cfg.dtype == "bf16":
        attn_roof = {"kernel": "ds_attn_pruned", "bound": "tensor", "achieved": a_tf, "peak": pk["bf16_tflops_sustained"],
                     "unit": "TFLOP/s", "frac": a_tf / pk["bf16_tflops_sustained"], "traffic": None,
                     "peak_source": pk["_source"] + " (sustained)", "algorithmic_flops": fl,
                     "hbm_frac": a_gbs / pk["hbm_gbs"]}
    else:
        attn_roof = {"kernel": "ds_attn_pruned", "bound": "hbm", "achieved": a_gbs, "peak": pk["hbm_gbs"],
                     "unit": "GB/s", "frac": a_gbs / pk["hbm_gbs"], "traffic": traffic.get("attn_bytes_per_launch"),
                     "peak_source": pk["_source"], "algorithmic_bytes": a_bytes, "tflops": a_tf,
                     "tensor_frac_of_sustained": a_tf / pk["bf16_tflops_sustained"]}
    line = {
        "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "Hq": cfg.Hq, "Hkv": cfg.Hkv, "D": cfg.D, "P": cfg.P,
                   "gen": cfg.gen, "K": cfg.K, "window_tokens": cfg.w, "Lq": Lq, "Lkv": cfg.P + Lq, "V": cfg.V,
                   "n_layers": cfg.n_layers, "tau0": cfg.tau0, "alpha": cfg.alpha, "parallelism": f"replicas x{world}",
                   "l2": "inputs larger than L2 (KV cache and logits of one step exceed 126 MB)"
                   if a_bytes * cfg.n_layers + c_bytes > 2 * 126e6 else "working set near L2 size"},
        "tokens_per_s": {"query_tokens": value * cfg.B * Lq,
                         "committed_tokens": value * float(step.sel["sel_cnt"].sum().item())},
        "stage_ms": {"attn_per_layer": a_ms, "confidence": stage_ms[1], "select": stage_ms[2]},
        "roofline": attn_roof,
        "roofline_confidence": {"kernel": "ds_confidence", "bound": "hbm", "achieved": c_gbs, "peak": pk["hbm_gbs"],
                                "unit": "GB/s", "frac": c_gbs / pk["hbm_gbs"],
                                "traffic": traffic.get("confidence_bytes_per_launch"), "peak_source": pk["_source"],
                                "algorithmic_bytes": c_bytes},
        "clocks": clocks, "gpu_launches": int(launches), "device_status": int(status),
    }
    if clocks.get("sm_mhz"):
        line["roofline"]["us_per_launch"] = a_ms * 1e3
        line["roofline"]["us_x_mhz"] = a_ms * 1e3 * clocks["sm_mhz"]
    if sustained is not None:
        # the same kernel over seconds of back-to-back launches: the power cap has settled the SM clock, so this is
        # the figure a long-running decode sees; time x clock says how much of the difference is the clock
        def entry(us, mhz):
            if attn_roof["bound"] == "hbm":
                ach, peak, unit = a_bytes / (us * 1e-6) / 1e9, pk["hbm_gbs"], "GB/s"
            else:
                ach, peak, unit = fl / (us * 1e-6) / 1e12, pk["bf16_tflops_sustained"], "TFLOP/s"
            return {"achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak, "us_per_launch": us, "sm_mhz": mhz,
                    "us_x_mhz": us * mhz if mhz else None}
        rs = entry(sustained["us_per_launch"], sustained["sm_mhz"])
        rs.update({"kernel": "ds_attn_pruned", "bound": attn_roof["bound"], "seconds": sustained["seconds"],
                   "launches": sustained["launches"], "reasons": sustained["reasons"], "peak_source": attn_roof["peak_source"],
                   "second_half": entry(sustained["second_half"]["us_per_launch"], sustained["second_half"]["sm_mhz"])})
        line["roofline_sustained"] = rs
    if args.stages != "attn,confidence,select":
        line["stages"] = args.stages          # partial step: a profiling run, not a bench value
    if e2e:
        line["e2e"] = e2e
    if not args.no_lmhead and args.stages == "attn,confidence,select":
        del step
        torch.cuda.empty_cache()
        r_ms, r_bytes = time_rope(cfg, device)
        line["rope_gather"] = {"what": "rotary encoding + gather of the retained rows; not part of `value`", "ms": r_ms,
                               "roofline": {"kernel": "ds_rope_gather", "bound": "hbm", "achieved": r_bytes / (r_ms * 1e-3) / 1e9,
                                            "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": r_bytes / (r_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                                            "algorithmic_bytes": r_bytes, "traffic": None, "peak_source": pk["_source"]}}
        torch.cuda.empty_cache()
        t, flops, hid, in_bytes = time_lmhead(cfg, device)
        tf = flops / (t["fused"] * 1e-3) / 1e12
        line["lmhead_confidence"] = {
            "what": "output projection fused with Eq. 4 (logits never stored); not part of `value`",
            "rows": cfg.rows, "hidden": hid, "V": cfg.V, "ms": t["fused"],
            "roofline": {"kernel": "ds_lmhead_confidence", "bound": "tensor", "achieved": tf, "peak": pk["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": tf / pk["bf16_tflops"], "peak_source": pk["_source"] + " (burst)",
                         "traffic": None},
            "weight_stream_gbs": in_bytes / (t["fused"] * 1e-3) / 1e9,
            "unfused_ms": t["unfused"], "unfused": "torch.matmul (library GEMM) to bf16 logits + ds_confidence"}
    if not args.no_decode_loop and world == 1 and args.stages == "attn,confidence,select":
        step = None
        torch.cuda.empty_cache()
        line["decode_loop"] = time_decode_loop(device)
        torch.cuda.empty_cache()
    if not args.no_cpu_baseline and world == 1:
        smp = OracleSample(cfg, 32, 128)
        full_s, spent = smp.time()
        # grow the sample towards ~10 s of CPU work (never beyond the whole workload)
        grow = max(1.0, min(10.0 / max(spent, 1e-3), 64.0))
        if grow > 1.5:
            smp = OracleSample(cfg, int(32 * grow), int(128 * grow))
            full_s, spent = smp.time()
        line["cpu_baseline"] = {"value": 1.0 / full_s, "unit": "steps/s", "cores": smp.cores, "kind": "oracle",
                                "sample": smp.sample, "sample_seconds": spent}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

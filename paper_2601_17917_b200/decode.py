"""Block scheduler of the decoding procedure (Preliminary Eq. 1-5, the selection rule Eq. 9-10 and
"Early Exit For Block Diffusion"): blocks in order, iterations of a block until none of its positions is
masked, later blocks skipped for sequences that predicted EOS with high confidence.

Everything the procedure decides lives on the device: which sequences still take part (``active_seq`` /
``active_cnt``), which logit rows still need Eq. 4 (``masked_rows`` / ``masked_cnt``), the early-exit flags.
The kernels of an iteration read those lists themselves, so the host can enqueue iterations without waiting
for the previous one; it only looks, ``lookahead`` iterations late and through pinned memory, at the number
of active sequences to know when to stop enqueueing iterations of a block.  ``lookahead = 0`` is the
synchronous loop (one host wait per iteration, no surplus launch); with ``lookahead = n`` at most n surplus
iterations per block are enqueued, and they find empty lists and do nothing.

The model itself (Eq. 3) is the caller's: ``forward(step)`` must leave the logits of the current block's
positions in ``step.logits`` using ``step.idx`` (retained rows, Eq. 7), ``step.refresh`` (first iteration of
a block: every position is a query and the prefix cache is rebuilt) and the device lists; it may instead
return a tensor of the same shape and type that already holds them.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import (ds_block_begin, ds_confidence_listed, ds_confidence_workspace, ds_unmask_select,
               retained_indices)


@dataclass
class Step:
    """What ``forward`` gets for one iteration.  All tensors are device tensors owned by the decoder."""
    n: int                      # block number
    t: int                      # iteration within the block
    refresh: bool               # first iteration of the block: full forward, rebuilds the prefix KV cache
    idx: torch.Tensor           # int32 tail-relative retained rows (Eq. 7); on refresh: every row of the tail
    active_seq: torch.Tensor    # int32 [B] sequences whose block still has masked positions (first *active_cnt)
    active_cnt: torch.Tensor    # int32 [1]
    x_block: torch.Tensor       # int32 [B, K] current tokens of the block ([MASK] where undecided)
    logits: torch.Tensor        # [B * K, V] to be filled for the rows of the active sequences


class BlockDecoder:
    def __init__(self, B: int, L: int, K: int, V: int, *, tau0: float, alpha: float, mask_id: int, eos_id: int = -1,
                 eos_tau: float = 0.9, w_tokens: int = 0, keep_last: bool = True, count_suffix: bool = False,
                 logits_dtype=torch.bfloat16, device="cuda:0", lookahead: int = 2):
        if L % K != 0:
            raise ValueError("the generation length must be a multiple of the block size (Eq. 2)")
        if lookahead < 0:
            raise ValueError("lookahead must be >= 0")
        dev = torch.device(device)
        self.B, self.L, self.K, self.V, self.N = B, L, K, V, L // K
        self.tau0, self.alpha, self.mask_id, self.eos_id, self.eos_tau = tau0, alpha, mask_id, eos_id, eos_tau
        self.count_suffix, self.lookahead, self.device = count_suffix, lookahead, dev
        i32 = dict(dtype=torch.int32, device=dev)
        self.x = torch.empty((B, L), **i32)
        self.masked = torch.empty((B, K), dtype=torch.uint8, device=dev)
        self.x_block = torch.empty((B, K), **i32)
        self.conf = torch.zeros(B * K, dtype=torch.float32, device=dev)
        self.tok = torch.zeros(B * K, **i32)
        self.logits = torch.zeros((B * K, V), dtype=logits_dtype, device=dev)
        self.eos_exit = torch.zeros(B, dtype=torch.uint8, device=dev)
        # the selection updates the active list in place: every call of the loop sees the same pointers, so
        # attention plans (and CUDA graphs of an iteration) made once stay valid for the whole block
        self.active = torch.zeros(max(B, 1), **i32)
        self.active_cnt = torch.zeros(1, **i32)
        self.masked_rows = torch.zeros(max(B * K, 1), **i32)
        self.masked_cnt = torch.zeros(1, **i32)
        self.sel = dict(sel_idx=torch.empty((B, K), **i32), sel_cnt=torch.zeros(B, **i32),
                        block_done=torch.zeros(B, dtype=torch.uint8, device=dev), eos_exit=self.eos_exit,
                        active_seq=self.active, active_cnt=self.active_cnt,
                        masked_rows=self.masked_rows, masked_cnt=self.masked_cnt)
        self.workspace = torch.empty(max(ds_confidence_workspace(B * K, V, logits_dtype), 1), dtype=torch.uint8,
                                     device=dev)
        # Eq. 7 per block: the retained rows of the pruned iterations and all rows for the refresh iteration
        self.idx, self.idx_all, self.extra = [], [], []
        for n in range(self.N):
            keep = retained_indices(L, K, n, w_tokens, keep_last)
            self.idx.append(torch.tensor(keep, **i32))
            self.idx_all.append(torch.arange(L - n * K, **i32))
            self.extra.append(len(keep) - K if count_suffix else 0)
        # slot j of a block: number of active sequences before iteration j, copied to pinned memory
        self.cnt_host = torch.zeros(K + 1, dtype=torch.int32).pin_memory()
        self.events = [torch.cuda.Event() for _ in range(K + 1)]
        self._graphs = {}

    def _publish(self, slot: int, cnt: torch.Tensor):
        self.cnt_host[slot:slot + 1].copy_(cnt, non_blocking=True)
        self.events[slot].record()

    def _iteration(self, forward, n: int, t: int):
        """One iteration of block n: the model callback, Eq. 4 at the rows still masked, the selection."""
        B, K = self.B, self.K
        z = forward(Step(n=n, t=t, refresh=(t == 0), idx=self.idx_all[n] if t == 0 else self.idx[n],
                         active_seq=self.active, active_cnt=self.active_cnt, x_block=self.x_block,
                         logits=self.logits))
        if z is None:
            z = self.logits
        elif z.shape != self.logits.shape or z.dtype != self.logits.dtype or z.device != self.logits.device:
            raise ValueError("forward returned logits of the wrong shape, type or device")
        ds_confidence_listed(z, self.masked_rows, self.masked_cnt, self.conf, self.tok,
                             n_listed_max=B * K, workspace=self.workspace)
        ds_unmask_select(self.conf.view(B, K), self.tok.view(B, K), self.masked, self.x_block, self.tau0,
                         self.alpha, ratio_extra=self.extra[n], eos_id=self.eos_id, eos_tau=self.eos_tau,
                         seq_list=self.active, n_seq=B, n_seq_dev=self.active_cnt, out=self.sel)

    def _graph(self, forward, n: int, refresh: bool):
        """The CUDA graph of an iteration of block n (one for the refresh iteration, one for all the others:
        nothing an iteration is launched with depends on t).  Before the first capture every kernel runs once
        on empty lists, so that no module is loaded while a capture is open."""
        key = (n, refresh)
        if key not in self._graphs:
            t = 0 if refresh else 1
            self.active_cnt.zero_()
            self.masked_cnt.zero_()
            self._iteration(forward, n, t)          # empty lists: launches everything, changes nothing
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._iteration(forward, n, t)
            self._graphs[key] = g
        return self._graphs[key]

    def capture(self, forward):
        """Captures the graphs of every block ahead of a ``decode(..., graphs=True)`` (which otherwise captures
        them on first use).  ``forward`` must be the callable later passed to ``decode``: it has to launch the
        same work on the same buffers whenever it is called for a given (block, refresh) and must not depend
        on the iteration number, allocate, or synchronise."""
        for n in range(self.N):
            self._graph(forward, n, True)
            self._graph(forward, n, False)

    def decode(self, forward, before_iteration=None, graphs: bool = False) -> dict:
        """Runs the whole procedure on the current stream.  Returns x [B, L] (device), steps [N] (iterations
        each block needed), launched [N] (iterations enqueued, >= steps) and eos_exit [B] (device).
        ``before_iteration(n, t)``, if given, runs eagerly ahead of every iteration (e.g. to stage inputs).
        With ``graphs`` an iteration is one CUDA-graph launch (see ``capture``)."""
        B, K, N = self.B, self.K, self.N
        if graphs:
            self.capture(forward)
        self.x.fill_(self.mask_id)
        self.eos_exit.zero_()
        steps, launched = [], []
        for n in range(N):
            ds_block_begin(self.eos_exit, self.masked, self.x_block, self.mask_id, self.eos_id, self.active,
                           self.active_cnt, self.masked_rows, self.masked_cnt)
            self._publish(0, self.active_cnt)
            t = 0
            while t < K:
                seen = t - self.lookahead            # the newest slot the host insists on having seen
                if seen >= 0:
                    self.events[seen].synchronize()
                    if int(self.cnt_host[seen]) == 0:
                        break
                if before_iteration is not None:
                    before_iteration(n, t)
                if graphs:
                    self._graphs[(n, t == 0)].replay()
                else:
                    self._iteration(forward, n, t)
                t += 1
                self._publish(t, self.active_cnt)
            self.events[t].synchronize()             # everything enqueued for this block has run
            need = next(j for j in range(t + 1) if int(self.cnt_host[j]) == 0)
            steps.append(need)
            launched.append(t)
            self.x[:, n * K:(n + 1) * K].copy_(self.x_block)
        return dict(x=self.x, steps=steps, launched=launched, eos_exit=self.eos_exit)

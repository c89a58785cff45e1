"""CPU ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Plain, slow, double-precision restatement of one suffix-pruned block-diffusion
denoising step, written from the paper's equations.  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import this package; the CUDA
library never does, and nothing here imports the CUDA package.

Contents
--------
* ``block_indices`` / ``retained_indices``: Eq. 2 and Eq. 7 as integer sets.
* ``attn`` (C, ``oracle_attn``): pruned bidirectional attention, Eq. 8 plus the
  query/key construction of "Dynamic Confidence Aware Parallel Decoding".
* ``attn_full`` (numpy, written separately): unpruned attention of the whole
  tail over prefix + whole tail, materialising every score row.  It exists to
  pin ``attn``: retaining every suffix position must reproduce it.
* ``confidence`` (C, ``oracle_confidence``): Eq. 4.
* ``rope_gather`` (C, ``oracle_rope_gather``): rotary encoding of the retained
  rows with their original position ids (Eq. 7 and the text around it: pruned
  tokens keep their place through their rotary position ids) and their gather
  into compact Q/K/V.
* ``lmhead_confidence`` (C, ``oracle_lmhead_confidence``): the output projection
  (the last of the components that turn attention outputs into logits,
  Method, "Dynamic Confidence Aware Parallel Decoding") composed with Eq. 4,
  logits kept in float64.
* ``threshold`` / ``select`` (C, float32, contraction off): Eq. 10, Eq. 9, Eq. 5,
  block termination and the early-exit flag.
* ``decode`` (Python loop over the above): the block-wise decoding procedure of
  the Preliminary section (Eq. 1-5) with the selection rule of Eq. 9-10 and
  "Early Exit For Block Diffusion", the model being a caller-supplied function
  that returns the current block's logits.

Pins (see tests, run with ``-m "not gpu"``): every function is checked against
closed forms, invariants, a library routine on the special case it reduces to,
hand-worked thresholds and exhaustive enumeration; none is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "ds_oracle.c"
_LIB = _HERE / "libds_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc.  ``-ffp-contract=off`` keeps every float32
    operation of the selection rule separately rounded."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-std=c99",
               "-shared", "-fPIC", "-o", str(_LIB), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        c_fp = ctypes.POINTER(ctypes.c_float)
        c_dp = ctypes.POINTER(ctypes.c_double)
        c_ip = ctypes.POINTER(ctypes.c_int32)
        c_bp = ctypes.POINTER(ctypes.c_uint8)
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_attn.restype = ctypes.c_int
        lib.oracle_attn.argtypes = [c_fp, c_fp, c_fp, c_fp, c_fp] + [ctypes.c_int] * 7 + [
            c_ip, ctypes.c_long, ctypes.c_double, c_dp, c_dp]
        lib.oracle_confidence.restype = ctypes.c_int
        lib.oracle_confidence.argtypes = [c_fp, ctypes.c_long, ctypes.c_long, ctypes.c_long, c_dp, c_ip]
        lib.oracle_lmhead_confidence.restype = ctypes.c_int
        lib.oracle_lmhead_confidence.argtypes = [c_fp, c_fp, ctypes.c_long, ctypes.c_long, ctypes.c_long, c_dp,
                                                 c_ip, c_dp]
        lib.oracle_rope_gather.restype = ctypes.c_int
        lib.oracle_rope_gather.argtypes = [c_fp, c_fp, c_fp] + [ctypes.c_int] * 6 + [
            c_ip, ctypes.c_long, ctypes.c_long, ctypes.c_double, c_dp, c_dp, c_dp]
        lib.oracle_threshold.restype = ctypes.c_float
        lib.oracle_threshold.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                         ctypes.c_float]
        lib.oracle_select.restype = ctypes.c_int
        lib.oracle_select.argtypes = [ctypes.c_int, ctypes.c_int, c_fp, c_ip, c_bp, c_ip,
                                      ctypes.c_float, ctypes.c_float, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_float, c_ip, ctypes.c_int, c_ip, c_ip, c_bp, c_bp,
                                      c_ip, c_ip, c_fp]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the C oracle uses (OpenMP maximum, honours OMP_NUM_THREADS)."""
    return int(_load().oracle_num_threads())


def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _ptr(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


# --------------------------------------------------------------------------
# Eq. 2 and Eq. 7: index sets
# --------------------------------------------------------------------------
def block_indices(p_L: int, K: int, n: int) -> list[int]:
    """Eq. 2: absolute positions of block n, I_n = {p_L + nK, ..., p_L + (n+1)K - 1}."""
    return list(range(p_L + n * K, p_L + (n + 1) * K))


def retained_indices(gen_len: int, K: int, c: int, w_tokens: int, keep_last: bool = True) -> list[int]:
    """Eq. 7 as tail-relative row numbers.

    The tail is everything from the current block c onward: row 0 is the first
    position of block c, row T-1 (T = gen_len - c*K) the last position of the
    sequence.  Retained = the current block I_c, the ``w_tokens`` suffix
    positions nearest to it, and the trailing position of the sequence (the
    paper writes p_L + L, one past Eq. 2's last 0-based position; the last
    position is meant).  A window that already reaches the end does not
    duplicate it.  Returned strictly ascending.
    """
    T = gen_len - c * K
    if T < K or w_tokens < 0:
        raise ValueError("bad block / window")
    keep = set(range(K))
    keep.update(range(K, min(K + w_tokens, T)))
    if keep_last and T > K:
        keep.add(T - 1)
    return sorted(keep)


# --------------------------------------------------------------------------
# attention
# --------------------------------------------------------------------------
def attn(q_tail, k_tail, v_tail, k_pre, v_pre, idx, scale, want_lse=False):
    """Pruned attention (C oracle).  Shapes: q_tail [B,Hq,T,D]; k_tail, v_tail
    [B,Hkv,T,D]; k_pre, v_pre [B,Hkv,P,D]; idx [Lq] or [B,Lq].  Returns out
    [B,Hq,Lq,D] float64 (and lse [B,Hq,Lq])."""
    lib = _load()
    q_tail, k_tail, v_tail, k_pre, v_pre = map(_f32, (q_tail, k_tail, v_tail, k_pre, v_pre))
    B, Hq, T, D = q_tail.shape
    Hkv = k_tail.shape[1]
    P = k_pre.shape[2]
    assert k_tail.shape == (B, Hkv, T, D) and v_tail.shape == (B, Hkv, T, D)
    assert k_pre.shape == (B, Hkv, P, D) and v_pre.shape == (B, Hkv, P, D)
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    if idx.ndim == 1:
        Lq, bstride = idx.shape[0], 0
    else:
        assert idx.shape[0] == B
        Lq, bstride = idx.shape[1], idx.shape[1]
    out = np.empty((B, Hq, Lq, D), dtype=np.float64)
    lse = np.empty((B, Hq, Lq), dtype=np.float64)
    rc = lib.oracle_attn(_ptr(q_tail, ctypes.c_float), _ptr(k_tail, ctypes.c_float),
                         _ptr(v_tail, ctypes.c_float), _ptr(k_pre, ctypes.c_float),
                         _ptr(v_pre, ctypes.c_float), B, Hq, Hkv, D, P, T, Lq,
                         _ptr(idx, ctypes.c_int32), bstride, float(scale),
                         _ptr(out, ctypes.c_double), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle_attn rejected its arguments ({rc})")
    return (out, lse) if want_lse else out


def attn_full(q_tail, k_tail, v_tail, k_pre, v_pre, scale):
    """Unpruned attention, brute force in numpy float64: every tail row queries
    the prefix and the WHOLE tail.  Written apart from ``attn`` (no index list,
    no shared helper) so that the two can check each other."""
    q = np.asarray(q_tail, dtype=np.float64)
    B, Hq, T, D = q.shape
    Hkv = np.asarray(k_tail).shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hq, T, D), dtype=np.float64)
    for b in range(B):
        for h in range(Hq):
            g = h // G
            keys = np.concatenate([np.asarray(k_pre, np.float64)[b, g], np.asarray(k_tail, np.float64)[b, g]], 0)
            vals = np.concatenate([np.asarray(v_pre, np.float64)[b, g], np.asarray(v_tail, np.float64)[b, g]], 0)
            for i in range(T):
                scores = scale * (keys @ q[b, h, i])
                e = np.exp(scores - scores.max())
                out[b, h, i] = (e / e.sum()) @ vals
    return out


# --------------------------------------------------------------------------
# confidence
# --------------------------------------------------------------------------
def confidence(logits):
    """Eq. 4 for every row of ``logits`` [rows, V] (float32 values; bf16 widened
    exactly by the caller).  Returns (conf float64 [rows], tok int32 [rows])."""
    lib = _load()
    z = _f32(logits)
    rows, V = z.shape
    conf = np.empty(rows, dtype=np.float64)
    tok = np.empty(rows, dtype=np.int32)
    rc = lib.oracle_confidence(_ptr(z, ctypes.c_float), rows, V, V, _ptr(conf, ctypes.c_double),
                               _ptr(tok, ctypes.c_int32))
    if rc != 0:
        raise ValueError("oracle_confidence rejected its arguments")
    return conf, tok


def rope_gather(q_raw, k_raw, v_raw, idx, pos_offset, theta=10000.0):
    """Rotary encoding (rotate-half pairing) of the retained tail rows with their original position ids
    ``pos_offset + idx[i]`` and gather into compact buffers.  q_raw [B,Hq,T,D]; k_raw, v_raw [B,Hkv,T,D];
    idx [Lq] or [B,Lq].  Returns float64 (q [B,Hq,Lq,D], k [B,Hkv,Lq,D], v [B,Hkv,Lq,D])."""
    lib = _load()
    q_raw, k_raw, v_raw = map(_f32, (q_raw, k_raw, v_raw))
    B, Hq, T, D = q_raw.shape
    Hkv = k_raw.shape[1]
    assert k_raw.shape == (B, Hkv, T, D) and v_raw.shape == (B, Hkv, T, D)
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    Lq, bstride = (idx.shape[0], 0) if idx.ndim == 1 else (idx.shape[1], idx.shape[1])
    q = np.empty((B, Hq, Lq, D)); k = np.empty((B, Hkv, Lq, D)); v = np.empty((B, Hkv, Lq, D))
    rc = lib.oracle_rope_gather(_ptr(q_raw, ctypes.c_float), _ptr(k_raw, ctypes.c_float), _ptr(v_raw, ctypes.c_float),
                                B, Hq, Hkv, D, T, Lq, _ptr(idx, ctypes.c_int32), bstride, int(pos_offset), float(theta),
                                _ptr(q, ctypes.c_double), _ptr(k, ctypes.c_double), _ptr(v, ctypes.c_double))
    if rc != 0:
        raise ValueError("oracle_rope_gather rejected its arguments")
    return q, k, v


def lmhead_confidence(hidden, weight, want_logits=False):
    """Output projection z = hidden @ weight.T in float64 followed by Eq. 4, the logits never rounded or
    stored in a narrower type.  hidden [rows, hid], weight [V, hid] (float32 values; bf16 widened exactly
    by the caller).  Returns (conf float64 [rows], tok int32 [rows]) and, on request, the logits."""
    lib = _load()
    h, w = _f32(hidden), _f32(weight)
    rows, hid = h.shape
    V = w.shape[0]
    assert w.shape == (V, hid)
    conf = np.empty(rows, dtype=np.float64)
    tok = np.empty(rows, dtype=np.int32)
    z = np.empty((rows, V), dtype=np.float64) if want_logits else None
    rc = lib.oracle_lmhead_confidence(_ptr(h, ctypes.c_float), _ptr(w, ctypes.c_float), rows, hid, V,
                                      _ptr(conf, ctypes.c_double), _ptr(tok, ctypes.c_int32),
                                      _ptr(z, ctypes.c_double) if want_logits else None)
    if rc != 0:
        raise ValueError("oracle_lmhead_confidence rejected its arguments")
    return (conf, tok, z) if want_logits else (conf, tok)


# --------------------------------------------------------------------------
# selection
# --------------------------------------------------------------------------
def threshold(n_masked: int, K: int, tau0: float, alpha: float, extra: int = 0) -> float:
    """Eq. 10 in float32."""
    return float(_load().oracle_threshold(int(n_masked), int(K), int(extra), float(tau0), float(alpha)))


def select(conf, tok, masked, x_block, tau0, alpha, ratio_extra=0, eos_id=-1, eos_tau=0.9,
           seq_list=None, eos_exit=None):
    """One selection step (Eq. 9, 10, 5 + flags).  Inputs are not modified.
    Returns a dict with the updated ``masked``/``x_block`` and ``sel_idx``
    [B,K] (-1 padded), ``sel_cnt``, ``block_done``, ``eos_exit``,
    ``active_seq`` (ascending), ``tau`` [B] (nan for unlisted sequences)."""
    lib = _load()
    conf = _f32(conf)
    B, K = conf.shape
    tok = np.ascontiguousarray(np.asarray(tok, dtype=np.int32))
    masked = np.ascontiguousarray(np.asarray(masked, dtype=np.uint8)).copy()
    x_block = np.ascontiguousarray(np.asarray(x_block, dtype=np.int32)).copy()
    assert tok.shape == (B, K) and masked.shape == (B, K) and x_block.shape == (B, K)
    sel_idx = np.full((B, K), -1, dtype=np.int32)
    sel_cnt = np.zeros(B, dtype=np.int32)
    block_done = np.zeros(B, dtype=np.uint8)
    eos = np.zeros(B, dtype=np.uint8) if eos_exit is None else np.asarray(eos_exit, np.uint8).copy()
    active = np.full(B, -1, dtype=np.int32)
    n_active = np.zeros(1, dtype=np.int32)
    tau = np.full(B, np.nan, dtype=np.float32)
    if seq_list is None:
        sl, ns = None, 0
    else:
        sl_arr = np.ascontiguousarray(np.asarray(seq_list, dtype=np.int32))
        sl, ns = _ptr(sl_arr, ctypes.c_int32), int(sl_arr.shape[0])
    rc = lib.oracle_select(B, K, _ptr(conf, ctypes.c_float), _ptr(tok, ctypes.c_int32),
                           _ptr(masked, ctypes.c_uint8), _ptr(x_block, ctypes.c_int32), float(tau0),
                           float(alpha), int(ratio_extra), int(eos_id), float(eos_tau), sl, ns,
                           _ptr(sel_idx, ctypes.c_int32), _ptr(sel_cnt, ctypes.c_int32),
                           _ptr(block_done, ctypes.c_uint8), _ptr(eos, ctypes.c_uint8),
                           _ptr(active, ctypes.c_int32), _ptr(n_active, ctypes.c_int32),
                           _ptr(tau, ctypes.c_float))
    if rc != 0:
        raise ValueError("oracle_select rejected its arguments")
    return dict(masked=masked, x_block=x_block, sel_idx=sel_idx, sel_cnt=sel_cnt, block_done=block_done,
                eos_exit=eos, active_seq=active[: int(n_active[0])].copy(), tau=tau)


# --------------------------------------------------------------------------
# the block-wise decoding procedure
# --------------------------------------------------------------------------
def decode(logits_fn, B: int, L: int, K: int, tau0: float, alpha: float, mask_id: int, eos_id: int = -1,
           eos_tau: float = 0.9, extra_fn=None, trace=None):
    """Block-wise diffusion decoding of B sequences (Preliminary, Eq. 1-5; selection by Eq. 9-10;
    "Early Exit For Block Diffusion").

    Eq. 1: the generated part starts as L [MASK] tokens, split (Eq. 2) into N = L / K blocks.  Block n is
    iterated until none of its positions is masked, then block n + 1 follows.  At iteration t of block n
    ``logits_fn(n, t)`` stands for Eq. 3 and returns the logits [B, K, V] of the block's positions;
    Eq. 4 gives confidences and tokens, Eq. 9-10 choose the positions to finalise, Eq. 5 updates them.
    Sequences whose block is finished are no longer processed (their logits are not looked at).
    Early exit: a sequence that finalised ``eos_id`` with confidence >= ``eos_tau`` finishes its current
    block and skips every later block; the skipped blocks are filled with ``eos_id`` (what they hold is not
    stated in the paper).
    ``extra_fn(n)`` = number of retained suffix rows counted as masked in Eq. 10's ratio (None: 0).

    Returns dict(x [B, L] int32, steps [N] iterations spent on each block, seq_steps [B, N] iterations
    each sequence took part in, eos_exit [B]).  ``trace``, if a list, receives one dict per iteration
    (n, t, conf, tau, masked before, active before).
    """
    if L % K != 0:
        raise ValueError("L must be a multiple of K")
    N = L // K
    x = np.full((B, L), mask_id, dtype=np.int32)
    steps = np.zeros(N, dtype=np.int32)
    seq_steps = np.zeros((B, N), dtype=np.int32)
    exited = np.zeros(B, dtype=np.uint8)
    for n in range(N):
        live = [b for b in range(B) if exited[b] == 0]
        masked = np.zeros((B, K), dtype=np.uint8)
        xb = np.full((B, K), eos_id, dtype=np.int32)
        masked[live] = 1
        xb[live] = mask_id
        extra = 0 if extra_fn is None else int(extra_fn(n))
        active = list(live)
        t = 0
        while active:
            z = np.asarray(logits_fn(n, t), dtype=np.float64)
            V = z.shape[-1]
            conf, tok = confidence(z.reshape(B * K, V))
            conf = conf.reshape(B, K).astype(np.float32)   # Eq. 9's comparison is taken in float32
            tok = tok.reshape(B, K)
            r = select(conf, tok, masked, xb, tau0, alpha, ratio_extra=extra, eos_id=eos_id, eos_tau=eos_tau,
                       seq_list=active, eos_exit=exited)
            if trace is not None:
                trace.append(dict(n=n, t=t, conf=conf, tau=r["tau"], masked=masked.copy(), active=list(active)))
            seq_steps[active, n] += 1
            masked, xb, exited = r["masked"], r["x_block"], r["eos_exit"]
            active = r["active_seq"].tolist()
            t += 1
        steps[n] = t
        x[:, n * K:(n + 1) * K] = xb
    return dict(x=x, steps=steps, seq_steps=seq_steps, eos_exit=exited)

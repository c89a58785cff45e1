"""B200-native suffix-pruned denoising step for block-diffusion LLM decoding.

Thin Python binding over the C-ABI library ``libds_b200.so`` (declared in
``include/ds.h``).  The functions here have the same names as the C entry
points and only marshal arguments: torch tensors supply device memory and the
current stream, every step of the path runs in the library's CUDA kernels.
There is no CPU or PyTorch fallback: if the library is not built, importing
succeeds but the first call raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

from . import workloads  # noqa: F401  (seeded synthetic inputs)

__all__ = [
    "lib", "retained_indices", "ds_attn_pruned", "ds_attn_pruned_workspace", "ds_confidence",
    "ds_confidence_workspace", "ds_confidence_static", "ds_lmhead_confidence", "ds_lmhead_confidence_workspace",
    "ds_rope_gather", "ds_unmask_select", "ds_read_status", "ds_strerror", "ds_version",
    "ds_launch_count", "ds_block_begin", "ds_confidence_listed", "AttnPlan", "ds_selftest_bounded_wait",
    "DsError", "DS_F32", "DS_BF16", "DS_DEV_INDEX", "DS_DEV_TIMEOUT",
    "DS_ATTN_KERNEL_AUTO", "DS_ATTN_KERNEL_ONE_TILE", "DS_ATTN_KERNEL_TWO_TILE",
]

DS_F32, DS_BF16 = 0, 1
DS_OK, DS_ERR_INVALID_ARG, DS_ERR_UNSUPPORTED, DS_ERR_WORKSPACE, DS_ERR_CUDA, DS_ERR_STATIC_LIMIT = range(6)
DS_CONFIDENCE_STATIC_MAX_ROWS = 4096
DS_DEV_INDEX, DS_DEV_TIMEOUT = 1, 2
DS_ATTN_KERNEL_AUTO, DS_ATTN_KERNEL_ONE_TILE, DS_ATTN_KERNEL_TWO_TILE = 0, 1, 2

_LIB_PATH = Path(__file__).resolve().parent / "libds_b200.so"
_lib = None


class DsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = ""
        if code == DS_ERR_CUDA:
            detail = f" [{lib().ds_last_cuda_error_name().decode()} = {lib().ds_last_cuda_error()}]"
        super().__init__(f"{where}: {ds_strerror(code)} (status {code}){detail}")


class _AttnParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("P", ctypes.c_int32), ("T", ctypes.c_int32), ("Lq", ctypes.c_int32), ("dtype", ctypes.c_int32),
        ("q_tail", ctypes.c_void_p), ("k_tail", ctypes.c_void_p), ("v_tail", ctypes.c_void_p),
        ("k_prefix", ctypes.c_void_p), ("v_prefix", ctypes.c_void_p),
        ("q_stride", ctypes.c_int64 * 3), ("kv_tail_stride", ctypes.c_int64 * 3),
        ("kv_prefix_stride", ctypes.c_int64 * 3), ("out_stride", ctypes.c_int64 * 3),
        ("idx", ctypes.c_void_p), ("idx_batch_stride", ctypes.c_int64), ("scale", ctypes.c_float),
        ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t), ("status", ctypes.c_void_p),
        ("seq_list", ctypes.c_void_p), ("n_seq", ctypes.c_int32), ("n_seq_dev", ctypes.c_void_p),
        ("kernel", ctypes.c_int32),
    ]


class _RopeParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("T", ctypes.c_int32), ("Lq", ctypes.c_int32),
        ("q_raw", ctypes.c_void_p), ("k_raw", ctypes.c_void_p), ("v_raw", ctypes.c_void_p),
        ("q_stride", ctypes.c_int64 * 3), ("kv_stride", ctypes.c_int64 * 3),
        ("idx", ctypes.c_void_p), ("idx_batch_stride", ctypes.c_int64),
        ("pos_offset", ctypes.c_int32), ("rope_theta", ctypes.c_float),
        ("q_out", ctypes.c_void_p), ("k_out", ctypes.c_void_p), ("v_out", ctypes.c_void_p),
        ("q_out_stride", ctypes.c_int64 * 3), ("kv_out_stride", ctypes.c_int64 * 3),
        ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p), ("cache_stride", ctypes.c_int64 * 3),
        ("cache_row0", ctypes.c_int32), ("n_append", ctypes.c_int32), ("status", ctypes.c_void_p),
    ]


class _BlockParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("mask_id", ctypes.c_int32), ("fill_id", ctypes.c_int32),
        ("eos_exit", ctypes.c_void_p), ("masked", ctypes.c_void_p), ("x_block", ctypes.c_void_p),
        ("active_seq", ctypes.c_void_p), ("active_cnt", ctypes.c_void_p), ("masked_rows", ctypes.c_void_p),
        ("masked_cnt", ctypes.c_void_p),
    ]


class _SelectParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("K", ctypes.c_int32), ("conf", ctypes.c_void_p), ("tok", ctypes.c_void_p),
        ("masked", ctypes.c_void_p), ("x_block", ctypes.c_void_p), ("tau0", ctypes.c_float),
        ("alpha", ctypes.c_float), ("ratio_extra", ctypes.c_int32), ("eos_id", ctypes.c_int32),
        ("eos_tau", ctypes.c_float), ("seq_list", ctypes.c_void_p), ("n_seq", ctypes.c_int32),
        ("n_seq_dev", ctypes.c_void_p), ("sel_idx", ctypes.c_void_p), ("sel_cnt", ctypes.c_void_p),
        ("block_done", ctypes.c_void_p), ("eos_exit", ctypes.c_void_p), ("active_seq", ctypes.c_void_p),
        ("active_cnt", ctypes.c_void_p), ("masked_rows", ctypes.c_void_p), ("masked_cnt", ctypes.c_void_p),
    ]


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2601_17917_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(str(_LIB_PATH))
        L.ds_attn_pruned_workspace.restype = ctypes.c_size_t
        L.ds_attn_pruned_workspace.argtypes = [ctypes.POINTER(_AttnParams)]
        L.ds_attn_pruned.restype = ctypes.c_int
        L.ds_attn_pruned.argtypes = [ctypes.POINTER(_AttnParams), ctypes.c_void_p]
        L.ds_attn_plan_create.restype = ctypes.c_int
        L.ds_attn_plan_create.argtypes = [ctypes.POINTER(_AttnParams), ctypes.POINTER(ctypes.c_void_p)]
        L.ds_attn_plan_launch.restype = ctypes.c_int
        L.ds_attn_plan_launch.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.ds_attn_plan_destroy.restype = None
        L.ds_attn_plan_destroy.argtypes = [ctypes.c_void_p]
        L.ds_confidence_workspace.restype = ctypes.c_size_t
        L.ds_confidence_workspace.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int32]
        L.ds_confidence.restype = ctypes.c_int
        L.ds_confidence.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.ds_confidence_listed.restype = ctypes.c_int
        L.ds_confidence_listed.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                           ctypes.c_void_p]
        L.ds_rope_gather.restype = ctypes.c_int
        L.ds_rope_gather.argtypes = [ctypes.POINTER(_RopeParams), ctypes.c_void_p]
        L.ds_lmhead_confidence_workspace.restype = ctypes.c_size_t
        L.ds_lmhead_confidence_workspace.argtypes = [ctypes.c_int64, ctypes.c_int64]
        L.ds_lmhead_confidence.restype = ctypes.c_int
        L.ds_lmhead_confidence.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int64] * 5 + [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
        L.ds_confidence_static.restype = ctypes.c_int
        L.ds_confidence_static.argtypes = [ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                           ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p]
        L.ds_block_begin.restype = ctypes.c_int
        L.ds_block_begin.argtypes = [ctypes.POINTER(_BlockParams), ctypes.c_void_p]
        L.ds_unmask_select.restype = ctypes.c_int
        L.ds_unmask_select.argtypes = [ctypes.POINTER(_SelectParams), ctypes.c_void_p]
        L.ds_read_status.restype = ctypes.c_int
        L.ds_read_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint32)]
        L.ds_selftest_bounded_wait.restype = ctypes.c_int
        L.ds_selftest_bounded_wait.argtypes = [ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.ds_last_cuda_error.restype = ctypes.c_int
        L.ds_last_cuda_error_name.restype = ctypes.c_char_p
        L.ds_strerror.restype = ctypes.c_char_p
        L.ds_strerror.argtypes = [ctypes.c_int]
        L.ds_version.restype = ctypes.c_int
        L.ds_launch_count.restype = ctypes.c_int64
        _lib = L
    return _lib


def ds_strerror(code: int) -> str:
    return lib().ds_strerror(int(code)).decode()


def ds_version() -> int:
    return int(lib().ds_version())


def ds_launch_count() -> int:
    return int(lib().ds_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DS_F32
    if t.dtype == torch.bfloat16:
        return DS_BF16
    raise TypeError(f"unsupported element type {t.dtype}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check_dev(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise ValueError("all tensors must live on a CUDA device")


def retained_indices(gen_len: int, K: int, c: int, w_tokens: int, keep_last: bool = True) -> list[int]:
    """Host step of the path: the retained set of Eq. 7 as tail-relative rows.

    The tail starts at the current block c and has T = gen_len - c*K rows.
    Kept: the K block rows, the next ``w_tokens`` rows (sliding window nearest
    the block; -1 keeps the whole suffix), and the trailing position T-1.  The
    list is strictly ascending, as ``ds_attn_pruned`` requires.
    """
    T = gen_len - c * K
    if K <= 0 or T < K or w_tokens < -1:
        raise ValueError("bad block / window")
    end = T if w_tokens < 0 else min(K + w_tokens, T)
    idx = list(range(end))
    if keep_last and end < T:
        idx.append(T - 1)
    return idx


def _attn_params(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out, lse, workspace, status,
                 seq_list=None, n_seq=None, n_seq_dev=None, kernel=DS_ATTN_KERNEL_AUTO):
    B, Hq, T, D = q_tail.shape
    Hkv = k_tail.shape[1]
    P = 0 if k_prefix is None else k_prefix.shape[2]
    for t in (q_tail, k_tail, v_tail, out) + ((k_prefix, v_prefix) if P else ()):
        if t.stride(-1) != 1:
            raise ValueError("the head dimension must be contiguous")
    if k_tail.stride() != v_tail.stride() or (P and k_prefix.stride() != v_prefix.stride()):
        raise ValueError("K and V must share strides")
    if idx.dtype != torch.int32:
        raise TypeError("idx must be int32")
    Lq = idx.shape[-1]
    p = _AttnParams()
    p.B, p.Hq, p.Hkv, p.D, p.P, p.T, p.Lq = B, Hq, Hkv, D, P, T, Lq
    p.dtype = _dtype_code(q_tail)
    p.q_tail, p.k_tail, p.v_tail = q_tail.data_ptr(), k_tail.data_ptr(), v_tail.data_ptr()
    p.k_prefix = k_prefix.data_ptr() if P else None
    p.v_prefix = v_prefix.data_ptr() if P else None
    p.q_stride[:] = q_tail.stride()[:3]
    p.kv_tail_stride[:] = k_tail.stride()[:3]
    if P:
        p.kv_prefix_stride[:] = k_prefix.stride()[:3]
    p.out_stride[:] = out.stride()[:3]
    p.idx = idx.data_ptr()
    p.idx_batch_stride = 0 if idx.dim() == 1 else idx.stride(0)
    p.scale = float(scale)
    p.out = out.data_ptr()
    p.lse = lse.data_ptr() if lse is not None else None
    p.workspace = workspace.data_ptr() if workspace is not None else None
    p.workspace_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    p.status = status.data_ptr() if status is not None else None
    if seq_list is not None:
        if seq_list.dtype != torch.int32 or (n_seq_dev is not None and n_seq_dev.dtype != torch.int32):
            raise TypeError("seq_list and n_seq_dev must be int32")
        if seq_list.numel() == 0:
            raise ValueError("seq_list must have room for at least one entry (use n_seq=0 for an empty list)")
        p.seq_list = seq_list.data_ptr()
        p.n_seq = seq_list.numel() if n_seq is None else min(int(n_seq), seq_list.numel())
        p.n_seq_dev = n_seq_dev.data_ptr() if n_seq_dev is not None else None
    p.kernel = int(kernel)
    return p


def ds_attn_pruned_workspace(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out,
                             kernel=DS_ATTN_KERNEL_AUTO) -> int:
    p = _attn_params(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out, None, None, None, kernel=kernel)
    return int(lib().ds_attn_pruned_workspace(ctypes.byref(p)))


def ds_attn_pruned(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out=None, lse=None,
                   workspace=None, status=None, stream=None, seq_list=None, n_seq=None, n_seq_dev=None,
                   kernel=DS_ATTN_KERNEL_AUTO):
    """Pruned attention (Eq. 7-8).  q_tail [B,Hq,T,D]; k_tail, v_tail [B,Hkv,T,D];
    k_prefix, v_prefix [B,Hkv,P,D] or None; idx int32 [Lq] or [B,Lq] on the device.
    seq_list (int32, ascending batch numbers; its first n_seq entries, or as many as the device scalar
    n_seq_dev says) restricts the call to those sequences.  ``kernel`` pins the bf16 kernel (DS_ATTN_KERNEL_*).
    Returns ``out`` [B,Hq,Lq,D].  Allocates ``out``/``workspace`` with torch when not given."""
    _check_dev(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, out, lse, workspace, status, seq_list, n_seq_dev)
    B, Hq, T, D = q_tail.shape
    if out is None:
        out = torch.empty((B, Hq, idx.shape[-1], D), dtype=q_tail.dtype, device=q_tail.device)
    p = _attn_params(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out, lse, workspace, status,
                     seq_list, n_seq, n_seq_dev, kernel)
    if workspace is None:
        need = int(lib().ds_attn_pruned_workspace(ctypes.byref(p)))
        if need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q_tail.device)
            p.workspace, p.workspace_bytes = workspace.data_ptr(), need
    rc = lib().ds_attn_pruned(ctypes.byref(p), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_attn_pruned")
    return out


class AttnPlan:
    """ds_attn_plan: the arguments of ds_attn_pruned validated and turned into kernel parameters once;
    ``launch`` then only enqueues the kernel.  The plan keeps references to the tensors it was made from
    (their contents are read at every launch).  ``out`` is allocated when not given."""

    def __init__(self, q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out=None, lse=None, workspace=None,
                 status=None, seq_list=None, n_seq=None, n_seq_dev=None, kernel=DS_ATTN_KERNEL_AUTO):
        _check_dev(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, out, lse, workspace, status, seq_list, n_seq_dev)
        B, Hq, T, D = q_tail.shape
        if out is None:
            out = torch.empty((B, Hq, idx.shape[-1], D), dtype=q_tail.dtype, device=q_tail.device)
        p = _attn_params(q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, scale, out, lse, workspace, status,
                         seq_list, n_seq, n_seq_dev, kernel)
        if workspace is None:
            need = int(lib().ds_attn_pruned_workspace(ctypes.byref(p)))
            if need:
                workspace = torch.empty(need, dtype=torch.uint8, device=q_tail.device)
                p.workspace, p.workspace_bytes = workspace.data_ptr(), need
        self.out = out
        self._keep = (q_tail, k_tail, v_tail, k_prefix, v_prefix, idx, out, lse, workspace, status, seq_list, n_seq_dev)
        self._h = ctypes.c_void_p()
        self._destroy = lib().ds_attn_plan_destroy
        self._launch = lib().ds_attn_plan_launch
        rc = lib().ds_attn_plan_create(ctypes.byref(p), ctypes.byref(self._h))
        if rc != DS_OK:
            raise DsError(rc, "ds_attn_plan_create")

    def launch(self, stream=None):
        rc = self._launch(self._h, _stream(stream))
        if rc != DS_OK:
            raise DsError(rc, "ds_attn_plan_launch")
        return self.out

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self._destroy(h)


def ds_confidence_workspace(rows: int, V: int, dtype) -> int:
    code = dtype if isinstance(dtype, int) else (DS_BF16 if dtype == torch.bfloat16 else DS_F32)
    return int(lib().ds_confidence_workspace(int(rows), int(V), code))


def ds_confidence(logits, row_list=None, conf=None, tok=None, workspace=None, stream=None):
    """Eq. 4 over ``logits`` [rows, V] (last dimension contiguous).  Returns (conf f32 [rows], tok i32 [rows])."""
    _check_dev(logits, row_list, conf, tok, workspace)
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [rows, V] with contiguous rows")
    rows, V = logits.shape
    if conf is None:
        conf = torch.empty(rows, dtype=torch.float32, device=logits.device)
    if tok is None:
        tok = torch.empty(rows, dtype=torch.int32, device=logits.device)
    if workspace is None:
        need = ds_confidence_workspace(rows, V, logits.dtype)
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=logits.device)
    if row_list is not None and row_list.dtype != torch.int32:
        raise TypeError("row_list must be int32")
    if row_list is not None and row_list.numel() == 0:
        return conf, tok      # no row listed: nothing is touched (a null list pointer would mean "all rows")
    rc = lib().ds_confidence(_ptr(logits), _dtype_code(logits), rows, V, logits.stride(0), _ptr(row_list),
                             0 if row_list is None else row_list.numel(), _ptr(conf), _ptr(tok),
                             _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_confidence")
    return conf, tok


def ds_confidence_listed(logits, row_list, n_listed_dev, conf, tok, n_listed_max=None, workspace=None, stream=None):
    """Eq. 4 over the first ``*n_listed_dev`` rows named in ``row_list`` (both on the device, int32), e.g.
    ds_unmask_select's masked_rows / masked_cnt.  conf/tok [rows] are updated at those rows only."""
    _check_dev(logits, row_list, n_listed_dev, conf, tok, workspace)
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [rows, V] with contiguous rows")
    if row_list.dtype != torch.int32 or n_listed_dev.dtype != torch.int32:
        raise TypeError("row_list and n_listed_dev must be int32")
    rows, V = logits.shape
    n_max = min(rows, row_list.numel()) if n_listed_max is None else int(n_listed_max)
    if workspace is None:
        need = ds_confidence_workspace(rows, V, logits.dtype)
        workspace = torch.empty(max(need, 1), dtype=torch.uint8, device=logits.device)
    rc = lib().ds_confidence_listed(_ptr(logits), _dtype_code(logits), rows, V, logits.stride(0), _ptr(row_list),
                                    n_max, _ptr(n_listed_dev), _ptr(conf), _ptr(tok), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_confidence_listed")
    return conf, tok


def ds_rope_gather(q_raw, k_raw, v_raw, idx, pos_offset, rope_theta=10000.0, q_out=None, k_out=None, v_out=None,
                   k_cache=None, v_cache=None, cache_row0=0, n_append=0, status=None, stream=None):
    """Rotary encoding of the retained tail rows with their original position ids and gather into compact
    buffers (Eq. 7-8); optionally appends the first ``n_append`` retained rows to the prefix cache.
    q_raw [B,Hq,T,D]; k_raw, v_raw [B,Hkv,T,D] bf16; idx int32 [Lq] or [B,Lq].  Returns (q, k, v) compact
    [B,H,Lq,D], ready for ``ds_attn_pruned`` with ``idx = arange(Lq)``."""
    _check_dev(q_raw, k_raw, v_raw, idx, q_out, k_out, v_out, k_cache, v_cache, status)
    B, Hq, T, D = q_raw.shape
    Hkv = k_raw.shape[1]
    Lq = idx.shape[-1]
    for t in (q_raw, k_raw, v_raw):
        if t.dtype != torch.bfloat16 or t.stride(-1) != 1:
            raise ValueError("inputs must be bf16 with a contiguous head dimension")
    if k_raw.stride() != v_raw.stride():
        raise ValueError("K and V must share strides")
    if idx.dtype != torch.int32:
        raise TypeError("idx must be int32")
    dev = q_raw.device
    if q_out is None:
        q_out = torch.empty((B, Hq, Lq, D), dtype=torch.bfloat16, device=dev)
    if k_out is None:
        k_out = torch.empty((B, Hkv, Lq, D), dtype=torch.bfloat16, device=dev)
    if v_out is None:
        v_out = torch.empty((B, Hkv, Lq, D), dtype=torch.bfloat16, device=dev)
    if k_out.stride() != v_out.stride():
        raise ValueError("k_out and v_out must share strides")
    p = _RopeParams()
    p.B, p.Hq, p.Hkv, p.D, p.T, p.Lq = B, Hq, Hkv, D, T, Lq
    p.q_raw, p.k_raw, p.v_raw = q_raw.data_ptr(), k_raw.data_ptr(), v_raw.data_ptr()
    p.q_stride[:] = q_raw.stride()[:3]
    p.kv_stride[:] = k_raw.stride()[:3]
    p.idx = idx.data_ptr()
    p.idx_batch_stride = 0 if idx.dim() == 1 else idx.stride(0)
    p.pos_offset, p.rope_theta = int(pos_offset), float(rope_theta)
    p.q_out, p.k_out, p.v_out = q_out.data_ptr(), k_out.data_ptr(), v_out.data_ptr()
    p.q_out_stride[:] = q_out.stride()[:3]
    p.kv_out_stride[:] = k_out.stride()[:3]
    if n_append:
        if k_cache is None or v_cache is None or k_cache.stride() != v_cache.stride():
            raise ValueError("appending needs k_cache and v_cache with equal strides")
        p.k_cache, p.v_cache = k_cache.data_ptr(), v_cache.data_ptr()
        p.cache_stride[:] = k_cache.stride()[:3]
    p.cache_row0, p.n_append = int(cache_row0), int(n_append)
    p.status = status.data_ptr() if status is not None else None
    rc = lib().ds_rope_gather(ctypes.byref(p), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_rope_gather")
    return q_out, k_out, v_out


def ds_lmhead_confidence_workspace(rows: int, V: int) -> int:
    return int(lib().ds_lmhead_confidence_workspace(int(rows), int(V)))


def ds_lmhead_confidence(hidden, weight, conf=None, tok=None, workspace=None, status=None, stream=None):
    """Output projection fused with Eq. 4: hidden bf16 [rows, hid], weight bf16 [V, hid] (last dimension
    contiguous).  Returns (conf f32 [rows], tok i32 [rows]); the logits are never stored."""
    _check_dev(hidden, weight, conf, tok, workspace, status)
    if hidden.dtype != torch.bfloat16 or weight.dtype != torch.bfloat16:
        raise TypeError("hidden and weight must be bf16")
    if hidden.dim() != 2 or weight.dim() != 2 or hidden.stride(1) != 1 or weight.stride(1) != 1:
        raise ValueError("hidden [rows, hid] and weight [V, hid] must have contiguous rows")
    rows, hid = hidden.shape
    V = weight.shape[0]
    if weight.shape[1] != hid:
        raise ValueError("hidden and weight disagree on the hidden size")
    if conf is None:
        conf = torch.empty(rows, dtype=torch.float32, device=hidden.device)
    if tok is None:
        tok = torch.empty(rows, dtype=torch.int32, device=hidden.device)
    if workspace is None:
        workspace = torch.empty(max(ds_lmhead_confidence_workspace(rows, V), 256), dtype=torch.uint8,
                                device=hidden.device)
    rc = lib().ds_lmhead_confidence(_ptr(hidden), _ptr(weight), rows, hid, V, hidden.stride(0), weight.stride(0),
                                    _ptr(conf), _ptr(tok), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                    _ptr(status), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_lmhead_confidence")
    return conf, tok


def ds_confidence_static(logits, conf, tok, row_list=None, stream=None):
    """Eq. 4 like ``ds_confidence``, through the entry point that needs no workspace: its scratch is a
    fixed array inside the library, so the call itself allocates nothing.  For callers that cannot
    allocate device memory where they call from.  ``conf`` f32 [rows] and ``tok`` i32 [rows] must be
    passed in (this wrapper creates no tensor either).  At most DS_CONFIDENCE_STATIC_MAX_ROWS rows are
    processed per call; calls that may overlap on the GPU must be ordered, they share the scratch."""
    _check_dev(logits, row_list, conf, tok)
    if logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits must be [rows, V] with contiguous rows")
    rows, V = logits.shape
    if conf.dtype != torch.float32 or tok.dtype != torch.int32 or conf.numel() < rows or tok.numel() < rows:
        raise ValueError("conf must be f32 [rows] and tok i32 [rows]")
    if row_list is not None and row_list.dtype != torch.int32:
        raise TypeError("row_list must be int32")
    if row_list is not None and row_list.numel() == 0:
        return conf, tok      # no row listed: nothing is touched (a null list pointer would mean "all rows")
    rc = lib().ds_confidence_static(_ptr(logits), _dtype_code(logits), rows, V, logits.stride(0), _ptr(row_list),
                                    0 if row_list is None else row_list.numel(), _ptr(conf), _ptr(tok),
                                    _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_confidence_static")
    return conf, tok


def ds_unmask_select(conf, tok, masked, x_block, tau0, alpha, ratio_extra=0, eos_id=-1, eos_tau=0.9,
                     seq_list=None, n_seq=None, n_seq_dev=None, out=None, stream=None):
    """Eq. 9-10 selection step.  conf f32 [B,K], tok i32 [B,K]; masked u8 [B,K] and
    x_block i32 [B,K] are updated in place.  Returns a dict of device tensors:
    sel_idx, sel_cnt, block_done, eos_exit, active_seq, active_cnt, masked_rows, masked_cnt
    (pass ``out`` to reuse them; masked_rows/masked_cnt are written when ``out`` holds them)."""
    _check_dev(conf, tok, masked, x_block, seq_list, n_seq_dev)
    B, K = conf.shape
    dev = conf.device
    for t, dt in ((conf, torch.float32), (tok, torch.int32), (masked, torch.uint8), (x_block, torch.int32)):
        if t.dtype != dt or not t.is_contiguous() or tuple(t.shape) != (B, K):
            raise ValueError("conf/tok/masked/x_block must be contiguous [B,K] of f32/i32/u8/i32")
    if out is None:
        out = dict(sel_idx=torch.empty((B, K), dtype=torch.int32, device=dev),
                   sel_cnt=torch.zeros(B, dtype=torch.int32, device=dev),
                   block_done=torch.zeros(B, dtype=torch.uint8, device=dev),
                   eos_exit=torch.zeros(B, dtype=torch.uint8, device=dev),
                   active_seq=torch.empty(max(B, 1), dtype=torch.int32, device=dev),
                   active_cnt=torch.zeros(1, dtype=torch.int32, device=dev),
                   masked_rows=torch.empty(max(B * K, 1), dtype=torch.int32, device=dev),
                   masked_cnt=torch.zeros(1, dtype=torch.int32, device=dev))
    p = _SelectParams()
    p.B, p.K = B, K
    p.conf, p.tok, p.masked, p.x_block = conf.data_ptr(), tok.data_ptr(), masked.data_ptr(), x_block.data_ptr()
    p.tau0, p.alpha, p.ratio_extra, p.eos_id, p.eos_tau = tau0, alpha, ratio_extra, eos_id, eos_tau
    if seq_list is not None:
        if seq_list.dtype != torch.int32:
            raise TypeError("seq_list must be int32")
        # an empty tensor has a null data pointer, which the C ABI reads as "no list": keep it non-null
        p.seq_list = seq_list.data_ptr() if seq_list.numel() else out["active_cnt"].data_ptr()
        p.n_seq = seq_list.numel() if n_seq is None else min(int(n_seq), seq_list.numel())
        p.n_seq_dev = n_seq_dev.data_ptr() if n_seq_dev is not None else None
    p.sel_idx, p.sel_cnt = out["sel_idx"].data_ptr(), out["sel_cnt"].data_ptr()
    p.block_done, p.eos_exit = out["block_done"].data_ptr(), out["eos_exit"].data_ptr()
    p.active_seq, p.active_cnt = out["active_seq"].data_ptr(), out["active_cnt"].data_ptr()
    if out.get("masked_rows") is not None:
        p.masked_rows, p.masked_cnt = out["masked_rows"].data_ptr(), out["masked_cnt"].data_ptr()
    rc = lib().ds_unmask_select(ctypes.byref(p), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_unmask_select")
    return out


def ds_block_begin(eos_exit, masked, x_block, mask_id, fill_id, active_seq, active_cnt, masked_rows=None,
                   masked_cnt=None, stream=None):
    """Start of a block (Eq. 1-2, early exit): fresh [MASK] state for the sequences that have not exited,
    ``fill_id`` for the others, and the device lists the step's entry points read."""
    _check_dev(eos_exit, masked, x_block, active_seq, active_cnt, masked_rows, masked_cnt)
    B, K = masked.shape
    if eos_exit.dtype != torch.uint8 or masked.dtype != torch.uint8 or x_block.dtype != torch.int32:
        raise TypeError("eos_exit/masked must be uint8 and x_block int32")
    if not (masked.is_contiguous() and x_block.is_contiguous()) or tuple(x_block.shape) != (B, K):
        raise ValueError("masked and x_block must be contiguous [B,K]")
    for t in (active_seq, active_cnt, masked_rows, masked_cnt):
        if t is not None and t.dtype != torch.int32:
            raise TypeError("the lists and counts must be int32")
    p = _BlockParams()
    p.B, p.K, p.mask_id, p.fill_id = B, K, int(mask_id), int(fill_id)
    p.eos_exit, p.masked, p.x_block = eos_exit.data_ptr(), masked.data_ptr(), x_block.data_ptr()
    p.active_seq, p.active_cnt = active_seq.data_ptr(), active_cnt.data_ptr()
    p.masked_rows = masked_rows.data_ptr() if masked_rows is not None else None
    p.masked_cnt = masked_cnt.data_ptr() if masked_cnt is not None else None
    rc = lib().ds_block_begin(ctypes.byref(p), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_block_begin")


def ds_selftest_bounded_wait(poll_limit: int, status=None, report=None, stream=None):
    """Runs the kernels' bounded wait on a barrier nobody arrives on (see ds.h).  status: int32/uint32 [1],
    report: int32 [3], both optional device tensors."""
    _check_dev(status, report)
    rc = lib().ds_selftest_bounded_wait(int(poll_limit), _ptr(status), _ptr(report), _stream(stream))
    if rc != DS_OK:
        raise DsError(rc, "ds_selftest_bounded_wait")


def ds_read_status(status: torch.Tensor, stream=None) -> int:
    host = ctypes.c_uint32(0)
    rc = lib().ds_read_status(_ptr(status), _stream(stream), ctypes.byref(host))
    if rc != DS_OK:
        raise DsError(rc, "ds_read_status")
    return int(host.value)

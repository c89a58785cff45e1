"""CPU-side checks of the boundary: the library loads without a GPU, exports every
symbol the header declares, the ctypes mirrors match the C structs, arguments
are validated before anything touches a device, and the host step (Eq. 7 index
list) agrees with the oracle's own construction."""
import ctypes
import re
import subprocess
import sys
from pathlib import Path

import pytest
import torch

import oracle
import paper_2601_17917_b200 as ds
from paper_2601_17917_b200 import build as ds_build

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def L():
    ds_build.build()
    return ds.lib()


def test_exports_every_declared_symbol(L):
    header = (ROOT / "include" / "ds.h").read_text()
    names = re.findall(r"DS_API\s+[\w\s\*]+?\b(ds_\w+)\s*\(", header)
    assert len(names) >= 9 and len(set(names)) == len(names)
    for n in names:
        assert hasattr(L, n), n
    assert L.ds_version() == 1000
    assert ds.ds_strerror(0) == "ok" and "workspace" in ds.ds_strerror(3)


def test_ctypes_structs_match_header(tmp_path):
    src = tmp_path / "layout.c"
    src.write_text(r'''
#include <stdio.h>
#include <stddef.h>
#include "ds.h"
int main(void) {
  printf("%zu %zu %zu %zu %zu %zu %zu\n", sizeof(ds_attn_params), offsetof(ds_attn_params, q_stride),
         offsetof(ds_attn_params, idx), offsetof(ds_attn_params, scale), offsetof(ds_attn_params, out),
         offsetof(ds_attn_params, status), offsetof(ds_attn_params, kernel));
  printf("%zu %zu %zu %zu %zu\n", sizeof(ds_select_params), offsetof(ds_select_params, tau0),
         offsetof(ds_select_params, seq_list), offsetof(ds_select_params, n_seq_dev),
         offsetof(ds_select_params, active_cnt));
  printf("%zu %zu %zu %zu %zu %zu\n", sizeof(ds_rope_params), offsetof(ds_rope_params, q_stride),
         offsetof(ds_rope_params, idx), offsetof(ds_rope_params, rope_theta), offsetof(ds_rope_params, k_cache),
         offsetof(ds_rope_params, status));
  return 0;
}''')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", str(ROOT / "include"), str(src), "-o", str(exe)], check=True)
    a, s, r = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.strip().splitlines()
    A, S, R = ds._AttnParams, ds._SelectParams, ds._RopeParams
    assert [int(v) for v in r.split()] == [ctypes.sizeof(R), R.q_stride.offset, R.idx.offset, R.rope_theta.offset,
                                           R.k_cache.offset, R.status.offset]
    assert [int(v) for v in a.split()] == [ctypes.sizeof(A), A.q_stride.offset, A.idx.offset, A.scale.offset,
                                           A.out.offset, A.status.offset, A.kernel.offset]
    assert [int(v) for v in s.split()] == [ctypes.sizeof(S), S.tau0.offset, S.seq_list.offset,
                                           S.n_seq_dev.offset, S.active_cnt.offset]


def test_header_compiles_as_c(tmp_path):
    src = tmp_path / "h.c"
    src.write_text('#include "ds.h"\nint main(void){return (int)DS_OK;}\n')
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", str(ROOT / "include"), "-c", str(src), "-o",
                    str(tmp_path / "h.o")], check=True)


def _attn(**kw):
    p = ds._AttnParams()
    p.B, p.Hq, p.Hkv, p.D, p.P, p.T, p.Lq, p.dtype = 1, 4, 4, 64, 0, 8, 4, ds.DS_BF16
    fake = 0x7f0000000000  # never dereferenced: validation fails first
    p.q_tail = p.k_tail = p.v_tail = p.out = fake
    p.idx = fake
    for s in (p.q_stride, p.kv_tail_stride, p.out_stride):
        s[:] = (4 * 8 * 64, 8 * 64, 64)
    p.scale = 0.125
    for k, v in kw.items():
        if isinstance(v, tuple):
            getattr(p, k)[:] = v
        else:
            setattr(p, k, v)
    return p


def test_attention_argument_validation_needs_no_gpu(L):
    bad = [dict(Hkv=3), dict(Lq=0), dict(Lq=9), dict(D=0), dict(dtype=7), dict(q_tail=None), dict(idx=None),
           dict(out=None), dict(q_tail=0x7f0000000004), dict(q_stride=(4 * 8 * 64, 8 * 64, 60)),
           dict(kv_tail_stride=(4 * 8 * 64, 8 * 64, 32)), dict(P=16), dict(idx_batch_stride=2),
           dict(scale=float("nan")), dict(T=0)]
    for kw in bad:
        p = _attn(**kw)
        assert L.ds_attn_pruned(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG, kw
        assert L.ds_attn_pruned_workspace(ctypes.byref(p)) == 0
    assert L.ds_attn_pruned(None, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_attn_pruned(ctypes.byref(_attn(D=48, q_stride=(4 * 8 * 48, 8 * 48, 48),
                                               kv_tail_stride=(4 * 8 * 48, 8 * 48, 48),
                                               out_stride=(4 * 8 * 48, 8 * 48, 48))), None) == ds.DS_ERR_UNSUPPORTED
    # B = 0 is a valid empty call
    assert L.ds_attn_pruned(ctypes.byref(_attn(B=0)), None) == ds.DS_OK


def test_attention_envelope_refuses_instead_of_rerouting(L):
    """bf16 is served by the tensor-core kernels only (D 64 or 128, positive scale) and fp32 by the CUDA-core
    kernel only (D 32, 64, 128, 256): a well-formed request outside that is DS_ERR_UNSUPPORTED, decided on
    the host before any device is touched.  The kernel choice is an explicit field, not an environment
    variable."""
    def shaped(D, **kw):
        st = (4 * 8 * D, 8 * D, D)
        return _attn(**{**dict(D=D, q_stride=st, kv_tail_stride=st, out_stride=st), **kw})
    for p in (shaped(96), shaped(32), shaped(160), shaped(256), shaped(128, scale=0.0), shaped(64, scale=-0.125),
              shaped(96, dtype=ds.DS_F32), shaped(224, dtype=ds.DS_F32),
              shaped(128, B=2, q_stride=(0, 8 * 128, 128))):            # a broadcast batch: no tensor map for it
        assert L.ds_attn_pruned(ctypes.byref(p), None) == ds.DS_ERR_UNSUPPORTED
        assert L.ds_attn_pruned_workspace(ctypes.byref(p)) == 0
        h = ctypes.c_void_p()
        assert L.ds_attn_plan_create(ctypes.byref(p), ctypes.byref(h)) == ds.DS_ERR_UNSUPPORTED and not h.value
    for k in (-1, 3, 100):
        assert L.ds_attn_pruned(ctypes.byref(_attn(kernel=k)), None) == ds.DS_ERR_INVALID_ARG
    import os
    os.environ["DS_ATTN_PATH"] = "simt"          # the library reads no environment
    try:
        assert L.ds_attn_pruned(ctypes.byref(shaped(96)), None) == ds.DS_ERR_UNSUPPORTED
    finally:
        del os.environ["DS_ATTN_PATH"]
    src = "".join(f.read_text() for f in (ROOT / "paper_2601_17917_b200" / "csrc").glob("*.cu*"))
    assert "getenv" not in src


def test_bounded_wait_selftest_argument_validation(L):
    fake = ctypes.c_void_p(0x7f0000000000)
    assert L.ds_selftest_bounded_wait(0, fake, fake, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_selftest_bounded_wait(1 << 20, fake, fake, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_selftest_bounded_wait(100, ctypes.c_void_p(0x7f0000000002), fake, None) == ds.DS_ERR_INVALID_ARG


def test_confidence_and_select_argument_validation(L):
    fake = ctypes.c_void_p(0x7f0000000000)
    assert L.ds_confidence(fake, 1, 4, 0, 0, None, 0, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence(fake, 1, 4, 100, 64, None, 0, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence(fake, 5, 4, 100, 100, None, 0, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence(None, 1, 4, 100, 100, None, 0, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence(fake, 1, 0, 100, 100, None, 0, fake, fake, None, 0, None) == ds.DS_OK
    assert L.ds_confidence_workspace(32, 126464, 1) > 0
    p = ds._SelectParams()
    assert L.ds_unmask_select(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG       # K = 0
    p.B, p.K = 2, 5000
    assert L.ds_unmask_select(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG
    p.K = 32
    p.active_cnt = 0x7f0000000000
    assert L.ds_unmask_select(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG       # null arrays
    assert L.ds_unmask_select(None, None) == ds.DS_ERR_INVALID_ARG


def test_loop_control_entry_points_validate_without_a_gpu(L):
    fake = ctypes.c_void_p(0x7f0000000000)
    # plans: an invalid description gives the error of ds_attn_pruned and no plan; destroying NULL is allowed
    h = ctypes.c_void_p(0x1234)
    assert L.ds_attn_plan_create(ctypes.byref(_attn(Lq=0)), ctypes.byref(h)) == ds.DS_ERR_INVALID_ARG
    assert not h.value
    assert L.ds_attn_plan_create(ctypes.byref(_attn()), None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_attn_plan_launch(None, None) == ds.DS_ERR_INVALID_ARG
    L.ds_attn_plan_destroy(None)
    # sequence lists
    p = _attn()
    p.seq_list, p.n_seq = 0x7f0000000000, p.B + 1
    assert L.ds_attn_pruned(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG
    p.n_seq = -1
    assert L.ds_attn_pruned(ctypes.byref(p), None) == ds.DS_ERR_INVALID_ARG
    # rows listed on the device
    assert L.ds_confidence_listed(fake, 1, 4, 100, 100, None, 4, fake, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence_listed(fake, 1, 4, 100, 100, fake, 4, None, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence_listed(fake, 1, 4, 100, 100, fake, 5, fake, fake, fake, None, 0, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_confidence_listed(fake, 1, 4, 100, 100, fake, 0, fake, fake, fake, None, 0, None) == ds.DS_OK
    # start of a block
    b = ds._BlockParams()
    assert L.ds_block_begin(None, None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_block_begin(ctypes.byref(b), None) == ds.DS_ERR_INVALID_ARG       # K = 0
    b.B, b.K, b.active_cnt = 2, 32, 0x7f0000000000
    assert L.ds_block_begin(ctypes.byref(b), None) == ds.DS_ERR_INVALID_ARG       # null arrays
    b.masked_rows = 0x7f0000000000                                                  # rows without their count
    assert L.ds_block_begin(ctypes.byref(b), None) == ds.DS_ERR_INVALID_ARG
    assert L.ds_last_cuda_error() == 0 and L.ds_last_cuda_error_name() == b"cudaSuccess"


def test_host_index_list_matches_oracle():
    for gen, K, c, w, last in [(256, 32, 0, 16, True), (256, 32, 0, 32, True), (1024, 32, 0, 64, True),
                               (4096, 64, 0, 0, False), (4096, 64, 0, 64, True), (4096, 64, 0, 256, True),
                               (4096, 64, 3, 256, True), (256, 32, 7, 64, True), (256, 32, 6, 32, True),
                               (256, 32, 6, 31, True), (128, 32, 1, 500, True), (128, 32, 1, 0, True)]:
        assert ds.retained_indices(gen, K, c, w, last) == oracle.retained_indices(gen, K, c, w, last)
    # -1 = whole suffix = the unpruned method
    assert ds.retained_indices(4096, 64, 0, -1) == list(range(4096)) == oracle.retained_indices(4096, 64, 0, 4032)
    with pytest.raises(ValueError):
        ds.retained_indices(64, 32, 2, 8)


def test_binding_rejects_host_tensors():
    z = torch.zeros(4, 64)
    with pytest.raises(ValueError):
        ds.ds_confidence(z)


def test_workload_generators_are_seeded():
    from paper_2601_17917_b200 import workloads as wl
    cfg = wl.CONFIGS["tiny"]
    a, b = wl.attention_inputs(cfg), wl.attention_inputs(cfg)
    assert all(torch.equal(a[k], b[k]) for k in a)
    assert a["q_tail"].shape == (1, 4, 256, 64) and a["k_pre"].shape == (1, 4, 64, 64)
    z = wl.logits(cfg)
    assert z.shape == (32, 1024) and torch.equal(z, wl.logits(cfg))
    assert 1.8 < z.std().item() < 2.3
    x, m = wl.block_state(cfg, "half")
    assert int(m.sum()) == 16 and (x[m.bool()] == cfg.V - 1).all()

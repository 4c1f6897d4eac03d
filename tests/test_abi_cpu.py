"""CPU-only checks of the boundary: the shared library loads, exports every function the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2609_19242_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            src = open(os.path.join(inc, f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(bdlm_[a-z0-9_]+)\s*\(", src))
    return names


def test_library_exports_every_declared_symbol():
    L = binding.lib()
    declared = _declared_functions()
    assert {"bdlm_attn_fwd", "bdlm_attn_bwd", "bdlm_lse_merge"} <= declared
    for name in declared:
        assert hasattr(L, name), name
    assert declared >= set(binding.EXPORTS)


def test_status_strings():
    assert binding.status_string(0) == "BDLM_OK"
    assert binding.status_string(-1) == "BDLM_ERR_INVALID_ARG"
    assert binding.status_string(-5) == "BDLM_ERR_DEVICE_TIMEOUT"
    assert binding.status_string(-99) == "BDLM_ERR_UNKNOWN"


@pytest.mark.parametrize("kw,code", [
    (dict(batch=0), -1), (dict(L=100, block_size=16), -1), (dict(H=6, H_kv=4), -1),
    (dict(d=96), -2), (dict(clean_mask_mode=3), -1), (dict(kv_range=(8, 4)), -1),
    (dict(kv_range=(0, 4096)), -1), (dict(scale=-1.0), -1), (dict(impl=7), -1),
])
def test_bad_parameters_are_rejected_without_a_device(kw, code):
    base = dict(batch=1, L=256, block_size=16, H=4, H_kv=2, d=64)
    base.update(kw)
    p = binding.make_params(**base)
    fake = ctypes.c_void_p(0x1000)   # never dereferenced: parameter checks come first
    rc = binding.lib().bdlm_attn_fwd(ctypes.byref(p), *([fake] * 10), None, 0, None)
    assert rc == code
    assert binding.bdlm_workspace_bytes(p, binding.BDLM_WS_BWD) == 0


def test_null_and_misaligned_pointers_are_rejected():
    p = binding.make_params(1, 256, 16, 4, 2, 64)
    ok = ctypes.c_void_p(0x1000)
    bad = ctypes.c_void_p(0x1004)
    L = binding.lib()
    assert L.bdlm_attn_fwd(ctypes.byref(p), None, ok, ok, None, ok, ok, ok, ok, ok, ok, None, 0, None) == -1
    assert L.bdlm_attn_fwd(ctypes.byref(p), ok, None, ok, ok, ok, ok, ok, ok, ok, ok, None, 0, None) == -1
    assert L.bdlm_attn_fwd(ctypes.byref(p), bad, ok, ok, ok, ok, ok, ok, ok, ok, ok, None, 0, None) == -1
    assert L.bdlm_attn_fwd(None, *([ok] * 10), None, 0, None) == -1
    args = [ok] * 18
    assert L.bdlm_attn_bwd(ctypes.byref(p), *args, None, 0, None) == -1           # null workspace
    assert L.bdlm_attn_bwd(ctypes.byref(p), *args, ok, 16, None) == -3            # workspace too small
    ps = binding.make_params(1, 256, 16, 4, 2, 64, kv_range=(0, 128))
    assert L.bdlm_attn_bwd(ctypes.byref(ps), *args, ok, 1 << 30, None) == -2       # sharded backward
    arr = (ctypes.c_void_p * 2)(0x1000, 0x2000)
    assert L.bdlm_lse_merge(0, 1, 8, 1, 64, arr, arr, 0, ok, ok, None) == -1
    assert L.bdlm_lse_merge(17, 1, 8, 1, 64, arr, arr, 0, ok, ok, None) == -1
    assert L.bdlm_lse_merge(2, 1, 8, 1, 60, arr, arr, 0, ok, ok, None) == -1
    assert L.bdlm_lse_merge(2, 1, 8, 1, 64, arr, arr, 0, ok, ctypes.c_void_p(0x2000), None) == -1  # lse aliasing


def test_workspace_size_formula():
    p = binding.make_params(2, 512, 32, 8, 2, 128, impl=binding.IMPL_PORTABLE)
    need = binding.bdlm_workspace_bytes(p, binding.BDLM_WS_BWD)
    assert need >= 2 * 2 * 8 * 512 * 4
    assert binding.bdlm_workspace_bytes(p, binding.BDLM_WS_FWD) == 0
    # the backward modes: two-pass needs the D rows only; fused and automatic add the fp32 dQ accumulators
    # (2 streams x batch x H x L x 128 floats) when the tensor-core kernels take the shape, nothing otherwise
    mk = lambda sp, **kw: binding.bdlm_workspace_bytes(binding.make_params(2, 512, 32, 8, 2, 128, bwd_single_pass=sp, **kw),
                                                      binding.BDLM_WS_BWD)
    d_rows = 2 * 2 * 8 * 512 * 4
    acc = 2 * 2 * 8 * 512 * 128 * 4
    assert mk(False) == d_rows and mk(True) == d_rows + acc and mk(None) == d_rows + acc
    assert mk(None, impl=binding.IMPL_PORTABLE) == d_rows
    # a length that is no multiple of the fused kernel's 64-row steps: the accumulators are padded to whole steps
    ragged = binding.make_params(1, 160, 32, 4, 2, 128, bwd_single_pass=True)
    assert binding.bdlm_workspace_bytes(ragged, binding.BDLM_WS_BWD) == 2 * 160 * 4 * 4 + 2 * 192 * 4 * 128 * 4
    # head dimension 64 takes the tensor-core kernels too; its accumulator rows keep 128 floats
    d64 = binding.make_params(1, 256, 16, 4, 2, 64, bwd_single_pass=None)
    assert binding.bdlm_workspace_bytes(d64, binding.BDLM_WS_BWD) == 2 * 4 * 256 * 4 + 2 * 256 * 4 * 128 * 4
    # a forced fused backward refuses a workspace that holds only the D rows; the automatic mode accepts it
    ok = ctypes.c_void_p(0x1000)
    forced = binding.make_params(2, 512, 32, 8, 2, 128, bwd_single_pass=True)
    assert binding.lib().bdlm_attn_bwd(ctypes.byref(forced), *([ok] * 18), ok, d_rows, None) == -3
    bad_mode = binding.make_params(2, 512, 32, 8, 2, 128)
    bad_mode.bwd_single_pass = 3
    assert binding.lib().bdlm_attn_bwd(ctypes.byref(bad_mode), *([ok] * 18), ok, 1 << 30, None) == -1
    assert binding.lib().bdlm_selftest_wait_timeout(0, None) == -1
    assert binding.lib().bdlm_selftest_wait_timeout(1 << 40, None) == -1


def test_packed_geometry_is_checked_without_a_device():
    """Bad packed geometries are rejected before any pointer is used."""
    L = binding.lib()
    p = binding.make_params(1, 256, 16, 4, 2, 64)
    fake = ctypes.c_void_p(0x1000)
    for kw, code in [(dict(Lq_clean=-1), -1), (dict(Lq_clean=200, clean_q_pos0=100), -1),
                     (dict(n_blocks=-2), -1), (dict(n_blocks=4, block_prefix=0x1002), -1)]:
        g = binding.BdlmPackedGeometry()
        g.Lq_clean, g.clean_q_pos0, g.n_blocks, g.block_prefix = 128, 0, 8, None
        for k, v in kw.items():
            setattr(g, k, v)
        rc = L.bdlm_attn_fwd_packed(ctypes.byref(p), ctypes.byref(g), *([fake] * 10), None)
        assert rc == code, kw
        assert L.bdlm_workspace_bytes_packed(ctypes.byref(p), ctypes.byref(g), binding.BDLM_WS_BWD) == 0
    g = binding.BdlmPackedGeometry()
    g.Lq_clean, g.clean_q_pos0, g.n_blocks, g.block_prefix = 128, 64, 8, None
    assert L.bdlm_workspace_bytes_packed(ctypes.byref(p), ctypes.byref(g), binding.BDLM_WS_BWD) >= 2 * 4 * 128 * 4
    assert L.bdlm_attn_fwd_packed(ctypes.byref(p), None, *([fake] * 10), None) == -1
    # a clean length that is not a multiple of the block size is fine in the packed form only
    p2 = binding.make_params(1, 250, 16, 4, 2, 64)
    assert L.bdlm_workspace_bytes_packed(ctypes.byref(p2), ctypes.byref(g), binding.BDLM_WS_BWD) > 0
    assert binding.bdlm_workspace_bytes(p2, binding.BDLM_WS_BWD) == 0


def test_linear_ce_arguments_are_checked_without_a_device():
    L = binding.lib()
    ok = ctypes.c_void_p(0x1000)
    good = binding.make_lce_params(256, 64, 512)
    assert binding.bdlm_linear_ce_workspace_bytes(good, binding.LCE_WS_FWD) >= 3 * 256 * 4
    assert binding.bdlm_linear_ce_workspace_bytes(good, binding.LCE_WS_BWD) == 256 * 512 * 2          # one chunk: dz only
    big = binding.make_lce_params(1000, 64, 512, token_chunk=256)
    assert binding.bdlm_linear_ce_workspace_bytes(big, binding.LCE_WS_BWD) == 256 * 512 * 2 + 512 * 64 * 4   # + fp32 dW
    for kw in (dict(T=0, D=64, V=512), dict(T=8, D=60, V=512), dict(T=8, D=64, V=500), dict(T=8, D=64, V=512, token_chunk=100),
               dict(T=8, D=64, V=512, grad_loss=float("nan"))):
        p = binding.make_lce_params(**kw)
        assert binding.bdlm_linear_ce_workspace_bytes(p, binding.LCE_WS_FWD) == 0
        assert L.bdlm_linear_ce_fwd(ctypes.byref(p), *([ok] * 7), ok, 1 << 30, None) == -1
        assert L.bdlm_linear_ce_bwd(ctypes.byref(p), *([ok] * 7), ok, 1 << 30, None) == -1
    assert L.bdlm_linear_ce_fwd(ctypes.byref(good), None, ok, ok, ok, ok, ok, ok, ok, 1 << 30, None) == -1     # null h
    assert L.bdlm_linear_ce_fwd(ctypes.byref(good), ctypes.c_void_p(0x1008), ok, ok, ok, ok, ok, ok, ok, 1 << 30, None) == -1
    assert L.bdlm_linear_ce_fwd(ctypes.byref(good), *([ok] * 7), ok, 64, None) == -3                             # workspace too small
    assert L.bdlm_linear_ce_bwd(ctypes.byref(good), *([ok] * 7), ok, 64, None) == -3
    assert L.bdlm_linear_ce_fwd(None, *([ok] * 7), ok, 1 << 30, None) == -1

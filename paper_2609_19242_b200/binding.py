"""ctypes binding of `libbdlm_attn.so` (declarations in include/bdlm_attn.h).

Argument marshalling only: PyTorch supplies device memory and the current stream; every
step of the computation runs in the library's kernels.  There is no fallback: if the
shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbdlm_attn.so")

BDLM_WS_FWD, BDLM_WS_BWD = 0, 1
IMPL_AUTO, IMPL_PORTABLE, IMPL_TCGEN05 = 0, 1, 2
PASS_DSUM, PASS_DKDV, PASS_DQ = 1, 2, 4
BWD_AUTO, BWD_FUSED, BWD_TWO_PASS = 0, 1, 2

EXPORTS = ("bdlm_workspace_bytes", "bdlm_attn_fwd", "bdlm_attn_bwd", "bdlm_lse_merge",
           "bdlm_status_string", "bdlm_get_device_status", "bdlm_set_trace_buffer",
           "bdlm_attn_bwd_static_scratch", "bdlm_workspace_bytes_packed", "bdlm_attn_fwd_packed",
           "bdlm_attn_bwd_packed", "bdlm_selftest_wait_timeout", "bdlm_linear_ce_workspace_bytes",
           "bdlm_linear_ce_fwd", "bdlm_linear_ce_bwd")
LCE_WS_FWD, LCE_WS_BWD = 0, 1
STATIC_SCRATCH_ROWS = 1 << 20
TRACE_SLOTS = 256


class BdlmError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class BdlmParams(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("L", ctypes.c_int32), ("block_size", ctypes.c_int32),
                ("H", ctypes.c_int32), ("H_kv", ctypes.c_int32), ("d", ctypes.c_int32),
                ("scale", ctypes.c_float), ("clean_mask_mode", ctypes.c_int32),
                ("kv_begin", ctypes.c_int32), ("kv_end", ctypes.c_int32),
                ("kv_range_set", ctypes.c_int32), ("include_noisy_diag", ctypes.c_int32),
                ("impl", ctypes.c_int32), ("bwd_passes", ctypes.c_int32), ("bwd_single_pass", ctypes.c_int32),
                ("window", ctypes.c_int32), ("reserved", ctypes.c_int32 * 2)]


class BdlmPackedGeometry(ctypes.Structure):
    _fields_ = [("Lq_clean", ctypes.c_int32), ("clean_q_pos0", ctypes.c_int32), ("n_blocks", ctypes.c_int32),
                ("kv_chunk_len", ctypes.c_int32), ("block_prefix", ctypes.c_void_p),
                ("kv_chunk_pos", ctypes.c_void_p), ("kv_pos_chunk", ctypes.c_void_p)]


class BdlmLceParams(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("D", ctypes.c_int32), ("V", ctypes.c_int32), ("token_chunk", ctypes.c_int32),
                ("grad_loss", ctypes.c_float), ("reserved", ctypes.c_int32 * 3)]


_lib = None


def lib():
    """The loaded shared library (loads it on first use; raises if it is not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is not built; run `python -m paper_2609_19242_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, pp = ctypes.c_void_p, ctypes.POINTER(BdlmParams)
        L.bdlm_workspace_bytes.restype = ctypes.c_size_t
        L.bdlm_workspace_bytes.argtypes = [pp, ctypes.c_int32]
        L.bdlm_attn_fwd.restype = ctypes.c_int
        L.bdlm_attn_fwd.argtypes = [pp] + [vp] * 10 + [vp, ctypes.c_size_t, vp]
        L.bdlm_attn_bwd.restype = ctypes.c_int
        L.bdlm_attn_bwd.argtypes = [pp] + [vp] * 18 + [vp, ctypes.c_size_t, vp]
        L.bdlm_lse_merge.restype = ctypes.c_int
        L.bdlm_lse_merge.argtypes = [ctypes.c_int32] * 5 + [ctypes.POINTER(vp), ctypes.POINTER(vp),
                                                             ctypes.c_int32, vp, vp, vp]
        L.bdlm_status_string.restype = ctypes.c_char_p
        L.bdlm_status_string.argtypes = [ctypes.c_int]
        L.bdlm_get_device_status.restype = ctypes.c_int
        L.bdlm_get_device_status.argtypes = [vp]
        L.bdlm_attn_bwd_static_scratch.restype = ctypes.c_int
        L.bdlm_attn_bwd_static_scratch.argtypes = [pp] + [vp] * 18 + [vp]
        L.bdlm_set_trace_buffer.restype = ctypes.c_int
        L.bdlm_set_trace_buffer.argtypes = [vp, ctypes.c_size_t]
        gp = ctypes.POINTER(BdlmPackedGeometry)
        L.bdlm_workspace_bytes_packed.restype = ctypes.c_size_t
        L.bdlm_workspace_bytes_packed.argtypes = [pp, gp, ctypes.c_int32]
        L.bdlm_attn_fwd_packed.restype = ctypes.c_int
        L.bdlm_attn_fwd_packed.argtypes = [pp, gp] + [vp] * 10 + [vp]
        L.bdlm_attn_bwd_packed.restype = ctypes.c_int
        L.bdlm_attn_bwd_packed.argtypes = [pp, gp] + [vp] * 18 + [vp, ctypes.c_size_t, vp]
        lp = ctypes.POINTER(BdlmLceParams)
        L.bdlm_linear_ce_workspace_bytes.restype = ctypes.c_size_t
        L.bdlm_linear_ce_workspace_bytes.argtypes = [lp, ctypes.c_int32]
        L.bdlm_linear_ce_fwd.restype = ctypes.c_int
        L.bdlm_linear_ce_fwd.argtypes = [lp] + [vp] * 7 + [vp, ctypes.c_size_t, vp]
        L.bdlm_linear_ce_bwd.restype = ctypes.c_int
        L.bdlm_linear_ce_bwd.argtypes = [lp] + [vp] * 7 + [vp, ctypes.c_size_t, vp]
        L.bdlm_selftest_wait_timeout.restype = ctypes.c_int
        L.bdlm_selftest_wait_timeout.argtypes = [ctypes.c_int64, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().bdlm_status_string(int(status)).decode()


bdlm_status_string = status_string


def make_params(batch, L, block_size, H, H_kv, d, scale=0.0, clean_mask_mode=0, kv_range=None,
                include_noisy_diag=True, impl=IMPL_AUTO, bwd_passes=0, bwd_single_pass=None, window=0) -> BdlmParams:
    """`bwd_single_pass`: None = automatic (BDLM_BWD_AUTO: the fused kernel when the workspace has room for it),
    True = the fused kernel (BDLM_BWD_FUSED), False = the two-pass kernels (BDLM_BWD_TWO_PASS)."""
    p = BdlmParams()
    p.batch, p.L, p.block_size, p.H, p.H_kv, p.d = batch, L, block_size, H, H_kv, d
    p.scale = float(scale)
    p.clean_mask_mode = clean_mask_mode
    if kv_range is None:
        p.kv_begin, p.kv_end, p.kv_range_set = 0, 0, 0
    else:
        p.kv_begin, p.kv_end, p.kv_range_set = int(kv_range[0]), int(kv_range[1]), 1
    p.include_noisy_diag = 1 if include_noisy_diag else 0
    p.impl = impl
    p.bwd_passes = bwd_passes
    p.bwd_single_pass = BWD_AUTO if bwd_single_pass is None else (BWD_FUSED if bwd_single_pass else BWD_TWO_PASS)
    p.window = int(window)
    return p


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _shape_params(q, k, block_size, **kw):
    batch, L, H, d = q.shape
    return make_params(batch, L, block_size, H, k.shape[2], d, **kw)


def bdlm_workspace_bytes(params: BdlmParams, which: int) -> int:
    return int(lib().bdlm_workspace_bytes(ctypes.byref(params), which))


def bdlm_attn_fwd(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, block_size, *,
                  out=None, scale=0.0, clean_mask_mode=0, kv_range=None, include_noisy_diag=True,
                  impl=IMPL_AUTO, window=0):
    """Forward of the layer.  Tensors: q [batch,L,H,d], k/v [batch,L,H_kv,d], bf16, on one CUDA
    device.  Either q may be None (that stream is skipped).  Returns
    (o_clean, lse_clean, o_noisy, lse_noisy); `out` may supply those four tensors."""
    qref = q_clean if q_clean is not None else q_noisy
    p = _shape_params(qref, k_clean, block_size, scale=scale, clean_mask_mode=clean_mask_mode,
                      kv_range=kv_range, include_noisy_diag=include_noisy_diag, impl=impl, window=window)
    dev = qref.device
    if out is None:
        mk_o = lambda q: None if q is None else torch.empty_like(q)
        mk_l = lambda q: None if q is None else torch.empty(p.batch, p.H, p.L, dtype=torch.float32, device=dev)
        out = (mk_o(q_clean), mk_l(q_clean), mk_o(q_noisy), mk_l(q_noisy))
    o_c, l_c, o_n, l_n = out
    rc = lib().bdlm_attn_fwd(ctypes.byref(p), _ptr(q_clean), _ptr(k_clean), _ptr(v_clean),
                             _ptr(q_noisy), _ptr(k_noisy), _ptr(v_noisy),
                             _ptr(o_c), _ptr(o_n), _ptr(l_c), _ptr(l_n), None, 0, _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_attn_fwd")
    return o_c, l_c, o_n, l_n


def bdlm_attn_bwd(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, lse_clean,
                  o_noisy, lse_noisy, do_clean, do_noisy, block_size, *, out=None, workspace=None,
                  scale=0.0, clean_mask_mode=0, impl=IMPL_AUTO, passes=0, single_pass=None, window=0):
    """Backward of the layer.  Returns (dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy).
    `single_pass=True` selects the fused one-kernel backward (dQ through fp32 add-reductions into a
    workspace accumulator: faster, dQ reproducible only up to fp32 summation order), `False` the two-pass
    kernels (every gradient bitwise reproducible); `None` (default) lets the library take the fused kernel
    whenever the workspace it is given has room for it -- the workspace allocated here always has."""
    p = _shape_params(q_clean, k_clean, block_size, scale=scale, clean_mask_mode=clean_mask_mode, impl=impl,
                      bwd_passes=passes, bwd_single_pass=single_pass, window=window)
    if out is None:
        out = tuple(torch.empty_like(t) for t in (q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy))
    need = bdlm_workspace_bytes(p, BDLM_WS_BWD)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=q_clean.device)
    dq_c, dk_c, dv_c, dq_n, dk_n, dv_n = out
    rc = lib().bdlm_attn_bwd(ctypes.byref(p), _ptr(q_clean), _ptr(k_clean), _ptr(v_clean),
                             _ptr(q_noisy), _ptr(k_noisy), _ptr(v_noisy), _ptr(o_clean), _ptr(o_noisy),
                             _ptr(lse_clean), _ptr(lse_noisy), _ptr(do_clean), _ptr(do_noisy),
                             _ptr(dq_c), _ptr(dk_c), _ptr(dv_c), _ptr(dq_n), _ptr(dk_n), _ptr(dv_n),
                             _ptr(workspace), workspace.numel(), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_attn_bwd")
    return out


def bdlm_attn_bwd_static_scratch(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, lse_clean,
                                 o_noisy, lse_noisy, do_clean, do_noisy, block_size, *, out,
                                 scale=0.0, clean_mask_mode=0, impl=IMPL_AUTO):
    """Backward through the entry point that takes no workspace: the library's built-in scratch
    array is used, so this wrapper allocates nothing either -- `out` (the six gradient tensors)
    must be supplied by the caller.  For callers that may not allocate device memory; limited to
    batch*H*L <= STATIC_SCRATCH_ROWS, and calls that overlap on the GPU must be serialised."""
    p = _shape_params(q_clean, k_clean, block_size, scale=scale, clean_mask_mode=clean_mask_mode, impl=impl)
    dq_c, dk_c, dv_c, dq_n, dk_n, dv_n = out
    rc = lib().bdlm_attn_bwd_static_scratch(
        ctypes.byref(p), _ptr(q_clean), _ptr(k_clean), _ptr(v_clean), _ptr(q_noisy), _ptr(k_noisy), _ptr(v_noisy),
        _ptr(o_clean), _ptr(o_noisy), _ptr(lse_clean), _ptr(lse_noisy), _ptr(do_clean), _ptr(do_noisy),
        _ptr(dq_c), _ptr(dk_c), _ptr(dv_c), _ptr(dq_n), _ptr(dk_n), _ptr(dv_n), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_attn_bwd_static_scratch")
    return out


_checked_prefix_tables = set()


def _packed_setup(q_clean, k_clean, q_noisy, block_size, block_prefix, clean_q_pos0, window, kv_chunks=None, **kw):
    """Parameters and geometry of a packed call.  `block_prefix` is an int32 CUDA tensor [n_blocks] (or None
    for b * block_size); its ordering rules are checked here on a host copy because the C library never reads
    device memory on the host."""
    batch, L, H_kv, d = k_clean.shape
    qref = q_clean if q_clean is not None else q_noisy
    H = qref.shape[2]
    p = make_params(batch, L, block_size, H, H_kv, d, window=window, **kw)
    g = BdlmPackedGeometry()
    g.Lq_clean = 0 if q_clean is None else q_clean.shape[1]
    g.clean_q_pos0 = int(clean_q_pos0)
    g.n_blocks = 0
    g.block_prefix = None
    g.kv_chunk_len, g.kv_chunk_pos, g.kv_pos_chunk = 0, None, None
    keep = []   # device tables must outlive the launch call
    if kv_chunks is not None:
        # kv_chunks = (chunk_len, positions): memory chunk m of the clean K/V holds positions[m] .. + chunk_len - 1
        chunk_len, positions = int(kv_chunks[0]), [int(x) for x in kv_chunks[1]]
        n = L // chunk_len if chunk_len > 0 else 0
        if chunk_len <= 0 or L % chunk_len != 0 or len(positions) != n:
            raise ValueError("kv_chunks: chunk_len must divide L and there must be L / chunk_len positions")
        if sorted(positions) != [c * chunk_len for c in range(n)]:
            raise ValueError("kv_chunks: positions must be a permutation of the multiples of chunk_len")
        inv = [0] * n
        for m, pos in enumerate(positions):
            inv[pos // chunk_len] = m
        t_pos = torch.tensor(positions, dtype=torch.int32, device=k_clean.device)
        t_inv = torch.tensor(inv, dtype=torch.int32, device=k_clean.device)
        keep += [t_pos, t_inv]
        g.kv_chunk_len, g.kv_chunk_pos, g.kv_pos_chunk = chunk_len, t_pos.data_ptr(), t_inv.data_ptr()
    if q_noisy is not None:
        if q_noisy.shape[1] % block_size != 0:
            raise ValueError("packed noisy rows must be a whole number of blocks")
        g.n_blocks = q_noisy.shape[1] // block_size
        if block_prefix is not None:
            assert block_prefix.is_cuda and block_prefix.dtype == torch.int32 and block_prefix.is_contiguous()
            if block_prefix.numel() != g.n_blocks:
                raise ValueError("block_prefix needs one entry per packed block")
            # the host copy synchronises the device: a table that was checked once (same storage, same version
            # counter, same rules) is not copied again on the calls of later steps
            key = (block_prefix.data_ptr(), block_prefix.numel(), block_prefix._version, L, block_size, window > 0)
            if key not in _checked_prefix_tables:
                host = block_prefix.cpu()
                step = host[1:] - host[:-1]
                if host.numel() and (int(host.min()) < 0 or int(host.max()) > L):
                    raise ValueError("block_prefix entries must lie in [0, L]")
                if step.numel() and int(step.min()) < 0:
                    raise ValueError("block_prefix must be non-decreasing (sort the packed blocks)")
                if window > 0 and step.numel() and int(step.min()) < block_size:
                    raise ValueError("with a sliding window the packed blocks must not overlap in position")
                if len(_checked_prefix_tables) >= 256:
                    _checked_prefix_tables.clear()
                _checked_prefix_tables.add(key)
            g.block_prefix = block_prefix.data_ptr()
    g._keep = keep
    return p, g


def bdlm_attn_fwd_packed(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, block_size, *,
                         block_prefix=None, clean_q_pos0=0, out=None, scale=0.0, clean_mask_mode=0,
                         kv_range=None, include_noisy_diag=True, impl=IMPL_AUTO, window=0, kv_chunks=None):
    """Forward of the packed form (one rank's launch of the CSBP schedule; DFlash2-style blocks).
    q_clean [batch, Lq, H, d] or None: clean queries at positions clean_q_pos0 .. ; q_noisy
    [batch, n_blocks*block_size, H, d] or None with k_noisy/v_noisy packed alike; k_clean/v_clean
    [batch, L, H_kv, d] complete.  Returns (o_clean, lse_clean, o_noisy, lse_noisy)."""
    p, g = _packed_setup(q_clean, k_clean, q_noisy, block_size, block_prefix, clean_q_pos0, window, kv_chunks,
                         scale=scale, clean_mask_mode=clean_mask_mode, kv_range=kv_range,
                         include_noisy_diag=include_noisy_diag, impl=impl)
    dev = k_clean.device
    if out is None:
        mk_o = lambda q: None if q is None else torch.empty_like(q)
        mk_l = lambda q: None if q is None else torch.empty(p.batch, p.H, q.shape[1], dtype=torch.float32, device=dev)
        out = (mk_o(q_clean), mk_l(q_clean), mk_o(q_noisy), mk_l(q_noisy))
    o_c, l_c, o_n, l_n = out
    rc = lib().bdlm_attn_fwd_packed(ctypes.byref(p), ctypes.byref(g), _ptr(q_clean), _ptr(k_clean), _ptr(v_clean),
                                    _ptr(q_noisy), _ptr(k_noisy), _ptr(v_noisy),
                                    _ptr(o_c), _ptr(o_n), _ptr(l_c), _ptr(l_n), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_attn_fwd_packed")
    return o_c, l_c, o_n, l_n


def bdlm_attn_bwd_packed(q_clean, k_clean, v_clean, q_noisy, k_noisy, v_noisy, o_clean, lse_clean,
                         o_noisy, lse_noisy, do_clean, do_noisy, block_size, *, block_prefix=None,
                         clean_q_pos0=0, out=None, workspace=None, scale=0.0, clean_mask_mode=0,
                         impl=IMPL_AUTO, passes=0, single_pass=None, window=0, kv_chunks=None):
    """Backward of the packed form.  Returns (dq_clean, dk_clean, dv_clean, dq_noisy, dk_noisy, dv_noisy);
    entries of a stream that was left out are None.  dk_clean/dv_clean are this call's contribution for
    every clean key.  `single_pass` as in bdlm_attn_bwd."""
    p, g = _packed_setup(q_clean, k_clean, q_noisy, block_size, block_prefix, clean_q_pos0, window, kv_chunks,
                         scale=scale, clean_mask_mode=clean_mask_mode, impl=impl, bwd_passes=passes,
                         bwd_single_pass=single_pass)
    if out is None:
        e = lambda t: None if t is None else torch.empty_like(t)
        out = (e(q_clean), torch.empty_like(k_clean), torch.empty_like(v_clean), e(q_noisy),
               e(k_noisy if q_noisy is not None else None), e(v_noisy if q_noisy is not None else None))
    need = int(lib().bdlm_workspace_bytes_packed(ctypes.byref(p), ctypes.byref(g), BDLM_WS_BWD))
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=k_clean.device)
    dq_c, dk_c, dv_c, dq_n, dk_n, dv_n = out
    rc = lib().bdlm_attn_bwd_packed(ctypes.byref(p), ctypes.byref(g), _ptr(q_clean), _ptr(k_clean), _ptr(v_clean),
                                    _ptr(q_noisy), _ptr(k_noisy), _ptr(v_noisy), _ptr(o_clean), _ptr(o_noisy),
                                    _ptr(lse_clean), _ptr(lse_noisy), _ptr(do_clean), _ptr(do_noisy),
                                    _ptr(dq_c), _ptr(dk_c), _ptr(dv_c), _ptr(dq_n), _ptr(dk_n), _ptr(dv_n),
                                    _ptr(workspace), workspace.numel(), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_attn_bwd_packed")
    return out


def bdlm_lse_merge(o_partials, lse_partials, *, out=None):
    """Merge normalised partial outputs [batch,L,H,d] (all bf16 or all fp32) with row LSEs
    [batch,H,L] over disjoint key sets.  Returns (o bf16, lse fp32)."""
    n = len(o_partials)
    batch, L, H, d = o_partials[0].shape
    dtype = 1 if o_partials[0].dtype == torch.float32 else 0
    if out is None:
        out = (torch.empty(batch, L, H, d, dtype=torch.bfloat16, device=o_partials[0].device),
               torch.empty(batch, H, L, dtype=torch.float32, device=o_partials[0].device))
    arr_t = ctypes.c_void_p * n
    o_arr = arr_t(*[t.data_ptr() for t in o_partials])
    l_arr = arr_t(*[t.data_ptr() for t in lse_partials])
    for t in list(o_partials) + list(lse_partials):
        assert t.is_cuda and t.is_contiguous()
    rc = lib().bdlm_lse_merge(n, batch, L, H, d, o_arr, l_arr, dtype, _ptr(out[0]), _ptr(out[1]), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_lse_merge")
    return out


def bdlm_get_device_status() -> int:
    return int(lib().bdlm_get_device_status(_stream()))


def bdlm_selftest_wait_timeout(limit_ticks: int) -> None:
    """Launches the library's bounded-wait self-test kernel: a wait that runs out after `limit_ticks`
    clock ticks; afterwards bdlm_get_device_status() reports BDLM_ERR_DEVICE_TIMEOUT once."""
    rc = lib().bdlm_selftest_wait_timeout(int(limit_ticks), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_selftest_wait_timeout")


def bdlm_set_trace_buffer(counters) -> None:
    """Switch kernel tracing on (an int64 CUDA tensor of TRACE_SLOTS zeros) or off (None)."""
    if counters is None:
        rc = lib().bdlm_set_trace_buffer(None, 0)
    else:
        assert counters.is_cuda and counters.dtype == torch.int64 and counters.numel() >= TRACE_SLOTS
        rc = lib().bdlm_set_trace_buffer(_ptr(counters), counters.numel() * 8)
    if rc != 0:
        raise BdlmError(rc, "bdlm_set_trace_buffer")


# ------------------------------------------------------------------------------------------
# token-chunked linear cross-entropy (include/bdlm_linear_ce.h)
# ------------------------------------------------------------------------------------------
def make_lce_params(T, D, V, token_chunk=0, grad_loss=1.0) -> BdlmLceParams:
    p = BdlmLceParams()
    p.T, p.D, p.V, p.token_chunk, p.grad_loss = int(T), int(D), int(V), int(token_chunk), float(grad_loss)
    return p


def bdlm_linear_ce_workspace_bytes(params: BdlmLceParams, which: int) -> int:
    return int(lib().bdlm_linear_ce_workspace_bytes(ctypes.byref(params), which))


def bdlm_linear_ce_fwd(h, w, labels, token_weight=None, *, out=None, workspace=None):
    """Forward of the linear cross-entropy: h [T, D] bf16, w [V, D] bf16, labels [T] int32 (negative = ignored),
    token_weight [T] fp32 or None.  Returns (loss [1] fp32, nll [T] fp32, lse [T] fp32), all on the device."""
    T, D = h.shape
    V = w.shape[0]
    p = make_lce_params(T, D, V)
    if out is None:
        out = (torch.empty(1, dtype=torch.float32, device=h.device), torch.empty(T, dtype=torch.float32, device=h.device),
               torch.empty(T, dtype=torch.float32, device=h.device))
    if workspace is None:
        workspace = torch.empty(max(bdlm_linear_ce_workspace_bytes(p, LCE_WS_FWD), 16), dtype=torch.uint8, device=h.device)
    assert labels.dtype == torch.int32
    rc = lib().bdlm_linear_ce_fwd(ctypes.byref(p), _ptr(h), _ptr(w), _ptr(labels), _ptr(token_weight), _ptr(out[0]),
                                  _ptr(out[1]), _ptr(out[2]), _ptr(workspace), workspace.numel(), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_linear_ce_fwd")
    return out


def bdlm_linear_ce_bwd(h, w, labels, lse, token_weight=None, *, grad_loss=1.0, token_chunk=0, out=None, workspace=None):
    """Backward of the linear cross-entropy for the upstream scalar gradient `grad_loss`.  Returns (dh [T, D] bf16,
    dw [V, D] bf16).  `token_chunk` (a multiple of 128, 0 = default) bounds the dz scratch to token_chunk * V bf16."""
    T, D = h.shape
    V = w.shape[0]
    p = make_lce_params(T, D, V, token_chunk=token_chunk, grad_loss=grad_loss)
    if out is None:
        out = (torch.empty_like(h), torch.empty_like(w))
    if workspace is None:
        workspace = torch.empty(max(bdlm_linear_ce_workspace_bytes(p, LCE_WS_BWD), 16), dtype=torch.uint8, device=h.device)
    assert labels.dtype == torch.int32
    rc = lib().bdlm_linear_ce_bwd(ctypes.byref(p), _ptr(h), _ptr(w), _ptr(labels), _ptr(token_weight), _ptr(lse),
                                  _ptr(out[0]), _ptr(out[1]), _ptr(workspace), workspace.numel(), _stream())
    if rc != 0:
        raise BdlmError(rc, "bdlm_linear_ce_bwd")
    return out

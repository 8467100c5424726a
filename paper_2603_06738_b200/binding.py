"""Thin Python binding of the C ABI in ``include/rib_window_attn.h``.

Argument marshalling only: torch supplies device memory and the current stream, every step of
the computation runs in the CUDA kernels of ``librib_window_attn.so``.  There is no CPU or
PyTorch fallback: if the shared library has not been built, importing this module's functions
raises ``RibLibraryMissing``.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "librib_window_attn.so"
_lib = None

RIB_OK = 0
RIB_ERR_DEVICE_WAIT = -7
RIB_PATH_NONE, RIB_PATH_GENERIC, RIB_PATH_SM100, RIB_PATH_SM100_EXACT = 0, 1, 2, 3

EXPORTS = (
    "rib_window_attn_fwd", "rib_window_attn_bwd", "rib_window_attn_bwd_workspace",
    "rib_query_status", "rib_status_string", "rib_set_path", "rib_last_path", "rib_kernel_launches",
    "rib_window_attn_bwd_noalloc", "rib_profile_begin", "rib_profile_end",
    "rib_generate_features", "rib_generate_features_bwd",
    "rib_window_attn_fwd_headwise", "rib_window_attn_bwd_headwise", "rib_window_attn_bwd_headwise_workspace",
    "rib_window_attn_fwd_padded", "rib_cla_gate", "rib_window_attn_fwd_gated",
    "rib_window_attn_bwd_padded", "rib_window_attn_bwd_padded_workspace",
    "rib_window_attn_fwd_masked", "rib_window_attn_bwd_masked", "rib_window_cycle_bwd", "rib_window_cycle_bwd_workspace",
    "rib_cla_product", "rib_cla_product_bwd", "rib_cla_gate_bwd", "rib_cla_gate_bwd_workspace",
    "rib_wait_probe", "rib_exp_probe", "rib_tensor_map_cache_counts", "rib_window_cycle_fwd",
)
KERNEL_NAMES = {1: "rib_fwd_sm100_kernel", 2: "rib_bwd_prepare_kernel", 3: "rib_bwd_sm100_kernel",
                4: "rib_bwd_finish_kernel", 6: "generic_fwd_kernel",
                7: "rowdot_kernel", 8: "generic_bwd_dq_kernel", 9: "generic_bwd_dkv_kernel",
                10: "rib_generator_fwd_kernel", 11: "rib_generator_bwd_kernel", 12: "rib_cla_gate_kernel",
                13: "rib_cla_bwd_pw_kernel", 14: "rib_cla_bwd_dw_kernel", 15: "rib_cla_product_kernel", 16: "rib_cla_bwd_tc_kernel"}
RIB_NOALLOC_SCRATCH_BYTES = 32 << 20


class RibLibraryMissing(RuntimeError):
    pass


class RibError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"rib call failed with {code}: {rib_status_string(code)}")


def library() -> ctypes.CDLL:
    """Load (once) the in-tree shared library and declare the C signatures."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RibLibraryMissing(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2603_06738_b200.build`")
        lib = ctypes.CDLL(str(_LIB_PATH))
        vp, ci, fp = ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p
        lib.rib_window_attn_fwd.restype = ci
        lib.rib_window_attn_fwd.argtypes = [vp] * 5 + [ci] * 8 + [vp, fp, vp]
        lib.rib_window_attn_bwd.restype = ci
        lib.rib_window_attn_bwd.argtypes = [vp] * 8 + [ci] * 8 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        ll = ctypes.c_longlong
        lib.rib_window_attn_fwd_headwise.restype = ci
        lib.rib_window_attn_fwd_headwise.argtypes = [vp] * 5 + [ll] + [ci] * 8 + [vp, fp, vp]
        lib.rib_window_attn_fwd_padded.restype = ci
        lib.rib_window_attn_fwd_padded.argtypes = [vp] * 5 + [ll] + [ci] * 8 + [vp, fp, vp]
        lib.rib_window_attn_bwd_padded.restype = ci
        lib.rib_window_attn_bwd_padded.argtypes = [vp] * 5 + [ll] + [vp] * 3 + [ci] * 8 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        lib.rib_window_cycle_bwd.restype = ci
        lib.rib_window_cycle_bwd.argtypes = [vp] * 8 + [vp, vp, ci] + [ci] * 6 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        lib.rib_window_cycle_bwd_workspace.restype = ctypes.c_size_t
        lib.rib_window_cycle_bwd_workspace.argtypes = [vp, ci] + [ci] * 6
        lib.rib_window_attn_fwd_masked.restype = ci
        lib.rib_window_attn_fwd_masked.argtypes = [vp] * 5 + [ll] + [ci] * 8 + [vp, fp, vp]
        lib.rib_window_attn_bwd_masked.restype = ci
        lib.rib_window_attn_bwd_masked.argtypes = [vp] * 5 + [ll] + [vp] * 3 + [ci] * 8 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        lib.rib_window_attn_bwd_padded_workspace.restype = ctypes.c_size_t
        lib.rib_window_attn_bwd_padded_workspace.argtypes = [ll] + [ci] * 7
        lib.rib_cla_gate.restype = ci
        lib.rib_cla_gate.argtypes = [vp] * 5 + [ci] * 4 + [vp, vp]
        lib.rib_cla_product.restype = ci
        lib.rib_cla_product.argtypes = [vp, vp, ll, vp, vp]
        lib.rib_cla_product_bwd.restype = ci
        lib.rib_cla_product_bwd.argtypes = [vp, vp, vp, ll, vp, vp, vp]
        lib.rib_cla_gate_bwd.restype = ci
        lib.rib_cla_gate_bwd.argtypes = [vp] * 6 + [ci] * 4 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        lib.rib_cla_gate_bwd_workspace.restype = ctypes.c_size_t
        lib.rib_cla_gate_bwd_workspace.argtypes = [ci] * 4
        lib.rib_window_attn_fwd_gated.restype = ci
        lib.rib_window_attn_fwd_gated.argtypes = [vp] * 5 + [ll, vp] + [ci] * 8 + [vp, fp, vp]
        lib.rib_window_attn_bwd_headwise.restype = ci
        lib.rib_window_attn_bwd_headwise.argtypes = [vp] * 5 + [ll] + [vp] * 3 + [ci] * 8 + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        lib.rib_window_attn_bwd_headwise_workspace.restype = ctypes.c_size_t
        lib.rib_window_attn_bwd_headwise_workspace.argtypes = [ll] + [ci] * 7
        lib.rib_window_attn_bwd_noalloc.restype = ci
        lib.rib_window_attn_bwd_noalloc.argtypes = [vp] * 8 + [ci] * 8 + [vp] * 5 + [vp]
        lib.rib_generate_features.restype = ci
        lib.rib_generate_features.argtypes = [vp] * 4 + [ci] * 4 + [vp] * 3
        lib.rib_generate_features_bwd.restype = ci
        lib.rib_generate_features_bwd.argtypes = [vp] * 6 + [ci] * 4 + [vp] * 5
        lib.rib_profile_begin.restype = ci
        lib.rib_profile_begin.argtypes = [ci]
        lib.rib_profile_end.restype = ci
        lib.rib_profile_end.argtypes = [ctypes.POINTER(ci), ctypes.POINTER(ctypes.c_float), ci]
        lib.rib_window_attn_bwd_workspace.restype = ctypes.c_size_t
        lib.rib_window_attn_bwd_workspace.argtypes = [ci] * 7
        lib.rib_query_status.restype = ci
        lib.rib_query_status.argtypes = [vp]
        lib.rib_status_string.restype = ctypes.c_char_p
        lib.rib_status_string.argtypes = [ci]
        lib.rib_set_path.restype = ci
        lib.rib_set_path.argtypes = [ci]
        lib.rib_last_path.restype = ci
        lib.rib_last_path.argtypes = []
        lib.rib_kernel_launches.restype = ctypes.c_longlong
        lib.rib_kernel_launches.argtypes = []
        lib.rib_window_cycle_fwd.restype = ci
        lib.rib_window_cycle_fwd.argtypes = [ctypes.POINTER(vp)] * 5 + [ctypes.POINTER(ci)] * 2 + [ci] * 7 + [ctypes.POINTER(vp)] * 2 + [vp]
        lib.rib_tensor_map_cache_counts.restype = None
        lib.rib_tensor_map_cache_counts.argtypes = [ctypes.POINTER(ctypes.c_longlong)] * 2
        lib.rib_wait_probe.restype = ci
        lib.rib_wait_probe.argtypes = [ctypes.c_ulonglong, vp]
        lib.rib_exp_probe.restype = ctypes.c_longlong
        lib.rib_exp_probe.argtypes = [vp, ci, ci, vp]
        _lib = lib
    return _lib


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _ptr(t) -> int | None:
    return None if t is None else int(t.data_ptr())


def _check_image(name, t, shape=None):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 5:
        raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor [B,H,W,heads,d]")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")


def _check_pos(name, t, n):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 2 or t.shape[0] != n:
        raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor [n={n}, r]")


def _check_pos_headwise(name, t, heads, n):
    if (t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 3
            or t.shape[0] != heads or t.shape[1] != n):
        raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor [heads={heads}, n={n}, r]")


def rib_status_string(code: int) -> str:
    return library().rib_status_string(int(code)).decode()


def rib_set_path(path: int) -> int:
    return int(library().rib_set_path(int(path)))


def rib_last_path() -> int:
    return int(library().rib_last_path())


def rib_kernel_launches() -> int:
    return int(library().rib_kernel_launches())


def rib_profile_begin(max_launches: int) -> None:
    rc = int(library().rib_profile_begin(int(max_launches)))
    if rc != RIB_OK:
        raise RibError(rc)


def rib_profile_end(capacity: int) -> list[tuple[int, float]]:
    """Ends the per-kernel timing session; returns [(kernel id, device milliseconds), ...] in launch order."""
    ids = (ctypes.c_int * capacity)()
    ms = (ctypes.c_float * capacity)()
    n = int(library().rib_profile_end(ids, ms, capacity))
    if n < 0:
        raise RibError(n)
    return [(int(ids[i]), float(ms[i])) for i in range(n)]


def rib_query_status(stream=None) -> int:
    return int(library().rib_query_status(_stream_ptr(stream)))


def rib_tensor_map_cache_counts() -> tuple[int, int]:
    """(hits, misses) of the library's tensor-map cache in this process."""
    h, m = ctypes.c_longlong(0), ctypes.c_longlong(0)
    library().rib_tensor_map_cache_counts(ctypes.byref(h), ctypes.byref(m))
    return int(h.value), int(m.value)


def rib_wait_probe(limit_ns: int, stream=None) -> None:
    """Enqueue the self-test kernel whose bounded wait runs out after `limit_ns` nanoseconds."""
    rc = int(library().rib_wait_probe(int(limit_ns), _stream_ptr(stream)))
    if rc != RIB_OK:
        raise RibError(rc)


def rib_exp_probe(sink, blocks: int, iters: int, stream=None) -> int:
    """Enqueue the exp-throughput kernel; returns the number of exponentials it evaluates."""
    n = int(library().rib_exp_probe(_ptr(sink), int(blocks), int(iters), _stream_ptr(stream)))
    if n < 0:
        raise RibError(n)
    return n


def rib_window_attn_bwd_workspace(B, H, W, heads, d, r, window) -> int:
    return int(library().rib_window_attn_bwd_workspace(B, H, W, heads, d, r, window))


def rib_window_attn_fwd(q, k, v, pq, pk, window, shift=0, out=None, lse=None, stream=None, want_lse=True):
    """Enqueue the forward pass; returns (out bf16 [B,H,W,heads,d], lse fp32 [B,heads,H,W] or None)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    _check_image("k", k, q.shape)
    _check_image("v", v, q.shape)
    n = window * window
    _check_pos("pq", pq, n)
    _check_pos("pk", pk, n)
    r = pq.shape[1]
    if out is None:
        out = torch.empty_like(q)
    if lse is None and want_lse:
        lse = torch.empty((B, heads, H, W), dtype=torch.float32, device=q.device)
    rc = library().rib_window_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), B, H, W, heads, d, r,
                                       window, shift, _ptr(out), _ptr(lse), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return out, lse


def rib_window_attn_bwd(q, k, v, pq, pk, out, lse, dout, window, shift=0, workspace=None, stream=None):
    """Enqueue the backward pass; returns (dq, dk, dv bf16, dpq, dpk fp32 [n,r])."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    for name, t in (("k", k), ("v", v), ("out", out), ("dout", dout)):
        _check_image(name, t, q.shape)
    n = window * window
    _check_pos("pq", pq, n)
    _check_pos("pk", pk, n)
    r = pq.shape[1]
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, heads, H, W) or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    need = rib_window_attn_bwd_workspace(B, H, W, heads, d, r, window)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dpq = torch.empty((n, r), dtype=torch.float32, device=q.device)
    dpk = torch.empty((n, r), dtype=torch.float32, device=q.device)
    rc = library().rib_window_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), _ptr(out), _ptr(lse),
                                       _ptr(dout), B, H, W, heads, d, r, window, shift, _ptr(dq), _ptr(dk),
                                       _ptr(dv), _ptr(dpq), _ptr(dpk), _ptr(workspace), workspace.numel(),
                                       _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dq, dk, dv, dpq, dpk


def rib_window_attn_bwd_headwise_workspace(pos_head_stride, B, H, W, heads, d, r, window) -> int:
    return int(library().rib_window_attn_bwd_headwise_workspace(pos_head_stride, B, H, W, heads, d, r, window))


def rib_window_attn_fwd_headwise(q, k, v, pq, pk, window, shift=0, stream=None, want_lse=True):
    """Forward pass with one Pq/Pk table per head: pq, pk bf16 [heads, n, r]; returns (out, lse)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    _check_image("k", k, q.shape)
    _check_image("v", v, q.shape)
    n = window * window
    _check_pos_headwise("pq", pq, heads, n)
    _check_pos_headwise("pk", pk, heads, n)
    r = pq.shape[2]
    out = torch.empty_like(q)
    lse = torch.empty((B, heads, H, W), dtype=torch.float32, device=q.device) if want_lse else None
    rc = library().rib_window_attn_fwd_headwise(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), n * r, B, H, W, heads,
                                                d, r, window, shift, _ptr(out), _ptr(lse), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return out, lse


def rib_window_attn_fwd_padded(q, k, v, pq, pk, window, shift=0, stream=None, want_lse=True):
    """Forward pass on a map whose sides need not be multiples of the window (positions of the extended map
    beyond H x W are not tokens); pq, pk are [n, r] or [heads, n, r].  Returns (out, lse)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    _check_image("k", k, q.shape)
    _check_image("v", v, q.shape)
    n = window * window
    headwise = pq.dim() == 3
    if headwise:
        _check_pos_headwise("pq", pq, heads, n)
        _check_pos_headwise("pk", pk, heads, n)
    else:
        _check_pos("pq", pq, n)
        _check_pos("pk", pk, n)
    r = pq.shape[-1]
    out = torch.empty_like(q)
    lse = torch.empty((B, heads, H, W), dtype=torch.float32, device=q.device) if want_lse else None
    rc = library().rib_window_attn_fwd_padded(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), n * r if headwise else 0,
                                              B, H, W, heads, d, r, window, shift, _ptr(out), _ptr(lse), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return out, lse


def rib_window_cycle_fwd(qs, ks, vs, pqs, pks, windows, shifts=None, stream=None, want_lse=True):
    """The cyclic window strategy in one call: layer l attends qs[l], ks[l], vs[l] in windows of side windows[l] with the tables
    pqs[l], pks[l] ([windows[l]^2, r]).  Returns (outs, lses), one tensor per layer."""
    layers = len(windows)
    if not (len(qs) == len(ks) == len(vs) == len(pqs) == len(pks) == layers) or (shifts is not None and len(shifts) != layers):
        raise ValueError("one q, k, v, pq, pk (and shift) per layer")
    _check_image("q", qs[0])
    B, H, W, heads, d = qs[0].shape
    r = pqs[0].shape[1]
    for l in range(layers):
        for name, t in (("q", qs[l]), ("k", ks[l]), ("v", vs[l])):
            _check_image(name, t, qs[0].shape)
        _check_pos("pq", pqs[l], windows[l] * windows[l])
        _check_pos("pk", pks[l], windows[l] * windows[l])
        if pqs[l].shape[1] != r or pks[l].shape[1] != r:
            raise ValueError("every layer uses the same rank")
    outs = [torch.empty_like(qs[0]) for _ in range(layers)]
    lses = [torch.empty((B, heads, H, W), dtype=torch.float32, device=qs[0].device) if want_lse else None for _ in range(layers)]
    arr = lambda ts: (ctypes.c_void_p * layers)(*[_ptr(t) for t in ts])
    ints = lambda xs: (ctypes.c_int * layers)(*[int(x) for x in xs])
    rc = library().rib_window_cycle_fwd(arr(qs), arr(ks), arr(vs), arr(pqs), arr(pks), ints(windows),
                                        ints(shifts) if shifts is not None else None, layers, B, H, W, heads, d, r,
                                        arr(outs), arr(lses) if want_lse else None, _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return outs, lses


def rib_window_cycle_bwd(qs, ks, vs, pqs, pks, outs, lses, douts, windows, shifts=None, workspace=None, stream=None):
    """Backward passes of the layers of rib_window_cycle_fwd.  Returns (dqs, dks, dvs, dpqs, dpks), one tensor per layer."""
    layers = len(windows)
    lists = (qs, ks, vs, pqs, pks, outs, lses, douts)
    if any(len(x) != layers for x in lists) or (shifts is not None and len(shifts) != layers):
        raise ValueError("one q, k, v, pq, pk, out, lse, dout (and shift) per layer")
    _check_image("q", qs[0])
    B, H, W, heads, d = qs[0].shape
    r = pqs[0].shape[1]
    for l in range(layers):
        for name, t in (("q", qs[l]), ("k", ks[l]), ("v", vs[l]), ("out", outs[l]), ("dout", douts[l])):
            _check_image(name, t, qs[0].shape)
        _check_pos("pq", pqs[l], windows[l] * windows[l])
        _check_pos("pk", pks[l], windows[l] * windows[l])
        if lses[l].dtype != torch.float32 or tuple(lses[l].shape) != (B, heads, H, W) or not lses[l].is_contiguous():
            raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    ints = lambda xs: (ctypes.c_int * layers)(*[int(x) for x in xs])
    arr = lambda ts: (ctypes.c_void_p * layers)(*[_ptr(t) for t in ts])
    need = int(library().rib_window_cycle_bwd_workspace(ints(windows), layers, B, H, W, heads, d, r))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=qs[0].device)
    dqs, dks, dvs = ([torch.empty_like(qs[0]) for _ in range(layers)] for _ in range(3))
    dpqs = [torch.empty(tuple(t.shape), dtype=torch.float32, device=t.device) for t in pqs]
    dpks = [torch.empty(tuple(t.shape), dtype=torch.float32, device=t.device) for t in pks]
    rc = library().rib_window_cycle_bwd(arr(qs), arr(ks), arr(vs), arr(pqs), arr(pks), arr(outs), arr(lses), arr(douts), ints(windows),
                                        ints(shifts) if shifts is not None else None, layers, B, H, W, heads, d, r,
                                        arr(dqs), arr(dks), arr(dvs), arr(dpqs), arr(dpks), _ptr(workspace), workspace.numel(),
                                        _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dqs, dks, dvs, dpqs, dpks


def rib_window_attn_bwd_padded(q, k, v, pq, pk, out, lse, dout, window, shift=0, workspace=None, stream=None):
    """Backward pass on a map whose sides need not be multiples of the window; pq, pk [n, r] or [heads, n, r].
    Returns (dq, dk, dv bf16, dpq, dpk fp32 of the shape of pq)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    for name, t in (("k", k), ("v", v), ("out", out), ("dout", dout)):
        _check_image(name, t, q.shape)
    n = window * window
    headwise = pq.dim() == 3
    if headwise:
        _check_pos_headwise("pq", pq, heads, n)
        _check_pos_headwise("pk", pk, heads, n)
    else:
        _check_pos("pq", pq, n)
        _check_pos("pk", pk, n)
    r = pq.shape[-1]
    stride = n * r if headwise else 0
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, heads, H, W) or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    need = int(library().rib_window_attn_bwd_padded_workspace(stride, B, H, W, heads, d, r, window))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dpq = torch.empty(tuple(pq.shape), dtype=torch.float32, device=q.device)
    dpk = torch.empty(tuple(pk.shape), dtype=torch.float32, device=q.device)
    rc = library().rib_window_attn_bwd_padded(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), stride, _ptr(out), _ptr(lse),
                                              _ptr(dout), B, H, W, heads, d, r, window, shift, _ptr(dq), _ptr(dk), _ptr(dv),
                                              _ptr(dpq), _ptr(dpk), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dq, dk, dv, dpq, dpk


def rib_window_attn_fwd_masked(q, k, v, pq, pk, window, shift=0, stream=None, want_lse=True):
    """Forward pass with shifted windows whose wrapped parts do not attend to each other (H, W multiples of the
    window); pq, pk are [n, r] or [heads, n, r].  Returns (out, lse)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    _check_image("k", k, q.shape)
    _check_image("v", v, q.shape)
    n = window * window
    headwise = pq.dim() == 3
    if headwise:
        _check_pos_headwise("pq", pq, heads, n)
        _check_pos_headwise("pk", pk, heads, n)
    else:
        _check_pos("pq", pq, n)
        _check_pos("pk", pk, n)
    r = pq.shape[-1]
    out = torch.empty_like(q)
    lse = torch.empty((B, heads, H, W), dtype=torch.float32, device=q.device) if want_lse else None
    rc = library().rib_window_attn_fwd_masked(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), n * r if headwise else 0,
                                              B, H, W, heads, d, r, window, shift, _ptr(out), _ptr(lse), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return out, lse


def rib_window_attn_bwd_masked(q, k, v, pq, pk, out, lse, dout, window, shift=0, workspace=None, stream=None):
    """Backward pass of rib_window_attn_fwd_masked; pq, pk [n, r] or [heads, n, r].
    Returns (dq, dk, dv bf16, dpq, dpk fp32 of the shape of pq)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    for name, t in (("k", k), ("v", v), ("out", out), ("dout", dout)):
        _check_image(name, t, q.shape)
    n = window * window
    headwise = pq.dim() == 3
    if headwise:
        _check_pos_headwise("pq", pq, heads, n)
        _check_pos_headwise("pk", pk, heads, n)
    else:
        _check_pos("pq", pq, n)
        _check_pos("pk", pk, n)
    r = pq.shape[-1]
    stride = n * r if headwise else 0
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, heads, H, W) or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    need = int(library().rib_window_attn_bwd_padded_workspace(stride, B, H, W, heads, d, r, window))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dpq = torch.empty(tuple(pq.shape), dtype=torch.float32, device=q.device)
    dpk = torch.empty(tuple(pk.shape), dtype=torch.float32, device=q.device)
    rc = library().rib_window_attn_bwd_masked(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), stride, _ptr(out), _ptr(lse),
                                              _ptr(dout), B, H, W, heads, d, r, window, shift, _ptr(dq), _ptr(dk), _ptr(dv),
                                              _ptr(dpq), _ptr(dpk), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dq, dk, dv, dpq, dpk


def rib_cla_gate(x, w_dw, b_dw, w_pw, b_pw, stream=None):
    """CLA gate (Eq. 8): x bf16 [B,H,W,D]; w_dw fp32 [D,3,3]; b_dw fp32 [D]; w_pw fp32 [D,D] (out, in); b_pw fp32 [D].
    Returns the gate, bf16 [B,H,W,D]."""
    if x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous() or x.dim() != 4:
        raise ValueError("x must be a contiguous CUDA bfloat16 tensor [B,H,W,D]")
    B, H, W, D = x.shape
    for name, t, shape in (("w_dw", w_dw, (D, 3, 3)), ("b_dw", b_dw, (D,)), ("w_pw", w_pw, (D, D)), ("b_pw", b_pw, (D,))):
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shape:
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor of shape {shape}")
    gate = torch.empty_like(x)
    rc = library().rib_cla_gate(_ptr(x), _ptr(w_dw), _ptr(b_dw), _ptr(w_pw), _ptr(b_pw), B, H, W, D, _ptr(gate), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return gate


def _check_bf16_like(name, t, like=None):
    if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA bfloat16 tensor")
    if like is not None and t.numel() != like.numel():
        raise ValueError(f"{name} must have as many elements as out")


def rib_cla_product(out, gate, stream=None):
    """Eq. 9 on its own: out [B,H,W,heads,d] (or [B,H,W,D]) times gate [B,H,W,D], both bf16; returns out's shape."""
    _check_bf16_like("out", out)
    _check_bf16_like("gate", gate, out)
    res = torch.empty_like(out)
    rc = library().rib_cla_product(_ptr(out), _ptr(gate), out.numel(), _ptr(res), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return res


def rib_cla_product_bwd(out, gate, dout_gated, stream=None):
    """Chain rule of Eq. 9: returns (dout in out's shape, dgate in gate's shape), bf16."""
    _check_bf16_like("out", out)
    _check_bf16_like("gate", gate, out)
    _check_bf16_like("dout_gated", dout_gated, out)
    dout = torch.empty_like(out)
    dgate = torch.empty_like(gate)
    rc = library().rib_cla_product_bwd(_ptr(out), _ptr(gate), _ptr(dout_gated), out.numel(), _ptr(dout), _ptr(dgate),
                                       _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dout, dgate


def rib_cla_gate_bwd(x, w_dw, b_dw, w_pw, b_pw, dgate, workspace=None, stream=None):
    """Chain rule of Eq. 8: x, dgate bf16 [B,H,W,D]; weights as for rib_cla_gate.
    Returns (dx bf16 [B,H,W,D], dw_dw [D,3,3], db_dw [D], dw_pw [D,D], db_pw [D] fp32)."""
    if x.dtype != torch.bfloat16 or not x.is_cuda or not x.is_contiguous() or x.dim() != 4:
        raise ValueError("x must be a contiguous CUDA bfloat16 tensor [B,H,W,D]")
    B, H, W, D = x.shape
    if dgate.dtype != torch.bfloat16 or not dgate.is_cuda or not dgate.is_contiguous() or dgate.shape != x.shape:
        raise ValueError("dgate must be a contiguous CUDA bfloat16 tensor of x's shape")
    for name, t, shape in (("w_dw", w_dw, (D, 3, 3)), ("b_dw", b_dw, (D,)), ("w_pw", w_pw, (D, D)), ("b_pw", b_pw, (D,))):
        if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shape:
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor of shape {shape}")
    need = library().rib_cla_gate_bwd_workspace(B, H, W, D)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=x.device)
    dx = torch.empty_like(x)
    grads = [torch.empty_like(t) for t in (w_dw, b_dw, w_pw, b_pw)]
    rc = library().rib_cla_gate_bwd(_ptr(x), _ptr(w_dw), _ptr(b_dw), _ptr(w_pw), _ptr(b_pw), _ptr(dgate), B, H, W, D, _ptr(dx),
                                    *[_ptr(g) for g in grads], _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return (dx, *grads)


def rib_window_attn_fwd_gated(q, k, v, pq, pk, gate, window, shift=0, stream=None, want_lse=True):
    """Forward pass whose output is multiplied by the CLA gate (Eq. 9); gate bf16 [B,H,W,heads*d]; pq, pk [n,r] or
    [heads,n,r].  Returns (out, lse)."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    _check_image("k", k, q.shape)
    _check_image("v", v, q.shape)
    if gate.dtype != torch.bfloat16 or not gate.is_cuda or not gate.is_contiguous() or tuple(gate.shape) != (B, H, W, heads * d):
        raise ValueError("gate must be a contiguous CUDA bfloat16 tensor [B,H,W,heads*d]")
    n = window * window
    headwise = pq.dim() == 3
    if headwise:
        _check_pos_headwise("pq", pq, heads, n)
        _check_pos_headwise("pk", pk, heads, n)
    else:
        _check_pos("pq", pq, n)
        _check_pos("pk", pk, n)
    r = pq.shape[-1]
    out = torch.empty_like(q)
    lse = torch.empty((B, heads, H, W), dtype=torch.float32, device=q.device) if want_lse else None
    rc = library().rib_window_attn_fwd_gated(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), n * r if headwise else 0, _ptr(gate),
                                             B, H, W, heads, d, r, window, shift, _ptr(out), _ptr(lse), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return out, lse


def rib_window_attn_bwd_headwise(q, k, v, pq, pk, out, lse, dout, window, shift=0, workspace=None, stream=None):
    """Backward pass with one Pq/Pk table per head; returns (dq, dk, dv bf16, dpq, dpk fp32 [heads, n, r])."""
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    for name, t in (("k", k), ("v", v), ("out", out), ("dout", dout)):
        _check_image(name, t, q.shape)
    n = window * window
    _check_pos_headwise("pq", pq, heads, n)
    _check_pos_headwise("pk", pk, heads, n)
    r = pq.shape[2]
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, heads, H, W) or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    need = rib_window_attn_bwd_headwise_workspace(n * r, B, H, W, heads, d, r, window)
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dpq = torch.empty((heads, n, r), dtype=torch.float32, device=q.device)
    dpk = torch.empty((heads, n, r), dtype=torch.float32, device=q.device)
    rc = library().rib_window_attn_bwd_headwise(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), n * r, _ptr(out),
                                                _ptr(lse), _ptr(dout), B, H, W, heads, d, r, window, shift, _ptr(dq),
                                                _ptr(dk), _ptr(dv), _ptr(dpq), _ptr(dpk), _ptr(workspace),
                                                workspace.numel(), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return dq, dk, dv, dpq, dpk


def rib_window_attn_bwd_noalloc(q, k, v, pq, pk, out, lse, dout, dq, dk, dv, dpq, dpk, window, shift=0, stream=None):
    """Backward pass into caller-provided result tensors, using the library's built-in scratch.

    For callers that must not allocate on the device: nothing is allocated here either, so every
    result tensor is passed in.  Shapes that need more than ``RIB_NOALLOC_SCRATCH_BYTES`` of
    scratch raise ``RibError`` (RIB_ERR_TOO_LARGE).  Calls on one device share the scratch: keep
    them on one stream.
    """
    _check_image("q", q)
    B, H, W, heads, d = q.shape
    for name, t in (("k", k), ("v", v), ("out", out), ("dout", dout), ("dq", dq), ("dk", dk), ("dv", dv)):
        _check_image(name, t, q.shape)
    n = window * window
    _check_pos("pq", pq, n)
    _check_pos("pk", pk, n)
    r = pq.shape[1]
    for name, t in (("dpq", dpq), ("dpk", dpk)):
        if t.dtype != torch.float32 or tuple(t.shape) != (n, r) or not t.is_contiguous() or not t.is_cuda:
            raise ValueError(f"{name} must be a contiguous CUDA fp32 tensor [n, r]")
    if lse.dtype != torch.float32 or tuple(lse.shape) != (B, heads, H, W) or not lse.is_contiguous():
        raise ValueError("lse must be a contiguous fp32 tensor [B,heads,H,W]")
    rc = library().rib_window_attn_bwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(pq), _ptr(pk), _ptr(out), _ptr(lse),
                                               _ptr(dout), B, H, W, heads, d, r, window, shift, _ptr(dq), _ptr(dk),
                                               _ptr(dv), _ptr(dpq), _ptr(dpk), _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)


def _check_f32(name, t, shape):
    if t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name} must be a contiguous CUDA float32 tensor of shape {tuple(shape)}")


def rib_generate_features(w_h, b_h, w_pq, w_pk, window, stream=None):
    """Pq, Pk (bf16 [window^2, r]) from the generator weights (Eq. 1-3); L is read off w_h's height 2 + 4 L."""
    rows, dh = w_h.shape
    L, r = (rows - 2) // 4, w_pq.shape[1]
    _check_f32("w_h", w_h, (2 + 4 * L, dh)); _check_f32("b_h", b_h, (dh,))
    _check_f32("w_pq", w_pq, (dh, r)); _check_f32("w_pk", w_pk, (dh, r))
    pq = torch.empty((window * window, r), dtype=torch.bfloat16, device=w_h.device)
    pk = torch.empty_like(pq)
    rc = library().rib_generate_features(_ptr(w_h), _ptr(b_h), _ptr(w_pq), _ptr(w_pk), window, L, dh, r, _ptr(pq), _ptr(pk),
                                         _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return pq, pk


def rib_generate_features_bwd(w_h, b_h, w_pq, w_pk, dpq, dpk, window, stream=None):
    """Gradients (dw_h, db_h, dw_pq, dw_pk) of the generator weights given dpq, dpk fp32 [window^2, r]."""
    rows, dh = w_h.shape
    L, r = (rows - 2) // 4, w_pq.shape[1]
    _check_f32("w_h", w_h, (2 + 4 * L, dh)); _check_f32("b_h", b_h, (dh,))
    _check_f32("w_pq", w_pq, (dh, r)); _check_f32("w_pk", w_pk, (dh, r))
    _check_f32("dpq", dpq, (window * window, r)); _check_f32("dpk", dpk, (window * window, r))
    outs = tuple(torch.empty_like(t) for t in (w_h, b_h, w_pq, w_pk))
    rc = library().rib_generate_features_bwd(_ptr(w_h), _ptr(b_h), _ptr(w_pq), _ptr(w_pk), _ptr(dpq), _ptr(dpk), window, L, dh, r,
                                             *[_ptr(t) for t in outs], _stream_ptr(stream))
    if rc != RIB_OK:
        raise RibError(rc)
    return outs

"""Thin Python binding of the C ABI declared in include/terra.h.

Argument marshalling only: tensors must already live on the GPU; every step of the path
(route, gather, attention, scatter) runs in the library's kernels.  There is no CPU
fallback: if the shared library is missing or no CUDA device is present, calls raise.
PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .build import LIB_PATH

TERRA_OK = 0
EXPORTS = ("terra_route_sizes", "terra_window_route", "terra_swin_workspace_bytes", "terra_swin_attn_fwd",
           "terra_swin_attn_fwd_noalloc", "terra_swin_attn_bwd", "terra_swin_check", "terra_strerror", "terra_last_cuda_error",
           "terra_launch_count", "terra_selftest_bounded_wait", "terra_profile_enable", "terra_profile_count", "terra_profile_get",
           "terra_fixed_assignment_padding", "terra_ragged_window_range", "terra_swin_attn_fwd_packed", "terra_swin_attn_bwd_packed",
           "terra_pad_grid", "terra_crop_grid")


class TerraError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"terra status {status}: {text}")
        self.status = status


class terra_swin_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "W", "heads", "head_dim", "window", "shift_h", "shift_w", "periodic_h", "periodic_w")] + \
               [("scale", ctypes.c_float), ("dtype", ctypes.c_int32)]

TERRA_DTYPE_BF16, TERRA_DTYPE_F16 = 0, 1


_lib = None


def load_library(path: str | None = None) -> ctypes.CDLL:
    """dlopen the CUDA library.  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or os.environ.get("TERRA_LIB_PATH") or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2608_15211_b200.build` "
                                "(the library has no CPU fallback)")
    lib = ctypes.CDLL(p)
    vp, i32p, i64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)
    dp = ctypes.POINTER(terra_swin_desc)
    lib.terra_route_sizes.argtypes = [dp, i64p, i32p, i32p]
    lib.terra_window_route.argtypes = [dp, vp, vp, vp, vp, vp, vp]
    lib.terra_swin_workspace_bytes.argtypes = [dp, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t)]
    lib.terra_swin_attn_fwd.argtypes = [dp] + [vp] * 6 + [vp, ctypes.c_size_t, vp]
    lib.terra_swin_attn_bwd.argtypes = [dp] + [vp] * 11 + [vp, ctypes.c_size_t, vp]
    lib.terra_swin_attn_fwd_noalloc.argtypes = [dp] + [vp] * 6 + [vp]
    lib.terra_swin_attn_fwd_packed.argtypes = [dp] + [vp] * 4 + [vp, ctypes.c_size_t, vp]
    lib.terra_swin_attn_bwd_packed.argtypes = [dp] + [vp] * 7 + [vp, ctypes.c_size_t, vp]
    for n in ("terra_route_sizes", "terra_window_route", "terra_swin_workspace_bytes", "terra_swin_attn_fwd",
              "terra_swin_attn_fwd_noalloc", "terra_swin_attn_bwd", "terra_swin_attn_fwd_packed", "terra_swin_attn_bwd_packed"):
        getattr(lib, n).restype = ctypes.c_int
    lib.terra_swin_check.argtypes = [vp]
    lib.terra_swin_check.restype = ctypes.c_int
    lib.terra_strerror.argtypes = [ctypes.c_int]
    lib.terra_strerror.restype = ctypes.c_char_p
    lib.terra_last_cuda_error.restype = ctypes.c_char_p
    lib.terra_launch_count.restype = ctypes.c_int64
    lib.terra_selftest_bounded_wait.argtypes = [ctypes.c_longlong, vp]
    lib.terra_selftest_bounded_wait.restype = ctypes.c_int
    lib.terra_profile_enable.argtypes = [ctypes.c_int]
    lib.terra_profile_count.restype = ctypes.c_int
    lib.terra_profile_get.argtypes = [ctypes.c_int, ctypes.c_char_p, ctypes.c_int, ctypes.POINTER(ctypes.c_float)]
    lib.terra_fixed_assignment_padding.argtypes = [ctypes.c_int64, ctypes.c_int64] + [ctypes.c_int32] * 5 + [i64p, i64p]
    lib.terra_fixed_assignment_padding.restype = ctypes.c_int
    lib.terra_ragged_window_range.argtypes = [ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, i64p, i64p]
    lib.terra_ragged_window_range.restype = ctypes.c_int
    for n in ("terra_pad_grid", "terra_crop_grid"):
        getattr(lib, n).argtypes = [vp, vp] + [ctypes.c_int32] * 5 + [ctypes.c_int64, vp]
        getattr(lib, n).restype = ctypes.c_int
    if path is None:
        _lib = lib
    return lib


def make_desc(cfg, scale: float = 0.0, dtype=torch.bfloat16) -> terra_swin_desc:
    """Descriptor from any object with B, H, W, heads, head_dim, window, shift_*, periodic_* fields; `dtype` is the
    element type of the activations (torch.bfloat16 or torch.float16)."""
    if dtype not in (torch.bfloat16, torch.float16):
        raise ValueError("terra: activations are bf16 or fp16")
    return terra_swin_desc(cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim, cfg.window, cfg.shift_h, cfg.shift_w,
                           cfg.periodic_h, cfg.periodic_w, float(scale),
                           TERRA_DTYPE_F16 if dtype == torch.float16 else TERRA_DTYPE_BF16)


def _act_dtype(desc):
    return torch.float16 if desc.dtype == TERRA_DTYPE_F16 else torch.bfloat16


def _check(status: int) -> None:
    if status != TERRA_OK:
        lib = load_library()
        text = lib.terra_strerror(status).decode()
        extra = lib.terra_last_cuda_error().decode()
        raise TerraError(status, text + (f" [{extra}]" if extra and status == 5 else ""))


def _ptr(t) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda:
        raise ValueError("terra: tensors must be CUDA tensors (the library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError("terra: tensors must be contiguous")
    if t.device.index != torch.cuda.current_device():
        # the library launches on the current device (its stream, SM count and built-in scratch are that device's)
        raise ValueError(f"terra: tensor lives on {t.device} but the current device is cuda:{torch.cuda.current_device()}; "
                         "make the tensors' device current (torch.cuda.device(...)) around the call")
    return ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def terra_swin_check() -> None:
    """Waits for the current stream; raises TerraError(6) if a kernel gave up on a bounded wait."""
    _check(load_library().terra_swin_check(_stream()))


def profile_enable(on: bool) -> None:
    load_library().terra_profile_enable(int(on))


def profile_read() -> list:
    """[(kernel name, milliseconds)] of every launch recorded since profile_enable(True)."""
    lib = load_library()
    out = []
    name = ctypes.create_string_buffer(64)
    ms = ctypes.c_float()
    for i in range(lib.terra_profile_count()):
        if lib.terra_profile_get(i, name, 64, ctypes.byref(ms)) == TERRA_OK:
            out.append((name.value.decode(), float(ms.value)))
    return out


def selftest_bounded_wait(limit_cycles: int = 1_000_000) -> None:
    """Launches the kernel whose bounded wait must expire (see include/terra.h); check with terra_swin_check()."""
    _check(load_library().terra_selftest_bounded_wait(int(limit_cycles), _stream()))


def launch_count() -> int:
    return int(load_library().terra_launch_count())


def terra_fixed_assignment_padding(H: int, W: int, p: int, alpha: int, w: int, m: int = 1, n: int = 1):
    """(H_hat, W_hat) of Eq. 3: the input field padded so that an m x n WP mesh holds equal window counts."""
    hh, ww = ctypes.c_int64(), ctypes.c_int64()
    _check(load_library().terra_fixed_assignment_padding(H, W, p, alpha, w, m, n, ctypes.byref(hh), ctypes.byref(ww)))
    return hh.value, ww.value


def terra_ragged_window_range(M: int, ranks: int, r: int):
    """[L, R) of Eq. 4: the row-major window range that rank r of `ranks` owns."""
    lo, hi = ctypes.c_int64(), ctypes.c_int64()
    _check(load_library().terra_ragged_window_range(M, ranks, r, ctypes.byref(lo), ctypes.byref(hi)))
    return lo.value, hi.value


def terra_route_sizes(desc: terra_swin_desc):
    nt, nw, mx = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().terra_route_sizes(ctypes.byref(desc), ctypes.byref(nt), ctypes.byref(nw), ctypes.byref(mx)))
    return nt.value, nw.value, mx.value


def terra_window_route(desc: terra_swin_desc, device="cuda") -> dict:
    """Allocates the five int32 route arrays on `device` and fills them."""
    nt, nw, _ = terra_route_sizes(desc)
    out = {k: torch.empty(nt, dtype=torch.int32, device=device) for k in ("perm", "inv_perm", "pos", "label")}
    out["win_offsets"] = torch.empty(nw + 1, dtype=torch.int32, device=device)
    _check(load_library().terra_window_route(ctypes.byref(desc), _ptr(out["perm"]), _ptr(out["inv_perm"]),
                                             _ptr(out["win_offsets"]), _ptr(out["pos"]), _ptr(out["label"]), _stream()))
    return out


def terra_swin_workspace_bytes(desc: terra_swin_desc, backward: bool) -> int:
    n = ctypes.c_size_t()
    _check(load_library().terra_swin_workspace_bytes(ctypes.byref(desc), int(backward), ctypes.byref(n)))
    return int(n.value)


def _expect(t, dtype, numel, name):
    if t.dtype != dtype or t.numel() != numel:
        raise ValueError(f"terra: {name} must be {dtype} with {numel} elements, got {t.dtype} x {t.numel()}")


def terra_swin_attn_fwd(desc, q, k, v, bias_table, o=None, lse=None, workspace=None):
    """Forward.  q, k, v bf16 [B, H, W, heads, head_dim]; bias_table fp32 [(2w-1)^2, heads].
    Returns (o bf16 like q, lse fp32 [B, H, W, heads]); pass o / lse / workspace to reuse buffers."""
    n = desc.B * desc.H * desc.W * desc.heads
    for name, t in (("q", q), ("k", k), ("v", v)):
        _expect(t, _act_dtype(desc), n * desc.head_dim, name)
    _expect(bias_table, torch.float32, (2 * desc.window - 1) ** 2 * desc.heads, "bias_table")
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((desc.B, desc.H, desc.W, desc.heads), dtype=torch.float32, device=q.device)
    _expect(o, _act_dtype(desc), n * desc.head_dim, "o")
    _expect(lse, torch.float32, n, "lse")
    if workspace is None:
        need = terra_swin_workspace_bytes(desc, False)
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device) if need else None
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load_library().terra_swin_attn_fwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(bias_table),
                                              _ptr(o), _ptr(lse), _ptr(workspace), ws_bytes, _stream()))
    return o, lse


def terra_swin_attn_fwd_noalloc(desc, q, k, v, bias_table, o, lse):
    """Forward into caller-provided o / lse with no workspace: the library's built-in scratch is used and
    nothing is allocated, by this binding or by the library (see include/terra.h for who needs this and
    for its limits: at most TERRA_NOALLOC_MAX_HEADS heads, calls on one device must not overlap)."""
    n = desc.B * desc.H * desc.W * desc.heads
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o)):
        _expect(t, _act_dtype(desc), n * desc.head_dim, name)
    _expect(bias_table, torch.float32, (2 * desc.window - 1) ** 2 * desc.heads, "bias_table")
    _expect(lse, torch.float32, n, "lse")
    _check(load_library().terra_swin_attn_fwd_noalloc(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(bias_table),
                                                      _ptr(o), _ptr(lse), _stream()))
    return o, lse


def terra_swin_attn_bwd(desc, q, k, v, bias_table, o, lse, d_o, dq=None, dk=None, dv=None, dbias=None,
                        workspace=None):
    """Backward.  Returns (dq, dk, dv bf16 like q, dbias fp32 like bias_table)."""
    n = desc.B * desc.H * desc.W * desc.heads
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o), ("d_o", d_o)):
        _expect(t, _act_dtype(desc), n * desc.head_dim, name)
    _expect(lse, torch.float32, n, "lse")
    _expect(bias_table, torch.float32, (2 * desc.window - 1) ** 2 * desc.heads, "bias_table")
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    dbias = torch.empty_like(bias_table) if dbias is None else dbias
    for name, t in (("dq", dq), ("dk", dk), ("dv", dv)):
        _expect(t, _act_dtype(desc), n * desc.head_dim, name)
    _expect(dbias, torch.float32, bias_table.numel(), "dbias")
    if workspace is None:
        workspace = torch.empty(terra_swin_workspace_bytes(desc, True), dtype=torch.uint8, device=q.device)
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(load_library().terra_swin_attn_bwd(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _ptr(bias_table),
                                              _ptr(o), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv),
                                              _ptr(dbias), _ptr(workspace), ws_bytes, _stream()))
    return dq, dk, dv, dbias


def terra_swin_attn_fwd_packed(desc, qkv, bias_table, o=None, lse=None, workspace=None):
    """Forward on the packed projection output.  qkv bf16 [B, H, W, 3, heads, head_dim] (q, k, v in that order);
    returns (o bf16 [B, H, W, heads, head_dim], lse fp32 [B, H, W, heads])."""
    n = desc.B * desc.H * desc.W * desc.heads
    _expect(qkv, _act_dtype(desc), 3 * n * desc.head_dim, "qkv")
    _expect(bias_table, torch.float32, (2 * desc.window - 1) ** 2 * desc.heads, "bias_table")
    if o is None:
        o = torch.empty((desc.B, desc.H, desc.W, desc.heads, desc.head_dim), dtype=_act_dtype(desc), device=qkv.device)
    if lse is None:
        lse = torch.empty((desc.B, desc.H, desc.W, desc.heads), dtype=torch.float32, device=qkv.device)
    _expect(o, _act_dtype(desc), n * desc.head_dim, "o")
    _expect(lse, torch.float32, n, "lse")
    if workspace is None:
        need = terra_swin_workspace_bytes(desc, False)
        workspace = torch.empty(need, dtype=torch.uint8, device=qkv.device) if need else None
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(load_library().terra_swin_attn_fwd_packed(ctypes.byref(desc), _ptr(qkv), _ptr(bias_table), _ptr(o), _ptr(lse),
                                                     _ptr(workspace), ws_bytes, _stream()))
    return o, lse


def terra_swin_attn_bwd_packed(desc, qkv, bias_table, o, lse, d_o, dqkv=None, dbias=None, workspace=None):
    """Backward on the packed layout.  Returns (dqkv bf16 like qkv, dbias fp32 like bias_table)."""
    n = desc.B * desc.H * desc.W * desc.heads
    _expect(qkv, _act_dtype(desc), 3 * n * desc.head_dim, "qkv")
    for name, t in (("o", o), ("d_o", d_o)):
        _expect(t, _act_dtype(desc), n * desc.head_dim, name)
    _expect(lse, torch.float32, n, "lse")
    _expect(bias_table, torch.float32, (2 * desc.window - 1) ** 2 * desc.heads, "bias_table")
    dqkv = torch.empty_like(qkv) if dqkv is None else dqkv
    dbias = torch.empty_like(bias_table) if dbias is None else dbias
    _expect(dqkv, _act_dtype(desc), 3 * n * desc.head_dim, "dqkv")
    _expect(dbias, torch.float32, bias_table.numel(), "dbias")
    if workspace is None:
        workspace = torch.empty(terra_swin_workspace_bytes(desc, True), dtype=torch.uint8, device=qkv.device)
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(load_library().terra_swin_attn_bwd_packed(ctypes.byref(desc), _ptr(qkv), _ptr(bias_table), _ptr(o), _ptr(lse),
                                                     _ptr(d_o), _ptr(dqkv), _ptr(dbias), _ptr(workspace), ws_bytes, _stream()))
    return dqkv, dbias


def padded_extent(extent: int, window: int) -> int:
    """The extent rounded up to complete windows."""
    return -(-extent // window) * window


def terra_pad_grid(x, H_pad: int, W_pad: int):
    """x [B, H, W, ...] -> zero-padded [B, H_pad, W_pad, ...] (complete-window mode, see include/terra.h)."""
    B, H, W = x.shape[:3]
    token_bytes = x[0, 0, 0].numel() * x.element_size()
    y = torch.empty((B, H_pad, W_pad) + tuple(x.shape[3:]), dtype=x.dtype, device=x.device)
    _check(load_library().terra_pad_grid(_ptr(x), _ptr(y), B, H, W, H_pad, W_pad, token_bytes, _stream()))
    return y


def terra_crop_grid(y, H: int, W: int):
    """y [B, H_pad, W_pad, ...] -> its top-left [B, H, W, ...] corner as a dense tensor."""
    B, H_pad, W_pad = y.shape[:3]
    token_bytes = y[0, 0, 0].numel() * y.element_size()
    x = torch.empty((B, H, W) + tuple(y.shape[3:]), dtype=y.dtype, device=y.device)
    _check(load_library().terra_crop_grid(_ptr(y), _ptr(x), B, H, W, H_pad, W_pad, token_bytes, _stream()))
    return x

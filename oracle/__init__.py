"""Python face of the CPU oracle (test infrastructure, not the product).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It compiles ``swin_oracle.c`` with gcc on first use and calls it
through ctypes.  Nothing here touches the CUDA library, and the CUDA package never
imports this one.

All results come back in the window-major layout of the token route (selected
windows in order, slots inside a window row-major over the window's extent);
``to_grid`` puts a full result back on the [B, H, W, ...] grid.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swin_oracle.c")
_LIB = os.path.join(_HERE, "libswin_oracle.so")
_lock = threading.Lock()
_lib = None


class _Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "W", "heads", "head_dim", "window", "shift_h", "shift_w",
                 "periodic_h", "periodic_w")] + [("scale", ctypes.c_double)]


def build(force: bool = False) -> str:
    """Compile the oracle's C file into a shared library beside it."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_num_threads.restype = ctypes.c_int
        for name in ("oracle_route_sizes", "oracle_window_route", "oracle_attn_fwd", "oracle_attn_bwd"):
            getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _desc(cfg, scale: float = 0.0) -> _Desc:
    return _Desc(cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim, cfg.window, cfg.shift_h, cfg.shift_w,
                 cfg.periodic_h, cfg.periodic_w, float(scale))


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def route_sizes(cfg):
    nt, nw, mx = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32()
    rc = _load().oracle_route_sizes(ctypes.byref(_desc(cfg)), ctypes.byref(nt), ctypes.byref(nw), ctypes.byref(mx))
    if rc:
        raise ValueError(f"oracle_route_sizes failed ({rc})")
    return nt.value, nw.value, mx.value


def window_route(cfg) -> dict:
    """int32 arrays perm, inv_perm, win_offsets, pos, label (per sample)."""
    nt, nw, _ = route_sizes(cfg)
    out = {k: np.empty(nt, dtype=np.int32) for k in ("perm", "inv_perm", "pos", "label")}
    out["win_offsets"] = np.empty(nw + 1, dtype=np.int32)
    rc = _load().oracle_window_route(ctypes.byref(_desc(cfg)), _ptr(out["perm"]), _ptr(out["inv_perm"]),
                                     _ptr(out["win_offsets"]), _ptr(out["pos"]), _ptr(out["label"]))
    if rc:
        raise ValueError(f"oracle_window_route failed ({rc})")
    return out


def _as_input(x):
    """torch bf16 tensor / numpy uint16 (bf16 bits) / numpy float64 -> (kind, contiguous numpy array)."""
    try:
        import torch
        if isinstance(x, torch.Tensor):
            if x.dtype == torch.bfloat16:
                return 0, x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
            return 1, x.detach().cpu().to(torch.float64).contiguous().numpy()
    except ImportError:  # pragma: no cover
        pass
    a = np.ascontiguousarray(x)
    if a.dtype == np.uint16:
        return 0, a
    return 1, np.ascontiguousarray(a, dtype=np.float64)


def _inputs(cfg, tensors):
    kinds, arrs = zip(*[_as_input(t) for t in tensors])
    if len(set(kinds)) != 1:
        raise ValueError("all activations must share one dtype (bf16 or float64)")
    n = cfg.tokens * cfg.heads * cfg.head_dim
    for a in arrs:
        if a.size != n:
            raise ValueError("activation has the wrong number of elements for this configuration")
    return kinds[0], arrs


def _selection(cfg, sel):
    _, nw, _ = route_sizes(cfg)
    offs = window_route(cfg)["win_offsets"].astype(np.int64)
    sizes = np.diff(offs)
    if sel is None:
        ids = np.arange(cfg.B * nw, dtype=np.int64)
    else:
        ids = np.ascontiguousarray(sel, dtype=np.int64)
    total = int(sizes[ids % nw].sum())
    return ids, total


def attn_fwd(cfg, q, k, v, bias, sel=None, scale: float = 0.0):
    """Forward over the selected (batch * n_windows + window) ids (all when None).

    Returns (o [S, heads, head_dim], lse [S, heads]) as float64, window-major."""
    kind, (qa, ka, va) = _inputs(cfg, (q, k, v))
    ba = np.ascontiguousarray(np.asarray(bias, dtype=np.float64))
    ids, total = _selection(cfg, sel)
    o = np.empty((total, cfg.heads, cfg.head_dim), dtype=np.float64)
    lse = np.empty((total, cfg.heads), dtype=np.float64)
    rc = _load().oracle_attn_fwd(ctypes.byref(_desc(cfg, scale)), ctypes.c_int(kind), _ptr(qa), _ptr(ka), _ptr(va),
                                 _ptr(ba), ctypes.c_int64(len(ids)), _ptr(ids), _ptr(o), _ptr(lse))
    if rc:
        raise ValueError(f"oracle_attn_fwd failed ({rc})")
    return o, lse


def attn_bwd(cfg, q, k, v, d_o, bias, sel=None, scale: float = 0.0):
    """Backward over the selected windows.  Returns dq, dk, dv [S, heads, head_dim] (window-major)
    and dbias [(2w-1)^2, heads] summed over the selection, float64."""
    kind, (qa, ka, va, ga) = _inputs(cfg, (q, k, v, d_o))
    ba = np.ascontiguousarray(np.asarray(bias, dtype=np.float64))
    ids, total = _selection(cfg, sel)
    dq = np.empty((total, cfg.heads, cfg.head_dim), dtype=np.float64)
    dk = np.empty_like(dq)
    dv = np.empty_like(dq)
    dbias = np.empty((cfg.bias_rows, cfg.heads), dtype=np.float64)
    rc = _load().oracle_attn_bwd(ctypes.byref(_desc(cfg, scale)), ctypes.c_int(kind), _ptr(qa), _ptr(ka), _ptr(va),
                                 _ptr(ga), _ptr(ba), ctypes.c_int64(len(ids)), _ptr(ids),
                                 _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbias))
    if rc:
        raise ValueError(f"oracle_attn_bwd failed ({rc})")
    return dq, dk, dv, dbias


def selection_tokens(cfg, sel=None):
    """Flat grid index (b * H * W + u * W + v) of every output slot of a selection, in output order."""
    r = window_route(cfg)
    nw = len(r["win_offsets"]) - 1
    ids = np.arange(cfg.B * nw, dtype=np.int64) if sel is None else np.asarray(sel, dtype=np.int64)
    parts = []
    for i in ids:
        b, g = divmod(int(i), nw)
        lo, hi = r["win_offsets"][g], r["win_offsets"][g + 1]
        parts.append(b * cfg.H * cfg.W + r["perm"][lo:hi].astype(np.int64))
    return np.concatenate(parts) if parts else np.empty(0, dtype=np.int64)


def to_grid(cfg, x_window_major):
    """Inverse route of a full (sel=None) window-major result back onto the [B, H, W, ...] grid."""
    tok = selection_tokens(cfg, None)
    out = np.empty_like(x_window_major)
    out[tok] = x_window_major
    return out.reshape((cfg.B, cfg.H, cfg.W) + x_window_major.shape[1:])

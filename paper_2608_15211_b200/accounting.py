"""Algorithmic work of one shifted-window attention step (used by the benchmark's roofline figures).

FLOP convention ("strict"): per allowed (query, key) pair per head 4*d FLOP forward (QK^T and PV) and
8*d FLOP backward (dP, dV, dQ, dK); masked pairs, padded tile slots and the backward's recomputation
of S are not counted.  The FlashAttention convention (10*d backward) is reported beside it.
Byte convention: per token per head the forward reads Q, K, V and writes O (4 * 2d bytes) plus one
fp32 LSE; the backward reads Q, K, V, dO and writes dQ, dK, dV (7 * 2d bytes) plus one fp32 LSE read.
"""
from __future__ import annotations


def _axis_groups(L: int, w: int, s: int, periodic: bool):
    """Per window index along one axis: sizes of the groups that may attend to each other."""
    s %= L
    out = []
    for lo in range(0, L, w):
        hi = min(L, lo + w)
        if periodic or s == 0:
            out.append([hi - lo])
        else:
            # rolled coordinates >= L - s hold the tokens that wrapped across the edge
            plain = max(0, min(hi, L - s) - lo)
            wrapped = (hi - lo) - plain
            out.append([x for x in (plain, wrapped) if x > 0])
    return out


def allowed_pairs(cfg) -> int:
    """Allowed (query, key) pairs per head per sample."""
    gh = _axis_groups(cfg.H, cfg.window, cfg.shift_h, bool(cfg.periodic_h))
    gw = _axis_groups(cfg.W, cfg.window, cfg.shift_w, bool(cfg.periodic_w))
    return sum(sum(x * x for x in g) for g in gh) * sum(sum(x * x for x in g) for g in gw)


def work(cfg) -> dict:
    pairs = allowed_pairs(cfg) * cfg.heads * cfg.B
    d = cfg.head_dim
    tensor_bytes = cfg.tokens * cfg.heads * d * 2
    lse_bytes = cfg.tokens * cfg.heads * 4
    return {
        "score_elements": pairs,
        "flop_fwd": 4 * d * pairs,
        "flop_bwd": 8 * d * pairs,
        "flop_bwd_fa": 10 * d * pairs,
        "bytes_fwd": 4 * tensor_bytes + lse_bytes,
        "bytes_bwd": 7 * tensor_bytes + lse_bytes,
        "tensor_bytes": tensor_bytes,
        "tokens": cfg.tokens,
    }

"""Pins for the oracle's backward pass: finite differences, autograd through a global-attention
restatement, and closed-form special cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_15211_b200.workloads import small_config
from tests._brute import rolled_geometry

CASES = [
    (6, 8, 4, 2, 2, 0, 1),
    (7, 10, 4, 2, 2, 0, 1),
    (9, 7, 4, 3, 3, 0, 1),
    (8, 8, 4, 2, 2, 0, 0),
]


def _cfg(H, W, w, sh, sw, ph, pw, heads=2, d=4, B=1):
    return small_config("t", B, H, W, heads, d, w, sh, sw, ph, pw)


def _rand(cfg, seed, n=4):
    rng = np.random.default_rng(seed)
    shape = (cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim)
    return [rng.normal(size=shape) for _ in range(n)]


def _bwd_grid(cfg, q, k, v, g, table):
    dq, dk, dv, dt = oracle.attn_bwd(cfg, q, k, v, g, table)
    return oracle.to_grid(cfg, dq), oracle.to_grid(cfg, dk), oracle.to_grid(cfg, dv), dt


def _loss(cfg, q, k, v, g, table):
    o, _ = oracle.attn_fwd(cfg, q, k, v, table)
    return float((oracle.to_grid(cfg, o) * g).sum())


@pytest.mark.parametrize("case", CASES[:3])
def test_central_finite_differences(case):
    cfg = _cfg(*case, B=2)
    q, k, v, g = _rand(cfg, 21)
    table = np.random.default_rng(22).normal(0, 0.5, size=(cfg.bias_rows, cfg.heads))
    dq, dk, dv, dt = _bwd_grid(cfg, q, k, v, g, table)
    rng = np.random.default_rng(23)
    h = 1e-5
    for name, x, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv), ("t", table, dt)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": q, "k": k, "v": v, "t": table}
            args_m = dict(args_p)
            args_p[name], args_m[name] = xp, xm
            fd = (_loss(cfg, args_p["q"], args_p["k"], args_p["v"], g, args_p["t"]) -
                  _loss(cfg, args_m["q"], args_m["k"], args_m["v"], g, args_m["t"])) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-7 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


@pytest.mark.parametrize("case", CASES)
def test_autograd_through_global_masked_attention(case):
    H, W, w, sh, sw, ph, pw = case
    cfg = _cfg(*case, B=2)
    q, k, v, g = _rand(cfg, 31)
    table = np.random.default_rng(32).normal(0, 0.5, size=(cfg.bias_rows, cfg.heads))
    dq, dk, dv, dt = _bwd_grid(cfg, q, k, v, g, table)
    win, lab, a, b = (torch.from_numpy(x.reshape(-1)) for x in rolled_geometry(H, W, w, sh, sw, ph, pw))
    allowed = (win[:, None] == win[None, :]) & (lab[:, None] == lab[None, :])
    rel = ((a[:, None] - a[None, :] + w - 1) * (2 * w - 1) + (b[:, None] - b[None, :] + w - 1))
    rel = rel.clamp(0, cfg.bias_rows - 1)               # pairs in different windows are masked below
    tq, tk, tv, tt = (torch.tensor(x, requires_grad=True) for x in (q, k, v, table))
    N = H * W
    qf, kf, vf = (x.reshape(cfg.B, N, cfg.heads, cfg.head_dim) for x in (tq, tk, tv))
    s = torch.einsum("bihc,bjhc->bhij", qf, kf) / np.sqrt(cfg.head_dim)
    s = s + tt[rel.reshape(-1)].reshape(N, N, cfg.heads).permute(2, 0, 1)[None]
    s = s.masked_fill(~allowed[None, None], float("-inf"))
    o = torch.einsum("bhij,bjhc->bihc", s.softmax(-1), vf)
    (o * torch.from_numpy(g).reshape(cfg.B, N, cfg.heads, cfg.head_dim)).sum().backward()
    np.testing.assert_allclose(dq, tq.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dk, tk.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dv, tv.grad.numpy(), atol=1e-12)
    np.testing.assert_allclose(dt, tt.grad.numpy(), atol=1e-12)


def test_bias_gradient_sums_to_zero_per_head():
    # sum_j dS_ij = 0 for every query row, hence sum_r dT[r, head] = 0
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1)
    q, k, v, g = _rand(cfg, 41)
    table = np.random.default_rng(42).normal(0, 0.5, size=(cfg.bias_rows, cfg.heads))
    _, _, _, dt = _bwd_grid(cfg, q, k, v, g, table)
    assert np.all(np.abs(dt.sum(axis=0)) < 1e-12)
    assert np.abs(dt).max() > 1e-3


def test_uniform_attention_gives_group_mean_value_gradient():
    # Q = 0, T = 0: P_ij = 1/n_group, so dV_j = mean over the group's queries of dO_i
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1)
    q, k, v, g = _rand(cfg, 51)
    dq, dk, dv, dt = _bwd_grid(cfg, np.zeros_like(q), k, v, g, np.zeros((cfg.bias_rows, cfg.heads)))
    win, lab, _, _ = rolled_geometry(7, 10, 4, 2, 2, 0, 1)
    key = win * 4 + lab
    for grp in np.unique(key):
        m = key == grp
        np.testing.assert_allclose(dv[0][m], np.broadcast_to(g[0][m].mean(axis=0), dv[0][m].shape), atol=1e-12)
    np.testing.assert_allclose(dk, 0.0, atol=1e-12)      # dK_j = scale sum_i dS_ij q_i with q = 0


def test_selection_and_bf16_inputs():
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1, B=2)
    gen = torch.Generator().manual_seed(5)
    q, k, v, g = (torch.randn(2, 7, 10, 2, 4, generator=gen).to(torch.bfloat16) for _ in range(4))
    table = np.random.default_rng(61).normal(0, 0.5, size=(cfg.bias_rows, cfg.heads))
    full = oracle.attn_bwd(cfg, q, k, v, g, table)
    dbl = oracle.attn_bwd(cfg, *(x.double().numpy() for x in (q, k, v, g)), table)
    for x, y in zip(full[:3], dbl[:3]):
        np.testing.assert_array_equal(x, y)
    np.testing.assert_allclose(full[3], dbl[3], atol=1e-13)
    nw = 6
    parts = [oracle.attn_bwd(cfg, q, k, v, g, table, sel=np.array([i])) for i in range(cfg.B * nw)]
    np.testing.assert_allclose(sum(p[3] for p in parts), full[3], atol=1e-12)
    np.testing.assert_array_equal(np.concatenate([p[0] for p in parts]), full[0])
    np.testing.assert_array_equal(np.concatenate([p[2] for p in parts]), full[2])

"""Pins for the oracle's forward pass: brute force, library special cases, invariants."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_15211_b200.workloads import small_config
from tests._brute import global_attention, random_bias_fn, rolled_geometry, table_from_fn

TINY = [
    (6, 8, 4, 2, 2, 0, 1),
    (7, 10, 4, 2, 2, 0, 1),
    (5, 9, 3, 1, 1, 0, 1),
    (9, 7, 4, 3, 3, 0, 1),
    (8, 8, 4, 2, 2, 0, 0),
    (8, 12, 4, 1, 3, 1, 1),
    (6, 6, 4, 0, 0, 0, 1),
]


def _cfg(H, W, w, sh, sw, ph, pw, heads=2, d=4, B=1):
    return small_config("t", B, H, W, heads, d, w, sh, sw, ph, pw)


def _rand(cfg, seed):
    rng = np.random.default_rng(seed)
    shape = (cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim)
    return [rng.normal(size=shape) for _ in range(3)]


def _fwd_grid(cfg, q, k, v, table, scale=0.0):
    o, lse = oracle.attn_fwd(cfg, q, k, v, table, scale=scale)
    return oracle.to_grid(cfg, o), oracle.to_grid(cfg, lse)


@pytest.mark.parametrize("case", TINY)
def test_equals_global_attention_under_membership_mask(case):
    H, W, w, sh, sw, ph, pw = case
    cfg = _cfg(*case, B=2)
    q, k, v = _rand(cfg, 1)
    fn = random_bias_fn(w, cfg.heads, 7)
    table = table_from_fn(w, cfg.heads, fn)
    o, lse = _fwd_grid(cfg, q, k, v, table)
    win, lab, a, b = rolled_geometry(H, W, w, sh, sw, ph, pw)
    for bi in range(cfg.B):
        eo, el, _ = global_attention(q[bi], k[bi], v[bi], win, lab, a, b, fn, 1.0 / np.sqrt(cfg.head_dim))
        np.testing.assert_allclose(o[bi], eo, rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[bi], el, rtol=0, atol=1e-12)


def test_bias_sign_and_axis_order_with_a_closed_form_table():
    # bias(da, db) = 0.3 da + 0.07 db with da = a_query - a_key: a transposed or sign-flipped index fails
    cfg = _cfg(5, 6, 8, 0, 0, 0, 0, heads=1, d=3)     # one window covers the grid
    q, k, v = _rand(cfg, 2)
    fn = lambda da, db, h: 0.3 * da + 0.07 * db
    table = table_from_fn(8, 1, fn)
    o, _ = _fwd_grid(cfg, q, k, v, table)
    uu, vv = np.meshgrid(np.arange(5), np.arange(6), indexing="ij")
    uu, vv = uu.reshape(-1), vv.reshape(-1)
    bias = 0.3 * (uu[:, None] - uu[None, :]) + 0.07 * (vv[:, None] - vv[None, :])
    tq, tk, tv = (torch.from_numpy(x[0, :, :, 0, :].reshape(30, 3)) for x in (q, k, v))
    exp = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None],
                                                           attn_mask=torch.from_numpy(bias)[None])
    np.testing.assert_allclose(o[0, :, :, 0, :].reshape(30, 3), exp[0].numpy(), atol=1e-12)


def test_zero_table_zero_shift_is_library_attention_per_tile():
    cfg = _cfg(8, 12, 4, 0, 0, 0, 1, heads=3, d=8)
    q, k, v = _rand(cfg, 3)
    table = np.zeros((49, 3))
    o, lse = _fwd_grid(cfg, q, k, v, table, scale=0.37)
    for r0 in range(0, 8, 4):
        for c0 in range(0, 12, 4):
            for h in range(3):
                tq, tk, tv = (torch.from_numpy(x[0, r0:r0 + 4, c0:c0 + 4, h, :].reshape(16, 8)) for x in (q, k, v))
                exp = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], scale=0.37)
                np.testing.assert_allclose(o[0, r0:r0 + 4, c0:c0 + 4, h, :].reshape(16, 8), exp[0].numpy(), atol=1e-12)
                el = torch.logsumexp(0.37 * tq @ tk.T, dim=1).numpy()
                np.testing.assert_allclose(lse[0, r0:r0 + 4, c0:c0 + 4, h].reshape(16), el, atol=1e-12)


def test_matches_swin_roll_and_region_mask_construction():
    """Both axes non-periodic on a divisible grid: the Swin Transformer's published recipe --
    roll the feature map by (-s, -s), partition into w x w tiles by reshaping, add a large negative
    number between tokens of different regions (three slices per axis: [0, L-w), [L-w, L-s), [L-s, L)),
    add the bias looked up through a pairwise relative-index matrix, softmax, merge tiles, roll back."""
    H, W, w, s, nh, d = 8, 12, 4, 2, 2, 4
    cfg = _cfg(H, W, w, s, s, 0, 0, heads=nh, d=d)
    q, k, v = (torch.from_numpy(x) for x in _rand(cfg, 4))
    table = torch.from_numpy(np.random.default_rng(5).normal(0, 0.5, size=((2 * w - 1) ** 2, nh)))

    def tiles(x):  # [H, W, C...] -> [tiles, w*w, C...]
        rest = x.shape[2:]
        x = x.reshape(H // w, w, W // w, w, *rest)
        x = x.permute(0, 2, 1, 3, *range(4, 4 + len(rest)))
        return x.reshape(-1, w * w, *rest)

    region = torch.zeros(H, W)
    cnt = 0
    for hs in (slice(0, H - w), slice(H - w, H - s), slice(H - s, H)):
        for ws in (slice(0, W - w), slice(W - w, W - s), slice(W - s, W)):
            region[hs, ws] = cnt
            cnt += 1
    reg_t = tiles(region)
    add_mask = torch.where(reg_t[:, :, None] != reg_t[:, None, :], -1.0e9, 0.0).double()
    coords = torch.stack(torch.meshgrid(torch.arange(w), torch.arange(w), indexing="ij")).flatten(1)
    rel = coords[:, :, None] - coords[:, None, :]
    rel_index = (rel[0] + w - 1) * (2 * w - 1) + (rel[1] + w - 1)
    bias = table[rel_index.reshape(-1)].reshape(w * w, w * w, nh).permute(2, 0, 1)

    roll = lambda x: torch.roll(x, shifts=(-s, -s), dims=(0, 1))
    qt, kt, vt = (tiles(roll(x[0])) for x in (q, k, v))              # [T, n, nh, d]
    att = torch.einsum("tihc,tjhc->thij", qt, kt) / np.sqrt(d) + bias[None] + add_mask[:, None]
    out = torch.einsum("thij,tjhc->tihc", att.softmax(-1), vt)       # [T, n, nh, d]
    out = out.reshape(H // w, W // w, w, w, nh, d).permute(0, 2, 1, 3, 4, 5).reshape(H, W, nh, d)
    out = torch.roll(out, shifts=(s, s), dims=(0, 1))

    o, _ = _fwd_grid(cfg, q.numpy(), k.numpy(), v.numpy(), table.numpy())
    np.testing.assert_allclose(o[0], out.numpy(), atol=1e-12)


def test_rows_sum_to_one_and_outputs_are_convex_combinations():
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1)
    q, k, v = _rand(cfg, 6)
    table = np.random.default_rng(8).normal(0, 0.5, size=(49, 2))
    o1, _ = _fwd_grid(cfg, q, k, np.ones_like(v), table)
    np.testing.assert_allclose(o1, 1.0, atol=1e-13)             # sum_j P_ij = 1
    o, _ = _fwd_grid(cfg, q, k, v, table)
    win, lab, _, _ = rolled_geometry(7, 10, 4, 2, 2, 0, 1)
    key = win * 4 + lab
    for grp in np.unique(key):
        m = key == grp
        vs, os_ = v[0][m], o[0][m]
        assert np.all(os_ <= vs.max(axis=0) + 1e-12) and np.all(os_ >= vs.min(axis=0) - 1e-12)


def test_constant_added_to_table_and_zero_query_cases():
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1)
    q, k, v = _rand(cfg, 9)
    table = np.random.default_rng(10).normal(0, 0.5, size=(49, 2))
    o, lse = _fwd_grid(cfg, q, k, v, table)
    o2, lse2 = _fwd_grid(cfg, q, k, v, table + np.array([1.5, -0.25]))
    np.testing.assert_allclose(o2, o, atol=1e-12)
    np.testing.assert_allclose(lse2 - lse, np.broadcast_to([1.5, -0.25], lse.shape), atol=1e-12)
    # Q = 0 and T = 0: uniform attention over the token's group -> group mean of V, LSE = ln(group size)
    o3, lse3 = _fwd_grid(cfg, np.zeros_like(q), k, v, np.zeros_like(table))
    win, lab, _, _ = rolled_geometry(7, 10, 4, 2, 2, 0, 1)
    key = win * 4 + lab
    for grp in np.unique(key):
        m = key == grp
        np.testing.assert_allclose(o3[0][m], np.broadcast_to(v[0][m].mean(axis=0), o3[0][m].shape), atol=1e-12)
        np.testing.assert_allclose(lse3[0][m], np.log(m.sum()), atol=1e-12)


def test_heads_and_batches_are_independent_and_mask_isolates_wrapped_rows():
    cfg = _cfg(9, 8, 4, 3, 2, 0, 1, B=2)
    q, k, v = _rand(cfg, 11)
    table = np.random.default_rng(12).normal(0, 0.5, size=(49, 2))
    o, _ = _fwd_grid(cfg, q, k, v, table)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[1], k2[1], v2[1] = 0.0, 5.0, -3.0                 # batch 1 changed
    k2[:, :, :, 1], v2[:, :, :, 1] = 2.0, 7.0            # head 1 changed
    o2, _ = _fwd_grid(cfg, q2, k2, v2, table)
    np.testing.assert_array_equal(o2[0, :, :, 0], o[0, :, :, 0])
    # poison K and V of the rows that wrapped across the latitude edge (u < shift_h)
    k3, v3 = k.copy(), v.copy()
    k3[:, :3], v3[:, :3] = 1e3, 1e6
    o3, _ = _fwd_grid(cfg, q, k3, v3, table)
    np.testing.assert_array_equal(o3[:, 3:], o[:, 3:])


@pytest.mark.parametrize("W,kshift", [(12, 5), (10, 3)])
def test_longitude_equivariance(W, kshift):
    # rolling the input along the periodic axis and shifting the window origin with it rolls the output
    base = _cfg(6, W, 4, 2, 2, 0, 1)
    q, k, v = _rand(base, 13)
    table = np.random.default_rng(14).normal(0, 0.5, size=(49, 2))
    o, _ = _fwd_grid(base, q, k, v, table)
    moved = _cfg(6, W, 4, 2, 2 + kshift, 0, 1)
    rq, rk, rv = (np.roll(x, kshift, axis=2) for x in (q, k, v))
    o2, _ = _fwd_grid(moved, rq, rk, rv, table)
    np.testing.assert_allclose(o2, np.roll(o, kshift, axis=2), atol=1e-13)


def test_truncated_window_equals_padded_window_with_masked_keys():
    # 6 x 6 grid, w = 4, no shift: the 2 x 2 corner window equals a 4 x 4 window whose padded keys are excluded
    cfg = _cfg(6, 6, 4, 0, 0, 0, 0, heads=1, d=4)
    q, k, v = _rand(cfg, 15)
    table = np.random.default_rng(16).normal(0, 0.5, size=(49, 1))
    o, _ = _fwd_grid(cfg, q, k, v, table)
    pad = lambda x: np.pad(x[0, 4:, 4:, 0], ((0, 2), (0, 2), (0, 0)))
    tq, tk, tv = (torch.from_numpy(pad(x).reshape(16, 4)) for x in (q, k, v))
    a, b = np.divmod(np.arange(16), 4)
    idx = (a[:, None] - a[None, :] + 3) * 7 + (b[:, None] - b[None, :] + 3)
    real = (a < 2) & (b < 2)
    mask = torch.from_numpy(np.where(real[None, :], table[idx, 0], -np.inf))
    exp = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], attn_mask=mask[None])[0]
    np.testing.assert_allclose(o[0, 4:, 4:, 0].reshape(4, 4), exp.numpy()[real], atol=1e-12)


def test_bf16_inputs_are_widened_exactly_and_selection_matches_full_run():
    cfg = _cfg(7, 10, 4, 2, 2, 0, 1, B=2)
    g = torch.Generator().manual_seed(3)
    q, k, v = (torch.randn(2, 7, 10, 2, 4, generator=g).to(torch.bfloat16) for _ in range(3))
    table = np.random.default_rng(17).normal(0, 0.5, size=(49, 2))
    o_b, l_b = oracle.attn_fwd(cfg, q, k, v, table)
    o_d, l_d = oracle.attn_fwd(cfg, q.double().numpy(), k.double().numpy(), v.double().numpy(), table)
    np.testing.assert_array_equal(o_b, o_d)
    sel = np.array([1 * 6 + 5, 0 * 6 + 2, 1 * 6 + 0])       # (batch, window) ids in arbitrary order
    o_s, l_s = oracle.attn_fwd(cfg, q, k, v, table, sel=sel)
    tok_all = oracle.selection_tokens(cfg, None)
    tok_sel = oracle.selection_tokens(cfg, sel)
    lookup = {t: i for i, t in enumerate(tok_all)}
    rows = np.array([lookup[t] for t in tok_sel])
    np.testing.assert_array_equal(o_s, o_b[rows])
    np.testing.assert_array_equal(l_s, l_b[rows])

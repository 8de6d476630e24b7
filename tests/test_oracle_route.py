"""Pins for the oracle's token route (integer work: everything is exact)."""
import numpy as np
import pytest

import oracle
from paper_2608_15211_b200.workloads import CONFIGS, small_config
from tests._brute import rolled_geometry

TINY = [
    # H, W, w, sh, sw, ph, pw
    (6, 8, 4, 2, 2, 0, 1),
    (7, 10, 4, 2, 2, 0, 1),
    (5, 9, 3, 1, 1, 0, 1),
    (9, 7, 4, 3, 3, 0, 1),      # 0 < H mod w < shift: the top rows split into two groups
    (8, 8, 4, 2, 2, 0, 0),
    (8, 12, 4, 1, 3, 1, 1),
    (10, 6, 4, 0, 0, 0, 1),
    (3, 5, 8, 1, 2, 0, 1),      # window larger than the grid
    (1, 7, 2, 0, 3, 0, 1),
]


def _cfg(H, W, w, sh, sw, ph, pw, heads=1, d=4, B=1):
    return small_config("t", B, H, W, heads, d, w, sh, sw, ph, pw)


@pytest.mark.parametrize("name,mh,mw,hist", [
    ("cfg1", 4, 8, {(8, 8): 32}),
    ("cfg2", 16, 32, {(8, 8): 512}),
    ("cfg3", 32, 68, {(16, 16): 2077, (16, 8): 31, (14, 16): 67, (14, 8): 1}),
    ("cfg4", 8, 16, {(32, 32): 128}),
    ("cfg5", 73, 155, {(14, 14): 11088, (14, 4): 72, (12, 14): 154, (12, 4): 1}),
])
def test_window_counts_closed_form(name, mh, mw, hist):
    cfg = CONFIGS[name]
    nt, nw, mx = oracle.route_sizes(cfg)
    assert nt == cfg.H * cfg.W
    assert nw == mh * mw == (-(-cfg.H // cfg.window)) * (-(-cfg.W // cfg.window))
    r = oracle.window_route(cfg)
    sizes = np.diff(r["win_offsets"])
    assert sizes.sum() == cfg.H * cfg.W
    assert sizes.max() == mx
    # class histogram: window rows are (extent_h, extent_w)
    got = {}
    for g, n in enumerate(sizes):
        wr, wc = divmod(g, mw)
        eh = min(cfg.window, cfg.H - wr * cfg.window)
        ew = min(cfg.window, cfg.W - wc * cfg.window)
        assert n == eh * ew
        got[(eh, ew)] = got.get((eh, ew), 0) + 1
    assert got == hist


def test_cfg3_token_sum_matches_hand_arithmetic():
    assert 2077 * 256 + 31 * 128 + 67 * 224 + 112 == 510 * 1080


@pytest.mark.parametrize("case", TINY)
def test_route_is_a_permutation_with_inverse(case):
    cfg = _cfg(*case)
    r = oracle.window_route(cfg)
    n = cfg.H * cfg.W
    assert sorted(r["perm"].tolist()) == list(range(n))
    assert np.array_equal(r["inv_perm"][r["perm"]], np.arange(n))
    assert np.all(np.diff(r["win_offsets"]) > 0)
    assert r["win_offsets"][0] == 0 and r["win_offsets"][-1] == n


@pytest.mark.parametrize("case", TINY)
def test_route_matches_physically_rolled_tiles(case):
    H, W, w, sh, sw, ph, pw = case
    cfg = _cfg(*case)
    r = oracle.window_route(cfg)
    win, lab, a, b = rolled_geometry(H, W, w, sh, sw, ph, pw)
    # per token: the slot's window, offset and label agree with the rolled picture
    slot = r["inv_perm"].reshape(H, W)
    gwin = np.searchsorted(r["win_offsets"], slot, side="right") - 1
    assert np.array_equal(gwin, win)
    assert np.array_equal(r["pos"][slot], a * w + b)
    assert np.array_equal(r["label"][slot], lab)
    # slot order: tiles of the rolled index array, read row-major, one after another
    idx = np.arange(H * W).reshape(H, W)
    rolled = np.roll(idx, shift=(-(sh % H), -(sw % W)), axis=(0, 1))
    expect = np.concatenate([rolled[r0:r0 + w, c0:c0 + w].reshape(-1)
                             for r0 in range(0, H, w) for c0 in range(0, W, w)])
    assert np.array_equal(r["perm"], expect)


def test_zero_shift_is_plain_tiling_with_no_labels():
    cfg = _cfg(10, 12, 4, 0, 0, 0, 0)
    r = oracle.window_route(cfg)
    idx = np.arange(120).reshape(10, 12)
    expect = np.concatenate([idx[r0:r0 + 4, c0:c0 + 4].reshape(-1)
                             for r0 in range(0, 10, 4) for c0 in range(0, 12, 4)])
    assert np.array_equal(r["perm"], expect)
    assert not r["label"].any()


@pytest.mark.parametrize("ph,pw", [(0, 1), (0, 0), (1, 1)])
def test_full_roll_is_the_identity(ph, pw):
    base = oracle.window_route(_cfg(9, 10, 4, 0, 0, ph, pw))
    full = oracle.window_route(_cfg(9, 10, 4, 9, 10, ph, pw))
    for k in base:
        assert np.array_equal(base[k], full[k]), k
    one = oracle.window_route(_cfg(9, 10, 4, 2, 3, ph, pw))
    more = oracle.window_route(_cfg(9, 10, 4, 2 + 9, 3 + 2 * 10, ph, pw))
    for k in one:
        assert np.array_equal(one[k], more[k]), k


def test_labels_only_on_non_periodic_axes():
    r = oracle.window_route(_cfg(8, 8, 4, 2, 2, 0, 1))
    assert set(np.unique(r["label"])) == {0, 2}
    r = oracle.window_route(_cfg(8, 8, 4, 2, 2, 1, 1))
    assert set(np.unique(r["label"])) == {0}
    r = oracle.window_route(_cfg(8, 8, 4, 2, 2, 0, 0))
    assert set(np.unique(r["label"])) == {0, 1, 2, 3}
    # wrapped tokens are exactly the first shift rows of the unrolled grid
    r = oracle.window_route(_cfg(8, 8, 4, 3, 0, 0, 1))
    lab_grid = r["label"][r["inv_perm"]].reshape(8, 8)
    assert np.all(lab_grid[:3] == 2) and np.all(lab_grid[3:] == 0)


def test_bad_descriptor_is_rejected():
    with pytest.raises(ValueError):
        oracle.window_route(_cfg(0, 8, 4, 0, 0, 0, 1))
    with pytest.raises(ValueError):
        oracle.window_route(_cfg(8, 8, 0, 0, 0, 0, 1))

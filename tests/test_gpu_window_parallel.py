"""Window-parallel execution on the GPU, one process standing in for R ranks one after the other (this machine has one
GPU; the ranks of a real run only differ in which windows they take): every rank cuts its window range into rectangles,
runs the library on each rectangle's sub-grid and writes the results at their grid positions.  The union must equal
the single call on the whole grid, and the oracle."""
import pytest
import torch

import paper_2608_15211_b200 as terra
from paper_2608_15211_b200 import window_parallel as wp
from paper_2608_15211_b200.workloads import CONFIGS, make_inputs, small_config
from tests.test_gpu_parity import _check_backward, _check_forward, _to_gpu

pytestmark = pytest.mark.gpu


def _lib_fwd(cfg, q, k, v, bias):
    return terra.terra_swin_attn_fwd(terra.make_desc(cfg), q, k, v, bias)


def _lib_bwd(cfg, q, k, v, bias, o, lse, d_o):
    return terra.terra_swin_attn_bwd(terra.make_desc(cfg), q, k, v, bias, o, lse, d_o)


def _run_all_ranks(cfg, xg, world):
    o = torch.full_like(xg["q"], float("nan"))
    lse = torch.full((cfg.B, cfg.H, cfg.W, cfg.heads), float("nan"), dtype=torch.float32, device="cuda")
    dq, dk, dv = (torch.full_like(xg["q"], float("nan")) for _ in range(3))
    dbias = torch.zeros_like(xg["bias"])
    for rank in range(world):
        plan = wp.WindowParallelPlan(cfg, world, rank)
        have = {n: wp.gather_rows_from_full(plan, xg[n]) for n in ("q", "k", "v", "do")}
        for rect in plan.rects:
            loc_cfg = wp.local_config(cfg, rect)
            loc = {n: plan.local_tensor(have[n], rect) for n in have}
            o_loc, lse_loc = _lib_fwd(loc_cfg, loc["q"], loc["k"], loc["v"], xg["bias"])
            g = _lib_bwd(loc_cfg, loc["q"], loc["k"], loc["v"], xg["bias"], o_loc, lse_loc, loc["do"])
            for full, part in ((o, o_loc), (lse, lse_loc), (dq, g[0]), (dk, g[1]), (dv, g[2])):
                wp.scatter_rows_to_full([(rect, part)], full)
            dbias += g[3]
    terra.terra_swin_check()
    return o, lse, dq, dk, dv, dbias


CASES = [
    ("wp_w16", 2, 45, 70, 3, 32, 16, 8, 8, 0, 1),            # ragged, latitude mask; ranks split window rows
    ("wp_w8_masks", 1, 30, 44, 2, 32, 8, 4, 4, 0, 0),         # masks on both axes
    ("wp_d64_w32", 1, 70, 100, 2, 64, 32, 16, 16, 0, 1),
]


@pytest.mark.parametrize("world", [2, 3, 5])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_ranks_together_equal_the_single_call_and_the_oracle(case, world):
    cfg = small_config(*case)
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0
    xg = _to_gpu(x)
    o, lse, dq, dk, dv, dbias = _run_all_ranks(cfg, xg, world)
    d = terra.make_desc(cfg)
    o1, lse1 = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    g1 = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o1, lse1, xg["do"])
    terra.terra_swin_check()
    # same kernels on the same windows: the per-window results agree to rounding of the last place at most
    for name, a, b in (("o", o, o1), ("lse", lse, lse1), ("dq", dq, g1[0]), ("dk", dk, g1[1]), ("dv", dv, g1[2])):
        assert torch.isfinite(a.float()).all(), name
        assert torch.allclose(a.float(), b.float(), rtol=2e-2, atol=2e-2 * float(b.float().abs().max())), name
    _check_forward(cfg, x, o, lse, None)
    _check_backward(cfg, x, (dq, dk, dv, dbias), None, True)


def test_config_3_on_four_ranks_matches_the_single_call():
    cfg = CONFIGS["cfg3"]
    xg = _to_gpu(make_inputs(cfg))
    o, lse, dq, dk, dv, dbias = _run_all_ranks(cfg, xg, 4)
    d = terra.make_desc(cfg)
    o1, lse1 = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    g1 = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o1, lse1, xg["do"])
    terra.terra_swin_check()
    assert torch.equal(o, o1) and torch.equal(lse, lse1)          # a window's rows do not depend on which call computed them
    for a, b in ((dq, g1[0]), (dk, g1[1]), (dv, g1[2])):
        assert torch.equal(a, b)
    assert torch.allclose(dbias, g1[3], rtol=1e-3, atol=1e-4 * float(g1[3].abs().max()))

"""Window-parallel execution (Section IV-C WP, Section V-A Eq. 4, Section IV-D token routes): the plan's integer
bookkeeping on the host, and two / three gloo ranks on the CPU that exchange grid rows, run the attention of their own
windows (the oracle stands in for the library, which has no CPU path) and route the results back."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2608_15211_b200 import window_parallel as wp
from paper_2608_15211_b200.workloads import make_inputs, small_config

CASES = [
    small_config("wp_a", 2, 20, 24, 2, 32, 4, 2, 2, 0, 1),        # latitude mask, periodic longitude
    small_config("wp_b", 1, 23, 31, 1, 32, 5, 2, 3, 0, 0),        # ragged on both axes, masks on both axes
    small_config("wp_c", 1, 9, 7, 2, 32, 4, 3, 3, 0, 1),          # 0 < H mod w < shift
    small_config("wp_d", 1, 16, 16, 1, 32, 8, 0, 0, 1, 1),        # no shift
]


@pytest.mark.parametrize("cfg", CASES, ids=[c.name for c in CASES])
@pytest.mark.parametrize("world", [1, 2, 3, 4, 7])
def test_plan_covers_every_window_once_and_the_exchange_lists_agree(cfg, world):
    mh, mw = -(-cfg.H // cfg.window), -(-cfg.W // cfg.window)
    seen = np.zeros((mh, mw), dtype=int)
    tokens = np.zeros((cfg.H, cfg.W), dtype=int)
    for r in range(world):
        plan = wp.WindowParallelPlan(cfg, world, r)
        assert plan.ranges[r] == wp.ragged_window_range(mh * mw, world, r)
        assert len(plan.rects) <= 3
        for rect in plan.rects:
            seen[rect.wr0:rect.wr1, rect.wc0:rect.wc1] += 1
            tokens[np.ix_(rect.rows, rect.cols)] += 1
            loc = wp.local_config(cfg, rect)
            assert loc.H == len(rect.rows) and loc.W == len(rect.cols)
        assert wp._sender_order_matches(plan)
        for src in range(world):
            for u in plan.fetch[r][src]:
                assert plan.stripes[src][0] <= u < plan.stripes[src][1] and src != r
    assert (seen == 1).all()            # every window owned once
    assert (tokens == 1).all()          # hence every token computed once


def test_window_counts_differ_by_at_most_one_and_boundary_rows_are_few():
    cfg = small_config("wp_e", 1, 128, 96, 1, 32, 8, 4, 4, 0, 1)
    world = 4
    counts = []
    for r in range(world):
        plan = wp.WindowParallelPlan(cfg, world, r)
        lo, hi = plan.ranges[r]
        counts.append(hi - lo)
        # stripes of 32 rows, window rows of 8, shift 4: a rank fetches a few rows at its stripe's edge, not the grid
        assert plan.rows_received() <= cfg.window + cfg.shift_h
    assert max(counts) - min(counts) <= 1


def _oracle_fwd(cfg, q, k, v, bias):
    o, lse = oracle.attn_fwd(cfg, q, k, v, bias.double().numpy())
    return (torch.from_numpy(oracle.to_grid(cfg, o)), torch.from_numpy(oracle.to_grid(cfg, lse)))


def _oracle_bwd(cfg, q, k, v, bias, o, lse, d_o):
    dq, dk, dv, db = oracle.attn_bwd(cfg, q, k, v, d_o, bias.double().numpy())
    g = lambda x: torch.from_numpy(oracle.to_grid(cfg, x))
    return g(dq), g(dk), g(dv), torch.from_numpy(db)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, cfg, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        x = {k: v.double() for k, v in make_inputs(cfg).items()}          # every rank draws the same seeded inputs ...
        x["bias"] = x["bias"] * 25.0
        plan = wp.WindowParallelPlan(cfg, world, rank)
        a, b = plan.stripes[rank]
        mine = {k: x[k][:, a:b].contiguous() for k in ("q", "k", "v", "do")}     # ... and keeps only its stripe
        o, lse = wp.wp_forward(plan, mine["q"], mine["k"], mine["v"], x["bias"], _oracle_fwd)
        dq, dk, dv, db = wp.wp_backward(plan, mine["q"], mine["k"], mine["v"], x["bias"], o, lse.double(), mine["do"], _oracle_bwd)
        out[rank] = dict(o=o.numpy(), lse=lse.numpy(), dq=dq.numpy(), dk=dk.numpy(), dv=dv.numpy(), db=db.numpy(),
                         recv=plan.rows_received())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("cfg", CASES[:3], ids=[c.name for c in CASES[:3]])
def test_gloo_ranks_reproduce_the_single_rank_result(cfg, world):
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), cfg, out), nprocs=world, join=True)
        res = dict(out)
    x = {k: v.double() for k, v in make_inputs(cfg).items()}
    x["bias"] = x["bias"] * 25.0
    ro, rl = _oracle_fwd(cfg, x["q"], x["k"], x["v"], x["bias"])
    rq, rk, rv, rb = _oracle_bwd(cfg, x["q"], x["k"], x["v"], x["bias"], None, None, x["do"])
    for name, ref in (("o", ro), ("lse", rl), ("dq", rq), ("dk", rk), ("dv", rv)):
        got = np.concatenate([res[r][name] for r in range(world)], axis=1)       # stripes back together along latitude
        tol = 1e-6 if name == "lse" else 1e-10       # lse travels and is stored as fp32, as in the library
        np.testing.assert_allclose(got, ref.numpy(), rtol=tol, atol=tol * 1e-2, err_msg=name)
    for r in range(world):
        np.testing.assert_allclose(res[r]["db"], rb.numpy(), rtol=1e-9, atol=1e-12)   # all-reduced: the same on every rank

"""Window-ownership helpers (Section V-A, Eq. 3 and Eq. 4): the oracle against the values the paper prints and
against the properties the paper states, then the library's host-side entry points against the oracle."""
import os
import random

import pytest

from oracle import assign
from paper_2608_15211_b200 import binding
from paper_2608_15211_b200.build import build

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "window_assignment.txt")


def _golden():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        left, right = line.split("->")
        kind, *args = left.split()
        rows.append((kind, {k: int(v) for k, v in (a.split("=") for a in args)},
                     dict(a.split("=") for a in right.split())))
    return rows


@pytest.mark.parametrize("kind,args,want", _golden())
def test_oracle_reproduces_the_printed_values(kind, args, want):
    if kind == "padding":
        hh, ww = assign.fixed_assignment_padding(**args)
        unit = args["p"] * args["alpha"] * args["w"]
        assert f"{hh // unit}x{ww // unit}" == want["grid"]
        assert round(100 * assign.padding_overhead(args["H"], args["W"], hh, ww), 1) == float(want["overhead_pct"])
    else:
        counts = sorted(b - a for a, b in (assign.ragged_window_range(args["M"], args["ranks"], r) for r in range(args["ranks"])))
        assert counts == [int(c) for c in want["counts_sorted"].split(",")]


def test_ragged_ranges_partition_the_windows_and_differ_by_at_most_one():
    """Section V-A: every complete window is assigned exactly once; any two ranks' counts differ by at most one."""
    for M in list(range(0, 40)) + [45, 128, 2176, 11315]:
        for ranks in (1, 2, 3, 4, 7, 8, 16, 33):
            rng = [assign.ragged_window_range(M, ranks, r) for r in range(ranks)]
            assert rng[0][0] == 0 and rng[-1][1] == M
            assert all(rng[r][1] == rng[r + 1][0] for r in range(ranks - 1))
            counts = [b - a for a, b in rng]
            assert min(counts) >= 0 and max(counts) - min(counts) <= 1
            # brute force: the owner of each window, from the inequalities solved for the rank
            for j in range(M):
                r = assign.ragged_owner(M, ranks, j)
                assert rng[r][0] <= j < rng[r][1]


def test_padding_is_the_smallest_multiple_that_covers_the_field():
    rnd = random.Random(7)
    for _ in range(200):
        H, W = rnd.randint(1, 5000), rnd.randint(1, 9000)
        p, alpha, w = rnd.choice((1, 2, 4)), rnd.choice((1, 2)), rnd.choice((4, 8, 16, 32, 128))
        m, n = rnd.randint(1, 4), rnd.randint(1, 8)
        hh, ww = assign.fixed_assignment_padding(H, W, p, alpha, w, m, n)
        uh, uw = p * alpha * w * m, p * alpha * w * n
        assert hh % uh == 0 and ww % uw == 0 and 0 <= hh - H < uh and 0 <= ww - W < uw
        # equal window ownership on the m x n mesh: the window grid divides by the mesh
        assert (hh // (p * alpha * w)) % m == 0 and (ww // (p * alpha * w)) % n == 0


@pytest.fixture(scope="module")
def lib():
    build()
    return binding.load_library()


def test_library_matches_the_oracle(lib):
    rnd = random.Random(11)
    for _ in range(300):
        H, W = rnd.randint(1, 10**6), rnd.randint(1, 10**6)
        p, alpha, w = rnd.choice((1, 2, 4, 8)), rnd.choice((1, 2, 3)), rnd.randint(1, 128)
        m, n = rnd.randint(1, 16), rnd.randint(1, 16)
        assert binding.terra_fixed_assignment_padding(H, W, p, alpha, w, m, n) == assign.fixed_assignment_padding(H, W, p, alpha, w, m, n)
    for _ in range(300):
        M, ranks = rnd.choice((0, 1, 10, 45, 2176, 11315, rnd.randint(0, 2**40), 2**62 + 12345)), rnd.randint(1, 4096)
        for r in {0, ranks - 1, rnd.randrange(ranks)}:
            assert binding.terra_ragged_window_range(M, ranks, r) == assign.ragged_window_range(M, ranks, r)


def test_library_rejects_bad_arguments(lib):
    for bad in ((0, 10, 1, 1, 1, 1, 1), (10, 10, 0, 1, 1, 1, 1), (10, 10, 1, 1, 1, 0, 1), (10, 10, 2**31 - 1, 2**31 - 1, 2**31 - 1, 2, 1)):
        with pytest.raises(binding.TerraError) as e:
            binding.terra_fixed_assignment_padding(*bad)
        assert e.value.status == 1
    for bad in ((-1, 4, 0), (10, 0, 0), (10, 4, 4), (10, 4, -1)):
        with pytest.raises(binding.TerraError) as e:
            binding.terra_ragged_window_range(*bad)
        assert e.value.status == 1


# ---- two gloo ranks: each asks the library for its own range; together they own every window once ----------

def _free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _owner_worker(rank: int, world: int, port: int, M: int, out):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = binding.terra_ragged_window_range(M, world, rank)
        mine = torch.tensor([lo, hi], dtype=torch.int64)
        both = [torch.zeros(2, dtype=torch.int64) for _ in range(world)]
        dist.all_gather(both, mine)
        out[rank] = [tuple(int(v) for v in t) for t in both]
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("M", [2176, 11315, 5])
def test_two_ranks_own_every_window_exactly_once(M):
    import torch.multiprocessing as mp
    build()
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_owner_worker, args=(world, _free_port(), M, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]                                   # every rank sees the same ownership table
    (l0, r0), (l1, r1) = res[0]
    assert l0 == 0 and r0 == l1 and r1 == M and abs((r0 - l0) - (r1 - l1)) <= 1
    assert [(l0, r0), (l1, r1)] == [assign.ragged_window_range(M, world, r) for r in range(world)]

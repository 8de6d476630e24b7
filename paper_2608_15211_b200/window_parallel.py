"""Window-parallel execution of the shifted-window attention block over several ranks (paper Section IV-C "WP",
Section IV-D token routes, Section V-A ragged window assignment, Eq. 4).

Every complete window is owned by exactly one rank: rank r of R owns the row-major window range
[floor(r M / R), floor((r + 1) M / R)) of the M = M_h x M_w windows (Eq. 4; the C ABI's
`terra_ragged_window_range`).  The activations live in the spatially contiguous layout, split along latitude:
rank r holds the grid rows [floor(r H / R), floor((r + 1) H / R)) of every tensor.  One step is

  1. token route in: each rank fetches the grid rows its windows touch and that it does not hold (rows near its
     stripe's edges, a few times the window side and the shift; with stripes and ranges lined up this is the
     boundary-only exchange of Section V-A) -- point-to-point copies into local memory;
  2. attention on the rank's windows: the window range is cut into at most three rectangles of windows (the tail
     of a window row, whole window rows, the head of a window row); each rectangle is a shifted-window problem of
     its own on a sub-grid, and is handed to the library call unchanged (see `Rect` for how the roll and the shift
     mask of the full grid carry over);
  3. token route out: outputs (or gradients) return to the ranks that hold their rows: the inverse mapping;
  4. backward only: the relative-position-bias gradient is summed over the ranks (one all-reduce).

The exchange uses torch.distributed point-to-point calls and works on any backend (NCCL between GPUs, gloo between
CPU processes in the tests).  The attention itself is injected (`fwd_fn`, `bwd_fn`): the library's binding on a GPU.
Nothing here holds arithmetic of the method; the plan is integer bookkeeping.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch
import torch.distributed as dist


def ragged_window_range(M: int, ranks: int, r: int):
    """Eq. 4: rank r of `ranks` owns windows [floor(r M / ranks), floor((r + 1) M / ranks))."""
    return (r * M) // ranks, ((r + 1) * M) // ranks


def stripe_rows(H: int, ranks: int, r: int):
    """Grid rows of the contiguous layout that rank r holds."""
    return (r * H) // ranks, ((r + 1) * H) // ranks


@dataclass(frozen=True)
class Rect:
    """A rectangle of windows [wr0, wr1) x [wc0, wc1) as a shifted-window problem of its own.

    In the rolled frame of the full grid the rectangle covers rows [wr0 w, min(H, wr1 w)) and columns
    [wc0 w, min(W, wc1 w)): windows tile it from its corner exactly as they tile the full frame, and its last window
    row / column is truncated exactly where the full grid's is.  `rows` / `cols` list the ORIGINAL grid rows / columns
    of the sub-grid in the order of the local tensor.  On a non-periodic axis whose rectangle mixes tokens that
    wrapped across the edge with tokens that did not, the wrapped ones come first and the local problem is given the
    shift `shift_h` (`shift_w`) = their number: the library's own roll then moves them behind the others, where the
    full frame has them, and its shift mask separates the two groups.  Otherwise the local order is the rolled order,
    the local shift is 0 and no mask is needed (all tokens belong to one group).
    """
    wr0: int
    wr1: int
    wc0: int
    wc1: int
    rows: tuple
    cols: tuple
    shift_h: int
    shift_w: int
    periodic_h: int
    periodic_w: int


def _axis(L: int, w: int, s: int, periodic: bool, lo_win: int, hi_win: int):
    """Original coordinates of rolled positions [lo_win w, min(L, hi_win w)) in local order, the local shift and the
    local periodic flag."""
    s %= L
    rolled = range(lo_win * w, min(L, hi_win * w))
    orig = [(x + s) % L for x in rolled]
    if periodic or s == 0:
        return tuple(orig), 0, 1
    wrapped = [c for x, c in zip(rolled, orig) if x >= L - s]      # tokens with original coordinate < s
    plain = [c for x, c in zip(rolled, orig) if x < L - s]
    if wrapped and plain:
        return tuple(wrapped + plain), len(wrapped), 0
    return tuple(orig), 0, 1


def window_rectangles(cfg, lo: int, hi: int):
    """The window range [lo, hi) (row-major) as at most three rectangles of windows."""
    mw = -(-cfg.W // cfg.window)
    out = []
    if hi <= lo:
        return out
    r0, r1 = lo // mw, (hi - 1) // mw
    spans = []
    if r0 == r1:
        spans.append((r0, r0 + 1, lo - r0 * mw, hi - r0 * mw))
    else:
        first_full = r0 if lo == r0 * mw else r0 + 1
        last_full = r1 + 1 if hi == (r1 + 1) * mw else r1
        if first_full > r0:
            spans.append((r0, r0 + 1, lo - r0 * mw, mw))
        if last_full > first_full:
            spans.append((first_full, last_full, 0, mw))
        if last_full <= r1:
            spans.append((r1, r1 + 1, 0, hi - r1 * mw))
    for wr0, wr1, wc0, wc1 in spans:
        rows, sh, ph = _axis(cfg.H, cfg.window, cfg.shift_h, bool(cfg.periodic_h), wr0, wr1)
        cols, sw, pw = _axis(cfg.W, cfg.window, cfg.shift_w, bool(cfg.periodic_w), wc0, wc1)
        out.append(Rect(wr0, wr1, wc0, wc1, rows, cols, sh, sw, ph, pw))
    return out


def local_config(cfg, rect: Rect):
    """The configuration of the rectangle's own shifted-window problem."""
    return replace(cfg, name=f"{cfg.name}[{rect.wr0}:{rect.wr1},{rect.wc0}:{rect.wc1}]", H=len(rect.rows), W=len(rect.cols),
                   shift_h=rect.shift_h, shift_w=rect.shift_w, periodic_h=rect.periodic_h, periodic_w=rect.periodic_w)


class WindowParallelPlan:
    """Who owns which windows, which grid rows each rank needs, and who sends which rows to whom."""

    def __init__(self, cfg, world: int, rank: int):
        self.cfg, self.world, self.rank = cfg, world, rank
        mh, mw = -(-cfg.H // cfg.window), -(-cfg.W // cfg.window)
        self.n_windows = mh * mw
        self.ranges = [ragged_window_range(self.n_windows, world, r) for r in range(world)]
        self.stripes = [stripe_rows(cfg.H, world, r) for r in range(world)]
        self.rects_of = [window_rectangles(cfg, lo, hi) for lo, hi in self.ranges]
        self.rects = self.rects_of[rank]
        # grid rows each rank needs (sorted, unique) and, of those, the ones it does not hold
        self.needed = [sorted({u for rect in rects for u in rect.rows}) for rects in self.rects_of]
        self.owner_of_row = [0] * cfg.H
        for r, (a, b) in enumerate(self.stripes):
            for u in range(a, b):
                self.owner_of_row[u] = r
        # fetch[dst][src] = rows that dst gets from src (sorted); the same lists drive the way back
        self.fetch = [[[] for _ in range(world)] for _ in range(world)]
        for dst in range(world):
            for u in self.needed[dst]:
                src = self.owner_of_row[u]
                if src != dst:
                    self.fetch[dst][src].append(u)

    # ---- sizes, for reporting (Section V-A: boundary-only exchange) -------------------------------------------
    def rows_received(self, rank=None) -> int:
        rank = self.rank if rank is None else rank
        return sum(len(v) for v in self.fetch[rank])

    def rows_sent(self, rank=None) -> int:
        rank = self.rank if rank is None else rank
        return sum(len(self.fetch[dst][rank]) for dst in range(self.world))

    # ---- token route in ----------------------------------------------------------------------------------------
    def gather_rows(self, stripe: torch.Tensor):
        """stripe [B, rows of this rank, W, ...] -> (pool [B, n, W, ...], position of grid row u in the pool) for every
        row this rank needs.  Rows held by other ranks arrive by point-to-point copies into local buffers; the pool is
        the stripe followed by those buffers."""
        a, b = self.stripes[self.rank]
        ops, recv_bufs, pos = [], [], {u: u - a for u in range(a, b)}
        n = b - a
        for src in range(self.world):
            rows = self.fetch[self.rank][src]
            if rows:
                buf = torch.empty((stripe.shape[0], len(rows)) + tuple(stripe.shape[2:]), dtype=stripe.dtype, device=stripe.device)
                recv_bufs.append(buf)
                for j, u in enumerate(rows):
                    pos[u] = n + j
                n += len(rows)
                ops.append(dist.P2POp(dist.irecv, buf, src))
        send_keep = []
        for dst in range(self.world):
            rows = self.fetch[dst][self.rank]
            if rows:
                idx = torch.tensor([u - a for u in rows], device=stripe.device)
                buf = stripe.index_select(1, idx).contiguous()
                send_keep.append(buf)
                ops.append(dist.P2POp(dist.isend, buf, dst))
        if ops:
            for req in dist.batch_isend_irecv(ops):
                req.wait()
        pool = torch.cat([stripe] + recv_bufs, dim=1) if recv_bufs else stripe
        return pool, pos

    def local_tensor(self, have, rect: Rect) -> torch.Tensor:
        """The rectangle's sub-grid [B, rows, cols, ...] from the gathered grid rows."""
        pool, pos = have
        rows = [pos[u] for u in rect.rows]
        x = pool
        if rows != list(range(pool.shape[1])):
            x = x.index_select(1, torch.tensor(rows, device=pool.device))
        if list(rect.cols) != list(range(pool.shape[2])):
            x = x.index_select(2, torch.tensor(rect.cols, device=pool.device))
        return x.contiguous()

    # ---- token route out ---------------------------------------------------------------------------------------
    def scatter_rows(self, parts: list, stripe_out: torch.Tensor) -> None:
        """parts = [(rect, local tensor [B, rows, cols, ...])]: every value goes to the rank that holds its grid row,
        at its grid position (the inverse of gather_rows + local_tensor).  Positions of `stripe_out` that no window of
        any rank covers do not exist: the windows tile the whole grid."""
        a, _ = self.stripes[self.rank]
        W = self.cfg.W
        tail = tuple(stripe_out.shape[3:])
        B = stripe_out.shape[0]
        # full-width rows of this rank's results, keyed by grid row: (columns, values)
        by_row = {}
        for rect, loc in parts:
            loc = loc.to(stripe_out.dtype)
            for j, u in enumerate(rect.rows):
                by_row.setdefault(u, []).append((rect.cols, loc[:, j]))
        ops, recv_bufs, send_keep = [], [], []
        # what this rank computed for rows held elsewhere: one message per destination, (row, column)-ordered
        out_msgs = {}
        for u in sorted(by_row):
            dst = self.owner_of_row[u]
            if dst != self.rank:
                out_msgs.setdefault(dst, []).append(u)
        for dst, rows in out_msgs.items():
            pieces = []
            for u in rows:
                for cols, val in by_row[u]:
                    pieces.append(val.reshape(B, len(cols), -1))
            buf = torch.cat(pieces, dim=1).contiguous()
            send_keep.append(buf)
            ops.append(dist.P2POp(dist.isend, buf, dst))
        # what other ranks computed for rows held here: the plan tells which (row, columns) come from whom
        for src in range(self.world):
            if src == self.rank:
                continue
            layout = []
            for rect in self.rects_of[src]:
                for u in rect.rows:
                    if self.owner_of_row[u] == self.rank:
                        layout.append((u, rect.cols))
            layout.sort(key=lambda t: t[0])        # stable: same order as the sender's (rows sorted, rectangles in order)
            if layout:
                n = sum(len(c) for _, c in layout)
                buf = torch.empty((B, n, math.prod(tail) if tail else 1), dtype=stripe_out.dtype, device=stripe_out.device)
                recv_bufs.append((layout, buf))
                ops.append(dist.P2POp(dist.irecv, buf, src))
        if ops:
            for req in dist.batch_isend_irecv(ops):
                req.wait()
        flat = stripe_out.reshape(B, stripe_out.shape[1], W, -1)
        for rect, loc in parts:        # rows of this rank's own results that it also holds: one indexed write per rectangle
            keep = [(j, u - a) for j, u in enumerate(rect.rows) if self.owner_of_row[u] == self.rank]
            if keep:
                src_rows = torch.tensor([j for j, _ in keep], device=flat.device)
                dst_rows = torch.tensor([d for _, d in keep], device=flat.device)
                cols = torch.tensor(rect.cols, device=flat.device)
                vals = loc.to(stripe_out.dtype).reshape(B, len(rect.rows), len(rect.cols), -1).index_select(1, src_rows)
                flat[:, dst_rows[:, None], cols[None, :]] = vals
        for layout, buf in recv_bufs:
            pos = 0
            for u, cols in layout:
                flat[:, u - a, torch.tensor(cols, device=flat.device)] = buf[:, pos:pos + len(cols)]
                pos += len(cols)


def gather_rows_from_full(plan: WindowParallelPlan, full: torch.Tensor) -> dict:
    """The rows a rank needs, taken from a tensor that holds the whole grid (inputs replicated on every rank, or one
    process standing in for all ranks): no exchange."""
    return full, {u: u for u in plan.needed[plan.rank]}


def scatter_rows_to_full(parts: list, full_out: torch.Tensor) -> None:
    """Writes a rank's results at their grid positions of a whole-grid tensor."""
    B, H, W = full_out.shape[:3]
    flat = full_out.reshape(B, H, W, -1)
    for rect, loc in parts:
        rows = torch.tensor(rect.rows, device=flat.device)
        cols = torch.tensor(rect.cols, device=flat.device)
        flat[:, rows[:, None], cols[None, :]] = loc.reshape(B, len(rect.rows), len(rect.cols), -1).to(flat.dtype)


def _sender_order_matches(plan: WindowParallelPlan) -> bool:
    """Self-check used by the tests: for every (src, dst) the receiver's layout lists the same (row, columns) items in
    the same order as the sender emits them."""
    for src in range(plan.world):
        by_row = {}
        for rect in plan.rects_of[src]:
            for u in rect.rows:
                by_row.setdefault(u, []).append(rect.cols)
        for dst in range(plan.world):
            if dst == src:
                continue
            sent = [(u, cols) for u in sorted(by_row) if plan.owner_of_row[u] == dst for cols in by_row[u]]
            layout = []
            for rect in plan.rects_of[src]:
                for u in rect.rows:
                    if plan.owner_of_row[u] == dst:
                        layout.append((u, rect.cols))
            layout.sort(key=lambda t: t[0])
            if sent != layout:
                return False
    return True


def wp_forward(plan: WindowParallelPlan, q, k, v, bias, fwd_fn):
    """Window-parallel forward.  q, k, v: this rank's stripes [B, rows, W, heads, d]; bias: the full table (replicated).
    fwd_fn(local_cfg, q, k, v, bias) -> (o [B, h, w, heads, d], lse [B, h, w, heads]).  Returns the stripes of o and lse."""
    hq, hk, hv = plan.gather_rows(q), plan.gather_rows(k), plan.gather_rows(v)
    o_parts, l_parts = [], []
    for rect in plan.rects:
        cfg_loc = local_config(plan.cfg, rect)
        o_loc, lse_loc = fwd_fn(cfg_loc, plan.local_tensor(hq, rect), plan.local_tensor(hk, rect), plan.local_tensor(hv, rect), bias)
        o_parts.append((rect, o_loc))
        l_parts.append((rect, lse_loc))
    o = torch.empty_like(q)
    lse = torch.empty(q.shape[:4], dtype=torch.float32, device=q.device)
    plan.scatter_rows(o_parts, o)
    plan.scatter_rows(l_parts, lse)
    return o, lse


def wp_backward(plan: WindowParallelPlan, q, k, v, bias, o, lse, d_o, bwd_fn):
    """Window-parallel backward.  Stripes in, stripes of dq, dk, dv out; dbias is summed over the ranks (all-reduce).
    bwd_fn(local_cfg, q, k, v, bias, o, lse, d_o) -> (dq, dk, dv, dbias)."""
    h = {n: plan.gather_rows(t) for n, t in (("q", q), ("k", k), ("v", v), ("o", o), ("lse", lse), ("do", d_o))}
    parts = {"dq": [], "dk": [], "dv": []}
    dbias = torch.zeros_like(bias)
    for rect in plan.rects:
        cfg_loc = local_config(plan.cfg, rect)
        loc = {n: plan.local_tensor(h[n], rect) for n in h}
        dq, dk, dv, db = bwd_fn(cfg_loc, loc["q"], loc["k"], loc["v"], bias, loc["o"], loc["lse"], loc["do"])
        parts["dq"].append((rect, dq))
        parts["dk"].append((rect, dk))
        parts["dv"].append((rect, dv))
        dbias += db
    out = {n: torch.empty_like(q) for n in parts}
    for n in parts:
        plan.scatter_rows(parts[n], out[n])
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(dbias)
    return out["dq"], out["dk"], out["dv"], dbias


def library_fns():
    """fwd_fn / bwd_fn that call the CUDA library through its binding (local tensors on the current GPU)."""
    from . import binding

    def fwd_fn(cfg, q, k, v, bias):
        return binding.terra_swin_attn_fwd(binding.make_desc(cfg, dtype=q.dtype), q, k, v, bias)

    def bwd_fn(cfg, q, k, v, bias, o, lse, d_o):
        return binding.terra_swin_attn_bwd(binding.make_desc(cfg, dtype=q.dtype), q, k, v, bias, o, lse, d_o)

    return fwd_fn, bwd_fn


def main():
    """One window-parallel forward + backward step over the ranks of the current torchrun job (NCCL), each rank on its
    own GPU with its latitude stripe of the seeded workload:

        python -m torch.distributed.run --nnodes=1 --nproc-per-node R --master-addr 127.0.0.1 --master-port P \\
            -m paper_2608_15211_b200.window_parallel --config cfg3

    Prints one JSON line per job: step time (maximum over ranks, CUDA events), windows and exchanged rows per rank.
    Without torchrun it runs as a single rank."""
    import argparse
    import json
    import os

    from .workloads import CONFIGS, make_activation, make_bias_table

    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--steps", type=int, default=5)
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    plan = WindowParallelPlan(cfg, world, rank)
    a, b = plan.stripes[rank]
    # every rank draws the same seeded tensors and keeps its stripe (a real model would produce the stripe in place)
    stripe = {n: make_activation(cfg, n, dev)[:, a:b].contiguous() for n in ("q", "k", "v", "do")}
    bias = make_bias_table(cfg, dev)
    fwd_fn, bwd_fn = library_fns()

    def step():
        o, lse = wp_forward(plan, stripe["q"], stripe["k"], stripe["v"], bias, fwd_fn)
        return wp_backward(plan, stripe["q"], stripe["k"], stripe["v"], bias, o, lse, stripe["do"], bwd_fn)

    step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    ms = torch.tensor([t0.elapsed_time(t1) / args.steps], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"config": cfg.name, "ranks": world, "ms_per_step_max_over_ranks": float(ms.item()),
                          "windows_per_rank": [hi - lo for lo, hi in plan.ranges],
                          "grid_rows_received_per_rank": [plan.rows_received(r) for r in range(world)],
                          "grid_rows_per_stripe": [hi - lo for lo, hi in plan.stripes]}), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

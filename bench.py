#!/usr/bin/env python
"""Benchmark of the shifted-window attention block (route + forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl reference]

One step = one pass of the whole hot path over one batch of seeded synthetic input: the token route
(index map), the fused forward, and the fused backward, all through the C ABI.  The default workload
is the Wenhai-shaped configuration (token grid 510 x 1080, 12 heads x 32, window 16, shift 8), the one
the headline metric is quoted on.  Nothing is sharded: with N > 1 every rank runs an independent
replica of the same workload ("replicas only") and the value is the aggregate over ranks.

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "shifted-window attn fwd+bwd TFLOP/s (bf16)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()       # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample_ids(cfg, count):
    """Evenly spaced (batch, window) ids: a bounded sample of the workload's windows."""
    import numpy as np
    mh, mw = -(-cfg.H // cfg.window), -(-cfg.W // cfg.window)
    total = cfg.B * mh * mw
    count = max(1, min(count, total))
    return np.unique(np.linspace(0, total - 1, count).astype(np.int64))


def oracle_sample_flops(cfg, ids):
    """Strict FLOP count of the sampled windows (forward + backward), from the route's labels."""
    import numpy as np
    import oracle
    r = oracle.window_route(cfg)
    nw = len(r["win_offsets"]) - 1
    pairs = 0
    for i in ids:
        g = int(i) % nw
        lab = r["label"][r["win_offsets"][g]:r["win_offsets"][g + 1]]
        pairs += int(sum(int((lab == v).sum()) ** 2 for v in np.unique(lab)))
    return 12 * cfg.head_dim * pairs * cfg.heads


def time_oracle(cfg, x, ids):
    import oracle
    table = x["bias"].double().numpy()
    t0 = time.perf_counter()
    oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], table, sel=ids)
    oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], table, sel=ids)
    return time.perf_counter() - t0


def oracle_probe_count(cfg):
    """Windows in the first timing probe of the oracle, or 0 if a single window of the workload is beyond any bounded
    sample (estimated from the window's score elements x head dim at about 3e8 per second, the oracle's order of
    magnitude on large windows)."""
    n = min(cfg.window, cfg.H) * min(cfg.window, cfg.W)
    est = cfg.heads * n * n * cfg.head_dim / 3.0e8
    if est > 40.0:
        return 0
    return int(max(1, min(8, 10.0 / max(est, 1e-6))))


def cpu_baseline(cfg, target_seconds=12.0):
    """The oracle, as it stands, timed on this machine's host cores on a bounded sample of windows."""
    import oracle
    from paper_2608_15211_b200.workloads import make_inputs
    n_probe = oracle_probe_count(cfg)
    if n_probe == 0:
        return {"value": None, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                "sample": f"not timed: one {cfg.window} x {cfg.window} window of {cfg.name} over {cfg.heads} heads takes the "
                          f"fp64 oracle minutes, beyond a bounded sample"}
    x = make_inputs(cfg)
    probe = oracle_sample_ids(cfg, n_probe)
    t_probe = time_oracle(cfg, x, probe)
    count = int(max(n_probe, min(len(probe) * target_seconds / max(t_probe, 1e-3), 4096)))
    ids = oracle_sample_ids(cfg, count)
    t = time_oracle(cfg, x, ids)
    flops = oracle_sample_flops(cfg, ids)
    return {"value": flops / t / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{len(ids)} of {cfg.B * (-(-cfg.H // cfg.window)) * (-(-cfg.W // cfg.window))} windows of "
                      f"{cfg.name}, forward + backward, fp64, {t:.1f} s wall"}


def run_reference(args, cfg):
    """--impl reference: the CPU oracle on a bounded sample per step, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2608_15211_b200.workloads import make_inputs
    n_probe = oracle_probe_count(cfg)
    if n_probe == 0:
        print(json.dumps({"impl": "reference", "unavailable": f"one window of {cfg.name} takes the fp64 oracle minutes: "
                                                              f"no bounded sample of this workload"}), flush=True)
        return
    x = make_inputs(cfg)
    probe = oracle_sample_ids(cfg, n_probe)
    t_probe = time_oracle(cfg, x, probe)
    budget = 120.0 / max(1, args.steps + args.warmup)          # whole run within a few minutes
    count = int(max(min(4, n_probe), min(len(probe) * min(budget, 10.0) / max(t_probe, 1e-3), 4096)))
    ids = oracle_sample_ids(cfg, count)
    flops = oracle_sample_flops(cfg, ids)
    for _ in range(args.warmup):
        time_oracle(cfg, x, ids)
    times = [time_oracle(cfg, x, ids) for _ in range(args.steps)]
    t = sum(times) / len(times)
    value = flops / t / 1e12
    sample = f"{len(ids)} windows of {cfg.name} per step, forward + backward, fp64"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg, "cpu oracle; no GPU work"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per (batch, window, head) item from the ncu
# captures summarised under profiles/ (config 3 cut to 254 token rows, 13 056 items); traffic grows in
# proportion to the item count, so a full launch is this figure times its items.  None = not captured.
TRAFFIC_SOURCE = "stored ncu capture (profiles/swin_*_cfg3_rows254.md), scaled by the item count; not measured in this run"
NCU_DRAM_BYTES_PER_ITEM = {
    "swin_fwd_tc_kernel": 63575,
    "swin_bwd_fused_kernel": 112166,
}


def ncu_traffic(kernel, cfg):
    per_item = NCU_DRAM_BYTES_PER_ITEM.get(kernel)
    if per_item is None or cfg.head_dim != 32 or cfg.window != 16:
        return None
    mh, mw = -(-cfg.H // cfg.window), -(-cfg.W // cfg.window)
    return per_item * cfg.B * mh * mw * cfg.heads


def workload_config(cfg, l2_note):
    return {"workload": f"{cfg.name}: B={cfg.B}, token grid {cfg.H}x{cfg.W}, {cfg.heads} heads x d={cfg.head_dim}, "
                        f"window {cfg.window}, shift {cfg.shift_h}, lat non-periodic / lon periodic, fwd+bwd",
            "l2": l2_note, "flop_convention": "strict: 12*d per allowed (query, key) pair per head",
            "parallelism": "replicas only (nothing sharded, no collectives)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="cfg3")
    ap.add_argument("--impl", default="terra", choices=["terra", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-packed", action="store_true", help="skip the packed-QKV leg")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp16"],
                    help="element type of the activations and gradients (the benchmark's metric is quoted on bf16)")
    ap.add_argument("--rows", type=int, default=0,
                    help="profiling aid: keep the configuration but use this many token rows (a smaller case of the "
                         "same kernels for ncu captures); the JSON names the changed grid")
    args = ap.parse_args()

    import dataclasses
    from paper_2608_15211_b200.workloads import CONFIGS
    cfg = CONFIGS[args.config]
    if args.rows > 0:
        cfg = dataclasses.replace(cfg, H=args.rows, name=f"{cfg.name}-rows{args.rows}")
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist

    import paper_2608_15211_b200 as terra
    from paper_2608_15211_b200.accounting import work
    from paper_2608_15211_b200.replicas import max_over_ranks, whole_job_tflops
    from paper_2608_15211_b200.build import build
    from paper_2608_15211_b200.workloads import make_activation, make_bias_table

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    terra.load_library()
    dev = f"cuda:{local_rank}"
    peaks, peak_kind = load_peaks()

    # inputs resident in HBM (seeded device generators)
    act_dtype = torch.float16 if args.dtype == "fp16" else torch.bfloat16
    q, k, v, d_o = (make_activation(cfg, t, dev).to(act_dtype) for t in ("q", "k", "v", "do"))
    bias = make_bias_table(cfg, dev)
    desc = terra.make_desc(cfg, dtype=act_dtype)
    nt, nw, _ = terra.terra_route_sizes(desc)
    route = {n: torch.empty(nt, dtype=torch.int32, device=dev) for n in ("perm", "inv_perm", "pos", "label")}
    route["win_offsets"] = torch.empty(nw + 1, dtype=torch.int32, device=dev)
    o = torch.empty_like(q)
    lse = torch.empty((cfg.B, cfg.H, cfg.W, cfg.heads), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dbias = torch.empty_like(bias)
    ws = torch.empty(max(16, terra.terra_swin_workspace_bytes(desc, True), terra.terra_swin_workspace_bytes(desc, False)),
                     dtype=torch.uint8, device=dev)
    lib = terra.load_library()
    import ctypes
    P = lambda t: ctypes.c_void_p(t.data_ptr())
    stream = torch.cuda.current_stream()
    sp = ctypes.c_void_p(stream.cuda_stream)

    def call_route():
        rc = lib.terra_window_route(ctypes.byref(desc), P(route["perm"]), P(route["inv_perm"]), P(route["win_offsets"]),
                                    P(route["pos"]), P(route["label"]), sp)
        assert rc == 0, rc

    def call_fwd():
        rc = lib.terra_swin_attn_fwd(ctypes.byref(desc), P(q), P(k), P(v), P(bias), P(o), P(lse), P(ws), ws.numel(), sp)
        assert rc == 0, rc

    def call_bwd():
        rc = lib.terra_swin_attn_bwd(ctypes.byref(desc), P(q), P(k), P(v), P(bias), P(o), P(lse), P(d_o),
                                     P(dq), P(dk), P(dv), P(dbias), P(ws), ws.numel(), sp)
        assert rc == 0, rc

    def step():
        call_route()
        call_fwd()
        call_bwd()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    terra.terra_swin_check()           # raises if any kernel of the warm-up gave up on a bounded wait

    wk = work(cfg)
    flops = wk["flop_fwd"] + wk["flop_bwd"]
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = terra.launch_count()
    terra.profile_enable(True)         # the library brackets each of its main kernels with CUDA events on this stream
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        ev[i][0].record(stream)
        call_route()
        ev[i][1].record(stream)
        call_fwd()
        ev[i][2].record(stream)
        call_bwd()
        ev[i][3].record(stream)
    t_end.record(stream)
    barrier()
    # a CTA whose bounded wait expired leaves its loops early and the launch still returns TERRA_OK: a timed
    # region that saw that is not a measurement, so it ends the run with an error instead of a line
    terra.terra_swin_check()
    launches = terra.launch_count() - launches0
    kernel_ms = {}
    for kname, kms in terra.profile_read():
        kernel_ms.setdefault(kname, []).append(kms)
    terra.profile_enable(False)
    clocks = sampler.stop()
    total_ms = max_over_ranks(t_start.elapsed_time(t_end), dev)     # the job is as slow as its slowest replica
    ms_step = total_ms / args.steps
    route_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    fwd_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
    bwd_ms = statistics.mean(e[2].elapsed_time(e[3]) for e in ev)
    value = whole_job_tflops(flops, world, ms_step)

    # the same step on the packed layout of a fused QKV projection ([B, H, W, 3, heads, d] in, the gradient in
    # the same layout out): same kernels, only the token stride differs
    packed = None
    if not args.no_packed:
        qkv = torch.stack([q, k, v], dim=3).contiguous()
        dqkv = torch.empty_like(qkv)
        for _ in range(3):
            terra.terra_swin_attn_fwd_packed(desc, qkv, bias, o, lse, ws)
            terra.terra_swin_attn_bwd_packed(desc, qkv, bias, o, lse, d_o, dqkv, dbias, ws)
        n_packed = max(4, min(args.steps, 20))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record()
        for _ in range(n_packed):
            terra.terra_swin_attn_fwd_packed(desc, qkv, bias, o, lse, ws)
            terra.terra_swin_attn_bwd_packed(desc, qkv, bias, o, lse, d_o, dqkv, dbias, ws)
        b.record()
        barrier()
        terra.terra_swin_check()
        packed_ms = max_over_ranks(a.elapsed_time(b) / n_packed, dev)
        packed = {"value": whole_job_tflops(flops, world, packed_ms), "unit": UNIT, "ms_per_step": packed_ms, "steps": n_packed,
                  "note": "terra_swin_attn_fwd_packed + terra_swin_attn_bwd_packed on qkv / dqkv [B, H, W, 3, heads, d]"}
        del qkv, dqkv
        # restore the outputs of the unpacked step for whatever reads them below
        call_fwd()
        call_bwd()

    # end to end through the C ABI from pinned HOST buffers: every step copies its inputs host -> device, runs, and
    # copies its results device -> host.  Two device buffer sets and three streams, as an application would do
    # it: the H2D copy of step i + 1 and the D2H copy of step i - 1 overlap step i's kernels.
    e2e = None
    if not args.no_e2e:
        in_names, out_names = ("q", "k", "v", "d_o", "bias"), ("o", "lse", "dq", "dk", "dv", "dbias")
        sets = [dict(q=q, k=k, v=v, d_o=d_o, bias=bias, o=o, lse=lse, dq=dq, dk=dk, dv=dv, dbias=dbias)]
        sets.append({n: torch.empty_like(t) for n, t in sets[0].items()})
        host_in = [torch.empty(sets[0][n].shape, dtype=sets[0][n].dtype, pin_memory=True).copy_(sets[0][n]) for n in in_names]
        host_out = [torch.empty(sets[0][n].shape, dtype=sets[0][n].dtype, pin_memory=True) for n in out_names]
        h2d = sum(x.numel() * x.element_size() for x in host_in)
        d2h = sum(x.numel() * x.element_size() for x in host_out)
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

        def run_set(S):
            call_route()
            rc = lib.terra_swin_attn_fwd(ctypes.byref(desc), P(S["q"]), P(S["k"]), P(S["v"]), P(S["bias"]), P(S["o"]), P(S["lse"]),
                                         P(ws), ws.numel(), sp)
            assert rc == 0, rc
            rc = lib.terra_swin_attn_bwd(ctypes.byref(desc), P(S["q"]), P(S["k"]), P(S["v"]), P(S["bias"]), P(S["o"]), P(S["lse"]),
                                         P(S["d_o"]), P(S["dq"]), P(S["dk"]), P(S["dv"]), P(S["dbias"]), P(ws), ws.numel(), sp)
            assert rc == 0, rc

        def e2e_steps(n, first, last):
            ev_c = [torch.cuda.Event() for _ in range(n)]
            ev_o = [torch.cuda.Event() for _ in range(n)]
            first.record(stream)
            s_in.wait_event(first)
            for i in range(n):
                S = sets[i % 2]
                ev_in = torch.cuda.Event()
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_c[i - 2])       # this set's inputs have been consumed
                    for name, src in zip(in_names, host_in):
                        S[name].copy_(src, non_blocking=True)
                    ev_in.record(s_in)
                stream.wait_event(ev_in)
                if i >= 2:
                    stream.wait_event(ev_o[i - 2])         # this set's results have been copied out
                run_set(S)
                ev_c[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_c[i])
                    for dst, name in zip(host_out, out_names):
                        dst.copy_(S[name], non_blocking=True)
                    ev_o[i].record(s_out)
            stream.wait_event(ev_o[n - 1])
            last.record(stream)

        n_e2e = max(4, min(args.steps, 10))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps(2, a, b)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_steps(n_e2e, a, b)
        barrier()
        terra.terra_swin_check()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / n_e2e, dev)
        e2e = {"value": whole_job_tflops(flops, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "note": "pinned host buffers; H2D, kernels and D2H of consecutive steps overlap (two device buffer sets)"}

    if rank == 0:
        peak_tf = peaks["bf16_tflops"]
        peak_bw = peaks["hbm_gbs"]
        sm_count = torch.cuda.get_device_properties(local_rank).multi_processor_count
        # Algorithmic FLOP per launch of each kernel (strict convention, per allowed pair per head):
        # forward 4d (QK^T, PV); one-pass backward 8d (dP, dV, dK, dQ; the recomputed S is not counted); the
        # two-kernel backward paths 4d each (key side: dV, dK; query side: dP, dQ).
        pairs = wk["score_elements"]
        d = cfg.head_dim
        kernel_flop = {"swin_fwd_tc_kernel": 4 * d * pairs, "swin_fwd_tc64_kernel": 4 * d * pairs, "swin_fwd_mma_kernel": 4 * d * pairs,
                       "swin_fwd_small_kernel": 4 * d * pairs,
                       "swin_bwd_fused_kernel": 8 * d * pairs, "swin_bwd_small_kernel": 8 * d * pairs,
                       "swin_bwd_mma_kernel<key tiles>": 4 * d * pairs, "swin_bwd_mma_kernel<query tiles>": 4 * d * pairs,
                       "swin_bwd_kv64_kernel": 4 * d * pairs, "swin_bwd_q64_kernel": 4 * d * pairs,
                       "swin_bwd_kv64_kernel<query side>": 4 * d * pairs,
                       "swin_bwd_delta_kernel": 0}
        kernels = []
        for kname, vals in kernel_ms.items():
            avg = statistics.mean(vals)
            kernels.append({"kernel": kname, "launches": len(vals), "avg_ms": avg,
                            "tflops": kernel_flop.get(kname, 0) / (avg * 1e-3) / 1e12,
                            "dram_bytes_ncu": ncu_traffic(kname, cfg)})
        kernels.sort(key=lambda r: -r["avg_ms"] * r["launches"])
        dom = kernels[0] if kernels else {"kernel": "none", "avg_ms": bwd_ms, "tflops": 0.0, "dram_bytes_ncu": None}
        achieved = dom["tflops"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
            "config": workload_config(cfg, "inputs exceed L2 (4 bf16 tensors of %.0f MB each)" % (wk["tensor_bytes"] / 1e6)),
            "tokens_per_s": world * cfg.tokens / (ms_step * 1e-3),
            "pct_of_bf16_peak": {"of_measured_burst": 100 * value / world / peaks["bf16_tflops"],
                                 "of_measured_sustained": 100 * value / world / peaks["bf16_tflops_sustained"],
                                 "of_nominal_2250": 100 * value / world / 2250.0, "peaks": peak_kind},
            "fa_convention_tflops": world * (wk["flop_fwd"] + wk["flop_bwd_fa"]) / (ms_step * 1e-3) / 1e12,
            "breakdown_ms": {"route": route_ms, "fwd": fwd_ms, "bwd": bwd_ms},
            "fwd_tflops": wk["flop_fwd"] / (fwd_ms * 1e-3) / 1e12,
            "bwd_tflops": wk["flop_bwd"] / (bwd_ms * 1e-3) / 1e12,
            "roofline": {"bound": "tensor", "kernel": dom["kernel"], "avg_ms": dom["avg_ms"],
                         "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved / peak_tf,
                         "traffic": dom["dram_bytes_ncu"], "traffic_source": TRAFFIC_SOURCE if dom["dram_bytes_ncu"] else None,
                         "peak_kind": f"{peak_kind} burst bf16",
                         "note": "dominant kernel by time; achieved = its algorithmic FLOP / its CUDA-event duration"},
            "kernels": kernels,
            "roofline_hbm": {"bound": "hbm", "achieved": (wk["bytes_fwd"] + wk["bytes_bwd"]) / (ms_step * 1e-3) / 1e9,
                             "peak": peak_bw, "unit": "GB/s",
                             "frac": (wk["bytes_fwd"] + wk["bytes_bwd"]) / (ms_step * 1e-3) / 1e9 / peak_bw,
                             "note": "algorithmic bytes of the whole step / step time"},
            # The tcgen05 kernels are limited by the elementwise warps, not by the tensor pipe: one exp2 per
            # (query, key) pair per head on the special-function unit (16 per clock per SM) and about 11 lane
            # instructions per pair (128 lanes per clock per SM) in the dominant kernel.
            "roofline_alu": {"bound": "alu", "kernel": dom["kernel"], "unit": "G pairs/s",
                             "achieved": pairs / (dom["avg_ms"] * 1e-3) / 1e9,
                             "peak_exp_unit": 16 * sm_count * (clocks.get("sm_mhz") or 1965.0) * 1e6 / 1e9,
                             "peak_issue_slots": 128 * sm_count * (clocks.get("sm_mhz") or 1965.0) * 1e6 / 11.0 / 1e9,
                             "note": "peaks derived from unit counts and the sampled SM clock; achieved = allowed pairs of one launch / its duration"},
            "clocks": clocks, "gpu_launches": launches, "e2e": e2e,
        }
        if packed is not None:
            line["packed_qkv"] = packed
        ra = line["roofline_alu"]
        ra["frac_exp_unit"] = ra["achieved"] / ra["peak_exp_unit"]
        ra["frac_issue_slots"] = ra["achieved"] / ra["peak_issue_slots"]
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(cfg)
        elif world > 1:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

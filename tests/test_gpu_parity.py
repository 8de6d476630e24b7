"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import CONFIGS, make_inputs, small_config
from tests._parity import gate, gpu_rows

pytestmark = pytest.mark.gpu

EDGE = [
    # name,            B, H,  W,  heads, d,  w,  sh, sw, ph, pw
    ("tiny_nonperiodic", 2, 8, 8, 2, 32, 4, 2, 2, 0, 0),
    ("tiny_periodic", 1, 8, 12, 1, 32, 4, 1, 3, 1, 1),
    ("ragged_small_rem", 1, 9, 7, 2, 32, 4, 3, 3, 0, 1),       # 0 < H mod w < shift
    ("window_gt_grid", 1, 3, 5, 2, 32, 8, 1, 2, 0, 1),
    ("single_row", 1, 1, 70, 1, 32, 6, 0, 5, 0, 1),
    ("no_shift", 3, 10, 12, 2, 64, 4, 0, 0, 0, 1),
    ("odd_window", 1, 23, 31, 3, 32, 5, 2, 3, 0, 1),
    ("w1", 1, 4, 6, 1, 32, 1, 0, 0, 0, 1),
    ("w32_d32", 1, 40, 70, 1, 32, 32, 16, 16, 0, 1),
    ("w20_d64", 2, 45, 50, 2, 64, 20, 10, 10, 0, 1),
    ("shift_ge_grid", 1, 12, 16, 2, 32, 4, 12 + 2, 16 * 3 + 1, 0, 1),
    ("w12_three_blocks", 2, 30, 40, 3, 32, 12, 6, 6, 0, 1),     # 144-token windows: two key tiles, an odd number of query blocks
    ("w16_wrap_and_rem", 1, 40, 48, 2, 32, 16, 8, 8, 0, 1),      # full, masked (latitude wrap) and truncated 16-wide windows
    ("w8_nonperiodic", 2, 24, 40, 2, 32, 8, 4, 4, 0, 0),         # 64-token windows, masks on both axes, several items per CTA
    # 16-wide windows whose rows are runs of consecutive tokens: the forward fetches them with tiled TMA copies
    ("tma_rows_wrap_lat", 2, 30, 56, 3, 32, 16, 8, 8, 0, 1),     # last column 8 wide, last row 14 high, latitude wrap + mask
    ("tma_nonperiodic", 1, 46, 64, 2, 32, 16, 8, 16, 0, 0),      # masks on both axes
    ("bulk64_w32", 1, 64, 96, 2, 64, 32, 16, 8, 0, 1),           # head dim 64, complete windows: rows by tiled bulk copies
    ("bulk64_w16", 2, 32, 48, 2, 64, 16, 8, 8, 0, 0),
    ("gather64_w32", 1, 64, 64, 2, 64, 32, 12, 20, 0, 0),        # complete windows, shifts not multiples of 8: rows gathered
    # 32-wide complete windows whose latitude shift is no multiple of 4: groups of window rows that would cross the
    # latitude wrap fall back to one bulk copy per window row; the last window column crosses the longitude seam
    ("bulk64_w32_odd_shift", 1, 64, 64, 2, 64, 32, 5, 24, 0, 1),
    ("bulk128_w32_odd_shift", 1, 64, 96, 1, 128, 32, 13, 8, 1, 1),
    ("tma_noshift", 1, 32, 40, 2, 32, 16, 0, 0, 0, 1),
]


def _to_gpu(x):
    return {k: v.cuda() for k, v in x.items()}


def _run_fwd(cfg, xg, scale=0.0):
    d = terra.make_desc(cfg, scale)
    o, lse = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    terra.terra_swin_check()          # synchronises; raises if a kernel gave up on a bounded wait
    return d, o, lse


def _run_bwd(cfg, d, xg, o, lse):
    out = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o, lse, xg["do"])
    terra.terra_swin_check()
    return out


def _check_forward(cfg, x, o, lse, sel, scale=0.0, strict=True):
    ro, rl = oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], x["bias"].double().numpy(), sel=sel, scale=scale)
    tok = oracle.selection_tokens(cfg, sel)
    gate("o", gpu_rows(o, cfg, tok), ro, strict)
    gate("lse", gpu_rows(lse, cfg, tok), rl, strict)


def _check_backward(cfg, x, grads, sel, dbias_ref_is_total, scale=0.0, strict=True):
    dq, dk, dv, dbias = grads
    rq, rk, rv, rb = oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], x["bias"].double().numpy(), sel=sel, scale=scale)
    tok = oracle.selection_tokens(cfg, sel)
    gate("dq", gpu_rows(dq, cfg, tok), rq, strict)
    gate("dk", gpu_rows(dk, cfg, tok), rk, strict)
    gate("dv", gpu_rows(dv, cfg, tok), rv, strict)
    if dbias_ref_is_total:
        gate("dbias", dbias.cpu().double().numpy(), rb, strict)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_route_bit_exact(name):
    cfg = CONFIGS[name]
    got = terra.terra_window_route(terra.make_desc(cfg))
    torch.cuda.synchronize()
    ref = oracle.window_route(cfg)
    for key, val in ref.items():
        assert np.array_equal(got[key].cpu().numpy(), val), key


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_route_bit_exact_edge_cases(case):
    cfg = small_config(*case)
    got = terra.terra_window_route(terra.make_desc(cfg))
    torch.cuda.synchronize()
    ref = oracle.window_route(cfg)
    for key, val in ref.items():
        assert np.array_equal(got[key].cpu().numpy(), val), key


def test_route_null_outputs_are_skipped():
    import ctypes
    cfg = CONFIGS["cfg1"]
    d = terra.make_desc(cfg)
    perm = torch.full((cfg.H * cfg.W,), -1, dtype=torch.int32, device="cuda")
    null = ctypes.c_void_p(0)
    lib = terra.load_library()
    assert lib.terra_window_route(ctypes.byref(d), ctypes.c_void_p(perm.data_ptr()), null, null, null, null, null) == 0
    torch.cuda.synchronize()
    assert np.array_equal(perm.cpu().numpy(), oracle.window_route(cfg)["perm"])


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_edge_cases_forward_backward(case):
    cfg = small_config(*case)
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0          # make the bias matter (std 0.5)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)


def test_explicit_scale_is_used():
    cfg = small_config("scale", 1, 12, 16, 2, 32, 4, 2, 2, 0, 1)
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg, scale=0.05)
    _check_forward(cfg, x, o, lse, None, scale=0.05)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True, scale=0.05)


def test_cfg1_forward_full():
    cfg = CONFIGS["cfg1"]
    x = make_inputs(cfg)
    d, o, lse = _run_fwd(cfg, _to_gpu(x))
    _check_forward(cfg, x, o, lse, None)


@pytest.mark.parametrize("name", ["cfg2", "cfg3"])
def test_full_tensors_forward_backward(name):
    cfg = CONFIGS[name]
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)


def test_cfg4_full_tensors_forward_backward():
    """Config 4 at full size, every one of its 128 windows against the oracle (O, LSE, dQ, dK, dV, dBias)."""
    cfg = CONFIGS["cfg4"]
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)


def test_cfg5_full_size_every_window_in_chunks():
    """Config 5 at full size: ONE forward and ONE backward launch over all 22 630 windows; the oracle then walks
    over the windows in chunks (its fp64 results for the whole problem would not fit in host memory at once).
    Every output row of every chunk is compared, and the oracle's bias gradient, which is additive over
    selections of windows, is summed over the chunks and compared with the launch's full dBias."""
    cfg = CONFIGS["cfg5"]
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    dq, dk, dv, dbias = _run_bwd(cfg, d, xg, o, lse)
    _, nw, _ = oracle.route_sizes(cfg)
    total = cfg.B * nw
    bias64 = x["bias"].double().numpy()
    rb_sum = np.zeros((cfg.bias_rows, cfg.heads))
    n_chunks = 24
    for c in range(n_chunks):
        sel = np.arange(c * total // n_chunks, (c + 1) * total // n_chunks, dtype=np.int64)
        tok = oracle.selection_tokens(cfg, sel)
        ro, rl = oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], bias64, sel=sel)
        gate(f"o[{c}]", gpu_rows(o, cfg, tok), ro)
        gate(f"lse[{c}]", gpu_rows(lse, cfg, tok), rl)
        del ro, rl
        rq, rk, rv, rb = oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], bias64, sel=sel)
        gate(f"dq[{c}]", gpu_rows(dq, cfg, tok), rq)
        gate(f"dk[{c}]", gpu_rows(dk, cfg, tok), rk)
        gate(f"dv[{c}]", gpu_rows(dv, cfg, tok), rv)
        rb_sum += rb
        del rq, rk, rv
    gate("dbias", dbias.cpu().double().numpy(), rb_sum)


# Activations far from N(0, 1): scores of tens to thousands of nats, a bias table with one entry of +200 and a
# wide spread, and grids whose windows mix shift-mask groups and end in truncated windows.  The keys a query may
# not see (the other mask group, slots past the window's extent) then carry scores that exceed every allowed one by
# hundreds of nats: a softmax that takes its maximum over them would underflow to 0 / 0.
LARGE = [
    # name,            B, H,  W,  heads, d,  w,  sh, sw, ph, pw, q/k factor
    ("x8_w16_masks", 1, 40, 56, 2, 32, 16, 8, 8, 0, 0, 8.0),
    ("x32_w16_masks", 1, 40, 56, 2, 32, 16, 8, 8, 0, 0, 32.0),
    ("x8_w14", 2, 37, 45, 3, 32, 14, 7, 7, 0, 1, 8.0),
    ("x32_w8", 1, 24, 40, 2, 32, 8, 4, 4, 0, 0, 32.0),
    ("x8_d64_w32", 1, 70, 80, 2, 64, 32, 16, 16, 0, 0, 8.0),
    ("x32_d64_w32", 1, 70, 80, 2, 64, 32, 16, 16, 0, 0, 32.0),
    ("x8_d64_w20", 1, 45, 50, 2, 64, 20, 10, 10, 0, 1, 8.0),
    ("x8_d128_w32", 1, 64, 64, 1, 128, 32, 16, 16, 0, 0, 8.0),
]


@pytest.mark.parametrize("case", LARGE, ids=[c[0] for c in LARGE])
def test_large_magnitude_scores_and_wide_bias_stay_finite_and_exact(case):
    cfg = small_config(*case[:-1])
    f = case[-1]
    x = make_inputs(cfg)
    x["q"] = (x["q"].float() * f).to(torch.bfloat16)
    x["k"] = (x["k"].float() * f).to(torch.bfloat16)
    x["bias"] = x["bias"] * 25.0
    x["bias"][3, 0] = 200.0                 # one entry far above the rest
    x["bias"][5, :] = -150.0                # and a row far below
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    _check_forward(cfg, x, o, lse, None)
    # backward: the two gates of the tolerance statement.  With nearly one-hot softmax rows dS = P (dP - delta) is
    # the difference of two nearly equal numbers, of which delta is taken from the saved bf16 O, so the tighter
    # diagnostic gate (which budgets only bf16 rounding of the outputs) does not apply here.
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True, strict=False)


def test_outputs_are_reproducible_and_inputs_untouched():
    cfg = CONFIGS["cfg2"]
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    keep = {k: v.clone() for k, v in xg.items()}
    d, o1, l1 = _run_fwd(cfg, xg)
    g1 = _run_bwd(cfg, d, xg, o1, l1)
    d, o2, l2 = _run_fwd(cfg, xg)
    g2 = _run_bwd(cfg, d, xg, o2, l2)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    for a, b in zip(g1[:3], g2[:3]):
        assert torch.equal(a, b)
    for k in xg:
        assert torch.equal(xg[k], keep[k])


def test_alignment_and_workspace_errors():
    cfg = CONFIGS["cfg1"]
    x = _to_gpu(make_inputs(small_config("e", 1, 32, 64, 3, 32, 8, 4, 4)))
    d = terra.make_desc(cfg)
    n = cfg.tokens * cfg.heads * cfg.head_dim
    buf = torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(terra.TerraError) as e:
        terra.terra_swin_attn_fwd(d, buf[1:n + 1], x["k"], x["v"], x["bias"])
    assert e.value.status == 3
    o, lse = terra.terra_swin_attn_fwd(d, x["q"], x["k"], x["v"], x["bias"])
    with pytest.raises(terra.TerraError) as e:
        terra.terra_swin_attn_bwd(d, x["q"], x["k"], x["v"], x["bias"], o, lse, x["do"],
                                  workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 4
    torch.cuda.synchronize()


def test_expired_bounded_wait_is_reported_and_the_context_stays_usable():
    """A kernel wait that nothing satisfies gives up after its cycle limit and the host sees it; afterwards the
    library works as before (no hang, no fault)."""
    terra.terra_swin_check()                       # clean slate
    terra.selftest_bounded_wait(2_000_000)         # about a millisecond of SM clocks
    with pytest.raises(terra.TerraError) as e:
        terra.terra_swin_check()
    assert e.value.status == 6
    terra.terra_swin_check()                       # the word was cleared by the failed check
    cfg = small_config("after", 1, 16, 16, 2, 32, 8, 4, 4)
    x = make_inputs(cfg)
    d, o, lse = _run_fwd(cfg, _to_gpu(x))
    _check_forward(cfg, x, o, lse, None)


def test_side_stream_and_interleaved_shapes_give_the_same_bits():
    """The calls are stream-ordered and keep no state between calls: results on a side stream, and with calls of
    another shape in between (same workspace reused), equal the plain results bit for bit."""
    cfg_a = small_config("sa", 2, 40, 48, 3, 32, 16, 8, 8, 0, 1)
    cfg_b = small_config("sb", 1, 45, 50, 2, 64, 20, 10, 10, 0, 1)          # the other kernel family
    cfg_c = small_config("sc", 1, 30, 44, 5, 32, 14, 7, 7, 0, 0)
    xs = {c.name: _to_gpu(make_inputs(c)) for c in (cfg_a, cfg_b, cfg_c)}
    descs = {c.name: terra.make_desc(c) for c in (cfg_a, cfg_b, cfg_c)}
    need = max(max(terra.terra_swin_workspace_bytes(d, True), terra.terra_swin_workspace_bytes(d, False)) for d in descs.values())
    ws = torch.empty(max(16, need), dtype=torch.uint8, device="cuda")

    def run(name):
        x, d = xs[name], descs[name]
        o, lse = terra.terra_swin_attn_fwd(d, x["q"], x["k"], x["v"], x["bias"], workspace=ws)
        grads = terra.terra_swin_attn_bwd(d, x["q"], x["k"], x["v"], x["bias"], o, lse, x["do"], workspace=ws)
        return (o, lse) + tuple(grads)

    ref = {n: run(n) for n in xs}
    terra.terra_swin_check()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        order = ["sa", "sb", "sc", "sa", "sc", "sb", "sa"]
        outs = [(n, run(n)) for n in order]
    side.synchronize()
    terra.terra_swin_check()
    for n, out in outs:
        names = ("o", "lse", "dq", "dk", "dv", "dbias")
        for nm, a, b in zip(names, out, ref[n]):
            if nm == "dbias" and n == "sb":
                # the register-tile backward sums the bias gradient with atomics: no fixed order
                assert torch.allclose(a, b, rtol=1e-4, atol=1e-5 * float(b.abs().max()))
            else:
                assert torch.equal(a, b), (n, nm)


LATE_MAXIMA = [
    # name,     B, H,  W,  heads, d,  w,  sh, sw, ph, pw
    ("late128", 1, 64, 64, 1, 128, 32, 0, 0, 0, 1),
    ("late64", 1, 64, 96, 2, 64, 32, 16, 8, 0, 1),
    ("late64_ragged", 1, 70, 80, 2, 64, 32, 16, 16, 0, 0),
    ("late128_w16", 1, 32, 48, 2, 128, 16, 8, 8, 0, 1),
]


@pytest.mark.parametrize("case", LATE_MAXIMA, ids=[c[0] for c in LATE_MAXIMA])
def test_forward_when_the_keys_streamed_last_dominate(case):
    """The large-window forward streams the keys once and keeps a running reference for the row maximum: here the keys
    in the lower half of every window are 24 times larger, so the chunks streamed last raise the row maxima by many
    octaves and the accumulated output has to be scaled down on the way (log-sum-exp up to 150 nats)."""
    cfg = small_config(*case)
    x = make_inputs(cfg)
    rows = torch.arange(cfg.H).view(1, cfg.H, 1, 1, 1)
    k = x["k"].float()
    x["k"] = torch.where(((rows - cfg.shift_h) % cfg.window) >= cfg.window // 2, k * 24.0, k).to(torch.bfloat16)
    x["bias"] = x["bias"] * 25.0
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)

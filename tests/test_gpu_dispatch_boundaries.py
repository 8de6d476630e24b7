"""Seeded random shapes (head dim, window side, grid extents complete or ragged, shifts, periodic flags): forward and
backward through the C ABI against the oracle.  The shapes cross every dispatch boundary of the library (windows of at
most 64 tokens, the small-window and the chunked tcgen05 kernels, bulk-copy and gathering loaders, register tiles)."""
import random

import pytest

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import make_inputs, small_config
from tests._parity import gate, gpu_rows

pytestmark = pytest.mark.gpu


def _random_config(rng, i):
    d = rng.choice([32, 64, 128, 128])
    w = rng.choice([4, 7, 8, 8, 12, 16, 16, 20, 32, 32])
    if rng.random() < 0.5:                                   # a grid of complete windows
        H, W = w * rng.randint(1, 3), w * rng.randint(1, 3)
    else:
        H, W = rng.randint(max(2, w // 2), 2 * w + 5), rng.randint(max(2, w // 2), 2 * w + 9)
    if H * W > 6000:
        H = max(2, 6000 // W)
    heads, B = rng.randint(1, 3), rng.randint(1, 2)
    sh = rng.choice([0, w // 2, rng.randint(0, w - 1), 8 * rng.randint(0, 3)]) % max(1, min(w, H))
    sw = rng.choice([0, w // 2, rng.randint(0, w - 1), 8 * rng.randint(0, 3)]) % max(1, min(w, W))
    return small_config(f"random{i}", B, H, W, heads, d, w, sh, sw, rng.randint(0, 1), rng.randint(0, 1))


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_forward_backward(seed):
    rng = random.Random(seed)
    for i in range(30):
        cfg = _random_config(rng, i)
        x = make_inputs(cfg)
        x["bias"] = x["bias"] * 25.0
        xg = {k: v.cuda() for k, v in x.items()}
        d = terra.make_desc(cfg)
        o, lse = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
        dq, dk, dv, dbias = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o, lse, xg["do"])
        terra.terra_swin_check()
        table = x["bias"].double().numpy()
        ro, rl = oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], table)
        rq, rk, rv, rb = oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], table)
        tok = oracle.selection_tokens(cfg, None)
        shape = f"B={cfg.B} H={cfg.H} W={cfg.W} heads={cfg.heads} d={cfg.head_dim} w={cfg.window}"
        for name, got, ref in (("o", gpu_rows(o, cfg, tok), ro), ("lse", gpu_rows(lse, cfg, tok), rl),
                               ("dq", gpu_rows(dq, cfg, tok), rq), ("dk", gpu_rows(dk, cfg, tok), rk),
                               ("dv", gpu_rows(dv, cfg, tok), rv), ("dbias", dbias.cpu().double().numpy(), rb)):
            gate(f"{shape} {name}", got, ref, strict=False)

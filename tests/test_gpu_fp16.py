"""fp16 activations and gradients (the paper trains in fp16 mixed precision, Section VII-A) through the C ABI against
the oracle, which receives the same fp16 values widened to fp64."""
import pytest
import torch

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import make_inputs, small_config
from tests._parity import gate, gpu_rows

pytestmark = pytest.mark.gpu

SHAPES = [
    # name,          B, H,  W,  heads, d,  w,  sh, sw, ph, pw
    ("f16_d32_w8", 2, 24, 40, 2, 32, 8, 4, 4, 0, 0),
    ("f16_d32_w16", 1, 40, 48, 3, 32, 16, 8, 8, 0, 1),
    ("f16_d64_w32", 1, 64, 96, 2, 64, 32, 16, 16, 0, 1),
    ("f16_d64_w20_ragged", 1, 45, 50, 2, 64, 20, 10, 10, 0, 1),
    ("f16_d128_w8", 1, 30, 44, 2, 128, 8, 4, 4, 0, 1),
    ("f16_d128_w32", 1, 40, 70, 1, 128, 32, 16, 16, 0, 0),
    # grids of complete windows: the bulk-copy loaders and the tcgen05 query side of the fp16 builds
    ("f16_d128_w32_complete", 1, 64, 64, 1, 128, 32, 16, 16, 0, 1),
    ("f16_d32_w16_complete", 2, 32, 64, 3, 32, 16, 8, 0, 0, 1),
    ("f16_d64_w16_complete", 1, 32, 48, 2, 64, 16, 8, 8, 0, 0),
    ("f16_d128_w64_complete", 1, 64, 128, 2, 128, 64, 16, 40, 0, 0),  # staged bias rows; query side by exchanged roles
    ("f16_d32_w12", 1, 40, 62, 2, 32, 12, 6, 6, 0, 1),                # 16 slots per window row, full-width and truncated windows
]


@pytest.mark.parametrize("case", SHAPES, ids=[c[0] for c in SHAPES])
def test_fp16_forward_backward(case):
    cfg = small_config(*case)
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0
    for name in ("q", "k", "v", "do"):
        x[name] = x[name].to(torch.float16)
    xg = {k: v.cuda() for k, v in x.items()}
    d = terra.make_desc(cfg, dtype=torch.float16)
    o, lse = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    assert o.dtype == torch.float16
    dq, dk, dv, dbias = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o, lse, xg["do"])
    terra.terra_swin_check()
    bias64 = x["bias"].double().numpy()
    ro, rl = oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], bias64)
    rq, rk, rv, rb = oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], bias64)
    tok = oracle.selection_tokens(cfg, None)
    for name, got, ref in (("o", gpu_rows(o, cfg, tok), ro), ("lse", gpu_rows(lse, cfg, tok), rl),
                           ("dq", gpu_rows(dq, cfg, tok), rq), ("dk", gpu_rows(dk, cfg, tok), rk),
                           ("dv", gpu_rows(dv, cfg, tok), rv), ("dbias", dbias.cpu().double().numpy(), rb)):
        gate(name, got, ref)


def test_fp16_descriptor_refuses_bf16_tensors_and_the_other_way_round():
    cfg = small_config("f16_types", 1, 16, 16, 2, 32, 8, 4, 4)
    x = {k: v.cuda() for k, v in make_inputs(cfg).items()}
    with pytest.raises(ValueError):
        terra.terra_swin_attn_fwd(terra.make_desc(cfg, dtype=torch.float16), x["q"], x["k"], x["v"], x["bias"])
    h = {k: (v.to(torch.float16) if v.dtype == torch.bfloat16 else v) for k, v in x.items()}
    with pytest.raises(ValueError):
        terra.terra_swin_attn_fwd(terra.make_desc(cfg), h["q"], h["k"], h["v"], h["bias"])

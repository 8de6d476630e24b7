"""Head dim 128, the per-head width of every model in the paper's Table V (1024 / 8, 4096 / 32, 8192 / 64 channels per
heads), with the window sides those models use (8 and 32): the CUDA path through the C ABI against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import CONFIGS, make_inputs, small_config
from tests._parity import gate, gpu_rows
from tests.test_gpu_parity import _check_backward, _check_forward, _run_bwd, _run_fwd, _to_gpu

pytestmark = pytest.mark.gpu

SHAPES = [
    # name,          B, H,  W,  heads, d,  w,  sh, sw, ph, pw
    ("d128_w8", 2, 24, 40, 2, 128, 8, 4, 4, 0, 1),
    ("d128_w8_masks", 1, 30, 44, 3, 128, 8, 4, 4, 0, 0),            # truncated on both axes, masks on both axes
    ("d128_w32", 1, 64, 96, 2, 128, 32, 16, 16, 0, 1),
    ("d128_w32_ragged", 1, 70, 45, 1, 128, 32, 20, 30, 0, 0),       # 13-wide last column, 6-high last row
    ("d128_w5", 1, 23, 31, 2, 128, 5, 2, 3, 0, 1),
    ("d128_w16_noshift", 1, 40, 48, 2, 128, 16, 0, 0, 0, 1),
    # complete windows and a longitude shift that is a multiple of 8: rows arrive by tiled bulk copies
    ("d128_w16_bulk", 1, 32, 48, 2, 128, 16, 8, 8, 0, 1),
    ("d128_w32_bulk_shift24", 1, 64, 64, 1, 128, 32, 8, 24, 0, 0),  # seam after 8 of a row's 32 tokens, masks on both axes
    ("d128_w32_bulk_noshift", 2, 32, 64, 2, 128, 32, 0, 0, 0, 1),
    # complete windows whose shifts are not multiples of 8: every row is gathered with 16-byte copies
    ("d128_w32_gather", 1, 64, 64, 1, 128, 32, 12, 12, 0, 1),
]


@pytest.mark.parametrize("case", SHAPES, ids=[c[0] for c in SHAPES])
def test_head_dim_128_forward_backward(case):
    cfg = small_config(*case)
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0          # make the bias matter (std 0.5)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)


def test_table_v_small_model_shape_full_tensors():
    """The small model's attention block at full size (288 x 544 tokens, 8 heads x 128, window 8): every output against
    the oracle."""
    cfg = CONFIGS["tv_small"]
    x = make_inputs(cfg)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)


def test_packed_qkv_head_dim_128_matches_the_separate_tensors():
    cfg = small_config("d128_packed", 1, 24, 40, 2, 128, 8, 4, 4, 0, 1)
    xg = _to_gpu(make_inputs(cfg))
    d = terra.make_desc(cfg)
    o, lse = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    dq, dk, dv, _ = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o, lse, xg["do"])
    qkv = torch.stack([xg["q"], xg["k"], xg["v"]], dim=3).contiguous()
    o2, lse2 = terra.terra_swin_attn_fwd_packed(d, qkv, xg["bias"])
    dqkv, _ = terra.terra_swin_attn_bwd_packed(d, qkv, xg["bias"], o2, lse2, xg["do"])
    terra.terra_swin_check()
    assert torch.equal(o, o2) and torch.equal(lse, lse2)
    for i, g in enumerate((dq, dk, dv)):
        assert torch.equal(dqkv[:, :, :, i], g)

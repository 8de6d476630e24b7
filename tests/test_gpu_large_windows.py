"""Windows of 64 and 128 tokens per side (4096 and 16 384 tokens per window), the sizes of the paper's window-assignment
study (Section VII-E), and sides between 32 and 128 in general: the CUDA path through the C ABI against the oracle."""
import pytest

from paper_2608_15211_b200.workloads import make_inputs, small_config
from tests.test_gpu_parity import _check_backward, _check_forward, _run_bwd, _run_fwd, _to_gpu

pytestmark = pytest.mark.gpu

SHAPES = [
    # name,             B, H,   W,   heads, d,  w,   sh, sw, ph, pw
    ("w64_d32_ragged", 1, 70, 130, 2, 32, 64, 32, 32, 0, 1),        # rows 64 + 6, columns 64 + 64 + 2, latitude mask
    ("w64_d64_masks", 1, 64, 128, 1, 64, 64, 20, 30, 0, 0),          # complete windows, masks on both axes
    ("w40_d32", 2, 50, 90, 2, 32, 40, 20, 20, 0, 1),                 # a side that is no multiple of 32
    ("w128_d32", 1, 130, 140, 1, 32, 128, 64, 64, 0, 1),             # one complete 128 x 128 window and three truncated ones
    ("w128_d128_one_window", 1, 128, 128, 1, 128, 128, 0, 0, 1, 1),  # 16 384 tokens, head dim 128
    # complete windows with a longitude shift that is a multiple of 8: the forward kernel that stages bias-table rows
    ("w64_d64_complete", 1, 128, 192, 2, 64, 64, 32, 40, 0, 1),      # latitude mask, rows that wrap around the seam
    ("w64_d128_complete", 2, 64, 128, 2, 128, 64, 16, 8, 0, 0),      # masks on both axes
    ("w128_d64_complete", 1, 128, 128, 2, 64, 128, 40, 16, 0, 0),
    ("w128_d128_masked", 1, 128, 256, 1, 128, 128, 64, 72, 0, 1),    # two windows, latitude mask, seam
]


@pytest.mark.parametrize("case", SHAPES, ids=[c[0] for c in SHAPES])
def test_large_window_forward_backward(case):
    cfg = small_config(*case)
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0          # make the bias matter (std 0.5)
    xg = _to_gpu(x)
    d, o, lse = _run_fwd(cfg, xg)
    _check_forward(cfg, x, o, lse, None)
    grads = _run_bwd(cfg, d, xg, o, lse)
    _check_backward(cfg, x, grads, None, True)

"""Packed-QKV entry points: the same kernels reading q, k, v as the three slots of one [B, H, W, 3, heads, d] tensor
and writing dq, dk, dv into the slots of another.  Checked against the oracle, and bit for bit against the calls on
separate tensors (same kernels, same arithmetic, only the addresses differ)."""
import pytest
import torch

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import CONFIGS, make_inputs, small_config
from tests._parity import gate, gpu_rows

pytestmark = pytest.mark.gpu

CASES = [
    small_config("packed_w16", 1, 40, 48, 2, 32, 16, 8, 8, 0, 1),      # tcgen05 kernels: full, masked and truncated windows
    small_config("packed_w8", 2, 24, 40, 3, 32, 8, 4, 4, 0, 0),        # tcgen05 kernels, several items per CTA
    small_config("packed_w14", 1, 45, 50, 2, 32, 14, 7, 7, 0, 1),      # generic table addressing
    small_config("packed_d64", 1, 45, 50, 2, 64, 20, 10, 10, 0, 1),    # register-tile kernels
    small_config("packed_d64_w32", 1, 64, 64, 2, 64, 32, 16, 16, 0, 1),  # chunked tcgen05 kernels, complete windows
    small_config("packed_noshift", 1, 32, 32, 2, 32, 16, 0, 0, 0, 1),  # the unshifted W-MSA sibling of the block
    small_config("packed_d64_w64", 1, 64, 128, 2, 64, 64, 32, 24, 0, 1),  # chunked tcgen05 kernels with staged bias rows
]


@pytest.mark.parametrize("cfg", CASES, ids=[c.name for c in CASES])
def test_packed_calls_match_the_oracle_and_the_unpacked_calls(cfg):
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0
    xg = {k: v.cuda() for k, v in x.items()}
    d = terra.make_desc(cfg)
    qkv = torch.stack([xg["q"], xg["k"], xg["v"]], dim=3).contiguous()          # [B, H, W, 3, heads, d]
    o, lse = terra.terra_swin_attn_fwd_packed(d, qkv, xg["bias"])
    dqkv, dbias = terra.terra_swin_attn_bwd_packed(d, qkv, xg["bias"], o, lse, xg["do"])
    terra.terra_swin_check()
    o2, lse2 = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    dq2, dk2, dv2, dbias2 = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o2, lse2, xg["do"])
    terra.terra_swin_check()
    assert torch.equal(o, o2) and torch.equal(lse, lse2)
    assert torch.equal(dqkv[:, :, :, 0], dq2) and torch.equal(dqkv[:, :, :, 1], dk2) and torch.equal(dqkv[:, :, :, 2], dv2)
    assert torch.equal(qkv[:, :, :, 0], xg["q"])                                 # inputs untouched
    bias64 = x["bias"].double().numpy()
    ro, rl = oracle.attn_fwd(cfg, x["q"], x["k"], x["v"], bias64)
    rq, rk, rv, rb = oracle.attn_bwd(cfg, x["q"], x["k"], x["v"], x["do"], bias64)
    tok = oracle.selection_tokens(cfg, None)
    for name, got, ref in (("o", gpu_rows(o, cfg, tok), ro), ("lse", gpu_rows(lse, cfg, tok), rl),
                           ("dq", gpu_rows(dqkv[:, :, :, 0].contiguous(), cfg, tok), rq),
                           ("dk", gpu_rows(dqkv[:, :, :, 1].contiguous(), cfg, tok), rk),
                           ("dv", gpu_rows(dqkv[:, :, :, 2].contiguous(), cfg, tok), rv),
                           ("dbias", dbias.cpu().double().numpy(), rb)):
        gate(name, got, ref, strict=False)
    if cfg.head_dim == 32 and 8 < cfg.window <= 16:
        assert torch.equal(dbias, dbias2)            # fixed summation order on the tcgen05 path (windows of more than 64 tokens)


def test_packed_full_size_config3_runs_at_the_same_speed():
    """Config 3 in the packed layout: outputs equal the unpacked run bit for bit; the kernels' times are reported."""
    cfg = CONFIGS["cfg3"]
    x = make_inputs(cfg)
    xg = {k: v.cuda() for k, v in x.items()}
    d = terra.make_desc(cfg)
    qkv = torch.stack([xg["q"], xg["k"], xg["v"]], dim=3).contiguous()
    o, lse = terra.terra_swin_attn_fwd_packed(d, qkv, xg["bias"])
    dqkv, dbias = terra.terra_swin_attn_bwd_packed(d, qkv, xg["bias"], o, lse, xg["do"])
    o2, lse2 = terra.terra_swin_attn_fwd(d, xg["q"], xg["k"], xg["v"], xg["bias"])
    dq2, dk2, dv2, dbias2 = terra.terra_swin_attn_bwd(d, xg["q"], xg["k"], xg["v"], xg["bias"], o2, lse2, xg["do"])
    terra.terra_swin_check()
    assert torch.equal(o, o2) and torch.equal(lse, lse2) and torch.equal(dbias, dbias2)
    assert torch.equal(dqkv[:, :, :, 0], dq2) and torch.equal(dqkv[:, :, :, 1], dk2) and torch.equal(dqkv[:, :, :, 2], dv2)

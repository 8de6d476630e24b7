"""Complete-window ("padded") mode (Section IV-B, Eq. 3): activations padded with zero tokens to a grid that the window
side divides, attention on the padded grid, results cropped back.  The padded tokens are ordinary tokens there, so the
reference is the oracle on the padded configuration with the padded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import make_inputs, small_config
from tests._parity import gate

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", [("pad_w16", 2, 45, 70, 2, 32, 16, 8, 8, 0, 1), ("pad_w8_d128", 1, 30, 43, 2, 128, 8, 4, 4, 0, 1)],
                         ids=["w16", "w8_d128"])
def test_padded_mode_matches_the_oracle_on_the_padded_grid(case):
    cfg = small_config(*case)
    Hp, Wp = terra.padded_extent(cfg.H, cfg.window), terra.padded_extent(cfg.W, cfg.window)
    assert (Hp, Wp) != (cfg.H, cfg.W)
    cfg_p = dataclasses.replace(cfg, H=Hp, W=Wp, name=cfg.name + "_padded")
    x = make_inputs(cfg)
    x["bias"] = x["bias"] * 25.0
    xg = {k: v.cuda() for k, v in x.items()}
    pad = {n: terra.terra_pad_grid(xg[n], Hp, Wp) for n in ("q", "k", "v", "do")}
    # the padding kernel against a plain tensor construction
    for n in pad:
        ref = torch.zeros_like(pad[n])
        ref[:, :cfg.H, :cfg.W] = xg[n]
        assert torch.equal(pad[n], ref)
    d = terra.make_desc(cfg_p)
    o, lse = terra.terra_swin_attn_fwd(d, pad["q"], pad["k"], pad["v"], xg["bias"])
    dq, dk, dv, dbias = terra.terra_swin_attn_bwd(d, pad["q"], pad["k"], pad["v"], xg["bias"], o, lse, pad["do"])
    terra.terra_swin_check()
    o_c = terra.terra_crop_grid(o, cfg.H, cfg.W)
    assert torch.equal(o_c, o[:, :cfg.H, :cfg.W])
    xp = {n: pad[n].cpu() for n in pad}
    bias64 = x["bias"].double().numpy()
    ro, rl = oracle.attn_fwd(cfg_p, xp["q"], xp["k"], xp["v"], bias64)
    rq, rk, rv, rb = oracle.attn_bwd(cfg_p, xp["q"], xp["k"], xp["v"], xp["do"], bias64)
    crop = lambda t: oracle.to_grid(cfg_p, t)[:, :cfg.H, :cfg.W]
    gate("o", o_c.float().cpu().numpy(), crop(ro))
    gate("lse", terra.terra_crop_grid(lse, cfg.H, cfg.W).cpu().numpy(), crop(rl))
    for name, got, ref in (("dq", dq, rq), ("dk", dk, rk), ("dv", dv, rv)):
        gate(name, terra.terra_crop_grid(got, cfg.H, cfg.W).float().cpu().numpy(), crop(ref))
    gate("dbias", dbias.cpu().double().numpy(), rb)
    # and it is a different function from the truncated mode: the padded zero tokens take part in the softmax
    o_t, _ = terra.terra_swin_attn_fwd(terra.make_desc(cfg), xg["q"], xg["k"], xg["v"], xg["bias"])
    assert not torch.allclose(o_t.float(), o_c.float(), atol=1e-2)

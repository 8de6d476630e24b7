"""The forward entry point that allocates nothing, against the regular forward entry point.

Some embedders may not request device memory at all (their buffers come from a pool they do not control, or
they run inside a loop that received all its memory up front), so they cannot supply the forward kernel's
workspace.  `terra_swin_attn_fwd_noalloc` keeps that scratch in a fixed array inside the library.  This test
calls it through the C ABI twice in a row, with different bias tables and head counts so that the second call
has to rewrite what the first left in the shared scratch, and compares each result with the regular entry
point on the same inputs: bit for bit where both run the same kernel (head dim 32, window <= 16), through the
tolerance gates otherwise.  "Allocates nothing" is checked on the device itself: after one warm-up call per
device (which is where the library's array becomes resident) the free device memory reported by the driver
must not drop across further calls; PyTorch's own counter would not see an allocation made inside the library.
It runs last (file name) so that a run that stops at the first failure has already executed every other test;
it also passes on its own in a fresh process.
"""
import ctypes

import pytest
import torch

import paper_2608_15211_b200 as terra
from paper_2608_15211_b200.workloads import make_inputs, small_config
from tests._parity import gate

pytestmark = pytest.mark.gpu


def _call_noalloc(d, x, o, lse):
    rc = terra.load_library().terra_swin_attn_fwd_noalloc(
        ctypes.byref(d), *(ctypes.c_void_p(t.data_ptr()) for t in (x["q"], x["k"], x["v"], x["bias"], o, lse)),
        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert rc == 0, terra.load_library().terra_strerror(rc)
    terra.terra_swin_check()


def _both_paths(cfg, extra):
    x = {k: v.cuda() for k, v in make_inputs(cfg, extra=extra).items()}
    x["bias"] = x["bias"] * 25.0
    d = terra.make_desc(cfg)
    o_ref, lse_ref = terra.terra_swin_attn_fwd(d, x["q"], x["k"], x["v"], x["bias"])
    o = torch.full_like(o_ref, float("nan"))
    lse = torch.full_like(lse_ref, float("nan"))
    _call_noalloc(d, x, o, lse)                         # warm-up: the first call on a device may make the array resident
    o.fill_(float("nan"))
    lse.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()          # the driver's count of free bytes: sees every kind of allocation
    mine_before = torch.cuda.memory_allocated()
    _call_noalloc(d, x, o, lse)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == mine_before  # this test itself allocated nothing in between ...
    assert free_after >= free_before, (free_before, free_after)   # ... so a drop would be the library's doing
    return (o, lse), (o_ref, lse_ref)


def test_noalloc_forward_matches_regular_forward_twice_in_a_row():
    # first call: 12 heads, window 16 (ragged grid, latitude mask); second call: 5 heads, window 8, other values
    for cfg, extra in ((small_config("na1", 1, 45, 70, 12, 32, 16, 8, 8), 1),
                       (small_config("na2", 2, 30, 40, 5, 32, 8, 4, 4), 2)):
        (o, lse), (o_ref, lse_ref) = _both_paths(cfg, extra)
        # the same kernel on the same inputs: stale contents of the shared scratch would show as different bits
        assert torch.equal(o, o_ref)
        assert torch.equal(lse, lse_ref)


def test_noalloc_forward_on_a_shape_without_scratch_and_its_limit():
    cfg = small_config("na3", 1, 40, 70, 2, 64, 20, 10, 10)         # head dim 64: the kernel needs no scratch
    (o, lse), (o_ref, lse_ref) = _both_paths(cfg, 3)
    gate("o", o.float().cpu().numpy(), o_ref.float().cpu().numpy())
    gate("lse", lse.cpu().numpy(), lse_ref.cpu().numpy())
    big = small_config("na4", 1, 16, 16, 65, 32, 16, 8, 8)            # one head more than the fixed scratch holds
    x = {k: v.cuda() for k, v in make_inputs(big).items()}
    d = terra.make_desc(big)
    o = torch.empty_like(x["q"])
    lse = torch.empty((big.B, big.H, big.W, big.heads), dtype=torch.float32, device="cuda")
    with pytest.raises(terra.TerraError) as e:
        terra.terra_swin_attn_fwd_noalloc(d, x["q"], x["k"], x["v"], x["bias"], o, lse)
    assert e.value.status == 7

"""Helpers of the GPU parity tests: tolerance gates and oracle-side gathering."""
import numpy as np
import torch

# Gates for bf16 outputs against the fp64 oracle (stated by the benchmark spec for this path):
#   G1  max |err| <= 2e-2 * max |ref|
#   G2  |err_i| <= 2e-2 * max |ref| + 3e-2 * |ref_i|  for every element
# G3 is a tighter diagnostic with the absolute term at 4e-3 * max |ref|: bf16 rounding of an output of
# magnitude max|ref| alone is up to 2e-3 * max|ref|, so this leaves a factor two for the bf16 P / dS operands.
G1_ABS, G2_REL, G3_ABS = 2e-2, 3e-2, 4e-3


def gate(name, got, ref, strict=True):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), f"{name}: non-finite values in the GPU result"
    err = np.abs(got - ref)
    if np.abs(ref).max() < 1e-9:
        # structurally zero reference (single-token windows: dQ = dK = 0).  The GPU value is the rounding
        # residue of dP - delta, where delta uses the saved bf16 O: |dO| |O| 2^-9 |k| scale ~ 1e-2 for N(0, 1) inputs
        assert err.max() <= 2e-2, f"{name}: zero reference, |got| up to {err.max():.3e}"
        return float(err.max())
    scale = np.abs(ref).max()
    assert err.max() <= G1_ABS * scale, f"{name}: G1 max|err| {err.max():.3e} > {G1_ABS * scale:.3e}"
    assert np.all(err <= G1_ABS * scale + G2_REL * np.abs(ref)), f"{name}: G2 failed"
    if strict:
        bad = err > G3_ABS * scale + G2_REL * np.abs(ref)
        assert not bad.any(), f"{name}: G3 failed on {bad.sum()} of {bad.size} (max err {err.max():.3e}, scale {scale:.3e})"
    return float(err.max() / scale) if scale > 0 else 0.0


def gpu_rows(t, cfg, tokens):
    """Rows of a grid-layout GPU tensor [B, H, W, heads, ...] at flat token indices, as float64 numpy."""
    flat = t.reshape(cfg.B * cfg.H * cfg.W, *t.shape[3:])
    idx = torch.from_numpy(np.asarray(tokens)).to(t.device)
    return flat[idx].float().cpu().double().numpy()

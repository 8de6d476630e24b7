"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
and rejects bad descriptors before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2608_15211_b200 as terra
from paper_2608_15211_b200 import binding
from paper_2608_15211_b200.build import build
from paper_2608_15211_b200.workloads import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build()
    return binding.load_library()


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(terra_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared_symbols()
    assert {"terra_window_route", "terra_swin_attn_fwd", "terra_swin_attn_bwd"} <= declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared >= set(binding.EXPORTS)


@pytest.mark.parametrize("name,expect", [
    ("cfg1", (2048, 32, 64)), ("cfg2", (32768, 512, 64)), ("cfg3", (550800, 2176, 256)),
    ("cfg4", (131072, 128, 1024)), ("cfg5", (2203200, 11315, 196)),
])
def test_route_sizes(lib, name, expect):
    assert terra.terra_route_sizes(terra.make_desc(CONFIGS[name])) == expect


def test_workspace_sizes(lib):
    cfg = CONFIGS["cfg3"]
    d = terra.make_desc(cfg)
    assert terra.terra_swin_workspace_bytes(d, False) >= cfg.heads * 8192     # prepared bias tables
    assert terra.terra_swin_workspace_bytes(terra.make_desc(CONFIGS["cfg4"]), False) >= CONFIGS["cfg4"].heads * 6048 * 4    # tables for window side 32
    assert terra.terra_swin_workspace_bytes(d, True) >= cfg.tokens * cfg.heads * 4


def _desc(**kw):
    base = dict(B=1, H=8, W=8, heads=2, head_dim=32, window=4, shift_h=2, shift_w=2, periodic_h=0, periodic_w=1)
    base.update(kw)
    return terra.terra_swin_desc(*[base[k] for k in ("B", "H", "W", "heads", "head_dim", "window", "shift_h",
                                                     "shift_w", "periodic_h", "periodic_w")], 0.0)


@pytest.mark.parametrize("kw,status", [
    (dict(H=0), 1), (dict(B=-1), 1), (dict(window=0), 1), (dict(shift_w=-1), 1), (dict(heads=0), 1),
    (dict(H=70000, W=70000), 1),
])
def test_bad_descriptor_is_rejected_on_the_host(lib, kw, status):
    with pytest.raises(terra.TerraError) as e:
        terra.terra_route_sizes(_desc(**kw))
    assert e.value.status == status


@pytest.mark.parametrize("kw", [dict(head_dim=48), dict(head_dim=256), dict(window=129)])
def test_unsupported_shapes(lib, kw):
    with pytest.raises(terra.TerraError) as e:
        terra.terra_swin_workspace_bytes(_desc(**kw), True)
    assert e.value.status == 2


def test_null_pointers_are_rejected_before_any_launch(lib):
    d = _desc()
    null = ctypes.c_void_p(0)
    before = terra.launch_count()
    rc = lib.terra_swin_attn_fwd(ctypes.byref(d), null, null, null, null, null, null, null, 0, null)
    assert rc == 1
    rc = lib.terra_swin_attn_bwd(ctypes.byref(d), *([null] * 11), null, 0, null)
    assert rc == 1
    assert lib.terra_swin_attn_fwd(None, null, null, null, null, null, null, null, 0, null) == 1
    assert terra.launch_count() == before
    assert b"invalid" in lib.terra_strerror(1)
    assert lib.terra_strerror(99) == b"unknown status"


def test_binding_refuses_cpu_tensors(lib):
    import torch
    cfg = CONFIGS["cfg1"]
    x = torch.zeros(cfg.B, cfg.H, cfg.W, cfg.heads, cfg.head_dim, dtype=torch.bfloat16)
    t = torch.zeros(cfg.bias_rows, cfg.heads)
    with pytest.raises(ValueError):
        terra.terra_swin_attn_fwd(terra.make_desc(cfg), x, x, x, t, o=x.clone(), lse=torch.zeros(cfg.B, cfg.H, cfg.W, cfg.heads))


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "absent.so"))

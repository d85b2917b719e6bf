"""Host-side checks of the C ABI that need no GPU: the library loads, exports every function
the header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest
import torch

from paper_2006_16668_b200 import CONFIGS
from paper_2006_16668_b200 import binding as B
from paper_2006_16668_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gshard_moe.h")


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_library()


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gshard_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert "gshard_moe_top2_forward" in names and "gshard_moe_top2_backward" in names
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in the header but not exported"
        assert n in B.EXPORTS, f"{n} has no Python binding"
    assert sorted(B.EXPORTS) == names


def test_version_and_status_strings():
    assert B.load().gshard_version() >= 100
    assert B.status_string(B.GSHARD_OK) == "ok"
    assert "workspace" in B.status_string(B.GSHARD_ERR_WORKSPACE_TOO_SMALL)
    assert B.status_string(12345) == "unknown status"


def test_workspace_sizes_for_the_paper_configs():
    for name, cfg in CONFIGS.items():
        shape = B.make_shape(cfg)
        fwd = B.gshard_moe_top2_workspace_bytes(shape)
        bwd = B.gshard_moe_top2_workspace_bytes(shape, True)
        ctx = B.gshard_moe_top2_context_bytes(shape)
        stg = B.gshard_moe_top2_host_staging_bytes(shape)
        es = 4 if cfg.dtype == "f32" else 2
        R = cfg.E * cfg.G * cfg.C
        # at least the dispatched inputs, hidden activations and expert outputs
        assert fwd >= R * (2 * cfg.M + cfg.H) * es
        assert ctx >= R * (cfg.M + cfg.H) * es
        assert stg >= 2 * cfg.N * cfg.M * es
        assert bwd > 0 and fwd % 256 == 0
    # MoE(2048E): everything (weights + scratch) must fit one B200 with room to spare
    c4 = CONFIGS["c4_2048e"]
    total = 2 * c4.E * c4.M * c4.H * 2 + B.gshard_moe_top2_workspace_bytes(B.make_shape(c4))
    assert total < 120e9


@pytest.mark.parametrize("kw,code", [
    (dict(G=0), B.GSHARD_ERR_INVALID_ARG), (dict(E=1), B.GSHARD_ERR_INVALID_ARG),
    (dict(C=0), B.GSHARD_ERR_INVALID_ARG), (dict(M=20), B.GSHARD_ERR_UNSUPPORTED_SHAPE),
    (dict(S=40000), B.GSHARD_ERR_UNSUPPORTED_SHAPE), (dict(E=20000), B.GSHARD_ERR_UNSUPPORTED_SHAPE),
    (dict(dtype="bf16", M=72), B.GSHARD_ERR_UNSUPPORTED_SHAPE),
    (dict(flags=131072), B.GSHARD_ERR_INVALID_ARG),
    # more (group, 128-token tile) pairs, or 64-row tiles of the CUDA-core GEMM, than a grid's y extent
    (dict(G=70000, S=1), B.GSHARD_ERR_UNSUPPORTED_SHAPE), (dict(G=600, S=16384), B.GSHARD_ERR_UNSUPPORTED_SHAPE),
    (dict(flags=B.GSHARD_FLAG_FUSED_FFN | B.GSHARD_FLAG_UNFUSED_FFN), B.GSHARD_ERR_INVALID_ARG),
])
def test_bad_shapes_are_rejected(kw, code):
    base = dict(G=2, S=64, M=64, H=256, E=16, C=16, dtype="f32", flags=0)
    base.update(kw)
    shape = B.make_shape(**base)
    assert B.gshard_moe_top2_workspace_bytes(shape) == 0
    fake = 0x10000
    rc = B.load().gshard_moe_top2_forward(ctypes.byref(shape), fake, fake, fake, fake, fake, fake, fake, None,
                                          None, fake, 1 << 40, None)
    assert rc == code


def test_bad_pointers_and_short_workspace():
    shape = B.make_shape(CONFIGS["c1_tiny"])
    need = B.gshard_moe_top2_workspace_bytes(shape)
    fake = 0x10000
    f = B.load().gshard_moe_top2_forward
    args = [fake] * 7
    assert f(ctypes.byref(shape), *args, None, None, fake, need - 1, None) == B.GSHARD_ERR_WORKSPACE_TOO_SMALL
    for i in range(7):
        bad = list(args)
        bad[i] = None
        assert f(ctypes.byref(shape), *bad, None, None, fake, need, None) == B.GSHARD_ERR_INVALID_ARG
    misaligned = list(args)
    misaligned[0] = fake + 4
    assert f(ctypes.byref(shape), *misaligned, None, None, fake, need, None) == B.GSHARD_ERR_INVALID_ARG
    assert f(ctypes.byref(shape), *args, None, None, fake + 16, need, None) == B.GSHARD_ERR_INVALID_ARG
    assert f(None, *args, None, None, fake, need, None) == B.GSHARD_ERR_INVALID_ARG
    # save-for-backward without a context buffer, or with one that is not 256-byte aligned
    shape_s = B.make_shape(CONFIGS["c1_tiny"], flags=B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
    assert B.load().gshard_moe_top2_backward(ctypes.byref(shape_s), *([fake] * 4), fake + 16, fake, 0.01,
                                             *([fake] * 5), 1 << 40, None) == B.GSHARD_ERR_INVALID_ARG
    if not torch.cuda.is_available():
        # with valid arguments the next check is the device: no GPU here, nothing is launched
        assert f(ctypes.byref(shape), *args, None, None, fake, need, None) in (B.GSHARD_ERR_CUDA, B.GSHARD_ERR_ARCH)
        assert B.load().gshard_moe_top2_backward(ctypes.byref(shape_s), *([fake] * 6), 0.01, *([fake] * 5),
                                                 1 << 40, None) in (B.GSHARD_ERR_CUDA, B.GSHARD_ERR_ARCH)


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libgshard_moe.so"))
    with pytest.raises(ImportError, match="no fallback"):
        B.load()

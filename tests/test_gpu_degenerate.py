"""Degenerate cases of the method on the GPU: exact ties (the lowest expert index must win, for
both picks), identical tokens (one expert takes everything and overflows), extreme values of the
random-routing noise, two experts, one token per group."""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import MoEConfig, make_inputs
from paper_2006_16668_b200 import binding as B
from parity_util import to_np
from test_gpu_forward import check_forward, run_forward

pytestmark = pytest.mark.gpu

PATHS = [("f32", 0), ("bf16", B.GSHARD_FLAG_SIMT_CONTRACTIONS), ("bf16", 0)]


# (dtype, flags, E): the gating kernels differ in where the twin of an expert lives - the same
# 32-column chunk (E = 32, one-SM kernel), another column part of a CTA (E = 256, CTA pairs),
# another column tile (E = 512), another CTA of the cluster (cluster kernel)
TIE_PATHS = [(d, f, 32) for d, f in PATHS] + [
    ("bf16", 0, 256), ("bf16", 0, 512), ("bf16", B.GSHARD_FLAG_GATE_ONE_SM, 512),
    ("bf16", B.GSHARD_FLAG_GATE_CLUSTER, 256), ("bf16", B.GSHARD_FLAG_GATE_CLUSTER, 1024),
]


@pytest.mark.parametrize("dtype,flags,E", TIE_PATHS)
def test_exact_ties_lowest_index_wins(dtype, flags, E):
    # every expert j < E/2 has a twin j + E/2 with identical gating weights: the two largest gates
    # of every token tie exactly, so Algorithm 1's top_2 must return (j, j + E/2), w1 = w2 = 1/2.
    cfg = MoEConfig("ties", G=2, S=192, M=64, H=64, E=E, C=12, dtype=dtype, seed=31)
    inp = make_inputs(cfg, "cuda")
    half = cfg.E // 2
    inp["wg"][:, half:] = inp["wg"][:, :half]
    y, l_aux, rt = run_forward(cfg, inp, flags)
    ei = to_np(rt["expert_idx"])
    logits = to_np(inp["x"]).astype(np.float64) @ to_np(inp["wg"]).astype(np.float64)[:, :half]
    top = logits.argmax(axis=-1)
    srt = np.sort(logits, axis=-1)
    clear = (srt[..., -1] - srt[..., -2]) > 1e-3              # tokens whose best expert is unambiguous
    assert np.array_equal(ei[..., 0][clear], top[clear])
    assert np.array_equal(ei[..., 1][clear], top[clear] + half)
    assert np.all(ei[..., 0] < half) and np.array_equal(ei[..., 1], ei[..., 0] + half)
    w = to_np(rt["weight"])
    assert np.all(w == 0.5)
    # wg = 0: all E gates tie; picks are (0, 1); only the first C tokens of a group keep anything
    inp["wg"].zero_()
    y, l_aux, rt = run_forward(cfg, inp, flags)
    ei = to_np(rt["expert_idx"])
    assert np.all(ei[..., 0] == 0) and np.all(ei[..., 1] == 1)
    slot = to_np(rt["slot"])
    expect = np.where(np.arange(cfg.S) < cfg.C, np.arange(cfg.S), -1)
    assert np.array_equal(slot[..., 0], np.broadcast_to(expect, (cfg.G, cfg.S)))
    assert np.array_equal(slot[..., 1], np.broadcast_to(expect, (cfg.G, cfg.S)))       # 2*w2 = 1 > u always
    assert float(l_aux) == pytest.approx(1.0 / cfg.E ** 2, rel=1e-5)
    assert not to_np(y)[:, cfg.C:].any()


@pytest.mark.parametrize("dtype,flags", PATHS)
def test_identical_tokens_overflow_one_expert(dtype, flags):
    cfg = MoEConfig("same", G=2, S=128, M=64, H=128, E=16, C=16, dtype=dtype, seed=32)
    inp = make_inputs(cfg, "cuda")
    inp["x"][:] = inp["x"][0, 0]
    y, l_aux, rt = run_forward(cfg, inp, flags)
    rep = {}
    check_forward(cfg, inp, y, l_aux, rt, range(cfg.G), cfg.S, report=rep)
    fc = to_np(rt["first_count"])
    assert np.all(fc.max(axis=1) == cfg.S)                    # one expert got every first choice
    assert int(rt["stats"][0]) == cfg.G * (cfg.S - cfg.C)     # everything beyond C is dropped
    _, p = orc.gates(to_np(inp["x"][0, :1]), to_np(inp["wg"]))
    assert float(l_aux) == pytest.approx(p.max() / cfg.E, rel=1e-4)    # closed form for identical tokens


@pytest.mark.parametrize("uval,expect_pass", [(0.0, "all"), (0.99999994, "half_only")])
def test_random_routing_extremes(uval, expect_pass):
    cfg = MoEConfig("u", G=2, S=256, M=64, H=64, E=16, C=64, dtype="f32", seed=33)
    inp = make_inputs(cfg, "cuda")
    inp["u"].fill_(uval)
    y, l_aux, rt = run_forward(cfg, inp)
    check_forward(cfg, inp, y, l_aux, rt, range(cfg.G), 16)
    passed = (to_np(rt["flags"]) & 2) != 0
    if expect_pass == "all":
        assert passed.all()
    else:
        assert not passed.any()        # 2*w2 <= 1 and equals 1 only at an exact tie


@pytest.mark.parametrize("name,G,S,M,H,E,C,dtype", [
    ("two_experts", 2, 200, 32, 64, 2, 200, "f32"),       # E = 2: both experts are always picked
    ("one_token_groups", 5, 1, 32, 64, 8, 1, "f32"),      # S = 1
    ("one_token_groups_bf16", 3, 1, 64, 64, 16, 1, "bf16"),
    ("capacity_above_s", 2, 64, 64, 128, 16, 100, "bf16"),  # C > S: nothing can overflow
])
def test_small_extremes(name, G, S, M, H, E, C, dtype):
    cfg = MoEConfig(name, G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, seed=34)
    inp = make_inputs(cfg, "cuda")
    y, l_aux, rt = run_forward(cfg, inp)
    check_forward(cfg, inp, y, l_aux, rt, range(G), S)
    if name == "capacity_above_s":
        assert int(rt["stats"][0]) == 0 and int(rt["stats"][2]) == 0
    if name == "two_experts":
        ei = to_np(rt["expert_idx"])
        assert np.all(ei[..., 0] + ei[..., 1] == 1)

"""Dense full-size parity of the dominant kernels against the oracle: more than a thousand sampled
tokens of the MoE(2048E) layer, and every row of whole experts of the expert FFN chosen to cover
the first and the last work units of several CTA groups and the ragged last wave.  (Routing of
every token at full size is covered by test_gpu_forward.test_full_size_sampled.)"""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import CONFIGS, make_inputs
from paper_2006_16668_b200 import binding as B
from parity_util import rel_fro, to_np
from test_gpu_forward import Y_TOL, check_forward, run_forward

pytestmark = pytest.mark.gpu


def test_c4_more_than_a_thousand_tokens():
    """Eight groups spread over the batch, 128 random tokens in each plus tokens with dropped
    choices: routing of those groups bit-exact, y against eq. (2)-(3) evaluated by the oracle."""
    cfg = CONFIGS["c4_2048e"]
    inp = make_inputs(cfg, "cuda")
    y, l_aux, rt = run_forward(cfg, inp)
    rep = {}
    check_forward(cfg, inp, y, l_aux, rt, list(range(1, cfg.G, 4)), 128, report=rep)
    assert rep["tokens"] >= 1024
    print(f"\n[c4] y rel. Frobenius error on {rep['tokens']} tokens: {rep['y_err']:.3e}")


def _whole_expert_check(cfg, experts, flags=0):
    """Stage calls at full size: dispatch, then the expert FFN in the form the layer uses; every
    output row of the chosen experts against the oracle's FFN of the same dispatched rows."""
    inp = make_inputs(cfg, "cuda")
    shape = B.make_shape(cfg, flags=flags)
    _, _, rt = run_forward(cfg, inp, flags)
    R = cfg.E * cfg.G * cfg.C
    buf = torch.empty(cfg.E, cfg.G * cfg.C, cfg.M, dtype=inp["x"].dtype, device="cuda")
    out = torch.empty_like(buf)
    ws = B.alloc_workspace(shape)
    B.gshard_moe_dispatch(shape, inp["x"], rt["slot_token"], buf)
    B.gshard_moe_expert_ffn(shape, buf, inp["wi"], inp["wo"], out, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    worst = 0.0
    for e in experts:
        rows = to_np(buf[e])
        ref = orc.ffn_rows(rows, to_np(inp["wi"][e]), to_np(inp["wo"][e]))
        got = to_np(out[e])
        empty = to_np(rt["slot_token"][e]).reshape(-1) < 0
        assert not got[empty].any(), "an empty slot's output row must be zero"
        assert (~empty).any()
        err = rel_fro(got, ref)
        worst = max(worst, err)
        assert err <= Y_TOL, (e, err)
    return worst


def test_c4_whole_experts_of_the_single_launch_ffn():
    """2048 work units over 37 groups of four CTAs: unit u belongs to group u mod 37, the last wave
    (units 2035..2047) reaches only 13 groups.  Experts: first units of the first, second and last
    group, the first group's second unit, the end of the last full wave, the first and last unit of
    the ragged wave, and two in the middle."""
    cfg = CONFIGS["c4_2048e"]
    worst = _whole_expert_check(cfg, (0, 1, 36, 37, 1000, 1023, 2034, 2035, 2047))
    print(f"\n[c4] worst whole-expert rel. Frobenius error: {worst:.3e}")


def test_c2_whole_experts_of_the_grouped_gemms():
    """1024 rows per expert on CTA pairs (four 256-row tiles): first, a middle and the last expert."""
    cfg = CONFIGS["c2_128e"]
    worst = _whole_expert_check(cfg, (0, 77, 127))
    print(f"\n[c2] worst whole-expert rel. Frobenius error: {worst:.3e}")

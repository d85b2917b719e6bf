"""GPU parity of the backward pass (gshard_moe_top2_backward) against the oracle's gradients of
L = <dy, y> + k*l_aux with the routing frozen.  Tolerance: relative Frobenius error 2e-2 per
gradient tensor (bf16 path); the fp32 path is held to 1e-4."""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import CONFIGS, MoEConfig, make_inputs
from paper_2006_16668_b200 import binding as B
from parity_util import rel_fro, to_np

pytestmark = pytest.mark.gpu

GRAD_TOL = 2e-2


def run_fwd_bwd(cfg, inp, flags=0):
    shape = B.make_shape(cfg, flags=flags | B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
    ws = B.alloc_workspace(shape)
    ctx = torch.empty(B.gshard_moe_top2_context_bytes(shape), dtype=torch.uint8, device="cuda")
    rt, rs = B.alloc_routing(shape)
    y = torch.empty_like(inp["x"])
    l_aux = torch.zeros(1, device="cuda")
    B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, rs, ctx, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    wsb = B.alloc_workspace(shape, for_backward=True)
    dx = torch.empty_like(inp["x"])
    dwg = torch.empty(cfg.M, cfg.E, dtype=torch.float32, device="cuda")
    dwi = torch.empty_like(inp["wi"])
    dwo = torch.empty_like(inp["wo"])
    B.gshard_moe_top2_backward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], ctx, inp["dy"], cfg.k_aux,
                               dx, dwg, dwi, dwo, wsb)
    assert B.gshard_moe_last_device_status(wsb) == B.GSHARD_OK
    return y, l_aux, rt, dx, dwg, dwi, dwo


def oracle_with_gpu_routing(cfg, inp, rt):
    """The oracle's forward record with the integer routing taken from the GPU run (the forward
    tests establish that it equals the oracle's up to near-ties); gradients are then the
    oracle's own arithmetic on that frozen routing."""
    f = orc.forward(to_np(inp["x"]), to_np(inp["wg"]), None, None, to_np(inp["u"]), cfg.C, want_y=False)
    agree = (f.expert_idx == to_np(rt["expert_idx"])).all(axis=-1).mean()
    assert agree > 0.995
    f.expert_idx = to_np(rt["expert_idx"])
    f.slot = to_np(rt["slot"])
    f.first_count = to_np(rt["first_count"])
    return f


BWD_CASES = [
    ("f32", 2, 48, 32, 64, 8, 8, "f32", 0, 1e-4),
    ("f32_ragged", 3, 50, 24, 40, 5, 6, "f32", 0, 1e-4),
    ("bf16_simt", 2, 128, 64, 128, 16, 12, "bf16", B.GSHARD_FLAG_SIMT_CONTRACTIONS, GRAD_TOL),
    ("bf16_umma", 2, 256, 128, 256, 16, 24, "bf16", 0, GRAD_TOL),
    ("bf16_umma_ragged", 3, 200, 192, 320, 32, 5, "bf16", 0, GRAD_TOL),
    ("bf16_umma_variant_a", 2, 256, 128, 256, 16, 20, "bf16", B.GSHARD_FLAG_SECOND_SKIP_FREES_SLOT, GRAD_TOL),
    # every grouped GEMM with more than 128 rows on CTA pairs (all four operand-layout variants)
    ("bf16_two_sm", 2, 384, 256, 512, 16, 80, "bf16", B.GSHARD_FLAG_TWO_SM_MMA, GRAD_TOL),
    # weight-gradient GEMMs on the resident-B kernel (contraction = rows per expert <= 256, at least
    # four row tiles): a ragged contraction (80 = 64 + 16) with a ragged last column block, and the
    # full four k-blocks
    ("bf16_wgrad_resident_ragged", 2, 256, 512, 640, 16, 40, "bf16", 0, GRAD_TOL),
    ("bf16_wgrad_resident_k256", 2, 1024, 512, 512, 16, 128, "bf16", 0, GRAD_TOL),
    # dwo on CTA pairs with the deep A ring (sixteen 256-row tiles per column block), dwi on single CTAs
    ("bf16_wgrad_pairs_deep_ring", 2, 512, 256, 4096, 16, 64, "bf16", 0, GRAD_TOL),
    # every weight gradient on pairs: few row tiles per column block, two resident B slices in turn
    ("bf16_wgrad_pairs_two_slices", 2, 1024, 512, 1024, 16, 128, "bf16", B.GSHARD_FLAG_TWO_SM_MMA, GRAD_TOL),
    # dh beside dwo and dbuf beside dwi, half of the multiprocessors each
    ("bf16_paired_gemms", 2, 1024, 512, 512, 16, 128, "bf16", B.GSHARD_FLAG_BWD_PAIRED_GEMMS, GRAD_TOL),
]


@pytest.mark.parametrize("name,G,S,M,H,E,C,dtype,flags,tol", BWD_CASES, ids=[c[0] for c in BWD_CASES])
def test_backward_small_every_element(name, G, S, M, H, E, C, dtype, flags, tol):
    cfg = MoEConfig(name, G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, seed=4242, backward=True, k_aux=0.01)
    inp = make_inputs(cfg, "cuda")
    y, l_aux, rt, dx, dwg, dwi, dwo = run_fwd_bwd(cfg, inp, flags)
    f = oracle_with_gpu_routing(cfg, inp, rt)
    rdx, rdwg, rdwi, rdwo = orc.backward(to_np(inp["x"]), to_np(inp["wg"]), to_np(inp["wi"]), to_np(inp["wo"]),
                                         f, to_np(inp["dy"]), cfg.k_aux)
    errs = {"dx": rel_fro(to_np(dx), rdx), "dwg": rel_fro(to_np(dwg), rdwg), "dwi": rel_fro(to_np(dwi), rdwi),
            "dwo": rel_fro(to_np(dwo), rdwo)}
    assert all(v <= tol for v in errs.values()), errs
    # experts that received no token get exactly zero weight gradients
    used = np.zeros(E, bool)
    used[np.unique(f.expert_idx[f.slot >= 0])] = True
    assert not to_np(dwi)[~used].any() and not to_np(dwo)[~used].any()


def test_backward_aux_loss_only():
    # dy = 0: only k*l_aux contributes; it reaches wg and x through the dense mean-gate term.
    cfg = MoEConfig("aux", G=2, S=64, M=32, H=64, E=8, C=16, dtype="f32", seed=9, backward=True, k_aux=1.0)
    inp = make_inputs(cfg, "cuda")
    inp["dy"].zero_()
    y, l_aux, rt, dx, dwg, dwi, dwo = run_fwd_bwd(cfg, inp)
    f = oracle_with_gpu_routing(cfg, inp, rt)
    rdx, rdwg, _, _ = orc.backward(to_np(inp["x"]), to_np(inp["wg"]), to_np(inp["wi"]), to_np(inp["wo"]), f,
                                   to_np(inp["dy"]), cfg.k_aux)
    assert not to_np(dwi).any() and not to_np(dwo).any()
    assert rel_fro(to_np(dwg), rdwg) < 1e-4 and rel_fro(to_np(dx), rdx) < 1e-4


def _token_grads(cfg, inp, ei, slot, fc, wg, g, s, k_aux, dy_row):
    """Oracle pieces for one token: (dx row from both paths, dlogit row)."""
    xs = to_np(inp["x"][g, s])
    dys = dy_row.astype(np.float64)
    _, p = orc.gates(xs[None, :], wg)
    p = p[0]
    a, b = p[ei[g, s, 0]], p[ei[g, s, 1]]
    dxs = np.zeros(cfg.M)
    dw = [0.0, 0.0]
    for k in range(2):
        if slot[g, s, k] < 0:
            continue
        e = int(ei[g, s, k])
        wi_e, wo_e = to_np(inp["wi"][e]), to_np(inp["wo"][e])
        o = orc.ffn_rows(xs[None, :], wi_e, wo_e)
        dw[k] = float(dys @ o[0])
        wk = (a if k == 0 else b) / (a + b)
        dxr, _, _ = orc.ffn_rows_backward(xs[None, :], (wk * dys)[None, :], wi_e, wo_e)
        dxs += dxr[0]
    dlogit = orc.gate_row_backward(p, ei[g, s, 0], ei[g, s, 1], dw[0], dw[1], fc[g], cfg.S, cfg.G, k_aux)
    dxs += dlogit @ wg.astype(np.float64).T          # dx += dlogit . wg^T
    return dxs, dlogit, xs


def test_backward_training_config_sampled():
    """MoE(512E) training step at full size.  The oracle cannot evaluate every expert, so:
    dwi/dwo are compared on sampled experts (all their rows), dx on sampled tokens, and dwg -
    a sum over all tokens - on a second run whose dy is non-zero only for the sampled tokens
    and whose l_aux weight is zero, so that only those tokens contribute."""
    cfg = CONFIGS["c5_512e_train"]
    inp = make_inputs(cfg, "cuda")
    rng = np.random.default_rng(11)
    toks = sorted({(int(rng.integers(cfg.G)), int(rng.integers(cfg.S))) for _ in range(132)})
    assert len(toks) >= 128
    y, l_aux, rt, dx, dwg, dwi, dwo = run_fwd_bwd(cfg, inp)
    # the forward that saves its context (two grouped-GEMM launches, h and out written into the
    # context) must give the layer output too: routing of three groups and y on sampled tokens
    from test_gpu_forward import check_forward
    rep = {}
    check_forward(cfg, inp, y, l_aux, rt, [0, 7, cfg.G - 1], 12, report=rep)
    print(f"\n[c5 forward with saved context] y rel. Frobenius error on {rep['tokens']} tokens: {rep['y_err']:.3e}")
    ei, slot, wt = to_np(rt["expert_idx"]), to_np(rt["slot"]), to_np(rt["weight"]).astype(np.float64)
    st = to_np(rt["slot_token"])
    fc = to_np(rt["first_count"])
    wg = to_np(inp["wg"])
    # 16 experts: the first and last of the batch, both sides of a CTA pair's tile boundary, and the
    # neighbours of the multiples of the SM count at which the persistent tile lists wrap
    for e in (0, 1, 7, 73, 74, 147, 148, 149, 255, 256, 295, 296, 300, 443, 510, 511):
        wi_e, wo_e = to_np(inp["wi"][e]), to_np(inp["wo"][e])
        rows_x, rows_dout = [], []
        for g in range(cfg.G):
            for c in range(cfg.C):
                s = st[e, g, c]
                if s < 0:
                    continue
                k = 0 if (ei[g, s, 0] == e and slot[g, s, 0] == c) else 1
                rows_x.append(to_np(inp["x"][g, s]))
                rows_dout.append(wt[g, s, k] * to_np(inp["dy"][g, s]).astype(np.float64))
        _, ref_dwi, ref_dwo = orc.ffn_rows_backward(np.stack(rows_x), np.stack(rows_dout), wi_e, wo_e)
        assert rel_fro(to_np(dwo[e]), ref_dwo) <= GRAD_TOL
        assert rel_fro(to_np(dwi[e]), ref_dwi) <= GRAD_TOL
    got, ref = [], []
    for (g, s) in toks:
        dxs, _, _ = _token_grads(cfg, inp, ei, slot, fc, wg, g, s, cfg.k_aux, to_np(inp["dy"][g, s]))
        got.append(to_np(dx[g, s]))
        ref.append(dxs)
    assert rel_fro(np.stack(got), np.stack(ref)) <= GRAD_TOL
    # dwg: dy restricted to the sampled tokens, k = 0
    dy_sparse = torch.zeros_like(inp["dy"])
    for (g, s) in toks:
        dy_sparse[g, s] = inp["dy"][g, s]
    inp2 = dict(inp)
    inp2["dy"] = dy_sparse
    del dwi, dwo, dx, y
    torch.cuda.empty_cache()
    _, _, rt2, _, dwg2, _, _ = run_fwd_bwd(cfg.scaled(k_aux=0.0), inp2)
    assert torch.equal(rt2["slot"], rt["slot"])
    ref_dwg = np.zeros((cfg.M, cfg.E))
    for (g, s) in toks:
        _, dlogit, xs = _token_grads(cfg, inp, ei, slot, fc, wg, g, s, 0.0, to_np(inp["dy"][g, s]))
        ref_dwg += np.outer(xs.astype(np.float64), dlogit)          # dwg = sum x^T dlogit
    assert rel_fro(to_np(dwg2), ref_dwg) <= GRAD_TOL


@pytest.mark.parametrize("dtype,tol", [("f32", 1e-5), ("bf16", 1e-2)])
def test_residual_connection_folded_into_combine_and_dx(dtype, tol):
    """GSHARD_FLAG_ADD_RESIDUAL: y = x + layer(x) and dx = dx_layer + dy, against the same layer without the
    flag (whose parity with the oracle the other tests establish)."""
    M, H = (64, 128)
    cfg = MoEConfig("res", G=2, S=128, M=M, H=H, E=16, C=12, dtype=dtype, seed=5, backward=True, k_aux=0.01)
    inp = make_inputs(cfg, "cuda")
    outs = {}
    for flag in (0, B.GSHARD_FLAG_ADD_RESIDUAL):
        shape = B.make_shape(cfg, flags=B.GSHARD_FLAG_SAVE_FOR_BACKWARD | flag)
        ws = B.alloc_workspace(shape, for_backward=True)
        wsf = B.alloc_workspace(shape)
        ctx = torch.empty(B.gshard_moe_top2_context_bytes(shape), dtype=torch.uint8, device="cuda")
        y = torch.empty_like(inp["x"])
        l_aux = torch.zeros(1, device="cuda")
        B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, None, ctx, wsf)
        dx = torch.empty_like(inp["x"])
        dwg = torch.empty(cfg.M, cfg.E, device="cuda")
        dwi, dwo = torch.empty_like(inp["wi"]), torch.empty_like(inp["wo"])
        B.gshard_moe_top2_backward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], ctx, inp["dy"], cfg.k_aux, dx, dwg,
                                   dwi, dwo, ws)
        assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
        outs[flag] = (y.float().cpu(), dx.float().cpu(), dwg.cpu(), dwi.float().cpu(), dwo.float().cpu())
    y0, dx0, dwg0, dwi0, dwo0 = outs[0]
    y1, dx1, dwg1, dwi1, dwo1 = outs[B.GSHARD_FLAG_ADD_RESIDUAL]
    x, dy = inp["x"].float().cpu(), inp["dy"].float().cpu()
    assert rel_fro(y1.numpy(), (y0 + x).numpy()) <= tol
    assert rel_fro(dx1.numpy(), (dx0 + dy).numpy()) <= tol
    # the weight gradients do not see the residual path
    assert torch.equal(dwg0, dwg1) and torch.equal(dwi0, dwi1) and torch.equal(dwo0, dwo1)

"""GPU parity of the individual stages (C-ABI stage calls) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import MoEConfig
from paper_2006_16668_b200 import binding as B
from parity_util import rel_fro, slot_token_from, to_np

pytestmark = pytest.mark.gpu


def _shape(G, S, M, H, E, C, dtype="f32", flags=0):
    return B.make_shape(G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, flags=flags)


CAP_CASES = [
    # G, S, E, C, variant_a, concentration (small = skewed routing)
    (2, 64, 8, 16, False, 1.0), (3, 1000, 5, 7, False, 0.3), (1, 4096, 2048, 4, False, 1.0),
    (2, 4096, 512, 16, True, 0.2), (4, 33, 4, 1, False, 1.0), (2, 2500, 128, 64, True, 1.0),
    (1, 31, 16384, 2, False, 1.0), (2, 4096, 4096, 2, False, 0.5),
]


@pytest.mark.parametrize("G,S,E,C,variant_a,conc", CAP_CASES)
def test_capacity_kernel_bit_exact(G, S, E, C, variant_a, conc):
    """The capacity kernel fed with the oracle's top-2 must reproduce Algorithm 1's two loops
    exactly.  Gates are float32 values on both sides, so the random-routing test is decided
    from identical numbers; tokens within 1e-6 of the threshold are forced to the GPU's
    outcome in the oracle's replay."""
    rng = np.random.default_rng(G * 1000 + S + E)
    flags = B.GSHARD_FLAG_SECOND_SKIP_FREES_SLOT if variant_a else 0
    shape = _shape(G, S, 8, 8, E, C, "f32", flags)
    # random top-2 picks with a skewed expert popularity, random float32 gate values g1 >= g2
    pop = rng.dirichlet(np.ones(E) * conc)
    e1 = rng.choice(E, size=(G, S), p=pop).astype(np.int32)
    e2 = (e1 + 1 + rng.integers(0, E - 1, size=(G, S))) % E
    e2 = e2.astype(np.int32)
    ga = rng.random((G, S)).astype(np.float32) * 0.5 + 1e-3
    gb = (ga * rng.random((G, S)).astype(np.float32)).astype(np.float32)
    gb = np.maximum(gb, np.float32(1e-6))
    u = rng.random((G, S)).astype(np.float32)
    m = rng.dirichlet(np.ones(E), size=G).astype(np.float32)
    dev = "cuda"
    ei = torch.from_numpy(np.stack([e1, e2], -1).copy()).to(dev)
    g12 = torch.from_numpy(np.stack([ga, gb], -1).copy()).to(dev)
    rt, rs = B.alloc_routing(shape)
    l_aux = torch.zeros(1, device=dev)
    ws = B.alloc_workspace(shape)
    B.gshard_moe_capacity(shape, ei, g12, torch.from_numpy(u).to(dev), torch.from_numpy(m).to(dev), rs, l_aux, ws)
    torch.cuda.synchronize()
    l_groups = []
    for g in range(G):
        gflags = to_np(rt["flags"][g])
        w2 = gb[g].astype(np.float64) / (ga[g].astype(np.float64) + gb[g].astype(np.float64))
        near = np.abs(2 * w2 - u[g]) < 1e-6
        override = np.where(near, ((gflags & 2) != 0).astype(np.int8), np.int8(-1)).astype(np.int8)
        r = orc.capacity(E, C, e1[g], e2[g], ga[g], gb[g], u[g], m[g], pass_override=override,
                         variant_a=variant_a)
        assert np.array_equal(to_np(rt["slot"][g]), r.slot)
        assert np.array_equal(gflags, r.flags)
        assert np.array_equal(to_np(rt["first_count"][g]), r.first_count)
        assert np.array_equal(to_np(rt["total_count"][g]), r.total_count)
        assert np.array_equal(to_np(rt["slot_token"][:, g, :]), slot_token_from(r, e1[g], e2[g], E, C))
        np.testing.assert_allclose(to_np(rt["weight"][g]), r.weight, rtol=1e-5)
        assert float(rt["l_aux_group"][g]) == pytest.approx(r.l_aux, rel=1e-5)
        l_groups.append(r.l_aux)
    assert float(l_aux) == pytest.approx(float(np.mean(l_groups)), rel=1e-5)


@pytest.mark.parametrize("bulk", [0, B.GSHARD_FLAG_BULK_DISPATCH], ids=["vector_loads", "tma_bulk"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_dispatch_and_combine(dtype, bulk):
    G, S, M, H, E, C = 3, 50, 72, 8, 6, 5
    rng = np.random.default_rng(5)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    shape = _shape(G, S, M, H, E, C, dtype, (B.GSHARD_FLAG_SIMT_CONTRACTIONS if dtype == "bf16" else 0) | bulk)
    x = torch.randn(G, S, M, device="cuda").to(tdt)
    # a valid routing from the oracle
    p = rng.dirichlet(np.ones(E), size=(G, S))
    st = np.full((E, G, C), -1, np.int32)
    ei = np.zeros((G, S, 2), np.int32)
    slot = np.zeros((G, S, 2), np.int32)
    weight = np.zeros((G, S, 2), np.float32)
    for g in range(G):
        e1, e2, g1, g2, _ = orc.top2(p[g])
        r = orc.capacity(E, C, e1, e2, g1, g2, rng.random(S).astype(np.float32), p[g].mean(0))
        st[:, g, :] = slot_token_from(r, e1, e2, E, C)
        ei[g, :, 0], ei[g, :, 1] = e1, e2
        slot[g], weight[g] = r.slot, r.weight
    buf = torch.full((E, G * C, M), 7.0, device="cuda").to(tdt)
    B.gshard_moe_dispatch(shape, x, torch.from_numpy(st).cuda(), buf)
    xn = to_np(x)
    expect = np.zeros((E, G, C, M), np.float32)
    for e in range(E):
        for g in range(G):
            for c in range(C):
                if st[e, g, c] >= 0:
                    expect[e, g, c] = xn[g, st[e, g, c]]
    assert np.array_equal(to_np(buf).reshape(E, G, C, M), expect)        # a copy: bit-exact
    # combine
    out = torch.randn(E, G * C, M, device="cuda").to(tdt)
    y = torch.empty(G, S, M, device="cuda", dtype=tdt)
    B.gshard_moe_combine(shape, out, torch.from_numpy(ei).cuda(), torch.from_numpy(slot).cuda(),
                         torch.from_numpy(weight).cuda(), y)
    on = to_np(out).reshape(E, G, C, M).astype(np.float64)
    yref = np.zeros((G, S, M))
    for g in range(G):
        for s in range(S):
            for k in range(2):
                if slot[g, s, k] >= 0:
                    yref[g, s] += np.float64(weight[g, s, k]) * on[ei[g, s, k], g, slot[g, s, k]]
    tol = 1e-6 if dtype == "f32" else 4e-3
    assert rel_fro(to_np(y), yref) < tol


FFN_CASES = [
    # E, G, C, M, H, dtype, flags
    (3, 2, 16, 64, 256, "f32", 0),
    (2, 1, 40, 128, 320, "bf16", B.GSHARD_FLAG_SIMT_CONTRACTIONS),
    (4, 1, 128, 1024, 8192, "bf16", 0),          # one full 128-row tile per expert (MoE(2048E) shape)
    (2, 2, 100, 1024, 2048, "bf16", 0),          # 200 rows: ragged second row tile
    (3, 1, 24, 192, 448, "bf16", 0),             # fewer rows than a tile, ragged column tile
    (1, 4, 96, 512, 1024, "bf16", 0),            # 384 rows
    # more than 128 rows run on CTA pairs by default: the same shapes on single CTAs
    (2, 2, 100, 1024, 2048, "bf16", B.GSHARD_FLAG_ONE_SM_MMA),
    (1, 4, 96, 512, 1024, "bf16", B.GSHARD_FLAG_ONE_SM_MMA),
    # the single-launch FFN (groups of four CTAs, h chunks handed over through an L2-resident ring)
    (40, 1, 128, 512, 2048, "bf16", B.GSHARD_FLAG_FUSED_FFN),
    (6, 2, 100, 256, 1024, "bf16", B.GSHARD_FLAG_FUSED_FFN),     # 200 rows: two row tiles per expert
    (3, 1, 24, 192, 3072, "bf16", B.GSHARD_FLAG_FUSED_FFN),      # 48 output columns per rank
    (37, 1, 1, 64, 1024, "bf16", B.GSHARD_FLAG_FUSED_FFN),       # one row per expert, 16 columns per rank
    (150, 1, 128, 1024, 1024, "bf16", B.GSHARD_FLAG_FUSED_FFN),  # more units than groups, uneven split
    (2, 3, 128, 448, 2048, "bf16", B.GSHARD_FLAG_FUSED_FFN),     # three full row tiles, 112 columns per rank
    # grouped GEMMs on CTA pairs (two-SM MMA): ragged 256-row tiles, odd tile counts
    (2, 2, 100, 1024, 2048, "bf16", B.GSHARD_FLAG_TWO_SM_MMA),   # 200 rows: second CTA of the pair ragged
    (3, 4, 96, 512, 1024, "bf16", B.GSHARD_FLAG_TWO_SM_MMA),     # 384 rows: two pair tiles, second half empty
    (5, 8, 128, 256, 1536, "bf16", B.GSHARD_FLAG_TWO_SM_MMA),    # 1024 rows, more tiles than pairs
]


@pytest.mark.parametrize("E,G,C,M,H,dtype,flags", FFN_CASES)
def test_expert_ffn_against_oracle(E, G, C, M, H, dtype, flags):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    umma = dtype == "bf16" and not (flags & B.GSHARD_FLAG_SIMT_CONTRACTIONS)
    shape = _shape(G, 4 * C, M, H, -(-max(E, 16) // 16) * 16 if umma else max(E, 2), C, dtype, flags)
    E_run = shape.E
    gen = torch.Generator(device="cuda").manual_seed(E * 100 + C)
    buf = torch.randn(E_run, G * C, M, generator=gen, device="cuda").to(tdt)
    wi = (torch.randn(E_run, M, H, generator=gen, device="cuda") * M ** -0.5).to(tdt)
    wo = (torch.randn(E_run, H, M, generator=gen, device="cuda") * H ** -0.5).to(tdt)
    out = torch.full((E_run, G * C, M), float("nan"), device="cuda").to(tdt)
    ws = B.alloc_workspace(shape)
    B.gshard_moe_expert_ffn(shape, buf, wi, wo, out, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    rows = min(G * C, 48)
    for e in sorted({0, E_run - 1, min(E - 1, E_run - 1)}):
        pick = np.unique(np.linspace(0, G * C - 1, rows).astype(int))
        ref = orc.ffn_rows(to_np(buf[e])[pick], to_np(wi[e]), to_np(wo[e]))
        got = to_np(out[e])[pick]
        assert np.all(np.isfinite(got))
        err = rel_fro(got, ref)
        assert err < (1e-5 if dtype == "f32" else 1e-2), (e, err)


CL = B.GSHARD_FLAG_GATE_CLUSTER
OS = B.GSHARD_FLAG_GATE_ONE_SM
GATE_CASES = [
    # G, S, M, E, flags    (cluster size of the fused gating kernel = ceil(E / 256))
    (2, 64, 128, 16, CL),                             # one CTA, a single 16-expert column tile
    (2, 96, 64, 128, CL),                             # one CTA; 96 tokens: ragged 128-token tile
    (3, 160, 128, 272, CL),                           # two CTAs, the second with 16 experts
    (2, 256, 1024, 512, CL),                          # two CTAs, full contraction depth
    (1, 288, 128, 768, CL),                           # three CTAs: two row quarters finalised by CTA 0
    (2, 128, 192, 1280, CL),                          # five CTAs
    (5, 544, 128, 2048, CL),                          # eight CTAs, more row tiles than clusters can hold at once
    (2, 100, 128, 512, CL),                           # S not a multiple of 32: the stored-logits form is chosen
    # default: stored logits + column-sum pass; on CTA pairs where E % 128 == 0
    (2, 256, 128, 2048, 0),                           # eight column tiles
    (3, 160, 1024, 128, 0),                           # one 128-expert tile, full contraction depth
    (1, 352, 192, 384, 0),                            # three row tiles: the last pair has an idle CTA; ragged second column tile
    (2, 100, 128, 272, 0),                            # E not a multiple of 128: the one-SM kernel is chosen
    (3, 96, 1024, 272, 0),
    (2, 256, 128, 2048, OS),                          # single CTAs forced
    (2, 200, 128, 384, OS),
]


@pytest.mark.parametrize("G,S,M,E,flags", GATE_CASES)
def test_gate_stage_against_oracle(G, S, M, E, flags):
    """Gating stage (softmax gates' top-2, raw gate values, mean gates m) against the fp64 oracle."""
    rng = np.random.default_rng(G * 7 + S + E)
    shape = _shape(G, S, M, 64, E, 2, "bf16", flags)
    x = torch.from_numpy(rng.standard_normal((G, S, M)).astype(np.float32)).to(torch.bfloat16).cuda()
    wg = torch.from_numpy((rng.standard_normal((M, E)) / np.sqrt(M)).astype(np.float32)).to(torch.bfloat16).cuda()
    ei = torch.full((G, S, 2), -1, dtype=torch.int32, device="cuda")
    g12 = torch.zeros(G, S, 2, device="cuda")
    m = torch.zeros(G, E, device="cuda")
    ws = B.alloc_workspace(shape)
    B.gshard_moe_gate(shape, x, wg, ei, g12, m, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    wg_np = to_np(wg)
    for g in range(G):
        _, p = orc.gates(to_np(x[g]), wg_np)
        e1, e2, g1, g2, g3 = orc.top2(p)
        margin = np.where(g3 >= 0, np.minimum(g1 - g2, g2 - g3), g1 - g2)
        ok = margin >= 1e-6
        got = to_np(ei[g])
        assert np.array_equal(got[ok, 0], e1[ok]) and np.array_equal(got[ok, 1], e2[ok])
        idx = np.arange(S)
        # raw gate values of the picks the GPU made (identical to the oracle's outside near-ties)
        np.testing.assert_allclose(to_np(g12[g])[:, 0], p[idx, got[:, 0]], rtol=2e-5, atol=1e-9)
        np.testing.assert_allclose(to_np(g12[g])[:, 1], p[idx, got[:, 1]], rtol=2e-5, atol=1e-9)
        np.testing.assert_allclose(to_np(m[g]), orc.mean_gates(p), rtol=1e-5, atol=1e-9)
    # bit-reproducible
    ei2, g122, m2 = torch.empty_like(ei), torch.empty_like(g12), torch.empty_like(m)
    B.gshard_moe_gate(shape, x, wg, ei2, g122, m2, ws)
    torch.cuda.synchronize()
    assert torch.equal(ei, ei2) and torch.equal(g12, g122) and torch.equal(m, m2)


@pytest.mark.parametrize("G,S,M,E,C,dtype", [(8, 300, 1024, 64, 40, "bf16"),     # 2 KB rows, 20480 rows: 17-18 per warp, the ring turns twice
                                             (4, 64, 4096, 16, 8, "f32"),        # 16 KB rows: ring too large, falls back
                                             (1, 16, 64, 16, 2, "bf16")])        # 128-byte rows, fewer rows than warps
def test_bulk_dispatch_is_the_same_copy(G, S, M, E, C, dtype):
    """GSHARD_FLAG_BULK_DISPATCH (rows through the TMA unit) against the definition: buf[e, g, c] is the
    token's row or zeros, bit for bit; invalid token indices count as empty slots."""
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(11)
    x = torch.randn(G, S, M, device="cuda", generator=gen).to(tdt)
    st = torch.randint(-1, S, (E, G, C), device="cuda", generator=gen, dtype=torch.int32)
    st[0, 0, 0], st[-1, -1, -1] = S, -5                                          # out of range: treated as empty
    shape = _shape(G, S, M, 64, E, C, dtype, B.GSHARD_FLAG_BULK_DISPATCH)
    buf = torch.full((E, G * C, M), 3.0, device="cuda").to(tdt)
    B.gshard_moe_dispatch(shape, x, st, buf)
    valid = (st >= 0) & (st < S)
    g_idx = torch.arange(G, device="cuda").view(1, G, 1).expand(E, G, C)
    expect = torch.where(valid.unsqueeze(-1), x[g_idx, st.clamp(0, S - 1).long()], torch.zeros((), device="cuda", dtype=tdt))
    assert torch.equal(buf.view(E, G, C, M), expect)


@pytest.mark.parametrize("G,S,M,H,E,C,extra", [(4, 512, 1024, 256, 64, 4, 0),                      # single-launch FFN, 2 KB rows
                                               (2, 256, 256, 512, 16, 40, 0),                      # CTA pairs
                                               (2, 256, 256, 512, 16, 40, B.GSHARD_FLAG_SAVE_FOR_BACKWARD)])
def test_forward_with_bulk_dispatch_has_the_same_bits(G, S, M, H, E, C, extra):
    from paper_2006_16668_b200 import MoEConfig, make_inputs
    cfg = MoEConfig("bulk", G=G, S=S, M=M, H=H, E=E, C=C, dtype="bf16", seed=31)
    inp = make_inputs(cfg, "cuda")
    ys = []
    for flags in (extra, extra | B.GSHARD_FLAG_BULK_DISPATCH):
        shape = B.make_shape(cfg, flags=flags)
        ws = B.alloc_workspace(shape)
        ctx = torch.empty(max(B.gshard_moe_top2_context_bytes(shape), 256), dtype=torch.uint8, device="cuda") if extra else None
        y, l_aux = torch.empty_like(inp["x"]), torch.zeros(1, device="cuda")
        B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, None, ctx, ws)
        assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
        ys.append((y, l_aux))
    assert torch.equal(ys[0][0].view(torch.int16), ys[1][0].view(torch.int16)) and torch.equal(ys[0][1], ys[1][1])

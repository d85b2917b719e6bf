"""Failure paths on the GPU that fault, trap or hang nothing: the give-up path of the bounded
device-side waits, and stage calls fed with index tensors that point outside their tensors."""
import numpy as np
import pytest
import torch

from oracle import gshard_oracle as orc
from paper_2006_16668_b200 import CONFIGS, make_inputs
from paper_2006_16668_b200 import binding as B
from parity_util import rel_fro, to_np

pytestmark = pytest.mark.gpu


def test_bounded_wait_gives_up_and_the_workspace_stays_usable():
    """A wait nothing will ever satisfy runs into its limit (200 us here), the kernel leaves through the
    teardown that the GEMM kernels share and the status word reads GSHARD_ERR_TIMEOUT; afterwards the
    same workspace runs a normal forward that matches the oracle."""
    cfg = CONFIGS["c1_tiny"]
    dev = "cuda"
    shape = B.make_shape(cfg)
    ws = B.alloc_workspace(shape, device=dev)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    B.gshard_moe_debug_wait_timeout(ws, limit_us=200)
    t1.record()
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_ERR_TIMEOUT
    assert t0.elapsed_time(t1) < 50.0          # milliseconds: the wait is bounded, nothing hung
    assert "wait" in B.status_string(B.GSHARD_ERR_TIMEOUT)
    # twice in a row: the first give-up left no tensor memory allocated and no barrier armed
    B.gshard_moe_debug_wait_timeout(ws, limit_us=50)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_ERR_TIMEOUT
    inp = make_inputs(cfg, dev)
    y = torch.empty_like(inp["x"])
    l_aux = torch.zeros(1, device=dev)
    B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, None, None, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK      # the forward resets the status word
    host = {k: to_np(v) for k, v in inp.items()}
    f = orc.forward(host["x"], host["wg"], host["wi"], host["wo"], host["u"], cfg.C)
    assert rel_fro(to_np(y), f.y) < 1e-5
    assert float(l_aux) == pytest.approx(f.l_aux, rel=1e-5)


def test_wait_probe_rejects_bad_arguments():
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    lib = B.load()
    assert lib.gshard_moe_debug_wait_timeout(None, 100, None) == B.GSHARD_ERR_INVALID_ARG
    assert lib.gshard_moe_debug_wait_timeout(ws.data_ptr(), 0, None) == B.GSHARD_ERR_INVALID_ARG
    assert lib.gshard_moe_debug_wait_timeout(ws.data_ptr(), 5000, None) == B.GSHARD_ERR_INVALID_ARG
    assert lib.gshard_moe_debug_wait_timeout(ws.data_ptr() + 16, 100, None) == B.GSHARD_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_dispatch_and_combine_skip_out_of_range_indices(dtype):
    """The stage calls take their index tensors from the caller.  Indices outside the tensors they
    address must be skipped (an empty slot / a dropped choice), never used: the rows they name would
    lie far outside the buffers.  Valid entries must still be served exactly."""
    G, S, M, H, E, C = 2, 40, 64, 64, 4, 6
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    flags = B.GSHARD_FLAG_SIMT_CONTRACTIONS if dtype == "bf16" else 0
    shape = B.make_shape(G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, flags=flags)
    rng = np.random.default_rng(7)
    x = torch.randn(G, S, M, device="cuda").to(tdt)
    st = rng.integers(-1, S, size=(E, G, C)).astype(np.int32)
    bad = rng.random((E, G, C)) < 0.3
    st_bad = np.where(bad, rng.choice([S, S + 1, 1 << 20, 2**31 - 1], size=st.shape), st).astype(np.int32)
    buf = torch.full((E, G * C, M), 7.0, device="cuda").to(tdt)
    B.gshard_moe_dispatch(shape, x, torch.from_numpy(st_bad).cuda(), buf)
    torch.cuda.synchronize()
    xb = to_np(x)
    want = np.zeros((E, G, C, M), np.float32)
    for e in range(E):
        for g in range(G):
            for c in range(C):
                if not bad[e, g, c] and st[e, g, c] >= 0:
                    want[e, g, c] = xb[g, st[e, g, c]]
    assert np.array_equal(to_np(buf).reshape(E, G, C, M), want)

    out = torch.randn(E, G * C, M, device="cuda").to(tdt)
    ei = rng.integers(0, E, size=(G, S, 2)).astype(np.int32)
    slot = rng.integers(-1, C, size=(G, S, 2)).astype(np.int32)
    w = rng.random((G, S, 2)).astype(np.float32)
    bad_e = rng.random((G, S, 2)) < 0.2
    bad_s = rng.random((G, S, 2)) < 0.2
    ei_bad = np.where(bad_e, rng.choice([-1, -5, E, E + 3, 1 << 24], size=ei.shape), ei).astype(np.int32)
    slot_bad = np.where(bad_s, rng.choice([C, C + 1, 1 << 24], size=slot.shape), slot).astype(np.int32)
    y = torch.empty(G, S, M, device="cuda").to(tdt)
    B.gshard_moe_combine(shape, out, torch.from_numpy(ei_bad).cuda(), torch.from_numpy(slot_bad).cuda(),
                         torch.from_numpy(w).cuda(), y)
    torch.cuda.synchronize()
    ob = to_np(out).reshape(E, G, C, M).astype(np.float64)
    ref = np.zeros((G, S, M), np.float64)
    for g in range(G):
        for s in range(S):
            for k in range(2):
                if bad_e[g, s, k] or bad_s[g, s, k] or slot[g, s, k] < 0:
                    continue
                ref[g, s] += float(w[g, s, k]) * ob[ei[g, s, k], g, slot[g, s, k]]
    assert rel_fro(to_np(y), ref) < (1e-6 if dtype == "f32" else 4e-3)


def test_debug_checks_pass_on_a_healthy_forward_and_catch_corrupted_routing():
    """GSHARD_FLAG_DEBUG_CHECKS verifies the routing tensors inside the forward (status stays OK, results
    are the same bits as without the flag); gshard_moe_check_routing, the same kernel on its own, must
    record GSHARD_ERR_INTERNAL for each kind of corruption - and survive indices that point far outside
    the tensors, because it bounds-checks before it dereferences."""
    from paper_2006_16668_b200 import MoEConfig
    cfg = MoEConfig("dbg", G=3, S=200, M=64, H=128, E=16, C=20, dtype="bf16", seed=12)
    inp = make_inputs(cfg, "cuda")
    outs = []
    for flags in (0, B.GSHARD_FLAG_DEBUG_CHECKS):
        shape = B.make_shape(cfg, flags=flags)
        ws = B.alloc_workspace(shape)
        rt, rs = B.alloc_routing(shape)
        y = torch.empty_like(inp["x"])
        l_aux = torch.zeros(1, device="cuda")
        B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, rs, None, ws)
        assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
        outs.append((y, rt, B.gshard_moe_last_launch_count()))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert outs[1][2] == outs[0][2] + 1                      # one more kernel: the check
    shape = B.make_shape(cfg)
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    good = outs[0][1]

    def status_of(**changed):
        t = {k: v.clone() for k, v in good.items()}
        for k, fn in changed.items():
            fn(t[k])
        B.gshard_moe_check_routing(shape, B.routing_struct(t), ws)
        return B.gshard_moe_last_device_status(ws)

    assert status_of() == B.GSHARD_OK
    kept = (good["slot"][..., 0] >= 0).nonzero()[0].tolist()           # a token whose first choice was kept
    g, s = kept

    def bump_slot(t):
        t[g, s, 0] = (t[g, s, 0] + 1) % cfg.C

    def far_expert(t):
        t[g, s, 1] = 1 << 24

    def same_experts(t):
        t[g, s, 1] = t[g, s, 0]

    def huge_slot(t):
        t[g, s, 0] = 1 << 20

    def wrong_token(t):
        e = int(good["expert_idx"][g, s, 0])
        t[e, g, int(good["slot"][g, s, 0])] = (s + 1) % cfg.S

    def far_token(t):
        t[0, 0, 0] = 1 << 28

    def bad_weight(t):
        t[g, s, 0] = 0.9
        t[g, s, 1] = 0.3

    def bad_flag(t):
        t[g, s] = t[g, s] ^ 1

    for change in (dict(slot=bump_slot), dict(expert_idx=far_expert), dict(expert_idx=same_experts),
                   dict(slot=huge_slot), dict(slot_token=wrong_token), dict(slot_token=far_token),
                   dict(weight=bad_weight), dict(flags=bad_flag)):
        assert status_of(**change) == B.GSHARD_ERR_INTERNAL, list(change)
    assert status_of() == B.GSHARD_OK                        # the workspace's status word is reset per call

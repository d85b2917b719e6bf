"""gshard_moe_top2_forward_ep on one GPU.

world = 1 must give the bits of gshard_moe_top2_forward.  For world = 2 and 4 the ranks are host
threads of this process that share the GPU, each with its own stream, inputs slice and workspace,
and the collectives are emulated on the host side: a rank's callback publishes its send buffer with
an event, meets the others at a host barrier and copies its slabs out of their buffers on its own
stream.  No kernel of one rank ever waits for a kernel of another (only streams wait on events), so
sharing the GPU is safe; what is tested is everything inside the library call: local gating and
capacity, the slab layout, the device-side regroup, the FFN over all groups' rows of the local
experts, the way back and the combine.  y and the routing must equal the single-GPU layer bit for
bit (whose parity with the oracle the other tests establish), l_aux to 1e-6 (the order of the sum
over groups differs)."""
import threading
import traceback

import pytest
import torch

from paper_2006_16668_b200 import MoEConfig, make_inputs
from paper_2006_16668_b200 import binding as B
from paper_2006_16668_b200 import ep

pytestmark = pytest.mark.gpu


def _single(cfg, inp, flags=0):
    shape = B.make_shape(cfg, flags=flags)
    ws = B.alloc_workspace(shape)
    rt, rs = B.alloc_routing(shape)
    y = torch.empty_like(inp["x"])
    l_aux = torch.zeros(1, device="cuda")
    B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, rs, None, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    return y, l_aux, rt


class _World:
    def __init__(self, n):
        self.n = n
        self.barrier = threading.Barrier(n, timeout=60)
        self.buf = [None] * n
        self.ready = [None] * n
        self.done = [None] * n


class _ThreadComm:
    """gshard_ep_comm for one emulated rank (a host thread with its own stream)."""

    def __init__(self, world, rank, tensors, stream):
        self.w, self.rank, self.tensors, self.stream = world, rank, [t for t in tensors if t is not None], stream
        self.error = None
        self._a2a = B.ALL_TO_ALL_FN(self._all_to_all)
        self._ar = B.ALL_REDUCE_FN(self._all_reduce)
        self.struct = B.gshard_ep_comm(self._a2a, self._ar, None)

    def _view(self, ptr, n):
        """The n bytes at ptr as a view of the tensor of this call that contains them."""
        for t in self.tensors:
            off = ptr - t.data_ptr()
            if 0 <= off and off + n <= t.numel() * t.element_size():
                return t.view(-1).view(torch.uint8)[off:off + n]
        raise AssertionError("collective buffer outside the tensors of the call")

    def _exchange(self, mine, consume):
        """Publish `mine`, wait until every rank has published, run consume(all buffers) on this
        rank's stream, and do not return before every rank has finished reading."""
        w, r = self.w, self.rank
        with torch.cuda.stream(self.stream):
            ev = torch.cuda.Event()
            ev.record(self.stream)
            w.buf[r], w.ready[r] = mine, ev
            w.barrier.wait()
            for s in range(w.n):
                self.stream.wait_event(w.ready[s])
            result = consume(list(w.buf))
            d = torch.cuda.Event()
            d.record(self.stream)
            w.done[r] = d
            w.barrier.wait()
            for s in range(w.n):
                self.stream.wait_event(w.done[s])
            w.barrier.wait()
        return result

    def _all_to_all(self, user, send, recv, bpp, stream):
        try:
            n, r = self.w.n, self.rank
            recv_v = self._view(recv, bpp * n)

            def consume(bufs):
                for s in range(n):
                    recv_v[s * bpp:(s + 1) * bpp].copy_(bufs[s][r * bpp:(r + 1) * bpp], non_blocking=True)
            self._exchange(self._view(send, bpp * n), consume)
            return 0
        except Exception:
            self.error = traceback.format_exc()
            return 1

    def _all_reduce(self, user, buf, count, stream):
        try:
            mine = self._view(buf, 4 * count).view(torch.float32)
            total = self._exchange(mine, lambda bufs: torch.stack([b.clone() for b in bufs]).sum(0))
            with torch.cuda.stream(self.stream):
                mine.copy_(total)
            return 0
        except Exception:
            self.error = traceback.format_exc()
            return 1


def _run_ranks(cfg, inp, world, flags=0):
    shape = B.make_shape(cfg, flags=flags)
    state = _World(world)
    results, errors = [None] * world, [None] * world

    def rank_main(rank):
        try:
            torch.cuda.set_device(0)
            lay = B.gshard_moe_ep_plan(shape, rank, world)
            gs, es = ep.local_slices(lay)
            stream = torch.cuda.Stream()
            x, u = inp["x"][gs].contiguous(), inp["u"][gs].contiguous()
            wi, wo = inp["wi"][es].contiguous(), inp["wo"][es].contiguous()
            ws = torch.empty(B.gshard_moe_ep_workspace_bytes(shape, world), dtype=torch.uint8, device="cuda")
            rt, rs = B.alloc_routing(lay.local)
            y = torch.empty_like(x)
            l_aux = torch.zeros(1, device="cuda")
            torch.cuda.synchronize()
            save = bool(flags & B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
            ctx = torch.empty(B.gshard_moe_ep_context_bytes(shape, world), dtype=torch.uint8, device="cuda") if save else None
            comm = _ThreadComm(state, rank, [ws, ctx, l_aux], stream)
            B.gshard_moe_top2_forward_ep(shape, rank, world, x, inp["wg"], wi, wo, u, y, l_aux, rs, comm.struct, ws,
                                         stream, context=ctx)
            assert comm.error is None, comm.error
            assert B.gshard_moe_last_device_status(ws, stream) == B.GSHARD_OK
            grads = None
            if save:
                dy = inp["dy"][gs].contiguous()
                wsb = torch.empty(B.gshard_moe_ep_backward_workspace_bytes(shape, world), dtype=torch.uint8, device="cuda")
                dx, dwi, dwo = torch.empty_like(x), torch.empty_like(wi), torch.empty_like(wo)
                dwg = torch.empty(cfg.M, cfg.E, dtype=torch.float32, device="cuda")
                torch.cuda.synchronize()
                comm_b = _ThreadComm(state, rank, [wsb, dwg], stream)
                B.gshard_moe_top2_backward_ep(shape, rank, world, x, inp["wg"], wi, wo, ctx, dy, cfg.k_aux, dx, dwg, dwi,
                                              dwo, comm_b.struct, wsb, stream)
                assert comm_b.error is None, comm_b.error
                assert B.gshard_moe_last_device_status(wsb, stream) == B.GSHARD_OK
                grads = (dx, dwg, dwi, dwo)
            stream.synchronize()
            results[rank] = (y, l_aux, rt, grads)
        except Exception:
            errors[rank] = traceback.format_exc()
            state.barrier.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=180)
    assert not any(errors), "\n".join(e for e in errors if e)
    assert all(r is not None for r in results)
    return results


CASES = [
    # name, G, S, M, H, E, C, dtype, flags
    ("f32", 4, 64, 32, 64, 8, 12, "f32", 0),
    ("bf16_single_launch_ffn", 8, 256, 256, 1024, 32, 16, "bf16", 0),          # 128 rows per expert
    ("bf16_cta_pairs", 8, 256, 256, 512, 16, 40, "bf16", 0),                   # 320 rows per expert
    ("bf16_variant_a", 4, 384, 128, 256, 64, 10, "bf16", B.GSHARD_FLAG_SECOND_SKIP_FREES_SLOT),
]


@pytest.mark.parametrize("name,G,S,M,H,E,C,dtype,flags", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("world", [1, 2, 4])
def test_expert_parallel_equals_single_gpu(world, name, G, S, M, H, E, C, dtype, flags):
    cfg = MoEConfig(name, G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, seed=4321)
    inp = make_inputs(cfg, "cuda")
    y_ref, l_ref, rt_ref = _single(cfg, inp, flags)
    results = _run_ranks(cfg, inp, world, flags)
    y = torch.cat([r[0] for r in results])
    assert torch.equal(y.view(torch.uint8), y_ref.view(torch.uint8)), "y differs from the single-GPU layer"
    for k in ("expert_idx", "slot", "weight", "flags", "first_count", "total_count", "m", "l_aux_group"):
        got = torch.cat([r[2][k] for r in results])
        assert torch.equal(got, rt_ref[k]), k
    st = torch.cat([r[2]["slot_token"] for r in results], dim=1)             # [E, Gl, C] per rank -> [E, G, C]
    assert torch.equal(st, rt_ref["slot_token"])
    assert int(sum(int(r[2]["stats"][4]) for r in results)) == int(rt_ref["stats"][4])
    for r in results:                                                          # the same l_aux on every rank
        if world == 1:
            assert torch.equal(r[1], l_ref)
        else:
            assert float(r[1]) == pytest.approx(float(l_ref), rel=1e-6)
            assert torch.equal(r[1], results[0][1])


BWD_CASES = [
    ("f32", 4, 64, 32, 64, 8, 12, "f32"),
    ("bf16_pairs", 4, 256, 256, 512, 16, 40, "bf16"),          # 160 rows per expert on one GPU, per rank the same
    ("bf16_resident_wgrad", 4, 512, 512, 512, 16, 64, "bf16"),  # 256 rows per expert: the weight-gradient kernel
]


@pytest.mark.parametrize("name,G,S,M,H,E,C,dtype", BWD_CASES, ids=[c[0] for c in BWD_CASES])
@pytest.mark.parametrize("world", [1, 2, 4])
def test_expert_parallel_backward_equals_single_gpu(world, name, G, S, M, H, E, C, dtype):
    """gshard_moe_top2_backward_ep after gshard_moe_top2_forward_ep with SAVE_FOR_BACKWARD.  The expert
    FFN sees the same rows in the same order as on one GPU and the token-wise kernels are row-wise, so
    dx, dwi, dwo must have the single-GPU bits (whose parity with the oracle test_gpu_backward.py
    establishes); dwg is a sum over tokens split differently (per-rank partial sums, then the
    all-reduce), compared to 1e-5 relative, and must be identical on all ranks."""
    from test_gpu_backward import run_fwd_bwd
    cfg = MoEConfig(name, G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, seed=2468, backward=True, k_aux=0.01)
    inp = make_inputs(cfg, "cuda")
    y_ref, l_ref, rt_ref, dx_ref, dwg_ref, dwi_ref, dwo_ref = run_fwd_bwd(cfg, inp)
    results = _run_ranks(cfg, inp, world, B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
    bits = lambda t: t.contiguous().view(torch.uint8)
    assert torch.equal(bits(torch.cat([r[0] for r in results])), bits(y_ref))
    assert torch.equal(bits(torch.cat([r[3][0] for r in results])), bits(dx_ref)), "dx"
    assert torch.equal(bits(torch.cat([r[3][2] for r in results])), bits(dwi_ref)), "dwi"
    assert torch.equal(bits(torch.cat([r[3][3] for r in results])), bits(dwo_ref)), "dwo"
    scale = float(dwg_ref.abs().max())
    for r in results:
        assert float((r[3][1] - dwg_ref).abs().max()) <= 1e-5 * scale + 1e-9, "dwg"
        assert torch.equal(r[3][1], results[0][3][1])
    for k in ("expert_idx", "slot", "weight", "first_count"):          # the routing the caller asked for
        assert torch.equal(torch.cat([r[2][k] for r in results]), rt_ref[k]), k


def test_expert_parallel_backward_against_the_oracle():
    """World 2 straight against the oracle's gradients (not through the single-GPU layer)."""
    import numpy as np
    from test_gpu_backward import GRAD_TOL, oracle_with_gpu_routing
    from oracle import gshard_oracle as orc
    from parity_util import rel_fro, to_np
    cfg = MoEConfig("ep_bwd_oracle", G=4, S=128, M=64, H=128, E=16, C=12, dtype="bf16", seed=99, backward=True, k_aux=0.01)
    inp = make_inputs(cfg, "cuda")
    results = _run_ranks(cfg, inp, 2, B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
    rt = {k: torch.cat([r[2][k] for r in results]) for k in ("expert_idx", "slot", "first_count")}
    f = oracle_with_gpu_routing(cfg, inp, rt)
    rdx, rdwg, rdwi, rdwo = orc.backward(to_np(inp["x"]), to_np(inp["wg"]), to_np(inp["wi"]), to_np(inp["wo"]), f,
                                         to_np(inp["dy"]), cfg.k_aux)
    errs = {"dx": rel_fro(to_np(torch.cat([r[3][0] for r in results])), rdx),
            "dwg": rel_fro(to_np(results[1][3][1]), rdwg),
            "dwi": rel_fro(to_np(torch.cat([r[3][2] for r in results])), rdwi),
            "dwo": rel_fro(to_np(torch.cat([r[3][3] for r in results])), rdwo)}
    assert all(v <= GRAD_TOL for v in errs.values()), errs


class _P2PRank:
    """gshard_ep_p2p for one emulated rank: the exchange buffers of all ranks live on the one GPU, so a
    peer's pointer is an ordinary pointer; the rendezvous records an event on this rank's stream, meets
    the other threads at a host barrier and makes the stream wait on every rank's event."""

    def __init__(self, world, rank, buffers, stream):
        self.w, self.rank, self.stream = world, rank, stream
        self.phases, self.error = [], None
        self._rv = B.RENDEZVOUS_FN(self._rendezvous)
        import ctypes
        self._ptrs = (ctypes.c_void_p * world.n)(*[b.data_ptr() for b in buffers])
        self.struct = B.gshard_ep_p2p(self._rv, None, self._ptrs)

    def _rendezvous(self, user, phase, stream):
        try:
            w, r = self.w, self.rank
            self.phases.append(phase)
            ev = torch.cuda.Event()
            ev.record(self.stream)
            w.ready[r] = ev
            w.barrier.wait()
            for s in range(w.n):
                self.stream.wait_event(w.ready[s])
            w.barrier.wait()                      # nobody overwrites its event before all have read it
            return 0
        except Exception:
            self.error = traceback.format_exc()
            return 1


def _run_ranks_p2p(cfg, inp, world, flags=0, steps=1):
    shape = B.make_shape(cfg, flags=flags)
    state = _World(world)
    nbytes = B.gshard_moe_ep_p2p_buffer_bytes(shape, world)
    assert nbytes > 0
    # poisoned, so that a row nobody wrote shows up
    buffers = [torch.full((nbytes,), 0x7F, dtype=torch.uint8, device="cuda") for _ in range(world)]
    torch.cuda.synchronize()
    results, errors = [None] * world, [None] * world

    def rank_main(rank):
        try:
            torch.cuda.set_device(0)
            lay = B.gshard_moe_ep_plan(shape, rank, world)
            gs, es = ep.local_slices(lay)
            stream = torch.cuda.Stream()
            x, u = inp["x"][gs].contiguous(), inp["u"][gs].contiguous()
            wi, wo = inp["wi"][es].contiguous(), inp["wo"][es].contiguous()
            ws = B.alloc_workspace(lay.local)
            rt, rs = B.alloc_routing(lay.local)
            y = torch.empty_like(x)
            l_aux = torch.zeros(1, device="cuda")
            torch.cuda.synchronize()
            p2p = _P2PRank(state, rank, buffers, stream)
            for _ in range(steps):
                B.gshard_moe_top2_forward_ep_p2p(shape, rank, world, x, inp["wg"], wi, wo, u, y, l_aux, rs, p2p.struct,
                                                 None, ws, stream)
            assert p2p.error is None, p2p.error
            assert p2p.phases == ([0, 1, 2] * steps if world > 1 else [])
            assert B.gshard_moe_last_device_status(ws, stream) == B.GSHARD_OK
            stream.synchronize()
            results[rank] = (y, l_aux, rt)
        except Exception:
            errors[rank] = traceback.format_exc()
            state.barrier.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=180)
    assert not any(errors), "\n".join(e for e in errors if e)
    assert all(r is not None for r in results)
    return results


@pytest.mark.parametrize("name,G,S,M,H,E,C,dtype,flags", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("world", [1, 2, 4])
def test_fused_exchange_equals_single_gpu(world, name, G, S, M, H, E, C, dtype, flags):
    """gshard_moe_top2_forward_ep_p2p: dispatch stores into the owners' buffers, combine loads out of
    them.  Same bits as the single-GPU layer; l_aux without a comm is the rank's share, so the shares
    must add up to the layer's l_aux.  Two steps in a row reuse the buffers (phase 0 protects them)."""
    cfg = MoEConfig(name, G=G, S=S, M=M, H=H, E=E, C=C, dtype=dtype, seed=977)
    inp = make_inputs(cfg, "cuda")
    y_ref, l_ref, rt_ref = _single(cfg, inp, flags)
    results = _run_ranks_p2p(cfg, inp, world, flags, steps=2)
    y = torch.cat([r[0] for r in results])
    assert torch.equal(y.view(torch.uint8), y_ref.view(torch.uint8)), "y differs from the single-GPU layer"
    for k in ("expert_idx", "slot", "weight", "flags", "first_count", "total_count", "m", "l_aux_group"):
        assert torch.equal(torch.cat([r[2][k] for r in results]), rt_ref[k]), k
    assert torch.equal(torch.cat([r[2]["slot_token"] for r in results], dim=1), rt_ref["slot_token"])
    assert sum(float(r[1]) for r in results) == pytest.approx(float(l_ref), rel=1e-6)


def test_fused_exchange_with_residual_and_bad_arguments():
    import ctypes
    cfg = MoEConfig("p2p_res", G=4, S=128, M=64, H=128, E=16, C=16, dtype="bf16", seed=5)
    inp = make_inputs(cfg, "cuda")
    y_ref, _, _ = _single(cfg, inp, B.GSHARD_FLAG_ADD_RESIDUAL)
    results = _run_ranks_p2p(cfg, inp, 2, B.GSHARD_FLAG_ADD_RESIDUAL)
    assert torch.equal(torch.cat([r[0] for r in results]).view(torch.int16), y_ref.view(torch.int16))
    shape = B.make_shape(cfg)
    lib = B.load()
    fake = 0x10000
    ptrs = (ctypes.c_void_p * 2)(fake, fake)
    no_rv = B.gshard_ep_p2p(B.RENDEZVOUS_FN(), None, ptrs)
    call = lambda rank, world, p2p, nbytes: lib.gshard_moe_top2_forward_ep_p2p(
        ctypes.byref(shape), rank, world, *([fake] * 7), None, p2p, None, fake, nbytes, None)
    assert call(0, 2, None, 1 << 40) == B.GSHARD_ERR_INVALID_ARG
    assert call(0, 2, ctypes.byref(no_rv), 1 << 40) == B.GSHARD_ERR_INVALID_ARG           # world > 1 needs a rendezvous
    assert call(0, 3, ctypes.byref(no_rv), 1 << 40) == B.GSHARD_ERR_UNSUPPORTED_SHAPE
    assert call(0, 1, ctypes.byref(no_rv), 16) == B.GSHARD_ERR_WORKSPACE_TOO_SMALL
    assert B.gshard_moe_ep_p2p_buffer_bytes(shape, 3) == 0


def test_world_one_at_full_size_is_the_single_gpu_layer():
    from paper_2006_16668_b200 import CONFIGS
    cfg = CONFIGS["c3_512e_skew"]
    inp = make_inputs(cfg, "cuda")
    y_ref, l_ref, _ = _single(cfg, inp)
    shape = B.make_shape(cfg)
    ws = torch.empty(B.gshard_moe_ep_workspace_bytes(shape, 1), dtype=torch.uint8, device="cuda")
    y = torch.empty_like(inp["x"])
    l_aux = torch.zeros(1, device="cuda")
    ep.forward(shape, 0, 1, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, None, ws)
    assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
    assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)) and torch.equal(l_aux, l_ref)


def test_bad_arguments():
    cfg = MoEConfig("bad", G=4, S=64, M=32, H=64, E=8, C=12, dtype="f32", seed=1)
    shape = B.make_shape(cfg)
    lib = B.load()
    fake = 0x10000
    import ctypes
    args = [fake] * 6
    fwd = lambda rank, world, ctx, nbytes, sh=shape: lib.gshard_moe_top2_forward_ep(
        ctypes.byref(sh), rank, world, *args, fake, None, ctx, None, fake, nbytes, None)
    assert fwd(0, 3, None, 1 << 40) == B.GSHARD_ERR_UNSUPPORTED_SHAPE
    assert fwd(2, 2, None, 1 << 40) == B.GSHARD_ERR_INVALID_ARG
    assert fwd(0, 2, None, 1 << 40) == B.GSHARD_ERR_INVALID_ARG                 # world > 1 needs the collectives
    assert fwd(0, 1, None, 16) == B.GSHARD_ERR_WORKSPACE_TOO_SMALL
    saving = B.make_shape(cfg, flags=B.GSHARD_FLAG_SAVE_FOR_BACKWARD)
    assert fwd(0, 1, None, 1 << 40, saving) == B.GSHARD_ERR_INVALID_ARG         # SAVE_FOR_BACKWARD needs a context
    bwd = lambda sh, nbytes: lib.gshard_moe_top2_backward_ep(ctypes.byref(sh), 0, 1, *([fake] * 6), 0.01, *([fake] * 4),
                                                            None, fake, nbytes, None)
    assert bwd(shape, 1 << 40) == B.GSHARD_ERR_INVALID_ARG                      # forward did not save
    assert bwd(saving, 16) == B.GSHARD_ERR_WORKSPACE_TOO_SMALL
    assert B.gshard_moe_ep_context_bytes(saving, 1) == B.gshard_moe_top2_context_bytes(saving)


def test_nccl_comm_single_rank():
    """The NCCL-backed collectives at world 1 (all that one GPU can run): the all-to-all is a group of
    one send and one receive to the rank itself, the all-reduce an identity; both are called through the
    function pointers the library fills in, then the expert-parallel forward runs with that comm."""
    import ctypes
    comm = ep.NcclComm(0, 1)
    try:
        stream = torch.cuda.current_stream().cuda_stream
        send = torch.randint(0, 255, (4096,), dtype=torch.uint8, device="cuda")
        recv = torch.zeros_like(send)
        assert comm.struct.all_to_all(comm.struct.user, send.data_ptr(), recv.data_ptr(), send.numel(), stream) == 0
        v = torch.tensor([1.5, -2.0], device="cuda")
        assert comm.struct.all_reduce_sum_f32(comm.struct.user, v.data_ptr(), 2, stream) == 0
        torch.cuda.synchronize()
        assert torch.equal(recv, send) and v.tolist() == [1.5, -2.0]
        cfg = MoEConfig("nccl1", G=4, S=128, M=64, H=128, E=16, C=16, dtype="bf16", seed=3)
        inp = make_inputs(cfg, "cuda")
        y_ref, l_ref, _ = _single(cfg, inp)
        shape = B.make_shape(cfg)
        ws = torch.empty(B.gshard_moe_ep_workspace_bytes(shape, 1), dtype=torch.uint8, device="cuda")
        y = torch.empty_like(inp["x"])
        l_aux = torch.zeros(1, device="cuda")
        ep.forward(shape, 0, 1, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l_aux, None, ws, comm=comm)
        assert B.gshard_moe_last_device_status(ws) == B.GSHARD_OK
        assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16)) and torch.equal(l_aux, l_ref)
    finally:
        comm.close()
    # without a communicator the constructor refuses
    lib = B.load()
    state, c = B.gshard_ep_nccl_state(), B.gshard_ep_comm()
    assert lib.gshard_ep_comm_from_nccl(None, 1, ctypes.byref(state), ctypes.byref(c)) == B.GSHARD_ERR_INVALID_ARG


_SYMM_SCRIPT = r"""
import torch, torch.distributed as dist
torch.cuda.set_device(0)
dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
from paper_2006_16668_b200 import MoEConfig, make_inputs, binding as B, ep
cfg = MoEConfig("symm1", G=4, S=128, M=64, H=128, E=16, C=16, dtype="bf16", seed=3)
shape = B.make_shape(cfg)
ex = ep.SymmetricExchange(shape, 0, 1)
assert ex.buffer.numel() == B.gshard_moe_ep_p2p_buffer_bytes(shape, 1)
for phase in (0, 1, 2):
    assert ex.struct.rendezvous(None, phase, None) == 0, ex.error
inp = make_inputs(cfg, "cuda")
ws = B.alloc_workspace(shape)
y, l = torch.empty_like(inp["x"]), torch.zeros(1, device="cuda")
ep.forward_p2p(shape, 0, 1, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y, l, ex, None, ws)
y2, l2 = torch.empty_like(y), torch.zeros(1, device="cuda")
B.gshard_moe_top2_forward(shape, inp["x"], inp["wg"], inp["wi"], inp["wo"], inp["u"], y2, l2, None, None, ws)
torch.cuda.synchronize()
assert torch.equal(y.view(torch.int16), y2.view(torch.int16)) and torch.equal(l, l2)
dist.destroy_process_group()
print("SYMM_OK")
"""


def test_symmetric_exchange_single_rank():
    """ep.SymmetricExchange (torch symmetric memory: peer pointer table + barrier as the rendezvous)
    at world 1, all that one GPU can run; in a child process because it needs a process group."""
    import os
    import socket
    import subprocess
    import sys
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), PYTHONPATH=root)
    out = subprocess.run([sys.executable, "-c", _SYMM_SCRIPT], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "SYMM_OK" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]

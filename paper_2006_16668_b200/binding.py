"""Thin ctypes binding of ``include/gshard_moe.h``: same names, argument marshalling only.

torch tensors supply device memory and the current stream; every step of the layer runs
inside the CUDA library.  If the library has not been built the first call raises - there
is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_float, c_int, c_int32, c_size_t, c_uint32, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgshard_moe.so")

GSHARD_OK = 0
GSHARD_ERR_INVALID_ARG = 1
GSHARD_ERR_UNSUPPORTED_SHAPE = 2
GSHARD_ERR_WORKSPACE_TOO_SMALL = 3
GSHARD_ERR_CUDA = 4
GSHARD_ERR_ARCH = 5
GSHARD_ERR_TIMEOUT = 6
GSHARD_ERR_INTERNAL = 7
GSHARD_F32 = 0
GSHARD_BF16 = 1
GSHARD_FLAG_SAVE_FOR_BACKWARD = 1
GSHARD_FLAG_SECOND_SKIP_FREES_SLOT = 2
GSHARD_FLAG_SIMT_CONTRACTIONS = 4
GSHARD_FLAG_FUSED_FFN = 8
GSHARD_FLAG_UNFUSED_FFN = 16
GSHARD_FLAG_TWO_SM_MMA = 32
GSHARD_FLAG_GATHER_DISPATCH = 64
GSHARD_FLAG_GATE_CLUSTER = 128
GSHARD_FLAG_GATE_ONE_SM = 256
GSHARD_FLAG_ONE_SM_MMA = 512
GSHARD_FLAG_ADD_RESIDUAL = 1024
GSHARD_FLAG_PLAIN_STORES = 2048
GSHARD_FLAG_BWD_PAIRED_GEMMS = 4096
GSHARD_FLAG_TF32_EXPERTS = 8192
GSHARD_FLAG_COMPACT_SLOTS = 16384
GSHARD_FLAG_DEBUG_CHECKS = 32768
GSHARD_FLAG_BULK_DISPATCH = 65536


class gshard_moe_shape(Structure):
    _fields_ = [("G", c_int32), ("S", c_int32), ("M", c_int32), ("H", c_int32), ("E", c_int32),
                ("C", c_int32), ("dtype", c_int32), ("flags", c_uint32)]


class gshard_moe_routing(Structure):
    _fields_ = [(n, c_void_p) for n in ("expert_idx", "slot", "weight", "flags", "first_count",
                                        "total_count", "slot_token", "m", "l_aux_group", "stats")]


class gshard_moe_ep_layout(Structure):
    _fields_ = [("rank", c_int32), ("world", c_int32), ("groups_local", c_int32), ("experts_local", c_int32),
                ("group_begin", c_int32), ("expert_begin", c_int32), ("rows_local", c_int32),
                ("row_bytes", c_size_t), ("bytes_per_peer", c_size_t), ("local", gshard_moe_shape),
                ("ffn", gshard_moe_shape)]


ALL_TO_ALL_FN = ctypes.CFUNCTYPE(c_int, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p)
ALL_REDUCE_FN = ctypes.CFUNCTYPE(c_int, c_void_p, c_void_p, c_size_t, c_void_p)


class gshard_ep_comm(Structure):
    _fields_ = [("all_to_all", ALL_TO_ALL_FN), ("all_reduce_sum_f32", ALL_REDUCE_FN), ("user", c_void_p)]


RENDEZVOUS_FN = ctypes.CFUNCTYPE(c_int, c_void_p, c_int, c_void_p)


class gshard_ep_p2p(Structure):
    _fields_ = [("rendezvous", RENDEZVOUS_FN), ("user", c_void_p), ("peer_buffers", POINTER(c_void_p))]


class gshard_ep_nccl_state(Structure):
    _fields_ = [("opaque", c_void_p * 8)]


EXPORTS = {
    # name: (restype, argtypes)
    "gshard_version": (c_int, []),
    "gshard_status_string": (ctypes.c_char_p, [c_int]),
    "gshard_moe_top2_workspace_bytes": (c_size_t, [POINTER(gshard_moe_shape), c_int]),
    "gshard_moe_top2_context_bytes": (c_size_t, [POINTER(gshard_moe_shape)]),
    "gshard_moe_top2_host_staging_bytes": (c_size_t, [POINTER(gshard_moe_shape)]),
    "gshard_moe_top2_forward": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 7 +
                                [POINTER(gshard_moe_routing), c_void_p, c_void_p, c_size_t, c_void_p]),
    "gshard_moe_top2_forward_host": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 7 +
                                     [POINTER(gshard_moe_routing), c_void_p, c_size_t, c_void_p]),
    "gshard_moe_top2_forward_host_async": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 7 +
                                           [POINTER(gshard_moe_routing), c_void_p, c_size_t, c_void_p, c_size_t] +
                                           [c_void_p] * 6),
    "gshard_moe_top2_backward": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 6 + [c_float] +
                                 [c_void_p] * 5 + [c_size_t, c_void_p]),
    "gshard_moe_gate": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 6 + [c_size_t, c_void_p]),
    "gshard_moe_capacity": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 4 +
                            [POINTER(gshard_moe_routing), c_void_p, c_void_p, c_size_t, c_void_p]),
    "gshard_moe_capacity_static": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 4 +
                                   [POINTER(gshard_moe_routing), c_void_p, c_void_p]),
    "gshard_moe_dispatch": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 4),
    "gshard_moe_expert_ffn": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 5 + [c_size_t, c_void_p]),
    "gshard_moe_combine": (c_int, [POINTER(gshard_moe_shape)] + [c_void_p] * 6),
    "gshard_moe_ep_plan": (c_int, [POINTER(gshard_moe_shape), c_int, c_int, POINTER(gshard_moe_ep_layout)]),
    "gshard_moe_ep_p2p_buffer_bytes": (c_size_t, [POINTER(gshard_moe_shape), c_int]),
    "gshard_moe_top2_forward_ep_p2p": (c_int, [POINTER(gshard_moe_shape), c_int, c_int] + [c_void_p] * 7 +
                                       [POINTER(gshard_moe_routing), POINTER(gshard_ep_p2p), POINTER(gshard_ep_comm),
                                        c_void_p, c_size_t, c_void_p]),
    "gshard_ep_comm_from_nccl": (c_int, [c_void_p, c_int, POINTER(gshard_ep_nccl_state), POINTER(gshard_ep_comm)]),
    "gshard_moe_ep_regroup_host": (c_int, [POINTER(gshard_moe_ep_layout), c_void_p, c_void_p, c_size_t, c_int]),
    "gshard_moe_ep_workspace_bytes": (c_size_t, [POINTER(gshard_moe_shape), c_int]),
    "gshard_moe_ep_context_bytes": (c_size_t, [POINTER(gshard_moe_shape), c_int]),
    "gshard_moe_ep_backward_workspace_bytes": (c_size_t, [POINTER(gshard_moe_shape), c_int]),
    "gshard_moe_top2_forward_ep": (c_int, [POINTER(gshard_moe_shape), c_int, c_int] + [c_void_p] * 7 +
                                   [POINTER(gshard_moe_routing), c_void_p, POINTER(gshard_ep_comm), c_void_p, c_size_t,
                                    c_void_p]),
    "gshard_moe_top2_backward_ep": (c_int, [POINTER(gshard_moe_shape), c_int, c_int] + [c_void_p] * 6 + [c_float] +
                                    [c_void_p] * 4 + [POINTER(gshard_ep_comm), c_void_p, c_size_t, c_void_p]),
    "gshard_dense_ffn_workspace_bytes": (c_size_t, [ctypes.c_int64, c_int32, c_int32, c_int32]),
    "gshard_dense_ffn_forward": (c_int, [ctypes.c_int64, c_int32, c_int32, c_int32, c_uint32] + [c_void_p] * 5 +
                                 [c_size_t, c_void_p]),
    "gshard_moe_debug_wait_timeout": (c_int, [c_void_p, c_uint32, c_void_p]),
    "gshard_moe_check_routing": (c_int, [POINTER(gshard_moe_shape), POINTER(gshard_moe_routing), c_void_p, c_void_p]),
    "gshard_moe_last_device_status": (c_int, [c_void_p, c_void_p]),
    "gshard_moe_last_launch_count": (c_int, []),
    "gshard_moe_time_expert_ffn": (c_int, [c_void_p, c_void_p]),
}

_lib = None


def load():
    """Load the CUDA library; raises if it is missing (build it with __graft_entry__.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build the CUDA library first "
                "(python -c 'import __graft_entry__ as g; g.build()'); there is no fallback path")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


class GshardError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def _check(code: int, where: str):
    if code != GSHARD_OK:
        raise GshardError(code, where)


def status_string(code: int) -> str:
    return load().gshard_status_string(int(code)).decode()


def make_shape(cfg=None, *, G=None, S=None, M=None, H=None, E=None, C=None, dtype=None, flags=0) -> gshard_moe_shape:
    """Shape struct from a MoEConfig or explicit sizes; dtype is "f32" | "bf16"."""
    if cfg is not None:
        G, S, M, H, E, C = cfg.G, cfg.S, cfg.M, cfg.H, cfg.E, cfg.C
        dtype = cfg.dtype if dtype is None else dtype
    code = {"f32": GSHARD_F32, "bf16": GSHARD_BF16}[dtype]
    return gshard_moe_shape(G, S, M, H, E, C, code, flags)


def _p(t):
    """Device/host pointer of a tensor (or None)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(stream=None):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def alloc_routing(shape: gshard_moe_shape, device="cuda"):
    """Allocate every optional routing output; returns (dict of tensors, struct)."""
    G, S, E, C = shape.G, shape.S, shape.E, shape.C
    t = {
        "expert_idx": torch.empty(G, S, 2, dtype=torch.int32, device=device),
        "slot": torch.empty(G, S, 2, dtype=torch.int32, device=device),
        "weight": torch.empty(G, S, 2, dtype=torch.float32, device=device),
        "flags": torch.empty(G, S, dtype=torch.uint8, device=device),
        "first_count": torch.empty(G, E, dtype=torch.int32, device=device),
        "total_count": torch.empty(G, E, dtype=torch.int32, device=device),
        "slot_token": torch.empty(E, G, C, dtype=torch.int32, device=device),
        "m": torch.empty(G, E, dtype=torch.float32, device=device),
        "l_aux_group": torch.empty(G, dtype=torch.float32, device=device),
        "stats": torch.zeros(8, dtype=torch.int64, device=device),
    }
    return t, routing_struct(t)


def routing_struct(tensors: dict) -> gshard_moe_routing:
    r = gshard_moe_routing()
    for name, _ in gshard_moe_routing._fields_:
        setattr(r, name, _p(tensors.get(name)))
    return r


def gshard_moe_top2_workspace_bytes(shape, for_backward=False) -> int:
    return int(load().gshard_moe_top2_workspace_bytes(ctypes.byref(shape), int(bool(for_backward))))


def gshard_moe_top2_context_bytes(shape) -> int:
    return int(load().gshard_moe_top2_context_bytes(ctypes.byref(shape)))


def gshard_moe_top2_host_staging_bytes(shape) -> int:
    return int(load().gshard_moe_top2_host_staging_bytes(ctypes.byref(shape)))


def alloc_workspace(shape, for_backward=False, host_staging=False, device="cuda") -> torch.Tensor:
    n = gshard_moe_top2_workspace_bytes(shape, for_backward)
    if n == 0:
        raise GshardError(GSHARD_ERR_UNSUPPORTED_SHAPE, "workspace_bytes")
    if host_staging:
        n += gshard_moe_top2_host_staging_bytes(shape)
    return torch.empty(n, dtype=torch.uint8, device=device)


def gshard_moe_top2_forward(shape, x, wg, wi, wo, u, y, l_aux, routing_out=None, context=None,
                            workspace=None, stream=None):
    rp = ctypes.byref(routing_out) if routing_out is not None else None
    _check(load().gshard_moe_top2_forward(ctypes.byref(shape), _p(x), _p(wg), _p(wi), _p(wo), _p(u), _p(y),
                                          _p(l_aux), rp, _p(context), _p(workspace), workspace.numel(),
                                          _stream(stream)), "gshard_moe_top2_forward")


def gshard_moe_top2_forward_host(shape, x_host, wg, wi, wo, u_host, y_host, l_aux_host, routing_out=None,
                                 workspace=None, stream=None):
    rp = ctypes.byref(routing_out) if routing_out is not None else None
    _check(load().gshard_moe_top2_forward_host(ctypes.byref(shape), _p(x_host), _p(wg), _p(wi), _p(wo),
                                               _p(u_host), _p(y_host), _p(l_aux_host), rp, _p(workspace),
                                               workspace.numel(), _stream(stream)),
           "gshard_moe_top2_forward_host")


def gshard_moe_top2_forward_host_async(shape, x_host, wg, wi, wo, u_host, y_host, l_aux_host, routing_out,
                                       workspace, staging, copy_in_stream, compute_stream, copy_out_stream,
                                       ev_in, ev_done, ev_out):
    """Pipelined host-buffer forward: streams are torch.cuda.Stream, events torch.cuda.Event that
    have been recorded once (so that their handles exist).  Nothing is synchronised."""
    rp = ctypes.byref(routing_out) if routing_out is not None else None
    _check(load().gshard_moe_top2_forward_host_async(
        ctypes.byref(shape), _p(x_host), _p(wg), _p(wi), _p(wo), _p(u_host), _p(y_host), _p(l_aux_host), rp,
        _p(workspace), workspace.numel(), _p(staging), staging.numel(), copy_in_stream.cuda_stream,
        compute_stream.cuda_stream, copy_out_stream.cuda_stream, ev_in.cuda_event, ev_done.cuda_event,
        ev_out.cuda_event), "gshard_moe_top2_forward_host_async")


def gshard_moe_top2_backward(shape, x, wg, wi, wo, context, dy, l_aux_weight, dx, dwg, dwi, dwo,
                             workspace=None, stream=None):
    _check(load().gshard_moe_top2_backward(ctypes.byref(shape), _p(x), _p(wg), _p(wi), _p(wo), _p(context),
                                           _p(dy), float(l_aux_weight), _p(dx), _p(dwg), _p(dwi), _p(dwo),
                                           _p(workspace), workspace.numel(), _stream(stream)),
           "gshard_moe_top2_backward")


def gshard_moe_gate(shape, x, wg, expert_idx, gate12, m, workspace, stream=None):
    _check(load().gshard_moe_gate(ctypes.byref(shape), _p(x), _p(wg), _p(expert_idx), _p(gate12), _p(m),
                                  _p(workspace), workspace.numel(), _stream(stream)), "gshard_moe_gate")


def gshard_moe_capacity(shape, expert_idx, gate12, u, m, routing_out, l_aux, workspace, stream=None):
    _check(load().gshard_moe_capacity(ctypes.byref(shape), _p(expert_idx), _p(gate12), _p(u), _p(m),
                                      ctypes.byref(routing_out), _p(l_aux), _p(workspace), workspace.numel(),
                                      _stream(stream)), "gshard_moe_capacity")


def gshard_moe_capacity_static(shape, expert_idx, gate12, u, m, routing_out, l_aux, stream=None):
    """Capacity assignment without a workspace: for callers that cannot allocate device memory
    (scratch is a fixed array inside the library; G <= 4096; every routing output required)."""
    _check(load().gshard_moe_capacity_static(ctypes.byref(shape), _p(expert_idx), _p(gate12), _p(u), _p(m),
                                             ctypes.byref(routing_out), _p(l_aux), _stream(stream)),
           "gshard_moe_capacity_static")


def gshard_moe_dispatch(shape, x, slot_token, buf, stream=None):
    _check(load().gshard_moe_dispatch(ctypes.byref(shape), _p(x), _p(slot_token), _p(buf), _stream(stream)),
           "gshard_moe_dispatch")


def gshard_moe_expert_ffn(shape, buf, wi, wo, out, workspace, stream=None):
    _check(load().gshard_moe_expert_ffn(ctypes.byref(shape), _p(buf), _p(wi), _p(wo), _p(out), _p(workspace),
                                        workspace.numel(), _stream(stream)), "gshard_moe_expert_ffn")


def gshard_moe_combine(shape, out, expert_idx, slot, weight, y, stream=None):
    _check(load().gshard_moe_combine(ctypes.byref(shape), _p(out), _p(expert_idx), _p(slot), _p(weight), _p(y),
                                     _stream(stream)), "gshard_moe_combine")


def gshard_moe_ep_plan(shape, rank, world) -> gshard_moe_ep_layout:
    """Host-only partitioning arithmetic of the expert-parallel form (works without a GPU)."""
    layout = gshard_moe_ep_layout()
    _check(load().gshard_moe_ep_plan(ctypes.byref(shape), int(rank), int(world), ctypes.byref(layout)),
           "gshard_moe_ep_plan")
    return layout


def gshard_moe_ep_regroup_host(layout, src, dst, inverse=False):
    """Permutes HOST tensors (rows of equal byte length) between the AllToAll layout and the expert
    FFN's layout; src and dst are contiguous CPU tensors of world * experts_local * rows_local rows."""
    rows = layout.world * layout.experts_local * layout.rows_local
    row_bytes = src.numel() * src.element_size() // rows
    assert src.is_contiguous() and dst.is_contiguous() and src.numel() == dst.numel()
    _check(load().gshard_moe_ep_regroup_host(ctypes.byref(layout), src.data_ptr(), dst.data_ptr(), row_bytes,
                                             int(bool(inverse))), "gshard_moe_ep_regroup_host")


def gshard_moe_ep_p2p_buffer_bytes(shape, world) -> int:
    return int(load().gshard_moe_ep_p2p_buffer_bytes(ctypes.byref(shape), int(world)))


def gshard_moe_top2_forward_ep_p2p(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local, l_aux,
                                   routing_out, p2p, comm, workspace, stream=None):
    rp = ctypes.byref(routing_out) if routing_out is not None else None
    cp = ctypes.byref(comm) if comm is not None else None
    _check(load().gshard_moe_top2_forward_ep_p2p(ctypes.byref(shape), int(rank), int(world), _p(x_local), _p(wg),
                                                 _p(wi_local), _p(wo_local), _p(u_local), _p(y_local), _p(l_aux), rp,
                                                 ctypes.byref(p2p), cp, _p(workspace), workspace.numel(), _stream(stream)),
           "gshard_moe_top2_forward_ep_p2p")


def gshard_ep_comm_from_nccl(nccl_comm: int, world: int):
    """(comm, state): a gshard_ep_comm whose collectives are NCCL calls on the given ncclComm_t handle;
    keep both objects (and the communicator) alive while the comm is in use."""
    state, comm = gshard_ep_nccl_state(), gshard_ep_comm()
    _check(load().gshard_ep_comm_from_nccl(nccl_comm, int(world), ctypes.byref(state), ctypes.byref(comm)),
           "gshard_ep_comm_from_nccl")
    return comm, state


def gshard_moe_ep_workspace_bytes(shape, world) -> int:
    return int(load().gshard_moe_ep_workspace_bytes(ctypes.byref(shape), int(world)))


def gshard_moe_ep_context_bytes(shape, world) -> int:
    return int(load().gshard_moe_ep_context_bytes(ctypes.byref(shape), int(world)))


def gshard_moe_ep_backward_workspace_bytes(shape, world) -> int:
    return int(load().gshard_moe_ep_backward_workspace_bytes(ctypes.byref(shape), int(world)))


def gshard_moe_top2_forward_ep(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local, l_aux,
                               routing_out=None, comm=None, workspace=None, stream=None, context=None):
    rp = ctypes.byref(routing_out) if routing_out is not None else None
    cp = ctypes.byref(comm) if comm is not None else None
    _check(load().gshard_moe_top2_forward_ep(ctypes.byref(shape), int(rank), int(world), _p(x_local), _p(wg),
                                             _p(wi_local), _p(wo_local), _p(u_local), _p(y_local), _p(l_aux), rp,
                                             _p(context), cp, _p(workspace), workspace.numel(), _stream(stream)),
           "gshard_moe_top2_forward_ep")


def gshard_moe_top2_backward_ep(shape, rank, world, x_local, wg, wi_local, wo_local, context, dy_local, l_aux_weight,
                                dx_local, dwg, dwi_local, dwo_local, comm=None, workspace=None, stream=None):
    cp = ctypes.byref(comm) if comm is not None else None
    _check(load().gshard_moe_top2_backward_ep(ctypes.byref(shape), int(rank), int(world), _p(x_local), _p(wg),
                                              _p(wi_local), _p(wo_local), _p(context), _p(dy_local),
                                              float(l_aux_weight), _p(dx_local), _p(dwg), _p(dwi_local), _p(dwo_local),
                                              cp, _p(workspace), workspace.numel(), _stream(stream)),
           "gshard_moe_top2_backward_ep")


def _dtype_code(t) -> int:
    return GSHARD_BF16 if t.dtype == torch.bfloat16 else GSHARD_F32


def gshard_dense_ffn_workspace_bytes(n_tokens, M, H, dtype_code) -> int:
    return int(load().gshard_dense_ffn_workspace_bytes(int(n_tokens), int(M), int(H), int(dtype_code)))


def gshard_dense_ffn_forward(x, wi, wo, y, workspace, stream=None, flags=0):
    """y = relu(x . wi) . wo for x [n, M], wi [M, H], wo [H, M] (the dense Transformer FFN)."""
    n, M = x.shape
    H = wi.shape[1]
    _check(load().gshard_dense_ffn_forward(n, M, H, _dtype_code(x), flags, _p(x), _p(wi), _p(wo), _p(y), _p(workspace),
                                           workspace.numel(), _stream(stream)), "gshard_dense_ffn_forward")


def gshard_moe_debug_wait_timeout(workspace, limit_us=200, stream=None):
    _check(load().gshard_moe_debug_wait_timeout(_p(workspace), int(limit_us), _stream(stream)),
           "gshard_moe_debug_wait_timeout")


def gshard_moe_check_routing(shape, routing, workspace, stream=None):
    _check(load().gshard_moe_check_routing(ctypes.byref(shape), ctypes.byref(routing), _p(workspace), _stream(stream)),
           "gshard_moe_check_routing")


def gshard_moe_last_device_status(workspace, stream=None) -> int:
    return int(load().gshard_moe_last_device_status(_p(workspace), _stream(stream)))


def gshard_moe_last_launch_count() -> int:
    return int(load().gshard_moe_last_launch_count())


def gshard_moe_time_expert_ffn(start_event, stop_event):
    """Arm torch.cuda.Event pair (enable_timing=True, already recorded once so that their handles
    exist) around the expert FFN of the next forward call; (None, None) disarms."""
    s = None if start_event is None else start_event.cuda_event
    e = None if stop_event is None else stop_event.cuda_event
    _check(load().gshard_moe_time_expert_ffn(s, e), "gshard_moe_time_expert_ffn")

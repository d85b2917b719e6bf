"""Expert-parallel forward over several GPUs, one process per GPU: the collectives of
``gshard_moe_top2_forward_ep`` backed by ``torch.distributed`` (NCCL over NVLink on GPUs).

The layer itself - gating, capacity, dispatch, the regrouping of received slabs, the expert FFN and
the combine - runs inside the CUDA library; this module only hands it two callbacks that move bytes
between ranks (Algorithm 2's AllToAll before and after the expert FFN, and the sum of the per-rank
shares of l_aux) and slices each rank's share out of global tensors.
"""
from __future__ import annotations

import ctypes
import traceback

import torch
import torch.distributed as dist

from . import binding as B


class TorchDistComm:
    """A ``gshard_ep_comm`` whose all-to-all and all-reduce are torch.distributed collectives.

    The library passes raw device pointers; they always point into a tensor of the call (workspace,
    context, the l_aux scalar, dwg), so they are turned back into views of the tensors registered
    here.  torch's NCCL collectives order themselves after the current stream and make it wait for
    their completion, which is the contract of the callbacks as long as the library call is made on
    torch's current stream.
    """

    def __init__(self, tensors, group=None):
        self.tensors = [t for t in tensors if t is not None]
        self.group = group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.error = None
        self._a2a = B.ALL_TO_ALL_FN(self._all_to_all)        # keep the thunks alive
        self._ar = B.ALL_REDUCE_FN(self._all_reduce)
        self.struct = B.gshard_ep_comm(self._a2a, self._ar, None)

    def _view(self, ptr: int, nbytes: int) -> torch.Tensor:
        for t in self.tensors:
            off = ptr - t.data_ptr()
            if 0 <= off and off + nbytes <= t.numel() * t.element_size():
                return t.view(-1).view(torch.uint8)[off:off + nbytes]
        raise ValueError("collective buffer outside the tensors of the call")

    def _all_to_all(self, user, send, recv, bytes_per_peer, stream):
        try:
            n = bytes_per_peer * self.world
            dist.all_to_all_single(self._view(recv, n), self._view(send, n), group=self.group)
            return 0
        except Exception:                                    # an exception must not cross the C frame
            self.error = traceback.format_exc()
            return 1

    def _all_reduce(self, user, buf, count, stream):
        try:
            dist.all_reduce(self._view(buf, 4 * count).view(torch.float32), op=dist.ReduceOp.SUM, group=self.group)
            return 0
        except Exception:
            self.error = traceback.format_exc()
            return 1


class NcclComm:
    """The collectives as direct NCCL calls from inside the library (no Python in the data path).

    Creates its own ncclComm_t with the NCCL library torch has loaded: rank 0 draws the unique id, the
    process group (any backend) carries it to the other ranks, every rank joins with
    ncclCommInitRank.  One GPU per process, the current device.
    """

    class _UniqueId(ctypes.Structure):
        _fields_ = [("internal", ctypes.c_byte * 128)]

    def __init__(self, rank: int, world: int, group=None):
        self.lib = self._load_nccl()
        self.rank, self.world = rank, world
        uid = self._UniqueId()
        if rank == 0:
            self._ok(self.lib.ncclGetUniqueId(ctypes.byref(uid)), "ncclGetUniqueId")
        if world > 1:
            payload = [bytes(uid.internal) if rank == 0 else None]
            dist.broadcast_object_list(payload, src=0, group=group)
            ctypes.memmove(ctypes.byref(uid), payload[0], 128)
        self.handle = ctypes.c_void_p()
        self.lib.ncclCommInitRank.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int, self._UniqueId, ctypes.c_int]
        self._ok(self.lib.ncclCommInitRank(ctypes.byref(self.handle), world, uid, rank), "ncclCommInitRank")
        self.struct, self._state = B.gshard_ep_comm_from_nccl(self.handle.value, world)

    @staticmethod
    def _load_nccl():
        import glob
        import os
        cands = []
        try:
            import nvidia.nccl
            for d in list(getattr(nvidia.nccl, "__path__", [])):       # a namespace package has no __file__
                cands += sorted(glob.glob(os.path.join(d, "lib", "libnccl.so*")))
        except ImportError:
            pass
        for path in cands + ["libnccl.so.2"]:
            try:
                return ctypes.CDLL(path, mode=ctypes.RTLD_GLOBAL)
            except OSError:
                continue
        raise ImportError("no NCCL library found")

    @staticmethod
    def _ok(code, what):
        if code != 0:
            raise RuntimeError(f"{what} failed with NCCL result {code}")

    def close(self):
        if self.handle:
            self.lib.ncclCommDestroy.argtypes = [ctypes.c_void_p]
            self.lib.ncclCommDestroy(self.handle)
            self.handle = ctypes.c_void_p()


class SymmetricExchange:
    """The exchange buffers and rendezvous of ``gshard_moe_top2_forward_ep_p2p`` on torch's symmetric
    memory: every rank allocates its buffer from the symmetric allocator, the rendezvous maps all of
    them into every process (``buffer_ptrs``), and the ordering callback is the allocation's own
    barrier, enqueued on the current stream (each rank runs on its own GPU, so the barrier kernels of
    different ranks never share one).  The library call must be made on torch's current stream.
    """

    def __init__(self, shape, rank: int, world: int, group=None):
        import torch.distributed._symmetric_memory as symm
        nbytes = B.gshard_moe_ep_p2p_buffer_bytes(shape, world)
        if nbytes == 0:
            raise ValueError("shape does not split over this many ranks")
        self.rank, self.world, self.error = rank, world, None
        self.buffer = symm.empty(nbytes, dtype=torch.uint8, device=torch.device("cuda", torch.cuda.current_device()))
        group = group if group is not None else dist.group.WORLD
        self.handle = symm.rendezvous(self.buffer, group.group_name)
        ptrs = [int(p) for p in self.handle.buffer_ptrs]
        if len(ptrs) != world or ptrs[rank] != self.buffer.data_ptr():
            raise RuntimeError("symmetric memory rendezvous returned an unexpected pointer table")
        self._ptrs = (ctypes.c_void_p * world)(*ptrs)
        self._rv = B.RENDEZVOUS_FN(self._rendezvous)
        self.struct = B.gshard_ep_p2p(self._rv, None, self._ptrs)

    def _rendezvous(self, user, phase, stream):
        try:
            self.handle.barrier(channel=int(phase))
            return 0
        except Exception:                                    # an exception must not cross the C frame
            self.error = traceback.format_exc()
            return 1


def forward_p2p(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local, l_aux, exchange,
                routing_out=None, workspace=None, comm=None):
    """One expert-parallel forward with the exchange fused into the dispatch and combine kernels
    (peer stores / peer loads through `exchange`, a SymmetricExchange); `comm` (a NcclComm) sums
    l_aux over the ranks, without it l_aux is this rank's share."""
    try:
        B.gshard_moe_top2_forward_ep_p2p(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local, l_aux,
                                         routing_out, exchange.struct, comm.struct if comm else None, workspace)
    except B.GshardError:
        if exchange.error:
            raise RuntimeError("the rendezvous of the expert-parallel forward failed:\n" + exchange.error)
        raise


def local_slices(layout: B.gshard_moe_ep_layout):
    """(group slice, expert slice) of this rank in the global tensors."""
    g0, e0 = layout.group_begin, layout.expert_begin
    return slice(g0, g0 + layout.groups_local), slice(e0, e0 + layout.experts_local)


def _call(fn, comm, what):
    try:
        fn(comm.struct if comm is not None else None)
    except B.GshardError:
        if comm is not None and getattr(comm, "error", None):
            raise RuntimeError(f"a collective of the expert-parallel {what} failed:\n" + comm.error)
        raise


def forward(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local, l_aux, routing_out=None,
            workspace=None, group=None, comm=None, context=None):
    """One expert-parallel forward on this rank (global `shape`); the process group must be
    initialised when world > 1.  Enqueues on torch's current stream.  comm: a NcclComm to reuse, else
    the collectives go through torch.distributed.  context: with SAVE_FOR_BACKWARD, a uint8 tensor of
    gshard_moe_ep_context_bytes(shape, world) for `backward`."""
    if comm is None and world > 1:
        comm = TorchDistComm([workspace, context, l_aux], group)
    _call(lambda c: B.gshard_moe_top2_forward_ep(shape, rank, world, x_local, wg, wi_local, wo_local, u_local, y_local,
                                                 l_aux, routing_out, c, workspace, context=context), comm, "forward")


def backward(shape, rank, world, x_local, wg, wi_local, wo_local, context, dy_local, l_aux_weight, dx_local, dwg,
             dwi_local, dwo_local, workspace=None, group=None, comm=None):
    """The backward of `forward` on this rank; dwg ends as the sum over the ranks."""
    if comm is None and world > 1:
        comm = TorchDistComm([workspace, dwg], group)
    _call(lambda c: B.gshard_moe_top2_backward_ep(shape, rank, world, x_local, wg, wi_local, wo_local, context, dy_local,
                                                  l_aux_weight, dx_local, dwg, dwi_local, dwo_local, c, workspace),
          comm, "backward")

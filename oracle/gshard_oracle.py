"""ctypes front end of the CPU oracle (``gshard_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, ``__graft_entry__.smoke()`` and the CPU-baseline
leg of ``bench.py`` are the only callers.  Nothing here touches CUDA or the
product package; arrays are numpy, floating point is double.

Each function marshals arguments for one C function; the arithmetic and the
citation of the passage it follows (Algorithm 1, eq. (1)-(3), Algorithm 2 of the
GShard paper) live in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gshard_oracle.c")
_SO = os.path.join(_HERE, "libgshard_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over tokens/rows only)."""
    stale = (not os.path.exists(_SO)) or os.path.getmtime(_SO) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _ptr(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.gso_capacity.restype = ctypes.c_double
        _lib.gso_forward.restype = ctypes.c_double
        _lib.gso_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().gso_num_threads())


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


c_f = ctypes.c_float
c_d = ctypes.c_double
c_i = ctypes.c_int32
c_u8 = ctypes.c_uint8
c_i8 = ctypes.c_int8


def gates(x, wg):
    """softmax(x . wg) for one group: x [S,M], wg [M,E] -> (logits, p) [S,E] float64."""
    x, wg = _f32(x), _f32(wg)
    S, M = x.shape
    E = wg.shape[1]
    logits = np.empty((S, E), np.float64)
    p = np.empty((S, E), np.float64)
    lib().gso_gates(_ptr(x, c_f), _ptr(wg, c_f), S, M, E, _ptr(logits, c_d), _ptr(p, c_d))
    return logits, p


def mean_gates(p):
    p = np.ascontiguousarray(p, np.float64)
    S, E = p.shape
    m = np.empty(E, np.float64)
    lib().gso_mean_gates(_ptr(p, c_d), S, E, _ptr(m, c_d))
    return m


def top2(p):
    """-> e1, e2 (int32), g1, g2, g3 (float64; g3 = third largest gate or -1)."""
    p = np.ascontiguousarray(p, np.float64)
    S, E = p.shape
    e1 = np.empty(S, np.int32)
    e2 = np.empty(S, np.int32)
    g1 = np.empty(S, np.float64)
    g2 = np.empty(S, np.float64)
    g3 = np.empty(S, np.float64)
    lib().gso_top2(_ptr(p, c_d), S, E, _ptr(e1, c_i), _ptr(e2, c_i), _ptr(g1, c_d),
                   _ptr(g2, c_d), _ptr(g3, c_d))
    return e1, e2, g1, g2, g3


@dataclass
class GroupRouting:
    slot: np.ndarray          # [S,2] int32
    weight: np.ndarray        # [S,2] float64
    flags: np.ndarray         # [S] uint8
    first_count: np.ndarray   # [E] int32
    total_count: np.ndarray   # [E] int32
    l_aux: float


def capacity(E, C, e1, e2, g1, g2, u, m, pass_override=None, variant_a=False) -> GroupRouting:
    """The two token loops of Algorithm 1 plus l_aux, for one group."""
    e1 = np.ascontiguousarray(e1, np.int32)
    e2 = np.ascontiguousarray(e2, np.int32)
    g1 = np.ascontiguousarray(g1, np.float64)
    g2 = np.ascontiguousarray(g2, np.float64)
    u = _f32(u)
    m = np.ascontiguousarray(m, np.float64)
    S = e1.shape[0]
    po = None if pass_override is None else np.ascontiguousarray(pass_override, np.int8)
    slot = np.empty((S, 2), np.int32)
    weight = np.empty((S, 2), np.float64)
    flags = np.empty(S, np.uint8)
    fc = np.empty(E, np.int32)
    tc = np.empty(E, np.int32)
    la = lib().gso_capacity(S, E, C, _ptr(e1, c_i), _ptr(e2, c_i), _ptr(g1, c_d), _ptr(g2, c_d),
                            _ptr(u, c_f), _ptr(m, c_d), _ptr(po, c_i8), int(bool(variant_a)),
                            _ptr(slot, c_i), _ptr(weight, c_d), _ptr(flags, c_u8),
                            _ptr(fc, c_i), _ptr(tc, c_i))
    return GroupRouting(slot, weight, flags, fc, tc, float(la))


def ffn_rows(xrows, wi_e, wo_e, want_h=False):
    """FFN_e(x) = wo_e . relu(wi_e . x) for each row: xrows [R,M], wi_e [M,H], wo_e [H,M]."""
    xrows, wi_e, wo_e = _f32(xrows), _f32(wi_e), _f32(wo_e)
    R, M = xrows.shape
    H = wi_e.shape[1]
    assert wi_e.shape == (M, H) and wo_e.shape == (H, M)
    out = np.empty((R, M), np.float64)
    h = np.empty((R, H), np.float64) if want_h else None
    lib().gso_ffn_rows(_ptr(xrows, c_f), R, _ptr(wi_e, c_f), _ptr(wo_e, c_f), M, H,
                       _ptr(out, c_d), _ptr(h, c_d))
    return (out, h) if want_h else out


@dataclass
class Forward:
    y: np.ndarray | None       # [G,S,M] float64
    l_aux: float
    expert_idx: np.ndarray     # [G,S,2]
    slot: np.ndarray           # [G,S,2]
    weight: np.ndarray         # [G,S,2] float64
    flags: np.ndarray          # [G,S]
    first_count: np.ndarray    # [G,E]
    total_count: np.ndarray    # [G,E]
    slot_token: np.ndarray     # [E,G,C]
    m: np.ndarray              # [G,E]
    l_aux_group: np.ndarray    # [G]


def forward(x, wg, wi, wo, u, C, variant_a=False, want_y=True) -> Forward:
    """Whole layer: x [G,S,M], wg [M,E], wi [E,M,H], wo [E,H,M], u [G,S]."""
    x, wg, u = _f32(x), _f32(wg), _f32(u)
    G, S, M = x.shape
    E = wg.shape[1]
    if want_y:
        wi, wo = _f32(wi), _f32(wo)
        H = wi.shape[2]
        assert wi.shape == (E, M, H) and wo.shape == (E, H, M)
    else:
        H = 0
    y = np.empty((G, S, M), np.float64) if want_y else None
    ei = np.empty((G, S, 2), np.int32)
    slot = np.empty((G, S, 2), np.int32)
    weight = np.empty((G, S, 2), np.float64)
    flags = np.empty((G, S), np.uint8)
    fc = np.empty((G, E), np.int32)
    tc = np.empty((G, E), np.int32)
    st = np.empty((E, G, C), np.int32)
    m = np.empty((G, E), np.float64)
    lg = np.empty(G, np.float64)
    la = lib().gso_forward(G, S, M, H, E, C, _ptr(x, c_f), _ptr(wg, c_f),
                           _ptr(wi if want_y else None, c_f), _ptr(wo if want_y else None, c_f),
                           _ptr(u, c_f), int(bool(variant_a)), _ptr(y, c_d), _ptr(ei, c_i),
                           _ptr(slot, c_i), _ptr(weight, c_d), _ptr(flags, c_u8), _ptr(fc, c_i),
                           _ptr(tc, c_i), _ptr(st, c_i), _ptr(m, c_d), _ptr(lg, c_d))
    return Forward(y, float(la), ei, slot, weight, flags, fc, tc, st, m, lg)


def ffn_rows_backward(xrows, dout, wi_e, wo_e):
    """Expert path backward for the rows of one expert -> (dxrows, dwi_e, dwo_e) float64."""
    xrows, wi_e, wo_e = _f32(xrows), _f32(wi_e), _f32(wo_e)
    dout = np.ascontiguousarray(dout, np.float64)
    R, M = xrows.shape
    H = wi_e.shape[1]
    dxr = np.zeros((R, M), np.float64)
    dwi = np.zeros((M, H), np.float64)
    dwo = np.zeros((H, M), np.float64)
    lib().gso_ffn_rows_backward(_ptr(xrows, c_f), _ptr(dout, c_d), R, _ptr(wi_e, c_f), _ptr(wo_e, c_f), M, H,
                                _ptr(dxr, c_d), _ptr(dwi, c_d), _ptr(dwo, c_d))
    return dxr, dwi, dwo


def gate_row_backward(p_row, e1, e2, dw1, dw2, first_count_g, S, G, k_aux):
    """Softmax/aux-loss backward of one token -> dlogit [E] float64."""
    p_row = np.ascontiguousarray(p_row, np.float64)
    fc = np.ascontiguousarray(first_count_g, np.int32)
    E = p_row.shape[0]
    dl = np.empty(E, np.float64)
    lib().gso_gate_row_backward(_ptr(p_row, c_d), E, int(e1), int(e2), ctypes.c_double(dw1), ctypes.c_double(dw2),
                                _ptr(fc, c_i), int(S), int(G), ctypes.c_double(k_aux), _ptr(dl, c_d))
    return dl


def backward(x, wg, wi, wo, fwd: Forward, dy, k_aux):
    """Gradients of <dy,y> + k_aux*l_aux with fwd's routing frozen -> dx, dwg, dwi, dwo."""
    x, wg, wi, wo, dy = _f32(x), _f32(wg), _f32(wi), _f32(wo), _f32(dy)
    G, S, M = x.shape
    E, _, H = wi.shape
    C = fwd.slot_token.shape[2]
    dx = np.empty((G, S, M), np.float64)
    dwg = np.empty((M, E), np.float64)
    dwi = np.empty((E, M, H), np.float64)
    dwo = np.empty((E, H, M), np.float64)
    ei = np.ascontiguousarray(fwd.expert_idx, np.int32)
    slot = np.ascontiguousarray(fwd.slot, np.int32)
    fc = np.ascontiguousarray(fwd.first_count, np.int32)
    lib().gso_backward(G, S, M, H, E, C, _ptr(x, c_f), _ptr(wg, c_f), _ptr(wi, c_f), _ptr(wo, c_f),
                       _ptr(ei, c_i), _ptr(slot, c_i), _ptr(fc, c_i), _ptr(dy, c_f),
                       ctypes.c_double(k_aux), _ptr(dx, c_d), _ptr(dwg, c_d), _ptr(dwi, c_d),
                       _ptr(dwo, c_d))
    return dx, dwg, dwi, dwo

"""ctypes wrapper around the C oracle (oracle/cmoe_oracle.c).  Test infrastructure only.

Every function takes the plain numpy arrays of a layer (the dict layout of the
seeded generator) and returns numpy arrays; no arithmetic happens here.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build


class _Desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("d", "d_ff", "E", "G", "r", "k")] + [
        ("C", C.c_void_p), ("R", C.c_void_p), ("b_c", C.c_void_p), ("b_e", C.c_void_p),
        ("B1", C.c_void_p), ("B2", C.c_void_p),
        ("U1q", C.c_void_p), ("V1q", C.c_void_p), ("U2q", C.c_void_p), ("V2q", C.c_void_p),
        ("U1s", C.c_void_p), ("V1s", C.c_void_p), ("U2s", C.c_void_p), ("V2s", C.c_void_p),
        ("base_is_bf16", C.c_int32),
    ]


_lib = None


def load(path: str):
    """Open an oracle shared object and declare its prototypes."""
    if True:
        L = C.CDLL(path)
        L.cmoe_ref_half_to_float.restype = C.c_float
        L.cmoe_ref_half_to_float.argtypes = [C.c_uint16]
        L.cmoe_ref_bf16_to_float.restype = C.c_float
        L.cmoe_ref_bf16_to_float.argtypes = [C.c_uint16]
        L.cmoe_ref_dequant.restype = C.c_float
        L.cmoe_ref_dequant.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.cmoe_ref_route.restype = C.c_int
        L.cmoe_ref_route.argtypes = [C.POINTER(_Desc), C.c_void_p, C.c_int32] + [C.c_void_p] * 5
        L.cmoe_ref_form_weight.restype = C.c_int
        L.cmoe_ref_form_weight.argtypes = [C.POINTER(_Desc), C.c_int32, C.c_int32, C.c_void_p]
        L.cmoe_ref_forward.restype = C.c_int
        L.cmoe_ref_forward.argtypes = [C.POINTER(_Desc), C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
        L.cmoe_ref_param_count.restype = None
        L.cmoe_ref_param_count.argtypes = [C.POINTER(_Desc), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.cmoe_ref_expert_stats.restype = C.c_int
        L.cmoe_ref_expert_stats.argtypes = [C.POINTER(_Desc), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_float, C.c_void_p]
        L.cmoe_ref_route_g1.restype = C.c_int
        L.cmoe_ref_route_g1.argtypes = [C.POINTER(_Desc), C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 3
        L.cmoe_ref_forward_g1.restype = C.c_int
        L.cmoe_ref_forward_g1.argtypes = [C.POINTER(_Desc), C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
        L.cmoe_ref_num_threads.restype = C.c_int
    return L


def lib():
    global _lib
    if _lib is None:
        _lib = load(_build.build())
    return _lib


def _ptr(a):
    return None if a is None or a.size == 0 else a.ctypes.data


class Layer:
    """Holds contiguous host copies of a layer's arrays and the C descriptor over them."""

    def __init__(self, layer: dict):
        s = layer["shape"]
        self.shape = s
        keep = {}
        bf16 = layer.get("base_dtype", "fp16") == "bf16"      # B1, B2 then hold bfloat16 bit patterns as uint16
        for name, dt in (("C", np.float32), ("R", np.float32), ("b_c", np.float32), ("b_e", np.float32),
                         ("B1", np.uint16 if bf16 else np.float16), ("B2", np.uint16 if bf16 else np.float16),
                         ("U1q", np.uint8), ("V1q", np.uint8), ("U2q", np.uint8), ("V2q", np.uint8),
                         ("U1s", np.float16), ("V1s", np.float16), ("U2s", np.float16), ("V2s", np.float16)):
            a = layer.get(name)
            keep[name] = None if a is None else np.ascontiguousarray(a, dtype=dt)
        self._keep = keep
        self.desc = _Desc(s.d, s.d_ff, s.E, s.G, s.r, s.k, *[_ptr(keep[n]) for n in (
            "C", "R", "b_c", "b_e", "B1", "B2", "U1q", "V1q", "U2q", "V2q", "U1s", "V1s", "U2s", "V2s")], 1 if bf16 else 0)

    def route(self, x: np.ndarray):
        """-> dict(cluster_id [T], expert_slot [T][k], gates [T][k], z [T][G], l [T][K])."""
        s = self.shape
        x = np.ascontiguousarray(x, dtype=np.float16)
        T = x.shape[0]
        cid = np.empty(T, np.int32)
        slot = np.empty((T, s.k), np.int32)
        gates = np.empty((T, s.k), np.float32)
        z = np.empty((T, s.G), np.float32)
        l = np.empty((T, s.K), np.float32)
        rc = lib().cmoe_ref_route(C.byref(self.desc), _ptr(x), T, _ptr(cid), _ptr(slot), _ptr(gates), _ptr(z), _ptr(l))
        if rc:
            raise ValueError("oracle rejected the descriptor")
        return dict(cluster_id=cid, expert_slot=slot, gates=gates, z=z, l=l)

    def forward(self, x: np.ndarray, token_idx=None) -> np.ndarray:
        """y (fp32) for all tokens, or for the listed ones."""
        s = self.shape
        x = np.ascontiguousarray(x, dtype=np.float16)
        T = x.shape[0]
        if token_idx is None:
            idx, n = None, T
        else:
            idx = np.ascontiguousarray(token_idx, dtype=np.int32)
            n = idx.size
        y = np.zeros((n, s.d), np.float32)
        rc = lib().cmoe_ref_forward(C.byref(self.desc), _ptr(x), T, _ptr(idx), n, _ptr(y))
        if rc:
            raise ValueError("oracle rejected its arguments")
        return y

    def route_g1(self, x: np.ndarray, g1: int):
        """g1 clusters per token -> dict(cluster_id [T][g1], expert_slot [T][g1][k], gates [T][g1][k])."""
        s = self.shape
        x = np.ascontiguousarray(x, dtype=np.float16)
        T = x.shape[0]
        cid = np.empty((T, g1), np.int32)
        slot = np.empty((T, g1, s.k), np.int32)
        gates = np.empty((T, g1, s.k), np.float32)
        if lib().cmoe_ref_route_g1(C.byref(self.desc), _ptr(x), T, g1, _ptr(cid), _ptr(slot), _ptr(gates)):
            raise ValueError("oracle rejected its arguments")
        return dict(cluster_id=cid, expert_slot=slot, gates=gates)

    def forward_g1(self, x: np.ndarray, g1: int, token_idx=None) -> np.ndarray:
        """y (fp32) with g1 clusters per token, for all tokens or for the listed ones."""
        s = self.shape
        x = np.ascontiguousarray(x, dtype=np.float16)
        T = x.shape[0]
        if token_idx is None:
            idx, n = None, T
        else:
            idx = np.ascontiguousarray(token_idx, dtype=np.int32)
            n = idx.size
        y = np.zeros((n, s.d), np.float32)
        if lib().cmoe_ref_forward_g1(C.byref(self.desc), _ptr(x), T, g1, _ptr(idx), n, _ptr(y)):
            raise ValueError("oracle rejected its arguments")
        return y

    def weight(self, e: int, which: int) -> np.ndarray:
        s = self.shape
        shp = (s.d, s.d_ff) if which == 1 else (s.d_ff, s.d)
        W = np.empty(shp, np.float32)
        rc = lib().cmoe_ref_form_weight(C.byref(self.desc), e, which, _ptr(W))
        if rc:
            raise ValueError("oracle rejected its arguments")
        return W

    def expert_stats(self, x: np.ndarray, mu: np.ndarray | None = None, beta: float = 0.05):
        """-> loads [E] int32, xbar [E][d] fp32, cov (float); `mu` ([E][d] fp32, contiguous) is updated in place."""
        s = self.shape
        x = np.ascontiguousarray(x, dtype=np.float16)
        loads = np.zeros(s.E, np.int32)
        xbar = np.zeros((s.E, s.d), np.float32)
        cov = np.zeros(1, np.float32)
        if mu is not None:
            assert mu.dtype == np.float32 and mu.flags.c_contiguous and mu.shape == (s.E, s.d)
        rc = lib().cmoe_ref_expert_stats(C.byref(self.desc), _ptr(x), x.shape[0], _ptr(loads), _ptr(xbar),
                                         None if mu is None else mu.ctypes.data, beta, _ptr(cov))
        if rc:
            raise ValueError("oracle rejected its arguments")
        return loads, xbar, float(cov[0])

    def param_count(self):
        a, b = C.c_int64(), C.c_int64()
        lib().cmoe_ref_param_count(C.byref(self.desc), C.byref(a), C.byref(b))
        return a.value, b.value


def bf16_to_float(bits: int) -> float:
    return float(lib().cmoe_ref_bf16_to_float(bits))


def half_to_float(bits: int) -> float:
    return float(lib().cmoe_ref_half_to_float(bits))


def dequant(q: np.ndarray, s: np.ndarray, idx: int) -> float:
    q = np.ascontiguousarray(q, np.uint8)
    s = np.ascontiguousarray(s, np.float16)
    return float(lib().cmoe_ref_dequant(_ptr(q), _ptr(s), idx))


def num_threads() -> int:
    return int(lib().cmoe_ref_num_threads())

"""CPU oracle of the adapter-aware MoE layer (test infrastructure only).

Thin ctypes marshalling over `ew_oracle.c`; numpy arrays in, numpy arrays out.  Nothing here is
imported by the product package.  `brute.py` holds an independent fp64 witness used to pin the C
code on tiny inputs; `stats.py` the closed-form memory metrics of Section 3.1.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

_lib = None


class _Cfg(C.Structure):
    _fields_ = [("H", C.c_int32), ("I", C.c_int32), ("M", C.c_int32), ("S", C.c_int32), ("k", C.c_int32),
                ("N", C.c_int32), ("E_max", C.c_int32), ("renormalize", C.c_int32),
                ("routed_scale", C.c_float)]


_U16P = C.POINTER(C.c_uint16)
_I32P = C.POINTER(C.c_int32)


class _Layer(C.Structure):
    _fields_ = [("router_w", _U16P), ("w_gate", _U16P), ("w_up", _U16P), ("w_down", _U16P),
                ("s_gate", _U16P), ("s_up", _U16P), ("s_down", _U16P), ("e", _I32P), ("loaded", _I32P),
                ("tuned", C.POINTER(_I32P)), ("a_gate", C.POINTER(_U16P)), ("a_up", C.POINTER(_U16P)),
                ("a_down", C.POINTER(_U16P))]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.ewo_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().ewo_num_threads())


def _u16(a):
    a = np.ascontiguousarray(a, dtype=np.uint16)
    return a, a.ctypes.data_as(_U16P)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_I32P)


@dataclasses.dataclass
class OracleConfig:
    H: int
    I: int
    M: int
    S: int
    k: int
    N: int
    E_max: int
    renormalize: int = 0
    routed_scale: float = 1.0

    def c(self) -> _Cfg:
        return _Cfg(self.H, self.I, self.M, self.S, self.k, self.N, self.E_max, self.renormalize,
                    self.routed_scale)

    @property
    def P(self) -> int:
        return self.M + self.N * self.E_max


class OracleLayer:
    """Host weights of one layer.  `adapters[i]` is None (not loaded) or (tuned_ids, w_gate, w_up, w_down)."""

    def __init__(self, cfg: OracleConfig, router_w, w_gate, w_up, w_down, s_gate, s_up, s_down,
                 adapters: Optional[Sequence] = None):
        self.cfg = cfg
        self._keep = []
        st = _Layer()
        for name, arr in (("router_w", router_w), ("w_gate", w_gate), ("w_up", w_up), ("w_down", w_down),
                          ("s_gate", s_gate), ("s_up", s_up), ("s_down", s_down)):
            if arr is None or np.asarray(arr).size == 0:
                arr = np.zeros(1, np.uint16)
            a, p = _u16(arr)
            self._keep.append(a)
            setattr(st, name, p)
            if name == "router_w":
                self.router_w = a
        N = cfg.N
        adapters = list(adapters) if adapters is not None else [None] * N
        assert len(adapters) == N
        self.e = np.zeros(N, np.int32)
        self.loaded = np.array([0 if a is None else 1 for a in adapters], np.int32)
        tuned_p = (_I32P * N)()
        ag, au, ad = (_U16P * N)(), (_U16P * N)(), (_U16P * N)()
        self.tuned: List[np.ndarray] = []
        for i, ad_i in enumerate(adapters):
            if ad_i is None:
                ids = np.zeros(0, np.int32)
                g = u = d = np.zeros(1, np.uint16)
            else:
                ids, g, u, d = ad_i
                ids = np.ascontiguousarray(ids, np.int32)
            self.e[i] = ids.shape[0]
            ids_pad = np.ascontiguousarray(np.concatenate([ids, np.zeros(1, np.int32)]))
            self.tuned.append(ids)
            self._keep.append(ids_pad)
            tuned_p[i] = ids_pad.ctypes.data_as(_I32P)
            for arr_p, arr in ((ag, g), (au, u), (ad, d)):
                a, p = _u16(arr)
                self._keep.append(a)
                arr_p[i] = p
        self._keep += [tuned_p, ag, au, ad]
        st.e = self.e.ctypes.data_as(_I32P)
        st.loaded = self.loaded.ctypes.data_as(_I32P)
        st.tuned = C.cast(tuned_p, C.POINTER(_I32P))
        st.a_gate = C.cast(ag, C.POINTER(_U16P))
        st.a_up = C.cast(au, C.POINTER(_U16P))
        st.a_down = C.cast(ad, C.POINTER(_U16P))
        self.st = st

    def build_map(self) -> np.ndarray:
        return build_map(self.cfg.M, self.cfg.N, self.cfg.E_max, self.tuned)


def build_map(M: int, N: int, E_max: int, tuned: Sequence[np.ndarray]) -> np.ndarray:
    """Pi[N, M] from the per-adapter ascending lists of tuned experts (empty list = identity row)."""
    e = np.array([len(t) for t in tuned], np.int32)
    keep = [np.ascontiguousarray(np.concatenate([np.asarray(t, np.int32), np.zeros(1, np.int32)])) for t in tuned]
    ptrs = (_I32P * N)(*[a.ctypes.data_as(_I32P) for a in keep])
    Pi = np.empty((N, M), np.int32)
    rc = lib().ewo_build_map(M, N, E_max, e.ctypes.data_as(_I32P), C.cast(ptrs, C.POINTER(_I32P)),
                             Pi.ctypes.data_as(_I32P))
    if rc != 0:
        raise ValueError(f"build_map failed: {rc}")
    return Pi


def reroute(ids: np.ndarray, aid: np.ndarray, Pi: np.ndarray, loaded: Optional[np.ndarray] = None,
            return_bad: bool = False):
    """Slot ids [B,k].  `loaded` [N] marks the adapters that are loaded (default: all); tokens whose adapter id
    is outside [-1,N) or not loaded are base-model tokens, and `return_bad` also returns how many there were."""
    ids, ip = _i32(ids)
    aid, ap = _i32(aid)
    Pi, pp = _i32(Pi)
    B, k = ids.shape
    N, M = Pi.shape
    lp = None
    if loaded is not None:
        loaded, lp = _i32(loaded)
        assert loaded.shape == (N,)
    out = np.empty((B, k), np.int32)
    bad = lib().ewo_reroute(B, k, M, N, ip, ap, pp, lp, out.ctypes.data_as(_I32P))
    return (out, int(bad)) if return_bad else out


def counts(slots: np.ndarray, P: int) -> np.ndarray:
    slots, sp = _i32(slots)
    out = np.empty(P, np.int32)
    lib().ewo_counts(slots.size, P, sp, out.ctypes.data_as(_I32P))
    return out


def gate_topk(cfg: OracleConfig, x: np.ndarray, router_w: np.ndarray, want_probs: bool = False):
    """-> ids [B,k] i32, w [B,k] f32, gap [B] f32 (p_(k) - p_(k+1)), probs [B,M] or None."""
    x, xp = _u16(x)
    rw, rp = _u16(router_w)
    B = x.shape[0]
    ids = np.empty((B, cfg.k), np.int32)
    w = np.empty((B, cfg.k), np.float32)
    gap = np.empty(B, np.float32)
    probs = np.empty((B, cfg.M), np.float32) if want_probs else None
    c = cfg.c()
    FP = C.POINTER(C.c_float)
    lib().ewo_gate_topk(C.byref(c), B, xp, rp, ids.ctypes.data_as(_I32P), w.ctypes.data_as(FP),
                        probs.ctypes.data_as(FP) if want_probs else None, gap.ctypes.data_as(FP))
    return ids, w, gap, probs


def topk_from_logits(cfg: OracleConfig, logits: np.ndarray):
    lg = np.ascontiguousarray(logits, np.float32)
    B = lg.shape[0]
    ids = np.empty((B, cfg.k), np.int32)
    w = np.empty((B, cfg.k), np.float32)
    gap = np.empty(B, np.float32)
    c = cfg.c()
    FP = C.POINTER(C.c_float)
    lib().ewo_topk_from_logits(C.byref(c), B, lg.ctypes.data_as(FP), ids.ctypes.data_as(_I32P),
                               w.ctypes.data_as(FP), gap.ctypes.data_as(FP))
    return ids, w, gap


def ffn_given_slots(layer: OracleLayer, x: np.ndarray, slots: np.ndarray, w: np.ndarray) -> np.ndarray:
    cfg = layer.cfg
    x, xp = _u16(x)
    slots, sp = _i32(slots)
    w = np.ascontiguousarray(w, np.float32)
    B = x.shape[0]
    out = np.empty((B, cfg.H), np.float32)
    c = cfg.c()
    FP = C.POINTER(C.c_float)
    rc = lib().ewo_ffn_given_slots(C.byref(c), C.byref(layer.st), B, xp, sp, w.ctypes.data_as(FP),
                                   out.ctypes.data_as(FP))
    if rc != 0:
        raise ValueError("a slot id pointed at an unmapped (padding) slot")
    return out


def layer_forward(layer: OracleLayer, x: np.ndarray, aid: np.ndarray, Pi: Optional[np.ndarray] = None):
    """Adapter-aware path -> out [B,H] f32, ids [B,k], w [B,k], slots [B,k]."""
    cfg = layer.cfg
    Pi = layer.build_map() if Pi is None else Pi
    x, xp = _u16(x)
    aid, ap = _i32(aid)
    Pi, pp = _i32(Pi)
    B = x.shape[0]
    out = np.empty((B, cfg.H), np.float32)
    ids = np.empty((B, cfg.k), np.int32)
    slots = np.empty((B, cfg.k), np.int32)
    w = np.empty((B, cfg.k), np.float32)
    c = cfg.c()
    FP = C.POINTER(C.c_float)
    rc = lib().ewo_layer_forward(C.byref(c), C.byref(layer.st), B, xp, ap, pp, out.ctypes.data_as(FP),
                                 ids.ctypes.data_as(_I32P), w.ctypes.data_as(FP), slots.ctypes.data_as(_I32P))
    if rc != 0:
        raise ValueError("a slot id pointed at an unmapped (padding) slot")
    return out, ids, w, slots


def layer_forward_merged(layer: OracleLayer, x: np.ndarray, aid: np.ndarray) -> np.ndarray:
    """The definition: every token through the merged model of its own adapter."""
    cfg = layer.cfg
    x, xp = _u16(x)
    aid, ap = _i32(aid)
    B = x.shape[0]
    out = np.empty((B, cfg.H), np.float32)
    c = cfg.c()
    lib().ewo_layer_forward_merged(C.byref(c), C.byref(layer.st), B, xp, ap,
                                   out.ctypes.data_as(C.POINTER(C.c_float)))
    return out

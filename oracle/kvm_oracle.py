"""ctypes wrapper around the C oracle (oracle/kvm_oracle.c).

Test infrastructure only: imported by tests/, by __graft_entry__.smoke() and by the CPU
baseline leg of bench.py.  It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from . import build as _build

GROWTH = {"fixed": 0, "sqrt": 1, "unbounded": 2, "power": 3, "saturating": 4}


class _Cfg(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
        ("C", C.c_int32), ("w", C.c_int32), ("S", C.c_int32), ("r", C.c_int32),
        ("growth_kind", C.c_int32), ("sqrt_coeff", C.c_int32), ("fixed_slots", C.c_int64),
        ("rope_base", C.c_double), ("ln_eps", C.c_double), ("norm_eps", C.c_double),
        ("radius_on", C.c_int32), ("reserved", C.c_int32),
        ("pow_num", C.c_int32), ("pow_den", C.c_int32), ("sat_half", C.c_int64),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        dp = C.POINTER(C.c_double)
        L.kvm_oracle_create.restype = C.c_void_p
        L.kvm_oracle_create.argtypes = [C.POINTER(_Cfg), dp, dp, dp, dp]
        L.kvm_oracle_free.argtypes = [C.c_void_p]
        L.kvm_oracle_forward.restype = C.c_int
        L.kvm_oracle_forward.argtypes = [C.c_void_p, dp, dp, dp, dp, C.c_int64, dp]
        for name in ("kvm_oracle_position", "kvm_oracle_rows", "kvm_oracle_nfolds"):
            getattr(L, name).restype = C.c_int64
            getattr(L, name).argtypes = [C.c_void_p]
        L.kvm_oracle_fold_log.argtypes = [C.c_void_p] + [C.POINTER(C.c_int64)] * 3
        L.kvm_oracle_export.argtypes = [C.c_void_p, dp, dp, dp, dp, C.POINTER(C.c_int32)]
        L.kvm_oracle_readout.argtypes = [C.c_void_p, dp, dp]
        L.kvm_oracle_assignments.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_uint8), dp]
        L.kvm_oracle_memory_keys.argtypes = [C.c_void_p, dp]
        L.kvm_oracle_threads.restype = C.c_int
        _lib = L
    return _lib


def _dp(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_double))


def _f64(a):
    return None if a is None else np.ascontiguousarray(np.asarray(a, dtype=np.float64))


@dataclass
class OracleConfig:
    B: int
    Hq: int
    Hkv: int
    d: int
    C: int
    w: int = 2
    S: int = 1
    r: int = 0
    growth: str = "fixed"
    fixed_slots: int = 0
    sqrt_coeff: int = 16
    pow_num: int = 1      # "power": floor(sqrt_coeff * e^(pow_num/pow_den))
    pow_den: int = 2
    sat_half: int = 0     # "saturating": floor(fixed_slots * e / (e + sat_half))
    rope_base: float = 10000.0
    ln_eps: float = 1e-5
    norm_eps: float = 1e-12
    radius_on: bool = True


class KVMOracle:
    """One layer state of the fp64 oracle; forward() consumes further tokens."""

    def __init__(self, cfg: OracleConfig, ln_w=None, ln_b=None, tau_s=None, tau_b=None):
        self.cfg = cfg
        c = _Cfg(cfg.B, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, cfg.w, cfg.S, cfg.r, GROWTH[cfg.growth],
                 cfg.sqrt_coeff, cfg.fixed_slots, cfg.rope_base, cfg.ln_eps, cfg.norm_eps,
                 1 if cfg.radius_on else 0, 0, cfg.pow_num, cfg.pow_den, cfg.sat_half)
        ln_w, ln_b, tau_s, tau_b = _f64(ln_w), _f64(ln_b), _f64(tau_s), _f64(tau_b)
        if ln_w is not None:
            assert ln_w.shape == (cfg.Hkv, cfg.d)
        if ln_b is not None:
            assert ln_b.shape == (cfg.Hkv, cfg.d)
        if tau_s is not None:
            assert tau_s.shape == (cfg.Hq,)
        if tau_b is not None:
            assert tau_b.shape == (cfg.Hq,)
        self._h = lib().kvm_oracle_create(C.byref(c), _dp(ln_w), _dp(ln_b), _dp(tau_s), _dp(tau_b))
        if not self._h:
            raise ValueError("invalid oracle configuration")

    def __del__(self):
        h = getattr(self, "_h", None)
        if h:
            lib().kvm_oracle_free(h)
            self._h = None

    @property
    def U(self):
        return self.cfg.B * self.cfg.Hkv

    def forward(self, q, k, v, gate=None):
        """q [B,Hq,n,d], k,v [B,Hkv,n,d], gate [B,Hkv,n] -> y [B,Hq,n,d] (float64)."""
        cfg = self.cfg
        q, k, v, gate = _f64(q), _f64(k), _f64(v), _f64(gate)
        n = q.shape[2]
        assert q.shape == (cfg.B, cfg.Hq, n, cfg.d), q.shape
        assert k.shape == (cfg.B, cfg.Hkv, n, cfg.d) and v.shape == k.shape
        if gate is not None:
            assert gate.shape == (cfg.B, cfg.Hkv, n)
        y = np.empty_like(q)
        rc = lib().kvm_oracle_forward(self._h, _dp(q), _dp(k), _dp(v), _dp(gate), n, _dp(y))
        if rc != 0:
            raise MemoryError("oracle allocation failed")
        return y

    @property
    def position(self):
        return lib().kvm_oracle_position(self._h)

    @property
    def rows(self):
        return lib().kvm_oracle_rows(self._h)

    @property
    def nfolds(self):
        return lib().kvm_oracle_nfolds(self._h)

    def fold_log(self):
        n = self.nfolds
        e = np.zeros(n, np.int64)
        m = np.zeros(n, np.int64)
        a = np.zeros(n, np.int64)
        p = C.POINTER(C.c_int64)
        lib().kvm_oracle_fold_log(self._h, e.ctypes.data_as(p), m.ctypes.data_as(p), a.ctypes.data_as(p))
        return e, m, a

    def export(self):
        U, m, d = self.U, self.rows, self.cfg.d
        sk = np.zeros((U, m, d)); sv = np.zeros((U, m, d))
        rho = np.zeros((U, m)); w = np.zeros((U, m)); cnt = np.zeros((U, m), np.int32)
        lib().kvm_oracle_export(self._h, _dp(sk), _dp(sv), _dp(rho), _dp(w),
                                cnt.ctypes.data_as(C.POINTER(C.c_int32)))
        return dict(sum_k=sk, sum_v=sv, radius=rho, weight=w, count=cnt)

    def readout(self):
        U, m, d = self.U, self.rows, self.cfg.d
        kh = np.zeros((U, m, d)); vh = np.zeros((U, m, d))
        lib().kvm_oracle_readout(self._h, _dp(kh), _dp(vh))
        return kh, vh

    def assignments(self):
        U, n = self.U, self.position
        slot = np.zeros((U, n), np.int32); app = np.zeros((U, n), np.uint8); mg = np.zeros((U, n))
        lib().kvm_oracle_assignments(self._h, slot.ctypes.data_as(C.POINTER(C.c_int32)),
                                     app.ctypes.data_as(C.POINTER(C.c_uint8)), _dp(mg))
        return slot, app, mg

    def memory_keys(self):
        U, n, d = self.U, self.position, self.cfg.d
        kb = np.zeros((U, n, d))
        lib().kvm_oracle_memory_keys(self._h, _dp(kb))
        return kb


def threads() -> int:
    return lib().kvm_oracle_threads()

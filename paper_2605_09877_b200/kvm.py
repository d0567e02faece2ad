"""Thin ctypes binding over the C ABI of libkvm.so (include/kvm.h).

Argument marshalling only: every step of the layer runs inside the CUDA library.  torch is
used for device memory and streams.  Importing this module raises if the library has not
been built (python -m paper_2605_09877_b200.build) -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvm.so")

KVM_OK = 0
STATUS = {0: "KVM_OK", 1: "KVM_ERR_INVALID_ARG", 2: "KVM_ERR_UNSUPPORTED", 3: "KVM_ERR_OOM",
          4: "KVM_ERR_CUDA", 5: "KVM_ERR_STATE_MISMATCH", 6: "KVM_ERR_CAPACITY", 7: "KVM_ERR_TIMEOUT"}
GROWTH_FIXED, GROWTH_SQRT, GROWTH_UNBOUNDED, GROWTH_POWER, GROWTH_SATURATING = 0, 1, 2, 3, 4
FLAG_NO_RADIUS, FLAG_RECORD_ASSIGN, FLAG_SIMT_ATTENTION, FLAG_SIMT_ROUTING, FLAG_MIN_KEY_SLOTS, FLAG_SERIAL_FOLDS, FLAG_FUSED_QK_LN = 1, 2, 4, 8, 16, 32, 64

EXPORTS = ["kvm_plan_capacity", "kvm_state_create", "kvm_prefill", "kvm_decode_step", "kvm_prefill_host",
           "kvm_decode_step_host", "kvm_state_free", "kvm_state_info", "kvm_state_check", "kvm_state_export",
           "kvm_debug_assignments", "kvm_launch_count", "kvm_status_string", "kvm_state_reset",
           "kvm_profile_enable", "kvm_profile_read", "kvm_debug_counters", "kvm_attend_rows_noalloc", "kvm_merge_gate", "kvm_head_layernorm",
           "kvm_state_snapshot_info", "kvm_state_export_window", "kvm_state_import", "kvm_debug_expire_wait"]


class KVMError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)}")


class Growth(C.Structure):
    _fields_ = [("kind", C.c_int32), ("sqrt_coeff", C.c_int32), ("fixed_slots", C.c_int64),
                ("pow_num", C.c_int32), ("pow_den", C.c_int32), ("sat_half", C.c_int64)]


class Strides(C.Structure):
    _fields_ = [("q", C.c_int64 * 4), ("k", C.c_int64 * 4), ("v", C.c_int64 * 4), ("out", C.c_int64 * 4)]


class SnapshotInfo(C.Structure):
    _fields_ = [("block", C.c_int32), ("rope_dims", C.c_int32), ("growth", Growth), ("n_slots", C.c_int64),
                ("position", C.c_int64), ("n_folds", C.c_int64), ("window_begin", C.c_int64), ("window_len", C.c_int64)]


class Config(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("n_bswa_chunks", C.c_int32), ("sink_len", C.c_int32),
        ("rope_base", C.c_float), ("ln_eps", C.c_float), ("norm_eps", C.c_float),
        ("ln_weight", C.POINTER(C.c_float)), ("ln_bias", C.POINTER(C.c_float)),
        ("tau_state", C.POINTER(C.c_float)), ("tau_bswa", C.POINTER(C.c_float)),
        ("max_block", C.c_int32), ("max_state_slots", C.c_int64), ("max_call_tokens", C.c_int64),
        ("max_seq_len", C.c_int64), ("device", C.c_int32), ("flags", C.c_uint32),
        ("qk_ln_eps", C.c_float),
        ("ln_q_weight", C.POINTER(C.c_float)), ("ln_q_bias", C.POINTER(C.c_float)),
        ("ln_k_weight", C.POINTER(C.c_float)), ("ln_k_bias", C.POINTER(C.c_float)),
    ]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2605_09877_b200.build` "
                          "(the KVM layer has no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp = C.c_void_p
    L.kvm_plan_capacity.restype = C.c_int64
    L.kvm_plan_capacity.argtypes = [C.c_int32, C.c_int32, Growth, C.c_int64]
    L.kvm_state_create.restype = C.c_int
    L.kvm_state_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    L.kvm_prefill.restype = C.c_int
    L.kvm_prefill.argtypes = [vp, vp, vp, vp, C.c_int32, Growth, C.c_int32, C.c_int64, vp, vp, C.POINTER(Strides), vp]
    L.kvm_decode_step.restype = C.c_int
    L.kvm_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.kvm_prefill_host.restype = C.c_int
    L.kvm_prefill_host.argtypes = [vp, vp, vp, vp, C.c_int32, Growth, C.c_int32, C.c_int64, vp, vp, vp]
    L.kvm_decode_step_host.restype = C.c_int
    L.kvm_decode_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.kvm_state_free.restype = C.c_int
    L.kvm_state_free.argtypes = [vp]
    L.kvm_state_info.restype = C.c_int
    L.kvm_state_info.argtypes = [vp, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.kvm_state_check.restype = C.c_int
    L.kvm_state_check.argtypes = [vp, vp]
    L.kvm_state_export.restype = C.c_int
    L.kvm_state_export.argtypes = [vp] * 9
    L.kvm_debug_assignments.restype = C.c_int
    L.kvm_debug_assignments.argtypes = [vp, C.c_int64, vp, vp, vp]
    L.kvm_state_reset.restype = C.c_int
    L.kvm_state_reset.argtypes = [vp]
    L.kvm_profile_enable.restype = C.c_int
    L.kvm_profile_enable.argtypes = [vp, C.c_int32]
    L.kvm_profile_read.restype = C.c_int
    L.kvm_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.kvm_debug_counters.restype = C.c_int
    L.kvm_debug_counters.argtypes = [vp, C.POINTER(C.c_int64), vp]
    L.kvm_launch_count.restype = C.c_int64
    L.kvm_launch_count.argtypes = [vp]
    L.kvm_attend_rows_noalloc.restype = C.c_int
    L.kvm_attend_rows_noalloc.argtypes = [vp, vp, vp, C.c_int32, C.c_int64, C.c_int32, C.c_float, vp, vp]
    L.kvm_merge_gate.restype = C.c_int
    L.kvm_merge_gate.argtypes = [vp, vp, C.c_int32, C.c_int64, C.c_int32, C.c_int32, vp, vp, vp]
    L.kvm_debug_expire_wait.restype = C.c_int
    L.kvm_debug_expire_wait.argtypes = [vp, C.c_int32, vp]
    L.kvm_head_layernorm.restype = C.c_int
    L.kvm_head_layernorm.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, C.c_int64, C.c_int32, C.c_float, vp]
    L.kvm_state_snapshot_info.restype = C.c_int
    L.kvm_state_snapshot_info.argtypes = [vp, C.POINTER(SnapshotInfo)]
    L.kvm_state_export_window.restype = C.c_int
    L.kvm_state_export_window.argtypes = [vp, vp, vp, vp, vp]
    L.kvm_state_import.restype = C.c_int
    L.kvm_state_import.argtypes = [vp, C.POINTER(SnapshotInfo)] + [vp] * 9
    L.kvm_status_string.restype = C.c_char_p
    L.kvm_status_string.argtypes = [C.c_int]
    return L


lib = _load()


def growth(kind: str, fixed_slots: int = 0, sqrt_coeff: int = 16, pow_num: int = 1, pow_den: int = 2,
           sat_half: int = 0) -> Growth:
    """fixed: B = fixed_slots; sqrt: floor(sqrt_coeff sqrt(e)); power: floor(sqrt_coeff e^(pow_num/pow_den));
    saturating: floor(fixed_slots e / (e + sat_half)); unbounded: no budget."""
    k = {"fixed": GROWTH_FIXED, "sqrt": GROWTH_SQRT, "unbounded": GROWTH_UNBOUNDED, "power": GROWTH_POWER,
         "saturating": GROWTH_SATURATING}[kind]
    return Growth(k, sqrt_coeff, fixed_slots, pow_num, pow_den, sat_half)


def merge_gate(x: "torch.Tensor", w_gate: "torch.Tensor", out=None, stream=None, status=None) -> "torch.Tensor":
    """g = 1 + ELU(x W_g): x bf16 [B, T, d_model], w_gate fp32 [Hkv, d_model] -> fp32 [B, Hkv, T]
    (argument marshalling only; the product runs in kvm_merge_gate).  `status`: optional int32 CUDA tensor
    of one element that receives KVM_ERR_TIMEOUT should a bounded device-side wait run out."""
    assert x.is_cuda and w_gate.is_cuda and x.dtype == torch.bfloat16 and w_gate.dtype == torch.float32
    assert x.is_contiguous() and w_gate.is_contiguous() and x.dim() == 3 and w_gate.dim() == 2
    B, T, dm = x.shape
    H = w_gate.shape[0]
    assert w_gate.shape[1] == dm
    if out is None:
        out = torch.empty((B, H, T), dtype=torch.float32, device=x.device)
    rc = lib.kvm_merge_gate(C.c_void_p(x.data_ptr()), C.c_void_p(w_gate.data_ptr()), B, T, dm, H,
                            C.c_void_p(out.data_ptr()), C.c_void_p(status.data_ptr()) if status is not None else None,
                            _stream_ptr(stream))
    if rc != 0:
        raise KVMError(rc, "kvm_merge_gate")
    return out


def head_layernorm(x: "torch.Tensor", weight=None, bias=None, eps: float = 1e-5, stream=None) -> "torch.Tensor":
    """LN_q / LN_k in place: x bf16 [B, H, T, d] contiguous; weight, bias fp32 [H, d] on the device or None."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, T, d = x.shape
    for t in (weight, bias):
        assert t is None or (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (H, d))
    rc = lib.kvm_head_layernorm(C.c_void_p(x.data_ptr()), C.c_void_p(weight.data_ptr() if weight is not None else 0),
                                C.c_void_p(bias.data_ptr() if bias is not None else 0), B, H, T, d, eps, _stream_ptr(stream))
    if rc != 0:
        raise KVMError(rc, "kvm_head_layernorm")
    return x


def kvm_plan_capacity(block: int, n_bswa_chunks: int, g: Growth, seq_len: int) -> int:
    return lib.kvm_plan_capacity(block, n_bswa_chunks, g, seq_len)


def _fp(a):
    if a is None:
        return None, None
    arr = np.ascontiguousarray(np.asarray(a, dtype=np.float32))
    return arr, arr.ctypes.data_as(C.POINTER(C.c_float))


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def attend_rows_noalloc(q, keys, values, scale: float, out=None, stream=None):
    """kvm_attend_rows_noalloc: out[h] = softmax(scale * q[h] . keys[h]^T) . values[h] for callers that may not
    allocate device memory inside the call (the split partials live in a fixed array of the library).
    q [H,d] fp16, keys/values [H,n,d] fp16 contiguous CUDA tensors; `out` [H,d] bf16 should be passed by such
    callers (it is only created here for convenience when omitted)."""
    assert q.dtype == torch.float16 and keys.dtype == torch.float16 and values.dtype == torch.float16
    assert q.is_contiguous() and keys.is_contiguous() and values.is_contiguous()
    H, n, d = keys.shape
    if out is None:
        out = torch.empty((H, d), dtype=torch.bfloat16, device=q.device)
    rc = lib.kvm_attend_rows_noalloc(C.c_void_p(q.data_ptr()), C.c_void_p(keys.data_ptr()), C.c_void_p(values.data_ptr()),
                                     H, n, d, scale, C.c_void_p(out.data_ptr()), _stream_ptr(stream))
    if rc != KVM_OK:
        raise KVMError(rc, "kvm_attend_rows_noalloc")
    return out


@dataclass
class LayerConfig:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    max_block: int
    max_state_slots: int
    max_call_tokens: int
    n_bswa_chunks: int = 2
    sink_len: int = 1
    rope_base: float = 10000.0
    ln_eps: float = 1e-5
    norm_eps: float = 1e-12
    max_seq_len: int = 0
    device: int = 0
    flags: int = 0


class KVMState:
    """Owns one kvm_state_t.  Methods map 1:1 to the C entry points of the same name."""

    def __init__(self, cfg: LayerConfig, ln_weight=None, ln_bias=None, tau_state=None, tau_bswa=None, qk_ln=None):
        """qk_ln: dict(eps, q_weight, q_bias, k_weight, k_bias) turns the fused front end on (KVM_FLAG_FUSED_QK_LN)."""
        self.cfg = cfg
        keep = [_fp(ln_weight), _fp(ln_bias), _fp(tau_state), _fp(tau_bswa)]
        flags, eps = cfg.flags, 0.0
        ln4 = [(None, None)] * 4
        if qk_ln is not None:
            flags |= FLAG_FUSED_QK_LN
            eps = float(qk_ln.get("eps", 1e-5))
            ln4 = [_fp(qk_ln.get(n)) for n in ("q_weight", "q_bias", "k_weight", "k_bias")]
        c = Config(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_bswa_chunks, cfg.sink_len,
                   cfg.rope_base, cfg.ln_eps, cfg.norm_eps, keep[0][1], keep[1][1], keep[2][1], keep[3][1],
                   cfg.max_block, cfg.max_state_slots, cfg.max_call_tokens, cfg.max_seq_len, cfg.device, flags,
                   eps, ln4[0][1], ln4[1][1], ln4[2][1], ln4[3][1])
        h = C.c_void_p()
        rc = lib.kvm_state_create(C.byref(c), C.byref(h))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_create")
        self._h = h
        self.U = cfg.batch * cfg.n_kv_heads

    def free(self):
        if getattr(self, "_h", None):
            lib.kvm_state_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    # -- kvm_prefill ---------------------------------------------------------------------
    def prefill(self, q, k, v, block: int, g: Growth, rope_dims: int, out=None, gate=None, stream=None):
        """q [B,Hq,n,d], k,v [B,Hkv,n,d] bf16 CUDA tensors (last dim contiguous)."""
        assert q.is_cuda and q.dtype == torch.bfloat16 and k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16
        n = q.shape[2]
        if out is None:
            out = torch.empty(q.shape, dtype=torch.bfloat16, device=q.device)
        st = Strides()
        for name, t in (("q", q), ("k", k), ("v", v), ("out", out)):
            arr = getattr(st, name)
            for i in range(4):
                arr[i] = t.stride(i)
        gp = None
        if gate is not None:
            assert gate.dtype == torch.float32 and gate.is_contiguous() and gate.is_cuda
            gp = C.c_void_p(gate.data_ptr())
        rc = lib.kvm_prefill(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()), self._h,
                             block, g, rope_dims, n, gp, C.c_void_p(out.data_ptr()), C.byref(st), _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_prefill")
        return out

    # -- kvm_decode_step -----------------------------------------------------------------
    def decode_step(self, q, k, v, out=None, gate=None, stream=None):
        """q [B,Hq,d], k,v [B,Hkv,d] contiguous bf16 CUDA tensors."""
        assert q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
        if out is None:
            out = torch.empty(q.shape, dtype=torch.bfloat16, device=q.device)
        gp = C.c_void_p(gate.data_ptr()) if gate is not None else None
        rc = lib.kvm_decode_step(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                 self._h, gp, C.c_void_p(out.data_ptr()), _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_decode_step")
        return out

    # -- host-buffer variants ------------------------------------------------------------
    def prefill_host(self, q, k, v, block: int, g: Growth, rope_dims: int, out, gate=None, stream=None):
        """Contiguous bf16 CPU tensors (pinned for speed); `out` is a CPU tensor that is filled."""
        for t in (q, k, v, out):
            assert (not t.is_cuda) and t.is_contiguous() and t.dtype == torch.bfloat16
        gp = C.c_void_p(gate.data_ptr()) if gate is not None else None
        rc = lib.kvm_prefill_host(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                  self._h, block, g, rope_dims, q.shape[2], gp, C.c_void_p(out.data_ptr()),
                                  _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_prefill_host")
        return out

    def decode_step_host(self, q, k, v, out, gate=None, stream=None):
        for t in (q, k, v, out):
            assert (not t.is_cuda) and t.is_contiguous() and t.dtype == torch.bfloat16
        gp = C.c_void_p(gate.data_ptr()) if gate is not None else None
        rc = lib.kvm_decode_step_host(C.c_void_p(q.data_ptr()), C.c_void_p(k.data_ptr()), C.c_void_p(v.data_ptr()),
                                      self._h, gp, C.c_void_p(out.data_ptr()), _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_decode_step_host")
        return out

    # -- inspection ----------------------------------------------------------------------
    def info(self):
        a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
        rc = lib.kvm_state_info(self._h, C.byref(a), C.byref(b), C.byref(c))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_info")
        return dict(n_slots=a.value, position=b.value, n_folds=c.value)

    def check(self, stream=None):
        return lib.kvm_state_check(self._h, _stream_ptr(stream))

    def reset(self):
        rc = lib.kvm_state_reset(self._h)
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_reset")

    def profile_enable(self, on=True):
        lib.kvm_profile_enable(self._h, 1 if on else 0)

    def profile_read(self):
        """Returns {phase: (milliseconds, bracket count)} accumulated since the last read."""
        ms = (C.c_double * 8)(); n = (C.c_int64 * 8)()
        rc = lib.kvm_profile_read(self._h, ms, n)
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_profile_read")
        names = ("ingest", "attention", "kbar", "route_filter", "fold_decide", "fold_apply", "decode")
        return {names[i]: (ms[i], n[i]) for i in range(7)}

    def debug_counters(self, stream=None):
        out = (C.c_int64 * 4)()
        rc = lib.kvm_debug_counters(self._h, out, _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_debug_counters")
        return dict(exhaustive_tokens=out[0], candidate_pairs=out[1], tokens=out[2], clamped_inputs=out[3])

    def debug_expire_wait(self, spins: int = 10000, stream=None):
        rc = lib.kvm_debug_expire_wait(self._h, spins, _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_debug_expire_wait")

    def launch_count(self):
        return lib.kvm_launch_count(self._h)

    def export(self, readout=True, stream=None):
        m, d, U = self.info()["n_slots"], self.cfg.head_dim, self.U
        sk = np.zeros((U, m, d), np.float64); sv = np.zeros((U, m, d), np.float32)
        rho = np.zeros((U, m), np.float32); w = np.zeros((U, m), np.float64); cnt = np.zeros((U, m), np.int32)
        kr = torch.zeros((U, m, d), dtype=torch.float16) if readout else None
        vr = torch.zeros((U, m, d), dtype=torch.float16) if readout else None
        p = lambda a: C.c_void_p(a.ctypes.data)
        rc = lib.kvm_state_export(self._h, p(sk), p(sv), p(rho), p(w), p(cnt),
                                  C.c_void_p(kr.data_ptr()) if readout else None,
                                  C.c_void_p(vr.data_ptr()) if readout else None, _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_export")
        return dict(sum_k=sk, sum_v=sv, radius=rho, weight=w, count=cnt, k_read=kr, v_read=vr)

    def snapshot(self, stream=None):
        """kvm_state_snapshot_info + kvm_state_export + kvm_state_export_window: everything kvm_state_import needs."""
        info = SnapshotInfo()
        rc = lib.kvm_state_snapshot_info(self._h, C.byref(info))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_snapshot_info")
        snap = self.export(readout=False, stream=stream)
        n, d = info.window_len, self.cfg.head_dim
        wk = torch.zeros((self.U, n, d), dtype=torch.float16); wv = torch.zeros((self.U, n, d), dtype=torch.float16)
        wg = np.zeros((self.U, n), np.float32)
        if info.block > 0:
            rc = lib.kvm_state_export_window(self._h, C.c_void_p(wk.data_ptr()), C.c_void_p(wv.data_ptr()),
                                             C.c_void_p(wg.ctypes.data), _stream_ptr(stream))
            if rc != KVM_OK:
                raise KVMError(rc, "kvm_state_export_window")
        snap.update(info=info, win_k=wk, win_v=wv, win_gate=wg)
        return snap

    def restore(self, snap, stream=None):
        """kvm_state_import of a snapshot() (possibly taken from another state of the same shape)."""
        p = lambda a: C.c_void_p(a.ctypes.data) if a is not None and a.size else None
        t = lambda a: C.c_void_p(a.data_ptr()) if a is not None and a.numel() else None
        rc = lib.kvm_state_import(self._h, C.byref(snap["info"]), p(snap["sum_k"]), p(snap["sum_v"]), p(snap["radius"]),
                                  p(snap["weight"]), p(snap["count"]), t(snap["win_k"]), t(snap["win_v"]),
                                  p(snap.get("win_gate")), _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_state_import")

    def assignments(self, n=None, stream=None):
        n = self.info()["position"] if n is None else n
        slot = np.zeros((self.U, n), np.int32); app = np.zeros((self.U, n), np.uint8)
        rc = lib.kvm_debug_assignments(self._h, n, C.c_void_p(slot.ctypes.data), C.c_void_p(app.ctypes.data),
                                       _stream_ptr(stream))
        if rc != KVM_OK:
            raise KVMError(rc, "kvm_debug_assignments")
        return slot, app

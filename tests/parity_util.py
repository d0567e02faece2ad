"""Helpers for the GPU parity tests: run the CUDA library and the fp64 oracle on the same
seeded bf16 inputs and compare.  The oracle side never touches CUDA; the CUDA side never
touches the oracle; this file only moves inputs and compares outputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle.kvm_oracle import KVMOracle, OracleConfig
from paper_2605_09877_b200 import synth

# tolerance stated for the layer: bf16 outputs and state means, fp32 accumulation
MAX_ABS = 2e-2
MEAN_ABS = 2e-3


def oracle_config(wl: synth.Workload, n_units=None, radius_on=True, ln_eps=1e-5) -> OracleConfig:
    if n_units is None:
        B, Hq, Hkv = wl.B, wl.Hq, wl.Hkv
    else:
        G = wl.Hq // wl.Hkv
        B, Hq, Hkv = 1, n_units * G, n_units
    return OracleConfig(B=B, Hq=Hq, Hkv=Hkv, d=wl.d, C=wl.C, w=wl.w, S=wl.S, r=wl.r, growth=wl.growth,
                        fixed_slots=wl.fixed_slots, sqrt_coeff=wl.sqrt_coeff, pow_num=wl.pow_num, pow_den=wl.pow_den,
                        sat_half=wl.sat_half, radius_on=radius_on, ln_eps=ln_eps)


def to_f64(t):
    return t.detach().cpu().double().numpy()


def select_units(wl, tensors, units, params):
    """Gathers the (batch, kv-head) units `units` into a B=1 problem for the oracle."""
    G = wl.Hq // wl.Hkv
    q = torch.stack([tensors["q"][b, h * G + g] for (b, h) in units for g in range(G)])[None]
    k = torch.stack([tensors["k"][b, h] for (b, h) in units])[None]
    v = torch.stack([tensors["v"][b, h] for (b, h) in units])[None]
    gate = None
    if tensors.get("gate") is not None:
        gate = torch.stack([tensors["gate"][b, h] for (b, h) in units])[None]
    sub = {}
    hk = [h for (_, h) in units]
    hq = [h * G + g for (_, h) in units for g in range(G)]
    for key, idx in (("ln_w", hk), ("ln_b", hk), ("tau_s", hq), ("tau_b", hq)):
        val = params.get(key)
        sub[key] = None if val is None else np.asarray(val, dtype=np.float32)[idx].astype(np.float64)
    return dict(q=q, k=k, v=v, gate=gate), sub


def gpu_layer(wl, params, flags=0, max_call_tokens=None, max_seq_len=None, radius_on=True, ln_eps=1e-5,
              extra_tokens=0):
    from paper_2605_09877_b200 import kvm
    g = kvm.growth(wl.growth, wl.fixed_slots, wl.sqrt_coeff, wl.pow_num, wl.pow_den, wl.sat_half)
    total = wl.T + extra_tokens
    cap = max(kvm.kvm_plan_capacity(wl.C, wl.w, g, total), wl.C)
    fl = flags | kvm.FLAG_RECORD_ASSIGN | (0 if radius_on else kvm.FLAG_NO_RADIUS)
    cfg = kvm.LayerConfig(batch=wl.B, n_q_heads=wl.Hq, n_kv_heads=wl.Hkv, head_dim=wl.d, max_block=wl.C,
                          max_state_slots=cap, max_call_tokens=max_call_tokens or wl.T, n_bswa_chunks=wl.w,
                          sink_len=wl.S, ln_eps=ln_eps, max_seq_len=max_seq_len or total, flags=fl)
    st = kvm.KVMState(cfg, ln_weight=params.get("ln_w"), ln_bias=params.get("ln_b"),
                      tau_state=params.get("tau_s"), tau_bswa=params.get("tau_b"))
    return st, g


def run_gpu(wl, tensors, params, cuts=None, flags=0, radius_on=True, decode_from=None, ln_eps=1e-5):
    """Prefill in segments given by `cuts` (token boundaries); tokens >= decode_from go through
    kvm_decode_step one at a time.  Returns (y [B,Hq,T,d] bf16 cpu, state handle)."""
    T = wl.T
    decode_from = T if decode_from is None else decode_from
    cuts = cuts or [0, decode_from]
    cuts = [c for c in cuts if c <= decode_from]
    if cuts[-1] != decode_from:
        cuts.append(decode_from)
    st, g = gpu_layer(wl, params, flags=flags, max_call_tokens=max(max(b - a for a, b in zip(cuts[:-1], cuts[1:])), 1),
                      radius_on=radius_on, ln_eps=ln_eps)
    dev = torch.device("cuda:0")
    q, k, v = (tensors[n].to(dev) for n in ("q", "k", "v"))
    gate = tensors.get("gate")
    gate = None if gate is None else gate.to(dev)
    y = torch.zeros_like(q)
    for a, b in zip(cuts[:-1], cuts[1:]):
        if b == a:
            continue
        gseg = None if gate is None else gate[:, :, a:b].contiguous()
        st.prefill(q[:, :, a:b], k[:, :, a:b], v[:, :, a:b], wl.C, g, wl.r, out=y[:, :, a:b], gate=gseg)
    for t in range(decode_from, T):
        gt = None if gate is None else gate[:, :, t].contiguous()
        yo = st.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), gate=gt)
        y[:, :, t] = yo
    torch.cuda.synchronize()
    assert st.check() == 0
    return y.cpu(), st


def run_oracle(wl, tensors, params, units=None, radius_on=True, ln_eps=1e-5):
    if units is not None:
        tensors, params = select_units(wl, tensors, units, params)
        cfg = oracle_config(wl, n_units=len(units), radius_on=radius_on, ln_eps=ln_eps)
    else:
        cfg = oracle_config(wl, radius_on=radius_on, ln_eps=ln_eps)
        params = {k: (None if v is None else np.asarray(v, dtype=np.float32).astype(np.float64)) for k, v in params.items()}
    o = KVMOracle(cfg, ln_w=params.get("ln_w"), ln_b=params.get("ln_b"), tau_s=params.get("tau_s"),
                  tau_b=params.get("tau_b"))
    gate = tensors.get("gate")
    y = o.forward(to_f64(tensors["q"]), to_f64(tensors["k"]), to_f64(tensors["v"]),
                  None if gate is None else to_f64(gate))
    return y, o


def compare(wl, y_gpu, st, y_ref, o, units=None, check_state=True):
    """Bit-exact: rows, folds, slot assignments, append flags, counts.  Tolerance: outputs,
    state means, readout caches."""
    G = wl.Hq // wl.Hkv
    yg = y_gpu.double().numpy()
    if units is not None:
        yg = np.stack([yg[b, h * G + g] for (b, h) in units for g in range(G)])[None]
        uidx = [b * wl.Hkv + h for (b, h) in units]
    else:
        uidx = list(range(wl.B * wl.Hkv))
    err = np.abs(yg - y_ref)
    stats = dict(max_abs=float(err.max()), mean_abs=float(err.mean()))
    assert np.isfinite(yg).all()
    assert stats["max_abs"] <= MAX_ABS, stats
    assert stats["mean_abs"] <= MEAN_ABS, stats
    info = st.info()
    assert info["n_slots"] == o.rows and info["n_folds"] == o.nfolds and info["position"] == o.position
    if not check_state:
        return stats
    slot_g, app_g = st.assignments()
    slot_o, app_o, margin = o.assignments()
    slot_g, app_g = slot_g[uidx], app_g[uidx]
    mism = np.argwhere(slot_g != slot_o)
    stats["slot_mismatches"] = int(len(mism))
    stats["min_margin"] = float(np.min(margin)) if margin.size else float("inf")
    assert len(mism) == 0, (mism[:10], [margin[tuple(i)] for i in mism[:10]])
    assert np.array_equal(app_g, app_o)
    if o.rows > 0:
        eg = st.export()
        eo = o.export()
        assert np.array_equal(eg["count"][uidx], eo["count"])
        np.testing.assert_allclose(eg["weight"][uidx], eo["weight"], rtol=1e-6, atol=1e-6)
        mean_k_g = eg["sum_k"][uidx] / eg["weight"][uidx][..., None]
        mean_v_g = eg["sum_v"][uidx].astype(np.float64) / eg["weight"][uidx][..., None]
        mean_k_o = eo["sum_k"] / eo["weight"][..., None]
        mean_v_o = eo["sum_v"] / eo["weight"][..., None]
        for a, b in ((mean_k_g, mean_k_o), (mean_v_g, mean_v_o)):
            e = np.abs(a - b)
            assert e.max() <= MAX_ABS and e.mean() <= MEAN_ABS, (e.max(), e.mean())
        stats["mean_k_err"] = float(np.abs(mean_k_g - mean_k_o).max())
        stats["mean_v_err"] = float(np.abs(mean_v_g - mean_v_o).max())
        np.testing.assert_allclose(eg["radius"][uidx], eo["radius"], rtol=1e-6)
        kh, vh = o.readout()
        ek = np.abs(eg["k_read"].double().numpy()[uidx] - kh)
        ev = np.abs(eg["v_read"].double().numpy()[uidx] - vh)
        # readout caches are fp16: half an ulp of the largest magnitude plus accumulation error
        assert ek.max() <= 2.0 ** -11 * max(1.0, np.abs(kh).max()) + 1e-4, ek.max()
        assert ev.max() <= 2.0 ** -11 * max(1.0, np.abs(vh).max()) + 1e-4, ev.max()
    return stats

"""GPU parity at the full sizes of the five configurations, in the launch configuration that
bench.py times (whole-sequence kvm_prefill on the default kernels), checked on sampled
(batch, head) units: units are independent end to end, so the oracle run on a unit alone gives that
unit's exact reference for every token, slot and state row.  Config 5 keeps its full length and
block structure (65536-token sqrt-growth prefill in segments, then 256 decode steps that end with a
fold) twice: on a reduced batch with every state tensor compared, and on the full batch (B64 x H32, the
state bench.py times: one readout copy, folds on the caller's stream, no fp64 memory keys) with outputs,
slots and append flags of sampled units compared (exporting the full state would move 17 GB to the host)."""
import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
CFG = synth.CONFIGS


def _full(name, units):
    wl = CFG[name]
    params = synth.make_layer_params(wl)
    tensors = synth.make_inputs(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units)
    stats = pu.compare(wl, y_gpu, st, y_ref, o, units=units)
    stats["counters"] = st.debug_counters()
    st.free()
    print(name, stats)
    return stats


def test_config2_full_size_sampled_units():
    _full("cfg2", [(0, 0), (0, 7), (1, 3), (1, 15)])


def test_config3_full_size_sampled_units():
    _full("cfg3", [(0, 5), (0, 31)])


def test_config4_full_size_sampled_unit():
    _full("cfg4", [(0, 2)])


@pytest.mark.parametrize("B,H,units", [(2, 2, [(0, 1), (1, 0)]), (64, 32, [(5, 30), (58, 3)])])
def test_config5_full_length_prefill_then_256_decode_steps(B, H, units):
    from paper_2605_09877_b200 import kvm
    wl = CFG["cfg5"].scaled(B=B, Hq=H, Hkv=H)
    full = B * H >= 256
    seg = 4096
    g = kvm.growth(wl.growth, wl.fixed_slots, wl.sqrt_coeff)
    total = wl.T + wl.decode_steps
    cap = kvm.kvm_plan_capacity(wl.C, wl.w, g, total)
    st = kvm.KVMState(kvm.LayerConfig(wl.B, wl.Hq, wl.Hkv, wl.d, wl.C, cap, seg, max_seq_len=total,
                                      flags=kvm.FLAG_RECORD_ASSIGN))
    from oracle.kvm_oracle import KVMOracle
    o = KVMOracle(pu.oracle_config(wl, n_units=len(units)))
    worst = dict(max_abs=0.0, mean_abs=0.0)

    def check(y_gpu, y_ref):
        yg = np.stack([y_gpu[u] for u in units])[None]
        err = np.abs(yg - y_ref)
        worst["max_abs"] = max(worst["max_abs"], float(err.max()))
        worst["mean_abs"] = max(worst["mean_abs"], float(err.mean()))
        assert err.max() <= pu.MAX_ABS and err.mean() <= pu.MEAN_ABS, (err.max(), err.mean())

    for s in range(wl.T // seg):
        t = synth.make_segment(wl, s, seg, device="cuda")
        y = st.prefill(t["q"], t["k"], t["v"], wl.C, g, wl.r)
        sub, _ = pu.select_units(wl, t, units, {})
        y_ref = o.forward(pu.to_f64(sub["q"]), pu.to_f64(sub["k"]), pu.to_f64(sub["v"]))
        check({u: y[u].double().cpu().numpy() for u in units}, y_ref)
        del t, y
    assert st.info()["n_slots"] == 4096 == o.rows
    for i in range(wl.decode_steps):
        d = synth.make_decode_inputs(wl, i, device="cuda")
        y = st.decode_step(d["q"], d["k"], d["v"])
        sub, _ = pu.select_units(wl, {k_: v_[:, :, None] for k_, v_ in d.items()}, units, {})
        y_ref = o.forward(pu.to_f64(sub["q"]), pu.to_f64(sub["k"]), pu.to_f64(sub["v"]))
        check({u: y[u].double().cpu().numpy()[None] for u in units}, y_ref)
    torch.cuda.synchronize()
    assert st.check() == 0
    info = st.info()
    assert info["n_slots"] == o.rows == 4103 and info["n_folds"] == o.nfolds and info["position"] == total
    uidx = [b * wl.Hkv + h for (b, h) in units]
    slot_g, app_g = st.assignments()
    slot_o, app_o, margin = o.assignments()
    assert np.array_equal(slot_g[uidx], slot_o) and np.array_equal(app_g[uidx], app_o)
    if full:
        print("cfg5 full batch", worst, "min routing margin", float(margin.min()), st.debug_counters())
        st.free()
        return
    eg, eo = st.export(), o.export()
    assert np.array_equal(eg["count"][uidx], eo["count"])
    mk = np.abs(eg["sum_k"][uidx] / eg["weight"][uidx][..., None] - eo["sum_k"] / eo["weight"][..., None])
    mv = np.abs(eg["sum_v"][uidx].astype(np.float64) / eg["weight"][uidx][..., None] - eo["sum_v"] / eo["weight"][..., None])
    assert mk.max() <= pu.MAX_ABS and mv.max() <= pu.MAX_ABS
    print("cfg5 full length", worst, "min routing margin", float(margin.min()), st.debug_counters())
    st.free()

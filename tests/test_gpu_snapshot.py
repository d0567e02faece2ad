"""Checkpoint / resume through the C ABI: prefill T1 tokens, take a snapshot (kvm_state_snapshot_info +
kvm_state_export + kvm_state_export_window), free the state, create a new one, kvm_state_import, and
continue with prefill and decode steps.  Everything after the cut must equal the uninterrupted run bit
for bit: outputs, sums, counts, radii and the slot of every later token."""
import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _continue(st, g, wl, q, k, v, gate, a, b, dec_from):
    y = torch.zeros_like(q[:, :, a:b])
    if dec_from > a:
        gs = None if gate is None else gate[:, :, a:dec_from].contiguous()
        st.prefill(q[:, :, a:dec_from], k[:, :, a:dec_from], v[:, :, a:dec_from], wl.C, g, wl.r, out=y[:, :, :dec_from - a], gate=gs)
    for t in range(max(dec_from, a), b):
        gt = None if gate is None else gate[:, :, t].contiguous()
        y[:, :, t - a] = st.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), gate=gt)
    torch.cuda.synchronize()
    return y.cpu()


SERIAL = 1 << 5   # KVM_FLAG_SERIAL_FOLDS


@pytest.mark.parametrize("wl,cut,params_trivial,use_gate,flags", [
    (synth.Workload("snapA", 2, 4, 2, 128, 256 * 6 + 90, 256, "sqrt", sqrt_coeff=10, r=32, seed=41), 256 * 3 + 77, False, True, 0),
    (synth.Workload("snapB", 1, 3, 3, 64, 64 * 20 + 5, 64, "fixed", fixed_slots=200, r=0, seed=42, kind="mixture"), 64 * 9, True, False, 0),
    (synth.Workload("snapC", 1, 2, 2, 64, 300, 32, "sqrt", sqrt_coeff=6, r=16, seed=43, w=3), 17, True, False, 0),   # cut before any fold
    (synth.Workload("snapD", 1, 40, 40, 128, 256 * 5 + 33, 256, "sqrt", r=0, seed=44), 256 * 4 + 1, True, False, 0),  # four-rows-per-warp apply
    # one readout copy, folds on the caller's stream
    (synth.Workload("snapF", 1, 4, 2, 128, 128 * 9 + 60, 128, "sqrt", sqrt_coeff=5, r=32, seed=46), 128 * 4 + 9, False, True, SERIAL),
    # the same with 64 units x block 128: no fp64 memory keys are kept, the import rebuilds the per-row statistics
    (synth.Workload("snapG", 2, 32, 32, 128, 128 * 8 + 50, 128, "sqrt", sqrt_coeff=5, r=32, seed=47), 128 * 5 + 3, False, False, SERIAL),
])
def test_snapshot_restore_continue_equals_uninterrupted_run(wl, cut, params_trivial, use_gate, flags):
    params = synth.make_layer_params(wl, trivial=params_trivial)
    tensors = synth.make_inputs(wl)
    gate_cpu = synth.make_gate(wl) if use_gate else None
    q, k, v = (tensors[n].cuda() for n in "qkv")
    gate = None if gate_cpu is None else gate_cpu.cuda()
    dec_from = wl.T - 40
    # uninterrupted: prefill [0, cut), prefill [cut, dec_from), decode the rest (same call boundaries as the resumed run)
    ref, g = pu.gpu_layer(wl, params, flags=flags)
    y0 = _continue(ref, g, wl, q, k, v, gate, 0, cut, cut)
    y_ref = _continue(ref, g, wl, q, k, v, gate, cut, wl.T, dec_from)
    e_ref = ref.export()
    slot_ref, app_ref = ref.assignments()
    ref.free()
    # interrupted: prefill [0, cut) -> snapshot -> free -> create -> import -> continue
    a, g = pu.gpu_layer(wl, params, flags=flags)
    y0b = _continue(a, g, wl, q, k, v, gate, 0, cut, cut)
    assert torch.equal(y0, y0b)
    snap = a.snapshot()
    info_a = a.info()
    a.free()
    b, g = pu.gpu_layer(wl, params, flags=flags)
    b.restore(snap)
    assert b.info() == info_a
    y_b = _continue(b, g, wl, q, k, v, gate, cut, wl.T, dec_from)
    assert b.check() == 0
    assert torch.equal(y_b, y_ref)
    e_b = b.export()
    for name in ("sum_k", "sum_v", "radius", "weight", "count"):
        assert np.array_equal(e_b[name], e_ref[name]), name
    assert torch.equal(e_b["k_read"], e_ref["k_read"]) and torch.equal(e_b["v_read"], e_ref["v_read"])
    slot_b, app_b = b.assignments()
    # tokens folded after the cut carry their slots; what was folded before the snapshot is not part of it
    later = slot_b >= 0
    assert later.sum() > 0 or wl.T - cut < wl.C
    assert np.array_equal(slot_b[later], slot_ref[later]) and np.array_equal(app_b[later], app_ref[later])
    # import into a state that is in use (implicit reset) gives the same continuation
    b.restore(snap)
    y_b2 = _continue(b, g, wl, q, k, v, gate, cut, wl.T, dec_from)
    assert torch.equal(y_b2, y_ref)
    b.free()


def test_import_rejects_inconsistent_snapshots_and_leaves_the_state_untouched():
    from paper_2605_09877_b200 import kvm
    wl = synth.Workload("snapE", 1, 2, 2, 64, 64 * 6, 64, "sqrt", sqrt_coeff=8, r=0, seed=45)
    params = synth.make_layer_params(wl)
    t = synth.make_inputs(wl)
    q, k, v = (t[n].cuda() for n in "qkv")
    st, g = pu.gpu_layer(wl, params)
    st.prefill(q, k, v, wl.C, g, wl.r)
    snap = st.snapshot()
    before = st.info()
    for field, val, code in (("n_slots", snap["info"].n_slots + 1, 1), ("n_folds", 0, 1), ("window_begin", 0, 1),
                             ("block", 60, 1), ("block", 512, 6), ("rope_dims", 3, 1), ("position", -1, 1)):
        bad = dict(snap)
        info = kvm.SnapshotInfo.from_buffer_copy(snap["info"])
        setattr(info, field, val)
        bad["info"] = info
        with pytest.raises(kvm.KVMError) as e:
            st.restore(bad)
        assert e.value.code == code, (field, e.value.code)
        assert st.info() == before
    small, _ = pu.gpu_layer(wl.scaled(T=64 * 3), params)   # capacity for three blocks only
    with pytest.raises(kvm.KVMError) as e:
        small.restore(snap)
    assert e.value.code == 6
    small.free()
    st.free()

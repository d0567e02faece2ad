"""Failure detection on the GPU without a GPU fault: a bounded device-side wait that runs out is reported
through the status word and leaves the context and the state usable; inputs outside the fp16 range that
the library works in are counted; host-side errors are covered in test_gpu_parity.py."""
import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_once_and_the_state_carries_on():
    """kvm_debug_expire_wait runs the library's bounded wait (10^4 spins) on a barrier nothing arrives at:
    the kernel returns normally, kvm_state_check reports KVM_ERR_TIMEOUT once, and the layer then finishes
    its sequence with results that match the oracle."""
    from paper_2605_09877_b200 import kvm
    wl = synth.Workload("fail", 1, 2, 2, 64, 64 * 7 + 9, 64, "sqrt", sqrt_coeff=6, r=16, seed=51)
    params = synth.make_layer_params(wl)
    tensors = synth.make_inputs(wl)
    q, k, v = (tensors[n].cuda() for n in "qkv")
    st, g = pu.gpu_layer(wl, params)
    y = torch.zeros_like(q)
    cut = 64 * 3 + 5
    st.prefill(q[:, :, :cut], k[:, :, :cut], v[:, :, :cut], wl.C, g, wl.r, out=y[:, :, :cut])
    assert st.check() == 0
    st.debug_expire_wait(10000)
    assert st.check() == 7          # KVM_ERR_TIMEOUT
    assert st.check() == 0          # reported once
    st.prefill(q[:, :, cut:], k[:, :, cut:], v[:, :, cut:], wl.C, g, wl.r, out=y[:, :, cut:])
    torch.cuda.synchronize()
    assert st.check() == 0
    y_ref, o = pu.run_oracle(wl, tensors, params)
    print(pu.compare(wl, y.cpu(), st, y_ref, o))
    with pytest.raises(kvm.KVMError) as e:
        st.debug_expire_wait(0)
    assert e.value.code == 1
    st.free()


def test_inputs_outside_the_fp16_range_are_clamped_and_counted():
    """bf16 inputs are carried as fp16 inside the library: magnitudes above 65504 saturate.  The debug counter
    says how many elements of q, k, v that hit, on the prefill path (16-byte and 4-byte ingest) and in
    decode steps; the outputs stay finite."""
    wl = synth.Workload("sat", 1, 2, 2, 64, 64 * 3 + 2, 64, "fixed", fixed_slots=64, r=0, seed=52)
    params = synth.make_layer_params(wl)
    tensors = synth.make_inputs(wl)
    tensors["q"][0, 0, 5, 3] = 1.0e5
    tensors["k"][0, 1, 70, 0] = -3.0e6
    tensors["v"][0, 0, 100, 63] = 7.0e4
    tensors["v"][0, 1, 64 * 3 + 1, 1] = -1.0e5        # a decode-step token
    tensors["q"][0, 1, 64 * 3, 9] = float("inf")       # a decode-step token
    y, st = pu.run_gpu(wl, tensors, params, decode_from=64 * 3)
    assert torch.isfinite(y.float()).all()
    assert st.debug_counters()["clamped_inputs"] == 5
    st.free()
    # rows that are not 16-byte aligned take the 4-byte ingest kernels: same count
    st, g = pu.gpu_layer(wl, params)
    pad = {n: torch.zeros((1, 2, wl.T, 68), dtype=torch.bfloat16, device="cuda") for n in "qkv"}
    for n in "qkv":
        pad[n][..., 2:66] = tensors[n].cuda()
    view = {n: pad[n][..., 2:66] for n in "qkv"}
    st.prefill(view["q"][:, :, :192], view["k"][:, :, :192], view["v"][:, :, :192], wl.C, g, wl.r)
    torch.cuda.synchronize()
    assert st.debug_counters()["clamped_inputs"] == 3
    st.free()


def test_gate_status_word_stays_clear_on_the_success_path():
    from paper_2605_09877_b200 import kvm
    g = torch.Generator().manual_seed(53)
    x = torch.randn((2, 512, 1024), generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn((16, 1024), generator=g) / 32).float().cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    gate = kvm.merge_gate(x, w, status=status)      # 16 heads, d_model % 64 == 0: the tensor-core path
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.isfinite(gate).all()

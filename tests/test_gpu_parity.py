"""GPU parity: the CUDA library (through the C ABI) against the fp64 oracle, element by element,
on the same seeded inputs.  Bit-exact for row counts, fold counts, slot assignments, append flags
and member counts; max-abs 2e-2 / mean-abs 2e-3 for bf16 outputs and state means."""
import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

CFG = synth.CONFIGS


def _run(wl, params=None, gate=False, cuts=None, decode_from=None, flags=0, radius_on=True, units=None,
         check_state=True):
    params = params or synth.make_layer_params(wl, trivial=True)
    tensors = synth.make_inputs(wl)
    if gate:
        tensors["gate"] = synth.make_gate(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params, cuts=cuts, flags=flags, radius_on=radius_on, decode_from=decode_from)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units, radius_on=radius_on)
    stats = pu.compare(wl, y_gpu, st, y_ref, o, units=units, check_state=check_state)
    st.free()
    return stats


def test_config1_full():
    """Config 1 exactly as stated: B1 H1 d64 T1024 C64, fixed 64 slots, no RoPE, seed 0."""
    stats = _run(CFG["cfg1"])
    print("cfg1", stats)


def test_config1_simt_paths():
    from paper_2605_09877_b200 import kvm
    _run(CFG["cfg1"], flags=kvm.FLAG_SIMT_ATTENTION | kvm.FLAG_SIMT_ROUTING)


def test_config2_reduced_several_tiles_and_ragged_tail():
    """Config 2's structure (fixed 512, C 128, partial RoPE 32, keys / sqrt(d)) at a size the
    oracle finishes in seconds; T is not a multiple of C so the last block stays in the window."""
    wl = CFG["cfg2"].scaled(B=2, Hq=3, Hkv=3, T=1500)
    print("cfg2-reduced", _run(wl))


def test_config3_reduced_sqrt_growth_mixture():
    wl = CFG["cfg3"].scaled(Hq=3, Hkv=3, T=3072 + 77)
    print("cfg3-reduced", _run(wl))


def test_config4_reduced_needles_rope_far_positions():
    wl = CFG["cfg4"].scaled(Hq=2, Hkv=2, T=4096)
    print("cfg4-reduced", _run(wl))


def test_config5_reduced_prefill_then_decode_with_fold():
    """Config 5's structure: sqrt-growth prefill, then single-token decode steps that cross a
    block boundary (the decode-time fold)."""
    wl = CFG["cfg5"].scaled(B=3, Hq=2, Hkv=2, T=2048 + 300)
    print("cfg5-reduced", _run(wl, decode_from=2048))


def test_segmented_prefill_equals_single_call():
    wl = CFG["cfg2"].scaled(B=1, Hq=2, Hkv=2, T=1100)
    print(_run(wl, cuts=[0, 1, 130, 131, 600, 1027, 1100], gate=True))


def test_decode_only_from_a_short_prefill():
    wl = CFG["cfg1"].scaled(T=400, r=16)
    print(_run(wl, decode_from=7))


@pytest.mark.parametrize("C,d,w,S", [(8, 64, 2, 1), (16, 128, 3, 0), (24, 64, 1, 3), (256, 128, 2, 1)])
def test_shapes_blocks_windows_sinks(C, d, w, S):
    wl = synth.Workload("t", 2, 2, 2, d, C * 9 + 3, C, "sqrt", sqrt_coeff=5, r=8, w=w, S=S, seed=11)
    print(_run(wl))


def test_affine_layernorm_temperatures_gate_gqa():
    wl = synth.Workload("t", 2, 4, 2, 128, 1280, 64, "fixed", fixed_slots=160, r=64, seed=12)
    params = synth.make_layer_params(wl, trivial=False)
    print(_run(wl, params=params, gate=True))


def test_unbounded_growth_never_merges():
    wl = synth.Workload("t", 1, 2, 2, 64, 640, 32, "unbounded", r=0, seed=13)
    stats = _run(wl)
    print(stats)


@pytest.mark.parametrize("kw", [dict(growth="power", sqrt_coeff=8, pow_num=2, pow_den=3),
                                dict(growth="power", sqrt_coeff=3, pow_num=3, pow_den=4),
                                dict(growth="saturating", fixed_slots=300, sat_half=1024)])
def test_power_law_and_saturating_budgets(kw):
    """The two further schedule shapes of Section 3.2 (exact integer budgets on both sides)."""
    wl = synth.Workload("t", 1, 2, 2, 64, 64 * 40 + 9, 64, r=16, seed=17, kind="mixture", **kw)
    print(_run(wl))


def test_attention_with_more_tiles_than_sms_splits_the_last_partial_wave():
    """160 (head, query tile) pairs on 148 SMs: the 12 tiles of the last wave run as two key splits each
    while the others keep one CTA; outputs must not show which tiles were split."""
    wl = synth.Workload("t", 1, 80, 80, 64, 256 * 5 + 60, 256, "sqrt", sqrt_coeff=16, r=16, seed=21)
    print(_run(wl))


def test_many_rows_per_fold_use_the_four_rows_per_warp_apply_kernel():
    """32 units x 256 tokens = 8192 rows per fold: the apply variant for large launches, head_dim 128,
    gates and affine LayerNorm included."""
    wl = synth.Workload("t", 2, 16, 16, 128, 256 * 4 + 70, 256, "sqrt", sqrt_coeff=12, r=32, seed=22, kind="mixture")
    params = synth.make_layer_params(wl, trivial=False)
    print(_run(wl, params=params, gate=True))


def test_radius_switch_off():
    wl = synth.Workload("t", 1, 2, 2, 64, 640, 32, "fixed", fixed_slots=48, seed=14)
    print(_run(wl, radius_on=False, gate=True))


def test_constructed_ties_route_to_lowest_eligible_row():
    """All keys equal: every similarity ties exactly; both sides must pick row S."""
    wl = synth.Workload("t", 1, 1, 1, 64, 256, 16, "fixed", fixed_slots=16, seed=15)
    tensors = synth.make_inputs(wl)
    tensors["k"] = torch.full_like(tensors["k"], 0.5)
    params = synth.make_layer_params(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params)
    y_ref, o = pu.run_oracle(wl, tensors, params)
    pu.compare(wl, y_gpu, st, y_ref, o)
    slot, app = st.assignments()
    merged = (slot >= 0) & (app == 0)
    assert merged.sum() > 0 and np.all(slot[merged] == 1)
    st.free()


def test_single_token_prefill_and_empty_state():
    wl = synth.Workload("t", 1, 1, 1, 64, 1, 16, "fixed", fixed_slots=16, seed=16)
    print(_run(wl))


def test_run_to_run_determinism():
    wl = CFG["cfg3"].scaled(Hq=2, Hkv=2, T=2048)
    tensors = synth.make_inputs(wl)
    params = synth.make_layer_params(wl)
    outs = []
    for _ in range(3):
        y, st = pu.run_gpu(wl, tensors, params)
        e = st.export()
        outs.append((y, e["sum_k"].copy(), e["sum_v"].copy()))
        st.free()
    for y, sk, sv in outs[1:]:
        assert torch.equal(y, outs[0][0]) and np.array_equal(sk, outs[0][1]) and np.array_equal(sv, outs[0][2])


def test_run_to_run_determinism_with_split_tail_and_four_row_apply():
    """The shape of the many-tiles test (key splits on the last wave, whose merge order is fixed by
    construction, and the apply variant for large launches): three runs, identical bits."""
    wl = synth.Workload("t", 1, 80, 80, 64, 256 * 4 + 30, 256, "sqrt", sqrt_coeff=16, r=16, seed=23)
    tensors = synth.make_inputs(wl)
    params = synth.make_layer_params(wl)
    outs = []
    for _ in range(3):
        y, st = pu.run_gpu(wl, tensors, params)
        e = st.export()
        outs.append((y, e["sum_k"].copy(), e["sum_v"].copy()))
        st.free()
    for y, sk, sv in outs[1:]:
        assert torch.equal(y, outs[0][0]) and np.array_equal(sk, outs[0][1]) and np.array_equal(sv, outs[0][2])


def test_host_buffer_entry_points_match_device_ones():
    from paper_2605_09877_b200 import kvm
    wl = CFG["cfg1"].scaled(T=300)
    tensors = synth.make_inputs(wl)
    params = synth.make_layer_params(wl)
    y_dev, st = pu.run_gpu(wl, tensors, params, decode_from=256)
    st.free()
    o256 = torch.zeros_like(tensors["q"][:, :, :256].contiguous())
    st3, g = pu.gpu_layer(wl, params, max_call_tokens=256)
    st3.prefill_host(tensors["q"][:, :, :256].contiguous(), tensors["k"][:, :, :256].contiguous(),
                     tensors["v"][:, :, :256].contiguous(), wl.C, g, wl.r, o256)
    assert torch.equal(o256, y_dev[:, :, :256])
    for t in range(256, 300):
        o1 = torch.zeros_like(tensors["q"][:, :, t].contiguous())
        st3.decode_step_host(tensors["q"][:, :, t].contiguous(), tensors["k"][:, :, t].contiguous(),
                             tensors["v"][:, :, t].contiguous(), o1)
        assert torch.equal(o1, y_dev[:, :, t])
    st3.free()


def test_host_prefill_pipelined_segments_match_device_prefill():
    """A long call through kvm_prefill_host is cut into segments whose copies overlap the compute;
    the result must equal the single device call bit for bit (gates included)."""
    wl = CFG["cfg2"].scaled(B=1, Hq=2, Hkv=2, T=128 * 33 + 5)
    tensors = synth.make_inputs(wl)
    tensors["gate"] = synth.make_gate(wl)
    params = synth.make_layer_params(wl)
    y_dev, st = pu.run_gpu(wl, tensors, params)
    ref = st.export()
    st.free()
    st2, g = pu.gpu_layer(wl, params)
    out = torch.zeros_like(tensors["q"])
    st2.prefill_host(tensors["q"].contiguous(), tensors["k"].contiguous(), tensors["v"].contiguous(), wl.C, g, wl.r, out,
                     gate=tensors["gate"].contiguous())
    assert torch.equal(out, y_dev)
    got = st2.export()
    assert np.array_equal(got["sum_k"], ref["sum_k"]) and np.array_equal(got["count"], ref["count"])
    st2.free()


def test_caller_stream_ordering_segments_and_decode_on_a_side_stream():
    """Everything is ordered on the caller's stream: segmented prefill and decode steps issued on a
    non-default stream, with no host synchronisation in between, equal the default-stream run with
    the same cuts bit for bit.  Against the single-call run the state is bit-equal too; the outputs
    agree to the bf16 tolerance only, since cuts inside a block shift the key tiles and with them
    the fp32 summation order."""
    wl = CFG["cfg3"].scaled(Hq=2, Hkv=2, T=256 * 7 + 40)
    tensors = synth.make_inputs(wl)
    params = synth.make_layer_params(wl)
    cuts = [0, 700, 1111, 256 * 7]
    y_one, st = pu.run_gpu(wl, tensors, params, decode_from=256 * 7)
    ref = st.export()
    st.free()
    y_cut, st = pu.run_gpu(wl, tensors, params, cuts=cuts, decode_from=256 * 7)
    st.free()
    st2, g = pu.gpu_layer(wl, params, max_call_tokens=700)
    dev = torch.device("cuda:0")
    q, k, v = (tensors[n].to(dev) for n in "qkv")
    y = torch.zeros_like(q)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for a, b in zip(cuts[:-1], cuts[1:]):
            st2.prefill(q[:, :, a:b], k[:, :, a:b], v[:, :, a:b], wl.C, g, wl.r, out=y[:, :, a:b], stream=side)
        for t in range(256 * 7, wl.T):
            y[:, :, t] = st2.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), stream=side)
    side.synchronize()
    assert st2.check() == 0
    assert torch.equal(y.cpu(), y_cut)
    err = (y.cpu().double() - y_one.double()).abs()
    assert float(err.max()) <= 2e-2 and float(err.mean()) <= 2e-3
    got = st2.export()
    for name in ("sum_k", "sum_v", "count"):
        assert np.array_equal(got[name], ref[name]), name
    st2.free()


def test_api_errors_leave_state_usable():
    from paper_2605_09877_b200 import kvm
    wl = CFG["cfg1"].scaled(T=128)
    params = synth.make_layer_params(wl)
    st, g = pu.gpu_layer(wl, params)
    t = synth.make_inputs(wl)
    q, k, v = (t[n].cuda() for n in "qkv")
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(q, k, v, 60, g, 0)          # block not a multiple of 8
    assert e.value.code == 1
    with pytest.raises(kvm.KVMError) as e:
        st.decode_step(q[:, :, 0].contiguous(), k[:, :, 0].contiguous(), v[:, :, 0].contiguous())
    assert e.value.code == 5                   # decode before any prefill fixed the block
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(q[:, :, :0], k[:, :, :0], v[:, :, :0], 64, g, 0)   # an empty call is rejected, not ignored
    assert e.value.code == 1
    st.prefill(q[:, :, :64], k[:, :, :64], v[:, :, :64], 64, g, 0)
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(q[:, :, 64:], k[:, :, 64:], v[:, :, 64:], 32, g, 0)
    assert e.value.code == 5
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(q[:, :, 64:], k[:, :, 64:], v[:, :, 64:], 64, g, 2)
    assert e.value.code == 5
    big = torch.zeros((1, 1, 129, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(big, big, big, 64, g, 0)
    assert e.value.code == 6
    st.prefill(q[:, :, 64:], k[:, :, 64:], v[:, :, 64:], 64, g, 0)
    assert st.info()["position"] == 128 and st.check() == 0
    st.free()
    # a failed first call binds nothing: the state takes another block / growth afterwards
    wl2 = wl.scaled(T=256)
    st, g = pu.gpu_layer(wl2, params)                      # rows for fixed 64 (rounded up to 128), calls of 256 tokens
    t2 = synth.make_inputs(wl2)
    q, k, v = (t2[n].cuda() for n in "qkv")
    with pytest.raises(kvm.KVMError) as e:
        st.prefill(q, k, v, 8, kvm.growth("unbounded"), 0)   # 256 tokens in blocks of 8, never merging: 248 rows
    assert e.value.code == 6
    assert st.info() == dict(n_slots=0, position=0, n_folds=0)
    # the host-buffer entry point validates the whole call before it copies anything
    hq, hk, hv = (t2[n].contiguous() for n in "qkv")
    ho = torch.zeros_like(hq)
    for bad_block in (0, -64, 60):
        with pytest.raises(kvm.KVMError) as e:
            st.prefill_host(hq, hk, hv, bad_block, g, 0, ho)
        assert e.value.code == 1
    with pytest.raises(kvm.KVMError) as e:
        st.prefill_host(hq, hk, hv, 8, kvm.growth("unbounded"), 0, ho)   # a later segment would exceed the capacity
    assert e.value.code == 6
    assert st.info() == dict(n_slots=0, position=0, n_folds=0) and float(ho.abs().sum()) == 0.0
    y = st.prefill(q, k, v, 64, g, 0)                        # and the state is still unbound and usable
    assert st.info()["position"] == 256 and st.check() == 0 and torch.isfinite(y.float()).all()
    st.free()
    with pytest.raises(kvm.KVMError):
        kvm.KVMState(kvm.LayerConfig(1, 1, 1, 96, 64, 64, 64))   # head_dim 96 unsupported

"""GPU parity for the kernel variants that only large launches select, each at the smallest shape that
still selects it, against the fp64 oracle on sampled (batch, head) units (units are independent end to
end, so the oracle run on a unit alone is that unit's exact reference):

  * the fold-decision kernel built for grids of more than 148 CTAs (two CTAs per SM, 64 registers);
  * the decode kernel's direct-output branch (one row split per head) at head_dim 128, with and without
    grouped queries;
  * config 5's structure at a batch wide enough to select the kernels that the full batch selects;
  * the minimum of two memory-key slots (one block of look-ahead), which very large batches run with;
  * what states that fill the GPU do: folds on the caller's stream with one readout copy, new-row products
    inside the decision kernel for folds that append few rows, memory keys recomputed from their fp16 copy.
"""
import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _sampled(wl, units, params=None, gate=False, decode_from=None, flags=0):
    params = params or synth.make_layer_params(wl)
    tensors = synth.make_inputs(wl)
    if gate:
        tensors["gate"] = synth.make_gate(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params, decode_from=decode_from, flags=flags)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units)
    stats = pu.compare(wl, y_gpu, st, y_ref, o, units=units)
    stats["counters"] = st.debug_counters()
    st.free()
    return stats


def test_fold_decide_two_ctas_per_sm_variant_head_dim_128():
    """160 units x block 256 at head_dim 128: one decision CTA per unit, 160 > 148 CTAs, so the 64-register
    build runs (the one every many-unit shape uses); gates and affine LayerNorm included."""
    wl = synth.Workload("t", 1, 160, 160, 128, 4 * 256 + 70, 256, "sqrt", sqrt_coeff=14, r=32, seed=31, kind="mixture")
    params = synth.make_layer_params(wl, trivial=False)
    print(_sampled(wl, [(0, 0), (0, 37), (0, 101), (0, 148), (0, 159)], params=params, gate=True))


def test_decode_direct_output_branch_head_dim_128():
    """640 query heads need no row split (nsplit == 1): the decode kernel writes its output directly.
    40 steps from position 1004 cross the block boundary at 1024, so one of them folds."""
    wl = synth.Workload("t", 20, 32, 32, 128, 1004 + 40, 256, "sqrt", r=0, seed=32)
    print(_sampled(wl, [(0, 0), (7, 13), (19, 31)], decode_from=1004))


def test_decode_grouped_queries_direct_and_split():
    """Four query heads per kv head: 640 query heads (direct output) and 8 query heads (row splits)."""
    wl = synth.Workload("t", 5, 128, 32, 128, 500 + 30, 128, "sqrt", r=32, seed=33)
    params = synth.make_layer_params(wl, trivial=False)
    print(_sampled(wl, [(0, 0), (2, 17), (4, 31)], params=params, decode_from=500))
    wl = synth.Workload("t", 1, 8, 2, 128, 700 + 30, 128, "sqrt", r=32, seed=34)
    print(_sampled(wl, [(0, 0), (0, 1)], decode_from=700))


def test_config5_structure_at_a_batch_that_selects_the_full_batch_kernels():
    """B8 x H32 = 256 units, block 256, sqrt growth, N(0,1) tokens, two prefill segments and a few decode
    steps: every kernel selection that depends on the number of units (decision kernel build, rows-per-warp
    apply, attention tail split, routing filter splits, decode without row splits) is the full batch's."""
    wl = synth.CONFIGS["cfg5"].scaled(B=8, T=3072 + 20)
    units = [(0, 0), (3, 9), (7, 31)]
    params = synth.make_layer_params(wl)
    tensors = synth.make_inputs(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params, cuts=[0, 2048, 3072], decode_from=3072)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units)
    print(pu.compare(wl, y_gpu, st, y_ref, o, units=units))
    st.free()


def test_two_memory_key_slots_one_block_of_look_ahead():
    """With only two memory-key slots every fold's keys are computed while the fold before it runs, and a
    slot is rewritten as soon as its fold is done: routing must still see its own block's keys."""
    from paper_2605_09877_b200 import kvm
    wl = synth.CONFIGS["cfg3"].scaled(Hq=3, Hkv=3, T=256 * 12 + 31)
    print(_sampled(wl, None, flags=kvm.FLAG_MIN_KEY_SLOTS))
    wl = synth.CONFIGS["cfg2"].scaled(B=2, Hq=2, Hkv=2, T=128 * 14)
    print(_sampled(wl, None, flags=kvm.FLAG_MIN_KEY_SLOTS, gate=True))


def test_serial_folds_one_readout_copy():
    """What states of 256 or more units do by themselves, forced on small shapes: folds on the caller's stream
    between the attention launches, one readout copy written in place; segmented prefill, gates, decode with a
    fold."""
    from paper_2605_09877_b200 import kvm
    wl = synth.CONFIGS["cfg3"].scaled(Hq=3, Hkv=3, T=256 * 9 + 31)
    print(_sampled(wl, None, flags=kvm.FLAG_SERIAL_FOLDS))
    wl = synth.Workload("t", 2, 4, 2, 128, 128 * 11 + 40, 128, "fixed", fixed_slots=400, r=32, seed=35)
    params = synth.make_layer_params(wl, trivial=False)
    tensors = synth.make_inputs(wl)
    tensors["gate"] = synth.make_gate(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params, cuts=[0, 300, 1000, 128 * 11], decode_from=128 * 11, flags=kvm.FLAG_SERIAL_FOLDS)
    y_ref, o = pu.run_oracle(wl, tensors, params)
    print(pu.compare(wl, y_gpu, st, y_ref, o))
    st.free()


def test_small_appends_compute_their_products_in_the_decision_kernel_and_keys_are_recomputed():
    """Serial states: a fold that appends at most 32 rows computes the products of its new rows with the block's
    keys itself (here every fold after the first: 4 sqrt(N) slots), larger ones use the batched launch (the
    second case, 16 sqrt(N): both kinds in one run).  64 units x block 128 is also the size from which no fp64
    memory keys are kept: every fp64 key the fold kernels use is recomputed from the fp16 key and the token's
    LayerNorm statistics.  Exact slots against the oracle say that the recomputed keys equal the stored ones."""
    from paper_2605_09877_b200 import kvm
    wl = synth.Workload("t", 2, 32, 32, 128, 128 * 12 + 31, 128, "sqrt", sqrt_coeff=4, r=32, seed=36)
    params = synth.make_layer_params(wl, trivial=False)
    stats = _sampled(wl, [(0, 0), (0, 19), (1, 7), (1, 31)], params=params, gate=True, flags=kvm.FLAG_SERIAL_FOLDS)
    print(stats)
    wl = synth.Workload("t", 2, 32, 32, 128, 128 * 40 + 77, 128, "sqrt", sqrt_coeff=16, r=32, seed=37, kind="mixture")
    print(_sampled(wl, [(0, 3), (1, 30)], flags=kvm.FLAG_SERIAL_FOLDS, decode_from=128 * 40 + 40))
    # the same small-append shape below the size threshold keeps its fp64 keys: products inside the kernel only
    wl = synth.Workload("t", 1, 3, 3, 64, 64 * 14 + 9, 64, "sqrt", sqrt_coeff=3, r=16, seed=38)
    print(_sampled(wl, None, flags=kvm.FLAG_SERIAL_FOLDS))


def test_bounds_first_decisions_head_dim_64_three_sink_rows_duplicated_keys():
    """More units than SMs: the decision kernel that ranks the tokens by the filter's bounds first and scores
    only the ones in doubt.  Head dimension 64, three sink rows (a sink row in reach takes a token's bounds
    away), mixture keys (near-duplicates inside a block: new rows in reach of many tokens), with the batched
    new-row products and with the products computed inside the kernel."""
    from paper_2605_09877_b200 import kvm
    wl = synth.Workload("t", 1, 160, 160, 64, 64 * 11 + 20, 64, "sqrt", sqrt_coeff=5, r=16, seed=39, kind="mixture", S=3)
    params = synth.make_layer_params(wl, trivial=False)
    units = [(0, 0), (0, 77), (0, 159)]
    print(_sampled(wl, units, params=params, gate=True))
    print(_sampled(wl, units, params=params, gate=True, flags=kvm.FLAG_SERIAL_FOLDS))
    wl = synth.Workload("t", 5, 32, 32, 128, 128 * 9 + 3, 128, "fixed", fixed_slots=300, r=32, seed=40, S=2)
    print(_sampled(wl, [(0, 0), (3, 11), (4, 31)], flags=kvm.FLAG_SERIAL_FOLDS))


def test_bounds_first_decisions_with_exactly_tied_scores():
    """More units than SMs, every key of a sequence equal (all similarities tie exactly) or every key repeated in
    the next block half (ties in pairs): the bounds decide nothing, every token is scored, and appended tokens,
    rows and merge targets must follow the tie rules (smaller token, lowest row) as in the oracle."""
    wl = synth.Workload("t", 1, 160, 160, 64, 32 * 9 + 5, 32, "sqrt", sqrt_coeff=3, r=0, seed=41)
    params = synth.make_layer_params(wl)
    units = [(0, 0), (0, 80), (0, 159)]
    tensors = synth.make_inputs(wl)
    tensors["k"] = torch.full_like(tensors["k"], 0.5)
    y_gpu, st = pu.run_gpu(wl, tensors, params)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units)
    print(pu.compare(wl, y_gpu, st, y_ref, o, units=units))
    st.free()
    tensors = synth.make_inputs(wl)
    k = tensors["k"]
    for b0 in range(0, wl.T - 31, 32):   # second half of every block repeats the first half
        k[:, :, b0 + 16:b0 + 32] = k[:, :, b0:b0 + 16]
    y_gpu, st = pu.run_gpu(wl, tensors, params)
    y_ref, o = pu.run_oracle(wl, tensors, params, units=units)
    print(pu.compare(wl, y_gpu, st, y_ref, o, units=units))
    st.free()


def test_many_units_run_to_run_and_across_variants_identical_bits():
    """256 units (bounds-first decisions, one readout copy, recomputed memory keys, one apply CTA per unit): three
    runs give identical bits, and the same problem run as 160 + 96 units in two states leaves the same state bit
    for bit (units are independent: the fold kernels chosen by the number of units must not change any unit's
    sums or counts)."""
    wl = synth.Workload("t", 8, 32, 32, 128, 256 * 6 + 77, 256, "sqrt", sqrt_coeff=12, r=32, seed=42, kind="mixture")
    tensors = synth.make_inputs(wl)
    params = synth.make_layer_params(wl)
    outs = []
    for _ in range(3):
        y, st = pu.run_gpu(wl, tensors, params)
        e = st.export()
        outs.append((y, e["sum_k"].copy(), e["sum_v"].copy(), e["count"].copy()))
        st.free()
    for y, sk, sv, c in outs[1:]:
        assert torch.equal(y, outs[0][0]) and np.array_equal(sk, outs[0][1]) and np.array_equal(sv, outs[0][2])
    # batch rows 0-4 (160 units: bounds-first kernel, two readout copies) and 5-7 (96 units: sliced decision kernel)
    for lo, hi in ((0, 5), (5, 8)):
        sub = wl.scaled(B=hi - lo)
        t = {k: v[lo:hi].contiguous() for k, v in tensors.items()}
        y, st = pu.run_gpu(sub, t, params)
        e = st.export()
        U0, U1 = lo * wl.Hkv, hi * wl.Hkv
        # (the attention launch may cut the last wave's tiles along the keys at one size and not at the other:
        #  outputs agree to the rounding of a different summation order, the state bit for bit)
        assert (y.float() - outs[0][0][lo:hi].float()).abs().max() <= 2e-2
        assert np.array_equal(e["sum_k"], outs[0][1][U0:U1]) and np.array_equal(e["sum_v"], outs[0][2][U0:U1])
        assert np.array_equal(e["count"], outs[0][3][U0:U1])
        st.free()


_SWEEP = [
    # (B, Hq, Hkv, d, C, blocks, extra, growth kwargs, r, S, w, kind, flags_serial, gate, decode)
    (5, 32, 32, 64, 16, 14, 3, dict(growth="sqrt", sqrt_coeff=2), 0, 0, 2, "normal", False, False, 0),
    (3, 64, 64, 64, 32, 10, 9, dict(growth="fixed", fixed_slots=96), 16, 2, 3, "mixture", True, True, 12),
    (10, 32, 16, 128, 64, 8, 1, dict(growth="power", sqrt_coeff=6, pow_num=2, pow_den=3), 32, 1, 2, "scaled_keys", False, True, 0),
    (6, 32, 32, 128, 128, 7, 50, dict(growth="saturating", fixed_slots=400, sat_half=600), 0, 4, 2, "needles", True, False, 20),
    (20, 8, 8, 64, 64, 9, 0, dict(growth="sqrt", sqrt_coeff=9), 16, 1, 4, "mixture", True, False, 0),
    (1, 150, 150, 128, 256, 4, 17, dict(growth="sqrt", sqrt_coeff=16), 32, 1, 2, "normal", True, True, 0),
]


@pytest.mark.parametrize("case", range(len(_SWEEP)))
def test_shape_sweep_with_more_units_than_sms(case):
    """Seeded sweep over the shapes the many-unit kernels meet: head dimension, block length from 16 to 256, every
    budget rule, sink rows from 0 to 4, window lengths, grouped queries, gates, rotary dimensions, with and without
    the serial-fold flag, prefill followed by decode steps; sampled units against the oracle."""
    from paper_2605_09877_b200 import kvm
    B, Hq, Hkv, d, C, nb, extra, gk, r, S, w, kind, serial, gate, dec = _SWEEP[case]
    T = C * nb + extra + dec
    wl = synth.Workload("sweep", B, Hq, Hkv, d, T, C, r=r, S=S, w=w, seed=100 + case, kind=kind, **gk)
    assert B * Hkv > 148
    params = synth.make_layer_params(wl, trivial=(case % 2 == 0))
    units = [(0, 0), (B // 2, Hkv // 2), (B - 1, Hkv - 1)]
    stats = _sampled(wl, units, params=params, gate=gate, decode_from=(T - dec) if dec else None,
                     flags=kvm.FLAG_SERIAL_FOLDS if serial else 0)
    print(case, stats)

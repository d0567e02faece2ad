"""Fused front end (KVM_FLAG_FUSED_QK_LN): LN_q / LN_k applied inside kvm_prefill / kvm_decode_step must give,
bit for bit, what kvm_head_layernorm on q and k followed by the plain calls gives - outputs, state sums,
slot of every token - and, through that chain, what the fp64 oracle gives within the layer's tolerance.
Also: grouped-query decode with 2 and 8 query heads per kv head."""
import numpy as np
import pytest
import torch

from oracle.frontend import head_layernorm as oracle_ln
from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _layer(wl, params, qk_ln=None, max_call_tokens=None):
    from paper_2605_09877_b200 import kvm
    g = kvm.growth(wl.growth, wl.fixed_slots, wl.sqrt_coeff)
    cap = max(kvm.kvm_plan_capacity(wl.C, wl.w, g, wl.T), wl.C)
    cfg = kvm.LayerConfig(wl.B, wl.Hq, wl.Hkv, wl.d, wl.C, cap, max_call_tokens or wl.T, max_seq_len=wl.T,
                          flags=kvm.FLAG_RECORD_ASSIGN)
    st = kvm.KVMState(cfg, ln_weight=params.get("ln_w"), ln_bias=params.get("ln_b"), tau_state=params.get("tau_s"),
                      tau_bswa=params.get("tau_b"), qk_ln=qk_ln)
    return st, g


def _run(st, g, wl, q, k, v, cuts, dec_from):
    y = torch.zeros_like(q)
    for a, b in zip(cuts[:-1], cuts[1:]):
        st.prefill(q[:, :, a:b], k[:, :, a:b], v[:, :, a:b], wl.C, g, wl.r, out=y[:, :, a:b])
    for t in range(dec_from, wl.T):
        y[:, :, t] = st.decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous())
    torch.cuda.synchronize()
    assert st.check() == 0
    return y.cpu()


@pytest.mark.parametrize("d,r,C", [(128, 32, 64), (64, 16, 32), (128, 0, 128)])
def test_fused_qk_layernorm_equals_standalone_kernel_then_plain_calls(d, r, C):
    from paper_2605_09877_b200 import kvm
    wl = synth.Workload("fe", 2, 4, 2, d, C * 6 + 7 + 12, C, "sqrt", sqrt_coeff=6, r=r, seed=61)
    params = synth.make_layer_params(wl, trivial=False)
    t = synth.make_inputs(wl)
    gen = torch.Generator().manual_seed(62)
    q = (t["q"].float() * 1.7 + 0.3).to(torch.bfloat16).cuda()      # off-centre rows: the normalisation has work to do
    k = (t["k"].float() * 0.6 - 0.2).to(torch.bfloat16).cuda()
    v = t["v"].cuda()
    wq = (1.0 + 0.2 * torch.randn((wl.Hq, d), generator=gen)).float()
    bq = (0.1 * torch.randn((wl.Hq, d), generator=gen)).float()
    wk = (1.0 + 0.2 * torch.randn((wl.Hkv, d), generator=gen)).float()
    eps = 1e-5
    dec_from = C * 6 + 7
    cuts = [0, C * 2 + 3, dec_from]
    # route A: the stand-alone kernel on copies of q and k, then the plain layer
    qa, ka = q.clone(), k.clone()
    kvm.head_layernorm(qa, wq.cuda(), bq.cuda(), eps)
    kvm.head_layernorm(ka, wk.cuda(), None, eps)
    sa, g = _layer(wl, params, max_call_tokens=dec_from)
    ya = _run(sa, g, wl, qa, ka, v, cuts, dec_from)
    ea, (slot_a, app_a) = sa.export(), sa.assignments()
    sa.free()
    # route B: the fused front end on the raw tensors
    sb, g = _layer(wl, params, qk_ln=dict(eps=eps, q_weight=wq.numpy(), q_bias=bq.numpy(), k_weight=wk.numpy()),
                   max_call_tokens=dec_from)
    yb = _run(sb, g, wl, q, k, v, cuts, dec_from)
    eb, (slot_b, app_b) = sb.export(), sb.assignments()
    assert torch.equal(ya, yb)
    for name in ("sum_k", "sum_v", "radius", "weight", "count"):
        assert np.array_equal(ea[name], eb[name]), name
    assert np.array_equal(slot_a, slot_b) and np.array_equal(app_a, app_b)
    # and against the oracle: fp64 LayerNorm (rounded to bf16 where the kernels round), then the fp64 layer
    qo = torch.from_numpy(oracle_ln(q.cpu().double().numpy(), wq.double().numpy(), bq.double().numpy(), eps)).to(torch.bfloat16)
    ko = torch.from_numpy(oracle_ln(k.cpu().double().numpy(), wk.double().numpy(), np.zeros((wl.Hkv, d)), eps)).to(torch.bfloat16)
    agree = (qo == qa.cpu()).float().mean().item()
    assert agree > 0.98     # (a value on a bf16 rounding boundary may fall either way after the fp32 error)
    y_ref, o = pu.run_oracle(wl, dict(q=qa.cpu(), k=ka.cpu(), v=v.cpu()), params)
    print(pu.compare(wl, yb, sb, y_ref, o))
    # rows that are not 16-byte aligned are refused by the fused front end
    pad = torch.zeros((wl.B, wl.Hq, 64, d + 4), dtype=torch.bfloat16, device="cuda")
    sb.reset()
    with pytest.raises(kvm.KVMError) as e:
        sb.prefill(pad[..., 2:d + 2], pad[:, :wl.Hkv, :, 2:d + 2], pad[:, :wl.Hkv, :, 2:d + 2], wl.C, g, wl.r)
    assert e.value.code == 1
    sb.free()


@pytest.mark.parametrize("G", [2, 8])
def test_decode_grouped_queries_share_a_cta(G):
    """G query heads per kv head: the decode kernel serves the whole group from one pass over the rows."""
    wl = synth.Workload("gq", 2, 2 * G, 2, 64 if G == 8 else 128, 300 + 70, 64, "sqrt", sqrt_coeff=7, r=16, seed=63 + G)
    params = synth.make_layer_params(wl, trivial=False)
    tensors = synth.make_inputs(wl)
    y_gpu, st = pu.run_gpu(wl, tensors, params, decode_from=300)
    y_ref, o = pu.run_oracle(wl, tensors, params)
    print(pu.compare(wl, y_gpu, st, y_ref, o))
    st.free()

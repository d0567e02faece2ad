"""kvm_attend_rows_noalloc against the regular decode entry point.

Some users of the library run where cudaMalloc is not allowed (all device memory belongs to their own
pool, or the section must not synchronise the device), so this entry point keeps the partial results
of its row splits in a fixed array inside the library instead of an allocated buffer.  The test feeds
it, through the C ABI, the very rows that kvm_decode_step attends over -- the state's readout cache
(kvm_state_export) followed by the window tokens -- and requires the same outputs within the layer's
tolerance, for two calls in a row (the second call finds the first call's leftovers in the array).
Collected last on purpose: a failure here stops nothing else under -x.
"""
import math

import numpy as np
import pytest
import torch

from paper_2605_09877_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _rows_for_step(st, k_all, v_all, t, wl):
    """Keys / values that decode step t attends over, per (batch, head): readout rows, then tokens [b, t]."""
    e = st.export()
    kr, vr = e["k_read"].cuda(), e["v_read"].cuda()                 # [U, m, d] fp16
    c = t // wl.C
    b = max(0, (c + 1) * wl.C - wl.w * wl.C)
    U = wl.B * wl.Hkv
    kw = k_all[:, :, b:t + 1].reshape(U, t + 1 - b, wl.d).to(torch.float16)   # bf16 -> fp16 is exact here (no RoPE)
    vw = v_all[:, :, b:t + 1].reshape(U, t + 1 - b, wl.d).to(torch.float16)
    return torch.cat([kr, kw], 1).contiguous(), torch.cat([vr, vw], 1).contiguous()


def test_noalloc_attention_matches_decode_step_twice():
    from paper_2605_09877_b200 import kvm
    # sqrt growth, no RoPE, 6 heads; 1500 prefill tokens leave a partial block in the window
    wl = synth.Workload("noalloc", 2, 3, 3, 128, 1500 + 2, 128, "sqrt", r=0, seed=21)
    t = synth.make_inputs(wl)
    q, k, v = (t[n].cuda() for n in "qkv")
    st, g = pu.gpu_layer(wl, synth.make_layer_params(wl), max_call_tokens=1500)
    st.prefill(q[:, :, :1500], k[:, :, :1500], v[:, :, :1500], wl.C, g, wl.r)
    scale = 1.0 / math.sqrt(wl.d)
    out = torch.empty((wl.B * wl.Hq, wl.d), dtype=torch.bfloat16, device="cuda")   # caller-owned output
    for step in range(2):
        pos = 1500 + step
        ref = st.decode_step(q[:, :, pos].contiguous(), k[:, :, pos].contiguous(), v[:, :, pos].contiguous())
        keys, vals = _rows_for_step(st, k, v, pos, wl)
        assert keys.shape[1] == st.info()["n_slots"] + (pos - 1280) + 1
        qh = q[:, :, pos].reshape(-1, wl.d).to(torch.float16).contiguous()
        kvm.attend_rows_noalloc(qh, keys, vals, scale, out=out)
        torch.cuda.synchronize()
        err = (out.double() - ref.reshape(-1, wl.d).double()).abs()
        assert torch.isfinite(out.double()).all()
        assert err.max().item() <= pu.MAX_ABS and err.mean().item() <= pu.MEAN_ABS, (step, err.max().item(), err.mean().item())
    st.free()


@pytest.mark.parametrize("d,heads,rows", [(128, 6, 1500), (64, 3, 8193), (64, 700, 300), (128, 40, 5000)])
def test_noalloc_attention_matches_the_fp64_definition_and_allocates_nothing(d, heads, rows):
    """The entry point against softmax(scale q K^T) V written out in fp64 on the same fp16 rows (so only the
    kernel's fp32 arithmetic and the bf16 rounding of the output separate the two), at both head sizes, with
    32 row splits of which the last ones are empty (8193 rows at head_dim 64), with one split per head
    (700 heads) and with two calls in a row; free device memory as the driver reports it is the same before
    and after the calls."""
    from oracle.attend_rows import attend_rows
    from paper_2605_09877_b200 import kvm
    g = torch.Generator().manual_seed(1000 + d + heads)
    q = torch.randn((heads, d), generator=g).to(torch.float16)
    keys = torch.randn((heads, rows, d), generator=g).to(torch.float16)
    vals = torch.randn((heads, rows, d), generator=g).to(torch.float16)
    keys[:, rows // 3] *= 3.0                      # one peaked row per head
    scale = 1.3 / math.sqrt(d)
    ref = attend_rows(q.numpy(), keys.numpy(), vals.numpy(), scale)
    qd, kd, vd = q.cuda(), keys.cuda(), vals.cuda()
    out = torch.empty((heads, d), dtype=torch.bfloat16, device="cuda")
    kvm.attend_rows_noalloc(qd, kd, vd, scale, out=out)      # (the first call on the device looks the array up)
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(2):
        out.zero_()
        kvm.attend_rows_noalloc(qd, kd, vd, scale, out=out)
        torch.cuda.synchronize()
        err = np.abs(out.double().cpu().numpy() - ref)
        # half a bf16 ulp of the output plus fp32 accumulation
        assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-4), float(err.max())
    assert torch.cuda.mem_get_info()[0] == free0


def test_noalloc_rejects_what_the_fixed_scratch_cannot_hold():
    from paper_2605_09877_b200 import kvm
    d = 128
    q = torch.zeros((16384, d), dtype=torch.float16, device="cuda")
    kv = torch.zeros((16384, 4, d), dtype=torch.float16, device="cuda")
    with pytest.raises(kvm.KVMError) as e:
        kvm.attend_rows_noalloc(q, kv, kv, 1.0)          # 16384 heads x 1 split > 8192 partial slots
    assert e.value.code == 6
    q96 = torch.zeros((2, 96), dtype=torch.float16, device="cuda")
    kv96 = torch.zeros((2, 4, 96), dtype=torch.float16, device="cuda")
    with pytest.raises(kvm.KVMError) as e:
        kvm.attend_rows_noalloc(q96, kv96, kv96, 1.0)
    assert e.value.code == 2

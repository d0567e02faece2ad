"""Merge gate g_t = 1 + ELU(x_t W_g) (Section 3.2 "KVM weight preparation", Eq. 2): pins of the fp64
oracle (closed forms, special cases, a library routine), then the CUDA entry point against it."""
import math

import numpy as np
import pytest
import torch

from oracle.frontend import elu, head_layernorm, merge_gate


def test_gate_closed_forms():
    # z = 0 -> g = 1 (a token that the gate neither damps nor amplifies); z > 0 -> 1 + z; z < 0 -> exp(z)
    x = np.array([[[0.0, 0.0], [2.0, 0.0], [-math.log(2.0), 0.0], [0.0, 5.0]]])   # [1, 4, 2]
    w = np.array([[1.0, 0.0]])                                                     # picks channel 0
    g = merge_gate(x, w)
    assert g.shape == (1, 1, 4)
    assert np.allclose(g[0, 0], [1.0, 3.0, 0.5, 1.0], rtol=0, atol=1e-15)
    # zero weights: every gate is exactly 1, the ungated layer
    assert np.all(merge_gate(np.random.default_rng(0).standard_normal((2, 7, 5)), np.zeros((3, 5))) == 1.0)


def test_gate_is_positive_monotone_and_continuous_at_zero():
    z = np.linspace(-30, 30, 2001)
    g = 1.0 + elu(z)
    assert np.all(g > 0) and np.all(np.diff(g) > 0)
    eps = 1e-9
    assert abs((1.0 + elu(np.array([eps]))[0]) - (1.0 + elu(np.array([-eps]))[0])) < 3e-9
    # derivative 1 on both sides of zero (ELU with alpha = 1 is C^1)
    assert abs((elu(np.array([1e-6]))[0] - elu(np.array([-1e-6]))[0]) / 2e-6 - 1.0) < 1e-6


def test_gate_matches_the_library_elu_and_a_plain_matmul():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 33, 48))
    w = rng.standard_normal((5, 48)) / math.sqrt(48)
    ref = 1.0 + torch.nn.functional.elu(torch.from_numpy(x) @ torch.from_numpy(w).T).permute(0, 2, 1).numpy()
    assert np.allclose(merge_gate(x, w), ref, rtol=1e-13, atol=1e-13)
    # layout: head h of batch b, token t uses W_g[h] and x[b, t]
    assert np.isclose(merge_gate(x, w)[1, 3, 17], 1.0 + elu(np.array([x[1, 17] @ w[3]]))[0])


@pytest.mark.gpu
@pytest.mark.parametrize("B,T,dm,H", [(2, 777, 1000, 3), (1, 64, 2048, 16), (3, 130, 72, 40), (2, 1, 256, 8),
                                      (1, 4096, 1024, 64), (2, 300, 512, 24), (1, 200, 256, 40), (2, 129, 64, 9),
                                      (1, 1, 4096, 32), (4, 19000, 128, 24), (2, 40000, 64, 40)])
def test_gate_kernel_against_the_oracle(B, T, dm, H):
    """Shapes cover both kernels (tensor cores when d_model is a multiple of 64 and there are more
    than 8 heads, else scalar cores), every head padding, ragged token tiles and a single token.
    Products of exactly converted bf16 inputs, sums in fp32, against fp64.  With |x| ~ 1 and
    |w| ~ 1/sqrt(d_model) a sum of d_model products in round-to-nearest fp32 carries an error of
    about sqrt(d_model) * 6e-8 in z; the tensor-core accumulator truncates instead of rounding, so
    its error grows like d_model * 2^-24 * |z| ~ 2.4e-4 |z| at d_model = 4096 in the worst case
    (measured: 3e-5).  On that path the weights enter as bf16 hi + bf16 lo (relative error 2^-17 per
    weight, products exact in fp32), which adds ~ 8e-6.  g = 1 + ELU(z) has slope <= max(1, g), hence
    the bound 2e-4 * max(1, g)."""
    from paper_2605_09877_b200 import kvm
    gen = torch.Generator().manual_seed(B * 1000 + T)
    x = torch.randn((B, T, dm), generator=gen).to(torch.bfloat16)
    w = (torch.randn((H, dm), generator=gen) / math.sqrt(dm)).float()
    g = kvm.merge_gate(x.cuda(), w.cuda())
    torch.cuda.synchronize()
    ref = merge_gate(x.double().numpy(), w.double().numpy())
    got = g.cpu().double().numpy()
    assert got.shape == ref.shape
    err = np.abs(got - ref) / np.maximum(1.0, ref)
    assert err.max() < 2e-4, err.max()


@pytest.mark.gpu
def test_gate_argument_checks():
    from paper_2605_09877_b200 import kvm
    x = torch.zeros((1, 8, 12), dtype=torch.bfloat16, device="cuda")   # d_model not a multiple of 8
    w = torch.zeros((2, 12), dtype=torch.float32, device="cuda")
    with pytest.raises(kvm.KVMError) as e:
        kvm.merge_gate(x, w)
    assert e.value.code == 1
    x = torch.zeros((1, 8, 16), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((65, 16), dtype=torch.float32, device="cuda")      # more than 64 heads
    with pytest.raises(kvm.KVMError) as e:
        kvm.merge_gate(x, w)
    assert e.value.code == 2
    g = kvm.merge_gate(x, torch.zeros((4, 16), dtype=torch.float32, device="cuda"))
    assert torch.all(g == 1.0)


# ---------------------------------------------------------------------------------------
# LN_q / LN_k

def test_head_layernorm_oracle_pins():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((2, 3, 5, 16)) * 3.0 + 1.5
    y = head_layernorm(x, eps=0.0)
    assert np.allclose(y.mean(-1), 0.0, atol=1e-14) and np.allclose((y ** 2).mean(-1), 1.0, atol=1e-13)
    # a constant row has no direction: with eps > 0 it maps to the bias
    b = rng.standard_normal((3, 16))
    yc = head_layernorm(np.full((1, 3, 2, 16), 7.0), bias=b, eps=1e-5)
    assert np.allclose(yc, b[None, :, None, :])
    # the library routine, head by head (weights are per head)
    w = rng.standard_normal((3, 16))
    ref = np.stack([torch.nn.functional.layer_norm(torch.from_numpy(x[:, h]), (16,), torch.from_numpy(w[h]),
                                                   torch.from_numpy(b[h]), 1e-5).numpy() for h in range(3)], axis=1)
    assert np.allclose(head_layernorm(x, w, b, 1e-5), ref, rtol=1e-12, atol=1e-12)
    # invariance to shift and positive scale of the input (eps = 0)
    assert np.allclose(head_layernorm(4.0 * x - 2.0, eps=0.0), y, atol=1e-12)


@pytest.mark.gpu
@pytest.mark.parametrize("B,H,T,d,affine", [(2, 3, 777, 128, True), (1, 5, 33, 64, True), (2, 2, 1, 128, False),
                                             (1, 16, 4096, 128, True)])
def test_head_layernorm_kernel_against_the_oracle(B, H, T, d, affine):
    """fp32 statistics of bf16 inputs, result rounded to bf16: within half a bf16 ulp of the fp64 value
    plus the fp32 error, i.e. |err| <= 2^-8 |y| + 1e-5 (the result of a rounding that may fall on
    either side of a tie)."""
    from paper_2605_09877_b200 import kvm
    gen = torch.Generator().manual_seed(7 * B + T)
    x = (torch.randn((B, H, T, d), generator=gen) * 2.0 + 0.5).to(torch.bfloat16)
    w = (1.0 + 0.3 * torch.randn((H, d), generator=gen)).float() if affine else None
    b = (0.2 * torch.randn((H, d), generator=gen)).float() if affine else None
    ref = head_layernorm(x.double().numpy(), None if w is None else w.double().numpy(),
                         None if b is None else b.double().numpy(), 1e-5)
    y = kvm.head_layernorm(x.cuda(), None if w is None else w.cuda(), None if b is None else b.cuda(), 1e-5)
    torch.cuda.synchronize()
    got = y.cpu().double().numpy()
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5)

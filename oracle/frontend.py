"""TEST INFRASTRUCTURE - fp64 oracle of the layer's front end.  Only tests/, __graft_entry__.smoke()
and bench.py's cpu_baseline leg may import this module; the product path never does.

head_layernorm: Appendix (time mixer of the backbone), "RoPE query / RoPE key": LN_q, LN_k are
LayerNorms over the head channels (biased variance, eps inside the root, per-head weight and bias).

merge_gate: Section 3.2 "KVM weight preparation", Eq. 2 (merge gate): g_t = 1 + ELU(x_t W_g), one
scalar per token and head.  ELU is the exponential linear unit with alpha = 1 (the paper names the
function without a parameter): ELU(z) = z for z > 0, exp(z) - 1 otherwise.  Written out from that
definition in numpy fp64; no blocking, no fusion.
"""
import numpy as np


def elu(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    return np.where(z > 0.0, z, np.expm1(np.minimum(z, 0.0)))


def merge_gate(x: np.ndarray, w_gate: np.ndarray) -> np.ndarray:
    """x [B, T, d_model], w_gate [H, d_model] (one d_model-vector W_g per head) -> g [B, H, T]."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w_gate, dtype=np.float64)
    assert x.ndim == 3 and w.ndim == 2 and x.shape[2] == w.shape[1]
    z = np.einsum("btc,hc->bht", x, w)
    return 1.0 + elu(z)


def head_layernorm(x: np.ndarray, weight=None, bias=None, eps: float = 1e-5) -> np.ndarray:
    """x [B, H, T, d] -> LayerNorm over d; weight, bias [H, d] or None."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    y = (x - mean) / np.sqrt(var + eps)
    if weight is not None:
        y = y * np.asarray(weight, dtype=np.float64)[None, :, None, :]
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :, None, :]
    return y

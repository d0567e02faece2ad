"""Pins of the fp64 gradient oracle (oracle/kvm_grad_oracle.py; CPU only): its forward against the C oracle,
its gradients against central finite differences of the C oracle's forward (an independent program), and the
never-compress limit against the textbook attention backward written out in numpy."""
import math

import numpy as np
import pytest

from oracle.kvm_grad_oracle import layer_forward, layer_grads
from oracle.kvm_oracle import KVMOracle, OracleConfig


def _inputs(cfg, T, seed, gate=True):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((cfg.B, cfg.Hq, T, cfg.d))
    k = rng.standard_normal((cfg.B, cfg.Hkv, T, cfg.d))
    v = rng.standard_normal((cfg.B, cfg.Hkv, T, cfg.d))
    g = 0.25 + 1.5 * rng.random((cfg.B, cfg.Hkv, T)) if gate else None
    dy = rng.standard_normal((cfg.B, cfg.Hq, T, cfg.d))
    params = dict(ln_w=1.0 + 0.2 * rng.standard_normal((cfg.Hkv, cfg.d)), ln_b=0.1 * rng.standard_normal((cfg.Hkv, cfg.d)),
                  tau_s=1.0 + 0.3 * rng.random(cfg.Hq), tau_b=0.8 + 0.3 * rng.random(cfg.Hq))
    return q, k, v, g, dy, params


def _c_forward(cfg, q, k, v, g, params):
    o = KVMOracle(cfg, **params)
    y = o.forward(q, k, v, g)
    slot, app, margin = o.assignments()
    return y, slot, app, margin


CASES = [
    OracleConfig(B=1, Hq=2, Hkv=1, d=8, C=4, w=2, S=1, r=4, growth="sqrt", sqrt_coeff=3),
    OracleConfig(B=2, Hq=2, Hkv=2, d=8, C=4, w=2, S=1, r=0, growth="fixed", fixed_slots=6),
    OracleConfig(B=1, Hq=1, Hkv=1, d=6, C=3, w=3, S=0, r=2, growth="sqrt", sqrt_coeff=2),
    OracleConfig(B=1, Hq=1, Hkv=1, d=8, C=4, w=2, S=1, r=4, growth="fixed", fixed_slots=5, radius_on=False),
]


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_forward_of_the_restatement_equals_the_c_oracle(ci):
    cfg = CASES[ci]
    T = cfg.C * 7 + 2
    q, k, v, g, dy, params = _inputs(cfg, T, 100 + ci)
    y_c, slot_c, app_c, _ = _c_forward(cfg, q, k, v, g, params)
    out = layer_grads(q, k, v, g, cfg, dy, **params)
    assert np.allclose(out["y"], y_c, rtol=1e-10, atol=1e-11)
    folded = slot_c >= 0
    assert np.array_equal(out["slots"][folded], slot_c[folded]) and np.array_equal(out["appended"][folded], app_c[folded] != 0)
    assert (out["slots"][~folded] == -1).all()


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_gradients_equal_central_differences_of_the_c_oracle(ci):
    """L = sum(y * dy).  Each sampled coordinate of q, k, v and the gate is moved by +-h in the C oracle; where
    the move leaves every routing decision as it was (it nearly always does), the difference quotient must
    equal the autograd gradient.  A dropped term - the radius, a LayerNorm statistic, the gate on merged
    tokens, the window/state temperature - shows up here."""
    cfg = CASES[ci]
    T = cfg.C * 6 + 1
    q, k, v, g, dy, params = _inputs(cfg, T, 200 + ci)
    out = layer_grads(q, k, v, g, cfg, dy, **params)
    _, slot0, app0, _ = _c_forward(cfg, q, k, v, g, params)
    rng = np.random.default_rng(300 + ci)
    h = 1e-6
    checked = 0
    for name, arr, grad in (("q", q, out["dq"]), ("k", k, out["dk"]), ("v", v, out["dv"]), ("gate", g, out["dgate"])):
        flat = arr.reshape(-1)
        for idx in rng.choice(flat.size, size=min(14, flat.size), replace=False):
            vals = []
            same = True
            for sgn in (+1.0, -1.0):
                old = flat[idx]
                flat[idx] = old + sgn * h
                y, slot, app, _ = _c_forward(cfg, q, k, v, g, params)
                flat[idx] = old
                same = same and np.array_equal(slot, slot0) and np.array_equal(app, app0)
                vals.append(float((y * dy).sum()))
            if not same:
                continue
            fd = (vals[0] - vals[1]) / (2 * h)
            an = float(grad.reshape(-1)[idx])
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(an), abs(fd)), (name, int(idx), fd, an)
            checked += 1
    assert checked >= 40
    # the tokens before the first fold only ever sit in the window: the gate cannot matter for tokens that were
    # appended (created rows are not gated) - their gate gradient is exactly zero
    if out["dgate"] is not None:
        assert np.all(out["dgate"].reshape(slot0.shape)[out["appended"] | (out["slots"] < 0)] == 0.0)


def test_never_compress_limit_equals_textbook_attention_backward():
    """Unbounded budget: nothing is ever merged, the layer is plain causal softmax attention over a transformed
    key set (window keys: RoPE(k); older keys: LN_s(LN_s(zero_r k))), with values unchanged (rho * v / ||v|| = v).
    dq and the part of dv that does not pass through the radius are then the textbook formulas
    dV = P^T dY, dP = dY V^T, dS = P * (dP - rowsum(dP * P)), dQ = dS K / sqrt(d)."""
    cfg = OracleConfig(B=1, Hq=1, Hkv=1, d=8, C=4, w=2, S=1, r=0, growth="unbounded")
    T = 23
    q, k, v, _, dy, _ = _inputs(cfg, T, 7, gate=False)
    out = layer_grads(q, k, v, None, cfg, dy)
    d, C, L = cfg.d, cfg.C, cfg.w * cfg.C

    def ln(x):
        mu = x.mean(-1, keepdims=True)
        return (x - mu) / np.sqrt(((x - mu) ** 2).mean(-1, keepdims=True) + cfg.ln_eps)

    K2 = ln(ln(k[0, 0]))                   # the key a token has once it sits in the state
    dq = np.zeros((T, d)); dvv = np.zeros((T, d))
    for t in range(T):
        e = (t // C + 1) * C
        wb = max(0, e - L)
        nstate = wb if e >= L else 0       # tokens [0, wb) sit in the state when block t//C is attended
        keys = np.concatenate([K2[:nstate], k[0, 0, wb:t + 1]])
        vals = np.concatenate([v[0, 0, :nstate], v[0, 0, wb:t + 1]])
        s = keys @ q[0, 0, t] / math.sqrt(d)
        p = np.exp(s - s.max()); p /= p.sum()
        assert np.allclose(p @ vals, out["y"][0, 0, t], atol=1e-10)
        dp = vals @ dy[0, 0, t]
        ds = p * (dp - (dp * p).sum())
        dq[t] = ds @ keys / math.sqrt(d)
        idx = np.concatenate([np.arange(nstate), np.arange(wb, t + 1)])
        np.add.at(dvv, idx, p[:, None] * dy[0, 0, t][None, :])
    assert np.allclose(out["dq"][0, 0], dq, atol=1e-10)
    # values: a state row reads out rho * v / ||v|| with rho = ||v||, i.e. v itself with derivative identity
    assert np.allclose(out["dv"][0, 0], dvv, atol=1e-9)

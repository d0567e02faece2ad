"""TEST INFRASTRUCTURE - fp64 gradient oracle of the KVM layer (training / backward pass, which the paper
benchmarks in Section 5 "Speed Benchmarks" next to prefill and decode).  Only tests/ may import it.

The layer is restated step by step in plain PyTorch CPU ops in float64 - partial RoPE, memory keys
LN_s(zero_r(k)) (Eq. 1), the single softmax over [state ; window] per block (Section 3.2 "Readout"), the
fold with append selection, merge routing and the gated merge update (Section 3.2 "Append", "Merge", budget
rule), value-radius readout - and differentiated by reverse-mode autograd.  The integer decisions of a fold
(which tokens are appended, which row a token merges into) are taken on detached values: the layer is
piecewise smooth in its inputs and the gradient is that of the piece the inputs lie in (routing held
constant), which is what a training step of the paper's model back-propagates.  Everything else carries
gradient, including the radius rho_i = ||v_creator|| of a row and the LayerNorm statistics.

Readings of open points are those of the forward oracle (oracle/kvm_oracle.c): half-split RoPE pairs with
angle t * base^(-2i/r); LayerNorm with biased variance over all d channels after zeroing the rotary ones;
budget floor(coeff * sqrt(e)) in integers, e = end of the block just attended; ties to the lowest index;
created rows ungated, merged tokens gated; eager folds.

Pins (tests/test_grad_oracle.py): the forward values and slot assignments of this restatement against the
C oracle; central finite differences of the C oracle's forward (an independent program) against these
gradients, coordinate by coordinate, away from routing ties; the never-compress limit against the textbook
softmax-attention backward formulas written out in numpy.
"""
from __future__ import annotations

import math

import torch


def _budget(cfg, e: int) -> int:
    if cfg.growth == "fixed":
        return cfg.fixed_slots
    if cfg.growth == "sqrt":
        return math.isqrt(cfg.sqrt_coeff * cfg.sqrt_coeff * e)
    if cfg.growth == "unbounded":
        return 1 << 60
    raise ValueError("gradient oracle: growth kinds fixed, sqrt, unbounded")


def _layer_norm(x, w, b, eps):
    mu = x.mean(dim=-1, keepdim=True)
    var = ((x - mu) ** 2).mean(dim=-1, keepdim=True)
    return w * (x - mu) / torch.sqrt(var + eps) + b


def _rope(x, t0: int, r: int, base: float):
    """x [n, d]: rows are positions t0, t0+1, ...; first r channels rotated, pairs (i, i + r/2)."""
    if r == 0:
        return x
    n = x.shape[0]
    half = r // 2
    i = torch.arange(half, dtype=torch.float64)
    ang = torch.arange(t0, t0 + n, dtype=torch.float64)[:, None] * base ** (-2.0 * i / r)[None, :]
    c, s = torch.cos(ang), torch.sin(ang)
    lo, hi = x[:, :half], x[:, half:r]
    return torch.cat([lo * c - hi * s, hi * c + lo * s, x[:, r:]], dim=1)


def layer_forward(q, k, v, gate, cfg, ln_w=None, ln_b=None, tau_s=None, tau_b=None):
    """Differentiable forward.  q [B,Hq,T,d], k, v [B,Hkv,T,d], gate [B,Hkv,T] or None: float64 tensors
    (requires_grad as the caller likes).  cfg: an OracleConfig (oracle/kvm_oracle.py).  Returns
    (y [B,Hq,T,d], slots [B*Hkv, T] int, appended [B*Hkv, T] bool)."""
    B, Hq, Hkv, d, C, w, S, r = cfg.B, cfg.Hq, cfg.Hkv, cfg.d, cfg.C, cfg.w, cfg.S, cfg.r
    T = q.shape[2]
    G = Hq // Hkv
    L = w * C
    f64 = torch.float64
    ln_w = torch.ones((Hkv, d), dtype=f64) if ln_w is None else torch.as_tensor(ln_w, dtype=f64)
    ln_b = torch.zeros((Hkv, d), dtype=f64) if ln_b is None else torch.as_tensor(ln_b, dtype=f64)
    tau_s = torch.ones(Hq, dtype=f64) if tau_s is None else torch.as_tensor(tau_s, dtype=f64)
    tau_b = torch.ones(Hq, dtype=f64) if tau_b is None else torch.as_tensor(tau_b, dtype=f64)
    zero_r = torch.ones(d, dtype=f64)
    zero_r[:r] = 0.0
    y = torch.zeros((B, Hq, T, d), dtype=f64)
    ys = [[None] * Hq for _ in range(B)]
    slots = torch.full((B * Hkv, T), -1, dtype=torch.int64)
    appended = torch.zeros((B * Hkv, T), dtype=torch.bool)
    for b in range(B):
        for hk in range(Hkv):
            u = b * Hkv + hk
            gw, gb = ln_w[hk], ln_b[hk]
            k_rot = _rope(k[b, hk], 0, r, cfg.rope_base)
            q_rot = [_rope(q[b, hk * G + g], 0, r, cfg.rope_base) for g in range(G)]
            kbar = _layer_norm(k[b, hk] * zero_r, gw, gb, cfg.ln_eps)          # Eq. 1, every token
            gt = torch.ones(T, dtype=f64) if gate is None else gate[b, hk]
            sK = sV = rho = wsum = None                                         # state rows of this unit
            out = [[] for _ in range(G)]
            for c in range((T + C - 1) // C):
                s0, e = c * C, (c + 1) * C
                s1 = min(e, T)
                wb = max(0, e - L)
                # ---- readout: one softmax over [state rows ; window tokens wb .. u] (causal in the window)
                nq = s1 - s0
                pos_q = torch.arange(s0, s1)
                pos_k = torch.arange(wb, s1)
                vis = pos_k[None, :] <= pos_q[:, None]
                if sK is not None:
                    k_state = _layer_norm(sK, gw, gb, cfg.ln_eps)
                    if cfg.radius_on:
                        v_state = rho[:, None] * sV / torch.clamp(sV.norm(dim=1, keepdim=True), min=cfg.norm_eps)
                    else:
                        v_state = sV / wsum[:, None]
                for g in range(G):
                    hq = hk * G + g
                    lw = tau_b[hq] * (q_rot[g][s0:s1] @ k_rot[wb:s1].T) / math.sqrt(d)
                    lw = lw.masked_fill(~vis, float("-inf"))
                    if sK is not None:
                        ls = tau_s[hq] * (q_rot[g][s0:s1] @ k_state.T) / math.sqrt(d)
                        p = torch.softmax(torch.cat([ls, lw], dim=1), dim=1)
                        o = p[:, :sK.shape[0]] @ v_state + p[:, sK.shape[0]:] @ v[b, hk, wb:s1]
                    else:
                        o = torch.softmax(lw, dim=1) @ v[b, hk, wb:s1]
                    out[g].append(o)
                # ---- fold of the overflow block [wb, wb + C) once the block is complete
                if s1 < e or c < w - 1:
                    continue
                om = slice(wb, wb + C)
                kb, vb, gb_ = kbar[om], v[b, hk, om], gt[om]
                if sK is None:                                                   # state initialisation
                    sK, sV, rho, wsum = kb.clone(), vb.clone(), vb.norm(dim=1), torch.ones(C, dtype=f64)
                    slots[u, om] = torch.arange(C)
                    appended[u, om] = True
                    continue
                m = sK.shape[0]
                with torch.no_grad():                                            # integer decisions: routing held constant
                    sim_old = kb @ _layer_norm(sK, gw, gb, cfg.ln_eps).T
                    score = sim_old.max(dim=1).values
                    bud = _budget(cfg, e)
                    n_a = min(max(m, min(bud, m + C)) - m, C)
                    order = sorted(range(C), key=lambda j: (score[j].item(), j))
                    app = sorted(order[:n_a])
                    rest = [j for j in range(C) if j not in set(app)]
                if n_a > 0:
                    ia = torch.tensor(app)
                    sK = torch.cat([sK, kb[ia]]); sV = torch.cat([sV, vb[ia]])
                    rho = torch.cat([rho, vb[ia].norm(dim=1)]); wsum = torch.cat([wsum, torch.ones(n_a, dtype=f64)])
                    slots[u, wb + ia] = m + torch.arange(n_a)
                    appended[u, wb + ia] = True
                if rest:
                    ir = torch.tensor(rest)
                    with torch.no_grad():
                        sim = kb[ir] @ _layer_norm(sK, gw, gb, cfg.ln_eps).T     # against s_+ before any merge of this fold
                        sim[:, :S] = float("-inf")
                        pi = sim.argmax(dim=1)                                   # (torch: first maximum = lowest row)
                        # argmax tie rule made explicit: lowest row among exact maxima
                        mx = sim.max(dim=1, keepdim=True).values
                        pi = (sim == mx).float().argmax(dim=1)
                    sK = sK.index_add(0, pi, gb_[ir, None] * kb[ir])
                    sV = sV.index_add(0, pi, gb_[ir, None] * vb[ir])
                    wsum = wsum.index_add(0, pi, gb_[ir])
                    slots[u, wb + ir] = pi
            for g in range(G):
                ys[b][hk * G + g] = torch.cat(out[g], dim=0)
    y = torch.stack([torch.stack(row) for row in ys])
    return y, slots, appended


def layer_grads(q, k, v, gate, cfg, dy, **params):
    """Gradients of L = sum(y * dy) with respect to q, k, v (and gate when given), routing held constant.
    Inputs are array-likes (float64); returns dict(y, dq, dk, dv, dgate, slots, appended) of numpy arrays."""
    tq = torch.tensor(q, dtype=torch.float64, requires_grad=True)
    tk = torch.tensor(k, dtype=torch.float64, requires_grad=True)
    tv = torch.tensor(v, dtype=torch.float64, requires_grad=True)
    tg = None if gate is None else torch.tensor(gate, dtype=torch.float64, requires_grad=True)
    y, slots, appended = layer_forward(tq, tk, tv, tg, cfg, **params)
    loss = (y * torch.as_tensor(dy, dtype=torch.float64)).sum()
    wrt = [tq, tk, tv] + ([tg] if tg is not None else [])
    grads = torch.autograd.grad(loss, wrt, allow_unused=True)
    z = lambda gr, ref: (torch.zeros_like(ref) if gr is None else gr).numpy()
    return dict(y=y.detach().numpy(), dq=z(grads[0], tq), dk=z(grads[1], tk), dv=z(grads[2], tv),
                dgate=None if tg is None else z(grads[3], tg), slots=slots.numpy(), appended=appended.numpy())

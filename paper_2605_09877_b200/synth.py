"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds only input generation (random draws, scaling, mixtures, needles) and
the workload shape table; none of the KVM arithmetic lives here.  It is the one module
shared by the CUDA tests/benchmark and the CPU oracle's tests, so that both sides consume
exactly the same bf16-rounded values.

The paper's speed benchmark (Section 5) is shape-only (32 heads x 128 channels, bf16,
block 256, contexts up to 32768) and uses no dataset, so seeded tensors stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    Hq: int
    Hkv: int
    d: int
    T: int
    C: int
    growth: str          # "fixed" | "sqrt" | "unbounded" | "power" | "saturating"
    fixed_slots: int = 0
    sqrt_coeff: int = 16
    pow_num: int = 1     # "power": budget floor(sqrt_coeff * e^(pow_num/pow_den))
    pow_den: int = 2
    sat_half: int = 0    # "saturating": budget floor(fixed_slots * e / (e + sat_half))
    r: int = 0           # rope_dims
    w: int = 2           # n_bswa_chunks
    S: int = 1           # sink rows
    seed: int = 0
    kind: str = "normal"  # "normal" | "scaled_keys" | "mixture" | "needles"
    decode_steps: int = 0

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations of the build's baseline description, in order.
CONFIGS = {
    "cfg1": Workload("cfg1", 1, 1, 1, 64, 1024, 64, "fixed", fixed_slots=64, r=0, seed=0, kind="normal"),
    "cfg2": Workload("cfg2", 2, 16, 16, 128, 8192, 128, "fixed", fixed_slots=512, r=32, seed=1,
                     kind="scaled_keys"),
    "cfg3": Workload("cfg3", 1, 32, 32, 128, 32768, 256, "sqrt", r=0, seed=2, kind="mixture"),
    "cfg4": Workload("cfg4", 1, 8, 8, 128, 131072, 256, "sqrt", r=32, seed=3, kind="needles"),
    "cfg5": Workload("cfg5", 64, 32, 32, 128, 65536, 256, "sqrt", r=0, seed=4, kind="normal",
                     decode_steps=256),
}

N_CENTROIDS = 4096
MIX_SIGMA = 0.3
NEEDLE_FRACTION = 0.01
NEEDLE_SCALE = 4.0


def _gen(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, g, device="cpu"):
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def make_inputs(wl: Workload, device="cpu"):
    """Returns dict(q=[B,Hq,T,d], k=[B,Hkv,T,d], v=[B,Hkv,T,d]) as bf16 tensors on `device`.

    Draw order is q, k, v, then auxiliaries; values are drawn in fp32 and rounded once to
    bf16.  With device="cpu" the result is independent of the machine.
    """
    g = _gen(wl.seed, device)
    B, Hq, Hkv, T, d = wl.B, wl.Hq, wl.Hkv, wl.T, wl.d
    if wl.kind in ("normal", "scaled_keys", "needles"):
        q = _randn((B, Hq, T, d), g, device)
        k = _randn((B, Hkv, T, d), g, device)
        v = _randn((B, Hkv, T, d), g, device)
        if wl.kind == "scaled_keys":
            k = k / (d ** 0.5)
        if wl.kind == "needles":
            perm = torch.randperm(T, generator=g, device=device)
            n_needles = max(1, int(T * NEEDLE_FRACTION))
            pos = perm[:n_needles]
            k[:, :, pos, :] = k[:, :, pos, :] * NEEDLE_SCALE
            onehot = torch.zeros((n_needles, d), device=device)
            onehot[torch.arange(n_needles, device=device), pos % d] = NEEDLE_SCALE
            v[:, :, pos, :] = onehot
    elif wl.kind == "mixture":
        eq = _randn((B, Hq, T, d), g, device)
        ek = _randn((B, Hkv, T, d), g, device)
        ev = _randn((B, Hkv, T, d), g, device)
        ck = _randn((N_CENTROIDS, d), g, device)
        cv = _randn((N_CENTROIDS, d), g, device)
        zk = torch.randint(0, N_CENTROIDS, (B, Hkv, T), generator=g, device=device)
        zq = torch.randint(0, N_CENTROIDS, (B, Hq, T), generator=g, device=device)
        q = ck[zq] + MIX_SIGMA * eq
        k = ck[zk] + MIX_SIGMA * ek
        v = cv[zk] + MIX_SIGMA * ev
    else:
        raise ValueError(wl.kind)
    return dict(q=q.to(torch.bfloat16), k=k.to(torch.bfloat16), v=v.to(torch.bfloat16))


def make_segment(wl: Workload, seg_index: int, n_tokens: int, device="cuda", units=None):
    """N(0,1) bf16 q,k,v for one prefill segment of a large workload, generated on `device`
    from seed (wl.seed, seg_index).  `units` (list of (b, h)) restricts nothing here; callers
    slice the returned tensors.  Used where whole tensors do not fit (config 5)."""
    g = _gen(wl.seed * 1000003 + seg_index, device)
    q = _randn((wl.B, wl.Hq, n_tokens, wl.d), g, device).to(torch.bfloat16)
    k = _randn((wl.B, wl.Hkv, n_tokens, wl.d), g, device).to(torch.bfloat16)
    v = _randn((wl.B, wl.Hkv, n_tokens, wl.d), g, device).to(torch.bfloat16)
    return dict(q=q, k=k, v=v)


def make_decode_inputs(wl: Workload, step: int, device="cpu", seed_offset=1):
    """Fresh N(0,1) bf16 q [B,Hq,d], k,v [B,Hkv,d] for decode step `step`."""
    g = _gen((wl.seed + seed_offset) * 7919 + step, device)
    q = _randn((wl.B, wl.Hq, wl.d), g, device).to(torch.bfloat16)
    k = _randn((wl.B, wl.Hkv, wl.d), g, device).to(torch.bfloat16)
    v = _randn((wl.B, wl.Hkv, wl.d), g, device).to(torch.bfloat16)
    return dict(q=q, k=k, v=v)


def make_gate(wl: Workload, device="cpu"):
    """A positive merge gate g_t in (0, 2) shaped [B,Hkv,T] (fp32), for gate tests."""
    g = _gen(wl.seed + 99991, device)
    return (0.25 + 1.5 * torch.rand((wl.B, wl.Hkv, wl.T), generator=g, device=device)).float()


def make_layer_params(wl: Workload, trivial=True):
    """LN_s weight/bias [Hkv,d] and per-head temperatures [Hq] (fp32).  trivial=True gives
    the defaults (1, 0, 1, 1); otherwise seeded values around them."""
    if trivial:
        return dict(ln_w=None, ln_b=None, tau_s=None, tau_b=None)
    g = _gen(wl.seed + 424243)
    return dict(
        ln_w=(1.0 + 0.2 * _randn((wl.Hkv, wl.d), g)).float(),
        ln_b=(0.1 * _randn((wl.Hkv, wl.d), g)).float(),
        tau_s=(1.0 + 0.3 * torch.rand((wl.Hq,), generator=g)).float(),
        tau_b=(0.8 + 0.3 * torch.rand((wl.Hq,), generator=g)).float(),
    )

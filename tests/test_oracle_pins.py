"""Pins of the fp64 oracle against what the paper and the mathematics fix (CPU only).

Each test names the passage it pins.  A plausible mistake in oracle/kvm_oracle.c (dropped
term, wrong sign or index, transposed operand, off-by-one block) is meant to fail at least
one of these; tests/test_oracle_mutations.py shows that for a list of planted mistakes.
"""
import os

import numpy as np
import pytest

from oracle.kvm_oracle import KVMOracle, OracleConfig

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def causal_softmax_attention(q, k, v, scale):
    """Textbook causal softmax attention, one head: q,k,v [T,d]."""
    T = q.shape[0]
    out = np.zeros_like(v)
    for t in range(T):
        logits = (k[: t + 1] @ q[t]) * scale
        p = np.exp(logits - logits.max())
        p /= p.sum()
        out[t] = p @ v[: t + 1]
    return out


def standardise(x):
    return (x - x.mean(-1, keepdims=True)) / x.std(-1, keepdims=True)


def rng(seed):
    return np.random.default_rng(seed)


def read_golden(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([int(x) for x in line.split()])
    return rows


# ---------------------------------------------------------------------------------------
# state sizes (Table 1; budget rule of Section 3.2; "16 sqrt(N)", "KVM 256" of Section 4)

def run_sizes(C, T, growth, fixed_slots=0, d=4, **kw):
    r = rng(0)
    cfg = OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, growth=growth, fixed_slots=fixed_slots, **kw)
    o = KVMOracle(cfg)
    step = 4096
    for t0 in range(0, T, step):
        n = min(step, T - t0)
        o.forward(r.standard_normal((1, 1, n, d)), r.standard_normal((1, 1, n, d)),
                  r.standard_normal((1, 1, n, d)))
    return o


def test_state_sizes_sqrt_schedule_golden():
    gold = read_golden("state_sizes_sqrt.txt")
    T = 32768
    o = run_sizes(256, T, "sqrt", d=2)
    e, m, _ = o.fold_log()
    got = dict(zip(e.tolist(), m.tolist()))
    checked = 0
    for ee, mm in gold:
        if ee <= T:
            assert got[ee] == mm, (ee, got[ee], mm)
            checked += 1
    assert checked >= 5
    # O(sqrt N) growth: never more than 16*sqrt(e), never shrinking, first state one chunk long
    assert m[0] == 256 and np.all(np.diff(m) >= 0)
    assert np.all(m <= np.maximum(256, np.floor(16 * np.sqrt(e.astype(np.float64))) + 1e-9))
    assert o.rows == 2896 and o.nfolds == T // 256 - 1


def test_state_sizes_fixed_schedule_golden():
    gold = read_golden("state_sizes_fixed.txt")
    o = run_sizes(128, 2048, "fixed", fixed_slots=512)
    e, m, a = o.fold_log()
    for idx, ee, mm in gold:
        assert e[idx] == ee and m[idx] == mm
    assert a.tolist()[:5] == [128, 128, 128, 128, 0]
    # O(1) state: constant after saturation
    assert np.all(m[3:] == 512)


def test_fixed_budget_below_block_is_clamped():
    # the first state is always one chunk long, and the budget never removes rows
    o = run_sizes(64, 640, "fixed", fixed_slots=16)
    _, m, a = o.fold_log()
    assert np.all(m == 64) and a[0] == 64 and np.all(a[1:] == 0)


def test_unbounded_budget_appends_everything():
    o = run_sizes(16, 160, "unbounded", d=4)
    e, m, a = o.fold_log()
    assert np.all(a == 16)
    assert np.all(m == e - 16)  # every token older than the (w-1)-block window is a row


def test_power_schedule_with_exponent_one_half_is_the_sqrt_schedule():
    """The power-law budget floor(a e^(p/q)) at a = 16, p/q = 1/2 is the paper's 16 sqrt(N)."""
    a = run_sizes(64, 8192, "sqrt", d=2)
    b = run_sizes(64, 8192, "power", d=2, sqrt_coeff=16, pow_num=1, pow_den=2)
    assert a.fold_log()[1].tolist() == b.fold_log()[1].tolist() and a.rows == b.rows


@pytest.mark.parametrize("a,p,q", [(8, 2, 3), (3, 3, 4), (40, 1, 3), (1, 1, 1), (5, 1, 4)])
def test_power_schedule_sizes_are_the_exact_integer_floor(a, p, q):
    """Whenever the budget lies between the rows held and rows + C, the state has exactly B(e) rows,
    and B(e) = n is pinned by its definition in integers: n^q <= a^q e^p < (n+1)^q."""
    C = 32
    o = run_sizes(C, 4096, "power", d=2, sqrt_coeff=a, pow_num=p, pow_den=q)
    e, m, na = o.fold_log()
    assert m[0] == C and np.all(np.diff(m) >= 0)
    seen = 0
    prev = 0
    for ee, mm, aa in zip(e.tolist(), m.tolist(), na.tolist()):
        if prev and prev < mm < prev + C:      # neither clamp of the budget rule is active: rows = B(e)
            assert mm ** q <= a ** q * ee ** p < (mm + 1) ** q, (ee, mm)
            seen += 1
        elif prev and mm == prev + C:           # capped by the overflow block: the budget is at least that
            assert (prev + C) ** q <= a ** q * ee ** p
        elif prev:                              # nothing appended: the budget is at most the rows held
            assert a ** q * ee ** p < (mm + 1) ** q
        prev = mm
    assert seen >= 3 or (a, p, q) == (1, 1, 1)


def test_saturating_schedule_sizes():
    """B(e) = floor(M e / (e + h)): half of M at e = h, below M for ever, never shrinking."""
    M, h, C = 300, 2048, 32
    o = run_sizes(C, 16384, "saturating", fixed_slots=M, d=2, sat_half=h)
    e, m, _ = o.fold_log()
    got = dict(zip(e.tolist(), m.tolist()))
    assert got[h] == M // 2                                  # 150 rows when e = h
    assert np.all(np.diff(m) >= 0) and m[0] == C and m[-1] < M
    for ee, mm in got.items():
        if mm > C:                                           # past the first state the rows follow the budget
            assert mm * (ee + h) <= M * ee < (mm + 1) * (ee + h), (ee, mm)
    assert got[16384] == (M * 16384) // (16384 + h) == 266


# ---------------------------------------------------------------------------------------
# attention regions

@pytest.mark.parametrize("T,C,w", [(8, 4, 2), (7, 4, 2), (24, 8, 3), (5, 16, 2)])
def test_first_L_tokens_are_exact_causal_attention(T, C, w):
    """Section 3.2: the first L0 = min(T, L) tokens use exact causal attention."""
    d = 8
    r = rng(1)
    q, k, v = (r.standard_normal((1, 1, T, d)) for _ in range(3))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, w=w, growth="fixed", fixed_slots=C))
    y = o.forward(q, k, v)
    ref = causal_softmax_attention(q[0, 0], k[0, 0], v[0, 0], 1 / np.sqrt(d))
    np.testing.assert_allclose(y[0, 0], ref, atol=1e-12)


@pytest.mark.parametrize("T,C,w,d", [(48, 4, 2, 8), (96, 8, 2, 16), (60, 4, 3, 8)])
def test_never_compressing_limit_equals_full_causal_attention(T, C, w, d):
    """If the budget allows it every overflow token is appended (Section 3.1), so nothing is
    ever merged.  With no RoPE, identity LN_s, eps -> 0 and keys that are already
    standardised per row, LN_s(LN_s(k)) = k and rho * v / ||v|| = v, hence the layer must
    equal plain full causal softmax attention (brute force)."""
    r = rng(2)
    q = r.standard_normal((1, 1, T, d))
    k = standardise(r.standard_normal((1, 1, T, d)))
    v = r.standard_normal((1, 1, T, d)) * r.uniform(0.2, 3.0, (1, 1, T, 1))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, w=w, growth="unbounded", ln_eps=0.0))
    y = o.forward(q, k, v)
    ref = causal_softmax_attention(q[0, 0], k[0, 0], v[0, 0], 1 / np.sqrt(d))
    np.testing.assert_allclose(y[0, 0], ref, atol=1e-10)
    assert o.rows == (T // C - (w - 1)) * C


def test_state_rows_are_position_free_but_window_is_rotated():
    """Section 3.1 "Positional Encoding": RoPE on q and window keys, rotary channels zeroed in
    the state.  Closed form with d = r = 2 inside the window: q_t . k_s = a^2 cos(t - s) for
    q = k = (a, 0), because channel pair (0, 1) rotates by t * base^0 = t radians."""
    T, C, a = 12, 8, 1.3
    q = np.zeros((1, 1, T, 2)); q[..., 0] = a
    k = q.copy()
    v = rng(3).standard_normal((1, 1, T, 2))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=2, C=C, r=2, growth="fixed", fixed_slots=C))
    y = o.forward(q, k, v)
    for t in range(T):
        logits = np.array([a * a * np.cos(t - s) / np.sqrt(2) for s in range(t + 1)])
        p = np.exp(logits - logits.max()); p /= p.sum()
        np.testing.assert_allclose(y[0, 0, t], p @ v[0, 0, : t + 1], atol=1e-12)


def test_rope_second_pair_frequency_and_direction():
    """d = r = 4: pairs (0,2) and (1,3); pair 1 turns by t * base^(-2/4) = t / 100 radians.
    q = e_1, k = e_3 gives q_t . k_s = sin((t - s)/100); q = k = e_1 gives cos((t - s)/100)."""
    T, C = 10, 16
    v = rng(4).standard_normal((1, 1, T, 4))
    for qc, kc, fn in ((1, 3, np.sin), (1, 1, np.cos), (3, 1, lambda x: -np.sin(x))):
        q = np.zeros((1, 1, T, 4)); q[..., qc] = 5.0
        k = np.zeros((1, 1, T, 4)); k[..., kc] = 5.0
        o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=4, C=C, r=4, growth="fixed", fixed_slots=C))
        y = o.forward(q, k, v)
        for t in range(T):
            logits = np.array([25.0 * fn((t - s) / 100.0) / 2.0 for s in range(t + 1)])
            p = np.exp(logits - logits.max()); p /= p.sum()
            np.testing.assert_allclose(y[0, 0, t], p @ v[0, 0, : t + 1], atol=1e-12)


def test_partial_rope_leaves_nope_channels_alone():
    """With r < d only the first r channels turn: a query/key pair living in the NoPE
    channels has a position-independent logit, so inside the window the output equals
    causal attention computed on the raw vectors."""
    T, C, d, r_ = 14, 8, 8, 4
    g = rng(5)
    q = np.zeros((1, 1, T, d)); k = np.zeros((1, 1, T, d))
    q[..., r_:] = g.standard_normal((1, 1, T, d - r_))
    k[..., r_:] = g.standard_normal((1, 1, T, d - r_))
    v = g.standard_normal((1, 1, T, d))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, r=r_, growth="fixed", fixed_slots=C))
    y = o.forward(q, k, v)
    ref = causal_softmax_attention(q[0, 0], k[0, 0], v[0, 0], 1 / np.sqrt(d))
    np.testing.assert_allclose(y[0, 0], ref, atol=1e-12)


# ---------------------------------------------------------------------------------------
# recurrence invariants

def run_random(T=320, C=16, d=16, growth="fixed", fixed_slots=24, r_=0, gate=False, seed=7, S=1,
               B=1, H=2, affine=False, w=2, ln_eps=1e-5):
    g = rng(seed)
    q = g.standard_normal((B, H, T, d)); k = g.standard_normal((B, H, T, d))
    v = g.standard_normal((B, H, T, d)) * g.uniform(0.3, 2.0, (B, H, T, 1))
    gt = g.uniform(0.2, 1.9, (B, H, T)) if gate else None
    kw = {}
    if affine:
        kw = dict(ln_w=1 + 0.3 * g.standard_normal((H, d)), ln_b=0.2 * g.standard_normal((H, d)),
                  tau_s=g.uniform(0.7, 1.4, H), tau_b=g.uniform(0.7, 1.4, H))
    cfg = OracleConfig(B=B, Hq=H, Hkv=H, d=d, C=C, w=w, S=S, r=r_, growth=growth,
                       fixed_slots=fixed_slots, ln_eps=ln_eps)
    o = KVMOracle(cfg, **kw)
    y = o.forward(q, k, v, gt)
    return o, y, (q, k, v, gt)


@pytest.mark.parametrize("gate,growth,r_", [(False, "fixed", 0), (True, "fixed", 4), (True, "sqrt", 0)])
def test_rows_are_weighted_sums_of_their_members(gate, growth, r_):
    """Merge update and Section 3.2's closing remark: each row is the creator's memory key /
    value plus the gate-weighted members; means = sums / weight; counts by-product."""
    o, _, (q, k, v, gt) = run_random(gate=gate, growth=growth, r_=r_, affine=True)
    st = o.export()
    slot, app, _ = o.assignments()
    kbar = o.memory_keys()
    U, T = slot.shape
    vv = v.reshape(U, T, -1)
    gg = np.ones((U, T)) if gt is None else gt.reshape(U, T)
    for u in range(U):
        m = o.rows
        sk = np.zeros((m, kbar.shape[-1])); sv = np.zeros_like(sk); w = np.zeros(m); n = np.zeros(m, int)
        for t in range(T):
            i = slot[u, t]
            if i < 0:
                continue
            wt = 1.0 if app[u, t] else gg[u, t]
            sk[i] += wt * kbar[u, t]; sv[i] += wt * vv[u, t]; w[i] += wt; n[i] += 1
        np.testing.assert_allclose(st["sum_k"][u], sk, atol=1e-10)
        np.testing.assert_allclose(st["sum_v"][u], sv, atol=1e-10)
        np.testing.assert_allclose(st["weight"][u], w, atol=1e-12)
        assert np.array_equal(st["count"][u], n)
        # every row was created exactly once, by an appended token
        creators = np.sort(slot[u][app[u] == 1])
        assert np.array_equal(creators, np.arange(m))
    # all tokens older than the window have been folded, the rest not
    n_folded = (o.nfolds) * o.cfg.C
    assert np.all(slot[:, :n_folded] >= 0) and np.all(slot[:, n_folded:] == -1)


def test_readout_key_is_layernorm_of_the_mean():
    """LN_s(sum) == LN_s(weighted mean) (Section 3.2, last paragraph): with eps = 0 and identity
    affine the readout key is the standardised mean vector."""
    o, _, _ = run_random(gate=True, ln_eps=0.0)
    st = o.export()
    khat, _ = o.readout()
    mean = st["sum_k"] / st["weight"][..., None]
    np.testing.assert_allclose(khat, standardise(mean), atol=1e-9)


def test_value_radius_is_preserved():
    """Value-radius preservation: ||s^V_hat_i|| equals the norm of the value that created row i,
    whatever was merged afterwards, and the direction is that of the running sum."""
    o, _, (q, k, v, gt) = run_random(gate=True, T=480)
    st = o.export()
    slot, app, _ = o.assignments()
    _, vhat = o.readout()
    U, T = slot.shape
    vv = v.reshape(U, T, -1)
    assert st["count"].max() > 3
    for u in range(U):
        for t in np.nonzero(app[u])[0]:
            i = slot[u, t]
            assert abs(np.linalg.norm(vhat[u, i]) - np.linalg.norm(vv[u, t])) < 1e-12
            assert abs(st["radius"][u, i] - np.linalg.norm(vv[u, t])) < 1e-13
        cosang = np.sum(vhat[u] * st["sum_v"][u], -1) / (
            np.linalg.norm(vhat[u], axis=-1) * np.linalg.norm(st["sum_v"][u], axis=-1))
        np.testing.assert_allclose(cosang, 1.0, atol=1e-12)


def test_sink_row_is_never_a_merge_target():
    o, _, (q, k, v, gt) = run_random(T=640)
    st = o.export()
    slot, app, _ = o.assignments()
    kbar = o.memory_keys()
    assert np.all(st["count"][:, 0] == 1)
    np.testing.assert_array_equal(st["sum_k"][:, 0], kbar[:, 0])
    merged = (slot >= 0) & (app == 0)
    assert merged.sum() > 0 and np.all(slot[merged] >= 1)
    # ablation switch S = 0: row 0 becomes eligible and does get used
    o0, _, _ = run_random(T=640, S=0)
    slot0, app0, _ = o0.assignments()
    assert np.any(slot0[(slot0 >= 0) & (app0 == 0)] == 0)


def test_routing_matches_brute_force_on_the_last_fold():
    """pi(j) = arg max_{i >= S} kbar_j . LN_s(s^K_i) for the overflow block [e - L, e - L + C),
    brute force from the state as it stood before that fold."""
    T, C, d, H = 160, 16, 16, 2
    g = rng(7)
    q, k, v = (g.standard_normal((1, H, T, d)) for _ in range(3))
    params = dict(ln_w=1 + 0.3 * g.standard_normal((H, d)), ln_b=0.2 * g.standard_normal((H, d)))
    cfg = OracleConfig(B=1, Hq=H, Hkv=H, d=d, C=C, growth="fixed", fixed_slots=24)
    full = KVMOracle(cfg, **params); prev = KVMOracle(cfg, **params)
    full.forward(q, k, v); prev.forward(q[:, :, : T - C], k[:, :, : T - C], v[:, :, : T - C])
    khat_prev, _ = prev.readout()
    kbar = full.memory_keys()
    slot, app, margin = full.assignments()
    b = T - 2 * C
    assert full.rows == prev.rows == 24  # fixed budget already saturated: merge only
    for u in range(full.U):
        for j in range(b, b + C):
            sims = khat_prev[u] @ kbar[u, j]
            sims[: cfg.S] = -np.inf
            assert slot[u, j] == int(np.argmax(sims)) and app[u, j] == 0
            top2 = np.sort(sims)[-2:]
            assert abs(margin[u, j] - (top2[1] - top2[0])) < 1e-12


def test_append_picks_least_redundant_tokens_brute_force():
    """A_e = the n_append overflow tokens with the smallest s_j = max_i kbar_j . LN_s(s^K_i)
    (sinks included); rows laid down in ascending token order; the rest merges into s_+."""
    T, C = 144, 16
    g = rng(21)
    q, k, v = (g.standard_normal((1, 1, T, 16)) for _ in range(3))
    cfg = OracleConfig(B=1, Hq=1, Hkv=1, d=16, C=C, growth="sqrt", sqrt_coeff=3)
    full = KVMOracle(cfg); prev = KVMOracle(cfg)
    full.forward(q, k, v); prev.forward(q[:, :, : T - C], k[:, :, : T - C], v[:, :, : T - C])
    n_a = full.rows - prev.rows
    assert 0 < n_a < C
    khat_prev, _ = prev.readout()
    kbar = full.memory_keys()[0]
    slot, app, _ = full.assignments()
    b = T - 2 * C
    scores = np.array([np.max(khat_prev[0] @ kbar[j]) for j in range(b, b + C)])
    chosen = np.sort(np.argsort(scores, kind="stable")[:n_a])
    assert np.array_equal(np.nonzero(app[0, b:b + C])[0], chosen)
    assert np.array_equal(slot[0, b + chosen], prev.rows + np.arange(n_a))
    # the remaining tokens route against old rows AND the rows appended in the same fold
    khat_full_rows = np.concatenate([khat_prev[0], standardise_ln(kbar[b + chosen], 1e-5)])
    for j in range(C):
        if j in chosen:
            continue
        sims = khat_full_rows @ kbar[b + j]
        sims[:1] = -np.inf
        assert slot[0, b + j] == int(np.argmax(sims))


def standardise_ln(x, eps):
    mu = x.mean(-1, keepdims=True)
    var = ((x - mu) ** 2).mean(-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps)


def test_constructed_ties_go_to_the_lowest_eligible_row():
    """All keys equal -> every similarity ties -> arg max takes the lowest row i >= S."""
    T, C, d = 64, 8, 8
    k = np.ones((1, 1, T, d)) * 0.5
    q = rng(30).standard_normal((1, 1, T, d)); v = rng(31).standard_normal((1, 1, T, d))
    for S in (0, 1, 3):
        o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, S=S, growth="fixed", fixed_slots=C))
        o.forward(q, k, v)
        slot, app, _ = o.assignments()
        merged = (slot[0] >= 0) & (app[0] == 0)
        assert merged.sum() == T - 2 * C  # every folded token after the first block merged
        assert np.all(slot[0][merged] == S)


def test_duplicates_are_not_appended_when_a_novel_token_exists():
    """Append picks the least redundant token: a block of copies of existing rows plus one
    new direction appends the new direction (budget grows by exactly one row)."""
    C, d = 8, 16
    g = rng(40)
    base = g.standard_normal((C, d))
    novel = g.standard_normal(d) * 3
    blk1 = base[g.permutation(C)].copy()
    jn = 5
    blk1[jn] = novel
    k = np.concatenate([base, blk1, g.standard_normal((2 * C, d))])[None, None]
    T = k.shape[2]
    q = g.standard_normal((1, 1, T, d)); v = g.standard_normal((1, 1, T, d))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, growth="fixed", fixed_slots=C + 1))
    o.forward(q[:, :, : 3 * C], k[:, :, : 3 * C], v[:, :, : 3 * C])
    slot, app, _ = o.assignments()
    assert o.rows == C + 1
    assert np.array_equal(np.nonzero(app[0, C:2 * C])[0], [jn])
    assert slot[0, C + jn] == C
    # each copy merged into the row holding its original (never the sink row 0: the copy of
    # row 0 goes to its next best row)
    for j in range(C):
        if j == jn:
            continue
        src = int(np.argmin(np.abs(base - blk1[j]).sum(-1)))
        if src != 0:
            assert slot[0, C + j] == src


# ---------------------------------------------------------------------------------------
# equivalences

@pytest.mark.parametrize("growth", ["fixed", "sqrt"])
def test_token_at_a_time_equals_chunked(growth):
    """The mask of Section 3.2 is per query, so decoding one token at a time, or prefilling in
    ragged segments, must give the same outputs and the same state as one prefill."""
    o1, y1, (q, k, v, gt) = run_random(T=200, growth=growth, gate=True, r_=4, affine=False)
    cfg = o1.cfg
    o2 = KVMOracle(cfg); o3 = KVMOracle(cfg)
    T = q.shape[2]
    y2 = np.concatenate([o2.forward(q[:, :, t:t + 1], k[:, :, t:t + 1], v[:, :, t:t + 1], gt[:, :, t:t + 1])
                         for t in range(T)], axis=2)
    cuts = [0, 5, 37, 38, 96, 150, T]
    y3 = np.concatenate([o3.forward(q[:, :, a:b], k[:, :, a:b], v[:, :, a:b], gt[:, :, a:b])
                         for a, b in zip(cuts[:-1], cuts[1:])], axis=2)
    np.testing.assert_array_equal(y1, y2)
    np.testing.assert_array_equal(y1, y3)
    for a, b in ((o1, o2), (o1, o3)):
        sa, sb = a.export(), b.export()
        for key in sa:
            np.testing.assert_array_equal(sa[key], sb[key])


def pseudocode_order_reference(q, k, v, C, n_chunks_window, sink_len, eps=1e-5, eps_norm=1e-12):
    """Independent numpy restatement in the ORDER of Appendix B (merge-only variant): per chunk,
    first merge the block that fell off in the previous iteration via a one-hot matrix product,
    then attend over [state ; window].  One head, no RoPE, identity LN affine, gate 1."""
    T, d = q.shape
    L = n_chunks_window * C
    ln = lambda x: (x - x.mean(-1, keepdims=True)) / np.sqrt(((x - x.mean(-1, keepdims=True)) ** 2).mean(-1, keepdims=True) + eps)
    s_k = s_v = s_len = None
    out = np.zeros_like(v)
    for c in range(T // C):
        bswa_end = (c + 1) * C
        bswa_begin = max(0, bswa_end - L)
        if bswa_begin >= C:  # a block fell off before this chunk
            o_k = ln(k[bswa_begin - C:bswa_begin]); o_v = v[bswa_begin - C:bswa_begin]
            if s_k is None:
                s_k, s_v, s_len = o_k.copy(), o_v.copy(), np.linalg.norm(o_v, axis=-1, keepdims=True)
            else:
                logits = o_k @ ln(s_k).T
                logits[:, :sink_len] = -np.inf
                onehot = np.zeros_like(logits)
                onehot[np.arange(C), logits.argmax(-1)] = 1.0
                s_k = s_k + onehot.T @ o_k
                s_v = s_v + onehot.T @ o_v
        a_q = q[bswa_end - C:bswa_end]
        a_k = k[bswa_begin:bswa_end]; a_v = v[bswa_begin:bswa_end]
        n_state = 0
        if s_k is not None:
            sv = s_v / np.maximum(np.linalg.norm(s_v, axis=-1, keepdims=True), eps_norm) * s_len
            a_k = np.concatenate([ln(s_k), a_k]); a_v = np.concatenate([sv, a_v]); n_state = len(s_k)
        logits = a_q @ a_k.T / np.sqrt(d)
        qpos = np.arange(bswa_end - C, bswa_end)[:, None]
        kpos = np.concatenate([np.full(n_state, -1), np.arange(bswa_begin, bswa_end)])[None]
        logits = np.where(kpos <= qpos, logits, -np.inf)
        p = np.exp(logits - logits.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
        out[bswa_end - C:bswa_end] = p @ a_v
    return out, s_k, s_v


@pytest.mark.parametrize("w", [2, 3])
def test_pseudocode_order_gives_the_same_outputs(w):
    """Appendix B processes "state first, lagging" and says this is equivalent to the main
    text's order; in the fixed-size regime (budget = C, merge only) both must agree."""
    T, C, d = 192, 16, 16
    g = rng(50)
    q, k, v = (g.standard_normal((T, d)) for _ in range(3))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, w=w, growth="fixed", fixed_slots=C))
    y = o.forward(q[None, None], k[None, None], v[None, None])
    ref, s_k, s_v = pseudocode_order_reference(q, k, v, C, w, 1)
    np.testing.assert_allclose(y[0, 0], ref, atol=1e-10)
    # the eager oracle has folded one block more than the lagging loop has
    o2 = KVMOracle(o.cfg)
    o2.forward(q[None, None, : T - C], k[None, None, : T - C], v[None, None, : T - C])
    np.testing.assert_allclose(o2.export()["sum_k"][0], s_k, atol=1e-10)
    np.testing.assert_allclose(o2.export()["sum_v"][0], s_v, atol=1e-10)


def test_temperatures_scale_their_own_region_only():
    """K^A = [tau_state * s^K_hat ; tau_bswa * k]: equal temperatures are the same as scaling
    the query; tau_state alone leaves the first L tokens (no state yet) untouched."""
    o1, y1, (q, k, v, _) = run_random(T=128)
    cfg = o1.cfg
    tau = np.array([1.7, 0.6])
    y2 = KVMOracle(cfg, tau_s=tau, tau_b=tau).forward(q, k, v)
    y3 = KVMOracle(cfg).forward(q * tau[None, :, None, None], k, v)
    np.testing.assert_allclose(y2, y3, atol=1e-12)
    y4 = KVMOracle(cfg, tau_s=tau).forward(q, k, v)
    L = cfg.w * cfg.C
    np.testing.assert_array_equal(y4[:, :, :L], y1[:, :, :L])
    assert np.abs(y4[:, :, L:] - y1[:, :, L:]).max() > 1e-3
    # the fold does not depend on the temperatures
    o5 = KVMOracle(cfg, tau_s=tau, tau_b=1 / tau)
    o5.forward(q, k, v)
    np.testing.assert_array_equal(o5.assignments()[0], o1.assignments()[0])


def test_grouped_queries_share_one_state():
    g = rng(60)
    T, C, d = 96, 8, 8
    q = g.standard_normal((1, 4, T, d)); k = g.standard_normal((1, 2, T, d)); v = g.standard_normal((1, 2, T, d))
    og = KVMOracle(OracleConfig(B=1, Hq=4, Hkv=2, d=d, C=C, growth="fixed", fixed_slots=12))
    yg = og.forward(q, k, v)
    of = KVMOracle(OracleConfig(B=1, Hq=4, Hkv=4, d=d, C=C, growth="fixed", fixed_slots=12))
    yf = of.forward(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1))
    np.testing.assert_array_equal(yg, yf)


def test_gate_of_one_is_no_gate_and_units_are_independent():
    o1, y1, (q, k, v, _) = run_random(T=160, B=2, H=2)
    y2 = KVMOracle(o1.cfg).forward(q, k, v, np.ones(q.shape[:3]))
    np.testing.assert_array_equal(y1, y2)
    # unit (1, 0) alone gives the same numbers
    cfg1 = OracleConfig(**{**o1.cfg.__dict__, "B": 1, "Hq": 1, "Hkv": 1})
    y3 = KVMOracle(cfg1).forward(q[1:2, 0:1], k[1:2, 0:1], v[1:2, 0:1])
    np.testing.assert_array_equal(y1[1:2, 0:1], y3)


def test_radius_switch_off_reads_out_the_mean_value():
    o, _, (q, k, v, gt) = run_random(gate=True)
    o2 = KVMOracle(OracleConfig(**{**o.cfg.__dict__, "radius_on": False}))
    o2.forward(q, k, v, gt)
    st = o2.export()
    _, vhat = o2.readout()
    np.testing.assert_allclose(vhat, st["sum_v"] / st["weight"][..., None], atol=1e-13)


# ---------------------------------------------------------------------------------------
# pins added for planted mistakes that the tests above did not see

def test_rope_frequency_exponent_runs_over_the_rotary_width():
    """Partial RoPE keeps base 10000 "even when applying across only 64 of 128 channels"
    (Appendix D): with d = 8, r = 4 the second pair (1, 3) turns by t * base^(-2/4) = t/100."""
    T, C, d = 10, 16, 8
    v = rng(70).standard_normal((1, 1, T, d))
    q = np.zeros((1, 1, T, d)); q[..., 1] = 5.0
    k = np.zeros((1, 1, T, d)); k[..., 1] = 5.0
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, r=4, growth="fixed", fixed_slots=C))
    y = o.forward(q, k, v)
    for t in range(T):
        logits = np.array([25.0 * np.cos((t - s) / 100.0) / np.sqrt(d) for s in range(t + 1)])
        p = np.exp(logits - logits.max()); p /= p.sum()
        np.testing.assert_allclose(y[0, 0, t], p @ v[0, 0, : t + 1], atol=1e-12)


def test_state_does_not_see_the_rotary_channels():
    """Eq. 1: the rotary subspace of a key is zeroed before it becomes a memory key, so the
    state rows and the routing are unchanged when only those channels of k change."""
    oa, _, (q, k, v, gt) = run_random(T=160, r_=4, gate=True)
    k2 = k.copy()
    k2[..., :4] = rng(71).standard_normal(k2[..., :4].shape)
    ob = KVMOracle(oa.cfg)
    ob.forward(q, k2, v, gt)
    sa, sb = oa.export(), ob.export()
    for key in sa:
        np.testing.assert_array_equal(sa[key], sb[key])
    np.testing.assert_array_equal(oa.assignments()[0], ob.assignments()[0])


def test_layernorm_affine_closed_forms():
    """LN_s is a LayerNorm WITH bias (Section 3.2 "KVM weight preparation").  A constant key
    normalises to beta; a +-1 alternating key has mean 0 and variance 1, so with eps = 0 it
    normalises to gamma * x + beta.  Rows are weight * that vector."""
    T, C, d, H = 48, 8, 8, 2
    g = rng(72)
    gamma = 1 + 0.3 * g.standard_normal((H, d)); beta = 0.2 * g.standard_normal((H, d))
    q = g.standard_normal((1, H, T, d)); v = g.standard_normal((1, H, T, d))
    cfg = OracleConfig(B=1, Hq=H, Hkv=H, d=d, C=C, growth="fixed", fixed_slots=C, ln_eps=0.0)
    pattern = np.where(np.arange(d) % 2 == 0, 1.0, -1.0)
    for x, expect in ((np.full(d, 0.7), beta), (3.0 * pattern, gamma * pattern + beta)):
        k = np.broadcast_to(x, (1, H, T, d)).copy()
        if np.ptp(x) == 0:
            cfg_x = OracleConfig(**{**cfg.__dict__, "ln_eps": 1e-5})  # constant vector: var = 0
        else:
            cfg_x = cfg
        o = KVMOracle(cfg_x, ln_w=gamma, ln_b=beta)
        o.forward(q, k, v)
        st = o.export()
        np.testing.assert_allclose(st["sum_k"], st["weight"][..., None] * expect[:, None, :], atol=1e-12)


def test_append_score_counts_the_sink_row():
    """s_j is a max over ALL rows (sinks included): a copy of the sink's key is fully
    redundant and must not be appended ahead of a half-new token."""
    C, d = 8, 32
    g = rng(73)
    base = g.standard_normal((C, d))
    blk1 = base.copy()
    j_half = 5
    blk1[j_half] = base[j_half] + 0.6 * g.standard_normal(d)   # similar to row 5, not identical
    k = np.concatenate([base, blk1, g.standard_normal((C, d))])[None, None]
    T = k.shape[2]
    q = g.standard_normal((1, 1, T, d)); v = g.standard_normal((1, 1, T, d))
    o = KVMOracle(OracleConfig(B=1, Hq=1, Hkv=1, d=d, C=C, growth="fixed", fixed_slots=C + 1))
    o.forward(q, k, v)
    slot, app, _ = o.assignments()
    assert np.array_equal(np.nonzero(app[0, C:2 * C])[0], [j_half])
    # the copy of the sink cannot merge into the sink; it goes to another row
    assert slot[0, C + 0] >= 1 and app[0, C + 0] == 0


def test_attend_rows_definition_closed_forms_and_library_routine():
    """oracle/attend_rows.py (single-query attention over given rows): equal keys give the plain mean of the
    values, a dominant key gives its value, and torch's scaled_dot_product_attention (a library routine,
    fp64) gives the same numbers; `scale` multiplies the logits (a transposed or unscaled product fails)."""
    import torch
    from oracle.attend_rows import attend_rows
    rng = np.random.default_rng(5)
    H, n, d = 3, 17, 8
    q = rng.standard_normal((H, d)); k = rng.standard_normal((H, n, d)); v = rng.standard_normal((H, n, d))
    same = np.repeat(k[:, :1], n, axis=1)
    assert np.allclose(attend_rows(q, same, v, 0.7), v.mean(axis=1), atol=1e-13)
    big = k.copy(); big[:, 5] = 50.0 * q
    assert np.allclose(attend_rows(q, big, v, 1.0), v[:, 5], atol=1e-9)
    ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q)[:, None], torch.from_numpy(k), torch.from_numpy(v),
                                                           scale=0.37)[:, 0].numpy()
    assert np.allclose(attend_rows(q, k, v, 0.37), ref, atol=1e-13)
    # two rows, by hand: logits (scale * q.k) = (ln 3, 0) -> weights (3/4, 1/4)
    q1 = np.array([[1.0, 0.0]]); k1 = np.array([[[np.log(3.0) / 2.0, 9.0], [0.0, -4.0]]]); v1 = np.array([[[4.0, 0.0], [0.0, 8.0]]])
    assert np.allclose(attend_rows(q1, k1, v1, 2.0), [[3.0, 2.0]], atol=1e-13)

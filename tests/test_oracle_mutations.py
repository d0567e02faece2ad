"""Shows that the pins in test_oracle_pins.py bite: each planted mistake (a one-line textual
change to a temporary COPY of oracle/kvm_oracle.c, compiled to a temporary library) must make
the pin suite fail.  Everything runs on the CPU; the committed oracle is never modified."""
import os
import subprocess
import sys
import tempfile
from concurrent.futures import ThreadPoolExecutor

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SRC = os.path.join(ROOT, "oracle", "kvm_oracle.c")

MUTATIONS = {
    "rope_sign": ("out[i] = a * cs - b * sn;", "out[i] = a * cs + b * sn;"),
    "rope_frequency_over_d": ("-2.0 * (double)i / (double)r", "-2.0 * (double)i / (double)d"),
    "rope_pairs_adjacent": ("double a = x[i], b = x[i + h];", "double a = x[i], b = x[(i + 1) % d];"),
    "memory_key_keeps_rotary": ("z[i] = (i < o->c.r) ? 0.0 : k[i];", "z[i] = k[i];"),
    "ln_unbiased_variance": ("var /= d;", "var /= (d - 1);"),
    "ln_drops_bias": ("((x[i] - mean) * rstd) + beta[i];", "((x[i] - mean) * rstd);"),
    "budget_cap_off_by_one": ("(Bud < m + C) ? Bud : m + C;", "(Bud < m + C - 1) ? Bud : m + C - 1;"),
    "append_picks_most_redundant": ("score[j] < score[pick]", "score[j] > score[pick]"),
    "append_score_skips_sinks": ("for (int64_t i = 0; i < m; ++i) {\n      double s = dot(kbar",
                                 "for (int64_t i = c->S; i < m; ++i) {\n      double s = dot(kbar"),
    "sinks_are_merge_targets": ("for (int64_t i = c->S; i < mp; ++i) {", "for (int64_t i = 0; i < mp; ++i) {"),
    "merge_ignores_new_rows": ("for (int64_t i = c->S; i < mp; ++i) {", "for (int64_t i = c->S; i < m; ++i) {"),
    "argmax_takes_last_of_ties": ("if (s > best) { second = best;", "if (s >= best) { second = best;"),
    "value_not_gated": ("u->sumV[i * d + x] += g * v[x];", "u->sumV[i * d + x] += v[x];"),
    "key_not_gated": ("u->sumK[i * d + x] += g * kbar[(size_t)j * d + x];",
                      "u->sumK[i * d + x] += kbar[(size_t)j * d + x];"),
    "radius_from_key": ("u->rho[row] = sqrt(dot(v, v, d));", "u->rho[row] = sqrt(dot(kbar, kbar, d));"),
    "radius_not_applied": ("vhat[i * d + x] = u->rho[i] * sv[x] / den;", "vhat[i * d + x] = sv[x] / den;"),
    "window_one_block_short": ("const int64_t b = (e - L > 0) ? e - L : 0;",
                               "const int64_t b = (e - L + C > 0) ? e - L + C : 0;"),
    "fold_one_chunk_late": ("(t1 == e) && (cidx >= c->w - 1);", "(t1 == e) && (cidx >= c->w);"),
    "window_excludes_self": ("const int64_t nwin = t - b + 1;", "const int64_t nwin = t - b;"),
    "scale_one_over_d": ("const double inv = 1.0 / sqrt((double)d);", "const double inv = 1.0 / (double)d;"),
    "state_temperature_on_window": ("s += q_rot[x] * (tb * kj[x]);", "s += q_rot[x] * (ts * kj[x]);"),
    "state_keys_not_normalised": ("layer_norm(u->sumK + i * d, o->ln_w + (size_t)hk * d, o->ln_b + (size_t)hk * d, o->c.ln_eps, d,\n               khat + i * d);",
                                  "memcpy(khat + i * d, u->sumK + i * d, sizeof(double) * d);"),
    "softmax_not_normalised": ("double p = logit[m + j] / den;", "double p = logit[m + j];"),
}


def _run(name):
    old, new = MUTATIONS[name]
    src = open(SRC).read()
    assert src.count(old) >= 1, f"mutation {name}: pattern not found"
    tmp = tempfile.mkdtemp(prefix="kvm_mut_")
    c = os.path.join(tmp, "mut.c")
    so = os.path.join(tmp, "libmut.so")
    with open(c, "w") as f:
        f.write(src.replace(old, new, 1))
    subprocess.run(["gcc", "-O1", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", so, c, "-lm"], check=True)
    env = dict(os.environ, KVM_ORACLE_LIB=so, OMP_NUM_THREADS="1")
    p = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-p", "no:cacheprovider",
                        os.path.join(ROOT, "tests", "test_oracle_pins.py")],
                       cwd=ROOT, env=env, capture_output=True, text=True)
    return name, p.returncode, p.stdout[-400:]


def test_every_planted_mistake_is_caught():
    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as ex:
        results = list(ex.map(_run, MUTATIONS))
    missed = [n for n, rc, _ in results if rc == 0]
    assert not missed, f"pins did not catch: {missed}"


def test_unmutated_copy_passes():
    """Control: the same harness with an identity 'mutation' passes."""
    MUTATIONS["__identity__"] = ("var /= d;", "var /= d;")
    try:
        name, rc, out = _run("__identity__")
    finally:
        del MUTATIONS["__identity__"]
    assert rc == 0, out

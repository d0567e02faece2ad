"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol that
include/kvm.h declares, and its host-side arithmetic (capacity planning, argument validation)
behaves.  No compute call is made without a GPU."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def kvm():
    from paper_2605_09877_b200 import build
    build.build()
    from paper_2605_09877_b200 import kvm as mod
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "kvm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvm_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(kvm):
    names = declared_symbols()
    assert len(names) >= 12
    raw = C.CDLL(kvm.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
    assert sorted(kvm.EXPORTS) == names


def test_status_strings(kvm):
    assert kvm.lib.kvm_status_string(0) == b"ok"
    assert b"capacity" in kvm.lib.kvm_status_string(6)


def test_plan_capacity_matches_the_budget_rule_closed_forms(kvm):
    g = kvm.growth("sqrt")
    for e, m in ((512, 256), (768, 443), (1024, 512), (8192, 1448), (32768, 2896), (65536, 4096), (131072, 5792)):
        assert kvm.kvm_plan_capacity(256, 2, g, e) == m
    assert kvm.kvm_plan_capacity(256, 2, g, 511) == 0
    gf = kvm.growth("fixed", fixed_slots=512)
    assert [kvm.kvm_plan_capacity(128, 2, gf, e) for e in (255, 256, 384, 512, 640, 8192)] == [0, 128, 256, 384, 512, 512]
    assert kvm.kvm_plan_capacity(64, 2, kvm.growth("fixed", fixed_slots=16), 1024) == 64
    assert kvm.kvm_plan_capacity(16, 2, kvm.growth("unbounded"), 160) == 144
    assert kvm.kvm_plan_capacity(0, 2, g, 100) == -1


def test_plan_capacity_power_and_saturating_schedules(kvm):
    # floor(16 e^(1/2)) is the sqrt schedule
    gp = kvm.growth("power", sqrt_coeff=16, pow_num=1, pow_den=2)
    for e, m in ((768, 443), (1024, 512), (32768, 2896), (131072, 5792)):
        assert kvm.kvm_plan_capacity(256, 2, gp, e) == m
    # exact integer floors: rows = the largest n with n^3 <= 8^3 e^2 once the budget has passed one block
    g23 = kvm.growth("power", sqrt_coeff=8, pow_num=2, pow_den=3)
    for e in (4096, 8192, 65536, 1 << 20):
        n = kvm.kvm_plan_capacity(32, 2, g23, e)
        assert n ** 3 <= 8 ** 3 * e ** 2 < (n + 1) ** 3, (e, n)
    gs = kvm.growth("saturating", fixed_slots=1024, sat_half=4096)
    assert kvm.kvm_plan_capacity(64, 2, gs, 4096) == 512
    assert kvm.kvm_plan_capacity(64, 2, gs, 1 << 22) == (1024 * (1 << 22)) // ((1 << 22) + 4096) == 1023
    # parameters outside the defined range
    assert kvm.kvm_plan_capacity(64, 2, kvm.growth("power", sqrt_coeff=16, pow_num=3, pow_den=2), 1024) == -1
    assert kvm.kvm_plan_capacity(64, 2, kvm.growth("power", sqrt_coeff=2000, pow_num=1, pow_den=2), 1024) == -1
    assert kvm.kvm_plan_capacity(64, 2, gp, 1 << 26) == -1
    assert kvm.kvm_plan_capacity(64, 2, kvm.growth("saturating", fixed_slots=100, sat_half=0), 1024) == -1


def test_create_validates_arguments_before_touching_the_device(kvm):
    h = C.c_void_p()
    assert kvm.lib.kvm_state_create(None, C.byref(h)) == 1
    bad = kvm.Config(1, 3, 2, 128, 2, 1, 10000.0, 1e-5, 1e-12, None, None, None, None, 64, 64, 64, 0, 0, 0)
    assert kvm.lib.kvm_state_create(C.byref(bad), C.byref(h)) == 1          # 3 q heads over 2 kv heads
    bad = kvm.Config(1, 2, 2, 96, 2, 1, 10000.0, 1e-5, 1e-12, None, None, None, None, 64, 64, 64, 0, 0, 0)
    assert kvm.lib.kvm_state_create(C.byref(bad), C.byref(h)) == 2          # head_dim 96
    bad = kvm.Config(1, 2, 2, 128, 2, 1, 10000.0, 1e-5, 1e-12, None, None, None, None, 512, 512, 64, 0, 0, 0)
    assert kvm.lib.kvm_state_create(C.byref(bad), C.byref(h)) == 2          # block > 256
    assert kvm.lib.kvm_state_free(None) == 0
    assert kvm.lib.kvm_state_info(None, None, None, None) == 1


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful without a GPU")
def test_no_cpu_fallback_without_a_device(kvm):
    h = C.c_void_p()
    ok = kvm.Config(1, 2, 2, 128, 2, 1, 10000.0, 1e-5, 1e-12, None, None, None, None, 64, 64, 64, 0, 0, 0)
    assert kvm.lib.kvm_state_create(C.byref(ok), C.byref(h)) == 4           # KVM_ERR_CUDA, loudly

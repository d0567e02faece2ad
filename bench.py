#!/usr/bin/env python
"""Benchmark of the KVM layer hot path on B200 (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5] [--impl reference]

A "step" is one pass of the whole hot path over one batch of synthetic input:
  cfg5 (default; the largest configuration: B64 H32 d128, 65536 tokens, block 256, 16 sqrt(N) budget):
      kvm_prefill of the whole sequence on an empty state, fed as 16 segments of 4096 tokens that are all
      resident in HBM (ingest, per-block attention over [state ; window], every fold); metric = prefill
      tokens/s.  The same JSON line carries a "decode" record: the 256 single-token decode steps that
      follow on that very state (us per step, HBM GB/s).
  prefill workloads (cfg1..cfg4, paper-speed): kvm_prefill of the full sequence in one call;
      metric = prefill tokens/s (batch * sequence tokens per second).
  decode workload (cfg5-decode): one kvm_decode_step for the whole batch on a state of
      m = 4096 rows plus a 256..511-token window built by a short fixed-budget prefill (a quick way to
      time the decode kernel alone); metric = decode us per step.
`value` is measured with inputs resident in HBM; `e2e` goes through the *_host entry points
with pinned host buffers (H2D and D2H inside the timed region).  With N > 1 every rank runs
the same per-GPU workload on its own units (weak scaling, no data-path collective).
"""
import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2605_09877_b200 import synth  # noqa: E402


# ------------------------------------------------------------------------------------------
# workload table and algorithmic work

def workload(name):
    c = synth.CONFIGS
    if name == "cfg5":
        return c[name], "prefill+decode"
    if name in c:
        return c[name], "prefill"
    if name == "paper-speed":   # the paper's speed-benchmark shape: B8 H32 d128 C256, KVM-sqrt, T=32768
        return synth.Workload("paper-speed", 8, 32, 32, 128, 32768, 256, "sqrt", r=0, seed=7), "prefill"
    if name == "cfg5-decode":
        return c["cfg5"], "decode"
    raise SystemExit(f"unknown workload {name}")


def fold_schedule(wl, T):
    """(e, m_before, n_append) per fold from the budget rule M* = max(m, min(B(e), m + C))."""
    out, m = [], 0
    for c in range(T // wl.C):
        e = (c + 1) * wl.C
        if c < wl.w - 1:
            continue
        if m == 0:
            out.append((e, 0, wl.C)); m = wl.C
            continue
        bud = wl.fixed_slots if wl.growth == "fixed" else (math.isqrt(wl.sqrt_coeff ** 2 * e) if wl.growth == "sqrt" else 1 << 60)
        na = min(max(m, min(bud, m + wl.C)) - m, wl.C)
        out.append((e, m, na)); m += na
    return out


def prefill_flops(wl, T):
    """Algorithmic flops of one prefill: attention 4*d per (query, visible key) with the causal
    triangle counted as a triangle, routing 2*d per (overflow token, state row) similarity."""
    folds = {e: (m0, na) for e, m0, na in fold_schedule(wl, T)}
    m, att_pairs, route_pairs = 0, 0, 0
    for c in range(T // wl.C):
        e = (c + 1) * wl.C
        win_prev = min(c, wl.w - 1) * wl.C
        att_pairs += wl.C * (m + win_prev) + wl.C * (wl.C + 1) // 2
        if e in folds:
            m0, na = folds[e]
            if m0 > 0:
                route_pairs += wl.C * m0 + (wl.C - na) * na
            m = m0 + na
    units_q, units_kv = wl.B * wl.Hq, wl.B * wl.Hkv
    return 4 * wl.d * att_pairs * units_q, 2 * wl.d * route_pairs * units_kv


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of the kernels that carry a roofline, from the ncu
# captures summarised under profiles/ncu_full_cfg5_small_case_prefill_and_decode_kernels.md.  The captures run a
# small case of the same kernels (256 units instead of 2048; 640 decode heads instead of 2048); both kernels read
# every key / value row of a (batch, head) unit once per launch, so the traffic of a launch grows in proportion to
# units x rows: the figure reported for a full-size launch is the algorithmic bytes of that launch times the
# measured ratio (traffic / algorithmic bytes) of the captured launches.
NCU_TRAFFIC_RATIO = {
    "attention": (268.54e6 + 13.6e6) / 278.2e6,   # captured: 268.5 MB read + 13.6 MB written; algorithmic 278.2 MB per launch
    "decode": 1.4320e9 / 1.4293e9,                # captured: 1.428 GB read + 4 MB written; algorithmic 1.4293 GB per launch
}


def attention_bytes_per_launch(wl, T):
    """Algorithmic bytes of an average attention launch of a prefill: per (batch, kv head) unit the fp16 readout rows
    K^, V^ of the state and the fp16 window keys and values the block can see, once; per (batch, q head) the block's
    fp16 queries read and its bf16 outputs written."""
    folds = {e: (m0, na) for e, m0, na in fold_schedule(wl, T)}
    m, tot, n = 0, 0, 0
    for c in range(T // wl.C):
        e = (c + 1) * wl.C
        win = min(c, wl.w - 1) * wl.C + wl.C
        tot += wl.B * wl.Hkv * (m + win) * wl.d * 2 * 2 + wl.B * wl.Hq * wl.C * wl.d * 2 * 2
        n += 1
        if e in folds:
            m = folds[e][0] + folds[e][1]
    return tot / max(n, 1)


def decode_bytes(wl, m, pos):
    """Algorithmic bytes of the decode step at position `pos`: fp16 readout rows K^, V^ of the m state rows plus
    the window tokens [b, pos] (keys and values), for every (batch, kv head)."""
    b = max(0, (pos // wl.C + 1) * wl.C - wl.w * wl.C)
    return wl.B * wl.Hkv * (m + pos - b + 1) * wl.d * 2 * 2


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tf_burst=d["bf16_tflops"], tf_sust=d["bf16_tflops_sustained"], src="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sust=1400.0, src="fallback")


# ------------------------------------------------------------------------------------------
# clocks

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.path = tempfile.mktemp(prefix="kvm_clocks_", suffix=".csv")
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        self.proc.wait()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        sm.sort()
        return dict(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))


# ------------------------------------------------------------------------------------------
# CPU oracle leg (reported baseline; the only place bench.py touches oracle/)

def oracle_sample(wl, mode, budget_s=20.0):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload."""
    from oracle import kvm_oracle as ko
    from tests.parity_util import oracle_config
    cores = ko.threads()
    if mode.startswith("prefill"):
        # sample: `n_units` (batch, head) units over a prefix of T_s tokens sized for ~budget_s
        n_units = min(cores, wl.B * wl.Hkv)
        T_s = wl.T
        att, rt = prefill_flops(wl.scaled(B=1, Hq=n_units * (wl.Hq // wl.Hkv), Hkv=n_units), T_s)
        rate = 1.6e9 * cores   # fp64 flop/s of the plain loops at the long end (3.2e9 on short prefixes); only sizes the sample
        while (att + rt) / rate > budget_s and T_s > 4 * wl.C:
            T_s = max(4 * wl.C, int(T_s * 0.75) // (4 * wl.C) * (4 * wl.C))
            att, rt = prefill_flops(wl.scaled(B=1, Hq=n_units * (wl.Hq // wl.Hkv), Hkv=n_units), T_s)
        small = wl.scaled(B=1, Hq=n_units * (wl.Hq // wl.Hkv), Hkv=n_units, T=T_s)
        t = synth.make_inputs(small)
        o = ko.KVMOracle(oracle_config(small))
        q, k, v = (t[n].double().numpy() for n in "qkv")
        t0 = time.perf_counter()
        o.forward(q, k, v)
        dt = time.perf_counter() - t0
        # tokens/s of the whole layer (all B*Hkv units) at the oracle's measured unit rate
        layer_tokens = wl.B * T_s * (n_units / (wl.B * wl.Hkv))
        return dict(value=layer_tokens / dt, unit="tokens/s", cores=cores, kind="oracle",
                    sample=f"{n_units} of {wl.B * wl.Hkv} (batch,head) units x first {T_s} of {wl.T} tokens, "
                           f"{dt:.1f} s wall; value = layer tokens/s at that unit rate"), dt
    # decode: oracle state built by a short unbounded-growth prefill to m rows, then timed steps
    n_units = min(cores, wl.B * wl.Hkv)
    small = synth.Workload("dec-sample", 1, n_units, n_units, wl.d, 4096 + 256 + 128, 256, "unbounded", seed=wl.seed)
    t = synth.make_inputs(small)
    o = ko.KVMOracle(oracle_config(small))
    q, k, v = (t[n].double().numpy() for n in "qkv")
    o.forward(q, k, v)
    steps = 8
    dq = synth.make_inputs(small.scaled(T=steps, seed=wl.seed + 1))
    q, k, v = (dq[n].double().numpy() for n in "qkv")
    t0 = time.perf_counter()
    for s in range(steps):
        o.forward(q[:, :, s:s + 1], k[:, :, s:s + 1], v[:, :, s:s + 1])
    dt = (time.perf_counter() - t0) / steps
    us_full = dt * 1e6 * (wl.B * wl.Hkv / n_units)
    return dict(value=us_full, unit="us/step", cores=cores, kind="oracle",
                sample=f"{n_units} of {wl.B * wl.Hkv} units, state of {o.rows} rows + window, {steps} steps; "
                       f"value = measured step time x {wl.B * wl.Hkv // n_units} (units are independent)"), dt * steps


# ------------------------------------------------------------------------------------------

def dist_setup(n, backend="nccl"):
    """One process per GPU (torchrun sets RANK / LOCAL_RANK / WORLD_SIZE).  The ranks are independent
    replicas of the per-GPU workload; the process group only serves the barrier and the max."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        else:
            dist.init_process_group(backend)
    return rank, world, local


def barrier(world, cuda=True):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if cuda:
        torch.cuda.synchronize()


def max_over_ranks(x, world, device="cuda"):
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate(mode, local_ms_per_step, units_per_step, world, device="cuda"):
    """Whole-job value from per-rank step times: every rank processes `units_per_step` units per step
    (weak scaling), the job's step time is the slowest rank's.  Returns (value, ms_per_step)."""
    ms = max_over_ranks(local_ms_per_step, world, device)
    if mode.startswith("prefill"):
        return world * units_per_step / (ms * 1e-3), ms     # tokens/s over all replicas
    return ms * 1e3, ms                                     # decode: us per step (each replica steps its batch)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl, mode = workload(args.workload)
    vals, last = [], None
    for i in range(args.warmup + args.steps):
        res, _ = oracle_sample(wl, mode, budget_s=8.0)
        if i >= args.warmup:
            vals.append(res["value"])
        last = res
    v = sum(vals) / len(vals)
    unit = last["unit"]
    pre = mode.startswith("prefill")
    ms = (wl.B * wl.T / v * 1e3) if pre else v / 1e3
    line = dict(metric="kvm_prefill_tokens_per_s" if pre else "kvm_decode_us_per_step", value=v, unit=unit,
                n_gpus=args.gpus, steps=args.steps, warmup=args.warmup, ms_per_step=ms,
                higher_is_better=pre, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=wl.name, mode=mode), impl="reference",
                cpu_baseline=dict(value=v, unit=unit, cores=last["cores"], kind="oracle", sample=last["sample"]),
                e2e=dict(value=v, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


def run_gate(args):
    """Front-end merge gate g = 1 + ELU(x W_g) (kvm_merge_gate): HBM-bound on reading x.  "gate": the
    default workload's layer (B2 T8192, d_model = Hq d = 2048, 16 kv heads); "gate-paper": the paper's
    speed shape (B8 T32768, d_model 4096, 32 heads; x is 2.1 GB)."""
    from paper_2605_09877_b200 import kvm
    rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    B, T, dm, H = (8, 32768, 4096, 32) if args.workload == "gate-paper" else (2, 8192, 2048, 16)
    pk = peaks()
    W, K = max(args.warmup, 3), args.steps
    gen = torch.Generator().manual_seed(100 + rank)
    x_host = torch.randn((B, T, dm), generator=gen).to(torch.bfloat16).pin_memory()
    w_host = (torch.randn((H, dm), generator=gen) / math.sqrt(dm)).float()
    x, w = x_host.to(dev), w_host.to(dev)
    gate = torch.empty((B, H, T), dtype=torch.float32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    bytes_step = B * T * dm * 2 + B * H * T * 4 + H * dm * 4   # x read once, gate written once, W_g read once
    for _ in range(W):
        kvm.merge_gate(x, w, out=gate)
    barrier(world)
    torch.cuda.synchronize()
    clocks = ClockSampler(local)
    clocks.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in ev:
        flush.zero_()
        a.record()
        kvm.merge_gate(x, w, out=gate)
        b.record()
    torch.cuda.synchronize()
    barrier(world)
    clk = clocks.stop()
    ms = sum(a.elapsed_time(b) for a, b in ev) / K
    ms_all = max_over_ranks(ms, world)
    # end to end: x from pinned host memory, the gates back to the host
    g_host = torch.empty((B, H, T), dtype=torch.float32).pin_memory()
    e2e = None
    if not args.no_e2e:
        t_e2e = []
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            xd = x_host.to(dev, non_blocking=True)
            kvm.merge_gate(xd, w, out=gate)
            g_host.copy_(gate, non_blocking=True)
            torch.cuda.synchronize()
            t_e2e.append(time.perf_counter() - t0)
        e2e = dict(value=world * B * T / min(t_e2e), unit="tokens/s", h2d_bytes_per_step=B * T * dm * 2,
                   d2h_bytes_per_step=B * H * T * 4)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle.frontend import merge_gate as oracle_gate
        nb = 1 if B * T * dm > (1 << 27) else B           # a bounded sample: one batch row of the large shape
        xs = x_host[:nb].double().numpy()
        t0 = time.perf_counter()
        ref = oracle_gate(xs, w_host.double().numpy())
        dt = time.perf_counter() - t0
        err = float(np.max(np.abs(gate[:nb].cpu().double().numpy() - ref) / np.maximum(1.0, ref)))
        assert err < 2e-4, err
        cpu = dict(value=nb * T / dt, unit="tokens/s", cores=os.cpu_count(), kind="oracle",
                   sample=f"{nb} of {B} batch rows x {T} tokens, {dt:.2f} s wall (numpy fp64); GPU result checked against it: max err {err:.1e}")
    if rank == 0:
        achieved = bytes_step / (ms * 1e-3) / 1e9
        line = dict(metric="kvm_merge_gate_tokens_per_s", value=world * B * T / (ms_all * 1e-3), unit="tokens/s",
                    n_gpus=world, steps=K, warmup=W, ms_per_step=ms_all, higher_is_better=True, scaling="weak",
                    vs_baseline=None, dtype="bf16 inputs, f32 accumulate", data="synthetic",
                    config=dict(workload=args.workload, mode="front end: merge gate", B=B, T=T, d_model=dm, Hkv=H,
                                l2="256 MiB flush between timed steps"),
                    clocks=clk, e2e=e2e, gpu_launches=K,
                    roofline=dict(bound="hbm", kernel="merge_gate", achieved=achieved, peak=pk["hbm"], unit="GB/s",
                                  frac=achieved / pk["hbm"], traffic=None, peak_source=pk["src"] + " copy bandwidth",
                                  bytes_per_step=bytes_step),
                    cpu_baseline=cpu)
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


def run_headln(args):
    """Front-end LN_q / LN_k (kvm_head_layernorm, in place): HBM-bound, every element read and written
    once.  "headln": the default workload's q (B2 H16 T8192 d128, 67 MB); "headln-paper": B8 H32 T32768
    d128 (2.1 GB)."""
    from paper_2605_09877_b200 import kvm
    rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    B, H, T, d = (8, 32, 32768, 128) if args.workload == "headln-paper" else (2, 16, 8192, 128)
    pk = peaks()
    W, K = max(args.warmup, 3), args.steps
    gen = torch.Generator().manual_seed(200 + rank)
    x_host = (torch.randn((B, H, T, d), generator=gen) * 2.0 + 0.5).to(torch.bfloat16).pin_memory()
    w = (1.0 + 0.3 * torch.randn((H, d), generator=gen)).float().to(dev)
    bia = (0.2 * torch.randn((H, d), generator=gen)).float().to(dev)
    x = x_host.to(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    bytes_step = 2 * B * H * T * d * 2
    for _ in range(W):
        x.copy_(x_host, non_blocking=True)
        kvm.head_layernorm(x, w, bia)
    barrier(world)
    clocks = ClockSampler(local)
    clocks.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in ev:
        x.copy_(x_host, non_blocking=True)   # (the kernel works in place: fresh inputs every step, outside the bracket)
        flush.zero_()
        a.record()
        kvm.head_layernorm(x, w, bia)
        b.record()
    torch.cuda.synchronize()
    barrier(world)
    clk = clocks.stop()
    ms = sum(a.elapsed_time(b) for a, b in ev) / K
    ms_all = max_over_ranks(ms, world)
    y_host = torch.empty_like(x_host).pin_memory()
    e2e = None
    if not args.no_e2e:
        t_e2e = []
        for _ in range(3):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            x.copy_(x_host, non_blocking=True)
            kvm.head_layernorm(x, w, bia)
            y_host.copy_(x, non_blocking=True)
            torch.cuda.synchronize()
            t_e2e.append(time.perf_counter() - t0)
        e2e = dict(value=world * B * T / min(t_e2e), unit="tokens/s", h2d_bytes_per_step=B * H * T * d * 2,
                   d2h_bytes_per_step=B * H * T * d * 2)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        from oracle.frontend import head_layernorm as oracle_ln
        nb = 1 if B * H * T * d > (1 << 27) else B
        hs = H if nb == B else 4                       # a bounded sample of the large shape: 4 heads of one batch row
        xs = x_host[:nb, :hs].double().numpy()
        t0 = time.perf_counter()
        ref = oracle_ln(xs, w[:hs].cpu().double().numpy(), bia[:hs].cpu().double().numpy(), 1e-5)
        dt = time.perf_counter() - t0
        got = y_host[:nb, :hs].double().numpy() if e2e else None
        if got is not None:
            assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-5)
        cpu = dict(value=nb * T * hs / H / dt, unit="tokens/s", cores=os.cpu_count(), kind="oracle",
                   sample=f"{hs} of {H} heads x {nb} of {B} batch rows x {T} tokens, {dt:.2f} s wall (numpy fp64; value = layer tokens/s at that rate)")
    if rank == 0:
        achieved = bytes_step / (ms * 1e-3) / 1e9
        line = dict(metric="kvm_head_layernorm_tokens_per_s", value=world * B * T / (ms_all * 1e-3), unit="tokens/s",
                    n_gpus=world, steps=K, warmup=W, ms_per_step=ms_all, higher_is_better=True, scaling="weak",
                    vs_baseline=None, dtype="bf16 in/out, f32 statistics", data="synthetic",
                    config=dict(workload=args.workload, mode="front end: LN_q / LN_k", B=B, H=H, T=T, d=d,
                                l2="256 MiB flush between timed steps"),
                    clocks=clk, e2e=e2e, gpu_launches=K,
                    roofline=dict(bound="hbm", kernel="head_layernorm", achieved=achieved, peak=pk["hbm"], unit="GB/s",
                                  frac=achieved / pk["hbm"], traffic=None, peak_source=pk["src"] + " copy bandwidth",
                                  bytes_per_step=bytes_step),
                    cpu_baseline=cpu)
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


def decode_record(st, wl, dev, stream, pk, world):
    """The decode half of the metric on the state the timed prefill left (position T, m rows, one block in the
    window): wl.decode_steps single-token steps with fresh inputs, every step between two CUDA events; the last
    one completes a block and folds.  The first half is timed as the user sees it (whole steps), the second
    half also with the library's per-kernel brackets (attention incl. its ingest, without the fold)."""
    n = wl.decode_steps
    info0 = st.info()
    dq = [synth.make_decode_inputs(wl.scaled(seed=wl.seed), i, device=dev) for i in range(n)]
    out = torch.empty_like(dq[0]["q"])
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    half = n // 2
    torch.cuda.synchronize()
    for i in range(n):
        if i == half:
            torch.cuda.synchronize()
            st.profile_enable(True)
            st.profile_read()
        d = dq[i]
        ev[i][0].record(stream)
        st.decode_step(d["q"], d["k"], d["v"], out=out)
        ev[i][1].record(stream)
    torch.cuda.synchronize()
    prof = st.profile_read()
    st.profile_enable(False)
    info1 = st.info()
    us = [1e3 * a.elapsed_time(b) for a, b in ev]
    plain = us[3:half]                                   # whole steps, user's view (the first three warm up)
    nbytes = [decode_bytes(wl, info0["n_slots"], info0["position"] + i) for i in range(n)]
    us_plain = sum(plain) / len(plain)
    gbs_plain = sum(nbytes[3:half]) / 1e9 / (sum(plain) * 1e-6)
    kern_ms, kern_n = prof["decode"]
    nfold = info1["n_folds"] - info0["n_folds"]
    kern_bytes = sum(nbytes[half:])
    gbs_kern = kern_bytes / 1e9 / (kern_ms * 1e-3) if kern_ms > 0 else None
    us_all = max_over_ranks(us_plain, world)
    return dict(metric="kvm_decode_us_per_step", value=us_all, unit="us/step", us_per_sequence_token=us_all / wl.B,
                steps=n, state_rows=info0["n_slots"], position0=info0["position"], folds_in_these_steps=nfold,
                fold_step_us=us[-1] if nfold else None, median_us=sorted(plain)[len(plain) // 2],
                min_us=min(plain), max_us=max(plain),
                roofline=dict(bound="hbm", kernel="decode", achieved=gbs_plain, peak=pk["hbm"], unit="GB/s",
                              frac=gbs_plain / pk["hbm"], frac_of_nominal_8TBs=gbs_plain / 8000.0,
                              traffic=sum(nbytes[3:half]) / len(plain) * NCU_TRAFFIC_RATIO["decode"],
                              peak_source=f"{pk['src']} copy bandwidth", bytes_per_step=sum(nbytes[3:half]) / len(plain),
                              what="whole decode steps (ingest + attention kernels), CUDA events around each step",
                              kernels_only_gbs=gbs_kern, kernels_only_us=1e3 * kern_ms / max(kern_n, 1)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg5")
    ap.add_argument("--impl", default="kvm")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle leg")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--simt", action="store_true", help="time the scalar-core cross-check kernels")
    ap.add_argument("--serial", action="store_true", help="force one readout copy and folds on the caller's stream")
    ap.add_argument("--tokens", type=int, default=0,
                    help="prefill workloads: shorten the sequence to this many tokens (small cases for ncu captures; "
                         "cfg5: a multiple of 4096)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (small cases for ncu captures)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.workload in ("gate", "gate-paper"):
        return run_gate(args)
    if args.workload in ("headln", "headln-paper"):
        return run_headln(args)

    from paper_2605_09877_b200 import kvm
    rank, world, local = dist_setup(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wl, mode = workload(args.workload)
    if args.batch:
        wl = wl.scaled(B=args.batch, name=f"{wl.name}-B{args.batch}")
    if args.tokens and mode == "prefill":
        wl = wl.scaled(T=args.tokens, name=f"{wl.name}-T{args.tokens}")
    pk = peaks()
    W, K = max(args.warmup, 3), args.steps
    g = kvm.growth(wl.growth, wl.fixed_slots, wl.sqrt_coeff)
    flags = (kvm.FLAG_SIMT_ATTENTION | kvm.FLAG_SIMT_ROUTING) if args.simt else 0
    if args.serial:
        flags |= kvm.FLAG_SERIAL_FOLDS
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    segs = None
    if mode == "prefill+decode":
        # the largest configuration: the sequence is fed in segments (q, k, v of all 65536 tokens are 103 GB,
        # all resident before the timed region starts); the outputs of a segment overwrite the previous one's
        T, seg = (args.tokens or wl.T), 4096
        assert T % seg == 0
        cap = kvm.kvm_plan_capacity(wl.C, wl.w, g, T + wl.decode_steps)
        st = kvm.KVMState(kvm.LayerConfig(wl.B, wl.Hq, wl.Hkv, wl.d, wl.C, max(cap, wl.C), seg, n_bswa_chunks=wl.w,
                                          sink_len=wl.S, device=local, flags=flags))
        segs = [synth.make_segment(wl.scaled(seed=wl.seed + 1000 * rank), i, seg, device=dev) for i in range(T // seg)]
        out = torch.empty_like(segs[0]["q"])
        if T != wl.T:
            wl = wl.scaled(T=T, name=f"{wl.name}-T{T}")

        def step():
            st.reset()
            for t in segs:
                st.prefill(t["q"], t["k"], t["v"], wl.C, g, wl.r, out=out)

        units_per_step = wl.B * T   # tokens
    elif mode == "prefill":
        T = wl.T
        cap = kvm.kvm_plan_capacity(wl.C, wl.w, g, T)
        st = kvm.KVMState(kvm.LayerConfig(wl.B, wl.Hq, wl.Hkv, wl.d, wl.C, max(cap, wl.C), T, n_bswa_chunks=wl.w,
                                          sink_len=wl.S, device=local, flags=flags))
        cpu = synth.make_inputs(wl.scaled(seed=wl.seed + 1000 * rank))
        q, k, v = (cpu[n].to(dev) for n in "qkv")
        out = torch.empty_like(q)

        def step():
            st.reset()
            st.prefill(q, k, v, wl.C, g, wl.r, out=out)

        units_per_step = wl.B * T   # tokens
    else:
        # state of m = 4096 rows (fixed budget 4096 reached by appends) and a one-block window
        m_rows, Tp = 4096, 5120   # 16 appending folds (e = 512 .. 4352), then 3 merging folds
        seg = 1024
        st = kvm.KVMState(kvm.LayerConfig(wl.B, wl.Hq, wl.Hkv, wl.d, wl.C, m_rows + 256, seg, n_bswa_chunks=wl.w,
                                          sink_len=wl.S, device=local, flags=flags))
        gfix = kvm.growth("fixed", fixed_slots=m_rows)
        for s in range(Tp // seg):
            t = synth.make_segment(wl, s, seg, device=dev)
            st.prefill(t["q"], t["k"], t["v"], wl.C, gfix, wl.r)
        torch.cuda.synchronize()
        assert st.info()["n_slots"] == m_rows
        dq = [synth.make_decode_inputs(wl, i % 8, device=dev) for i in range(8)]
        out = torch.empty_like(dq[0]["q"])
        cnt = [0]

        def step():
            d = dq[cnt[0] % 8]
            cnt[0] += 1
            st.decode_step(d["q"], d["k"], d["v"], out=out)

        units_per_step = wl.B       # sequence-tokens per step

    for _ in range(W):
        step()
    barrier(world)
    sampler = ClockSampler(local)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    l0 = st.launch_count()
    for i in range(K):
        flush.fill_(i & 0xff)             # L2 flush between timed iterations (untimed)
        ev[i][0].record(stream)
        step()
        ev[i][1].record(stream)
    barrier(world)
    launches = st.launch_count() - l0
    clocks = sampler.stop()
    times = [a.elapsed_time(b) for a, b in ev]
    value, ms_step = aggregate(mode, sum(times) / K, units_per_step, world)

    decode_rec = None
    if mode == "prefill+decode":
        decode_rec = decode_record(st, wl, dev, stream, pk, world)

    # per-phase device time (separate pass with event brackets) -> roofline of the dominant phase
    st.profile_enable(True)
    st.profile_read()
    nprof = 1 if mode == "prefill+decode" else min(K, 3)
    for i in range(nprof):
        flush.fill_(i)
        step()
    prof = st.profile_read()
    st.profile_enable(False)

    if mode.startswith("prefill"):
        att_f, rt_f = prefill_flops(wl, wl.T)
        per_kernel = {k_: v_[0] / nprof for k_, v_ in prof.items()}
        # the dominant kernel by device time; the two tensor-core kernels have an algorithmic flop count
        dom = max(per_kernel, key=per_kernel.get)
        if dom not in ("attention", "route_filter"):
            dom = "attention"   # decide / apply / kbar are latency-bound helpers without a flop model
        dom_ms = per_kernel[dom]
        n_dom = prof[dom][1] / nprof
        ach = ((att_f if dom == "attention" else rt_f) / 1e12) / (dom_ms * 1e-3)
        peak = pk["tf_sust"]
        roof = dict(bound="tensor", kernel=dom, achieved=ach, peak=peak, unit="TFLOP/s", frac=ach / peak,
                    traffic=(attention_bytes_per_launch(wl, wl.T) * NCU_TRAFFIC_RATIO["attention"]) if dom == "attention" else None,
                    traffic_source="algorithmic bytes of an average launch x (DRAM traffic / algorithmic bytes) of the ncu small-case capture (profiles/)",
                    algorithmic_bytes_per_launch=attention_bytes_per_launch(wl, wl.T) if dom == "attention" else None,
                    peak_source=f"{pk['src']} bf16 sustained (fp16 operands run at the bf16 rate)",
                    frac_of_burst=ach / pk["tf_burst"], frac_of_nominal_2250=ach / 2250.0,
                    launches_per_step=n_dom, avg_launch_us=1e3 * dom_ms / max(n_dom, 1),
                    share_of_device_time=dom_ms / max(sum(per_kernel.values()), 1e-9),
                    whole_step_tflops=(att_f + rt_f) / 1e12 / (ms_step * 1e-3),
                    whole_step_frac_of_burst=(att_f + rt_f) / 1e12 / (ms_step * 1e-3) / pk["tf_burst"],
                    phase_ms={k_: v_[0] / nprof for k_, v_ in prof.items()})
        metric, unit, hib = "kvm_prefill_tokens_per_s", "tokens/s", True
    else:
        info = st.info()
        # window tokens seen by the profiled steps (the last `nprof` ones): positions t attend [b, t]
        pos_end = info["position"]
        steps_t = range(pos_end - nprof, pos_end)
        nwin_avg = sum(t - max(0, (t // wl.C + 1) * wl.C - wl.w * wl.C) + 1 for t in steps_t) / nprof
        bytes_step = wl.B * wl.Hkv * (info["n_slots"] + nwin_avg) * wl.d * 2 * 2
        dec_ms = prof["decode"][0] / max(prof["decode"][1], 1)
        ach = bytes_step / 1e9 / (dec_ms * 1e-3)
        roof = dict(bound="hbm", kernel="decode", achieved=ach, peak=pk["hbm"], unit="GB/s", frac=ach / pk["hbm"],
                    traffic=bytes_step * NCU_TRAFFIC_RATIO["decode"], peak_source=f"{pk['src']} copy bandwidth",
                    bytes_per_step=bytes_step,
                    frac_of_nominal_8TBs=ach / 8000.0, phase_ms={k_: v_[0] / max(v_[1], 1) for k_, v_ in prof.items()})
        metric, unit, hib = "kvm_decode_us_per_step", "us/step", False

    # end to end through the host-buffer entry points (pinned memory)
    e2e = None
    if not args.no_e2e:
        if mode == "prefill+decode":
            # host buffers of two segments (pinned), sent alternately: a step copies every segment's q, k, v in
            # and its outputs out (the host buffers of all 16 segments would be 137 GB of pinned memory)
            hseg = [{n: segs[i][n].cpu().pin_memory() for n in "qkv"} for i in range(2)]
            hout = torch.empty_like(hseg[0]["q"]).pin_memory()
            nseg_ = len(segs)
            def estep():
                st.reset()
                for i in range(nseg_):
                    h = hseg[i & 1]
                    st.prefill_host(h["q"], h["k"], h["v"], wl.C, g, wl.r, hout)
            bi = nseg_ * sum(hseg[0][n].numel() for n in "qkv") * 2
            bo = nseg_ * hout.numel() * 2
        elif mode == "prefill":
            hq, hk, hv = (cpu[n].contiguous().pin_memory() for n in "qkv")
            hout = torch.empty_like(hq).pin_memory()
            def estep():
                st.reset()
                st.prefill_host(hq, hk, hv, wl.C, g, wl.r, hout)
            bi = (hq.numel() + hk.numel() + hv.numel()) * 2
            bo = hout.numel() * 2
        else:
            hd = {n: dq[0][n].cpu().pin_memory() for n in "qkv"}
            hout = torch.empty_like(hd["q"]).pin_memory()
            def estep():
                st.decode_step_host(hd["q"], hd["k"], hd["v"], hout)
            bi = sum(hd[n].numel() for n in "qkv") * 2
            bo = hout.numel() * 2
        ne = 2 if mode == "prefill+decode" else min(K, 5)
        for _ in range(1 if mode == "prefill+decode" else 2):
            estep()
        barrier(world)
        t0 = time.perf_counter()
        for _ in range(ne):
            estep()
        torch.cuda.synchronize()
        dt = max_over_ranks((time.perf_counter() - t0) / ne, world)
        ev_ = world * units_per_step / dt if mode.startswith("prefill") else dt * 1e6
        e2e = dict(value=ev_, unit=unit, h2d_bytes_per_step=bi, d2h_bytes_per_step=bo)

    cpu_base = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu_base, _ = oracle_sample(wl, mode)

    if rank == 0:
        line = dict(metric=metric, value=value, unit=unit, n_gpus=world, steps=K, warmup=W, ms_per_step=ms_step,
                    higher_is_better=hib, scaling="weak", vs_baseline=None, dtype="f16 operands, f32 accumulate, f64 routing",
                    data="synthetic",
                    config=dict(workload=wl.name, mode=mode, B=wl.B, Hq=wl.Hq, Hkv=wl.Hkv, d=wl.d, T=wl.T, C=wl.C,
                                growth=wl.growth, rope_dims=wl.r, l2="256 MiB flush between timed steps",
                                kernels="simt" if args.simt else "default"),
                    clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roof, cpu_baseline=cpu_base)
        if segs is not None:
            line["config"]["segments"] = f"{len(segs)} kvm_prefill calls of 4096 tokens per step, all inputs resident in HBM"
        if decode_rec is not None:
            line["decode"] = decode_rec
        print(json.dumps(line))
    st.free()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

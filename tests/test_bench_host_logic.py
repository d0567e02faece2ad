"""Host-side logic of bench.py without a GPU: flop accounting from the budget rule, and the N > 1
aggregation (replicas only: max-over-ranks step time, summed tokens) on two gloo ranks."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["KVM_ROOT"])
import bench
rank, world, local = bench.dist_setup(2, backend="gloo")
bench.barrier(world, cuda=False)
local_ms = 10.0 if rank == 0 else 12.5          # the slower rank sets the job's step time
v, ms = bench.aggregate("prefill", local_ms, 1000, world, device="cpu")
vd, msd = bench.aggregate("decode", local_ms, 64, world, device="cpu")
if rank == 0:
    print(json.dumps(dict(world=world, v=v, ms=ms, vd=vd, msd=msd)))
import torch.distributed as dist
dist.destroy_process_group()
"""


def test_two_rank_aggregation_over_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, KVM_ROOT=ROOT, MASTER_ADDR="127.0.0.1")
    p = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", "29613", str(script)],
                       capture_output=True, text=True, env=env, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    line = [l for l in p.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["world"] == 2
    assert d["ms"] == pytest.approx(12.5) and d["v"] == pytest.approx(2 * 1000 / 12.5e-3)
    assert d["vd"] == pytest.approx(12500.0)


def test_flop_accounting_matches_hand_counts():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2605_09877_b200 import synth
    # tiny case by hand: C=4, w=2, T=12, fixed budget 4, one head, d=8
    wl = synth.Workload("t", 1, 1, 1, 8, 12, 4, "fixed", fixed_slots=4)
    att, rt = bench.prefill_flops(wl, 12)
    # chunk 0: 4*5/2 = 10 pairs; chunk 1: 4*4 (prev block) + 10; chunk 2: 4*(4 state + 4) + 10 = 42
    assert att == 4 * 8 * (10 + 26 + 42)
    # folds at e=8 (initialisation, no routing) and e=12 (4 tokens x 4 rows)
    assert rt == 2 * 8 * 16
    assert bench.fold_schedule(synth.CONFIGS["cfg3"], 32768)[-1][1:] == (2884, 12)
    assert [f[2] for f in bench.fold_schedule(synth.CONFIGS["cfg2"], 8192)[:5]] == [128, 128, 128, 128, 0]

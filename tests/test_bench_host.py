"""Host-side logic of bench.py: byte accounting, peak lookup, and the multi-process aggregation (2 gloo ranks on CPU)."""
import json
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2012_15469_b200 import synth  # noqa: E402


def test_algorithmic_bytes_c5():
    w = synth.workload("C5")
    ab = bench.algorithmic_bytes_per_iteration(w, synth.RULE_CADA2, uploads_per_iter=128.0)
    x_rows = 256 * 512 * 4096 * 4
    assert ab["grad_kernel"] == x_rows + 256 * 512 * 4 + 4096 * 4 * (1 + 256)
    assert ab["total"] == ab["grad_kernel"] + 128 * 4096 * 8 + 256 * 4096 * 4 + 24 * 4096
    # X is counted once although two gradients are taken
    assert ab["grad_kernel"] < 1.01 * x_rows
    a1 = bench.algorithmic_bytes_per_iteration(w, synth.RULE_CADA1, uploads_per_iter=0.0)
    assert a1["total"] - a1["grad_kernel"] == 2 * 256 * 4096 * 4 + 24 * 4096      # stored innovations + aggregate + optimiser


def test_bf16_rows_are_two_bytes():
    w = synth.workload("C4")
    ab = bench.algorithmic_bytes_per_iteration(w, synth.RULE_CADA2, 0.0)
    assert ab["grad_kernel"] >= 10 * 128 * 784 * 2 and ab["grad_kernel"] < 10 * 128 * 784 * 2 + 8e6


def test_measured_peaks_has_a_source():
    p = bench.measured_peaks()
    assert p["source"] in ("measured", "fallback") and p["hbm_gbs"] > 1000


def test_aggregate_single_process():
    assert bench.aggregate_over_ranks(100, 12.5, None) == (100, 12.5)


def test_aggregate_two_gloo_ranks(tmp_path):
    """Replicas: iterations add up over ranks, the time is the slowest rank's."""
    script = tmp_path / "agg.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r = dist.get_rank()
        tot, ms = bench.aggregate_over_ranks(100 + r, 10.0 + 5.0 * r, dist)
        if r == 0:
            print(json.dumps({{"tot": tot, "ms": ms}}))
        dist.destroy_process_group()
    """))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29617", str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    res = json.loads(line)
    assert res == {"tot": 201, "ms": 15.0}


def test_shard_workers_partitions_every_worker_once():
    for M, world in ((20, 2), (20, 8), (10, 4), (7, 3), (3, 8)):
        seen = []
        for r in range(world):
            sh = bench.shard_workers(M, r, world)
            assert sh["M_total"] == M and sh["m_first"] == r and sh["m_stride"] == world
            assert sh["workers"] == [sh["m_first"] + i * sh["m_stride"] for i in range(len(sh["workers"]))]
            seen += sh["workers"]
        assert sorted(seen) == list(range(M))


def test_sharded_step_two_gloo_ranks(tmp_path):
    """The exchange step of the worker-sharded mode on 2 CPU ranks: a stand-in for the library computes each rank's partial
    sum of Eq. 2a over ITS workers; after bench.sharded_step every rank has applied the SAME total, which equals the sum over
    all workers, and the uploads counted on the ranks add up to the one-server count."""
    script = tmp_path / "shard.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch
        import torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        r, world = dist.get_rank(), dist.get_world_size()
        M, p = 7, 5
        G = np.arange(M * p, dtype=np.float32).reshape(M, p) + 1.0           # the stored gradients of the one-server run
        sh = bench.shard_workers(M, r, world)

        class FakeHandle:                                                     # worker side: sum over this rank's workers
            def __init__(self): self.applied, self.uploads = [], 0
            def step_local(self, out):
                out.copy_(torch.from_numpy(G[sh["workers"]].sum(axis=0))); self.uploads += len(sh["workers"])
            def step_apply(self, total): self.applied.append(total.clone())

        h = FakeHandle()
        buf = torch.zeros(p)
        for _ in range(3):
            bench.sharded_step(h, buf, dist)
        ups = torch.tensor([h.uploads]); dist.all_reduce(ups)
        ok = all(np.array_equal(a.numpy(), G.sum(axis=0)) for a in h.applied)
        gathered = [None] * world
        dist.all_gather_object(gathered, [a.tolist() for a in h.applied])
        if r == 0:
            print(json.dumps({{"ok": ok, "same": gathered[0] == gathered[1], "uploads": int(ups.item()), "workers": sh["workers"]}}))
        dist.destroy_process_group()
    """))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29619", str(script)],
                         capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    res = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert res == {"ok": True, "same": True, "uploads": 21, "workers": [0, 2, 4, 6]}


def test_reference_arm_prints_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "C1",
                          "--steps", "5", "--warmup", "3"], capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["value"] > 0 and d["config"]["workload"] == bench.workload_label(synth.workload("C1"))

"""Host logic of the benchmark that needs no GPU: the max-over-ranks reduction on
two gloo ranks, the row sampling of the CPU baseline, the reference arm's line."""
import json
import os
import subprocess
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
r = dist.get_rank()
out = bench.max_over_ranks([10.0 + r, 5.0 - r])
if r == 0:
    print(json.dumps(out))
dist.destroy_process_group()
""" % ROOT


def test_max_over_ranks_two_gloo_processes(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [l for l in res.stdout.splitlines() if l.startswith("[")][-1]
    assert json.loads(line) == [11.0, 5.0]


def test_max_over_ranks_single_process():
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


def test_row_sample_is_a_prefix_of_the_inputs():
    shapes = bench.scaled(bench.FULL, 0.0002)
    shapes["outer"]["cols"] = 500
    host = bench.make_host_inputs(shapes, pinned=False)
    sub, sh = bench.row_sample(host, shapes, 0.5)
    assert sh["magg"]["rows"] == shapes["magg"]["rows"] // 2
    assert sub["magg.X"].shape[0] == sh["magg"]["rows"]
    assert torch.equal(sub["row_dense.X"], host["row_dense.X"][:sh["row_dense"]["rows"]])
    r = sh["row_csr"]["rows"]
    assert sub["row_csr.rowptr"].numel() == r + 1
    assert sub["row_csr.vals"].numel() == int(host["row_csr.rowptr"][r])
    assert sub["outer.V"].shape == host["outer.V"].shape          # all of V stays
    assert sub["outer.U"].shape[0] == sh["outer"]["rows"]
    nb = bench.algorithmic_bytes(sh, sub)
    assert all(v > 0 for v in nb.values())
    t, res = bench.oracle_step(bench.numpy_inputs(sub), sh)
    assert set(t) == set(bench.OPS) and np.isfinite(res["outer"])


def test_reference_arm_prints_one_json_line():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
           "--warmup", "0", "--ref-frac", "0.001"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "GB/s" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["cpu_baseline"]["kind"] == "oracle"

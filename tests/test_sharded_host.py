"""The multi-GPU form of the path is row-block sharding plus one small all-reduce.  Its
host logic - which rows go to which rank, and how the pieces combine - runs here on two
`gloo` ranks on CPU, with the CPU checker standing in for the single-GPU call on each
rank's block; the combined result must be the checker's result on the whole input."""
import os
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_1801_00829_b200 import sharded  # noqa: E402


def test_row_blocks_cover_the_rows_once():
    for rows, world in ((10, 3), (7, 8), (0, 2), (1_000_003, 8)):
        cover = [sharded.row_block(rows, r, world) for r in range(world)]
        assert cover[0][0] == 0 and cover[-1][1] == rows
        assert all(a[1] == b[0] for a, b in zip(cover, cover[1:]))
        sizes = [hi - lo for lo, hi in cover]
        assert max(sizes) - min(sizes) <= 1


def test_csr_blocks_balance_the_stored_cells():
    rng = np.random.default_rng(5)
    lens = rng.integers(0, 40, size=5000)
    lens[100:200] = 0                       # a run of empty rows
    lens[4000] = 3000                       # one heavy row
    rowptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    for world in (1, 2, 3, 8):
        b = sharded.csr_row_blocks(rowptr, world)
        assert b[0] == 0 and b[-1] == 5000 and all(x <= y for x, y in zip(b, b[1:]))
        shares = [int(rowptr[b[r + 1]] - rowptr[b[r]]) for r in range(world)]
        assert sum(shares) == int(rowptr[-1])
        assert max(shares) <= int(rowptr[-1]) / world + 3000 + 40     # within one (heaviest) row of the ideal share
    rp, ci, va = sharded.csr_block(rowptr, np.arange(rowptr[-1]), np.arange(rowptr[-1], dtype=np.float64), 150, 4001)
    assert rp[0] == 0 and rp[-1] == len(ci) == len(va) == int(rowptr[4001] - rowptr[150])
    assert ci[0] == rowptr[150]


WORKER = textwrap.dedent("""
    import os, sys, json
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, %(root)r)
    import datagen, oracle
    from paper_1801_00829_b200 import sharded
    dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
    rank, world = dist.get_rank(), dist.get_world_size()
    out = {}
    # Cell full_agg / col_agg / row_agg over a dense input
    w = datagen.cell_workload(301, 57, seed=81)
    lo, hi = sharded.row_block(301, rank, world)
    XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
    sides = [("cell", w["Y"][lo:hi]), ("cell", w["Z"][lo:hi])]
    for agg in ("full", "col", "row"):
        res = sharded.sharded("cell", agg, lambda: torch.as_tensor(
            np.atleast_1d(oracle.cell(XYZ, "t1", w["X"][lo:hi], sides, agg=agg))))
        out["cell_" + agg] = res.tolist()
    # Row over CSR blocks balanced by stored cells: q = t(X) (w * (X v))
    c = datagen.row_csr_workload(4000, 300, 0.02, seed=82)
    b = sharded.csr_row_blocks(c["rowptr"], world)
    rp, ci, va = sharded.csr_block(c["rowptr"], c["colidx"], c["vals"], b[rank], b[rank + 1])
    Xl = dict(rows=b[rank + 1] - b[rank], cols=300, rowptr=rp, colidx=ci, vals=va)
    res = sharded.sharded("row", "col_t", lambda: torch.as_tensor(
        oracle.row_chain_csr(Xl, c["v"], c["w"][b[rank]:b[rank + 1]])))
    out["row_col_t"] = res.tolist()
    # Outer full_agg: rows of X and U partitioned, V replicated
    o = datagen.outer_workload(500, 400, 8, 0.05, seed=83)
    b = sharded.csr_row_blocks(o["rowptr"], world)
    rp, ci, va = sharded.csr_block(o["rowptr"], o["colidx"], o["vals"], b[rank], b[rank + 1])
    Xl = dict(rows=b[rank + 1] - b[rank], cols=400, rowptr=rp, colidx=ci, vals=va)
    res = sharded.sharded("outer", "full", lambda: torch.as_tensor(
        [oracle.outer_wsloss_masked(Xl, o["U"][b[rank]:b[rank + 1]], o["V"])], dtype=torch.float64))
    out["outer_full"] = res.tolist()
    out["rows_here"] = [lo, hi]
    print("RESULT " + json.dumps(out))
    dist.destroy_process_group()
""")


def test_two_ranks_combine_to_the_whole_result(tmp_path):
    import json
    import datagen
    import oracle
    script = tmp_path / "worker.py"
    script.write_text(WORKER % {"root": ROOT})
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29613", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        so, se = p.communicate(timeout=300)
        assert p.returncode == 0, se[-2000:]
        outs.append(json.loads([ln for ln in so.splitlines() if ln.startswith("RESULT ")][-1][7:]))
    w = datagen.cell_workload(301, 57, seed=81)
    XYZ = [("mul", "t0", "a", "side0"), ("mul", "t1", "t0", "side1")]
    sides = [("cell", w["Y"]), ("cell", w["Z"])]
    for r in range(2):                                   # the reduced results are the same on every rank
        assert np.allclose(outs[r]["cell_full"], [oracle.cell(XYZ, "t1", w["X"], sides, agg="full")], rtol=1e-13)
        assert np.allclose(outs[r]["cell_col"], oracle.cell(XYZ, "t1", w["X"], sides, agg="col"), rtol=1e-13)
    rows = np.concatenate([outs[0]["cell_row"], outs[1]["cell_row"]])      # row results stay partitioned
    assert outs[0]["rows_here"][1] == outs[1]["rows_here"][0]
    assert np.allclose(rows, oracle.cell(XYZ, "t1", w["X"], sides, agg="row"), rtol=1e-13)
    c = datagen.row_csr_workload(4000, 300, 0.02, seed=82)
    Xc = {k: c[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    ref = oracle.row_chain_csr(Xc, c["v"], c["w"])
    scale = oracle.row_chain_csr(dict(Xc, vals=np.abs(c["vals"])), np.abs(c["v"]), c["w"])
    assert np.all(np.abs(np.asarray(outs[0]["row_col_t"]) - ref) <= 1e-12 * scale)
    o = datagen.outer_workload(500, 400, 8, 0.05, seed=83)
    Xo = {k: o[k] for k in ("rows", "cols", "rowptr", "colidx", "vals")}
    assert np.allclose(outs[1]["outer_full"], [oracle.outer_wsloss_masked(Xo, o["U"], o["V"])], rtol=1e-13)

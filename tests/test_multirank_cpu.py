"""The N > 1 logic of bench.py on CPU: two gloo ranks agree on the max-over-ranks time, the
whole-job value counts every replica, and the reference arm prints one line from rank 0."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    dist.barrier()
    slowest = bench.max_over_ranks(local_ms, dist, "cpu")
    value = bench.whole_job_value(1e9, world, slowest / 5)
    with open(out + ".%d" % rank, "w") as fh:
        json.dump({"slowest": slowest, "value": value}, fh)
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    out = str(tmp_path / "r")
    mp.spawn(_rank_main, args=(2, 29517, out), nprocs=2, join=True)
    got = [json.load(open(out + ".%d" % r)) for r in range(2)]
    assert got[0] == got[1]
    assert got[0]["slowest"] == 15.0
    # 2 replicas x 1 GB per step, 3 ms per step -> 666.7 GB/s
    assert got[0]["value"] == pytest.approx(2 * 1e9 / 3e-3 / 1e9)


def test_reference_arm_prints_one_line_from_rank_zero():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29519",
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "flat_1m", "--steps", "1", "--warmup", "0"]
    res = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def _sharded_rank(rank, world, port, out):
    """Each rank plays the worker side of its own workers (with the oracle, on CPU), lays its
    messages out as rows of the job-wide exchange buffer — k pairs, then the tile directory,
    padded to an even number of words, rows back to back — and all-gathers them with the
    binding's helper in ONE collective; the server side then has to see the single-process
    result.  Two rounds with different k (a policy change between iterations): the rows of the
    second round have another length inside the same buffer."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import dd_ef_sgd as O
    from paper_2507_17346_b200 import binding as B
    d, n_total, k_cap, tile = 20_000, 4, 120, 8192
    per = n_total // world
    rng = np.random.default_rng(3)
    ntiles = (d + tile - 1) // tile

    def row_words(k):
        return (2 * k + ntiles + 1 + 1) // 2 * 2

    buf = torch.zeros(n_total * row_words(k_cap), dtype=torch.int32)     # sized for k_cap
    ok = True
    for k in (37, 120, 5):
        a = rng.standard_normal((n_total, d)).astype(np.float32)          # same on every rank
        rw = row_words(k)
        rows = buf[:n_total * rw].view(n_total, rw)                       # contiguous prefix
        rows.zero_()
        for w in range(rank * per, (rank + 1) * per):                      # the local workers only
            sel, vals, _ = O.compress(a[w], k)
            rows[w, 0:2 * k:2] = torch.from_numpy(sel.astype(np.int64).astype(np.int32))
            rows[w, 1:2 * k:2] = torch.from_numpy(vals.view(np.int32))
            rows[w, 2 * k:2 * k + ntiles + 1] = torch.from_numpy(
                np.searchsorted(sel, np.arange(ntiles + 1) * tile).astype(np.int32))
        B.all_gather_rows(rows, rank * per, per)
        got = [(rows[w, 0:2 * k:2].numpy().astype(np.uint32),
                rows[w, 1:2 * k:2].numpy().copy().view(np.float32)) for w in range(n_total)]
        S, _ = O.aggregate(got, d)
        want = [O.compress(a[w], k)[:2] for w in range(n_total)]
        S_want, _ = O.aggregate(want, d)
        ok = ok and bool(np.array_equal(S.view(np.uint32), S_want.view(np.uint32)))
        for w in range(n_total):
            ok = ok and rows[w, 2 * k + ntiles].item() == k and np.array_equal(got[w][0], want[w][0])
            ok = ok and rows[w, 2 * k].item() == 0
    with open(out + ".%d" % rank, "w") as fh:
        json.dump({"ok": ok}, fh)
    dist.destroy_process_group()


def test_sharded_exchange_layout_with_two_ranks(tmp_path):
    out = str(tmp_path / "s")
    mp.spawn(_sharded_rank, args=(2, 29523, out), nprocs=2, join=True)
    assert all(json.load(open(out + ".%d" % r))["ok"] for r in range(2))

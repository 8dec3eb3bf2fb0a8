"""CPU-side regression checks: the stored config-1 fixture (generator + oracle determinism) and the
benchmark's oracle arm, single process and as two ranks (replicas: rank 0 alone reports)."""
import json
import os
import subprocess
import sys

import numpy as np

from oracle import dyspec_oracle as orc
from paper_2410_11744_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _fixture():
    rows = {}
    outs = []
    with open(os.path.join(ROOT, "tests", "golden", "config1_oracle.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            if key == "out":
                outs.append((int(vals[0]), int(vals[1]), [float(x) for x in vals[2:]]))
            else:
                rows[key] = vals
    return rows, outs


def test_config1_matches_stored_fixture():
    """The fixture was written by tests/golden/make_golden.py (generator + oracle only)."""
    rows, outs = _fixture()
    w = wl.make_config(1)
    assert [int(x) for x in rows["parents"]] == w.parents[0].tolist()
    bits, depths = orc.build_tree_mask(w.parents[0], 4)
    assert [int(x) for x in rows["depths"]] == depths.tolist()
    assert [int(x, 16) for x in rows["mask_word0"]] == [int(x) for x in bits[:, 0]]
    assert [int(x, 16) for x in rows["q_bits_first8"]] == [int(x) for x in w.q.reshape(-1)[:8]]
    assert int(rows["k_bits_sum"][0]) == int(w.k.astype(np.uint64).sum())
    assert int(rows["v_bits_sum"][0]) == int(w.v.astype(np.uint64).sum())
    out = orc.tree_attention(w.q, w.k, w.v, int(w.prefix_len[0]), w.parents[0])
    for i, h, vals in outs:
        assert np.allclose(out[i, h, :len(vals)], vals, rtol=0, atol=1e-13)
    assert abs(np.abs(out).sum() - float(rows["out_abs_sum"][0])) < 1e-8
    # structure the definitions fix, independent of the stored numbers
    assert w.parents[0][0] == -1 and depths[0] == 0 and int(bits[0, 0]) == 1


def _json_lines(text):
    return [json.loads(ln) for ln in text.splitlines() if ln.startswith("{")]


def test_reference_arm_prints_one_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--warmup", "1", "--config", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr
    lines = _json_lines(r.stdout)
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["metric"] and d["unit"] == "tree tokens/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["config"]["workload"].startswith("c1_")


def test_reference_arm_under_torchrun_two_ranks():
    """N > 1: the path does not shard (replicas only); rank 0 alone runs and prints, the others exit 0."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29731", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0", "--config", "1"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2


def _throughput_rank(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    local_ms = 10.0 if rank == 0 else 25.0                      # rank 1 is the slow one
    value, max_ms = bench.whole_job_throughput(local_ms, 64, 100, world, dist, "cpu")
    q.put((rank, value, max_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_whole_job_throughput_is_all_units_over_the_slowest_rank():
    """N > 1 (replicas, gloo, two CPU ranks): the units of all ranks divided by the maximum over ranks of the time."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_throughput_rank, args=(r, 2, 29741, q)) for r in range(2)]
    for p_ in procs:
        p_.start()
    got = sorted(q.get(timeout=300) for _ in procs)
    for p_ in procs:
        p_.join(timeout=60)
        assert p_.exitcode == 0
    for rank, value, max_ms in got:
        assert max_ms == 25.0 and abs(value - 2 * 64 * 100 / 25e-3) < 1e-6
    sys.path.insert(0, ROOT)
    import bench
    value, max_ms = bench.whole_job_throughput(10.0, 64, 100, 1)
    assert max_ms == 10.0 and abs(value - 64 * 100 / 10e-3) < 1e-6

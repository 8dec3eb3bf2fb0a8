#!/usr/bin/env python
"""Benchmark of the tree-verify attention hot path (mask build + tree attention + split-KV combine).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2] [--no-per-config]

Prints ONE JSON line.  A step is one pass of the whole hot path over one synthetic batch (default:
config 5, the ragged batch of 8 Llama2-70B-shaped requests, the largest single-GPU workload).  Inputs
are resident in HBM; between steps the path rotates through enough independent copies of (Q, K, V, out)
that no step finds its inputs in L2.  `roofline` grades the attention call by its ISOLATED duration (one
call at a time on an idle GPU, cold inputs, median) and carries, in `per_config`, the same figures for
all five configs next to the back-to-back ones (in which consecutive calls overlap).  `e2e` repeats the
measurement with host buffers (pinned), copies inside the timed region.  `--impl reference` times the
fp64 CPU oracle instead (rank 0 only).  With N > 1 (torchrun) every rank runs an independent replica:
the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree_verify_attention_tree_tokens_per_s"
UNIT = "tree tokens/s"
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (tree_attn_small_c2_*.md, tree_attn_tc_c3_*.md, ..._c4_*.md, ..._c5_*.md)
NCU_TRAFFIC_BYTES = {"c2_llama2_7b_L1024_n64": 18411264, "c3_llama2_7b_L4096_n256": 77289216,
                     "c4_llama2_70b_L2048_n512": 18981120, "c5_ragged8_llama2_70b": 154391040}
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def algorithmic_cost(w, words_per_row):
    """Bytes: K and V once, Q in, O out, mask rows.  Flops: 4*D per visible (query, key) pair per head."""
    D, hq, hkv = w.head_dim, w.n_q_heads, w.n_kv_heads
    rows = int((w.prefix_len.astype(np.int64) + w.n_nodes).sum())
    n = w.total_nodes
    nbytes = 2 * rows * hkv * D * 2 + 2 * n * hq * D * 2 + n * words_per_row * 4
    pairs = 0
    for L, p in zip(w.prefix_len, w.parents):
        depth = np.zeros(len(p), dtype=np.int64)
        for i in range(len(p)):
            depth[i] = 0 if p[i] < 0 else depth[p[i]] + 1
        pairs += int((int(L) + depth + 1).sum())
    flops = 4 * hq * D * pairs
    return nbytes, flops


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def lines(self):
        try:
            with open(self.file.name) as f:
                return [ln.strip() for ln in f if ln.strip()]
        except Exception:
            return []

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
        lines = self.lines()
        try:
            os.unlink(self.file.name)
        except Exception:
            pass
        return lines

    @staticmethod
    def summarise(lines, note=""):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "note": "nvidia-smi gave no samples"}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "note": note}


def whole_job_throughput(local_ms, units_per_step_per_rank, steps, world, dist=None, device="cpu"):
    """Replicas: every rank runs the same workload; the job's time is the slowest rank's, its work the
    sum over ranks.  `dist` = torch.distributed (initialised) when world > 1.  Returns (value, max_ms)."""
    import torch
    ms = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    if dist is not None and world > 1:
        dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    max_ms = float(ms.item())
    return units_per_step_per_rank * world * steps / (max_ms * 1e-3), max_ms


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        n = 1
    try:
        n = min(n, len(os.sched_getaffinity(0)))
    except Exception:
        pass
    return n


def time_oracle(w, budget_s=12.0, max_passes=20):
    """The oracle as it stands on this workload: whole passes (mask + attention) until ~budget_s is used."""
    from oracle import dyspec_oracle as orc
    W = 4 * ((max(int(w.n_nodes.max()), 1) + 127) // 128)
    times = []
    t_start = time.perf_counter()
    while len(times) < max_passes and (not times or time.perf_counter() - t_start < budget_s):
        t0 = time.perf_counter()
        orc.build_tree_mask_ragged(w.parents, W)
        orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        times.append(time.perf_counter() - t0)
    return times


def time_oracle_request(w, r):
    """The oracle on ONE request of the batch (mask + attention): the bounded sample the reference arm
    takes per step.  Requests are independent, so the batch's time is the sum over its requests."""
    from oracle import dyspec_oracle as orc
    W = 4 * ((max(int(w.n_nodes.max()), 1) + 127) // 128)
    t0 = time.perf_counter()
    orc.build_tree_mask_ragged([w.parents[r]], W)
    n0 = int(w.node_offsets[r])
    n = int(w.n_nodes[r])
    orc.tree_attention_ragged(w.q[n0:n0 + n], w.k, w.v, w.prefix_len[r:r + 1], w.n_nodes[r:r + 1], w.kv_row_offset[r:r + 1],
                              [w.parents[r]])
    return time.perf_counter() - t0, n


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    from paper_2410_11744_b200 import workloads
    w = workloads.make_config(args.config)
    n_warm = min(args.warmup, 2)
    for i in range(n_warm):
        time_oracle_request(w, i % w.n_req)
    steps = max(1, args.steps)
    budget = 150.0
    secs, toks = [], []
    t_begin = time.perf_counter()
    for i in range(steps):
        sec, n = time_oracle_request(w, i % w.n_req)      # one request per step, round robin over the batch
        secs.append(sec)
        toks.append(n)
        if time.perf_counter() - t_begin > budget:
            break
    value = sum(toks) / sum(secs)
    cores = oracle_threads()
    sample = (f"{len(secs)} steps, each the oracle (mask + attention) on one request of {w.name}, round robin over its "
              f"{w.n_req} request(s); value = tree tokens of the sampled requests / their time")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": len(secs),
        "warmup": n_warm, "ms_per_step": sum(secs) / len(secs) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "fp64 numpy oracle; " + sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def _graph_of(torch, fn):
    """Capture `fn` (which only enqueues library calls on the current stream) into a CUDA graph."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g


def _time_replays(torch, graph, replays, tail=None):
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(replays):
        graph.replay()
    if tail is not None:
        tail()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


ROOFLINE_MIN_CALLS = 240      # calls per back-to-back figure, whatever --steps is
ISOLATED_CALLS = 64           # single calls timed one at a time (the first 8 are dropped)


def _median(xs):
    return float(statistics.median(xs))


def measure_config(torch, runner, w, steps, warmup, device, sparse=False, paged=None, isolated=True):
    """Device-resident timing of exactly `steps` steps, rotating over independent copies of the inputs
    that together exceed 2x L2.  The launch sequence of one rotation is captured in a CUDA graph so
    that the host's launch overhead (python, ctypes) does not starve the GPU.

    Besides the step time it measures the attention call three ways, each with its own repeat count
    (independent of `steps`):
      chain      calls on independent buffers back to back; consecutive calls overlap (programmatic
                 dependent launch), so this is a period, not a duration;
      dependent  the same chain with a tiny ordinary kernel after every call, which serialises the
                 stream the way the next layer's GEMM does (the tiny kernel's own period is subtracted);
      isolated   one call at a time: a kernel that only spins (no memory traffic, ~50 us) keeps the GPU busy
                 while the host enqueues an event, the single attention call and an event behind it, so
                 the host's launch latency is not in the figure; nothing else is on the GPU while the call
                 runs, and its inputs are cold (calls rotate over the buffer copies).  Median of the
                 calls: the duration the roofline fraction is graded on.
    The back-to-back figures are taken in five interleaved rounds (step, attention, mask, ...) and
    reported as medians, so that a clock or power state that drifts during the run hits all alike."""
    first = runner.DeviceBatch(w, device=device, sparse=sparse, paged=paged)
    nbytes, flops = algorithmic_cost(w, first.W)
    copies = max(2, min(64, int(np.ceil(2.0 * L2_BYTES / max(nbytes, 1)))))
    batches = [first] + [runner.DeviceBatch(w, device=device, plan=first.plan, sparse=sparse, paged=paged)
                         for _ in range(copies - 1)]
    info = first.plan.describe()
    launches_per_step = 1 + 1 + (1 if info["split_groups"] > 0 and info.get("combine_launch", 1) else 0)
    for i in range(max(warmup, 3)):
        batches[i % copies].step()
    torch.cuda.synchronize()
    tick = torch.zeros(32, dtype=torch.float32, device=device)

    def attn_then_tick():
        for b in batches:
            b.attention()
            tick.add_(1.0)

    g_step = _graph_of(torch, lambda: [b.step() for b in batches])
    g_attn = _graph_of(torch, lambda: [b.attention() for b in batches])
    g_mask = _graph_of(torch, lambda: [b.build_mask() for b in batches])
    g_dep = _graph_of(torch, attn_then_tick)
    g_tick = _graph_of(torch, lambda: [tick.add_(1.0) for _ in batches])
    for g in (g_step, g_attn, g_mask, g_dep, g_tick):
        g.replay()
    torch.cuda.synchronize()
    replays, rem = divmod(steps, copies)
    total_ms = _time_replays(torch, g_step, replays, tail=lambda: [batches[i].step() for i in range(rem)])
    # ---- the attention call and the mask builder by themselves: own repeat count, interleaved rounds
    rounds = 5
    r2 = max(1, int(np.ceil(ROOFLINE_MIN_CALLS / (rounds * copies))))
    per = {"step": [], "attn": [], "mask": [], "dep": [], "tick": []}
    for _ in range(rounds):
        for key, g in (("step", g_step), ("attn", g_attn), ("mask", g_mask), ("dep", g_dep), ("tick", g_tick)):
            per[key].append(_time_replays(torch, g, r2) / (r2 * copies))
    step_chain_ms, attn_ms, mask_ms = _median(per["step"]), _median(per["attn"]), _median(per["mask"])
    dep_ms = max(_median(per["dep"]) - _median(per["tick"]), 0.0)
    # ---- one call at a time
    iso_ms = None
    if isolated:
        stream = torch.cuda.current_stream()
        ts = []
        for i in range(ISOLATED_CALLS):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            torch.cuda._sleep(100000)       # ~50 us of spinning: the three enqueues below land while it runs
            e0.record(stream)
            batches[i % copies].attention()
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        iso_ms = _median(ts[8:])
    status = int(first.status.item())
    return dict(batches=batches, total_ms=total_ms, ms_per_step=total_ms / steps, step_chain_ms=step_chain_ms,
                attn_ms=attn_ms, mask_ms=mask_ms, dep_ms=dep_ms, iso_ms=iso_ms, chain_calls=rounds * r2 * copies,
                bytes=nbytes, flops=flops, copies=copies, info=info, launches_per_step=launches_per_step, status=status,
                graph=g_step)


def isolated_floor(torch):
    """What the isolated protocol reads for a kernel that does nothing, and for no kernel at all: the same
    spin kernel, events and median as in measure_config, around torch's one-cycle spin kernel and around
    nothing.  Context for the isolated durations (every one of them contains this much launch and event
    latency); the graded figures are not corrected by it."""
    stream = torch.cuda.current_stream()
    out = {}
    for label, fn in (("empty_kernel_us", lambda: torch.cuda._sleep(1)), ("event_pair_us", lambda: None)):
        ts = []
        for _ in range(ISOLATED_CALLS):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            torch.cuda._sleep(100000)
            e0.record(stream)
            fn()
            e1.record(stream)
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        out[label] = _median(ts[8:]) * 1e3
    return out


def random_tree_experiment(torch, runner, workloads, B, peaks, device, sizes=(256, 512, 1024, 2048), steps=200):
    """The paper's random-tree attention experiment (App. C.1, Table 5: one request, 64 heads x 128,
    no prefix, uniform random recursive trees): block counts and attention time in creation order
    (dense call) and after the GPU's DFS renumbering with empty tree tiles skipped."""
    rows = []
    for n in sizes:
        w = workloads.make_random_tree_case(n)
        probe = runner.DeviceBatch(w, device=device)
        order, _, new_parents = probe.dfs_reorder()
        w2 = workloads.permute_tree_tokens(w, [order], [new_parents])
        count = torch.zeros(1, dtype=torch.int64, device=device)
        blocks = []
        for batch in (probe, runner.DeviceBatch(w2, device=device, plan=probe.plan)):
            batch.build_mask()
            B.dyspec_mask_block_count(batch.bits, n, batch.W, 32, count)
            torch.cuda.synchronize()
            blocks.append(int(count.item()))
        # the reorder kernel alone, from resident parents
        order_d = torch.empty(n, dtype=torch.int32, device=device)
        newp_d = torch.empty(n, dtype=torch.int32, device=device)
        g_re = _graph_of(torch, lambda: [B.dyspec_plan_dfs_reorder(probe.plan, probe.parents, order_d, None, newp_d, None)
                                         for _ in range(20)])
        g_re.replay()
        torch.cuda.synchronize()
        reorder_us = _time_replays(torch, g_re, 10) / 200 * 1e3
        del probe
        m1 = measure_config(torch, runner, w, steps, 3, device)
        m2 = measure_config(torch, runner, w2, steps, 3, device, sparse=True)
        t_hbm_us = m1["bytes"] / (peaks["hbm_gbs"] * 1e9) * 1e6
        rows.append({"tree_size": n, "workload": w.name, "blocks32": {"creation_order": blocks[0], "dfs_order": blocks[1]},
                     "attention_call_us": {"creation_order_dense": m1["attn_ms"] * 1e3,
                                           "dfs_order_skipping": m2["attn_ms"] * 1e3},
                     "attention_call_isolated_us": {"creation_order_dense": m1["iso_ms"] * 1e3,
                                                    "dfs_order_skipping": m2["iso_ms"] * 1e3},
                     "mask_us": {"plain": m1["mask_ms"] * 1e3, "with_tile_sets": m2["mask_ms"] * 1e3},
                     "reorder_us": reorder_us, "bytes": m1["bytes"], "hbm_floor_us": t_hbm_us,
                     "frac_of_hbm_floor": {"creation_order_dense": t_hbm_us / (m1["attn_ms"] * 1e3),
                                           "dfs_order_skipping": t_hbm_us / (m2["attn_ms"] * 1e3)},
                     "plan": m1["info"], "status": [m1["status"], m2["status"]]})
        del m1, m2
        torch.cuda.empty_cache()
    return rows


def verification_experiment(torch, workloads, B, peaks, device):
    """Tree verification (Algorithm 3) on the device: Llama2 vocabulary (32000), the 64-node tree shape of
    config 2 for one request (the paper's batch size) and a batch of 8 requests with 256-node trees.
    Inputs rotate over copies that exceed 2x L2; algorithmic bytes = the draft and target rows of the
    visited nodes."""
    rows = []
    rng = np.random.default_rng(workloads.MASTER_SEED + 7000)
    tree64 = [workloads.greedy_tree(rng, 64, 8, 0.3)]
    for label, trees, disagreement in (
            ("1 request, 64 nodes", tree64, 1.0),
            ("8 requests, 256 nodes", [workloads.greedy_tree(rng, 256, 8, 0.1) for _ in range(8)], 1.0),
            # a draft close to the target (the regime speculative decoding is run in): first branches are accepted
            # and the walk needs two numbers per node instead of two rows
            ("1 request, 64 nodes, draft close to target", tree64, 0.05)):
        case = workloads.make_verify_case(workloads.MASTER_SEED + 7001, 32000, trees, sharpness=3.0, disagreement=disagreement)
        n_req = len(trees)
        N = int(case.node_offsets[-1])
        row_bytes = 2 * N * case.vocab * 4
        copies = max(2, min(32, int(np.ceil(2.0 * L2_BYTES / row_bytes))))
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
        parents, tokens = t(np.concatenate(case.parents)), t(np.concatenate(case.tokens))
        offs, au, su = t(case.node_offsets), t(case.accept_u), t(case.sample_u)
        bufs = [(t(case.draft_probs), t(case.target_probs)) for _ in range(copies)]
        out_t = torch.zeros((n_req, 64), dtype=torch.int32, device=device)
        out_n = torch.zeros((n_req, 64), dtype=torch.int32, device=device)
        cnt = torch.zeros((n_req,), dtype=torch.int32, device=device)
        status = torch.zeros(1, dtype=torch.int32, device=device)
        max_nodes = max(len(p) for p in trees)

        def call(d, tg):
            B.dyspec_verify_tree(parents, tokens, d, tg, au, su, offs, n_req, max_nodes, case.vocab, out_t, out_n, cnt, 64,
                                 bonus_at_leaf=True, status=status)
        for d, tg in bufs:
            call(d, tg)
        torch.cuda.synchronize()
        g = _graph_of(torch, lambda: [call(d, tg) for d, tg in bufs])
        g.replay()
        torch.cuda.synchronize()
        us = _time_replays(torch, g, 20) / (20 * copies) * 1e3
        emitted = cnt.cpu().numpy()
        visited = int(emitted.sum())                       # an upper bound of the nodes whose rows were read (a node whose first branch
                                                           # is accepted reads two numbers, not its rows)
        nbytes = visited * 2 * case.vocab * 4
        rows.append({"case": label, "vocab": case.vocab, "call_us": us, "us_per_token": us / max(1, int(emitted.max())),
                     "tokens_emitted": emitted.tolist(),
                     "rows_read_at_most": visited, "bytes_at_most": nbytes, "achieved_gbs": nbytes / (us * 1e-6) / 1e9,
                     "frac_of_hbm": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"], "copies": copies,
                     "status": int(status.item())})
        del bufs
        torch.cuda.empty_cache()
    return rows


def construction_experiment(torch, workloads, B, peaks, device):
    """Tree construction (Algorithms 1 and 2) on the device over the table-lookup draft model: vocabulary
    32000, 64 language-model-like (Zipf) table rows; the paper's two tree sizes (64 and 768 guesses) for one request, and the
    threshold form at the value of the greedy tree's last node.  Algorithmic bytes = one draft row
    (vocab * 4) per guess (greedy) or per expanded position (threshold)."""
    rows_np, uni_np = workloads.make_draft_table(workloads.MASTER_SEED + 8000, 64, 32000, zipf=True)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(device)
    rows, uni = t(rows_np), t(uni_np)
    root = torch.zeros(1, dtype=torch.int32, device=device)
    out = []
    for m in (64, 768):
        S = m + 1
        bufs = [torch.zeros((1, S), dtype=torch.int32, device=device) for _ in range(3)]
        vals = [torch.zeros((1, S), dtype=torch.float32, device=device) for _ in range(2)]
        cnt = torch.zeros(1, dtype=torch.int32, device=device)
        greedy = lambda: B.dyspec_build_tree_greedy(rows, 64, 32000, uni, len(uni_np), root, 1, m, bufs[0], bufs[1], vals[0],
                                                    vals[1], bufs[2], cnt)
        greedy()
        torch.cuda.synchronize()
        thr = float(vals[0][0, m].item())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(5):
            greedy()
        e1.record()
        torch.cuda.synchronize()
        g_us = e0.elapsed_time(e1) / 5 * 1e3
        parents = bufs[0][0].cpu().numpy()
        cap = 4 * m if 4 * m < 2047 else 2047
        tb = [torch.zeros((1, cap + 1), dtype=torch.int32, device=device) for _ in range(3)]
        tv = [torch.zeros((1, cap + 1), dtype=torch.float32, device=device) for _ in range(2)]
        layered = lambda: B.dyspec_build_tree_threshold(rows, 64, 32000, uni, len(uni_np), root, 1, thr, cap, tb[0], tb[1],
                                                        tv[0], tv[1], tb[2], cnt)
        layered()
        torch.cuda.synchronize()
        n_thr = int(cnt.item()) - 1
        e0.record()
        for _ in range(5):
            layered()
        e1.record()
        torch.cuda.synchronize()
        t_us = e0.elapsed_time(e1) / 5 * 1e3
        tp = tb[0][0, :n_thr + 1].cpu().numpy()
        positions = len(set(int(x) for x in tp[1:]))
        depth = np.zeros(m + 1, int)
        for k in range(1, m + 1):
            depth[k] = depth[parents[k]] + 1
        out.append({"guesses": m, "vocab": 32000, "greedy_us": g_us, "greedy_us_per_guess": g_us / m,
                    "greedy_gbs": m * 32000 * 4 / (g_us * 1e-6) / 1e9, "depth": int(depth.max()),
                    "threshold": thr, "threshold_guesses": n_thr, "threshold_positions": positions, "threshold_us": t_us,
                    "threshold_gbs": positions * 32000 * 4 / (t_us * 1e-6) / 1e9})
    return out


def compaction_experiment(torch, B, peaks, device):
    """Accepted-path KV compaction: 8 accepted nodes per request, Llama2-7B rows (32 x 128 bf16 = 8 KB) for
    1 request and Llama2-70B rows (8 x 128 = 2 KB) for a batch of 64; algorithmic bytes = rows moved x 2
    (read + write) x 2 (K and V)."""
    out = []
    for label, n_req, hkv in (("1 request, 32 kv heads", 1, 32), ("64 requests, 8 kv heads", 64, 8)):
        d, L, n, max_out = 128, 1024, 64, 16
        rows = n_req * (L + n)
        k = torch.zeros((rows, hkv, d), dtype=torch.bfloat16, device=device)
        v = torch.zeros((rows, hkv, d), dtype=torch.bfloat16, device=device)
        offs = torch.arange(n_req, dtype=torch.int64, device=device) * (L + n)
        Ls = torch.full((n_req,), L, dtype=torch.int32, device=device)
        acc = torch.tensor([[1, 4, 9, 17, 22, 30, 41, 55, -1] + [0] * (max_out - 9)] * n_req, dtype=torch.int32, device=device)
        cnt = torch.full((n_req,), 9, dtype=torch.int32, device=device)
        newL = torch.zeros(n_req, dtype=torch.int32, device=device)
        call = lambda: B.dyspec_compact_kv(k, v, offs, Ls, acc, cnt, n_req, max_out, hkv, d, newL)
        call()
        torch.cuda.synchronize()
        g = _graph_of(torch, lambda: [call() for _ in range(20)])
        g.replay()
        torch.cuda.synchronize()
        us = _time_replays(torch, g, 20) / 400 * 1e3
        nbytes = n_req * 8 * hkv * d * 2 * 2 * 2
        out.append({"case": label, "call_us": us, "bytes": nbytes, "achieved_gbs": nbytes / (us * 1e-6) / 1e9,
                    "frac_of_hbm": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]})
    return out


def paged_experiment(torch, runner, workloads, B, peaks, device, configs=(2, 3, 4, 5), page_size=256, steps=400):
    """The same step with the cache in shuffled pages of page_size rows beside the contiguous layout: prefix
    through a page table and tree rows in a run of their own ("paged"), and prefix and tree rows both in the
    pages ("in_sequence": key tiles follow the sequence, mask slices are shifted by L modulo the tile size;
    configs 2 - 4 have L on a tile boundary, the ragged batch does not).  Same algorithmic bytes, so the
    times should agree.  After it, the paged accepted-path compaction (8 accepted nodes, 64 requests)."""
    out = {"page_size": page_size, "configs": []}
    for idx in configs:
        w = workloads.make_config(idx)
        mc = measure_config(torch, runner, w, steps, 3, device, isolated=False)
        t_c = (mc["step_chain_ms"], mc["attn_ms"])
        del mc
        torch.cuda.empty_cache()
        mp = measure_config(torch, runner, w, steps, 3, device, paged=workloads.to_paged(w, page_size, idx), isolated=False)
        entry = {"config": idx, "workload": w.name, "contiguous_step_us": t_c[0] * 1e3,
                 "contiguous_attention_us": t_c[1] * 1e3, "paged_step_us": mp["step_chain_ms"] * 1e3,
                 "paged_attention_us": mp["attn_ms"] * 1e3, "bytes": mp["bytes"], "status": mp["status"]}
        del mp
        torch.cuda.empty_cache()
        ms = measure_config(torch, runner, w, steps, 3, device,
                            paged=workloads.to_paged(w, page_size, idx, tree_in_pages=True), isolated=False)
        entry.update({"in_sequence_step_us": ms["step_chain_ms"] * 1e3, "in_sequence_attention_us": ms["attn_ms"] * 1e3,
                      "in_sequence_status": ms["status"]})
        out["configs"].append(entry)
        del ms
        torch.cuda.empty_cache()
    n_req, hkv, d, L, n, max_out = 64, 8, 128, 1024, 64, 16
    pages_per_req = (L + n + page_size - 1) // page_size
    n_pages = n_req * pages_per_req
    rows = n_pages * page_size + n_req * n
    k = torch.zeros((rows, hkv, d), dtype=torch.bfloat16, device=device)
    v = torch.zeros((rows, hkv, d), dtype=torch.bfloat16, device=device)
    table = torch.randperm(n_pages, device=device).to(torch.int32).reshape(n_req, pages_per_req).contiguous()
    tree0 = n_pages * page_size + torch.arange(n_req, dtype=torch.int64, device=device) * n
    Ls = torch.full((n_req,), L, dtype=torch.int32, device=device)
    acc = torch.tensor([[1, 4, 9, 17, 22, 30, 41, 55, -1] + [0] * (max_out - 9)] * n_req, dtype=torch.int32, device=device)
    cnt = torch.full((n_req,), 9, dtype=torch.int32, device=device)
    newL = torch.zeros(n_req, dtype=torch.int32, device=device)
    call = lambda: B.dyspec_compact_kv_paged(k, v, tree0, table, pages_per_req, page_size, Ls, acc, cnt, n_req, max_out,
                                             hkv, d, newL)
    call()
    torch.cuda.synchronize()
    g = _graph_of(torch, lambda: [call() for _ in range(20)])
    g.replay()
    torch.cuda.synchronize()
    us = _time_replays(torch, g, 20) / 400 * 1e3
    nbytes = n_req * 8 * hkv * d * 2 * 2 * 2
    out["compaction"] = {"case": "64 requests, 8 kv heads, 8 accepted nodes", "call_us": us, "bytes": nbytes,
                         "achieved_gbs": nbytes / (us * 1e-6) / 1e9}
    # the same move with the tree rows inside the pages (node a = token L + a): in place
    call = lambda: B.dyspec_compact_kv_paged(k, v, None, table, pages_per_req, page_size, Ls, acc, cnt, n_req, max_out,
                                             hkv, d, newL)
    call()
    torch.cuda.synchronize()
    g = _graph_of(torch, lambda: [call() for _ in range(20)])
    g.replay()
    torch.cuda.synchronize()
    out["compaction"]["in_place_call_us"] = _time_replays(torch, g, 20) / 400 * 1e3
    return out


def small_tree_batch_experiment(torch, runner, workloads, peaks, device, steps=100):
    """The small-tree regime at a size where its rate, not its latency, shows: 8 requests of the Llama2-7B
    shape (32 heads x 128, 64-node greedy trees as in config 2) over 4096-token prefixes, and a ragged batch
    of 16 requests (prefix 200 - 3000, 32-node trees).  HBM-bound: achieved bytes/s against the measured copy peak."""
    rng = np.random.default_rng(workloads.MASTER_SEED + 77)
    cases = [
        ("8 requests, 32 heads, prefix 4096, 64-node trees",
         workloads.make_custom(1, 32, 32, 128, [4096] * 8, [workloads.greedy_tree(rng, 64, 8, 0.3) for _ in range(8)])),
        ("16 requests, 32 heads, prefix 200-3000, 32-node trees",
         workloads.make_custom(3, 32, 32, 128, [int(x) for x in rng.integers(200, 3000, 16)],
                               [workloads.greedy_tree(rng, 32, 8, 0.3) for _ in range(16)])),
    ]
    out = []
    for label, w in cases:
        m = measure_config(torch, runner, w, steps, 3, device, isolated=False)
        gbs = m["bytes"] / (m["attn_ms"] * 1e-3) / 1e9
        out.append({"case": label, "tree_tokens": w.total_nodes, "attention_call_us": m["attn_ms"] * 1e3,
                    "step_us": m["step_chain_ms"] * 1e3, "bytes": m["bytes"], "achieved_gbs": gbs,
                    "frac_of_hbm": gbs / peaks["hbm_gbs"], "plan": m["info"], "status": m["status"]})
        del m
        torch.cuda.empty_cache()
    return out


def roofline_entry(m, peaks, peaks_kind):
    """Roofline of one attention call: t_roof = max(bytes / HBM, flops / bf16 peak); the graded
    duration is the isolated one (falls back to the back-to-back period when that was not taken)."""
    t_hbm = m["bytes"] / (peaks["hbm_gbs"] * 1e9)
    t_tc = m["flops"] / (peaks["bf16_tflops"] * 1e12)
    graded = "isolated" if m.get("iso_ms") else "chain"
    dur = (m["iso_ms"] if graded == "isolated" else m["attn_ms"]) * 1e-3
    chain = m["attn_ms"] * 1e-3
    # nominal figures (HGX B200: 8 TB/s HBM3e as the workload definition quotes it, 2.25 PFLOP/s dense bf16): context only
    common = {"traffic": None, "kernel": "tree attention call (main kernel + any combine launch)",
              "duration": graded + (": one call alone on the GPU (cold inputs), events around it, median of %d" % (ISOLATED_CALLS - 8)
                                    if graded == "isolated" else ": back-to-back period"),
              "launch_us": dur * 1e6, "chain_us": chain * 1e6, "dependent_chain_us": m["dep_ms"] * 1e3,
              "chain_note": "back-to-back calls on independent buffers overlap (programmatic dependent launch): a period, "
                            "not a duration; dependent_chain = the same with a serialising tiny kernel after every call",
              "bytes": m["bytes"], "flops": m["flops"], "roof_us": max(t_hbm, t_tc) * 1e6}
    if t_hbm >= t_tc:
        ach = m["bytes"] / dur / 1e9
        common.update({"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                       "frac_chain": m["bytes"] / chain / 1e9 / peaks["hbm_gbs"], "peak_kind": peaks_kind,
                       "frac_of_nominal": ach / NOMINAL_HBM_GBS, "nominal_peak": NOMINAL_HBM_GBS})
        return common
    ach = m["flops"] / dur / 1e12
    common.update({"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                   "frac": ach / peaks["bf16_tflops"], "frac_chain": m["flops"] / chain / 1e12 / peaks["bf16_tflops"],
                   "peak_kind": peaks_kind + " (burst)",
                   "frac_of_sustained": ach / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                   "frac_of_nominal": ach / NOMINAL_BF16_TFLOPS, "nominal_peak": NOMINAL_BF16_TFLOPS})
    return common


def compact_roofline(idx, wi, mi, ri):
    """One per-config entry of roofline.per_config: everything needed to recompute the fraction by hand."""
    return {"config": idx, "workload": wi.name, "bound": ri["bound"], "bytes": mi["bytes"], "flops": mi["flops"],
            "roof_us": ri["roof_us"], "isolated_us": None if mi["iso_ms"] is None else mi["iso_ms"] * 1e3,
            "chain_us": mi["attn_ms"] * 1e3, "dependent_chain_us": mi["dep_ms"] * 1e3, "frac": ri["frac"],
            "traffic": NCU_TRAFFIC_BYTES.get(wi.name),
            "frac_chain": ri["frac_chain"], "graded_on": ri["duration"].split(":")[0]}


def run_ours(args):
    import torch
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback for the CUDA path)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2410_11744_b200 import build as _build
    if rank == 0:
        _build.build()
    if use_dist:
        dist.barrier()
    from paper_2410_11744_b200 import runner, workloads

    peaks, peaks_kind = load_peaks()
    w = workloads.make_config(args.config)
    sampler = ClockSampler(local) if rank == 0 else None

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident measurement (the headline `value`)
    barrier()
    m = measure_config(torch, runner, w, args.steps, args.warmup, device)
    barrier()
    n_lines_after_timed = len(sampler.lines()) if sampler else 0
    value, total_ms = whole_job_throughput(m["total_ms"], w.total_nodes, args.steps, world, dist if use_dist else None, device)
    tokens_per_step = w.total_nodes * world

    # ---- clocks: the timed region can be shorter than one nvidia-smi period; if so keep the same
    #      loop running (untimed) until a few samples exist, and say so.
    clocks_note = "sampled during warm-up + timed region"
    if sampler:
        if n_lines_after_timed < 4:
            t_end = time.time() + 1.0
            while time.time() < t_end:
                for i in range(200):
                    m["graph"].replay()
                torch.cuda.synchronize()
            clocks_note = "timed region shorter than the sampling period: sampled while the same loop kept running"
        clocks = ClockSampler.summarise(sampler.lines(), clocks_note)
    else:
        clocks = None

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    b0 = m["batches"][0]
    host_in = [t.cpu().pin_memory() for t in (b0.parents, b0.q, b0.k, b0.v)]
    host_out = torch.empty_like(b0.out, device="cpu").pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = host_out.numel() * host_out.element_size()
    e2e_steps = max(3, min(args.steps, 200))
    stream = torch.cuda.current_stream()

    def e2e_step(b):
        b.parents.copy_(host_in[0], non_blocking=True)
        b.q.copy_(host_in[1], non_blocking=True)
        b.k.copy_(host_in[2], non_blocking=True)
        b.v.copy_(host_in[3], non_blocking=True)
        b.step()
        host_out.copy_(b.out, non_blocking=True)
        stream.synchronize()

    for i in range(3):
        e2e_step(m["batches"][i % m["copies"]])
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(e2e_steps):
        e2e_step(m["batches"][i % m["copies"]])
    e1.record(stream)
    torch.cuda.synchronize()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)
    e2e_value, _ = whole_job_throughput(e2e_ms, w.total_nodes, e2e_steps, world, dist if use_dist else None, device)

    if rank != 0:
        if use_dist:
            dist.barrier()
            dist.destroy_process_group()
        return

    roof = roofline_entry(m, peaks, peaks_kind)
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(w.name)
    # the same call on ONE buffer set over and over: inputs stay in L2 (not the graded number)
    b_warm = m["batches"][0]
    g_warm = _graph_of(torch, lambda: [b_warm.attention() for _ in range(20)])
    g_warm.replay()
    torch.cuda.synchronize()
    warm_us = _time_replays(torch, g_warm, 20) / 400 * 1e3
    del g_warm

    # ---- all five configs, same protocol: compact entries inside `roofline`, the longer ones in `per_config`
    per_config, roof_rows = [], []
    if not args.no_per_config:
        for idx in (1, 2, 3, 4, 5):
            wi = w if idx == args.config else workloads.make_config(idx)
            mi = m if idx == args.config else measure_config(torch, runner, wi, 60, 3, device)
            ri = roofline_entry(mi, peaks, peaks_kind)
            roof_rows.append(compact_roofline(idx, wi, mi, ri))
            per_config.append({"config": idx, "workload": wi.name, "tree_tokens": wi.total_nodes,
                               "step_us": mi["step_chain_ms"] * 1e3, "attention_call_us": mi["attn_ms"] * 1e3,
                               "attention_call_isolated_us": mi["iso_ms"] * 1e3, "mask_us": mi["mask_ms"] * 1e3,
                               "tokens_per_s": wi.total_nodes / (mi["step_chain_ms"] * 1e-3),
                               "bytes": mi["bytes"], "flops": mi["flops"], "bound": ri["bound"], "achieved": ri["achieved"],
                               "unit": ri["unit"], "frac": ri["frac"], "plan": mi["info"], "status": mi["status"]})
            if idx != args.config:
                del mi["batches"], mi["graph"]
                torch.cuda.empty_cache()
    else:
        roof_rows.append(compact_roofline(args.config, w, m, roof))
    roof["per_config"] = roof_rows
    roof["isolated_floor"] = isolated_floor(torch)

    random_tree = None
    if not args.no_per_config and world == 1:
        from paper_2410_11744_b200 import binding
        random_tree = random_tree_experiment(torch, runner, workloads, binding, peaks, device)

    verification = None
    if not args.no_per_config and world == 1:
        verification = verification_experiment(torch, workloads, binding, peaks, device)

    construction = None
    if not args.no_per_config and world == 1:
        construction = construction_experiment(torch, workloads, binding, peaks, device)

    compaction = None
    if not args.no_per_config and world == 1:
        compaction = compaction_experiment(torch, binding, peaks, device)

    paged = None
    if not args.no_per_config and world == 1:
        paged = paged_experiment(torch, runner, workloads, binding, peaks, device)

    small_batch = None
    if not args.no_per_config and world == 1:
        small_batch = small_tree_batch_experiment(torch, runner, workloads, peaks, device)

    # ---- the oracle on the host cores, bounded sample of the same workload
    times = time_oracle(w, budget_s=12.0)
    cpu_sec = sum(times) / len(times)
    cpu_baseline = {"value": w.total_nodes / cpu_sec, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                    "sample": f"{len(times)} full passes (mask + attention) of {w.name}, {cpu_sec * 1e3:.1f} ms each"}
    # parity of the timed configuration against the oracle (whole output, one more oracle pass)
    parity = None
    try:
        from oracle import dyspec_oracle as orc
        b_par = m["batches"][0]
        b_par.step()
        bits_g, depths_g, out_g, st_g = b_par.results()
        ref_bits, ref_depths = orc.build_tree_mask_ragged(w.parents, b_par.W)
        ref = orc.tree_attention_ragged(w.q, w.k, w.v, w.prefix_len, w.n_nodes, w.kv_row_offset, w.parents)
        err = np.abs(orc.bf16_bits_to_f64(out_g) - ref)
        parity = {"mask_bit_exact": bool(np.array_equal(bits_g, ref_bits)), "depths_exact": bool(np.array_equal(depths_g, ref_depths)),
                  "attention_max_abs_err": float(err.max()), "attention_mean_abs_err": float(err.mean()),
                  "tolerance": {"max_abs": 2e-2, "mean_abs": 2e-3}, "device_status": st_g}
    except Exception as e:                # the measurement stands without it
        parity = {"error": repr(e)}
    try:                                  # the same on one thread (the oracle's only parallelism is its BLAS calls),
        from threadpoolctl import threadpool_limits   # on the batch's smallest request so that it stays bounded
        r_small = int(np.argmin(w.n_nodes.astype(np.int64) * (w.prefix_len.astype(np.int64) + w.n_nodes)))
        with threadpool_limits(limits=1):
            sec1, n1 = time_oracle_request(w, r_small)
        cpu_baseline["value_1_thread"] = n1 / sec1
        cpu_baseline["sample_1_thread"] = f"request {r_small} of the batch ({n1} tree tokens), one pass"
    except Exception:
        pass

    if sampler:
        sampler.stop()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads, "head_dim": w.head_dim,
                   "prefix_len": w.prefix_len.tolist(), "n_nodes": w.n_nodes.tolist(), "parallelism": "replicas only",
                   "l2": f"inputs rotate over {m['copies']} independent copies ({m['copies'] * m['bytes'] / 1e6:.0f} MB > 2x L2)",
                   "step": "mask build + tree attention (split-KV merge included)", "plan": m["info"]},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": m["launches_per_step"] * args.steps,
        "roofline": roof,
        "cpu_baseline": cpu_baseline,
        "kernel_us": {"mask_build": m["mask_ms"] * 1e3, "attention_call": m["attn_ms"] * 1e3,
                      "attention_call_L2_resident": warm_us, "attention_call_isolated": m["iso_ms"] * 1e3,
                      "attention_call_dependent_chain": m["dep_ms"] * 1e3, "step_back_to_back": m["step_chain_ms"] * 1e3,
                      "calls_per_back_to_back_figure": m["chain_calls"]},
        "device_status": m["status"],
        "parity_vs_oracle": parity,
    }
    if per_config:
        line["per_config"] = per_config
    if random_tree:
        line["random_tree_experiment"] = random_tree
    if verification:
        line["verification_experiment"] = verification
    if construction:
        line["construction_experiment"] = construction
    if compaction:
        line["compaction_experiment"] = compaction
    if paged:
        line["paged_cache_experiment"] = paged
    if small_batch:
        line["small_tree_batch_experiment"] = small_batch
    print(json.dumps(line), flush=True)
    if use_dist:
        dist.barrier()
        dist.destroy_process_group()


def run_profile(args):
    """A short eager run for profilers: no graphs, no timing, no oracle.  --profile-op step (default):
    mask build + attention of --config; sparse: DFS reorder + mask with tile sets + tile-skipping
    attention on the 2048-token random tree; small_batch: the 8-request small-tree batch; verify /
    construct: those kernels on small cases."""
    import torch
    from paper_2410_11744_b200 import build as _build
    _build.build()
    from paper_2410_11744_b200 import binding as B, runner, workloads
    dev = torch.device("cuda", 0)
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    if args.profile_op == "step":
        w = workloads.make_config(args.config)
        first = runner.DeviceBatch(w)
        nbytes, _ = algorithmic_cost(w, first.W)
        copies = max(2, min(8, int(np.ceil(1.2 * L2_BYTES / max(nbytes, 1)))))
        batches = [first] + [runner.DeviceBatch(w, plan=first.plan) for _ in range(copies - 1)]
        for i in range(args.profile):
            batches[i % copies].step()
        torch.cuda.synchronize()
        info = {"workload": w.name, "copies": copies, "plan": first.plan.describe(), "status": int(first.status.item())}
    elif args.profile_op == "small_batch":
        # the first case of small_tree_batch_experiment: 8 requests x 32 heads x 4096 prefix keys x 64-node trees (554 MB)
        rng = np.random.default_rng(workloads.MASTER_SEED + 77)
        w = workloads.make_custom(1, 32, 32, 128, [4096] * 8, [workloads.greedy_tree(rng, 64, 8, 0.3) for _ in range(8)])
        batches = [runner.DeviceBatch(w) for _ in range(2)]
        for i in range(args.profile):
            batches[i % 2].step()
        torch.cuda.synchronize()
        info = {"workload": "8 requests, 32 heads, prefix 4096, 64-node trees", "copies": 2,
                "plan": batches[0].plan.describe(), "status": int(batches[0].status.item())}
    elif args.profile_op == "sparse":
        w = workloads.make_random_tree_case(2048)
        probe = runner.DeviceBatch(w)
        order, _, new_parents = probe.dfs_reorder()
        w2 = workloads.permute_tree_tokens(w, [order], [new_parents])
        batches = [runner.DeviceBatch(w2, plan=probe.plan, sparse=True) for _ in range(2)]     # 2 x 134 MB > L2
        order_d = torch.empty(2048, dtype=torch.int32, device=dev)
        newp_d = torch.empty(2048, dtype=torch.int32, device=dev)
        for i in range(args.profile):
            B.dyspec_plan_dfs_reorder(probe.plan, probe.parents, order_d, None, newp_d, None)
            batches[i % 2].step()
        torch.cuda.synchronize()
        info = {"workload": w2.name, "copies": 2, "plan": probe.plan.describe(), "status": int(batches[0].status.item())}
    elif args.profile_op == "verify":
        rng = np.random.default_rng(workloads.MASTER_SEED + 7000)
        trees = [workloads.greedy_tree(rng, 256, 8, 0.1) for _ in range(8)]
        case = workloads.make_verify_case(workloads.MASTER_SEED + 7001, 32000, trees, sharpness=3.0, disagreement=1.0)
        d, tg = t(case.draft_probs), t(case.target_probs)
        out_t = torch.zeros((8, 64), dtype=torch.int32, device=dev)
        out_n = torch.zeros((8, 64), dtype=torch.int32, device=dev)
        cnt = torch.zeros(8, dtype=torch.int32, device=dev)
        args_ = (t(np.concatenate(case.parents)), t(np.concatenate(case.tokens)), d, tg, t(case.accept_u), t(case.sample_u),
                 t(case.node_offsets), 8, 256, 32000, out_t, out_n, cnt, 64)
        for _ in range(args.profile):
            B.dyspec_verify_tree(*args_, bonus_at_leaf=True)
        torch.cuda.synchronize()
        info = {"workload": "verify 8 requests x 256 nodes, vocab 32000", "emitted": cnt.cpu().numpy().tolist()}
    else:
        rows_np, uni_np = workloads.make_draft_table(workloads.MASTER_SEED + 8000, 64, 32000, zipf=True)
        rows, uni = t(rows_np), t(uni_np)
        root = torch.arange(8, dtype=torch.int32, device=dev)
        m = 64
        bufs = [torch.zeros((8, m + 1), dtype=torch.int32, device=dev) for _ in range(3)]
        vals = [torch.zeros((8, m + 1), dtype=torch.float32, device=dev) for _ in range(2)]
        cnt = torch.zeros(8, dtype=torch.int32, device=dev)
        for _ in range(args.profile):
            B.dyspec_build_tree_greedy(rows, 64, 32000, uni, len(uni_np), root, 8, m, bufs[0], bufs[1], vals[0], vals[1],
                                       bufs[2], cnt)
            B.dyspec_build_tree_threshold(rows, 64, 32000, uni, len(uni_np), root, 8, 0.05, 200, *[
                torch.zeros((8, 201), dtype=(torch.float32 if i in (2, 3) else torch.int32), device=dev) for i in range(5)], cnt)
        torch.cuda.synchronize()
        info = {"workload": "construct 8 requests, 64 guesses, vocab 32000"}
    info.update({"profiled_steps": args.profile, "op": args.profile_op})
    print(json.dumps(info))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--profile", type=int, default=0,
                    help="run only this many plain (eager) steps of --config and exit: the command to put under ncu")
    ap.add_argument("--profile-op", default="step", choices=["step", "sparse", "small_batch", "verify", "construct"])
    args = ap.parse_args()
    if args.profile > 0:
        return run_profile(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

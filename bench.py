#!/usr/bin/env python
"""Benchmark of the ClusterAttention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload tabular|video480|video720|sweep|tiny] [--no-cpu-baseline]

One "step" is one pass of the whole hot path (cluster_qk + select_blocks +
cluster_attention_fwd) over one batch of seeded synthetic input.  The default
workload is the tabular-shaped configuration (8 heads, d=64, bf16, 16,384
queries attending to 131,072 keys, clusters of 128, 1/8 of the key clusters
kept, compensation on).  The metric is the throughput of the whole path in
TFLOP/s over the computed blocks: 4*N_q*d*(keep*c + padded centroid columns)
flops per head divided by the time of the step.

With N > 1 (launched under torch.distributed.run) every rank runs an
independent replica on its own GPU: heads are independent problems and the
path has no exchange step, so there is no collective on the data path.

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same
workload instead.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "clusterattention_hot_path_block_tflops"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# DRAM bytes per launch of the dominant kernel from the ncu captures summarised under profiles/
# (4- and 8-head captures scaled by the head count).  Each figure is tied to the kernel source it
# was captured from: sha256 of csrc/attn_tc.cu + csrc/tc_ptx.cuh, first 16 hex digits.  When the
# source has changed since, the bench prints null instead of a stale figure.
NCU_TRAFFIC = {
    "tabular": {"bytes": 577.2e6, "source": "932f684fa31e5a09", "commit": "3110b1f"},
    "video480": {"bytes": 1264.8e6, "source": "932f684fa31e5a09", "commit": "3110b1f"},
}
# FP32 FMA rate of the CUDA cores, the roof of kernels bound by plain arithmetic (centroid scoring,
# the fp32 attention kernel): 148 SMs x 128 FMA lanes x 2 flops x 1.965 GHz (the maximum SM clock).
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def attn_source_digest():
    import hashlib
    h = hashlib.sha256()
    for name in ("attn_tc.cu", "tc_ptx.cuh"):
        with open(os.path.join(ROOT, "paper_2608_26965_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload_name):
    rec = NCU_TRAFFIC.get(workload_name)
    if rec is None or rec["source"] != attn_source_digest():
        return None, None
    return rec["bytes"], rec["commit"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="tabular")
    ap.add_argument("--keep", type=int, default=0, help="override kept key clusters per query cluster")
    ap.add_argument("--heads", type=int, default=0, help="run only the first HEADS heads (profiling captures)")
    ap.add_argument("--n-q", type=int, default=0, help="override the number of query rows per head")
    ap.add_argument("--n-k", type=int, default=0, help="override the number of key rows per head")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="sweep workload: cluster size x kept fraction x compensation, one JSON line with all points")
    ap.add_argument("--adaptive", type=float, default=0.0, metavar="RECALL",
                    help="adaptive mass-recall selection with this recall threshold (min count 16) and the "
                         "un-normalised query representation, instead of a fixed count per query cluster")
    ap.add_argument("--basic", type=int, default=-1, metavar="ITERATIONS",
                    help="cluster with basic recursive splitting (power iteration with the injected metric, "
                         "this many iterations per split) instead of the diagonalized variant")
    ap.add_argument("--scaling", action="store_true",
                    help="token-count sweep 8k..1M with per-stage times (64 kept blocks, and 10 %% of the blocks), "
                         "eager launches and one replayed CUDA graph, against dense attention")
    ap.add_argument("--max-tokens", type=int, default=1 << 20)
    ap.add_argument("--bare", action="store_true",
                    help="timed steps only: no sustained leg, no per-kernel timers (for captures under a profiler)")
    ap.add_argument("--fp8-qk", action="store_true",
                    help="attention with Q K^T on E4M3 codes (CA_ATTN_FP8_QK; head dimension 128 only)")
    ap.add_argument("--secondary", default="video480", metavar="WORKLOAD",
                    help="also report stage times and the attention roofline of this workload (10 steps); "
                         "'' switches it off")
    return ap.parse_args()


def block_flops(w, heads, keep=None):
    """Flops over the computed blocks: selected key rows plus centroid columns (padded to 128)."""
    keep = w.keep if keep is None else keep
    cols = keep * w.cluster + (-(-w.n_kc // 128) * 128 if w.compensate else 0)
    return 4.0 * w.n_q * w.head_dim * cols * heads


def dense_flops(w, heads):
    return 4.0 * w.n_q * w.n_k * w.head_dim * heads


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------
# CPU oracle on a bounded sample (the reference arm and the cpu_baseline leg)
# ------------------------------------------------------------------------------
def oracle_sample_step(w, Q, K, V, n_query_clusters=8, budget_rows=32768):
    """One oracle pass on a sample: a prefix of one head's rows (so clustering
    stays within seconds) and `n_query_clusters` query clusters of attention.
    Returns (flops over the blocks computed, seconds)."""
    from oracle import clusterattn_oracle as orc
    n_k = min(w.n_k, budget_rows)
    n_q = min(w.n_q, budget_rows)
    c = w.cluster
    n_kc = -(-n_k // c)
    keep = max(1, min(n_kc, round(w.keep * n_kc / w.n_kc)))
    Qs, Ks, Vs = Q[:n_q], K[:n_k], V[:n_k]
    t0 = time.perf_counter()
    cl = orc.cluster_qk(Qs, Ks, Vs, c, c)
    idx = orc.select_blocks(cl["cq"], cl["ck"], keep)
    n_qc = -(-n_q // c)
    sample = list(range(0, n_qc, max(1, n_qc // n_query_clusters)))[:n_query_clusters]
    orc.cluster_attention(Qs, Ks, Vs, cl["perm_q"], cl["perm_k"], c, c, idx, w.compensate, ck=cl["ck"],
                          cv=cl["cv"], count_k=cl["count_k"], query_clusters=sample)
    dt = time.perf_counter() - t0
    cols = keep * c + (n_kc if w.compensate else 0)
    flops = 4.0 * len(sample) * c * w.head_dim * cols
    desc = (f"1 head, first {n_q} queries x {n_k} keys of the workload: clustering and selection in full, "
            f"attention on {len(sample)} of {n_qc} query clusters, keep={keep} of {n_kc}")
    return flops, dt, desc


def decision_report(w, keep, flags, Qh, Kh, Vh, dev, head=0):
    """Part of the cpu_baseline leg: the integer decisions the device takes for one head of the timed
    workload (cluster permutations, block lists) against the oracle -- bit for bit against its
    float32 restatement on the device's own coordinates and centroids, and counted against its
    float64 definitions (differing split nodes, rows that end in another cluster, differing lists)."""
    import numpy as np
    import torch

    from oracle import clusterattn_oracle as orc
    from paper_2608_26965_b200 import binding
    from tests import decisions as dec

    w1 = w.scaled(heads=1)
    p1 = binding.problem_from_workload(w1, keep=keep, flags=flags)
    plan = binding.Plan(p1, dev, keep_y=True)
    dt = binding.torch_dtype(p1)
    Q, K, V = (torch.from_numpy(a[head:head + 1][None]).to(dt).to(dev) for a in (Qh, Kh, Vh))
    plan.cluster_qk(Q, K, V)
    plan.select_blocks()
    torch.cuda.synchronize()
    c = w.cluster
    out = {"head": head, "sides": {}}
    for side, Y, perm in (("queries", plan.Yq, plan.perm_q), ("keys", plan.Yk, plan.perm_k)):
        Yh, ph = Y[0, 0].cpu().numpy(), perm[0, 0].cpu().numpy()
        exact = bool(np.array_equal(ph, orc.recursive_split_f32(Yh, c)))
        rec = {"permutation_equals_float32_restatement": exact}
        if exact:
            a = dec.split_agreement(Yh, c, ph)
            rec.update(rows=a["rows"], split_nodes=a["nodes"], nodes_differing_from_float64=a["differing_nodes"],
                       of_them_not_near_ties=a["differing_nodes_not_near_tie"],
                       rows_in_another_cluster=a["rows_moved"],
                       rows_near_a_threshold=a["near_threshold_rows"], near_means="within 1e-6 of the spread of the set's keys")
        out["sides"][side] = rec
    cq, ck = plan.cq[0, 0].cpu().numpy(), plan.ck[0, 0].cpu().numpy()
    idx = plan.block_idx[0, 0].cpu().numpy()
    exact = bool(np.array_equal(idx, orc.select_blocks_f32(cq, ck, keep)))
    sel = {"lists_equal_float32_restatement": exact}
    if exact:
        a = dec.selection_agreement(cq, ck, keep, idx)
        sel.update(lists=a["lists"], lists_differing_from_float64=a["differing_lists"],
                   of_them_not_near_ties=a["differing_lists_not_near_tie"], near_tie_lists=a["near_tie_lists"])
    out["selection"] = sel
    return out


def run_reference(args, w):
    from paper_2608_26965_b200 import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    Q, K, V = inputs.generate_head(w, 0)
    times, flops, desc = [], 0.0, ""
    for i in range(args.warmup + args.steps):
        flops, dt, desc = oracle_sample_step(w, Q, K, V, n_query_clusters=4, budget_rows=16384)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = flops * len(times) / total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": host_cores(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.path = tempfile.mktemp(suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(device_index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------
# per-kernel rooflines of the clustering and selection stages
# ------------------------------------------------------------------------------
def split_level_counts(n, c):
    """(levels run as per-level launches over whole sets, levels finished inside the subtree kernel):
    sets of more than min(32 c, 4096) rows take a launch per level."""
    def nxt(big):
        L = c * ((big + c) // (2 * c))
        return max(L, big - L)
    levels, top, big = 0, 0, n
    tail_rows = min(32 * c, 4096)
    while big > c:
        if big > tail_rows:
            top += 1
        levels += 1
        big = nxt(big)
    return top, levels - top


def stage_rooflines(w, heads, group_ms, hbm_gbs, peak_kind):
    """Algorithmic bytes (flops for the scoring) of every kernel group of cluster_qk and
    select_blocks, its device time per step (the library's own CUDA-event timers, each group timed
    alone), and the fraction of the roof that bounds it."""
    b = 2 if w.dtype == "bf16" else 4
    d, nq, nk, c = w.head_dim, w.n_q, w.n_k, w.cluster
    top_q, tail_q = split_level_counts(nq, c)
    top_k, tail_k = split_level_counts(nk, c)
    sub = lambda nodes: nodes * d * d * 4                      # subsample rows read by `nodes` sets
    algo = {
        # Gram matrices of Q, K and of the query representation r(q) (stored as two bf16 halves / fp32)
        "gram": heads * ((nq + nk) * d * b + nq * d * 4),
        # Q -> r(q) (4 bytes per element out), r(q) -> Y_q, K -> Y_k (fp32 coordinates out)
        "transform": heads * (nq * d * (b + 4) + nq * d * 8 + nk * d * (b + 4)),
        # per level and side: a key and a row index read, a row index written, plus the subsample tiles
        "split_levels": heads * (12 * (nq * top_q + nk * top_k) + sub((1 << top_q) - 1) + sub((1 << top_k) - 1)),
        "split_tail": heads * (12 * (nq * tail_q + nk * tail_k)
                               + sub(max(0, w.n_qc - (1 << top_q))) + sub(max(0, w.n_kc - (1 << top_k)))),
        # Q, K and V rows read once and written once in cluster order
        "permute_centroid": heads * 2 * (nq + 2 * nk) * d * b,
    }
    out = {}
    for name, nbytes in algo.items():
        ms = group_ms.get(name)
        if not ms:
            continue
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[name] = {"bound": "hbm", "algorithmic_bytes": nbytes, "ms": ms, "achieved": gbs, "unit": "GB/s",
                     "peak": hbm_gbs, "peak_source": f"{peak_kind} HBM copy", "frac": gbs / hbm_gbs}
    for name in ("cholesky_factor", "principal_components"):
        if group_ms.get(name):
            out[name] = {"bound": "latency", "ms": group_ms[name],
                         "note": "d x d work on one CTA per head and side: no roofline, wall time only"}
    ms = group_ms.get("score_select")
    if ms:
        flops = 2.0 * w.n_qc * w.n_kc * d * heads
        tf = flops / (ms * 1e-3) / 1e12
        out["score_select"] = {"bound": "alu", "algorithmic_flops": flops, "ms": ms, "achieved": tf, "unit": "TFLOP/s",
                               "peak": FP32_ALU_TFLOPS, "peak_source": "148 SMs x 128 FMA lanes x 2 x 1.965 GHz",
                               "frac": tf / FP32_ALU_TFLOPS,
                               "algorithmic_bytes": heads * ((w.n_qc + w.n_kc) * d * 4 + w.n_qc * w.keep * 4),
                               "hbm_frac": heads * ((w.n_qc + w.n_kc) * d * 4 + w.n_qc * w.keep * 4) / (ms * 1e-3) / 1e9 / hbm_gbs}
    return out


def library_dense_ms(torch, binding, w, Q, K, V, dev, reps=3):
    """Dense attention through the library's own kernel: every key cluster kept, compensation off,
    identity permutation (the inputs themselves are the cluster-ordered tensors)."""
    p = binding.problem_from_workload(w, keep=w.n_kc, compensate=False)
    plan = binding.Plan(p, dev)
    c = w.cluster
    for dst, src, n in ((plan.Qp, Q, w.n_q), (plan.Kp, K, w.n_k), (plan.Vp, V, w.n_k)):
        dst.zero_()
        dst[:, :, :n].copy_(src)
    plan.perm_q.copy_(torch.arange(w.n_q, dtype=torch.int32, device=dev).expand_as(plan.perm_q))
    counts = torch.full((w.n_kc,), c, dtype=torch.int32, device=dev)
    counts[-1] = w.n_k - (w.n_kc - 1) * c
    plan.count_k.copy_(counts.expand_as(plan.count_k))
    plan.block_idx.copy_(torch.arange(w.n_kc, dtype=torch.int32, device=dev).expand_as(plan.block_idx))
    plan.ck.zero_()
    plan.cv.zero_()
    plan.cluster_attention_fwd(want_lse=False)
    torch.cuda.synchronize()
    a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        plan.cluster_attention_fwd(want_lse=False)
    b_.record()
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    return a.elapsed_time(b_) / reps


def secondary_workload(torch, binding, inputs, name, dev, steps, peaks):
    """Stage times and the attention roofline fraction of another workload (d = 128), so that the
    record of the default run also carries the video-shaped configuration."""
    w = inputs.WORKLOADS[name]
    p = binding.problem_from_workload(w)
    dt = binding.torch_dtype(p)
    Q, K, V = (torch.from_numpy(a[None]).to(dt).to(dev) for a in inputs.generate(w))
    plan = binding.Plan(p, dev)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        plan.forward(Q, K, V)
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    for e in ev:
        e[0].record(stream)
        plan.cluster_qk(Q, K, V)
        e[1].record(stream)
        plan.select_blocks()
        e[2].record(stream)
        plan.cluster_attention_fwd(want_lse=False)
        e[3].record(stream)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values()) and plan.recomputed_clusters() == 0
    stage = {"cluster_qk": float(np.mean([e[0].elapsed_time(e[1]) for e in ev])),
             "select_blocks": float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
             "cluster_attention_fwd": float(np.mean([e[2].elapsed_time(e[3]) for e in ev]))}
    flops = block_flops(w, w.heads)
    tf = flops / (stage["cluster_attention_fwd"] * 1e-3) / 1e12
    return {"workload": name, "heads": w.heads, "head_dim": w.head_dim, "n_q": w.n_q, "n_k": w.n_k, "keep": w.keep,
            "steps": steps, "stage_ms": stage, "ms_per_step": float(np.mean([e[0].elapsed_time(e[3]) for e in ev])),
            "block_flops_per_step": flops,
            "roofline": {"kernel": "cluster_attention_fwd", "bound": "tensor", "achieved": tf,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"]}}


# ------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------
def run_ours(args, w):
    import torch

    from paper_2608_26965_b200 import binding, build, inputs, replicas

    rank, local, world = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    device = torch.device(dev)
    distributed = replicas.init("nccl", device)
    if rank == 0:
        build.build()
    replicas.barrier(device)
    binding.load_library()

    keep = args.keep or w.keep
    heads = w.heads
    adaptive = args.adaptive > 0.0
    p = binding.problem_from_workload(w, keep=keep, flags=(binding.CA_QUERY_UNNORMALIZED if adaptive else 0) |
                                      (binding.CA_ATTN_FP8_QK if args.fp8_qk else 0))
    dt = binding.torch_dtype(p)
    Qh, Kh, Vh = inputs.generate(w)                        # every replica runs the same seeded batch
    pin = lambda a: torch.from_numpy(a[None]).to(dt).pin_memory()
    Q_host, K_host, V_host = pin(Qh), pin(Kh), pin(Vh)
    Q, K, V = (t.to(dev, non_blocking=True) for t in (Q_host, K_host, V_host))
    plan = binding.Plan(p, dev)
    O_host = torch.empty(plan.O.shape, dtype=dt).pin_memory()
    stream = torch.cuda.current_stream()

    def barrier():
        replicas.barrier(device)

    def max_over_ranks(x):
        return replicas.max_over_ranks(x, device)

    basic = args.basic >= 0
    if basic:
        rows_q, rows_k, _ = plan.basic_noise_rows()
        gen = torch.Generator(device=dev)
        gen.manual_seed(26082696)
        noise_q = torch.randn((1, heads, rows_q, w.head_dim), generator=gen, device=dev)
        noise_k = torch.randn((1, heads, rows_k, w.head_dim), generator=gen, device=dev)

    def clustering(Qd, Kd, Vd):
        if basic:
            plan.cluster_qk_basic(Qd, Kd, Vd, noise_q, noise_k, args.basic)
        else:
            plan.cluster_qk(Qd, Kd, Vd)

    def step(events=None):
        if events is not None:
            events[0].record(stream)
        clustering(Q, K, V)
        if events is not None:
            events[1].record(stream)
        if adaptive:
            plan.select_blocks_adaptive(args.adaptive, 16)
        else:
            plan.select_blocks()
        if events is not None:
            events[2].record(stream)
        if adaptive:
            plan.cluster_attention_fwd_ragged(want_lse=False)
        else:
            plan.cluster_attention_fwd(want_lse=False)
        if events is not None:
            events[3].record(stream)

    # the clock sampler runs from before the warm-up until after the sustained leg below, so that a
    # short timed region still has clock samples under the same load around it
    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    assert all(v == 0 for v in plan.last_status().values()), plan.last_status()

    # ---- timed region: device-resident inputs (larger than L2, so no flush is needed)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches0 = binding.kernel_launches()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for i in range(args.steps):
        step(ev[i])
    t_end.record(stream)
    barrier()
    launches = binding.kernel_launches() - launches0
    # ---- sustained leg (not the headline): the same step back to back for about a second, so that the
    # clock sampler sees this load for long enough; its time per step is reported beside the headline
    sustained = None
    if rank == 0 and not args.bare:
        n_sus = max(args.steps, int(1000.0 / max(t_start.elapsed_time(t_end) / args.steps, 0.05)))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record(stream)
        for _ in range(n_sus):
            step()
        s1.record(stream)
        torch.cuda.synchronize()
        sustained = {"steps": n_sus, "ms_per_step": s0.elapsed_time(s1) / n_sus}
    clocks = sampler.stop() if sampler else None
    if clocks is not None:
        clocks["window"] = "warm-up, timed region and the sustained leg (same step, about one second)"
        clocks["sustained_leg"] = sustained
    recomputed = plan.recomputed_clusters()           # 0 over every step so far: nothing left the tensor-core kernel
    # ---- per-kernel times of the clustering and selection stages (the library's own timers, each
    # kernel group alone on the stream), outside the timed region
    group_ms = {}
    if rank == 0 and not basic and not args.bare:
        binding.profile(True)
        n_prof = 5
        for _ in range(n_prof):
            step()
        group_ms = {k: v["ms"] / n_prof for k, v in binding.profile_read().items() if v["scopes"]}
        binding.profile(False)
    total_ms = max_over_ranks(t_start.elapsed_time(t_end))
    ms_per_step = total_ms / args.steps
    stage_ms = {
        "cluster_qk": float(np.mean([e[0].elapsed_time(e[1]) for e in ev])),
        "select_blocks": float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
        "cluster_attention_fwd": float(np.mean([e[2].elapsed_time(e[3]) for e in ev])),
    }
    mean_keep = float(plan.keep_count.float().mean().item()) if adaptive else float(keep)
    flops_step = block_flops(w, heads, mean_keep)
    value = world * flops_step / (ms_per_step * 1e-3) / 1e12

    # ---- end to end through the same calls with HOST buffers (pinned), copies inside the region
    e2e = None
    if not args.no_e2e:
        # Inputs are double-buffered on the device: the copy of step i+1 (side stream) runs under
        # the kernels of step i, and the result goes back on a third stream.  Every copy is inside
        # the timed region and ordered against the kernels with events.
        sets = [(Q, K, V), tuple(torch.empty_like(t) for t in (Q, K, V))]
        h2d, d2h = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(2)]        # inputs of set b are on the device
        ev_free = [torch.cuda.Event() for _ in range(2)]      # kernels have finished reading set b
        ev_out = torch.cuda.Event()                           # O has been written
        ev_read = torch.cuda.Event()                          # O has been copied to the host
        state = {"i": 0}

        def e2e_step():
            i = state["i"]
            bsel = i & 1
            with torch.cuda.stream(h2d):
                if i >= 2:
                    h2d.wait_event(ev_free[bsel])
                for dst, src in zip(sets[bsel], (Q_host, K_host, V_host)):
                    dst.copy_(src, non_blocking=True)
                ev_in[bsel].record(h2d)
            stream.wait_event(ev_in[bsel])
            Qd, Kd, Vd = sets[bsel]
            clustering(Qd, Kd, Vd)
            ev_free[bsel].record(stream)                      # only the clustering stage reads the inputs
            if adaptive:
                plan.select_blocks_adaptive(args.adaptive, 16)
            else:
                plan.select_blocks()
            if i >= 1:
                stream.wait_event(ev_read)                    # the previous result has left plan.O
            if adaptive:
                plan.cluster_attention_fwd_ragged(want_lse=False)
            else:
                plan.cluster_attention_fwd(want_lse=False)
            ev_out.record(stream)
            with torch.cuda.stream(d2h):
                d2h.wait_event(ev_out)
                O_host.copy_(plan.O, non_blocking=True)
                ev_read.record(d2h)
            state["i"] = i + 1

        def drain():
            stream.wait_stream(h2d)
            stream.wait_stream(d2h)

        for _ in range(2):
            e2e_step()
        drain()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        h2d.wait_event(a)
        d2h.wait_event(a)
        for _ in range(args.steps):
            e2e_step()
        drain()
        b.record(stream)
        barrier()
        e2e_ms = max_over_ranks(a.elapsed_time(b)) / args.steps
        nbytes = lambda t: t.numel() * t.element_size()
        e2e = {"value": world * flops_step / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": nbytes(Q_host) + nbytes(K_host) + nbytes(V_host),
               "d2h_bytes_per_step": nbytes(O_host),
               "overlap": "inputs double-buffered on the device; copies on side streams under the kernels"}

    # ---- dense attention on the same GPU (library kernel with every block kept, and torch SDPA)
    dense = None
    if not args.no_dense and rank == 0:
        dense = {}
        try:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.no_grad():
                for _ in range(2):
                    torch.nn.functional.scaled_dot_product_attention(Q, K, V)
                torch.cuda.synchronize()
                a.record(stream)
                for _ in range(5):
                    torch.nn.functional.scaled_dot_product_attention(Q, K, V)
                b.record(stream)
                torch.cuda.synchronize()
            dense["torch_sdpa_ms"] = a.elapsed_time(b) / 5
            dense["torch_sdpa_tflops"] = dense_flops(w, heads) / (dense["torch_sdpa_ms"] * 1e-3) / 1e12
            dense["speedup_vs_torch_sdpa"] = dense["torch_sdpa_ms"] / ms_per_step
        except Exception as exc:  # noqa: BLE001
            dense["torch_sdpa_error"] = str(exc)[:200]
        if w.dtype == "bf16":
            dense["library_ms"] = library_dense_ms(torch, binding, w, Q, K, V, dev)
            dense["library_tflops"] = dense_flops(w, heads) / (dense["library_ms"] * 1e-3) / 1e12
        candidates = [dense[k] for k in ("torch_sdpa_ms", "library_ms") if k in dense]
        if candidates:
            dense["fastest_ms"] = min(candidates)
            dense["speedup_vs_fastest_dense"] = dense["fastest_ms"] / ms_per_step

    barrier()
    if rank != 0:
        replicas.shutdown()
        return

    # ---- supplementary: the same steps (a) replayed from one CUDA graph, (b) with two steps in
    # flight on two streams and two sets of buffers.  Neither is the headline; both say how much of a
    # step is launch gaps and latency-bound clustering that another step could fill.
    overlap = None
    if not (args.no_e2e or adaptive or basic):
        def timed_steps(fn, n):
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn(n)
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / n
        overlap = {}
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                plan.forward(Q, K, V, stream=side)
                side.synchronize()
                with torch.cuda.graph(graph, stream=side):
                    plan.forward(Q, K, V, stream=side)
            overlap["cuda_graph_ms_per_step"] = timed_steps(lambda n: [graph.replay() for _ in range(n)], args.steps)
            del graph
        except Exception as exc:                               # noqa: BLE001
            overlap["cuda_graph_ms_per_step"] = f"capture failed: {str(exc)[:120]}"
        plans = [plan, binding.Plan(p, dev)]
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]

        def two_in_flight(n):
            for st_ in streams:
                st_.wait_stream(torch.cuda.current_stream())
            for i in range(n):
                plans[i & 1].forward(Q, K, V, stream=streams[i & 1])
            for st_ in streams:
                torch.cuda.current_stream().wait_stream(st_)
        two_in_flight(4)
        overlap["two_steps_in_flight_ms_per_step"] = timed_steps(two_in_flight, args.steps)
        assert all(v == 0 for pl in plans for v in pl.last_status().values())
        del plans[1]

    peaks, peak_kind = load_peaks()
    attn_ms = stage_ms["cluster_attention_fwd"]
    attn_tflops = flops_step / (attn_ms * 1e-3) / 1e12
    traffic, traffic_commit = (None, None) if (adaptive or basic or args.keep or args.n_q or args.n_k or args.heads) \
        else ncu_traffic(w.name)
    if w.dtype == "bf16":
        roofline = {"kernel": "cluster_attention_fwd", "bound": "tensor", "achieved": attn_tflops,
                    "peak": peaks["bf16_tflops"], "peak_source": f"{peak_kind} bf16 burst", "unit": "TFLOP/s",
                    "frac": attn_tflops / peaks["bf16_tflops"], "traffic": traffic, "traffic_capture_commit": traffic_commit}
    else:           # fp32 storage runs the CUDA-core kernel: bound by the FP32 FMA rate
        roofline = {"kernel": "cluster_attention_fwd", "bound": "alu", "achieved": attn_tflops, "peak": FP32_ALU_TFLOPS,
                    "peak_source": "148 SMs x 128 FMA lanes x 2 x 1.965 GHz", "unit": "TFLOP/s",
                    "frac": attn_tflops / FP32_ALU_TFLOPS, "traffic": None}
    if w.dtype == "bf16" and w.head_dim == 64:
        # At d = 64 the exponentials bound the kernel before the tensor pipe does: a half-step of 64 keys
        # is 2 x (128 x 64 x 64) multiply-adds = 2^21 flops of tensor work per query tile and
        # 128 x 64 = 8192 exponentials, which the special-function unit of an SM takes 512 cycles for
        # (16 per cycle: 4 sub-cores x 1 warp instruction per 8 cycles): at most 4096 flops per cycle
        # and SM, i.e. 148 SMs x 4096 x 1.965 GHz.
        sfu_peak = 148 * 4096 * 1.965e9 / 1e12
        roofline["second_bound"] = {"name": "special-function unit (exp2 of the softmax)", "peak": sfu_peak,
                                    "unit": "TFLOP/s", "frac": attn_tflops / sfu_peak,
                                    "derivation": "8192 exp2 per 2^21 tensor flops; 16 exp2 per cycle and SM; "
                                                  "148 SMs x 4096 flops/cycle x 1.965 GHz"}
    stages = stage_rooflines(w.scaled(keep=keep), heads, group_ms, peaks["hbm_gbs"], peak_kind) if group_ms else None
    secondary = None
    if args.secondary and args.secondary != w.name and world == 1 and w.name == "tabular" \
            and not (adaptive or basic or args.keep or args.n_q or args.n_k or args.heads):
        secondary = secondary_workload(torch, binding, inputs, args.secondary, dev, 10, peaks)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "heads": heads, "head_dim": w.head_dim, "n_q": w.n_q, "n_k": w.n_k,
                   "cluster": w.cluster, "keep": mean_keep if adaptive else keep, "n_kc": w.n_kc,
                   "selection": f"adaptive recall {args.adaptive} min 16" if adaptive else "top-k",
                   "qk_operands": "e4m3 (per-row / per-cluster scales)" if args.fp8_qk else w.dtype,
                   "clustering": f"basic recursive splitting, {args.basic} power iterations" if basic
                   else "diagonalized recursive splitting", "compensate": w.compensate,
                   "parallelism": "replicas" if world > 1 else "single",
                   "l2": "inputs larger than L2 (no flush)"},
        "stage_ms": stage_ms, "block_flops_per_step": flops_step, "dense_flops": dense_flops(w, heads),
        "roofline": roofline, "stage_rooflines": stages, "kernel_group_ms": group_ms or None,
        "e2e": e2e, "gpu_launches": int(launches), "recomputed_clusters": int(recomputed),
        "clocks": clocks, "dense": dense,
        "overlap": overlap, "secondary": secondary,
    }
    if not args.no_cpu_baseline:
        # the oracle as it stands on whole heads until about 10 s of CPU work are spent
        flops = secs = 0.0
        used = 0
        for h in range(heads):
            f, s_, desc = oracle_sample_step(w, Qh[h], Kh[h], Vh[h], n_query_clusters=1 << 30,
                                             budget_rows=1 << 30)
            flops, secs, used = flops + f, secs + s_, used + 1
            if secs > 10.0:
                break
        line["cpu_baseline"] = {"value": flops / secs / 1e12, "unit": UNIT, "cores": host_cores(),
                                "kind": "oracle", "seconds": secs,
                                "sample": f"{used} of {heads} heads in full (all stages, fp64 numpy)"}
        if not adaptive and not basic:
            line["decisions_vs_oracle"] = decision_report(w, keep, p.flags, Qh, Kh, Vh, dev)
    print(json.dumps(line))
    replicas.shutdown()


def run_sweep(args):
    """Cluster size 64/128/256 x kept fraction 1/32..1/2 x compensation on/off on the sweep
    workload (16 heads, d=128, 131,072 tokens), plus dense attention on the same tensors."""
    import torch

    from paper_2608_26965_b200 import binding, build, inputs

    build.build()
    binding.load_library()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    base = inputs.WORKLOADS["sweep"]
    if args.heads:
        base = base.scaled(heads=args.heads)
    Qh, Kh, Vh = inputs.generate(base)
    dt = torch.bfloat16
    Q, K, V = (torch.from_numpy(a[None]).to(dt).to(dev) for a in (Qh, Kh, Vh))
    stream = torch.cuda.current_stream()
    peaks, peak_kind = load_peaks()

    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    with torch.no_grad():
        dense_ms = timed(lambda: torch.nn.functional.scaled_dot_product_attention(Q, K, V), 3)
    points = []
    for c in (64, 128, 256):
        n_kc = base.n_k // c
        first = True
        for frac in (1 / 32, 1 / 16, 1 / 8, 1 / 4, 1 / 2):
            keep = inputs.keep_from_fraction(n_kc, frac)
            for comp in (True, False):
                w = base.scaled(cluster=c, keep=keep, compensate=comp)
                p = binding.problem_from_workload(w)
                plan = binding.Plan(p, dev)
                if first:
                    cluster_ms = timed(lambda: plan.cluster_qk(Q, K, V), args.steps)
                    first = False
                    kept = plan                      # clustering does not depend on keep / compensation
                else:
                    for name in ("perm_q", "perm_k", "Qp", "Kp", "Vp", "cq", "ck", "cv", "count_q", "count_k"):
                        setattr(plan, name, getattr(kept, name))
                select_ms = timed(lambda: plan.select_blocks(), args.steps)
                attn_ms = timed(lambda: plan.cluster_attention_fwd(want_lse=False), args.steps)
                assert all(v == 0 for v in plan.last_status().values())
                flops = block_flops(w, w.heads, keep)
                total = cluster_ms + select_ms + attn_ms
                points.append({"cluster": c, "fraction": frac, "keep": keep, "compensate": comp,
                               "cluster_qk_ms": cluster_ms, "select_ms": select_ms, "attn_ms": attn_ms,
                               "total_ms": total, "attn_tflops": flops / attn_ms / 1e9,
                               "attn_frac_of_peak": flops / attn_ms / 1e9 / peaks["bf16_tflops"],
                               "speedup_vs_dense": dense_ms / total})
                del plan
    print(json.dumps({"metric": METRIC, "workload": "sweep", "heads": base.heads, "n": base.n_q,
                      "head_dim": base.head_dim, "dense_sdpa_ms": dense_ms,
                      "dense_sdpa_tflops": dense_flops(base, base.heads) / dense_ms / 1e9,
                      "peak_tflops": peaks["bf16_tflops"], "peak_source": peak_kind, "points": points}))


def run_scaling(args):
    """Token counts 8,192 .. 1,048,576 (self-attention, d = 64, 128-row clusters): per-stage
    times with 64 kept blocks and with 10 % of the blocks kept, the same step replayed from a
    CUDA graph, and dense attention on the same tensors."""
    import torch

    from paper_2608_26965_b200 import binding, build, inputs

    build.build()
    binding.load_library()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    heads = args.heads or 4
    stream = torch.cuda.current_stream()
    points = []
    n = 8192
    while n <= args.max_tokens:
        base = inputs.WORKLOADS["tabular"].scaled(n_q=n, n_k=n, heads=heads)
        Qh, Kh, Vh = inputs.generate(base)
        Q, K, V = (torch.from_numpy(a[None]).to(torch.bfloat16).to(dev) for a in (Qh, Kh, Vh))
        reps = max(2, min(args.steps, (1 << 22) // n))

        def timed(fn, reps):
            fn()
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps

        with torch.no_grad():
            dense_ms = timed(lambda: torch.nn.functional.scaled_dot_product_attention(Q, K, V), 1 if n > 200000 else 3)
        n_kc = base.n_kc
        for label, keep in (("64 blocks", min(64, n_kc)), ("10 %", max(1, round(0.1 * n_kc)))):
            w = base.scaled(keep=keep)
            plan = binding.Plan(binding.problem_from_workload(w), dev)
            cluster_ms = timed(lambda: plan.cluster_qk(Q, K, V), reps)
            select_ms = timed(lambda: plan.select_blocks(), reps)
            attn_ms = timed(lambda: plan.cluster_attention_fwd(want_lse=False), reps)
            eager_ms = timed(lambda: plan.forward(Q, K, V), reps)
            assert all(v == 0 for v in plan.last_status().values())
            # the same step captured once and replayed: no per-launch host cost
            graph_ms = None
            try:
                side = torch.cuda.Stream()
                side.wait_stream(stream)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    plan.forward(Q, K, V, stream=side)
                    side.synchronize()
                    with torch.cuda.graph(graph, stream=side):
                        plan.forward(Q, K, V, stream=side)
                stream.wait_stream(side)
                graph_ms = timed(graph.replay, reps)
                del graph
            except Exception as exc:  # noqa: BLE001
                graph_ms = f"capture failed: {str(exc)[:120]}"
            points.append({"n": n, "kept": label, "keep": keep, "cluster_qk_ms": cluster_ms, "select_ms": select_ms,
                           "attn_ms": attn_ms, "step_ms": eager_ms, "graph_step_ms": graph_ms, "dense_sdpa_ms": dense_ms,
                           "speedup_vs_dense": dense_ms / eager_ms})
            del plan
        del Q, K, V
        torch.cuda.empty_cache()
        n *= 2
    print(json.dumps({"metric": METRIC, "workload": "scaling", "heads": heads, "head_dim": 64, "cluster": 128,
                      "points": points}))


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.scaling:
        run_scaling(args)
        return
    from paper_2608_26965_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.heads:
        w = w.scaled(heads=args.heads)
    if args.n_q or args.n_k:
        w = w.scaled(n_q=args.n_q or w.n_q, n_k=args.n_k or w.n_k)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

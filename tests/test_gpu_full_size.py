"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 oracle cannot run whole workloads of this size, so each stage is
checked on samples the oracle computes one by one, against the device's own
intermediate results (the stage inputs are then identical on both sides):
  * splitter: the oracle's splitter on the device's fp32 coordinates of sampled
    heads must give the same permutation, bit for bit;
  * selection: exact lists on the device's centroids of sampled heads;
  * attention: sampled query clusters, oracle attention on the device's
    permutation, centroids and block lists;
  * invariants that hold at any size for every head: the permutation is a
    permutation, counts sum to n, block lists are strictly ascending.
"""
import numpy as np
import pytest
import torch

from oracle import clusterattn_oracle as orc
from paper_2608_26965_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_workload(name, keep=None):
    build.build()
    w = inputs.WORKLOADS[name]
    if keep is not None:
        w = w.scaled(keep=keep)
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV, keep_y=True)
    dev = lambda a: torch.from_numpy(a[None]).to(dt).to(DEV)
    O = plan.forward(dev(Q), dev(K), dev(V), want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    assert plan.recomputed_clusters() == 0          # everything stayed on the tensor-core kernel
    return w, Q, K, V, plan, O


def check_workload(name, sample_heads, clusters_per_head, split_heads, keep=None):
    w, Q, K, V, plan, O = run_workload(name, keep)
    c = w.cluster
    # ---- invariants for every head
    perm_q, perm_k = plan.perm_q[0], plan.perm_k[0]
    for perm, n in ((perm_q, w.n_q), (perm_k, w.n_k)):
        srt = torch.sort(perm, dim=1).values
        assert torch.equal(srt, torch.arange(n, device=DEV, dtype=torch.int32).expand_as(srt))
    assert int(plan.count_k.sum()) == w.heads * w.n_k and int(plan.count_q.sum()) == w.heads * w.n_q
    assert int(plan.count_k.min()) >= min(c, w.n_k % c or c)
    idx_all = plan.block_idx[0]
    assert bool((idx_all[..., 1:] > idx_all[..., :-1]).all()) and int(idx_all.min()) >= 0 and int(idx_all.max()) < w.n_kc
    assert bool(torch.isfinite(O.float()).all())
    r = np.random.default_rng(w.config_id)
    # ---- splitter at full size
    for h in split_heads:
        Yk = plan.Yk[0, h].cpu().numpy()
        assert np.array_equal(perm_k[h].cpu().numpy(), orc.recursive_split(Yk, c)), f"key split differs, head {h}"
        Yq = plan.Yq[0, h].cpu().numpy()
        assert np.array_equal(perm_q[h].cpu().numpy(), orc.recursive_split(Yq, c)), f"query split differs, head {h}"
    worst_abs, worst_rel = 0.0, 0.0
    for h in sample_heads:
        pq, pk = perm_q[h].cpu().numpy(), perm_k[h].cpu().numpy()
        ck, cv = plan.ck[0, h].cpu().numpy(), plan.cv[0, h].cpu().numpy()
        cq = plan.cq[0, h].cpu().numpy()
        idx = plan.block_idx[0, h].cpu().numpy()
        # ---- centroids of sampled clusters and the whole selection of this head
        for j in r.choice(w.n_kc, 4, replace=False):
            rows = pk[j * c:min((j + 1) * c, w.n_k)]
            assert np.abs(ck[j] - K[h][rows].astype(np.float64).mean(0)).max() < 1e-5
            assert np.abs(cv[j] - V[h][rows].astype(np.float64).mean(0)).max() < 1e-5
        assert np.array_equal(idx, orc.select_blocks(cq, ck, w.keep)), f"block lists differ, head {h}"
        # ---- attention on sampled query clusters
        qcs = sorted(r.choice(w.n_qc, clusters_per_head, replace=False).tolist())
        if w.n_q % c:
            qcs[-1] = w.n_qc - 1                 # include the short cluster
        o_ref, lse_ref = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, c, c, idx, w.compensate, ck=ck, cv=cv,
                                               count_k=plan.count_k[0, h].cpu().numpy(), query_clusters=qcs)
        rows = np.concatenate([pq[i * c:min((i + 1) * c, w.n_q)] for i in qcs])
        got = O[0, h].float().cpu().numpy()[rows]
        worst_abs = max(worst_abs, np.abs(got - o_ref[rows]).max())
        worst_rel = max(worst_rel, np.linalg.norm(got - o_ref[rows]) / np.linalg.norm(o_ref[rows]))
        assert np.abs(plan.lse[0, h].cpu().numpy()[rows] - lse_ref[rows]).max() < 2e-2
    print(f"{name}: sampled attention max-abs {worst_abs:.3e}, relative Frobenius {worst_rel:.3e}")
    assert worst_abs <= 2e-2 and worst_rel <= 5e-3


def test_tabular_full_size():
    check_workload("tabular", sample_heads=[0, 5], clusters_per_head=6, split_heads=[3])


def test_video480_full_size():
    check_workload("video480", sample_heads=[0, 17, 39], clusters_per_head=4, split_heads=[11])


def test_video720_full_size_both_densities():
    check_workload("video720", sample_heads=[2, 31], clusters_per_head=3, split_heads=[20])          # 1/8
    check_workload("video720", sample_heads=[7], clusters_per_head=3, split_heads=[], keep=37)        # 1/16


def test_sweep_full_size_one_eighth():
    check_workload("sweep", sample_heads=[1, 14], clusters_per_head=4, split_heads=[9])


def test_tabular_full_size_adaptive_selection():
    """The adaptive path at the benchmark size, as `bench.py --adaptive 0.5` launches it:
    un-normalised query representation, mass-recall selection, attention over ragged lists."""
    build.build()
    w = inputs.WORKLOADS["tabular"]
    Q, K, V = inputs.generate(w)
    scale = float(np.float32(1.0 / np.sqrt(w.head_dim)))
    p = binding.problem_from_workload(w, flags=binding.CA_QUERY_UNNORMALIZED, softmax_scale=scale)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV, keep_y=True)
    dev = lambda a: torch.from_numpy(a[None]).to(dt).to(DEV)
    O, lse = plan.forward_adaptive(dev(Q), dev(K), dev(V), recall=0.5, min_count=16, want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    assert plan.recomputed_clusters() == 0          # everything stayed on the tensor-core kernel
    c = w.cluster
    keep_all = plan.keep_count[0]
    assert int(keep_all.min()) >= 16 and int(keep_all.max()) <= w.n_kc
    idx_all = plan.block_idx_ragged[0]
    pos = torch.arange(w.n_kc, device=DEV)[None, None, :]
    live = pos < keep_all[..., None]
    assert bool(((idx_all[..., 1:] > idx_all[..., :-1]) | ~live[..., 1:]).all())       # ascending inside the list
    assert bool((idx_all[~live] == -1).all())                                          # padding behind it
    r = np.random.default_rng(77)
    for h in (1, 6):
        Yq = plan.Yq[0, h].cpu().numpy()
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, orc.recursive_split(Yq, c))
        ck, cv, cq = (t[0, h].cpu().numpy() for t in (plan.ck, plan.cv, plan.cq))
        cnt = plan.count_k[0, h].cpu().numpy()
        lists = orc.select_blocks_adaptive(cq, ck, cnt, 0.5, 16, scale=scale)
        keep = keep_all[h].cpu().numpy()
        idx = idx_all[h].cpu().numpy()
        for i, row in enumerate(lists):
            assert keep[i] == len(row) and np.array_equal(idx[i, :len(row)], row), (h, i)
        qcs = sorted(r.choice(w.n_qc, 4, replace=False).tolist())
        o_ref, lse_ref = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, c, c, lists, True, ck=ck, cv=cv,
                                               count_k=cnt, query_clusters=qcs)
        rows = np.concatenate([pq[i * c:(i + 1) * c] for i in qcs])
        got = O[0, h].float().cpu().numpy()[rows]
        assert np.abs(got - o_ref[rows]).max() <= 2e-2
        assert np.linalg.norm(got - o_ref[rows]) <= 5e-3 * np.linalg.norm(o_ref[rows])
        assert np.abs(lse[0, h].cpu().numpy()[rows] - lse_ref[rows]).max() < 2e-2


def test_tabular_full_size_basic_splitting():
    """Basic recursive splitting at the benchmark size, as `bench.py --basic 3` launches it: the
    oracle's splitter on the device's metric matrices reproduces the permutation of 131,072 keys and
    16,384 queries of a sampled head bit for bit; invariants on every head."""
    build.build()
    w = inputs.WORKLOADS["tabular"]
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV)
    rows_q, rows_k, _ = plan.basic_noise_rows()
    r = np.random.default_rng(11)
    nq = r.standard_normal((w.heads, rows_q, w.head_dim)).astype(np.float32)
    nk = r.standard_normal((w.heads, rows_k, w.head_dim)).astype(np.float32)
    dev = lambda a, t=torch.float32: torch.from_numpy(a[None]).to(t).to(DEV)
    plan.cluster_qk_basic(dev(Q, dt), dev(K, dt), dev(V, dt), dev(nq), dev(nk), 3)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    assert plan.recomputed_clusters() == 0          # everything stayed on the tensor-core kernel
    for perm, n in ((plan.perm_q[0], w.n_q), (plan.perm_k[0], w.n_k)):
        srt = torch.sort(perm, dim=1).values
        assert torch.equal(srt, torch.arange(n, device=DEV, dtype=torch.int32).expand_as(srt))
    assert int(plan.count_k.sum()) == w.heads * w.n_k and int(plan.count_k.min()) == w.cluster
    h = 4
    A_q, A_k = plan.A_q[0, h].cpu().numpy(), plan.A_k[0, h].cpu().numpy()
    assert np.array_equal(plan.perm_k[0, h].cpu().numpy(), orc.basic_recursive_split(K[h], A_k, nk[h], w.cluster, 3))
    assert np.array_equal(plan.perm_q[0, h].cpu().numpy(), orc.basic_recursive_split(Q[h], A_q, nq[h], w.cluster, 3))

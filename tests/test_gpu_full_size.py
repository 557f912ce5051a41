"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The fp64 oracle cannot run whole workloads of this size, so each stage is
checked on samples the oracle computes one by one, against the device's own
intermediate results (the stage inputs are then identical on both sides):
  * coordinates: the device's split coordinates of a sampled head against the
    oracle's own chain from Q and K (metric, root, transform, principal
    components), column by column, and the first split of the two chains;
  * splitter: the oracle's splitter with float32 coordinate choices on the
    device's fp32 coordinates of sampled heads must give the same permutation,
    bit for bit; against the float64 choices the differences are counted and
    must all sit at near-ties, below 0.1 % of the rows;
  * selection: exact lists on the device's centroids of sampled heads (float32
    scores), differences from the float64 selection counted, near-ties only;
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
from tests import decisions

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


_GENERATED = {}


def generated(w):
    """Host copies of a workload's inputs, generated once per (workload, shape)."""
    key = (w.name, w.heads, w.n_q, w.n_k, w.head_dim)
    if key not in _GENERATED:
        _GENERATED.clear()                       # one workload at a time: they are large
        _GENERATED[key] = inputs.generate(w)
    return _GENERATED[key]


def run_workload(name, keep=None, cluster=None, compensate=None, flags=0, **shape):
    build.build()
    w = inputs.WORKLOADS[name]
    if shape:
        w = w.scaled(**shape)
    if cluster is not None:
        w = w.scaled(cluster=cluster)
    if keep is not None:
        w = w.scaled(keep=keep)
    if compensate is not None:
        w = w.scaled(compensate=compensate)
    Q, K, V = generated(w)
    p = binding.problem_from_workload(w, flags=flags)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV, keep_y=True)
    dev = lambda a: torch.from_numpy(a[None]).to(dt).to(DEV)
    O = plan.forward(dev(Q), dev(K), dev(V), want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    assert plan.recomputed_clusters() == 0          # everything stayed on the tensor-core kernel
    return w, Q, K, V, plan, O


def check_workload(name, sample_heads, clusters_per_head, split_heads, keep=None, cluster=None, compensate=None,
                   chain_heads=(), quantized=False, **shape):
    w, Q, K, V, plan, O = run_workload(name, keep, cluster, compensate,
                                       flags=binding.CA_ATTN_FP8_QK if quantized else 0, **shape)
    c = w.cluster
    label = f"{name} c={c} keep={w.keep}"
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
    # ---- splitter at full size: bit for bit the float32 restatement; counted against float64
    for h in split_heads:
        for side, perm, Y, n in (("keys", perm_k, plan.Yk, w.n_k), ("queries", perm_q, plan.Yq, w.n_q)):
            Yh, ph = Y[0, h].cpu().numpy(), perm[h].cpu().numpy()
            assert np.array_equal(ph, orc.recursive_split_f32(Yh, c)), f"{side} split differs, head {h}"
            decisions.check_split_agreement(Yh, c, ph, f"{label} {side}, head {h}")
    # ---- the chain from Q and K to the coordinates against the oracle's
    for h in chain_heads:
        decisions.check_coordinates(f"{label} head {h}", w, Q[h], K[h], plan.Yq[0, h].cpu().numpy(), plan.Yk[0, h].cpu().numpy(),
                          perm_q[h].cpu().numpy(), perm_k[h].cpu().numpy())
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
        assert np.array_equal(idx, orc.select_blocks_f32(cq, ck, w.keep)), f"block lists differ, head {h}"
        decisions.check_selection_agreement(cq, ck, w.keep, idx, f"{label}, head {h}")
        # ---- attention on sampled query clusters
        qcs = sorted(r.choice(w.n_qc, clusters_per_head, replace=False).tolist())
        if w.n_q % c:
            qcs[-1] = w.n_qc - 1                 # include the short cluster
        attend = orc.cluster_attention_quantized_qk if quantized else orc.cluster_attention
        o_ref, lse_ref = attend(Q[h], K[h], V[h], pq, pk, c, c, idx, w.compensate, ck=ck, cv=cv,
                                count_k=plan.count_k[0, h].cpu().numpy(), query_clusters=qcs)
        rows = np.concatenate([pq[i * c:min((i + 1) * c, w.n_q)] for i in qcs])
        got = O[0, h].float().cpu().numpy()[rows]
        worst_abs = max(worst_abs, np.abs(got - o_ref[rows]).max())
        worst_rel = max(worst_rel, np.linalg.norm(got - o_ref[rows]) / np.linalg.norm(o_ref[rows]))
        assert np.abs(plan.lse[0, h].cpu().numpy()[rows] - lse_ref[rows]).max() < 2e-2
    print(f"{label}: sampled attention max-abs {worst_abs:.3e}, relative Frobenius {worst_rel:.3e}")
    assert worst_abs <= 2e-2 and worst_rel <= 5e-3
    return plan


def test_tabular_full_size():
    check_workload("tabular", sample_heads=[0, 5], clusters_per_head=6, split_heads=[3], chain_heads=[3])


def test_video480_full_size():
    check_workload("video480", sample_heads=[0, 17, 39], clusters_per_head=4, split_heads=[11], chain_heads=[11])


def test_video480_full_size_quantised_qk():
    """The video-shaped workload with Q K^T on E4M3 codes (CA_ATTN_FP8_QK), as `bench.py --workload
    video480 --fp8-qk` launches it; sampled query clusters against the oracle's quantised attention."""
    check_workload("video480", sample_heads=[5, 33], clusters_per_head=4, split_heads=[], quantized=True)


def test_video720_full_size_both_densities():
    check_workload("video720", sample_heads=[2, 31], clusters_per_head=3, split_heads=[20], chain_heads=[20])   # 1/8
    check_workload("video720", sample_heads=[7], clusters_per_head=3, split_heads=[], keep=37)        # 1/16


def test_sweep_full_size_one_eighth():
    check_workload("sweep", sample_heads=[1, 14], clusters_per_head=4, split_heads=[9], chain_heads=[9])


@pytest.mark.parametrize("cluster,fraction,compensate", [(64, 1 / 32, True), (64, 1 / 2, False),
                                                         (256, 1 / 32, False), (256, 1 / 2, True)])
def test_sweep_full_size_other_cluster_sizes(cluster, fraction, compensate):
    """The sweep workload at 131,072 tokens with 64-row clusters (2,048 clusters per side: the tiled
    selection, half-filled query tiles) and 256-row clusters (two CTAs per query cluster), at the
    lowest and the highest density of the sweep, with and without compensation."""
    n_kc = inputs.WORKLOADS["sweep"].n_k // cluster
    check_workload("sweep", sample_heads=[3], clusters_per_head=3, split_heads=[3], cluster=cluster,
                   keep=inputs.keep_from_fraction(n_kc, fraction), compensate=compensate)


def test_long_sequence_half_a_million_tokens():
    """One head of 524,288 tokens (d = 64, 128-row clusters, 64 kept blocks, compensation on), the
    regime of the token-count sweep in which the 4,096 centroid columns per query outweigh the kept
    blocks: 12 split levels, selection in score tiles, attention with 64 half-steps of centroids."""
    check_workload("tabular", sample_heads=[0], clusters_per_head=3, split_heads=[0], keep=64,
                   heads=1, n_q=524288, n_k=524288)


def test_replayed_cuda_graph_writes_the_same_output():
    """The step captured into a CUDA graph the way bench.py does it, replayed on new inputs in the
    same buffers: output, permutations and block lists equal those of the eager calls bit for bit."""
    build.build()
    w = inputs.WORKLOADS["tabular"].scaled(heads=2, n_q=4096, n_k=16384, keep=16)
    p = binding.problem_from_workload(w)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV)
    first = [torch.from_numpy(a[None]).to(dt).to(DEV) for a in inputs.generate(w)]
    second = [torch.from_numpy(a[None]).to(dt).to(DEV) for a in inputs.generate(w.scaled(config_id=w.config_id + 100))]
    bufs = [t.clone() for t in first]
    stream = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(stream)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        plan.forward(*bufs, want_lse=True, stream=side)            # first call on the device: before the capture
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            plan.forward(*bufs, want_lse=True, stream=side)
    stream.wait_stream(side)
    for inputs_now in (second, first):
        for b, t in zip(bufs, inputs_now):
            b.copy_(t)
        for t in (plan.O, plan.lse, plan.perm_q, plan.perm_k, plan.block_idx):
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        replayed = [t.clone() for t in (plan.O, plan.lse, plan.perm_q, plan.perm_k, plan.block_idx)]
        for t in (plan.O, plan.lse, plan.perm_q, plan.perm_k, plan.block_idx):
            t.zero_()
        plan.forward(*inputs_now, want_lse=True)
        torch.cuda.synchronize()
        assert all(v == 0 for v in plan.last_status().values())
        for got, want in zip(replayed, (plan.O, plan.lse, plan.perm_q, plan.perm_k, plan.block_idx)):
            assert torch.equal(got, want)
    assert not torch.equal(replayed[0], torch.zeros_like(replayed[0]))


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
        assert np.array_equal(pq, orc.recursive_split_f32(Yq, c))
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

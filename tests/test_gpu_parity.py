"""Parity of the CUDA path (through the C ABI) against the fp64 oracle.

Integer results (permutations, block lists, counts, gathered rows) must match
bit for bit; floating point within the tolerances stated in each test.
"""
import numpy as np
import pytest
import torch

from oracle import clusterattn_oracle as orc
from paper_2608_26965_b200 import binding, build, inputs
from tests import decisions

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load_library()


def to_dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.to(DEV).contiguous()


def store(problem, a):
    """float32 host array -> device tensor in the problem's storage type ([1,H,n,d])."""
    return to_dev(a[None], binding.torch_dtype(problem))


def random_y(seed, H, n, d, ties=False):
    r = np.random.default_rng(seed)
    y = (r.standard_normal((H, n, d)) * np.linspace(2.0, 0.2, d)).astype(np.float32)
    if ties:
        y = np.round(y * 2.0) / 2.0                 # heavy duplication, includes +-0
        y[:, ::5, :] = -0.0
    return y


# ----------------------------------------------------------------------------
# Splitter on the oracle's own fp32 coordinates: bit-exact permutation,
# gathered rows, counts; centroids to fp32 rounding.
# ----------------------------------------------------------------------------
SPLIT_CASES = [
    # H, n_q, n_k, d, c_q, c_k, dtype, ties
    (2, 1024, 1024, 64, 64, 64, "fp32", False),       # the tiny configuration's shape
    (2, 1000, 1531, 64, 64, 32, "fp32", False),       # ragged: short last clusters
    (1, 50, 200, 64, 64, 128, "bf16", False),         # n <= c on one side, one split on the other
    (2, 3000, 4099, 128, 128, 128, "bf16", True),     # many exact ties
    (1, 2048, 40000, 64, 128, 128, "bf16", False),    # sets larger than the shared-memory window
    (1, 640, 704, 128, 256, 16, "bf16", False),       # extreme cluster sizes
    (1, 16384, 131072, 64, 128, 128, "bf16", False),  # one head of the tabular shape: 8-CTA clusters at the top
    (1, 5000, 200000, 64, 64, 128, "bf16", True),     # slices beyond the shared-memory window, with ties
    (2, 32760, 32760, 128, 128, 128, "bf16", False),  # the video shape: odd cluster counts, short last cluster
    (1, 4096, 1048576, 64, 128, 128, "bf16", False),  # a million rows: 13 levels, 8 with thread-block clusters
]


@pytest.mark.parametrize("H,n_q,n_k,d,c_q,c_k,dtype,ties", SPLIT_CASES)
def test_split_and_gather_bit_exact(H, n_q, n_k, d, c_q, c_k, dtype, ties):
    r = np.random.default_rng(n_q + n_k)
    Yq, Yk = random_y(1, H, n_q, d, ties), random_y(2, H, n_k, d, ties)
    Q = r.standard_normal((H, n_q, d)).astype(np.float32)
    K = r.standard_normal((H, n_k, d)).astype(np.float32)
    V = r.standard_normal((H, n_k, d)).astype(np.float32)
    if dtype == "bf16":
        Q, K, V = (inputs.round_to_bf16(x) for x in (Q, K, V))
    p = binding.make_problem(1, H, n_q, n_k, d, dtype, c_q, c_k, 1, flags=binding.CA_Y_IN)
    plan = binding.Plan(p, DEV)
    plan.cluster_qk(store(p, Q), store(p, K), store(p, V), Yq=to_dev(Yq[None]), Yk=to_dev(Yk[None]))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(H):
        # bit for bit the float32 restatement of the split decisions ...
        ref = orc.cluster_qk(Q[h], K[h], V[h], c_q, c_k, Yq32=Yq[h], Yk32=Yk[h], f32_decisions=True)
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, ref["perm_q"]), "query permutation differs"
        assert np.array_equal(pk, ref["perm_k"]), "key permutation differs"
        # ... and against the float64 definition: differences only at near-ties, < 0.1 % of the rows
        if n_k <= 200000:
            decisions.check_split_agreement(Yq[h], c_q, pq, f"queries {n_q} x {d}, head {h}")
            decisions.check_split_agreement(Yk[h], c_k, pk, f"keys {n_k} x {d}, head {h}")
        assert np.array_equal(plan.count_q[0, h].cpu().numpy(), ref["count_q"])
        assert np.array_equal(plan.count_k[0, h].cpu().numpy(), ref["count_k"])
        for got, src, perm, n, c in ((plan.Qp, Q, pq, n_q, c_q), (plan.Kp, K, pk, n_k, c_k),
                                     (plan.Vp, V, pk, n_k, c_k)):
            g = got[0, h].float().cpu().numpy()
            assert np.array_equal(g[:n], src[h][perm])            # rows moved, never changed
            assert np.all(g[n:] == 0)                             # padding of the short cluster
        for got, want in ((plan.cq, ref["cq"]), (plan.ck, ref["ck"]), (plan.cv, ref["cv"])):
            assert np.abs(got[0, h].cpu().numpy() - want).max() < 2e-6 * max(1.0, np.abs(want).max())


# Coordinates whose columns are permutations of one set of values: every column has the same
# variance in exact arithmetic, so which coordinate a set is split on is decided by the last bit of
# every rounding in the variance estimate.  A device sum that rounds once where the float32
# restatement rounds twice (a multiply and an add merged into a fused multiply-add) picks another
# coordinate for about two sets in three.  Shapes: sets with fewer rows than coordinates (a partly
# filled subsample), sets with at least d rows, and sets large enough for the per-level kernels.
EQUAL_VARIANCE_CASES = [
    # n, d, c
    (96, 128, 32), (300, 64, 16), (1500, 128, 16), (4096, 64, 128), (5000, 128, 64), (40000, 64, 128), (20000, 128, 128),
]


@pytest.mark.parametrize("n,d,c", EQUAL_VARIANCE_CASES)
def test_split_follows_the_float32_restatement_when_every_column_has_the_same_variance(n, d, c):
    H = 2
    r = np.random.default_rng(n * 131 + d)
    Y = np.empty((H, n, d), np.float32)
    for h in range(H):
        base = r.standard_normal(n).astype(np.float32)
        if h == 1:
            base = np.round(base * 4.0) / 4.0            # repeated values on top
        for t in range(d):
            Y[h, :, t] = r.permutation(base)
    X = inputs.round_to_bf16(r.standard_normal((H, n, d)).astype(np.float32))
    p = binding.make_problem(1, H, n, n, d, "bf16", c, c, 1, flags=binding.CA_Y_IN)
    plan = binding.Plan(p, DEV)
    plan.cluster_qk(store(p, X), store(p, X), store(p, X), Yq=to_dev(Y[None]), Yk=to_dev(Y[None, :, ::-1].copy()))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(H):
        assert np.array_equal(plan.perm_q[0, h].cpu().numpy(), orc.recursive_split_f32(Y[h], c)), f"queries, head {h}"
        assert np.array_equal(plan.perm_k[0, h].cpu().numpy(), orc.recursive_split_f32(Y[h, ::-1], c)), f"keys, head {h}"


# ----------------------------------------------------------------------------
# Full clustering stage: the device computes its own coordinates.  The oracle's
# splitter run on the device's coordinates must give the same permutation, and
# the coordinates must satisfy the basis-independent identities of the method.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("name,H,n_q,n_k", [("tiny", 2, 1024, 1024), ("tabular", 1, 2048, 6000),
                                             ("video480", 1, 4000, 4000)])
def test_cluster_qk_transforms_and_split(name, H, n_q, n_k):
    w = inputs.WORKLOADS[name].scaled(heads=H, n_q=n_q, n_k=n_k)
    if w.kind == "video":
        w = w.scaled(grid=(5, 25, 32))
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w, keep=min(w.keep, w.n_kc))
    plan = binding.Plan(p, DEV, keep_y=True)
    plan.cluster_qk(store(p, Q), store(p, K), store(p, V))
    torch.cuda.synchronize()
    d = w.head_dim
    for h in range(H):
        Yq, Yk = plan.Yq[0, h].cpu().numpy(), plan.Yk[0, h].cpu().numpy()
        # same split decisions as the oracle's splitter on these very coordinates
        assert np.array_equal(plan.perm_q[0, h].cpu().numpy(), orc.recursive_split_f32(Yq, w.cluster))
        assert np.array_equal(plan.perm_k[0, h].cpu().numpy(), orc.recursive_split_f32(Yk, w.cluster))
        decisions.check_split_agreement(Yq, w.cluster, plan.perm_q[0, h].cpu().numpy(), f"{name} queries, head {h}")
        decisions.check_split_agreement(Yk, w.cluster, plan.perm_k[0, h].cpu().numpy(), f"{name} keys, head {h}")
        # key coordinates are an isometry of the query-aware metric:
        # |Y_i - Y_j|^2 == (k_i - k_j)^T M (k_i - k_j), M = Q^T Q / n   (Section 3.2.2)
        M = orc.metric_q(Q[h])
        r = np.random.default_rng(h)
        i, j = r.integers(0, n_k, 200), r.integers(0, n_k, 200)
        dk = K[h][i].astype(np.float64) - K[h][j]
        want = np.einsum("nd,de,ne->n", dk, M, dk)
        got = ((Yk[i].astype(np.float64) - Yk[j]) ** 2).sum(1)
        assert np.abs(got - want).max() <= 2e-3 * want.max()
        # query coordinates are an isometry of r(q) = R_k q / |R_k q|
        R_k = orc.psd_root(orc.centered_scatter(K[h]))
        rq = orc.query_representation(Q[h], R_k)
        i, j = r.integers(0, n_q, 200), r.integers(0, n_q, 200)
        want = ((rq[i] - rq[j]) ** 2).sum(1)
        got = ((Yq[i].astype(np.float64) - Yq[j]) ** 2).sum(1)
        assert np.abs(got - want).max() <= 2e-3 * max(want.max(), 1e-12)
        # principal components: centred, decorrelated, variance in descending order
        for Y, ref in ((Yk, orc.diagonalize(orc.transform_keys(K[h], orc.psd_root(M)))[1]),
                       (Yq, orc.diagonalize(rq)[1])):
            Y = Y.astype(np.float64)
            scale = ref[0]
            assert np.abs(Y.mean(0)).max() < 1e-3 * np.sqrt(scale)
            cov = (Y.T @ Y) / Y.shape[0]
            assert np.abs(np.diag(cov) - ref).max() < 2e-3 * scale          # eigenvalues
            off = cov - np.diag(np.diag(cov))
            assert np.abs(off).max() < 2e-3 * scale
        # and the chain as a whole against the oracle's: coordinates column by column, the first split
        decisions.check_coordinates(f"{name} head {h}", w, Q[h], K[h], Yq, Yk, plan.perm_q[0, h].cpu().numpy(),
                                    plan.perm_k[0, h].cpu().numpy())
    assert all(v == 0 for v in plan.last_status().values())


# ----------------------------------------------------------------------------
# Block selection on the oracle's centroids (rounded to fp32): exact lists.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("H,n_qc,n_kc,d,keep", [(2, 16, 16, 64, 4), (1, 37, 300, 128, 1), (1, 5, 300, 64, 300),
                                                  (2, 130, 1024, 64, 128), (1, 9, 2049, 128, 77)])
def test_select_blocks_exact(H, n_qc, n_kc, d, keep):
    r = np.random.default_rng(n_qc * n_kc)
    cq = r.standard_normal((H, n_qc, d)).astype(np.float32)
    ck = r.standard_normal((H, n_kc, d)).astype(np.float32)
    ck[:, 3] = ck[:, 1]                      # duplicate centroids: exact score ties
    ck[:, n_kc - 1] = ck[:, 1]
    if n_qc > 4:
        cq[:, 4] = 0.0                       # a zero query centroid: every score ties at 0
    c = 16
    p = binding.make_problem(1, H, n_qc * c, n_kc * c, d, "fp32", c, c, keep)
    plan = binding.Plan(p, DEV)
    got = plan.select_blocks(to_dev(cq[None]), to_dev(ck[None])).cpu().numpy()[0]
    torch.cuda.synchronize()
    for h in range(H):
        # the scores are float32 with a fixed operation order on both sides: the lists are equal;
        # against the float64 scores they differ only where the k-th and (k+1)-th score tie
        assert np.array_equal(got[h], orc.select_blocks_f32(cq[h], ck[h], keep)), h
        decisions.check_selection_agreement(cq[h], ck[h], keep, got[h], f"{n_qc} x {n_kc}, keep {keep}, head {h}")


# ----------------------------------------------------------------------------
# Attention on the oracle's permutation and block lists.
# ----------------------------------------------------------------------------
def attention_case(w, H, keep, compensate, flags=0, perm_seed=None, cluster_k=None, adaptive=None, quantized=False):
    Q, K, V = inputs.generate(w.scaled(heads=H))
    c_q, c_k = w.cluster, (cluster_k or w.cluster)
    p = binding.problem_from_workload(w, heads=H, keep=keep, compensate=compensate, flags=flags,
                                      cluster_q=c_q, cluster_k=c_k)
    plan = binding.Plan(p, DEV)
    refs = []
    arrs = {k: [] for k in ("perm_q", "Qp", "Kp", "Vp", "ck", "cv", "count_k", "idx")}
    for h in range(H):
        if perm_seed is None:
            cl = orc.cluster_qk(Q[h], K[h], V[h], c_q, c_k)
        else:                                # any valid permutation must work
            r = np.random.default_rng(perm_seed + h)
            pq, pk = r.permutation(w.n_q), r.permutation(w.n_k)
            cq_, nq_ = orc.centroids(Q[h], pq, c_q)
            ck_, nk_ = orc.centroids(K[h], pk, c_k)
            cv_, _ = orc.centroids(V[h], pk, c_k)
            cl = dict(perm_q=pq, perm_k=pk, cq=cq_, ck=ck_, cv=cv_, count_q=nq_, count_k=nk_)
        if adaptive is None:
            idx = orc.select_blocks(cl["cq"], cl["ck"], keep)
        else:                                # lists of different lengths (Section 3.3.2)
            idx = orc.select_blocks_adaptive(cl["cq"], cl["ck"], cl["count_k"], adaptive[0], adaptive[1])
        ck32, cv32 = cl["ck"].astype(np.float32), cl["cv"].astype(np.float32)
        attend = orc.cluster_attention_quantized_qk if quantized else orc.cluster_attention
        o, lse = attend(Q[h], K[h], V[h], cl["perm_q"], cl["perm_k"], c_q, c_k, idx, compensate,
                        ck=ck32, cv=cv32, count_k=cl["count_k"])
        refs.append((o, lse))

        def pad(x, perm, n, c):
            out = np.zeros((-(-n // c) * c, x.shape[1]), np.float32)
            out[:n] = x[perm]
            return out
        arrs["perm_q"].append(cl["perm_q"].astype(np.int32))
        arrs["Qp"].append(pad(Q[h], cl["perm_q"], w.n_q, c_q))
        arrs["Kp"].append(pad(K[h], cl["perm_k"], w.n_k, c_k))
        arrs["Vp"].append(pad(V[h], cl["perm_k"], w.n_k, c_k))
        arrs["ck"].append(ck32)
        arrs["cv"].append(cv32)
        arrs["count_k"].append(cl["count_k"].astype(np.int32))
        if adaptive is None:
            arrs["idx"].append(idx.astype(np.int32))
        else:
            padded = np.full((len(idx), p.n_kc), -1, np.int32)
            for i, row in enumerate(idx):
                padded[i, :len(row)] = row
            arrs["idx"].append(padded)
            arrs.setdefault("keep_count", []).append(np.array([len(row) for row in idx], np.int32))
    st = {k: np.stack(v)[None] for k, v in arrs.items()}
    dt = binding.torch_dtype(p)
    if adaptive is None:
        O, lse = plan.cluster_attention_fwd(to_dev(st["Qp"], dt), to_dev(st["Kp"], dt), to_dev(st["Vp"], dt),
                                            to_dev(st["ck"]), to_dev(st["cv"]), to_dev(st["count_k"]),
                                            to_dev(st["idx"]), to_dev(st["perm_q"]))
    else:
        O, lse = plan.cluster_attention_fwd_ragged(to_dev(st["idx"]), to_dev(st["keep_count"]),
                                                   to_dev(st["Qp"], dt), to_dev(st["Kp"], dt), to_dev(st["Vp"], dt),
                                                   to_dev(st["ck"]), to_dev(st["cv"]), to_dev(st["count_k"]),
                                                   to_dev(st["perm_q"]))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    return O[0].float().cpu().numpy(), lse[0].cpu().numpy(), refs


@pytest.mark.parametrize("compensate", [True, False])
def test_attention_fp32_tiny_configuration(compensate):
    w = inputs.WORKLOADS["tiny"]
    O, lse, refs = attention_case(w, 2, w.keep, compensate)
    for h, (o_ref, lse_ref) in enumerate(refs):
        assert np.abs(O[h] - o_ref).max() < 1e-5
        assert np.abs(lse[h] - lse_ref).max() < 1e-5 * max(1.0, np.abs(lse_ref).max())


@pytest.mark.parametrize("n_q,n_k,c,keep", [(1000, 1531, 64, 5), (300, 300, 128, 3), (260, 4000, 32, 125)])
def test_attention_fp32_ragged_and_arbitrary_permutation(n_q, n_k, c, keep):
    w = inputs.WORKLOADS["tiny"].scaled(n_q=n_q, n_k=n_k, cluster=c)
    O, lse, refs = attention_case(w, 1, keep, True, perm_seed=7)
    assert np.abs(O[0] - refs[0][0]).max() < 1e-5
    assert np.abs(lse[0] - refs[0][1]).max() < 1e-5 * max(1.0, np.abs(refs[0][1]).max())


def bf16_close(O, o_ref):
    return np.abs(O - o_ref).max() <= 2e-2 and np.linalg.norm(O - o_ref) <= 5e-3 * np.linalg.norm(o_ref)


@pytest.mark.parametrize("name,n_q,n_k,keep,compensate,flags", [
    ("tabular", 1024, 4096, 4, True, 0), ("tabular", 1024, 4096, 4, False, 0),
    ("video480", 1000, 1000, 2, True, 0), ("sweep", 2048, 2048, 16, True, 0),
    ("tabular", 512, 2048, 4, True, binding.CA_ATTN_FP32),
    ("sweep64", 1100, 3000, 9, True, 0),          # 64-row clusters on both sides, short last clusters
    ("sweep256", 1024, 2100, 3, True, 0),         # 256-row clusters: two CTAs per query cluster
    ("sweep32k", 640, 1000, 11, False, 0),        # 32-row key clusters packed four to a tile
    ("sweep64x128", 1100, 3000, 5, True, 0),      # 64 query rows x 128 key rows: the paper's block shape
])
def test_attention_bf16(name, n_q, n_k, keep, compensate, flags):
    variants = {"sweep64": ("sweep", 64, 64), "sweep256": ("sweep", 256, 256), "sweep32k": ("sweep", 128, 32),
                "sweep64x128": ("sweep", 64, 128)}
    cluster_k = None
    if name in variants:
        name, cq_, cluster_k = variants[name]
        w = inputs.WORKLOADS[name].scaled(n_q=n_q, n_k=n_k, cluster=cq_)
    else:
        w = inputs.WORKLOADS[name].scaled(n_q=n_q, n_k=n_k)
    if w.kind == "video":
        w = w.scaled(grid=(5, 10, 20))
    O, lse, refs = attention_case(w, 2, keep, compensate, flags=flags, cluster_k=cluster_k)
    for h, (o_ref, lse_ref) in enumerate(refs):
        assert bf16_close(O[h], o_ref), (np.abs(O[h] - o_ref).max(),
                                         np.linalg.norm(O[h] - o_ref) / np.linalg.norm(o_ref))
        assert np.abs(lse[h] - lse_ref).max() < 2e-2


@pytest.mark.parametrize("name,n_q,n_k,c_q,c_k,keep,compensate,perm_seed", [
    ("video480", 1000, 1000, 128, 128, 2, True, None),     # short last clusters, centroid columns
    ("sweep", 2048, 2048, 128, 128, 16, True, None),       # all blocks kept but none short
    ("sweep", 1100, 3000, 64, 64, 9, True, 5),             # 64-row clusters: one key scale per half-step
    ("sweep", 1100, 3000, 64, 128, 5, False, None),        # the paper's block shape, no compensation
    ("sweep", 1024, 2100, 256, 256, 3, True, 6),           # two CTAs per query cluster, two tiles per key cluster
])
def test_attention_with_quantised_qk(name, n_q, n_k, c_q, c_k, keep, compensate, perm_seed):
    """CA_ATTN_FP8_QK: Q K^T on E4M3 codes with a scale per query row, per key cluster and per run
    of 64 key centroids (Section 3.1 / 5.1: the paper's kernel is a quantised one).  The codes are
    taken in float32 the same way on both sides and their products are exact, so the result is held
    to the bf16 tolerances against the oracle's attention on the de-quantised tensors -- and it
    differs visibly from the unquantised attention."""
    w = inputs.WORKLOADS[name].scaled(n_q=n_q, n_k=n_k, cluster=c_q)
    if w.kind == "video":
        w = w.scaled(grid=(5, 10, 20))
    O, lse, refs = attention_case(w, 2, keep, compensate, flags=binding.CA_ATTN_FP8_QK, cluster_k=c_k,
                                  perm_seed=perm_seed, quantized=True)
    _, _, plain = attention_case(w, 2, keep, compensate, cluster_k=c_k, perm_seed=perm_seed)
    for h, (o_ref, lse_ref) in enumerate(refs):
        assert bf16_close(O[h], o_ref), (np.abs(O[h] - o_ref).max(), np.linalg.norm(O[h] - o_ref) / np.linalg.norm(o_ref))
        assert np.abs(lse[h] - lse_ref).max() < 2e-2
        # the quantisation itself is a larger step than the tolerance of the comparison
        assert np.linalg.norm(plain[h][0] - o_ref) > 2 * np.linalg.norm(O[h] - o_ref)


def test_quantised_qk_is_refused_where_it_is_not_built():
    p = binding.make_problem(1, 1, 512, 512, 64, "bf16", 128, 128, 2, flags=binding.CA_ATTN_FP8_QK)
    plan = binding.Plan(p.copy(flags=0), DEV)
    plan.problem = p
    with pytest.raises(binding.ClusterAttnError, match="CA_ERR_UNSUPPORTED"):
        plan.cluster_attention_fwd()


def test_all_blocks_kept_is_dense_attention_on_device():
    w = inputs.WORKLOADS["tiny"]
    O, lse, _ = attention_case(w, 1, w.n_kc, False)
    Q, K, V = inputs.generate(w.scaled(heads=1))
    od, lsed = orc.dense_attention(Q[0], K[0], V[0], return_lse=True)
    assert np.abs(O[0] - od).max() < 1e-5 and np.abs(lse[0] - lsed).max() < 1e-5


# ----------------------------------------------------------------------------
# The whole path on the tiny configuration, every stage on the device.
# ----------------------------------------------------------------------------
def test_end_to_end_tiny_configuration():
    w = inputs.WORKLOADS["tiny"]
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w)
    plan = binding.Plan(p, DEV, keep_y=True)
    O = plan.forward(store(p, Q), store(p, K), store(p, V), want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(w.heads):
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        idx = plan.block_idx[0, h].cpu().numpy()
        # selection agrees with the oracle's on the device's own centroids
        want_idx = orc.select_blocks_f32(plan.cq[0, h].cpu().numpy(), plan.ck[0, h].cpu().numpy(), w.keep)
        assert np.array_equal(idx, want_idx)
        decisions.check_selection_agreement(plan.cq[0, h].cpu().numpy(), plan.ck[0, h].cpu().numpy(), w.keep, idx,
                                            f"tiny head {h}")
        # attention agrees with the oracle's on the device's own clustering and selection
        o_ref, lse_ref = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, w.cluster, w.cluster, idx, True,
                                               ck=plan.ck[0, h].cpu().numpy(), cv=plan.cv[0, h].cpu().numpy(),
                                               count_k=plan.count_k[0, h].cpu().numpy())
        assert np.abs(O[0, h].cpu().numpy() - o_ref).max() < 1e-5
        # the split decisions against the float64 definition, and the whole chain from Q and K to the
        # coordinates against the oracle's own chain
        Yq, Yk = plan.Yq[0, h].cpu().numpy(), plan.Yk[0, h].cpu().numpy()
        decisions.check_split_agreement(Yq, w.cluster, pq, f"tiny queries, head {h}")
        decisions.check_split_agreement(Yk, w.cluster, pk, f"tiny keys, head {h}")
        decisions.check_coordinates(f"tiny head {h}", w, Q[h], K[h], Yq, Yk, pq, pk)


# ----------------------------------------------------------------------------
# Adaptive selection (Section 3.3.2): float32 mass estimates with a fixed recipe
# on both sides, so lists and their lengths are equal bit for bit.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("H,n_qc,n_kc,d,spread", [(2, 16, 16, 64, 1.0), (1, 37, 300, 128, 1.0),
                                                    (2, 130, 1024, 64, 3.0), (1, 9, 2049, 128, 0.2),
                                                    (1, 20, 1500, 64, 12.0)])
@pytest.mark.parametrize("recall,min_count", [(0.5, 1), (0.9, 16), (0.999, 4), (1.0, 1)])
def test_select_blocks_adaptive_exact(H, n_qc, n_kc, d, spread, recall, min_count):
    r = np.random.default_rng(n_qc * n_kc + d)
    cq = (r.standard_normal((H, n_qc, d)) * spread).astype(np.float32)
    ck = r.standard_normal((H, n_kc, d)).astype(np.float32)
    ck[:, 3] = ck[:, 1]                      # duplicate centroids: equal masses, ordered by index
    ck[:, n_kc - 1] = ck[:, 1]
    if n_qc > 4:
        cq[:, 4] = 0.0                       # every score equal: the mass is the member count alone
    c = 16
    count = np.full((H, n_kc), c, np.int32)
    count[:, -1] = 5                         # a short last cluster weighs less
    scale = float(np.float32(1.0 / np.sqrt(d)))
    p = binding.make_problem(1, H, n_qc * c, n_kc * c - 11, d, "fp32", c, c, 1, softmax_scale=scale)
    plan = binding.Plan(p, DEV)
    idx, keep = plan.select_blocks_adaptive(recall, min_count, to_dev(cq[None]), to_dev(ck[None]),
                                            to_dev(count[None]))
    torch.cuda.synchronize()
    idx, keep = idx.cpu().numpy()[0], keep.cpu().numpy()[0]
    lengths = set()
    for h in range(H):
        want = orc.select_blocks_adaptive(cq[h], ck[h], count[h], recall, min_count, scale=scale)
        for i, row in enumerate(want):
            assert keep[h, i] == len(row), (h, i, keep[h, i], len(row))
            assert np.array_equal(idx[h, i, :len(row)], row), (h, i)
            assert (idx[h, i, len(row):] == -1).all()
            lengths.add(len(row))
    if recall < 1.0 and spread >= 1.0 and n_kc > 16:
        assert len(lengths) > 1              # the case does exercise lists of different lengths


@pytest.mark.parametrize("name,n_q,n_k,dtype_flags,recall", [
    ("tiny", 1024, 1024, 0, 0.9),                      # fp32 storage: CUDA-core kernel
    ("tabular", 1024, 4096, 0, 0.8),                   # bf16 on the tensor cores
    ("tabular", 1000, 4000, binding.CA_ATTN_FP32, 0.95),
    ("video480", 1000, 1000, 0, 0.9),
    ("sweep64", 1100, 3000, 0, 0.9),
])
def test_attention_ragged_lists(name, n_q, n_k, dtype_flags, recall):
    if name == "sweep64":
        w = inputs.WORKLOADS["sweep"].scaled(n_q=n_q, n_k=n_k, cluster=64)
    else:
        w = inputs.WORKLOADS[name].scaled(n_q=n_q, n_k=n_k)
    if w.kind == "video":
        w = w.scaled(grid=(5, 10, 20))
    O, lse, refs = attention_case(w, 2, 1, True, flags=dtype_flags, adaptive=(recall, 2))
    for h, (o_ref, lse_ref) in enumerate(refs):
        if w.dtype == "fp32":
            assert np.abs(O[h] - o_ref).max() < 1e-5 and np.abs(lse[h] - lse_ref).max() < 1e-5
        else:
            assert bf16_close(O[h], o_ref)
            assert np.abs(lse[h] - lse_ref).max() < 2e-2


def test_end_to_end_adaptive_tiny_configuration():
    """cluster_qk with the un-normalised query representation (Appendix B.1), adaptive
    selection and attention over the resulting ragged lists, every stage on the device."""
    w = inputs.WORKLOADS["tiny"]
    Q, K, V = inputs.generate(w)
    scale = float(np.float32(1.0 / np.sqrt(w.head_dim)))
    p = binding.problem_from_workload(w, flags=binding.CA_QUERY_UNNORMALIZED, softmax_scale=scale)
    plan = binding.Plan(p, DEV, keep_y=True)
    O, lse = plan.forward_adaptive(store(p, Q), store(p, K), store(p, V), recall=0.9, min_count=2, want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(w.heads):
        Yq = plan.Yq[0, h].cpu().numpy()
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, orc.recursive_split_f32(Yq, w.cluster))
        # query coordinates are an isometry of r(q) = R_k q, R_k = sqrt(K_c^T K_c / n)
        R_k = orc.psd_root(orc.centered_scatter(K[h]) / w.n_k)
        rq = orc.query_representation(Q[h], R_k, normalize=False)
        r = np.random.default_rng(h)
        i, j = r.integers(0, w.n_q, 200), r.integers(0, w.n_q, 200)
        want = ((rq[i] - rq[j]) ** 2).sum(1)
        got = ((Yq[i].astype(np.float64) - Yq[j]) ** 2).sum(1)
        assert np.abs(got - want).max() <= 2e-3 * want.max()
        decisions.check_coordinates(f"tiny, un-normalised queries, head {h}", w, Q[h], K[h], Yq,
                                    plan.Yk[0, h].cpu().numpy(), pq, pk, adaptive=True)
        lists = orc.select_blocks_adaptive(plan.cq[0, h].cpu().numpy(), plan.ck[0, h].cpu().numpy(),
                                           plan.count_k[0, h].cpu().numpy(), 0.9, 2, scale=scale)
        keep = plan.keep_count[0, h].cpu().numpy()
        idx = plan.block_idx_ragged[0, h].cpu().numpy()
        for i, row in enumerate(lists):
            assert keep[i] == len(row) and np.array_equal(idx[i, :len(row)], row)
        o_ref, lse_ref = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, w.cluster, w.cluster, lists, True,
                                               ck=plan.ck[0, h].cpu().numpy(), cv=plan.cv[0, h].cpu().numpy(),
                                               count_k=plan.count_k[0, h].cpu().numpy())
        assert np.abs(O[0, h].cpu().numpy() - o_ref).max() < 1e-5
        assert np.abs(lse[0, h].cpu().numpy() - lse_ref).max() < 1e-5


def test_end_to_end_asymmetric_clusters_64_by_128():
    """The block shape of the paper's attention kernel (64 query rows x 128 key rows) through every
    stage on the device, bf16, d = 64: clustering with different cluster sizes on the two sides,
    selection, attention; each stage checked against the oracle on the device's own inputs."""
    w = inputs.WORKLOADS["tabular"].scaled(heads=2, n_q=2000, n_k=6000)
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w, cluster_q=64, cluster_k=128, keep=6)
    plan = binding.Plan(p, DEV, keep_y=True)
    O = plan.forward(store(p, Q), store(p, K), store(p, V), want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(w.heads):
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, orc.recursive_split_f32(plan.Yq[0, h].cpu().numpy(), 64))
        assert np.array_equal(pk, orc.recursive_split_f32(plan.Yk[0, h].cpu().numpy(), 128))
        idx = plan.block_idx[0, h].cpu().numpy()
        assert np.array_equal(idx, orc.select_blocks_f32(plan.cq[0, h].cpu().numpy(), plan.ck[0, h].cpu().numpy(), 6))
        o_ref, _ = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, 64, 128, idx, True,
                                         ck=plan.ck[0, h].cpu().numpy(), cv=plan.cv[0, h].cpu().numpy(),
                                         count_k=plan.count_k[0, h].cpu().numpy())
        assert bf16_close(O[0, h].float().cpu().numpy(), o_ref)


# ----------------------------------------------------------------------------
# Selection on random shapes: both the fused kernel and, from 2,048 key clusters
# on, the tiled scores + one row per CTA; top-k and adaptive, exact lists.
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_selection_random_shapes_exact(seed):
    r = np.random.default_rng(1000 + seed)
    d = int(r.choice([64, 128]))
    H = int(r.integers(1, 3))
    n_qc = int(r.integers(1, 200))
    n_kc = int(r.choice([r.integers(1, 300), r.integers(2048, 2600)]))
    keep = int(r.integers(1, n_kc + 1))
    cq = (r.standard_normal((H, n_qc, d)) * r.uniform(0.2, 4.0)).astype(np.float32)
    ck = r.standard_normal((H, n_kc, d)).astype(np.float32)
    dup = r.integers(0, n_kc, max(1, n_kc // 10))
    ck[:, dup] = ck[:, dup[0]][:, None, :]                  # a tenth of the key centroids coincide
    count = r.integers(1, 17, (H, n_kc)).astype(np.int32)
    c = 16
    scale = float(np.float32(1.0 / np.sqrt(d)))
    p = binding.make_problem(1, H, n_qc * c, n_kc * c, d, "fp32", c, c, keep, softmax_scale=scale)
    plan = binding.Plan(p, DEV)
    got = plan.select_blocks(to_dev(cq[None]), to_dev(ck[None])).cpu().numpy()[0]
    recall = float(r.choice([0.3, 0.7, 0.95]))
    min_count = int(r.integers(1, 20))
    idx, kc = plan.select_blocks_adaptive(recall, min_count, to_dev(cq[None]), to_dev(ck[None]), to_dev(count[None]))
    torch.cuda.synchronize()
    idx, kc = idx.cpu().numpy()[0], kc.cpu().numpy()[0]
    for h in range(H):
        assert np.array_equal(got[h], orc.select_blocks_f32(cq[h], ck[h], keep)), (seed, h)
        decisions.check_selection_agreement(cq[h], ck[h], keep, got[h], f"seed {seed}, head {h}")
        want = orc.select_blocks_adaptive(cq[h], ck[h], count[h], recall, min_count, scale=scale)
        for i, row in enumerate(want):
            assert kc[h, i] == len(row) and np.array_equal(idx[h, i, :len(row)], row), (seed, h, i)


@pytest.mark.parametrize("seed", range(10))
def test_attention_random_shapes(seed):
    """Random sizes, cluster sizes, densities and arbitrary permutations (ragged tails on both
    sides); bf16 on the tensor-core kernel and fp32 on the CUDA-core kernel."""
    r = np.random.default_rng(2000 + seed)
    base = "tabular" if r.integers(0, 2) == 0 else "sweep"              # d = 64 / d = 128
    c_q = int(r.choice([64, 128, 256]))
    c_k = int(r.choice([16, 32, 64, 128, 256]))
    n_q = int(r.integers(c_q // 2, 5 * c_q))
    n_k = int(r.integers(c_k, 40 * c_k))
    n_kc = -(-n_k // c_k)
    keep = int(r.integers(1, n_kc + 1))
    compensate = bool(r.integers(0, 2))
    w = inputs.WORKLOADS[base].scaled(n_q=n_q, n_k=n_k, cluster=c_q)
    if seed % 5 == 4:
        w = w.scaled(dtype="fp32")
    O, lse, refs = attention_case(w, 2, keep, compensate, perm_seed=seed, cluster_k=c_k)
    for h, (o_ref, lse_ref) in enumerate(refs):
        if w.dtype == "fp32":
            assert np.abs(O[h] - o_ref).max() < 1e-5 and np.abs(lse[h] - lse_ref).max() < 1e-5, (seed, h)
        else:
            assert bf16_close(O[h], o_ref), (seed, h, c_q, c_k, n_q, n_k, keep, compensate,
                                             np.abs(O[h] - o_ref).max())
            assert np.abs(lse[h] - lse_ref).max() < 2e-2

"""Basic recursive splitting with the injected metric (Section 3.2.1, Section 5.2): the device
against the oracle, through the C ABI.  Both sides take every floating-point step in float32 with
the same operation order, so permutations are compared bit for bit."""
import numpy as np
import pytest
import torch

from oracle import clusterattn_oracle as orc
from paper_2608_26965_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load_library()


def dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a)).to(dtype).to(DEV)


def noise_for(r, H, rows, d):
    return r.standard_normal((H, rows, d)).astype(np.float32)


CASES = [
    # H, n_q, n_k, d, c_q, c_k, dtype, iterations
    (2, 1024, 1024, 64, 64, 64, "fp32", 3),
    (2, 1000, 1531, 64, 64, 32, "fp32", 2),          # ragged sizes, short last clusters
    (1, 50, 200, 64, 64, 128, "bf16", 3),            # no split on one side, one on the other
    (1, 3000, 4099, 128, 128, 128, "bf16", 3),
    (1, 2048, 40000, 64, 128, 128, "bf16", 1),       # sets larger than the shared-memory window
    (1, 640, 704, 128, 256, 16, "bf16", 0),          # no iteration: the start vectors decide
    (1, 700, 5000, 128, 64, 128, "fp32", 2),         # float32 rows at d = 128: two subsets staged per round
]


@pytest.mark.parametrize("H,n_q,n_k,d,c_q,c_k,dtype,iterations", CASES)
def test_basic_split_with_given_metrics_is_bit_exact(H, n_q, n_k, d, c_q, c_k, dtype, iterations):
    r = np.random.default_rng(n_q + n_k + d)
    spread = np.linspace(2.0, 0.3, d)
    Q = (r.standard_normal((H, n_q, d)) * spread).astype(np.float32)
    K = (r.standard_normal((H, n_k, d)) * spread[::-1] + 0.5).astype(np.float32)
    V = r.standard_normal((H, n_k, d)).astype(np.float32)
    if dtype == "bf16":
        Q, K, V = (inputs.round_to_bf16(x) for x in (Q, K, V))
        Q[:, ::7] = Q[:, :1]                             # duplicated rows: exact ties in every projection
    p = binding.make_problem(1, H, n_q, n_k, d, dtype, c_q, c_k, 1, flags=binding.CA_METRIC_IN)
    plan = binding.Plan(p, DEV)
    rows_q, rows_k, _ = plan.basic_noise_rows()
    assert rows_q == (1 << max(1, orc.split_levels(n_q, c_q))) - 1
    assert rows_k == (1 << max(1, orc.split_levels(n_k, c_k))) - 1
    nq, nk = noise_for(r, H, rows_q, d), noise_for(r, H, rows_k, d)
    A_q = np.stack([orc.basic_metrics(Q[h], K[h])[0] for h in range(H)]).astype(np.float32)
    A_k = np.stack([orc.basic_metrics(Q[h], K[h])[1] for h in range(H)]).astype(np.float32)
    dt = binding.torch_dtype(p)
    plan.cluster_qk_basic(dev(Q[None], dt), dev(K[None], dt), dev(V[None], dt), dev(nq[None]), dev(nk[None]),
                          iterations, A_q=dev(A_q[None]), A_k=dev(A_k[None]))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(H):
        want_q = orc.basic_recursive_split(Q[h], A_q[h], nq[h], c_q, iterations)
        want_k = orc.basic_recursive_split(K[h], A_k[h], nk[h], c_k, iterations)
        assert np.array_equal(plan.perm_q[0, h].cpu().numpy(), want_q), f"query permutation, head {h}"
        assert np.array_equal(plan.perm_k[0, h].cpu().numpy(), want_k), f"key permutation, head {h}"
        # gathered rows and counts follow the permutation
        Kp = plan.Kp[0, h].float().cpu().numpy()
        assert np.array_equal(Kp[:n_k], K[h][want_k])
        cnt = plan.count_k[0, h].cpu().numpy()
        assert cnt.sum() == n_k and (cnt[:-1] == c_k).all()
        ck_ref, _ = orc.centroids(K[h], want_k, c_k)
        assert np.abs(plan.ck[0, h].cpu().numpy() - ck_ref).max() < 2e-6 * max(1.0, np.abs(ck_ref).max())


@pytest.mark.parametrize("name,H,n_q,n_k", [("tiny", 2, 1024, 1024), ("tabular", 1, 2048, 6000)])
def test_basic_split_with_device_metrics_and_attention(name, H, n_q, n_k):
    """The device computes the metric matrices itself; the oracle's splitter on those matrices gives
    the same permutation, the matrices are the paper's (Section 3.2.2), and selection + attention on
    the resulting clustering agree with the oracle."""
    w = inputs.WORKLOADS[name].scaled(heads=H, n_q=n_q, n_k=n_k)
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w, keep=min(w.keep, w.n_kc))
    plan = binding.Plan(p, DEV)
    rows_q, rows_k, _ = plan.basic_noise_rows()
    r = np.random.default_rng(3)
    nq, nk = noise_for(r, H, rows_q, w.head_dim), noise_for(r, H, rows_k, w.head_dim)
    dt = binding.torch_dtype(p)
    plan.cluster_qk_basic(dev(Q[None], dt), dev(K[None], dt), dev(V[None], dt), dev(nq[None]), dev(nk[None]), 3)
    plan.select_blocks()
    O, lse = plan.cluster_attention_fwd(want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    c = w.cluster
    for h in range(H):
        A_q, A_k = plan.A_q[0, h].cpu().numpy(), plan.A_k[0, h].cpu().numpy()
        ref_q, ref_k = orc.basic_metrics(Q[h], K[h])
        assert np.abs(A_q - ref_q).max() < 1e-4 * np.abs(ref_q).max()
        assert np.abs(A_k - ref_k).max() < 1e-4 * np.abs(ref_k).max()
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, orc.basic_recursive_split(Q[h], A_q, nq[h], c, 3))
        assert np.array_equal(pk, orc.basic_recursive_split(K[h], A_k, nk[h], c, 3))
        idx = plan.block_idx[0, h].cpu().numpy()
        assert np.array_equal(idx, orc.select_blocks_f32(plan.cq[0, h].cpu().numpy(), plan.ck[0, h].cpu().numpy(), p.keep))
        o_ref, lse_ref = orc.cluster_attention(Q[h], K[h], V[h], pq, pk, c, c, idx, True,
                                               ck=plan.ck[0, h].cpu().numpy(), cv=plan.cv[0, h].cpu().numpy(),
                                               count_k=plan.count_k[0, h].cpu().numpy())
        got = O[0, h].float().cpu().numpy()
        if w.dtype == "fp32":
            assert np.abs(got - o_ref).max() < 1e-5
        else:
            assert np.abs(got - o_ref).max() <= 2e-2 and np.linalg.norm(got - o_ref) <= 5e-3 * np.linalg.norm(o_ref)
        # the clusters are tighter than random ones even in the plain Euclidean sense
        Kh = K[h].astype(np.float64)
        tight = np.mean([Kh[pk[j * c:(j + 1) * c]].var(0).sum() for j in range(w.n_kc)])
        rand = np.mean([Kh[r.permutation(n_k)[:c]].var(0).sum() for _ in range(20)])
        assert tight < 0.95 * rand

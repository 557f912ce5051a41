"""Random shapes through the splitters (Section 3.2.1), bit for bit against the oracle.

The fixed cases of test_gpu_parity.py pin the paths the full-size launches take; these draw the
sizes, cluster sizes, head dimension, storage type and the amount of repeated values from a seeded
generator, so that partly filled subsamples, one-row tails, sets just above and just below the
sizes at which the kernels change paths, and exact ties all occur in combinations nobody listed.
"""
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


def _to_dev(a, dtype=torch.float32):
    return torch.from_numpy(np.ascontiguousarray(a[None])).to(dtype).to(DEV)


def _draw(seed):
    r = np.random.default_rng(26965 + seed)
    d = int(r.choice([64, 128]))
    c_q = int(r.choice([16, 32, 64, 128, 256]))
    c_k = int(r.choice([16, 32, 64, 128, 256]))
    n_q = int(r.integers(1, 20000))
    n_k = int(r.integers(1, 50000))
    H = int(r.integers(1, 3))
    dtype = str(r.choice(["bf16", "fp32"]))
    ties = int(r.integers(0, 3))                     # 0: none, 1: quarters, 2: halves with signed zeros
    return r, d, c_q, c_k, n_q, n_k, H, dtype, ties


@pytest.mark.parametrize("seed", range(16))
def test_diagonalized_split_on_random_shapes(seed):
    r, d, c_q, c_k, n_q, n_k, H, dtype, ties = _draw(seed)
    Yq = r.standard_normal((H, n_q, d)).astype(np.float32)
    Yk = r.standard_normal((H, n_k, d)).astype(np.float32)
    if ties == 1:
        Yq, Yk = np.round(Yq * 4) / 4, np.round(Yk * 4) / 4
    elif ties == 2:
        Yq, Yk = np.round(Yq * 2) / 2, np.round(Yk * 2) / 2
        Yk[:, ::5, :] = -0.0
    Q = r.standard_normal((H, n_q, d)).astype(np.float32)
    K = r.standard_normal((H, n_k, d)).astype(np.float32)
    if dtype == "bf16":
        Q, K = inputs.round_to_bf16(Q), inputs.round_to_bf16(K)
    p = binding.make_problem(1, H, n_q, n_k, d, dtype, c_q, c_k, 1, flags=binding.CA_Y_IN)
    plan = binding.Plan(p, DEV)
    dt = binding.torch_dtype(p)
    plan.cluster_qk(_to_dev(Q, dt), _to_dev(K, dt), _to_dev(K, dt), Yq=_to_dev(Yq), Yk=_to_dev(Yk))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    what = f"d={d} c=({c_q},{c_k}) n=({n_q},{n_k}) {dtype} ties={ties}"
    for h in range(H):
        pq, pk = plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(pq, orc.recursive_split_f32(Yq[h], c_q)), f"queries, head {h}: {what}"
        assert np.array_equal(pk, orc.recursive_split_f32(Yk[h], c_k)), f"keys, head {h}: {what}"
        assert np.array_equal(plan.Kp[0, h, :n_k].float().cpu().numpy(), K[h][pk]), f"gathered keys, head {h}: {what}"


@pytest.mark.parametrize("seed", range(8))
def test_basic_split_on_random_shapes(seed):
    r, d, c_q, c_k, n_q, n_k, H, dtype, _ = _draw(100 + seed)
    n_q, n_k = min(n_q, 6000), min(n_k, 12000)
    c_q, c_k = max(c_q, 32), max(c_k, 32)
    iterations = int(r.integers(0, 4))
    Q = r.standard_normal((H, n_q, d)).astype(np.float32)
    K = r.standard_normal((H, n_k, d)).astype(np.float32)
    if dtype == "bf16":
        Q, K = inputs.round_to_bf16(Q), inputs.round_to_bf16(K)
    p = binding.make_problem(1, H, n_q, n_k, d, dtype, c_q, c_k, 1, flags=binding.CA_METRIC_IN)
    plan = binding.Plan(p, DEV)
    dt = binding.torch_dtype(p)
    rows_q, rows_k, _ = plan.basic_noise_rows()
    noise_q = r.standard_normal((H, rows_q, d)).astype(np.float32)
    noise_k = r.standard_normal((H, rows_k, d)).astype(np.float32)
    A_q = np.stack([np.cov(r.standard_normal((3 * d, d)).T) for _ in range(H)]).astype(np.float32)
    A_k = np.stack([np.cov(r.standard_normal((3 * d, d)).T) for _ in range(H)]).astype(np.float32)
    plan.cluster_qk_basic(_to_dev(Q, dt), _to_dev(K, dt), _to_dev(K, dt), _to_dev(noise_q), _to_dev(noise_k),
                          iterations, A_q=_to_dev(A_q), A_k=_to_dev(A_k))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    what = f"d={d} c=({c_q},{c_k}) n=({n_q},{n_k}) {dtype} iterations={iterations}"
    for h in range(H):
        ref_q = orc.basic_recursive_split(Q[h], A_q[h], noise_q[h], c_q, iterations)
        ref_k = orc.basic_recursive_split(K[h], A_k[h], noise_k[h], c_k, iterations)
        assert np.array_equal(plan.perm_q[0, h].cpu().numpy(), ref_q), f"queries, head {h}: {what}"
        assert np.array_equal(plan.perm_k[0, h].cpu().numpy(), ref_k), f"keys, head {h}: {what}"

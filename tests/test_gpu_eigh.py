"""The eigen-decomposition of the principal-component kernel (Section 3.2.1, diagonalized variant) on
matrices with known or awkward spectra, against LAPACK (numpy.linalg.eigh in float64) and against
what defines an eigen-decomposition: orthonormal columns, A W = W diag(lambda), descending order.
The kernel works in float32: the bounds are a few units of float32 rounding times the size of A."""
import numpy as np
import pytest
import torch

from paper_2608_26965_b200 import binding

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run(mats):
    A = torch.from_numpy(np.ascontiguousarray(np.stack(mats))).to(torch.float64).to(DEV)
    W, ev = binding.debug_eigh(A)
    torch.cuda.synchronize()
    return W.cpu().numpy().astype(np.float64), ev.cpu().numpy()


def check(A, W, ev, label, vectors_unique=True):
    d = A.shape[0]
    size = max(np.abs(A).max(), 1e-30)
    ref = np.linalg.eigvalsh(A)[::-1]
    assert np.all(np.diff(ev) <= 1e-6 * size), f"{label}: eigenvalues not descending"
    assert np.abs(ev - ref).max() <= 2e-5 * size, f"{label}: eigenvalues off by {np.abs(ev - ref).max() / size:.2e}"
    assert np.abs(W.T @ W - np.eye(d)).max() <= 2e-5, f"{label}: columns not orthonormal ({np.abs(W.T @ W - np.eye(d)).max():.2e})"
    resid = np.abs(A @ W - W * ev[None, :]).max()
    assert resid <= 3e-5 * size, f"{label}: residual {resid / size:.2e}"
    # sign rule: the entry of largest magnitude of every column is positive
    big = np.abs(W).argmax(0)
    assert np.all(W[big, np.arange(d)] > 0), f"{label}: sign rule"
    if vectors_unique:
        _, V = np.linalg.eigh(A)
        V = V[:, ::-1]
        cos = np.abs((V * W).sum(0))
        # a vector is determined only as well as its eigenvalue is separated: weigh by the gap
        gap = np.minimum(np.abs(np.diff(ref, prepend=np.inf)), np.abs(np.diff(ref, append=-np.inf))) / size
        assert np.all((1 - cos) * np.minimum(gap, 1.0) <= 1e-5), f"{label}: eigenvectors"


@pytest.mark.parametrize("d", [64, 128])
def test_random_covariances_and_graded_spectra(d):
    r = np.random.default_rng(d)
    mats, labels = [], []
    X = r.standard_normal((4 * d, d)) * np.linspace(3.0, 0.2, d)
    mats.append(X.T @ X / X.shape[0]); labels.append("covariance")
    Qm, _ = np.linalg.qr(r.standard_normal((d, d)))
    mats.append(Qm @ np.diag(10.0 ** np.linspace(0, -7, d)) @ Qm.T); labels.append("graded 1e0..1e-7")
    mats.append(Qm @ np.diag(np.concatenate([np.full(d // 2, 2.0), np.linspace(1.0, 0.5, d - d // 2)])) @ Qm.T)
    labels.append("half of the spectrum equal")
    mats.append(Qm @ np.diag(1.0 + 1e-6 * np.arange(d)) @ Qm.T); labels.append("cluster of width 1e-4")
    mats.append(1e6 * mats[0]); labels.append("large scale")
    mats.append(1e-9 * mats[0]); labels.append("small scale")
    mats = [(m + m.T) / 2 for m in mats]
    W, ev = run(mats)
    for A, w, e, lab in zip(mats, W, ev, labels):
        check(A, w, e, f"d={d} {lab}", vectors_unique=lab in ("covariance", "graded 1e0..1e-7", "large scale", "small scale"))


@pytest.mark.parametrize("d", [64, 128])
def test_degenerate_and_structured_matrices(d):
    r = np.random.default_rng(7 * d)
    u = r.standard_normal(d)
    lap = 2 * np.eye(d) - np.eye(d, k=1) - np.eye(d, k=-1)        # already tridiagonal: closed-form spectrum
    blocks = np.zeros((d, d))
    for q in range(4):                                             # no coupling at the quarter cuts
        B = r.standard_normal((d // 4, d // 4))
        blocks[q * d // 4:(q + 1) * d // 4, q * d // 4:(q + 1) * d // 4] = B @ B.T
    low = r.standard_normal((d, 3))
    mats = [np.zeros((d, d)), np.eye(d), np.outer(u, u), lap, blocks, low @ low.T, np.diag(np.arange(d, 0, -1.0))]
    labels = ["zero", "identity", "rank one", "1-D Laplacian", "four uncoupled blocks", "rank three", "diagonal"]
    W, ev = run(mats)
    for A, w, e, lab in zip(mats, W, ev, labels):
        check(A, w, e, f"d={d} {lab}", vectors_unique=lab in ("1-D Laplacian", "diagonal"))
    # the Laplacian's eigenvalues: 2 - 2 cos(k pi / (d + 1))
    want = np.sort(2 - 2 * np.cos(np.arange(1, d + 1) * np.pi / (d + 1)))[::-1]
    assert np.abs(ev[3] - want).max() <= 1e-5


def test_many_matrices_in_one_launch_are_independent():
    r = np.random.default_rng(99)
    d = 64
    mats = []
    for i in range(40):
        X = r.standard_normal((300, d)) * r.uniform(0.1, 2.0, d)
        mats.append(X.T @ X / 300)
    W, ev = run(mats)
    W1, ev1 = run(mats[17:18])
    assert np.array_equal(W[17], W1[0]) and np.array_equal(ev[17], ev1[0])
    for i in (0, 17, 39):
        check(mats[i], W[i], ev[i], f"matrix {i}")


def test_argument_errors():
    A = torch.zeros((1, 32, 32), dtype=torch.float64, device=DEV)
    with pytest.raises(binding.ClusterAttnError):
        binding.debug_eigh(A)                                      # d = 32 is not built

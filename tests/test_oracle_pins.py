"""Pins of the fp64 oracle against what the paper and the mathematics fix.

Each test checks an oracle function against something other than itself: an
identity printed in the paper, a closed form, a brute-force enumeration, a
special case that reduces to a textbook routine, or a library routine.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import clusterattn_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- dense (Eq. 1)
def test_dense_matches_torch_sdpa_fp64():
    r = rng(0)
    Q, K, V = r.standard_normal((37, 16)), r.standard_normal((53, 16)), r.standard_normal((53, 16))
    o = orc.dense_attention(Q, K, V)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(Q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None])[0].numpy()
    assert np.abs(o - ref).max() < 1e-13


def test_dense_two_keys_closed_form():
    # one query, two keys: weights are a logistic function of the logit gap / sqrt(d)
    q = np.array([[2.0, 0.0, 0.0, 0.0]])
    K = np.array([[1.0, 0, 0, 0], [-1.0, 0, 0, 0]])
    V = np.array([[1.0, 0, 0, 0], [0.0, 1.0, 0, 0]])
    o, lse = orc.dense_attention(q, K, V, return_lse=True)
    w0 = 1.0 / (1.0 + np.exp(-(2.0 - (-2.0)) / 2.0))     # sqrt(4) = 2
    assert np.allclose(o[0, :2], [w0, 1 - w0], atol=1e-15)
    assert np.isclose(lse[0], np.log(np.exp(1.0) + np.exp(-1.0)), atol=1e-15)


# ------------------------------------------------- key metric (Section 3.2.2)
def test_key_metric_root_gives_mean_squared_logit_difference():
    r = rng(1)
    Q = r.standard_normal((200, 12)) @ r.standard_normal((12, 12))
    R = orc.psd_root(orc.metric_q(Q))
    assert np.allclose(R, R.T, atol=1e-12)
    for _ in range(20):
        k1, k2 = r.standard_normal(12), r.standard_normal(12)
        lhs = np.sum((R @ (k1 - k2)) ** 2)
        rhs = np.sum((Q @ (k1 - k2)) ** 2) / Q.shape[0]
        assert np.isclose(lhs, rhs, rtol=1e-10)
        # inner product in the metric space
        assert np.isclose((R @ k1) @ (R @ k2), k1 @ orc.metric_q(Q) @ k2, rtol=1e-9, atol=1e-9)
    # rows of transform_keys are R_q k
    K = r.standard_normal((5, 12))
    assert np.allclose(orc.transform_keys(K, R), (R @ K.T).T, atol=1e-12)


def test_psd_root_clamps_negative_eigenvalues_and_handles_rank_deficiency():
    r = rng(2)
    B = r.standard_normal((6, 3))
    A = B @ B.T                                  # rank 3 of 6: zero-distance directions exist
    R = orc.psd_root(A)
    assert np.allclose(R @ R, A, atol=1e-10)
    A_bad = A - 1e-9 * np.eye(6)                 # slightly indefinite
    R2 = orc.psd_root(A_bad)
    lam = np.linalg.eigvalsh(R2)
    assert lam.min() > -1e-12 and np.allclose(R2 @ R2, A, atol=1e-7)
    # diagonal case: root is the elementwise square root
    D = np.diag([4.0, 9.0, 0.0, 1.0])
    assert np.allclose(orc.psd_root(D), np.diag([2.0, 3.0, 0.0, 1.0]), atol=1e-14)


# ------------------------------------------- query metric (Appendix B.1 / B.2)
def test_pair_difference_operator_is_2n_times_centered_scatter():
    r = rng(3)
    n, d = 9, 4
    K = r.standard_normal((n, d)) + 3.0
    D = np.array([K[a] - K[b] for a in range(n) for b in range(n)])   # all ordered pairs
    assert np.allclose(D.T @ D, 2 * n * orc.centered_scatter(K), atol=1e-10)


def test_centered_key_representation_ignores_softmax_invariant_shifts():
    r = rng(4)
    n, d = 30, 6
    K = r.standard_normal((n, d))
    K[:, 5] = 0.7                                   # zero-variance direction: K e_5 = 0.7 * 1
    delta = np.zeros(d)
    delta[5] = 2.5
    assert np.allclose(K @ delta, (0.7 * 2.5) * np.ones(n))
    C = orc.centered_scatter(K)
    R_k = orc.psd_root(C)
    q = r.standard_normal(d)
    Kc = K - K.mean(0)
    assert np.allclose(Kc @ (q + delta), Kc @ q, atol=1e-12)
    # same invariance through the root matrix: ||R_k delta|| = ||K_c delta|| = 0
    assert np.linalg.norm(R_k @ delta) < 1e-6
    # and softmax over the keys is indeed unchanged by the shift
    a, b = K @ q, K @ (q + delta)
    sa, sb = np.exp(a - a.max()), np.exp(b - b.max())
    assert np.allclose(sa / sa.sum(), sb / sb.sum(), atol=1e-12)


def test_query_representation_is_scale_invariant_and_unit_norm():
    r = rng(5)
    K = r.standard_normal((50, 8)) * np.arange(1, 9)
    R_k = orc.psd_root(orc.centered_scatter(K))
    Q = r.standard_normal((10, 8))
    scales = r.uniform(0.1, 10.0, size=(10, 1))
    a = orc.query_representation(Q, R_k)
    b = orc.query_representation(Q * scales, R_k)
    assert np.allclose(a, b, atol=1e-12)
    assert np.allclose(np.linalg.norm(a, axis=1), 1.0, atol=1e-12)
    assert np.allclose(a[0], (R_k @ Q[0]) / np.linalg.norm(R_k @ Q[0]), atol=1e-12)
    zero = orc.query_representation(np.zeros((1, 8)), R_k)
    assert np.all(zero == 0.0)


# ---------------------------------------- diagonalization (Section 3.2.1, PCA)
def test_diagonalize_is_pca_of_the_rows():
    r = rng(6)
    X = r.standard_normal((500, 7)) @ r.standard_normal((7, 7)) + 5.0
    Y, lam, E = orc.diagonalize(X)
    assert np.allclose(E.T @ E, np.eye(7), atol=1e-12)
    assert np.all(np.diff(lam) <= 1e-12)                       # descending
    cov = (Y.T @ Y) / X.shape[0]
    assert np.allclose(cov, np.diag(lam), atol=1e-9)           # decorrelated, variances = eigenvalues
    assert np.allclose(Y.mean(0), 0.0, atol=1e-10)
    # pairwise distances are preserved (pure rotation of the centred rows)
    assert np.isclose(np.linalg.norm(Y[3] - Y[11]), np.linalg.norm(X[3] - X[11]), rtol=1e-12)
    # equivalent to the SVD of the centred data matrix up to column signs
    _, s, Vt = np.linalg.svd(X - X.mean(0), full_matrices=False)
    assert np.allclose(s ** 2 / X.shape[0], lam, rtol=1e-10)
    assert np.allclose(np.abs(Vt), np.abs(E.T), atol=1e-8)
    # sign convention
    for t in range(7):
        assert E[np.argmax(np.abs(E[:, t])), t] > 0


def test_split_coordinates_do_not_depend_on_the_form_of_the_root():
    # using E sqrt(L), or a Cholesky factor, instead of E sqrt(L) E^T rotates the
    # transformed keys; the principal-component coordinates are the same, and with the
    # sign taken from the map out of the original space (lift) the signs are the same too.
    r = rng(7)
    Q = r.standard_normal((300, 6)) * np.array([3, 2, 1.5, 1, 0.5, 0.2])
    K = r.standard_normal((400, 6)) @ r.standard_normal((6, 6))
    M = orc.metric_q(Q)
    lam, E = np.linalg.eigh(M)
    R_sym = orc.psd_root(M)
    R_alt = E * np.sqrt(np.maximum(lam, 0))
    R_chol = np.linalg.cholesky(M)
    assert np.allclose(R_alt @ R_alt.T, M) and np.allclose(R_chol @ R_chol.T, M)
    Y1, l1, _ = orc.diagonalize(K @ R_sym)
    Y2, l2, _ = orc.diagonalize(K @ R_alt)
    assert np.allclose(l1, l2, rtol=1e-9)
    assert np.allclose(np.abs(Y1), np.abs(Y2), atol=1e-8)
    Y1, _, E1 = orc.diagonalize(K @ R_sym, lift=R_sym)
    for R in (R_alt, R_chol):
        Y2, _, E2 = orc.diagonalize(K @ R, lift=R)
        assert np.allclose(Y1, Y2, atol=1e-8)                 # signs included
        assert np.allclose(R_sym @ E1, R @ E2, atol=1e-8)     # the map from the original space is the same
    W = R_sym @ E1
    for t in range(6):
        assert W[np.argmax(np.abs(W[:, t])), t] > 0


# ---------------------------- the clustering stage's coordinates (Section 3.2.2, Appendix B)
@pytest.mark.parametrize("adaptive", [False, True])
def test_split_coordinates_carry_the_two_metrics(adaptive):
    """Keys are compared in the metric of the queries and queries in the metric of the centred
    keys: which root goes to which side, the 1/n of the un-normalised form and the normalisation
    of the ranking form are all fixed by distances written WITHOUT any matrix root."""
    r = rng(70 + adaptive)
    d, n_q, n_k = 7, 90, 130
    Q = (r.standard_normal((n_q, d)) * np.linspace(3.0, 0.3, d)) @ r.standard_normal((d, d)) + 0.5
    K = (r.standard_normal((n_k, d)) * np.linspace(0.2, 2.0, d)) @ r.standard_normal((d, d)) - 1.0
    Yq, Yk = orc.split_coordinates(Q, K, adaptive=adaptive)
    assert Yq.dtype == np.float32 and Yk.dtype == np.float32
    assert Yq.shape == (n_q, d) and Yk.shape == (n_k, d)
    Yq, Yk = Yq.astype(np.float64), Yk.astype(np.float64)
    Kc = K - K.mean(0)
    # keys: |y_i - y_j|^2 = |Q (k_i - k_j)|^2 / n_q      (Section 3.2.2, key clustering)
    for i, j in zip(r.integers(0, n_k, 40), r.integers(0, n_k, 40)):
        want = ((Q @ (K[i] - K[j])) ** 2).sum() / n_q
        assert np.isclose(((Yk[i] - Yk[j]) ** 2).sum(), want, rtol=2e-5, atol=1e-9)
    for i, j in zip(r.integers(0, n_q, 40), r.integers(0, n_q, 40)):
        a, b = Kc @ Q[i], Kc @ Q[j]                     # K_c q: the logits up to a per-query shift
        if adaptive:                                    # Appendix B.1: |K_c (q_i - q_j)|^2 / n_k
            want = ((a - b) ** 2).sum() / n_k
        else:                                           # Appendix B.2: unit vectors K_c q / |K_c q|
            want = 2.0 - 2.0 * (a @ b) / np.sqrt((a @ a) * (b @ b))
        assert np.isclose(((Yq[i] - Yq[j]) ** 2).sum(), want, rtol=2e-5, atol=1e-7)
    # both sets are centred and decorrelated with variances in descending order
    for Y in (Yq, Yk):
        cov = Y.T @ Y / Y.shape[0]
        off = cov - np.diag(np.diag(cov))
        assert np.abs(Y.mean(0)).max() < 1e-5 * np.sqrt(cov[0, 0])
        assert np.abs(off).max() < 1e-5 * cov[0, 0] and np.all(np.diff(np.diag(cov)) <= 1e-6 * cov[0, 0])
    # swapping the sides must fail the same checks (the two metrics differ on this input)
    Yq_s, Yk_s = (y.astype(np.float64) for y in orc.split_coordinates(K[:n_q], Q, adaptive=adaptive))
    i, j = 3, 11
    assert not np.isclose(((Yk_s[i] - Yk_s[j]) ** 2).sum(), ((Q @ (Q[i] - Q[j])) ** 2).sum() / n_q, rtol=1e-2)


# ------------------------------------------------------ split sizes (Section 3.1)
def test_split_point_rule_and_golden_shapes():
    for c in (1, 2, 64, 128, 256):
        for s in list(range(c + 1, 12 * c + 3)) + [32760, 75600, 131072]:
            if s <= c:
                continue
            L = orc.split_point(s, c)
            assert L % c == 0 and c <= L < s
            # closest multiple of c to s/2; the half-way case goes up
            cands = [m * c for m in range(1, s // c + 1) if m * c < s]
            best = min(cands, key=lambda x: (abs(2 * x - s), -x))
            assert L == best, (s, c, L, best)
    with open(os.path.join(GOLDEN, "split_shapes.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for N, c, n_clusters, short, levels in ((int(x) for x in r_) for r_ in rows):
        sizes, depth = [N], 0
        while any(s > c for s in sizes):
            nxt = []
            for s in sizes:
                if s > c:
                    L = orc.split_point(s, c)
                    nxt += [L, s - L]
                else:
                    nxt.append(s)
            sizes, depth = nxt, depth + 1
        assert len(sizes) == n_clusters and depth == levels
        shorts = [s for s in sizes if s != c]
        assert shorts == ([short] if short else [])
        assert sizes[-1] == (short if short else c)     # the short cluster is the last one


# ------------------------------------------------- recursive split (Section 3.2.1)
@pytest.mark.parametrize("N,c,d", [(1024, 64, 8), (1000, 64, 5), (777, 32, 3), (130, 128, 4),
                                   (64, 64, 4), (50, 64, 4), (5 * 16 + 3, 16, 2)])
def test_recursive_split_invariants(N, c, d):
    r = rng(N + c)
    Y = (r.standard_normal((N, d)) * np.linspace(3, 0.5, d)).astype(np.float32)
    perm, tree = orc.recursive_split(Y, c, return_tree=True)
    assert sorted(perm.tolist()) == list(range(N))              # clusters partition the rows
    for lo, hi, t, L in tree:
        assert L % c == 0 and 0 < L < hi - lo                   # lower side: multiple of c
        left, right = perm[lo:lo + L], perm[lo + L:hi]
        # ordered by (value, row): every row below sorts before every row above, along t
        kl = max((Y[i, t], i) for i in left)
        kr = min((Y[i, t], i) for i in right)
        assert kl < kr
    n_c = -(-N // c)
    for j in range(n_c):
        members = perm[j * c:(j + 1) * c]
        assert len(members) == (c if j < n_c - 1 or N % c == 0 else N % c)
        assert np.all(np.diff(members) > 0)                     # ascending original order inside a set


def test_recursive_split_one_dimension_is_sort_and_chunk():
    r = rng(11)
    for N, c in [(256, 16), (250, 16), (96, 32)]:
        y = r.standard_normal((N, 1)).astype(np.float32)
        y[::7] = y[3]                                           # duplicates: ties go to the lower row
        perm = orc.recursive_split(y, c)
        order = sorted(range(N), key=lambda i: (y[i, 0], i))
        for j in range(-(-N // c)):
            assert sorted(order[j * c:(j + 1) * c]) == perm[j * c:(j + 1) * c].tolist()


def test_recursive_split_single_level_is_median_cut_along_top_variance_coordinate():
    # N = 2c: one PDDP-style step along the coordinate with the largest sampled variance
    r = rng(12)
    c, d = 8, 3
    Y = r.standard_normal((2 * c, d)).astype(np.float32) * np.array([1.0, 4.0, 2.0], np.float32)
    perm, tree = orc.recursive_split(Y, c, return_tree=True)
    # brute force, written independently: subsample rows floor(j*s/m), m = min(d, s)
    s, m = 2 * c, min(d, 2 * c)
    sample = [Y[(j * s) // m].astype(np.float64) for j in range(m)]
    var = []
    for t in range(d):
        vals = [row[t] for row in sample]
        mu = sum(vals) / m
        var.append(sum((v - mu) ** 2 for v in vals) / m)
    t_star = max(range(d), key=lambda t: (var[t], -t))
    assert tree == [(0, 2 * c, t_star, c)]
    ranked = sorted(range(2 * c), key=lambda i: (Y[i, t_star], i))
    assert sorted(ranked[:c]) == perm[:c].tolist() and sorted(ranked[c:]) == perm[c:].tolist()


def test_choose_coordinate_ties_go_to_lowest_coordinate():
    sub = np.zeros((4, 5))
    sub[:, 2] = [1, -1, 1, -1]
    sub[:, 4] = [1, -1, 1, -1]
    for choose in (orc.choose_coordinate, orc.choose_coordinate_f32):
        t, var = choose(sub)
        assert t == 2 and var[2] == var[4] == 1.0
    assert orc.subsample_positions(10, 4).tolist() == [0, 2, 5, 7]


def test_choose_coordinate_is_the_population_variance_argmax():
    r = rng(17)
    sub = r.standard_normal((9, 6)) * np.array([1.0, 3.0, 2.0, 3.5, 0.1, 1.0]) + 10.0
    t, var = orc.choose_coordinate(sub)
    brute = [sum((x - sum(col) / 9) ** 2 for x in col) / 9 for col in sub.T.tolist()]
    assert np.allclose(var, brute, rtol=1e-12) and t == int(np.argmax(brute))
    assert np.allclose(var, np.var(sub, axis=0), rtol=1e-12)       # library routine, ddof = 0


def test_interleaved_sum32_follows_the_stated_order():
    """Inputs on which the order of the float32 additions decides the bits.  Expected values
    worked out by hand from: 2^24 + 1 rounds to 2^24 (tie to even), 2^24 + 2 is exact."""
    big = np.float32(2.0 ** 24)

    def column(m, **rows):
        x = np.zeros((m, 1), np.float32)
        for k, v in rows.items():
            x[int(k[1:])] = v
        return x
    # rows 0 and 8 feed partial sum p0, rows 1 and 9 feed p1:
    # p0 = rn(2^24 + 1) = 2^24, p1 = 1 + 1 = 2, total 2^24 + 2 (row after row: stays at 2^24)
    x = column(16, r0=big, r8=1.0, r1=1.0, r9=1.0)
    assert orc.interleaved_sum32(x)[0] == big + np.float32(2.0)
    assert np.cumsum(x[:, 0], dtype=np.float32)[-1] == big
    # p0 = rn(2^24 + 1) = 2^24, p1 = 1: rn(2^24 + 1) = 2^24
    # (partial sums over blocks of consecutive rows would add rows 8 and 9 first: 2^24 + 2)
    assert orc.interleaved_sum32(column(16, r0=big, r8=1.0, r9=1.0))[0] == big
    # the tree ((p0+p1)+(p2+p3)) + ((p4+p5)+(p6+p7)) with p0 = 2^24 and seven ones:
    # (2^24 + 2) + 4 = 2^24 + 6 (left to right over the partial sums: stays at 2^24)
    y = np.ones((8, 1), np.float32)
    y[0] = big
    assert orc.interleaved_sum32(y)[0] == big + np.float32(6.0)
    # p0 = 2^24, p1 = p5 = 1: (2^24 + 1 -> 2^24) + (0 + 1) -> 2^24
    # (pairing p0 with p4 and p1 with p5 first would give 2^24 + 2)
    assert orc.interleaved_sum32(column(8, r0=big, r1=1.0, r5=1.0))[0] == big
    # p0 = 2^24, p1 = p3 = 1: ((2^24 + 1 -> 2^24) + (0 + 1)) -> 2^24
    # (pairing p0 with p2 and p1 with p3 first would give 2^24 + 2)
    assert orc.interleaved_sum32(column(8, r0=big, r1=1.0, r3=1.0))[0] == big
    # fewer than eight rows, and one sum per column
    w = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]], np.float32)
    assert orc.interleaved_sum32(w).tolist() == [9.0, 12.0]


def test_float32_coordinate_choice_differs_from_the_definition_only_at_near_ties():
    """Two columns whose variances are almost equal: the float32 restatement may pick the other
    one, and when it does the two variances lie within the rounding error of a float32 sum."""
    r = rng(18)
    differ = 0
    for trial in range(3000):
        m = int(r.choice([16, 64, 128]))
        col = r.standard_normal(m)
        other = r.permutation(col) * (1.0 + r.uniform(-3e-7, 3e-7))
        sub = np.stack([col, other, 0.3 * r.standard_normal(m)], axis=1).astype(np.float32)
        t64, v64 = orc.choose_coordinate(sub)
        t32, _ = orc.choose_coordinate_f32(sub)
        if t64 != t32:
            differ += 1
            top = np.sort(v64)[::-1]
            assert (top[0] - top[1]) <= (m / 8 + 8) * 2.0 ** -23 * top[0]
    assert differ > 0                                          # the search does reach disagreements
    # well separated variances: the same decision
    for trial in range(200):
        sub = (r.standard_normal((64, 8)) * np.linspace(2.0, 0.5, 8)).astype(np.float32)
        assert orc.choose_coordinate(sub)[0] == orc.choose_coordinate_f32(sub)[0]


def test_recursive_split_clusters_are_tighter_than_random_clusters():
    # qualitative: Section 1.2 contrasts the method with random equal-size clusters
    r = rng(13)
    means = 3 * r.standard_normal((8, 16))
    X = means[r.integers(0, 8, 2048)] + 0.3 * r.standard_normal((2048, 16))
    Y, _, _ = orc.diagonalize(X)
    perm = orc.recursive_split(Y.astype(np.float32), 64)

    def within(p):
        return sum(X[p[j * 64:(j + 1) * 64]].var(axis=0).sum() for j in range(32)) / 32
    assert within(perm) < 0.5 * within(r.permutation(2048))


# -------------------------------------------- basic recursive splitting (Section 3.2.1, Section 5.2)
def test_basic_direction_converges_to_the_first_principal_component():
    # identity metric, many iterations: the textbook power iteration on the centred covariance
    r = rng(50)
    sub = (r.standard_normal((12, 12)) * np.linspace(4, 0.2, 12)).astype(np.float32)
    u = orc.basic_direction(sub, np.eye(12, dtype=np.float32), r.standard_normal(12).astype(np.float32), 200)
    Z = sub.astype(np.float64) - sub.astype(np.float64).mean(0)
    lam, E = np.linalg.eigh(Z.T @ Z)
    assert abs(float(np.linalg.norm(u)) - 1) < 1e-5
    assert abs(float(u.astype(np.float64) @ E[:, -1])) > 1 - 1e-4


def test_basic_direction_with_injected_metric_equals_transforming_the_rows():
    # u <- A C u on the rows x  ==  R (w <- C' w on the rows x R),  A = R R   (Section 5.2)
    r = rng(51)
    d = 10
    B = r.standard_normal((d, d))
    R = orc.psd_root(B @ B.T / d + 0.5 * np.eye(d))
    A = R @ R
    sub = r.standard_normal((d, d)) @ r.standard_normal((d, d))
    u0 = r.standard_normal(d)
    for p_iter in (1, 3, 6):
        u = orc.basic_direction(sub.astype(np.float32), A.astype(np.float32), u0.astype(np.float32), p_iter)
        w = orc.basic_direction((sub @ R).astype(np.float32), np.eye(d, dtype=np.float32),
                                np.linalg.solve(R, u0).astype(np.float32), p_iter)
        v = R @ w.astype(np.float64)
        v /= np.linalg.norm(v)
        assert np.abs(u.astype(np.float64) - v).max() < 2e-3
        # and the projections order the rows alike: x . u  ~  (x R) . w
        x = r.standard_normal((5, d))
        assert np.allclose(x @ u.astype(np.float64), (x @ R) @ w.astype(np.float64) / np.linalg.norm(R @ w), atol=5e-3)


def test_basic_split_tree_partitions_by_its_projections():
    r = rng(52)
    means = 3 * r.standard_normal((6, 8))
    X = (means[r.integers(0, 6, 1000)] + 0.4 * r.standard_normal((1000, 8))).astype(np.float32)
    c = 32
    levels = orc.split_levels(1000, c)
    noise = r.standard_normal(((1 << levels) - 1, 8)).astype(np.float32)
    perm, tree = orc.basic_recursive_split(X, np.eye(8, dtype=np.float32), noise, c, 3, return_tree=True)
    assert sorted(perm.tolist()) == list(range(1000))
    sizes = [len(perm[j * c:(j + 1) * c]) for j in range(-(-1000 // c))]
    assert sizes[:-1] == [c] * (len(sizes) - 1) and sizes[-1] == 1000 % c      # one short cluster, the last
    for j in range(len(sizes)):
        assert np.all(np.diff(perm[j * c:(j + 1) * c]) > 0)                     # ascending inside a set
    # replay: every node sends down exactly the L smallest (projection, row) pairs of its set
    check = np.arange(1000)
    for level, slot, lo, hi, L, u in tree:
        rows = check[lo:hi].copy()
        t = (X[rows].astype(np.float64) @ u.astype(np.float64))
        assert L == orc.split_point(hi - lo, c) and abs(float(np.linalg.norm(u)) - 1) < 1e-5
        order = np.lexsort((rows, orc._seq_dot_rows(X[rows], u)))
        down = np.sort(rows[order[:L]])
        up = np.sort(rows[order[L:]])
        assert t[np.isin(rows, down)].max() <= t[np.isin(rows, up)].min() + 1e-4   # a hyperplane cut
        check[lo:lo + L], check[lo + L:hi] = down, up
    assert np.array_equal(check, perm)

    def within(p):
        return sum(X[p[j * c:(j + 1) * c]].var(axis=0).sum() for j in range(31)) / 31
    assert within(perm) < 0.5 * within(r.permutation(1000))


def test_basic_split_start_vectors_and_one_dimension():
    r = rng(53)
    X = r.standard_normal((300, 4)).astype(np.float32)
    levels = orc.split_levels(300, 50)
    noise = r.standard_normal(((1 << levels) - 1, 4)).astype(np.float32)
    _, tree = orc.basic_recursive_split(X, np.eye(4, dtype=np.float32), noise, 50, iterations=0, return_tree=True)
    by_node = {(lv, sl): u for lv, sl, _, _, _, u in tree}
    g0 = noise[0].astype(np.float64)
    assert np.allclose(by_node[(0, 0)], g0 / np.linalg.norm(g0), atol=1e-6)       # the root starts at the noise
    for (lv, sl), u in by_node.items():
        if lv == 0:
            continue
        g = noise[(1 << lv) - 1 + sl].astype(np.float64)
        want = 0.5 * (by_node[(lv - 1, sl >> 1)].astype(np.float64) + g / np.linalg.norm(g))
        assert np.allclose(u, want, atol=1e-6)                                   # mean of parent and noise
    # d = 1 with positive noise: the direction is +1 at every node (a one-row subsample has no
    # variance, the start vector stays), so the method is "sort and cut into chunks"
    x = r.standard_normal((257, 1)).astype(np.float32)
    lv1 = orc.split_levels(257, 16)
    perm = orc.basic_recursive_split(x, np.ones((1, 1), np.float32),
                                     np.abs(r.standard_normal(((1 << lv1) - 1, 1))).astype(np.float32) + 0.1, 16, 2)
    spans = sorted((x[perm[j * 16:(j + 1) * 16], 0].min(), x[perm[j * 16:(j + 1) * 16], 0].max()) for j in range(17))
    assert all(spans[j][1] <= spans[j + 1][0] for j in range(16))


def test_basic_metrics_are_the_two_metric_matrices():
    r = rng(54)
    Q, K = r.standard_normal((40, 5)), r.standard_normal((60, 5)) + 1.0
    A_q, A_k = orc.basic_metrics(Q, K)
    assert np.allclose(A_k, Q.T @ Q / 40)                         # keys in the query metric
    Kc = K - K.mean(0)
    assert np.allclose(A_q, Kc.T @ Kc / 60)                       # queries in the centred key metric
    assert orc.split_levels(131072, 128) == 10 and orc.split_levels(32760, 128) == 8 and orc.split_levels(100, 128) == 0


# -------------------------------------------- centroids and scores (Section 3.3.1)
def test_centroid_score_is_mean_pairwise_logit_and_jensen_bound():
    r = rng(14)
    N, d, c = 96, 8, 16
    Q, K = r.standard_normal((N, d)), r.standard_normal((N + 5, d))
    pq, pk = r.permutation(N), r.permutation(N + 5)
    cq, nq = orc.centroids(Q, pq, c)
    ck, nk = orc.centroids(K, pk, c)
    assert nk.tolist() == [16] * 6 + [5] and nq.tolist() == [16] * 6
    S = orc.centroid_scores(cq, ck)
    for i, j in itertools.product(range(6), range(7)):
        qs, ks = Q[pq[i * c:(i + 1) * c]], K[pk[j * c:min((j + 1) * c, N + 5)]]
        pair = qs @ ks.T
        assert np.isclose(S[i, j], pair.mean(), atol=1e-12)
        assert np.exp(pair / np.sqrt(d)).mean() >= np.exp(S[i, j] / np.sqrt(d)) - 1e-12


def test_float32_scores_follow_the_exact_scores():
    r = rng(16)
    cq, ck = r.standard_normal((9, 64)), r.standard_normal((40, 64))
    S64 = orc.centroid_scores(cq.astype(np.float32), ck.astype(np.float32))
    S32 = orc.centroid_scores_f32(cq, ck)
    assert S32.dtype == np.float32 and np.abs(S32 - S64).max() < 2e-5 * np.abs(S64).max()
    # brute force of the stated order on one entry
    acc = np.float32(0)
    for k in range(64):
        acc = np.float32(acc + np.float32(np.float32(cq[3, k]) * np.float32(ck[7, k])))
    assert acc == S32[3, 7]
    # well separated scores: the float32 restatement selects what the definition selects
    assert np.array_equal(orc.select_blocks_f32(cq, ck, 5), orc.select_topk(S64, 5))
    assert np.array_equal(orc.select_blocks(cq.astype(np.float32), ck.astype(np.float32), 5), orc.select_topk(S64, 5))


def test_select_topk_matches_full_sort_with_index_tie_break():
    r = rng(15)
    S = r.standard_normal((7, 20))
    S[2, 5] = S[2, 9] = S[2, 14] = S[2].max() + 1.0          # three-way tie at the top
    S[4, :] = 1.0                                             # all equal
    for keep in (1, 2, 5, 20):
        got = orc.select_topk(S, keep)
        for i in range(7):
            ranked = sorted(range(20), key=lambda j: (-S[i, j], j))
            assert got[i].tolist() == sorted(ranked[:keep])
    assert orc.select_topk(S, 2)[2].tolist() == [5, 9]
    assert orc.select_topk(S, 3)[4].tolist() == [0, 1, 2]


# ------------------------------------------------ adaptive selection (Section 3.3.2)
def test_exp2_recipe_is_accurate_and_exact_on_integers():
    x = np.linspace(-40, 10, 20001).astype(np.float32)
    got = orc.exp2_f32(x).astype(np.float64)
    assert np.abs(got / np.exp2(x.astype(np.float64)) - 1).max() < 1e-4
    ints = np.arange(-20, 10).astype(np.float32)
    assert np.abs(orc.exp2_f32(ints) / np.exp2(ints.astype(np.float64)) - 1).max() < 1e-4
    assert orc.exp2_f32(np.float32(-1000.0)) < 1e-29            # clamped, no wrap-around


def test_adaptive_selection_recall_minimality_and_limits():
    r = rng(40)
    d, n_qc, n_kc = 16, 7, 60
    cq, ck = r.standard_normal((n_qc, d)) * 2, r.standard_normal((n_kc, d)) * 2
    counts = r.integers(1, 9, n_kc)
    scale = 1 / np.sqrt(d)
    S = orc.centroid_scores(cq.astype(np.float32), ck.astype(np.float32))
    exact_mass = counts[None, :] * np.exp(scale * (S - S.max(1, keepdims=True)))
    for recall in (0.5, 0.9, 0.99):
        lists = orc.select_blocks_adaptive(cq, ck, counts, recall, min_count=4, scale=scale)
        for i, sel in enumerate(lists):
            assert np.all(np.diff(sel) > 0) and len(sel) >= 4
            m = exact_mass[i]
            share = m[sel].sum() / m.sum()
            assert share >= recall - 1e-3                       # reaches the recall (estimate precision 1e-4)
            # greedy: every selected cluster is at least as massive as every excluded one
            out = np.setdiff1d(np.arange(n_kc), sel)
            assert m[sel].min() >= m[out].max() * (1 - 1e-3)
            # minimal: without its least massive member the recall is missed (unless at the minimum count)
            if len(sel) > 4:
                assert (m[sel].sum() - m[sel].min()) / m.sum() < recall + 1e-3
    # recall 1 takes everything, recall 0 takes the minimum count
    assert all(len(x) == n_kc for x in orc.select_blocks_adaptive(cq, ck, counts, 1.0, 4, scale))
    low = orc.select_blocks_adaptive(cq, ck, counts, 0.0, 5, scale)
    assert all(len(x) == 5 for x in low)
    # with equal cluster sizes the mass order is the score order: the minimum-count list is the top-k list
    same = orc.select_blocks_adaptive(cq, ck, np.full(n_kc, 8), 0.0, 5, scale)
    topk = orc.select_blocks(cq, ck, 5)
    assert all(np.array_equal(a, b) for a, b in zip(same, topk))


def test_unnormalised_query_representation_is_the_centred_key_metric():
    # Appendix B.1: |r(q1) - r(q2)|^2 = |K_c (q1 - q2)|^2 / n, and softmax-invariant shifts vanish
    r = rng(41)
    K = r.standard_normal((80, 6)) @ r.standard_normal((6, 6)) + 2.0
    n = K.shape[0]
    R_k = orc.psd_root(orc.centered_scatter(K) / n)
    Q = r.standard_normal((5, 6))
    Z = orc.query_representation(Q, R_k, normalize=False)
    Kc = K - K.mean(0)
    for a in range(5):
        for b in range(5):
            assert np.isclose(((Z[a] - Z[b]) ** 2).sum(), ((Kc @ (Q[a] - Q[b])) ** 2).sum() / n, rtol=1e-9, atol=1e-12)
    Yq, Yk = orc.split_coordinates(Q.repeat(20, 0) + 0.1 * r.standard_normal((100, 6)), K, adaptive=True)
    assert Yq.dtype == np.float32 and Yq.shape == (100, 6)


# ------------------------------------------------ attention (Section 1.2, Appendix A)
def _setup(seed, N_q=48, N_k=60, d=8, c=4):
    r = rng(seed)
    Q, K, V = r.standard_normal((N_q, d)), 1.5 * r.standard_normal((N_k, d)), r.standard_normal((N_k, d))
    return r, Q, K, V, r.permutation(N_q), r.permutation(N_k), c


def test_all_blocks_kept_equals_dense():
    r, Q, K, V, pq, pk, c = _setup(20, N_k=62)                 # 62 = 15*4 + 2: short key cluster
    n_kc, n_qc = 16, 12
    idx = np.tile(np.arange(n_kc), (n_qc, 1))
    for comp in (False, True):
        o, lse = orc.cluster_attention(Q, K, V, pq, pk, c, c, idx, comp)
        od, lsed = orc.dense_attention(Q, K, V, return_lse=True)
        assert np.abs(o - od).max() < 1e-12 and np.abs(lse - lsed).max() < 1e-12


def test_cluster_size_one_makes_compensation_exact():
    r, Q, K, V, pq, pk, _ = _setup(21, N_q=10, N_k=23)
    idx = np.stack([np.sort(r.choice(23, 5, replace=False)) for _ in range(10)])
    o, lse = orc.cluster_attention(Q, K, V, pq, pk, 1, 1, idx, True)
    od, lsed = orc.dense_attention(Q, K, V, return_lse=True)
    assert np.abs(o - od).max() < 1e-12 and np.abs(lse - lsed).max() < 1e-12
    o_nc, _ = orc.cluster_attention(Q, K, V, pq, pk, 1, 1, idx, False)
    assert np.abs(o_nc - od).max() > 1e-3                      # and it matters


def test_uncompensated_output_and_error_split():
    # eqs. (2)-(4): o_S over the selected keys; o - o_S = (1 - w_S)(o_Sbar - o_S)
    r, Q, K, V, pq, pk, c = _setup(22)
    n_kc, n_qc, keep = 15, 12, 4
    idx = np.stack([np.sort(r.choice(n_kc, keep, replace=False)) for _ in range(n_qc)])
    o_S, _ = orc.cluster_attention(Q, K, V, pq, pk, c, c, idx, False)
    scale = 1 / np.sqrt(Q.shape[1])
    for i in range(n_qc):
        S = np.concatenate([pk[j * c:(j + 1) * c] for j in idx[i]])
        Sbar = np.setdiff1d(np.arange(60), S)
        for row in pq[i * c:(i + 1) * c]:
            w = np.exp(scale * K @ Q[row])
            w /= w.sum()
            oS = (w[S] @ V[S]) / w[S].sum()
            oSb = (w[Sbar] @ V[Sbar]) / w[Sbar].sum()
            o = w @ V
            assert np.allclose(o_S[row], oS, atol=1e-13)
            assert np.allclose(o - o_S[row], (1 - w[S].sum()) * (oSb - oS), atol=1e-13)


def test_compensated_error_decomposition():
    # Appendix A: o - o_hat = sum_c |c| (delta_c (vbar_c - o_hat) + Cov_c(w, v)),
    # the 1/d_hat form with (vbar_c - o), d_hat = 1 - sum_c |c| delta_c, delta_c >= 0.
    r, Q, K, V, pq, pk, c = _setup(23, N_k=58)                 # last key cluster has 2 rows
    N_k, n_kc, n_qc, keep = 58, 15, 12, 3
    idx = np.stack([np.sort(r.choice(n_kc, keep, replace=False)) for _ in range(n_qc)])
    o_hat, lse_hat = orc.cluster_attention(Q, K, V, pq, pk, c, c, idx, True)
    od, lsed = orc.dense_attention(Q, K, V, return_lse=True)
    scale = 1 / np.sqrt(Q.shape[1])
    for i in range(n_qc):
        excluded = np.setdiff1d(np.arange(n_kc), idx[i])
        for row in pq[i * c:(i + 1) * c]:
            e = np.exp(scale * K @ Q[row])
            Z = e.sum()
            w = e / Z
            o = w @ V
            jensen_hat, jensen_o, cov_sum, d_hat = 0.0, 0.0, 0.0, 1.0
            for j in excluded:
                mem = pk[j * c:min((j + 1) * c, N_k)]
                n = len(mem)
                kbar, vbar = K[mem].mean(0), V[mem].mean(0)
                w_c = np.exp(scale * kbar @ Q[row]) / Z          # centroid weight, dense-normalised
                delta = w[mem].mean() - w_c
                assert delta >= -1e-15
                cov = ((w[mem] - w[mem].mean())[:, None] * (V[mem] - vbar)).mean(0)
                jensen_hat = jensen_hat + n * delta * (vbar - o_hat[row])
                jensen_o = jensen_o + n * delta * (vbar - o)
                cov_sum = cov_sum + n * cov
                d_hat -= n * delta
            assert np.allclose(o - o_hat[row], jensen_hat + cov_sum, atol=1e-13)
            assert np.allclose(o - o_hat[row], (jensen_o + cov_sum) / d_hat, atol=1e-13)
            # the compensated denominator is d_hat times the dense one
            assert np.isclose(lse_hat[row], lsed[row] + np.log(d_hat), atol=1e-12)


def test_attention_accepts_ragged_lists():
    r, Q, K, V, pq, pk, c = _setup(24)
    lists = [np.sort(r.choice(15, int(r.integers(1, 15)), replace=False)) for _ in range(12)]
    o, lse = orc.cluster_attention(Q, K, V, pq, pk, c, c, lists, True)
    # each query cluster equals the fixed-width call with its own list
    for i, sel in enumerate(lists):
        idx = np.tile(sel, (12, 1))
        o_i, _ = orc.cluster_attention(Q, K, V, pq, pk, c, c, idx, True, query_clusters=[i])
        rows = pq[i * c:(i + 1) * c]
        assert np.abs(o[rows] - o_i[rows]).max() < 1e-14


def test_forward_pipeline_shapes_and_convergence_to_dense():
    # whole path on a small mixture: more kept blocks -> closer to dense; SMC helps
    r = rng(30)
    means = 3 * r.standard_normal((4, 16)) / 4
    Q = means[r.integers(0, 4, 256)] + 0.5 * r.standard_normal((256, 16))
    K = means[r.integers(0, 4, 256)] + 0.5 * r.standard_normal((256, 16))
    V = r.standard_normal((256, 16))
    od = orc.dense_attention(Q, K, V)
    errs = []
    for keep in (2, 8, 16):
        o, _, cl, idx = orc.clusterattention_forward(Q, K, V, 16, 16, keep, True)
        assert idx.shape == (16, keep) and np.all(np.diff(idx, axis=1) > 0)
        assert sorted(cl["perm_k"].tolist()) == list(range(256))
        errs.append(np.abs(o - od).max())
    assert errs[2] < 1e-12 and errs[0] > errs[1] > errs[2]


# ------------------------------------------------ quantised Q K^T (Section 3.1, Section 5.1)
def _all_e4m3_values():
    """Every finite non-negative E4M3 number from the format's definition: 4 exponent bits (bias 7),
    3 mantissa bits, exponent field 0 = subnormals, the all-ones code is not a number."""
    vals = [m / 8.0 * 2.0 ** -6 for m in range(8)]
    for e in range(1, 16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            vals.append((1 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals)


def test_e4m3_rounding_matches_the_format():
    vals = _all_e4m3_values()
    assert len(vals) == 127 and vals.max() == 448.0 and vals[1] == 2.0 ** -9
    # representable numbers are fixed points, both signs
    assert np.array_equal(orc.round_to_minifloat(vals), vals)
    assert np.array_equal(orc.round_to_minifloat(-vals), -vals)
    # every real rounds to the nearest table entry; exact halves go to the even mantissa
    r = rng(60)
    y = np.concatenate([r.uniform(0, 460, 4000), r.uniform(0, 0.05, 2000), 2.0 ** r.uniform(-12, 9, 2000)])
    got = orc.round_to_minifloat(y)
    nearest = vals[np.abs(y[:, None] - vals[None, :]).argmin(axis=1)]
    assert np.array_equal(got, nearest)
    assert orc.round_to_minifloat(1.0625) == 1.0            # half-way between 1 (mantissa 000) and 1.125 (001)
    assert orc.round_to_minifloat(1.1875) == 1.25           # half-way between 1.125 (001) and 1.25 (010)
    assert orc.round_to_minifloat(2.0 ** -10) == 0.0        # half-way between 0 and the smallest subnormal
    assert orc.round_to_minifloat(3 * 2.0 ** -10) == 2.0 ** -8
    assert orc.round_to_minifloat(1e9) == 448.0 and orc.round_to_minifloat(-465.0) == -448.0
    assert orc.round_to_minifloat(464.0) == 448.0           # beyond the largest number: saturates


def test_group_quantisation_scales_the_largest_magnitude_to_448():
    x = np.array([[0.5, -3.0, 1.0], [0.0, 2.9, -0.011]], np.float32)
    s, code = orc.quantize_group_e4m3(x)
    assert s == np.float32(3.0) / np.float32(448.0) and code[0, 1] == -448.0
    # by hand: inv = 448/3; 0.5 * inv = 74.67 -> spacing 8 in [64, 128): 72;  1.0 * inv = 149.33 -> spacing 16: 144
    assert code[0, 0] == 72.0 and code[0, 2] == 144.0 and code[1, 0] == 0.0
    assert code[1, 1] == 448.0                              # 433.07 -> spacing 32 in [256, 512): 416 or 448, nearer 448
    assert code[1, 2] == -1.625                             # -1.6427 -> spacing 0.125 in [1, 2): -1.625
    zero_s, zero_code = orc.quantize_group_e4m3(np.zeros((2, 3), np.float32))
    assert zero_s == 0 and not zero_code.any()


def test_quantised_attention_two_by_two_by_hand():
    # one query, two keys in two clusters of one key each, d = 2, both kept
    Q = np.array([[1.0, 0.3]], np.float32)
    K = np.array([[2.0, 0.1], [-1.0, 1.0]], np.float32)
    V = np.array([[1.0, 0.0], [0.0, 1.0]])
    o, lse = orc.cluster_attention_quantized_qk(Q, K, V, np.arange(1), np.arange(2), 1, 1, np.array([[0, 1]]), False,
                                                scale=1.0)
    # query row: amax 1, inv 448: codes (448, 134.4 -> spacing 16: 128) -> (1, 128/448)
    # key 0: amax 2: codes (448, 22.4 -> spacing 2 in [16, 32): 22) -> (2, 2 * 22/448);  key 1: amax 1: (-1, 1) exact
    q = np.array([1.0, 128.0 / 448.0])
    k0 = np.array([2.0, 2.0 * 22.0 / 448.0])
    k1 = np.array([-1.0, 1.0])
    l0, l1 = q @ k0, q @ k1
    w0 = 1.0 / (1.0 + np.exp(l1 - l0))
    assert np.allclose(o[0], [w0, 1 - w0], atol=1e-6)       # float32 scales: 1e-7 relative
    assert np.isclose(lse[0], np.log(np.exp(l0) + np.exp(l1)), atol=1e-6)


def test_quantised_attention_tends_to_the_unquantised_one():
    r, Q, K, V, pq, pk, c = _setup(61, N_k=58)
    Q, K = Q.astype(np.float32), K.astype(np.float32)
    idx = np.stack([np.sort(r.choice(15, 4, replace=False)) for _ in range(12)])
    ck, cnt = orc.centroids(K, pk, c)
    ck32 = ck.astype(np.float32)
    exact, lse_exact = orc.cluster_attention(Q, K, V, pq, pk, c, c, idx, True, ck=ck32, count_k=cnt)
    errs = []
    for bits in (3, 7, 12, 23):
        o, lse = orc.cluster_attention_quantized_qk(Q, K, V, pq, pk, c, c, idx, True, ck=ck32, count_k=cnt, man_bits=bits)
        errs.append(np.abs(o - exact).max())
    assert errs[0] > errs[1] > errs[2] > errs[3]            # every added mantissa bit brings it closer
    assert errs[0] > 1e-3 and errs[3] < 2e-6                # 3 bits matter; 23 bits leave float32 rounding of the scales
    # the scales alone do not change anything that the codes do not: a tensor of representable
    # numbers with group maximum 448 passes through unchanged
    vals = _all_e4m3_values()
    X = r.choice(vals, (6, 8)).astype(np.float32)
    X[:, 0] = 448.0
    Qd, Kd, _ = orc.quantize_qk(X, X, np.arange(6), 2)
    assert np.array_equal(Qd, X.astype(np.float64)) and np.array_equal(Kd, X.astype(np.float64))

"""Plain fp64 statement of ClusterAttention* (transforms + diagonalized
recursive splitting + top-k selection + striped mean-compensation).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the product path.  Shares no code with
the CUDA kernels.

Every function works on ONE attention head (the method is per head, Section 3.1
"Overview") and takes numpy arrays that it widens to float64.  The steps follow
the paper's order and notation; no blocking, fusion or reordering is applied.
numpy's `eigh`, `matmul` and `lexsort` serve as library steps.

Pins (tests/test_oracle_*.py):
  dense_attention ........ torch fp64 SDPA; hand-computed 2-key case
  metric_q / psd_root .... ||R_q(k1-k2)||^2 == ||Q(k1-k2)||^2/n  (Section 3.2.2)
  centered_scatter ....... D^T D == 2n K_c^T K_c by pair enumeration (Appendix B.2),
                           shift invariance K_c(q+delta) == K_c q (Appendix B.1)
  query_representation ... invariance to positive rescaling of q (Appendix B.2)
  diagonalize ............ decorrelated coordinates, descending variance, isometry
  split_point / recursive_split ... partition + size invariants (Section 3.1),
                           d=1 closed form "sort and chunk", brute-force one-level cut
  split_coordinates ...... squared distances of the key coordinates == (k1-k2)^T (Q^T Q/n) (k1-k2)
                           and of the query coordinates == the distance of r(q) written with
                           K_c alone (no root), both query representations (Section 3.2.2,
                           Appendix B.1 / B.2); sign rule independent of the root's form
  centroids / centroid_scores ..... mean pairwise logit identity, Jensen bound (Section 3.3.1)
  select_topk ............ brute-force full sort
  cluster_attention ...... all blocks kept == dense; c=1 == dense; eqs. (2)-(4);
                           exact SMC error decomposition (Appendix A)
  *_f32 helpers .......... hand-computed sums whose bits depend on the order of the additions;
                           the fp64 decisions on inputs without near-ties
  round_to_minifloat / quantize_* / cluster_attention_quantized_qk ... the table of all E4M3
                           numbers written out from the format's definition, hand-rounded values,
                           a hand-computed 2 x 2 case, and the limit of many mantissa bits
                           (= the unquantised attention)
Decisions (which coordinate a split takes, which key clusters are kept) are DEFINED by the
float64 functions `choose_coordinate`, `centroid_scores` + `select_topk`.  The `_f32` functions
beside them restate the same quantities in float32 with a fixed operation order; they exist so
that a float32 implementation can be compared bit for bit, and the tests count where the two
decisions differ (only at near-ties).
Conventions of this build that the paper leaves open (subsample positions,
round-half-up split point, fp32 rounding of the split coordinates, eigenvector
sign) are "parity unpinned" by the paper: the oracle is their definition.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# Eq. (1): dense bidirectional attention, softmax includes the 1/sqrt(d) scale
# (Section 3.2.2 first paragraph; Section 3.3.1).
# --------------------------------------------------------------------------
def dense_attention(Q, K, V, scale=None, return_lse=False):
    Q = np.asarray(Q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    if scale is None:
        scale = 1.0 / np.sqrt(Q.shape[1])
    logits = scale * (Q @ K.T)
    mx = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - mx)
    z = e.sum(axis=1, keepdims=True)
    o = (e / z) @ V
    if return_lse:
        return o, (mx + np.log(z))[:, 0]
    return o


# --------------------------------------------------------------------------
# Section 3.2.2 "Key clustering": M = Q^T Q / n.
# --------------------------------------------------------------------------
def metric_q(Q):
    Q = np.asarray(Q, F64)
    return (Q.T @ Q) / Q.shape[0]


# --------------------------------------------------------------------------
# Section 3.2.2 "Query clustering" / Appendix B.2: K_c^T K_c with K_c the key
# matrix after subtracting the mean row.
# --------------------------------------------------------------------------
def centered_scatter(K):
    K = np.asarray(K, F64)
    Kc = K - K.mean(axis=0, keepdims=True)
    return Kc.T @ Kc


# --------------------------------------------------------------------------
# Section 3.2.2: root of a PSD matrix by eigendecomposition, negative
# eigenvalues clamped to zero; symmetric form E sqrt(L) E^T.
# --------------------------------------------------------------------------
def psd_root(A):
    A = np.asarray(A, F64)
    lam, E = np.linalg.eigh(0.5 * (A + A.T))
    lam = np.maximum(lam, 0.0)
    return (E * np.sqrt(lam)) @ E.T


# Keys go to query space through R_q (Section 3.2.2, "project all keys through R_q").
def transform_keys(K, R_q):
    return np.asarray(K, F64) @ np.asarray(R_q, F64)   # rows: (R_q k)^T, R_q symmetric


# r(q) = R_k q / |R_k q|  (Section 3.2.2, ranking form; Appendix B.2).
# A row whose transformed norm underflows maps to the zero vector.
def query_representation(Q, R_k, normalize=True):
    Z = np.asarray(Q, F64) @ np.asarray(R_k, F64)
    if not normalize:        # adaptive-selection form (Section 3.2.2, Appendix B.1): r(q) = R_k q
        return Z
    nrm = np.sqrt((Z * Z).sum(axis=1, keepdims=True))
    out = np.zeros_like(Z)
    ok = nrm[:, 0] >= 1e-30
    out[ok] = Z[ok] / nrm[ok]
    return out


# --------------------------------------------------------------------------
# Section 3.2.1 "Diagonalized recursive splitting": project the (transformed)
# rows onto the principal components of the full set.  Centred covariance,
# components in descending eigenvalue order.  The paper leaves the sign of a
# component open; it is fixed here through the map from the ORIGINAL space:
# with `lift` = the matrix R that produced the transformed rows (keys: x R_q,
# queries: R_k q before normalisation), component t is oriented so that the
# entry of largest magnitude (lowest index on ties) of column t of R E is
# positive.  R E does not change when R is replaced by another root R U of the
# same metric (E becomes U^T E), so the coordinates, signs included, are a
# function of the metric alone.  Without `lift` the rule applies to E itself.
# Returns (Y, eigenvalues, basis).
# --------------------------------------------------------------------------
def principal_basis(C, lift=None):
    lam, E = np.linalg.eigh(0.5 * (C + C.T))
    order = np.argsort(-lam, kind="stable")
    lam, E = lam[order], E[:, order]
    W = E if lift is None else np.asarray(lift, F64) @ E
    for t in range(E.shape[1]):
        j = int(np.argmax(np.abs(W[:, t])))
        if W[j, t] < 0:
            E[:, t] = -E[:, t]
    return lam, E


def diagonalize(X, lift=None):
    X = np.asarray(X, F64)
    mu = X.mean(axis=0, keepdims=True)
    Xc = X - mu
    C = (Xc.T @ Xc) / X.shape[0]
    lam, E = principal_basis(C, lift)
    return Xc @ E, lam, E


# --------------------------------------------------------------------------
# Section 3.2.1: the lower side of a split holds the multiple of c closest to
# half of the set (half-way cases go up), so at most one final cluster is short
# (Section 3.1).
# --------------------------------------------------------------------------
def split_point(s, c):
    return c * ((s + c) // (2 * c))


def subsample_positions(s, m):
    """m evenly spaced positions inside a segment of s rows: floor(j*s/m)."""
    return (np.arange(m, dtype=np.int64) * s) // m


def interleaved_sum32(x):
    """Column sums of a float32 array x [m, d] in float32, in a fixed order: eight
    partial sums over the rows j = r, r+8, r+16, ... (each taken row after row),
    combined as ((p0+p1)+(p2+p3)) + ((p4+p5)+(p6+p7)).  Every addition is one
    IEEE single-precision operation, so any implementation that follows the
    order gets the same bits."""
    assert x.dtype == np.float32
    zero = np.zeros(x.shape[1], np.float32)
    parts = [np.cumsum(x[r::8], axis=0, dtype=np.float32)[-1] if x[r::8].shape[0] else zero for r in range(8)]
    return ((parts[0] + parts[1]) + (parts[2] + parts[3])) + ((parts[4] + parts[5]) + (parts[6] + parts[7]))


def choose_coordinate(sub):
    """Section 3.2.1: the coordinate of highest variance over the subsample rows
    `sub` [m, d] (population variance, float64); lowest coordinate on exact ties.
    This is the definition of the decision."""
    sub = np.asarray(sub, F64)
    var = ((sub - sub.mean(axis=0, keepdims=True)) ** 2).mean(axis=0)
    return int(np.argmax(var)), var


def choose_coordinate_f32(sub):
    """The same decision restated in float32 with a fixed operation order
    (`interleaved_sum32`; no fused multiply-add): mean first, then squared
    deviations.  Not a definition: a helper against which a float32
    implementation can be compared bit for bit.  It can differ from
    `choose_coordinate` only where the two largest variances lie within the
    rounding error of a float32 sum of m terms."""
    sub = np.ascontiguousarray(sub, dtype=np.float32)
    m = np.float32(sub.shape[0])
    mean = interleaved_sum32(sub) / m
    dev = sub - mean
    var = interleaved_sum32(dev * dev) / m
    return int(np.argmax(var)), var


def recursive_split(Y32, c, return_tree=False, choose=choose_coordinate):
    """Diagonalized recursive splitting (Section 3.2.1) on fp32 coordinates.

    Y32 [N, d] float32: rows in principal-component coordinates.  Returns
    perm [N] (position -> original row); cluster j is perm[j*c:(j+1)*c].
    Every set keeps its rows in ascending original order, a split orders the
    set by (coordinate value, original row) and sends the first L rows down.
    `choose` picks the split coordinate from the subsample (the float64
    definition unless the float32 restatement is asked for).
    """
    Y32 = np.asarray(Y32)
    assert Y32.dtype == np.float32
    N, d = Y32.shape
    perm = np.arange(N, dtype=np.int64)
    work = [(0, N)]
    tree = []
    while work:
        nxt = []
        for lo, hi in work:
            s = hi - lo
            if s <= c:
                continue
            rows = perm[lo:hi].copy()
            m = min(d, s)
            sub = Y32[rows[subsample_positions(s, m)]]
            t, _ = choose(sub)
            L = split_point(s, c)
            keys = Y32[rows, t]
            order = np.lexsort((rows, keys))        # by value, then original row
            below = np.zeros(s, dtype=bool)
            below[order[:L]] = True
            perm[lo:lo + L] = rows[below]           # stable two-sided partition
            perm[lo + L:hi] = rows[~below]
            tree.append((lo, hi, t, L))
            nxt.append((lo, lo + L))
            nxt.append((lo + L, hi))
        work = nxt
    if return_tree:
        return perm, tree
    return perm


# --------------------------------------------------------------------------
# Section 3.2.1 "Basic recursive splitting" (the variant of principal direction
# divisive partitioning) with the metric injected into the power iteration, as
# Section 5.2 proposes: no eigendecomposition, no transformed copy of the rows.
# For rows x compared in the metric A = R R (R symmetric), the transformed rows
# are x R and their first principal direction w satisfies w ~ (R C R) w with C
# the covariance of the untransformed rows; in terms of u = R w the iteration is
# u <- A C u and the projection of a row is x . u, so only A is needed.
#
# Every step is float32 with sequential sums (left to right from zero, each
# product and sum rounded on its own), because the projections decide the
# partition:
#   subsample: m = min(d, s) rows at positions floor(j s / m) of the set;
#   mean mu_k = (sum_i x_ik) / m;  z = x - mu;
#   start: g = noise row of the node, gn = g / |g|; the root starts at gn, any
#     other node at (u_parent + gn) / 2  (the parent's estimate and a random
#     vector of the same norm, averaged);
#   one iteration: v_i = sum_k z_ik u_k;  w_k = sum_i z_ik v_i;
#     y_j = sum_k A_jk w_k;  u = y / |y|  (u is kept when |y| is 0 or not finite);
#   projection of every row of the set: t = sum_k x_k u_k;
#   split as in the diagonalized variant: order by (t, row), the first
#   L = c floor((s + c) / (2c)) rows go down, both sides keep ascending row order.
# Nodes are numbered level by level: node = 2^level - 1 + slot, where the bits of
# slot, most significant first, are the path from the root (0 = lower side).
# --------------------------------------------------------------------------
def _seq_dot_rows(Z32, u32):
    """sum_k Z[:, k] u[k] in float32, k ascending, product and sum rounded separately."""
    acc = np.zeros(Z32.shape[0], np.float32)
    for k in range(Z32.shape[1]):
        acc = acc + Z32[:, k] * u32[k]
    return acc


def _seq_norm(v32):
    s = np.float32(0.0)
    for x in v32:
        s = np.float32(s + np.float32(x * x))
    return np.float32(np.sqrt(s))


def basic_direction(sub32, A32, start32, iterations):
    """Power iteration for the first principal direction of the subsample in the metric A
    (dual form u <- A C u), float32 with the operation order stated above."""
    sub32 = np.asarray(sub32, np.float32)
    A32 = np.asarray(A32, np.float32)
    m, d = sub32.shape
    mu = np.zeros(d, np.float32)
    for i in range(m):
        mu = mu + sub32[i]
    mu = mu / np.float32(m)
    z = sub32 - mu[None, :]
    u = np.asarray(start32, np.float32).copy()
    for _ in range(iterations):
        v = _seq_dot_rows(z, u)                        # [m]
        w = np.zeros(d, np.float32)
        for i in range(m):
            w = w + z[i, :] * v[i]
        y = _seq_dot_rows(A32, w)                      # y_j = sum_k A[j, k] w[k]
        nrm = _seq_norm(y)
        if nrm > 0 and np.isfinite(nrm):
            u = y / nrm
    return u


def basic_start(noise_row32, parent_u32):
    g = np.asarray(noise_row32, np.float32)
    gn = g / _seq_norm(g)
    if parent_u32 is None:
        return gn
    return (np.asarray(parent_u32, np.float32) + gn) * np.float32(0.5)


def basic_recursive_split(X32, A32, noise32, c, iterations=3, return_tree=False):
    """X32 [N, d] float32 rows (the stored values), A32 [d, d] metric, noise32
    [2^levels - 1, d] normal deviates, one row per node.  Returns perm [N]."""
    X32 = np.asarray(X32)
    assert X32.dtype == np.float32
    N, d = X32.shape
    perm = np.arange(N, dtype=np.int64)
    work = [(0, N, 0, None)]                # lo, hi, slot, parent direction
    level = 0
    tree = []
    while work:
        nxt = []
        for lo, hi, slot, parent_u in work:
            s = hi - lo
            if s <= c:
                continue
            rows = perm[lo:hi].copy()
            m = min(d, s)
            node = (1 << level) - 1 + slot
            u = basic_direction(X32[rows[subsample_positions(s, m)]], A32,
                                basic_start(noise32[node], parent_u), iterations)
            keys = _seq_dot_rows(X32[rows], u)
            keys = np.where(keys == 0, np.float32(0.0), keys)      # -0 = +0
            L = split_point(s, c)
            order = np.lexsort((rows, keys))
            below = np.zeros(s, dtype=bool)
            below[order[:L]] = True
            perm[lo:lo + L] = rows[below]
            perm[lo + L:hi] = rows[~below]
            tree.append((level, slot, lo, hi, L, u))
            nxt.append((lo, lo + L, 2 * slot, u))
            nxt.append((lo + L, hi, 2 * slot + 1, u))
        work = nxt
        level += 1
    if return_tree:
        return perm, tree
    return perm


def recursive_split_f32(Y32, c, return_tree=False):
    """`recursive_split` with every coordinate chosen by `choose_coordinate_f32`."""
    return recursive_split(Y32, c, return_tree, choose=choose_coordinate_f32)


def split_levels(n, c):
    """Depth of the split tree: the largest set follows the larger child."""
    levels, big = 0, n
    while big > c:
        L = split_point(big, c)
        big = max(L, big - L)
        levels += 1
    return levels


def basic_metrics(Q, K):
    """Metrics of the basic variant: keys are compared in M = Q^T Q / n_q (Section 3.2.2),
    queries in K_c^T K_c / n_k (the un-normalised representation, Appendix B.1); fp64."""
    return centered_scatter(K) / np.asarray(K).shape[0], metric_q(Q)


# --------------------------------------------------------------------------
# Section 3.1 / 3.3.1 / Appendix A: centroids are means over the actual members
# in the ORIGINAL space; |c| is the member count.
# --------------------------------------------------------------------------
def centroids(X, perm, c):
    X = np.asarray(X, F64)
    N = X.shape[0]
    n_c = -(-N // c)
    cen = np.zeros((n_c, X.shape[1]), F64)
    cnt = np.zeros(n_c, np.int64)
    for j in range(n_c):
        rows = perm[j * c:min((j + 1) * c, N)]
        cen[j] = X[rows].mean(axis=0)
        cnt[j] = len(rows)
    return cen, cnt


# Section 3.3.1: score = dot product of the two centroids.
def centroid_scores(cq, ck):
    return np.asarray(cq, F64) @ np.asarray(ck, F64).T


def centroid_scores_f32(cq, ck):
    """The same scores restated in float32 with a fixed operation order: centroids
    rounded to float32, terms added for k = 0, 1, ... with the product and the sum
    rounded separately (no fused multiply-add).  Not a definition: a helper against
    which a float32 implementation can be compared bit for bit; the selection it
    leads to can differ from that of `centroid_scores` only where the k-th and
    (k+1)-th scores lie within float32 rounding of each other."""
    cq = np.ascontiguousarray(cq, dtype=np.float32)
    ck = np.ascontiguousarray(ck, dtype=np.float32)
    S = np.zeros((cq.shape[0], ck.shape[0]), np.float32)
    for k in range(cq.shape[1]):
        S = S + cq[:, k:k + 1] * ck[:, k][None, :]
    return S


# Section 3.3.2 top-k: the k best-scoring key clusters for each query cluster,
# ties to the lower index, listed in ascending index order.
def select_topk(scores, keep):
    scores = np.asarray(scores, F64)
    n_qc, n_kc = scores.shape
    out = np.zeros((n_qc, keep), np.int64)
    idx = np.arange(n_kc)
    for i in range(n_qc):
        order = np.lexsort((idx, -scores[i]))
        out[i] = np.sort(order[:keep])
    return out


# --------------------------------------------------------------------------
# Section 3.3.2, adaptive selection: estimate the attention mass of every key
# cluster from the centroids, |c_j| exp(qbar_i . kbar_j / sqrt(d)), and take the
# most massive clusters until their share of the estimated mass reaches the
# recall threshold, but never fewer than `min_count` (16 in the paper).  The
# paper reaches this set through a two-pass 128-bin histogram; the definition
# written out here is the exact greedy rule that the histogram approximates.
#
# The estimate only feeds discrete decisions (an order and a threshold
# crossing), so it is taken in float32 with operations that any implementation
# can reproduce bit for bit: 2^x by `exp2_f32` below, products and sums rounded
# separately, the running sum taken in the order of decreasing mass.
# --------------------------------------------------------------------------
_EXP2_C = np.array([0.99992806, 0.69326097, 0.24261113, 0.05517165], np.float32)
_LOG2E = np.float32(1.4426950408889634)


def exp2_f32(x):
    """2^x in float32 by a fixed recipe: clamp to [-100, 100], split x = n + f with n
    the nearest integer (adding and subtracting 1.5 * 2^23), cubic polynomial in f
    by Horner's rule with every product and sum rounded separately, scaling by
    2^n.  Relative error 7.5e-5."""
    x = np.minimum(np.maximum(np.asarray(x, np.float32), np.float32(-100.0)), np.float32(100.0))
    magic = np.float32(12582912.0)
    n = (x + magic) - magic
    f = x - n
    p = _EXP2_C[3] * f + _EXP2_C[2]
    p = p * f + _EXP2_C[1]
    p = p * f + _EXP2_C[0]
    return np.ldexp(p, n.astype(np.int32)).astype(np.float32)


def cluster_mass_f32(scores_f32, count_k, scale):
    """Estimated attention mass of every key cluster for every query cluster,
    relative to the row's best score: |c_j| 2^((s_ij - max_j s_ij) scale log2 e)."""
    S = np.asarray(scores_f32, np.float32)
    c = np.float32(np.float32(scale) * _LOG2E)
    rel = (S - S.max(axis=1, keepdims=True)) * c
    return exp2_f32(rel) * np.asarray(count_k, np.float32)[None, :]


def select_adaptive(mass_f32, recall, min_count):
    """Per query cluster: clusters in order of decreasing mass (ties: lower index);
    the shortest prefix whose running float32 sum reaches recall * total, where the
    total is the same running sum over all clusters; at least min_count clusters.
    Returns a list of ascending index arrays (ragged)."""
    mass = np.asarray(mass_f32, np.float32)
    n_qc, n_kc = mass.shape
    idx = np.arange(n_kc)
    lists = []
    for i in range(n_qc):
        order = np.lexsort((idx, -mass[i]))
        run = np.cumsum(mass[i][order], dtype=np.float32)
        target = np.float32(np.float32(recall) * run[-1])
        need = int(np.searchsorted(run, target, side="left")) + 1     # first prefix with run >= target
        if recall >= 1.0:
            need = n_kc                                               # full recall: every cluster, whatever rounding absorbs
        need = min(n_kc, max(need, min_count))
        lists.append(np.sort(order[:need]))
    return lists


def select_blocks_adaptive(cq, ck, count_k, recall, min_count=16, scale=None):
    if scale is None:
        scale = 1.0 / np.sqrt(np.asarray(cq).shape[1])
    return select_adaptive(cluster_mass_f32(centroid_scores_f32(cq, ck), count_k, scale), recall, min_count)


# --------------------------------------------------------------------------
# Sparse attention over the selected clusters (eq. 2) with optional striped
# mean-compensation (Appendix A, the expression for o-hat_S): an excluded
# cluster enters numerator and denominator through its centroid key and value
# with weight |c| * exp(q . k-bar / sqrt(d)).
# `rows_of_cluster` lets the caller evaluate a sample of query clusters only.
# --------------------------------------------------------------------------
def cluster_attention(Q, K, V, perm_q, perm_k, c_q, c_k, block_idx, compensate,
                      ck=None, cv=None, count_k=None, scale=None, query_clusters=None):
    Q = np.asarray(Q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    N_q, d = Q.shape
    N_k = K.shape[0]
    n_kc = -(-N_k // c_k)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    if compensate:
        if ck is None:
            ck, count_k = centroids(K, perm_k, c_k)
        if cv is None:
            cv, _ = centroids(V, perm_k, c_k)
        ck = np.asarray(ck, F64)
        cv = np.asarray(cv, F64)
        count_k = np.asarray(count_k, F64)
    O = np.zeros((N_q, V.shape[1]), F64)
    lse = np.zeros(N_q, F64)
    n_qc = -(-N_q // c_q)
    todo = range(n_qc) if query_clusters is None else query_clusters
    for i in todo:
        rows = perm_q[i * c_q:min((i + 1) * c_q, N_q)]
        sel = np.asarray(block_idx[i], np.int64)
        members = (np.concatenate([perm_k[j * c_k:min((j + 1) * c_k, N_k)] for j in sel]) if len(sel)
                   else np.zeros(0, np.int64))          # S empty: with compensation every cluster enters by its centroid
        logits = scale * (Q[rows] @ K[members].T)
        values = V[members]
        if compensate:
            excluded = np.setdiff1d(np.arange(n_kc), sel)
            if len(excluded):
                lc = scale * (Q[rows] @ ck[excluded].T) + np.log(count_k[excluded])[None, :]
                logits = np.concatenate([logits, lc], axis=1)
                values = np.concatenate([values, cv[excluded]], axis=0)
        mx = logits.max(axis=1, keepdims=True)
        e = np.exp(logits - mx)
        z = e.sum(axis=1, keepdims=True)
        O[rows] = (e / z) @ values
        lse[rows] = (mx + np.log(z))[:, 0]
    return O, lse


# --------------------------------------------------------------------------
# Quantised Q K^T (Section 3.1: the block-sparse kernel the paper runs is a
# quantised one; Section 5.1 names "the quantization in the kernel we use" as a
# source of its error).  The paper does not print that kernel's scheme; the
# variant defined here is: queries and keys are stored as 8-bit floating point
# numbers with 4 exponent and 3 mantissa bits (E4M3: bias 7, largest finite
# value 448, no infinities, subnormals down to 2^-9), each query ROW with its own
# scale, each key CLUSTER with one scale, the key centroids of the compensation
# with one scale per run of 64 centroids; probabilities and values are not
# quantised.  A scale maps the largest magnitude of its group to 448.  Because
# floating point decides the stored codes, scales and scaled values are taken in
# float32 with IEEE operations that any implementation reproduces bit for bit:
#   amax = max |x| over the group;  inv = 448 / amax;  s = amax / 448
#   (both 0 when amax is 0);  code = E4M3(x * inv), round to nearest, ties to
#   even, saturating;  the value the logits see is  s * code.
# Products of two such values and their sums are then exact in float64, so the
# quantised attention is `cluster_attention` on the de-quantised tensors.
# `man_bits` generalises the format (more mantissa bits, same exponent range):
# with enough of them the quantisation disappears, which pins the rest.
# --------------------------------------------------------------------------
def round_to_minifloat(y, man_bits=3, min_exp=-6, max_value=448.0):
    """Rounds float values to the nearest number of the form +-(1 + m / 2^man_bits) 2^e,
    e >= min_exp, or +-(m / 2^man_bits) 2^min_exp below that (subnormals); ties go to the even
    mantissa; magnitudes beyond max_value saturate.  Exact arithmetic in float64."""
    y = np.asarray(y, F64)
    mag = np.abs(y)
    e = np.floor(np.log2(np.where(mag > 0, mag, 1.0)))
    e = np.maximum(e, min_exp)
    step = np.exp2(e - man_bits)                    # spacing of the representable numbers around |y|
    q = np.rint(mag / step) * step                  # np.rint rounds halves to even
    q = np.minimum(q, max_value)
    return np.sign(y) * q


def quantize_group_e4m3(x32, man_bits=3):
    """One group with one scale.  Returns (s, codes) with the de-quantised values s * codes."""
    x32 = np.asarray(x32, np.float32)
    amax = np.float32(np.abs(x32).max()) if x32.size else np.float32(0)
    if amax == 0:
        return np.float32(0), np.zeros(x32.shape, F64)
    inv = np.float32(448.0) / amax                  # float32 division
    s = amax / np.float32(448.0)
    scaled = (x32 * inv).astype(np.float32)         # float32 product
    return s, round_to_minifloat(scaled, man_bits)


def quantize_qk(Q, K, perm_k, c_k, ck=None, man_bits=3):
    """De-quantised (Q~, K~, ck~) of the scheme above: per query row, per key cluster (the rows
    perm_k[j c_k : (j+1) c_k]), per run of 64 key centroids.  float64 arrays."""
    Q = np.asarray(Q, np.float32)
    K = np.asarray(K, np.float32)
    Qd = np.zeros(Q.shape, F64)
    for r in range(Q.shape[0]):
        s, code = quantize_group_e4m3(Q[r], man_bits)
        Qd[r] = F64(s) * code
    Kd = np.zeros(K.shape, F64)
    N_k = K.shape[0]
    for j in range(-(-N_k // c_k)):
        rows = perm_k[j * c_k:min((j + 1) * c_k, N_k)]
        s, code = quantize_group_e4m3(K[rows], man_bits)
        Kd[rows] = F64(s) * code
    ckd = None
    if ck is not None:
        ck = np.asarray(ck, np.float32)
        ckd = np.zeros(ck.shape, F64)
        for j0 in range(0, ck.shape[0], 64):
            s, code = quantize_group_e4m3(ck[j0:j0 + 64], man_bits)
            ckd[j0:j0 + 64] = F64(s) * code
    return Qd, Kd, ckd


def cluster_attention_quantized_qk(Q, K, V, perm_q, perm_k, c_q, c_k, block_idx, compensate,
                                   ck=None, cv=None, count_k=None, scale=None, query_clusters=None, man_bits=3):
    """`cluster_attention` with Q K^T (and the centroid logits) taken on the quantised queries, keys
    and key centroids; values, value centroids and counts as given."""
    if compensate and ck is None:
        ck, count_k = centroids(K, perm_k, c_k)
        ck = ck.astype(np.float32)
    if compensate and cv is None:
        cv, _ = centroids(V, perm_k, c_k)
    Qd, Kd, ckd = quantize_qk(Q, K, perm_k, c_k, ck if compensate else None, man_bits)
    return cluster_attention(Qd, Kd, V, perm_q, perm_k, c_q, c_k, block_idx, compensate, ck=ckd, cv=cv,
                             count_k=count_k, scale=scale, query_clusters=query_clusters)


# --------------------------------------------------------------------------
# The clustering stage for one head, steps in the paper's order:
# metrics -> roots -> transforms -> global principal components -> fp32
# coordinates -> recursive split -> centroids in the original space.
# --------------------------------------------------------------------------
def split_coordinates(Q, K, adaptive=False, return_maps=False):
    """Returns (Yq32, Yk32): the fp32 coordinates the splitter reads.  `adaptive`
    selects the query representation that goes with adaptive selection: the
    metric K_c^T K_c / n without normalisation (Appendix B.1) instead of the
    normalised ranking form (Appendix B.2).  With `return_maps` also the two
    matrices R E (root times principal directions) whose columns fix the signs."""
    R_q = psd_root(metric_q(Q))
    if adaptive:
        R_k = psd_root(centered_scatter(K) / np.asarray(K).shape[0])
    else:
        R_k = psd_root(centered_scatter(K))
    Yk, _, Ek = diagonalize(transform_keys(K, R_q), lift=R_q)
    Yq, _, Eq = diagonalize(query_representation(Q, R_k, normalize=not adaptive), lift=R_k)
    if return_maps:
        return Yq.astype(np.float32), Yk.astype(np.float32), R_k @ Eq, R_q @ Ek
    return Yq.astype(np.float32), Yk.astype(np.float32)


def cluster_qk(Q, K, V, c_q, c_k, Yq32=None, Yk32=None, adaptive=False, f32_decisions=False):
    if Yq32 is None or Yk32 is None:
        Yq32, Yk32 = split_coordinates(Q, K, adaptive)
    choose = choose_coordinate_f32 if f32_decisions else choose_coordinate
    perm_q = recursive_split(Yq32, c_q, choose=choose)
    perm_k = recursive_split(Yk32, c_k, choose=choose)
    cq, count_q = centroids(Q, perm_q, c_q)
    ck, count_k = centroids(K, perm_k, c_k)
    cv, _ = centroids(V, perm_k, c_k)
    return dict(perm_q=perm_q, perm_k=perm_k, cq=cq, ck=ck, cv=cv,
                count_q=count_q, count_k=count_k, Yq32=Yq32, Yk32=Yk32)


def select_blocks(cq, ck, keep):
    """Section 3.3: the `keep` best key clusters per query cluster by the float64 scores."""
    return select_topk(centroid_scores(cq, ck), keep)


def select_blocks_f32(cq, ck, keep):
    """The same selection on the float32 restatement of the scores (`centroid_scores_f32`)."""
    return select_topk(centroid_scores_f32(cq, ck), keep)


def clusterattention_forward(Q, K, V, c_q, c_k, keep, compensate, scale=None):
    """Whole hot path for one head; returns (O, lse, clustering dict, block_idx)."""
    cl = cluster_qk(Q, K, V, c_q, c_k)
    block_idx = select_blocks(cl["cq"], cl["ck"], keep)
    O, lse = cluster_attention(Q, K, V, cl["perm_q"], cl["perm_k"], c_q, c_k, block_idx,
                               compensate, ck=cl["ck"], cv=cl["cv"], count_k=cl["count_k"],
                               scale=scale)
    return O, lse, cl, block_idx

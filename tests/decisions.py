"""How far float32 decisions are from the float64 definitions (test helper).

The device takes its discrete decisions in float32: which coordinate a split
takes (a variance estimate over a subsample) and which key clusters are kept
(centroid scores).  The oracle DEFINES both in float64 and restates them in
float32 with a fixed operation order.  A float32 implementation is compared
  * bit for bit with the float32 restatement, and
  * with the float64 definition through the counts computed here: where the
    two decisions differ, how many rows / lists that touches, and whether every
    difference sits at a near-tie (the two largest variances, or the k-th and
    (k+1)-th scores, closer than float32 rounding can resolve).
Only `oracle/` is used; nothing here comes from the CUDA path.
"""
import numpy as np

from oracle import clusterattn_oracle as orc

# Relative gap of the two largest subsample variances below which a float32 sum of m terms (eight
# partial sums of m/8 terms, a three-level tree, mean and squared deviations each rounded once more)
# can order them differently from float64: each variance carries at most (m/8 + 8) roundings of
# relative size 2^-24, so two of them can cross when they are closer than twice that.
def variance_gap_limit(m):
    return (m / 8 + 8) * 2.0 ** -23

# Scores are float32 sums of d products: a near-tie of the k-th and (k+1)-th score is a gap below
# 1e-5 of the largest score magnitude of the row set (d * 2^-24 = 7.6e-6 at d = 128).
SCORE_GAP = 1e-5
# Rows whose split key lies this close (relative to the spread of the keys of their set) to the
# threshold are reported as near-threshold rows.
KEY_GAP = 1e-6


def split_agreement(Y32, c, perm_f32):
    """`perm_f32`: a permutation produced with float32 coordinate choices on the coordinates Y32
    (it must equal `orc.recursive_split_f32(Y32, c)`, which the caller checks).  Returns the counts
    that relate it to the float64 definition `orc.recursive_split(Y32, c)`."""
    Y32 = np.asarray(Y32)
    N = Y32.shape[0]
    nodes = []

    def both(sub):
        t64, v64 = orc.choose_coordinate(sub)
        t32, _ = orc.choose_coordinate_f32(sub)
        top = np.sort(v64)[::-1]
        gap = (top[0] - top[1]) / top[0] if len(top) > 1 and top[0] > 0 else 0.0
        nodes.append((t64 != t32, gap, sub.shape[0]))
        return t32, None

    perm_walk, tree = orc.recursive_split(Y32, c, return_tree=True, choose=both)
    assert np.array_equal(perm_walk, np.asarray(perm_f32)), "not the float32 restatement's permutation"
    perm64, tree64 = orc.recursive_split(Y32, c, return_tree=True)
    # positions below a node where the two decisions differ (the float32 walk's nodes)
    touched = np.zeros(N, bool)
    differing_nodes, worst_gap, not_near_tie = 0, 0.0, 0
    for (differs, gap, m), (lo, hi, _t, _L) in zip(nodes, tree):
        if differs:
            differing_nodes += 1
            worst_gap = max(worst_gap, gap)
            touched[lo:hi] = True
            if gap > variance_gap_limit(m):
                not_near_tie += 1
    # rows whose cluster differs between the two permutations (same tree shape: cluster = position // c)
    cluster32 = np.empty(N, np.int64)
    cluster64 = np.empty(N, np.int64)
    cluster32[np.asarray(perm_f32)] = np.arange(N) // c
    cluster64[perm64] = np.arange(N) // c
    moved = cluster32 != cluster64
    pos32 = np.empty(N, np.int64)
    pos32[np.asarray(perm_f32)] = np.arange(N)
    moved_outside = int((moved & ~touched[pos32]).sum())
    # rows whose key lies within KEY_GAP of their set's threshold (float64 tree), for the record
    near_threshold = 0
    for lo, hi, t, L in tree64:
        # the set of a node of the float64 tree: its rows are those of positions [lo, hi) in the
        # final permutation (later splits only reorder inside)
        keys = Y32[perm64[lo:hi], t].astype(np.float64)
        thr = np.partition(keys, L - 1)[L - 1]
        spread = keys.std()
        near_threshold += int((np.abs(keys - thr) <= KEY_GAP * spread).sum()) - 1 if spread > 0 else 0
    return dict(rows=N, nodes=len(tree), differing_nodes=differing_nodes, worst_gap=worst_gap,
                differing_nodes_not_near_tie=not_near_tie, rows_moved=int(moved.sum()),
                rows_moved_outside_differing_nodes=moved_outside, near_threshold_rows=near_threshold)


def check_split_agreement(Y32, c, perm_f32, label=""):
    """Asserts the bar: every differing decision is a near-tie, every moved row descends from one,
    and fewer than 0.1 % of the rows end in another cluster.  Prints the counts."""
    a = split_agreement(Y32, c, perm_f32)
    print(f"split decisions {label}: {a['nodes']} nodes, float32 and float64 choose another coordinate at "
          f"{a['differing_nodes']} (largest relative variance gap there {a['worst_gap']:.2e}); "
          f"{a['rows_moved']} of {a['rows']} rows end in another cluster; "
          f"{a['near_threshold_rows']} rows lie within {KEY_GAP:g} of a split threshold")
    assert a["differing_nodes_not_near_tie"] == 0
    assert a["rows_moved_outside_differing_nodes"] == 0
    assert a["rows_moved"] < 1e-3 * a["rows"]
    return a


def selection_agreement(cq32, ck32, keep, idx_f32):
    """`idx_f32` [n_qc, keep]: lists selected on float32 scores (the caller checks that they equal
    `orc.select_blocks_f32`).  Returns the counts that relate them to the float64 definition."""
    cq32 = np.asarray(cq32, np.float32)
    ck32 = np.asarray(ck32, np.float32)
    S = orc.centroid_scores(cq32, ck32)
    idx64 = orc.select_topk(S, keep)
    n_qc, n_kc = S.shape
    scale = np.abs(S).max()
    differing, near_tie_lists, unexplained = 0, 0, 0
    for i in range(n_qc):
        ranked = np.sort(S[i])[::-1]
        kth = ranked[keep - 1]
        gap = kth - ranked[keep] if keep < n_kc else np.inf
        near = gap < SCORE_GAP * scale
        near_tie_lists += int(near)
        a, b = set(np.asarray(idx_f32[i]).tolist()), set(idx64[i].tolist())
        if a != b:
            differing += 1
            # the entries that differ must all be candidates of the near-tie
            odd = np.array(sorted(a ^ b))
            if not near or np.abs(S[i, odd] - kth).max() >= SCORE_GAP * scale:
                unexplained += 1
    return dict(lists=n_qc, differing_lists=differing, near_tie_lists=near_tie_lists,
                differing_lists_not_near_tie=unexplained)


def check_selection_agreement(cq32, ck32, keep, idx_f32, label=""):
    a = selection_agreement(cq32, ck32, keep, idx_f32)
    print(f"block lists {label}: {a['differing_lists']} of {a['lists']} differ from the float64 selection; "
          f"{a['near_tie_lists']} lists have their k-th and (k+1)-th score within {SCORE_GAP:g} of the largest score")
    assert a["differing_lists_not_near_tie"] == 0
    return a


def coordinates_agreement(Y_dev, Y_orc):
    """Split coordinates computed by a float32 pipeline against the oracle's (float64, rounded to
    float32), column by column.  Both sides orient every component by the same rule (the column of
    the map from the original space, see `orc.principal_basis`), so well-separated components must
    agree element by element.  A component whose variance is close to its neighbour's is defined
    only up to a rotation inside that pair: its error is reported against the relative gap.
    Returns per-column arrays: variance (oracle), relative gap to the nearest neighbour, maximum
    absolute deviation in units of sqrt(largest variance), and the cosine between the two columns."""
    Yd = np.asarray(Y_dev, np.float64)
    Yo = np.asarray(Y_orc, np.float64)
    var = (Yo * Yo).mean(axis=0)
    d = var.shape[0]
    gap = np.empty(d)
    for t in range(d):
        near = [abs(var[t] - var[u]) for u in (t - 1, t + 1) if 0 <= u < d]
        gap[t] = min(near) / var[0]
    dev = np.abs(Yd - Yo).max(axis=0) / np.sqrt(var[0])
    cos = (Yd * Yo).sum(axis=0) / np.maximum(np.sqrt((Yd * Yd).sum(axis=0) * (Yo * Yo).sum(axis=0)), 1e-300)
    return dict(var=var, gap=gap, dev=dev, cos=cos)


def root_split_agreement(Y_dev, Y_orc, c):
    """The first split of the two pipelines, before any difference can cascade: the coordinate each
    side chooses, the rows that land on different sides, and how far those rows are from the
    oracle's threshold (in units of the key's spread).  Rows can only change sides when the
    difference of the two key columns reaches their distance from the threshold."""
    Y_dev, Y_orc = np.asarray(Y_dev), np.asarray(Y_orc)
    N, d = Y_orc.shape
    m = min(d, N)
    pos = orc.subsample_positions(N, m)
    t_dev, _ = orc.choose_coordinate(Y_dev[pos])
    t_orc, _ = orc.choose_coordinate(Y_orc[pos])
    out = dict(t_dev=t_dev, t_orc=t_orc, rows=N)
    if t_dev != t_orc or N <= c:
        return out
    L = orc.split_point(N, c)
    idx = np.arange(N)
    below = []
    for Y in (Y_dev, Y_orc):
        order = np.lexsort((idx, Y[:, t_orc]))
        b = np.zeros(N, bool)
        b[order[:L]] = True
        below.append(b)
    flipped = below[0] != below[1]
    keys = Y_orc[:, t_orc].astype(np.float64)
    thr = np.partition(keys, L - 1)[L - 1]
    spread = keys.std()
    out.update(flipped=int(flipped.sum()),
               flipped_max_distance=float(np.abs(keys[flipped] - thr).max() / spread) if flipped.any() else 0.0,
               key_max_difference=float(np.abs(Y_dev[:, t_orc].astype(np.float64) - keys).max() / spread),
               near_threshold_rows=int((np.abs(keys - thr) <= KEY_GAP * spread).sum()) - 1)
    return out


def within_cluster_scatter(Y, perm, c):
    """Mean squared distance of the rows to their cluster's mean, in the coordinates Y."""
    Y = np.asarray(Y, np.float64)
    N = Y.shape[0]
    total = 0.0
    for j in range(-(-N // c)):
        rows = perm[j * c:min((j + 1) * c, N)]
        total += ((Y[rows] - Y[rows].mean(axis=0)) ** 2).sum()
    return total / N


# The orientation of a component is itself a decision taken in floating point: the sign of the entry
# of largest magnitude of a column of R E.  Where the two largest magnitudes of that column lie this
# close (relative) and carry opposite signs, either orientation is a valid outcome of the rule.
SIGN_GAP = 2e-3


def check_coordinates(label, w, Qh, Kh, Yq_dev, Yk_dev, pq_dev, pk_dev, adaptive=False):
    """The device's chain from Q and K to the split coordinates against the oracle's own chain.
    Components whose variance is separated from both neighbours by more than 1 % of the largest
    variance must agree element by element (the sign rule is the same on both sides); closer ones
    may rotate inside their pair, in proportion to float32 rounding over the gap, and must still
    point the same way.  A component that comes out mirrored is accepted only where the sign rule
    itself is at a near-tie (counted and printed); it is mirrored back for the checks that follow.
    The first split of the two chains is compared before differences can cascade: same coordinate,
    and the rows that change sides lie no further from the threshold than the two key columns
    differ.  Last, the two clusterings are equally tight."""
    Yq_orc, Yk_orc, Wq, Wk = orc.split_coordinates(Qh, Kh, adaptive=adaptive, return_maps=True)
    for side, Yd, Yo, Wmap, perm, n in (("queries", Yq_dev, Yq_orc, Wq, pq_dev, w.n_q),
                                        ("keys", Yk_dev, Yk_orc, Wk, pk_dev, w.n_k)):
        a = coordinates_agreement(Yd, Yo)
        mirrored = np.nonzero((a["cos"] < 0) & (a["gap"] > 1e-4))[0]
        if len(mirrored):
            for t in mirrored:
                col = Wmap[:, t]
                top = np.argsort(-np.abs(col))[:2]
                rel = (abs(col[top[0]]) - abs(col[top[1]])) / abs(col[top[0]])
                print(f"{label} {side}: component {t} is mirrored; the two largest entries of its column of R E "
                      f"differ by {rel:.2e} (relative) with signs {np.sign(col[top[0]]):+.0f} / {np.sign(col[top[1]]):+.0f}")
                assert rel < SIGN_GAP and col[top[0]] * col[top[1]] < 0, "a mirrored component away from a sign near-tie"
            Yd = np.array(Yd, copy=True)
            Yd[:, mirrored] *= -1.0
            a = coordinates_agreement(Yd, Yo)
        sep = a["gap"] > 1e-2
        print(f"{label} {side}: {int(sep.sum())} of {len(sep)} components separated by > 1 % of the largest variance: "
              f"max deviation {a['dev'][sep].max() if sep.any() else 0:.2e} sqrt(var0); all components: "
              f"max deviation x gap {np.max(a['dev'] * np.maximum(a['gap'], 1e-7)):.2e}, min cosine {a['cos'].min():.6f}")
        assert (a["dev"][sep] < 2e-3).all()
        # a rotation inside a near-degenerate pair: error ~ (rounding of the covariance, 2e-6) / gap
        assert (a["dev"] * np.maximum(a["gap"], 1e-7) < 4e-5).all()
        assert (a["cos"][a["gap"] > 1e-4] > 0.5).all()
        root = root_split_agreement(Yd, Yo, w.cluster)
        print(f"{label} {side}: first split on coordinate {root['t_dev']} (device) / {root['t_orc']} (oracle); "
              f"{root.get('flipped', 'n/a')} of {n} rows change sides, the farthest {root.get('flipped_max_distance', 0):.2e} "
              f"spreads from the threshold (keys differ by at most {root.get('key_max_difference', 0):.2e}); "
              f"{root.get('near_threshold_rows', 0)} rows within {KEY_GAP:g} of the threshold")
        assert root["t_dev"] == root["t_orc"]
        if "flipped" in root:
            assert root["flipped_max_distance"] <= 2 * root["key_max_difference"] + 1e-12
            assert root["flipped"] < 1e-3 * n
        # equally tight clusters, measured in the oracle's coordinates
        mine = within_cluster_scatter(Yo, perm, w.cluster)
        theirs = within_cluster_scatter(Yo, orc.recursive_split(Yo, w.cluster), w.cluster)
        print(f"{label} {side}: within-cluster scatter {mine:.5g} (device clustering) / {theirs:.5g} (oracle clustering)")
        assert abs(mine / theirs - 1) < 0.03

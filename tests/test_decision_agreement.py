"""The float32 restatements of the oracle's decisions against their float64 definitions on
the synthetic workloads (CPU only): the counts that the GPU tests report for the device's
results, here for the oracle's own float32 helpers."""
import numpy as np

from oracle import clusterattn_oracle as orc
from paper_2608_26965_b200 import inputs
from tests import decisions


def test_tiny_workload_decisions_agree():
    w = inputs.WORKLOADS["tiny"]
    Q, K, V = inputs.generate(w)
    for h in range(w.heads):
        Yq, Yk = orc.split_coordinates(Q[h], K[h])
        for Y in (Yq, Yk):
            a = decisions.check_split_agreement(Y, w.cluster, orc.recursive_split_f32(Y, w.cluster), f"tiny head {h}")
            assert a["nodes"] == 15
        cl = orc.cluster_qk(Q[h], K[h], V[h], w.cluster, w.cluster)
        cq, ck = cl["cq"].astype(np.float32), cl["ck"].astype(np.float32)
        decisions.check_selection_agreement(cq, ck, w.keep, orc.select_blocks_f32(cq, ck, w.keep), f"tiny head {h}")


def test_split_agreement_counts_a_forced_near_tie():
    """Two coordinates that mirror each other up to 1e-7 (equal variances, opposite order):
    wherever the float32 estimate picks the other one, the node is counted, its rows are the only
    ones that move, and the gap is inside the near-tie limit."""
    r = np.random.default_rng(5)
    found = False
    for trial in range(400):
        n, c = 256, 64
        col = r.standard_normal(n)
        Y = np.stack([col, -col * (1 + r.uniform(-2e-7, 2e-7)), 0.2 * r.standard_normal(n)],
                     axis=1).astype(np.float32)
        a = decisions.split_agreement(Y, c, orc.recursive_split_f32(Y, c))
        assert a["differing_nodes_not_near_tie"] == 0 and a["rows_moved_outside_differing_nodes"] == 0
        if a["differing_nodes"]:
            found = True
            assert a["worst_gap"] <= decisions.variance_gap_limit(3) and a["rows_moved"] > 0
            break
    assert found


def test_selection_agreement_counts_a_forced_near_tie():
    r = np.random.default_rng(6)
    cq = r.standard_normal((5, 64)).astype(np.float32)
    ck = r.standard_normal((12, 64)).astype(np.float32)
    a = decisions.selection_agreement(cq, ck, 4, orc.select_blocks_f32(cq, ck, 4))
    assert a["differing_lists"] == 0 and a["differing_lists_not_near_tie"] == 0
    # a list that swaps a clearly better cluster for a clearly worse one is not explained by a near-tie
    S = orc.centroid_scores(cq, ck)
    bad = orc.select_topk(S, 4).copy()
    worst = int(np.argmin(S[2]))
    bad[2] = np.sort(np.append(bad[2][1:], worst)) if worst not in bad[2] else bad[2]
    b = decisions.selection_agreement(cq, ck, 4, bad)
    assert b["differing_lists"] == 1 and b["differing_lists_not_near_tie"] == 1

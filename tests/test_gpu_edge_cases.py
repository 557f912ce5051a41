"""Degenerate inputs and argument errors, through the C ABI on the device."""
import ctypes

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


def test_identical_keys_give_the_mean_of_the_values():
    """Every key equal (zero covariance: all pivots of the factorisation drop out, every split
    coordinate ties and rows split in index order).  All logits of a query are equal, so the
    compensated output is the plain mean of V whatever is selected (Appendix A: the centroid
    stands for its members exactly when their weights are equal)."""
    r = np.random.default_rng(5)
    H, n_q, n_k, d, c = 2, 300, 1000, 64, 64
    Q = r.standard_normal((H, n_q, d)).astype(np.float32)
    K = np.tile(r.standard_normal((H, 1, d)).astype(np.float32), (1, n_k, 1))
    V = r.standard_normal((H, n_k, d)).astype(np.float32)
    p = binding.make_problem(1, H, n_q, n_k, d, "fp32", c, c, 3)
    plan = binding.Plan(p, DEV)
    O = plan.forward(dev(Q[None]), dev(K[None]), dev(V[None]), want_lse=True)
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    for h in range(H):
        perm_k = plan.perm_k[0, h].cpu().numpy()
        assert np.array_equal(np.sort(perm_k), np.arange(n_k))
        assert np.array_equal(perm_k, np.arange(n_k))            # ties everywhere: index order survives
        want = V[h].astype(np.float64).mean(0)
        assert np.abs(O[0, h].cpu().numpy() - want).max() < 1e-5
        # the oracle agrees on the clustering of the queries computed by the device
        o_ref, _ = orc.cluster_attention(Q[h], K[h], V[h], plan.perm_q[0, h].cpu().numpy(), perm_k, c, c,
                                         plan.block_idx[0, h].cpu().numpy(), True)
        assert np.abs(O[0, h].cpu().numpy() - o_ref).max() < 1e-5


def test_zero_queries_and_a_single_cluster():
    """Q = 0: the metric is zero, r(q) is the zero vector, every score ties; n_k <= c: one key
    cluster, kept by every query cluster; the result is dense attention with equal weights."""
    r = np.random.default_rng(6)
    H, n_q, n_k, d, c = 1, 200, 100, 128, 128
    Q = np.zeros((H, n_q, d), np.float32)
    K = r.standard_normal((H, n_k, d)).astype(np.float32)
    V = r.standard_normal((H, n_k, d)).astype(np.float32)
    p = binding.make_problem(1, H, n_q, n_k, d, "bf16", c, c, 1)
    plan = binding.Plan(p, DEV)
    O = plan.forward(dev(Q[None], torch.bfloat16), dev(K[None], torch.bfloat16), dev(V[None], torch.bfloat16))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    assert int(plan.count_k[0, 0, 0]) == n_k and plan.count_k.numel() == 1
    want = inputs.round_to_bf16(V[0]).astype(np.float64).mean(0)
    assert np.abs(O[0, 0].float().cpu().numpy() - want).max() < 2e-2


def test_argument_errors_enqueue_nothing():
    lib = binding.load_library()
    good = binding.make_problem(1, 1, 256, 256, 64, "bf16", 64, 64, 2)
    plan = binding.Plan(good, DEV)
    launches = binding.kernel_launches()

    def attn(problem, ws=None, ws_bytes=None, block_idx=None):
        ws = plan.ws["attn"] if ws is None else ws
        args = [plan.Qp, plan.Kp, plan.Vp, plan.ck, plan.cv, plan.count_k,
                plan.block_idx if block_idx is None else block_idx, plan.perm_q]
        return lib.cluster_attention_fwd(ctypes.byref(problem), *[ctypes.c_void_p(t.data_ptr()) for t in args],
                                         ctypes.c_void_p(plan.O.data_ptr()), None, ctypes.c_void_p(ws.data_ptr()),
                                         ws.numel() if ws_bytes is None else ws_bytes, None)

    assert attn(good.copy(keep=5)) == binding.CA_ERR_INVALID_ARG            # more than n_kc = 4
    assert attn(good.copy(keep=0)) == binding.CA_ERR_INVALID_ARG
    assert attn(good.copy(cluster_k=96)) == binding.CA_ERR_INVALID_ARG      # not a power of two
    assert attn(good.copy(head_dim=96)) == binding.CA_ERR_UNSUPPORTED
    assert attn(good.copy(n_q=0)) == binding.CA_ERR_INVALID_ARG
    assert attn(good, ws_bytes=16) == binding.CA_ERR_WORKSPACE
    odd = torch.empty(plan.block_idx.numel() + 1, dtype=torch.int32, device=DEV)[1:]   # 4-byte aligned only
    assert attn(good, block_idx=odd) == binding.CA_ERR_INVALID_ARG
    rc = lib.select_blocks_adaptive(ctypes.byref(good), ctypes.c_void_p(plan.cq.data_ptr()),
                                    ctypes.c_void_p(plan.ck.data_ptr()), ctypes.c_void_p(plan.count_k.data_ptr()),
                                    0.0, 16, ctypes.c_void_p(plan.block_idx.data_ptr()),
                                    ctypes.c_void_p(plan.count_q.data_ptr()), ctypes.c_void_p(plan.ws["select"].data_ptr()),
                                    plan.ws["select"].numel(), None)
    assert rc == binding.CA_ERR_INVALID_ARG                                  # recall must be positive
    torch.cuda.synchronize()
    assert binding.kernel_launches() == launches                            # nothing was enqueued


def _bf16_round(a):
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).float().numpy()


@pytest.mark.parametrize("d,c_q,c_k,compensate", [(64, 128, 128, False), (64, 128, 32, True), (128, 128, 128, True),
                                                  (128, 128, 32, False), (64, 128, 64, True),
                                                  (64, 256, 128, True),      # two CTAs per query cluster
                                                  (128, 64, 128, False)])    # half-filled query tile
def test_attention_scores_that_rise_along_the_list(d, c_q, c_k, compensate):
    """Key blocks listed in an order in which the scores of a row climb by tens and by hundreds of
    binary orders of magnitude from one block to the next, and fall by as much for other rows: the
    running reference of the online softmax (Section 3.1: exact softmax over the kept blocks) has
    to follow without overflow, whatever it was before.  With 32-row key clusters the climb happens
    in the middle of a 64-column half-step."""
    r = np.random.default_rng(31 + d + c_k)
    H, n_q = 1, 300 if c_q < 256 else 700
    gains = np.array([0.0, 2.0, 4.0, 60.0, 62.0, 30.0, 600.0, 610.0, 100.0, 1200.0, 1.0, 3.0])
    n_kc = len(gains)
    n_k = n_kc * c_k - 5                                     # short last cluster
    e = np.zeros(d); e[:4] = 0.5                             # unit direction
    a = r.uniform(2.0, 5.0, n_q) * np.where(r.random(n_q) < 0.25, -1.0, 1.0)
    Q = _bf16_round(a[:, None] * e[None] + 0.3 * r.standard_normal((n_q, d)))
    K = _bf16_round(np.repeat(gains, c_k)[:n_k, None] * e[None] + 0.3 * r.standard_normal((n_k, d)))
    V = _bf16_round(r.standard_normal((n_k, d)))
    perm_q, perm_k = np.arange(n_q), np.arange(n_k)
    n_qc = -(-n_q // c_q)
    keep = 10
    lists = [np.arange(keep), np.arange(keep), np.r_[np.arange(5, keep), np.arange(5)]]
    idx = np.stack([lists[i % 3] for i in range(n_qc)]).astype(np.int32)
    ck, count_k = orc.centroids(K, perm_k, c_k)
    cv, _ = orc.centroids(V, perm_k, c_k)
    ck32, cv32 = ck.astype(np.float32), cv.astype(np.float32)
    o_ref, lse_ref = orc.cluster_attention(Q, K, V, perm_q, perm_k, c_q, c_k, idx, compensate,
                                           ck=ck32, cv=cv32, count_k=count_k)
    p = binding.make_problem(1, H, n_q, n_k, d, "bf16", c_q, c_k, keep, compensate)
    plan = binding.Plan(p, DEV)

    def pad(x, n, c):
        out = np.zeros((-(-n // c) * c, x.shape[1]), np.float32)
        out[:n] = x
        return out
    bf = torch.bfloat16
    O, lse = plan.cluster_attention_fwd(dev(pad(Q, n_q, c_q)[None, None], bf), dev(pad(K, n_k, c_k)[None, None], bf),
                                        dev(pad(V, n_k, c_k)[None, None], bf), dev(ck32[None, None]),
                                        dev(cv32[None, None]), dev(count_k[None, None], torch.int32),
                                        dev(idx[None, None], torch.int32), dev(perm_q[None, None], torch.int32))
    torch.cuda.synchronize()
    assert all(v == 0 for v in plan.last_status().values())
    O, lse = O[0, 0].float().cpu().numpy(), lse[0, 0].cpu().numpy()
    assert np.isfinite(O).all() and np.isfinite(lse).all()
    # the climbs of 2^300 and 2^600 leave the range of the tensor-core kernel's late reference:
    # those query clusters went through the second pass
    assert plan.recomputed_clusters() > 0
    assert np.abs(O - o_ref).max() <= 2e-2 and np.linalg.norm(O - o_ref) <= 5e-3 * np.linalg.norm(o_ref)
    assert np.abs(lse - lse_ref).max() <= 2e-2 + 1e-4 * np.abs(lse_ref).max()

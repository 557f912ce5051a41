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


# ----------------------------------------------------------------------------
# Indices that come from the caller are checked before use; waits are bounded.
# ----------------------------------------------------------------------------
def _attention_inputs(dtype, d, n_q, n_k, c, keep, seed):
    """A valid attention problem on an arbitrary permutation: host arrays + device tensors."""
    r = np.random.default_rng(seed)
    Q = _bf16_round(r.standard_normal((n_q, d)))
    K = _bf16_round(r.standard_normal((n_k, d)))
    V = _bf16_round(r.standard_normal((n_k, d)))
    perm_q, perm_k = r.permutation(n_q), r.permutation(n_k)
    n_qc, n_kc = -(-n_q // c), -(-n_k // c)
    idx = np.stack([np.sort(r.choice(n_kc, keep, replace=False)) for _ in range(n_qc)]).astype(np.int32)
    ck, count_k = orc.centroids(K, perm_k, c)
    cv, _ = orc.centroids(V, perm_k, c)

    def pad(x, perm, n):
        out = np.zeros((-(-n // c) * c, d), np.float32)
        out[:n] = x[perm]
        return out
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    t = dict(Qp=dev(pad(Q, perm_q, n_q)[None, None], dt), Kp=dev(pad(K, perm_k, n_k)[None, None], dt),
             Vp=dev(pad(V, perm_k, n_k)[None, None], dt), ck=dev(ck.astype(np.float32)[None, None]),
             cv=dev(cv.astype(np.float32)[None, None]), count_k=dev(count_k[None, None], torch.int32))
    host = dict(Q=Q, K=K, V=V, perm_q=perm_q, perm_k=perm_k, idx=idx, ck=ck.astype(np.float32),
                cv=cv.astype(np.float32), count_k=count_k)
    return host, t


@pytest.mark.parametrize("dtype,d,c", [("bf16", 64, 128), ("bf16", 128, 32), ("fp32", 64, 64)])
def test_forged_indices_are_reported_and_skipped(dtype, d, c):
    """A block list with entries that are no key clusters and a perm_q entry that is no row of O:
    the call reports CA_ERR_BAD_INDEX in the status word, treats the forged clusters as absent (the
    oracle on the list without them gives the same rows) and leaves the forged row unwritten."""
    n_q, n_k, keep = 5 * c + 17, 9 * c + 3, 4
    host, t = _attention_inputs(dtype, d, n_q, n_k, c, keep, seed=91)
    n_kc = -(-n_k // c)
    idx = host["idx"].copy()
    idx[2, 1] = n_kc + 5
    idx[2, 3] = -7
    perm_q = host["perm_q"].astype(np.int32).copy()
    forged_pos = 3 * c + 5
    lost_row = int(perm_q[forged_pos])
    perm_q[forged_pos] = n_q + 3
    p = binding.make_problem(1, 1, n_q, n_k, d, dtype, c, c, keep, True)
    plan = binding.Plan(p, DEV)
    plan.O.fill_(7.0)
    plan.lse.fill_(7.0)
    O, lse = plan.cluster_attention_fwd(t["Qp"], t["Kp"], t["Vp"], t["ck"], t["cv"], t["count_k"],
                                        dev(idx[None, None], torch.int32), dev(perm_q[None, None], torch.int32))
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == binding.CA_ERR_BAD_INDEX
    O, lse = O[0, 0].float().cpu().numpy(), lse[0, 0].cpu().numpy()
    assert np.isfinite(O).all() and np.isfinite(lse).all()
    assert (O[lost_row] == 7.0).all() and lse[lost_row] == 7.0          # not written
    lists = [row[(row >= 0) & (row < n_kc)] for row in idx]
    o_ref, lse_ref = orc.cluster_attention(host["Q"], host["K"], host["V"], host["perm_q"], host["perm_k"], c, c,
                                           lists, True, ck=host["ck"], cv=host["cv"], count_k=host["count_k"])
    rows = np.setdiff1d(np.arange(n_q), [lost_row])
    tol = 1e-5 if dtype == "fp32" else 2e-2
    assert np.abs(O[rows] - o_ref[rows]).max() <= tol and np.abs(lse[rows] - lse_ref[rows]).max() <= tol
    # the next call on the same workspace with valid indices is clean
    plan.cluster_attention_fwd(t["Qp"], t["Kp"], t["Vp"], t["ck"], t["cv"], t["count_k"],
                               dev(host["idx"][None, None], torch.int32),
                               dev(host["perm_q"].astype(np.int32)[None, None], torch.int32))
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == 0


@pytest.mark.parametrize("dtype,compensate", [("bf16", True), ("bf16", False), ("fp32", False)])
def test_ragged_list_lengths_of_zero_and_beyond_the_row(dtype, compensate):
    """cluster_attention_fwd_ragged with a list of length 0 (with compensation: centroids only;
    without: no entry at all, the rows are zeros with lse = -inf) and with a length beyond the row
    (clamped to the row and reported)."""
    d, c, n_q, n_k = 64, 64, 4 * 64, 6 * 64
    host, t = _attention_inputs(dtype, d, n_q, n_k, c, 6, seed=92)
    n_kc = 6
    idx = np.tile(np.arange(n_kc, dtype=np.int32), (4, 1))
    keep_count = np.array([3, 0, 6, 2], np.int32)
    p = binding.make_problem(1, 1, n_q, n_k, d, dtype, c, c, 1, compensate)
    plan = binding.Plan(p, DEV)
    args = (t["Qp"], t["Kp"], t["Vp"], t["ck"], t["cv"], t["count_k"], dev(host["perm_q"].astype(np.int32)[None, None], torch.int32))
    O, lse = plan.cluster_attention_fwd_ragged(dev(idx[None, None], torch.int32), dev(keep_count[None, None], torch.int32), *args)
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == 0
    O, lse = O[0, 0].float().cpu().numpy(), lse[0, 0].cpu().numpy()
    lists = [idx[i, :keep_count[i]] for i in range(4)]
    tol = 1e-5 if dtype == "fp32" else 2e-2
    empty_rows = host["perm_q"][c:2 * c]
    others = np.setdiff1d(np.arange(n_q), empty_rows)
    if compensate:
        o_ref, lse_ref = orc.cluster_attention(host["Q"], host["K"], host["V"], host["perm_q"], host["perm_k"], c, c,
                                               lists, True, ck=host["ck"], cv=host["cv"], count_k=host["count_k"])
        assert np.abs(O - o_ref).max() <= tol and np.abs(lse - lse_ref).max() <= tol
    else:
        lists_ne = [l if len(l) else np.array([0]) for l in lists]
        o_ref, lse_ref = orc.cluster_attention(host["Q"], host["K"], host["V"], host["perm_q"], host["perm_k"], c, c,
                                               lists_ne, False)
        assert np.abs(O[others] - o_ref[others]).max() <= tol
        assert (O[empty_rows] == 0).all() and np.isneginf(lse[empty_rows]).all()
    # a length beyond the row: reported, clamped to the row
    keep_count[3] = n_kc + 4
    O2, _ = plan.cluster_attention_fwd_ragged(dev(idx[None, None], torch.int32), dev(keep_count[None, None], torch.int32), *args)
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == binding.CA_ERR_BAD_INDEX
    lists[3] = idx[3]
    o_ref, _ = orc.cluster_attention(host["Q"], host["K"], host["V"], host["perm_q"], host["perm_k"], c, c,
                                     [l if len(l) else np.array([0]) for l in lists], compensate,
                                     ck=host["ck"], cv=host["cv"], count_k=host["count_k"])
    rows = host["perm_q"][3 * c:4 * c]
    assert np.abs(O2[0, 0].float().cpu().numpy()[rows] - o_ref[rows]).max() <= tol


@pytest.mark.parametrize("d", [64, 128])
def test_a_wait_that_runs_out_ends_the_kernel_with_a_status(d):
    """The loader of the tensor-core attention kernel is told (diagnostic hook) to leave out the key
    rows of one half-step, with the limit of the device-side waits set to about a millisecond: the
    waits for those rows run out, the kernel records CA_ERR_TIMEOUT, releases its tensor memory and
    returns.  With the hook cleared the next call on the same workspace is correct again."""
    lib = binding.load_library()
    c, n_q, n_k, keep = 128, 512, 1024, 3
    host, t = _attention_inputs("bf16", d, n_q, n_k, c, keep, seed=93)
    p = binding.make_problem(1, 1, n_q, n_k, d, "bf16", c, c, keep, True)
    plan = binding.Plan(p, DEV)
    args = (t["Qp"], t["Kp"], t["Vp"], t["ck"], t["cv"], t["count_k"], dev(host["idx"][None, None], torch.int32),
            dev(host["perm_q"].astype(np.int32)[None, None], torch.int32))
    good = plan.cluster_attention_fwd(*args)[0].clone()
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == 0
    try:
        lib.ca_debug_attn_wait(2_000_000, 2)
        plan.cluster_attention_fwd(*args)
        torch.cuda.synchronize()
        assert plan.last_status()["attn"] == binding.CA_ERR_TIMEOUT
    finally:
        lib.ca_debug_attn_wait(0, -1)
    again = plan.cluster_attention_fwd(*args)[0]
    torch.cuda.synchronize()
    assert plan.last_status()["attn"] == 0
    assert torch.equal(again, good)
    o_ref, _ = orc.cluster_attention(host["Q"], host["K"], host["V"], host["perm_q"], host["perm_k"], c, c,
                                     host["idx"], True, ck=host["ck"], cv=host["cv"], count_k=host["count_k"])
    assert np.abs(again[0, 0].float().cpu().numpy() - o_ref).max() <= 2e-2


def test_two_host_threads_on_two_streams_give_the_sequential_results():
    """Two plans driven from two host threads on their own streams at the same time (the library's
    side streams come from a pool, its launch counter is atomic): every output equals the one of the
    same call made alone."""
    import threading
    w = inputs.WORKLOADS["tabular"].scaled(heads=2, n_q=4096, n_k=16384, keep=16)
    data = [inputs.generate(w.scaled(config_id=w.config_id + 7 * i)) for i in range(2)]
    p = binding.problem_from_workload(w)
    tensors = [[torch.from_numpy(a[None]).to(torch.bfloat16).to(DEV) for a in d] for d in data]
    alone = []
    for t in tensors:
        plan = binding.Plan(p, DEV)
        O = plan.forward(*t, want_lse=True)
        torch.cuda.synchronize()
        alone.append([x.clone() for x in (O, plan.lse, plan.perm_q, plan.perm_k, plan.block_idx)])
    plans = [binding.Plan(p, DEV) for _ in range(2)]
    streams = [torch.cuda.Stream() for _ in range(2)]
    errors = []

    def work(i):
        try:
            with torch.cuda.device(0):
                for _ in range(5):
                    plans[i].forward(*tensors[i], want_lse=True, stream=streams[i])
                streams[i].synchronize()
        except Exception as exc:      # noqa: BLE001
            errors.append(exc)
    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for i in range(2):
        assert all(v == 0 for v in plans[i].last_status().values())
        got = (plans[i].O, plans[i].lse, plans[i].perm_q, plans[i].perm_k, plans[i].block_idx)
        for a, b in zip(got, alone[i]):
            assert torch.equal(a, b)

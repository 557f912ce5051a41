"""cluster_attention_fwd_static: the attention stage for callers that cannot
allocate device memory (no workspace argument; the library's fixed scratch
array is used instead).  Checked here against the regular entry point on two
calls in a row that use different problems, so that whatever the first call
left in the shared scratch must not leak into the second.

This file is collected last on purpose: a run that stops at the first failure
has then already been through every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import clusterattn_oracle as orc
from paper_2608_26965_b200 import binding, build, inputs

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def prepared_plan(name, heads, n_q, n_k, keep, compensate):
    """Clustering and selection through the regular entry points; returns the plan
    holding every input of the attention stage."""
    w = inputs.WORKLOADS[name].scaled(heads=heads, n_q=n_q, n_k=n_k)
    Q, K, V = inputs.generate(w)
    p = binding.problem_from_workload(w, keep=keep, compensate=compensate)
    dt = binding.torch_dtype(p)
    plan = binding.Plan(p, DEV)
    dev = lambda a: torch.from_numpy(a[None]).to(dt).to(DEV)
    plan.cluster_qk(dev(Q), dev(K), dev(V))
    plan.select_blocks()
    plan.host_inputs = (Q, K, V, w)
    return plan


def run_both(plan):
    p = plan.problem
    O_ref, lse_ref = plan.cluster_attention_fwd(want_lse=True)
    O_ref, lse_ref = O_ref.clone(), lse_ref.clone()
    O = torch.full_like(plan.O, float("nan"))
    lse = torch.full_like(plan.lse, float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    binding.cluster_attention_fwd_static(p, plan.Qp, plan.Kp, plan.Vp, plan.ck, plan.cv, plan.count_k,
                                         plan.block_idx, plan.perm_q, O, lse)
    torch.cuda.synchronize()
    taken = free_before - torch.cuda.mem_get_info()[0]      # device memory the call itself took
    assert binding.load_library().ca_static_last_status() == 0
    return O.float().cpu().numpy(), lse.cpu().numpy(), O_ref.float().cpu().numpy(), lse_ref.cpu().numpy(), taken


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    build.build()
    assert binding.static_scratch_bytes() == 32 << 20
    # first call: bf16 tensor-core path, 32 key clusters, compensation on
    first = prepared_plan("tabular", 2, 1024, 4096, 4, True)
    # second call: more key clusters than the first, different head count and keep (its
    # centroid copies overwrite, and extend beyond, what the first call left behind)
    second = prepared_plan("sweep", 3, 640, 6000, 7, True)
    # third: fp32 storage (FP32 kernel; only the status word of the scratch is used)
    third = prepared_plan("tiny", 2, 1024, 1024, 4, True)
    for n, (plan, tol) in enumerate(((first, 2e-2), (second, 2e-2), (first, 2e-2), (third, 1e-5))):
        O, lse, O_ref, lse_ref, taken = run_both(plan)
        assert np.isfinite(O).all() and np.isfinite(lse).all()
        assert np.abs(O - O_ref).max() <= tol
        assert np.abs(lse - lse_ref).max() <= tol
        # same kernels on the same inputs: the two entry points agree exactly
        assert np.array_equal(O, O_ref) and np.array_equal(lse, lse_ref)
        # once a first call in this process has looked the scratch array up (which may be what loads
        # the library's device code and reserves the array), a call takes no device memory
        if n > 0:
            assert taken == 0
        if n == 0:
            # and against the oracle: attention on the device's own clustering and block lists
            Q, K, V, w = plan.host_inputs
            c = w.cluster
            for h in range(plan.problem.heads):
                o_ref, lse_o = orc.cluster_attention(
                    Q[h], K[h], V[h], plan.perm_q[0, h].cpu().numpy(), plan.perm_k[0, h].cpu().numpy(), c, c,
                    plan.block_idx[0, h].cpu().numpy(), True, ck=plan.ck[0, h].cpu().numpy(),
                    cv=plan.cv[0, h].cpu().numpy(), count_k=plan.count_k[0, h].cpu().numpy())
                assert np.abs(O[0, h] - o_ref).max() <= 2e-2
                assert np.linalg.norm(O[0, h] - o_ref) <= 5e-3 * np.linalg.norm(o_ref)
                assert np.abs(lse[0, h] - lse_o).max() <= 2e-2


def test_static_scratch_entry_point_rejects_problems_beyond_its_fixed_size():
    build.build()
    lib = binding.load_library()
    # 64 heads x 1024 key clusters x d=128: 50 MB of centroid copies > 32 MiB
    p = binding.make_problem(1, 64, 131072, 131072, 128, "bf16", 128, 128, 128)
    assert binding.workspace_bytes(p)["attn"] > binding.static_scratch_bytes()
    dummy = torch.zeros(64, device=DEV)
    ptr = ctypes.c_void_p(dummy.data_ptr())
    rc = lib.cluster_attention_fwd_static(ctypes.byref(p), *([ptr] * 9), None, None)
    assert rc == 3      # CA_ERR_WORKSPACE, nothing enqueued
    torch.cuda.synchronize()

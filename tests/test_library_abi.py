"""CPU-side checks of the C boundary: the library builds, loads and exports
every symbol the public header declares; argument validation returns error
codes without touching a device."""
import ctypes
import os
import re

import pytest

from paper_2608_26965_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cluster_attention.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(?:int|void|const char\*|unsigned long long|size_t)\s+(\w+)\s*\(", text)))


def test_header_declarations_are_exported(lib):
    names = declared_functions()
    assert set(binding.EXPORTS) <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    assert b"sm_100a" in lib.ca_version()


def test_struct_layout_matches_header():
    assert ctypes.sizeof(binding.CaProblem) == 12 * 4


def test_workspace_query_and_validation(lib):
    p = binding.make_problem(1, 8, 16384, 131072, 64, "bf16", 128, 128, 128)
    sizes = binding.workspace_bytes(p)
    assert sizes["cluster"] > 8 * (16384 + 131072) * 4 and sizes["select"] >= 256 and sizes["attn"] >= 256
    bad = [p.copy(head_dim=96), p.copy(dtype=7), p.copy(cluster_k=100), p.copy(keep=0),
           p.copy(keep=1025), p.copy(n_q=0), p.copy(cluster_q=512)]
    for b in bad:
        rc = lib.ca_workspace_bytes(ctypes.byref(b), None, None, None)
        assert rc in (1, 2), rc
    # null data pointers are rejected before anything is enqueued
    rc = lib.cluster_qk(ctypes.byref(p), *([None] * 16), 0, None)
    assert rc == 1
    rc = lib.select_blocks(ctypes.byref(p), None, None, None, None, 0, None)
    assert rc == 1
    rc = lib.cluster_attention_fwd(ctypes.byref(p), *([None] * 11), 0, None)
    assert rc == 1


def test_binding_refuses_cpu_tensors(lib):
    import torch
    p = binding.make_problem(1, 1, 64, 64, 64, "fp32", 16, 16, 2)
    if torch.cuda.is_available():
        pytest.skip("CPU-only check")
    with pytest.raises(binding.ClusterAttnError):
        binding.Plan(p)

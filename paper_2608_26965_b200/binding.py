"""ctypes binding of libclusterattn.so: argument marshalling only.

The functions mirror the C entry points (`cluster_qk`, `select_blocks`,
`cluster_attention_fwd`).  torch provides device memory and streams; every
step of the computation runs inside the library's CUDA kernels.  There is no
CPU fallback: if the library is missing or no CUDA device is present the calls
raise.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Dict, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libclusterattn.so")

CA_OK = 0
CA_ERR_INVALID_ARG, CA_ERR_UNSUPPORTED, CA_ERR_WORKSPACE, CA_ERR_CUDA, CA_ERR_TIMEOUT = 1, 2, 3, 4, 5
CA_ERR_BAD_INDEX = 6
ERRORS = {1: "CA_ERR_INVALID_ARG", 2: "CA_ERR_UNSUPPORTED", 3: "CA_ERR_WORKSPACE", 4: "CA_ERR_CUDA",
          5: "CA_ERR_TIMEOUT", 6: "CA_ERR_BAD_INDEX"}
CA_DTYPE_FP32, CA_DTYPE_BF16 = 0, 1
CA_Y_IN, CA_ATTN_FP32, CA_QUERY_UNNORMALIZED, CA_METRIC_IN, CA_ATTN_FP8_QK = 1, 2, 4, 8, 16

EXPORTS = ("ca_workspace_bytes", "cluster_qk", "select_blocks", "cluster_attention_fwd",
           "ca_last_status", "ca_attn_recomputed", "ca_version", "ca_kernel_launches", "cluster_attention_fwd_static",
           "ca_static_scratch_bytes", "ca_static_last_status", "select_blocks_adaptive",
           "cluster_attention_fwd_ragged", "ca_basic_workspace_bytes", "cluster_qk_basic", "ca_debug_attn_wait", "ca_debug_eigh",
           "ca_profile", "ca_profile_read")


class CaProblem(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("n_q", ctypes.c_int32),
                ("n_k", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("cluster_q", ctypes.c_int32), ("cluster_k", ctypes.c_int32), ("keep", ctypes.c_int32),
                ("compensate", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("flags", ctypes.c_int32)]

    @property
    def n_qc(self) -> int:
        return -(-self.n_q // self.cluster_q)

    @property
    def n_kc(self) -> int:
        return -(-self.n_k // self.cluster_k)

    def copy(self, **kw) -> "CaProblem":
        vals = {f: getattr(self, f) for f, _ in self._fields_}
        vals.update(kw)
        return CaProblem(**vals)


class ClusterAttnError(RuntimeError):
    pass


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libclusterattn.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ClusterAttnError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_26965_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, sz = ctypes.c_void_p, ctypes.c_size_t
    pp = ctypes.POINTER(CaProblem)
    lib.ca_workspace_bytes.argtypes = [pp, ctypes.POINTER(sz), ctypes.POINTER(sz), ctypes.POINTER(sz)]
    lib.ca_workspace_bytes.restype = ctypes.c_int
    lib.cluster_qk.argtypes = [pp] + [vp] * 16 + [sz, vp]
    lib.cluster_qk.restype = ctypes.c_int
    lib.select_blocks.argtypes = [pp, vp, vp, vp, vp, sz, vp]
    lib.select_blocks.restype = ctypes.c_int
    lib.cluster_attention_fwd.argtypes = [pp] + [vp] * 11 + [sz, vp]
    lib.cluster_attention_fwd.restype = ctypes.c_int
    lib.select_blocks_adaptive.argtypes = [pp, vp, vp, vp, ctypes.c_float, ctypes.c_int32, vp, vp, vp, sz, vp]
    lib.select_blocks_adaptive.restype = ctypes.c_int
    lib.cluster_attention_fwd_ragged.argtypes = [pp] + [vp] * 8 + [ctypes.c_int32] + [vp] * 4 + [sz, vp]
    lib.cluster_attention_fwd_ragged.restype = ctypes.c_int
    lib.ca_basic_workspace_bytes.argtypes = [pp, ctypes.POINTER(sz), ctypes.POINTER(ctypes.c_int32),
                                             ctypes.POINTER(ctypes.c_int32)]
    lib.ca_basic_workspace_bytes.restype = ctypes.c_int
    lib.cluster_qk_basic.argtypes = [pp] + [vp] * 5 + [ctypes.c_int32] + [vp] * 13 + [sz, vp]
    lib.cluster_qk_basic.restype = ctypes.c_int
    lib.ca_last_status.argtypes = [vp]
    lib.ca_last_status.restype = ctypes.c_int
    lib.ca_attn_recomputed.argtypes = [vp]
    lib.ca_attn_recomputed.restype = ctypes.c_int
    lib.ca_version.argtypes = []
    lib.ca_version.restype = ctypes.c_char_p
    lib.ca_kernel_launches.argtypes = []
    lib.ca_kernel_launches.restype = ctypes.c_ulonglong
    lib.cluster_attention_fwd_static.argtypes = [pp] + [vp] * 10 + [vp]
    lib.cluster_attention_fwd_static.restype = ctypes.c_int
    lib.ca_static_scratch_bytes.argtypes = []
    lib.ca_static_scratch_bytes.restype = ctypes.c_size_t
    lib.ca_static_last_status.argtypes = []
    lib.ca_static_last_status.restype = ctypes.c_int
    lib.ca_debug_attn_wait.argtypes = [ctypes.c_longlong, ctypes.c_int]
    lib.ca_debug_attn_wait.restype = None
    lib.ca_debug_eigh.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                  ctypes.c_void_p]
    lib.ca_debug_eigh.restype = ctypes.c_int
    lib.ca_profile.argtypes = [ctypes.c_int]
    lib.ca_profile.restype = ctypes.c_int
    lib.ca_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float),
                                    ctypes.POINTER(ctypes.c_int)]
    lib.ca_profile_read.restype = ctypes.c_int
    _lib = lib
    return lib


def profile(enable: bool) -> None:
    """Switches the library's per-kernel-group timers on or off (ca_profile)."""
    _check(load_library().ca_profile(1 if enable else 0), "ca_profile")


def profile_read() -> Dict[str, Dict[str, float]]:
    """Device time in ms and number of timed scopes per kernel group since the timers were switched
    on or last read (ca_profile_read; synchronises the device)."""
    lib = load_library()
    n = 16
    names = (ctypes.c_char_p * n)()
    ms = (ctypes.c_float * n)()
    scopes = (ctypes.c_int * n)()
    got = lib.ca_profile_read(n, names, ms, scopes)
    if got < 0:
        _check(-got, "ca_profile_read")
    return {names[i].decode(): {"ms": float(ms[i]), "scopes": int(scopes[i])} for i in range(got)}


def kernel_launches() -> int:
    """Kernels the library has enqueued since it was loaded."""
    return int(load_library().ca_kernel_launches())


def _check(rc: int, what: str) -> None:
    if rc != CA_OK:
        raise ClusterAttnError(f"{what} failed: {ERRORS.get(rc, rc)}")


def _require_cuda(t: torch.Tensor, name: str) -> None:
    if not t.is_cuda:
        raise ClusterAttnError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if not t.is_contiguous():
        raise ClusterAttnError(f"{name} must be contiguous")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def torch_dtype(problem: CaProblem) -> torch.dtype:
    return torch.bfloat16 if problem.dtype == CA_DTYPE_BF16 else torch.float32


def make_problem(batch: int, heads: int, n_q: int, n_k: int, head_dim: int, dtype: str, cluster_q: int,
                 cluster_k: int, keep: int, compensate: bool = True, softmax_scale: float = 0.0,
                 flags: int = 0) -> CaProblem:
    code = {"fp32": CA_DTYPE_FP32, "bf16": CA_DTYPE_BF16}[dtype]
    return CaProblem(batch, heads, n_q, n_k, head_dim, code, cluster_q, cluster_k, keep,
                     1 if compensate else 0, float(softmax_scale), flags)


def problem_from_workload(w, heads: Optional[int] = None, **kw) -> CaProblem:
    args = dict(batch=1, heads=heads if heads is not None else w.heads, n_q=w.n_q, n_k=w.n_k,
                head_dim=w.head_dim, dtype=w.dtype, cluster_q=w.cluster, cluster_k=w.cluster, keep=w.keep,
                compensate=w.compensate)
    args.update(kw)
    return make_problem(**args)


def debug_eigh(A: torch.Tensor, stream=None):
    """ca_debug_eigh of the C library: A [count, d, d] float64 symmetric (CUDA).  Returns
    (W [count, d, d] float32 with eigenvector t in column t, evals [count, d] float64, descending)."""
    _require_cuda(A, "A")
    if A.dtype != torch.float64 or A.dim() != 3 or A.shape[1] != A.shape[2]:
        raise ClusterAttnError("A must be [count, d, d] float64")
    lib = load_library()
    count, d = int(A.shape[0]), int(A.shape[1])
    W = torch.empty((count, d, d), dtype=torch.float32, device=A.device)
    ev = torch.empty((count, d), dtype=torch.float64, device=A.device)
    _check(lib.ca_debug_eigh(_ptr(A), count, d, _ptr(W), _ptr(ev), _stream_ptr(stream)), "ca_debug_eigh")
    return W, ev


def workspace_bytes(problem: CaProblem) -> Dict[str, int]:
    lib = load_library()
    a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib.ca_workspace_bytes(ctypes.byref(problem), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
           "ca_workspace_bytes")
    return {"cluster": a.value, "select": b.value, "attn": c.value}


class Plan:
    """Device buffers for one problem shape: outputs of each stage and the
    workspaces the library asks for.  Holds memory only; all compute is in the
    library calls."""

    def __init__(self, problem: CaProblem, device: str = "cuda:0", keep_y: bool = False):
        if not torch.cuda.is_available():
            raise ClusterAttnError("no CUDA device: libclusterattn has no CPU path")
        load_library()
        self.problem = problem
        self.device = torch.device(device)
        p = problem
        dt = torch_dtype(p)
        B, H, D = p.batch, p.heads, p.head_dim
        dev = self.device
        i32, f32 = torch.int32, torch.float32
        self.perm_q = torch.empty((B, H, p.n_q), dtype=i32, device=dev)
        self.perm_k = torch.empty((B, H, p.n_k), dtype=i32, device=dev)
        self.Qp = torch.empty((B, H, p.n_qc * p.cluster_q, D), dtype=dt, device=dev)
        self.Kp = torch.empty((B, H, p.n_kc * p.cluster_k, D), dtype=dt, device=dev)
        self.Vp = torch.empty((B, H, p.n_kc * p.cluster_k, D), dtype=dt, device=dev)
        self.cq = torch.empty((B, H, p.n_qc, D), dtype=f32, device=dev)
        self.ck = torch.empty((B, H, p.n_kc, D), dtype=f32, device=dev)
        self.cv = torch.empty((B, H, p.n_kc, D), dtype=f32, device=dev)
        self.count_q = torch.empty((B, H, p.n_qc), dtype=i32, device=dev)
        self.count_k = torch.empty((B, H, p.n_kc), dtype=i32, device=dev)
        self.block_idx = torch.empty((B, H, p.n_qc, p.keep), dtype=i32, device=dev)
        self.block_idx_ragged = None
        self.keep_count = None
        self.O = torch.empty((B, H, p.n_q, D), dtype=dt, device=dev)
        self.lse = torch.empty((B, H, p.n_q), dtype=f32, device=dev)
        self.Yq = torch.empty((B, H, p.n_q, D), dtype=f32, device=dev) if keep_y else None
        self.Yk = torch.empty((B, H, p.n_k, D), dtype=f32, device=dev) if keep_y else None
        sizes = workspace_bytes(p)
        self.ws = {k: torch.zeros(max(v, 256), dtype=torch.uint8, device=dev) for k, v in sizes.items()}

    # -- the three entry points ------------------------------------------------
    def cluster_qk(self, Q, K, V, Yq=None, Yk=None, stream=None):
        """cluster_qk of the C library.  With Yq/Yk given and CA_Y_IN set in the
        problem's flags the split coordinates are taken from the caller."""
        p = self.problem
        for name, t in (("Q", Q), ("K", K), ("V", V)):
            _require_cuda(t, name)
        yq = Yq if Yq is not None else self.Yq
        yk = Yk if Yk is not None else self.Yk
        if p.flags & CA_Y_IN:
            _require_cuda(yq, "Yq")
            _require_cuda(yk, "Yk")
        lib = load_library()
        ws = self.ws["cluster"]
        rc = lib.cluster_qk(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(self.perm_q), _ptr(self.perm_k),
                            _ptr(self.Qp), _ptr(self.Kp), _ptr(self.Vp), _ptr(self.cq), _ptr(self.ck),
                            _ptr(self.cv), _ptr(self.count_q), _ptr(self.count_k), _ptr(yq), _ptr(yk),
                            _ptr(ws), ws.numel(), _stream_ptr(stream))
        _check(rc, "cluster_qk")
        return self

    def select_blocks(self, cq=None, ck=None, stream=None):
        lib = load_library()
        cq = self.cq if cq is None else cq
        ck = self.ck if ck is None else ck
        _require_cuda(cq, "cq")
        _require_cuda(ck, "ck")
        ws = self.ws["select"]
        rc = lib.select_blocks(ctypes.byref(self.problem), _ptr(cq), _ptr(ck), _ptr(self.block_idx), _ptr(ws),
                               ws.numel(), _stream_ptr(stream))
        _check(rc, "select_blocks")
        return self.block_idx

    def cluster_attention_fwd(self, Qp=None, Kp=None, Vp=None, ck=None, cv=None, count_k=None,
                              block_idx=None, perm_q=None, want_lse=True, stream=None):
        lib = load_library()
        args = [self.Qp if Qp is None else Qp, self.Kp if Kp is None else Kp, self.Vp if Vp is None else Vp,
                self.ck if ck is None else ck, self.cv if cv is None else cv,
                self.count_k if count_k is None else count_k,
                self.block_idx if block_idx is None else block_idx,
                self.perm_q if perm_q is None else perm_q]
        for i, t in enumerate(args):
            _require_cuda(t, f"arg{i}")
        ws = self.ws["attn"]
        rc = lib.cluster_attention_fwd(ctypes.byref(self.problem), *[_ptr(t) for t in args], _ptr(self.O),
                                       _ptr(self.lse if want_lse else None), _ptr(ws), ws.numel(),
                                       _stream_ptr(stream))
        _check(rc, "cluster_attention_fwd")
        return self.O, (self.lse if want_lse else None)

    def basic_noise_rows(self):
        """Rows of normal deviates per head that cluster_qk_basic reads (queries, keys)."""
        lib = load_library()
        b, rq, rk = ctypes.c_size_t(), ctypes.c_int32(), ctypes.c_int32()
        _check(lib.ca_basic_workspace_bytes(ctypes.byref(self.problem), ctypes.byref(b), ctypes.byref(rq),
                                            ctypes.byref(rk)), "ca_basic_workspace_bytes")
        return rq.value, rk.value, b.value

    def cluster_qk_basic(self, Q, K, V, noise_q, noise_k, iterations: int = 3, A_q=None, A_k=None, stream=None):
        """cluster_qk_basic of the C library: basic recursive splitting with the metric injected into
        the power iteration.  noise_q/noise_k: normal deviates [B,H,rows,d] (rows from basic_noise_rows).
        A_q/A_k are inputs when the problem has CA_METRIC_IN, otherwise they are written."""
        lib = load_library()
        p = self.problem
        for name, t in (("Q", Q), ("K", K), ("V", V), ("noise_q", noise_q), ("noise_k", noise_k)):
            _require_cuda(t, name)
        rq, rk, nbytes = self.basic_noise_rows()
        if tuple(noise_q.shape[-2:]) != (rq, p.head_dim) or tuple(noise_k.shape[-2:]) != (rk, p.head_dim):
            raise ClusterAttnError(f"noise must be [B,H,{rq},{p.head_dim}] and [B,H,{rk},{p.head_dim}]")
        if p.flags & CA_METRIC_IN and (A_q is None or A_k is None):
            raise ClusterAttnError("CA_METRIC_IN needs A_q and A_k")
        shape = (p.batch, p.heads, p.head_dim, p.head_dim)
        self.A_q = A_q if A_q is not None else torch.empty(shape, dtype=torch.float32, device=self.device)
        self.A_k = A_k if A_k is not None else torch.empty(shape, dtype=torch.float32, device=self.device)
        if self.ws.get("basic") is None or self.ws["basic"].numel() < nbytes:
            self.ws["basic"] = torch.zeros(max(nbytes, 256), dtype=torch.uint8, device=self.device)
        ws = self.ws["basic"]
        rc = lib.cluster_qk_basic(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(noise_q), _ptr(noise_k),
                                  int(iterations), _ptr(self.A_q), _ptr(self.A_k), _ptr(self.perm_q),
                                  _ptr(self.perm_k), _ptr(self.Qp), _ptr(self.Kp), _ptr(self.Vp), _ptr(self.cq),
                                  _ptr(self.ck), _ptr(self.cv), _ptr(self.count_q), _ptr(self.count_k), _ptr(ws),
                                  ws.numel(), _stream_ptr(stream))
        _check(rc, "cluster_qk_basic")
        return self

    def select_blocks_adaptive(self, recall: float, min_count: int = 16, cq=None, ck=None, count_k=None,
                               stream=None):
        """Adaptive assignment: returns (block_idx [B,H,n_qc,n_kc] padded with -1, keep_count [B,H,n_qc])."""
        lib = load_library()
        cq = self.cq if cq is None else cq
        ck = self.ck if ck is None else ck
        count_k = self.count_k if count_k is None else count_k
        for name, t in (("cq", cq), ("ck", ck), ("count_k", count_k)):
            _require_cuda(t, name)
        pr = self.problem
        if getattr(self, "block_idx_ragged", None) is None:
            self.block_idx_ragged = torch.empty((pr.batch, pr.heads, pr.n_qc, pr.n_kc), dtype=torch.int32,
                                                device=self.device)
            self.keep_count = torch.empty((pr.batch, pr.heads, pr.n_qc), dtype=torch.int32, device=self.device)
        ws = self.ws["select"]
        rc = lib.select_blocks_adaptive(ctypes.byref(pr), _ptr(cq), _ptr(ck), _ptr(count_k), float(recall),
                                        int(min_count), _ptr(self.block_idx_ragged), _ptr(self.keep_count),
                                        _ptr(ws), ws.numel(), _stream_ptr(stream))
        _check(rc, "select_blocks_adaptive")
        return self.block_idx_ragged, self.keep_count

    def cluster_attention_fwd_ragged(self, block_idx=None, keep_count=None, Qp=None, Kp=None, Vp=None, ck=None,
                                     cv=None, count_k=None, perm_q=None, want_lse=True, stream=None):
        lib = load_library()
        block_idx = self.block_idx_ragged if block_idx is None else block_idx
        keep_count = self.keep_count if keep_count is None else keep_count
        args = [self.Qp if Qp is None else Qp, self.Kp if Kp is None else Kp, self.Vp if Vp is None else Vp,
                self.ck if ck is None else ck, self.cv if cv is None else cv,
                self.count_k if count_k is None else count_k, block_idx, keep_count]
        perm_q = self.perm_q if perm_q is None else perm_q
        for i, t in enumerate(args + [perm_q]):
            _require_cuda(t, f"arg{i}")
        ws = self.ws["attn"]
        rc = lib.cluster_attention_fwd_ragged(ctypes.byref(self.problem), *[_ptr(t) for t in args],
                                              int(block_idx.shape[-1]), _ptr(perm_q), _ptr(self.O),
                                              _ptr(self.lse if want_lse else None), _ptr(ws), ws.numel(),
                                              _stream_ptr(stream))
        _check(rc, "cluster_attention_fwd_ragged")
        return self.O, (self.lse if want_lse else None)

    def forward_adaptive(self, Q, K, V, recall: float, min_count: int = 16, want_lse=False, stream=None):
        self.cluster_qk(Q, K, V, stream=stream)
        self.select_blocks_adaptive(recall, min_count, stream=stream)
        return self.cluster_attention_fwd_ragged(want_lse=want_lse, stream=stream)

    def forward(self, Q, K, V, want_lse=False, stream=None):
        """The whole hot path: clustering, block selection, attention."""
        self.cluster_qk(Q, K, V, stream=stream)
        self.select_blocks(stream=stream)
        return self.cluster_attention_fwd(want_lse=want_lse, stream=stream)[0]

    def last_status(self) -> Dict[str, int]:
        lib = load_library()
        return {k: lib.ca_last_status(_ptr(v)) for k, v in self.ws.items()}

    def recomputed_clusters(self) -> int:
        """Query clusters that the second pass of the attention calls on this plan has recomputed
        with the fp32 kernel, summed over all calls since the plan was made (ca_attn_recomputed)."""
        lib = load_library()
        n = lib.ca_attn_recomputed(_ptr(self.ws["attn"]))
        if n < 0:
            _check(-n, "ca_attn_recomputed")
        return n


# -- functional forms with the C names ------------------------------------------
def cluster_qk(problem: CaProblem, Q, K, V, Yq=None, Yk=None, plan: Optional[Plan] = None) -> Plan:
    plan = plan or Plan(problem, device=str(Q.device), keep_y=Yq is None)
    return plan.cluster_qk(Q, K, V, Yq=Yq, Yk=Yk)


def select_blocks(problem: CaProblem, cq, ck, plan: Optional[Plan] = None):
    plan = plan or Plan(problem, device=str(cq.device))
    return plan.select_blocks(cq, ck)


def cluster_attention_fwd(problem: CaProblem, Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q,
                          plan: Optional[Plan] = None):
    plan = plan or Plan(problem, device=str(Qp.device))
    if tuple(block_idx.shape[-2:]) != (problem.n_qc, problem.keep):
        raise ClusterAttnError("block_idx must be [B,H,n_qc,keep]")
    return plan.cluster_attention_fwd(Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q)


def select_blocks_adaptive(problem: CaProblem, cq, ck, count_k, recall: float, min_count: int = 16,
                           plan: Optional[Plan] = None):
    plan = plan or Plan(problem, device=str(cq.device))
    return plan.select_blocks_adaptive(recall, min_count, cq, ck, count_k)


def cluster_attention_fwd_ragged(problem: CaProblem, Qp, Kp, Vp, ck, cv, count_k, block_idx, keep_count, perm_q,
                                 plan: Optional[Plan] = None):
    plan = plan or Plan(problem, device=str(Qp.device))
    return plan.cluster_attention_fwd_ragged(block_idx, keep_count, Qp, Kp, Vp, ck, cv, count_k, perm_q)


def cluster_attention_fwd_static(problem: CaProblem, Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q, O,
                                 lse=None, stream=None):
    """The attention stage for callers that cannot allocate device memory (no
    workspace argument: the library's fixed 32 MiB scratch array is used).  The
    caller passes every input and the output tensors; nothing is allocated here
    either.  Calls on one device share the scratch and must not overlap."""
    lib = load_library()
    args = [Qp, Kp, Vp, ck, cv, count_k, block_idx, perm_q, O]
    for i, t in enumerate(args):
        _require_cuda(t, f"arg{i}")
    rc = lib.cluster_attention_fwd_static(ctypes.byref(problem), *[_ptr(t) for t in args], _ptr(lse),
                                          _stream_ptr(stream))
    _check(rc, "cluster_attention_fwd_static")
    return O, lse


def static_scratch_bytes() -> int:
    return int(load_library().ca_static_scratch_bytes())


def default_scale(problem: CaProblem) -> float:
    return problem.softmax_scale if problem.softmax_scale > 0 else 1.0 / math.sqrt(problem.head_dim)

"""Thin ctypes binding of the C-ABI library (`include/branch_attn.h`).

Argument marshalling only: torch provides device memory and streams, every
step of the computation runs in the library's CUDA kernels.  Importing this
module fails loudly if the compiled library is missing -- there is no CPU or
framework fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

BA_BF16, BA_FP32 = 0, 1
PART_MAIN, PART_BRANCH, PART_ALL = 1, 2, 3
OP_FWD, OP_BWD, OP_BWD_FUSED, OP_BWD_DEPTH = 0, 1, 2, 3
STAGE_PREP, STAGE_DQ, STAGE_DKDV, STAGE_ALL = 1, 2, 4, 7
STAGE_FUSED, STAGE_ALL_FUSED = 8, 9
IMPL_AUTO, IMPL_SIMT, IMPL_TC = 0, 1, 2

_DT = {"bf16": (BA_BF16, torch.bfloat16), "fp32": (BA_FP32, torch.float32)}


class BranchAttnError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {_lib().ba_status_string(code).decode()} (status {code}, "
                         f"cuda error {_lib().ba_last_cuda_error()})")


class _Problem(C.Structure):
    _fields_ = [
        ("n_main", C.c_int64), ("n_branch", C.c_int64),
        ("num_seqs", C.c_int32), ("num_branches", C.c_int32),
        ("h_q", C.c_int32), ("h_kv", C.c_int32), ("head_dim", C.c_int32),
        ("dtype", C.c_int32), ("softmax_scale", C.c_float),
        ("mask_kind", C.c_int32), ("uniform_len", C.c_int32), ("impl", C.c_int32),
        ("cu_seqlens", C.c_void_p), ("anchor_idx", C.c_void_p),
        ("branch_offsets", C.c_void_p), ("parent", C.c_void_p),
    ]


_LIB = None
EXPORTS = ("ba_status_string", "ba_last_cuda_error", "ba_plan_bytes", "ba_plan_create",
           "ba_plan_destroy", "ba_workspace_bytes", "ba_plan_pairs", "ba_plan_impl", "ba_plan_check", "branch_attn_fwd",
           "branch_attn_fwd_partial", "branch_attn_fwd_partial_merge", "lse_merge", "branch_attn_bwd", "branch_attn_bwd_stages",
           "branch_attn_bwd_static", "ba_finalize_grads", "ba_selftest_bounded_wait",
           "branch_attn_fwd_depth", "branch_attn_bwd_depth", "branch_attn_fwd_shard", "branch_attn_bwd_shard")


def _lib():
    global _LIB
    if _LIB is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise ImportError(f"{path} is missing: build it with "
                              "`python -m paper_2609_07108_b200.build` (needs nvcc); "
                              "there is no fallback path")
        lib = C.CDLL(path)
        lib.ba_status_string.restype = C.c_char_p
        lib.ba_status_string.argtypes = [C.c_int]
        lib.ba_last_cuda_error.restype = C.c_int
        lib.ba_plan_bytes.restype = C.c_size_t
        lib.ba_plan_bytes.argtypes = [C.POINTER(_Problem)]
        lib.ba_plan_create.restype = C.c_int
        lib.ba_plan_create.argtypes = [C.POINTER(_Problem), C.c_void_p, C.c_size_t, C.c_void_p,
                                       C.POINTER(C.c_void_p)]
        lib.ba_plan_destroy.restype = C.c_int
        lib.ba_plan_destroy.argtypes = [C.c_void_p]
        lib.ba_workspace_bytes.restype = C.c_size_t
        lib.ba_workspace_bytes.argtypes = [C.c_void_p, C.c_int]
        lib.ba_plan_pairs.restype = C.c_int64
        lib.ba_plan_pairs.argtypes = [C.c_void_p]
        lib.ba_plan_impl.restype = C.c_int
        lib.ba_plan_impl.argtypes = [C.c_void_p]
        lib.ba_plan_check.restype = C.c_int
        lib.ba_plan_check.argtypes = [C.c_void_p, C.c_void_p]
        vp, i64 = C.c_void_p, C.c_int64
        lib.branch_attn_fwd.restype = C.c_int
        lib.branch_attn_fwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp]
        lib.branch_attn_fwd_partial.restype = C.c_int
        lib.branch_attn_fwd_partial.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64,
                                                C.c_int, vp, vp, vp, C.c_size_t, vp]
        lib.branch_attn_fwd_partial_merge.restype = C.c_int
        lib.branch_attn_fwd_partial_merge.argtypes = lib.branch_attn_fwd_partial.argtypes
        lib.lse_merge.restype = C.c_int
        lib.lse_merge.argtypes = [i64, C.c_int, vp, vp, vp, vp, vp, C.c_int, vp, vp]
        lib.branch_attn_bwd.restype = C.c_int
        lib.branch_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64,
                                        C.c_int, C.c_int, vp, vp, vp, vp, vp, C.c_size_t, vp]
        lib.branch_attn_bwd_stages.restype = C.c_int
        lib.branch_attn_bwd_stages.argtypes = lib.branch_attn_bwd.argtypes + [C.c_int]
        lib.branch_attn_bwd_static.restype = C.c_int
        lib.branch_attn_bwd_static.argtypes = lib.branch_attn_bwd.argtypes[:-3] + [vp]
        lib.ba_finalize_grads.restype = C.c_int
        lib.ba_finalize_grads.argtypes = [vp, vp, i64, C.c_int, vp]
        lib.branch_attn_fwd_depth.restype = C.c_int
        lib.branch_attn_fwd_depth.argtypes = [vp, C.c_int, vp, vp, vp, i64, i64, vp, vp, vp]
        lib.branch_attn_bwd_depth.restype = C.c_int
        lib.branch_attn_bwd_depth.argtypes = [vp, C.c_int, vp, vp, vp, vp, vp, vp, i64, i64, vp, vp, vp, vp,
                                              C.c_size_t, vp]
        lib.branch_attn_fwd_shard.restype = C.c_int
        lib.branch_attn_fwd_shard.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64, C.c_int, vp, vp, vp]
        lib.branch_attn_bwd_shard.restype = C.c_int
        lib.branch_attn_bwd_shard.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i64,
                                              vp, vp, vp, vp, vp, C.c_size_t, vp, C.c_int]
        lib.ba_selftest_bounded_wait.restype = C.c_int
        lib.ba_selftest_bounded_wait.argtypes = [vp, i64, vp]
        _LIB = lib
    return _LIB


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _expect(name, t, shape, dtype, device, optional=False):
    """A tensor handed to the library must be exactly what the kernels and tensor
    maps assume: on the plan's device, contiguous, of the stated dtype and shape.
    (The library sees only a raw pointer; a strided view or a wrong dtype would
    make it read or write outside the allocation.)"""
    if t is None:
        if optional:
            return
        raise ValueError(f"{name}: tensor required")
    if not t.is_cuda or (device is not None and t.device != device):
        raise ValueError(f"{name}: on {t.device}, expected {device}")
    if t.dtype != dtype:
        raise ValueError(f"{name}: dtype {t.dtype}, expected {dtype}")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: shape {tuple(t.shape)}, expected {tuple(shape)}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: not contiguous")


def _expect_inputs(plan, q_main, q_branch, k, v, q_main_optional=True):
    p, dt, dev = plan.problem, plan.torch_dtype, plan.device
    _expect("q_main", q_main, (p.n_main, p.h_q, p.head_dim), dt, dev, optional=q_main_optional)
    _expect("q_branch", q_branch, (p.n_branch, p.h_q, p.head_dim), dt, dev, optional=p.n_branch == 0)
    _expect("k", k, (p.rows, p.h_kv, p.head_dim), dt, dev)
    _expect("v", v, (p.rows, p.h_kv, p.head_dim), dt, dev)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, what):
    if rc != 0:
        raise BranchAttnError(rc, what)


def _dev_i32(a, device):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(device)


class Plan:
    """ba_plan_create: metadata builder for one packed batch.

    `problem` is a `workloads.Problem` (host numpy metadata); the arrays are
    copied to the device, validated and expanded there.
    """

    def __init__(self, problem, device="cuda", impl=IMPL_AUTO):
        lib = _lib()
        self.problem = problem
        self.device = torch.device(device)
        if self.device.type == "cuda" and self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self.dtype_code, self.torch_dtype = _DT[problem.dtype]
        offs = np.asarray(problem.branch_offsets, dtype=np.int64)
        lens = np.diff(offs)
        uniform = int(lens[0]) if len(lens) and lens[0] > 0 and (lens == lens[0]).all() else 0
        self._cu = _dev_i32(problem.cu_seqlens, self.device)
        self._anchor = _dev_i32(problem.anchor_idx, self.device)
        self._offs = _dev_i32(offs, self.device)
        self._parent = _dev_i32(problem.parent, self.device) if problem.parent is not None else None
        self.c = _Problem(problem.n_main, problem.n_branch, problem.num_seqs, problem.num_branches,
                          problem.h_q, problem.h_kv, problem.head_dim, self.dtype_code,
                          float(problem.scale), int(problem.kind), uniform, impl,
                          self._cu.data_ptr(), self._anchor.data_ptr() if len(self._anchor) else None,
                          self._offs.data_ptr() if problem.num_branches else None,   # A = 0: no branch arrays
                          self._parent.data_ptr() if self._parent is not None and len(self._parent) else None)
        nbytes = lib.ba_plan_bytes(C.byref(self.c))
        if nbytes == 0:
            raise BranchAttnError(-2, "ba_plan_bytes")
        self._mem = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        handle = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = lib.ba_plan_create(C.byref(self.c), _p(self._mem), nbytes, _stream(), C.byref(handle))
        _check(rc, "ba_plan_create")
        self.handle = handle
        self.pairs = int(lib.ba_plan_pairs(handle))
        self.impl = int(lib.ba_plan_impl(handle))
        self._ws = {}

    def workspace(self, op):
        if op not in self._ws:
            n = _lib().ba_workspace_bytes(self.handle, op)
            self._ws[op] = torch.empty(max(n, 256), dtype=torch.uint8, device=self.device)
        return self._ws[op]

    def check(self):
        """Synchronise and raise if a kernel of this plan gave up a bounded wait."""
        _check(_lib().ba_plan_check(self.handle, _stream()), "ba_plan_check")

    def selftest_bounded_wait(self, limit_cycles=100000):
        """Launch the probe whose wait runs out; the next `check()` raises BA_ETIMEOUT."""
        _check(_lib().ba_selftest_bounded_wait(self.handle, limit_cycles, _stream()), "ba_selftest_bounded_wait")

    def close(self):
        if getattr(self, "handle", None):
            _lib().ba_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # sizes
    @property
    def n(self):
        return self.problem.n_main

    @property
    def m(self):
        return self.problem.n_branch

    def token_range(self, br_begin, br_end):
        o = self.problem.branch_offsets
        return int(o[br_begin]), int(o[br_end])


def branch_attn_fwd(plan, q_main, q_branch, k, v, out=None, lse=None):
    """(O [N+M, h_q, D] input dtype, LSE [N+M, h_q] fp32); q_main may be None."""
    p = plan.problem
    if out is None:
        out = torch.empty((p.rows, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=plan.device)
    if lse is None:
        lse = torch.empty((p.rows, p.h_q), dtype=torch.float32, device=plan.device)
    _expect_inputs(plan, q_main, q_branch, k, v)
    _expect("out", out, (p.rows, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("lse", lse, (p.rows, p.h_q), torch.float32, plan.device)
    ws = plan.workspace(OP_FWD)
    rc = _lib().branch_attn_fwd(plan.handle, _p(q_main), _p(q_branch), _p(k), _p(v), _p(out), _p(lse),
                                _p(ws), ws.numel(), _stream())
    _check(rc, "branch_attn_fwd")
    return out, lse


def branch_attn_fwd_partial(plan, q_main, q_branch, k, v, qm_range, br_range, kv_range, parts,
                            out=None, lse=None):
    """Compact fp32 (O_part, LSE_part) of the selected queries over the selected key set."""
    p = plan.problem
    t0, t1 = plan.token_range(*br_range)
    rows = (qm_range[1] - qm_range[0]) + (t1 - t0)
    if out is None:
        out = torch.empty((rows, p.h_q, p.head_dim), dtype=torch.float32, device=plan.device)
    if lse is None:
        lse = torch.empty((rows, p.h_q), dtype=torch.float32, device=plan.device)
    _expect_inputs(plan, q_main, q_branch, k, v)
    _expect("out", out, (rows, p.h_q, p.head_dim), torch.float32, plan.device)
    _expect("lse", lse, (rows, p.h_q), torch.float32, plan.device)
    ws = plan.workspace(OP_FWD)
    rc = _lib().branch_attn_fwd_partial(plan.handle, _p(q_main), _p(q_branch), _p(k), _p(v),
                                        qm_range[0], qm_range[1], br_range[0], br_range[1],
                                        kv_range[0], kv_range[1], parts, _p(out), _p(lse),
                                        _p(ws), ws.numel(), _stream())
    _check(rc, "branch_attn_fwd_partial")
    return out, lse


def branch_attn_fwd_partial_merge(plan, q_main, q_branch, k, v, qm_range, br_range, kv_range, parts, acc_o, acc_lse):
    """Partial forward whose epilogue merges into the compact fp32 (acc_o, acc_lse) in place."""
    p = plan.problem
    t0, t1 = plan.token_range(*br_range)
    rows = (qm_range[1] - qm_range[0]) + (t1 - t0)
    _expect_inputs(plan, q_main, q_branch, k, v)
    _expect("acc_o", acc_o, (rows, p.h_q, p.head_dim), torch.float32, plan.device)
    _expect("acc_lse", acc_lse, (rows, p.h_q), torch.float32, plan.device)
    ws = plan.workspace(OP_FWD)
    rc = _lib().branch_attn_fwd_partial_merge(plan.handle, _p(q_main), _p(q_branch), _p(k), _p(v),
                                              qm_range[0], qm_range[1], br_range[0], br_range[1],
                                              kv_range[0], kv_range[1], parts, _p(acc_o), _p(acc_lse),
                                              _p(ws), ws.numel(), _stream())
    _check(rc, "branch_attn_fwd_partial_merge")
    return acc_o, acc_lse


def lse_merge(o_a, lse_a, o_b, lse_b, out=None, lse_out=None, out_dtype=torch.float32):
    """Eq. (lse-merge); `out` may be `o_a` (fp32, in place)."""
    d = o_a.shape[-1]
    items = lse_a.numel()
    if out is None:
        out = torch.empty(o_a.shape, dtype=out_dtype, device=o_a.device)
    if lse_out is None:
        lse_out = torch.empty_like(lse_a)
    dev = o_a.device
    _expect("o_a", o_a, None, torch.float32, dev)
    _expect("o_b", o_b, o_a.shape, torch.float32, dev)
    _expect("lse_a", lse_a, o_a.shape[:-1], torch.float32, dev)
    _expect("lse_b", lse_b, o_a.shape[:-1], torch.float32, dev)
    _expect("out", out, o_a.shape, out.dtype, dev)
    _expect("lse_out", lse_out, o_a.shape[:-1], torch.float32, dev)
    if out.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"out: dtype {out.dtype} not supported")
    code = BA_BF16 if out.dtype == torch.bfloat16 else BA_FP32
    rc = _lib().lse_merge(items, d, _p(o_a), _p(lse_a), _p(o_b), _p(lse_b), _p(out), code,
                          _p(lse_out), _stream())
    _check(rc, "lse_merge")
    return out, lse_out


def _expect_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, accumulate, grads):
    p, dt, dev = plan.problem, plan.torch_dtype, plan.device
    _expect_inputs(plan, q_main, q_branch, k, v)
    _expect("o", o, (p.rows, p.h_q, p.head_dim), dt, dev)
    _expect("lse", lse, (p.rows, p.h_q), torch.float32, dev)
    _expect("d_o", d_o, (p.rows, p.h_q, p.head_dim), dt, dev)
    gdt = torch.float32 if accumulate else dt
    _expect("dQ_main", grads[0], (p.n_main, p.h_q, p.head_dim), gdt, dev, optional=q_main is None)
    _expect("dQ_branch", grads[1], (p.n_branch, p.h_q, p.head_dim), gdt, dev, optional=p.n_branch == 0)
    _expect("dK", grads[2], (p.rows, p.h_kv, p.head_dim), gdt, dev)
    _expect("dV", grads[3], (p.rows, p.h_kv, p.head_dim), gdt, dev)


def branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, qm_range=None, br_range=None,
                    kv_range=None, parts=PART_ALL, accumulate=False, grads=None, stages=STAGE_ALL,
                    fused_scratch=False):
    """(dQ_main, dQ_branch, dK, dV).  With `accumulate`, `grads` must hold four
    zero-initialised fp32 tensors which receive the selected terms.  `fused_scratch`:
    this call prepares (STAGE_PREP) a backward whose STAGE_FUSED call follows
    separately with accumulate=False."""
    p = plan.problem
    qm_range = (0, p.n_main) if qm_range is None else qm_range
    br_range = (0, p.num_branches) if br_range is None else br_range
    kv_range = (0, p.n_main) if kv_range is None else kv_range
    if grads is None:
        dt = torch.float32 if accumulate else plan.torch_dtype
        mk = torch.zeros if accumulate else torch.empty
        grads = (mk((p.n_main, p.h_q, p.head_dim), dtype=dt, device=plan.device)
                 if q_main is not None else None,
                 mk((p.n_branch, p.h_q, p.head_dim), dtype=dt, device=plan.device),
                 mk((p.rows, p.h_kv, p.head_dim), dtype=dt, device=plan.device),
                 mk((p.rows, p.h_kv, p.head_dim), dtype=dt, device=plan.device))
    _expect_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, accumulate, grads)
    # every stage of one backward must see the same workspace: once a plan has been
    # used for the one-kernel backward with gradients in the input dtype (which keeps
    # an fp32 dQ accumulator in the workspace), all its backward calls use that buffer
    if fused_scratch or ((stages & STAGE_FUSED) and not accumulate):
        plan._fused_ws = True
    ws = plan.workspace(OP_BWD_FUSED if getattr(plan, "_fused_ws", False) else OP_BWD)
    args = (plan.handle, _p(q_main), _p(q_branch), _p(k), _p(v), _p(o), _p(lse),
            _p(d_o), qm_range[0], qm_range[1], br_range[0], br_range[1],
            kv_range[0], kv_range[1], parts, 1 if accumulate else 0,
            _p(grads[0]), _p(grads[1]), _p(grads[2]), _p(grads[3]), _p(ws), ws.numel(), _stream())
    if stages == STAGE_ALL:
        rc = _lib().branch_attn_bwd(*args)
    else:
        rc = _lib().branch_attn_bwd_stages(*args, stages)
    _check(rc, "branch_attn_bwd")
    return grads


STATIC_SCRATCH_BYTES = 8 << 20


def branch_attn_bwd_static(plan, q_main, q_branch, k, v, o, lse, d_o, qm_range=None, br_range=None,
                           kv_range=None, parts=PART_ALL, accumulate=False, grads=None):
    """branch_attn_bwd for callers that cannot allocate device scratch at call
    time: the library's built-in 8 MiB array serves as workspace (problems whose
    backward scratch is larger raise BA_EWORKSPACE).  `grads` must be given: this
    wrapper allocates nothing either.  Calls that may overlap on the GPU must be
    serialised by the caller, they share the one array."""
    p = plan.problem
    qm_range = (0, p.n_main) if qm_range is None else qm_range
    br_range = (0, p.num_branches) if br_range is None else br_range
    kv_range = (0, p.n_main) if kv_range is None else kv_range
    if grads is None:
        raise ValueError("branch_attn_bwd_static writes into caller-provided gradient tensors")
    _expect_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, accumulate, grads)
    rc = _lib().branch_attn_bwd_static(plan.handle, _p(q_main), _p(q_branch), _p(k), _p(v), _p(o), _p(lse),
                                       _p(d_o), qm_range[0], qm_range[1], br_range[0], br_range[1],
                                       kv_range[0], kv_range[1], parts, 1 if accumulate else 0,
                                       _p(grads[0]), _p(grads[1]), _p(grads[2]), _p(grads[3]), _stream())
    _check(rc, "branch_attn_bwd_static")
    return grads


def ba_finalize_grads(src, dst=None, dtype=torch.bfloat16):
    if dst is None:
        dst = torch.empty(src.shape, dtype=dtype, device=src.device)
    _expect("src", src, None, torch.float32, src.device)
    _expect("dst", dst, src.shape, dst.dtype, src.device)
    if dst.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"dst: dtype {dst.dtype} not supported")
    code = BA_BF16 if dst.dtype == torch.bfloat16 else BA_FP32
    rc = _lib().ba_finalize_grads(_p(src), _p(dst), src.numel(), code, _stream())
    _check(rc, "ba_finalize_grads")
    return dst


# ---------------------------------------------------------------- step-major (per-depth) calls

def _expect_depth(plan, q_depth, k, v):
    p, dt, dev = plan.problem, plan.torch_dtype, plan.device
    a = p.num_branches
    _expect("q_depth", q_depth, (a, p.h_q, p.head_dim), dt, dev)
    _expect("k", k, (p.rows, p.h_kv, p.head_dim), dt, dev)
    _expect("v", v, (p.rows, p.h_kv, p.head_dim), dt, dev)


def branch_attn_fwd_depth(plan, depth, q_depth, k, v, br_range=None, out=None, lse=None):
    """Forward of the depth-`depth` tokens (one per branch) against the main prefix and the
    tokens of depths <= depth of the own branch; k, v hold the branch tokens depth-major.
    Returns (O_depth [A, h_q, D], LSE_depth [A, h_q])."""
    p = plan.problem
    a = p.num_branches
    br_range = (0, a) if br_range is None else br_range
    if out is None:
        out = torch.empty((a, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=plan.device)
    if lse is None:
        lse = torch.empty((a, p.h_q), dtype=torch.float32, device=plan.device)
    _expect_depth(plan, q_depth, k, v)
    _expect("out", out, (a, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("lse", lse, (a, p.h_q), torch.float32, plan.device)
    rc = _lib().branch_attn_fwd_depth(plan.handle, depth, _p(q_depth), _p(k), _p(v), br_range[0], br_range[1],
                                      _p(out), _p(lse), _stream())
    _check(rc, "branch_attn_fwd_depth")
    return out, lse


def branch_attn_bwd_depth(plan, depth, q_depth, k, v, o_depth, lse_depth, d_o_depth, dk, dv, br_range=None, dq=None):
    """Backward of one depth: dQ_depth (input dtype) is returned, the terms of dK / dV
    (fp32, depth-major like k, v) are added to `dk`, `dv`."""
    p = plan.problem
    a = p.num_branches
    br_range = (0, a) if br_range is None else br_range
    if dq is None:
        dq = torch.empty((a, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=plan.device)
    _expect_depth(plan, q_depth, k, v)
    _expect("o_depth", o_depth, (a, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("lse_depth", lse_depth, (a, p.h_q), torch.float32, plan.device)
    _expect("d_o_depth", d_o_depth, (a, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("dq", dq, (a, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("dk", dk, (p.rows, p.h_kv, p.head_dim), torch.float32, plan.device)
    _expect("dv", dv, (p.rows, p.h_kv, p.head_dim), torch.float32, plan.device)
    ws = plan.workspace(OP_BWD_DEPTH)
    rc = _lib().branch_attn_bwd_depth(plan.handle, depth, _p(q_depth), _p(k), _p(v), _p(o_depth), _p(lse_depth),
                                      _p(d_o_depth), br_range[0], br_range[1], _p(dq), _p(dk), _p(dv),
                                      _p(ws), ws.numel(), _stream())
    _check(rc, "branch_attn_bwd_depth")
    return dq


# ---------------------------------------------------------------- ring steps on a received K/V shard

def _expect_shard(plan, q_main, q_branch, k_shard, v_shard, kv_range):
    p, dt, dev = plan.problem, plan.torch_dtype, plan.device
    rows = kv_range[1] - kv_range[0]
    _expect("q_main", q_main, (p.n_main, p.h_q, p.head_dim), dt, dev, optional=True)
    _expect("q_branch", q_branch, (p.n_branch, p.h_q, p.head_dim), dt, dev, optional=p.n_branch == 0)
    _expect("k_shard", k_shard, (rows, p.h_kv, p.head_dim), dt, dev)
    _expect("v_shard", v_shard, (rows, p.h_kv, p.head_dim), dt, dev)


def branch_attn_fwd_shard(plan, q_main, q_branch, k_shard, v_shard, qm_range, br_range, kv_range, acc_o, acc_lse,
                          merge):
    """Partial forward over the main keys [kv_range) held in (k_shard, v_shard) only;
    writes (merge=False) or merges into (merge=True) the compact fp32 (acc_o, acc_lse)."""
    p = plan.problem
    t0, t1 = plan.token_range(*br_range)
    rows = (qm_range[1] - qm_range[0]) + (t1 - t0)
    _expect_shard(plan, q_main, q_branch, k_shard, v_shard, kv_range)
    _expect("acc_o", acc_o, (rows, p.h_q, p.head_dim), torch.float32, plan.device)
    _expect("acc_lse", acc_lse, (rows, p.h_q), torch.float32, plan.device)
    rc = _lib().branch_attn_fwd_shard(plan.handle, _p(q_main), _p(q_branch), _p(k_shard), _p(v_shard),
                                      qm_range[0], qm_range[1], br_range[0], br_range[1], kv_range[0], kv_range[1],
                                      1 if merge else 0, _p(acc_o), _p(acc_lse), _stream())
    _check(rc, "branch_attn_fwd_shard")
    return acc_o, acc_lse


def branch_attn_bwd_shard(plan, q_main, q_branch, k_shard, v_shard, o, lse, d_o, qm_range, br_range, kv_range,
                          dq_main, dq_branch, dk_shard, dv_shard, stages=STAGE_DQ | STAGE_DKDV):
    """Partial backward over the main keys [kv_range) held in the shard: adds to the local
    fp32 dQ accumulators and to the shard's fp32 dK / dV accumulators."""
    p = plan.problem
    rows = kv_range[1] - kv_range[0]
    _expect_shard(plan, q_main, q_branch, k_shard, v_shard, kv_range)
    _expect("o", o, (p.rows, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("lse", lse, (p.rows, p.h_q), torch.float32, plan.device)
    _expect("d_o", d_o, (p.rows, p.h_q, p.head_dim), plan.torch_dtype, plan.device)
    _expect("dq_main", dq_main, (p.n_main, p.h_q, p.head_dim), torch.float32, plan.device, optional=q_main is None)
    _expect("dq_branch", dq_branch, (p.n_branch, p.h_q, p.head_dim), torch.float32, plan.device, optional=p.n_branch == 0)
    _expect("dk_shard", dk_shard, (rows, p.h_kv, p.head_dim), torch.float32, plan.device)
    _expect("dv_shard", dv_shard, (rows, p.h_kv, p.head_dim), torch.float32, plan.device)
    ws = plan.workspace(OP_BWD_FUSED if getattr(plan, "_fused_ws", False) else OP_BWD)
    rc = _lib().branch_attn_bwd_shard(plan.handle, _p(q_main), _p(q_branch), _p(k_shard), _p(v_shard), _p(o), _p(lse),
                                      _p(d_o), qm_range[0], qm_range[1], br_range[0], br_range[1], kv_range[0],
                                      kv_range[1], _p(dq_main), _p(dq_branch), _p(dk_shard), _p(dv_shard),
                                      _p(ws), ws.numel(), _stream(), stages)
    _check(rc, "branch_attn_bwd_shard")

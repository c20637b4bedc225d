"""numpy front end of the fp64 CPU oracle -- TEST INFRASTRUCTURE ONLY.

Loads `liboracle.so` (built from `branch_attn_oracle.c` by `build()`) through
ctypes.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import this module; the CUDA product never does, and this module imports
nothing from the product package.

A `problem` is any object with the attributes `cu_seqlens`, `anchor_idx`,
`branch_offsets`, `kind` (0 chain, 1 block, 2 tree), `parent`, `h_q`, `h_kv`,
`head_dim`, `softmax_scale`.  Query rows and key rows are numbered "main rows
[0, N) then branch tokens [N, N+M)".

The functions follow the paper's Section 3.2: two key sets per branch query
(causal main prefix up to the anchor, own-branch keys under the branch mask),
the merge of Eq. (lse-merge), and gradients accumulated over key chunks.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "branch_attn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None

PART_MAIN, PART_BRANCH, PART_ALL = 1, 2, 3


class _Problem(C.Structure):
    _fields_ = [
        ("n_main", C.c_int64), ("n_branch", C.c_int64),
        ("num_seqs", C.c_int64), ("num_branches", C.c_int64),
        ("cu_seqlens", C.c_void_p), ("anchor_idx", C.c_void_p),
        ("branch_offsets", C.c_void_p), ("parent", C.c_void_p),
        ("kind", C.c_int32), ("h_q", C.c_int32), ("h_kv", C.c_int32), ("d", C.c_int32),
        ("scale", C.c_double),
        ("parts", C.c_int32),
        ("kv_begin", C.c_int64), ("kv_end", C.c_int64),
    ]


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                               "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        for name in ("oracle_visibility", "oracle_forward", "oracle_lse_merge", "oracle_backward"):
            getattr(_lib, name).restype = C.c_int
    return _lib


def _ptr(a):
    return C.c_void_p(a.ctypes.data) if a is not None and a.size else C.c_void_p(0)


class _Ctx:
    """Keeps the int32 metadata arrays alive next to the C struct."""

    def __init__(self, p, parts=PART_ALL, kv_range=None):
        self.cu = np.ascontiguousarray(p.cu_seqlens, dtype=np.int32)
        self.anchor = np.ascontiguousarray(p.anchor_idx, dtype=np.int32)
        self.offs = np.ascontiguousarray(p.branch_offsets, dtype=np.int32)
        self.parent = (np.ascontiguousarray(p.parent, dtype=np.int32)
                       if p.parent is not None else None)
        self.n = int(self.cu[-1])
        self.m = int(self.offs[-1]) if len(self.offs) else 0
        kb, ke = (0, self.n) if kv_range is None else kv_range
        self.s = _Problem(self.n, self.m, len(self.cu) - 1, len(self.anchor),
                          _ptr(self.cu), _ptr(self.anchor), _ptr(self.offs), _ptr(self.parent),
                          int(p.kind), int(p.h_q), int(p.h_kv), int(p.head_dim),
                          float(p.softmax_scale), int(parts), int(kb), int(ke))

    def rows(self, rows):
        if rows is None:
            rows = np.arange(self.n + self.m, dtype=np.int64)
        return np.ascontiguousarray(rows, dtype=np.int64)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def gather_q(p, q_main, q_branch, rows=None):
    """Query vectors [n_rows, h_q, d] (fp64) of the listed global rows."""
    n = int(p.cu_seqlens[-1])
    if rows is None:
        return _f64(np.concatenate([q_main, q_branch], axis=0))
    rows = np.asarray(rows, dtype=np.int64)
    out = np.empty((len(rows), p.h_q, p.head_dim), dtype=np.float64)
    is_b = rows >= n
    if (~is_b).any():
        out[~is_b] = q_main[rows[~is_b]]
    if is_b.any():
        out[is_b] = q_branch[rows[is_b] - n]
    return out


def visibility(p, rows=None, parts=PART_ALL, kv_range=None) -> np.ndarray:
    """Dense boolean matrix [n_rows, N+M]: may query row r see key row x?"""
    ctx = _Ctx(p, parts, kv_range)
    rows = ctx.rows(rows)
    out = np.zeros((len(rows), ctx.n + ctx.m), dtype=np.uint8)
    rc = _load().oracle_visibility(C.byref(ctx.s), C.c_int64(len(rows)), _ptr(rows), _ptr(out))
    assert rc == 0
    return out.astype(bool)


def forward(p, q_rows, k, v, rows=None, parts=PART_ALL, kv_range=None):
    """(O [n_rows,h_q,d], LSE [n_rows,h_q]) in fp64 for the listed rows.

    `q_rows` holds the query vectors of exactly those rows (see `gather_q`).
    """
    ctx = _Ctx(p, parts, kv_range)
    rows = ctx.rows(rows)
    q_rows, k, v = _f64(q_rows), _f64(k), _f64(v)
    assert q_rows.shape == (len(rows), p.h_q, p.head_dim)
    assert k.shape == v.shape == (ctx.n + ctx.m, p.h_kv, p.head_dim)
    o = np.zeros_like(q_rows)
    lse = np.zeros((len(rows), p.h_q), dtype=np.float64)
    rc = _load().oracle_forward(C.byref(ctx.s), C.c_int64(len(rows)), _ptr(rows),
                                _ptr(q_rows), _ptr(k), _ptr(v), _ptr(o), _ptr(lse))
    assert rc == 0
    return o, lse


def lse_merge(o_a, lse_a, o_b, lse_b):
    """Eq. (lse-merge) on fp64 arrays [..., d] / [...]."""
    o_a, o_b, lse_a, lse_b = _f64(o_a), _f64(o_b), _f64(lse_a), _f64(lse_b)
    assert o_a.shape == o_b.shape and lse_a.shape == lse_b.shape == o_a.shape[:-1]
    o = np.zeros_like(o_a)
    lse = np.zeros_like(lse_a)
    rc = _load().oracle_lse_merge(C.c_int64(lse_a.size), C.c_int(o_a.shape[-1]),
                                  _ptr(o_a), _ptr(lse_a), _ptr(o_b), _ptr(lse_b),
                                  _ptr(o), _ptr(lse))
    assert rc == 0
    return o, lse


def backward(p, q_rows, k, v, d_o_rows, rows=None, parts=PART_ALL, kv_range=None):
    """(dQ [n_rows,h_q,d], dK, dV [N+M,h_kv,d]) for the loss sum_r <dO_r, O_r>
    over the listed rows.  The log-sum-exp and delta = <dO, O> always come from
    the complete visible set; `parts` / `kv_range` select which keys' gradient
    terms are summed (gradients are additive over key chunks)."""
    full = _Ctx(p)
    rows = full.rows(rows)
    q_rows, k, v, d_o_rows = _f64(q_rows), _f64(k), _f64(v), _f64(d_o_rows)
    o, lse = forward(p, q_rows, k, v, rows)
    delta = np.ascontiguousarray((o * d_o_rows).sum(axis=-1))
    ctx = _Ctx(p, parts, kv_range)
    dq = np.zeros_like(q_rows)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    rc = _load().oracle_backward(C.byref(ctx.s), C.c_int64(len(rows)), _ptr(rows),
                                 _ptr(q_rows), _ptr(k), _ptr(v), _ptr(d_o_rows),
                                 _ptr(lse), _ptr(delta), _ptr(dq), _ptr(dk), _ptr(dv))
    assert rc == 0
    return dq, dk, dv

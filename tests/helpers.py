"""Shared helpers of the GPU parity tests: run the CUDA library through its
binding, run the CPU oracle on the same seeded inputs, compare."""
from __future__ import annotations

import copy

import numpy as np
import torch

from paper_2609_07108_b200 import workloads as W

# Tolerances (max abs on O/dQ/dK/dV; LSE relative to max(1, |lse|)).
TOL = {"bf16": 2e-2, "fp32": 1e-4}
LSE_RTOL = 1e-3


def to_dev(p, t, device="cuda"):
    dt = torch.bfloat16 if p.dtype == "bf16" else torch.float32
    return {k: torch.from_numpy(v).to(device=device, dtype=dt) for k, v in t.items()}


def f32(x):
    return x.detach().float().cpu().numpy()


def head_slice(p, groups):
    """Problem restricted to the listed KV-head groups (heads are independent)."""
    g = p.h_q // p.h_kv
    q_heads = np.concatenate([np.arange(k * g, (k + 1) * g) for k in groups])
    p2 = copy.copy(p)
    p2.h_kv = len(groups)
    p2.h_q = len(q_heads)
    return p2, q_heads, np.asarray(groups)


def assert_close(name, got, want, tol):
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == np.shape(want), f"{name}: shape {got.shape} vs {np.shape(want)}"
    if got.size == 0:
        return
    err = np.abs(got - want)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    assert err.max() <= tol, f"{name}: max abs err {err.max():.3e} > {tol:.1e} at {np.unravel_index(err.argmax(), err.shape)}"


def assert_lse_close(got, want):
    got = np.asarray(got, dtype=np.float64)
    neg = np.isneginf(want)
    assert (np.isneginf(got) == neg).all(), "LSE: -inf pattern differs"
    err = np.abs(got[~neg] - want[~neg]) / np.maximum(1.0, np.abs(want[~neg]))
    if err.size:
        assert err.max() <= LSE_RTOL, f"LSE: max rel err {err.max():.3e}"


def oracle_fwd_bwd(oracle, p, t, groups=None, rows=None, backward=True, parts=3, kv_range=None):
    """Oracle results on a KV-group subset and/or row subset.

    Returns dict with o, lse (rows x subset heads), and dq, dk, dv if asked.
    """
    groups = list(range(p.h_kv)) if groups is None else list(groups)
    p2, qh, kvh = head_slice(p, groups)
    k = t["k"][:, kvh]
    v = t["v"][:, kvh]
    q_rows = oracle.gather_q(p, t["q_main"][:, qh], t["q_branch"][:, qh], rows)
    out = {"q_heads": qh, "kv_heads": kvh}
    out["o"], out["lse"] = oracle.forward(p2, q_rows, k, v, rows=rows, parts=parts, kv_range=kv_range)
    if backward:
        go = t["d_o"][:, qh] if rows is None else t["d_o"][np.asarray(rows)][:, qh]
        out["dq"], out["dk"], out["dv"] = oracle.backward(p2, q_rows, k, v, go, rows=rows,
                                                          parts=parts, kv_range=kv_range)
    return out

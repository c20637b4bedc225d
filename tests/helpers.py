"""Shared helpers of the GPU parity tests: run the CUDA library through its
binding, run the CPU oracle on the same seeded inputs, compare."""
from __future__ import annotations

import copy

import numpy as np
import torch

from paper_2609_07108_b200 import workloads as W

# Tolerances.  The absolute bound on O / dQ / dK / dV and the relative bound on
# LSE are the stated acceptance bounds.  At long context most outputs are far
# smaller than the absolute bound (|O| ~ 1e-2, |dQ| ~ 1e-4 at 32K-256K keys), so
# every comparison is additionally gated relative to the data:
#   rel-RMS  ||got - want||_2 / ||want||_2 per tensor,
#   per row  max|err_row| <= ROW_RTOL * max(max|want_row|, ROW_FLOOR * max|want|),
#   LSE      |got - want| <= LSE_ATOL absolutely (one dropped 128-key tile out of
#            2,048 moves LSE by 4.9e-4).
TOL = {"bf16": 2e-2, "fp32": 1e-4}
REL_RMS = {"bf16": 1e-2, "fp32": 1e-5}
ROW_RTOL = {"bf16": 2e-2, "fp32": 1e-4}
ROW_FLOOR = 1e-3
# The backward takes O in the input dtype, so delta = <dO, O> carries O's rounding
# (relative 2^-9 in bf16).  In a row with n visible keys that error reaches dQ as
# about 2e-3 / sqrt(n) of |dQ_row|; for a one-key row dQ is exactly zero in exact
# arithmetic.  Rows with fewer keys than this are held to the absolute bound only.
ROW_GATE_MIN_KEYS = 8
LSE_RTOL = 1e-3
LSE_ATOL = 1e-4

REPORT = []   # (name, max abs err, rel-RMS) of every comparison, for the test log


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


def dtype_of_tol(tol):
    return "fp32" if tol <= 1e-3 else "bf16"


def error_metrics(got, want):
    """(max abs error, rel-RMS error) of one tensor."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    if got.size == 0:
        return 0.0, 0.0
    err = got - want
    den = float(np.sqrt(np.mean(want * want)))
    num = float(np.sqrt(np.mean(err * err)))
    return float(np.abs(err).max()), (num / den if den > 0 else (0.0 if num == 0 else np.inf))


def assert_close(name, got, want, tol, row_keys=None, relative=True):
    """Absolute bound `tol`, plus (relative=True) the rel-RMS gate and the per-row
    scaled gate.  A "row" is one vector along the last axis.  `row_keys`: visible
    keys of each index of axis 0 (rows with fewer than ROW_GATE_MIN_KEYS are
    exempt from the per-row gate)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == np.shape(want), f"{name}: shape {got.shape} vs {np.shape(want)}"
    if got.size == 0:
        return
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    err = np.abs(got - want)
    max_abs, rel_rms = error_metrics(got, want)
    REPORT.append((name, max_abs, rel_rms))
    print(f"[parity] {name}: max abs err {max_abs:.3e}, rel-RMS {rel_rms:.3e}, max |want| {np.abs(want).max():.3e}")
    assert max_abs <= tol, f"{name}: max abs err {max_abs:.3e} > {tol:.1e} at {np.unravel_index(err.argmax(), err.shape)}"
    if not relative:
        return
    kind = dtype_of_tol(tol)
    assert rel_rms <= REL_RMS[kind], f"{name}: rel-RMS err {rel_rms:.3e} > {REL_RMS[kind]:.0e}"
    if got.ndim >= 2:
        row_err = err.max(axis=-1)
        row_mag = np.abs(want).max(axis=-1)
        floor = ROW_FLOOR * float(np.abs(want).max())
        bound = ROW_RTOL[kind] * np.maximum(row_mag, floor)
        bad = row_err > bound
        if row_keys is not None:
            few = np.asarray(row_keys) < ROW_GATE_MIN_KEYS
            bad &= ~few.reshape((-1,) + (1,) * (bad.ndim - 1))
        if bad.any():
            i = np.unravel_index(np.argmax(np.where(bad, row_err / np.maximum(bound, 1e-300), 0)), bad.shape)
            raise AssertionError(f"{name}: row {i}: max err {row_err[i]:.3e} > {bound[i]:.3e} "
                                 f"(row max |want| {row_mag[i]:.3e}); {int(bad.sum())} rows over the scaled bound")


def assert_lse_close(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    neg = np.isneginf(want)
    assert (np.isneginf(got) == neg).all(), "LSE: -inf pattern differs"
    if (~neg).any():
        d = np.abs(got[~neg] - want[~neg])
        rel = d / np.maximum(1.0, np.abs(want[~neg]))
        print(f"[parity] LSE: max abs err {d.max():.3e}")
        assert rel.max() <= LSE_RTOL, f"LSE: max rel err {rel.max():.3e}"
        assert d.max() <= LSE_ATOL, f"LSE: max abs err {d.max():.3e} > {LSE_ATOL:.0e}"


def visible_counts(p):
    """Visible keys of every query row (main rows, then branch tokens), from the
    metadata alone."""
    cu = p.cu_seqlens.astype(np.int64)
    n = p.n_main
    pos = np.arange(n, dtype=np.int64)
    seq = np.searchsorted(cu, pos, side="right") - 1
    main = pos - cu[seq] + 1
    if p.num_branches == 0:
        return main
    anchors = p.anchor_idx.astype(np.int64)
    aseq = np.searchsorted(cu, anchors, side="right") - 1
    prefix = anchors - cu[aseq] + 1
    blen = np.diff(p.branch_offsets.astype(np.int64))
    local = W._uniform_local_counts(p)
    if local is None:
        local = W.branch_local_counts(p)
    return np.concatenate([main, np.repeat(prefix, blen) + local])


def key_viewer_counts(p):
    """For every key (main keys, then branch tokens): an upper bound on the largest
    visible-set size among the query rows that can see it -- the longest row of its
    sequence for a main key, the longest row of its own branch for a branch key.  Keys
    whose every viewer has only a few keys inherit the cancellation described at
    ROW_GATE_MIN_KEYS."""
    cu = p.cu_seqlens.astype(np.int64)
    pos = np.arange(p.n_main, dtype=np.int64)
    seq = np.searchsorted(cu, pos, side="right") - 1
    main = cu[seq + 1] - cu[seq]
    if p.num_branches == 0:
        return main
    nk = visible_counts(p)[p.n_main:]
    offs = p.branch_offsets.astype(np.int64)
    blen = np.diff(offs)
    longest = np.zeros(p.num_branches, dtype=np.int64)
    nonempty = blen > 0
    longest[nonempty] = np.maximum.reduceat(nk, offs[:-1][nonempty])
    return np.concatenate([main, np.repeat(longest, blen)])


# Closed forms of the visible sets (q = 0 probes of the full-size tests), from the metadata alone.

def branch_visibility(p):
    """[M, L] bool: token t sees token u of its own branch (uniform branch length L),
    written out from the three mask definitions."""
    a = p.num_branches
    offs = p.branch_offsets.astype(np.int64)
    length = int(offs[1] - offs[0])
    assert (np.diff(offs) == length).all(), "closed-form probe: uniform branch length only"
    i = np.arange(length)
    if p.kind == W.CHAIN:
        one = i[None, :] <= i[:, None]
        return np.broadcast_to(one, (a, length, length)).reshape(a * length, length)
    if p.kind == W.BLOCK:
        return np.ones((a * length, length), dtype=bool)
    par = p.parent.reshape(a, length).astype(np.int64)
    anc = np.zeros((a, length, length), dtype=bool)
    ar = np.arange(a)
    for j in range(length):
        anc[:, j, j] = True
        has = par[:, j] >= 0
        anc[has, j, :] |= anc[ar[has], par[has, j], :]
    return anc.reshape(a * length, length)


def count_bit_below(x, b):
    """How many integers in [0, x) have bit b set."""
    x = np.asarray(x, dtype=np.int64)
    period = np.int64(1) << (b + 1)
    half = np.int64(1) << b
    return (x // period) * half + np.maximum(0, (x % period) - half)


N_BITS = 24
GROUP_OFFSET = 1000003     # key x of KV head g carries the bits of x + g * GROUP_OFFSET


def index_bit_values(p, device):
    """V [N+M, h_kv, D] bf16 with column c < 24 = bit c of (key index + head offset), column D-1 = 1."""
    x = torch.arange(p.rows, device=device, dtype=torch.int64)
    v = torch.zeros((p.rows, p.h_kv, p.head_dim), dtype=torch.bfloat16, device=device)
    for g in range(p.h_kv):
        code = x + g * GROUP_OFFSET
        for c in range(N_BITS):
            v[:, g, c] = ((code >> c) & 1).to(torch.bfloat16)
    v[:, :, p.head_dim - 1] = 1.0
    return v


def expected_bit_fractions(p, g):
    """[N+M, 24] float64: fraction of each row's visible keys whose code has bit c set (KV head g)."""
    cu = p.cu_seqlens.astype(np.int64)
    n = p.n_main
    off = g * GROUP_OFFSET
    pos = np.arange(n, dtype=np.int64)
    seq = np.searchsorted(cu, pos, side="right") - 1
    lo_main, hi_main = cu[seq], pos
    anchors = p.anchor_idx.astype(np.int64)
    blen = np.diff(p.branch_offsets.astype(np.int64))
    aseq = np.searchsorted(cu, anchors, side="right") - 1
    lo = np.concatenate([lo_main, np.repeat(cu[aseq], blen)])
    hi = np.concatenate([hi_main, np.repeat(anchors, blen)])
    counts = visible_counts(p).astype(np.float64)
    out = np.empty((p.rows, N_BITS), dtype=np.float64)
    vis = branch_visibility(p) if p.num_branches else None
    if vis is not None:
        length = vis.shape[1]
        start = np.repeat(p.branch_offsets[:-1].astype(np.int64), blen)
        codes = n + start[:, None] + np.arange(length)[None, :] + off          # [M, L]
    for c in range(N_BITS):
        cnt = count_bit_below(hi + 1 + off, c) - count_bit_below(lo + off, c)
        if vis is not None:
            cnt[n:] += (vis & (((codes >> c) & 1) == 1)).sum(axis=1)
        out[:, c] = cnt / counts
    return out



class Guarded:
    """Output tensor embedded in a larger allocation whose margins hold a sentinel:
    a kernel that writes outside its output changes a margin byte."""

    MARGIN = 4096      # bytes on each side (keeps 256-byte alignment of the payload)

    def __init__(self, shape, dtype, device="cuda", fill=None):
        numel = int(np.prod(shape))
        esz = torch.empty(0, dtype=dtype).element_size()
        nbytes = (numel * esz + 255) // 256 * 256
        self.raw = torch.full((nbytes + 2 * self.MARGIN,), 0xA5, dtype=torch.uint8, device=device)
        self.nbytes = numel * esz
        self.t = self.raw[self.MARGIN:self.MARGIN + numel * esz].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, name):
        head = self.raw[:self.MARGIN]
        tail = self.raw[self.MARGIN + self.nbytes:]
        assert bool((head == 0xA5).all()), f"{name}: bytes before the output were overwritten"
        assert bool((tail == 0xA5).all()), f"{name}: bytes after the output were overwritten"


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

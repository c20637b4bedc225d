"""Zigzag context-parallel layout, emulated on one GPU (host-side driver).

Paper Section 3.2 / Figure 1: the causal prefix is zigzag-sharded across C
context-parallel ranks, branch-local keys stay on the rank that owns the anchor,
and each rank merges its ring-step partial results with Eq. (lse-merge).  Here
the "ranks" are loop iterations on one device: the sequence is cut into 2C equal
chunks, rank r owns chunks r and 2C-1-r (and the branches anchored in them);
at ring step s it attends to the chunks of rank (r - s) mod C through the
library's partial forward / backward, with the branch-local part done in the
local step (s = 0).

`schedule` is pure integer bookkeeping (testable without a GPU); `forward` and
`backward` issue the library calls.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np


@dataclass(frozen=True)
class Block:
    rank: int
    step: int
    q_chunk: int
    kv_chunk: int
    qm: Tuple[int, int]       # main query rows
    br: Tuple[int, int]       # branch index range anchored in the q chunk
    kv: Tuple[int, int]       # main key rows
    branch_part: bool         # this call also covers the branch-local keys
    diagonal: bool            # q chunk == kv chunk


def chunk_bounds(n: int, cp: int) -> List[Tuple[int, int]]:
    """2*cp equal chunks of [0, n) (n must divide evenly)."""
    nc = 2 * cp
    if n % nc:
        raise ValueError(f"{n} tokens do not split into {nc} equal chunks")
    c = n // nc
    return [(i * c, (i + 1) * c) for i in range(nc)]


def rank_chunks(rank: int, cp: int) -> Tuple[int, int]:
    return rank, 2 * cp - 1 - rank


def schedule(problem, cp: int) -> List[Block]:
    """All (rank, ring step, q chunk, kv chunk) calls that carry work, for a
    single packed sequence.  A (q chunk, kv chunk) pair whose keys all lie after
    every query of the chunk is fully masked and skipped on the host."""
    if problem.num_seqs != 1:
        raise ValueError("the emulated zigzag layout is defined for one sequence")
    n = problem.n_main
    bounds = chunk_bounds(n, cp)
    anchors = np.asarray(problem.anchor_idx, dtype=np.int64)
    out = []
    for rank in range(cp):
        for step in range(cp):
            src = (rank - step) % cp
            for qc in rank_chunks(rank, cp):
                q0, q1 = bounds[qc]
                b0 = int(np.searchsorted(anchors, q0, side="left"))
                b1 = int(np.searchsorted(anchors, q1, side="left"))
                for kc in rank_chunks(src, cp):
                    if kc > qc:
                        continue                      # keys after every query: fully masked
                    out.append(Block(rank, step, qc, kc, (q0, q1), (b0, b1), bounds[kc],
                                     branch_part=(kc == qc), diagonal=(kc == qc)))
    return out


def pairs_per_rank(problem, cp: int) -> List[int]:
    """Visible (query, main key) pairs each emulated rank processes (branch-local
    pairs excluded): the quantity zigzag sharding balances."""
    n = problem.n_main
    bounds = chunk_bounds(n, cp)
    anchors = np.asarray(problem.anchor_idx, dtype=np.int64)
    blen = np.diff(np.asarray(problem.branch_offsets, dtype=np.int64))
    # weight of a main position = 1 (own row) + branch tokens anchored there
    w = np.ones(n, dtype=np.int64)
    np.add.at(w, anchors, blen)
    out = []
    for rank in range(cp):
        tot = 0
        for qc in rank_chunks(rank, cp):
            q0, q1 = bounds[qc]
            pos = np.arange(q0, q1, dtype=np.int64)
            tot += int((w[q0:q1] * (pos + 1)).sum())
        out.append(tot)
    return out


class Workspace:
    """Device buffers of the emulated layout, allocated once and reused by every
    step: the two compact fp32 (O, LSE) accumulators of a query chunk, and for the
    backward the four fp32 gradient accumulators plus the gradients in the input
    dtype.  (A step zeroes the accumulators with one memset each.)"""

    def __init__(self, ba, plan, cp, backward=True):
        import torch
        p = plan.problem
        self.cp = cp
        dev = plan.device
        csize = p.n_main // (2 * cp)
        max_rows = 0
        for b in schedule(p, cp):
            t0, t1 = plan.token_range(*b.br)
            max_rows = max(max_rows, csize + t1 - t0)
        f32 = dict(dtype=torch.float32, device=dev)
        self.acc_o = torch.empty((max_rows, p.h_q, p.head_dim), **f32)
        self.acc_l = torch.empty((max_rows, p.h_q), **f32)
        self.inc_o = self.inc_l = None
        if plan.impl != ba.IMPL_TC:       # the plain-FMA path merges in a pass of its own
            self.inc_o, self.inc_l = torch.empty_like(self.acc_o), torch.empty_like(self.acc_l)
        self.grads = self.outs = None
        if backward:
            shapes = ((p.n_main, p.h_q, p.head_dim), (p.n_branch, p.h_q, p.head_dim),
                      (p.rows, p.h_kv, p.head_dim), (p.rows, p.h_kv, p.head_dim))
            self.grads = tuple(torch.empty(s, **f32) for s in shapes)
            self.outs = tuple(torch.empty(s, dtype=plan.torch_dtype, device=dev) for s in shapes)


def chunk_order(cp: int) -> List[int]:
    """Query chunks in the order the drivers work through them (rank by rank)."""
    return [qc for rank in range(cp) for qc in rank_chunks(rank, cp)]


def forward(ba, plan, q_main, q_branch, k, v, cp, out=None, lse=None, ws=None, hooks=None):
    """Emulated CP forward: per (rank, step) partial calls, each merged into the
    running (O, LSE) by Eq. (lse-merge) -- in the kernel's epilogue on tensor-core
    plans, by `lse_merge` otherwise.  `out` may be fp32 (no rounding of O).
    `hooks.q_ready(qc)`, if given, is called before the first call that reads the
    query rows of chunk qc (a caller that streams the queries in waits there).
    Returns (O [N+M,h_q,D], LSE fp32, number of library launches)."""
    import torch
    p = plan.problem
    n = p.n_main
    if out is None:
        out = torch.empty((p.rows, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=plan.device)
    if lse is None:
        lse = torch.empty((p.rows, p.h_q), dtype=torch.float32, device=plan.device)
    if ws is None:
        ws = Workspace(ba, plan, cp, backward=False)
    blocks = schedule(p, cp)
    launches = 0
    # two compact fp32 buffers (accumulated, incoming) reused by every q chunk
    csize = n // (2 * cp)
    acc_o, acc_l, inc_o, inc_l = ws.acc_o, ws.acc_l, ws.inc_o, ws.inc_l
    # tensor-core plans merge each later ring step into the accumulators in the kernel's
    # epilogue; the plain-FMA path writes the step's partial result and merges it in a pass of its own
    in_kernel = plan.impl == ba.IMPL_TC
    for rank in range(cp):
        for qc in rank_chunks(rank, cp):
            mine = [b for b in blocks if b.rank == rank and b.q_chunk == qc]
            if hooks is not None:
                hooks.q_ready(qc)
            t0, t1 = plan.token_range(*mine[0].br)
            rows = csize + t1 - t0
            a_o, a_l = acc_o[:rows], acc_l[:rows]
            for j, b in enumerate(mine):
                parts = ba.PART_MAIN | (ba.PART_BRANCH if b.branch_part else 0)
                if j > 0 and in_kernel:
                    ba.branch_attn_fwd_partial_merge(plan, q_main, q_branch, k, v, b.qm, b.br, b.kv, parts, a_o, a_l)
                    launches += 1
                    continue
                i_o, i_l = (None, None) if in_kernel else (inc_o[:rows], inc_l[:rows])
                dst = (a_o, a_l) if j == 0 else (i_o, i_l)
                ba.branch_attn_fwd_partial(plan, q_main, q_branch, k, v, b.qm, b.br, b.kv, parts,
                                           out=dst[0], lse=dst[1])
                launches += 1
                if j > 0:
                    ba.lse_merge(a_o, a_l, i_o, i_l, out=a_o, lse_out=a_l)
                    launches += 1
            q0, q1 = mine[0].qm
            # fp32 compact -> output dtype, global layout (main rows, then the branch rows)
            ba.ba_finalize_grads(a_o[:csize], dst=out[q0:q1])
            ba.ba_finalize_grads(a_l[:csize], dst=lse[q0:q1])
            launches += 2
            if t1 > t0:
                ba.ba_finalize_grads(a_o[csize:], dst=out[n + t0:n + t1])
                ba.ba_finalize_grads(a_l[csize:], dst=lse[n + t0:n + t1])
                launches += 2
    return out, lse, launches


def backward(ba, plan, q_main, q_branch, k, v, o, lse, d_o, cp, fused=False, ws=None, hooks=None):
    """Emulated CP backward: the same (rank, step) blocks, gradients accumulated
    in fp32 and converted once at the end.  Returns (dQ_main, dQ_branch, dK, dV,
    launches) in the input dtype.  `fused`: one kernel per block for dQ, dK and
    dV (dQ summed with atomic adds) instead of a dQ and a dK/dV kernel.
    The per-row scalars (delta and -LSE log2 e) of a query chunk are prepared once,
    before the chunk's first block, not once per block.  dQ of a query chunk is
    complete when the chunk's last block is done (as on the rank that owns it) and is
    converted right then; `hooks.dq_done(qc, (q0, q1), (t0, t1))`, if given, is called
    after that (a caller that streams the gradients out starts there).  dK and dV
    are complete, and converted, at the end."""
    p = plan.problem
    if ws is None or ws.grads is None:
        ws = Workspace(ba, plan, cp, backward=True)
    grads = ws.grads
    for g in grads:
        g.zero_()
    launches = 0
    common = dict(accumulate=True, grads=grads)
    blocks = schedule(p, cp)
    for rank in range(cp):
        for qc in rank_chunks(rank, cp):
            mine = [b for b in blocks if b.rank == rank and b.q_chunk == qc]
            ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, qm_range=mine[0].qm, br_range=mine[0].br,
                               kv_range=(0, 0), parts=0, stages=ba.STAGE_PREP, **common)
            launches += 1
            for b in mine:
                parts = ba.PART_MAIN | (ba.PART_BRANCH if b.branch_part else 0)
                rng = dict(qm_range=b.qm, br_range=b.br, kv_range=b.kv, parts=parts)
                if fused:
                    ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, stages=ba.STAGE_FUSED, **rng, **common)
                    launches += 1
                else:
                    ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, stages=ba.STAGE_DQ, **rng, **common)
                    ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, stages=ba.STAGE_DKDV, **rng, **common)
                    launches += 2
            q0, q1 = mine[0].qm
            t0, t1 = plan.token_range(*mine[0].br)
            ba.ba_finalize_grads(grads[0][q0:q1], dst=ws.outs[0][q0:q1])
            launches += 1
            if t1 > t0:
                ba.ba_finalize_grads(grads[1][t0:t1], dst=ws.outs[1][t0:t1])
                launches += 1
            if hooks is not None:
                hooks.dq_done(qc, (q0, q1), (t0, t1))
    ba.ba_finalize_grads(grads[2], dst=ws.outs[2])
    ba.ba_finalize_grads(grads[3], dst=ws.outs[3])
    return (*ws.outs, launches + 2)

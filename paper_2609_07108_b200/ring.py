"""Zigzag K/V ring with a local double buffer (host-side driver).

Paper Section 3.2, "Communication cost and overlap": in the context-parallel
layout the queries stay on their rank while the K/V shards travel around a ring,
one hop per step, and the transfer of the next shard is hidden behind the
attention of the current one (step time = max(t_comm, t_attn)); per rank the
forward moves 2 (C - 1) (N / C) d_kv b bytes (Eq. cp-comm).  The backward
replays the same ring, and the gradient accumulators of a shard travel with it
back to its owner.

This module is that schedule in the form one GPU can run and test: the ranks are
loop iterations, "receiving" the next shard is a device copy (one cudaMemcpyAsync
per shard tensor, issued through torch on a side stream) from the memory that
stands for the peer into a local double buffer, and event hand-offs order copy
and compute exactly as a transport would: the kernels of a ring step read only
the local buffer (`branch_attn_fwd_shard` / `branch_attn_bwd_shard`), and a buffer
slot is refilled only after the step that read it has finished.  Step 0 of a
rank uses its own K/V (and its branch-local keys, which never move).  No kernel
reads another device's memory and nothing here needs more than one device; over
NVLink the copy would be a peer copy or a send/recv into the same buffer.

`hand_off_plan` is the pure schedule (testable on CPU, also by ranks that really
exchange shards through torch.distributed); `forward` / `backward` run it on the
device through the library and give results bit-identical to `zigzag.forward` /
`zigzag.backward` (same kernels, same accumulation order).
"""
from __future__ import annotations

from typing import Dict, List, Tuple

from . import zigzag


def shard_owner_chunks(rank: int, step: int, cp: int) -> Tuple[int, Tuple[int, int]]:
    """At ring step `step`, rank `rank` holds the shard of rank (rank - step) mod cp."""
    src = (rank - step) % cp
    return src, zigzag.rank_chunks(src, cp)


def hand_off_plan(rank: int, cp: int) -> List[tuple]:
    """Ordered actions of one rank for one pass over the ring.

    ("recv", step, src, slot)     start receiving the shard of `src`, needed at `step`, into `slot`
    ("wait", step, slot)          the compute stream waits until that shard has arrived
    ("compute", step, src, slot)  ring step on the shard in `slot` (slot None: the rank's own K/V)
    ("free", step, slot)          the step's kernels are done with `slot`; it may be refilled
    Slot of step s is s % 2; the receive for step s + 1 is issued before the compute of step s,
    and only after the "free" of step s - 1, which used the same slot."""
    plan = []
    for step in range(cp):
        if step + 1 < cp:
            nxt, _ = shard_owner_chunks(rank, step + 1, cp)
            plan.append(("recv", step + 1, nxt, (step + 1) % 2))
        src, _ = shard_owner_chunks(rank, step, cp)
        if step > 0:
            plan.append(("wait", step, step % 2))
        plan.append(("compute", step, src, None if step == 0 else step % 2))
        if step > 0:
            plan.append(("free", step, step % 2))
    return plan


def check_plan(plan: List[tuple]) -> None:
    """A slot is never refilled while a step may still read it, and never read before it arrived."""
    state = {0: "free", 1: "free"}       # free -> filling -> ready -> free
    for act in plan:
        kind = act[0]
        if kind == "recv":
            slot = act[3]
            assert state[slot] == "free", f"slot {slot} refilled while {state[slot]}"
            state[slot] = "filling"
        elif kind == "wait":
            slot = act[2]
            assert state[slot] == "filling"
            state[slot] = "ready"
        elif kind == "compute" and act[3] is not None:
            assert state[act[3]] == "ready", f"step {act[1]} reads slot {act[3]} that is {state[act[3]]}"
        elif kind == "free":
            assert state[act[2]] == "ready"
            state[act[2]] = "free"


def shard_bytes_per_rank(problem, cp: int, elem_bytes: int = 2) -> int:
    """Eq. (cp-comm): 2 (C - 1) (N / C) d_kv b with d_kv = h_kv * head_dim (K and V)."""
    return 2 * (cp - 1) * (problem.n_main // cp) * problem.h_kv * problem.head_dim * elem_bytes


class RingBuffers:
    """Local double buffer of one rank: two slots, each holding the K and V rows of the two
    chunks of a shard.  Allocated once; the emulated ranks reuse it in turn."""

    def __init__(self, plan, cp):
        import torch
        p = plan.problem
        self.csize = p.n_main // (2 * cp)
        shape = (2, 2, self.csize, p.h_kv, p.head_dim)      # [slot, chunk of the shard, rows, h_kv, d]
        self.k = torch.empty(shape, dtype=plan.torch_dtype, device=plan.device)
        self.v = torch.empty(shape, dtype=plan.torch_dtype, device=plan.device)
        self.side = torch.cuda.Stream(device=plan.device)


def new_stats() -> Dict:
    return {"copies": [], "copied_bytes": 0}


def copy_ms(stats) -> float:
    """Summed device time of the shard copies (after a synchronize)."""
    return sum(a.elapsed_time(b) for a, b in stats["copies"])


def forward(ba, plan, q_main, q_branch, k, v, cp, out=None, lse=None, ws=None, bufs=None, stats=None):
    """Ring forward.  Same result as `zigzag.forward`, bit for bit; K/V of the remote steps are
    read from the local double buffer only.  Returns (O, LSE, library launches)."""
    import torch
    p = plan.problem
    n = p.n_main
    if out is None:
        out = torch.empty((p.rows, p.h_q, p.head_dim), dtype=plan.torch_dtype, device=plan.device)
    if lse is None:
        lse = torch.empty((p.rows, p.h_q), dtype=torch.float32, device=plan.device)
    if plan.impl != ba.IMPL_TC:
        raise ValueError("the ring driver merges in the kernel epilogue: tensor-core plans only")
    bufs = bufs or RingBuffers(plan, cp)
    ws = ws or zigzag.Workspace(ba, plan, cp, backward=False)
    csize = n // (2 * cp)
    # a rank works on its two query chunks in every step: one compact accumulator pair for each
    if getattr(ws, "acc2_o", None) is None:
        ws.acc2_o, ws.acc2_l = torch.empty_like(ws.acc_o), torch.empty_like(ws.acc_l)
    launches = [0]
    state = {}

    def compute(b, k_src, v_src, shard):
        first = b.q_chunk not in state["started"]
        t0, t1 = plan.token_range(*b.br)
        rows = csize + t1 - t0
        acc = state["acc"][b.q_chunk]
        a_o, a_l = acc[0][:rows], acc[1][:rows]
        if shard:
            ba.branch_attn_fwd_shard(plan, q_main, q_branch, k_src, v_src, b.qm, b.br, b.kv, a_o, a_l, merge=not first)
        else:
            parts = ba.PART_MAIN | (ba.PART_BRANCH if b.branch_part else 0)
            if first:
                ba.branch_attn_fwd_partial(plan, q_main, q_branch, k_src, v_src, b.qm, b.br, b.kv, parts, out=a_o, lse=a_l)
            else:
                ba.branch_attn_fwd_partial_merge(plan, q_main, q_branch, k_src, v_src, b.qm, b.br, b.kv, parts, a_o, a_l)
        state["started"].add(b.q_chunk)
        launches[0] += 1

    blocks = zigzag.schedule(p, cp)
    # one rank at a time: run its ring, then write its two query chunks out
    for rank in range(cp):
        qa, qb = zigzag.rank_chunks(rank, cp)
        state["started"] = set()
        state["acc"] = {qa: (ws.acc_o, ws.acc_l), qb: (ws.acc2_o, ws.acc2_l)}
        _run_one_rank(ba, plan, cp, rank, k, v, bufs, stats, compute, blocks)
        for qc in (qa, qb):
            mine = [b for b in blocks if b.rank == rank and b.q_chunk == qc]
            t0, t1 = plan.token_range(*mine[0].br)
            a_o, a_l = state["acc"][qc]
            q0, q1 = mine[0].qm
            ba.ba_finalize_grads(a_o[:csize], dst=out[q0:q1])
            ba.ba_finalize_grads(a_l[:csize], dst=lse[q0:q1])
            launches[0] += 2
            if t1 > t0:
                rows = csize + t1 - t0
                ba.ba_finalize_grads(a_o[csize:rows], dst=out[n + t0:n + t1])
                ba.ba_finalize_grads(a_l[csize:rows], dst=lse[n + t0:n + t1])
                launches[0] += 2
    torch.cuda.current_stream().wait_stream(bufs.side)
    return out, lse, launches[0]


def _run_one_rank(ba, plan, cp, rank, k, v, bufs, stats, compute, blocks):
    import torch
    p = plan.problem
    bounds = zigzag.chunk_bounds(p.n_main, cp)
    main = torch.cuda.current_stream()
    side = bufs.side
    if not hasattr(bufs, "freed"):
        bufs.freed = {0: None, 1: None}
    arrived = {}
    timing = stats is not None
    for act in hand_off_plan(rank, cp):
        kind = act[0]
        if kind == "recv":
            _, step, src, slot = act
            if bufs.freed[slot] is None:                      # first use: order after the work already queued
                ev0 = torch.cuda.Event()
                ev0.record(main)
                bufs.freed[slot] = ev0
            with torch.cuda.stream(side):
                side.wait_event(bufs.freed[slot])             # the step that read this slot has finished
                t0 = torch.cuda.Event(enable_timing=timing)
                t0.record(side)
                for i, c in enumerate(zigzag.rank_chunks(src, cp)):       # one copy per shard tensor
                    a, b = bounds[c]
                    bufs.k[slot, i].copy_(k[a:b], non_blocking=True)
                    bufs.v[slot, i].copy_(v[a:b], non_blocking=True)
                ev = torch.cuda.Event(enable_timing=timing)
                ev.record(side)
            arrived[step] = ev
            if timing:
                stats["copies"].append((t0, ev))
                stats["copied_bytes"] += 4 * bufs.csize * p.h_kv * p.head_dim * k.element_size()
        elif kind == "wait":
            main.wait_event(arrived[act[1]])
        elif kind == "compute":
            _, step, src, slot = act
            chunks = zigzag.rank_chunks(src, cp)
            for b in (b for b in blocks if b.rank == rank and b.step == step):
                if slot is None:
                    compute(b, k, v, False)
                else:
                    i = chunks.index(b.kv_chunk)
                    compute(b, bufs.k[slot, i], bufs.v[slot, i], True)
        elif kind == "free":
            ev = torch.cuda.Event()
            ev.record(main)
            bufs.freed[act[2]] = ev


def backward(ba, plan, q_main, q_branch, k, v, o, lse, d_o, cp, fused=False, ws=None, bufs=None, stats=None):
    """Ring backward: replays the K/V ring; the fp32 dK / dV accumulators of a shard travel with
    it and return to their owner -- on one device the travelling accumulator of a chunk is the slice
    of the global accumulator it returns into, so the return trip is the identity.  Same result as
    `zigzag.backward` (bit for bit with the two-kernel backward)."""
    p = plan.problem
    bufs = bufs or RingBuffers(plan, cp)
    if ws is None or ws.grads is None:
        ws = zigzag.Workspace(ba, plan, cp, backward=True)
    grads = ws.grads
    for g in grads:
        g.zero_()
    launches = [0]
    blocks = zigzag.schedule(p, cp)
    stages = (ba.STAGE_FUSED,) if fused else (ba.STAGE_DQ, ba.STAGE_DKDV)

    def compute(b, k_src, v_src, shard):
        for st in stages:
            if shard:
                k0, k1 = b.kv
                ba.branch_attn_bwd_shard(plan, q_main, q_branch, k_src, v_src, o, lse, d_o, b.qm, b.br, b.kv,
                                         grads[0], grads[1], grads[2][k0:k1], grads[3][k0:k1], stages=st)
            else:
                parts = ba.PART_MAIN | (ba.PART_BRANCH if b.branch_part else 0)
                ba.branch_attn_bwd(plan, q_main, q_branch, k_src, v_src, o, lse, d_o, qm_range=b.qm, br_range=b.br,
                                   kv_range=b.kv, parts=parts, accumulate=True, grads=grads, stages=st)
            launches[0] += 1

    for rank in range(cp):
        for qc in zigzag.rank_chunks(rank, cp):        # per-row scalars of the rank's query chunks, once
            mine = [b for b in blocks if b.rank == rank and b.q_chunk == qc]
            ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, qm_range=mine[0].qm, br_range=mine[0].br,
                               kv_range=(0, 0), parts=0, accumulate=True, grads=grads, stages=ba.STAGE_PREP)
            launches[0] += 1
        _run_one_rank(ba, plan, cp, rank, k, v, bufs, stats, compute, blocks)
    import torch
    torch.cuda.current_stream().wait_stream(bufs.side)
    outs = tuple(ba.ba_finalize_grads(g, dst=d) for g, d in zip(grads, ws.outs))
    return (*outs, launches[0] + 4)

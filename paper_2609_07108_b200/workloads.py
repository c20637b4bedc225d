"""Seeded synthetic workloads for draft branch attention.

This module only produces *inputs*: packed sequence lengths, anchors, branch
shapes, random trees and random tensors.  It holds none of the attention
arithmetic, so both the CPU oracle's tests and the CUDA path's tests draw from
it without sharing any code of the method itself.

The five named configurations follow the paper's workload families (Section
3.2, "draft families": an EAGLE-3 training-time-test chain at every position,
a DFlash block per anchor, plus a general tree given by parent indices) on
packed variable-length batches as in the paper's Section 4.4 operator
benchmark (variable-length batches, fixed global lengths up to 256K tokens).
The paper's own data (RL rollouts) is not used; these inputs stand in for it.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

CHAIN, BLOCK, TREE = 0, 1, 2
KIND_NAMES = {CHAIN: "chain", BLOCK: "block", TREE: "tree"}

PART_MAIN, PART_BRANCH = 1, 2


@dataclass
class Problem:
    """Shape and metadata of one packed batch (no tensors)."""

    cu_seqlens: np.ndarray          # int32 [B+1]
    anchor_idx: np.ndarray          # int32 [A], global packed index, non-decreasing
    branch_offsets: np.ndarray      # int32 [A+1], branch-major token offsets
    kind: int                       # CHAIN / BLOCK / TREE
    parent: Optional[np.ndarray]    # int32 [M] branch-local parent (-1 = root), TREE only
    h_q: int
    h_kv: int
    head_dim: int
    dtype: str = "bf16"             # "bf16" or "fp32"
    scale: float = 0.0              # 0 => 1/sqrt(head_dim)
    name: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def n_main(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def num_seqs(self) -> int:
        return len(self.cu_seqlens) - 1

    @property
    def num_branches(self) -> int:
        return len(self.anchor_idx)

    @property
    def n_branch(self) -> int:
        return int(self.branch_offsets[-1])

    @property
    def rows(self) -> int:
        return self.n_main + self.n_branch

    @property
    def softmax_scale(self) -> float:
        return self.scale if self.scale > 0 else 1.0 / float(np.sqrt(self.head_dim))


# --------------------------------------------------------------------------
# building blocks
# --------------------------------------------------------------------------

def lognormal_lengths(rng: np.random.Generator, num_seqs: int, total: int,
                      median: float, sigma: float = 0.5, min_len: int = 16) -> np.ndarray:
    """`num_seqs` lengths summing to `total`, log-normal around `median`."""
    raw = rng.lognormal(mean=np.log(median), sigma=sigma, size=num_seqs)
    lens = np.maximum(min_len, np.rint(raw * (total / raw.sum()))).astype(np.int64)
    lens[np.argmax(lens)] += total - lens.sum()
    assert lens.sum() == total and lens.min() >= 1
    return lens


def cu_from_lengths(lens) -> np.ndarray:
    cu = np.zeros(len(lens) + 1, dtype=np.int64)
    cu[1:] = np.cumsum(np.asarray(lens, dtype=np.int64))
    return cu.astype(np.int32)


def uniform_branch_offsets(num_branches: int, length: int) -> np.ndarray:
    return (np.arange(num_branches + 1, dtype=np.int64) * length).astype(np.int32)


def random_tree_parents(rng: np.random.Generator, nodes: int, max_depth: int) -> np.ndarray:
    """Parent indices of one random tree: parent[0] = -1, parent[i] < i, and
    no root-to-node path holds more than `max_depth` tokens (root depth 1)."""
    parent = np.full(nodes, -1, dtype=np.int32)
    depth = np.ones(nodes, dtype=np.int32)
    for i in range(1, nodes):
        cand = np.nonzero(depth[:i] <= max_depth - 1)[0]
        p = int(cand[rng.integers(len(cand))])
        parent[i] = p
        depth[i] = depth[p] + 1
    return parent


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even), returned as fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit pattern of values already rounded with `round_to_bf16`."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def make_tensors(p: Problem, seed: int = 0, std: float = 1.0, cot_std: float = 0.1,
                 with_cotangent: bool = True) -> dict:
    """Q (main, branch), K, V and the output cotangent dO as fp32 arrays.

    For bf16 problems every value is rounded to bf16 once, so the oracle
    (promoting to fp64) and the GPU (reading bf16) see identical numbers.
    """
    rng = np.random.default_rng(seed)
    n, m, hq, hkv, d = p.n_main, p.n_branch, p.h_q, p.h_kv, p.head_dim

    def draw(r, shape, s):
        x = r.standard_normal(shape, dtype=np.float32) * np.float32(s)
        return round_to_bf16(x) if p.dtype == "bf16" else x

    t = {
        "q_main": draw(rng, (n, hq, d), std),
        "q_branch": draw(rng, (m, hq, d), std),
        "k": draw(rng, (n + m, hkv, d), std),
        "v": draw(rng, (n + m, hkv, d), std),
    }
    if with_cotangent:
        rng2 = np.random.default_rng(seed + 1)
        t["d_o"] = draw(rng2, (n + m, hq, d), cot_std)
    return t


# --------------------------------------------------------------------------
# the five named configurations (optionally scaled down by `shrink`)
# --------------------------------------------------------------------------

def _anchors_every(cu: np.ndarray, stride: int) -> np.ndarray:
    out = []
    for s in range(len(cu) - 1):
        out.append(np.arange(cu[s], cu[s + 1], stride, dtype=np.int64))
    return np.concatenate(out).astype(np.int32) if out else np.zeros(0, np.int32)


def config1() -> Problem:
    """Tiny fp32 case: sequences of 256 and 384 tokens, 4 heads, head_dim 64,
    depth-3 chains rooted at every 16th position of each sequence."""
    cu = cu_from_lengths([256, 384])
    anchors = _anchors_every(cu, 16)
    return Problem(cu, anchors, uniform_branch_offsets(len(anchors), 3), CHAIN, None,
                   4, 4, 64, dtype="fp32", name="config1_tiny_fp32_chain")


def config2(shrink: int = 1) -> Problem:
    """EAGLE-3 training-time-test shape: 8 packed log-normal sequences,
    8,192 tokens, 32/8 heads, head_dim 128, depth-3 chain at every position."""
    rng = np.random.default_rng(0)
    total = 8192 // shrink
    lens = lognormal_lengths(rng, 8, total, median=1024 / shrink)
    cu = cu_from_lengths(lens)
    anchors = np.arange(total, dtype=np.int32)
    return Problem(cu, anchors, uniform_branch_offsets(total, 3), CHAIN, None,
                   32, 8, 128, name=f"config2_eagle3_chain_{total}")


def config3(shrink: int = 1) -> Problem:
    """DFlash-style block draft: 32,768 tokens in 16 sequences, 512 anchors,
    16-token bidirectional blocks."""
    rng = np.random.default_rng(0)
    total = 32768 // shrink
    lens = lognormal_lengths(rng, 16, total, median=2048 / shrink)
    cu = cu_from_lengths(lens)
    na = max(1, 512 // shrink)
    anchors = np.sort(rng.choice(total, size=na, replace=False)).astype(np.int32)
    return Problem(cu, anchors, uniform_branch_offsets(na, 16), BLOCK, None,
                   32, 8, 128, name=f"config3_dflash_block_{total}")


def config4(shrink: int = 1) -> Problem:
    """General tree branch: 65,536 tokens in 16 sequences, 1,024 anchors each
    with a 31-node random tree of depth at most 6."""
    rng = np.random.default_rng(0)
    total = 65536 // shrink
    lens = lognormal_lengths(rng, 16, total, median=4096 / shrink)
    cu = cu_from_lengths(lens)
    na = max(1, 1024 // shrink)
    anchors = np.sort(rng.choice(total, size=na, replace=False)).astype(np.int32)
    trng = np.random.default_rng(1)
    parent = np.concatenate([random_tree_parents(trng, 31, 6) for _ in range(na)]).astype(np.int32)
    return Problem(cu, anchors, uniform_branch_offsets(na, 31), TREE, parent,
                   32, 8, 128, name=f"config4_tree_{total}")


def config5(shrink: int = 1) -> Problem:
    """Long-context single sequence: 262,144 tokens, depth-3 chain at every
    position; run through the 16-chunk zigzag layout of an 8-way split."""
    total = 262144 // shrink
    cu = cu_from_lengths([total])
    anchors = np.arange(total, dtype=np.int32)
    return Problem(cu, anchors, uniform_branch_offsets(total, 3), CHAIN, None,
                   32, 8, 128, name=f"config5_long_chain_{total}", extra={"cp": 8})


def varlen_ttt(shrink: int = 1) -> Problem:
    """Shape of the paper's operator benchmark (Section 4.4): a packed
    variable-length batch whose longest sequence has 20,480 tokens and whose
    padded-to-longest size is about 2.25 times its real size, EAGLE-3
    training-time test with three draft passes (depth-3 chain at every
    position).  Eight sequences, 73,728 tokens; the paper gives no length
    distribution beyond those two figures."""
    lens = [20480, 14336, 11264, 9216, 7168, 5120, 4096, 2048]
    lens = [max(1, x // shrink) for x in lens]
    total = int(sum(lens))
    cu = cu_from_lengths(lens)
    anchors = np.arange(total, dtype=np.int32)
    return Problem(cu, anchors, uniform_branch_offsets(total, 3), CHAIN, None,
                   32, 8, 128, name=f"varlen_ttt_chain_{total}")


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5, 6: varlen_ttt}


def odd_shapes(kind: int, seed: int = 0, h_q: int = 4, h_kv: int = 2, head_dim: int = 64,
               dtype: str = "fp32") -> Problem:
    """Correctness-only batch: sequence lengths 1, 17, 130, 0 and 257; anchors on
    the first and last token of a sequence; two branches on one anchor; branch
    lengths from 1 to 64."""
    rng = np.random.default_rng(seed)
    lens = [1, 17, 130, 0, 257]
    cu = cu_from_lengths(lens)
    anchors = [0, 1, 1, 9, 17, 18, 18 + 64, 18 + 129, 148, 148, 148 + 100, 148 + 256]
    anchors = np.array(sorted(anchors), dtype=np.int32)
    blens = np.array([1, 2, 64, 3, 17, 5, 33, 64, 7, 1, 31, 12], dtype=np.int64)
    offs = np.zeros(len(blens) + 1, dtype=np.int64)
    offs[1:] = np.cumsum(blens)
    parent = None
    if kind == TREE:
        parent = np.concatenate([random_tree_parents(rng, int(n), 6) for n in blens]).astype(np.int32)
    return Problem(cu, anchors, offs.astype(np.int32), kind, parent, h_q, h_kv, head_dim,
                   dtype=dtype, name=f"odd_{KIND_NAMES[kind]}")


# --------------------------------------------------------------------------
# pair counts and the zigzag chunk layout (integer bookkeeping only)
# --------------------------------------------------------------------------

def branch_local_counts(p: Problem) -> np.ndarray:
    """Per branch token, how many tokens of its own branch it may see."""
    m = p.n_branch
    out = np.zeros(m, dtype=np.int64)
    for b in range(p.num_branches):
        s, e = int(p.branch_offsets[b]), int(p.branch_offsets[b + 1])
        n = e - s
        if p.kind == CHAIN:
            out[s:e] = np.arange(1, n + 1)
        elif p.kind == BLOCK:
            out[s:e] = n
        else:
            depth = np.zeros(n, dtype=np.int64)
            for i in range(n):
                pi = int(p.parent[s + i])
                depth[i] = 1 if pi < 0 else depth[pi] + 1
            out[s:e] = depth
    return out


def _uniform_local_counts(p: Problem):
    """Fast path for uniform chain/block shapes (all branches equal length)."""
    a = p.num_branches
    if a == 0 or p.kind == TREE:
        return None
    n = int(p.branch_offsets[1] - p.branch_offsets[0])
    if not np.all(np.diff(p.branch_offsets.astype(np.int64)) == n):
        return None
    per = np.arange(1, n + 1, dtype=np.int64) if p.kind == CHAIN else np.full(n, n, np.int64)
    return np.tile(per, a)


def useful_pairs(p: Problem, with_main_queries: bool = True) -> int:
    """Number of (query row, visible key) pairs per query head."""
    cu = p.cu_seqlens.astype(np.int64)
    lens = np.diff(cu)
    pairs = int((lens * (lens + 1) // 2).sum()) if with_main_queries else 0
    if p.num_branches:
        anchors = p.anchor_idx.astype(np.int64)
        seq = np.searchsorted(cu, anchors, side="right") - 1
        prefix = anchors - cu[seq] + 1
        blen = np.diff(p.branch_offsets.astype(np.int64))
        pairs += int((prefix * blen).sum())
        loc = _uniform_local_counts(p)
        if loc is None:
            loc = branch_local_counts(p)
        pairs += int(loc.sum())
    return pairs

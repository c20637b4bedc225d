"""Pins for the fp64 CPU oracle: every check here compares the oracle with
something other than itself -- hand-written matrices, a brute-force Python
restatement, closed forms, a library attention routine, the merge equation's
invariants, finite differences.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "visibility_tiny.txt")


def tiny_problem(kind, h_q=2, h_kv=1, d=8, seed=0):
    """Two sequences (5 and 9 tokens) with four branches of unequal length."""
    rng = np.random.default_rng(seed)
    cu = W.cu_from_lengths([5, 9])
    anchors = np.array([0, 3, 3, 13], dtype=np.int32)
    lens = [2, 4, 1, 5]
    offs = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    parent = None
    if kind == W.TREE:
        parent = np.concatenate([W.random_tree_parents(rng, n, 3) for n in lens]).astype(np.int32)
    return W.Problem(cu, anchors, offs, kind, parent, h_q, h_kv, d, dtype="fp32")


def rand_tensors(p, seed=0, std=1.0):
    rng = np.random.default_rng(seed)
    n, m = p.n_main, p.n_branch
    q = rng.standard_normal((n + m, p.h_q, p.head_dim)) * std
    k = rng.standard_normal((n + m, p.h_kv, p.head_dim)) * std
    v = rng.standard_normal((n + m, p.h_kv, p.head_dim)) * std
    d_o = rng.standard_normal((n + m, p.h_q, p.head_dim))
    return q, k, v, d_o


# ---------------------------------------------------------------- visibility

def _parse_golden():
    cases, cur, section = {}, None, None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("[case"):
            cur = {"rows": {}}
            cases[line[6:-1]] = cur
            continue
        tok = line.split()
        if tok[0] in ("cu_seqlens", "anchors", "branch_offsets", "tree_parent"):
            cur[tok[0]] = np.array([int(t) for t in tok[1:]], dtype=np.int32)
        elif tok[0] in ("main", "chain", "block", "tree"):
            section = tok[0]
            cur["rows"][section] = []
        else:
            cur["rows"][section].append([int(c) for c in "".join(tok)])
    return cases


@pytest.mark.parametrize("case", ["two_seqs", "seven_node_tree"])
def test_visibility_matches_hand_written_matrices(oracle, case):
    c = _parse_golden()[case]
    for name, kind in (("chain", W.CHAIN), ("block", W.BLOCK), ("tree", W.TREE)):
        if name not in c["rows"]:
            continue
        p = W.Problem(c["cu_seqlens"], c["anchors"], c["branch_offsets"], kind,
                      c["tree_parent"] if kind == W.TREE else None, 1, 1, 4)
        want = np.array(c["rows"]["main"] + c["rows"][name], dtype=bool)
        got = oracle.visibility(p)
        assert got.shape == want.shape
        assert (got == want).all(), f"{case}/{name}"


def brute_visibility(p, parts=3, kv_range=None):
    """Second, independent restatement in plain Python loops."""
    n, m = p.n_main, p.n_branch
    kb, ke = (0, n) if kv_range is None else kv_range
    cu = [int(c) for c in p.cu_seqlens]

    def seq(i):
        return max(s for s in range(len(cu) - 1) if cu[s] <= i)  # last start <= i

    def seq_strict(i):
        for s in range(len(cu) - 1):
            if cu[s] <= i < cu[s + 1]:
                return s
        raise AssertionError

    vis = np.zeros((n + m, n + m), dtype=bool)
    for r in range(n):
        s = seq_strict(r)
        for x in range(cu[s], r + 1):
            vis[r, x] = bool(parts & 1) and kb <= x < ke
    for b in range(p.num_branches):
        a = int(p.anchor_idx[b])
        s = seq_strict(a)
        t0, t1 = int(p.branch_offsets[b]), int(p.branch_offsets[b + 1])
        for i in range(t1 - t0):
            r = n + t0 + i
            for x in range(cu[s], a + 1):
                vis[r, x] = bool(parts & 1) and kb <= x < ke
            if p.kind == W.CHAIN:
                local = set(range(i + 1))
            elif p.kind == W.BLOCK:
                local = set(range(t1 - t0))
            else:
                local, node = set(), i
                while node != -1:
                    local.add(node)
                    node = int(p.parent[t0 + node])
            for u in local:
                vis[r, n + t0 + u] = bool(parts & 2)
    return vis


@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
def test_visibility_matches_brute_force(oracle, kind):
    for p in (tiny_problem(kind), W.odd_shapes(kind)):
        assert (oracle.visibility(p) == brute_visibility(p)).all()
        for parts, rng_ in ((1, (3, 11)), (2, None), (3, (0, 4)), (1, (6, 6))):
            got = oracle.visibility(p, parts=parts, kv_range=rng_)
            assert (got == brute_visibility(p, parts, rng_)).all()


def test_visible_counts_match_pair_formula(oracle):
    """`useful_pairs` (closed form over lengths/anchors) equals the number of
    ones in the oracle's visibility matrix."""
    for kind in (W.CHAIN, W.BLOCK, W.TREE):
        for p in (tiny_problem(kind), W.odd_shapes(kind)):
            vis = oracle.visibility(p)
            assert int(vis.sum()) == W.useful_pairs(p)
            assert int(vis[p.n_main:].sum()) == W.useful_pairs(p, with_main_queries=False)
    p = W.config1()
    assert int(oracle.visibility(p).sum()) == W.useful_pairs(p) == 126184


# -------------------------------------------------------------- closed forms

@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
def test_zero_queries_give_log_count_and_mean_value(oracle, kind):
    """q = 0: every visible key gets the same weight, so LSE = log |U(r)| and
    O is the plain mean of the visible values (index-coded here)."""
    p = W.odd_shapes(kind)
    vis = brute_visibility(p)
    nk = p.rows
    q = np.zeros((nk, p.h_q, p.head_dim))
    rng = np.random.default_rng(1)
    k = rng.standard_normal((nk, p.h_kv, p.head_dim))
    v = np.zeros((nk, p.h_kv, p.head_dim))
    v[:, :, 0] = np.arange(nk)[:, None]          # value = key index
    v[:, :, 1] = 1.0                             # rows of P sum to one
    o, lse = oracle.forward(p, q, k, v)
    cnt = vis.sum(1)
    assert np.allclose(lse, np.log(cnt)[:, None], atol=1e-12)
    mean_idx = (vis * np.arange(nk)[None, :]).sum(1) / cnt
    assert np.allclose(o[:, :, 0], mean_idx[:, None], atol=1e-9)
    assert np.allclose(o[:, :, 1], 1.0, atol=1e-12)
    assert np.allclose(o[:, :, 2:], 0.0)


def test_one_hot_scores_pick_one_key(oracle):
    """A query aligned with exactly one visible key (huge score) returns that
    key's value; aligned with an invisible key it does not."""
    p = tiny_problem(W.CHAIN)
    p = W.Problem(p.cu_seqlens, p.anchor_idx, p.branch_offsets, W.CHAIN, None, 1, 1, 32, scale=1.0)
    nk = p.rows                                   # 26 rows: key x = unit vector e_x
    k = np.zeros((nk, 1, 32))
    for x in range(nk):
        k[x, 0, x] = 1.0
    v = np.random.default_rng(0).standard_normal((nk, 1, 32))
    vis = brute_visibility(p)
    for r in (2, 7, 13, 14 + 3, 14 + 11):
        for x in (0, 3, 6, 14 + 2, 14 + 3, 14 + 11):
            q = np.zeros((1, 1, 32))
            q[0, 0, x] = 200.0
            o, _ = oracle.forward(p, q, k, v, rows=[r])
            if vis[r, x]:
                assert np.allclose(o[0, 0], v[x, 0], atol=1e-12)
            else:
                assert not np.allclose(o[0, 0], v[x, 0], atol=1e-3)


# ------------------------------------------------------ library special cases

def _sdpa_causal(q, k, v, scale):
    """[L, H, D] fp64 arrays -> (O, LSE) by torch's library attention."""
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(a)).permute(1, 0, 2)[None] for a in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def test_no_branches_reduces_to_causal_attention(oracle):
    """Branch length 0: packed varlen causal attention, sequence by sequence."""
    lens = [7, 1, 33, 20]
    cu = W.cu_from_lengths(lens)
    p = W.Problem(cu, np.zeros(0, np.int32), np.zeros(1, np.int32), W.CHAIN, None, 4, 4, 16)
    q, k, v, _ = rand_tensors(p, 3)
    o, lse = oracle.forward(p, q, k, v)
    for s in range(len(lens)):
        a, b = cu[s], cu[s + 1]
        ref = _sdpa_causal(q[a:b], k[a:b], v[a:b], p.softmax_scale)
        assert np.allclose(o[a:b], ref, atol=1e-12)
    # LSE of the first token of each sequence is its single score
    for s in range(len(lens)):
        a = cu[s]
        s0 = p.softmax_scale * (q[a] * k[a]).sum(-1)
        assert np.allclose(lse[a], s0, atol=1e-12)


def test_single_chain_token_is_last_row_of_a_longer_causal_sequence(oracle):
    """One 1-token branch anchored at local position a: its output equals the
    last row of causal attention over [main 0..a, branch token]."""
    L, a = 12, 6
    cu = W.cu_from_lengths([4, L])
    p = W.Problem(cu, np.array([4 + a], np.int32), np.array([0, 1], np.int32), W.CHAIN, None, 2, 2, 8)
    q, k, v, _ = rand_tensors(p, 5)
    n = p.n_main
    o, _ = oracle.forward(p, q[n:], k, v, rows=[n])
    kk = np.concatenate([k[4:4 + a + 1], k[n:]], 0)
    vv = np.concatenate([v[4:4 + a + 1], v[n:]], 0)
    qq = np.concatenate([q[4:4 + a + 1], q[n:]], 0)
    ref = _sdpa_causal(qq, kk, vv, p.softmax_scale)
    assert np.allclose(o[0], ref[-1], atol=1e-12)


def test_block_branch_equals_dense_attention_over_union(oracle):
    """A block token's output is ordinary softmax attention over the explicit
    concatenation [prefix keys, block keys] (library matmul + softmax)."""
    p = tiny_problem(W.BLOCK, h_q=2, h_kv=2, d=8)
    q, k, v, _ = rand_tensors(p, 9)
    n = p.n_main
    o, lse = oracle.forward(p, q, k, v)
    b = 1                                                     # anchor 3, 4 tokens
    t0, t1 = p.branch_offsets[b], p.branch_offsets[b + 1]
    keys = np.concatenate([np.arange(0, 4), n + np.arange(t0, t1)])
    for i in range(t0, t1):
        for h in range(2):
            s = torch.from_numpy(k[keys, h] @ q[n + i, h]) * p.softmax_scale
            pr = torch.softmax(s, 0).numpy()
            assert np.allclose(o[n + i, h], pr @ v[keys, h], atol=1e-12)
            assert math.isclose(lse[n + i, h], float(torch.logsumexp(s, 0)), abs_tol=1e-12)


# ------------------------------------------------------------------- merge

def test_merge_hand_values(oracle):
    """Eq. (lse-merge) on values worked by hand."""
    inf = np.inf
    o_a = np.array([[1.0, 3.0], [2.0, 2.0], [5.0, 5.0], [0.0, 0.0]])
    o_b = np.array([[3.0, 1.0], [4.0, 0.0], [0.0, 0.0], [0.0, 0.0]])
    l_a = np.array([0.0, math.log(3.0), 1.5, -inf])
    l_b = np.array([0.0, 0.0, -inf, -inf])
    o, l = oracle.lse_merge(o_a, l_a, o_b, l_b)
    assert np.allclose(l[:3], [math.log(2.0), math.log(4.0), 1.5], atol=1e-15)
    assert l[3] == -inf
    assert np.allclose(o, [[2.0, 2.0], [2.5, 1.5], [5.0, 5.0], [0.0, 0.0]], atol=1e-15)
    assert not np.isnan(o).any()


@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
def test_main_part_merged_with_branch_part_is_union_attention(oracle, kind):
    """The paper's decomposition: attention over the main prefix and attention
    over the branch keys, merged by Eq. (lse-merge), equals attention over the
    union of both key sets."""
    p = W.odd_shapes(kind)
    q, k, v, _ = rand_tensors(p, 2, std=1.5)
    o, lse = oracle.forward(p, q, k, v)
    om, lm = oracle.forward(p, q, k, v, parts=1)
    ob, lb = oracle.forward(p, q, k, v, parts=2)
    n = p.n_main
    assert np.isneginf(lb[:n]).all() and (ob[:n] == 0).all()      # main queries: no branch keys
    o2, l2 = oracle.lse_merge(om, lm, ob, lb)
    assert np.allclose(o2, o, atol=1e-12) and np.allclose(l2, lse, atol=1e-12)


def test_merge_over_any_chunk_partition_and_order(oracle):
    p = W.odd_shapes(W.TREE)
    q, k, v, _ = rand_tensors(p, 4)
    o, lse = oracle.forward(p, q, k, v)
    n = p.n_main
    rng = np.random.default_rng(0)
    cuts = np.sort(rng.choice(np.arange(1, n), size=6, replace=False))
    bounds = [0, *cuts.tolist(), n]
    pieces = [oracle.forward(p, q, k, v, parts=1, kv_range=(bounds[i], bounds[i + 1]))
              for i in range(len(bounds) - 1)]
    pieces.append(oracle.forward(p, q, k, v, parts=2))
    for trial in range(3):
        order = rng.permutation(len(pieces))
        acc_o, acc_l = pieces[order[0]]
        for j in order[1:]:
            acc_o, acc_l = oracle.lse_merge(acc_o, acc_l, *pieces[j])
        assert np.allclose(acc_o, o, atol=1e-12) and np.allclose(acc_l, lse, atol=1e-12)


# -------------------------------------------------------------- invariances

def test_key_and_value_shift_invariance(oracle):
    p = tiny_problem(W.TREE, h_q=4, h_kv=2, d=8)
    q, k, v, _ = rand_tensors(p, 6)
    o, lse = oracle.forward(p, q, k, v)
    c = np.random.default_rng(7).standard_normal(8)
    o1, lse1 = oracle.forward(p, q, k + c, v)
    assert np.allclose(o1, o, atol=1e-12)
    assert np.allclose(lse1 - lse, p.softmax_scale * (q @ c), atol=1e-12)
    o2, lse2 = oracle.forward(p, q, k, v + c)
    assert np.allclose(o2, o + c, atol=1e-12) and np.allclose(lse2, lse, atol=1e-13)


def test_gqa_equals_repeated_kv_heads(oracle):
    p = tiny_problem(W.CHAIN, h_q=4, h_kv=2, d=8)
    q, k, v, d_o = rand_tensors(p, 8)
    o, lse = oracle.forward(p, q, k, v)
    dq, dk, dv = oracle.backward(p, q, k, v, d_o)
    p2 = tiny_problem(W.CHAIN, h_q=4, h_kv=4, d=8)
    k2, v2 = np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1)
    o2, lse2 = oracle.forward(p2, q, k2, v2)
    dq2, dk2, dv2 = oracle.backward(p2, q, k2, v2, d_o)
    assert np.allclose(o, o2, atol=1e-13) and np.allclose(lse, lse2, atol=1e-13)
    assert np.allclose(dq, dq2, atol=1e-13)
    assert np.allclose(dk, dk2.reshape(-1, 2, 2, 8).sum(2), atol=1e-12)
    assert np.allclose(dv, dv2.reshape(-1, 2, 2, 8).sum(2), atol=1e-12)


# ----------------------------------------------------------------- backward

@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
def test_gradients_match_central_finite_differences(oracle, kind):
    p = tiny_problem(kind, h_q=4, h_kv=2, d=8)
    q, k, v, d_o = rand_tensors(p, 11)
    dq, dk, dv = oracle.backward(p, q, k, v, d_o)

    def loss(q_, k_, v_):
        o, _ = oracle.forward(p, q_, k_, v_)
        return float((o * d_o).sum())

    rng = np.random.default_rng(0)
    h = 1e-5
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        flat_idx = rng.choice(arr.size, size=40, replace=False)
        # make sure both main rows and branch rows are probed
        for fi in flat_idx:
            idx = np.unravel_index(fi, arr.shape)
            plus = [q.copy(), k.copy(), v.copy()]
            minus = [q.copy(), k.copy(), v.copy()]
            j = "qkv".index(name)
            plus[j][idx] += h
            minus[j][idx] -= h
            fd = (loss(*plus) - loss(*minus)) / (2 * h)
            assert math.isclose(fd, grad[idx], rel_tol=1e-6, abs_tol=1e-8), (name, idx, fd, grad[idx])
        assert np.abs(grad).max() > 1e-3


def test_gradient_chunks_add_up_and_are_linear_in_cotangent(oracle):
    p = W.odd_shapes(W.BLOCK, h_q=2, h_kv=1, head_dim=8)
    q, k, v, d_o = rand_tensors(p, 12)
    dq, dk, dv = oracle.backward(p, q, k, v, d_o)
    n = p.n_main
    parts = [oracle.backward(p, q, k, v, d_o, parts=1, kv_range=(0, 100)),
             oracle.backward(p, q, k, v, d_o, parts=1, kv_range=(100, 101)),
             oracle.backward(p, q, k, v, d_o, parts=1, kv_range=(101, n)),
             oracle.backward(p, q, k, v, d_o, parts=2)]
    for got, want in zip((sum(x[i] for x in parts) for i in range(3)), (dq, dk, dv)):
        assert np.allclose(got, want, atol=1e-12)
    # a chunk's dK/dV are zero outside the chunk
    assert (parts[0][1][100:] == 0).all() and (parts[3][2][:n] == 0).all()
    dq3, dk3, dv3 = oracle.backward(p, q, k, v, -2.5 * d_o)
    assert np.allclose(dq3, -2.5 * dq, atol=1e-12)
    assert np.allclose(dk3, -2.5 * dk, atol=1e-12) and np.allclose(dv3, -2.5 * dv, atol=1e-12)


def test_row_subset_gives_the_same_rows(oracle):
    p = W.odd_shapes(W.CHAIN, h_q=2, h_kv=1, head_dim=8)
    q, k, v, d_o = rand_tensors(p, 13)
    o, lse = oracle.forward(p, q, k, v)
    rows = np.array([0, 5, 17, 147, 404, p.n_main, p.n_main + 70, p.rows - 1])
    o_s, lse_s = oracle.forward(p, q[rows], k, v, rows=rows)
    assert np.array_equal(o_s, o[rows]) and np.array_equal(lse_s, lse[rows])
    # sparse cotangent: gradients of the listed rows only
    d_sparse = np.zeros_like(d_o)
    d_sparse[rows] = d_o[rows]
    dq, dk, dv = oracle.backward(p, q, k, v, d_sparse)
    dq_s, dk_s, dv_s = oracle.backward(p, q[rows], k, v, d_o[rows], rows=rows)
    assert np.allclose(dq_s, dq[rows], atol=1e-13)
    assert np.allclose(dk_s, dk, atol=1e-13) and np.allclose(dv_s, dv, atol=1e-13)

"""GPU parity of the step-major (per-depth) calls: the depth-d tokens of every
branch attend to their causal main prefix and to depths 1..d of their own branch,
with the branch tokens stored depth-major.  The oracle needs no new arithmetic:
it is the chain problem evaluated on the rows of depth d, with K / V permuted
from depth-major to the oracle's branch-major order by plain indexing."""
import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W
from helpers import (TOL, assert_close, assert_lse_close, f32, key_viewer_counts, oracle_fwd_bwd, to_dev,
                     visible_counts)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ba():
    from paper_2609_07108_b200 import binding
    assert torch.cuda.is_available()
    return binding


def depth_major(x, n, a, length):
    """[N + A*L, ...] with branch-major branch rows -> the same rows depth-major."""
    br = x[n:].reshape(a, length, *x.shape[1:])
    return torch.cat([x[:n], br.transpose(0, 1).reshape(a * length, *x.shape[1:])], 0).contiguous()


def branch_major(x, n, a, length):
    br = x[n:].reshape(length, a, *x.shape[1:])
    return torch.cat([x[:n], br.transpose(0, 1).reshape(a * length, *x.shape[1:])], 0).contiguous()


def chain_problem(seq_lens, anchors, length, h_q=4, h_kv=2):
    anchors = np.asarray(sorted(anchors), dtype=np.int32)
    return W.Problem(W.cu_from_lengths(seq_lens), anchors, W.uniform_branch_offsets(len(anchors), length), W.CHAIN,
                     None, h_q, h_kv, 128, name="chain_for_depth_calls")


def run_depth_case(ba, oracle, p, seed, splits=None, groups=None):
    n, a, length = p.n_main, p.num_branches, int(p.branch_offsets[1])
    t = W.make_tensors(p, seed=seed, std=0.5)
    t["d_o"][:n] = 0                      # the loss of this test is over the branch rows only
    d = to_dev(p, t)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    ref = oracle_fwd_bwd(oracle, p, t, groups=groups)
    qh, kvh = ref["q_heads"], ref["kv_heads"]
    k_dm, v_dm = depth_major(d["k"], n, a, length), depth_major(d["v"], n, a, length)
    q_br = d["q_branch"].reshape(a, length, p.h_q, p.head_dim)
    go_br = d["d_o"][n:].reshape(a, length, p.h_q, p.head_dim)
    nk, kk = visible_counts(p), key_viewer_counts(p)
    tol = TOL["bf16"]
    splits = splits or [(0, a)]
    outs = []
    for depth in range(1, length + 1):
        # rows of later depths "do not exist yet": poison them, the call must not read them
        k_now, v_now = k_dm.clone(), v_dm.clone()
        k_now[n + depth * a:] = float("nan")
        v_now[n + depth * a:] = float("nan")
        q_d = q_br[:, depth - 1].contiguous()
        o_d = torch.full((a, p.h_q, p.head_dim), 7.0, dtype=torch.bfloat16, device="cuda")
        lse_d = torch.full((a, p.h_q), 7.0, dtype=torch.float32, device="cuda")
        for br in splits:
            ba.branch_attn_fwd_depth(plan, depth, q_d, k_now, v_now, br_range=br, out=o_d, lse=lse_d)
        plan.check()
        rows = n + np.arange(a) * length + (depth - 1)
        assert_close(f"O depth {depth}", f32(o_d)[:, qh], ref["o"][rows], tol, row_keys=nk[rows])
        assert_lse_close(f32(lse_d)[:, qh], ref["lse"][rows])
        outs.append((q_d, o_d, lse_d, k_now, v_now))
    # backward, deepest first, all into the same depth-major fp32 accumulators
    dk = torch.zeros((p.rows, p.h_kv, p.head_dim), dtype=torch.float32, device="cuda")
    dv = torch.zeros_like(dk)
    for depth in range(length, 0, -1):
        q_d, o_d, lse_d, k_now, v_now = outs[depth - 1]
        go_d = go_br[:, depth - 1].contiguous()
        dq_d = torch.full((a, p.h_q, p.head_dim), 7.0, dtype=torch.bfloat16, device="cuda")
        for br in splits:
            ba.branch_attn_bwd_depth(plan, depth, q_d, k_now, v_now, o_d, lse_d, go_d, dk, dv, br_range=br, dq=dq_d)
        plan.check()
        rows = n + np.arange(a) * length + (depth - 1)
        assert_close(f"dQ depth {depth}", f32(dq_d)[:, qh], ref["dq"][rows], tol, row_keys=nk[rows])
    dk_bm, dv_bm = branch_major(dk, n, a, length), branch_major(dv, n, a, length)
    assert_close("dK (all depths accumulated)", f32(dk_bm)[:, kvh], ref["dk"], tol, row_keys=kk)
    assert_close("dV (all depths accumulated)", f32(dv_bm)[:, kvh], ref["dv"], tol, row_keys=kk)
    return plan, d, k_dm, v_dm


def test_depth_calls_match_the_oracle_every_position_anchored(ba, oracle):
    p = W.varlen_ttt(shrink=64)                        # eight sequences, a depth-3 chain at every position
    run_depth_case(ba, oracle, p, seed=31, groups=[0, p.h_kv - 1])


def test_depth_calls_sparse_anchors_shared_anchors_and_branch_ranges(ba, oracle):
    rng = np.random.default_rng(5)
    lens = [1, 130, 0, 257, 300]
    total = sum(lens)
    anchors = rng.choice(total, size=150, replace=True).tolist() + [0, 0, total - 1, total - 1, 130, 131]
    p = chain_problem(lens, anchors, length=4)
    a = p.num_branches
    run_depth_case(ba, oracle, p, seed=32, splits=[(0, 37), (37, 37), (37, 130), (130, a)])


def test_depth_calls_reject_what_they_cannot_do(ba):
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16")          # branches of unequal length
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    lib = ba._lib()
    x = torch.zeros(16, device="cuda")
    assert lib.branch_attn_fwd_depth(plan.handle, 1, ba._p(x), ba._p(x), ba._p(x), 0, 1, ba._p(x), ba._p(x), ba._stream()) == -2
    q = W.config3(shrink=16)                                         # block mask
    assert lib.branch_attn_fwd_depth(ba.Plan(q, impl=ba.IMPL_TC).handle, 1, ba._p(x), ba._p(x), ba._p(x), 0, 1, ba._p(x),
                                     ba._p(x), ba._stream()) == -2
    c = W.config2(shrink=16)
    cp = ba.Plan(c, impl=ba.IMPL_TC)
    for depth, br in ((0, (0, 1)), (4, (0, 1)), (1, (0, c.num_branches + 1)), (1, (5, 4))):
        assert lib.branch_attn_fwd_depth(cp.handle, depth, ba._p(x), ba._p(x), ba._p(x), br[0], br[1], ba._p(x), ba._p(x),
                                         ba._stream()) == -1
    assert lib.branch_attn_fwd_depth(cp.handle, 1, None, None, None, 3, 3, None, None, ba._stream()) == 0   # empty range
    torch.cuda.synchronize()


def test_stepwise_equals_all_depths_call_full_size(ba):
    """The paper's packed variable-length benchmark shape at full size: depth 1, 2, 3 in turn
    against the all-depths forward and backward (itself checked against the oracle at this
    size), on every branch row and every key."""
    p = W.varlen_ttt()
    n, a, length = p.n_main, p.num_branches, 3
    g = torch.Generator(device="cuda")
    g.manual_seed(41)

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    q_main, q_branch = draw((n, p.h_q, 128), 0.5), draw((a * length, p.h_q, 128), 0.5)
    k, v = draw((p.rows, p.h_kv, 128), 0.5), draw((p.rows, p.h_kv, 128), 0.5)
    d_o = draw((p.rows, p.h_q, 128), 0.1)
    d_o[:n] = 0
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, q_main, q_branch, k, v)
    gq, gb, gk, gv = ba.branch_attn_bwd(plan, q_main, q_branch, k, v, o, lse, d_o, accumulate=True,
                                        stages=ba.STAGE_ALL_FUSED)
    plan.check()
    assert float(gq.abs().max()) == 0.0
    k_dm, v_dm = depth_major(k, n, a, length), depth_major(v, n, a, length)
    nk, kk = visible_counts(p), key_viewer_counts(p)
    o_br = o[n:].reshape(a, length, p.h_q, 128)
    lse_br = lse[n:].reshape(a, length, p.h_q)
    dk = torch.zeros((p.rows, p.h_kv, 128), dtype=torch.float32, device="cuda")
    dv = torch.zeros_like(dk)
    want_count = nk[n:].reshape(a, length)
    for depth in (1, 2, 3):
        q_d = q_branch.reshape(a, length, p.h_q, 128)[:, depth - 1].contiguous()
        o_d, lse_d = ba.branch_attn_fwd_depth(plan, depth, q_d, k_dm, v_dm)
        plan.check()
        rk = want_count[:, depth - 1]
        assert_close(f"O depth {depth} vs all-depths call", f32(o_d), f32(o_br[:, depth - 1]).astype(np.float64), 2e-2,
                     row_keys=rk)
        assert float((lse_d - lse_br[:, depth - 1]).abs().max()) <= 1e-5
        # the backward takes the all-depths forward's O and LSE, as the all-depths backward did
        go_d = d_o[n:].reshape(a, length, p.h_q, 128)[:, depth - 1].contiguous()
        dq_d = ba.branch_attn_bwd_depth(plan, depth, q_d, k_dm, v_dm, o_br[:, depth - 1].contiguous(),
                                        lse_br[:, depth - 1].contiguous(), go_d, dk, dv)
        plan.check()
        want = gb.reshape(a, length, p.h_q, 128)[:, depth - 1]
        assert_close(f"dQ depth {depth} vs all-depths call", f32(dq_d), f32(want).astype(np.float64), 2e-2, row_keys=rk)
    assert_close("dK vs all-depths call", f32(branch_major(dk, n, a, length)), f32(gk).astype(np.float64), 2e-2, row_keys=kk)
    assert_close("dV vs all-depths call", f32(branch_major(dv, n, a, length)), f32(gv).astype(np.float64), 2e-2, row_keys=kk)
    # closed form over every branch row: q = 0  =>  LSE = log |visible set|
    zero = torch.zeros((a, p.h_q, 128), dtype=torch.bfloat16, device="cuda")
    for depth in (1, 2, 3):
        _, lse0 = ba.branch_attn_fwd_depth(plan, depth, zero, k_dm, v_dm)
        err = np.abs(f32(lse0).astype(np.float64) - np.log(want_count[:, depth - 1].astype(np.float64))[:, None])
        assert err.max() <= 2e-5, f"depth {depth}: q=0 LSE closed form off by {err.max():.2e}"
    plan.check()

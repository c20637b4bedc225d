"""GPU parity of the one-kernel backward (BA_STAGE_FUSED: dQ, dK, dV from one
key-stationary tensor-core kernel, dQ summed with fp32 atomic adds) against the
fp64 CPU oracle, element by element on the same seeded inputs."""
import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W
from helpers import TOL, assert_close, f32, key_viewer_counts, oracle_fwd_bwd, to_dev, visible_counts

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ba():
    from paper_2609_07108_b200 import binding
    assert torch.cuda.is_available()
    return binding


def fused_grads(ba, plan, d, o, lse, q_main=True, grads=None, **ranges):
    qm = d["q_main"] if q_main else None
    return ba.branch_attn_bwd(plan, qm, d["q_branch"], d["k"], d["v"], o, lse, d["d_o"], accumulate=True,
                              grads=grads, stages=ba.STAGE_ALL_FUSED, **ranges)


def check_fused(ba, oracle, p, seed=0, std=0.5, groups=None, q_main=True, mutate=None, relative_grads=True):
    t = W.make_tensors(p, seed=seed, std=std)
    if mutate:
        mutate(t)
    n = p.n_main
    if not q_main:
        t["d_o"][:n] = 0
    d = to_dev(p, t)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"] if q_main else None, d["q_branch"], d["k"], d["v"])
    ref = oracle_fwd_bwd(oracle, p, t, groups=groups)
    qh, kvh = ref["q_heads"], ref["kv_heads"]
    dqm, dqb, dk, dv = fused_grads(ba, plan, d, o, lse, q_main=q_main)
    plan.check()
    tol = TOL["bf16"]
    nk, kk = visible_counts(p), key_viewer_counts(p)
    rel = relative_grads
    if q_main:
        assert_close("dQ_main", f32(dqm)[:, qh], ref["dq"][:n], tol, row_keys=nk[:n], relative=rel)
    assert_close("dQ_branch", f32(dqb)[:, qh], ref["dq"][n:], tol, row_keys=nk[n:], relative=rel)
    assert_close("dK", f32(dk)[:, kvh], ref["dk"], tol, row_keys=kk, relative=rel)
    assert_close("dV", f32(dv)[:, kvh], ref["dv"], tol, row_keys=kk)
    # the split kernels on the same inputs: same sums up to the order of the dQ terms
    split = ba.branch_attn_bwd(plan, d["q_main"] if q_main else None, d["q_branch"], d["k"], d["v"], o, lse,
                               d["d_o"], accumulate=True)
    for name, a, b in zip(("dQm", "dQb", "dK", "dV"), (dqm, dqb, dk, dv), split):
        if a is not None:
            assert_close(name + " fused vs split", f32(a), f32(b).astype(np.float64), 5e-3, relative=False)
    plan.check()
    # gradients in the input dtype: dQ summed in the workspace and converted, dK / dV stored directly
    gq, gb, gk, gv = ba.branch_attn_bwd(plan, d["q_main"] if q_main else None, d["q_branch"], d["k"], d["v"], o, lse,
                                        d["d_o"], stages=ba.STAGE_ALL_FUSED)
    plan.check()
    assert gb.dtype == torch.bfloat16 and gk.dtype == torch.bfloat16
    if q_main:
        assert_close("dQ_main bf16", f32(gq)[:, qh], ref["dq"][:n], tol, row_keys=nk[:n], relative=rel)
    assert_close("dQ_branch bf16", f32(gb)[:, qh], ref["dq"][n:], tol, row_keys=nk[n:], relative=rel)
    assert_close("dK bf16", f32(gk)[:, kvh], ref["dk"], tol, row_keys=kk, relative=rel)
    assert_close("dV bf16", f32(gv)[:, kvh], ref["dv"], tol, row_keys=kk)


@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
def test_odd_shapes_all_masks(ba, oracle, kind):
    check_fused(ba, oracle, W.odd_shapes(kind, head_dim=128, dtype="bf16"), seed=3)


@pytest.mark.parametrize("cfg,shrink", [(3, 16), (4, 16), (5, 128), (6, 64)])
def test_shrunken_configs(ba, oracle, cfg, shrink):
    p = W.CONFIGS[cfg](shrink)
    check_fused(ba, oracle, p, seed=0, groups=[0, p.h_kv - 1])


@pytest.mark.parametrize("h_q,h_kv", [(2, 2), (3, 1), (5, 1), (6, 2)])
def test_head_group_sizes(ba, oracle, h_q, h_kv):
    check_fused(ba, oracle, W.odd_shapes(W.BLOCK, head_dim=128, dtype="bf16", h_q=h_q, h_kv=h_kv), seed=8)


@pytest.mark.parametrize("kind", [W.CHAIN, W.TREE])
def test_branch_queries_only(ba, oracle, kind):
    check_fused(ba, oracle, W.odd_shapes(kind, head_dim=128, dtype="bf16"), seed=4, q_main=False)


def _sharp(t):          # near one-hot softmax rows
    t["q_main"] *= 8
    t["q_branch"] *= 8


def _offset(t):         # a large common component in every key: scores far from zero
    rng = np.random.default_rng(99)
    c = W.round_to_bf16(rng.standard_normal(t["k"].shape[-1]).astype(np.float32) * 4)
    t["k"] += c
    t["k"][:] = W.round_to_bf16(t["k"])


def _late_outlier(t):   # one key aligned with a late query
    t["k"][400] = W.round_to_bf16(t["q_main"][404, 0] * 3)


@pytest.mark.parametrize("mutate", [_sharp, _offset, _late_outlier])
def test_stress_inputs(ba, oracle, mutate):
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16", h_q=4, h_kv=2)
    check_fused(ba, oracle, p, seed=6, mutate=mutate, relative_grads=False)


def test_unaligned_ranges_with_gradients_in_the_input_dtype(ba, oracle):
    """Query and key ranges that start and end inside tiles; rows and keys outside the
    ranges keep what the output tensors held."""
    p = W.odd_shapes(W.BLOCK, head_dim=128, dtype="bf16")
    t = W.make_tensors(p, seed=15, std=0.5)
    d = to_dev(p, t)
    n, a = p.n_main, p.num_branches
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
    qm, br, kv = (37, 301), (1, a - 1), (13, 333)
    t0, t1 = plan.token_range(*br)
    rows = np.concatenate([np.arange(*qm), n + np.arange(t0, t1)])
    ref_dq, ref_dk, ref_dv = oracle.backward(p, oracle.gather_q(p, t["q_main"], t["q_branch"], rows), t["k"], t["v"],
                                             t["d_o"][rows], rows=rows, parts=3, kv_range=kv)
    grads = tuple(torch.full(x.shape, 7.0, dtype=torch.bfloat16, device="cuda")
                  for x in (d["q_main"], d["q_branch"], d["k"], d["v"]))
    ba.branch_attn_bwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"], qm_range=qm, br_range=br,
                       kv_range=kv, grads=grads, stages=ba.STAGE_ALL_FUSED)
    plan.check()
    dq = torch.cat([grads[0], grads[1]], 0)
    nk, kk = visible_counts(p), key_viewer_counts(p)
    assert_close("dQ (selected rows)", f32(dq)[rows], ref_dq, TOL["bf16"], row_keys=nk[rows])
    other = np.ones(p.rows, bool); other[rows] = False
    assert float((dq[torch.from_numpy(other).cuda()].float() - 7.0).abs().max()) == 0.0
    keys = np.concatenate([np.arange(*kv), n + np.arange(t0, t1)])       # the key set of the call
    assert_close("dK (key set)", f32(grads[2])[keys], ref_dk[keys], TOL["bf16"], row_keys=kk[keys])
    assert_close("dV (key set)", f32(grads[3])[keys], ref_dv[keys], TOL["bf16"], row_keys=kk[keys])


def test_no_branches(ba, oracle):
    cu = W.cu_from_lengths([100, 300, 29])
    p = W.Problem(cu, np.zeros(0, np.int32), np.zeros(1, np.int32), W.CHAIN, None, 4, 2, 128, dtype="bf16")
    check_fused(ba, oracle, p, seed=5)


def test_key_chunks_and_query_ranges_accumulate(ba, oracle):
    """Ring-style use: one call per (key chunk, query range), all into the same accumulators."""
    p = W.odd_shapes(W.TREE, head_dim=128, dtype="bf16")
    t = W.make_tensors(p, seed=11, std=0.5)
    d = to_dev(p, t)
    n, a = p.n_main, p.num_branches
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
    grads = None
    for i, kv in enumerate([(0, 17), (17, 18), (18, 150), (150, 150), (150, n)]):
        parts = ba.PART_MAIN | (ba.PART_BRANCH if i == 2 else 0)
        for qmr, brr in (((0, 100), (0, 5)), ((100, n), (5, a))):
            grads = fused_grads(ba, plan, d, o, lse, grads=grads, qm_range=qmr, br_range=brr, kv_range=kv,
                                parts=parts)
    plan.check()
    ref = oracle_fwd_bwd(oracle, p, t)
    want = (ref["dq"][:n], ref["dq"][n:], ref["dk"], ref["dv"])
    nk, kk = visible_counts(p), key_viewer_counts(p)
    for name, g, w, rk in zip(("dQm", "dQb", "dK", "dV"), grads, want, (nk[:n], nk[n:], kk, kk)):
        assert_close(name, f32(g), w, TOL["bf16"], row_keys=rk)
        assert_close(name + " finalized", f32(ba.ba_finalize_grads(g, dtype=torch.bfloat16)), w, TOL["bf16"], row_keys=rk)


def test_dk_dv_bit_identical_dq_close_run_to_run(ba):
    p = W.CONFIGS[3](16)
    t = W.make_tensors(p, seed=2, std=0.5)
    d = to_dev(p, t)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
    g1 = fused_grads(ba, plan, d, o, lse)
    g2 = fused_grads(ba, plan, d, o, lse)
    plan.check()
    assert torch.equal(g1[2], g2[2]) and torch.equal(g1[3], g2[3])
    for a, b in zip(g1[:2], g2[:2]):
        assert (a - b).abs().max().item() <= 1e-4 * max(1.0, a.abs().max().item())


def test_rejects_what_it_cannot_do(ba):
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16")
    d = to_dev(p, W.make_tensors(p, seed=1, std=0.5))
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
    # gradients in the input dtype need the larger workspace (fp32 dQ accumulator)
    assert ba._lib().ba_workspace_bytes(plan.handle, ba.OP_BWD_FUSED) > ba._lib().ba_workspace_bytes(plan.handle, ba.OP_BWD)
    small = plan.workspace(ba.OP_BWD)
    grads = [torch.empty_like(x) for x in (d["q_main"], d["q_branch"], d["k"], d["v"])]
    rc = ba._lib().branch_attn_bwd_stages(plan.handle, *(ba._p(x) for x in (d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"])),
                                          0, p.n_main, 0, p.num_branches, 0, p.n_main, ba.PART_ALL, 0,
                                          *(ba._p(g) for g in grads), ba._p(small), small.numel(), ba._stream(),
                                          ba.STAGE_ALL_FUSED)
    assert rc == -3   # BA_EWORKSPACE
    with pytest.raises(ba.BranchAttnError) as e:   # fused replaces the dQ and dK/dV stages
        ba.branch_attn_bwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"], accumulate=True,
                           stages=ba.STAGE_FUSED | ba.STAGE_DQ)
    assert e.value.code == -1   # BA_EINVAL
    simt = ba.Plan(p, impl=ba.IMPL_SIMT)
    with pytest.raises(ba.BranchAttnError) as e:
        ba.branch_attn_bwd(simt, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"], accumulate=True,
                           stages=ba.STAGE_ALL_FUSED)
    assert e.value.code == -2   # BA_EUNSUPPORTED
    plan.check()

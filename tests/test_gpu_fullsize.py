"""GPU parity at the full sizes of the named configurations, in the launch
configuration the benchmark times.  The oracle cannot afford every output at
these sizes, so each case checks (i) exact oracle values on sampled query rows
(O, LSE, dQ are row-local), (ii) dK / dV for ALL keys under a cotangent that is
zero outside the sampled rows (the backward is linear in dO, so the oracle
needs only those rows), and (iii) a closed form that holds at any size: with
q = 0 every visible key weighs the same, so LSE = log(size of the visible set)
for every one of the N + M rows."""
import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W
from paper_2609_07108_b200 import zigzag
from helpers import TOL, assert_close, assert_lse_close, f32, head_slice

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ba():
    from paper_2609_07108_b200 import binding
    assert torch.cuda.is_available()
    return binding


def device_inputs(p, seed):
    """Seeded bf16 inputs drawn on the device (N(0,1)*0.5; cotangent N(0,1)*0.1)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    n, m = p.n_main, p.n_branch
    return {"q_main": draw((n, p.h_q, p.head_dim), 0.5), "q_branch": draw((m, p.h_q, p.head_dim), 0.5),
            "k": draw((n + m, p.h_kv, p.head_dim), 0.5), "v": draw((n + m, p.h_kv, p.head_dim), 0.5),
            "d_o": draw((n + m, p.h_q, p.head_dim), 0.1)}


def sample_rows(p, count, seed, edges=()):
    """Random query rows plus the given main positions (tile / chunk edges) and
    the branch rows anchored there."""
    rng = np.random.default_rng(seed)
    rows = set(rng.choice(p.rows, size=count, replace=False).tolist())
    anchors = p.anchor_idx.astype(np.int64)
    for e in edges:
        if 0 <= e < p.n_main:
            rows.add(int(e))
            b = int(np.searchsorted(anchors, e, side="left"))
            if b < len(anchors) and anchors[b] == e:
                rows.update(range(p.n_main + int(p.branch_offsets[b]), p.n_main + int(p.branch_offsets[b + 1])))
    return np.array(sorted(rows), dtype=np.int64)


def visible_counts(p):
    cu = p.cu_seqlens.astype(np.int64)
    n = p.n_main
    pos = np.arange(n, dtype=np.int64)
    seq = np.searchsorted(cu, pos, side="right") - 1
    main = pos - cu[seq] + 1
    anchors = p.anchor_idx.astype(np.int64)
    aseq = np.searchsorted(cu, anchors, side="right") - 1
    prefix = anchors - cu[aseq] + 1
    blen = np.diff(p.branch_offsets.astype(np.int64))
    local = W._uniform_local_counts(p)
    if local is None:
        local = W.branch_local_counts(p)
    return np.concatenate([main, np.repeat(prefix, blen) + local])


def check_sampled(ba, oracle, p, cp, groups, n_rows, seed, backward=True, edges=(), fused=False):
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    assert plan.impl == ba.IMPL_TC
    t = device_inputs(p, seed)
    rows = sample_rows(p, n_rows, seed, edges)
    rows_t = torch.from_numpy(rows).cuda()
    n = p.n_main
    tol = TOL["bf16"]

    def fwd():
        if cp:
            o, lse, _ = zigzag.forward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], cp)
            return o, lse
        return ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])

    o, lse = fwd()
    plan.check()
    # --- oracle on the sampled rows, selected KV groups
    p2, qh, kvh = head_slice(p, groups)
    qh_t, kvh_t = torch.from_numpy(qh).cuda(), torch.from_numpy(kvh).cuda()
    k_h = f32(t["k"][:, kvh_t])
    v_h = f32(t["v"][:, kvh_t])
    is_b = rows >= n
    q_rows = np.empty((len(rows), len(qh), p.head_dim), dtype=np.float64)
    if (~is_b).any():
        q_rows[~is_b] = f32(t["q_main"][torch.from_numpy(rows[~is_b]).cuda()][:, qh_t])
    if is_b.any():
        q_rows[is_b] = f32(t["q_branch"][torch.from_numpy(rows[is_b] - n).cuda()][:, qh_t])
    ref_o, ref_lse = oracle.forward(p2, q_rows, k_h, v_h, rows=rows)
    assert_close("O (sampled rows)", f32(o[rows_t][:, qh_t]), ref_o, tol)
    assert_lse_close(f32(lse[rows_t][:, qh_t]), ref_lse)

    if backward:
        # cotangent zero outside the sampled rows: dK/dV of every key are then exact from those rows
        d_o = torch.zeros_like(t["d_o"])
        d_o[rows_t] = t["d_o"][rows_t]
        if cp:
            dqm, dqb, dk, dv, _ = zigzag.backward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, d_o, cp,
                                                  fused=fused)
        else:
            dqm, dqb, dk, dv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, d_o)
        plan.check()
        go_rows = f32(d_o[rows_t][:, qh_t])
        ref_dq, ref_dk, ref_dv = oracle.backward(p2, q_rows, k_h, v_h, go_rows, rows=rows)
        dq_all = torch.cat([dqm, dqb], 0)
        assert_close("dQ (sampled rows)", f32(dq_all[rows_t][:, qh_t]), ref_dq, tol)
        assert_close("dK (all keys)", f32(dk[:, kvh_t]), ref_dk, tol)
        assert_close("dV (all keys)", f32(dv[:, kvh_t]), ref_dv, tol)
        # rows with zero cotangent get exactly zero dQ
        other = torch.ones(p.rows, dtype=torch.bool, device="cuda")
        other[rows_t] = False
        assert float(dq_all[other].abs().max()) == 0.0
        del dq_all, dk, dv, dqm, dqb, d_o

    # --- closed form over every row: q = 0  =>  LSE = log |visible set|
    t["q_main"].zero_()
    t["q_branch"].zero_()
    _, lse0 = fwd()
    plan.check()
    want = np.log(visible_counts(p).astype(np.float64))
    got = f32(lse0).astype(np.float64)
    err = np.abs(got - want[:, None]) / np.maximum(1.0, want[:, None])
    assert err.max() <= 1e-3, f"q=0 LSE closed form: max rel err {err.max():.2e} at {np.unravel_index(err.argmax(), err.shape)}"
    torch.cuda.synchronize()


def tile_edges(p):
    cu = p.cu_seqlens.astype(np.int64)
    e = [0, 1, 127, 128, p.n_main - 1, p.n_main - 128]
    for c in cu[1:-1]:
        e += [int(c) - 1, int(c)]
    return e


def test_config2_full_size_forward(ba, oracle):
    p = W.config2()
    check_sampled(ba, oracle, p, cp=0, groups=[0, 7], n_rows=2048, seed=0, backward=False, edges=tile_edges(p))


def test_config3_full_size(ba, oracle):
    p = W.config3()
    check_sampled(ba, oracle, p, cp=0, groups=[1, 6], n_rows=768, seed=1, edges=tile_edges(p))


def test_config4_full_size(ba, oracle):
    p = W.config4()
    check_sampled(ba, oracle, p, cp=0, groups=[2, 5], n_rows=512, seed=2, edges=tile_edges(p))


def test_varlen_ttt_full_size(ba, oracle):
    """The paper's packed variable-length operator-benchmark shape (eight sequences, longest 20,480 tokens)."""
    p = W.varlen_ttt()
    assert p.n_main == 73728 and int(np.diff(p.cu_seqlens).max()) == 20480
    check_sampled(ba, oracle, p, cp=0, groups=[0, 7], n_rows=256, seed=5, edges=tile_edges(p))


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_config5_full_size_zigzag(ba, oracle, fused):
    """256K tokens through the emulated 8-way zigzag layout: partial forward +
    lse_merge, partial backward with fp32 accumulation (dQ kernel + dK/dV kernel, or
    the one-kernel backward that bench.py times)."""
    p = W.config5()
    chunk = p.n_main // 16
    edges = [0, 1, p.n_main - 1]
    for c in range(16):
        edges += [c * chunk, (c + 1) * chunk - 1]
    check_sampled(ba, oracle, p, cp=8, groups=[3], n_rows=160, seed=3, edges=edges, fused=fused)


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_zigzag_equals_monolithic_small(ba, fused):
    """Self-consistency of the two launch configurations on the GPU."""
    p = W.config5(shrink=16)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 4)
    o1, l1 = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])
    o2, l2, _ = zigzag.forward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], 8)
    assert float((o1.float() - o2.float()).abs().max()) <= 2e-2
    assert float((l1 - l2).abs().max()) <= 1e-3
    g1 = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o1, l1, t["d_o"])
    g2 = zigzag.backward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o1, l1, t["d_o"], 8, fused=fused)
    for a, b in zip(g1, g2[:4]):
        assert float((a.float() - b.float()).abs().max()) <= 2e-2
    plan.check()


def test_config3_full_size_dense_cotangent_one_group(ba, oracle):
    """Dense dO at full size: every gradient of one KV-head group of the
    32,768-token DFlash batch against the oracle (all rows, all keys)."""
    p = W.config3()
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 11)
    o, lse = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])
    dqm, dqb, dk, dv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"])
    plan.check()
    p2, qh, kvh = head_slice(p, [4])
    qh_t = torch.from_numpy(qh).cuda()
    q_all = np.concatenate([f32(t["q_main"][:, qh_t]), f32(t["q_branch"][:, qh_t])], 0)
    k_h, v_h = f32(t["k"][:, 4:5]), f32(t["v"][:, 4:5])
    ref_o, ref_lse = oracle.forward(p2, q_all, k_h, v_h)
    ref_dq, ref_dk, ref_dv = oracle.backward(p2, q_all, k_h, v_h, f32(t["d_o"][:, qh_t]))
    tol = TOL["bf16"]
    assert_close("O", f32(o[:, qh_t]), ref_o, tol)
    assert_lse_close(f32(lse[:, qh_t]), ref_lse)
    assert_close("dQ", f32(torch.cat([dqm, dqb], 0)[:, qh_t]), ref_dq, tol)
    assert_close("dK", f32(dk[:, 4:5]), ref_dk, tol)
    assert_close("dV", f32(dv[:, 4:5]), ref_dv, tol)
    # the one-kernel backward on the same dense cotangent (fp32 accumulators, dQ by atomic adds)
    del dqm, dqb, dk, dv
    fq, fb, fk, fv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"],
                                        accumulate=True, stages=ba.STAGE_ALL_FUSED)
    plan.check()
    assert_close("dQ fused", f32(torch.cat([fq, fb], 0)[:, qh_t]), ref_dq, tol)
    assert_close("dK fused", f32(fk[:, 4:5]), ref_dk, tol)
    assert_close("dV fused", f32(fv[:, 4:5]), ref_dv, tol)


def test_results_are_bit_identical_from_run_to_run(ba):
    """Forward and the two-kernel backward: every output element has one owning CTA
    and a fixed summation order.  (The one-kernel backward sums dQ with atomic adds;
    its dK / dV are bit-identical, its dQ only close: test_gpu_fused_bwd.py.)"""
    p = W.config4(shrink=8)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 12)
    runs = []
    for _ in range(2):
        o, lse = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])
        g = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"])
        runs.append((o, lse, *g))
    torch.cuda.synchronize()
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    plan.check()

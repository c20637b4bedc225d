"""GPU parity at the full sizes of the named configurations, in the launch
configuration the benchmark times.  The oracle cannot afford every output at
these sizes, so each case checks
(i)   exact oracle values on sampled query rows (O, LSE, dQ are row-local), gated
      absolutely AND relative to the data (per tensor rel-RMS, per row scaled bound:
      at these lengths the values are far below the absolute bound),
(ii)  dK / dV for ALL keys under a cotangent that is zero outside the sampled rows
      (the backward is linear in dO, so the oracle needs only those rows),
(iii) two closed forms that hold for every one of the N + M rows: with q = 0 every
      visible key weighs the same, so LSE = log(size of the visible set), and with
      V columns holding the bits of the key index, O[bit] = fraction of visible
      keys whose index has that bit set -- a dropped, duplicated or misplaced key
      tile anywhere changes both,
(iv)  sentinel margins around every output buffer."""
import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W
from paper_2609_07108_b200 import zigzag
from helpers import (N_BITS, TOL, Guarded, assert_close, assert_lse_close, expected_bit_fractions, f32, head_slice,
                     index_bit_values, key_viewer_counts, visible_counts)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ba():
    from paper_2609_07108_b200 import binding
    assert torch.cuda.is_available()
    return binding


def device_inputs(p, seed, q_scale=1.0):
    """Seeded bf16 inputs drawn on the device (N(0,1)*0.5; cotangent N(0,1)*0.1)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    n, m = p.n_main, p.n_branch
    return {"q_main": draw((n, p.h_q, p.head_dim), 0.5 * q_scale), "q_branch": draw((m, p.h_q, p.head_dim), 0.5 * q_scale),
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


def check_closed_forms(ba, plan, p, t, cp, ws=None):
    """q = 0, index-coded V, fp32 output: LSE and O of every row against their closed forms."""
    t["q_main"].zero_()
    t["q_branch"].zero_()
    v_code = index_bit_values(p, "cuda")
    if cp:
        o32 = torch.empty((p.rows, p.h_q, p.head_dim), dtype=torch.float32, device="cuda")
        o32, lse0, _ = zigzag.forward(ba, plan, t["q_main"], t["q_branch"], t["k"], v_code, cp, out=o32, ws=ws)
    else:
        o32, lse0 = ba.branch_attn_fwd_partial(plan, t["q_main"], t["q_branch"], t["k"], v_code, (0, p.n_main),
                                               (0, p.num_branches), (0, p.n_main), ba.PART_ALL)
    plan.check()
    want = np.log(visible_counts(p).astype(np.float64))
    got = f32(lse0).astype(np.float64)
    err = np.abs(got - want[:, None])
    print(f"[parity] q=0 LSE closed form, all rows: max abs err {err.max():.3e}")
    assert err.max() <= 2e-5, f"q=0 LSE closed form: max abs err {err.max():.2e} at {np.unravel_index(err.argmax(), err.shape)}"
    grp = p.h_q // p.h_kv
    worst = 0.0
    for g in range(p.h_kv):
        exp = torch.from_numpy(expected_bit_fractions(p, g)).to("cuda", torch.float32)
        for h in range(g * grp, (g + 1) * grp):
            d = (o32[:, h, :N_BITS] - exp).abs()
            e = float(d.max())
            assert e <= 1e-5, (f"index-bit closed form: head {h}: max abs err {e:.2e} at row/bit "
                               f"{np.unravel_index(int(d.argmax()), tuple(d.shape))}")
            worst = max(worst, e)
            e1 = float((o32[:, h, p.head_dim - 1] - 1.0).abs().max())
            assert e1 <= 1e-5, f"constant column: head {h}: {e1:.2e}"
            assert float(o32[:, h, N_BITS:p.head_dim - 1].abs().max()) == 0.0
    print(f"[parity] index-bit closed form, all rows and heads: max abs err {worst:.3e}")
    del o32, v_code
    torch.cuda.synchronize()


# ------------------------------------------------------------ sampled rows

def check_sampled(ba, oracle, p, cp, groups, n_rows, seed, backward=True, edges=(), fused=False, q_scale=1.0,
                  closed_forms=True):
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    assert plan.impl == ba.IMPL_TC
    t = device_inputs(p, seed, q_scale)
    rows = sample_rows(p, n_rows, seed, edges)
    rows_t = torch.from_numpy(rows).cuda()
    n = p.n_main
    tol = TOL["bf16"]
    nk, kk = visible_counts(p), key_viewer_counts(p)
    ws = zigzag.Workspace(ba, plan, cp, backward=backward) if cp else None
    g_o = Guarded((p.rows, p.h_q, p.head_dim), torch.bfloat16)
    g_lse = Guarded((p.rows, p.h_q), torch.float32)

    if cp:
        o, lse, _ = zigzag.forward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], cp, out=g_o.t, lse=g_lse.t, ws=ws)
    else:
        o, lse = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], out=g_o.t, lse=g_lse.t)
    plan.check()
    g_o.check("O")
    g_lse.check("LSE")
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
    assert_close("O (sampled rows)", f32(o[rows_t][:, qh_t]), ref_o, tol, row_keys=nk[rows])
    assert_lse_close(f32(lse[rows_t][:, qh_t]), ref_lse)

    if backward:
        # cotangent zero outside the sampled rows: dK/dV of every key are then exact from those rows
        d_o = torch.zeros_like(t["d_o"])
        d_o[rows_t] = t["d_o"][rows_t]
        shapes = ((p.n_main, p.h_q, p.head_dim), (p.n_branch, p.h_q, p.head_dim),
                  (p.rows, p.h_kv, p.head_dim), (p.rows, p.h_kv, p.head_dim))
        guards = tuple(Guarded(s, torch.bfloat16) for s in shapes)
        if cp:
            ws.outs = tuple(g.t for g in guards)
            dqm, dqb, dk, dv, _ = zigzag.backward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, d_o, cp,
                                                  fused=fused, ws=ws)
        else:
            dqm, dqb, dk, dv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, d_o,
                                                  grads=tuple(g.t for g in guards),
                                                  stages=ba.STAGE_ALL_FUSED if fused else ba.STAGE_ALL)
        plan.check()
        for name, g in zip(("dQ_main", "dQ_branch", "dK", "dV"), guards):
            g.check(name)
        go_rows = f32(d_o[rows_t][:, qh_t])
        ref_dq, ref_dk, ref_dv = oracle.backward(p2, q_rows, k_h, v_h, go_rows, rows=rows)
        dq_all = torch.cat([dqm, dqb], 0)
        # sharp scores: near one-hot rows make dS a cancellation, so dQ and dK keep the absolute bound only
        rel = q_scale == 1.0
        assert_close("dQ (sampled rows)", f32(dq_all[rows_t][:, qh_t]), ref_dq, tol, row_keys=nk[rows], relative=rel)
        assert_close("dK (all keys)", f32(dk[:, kvh_t]), ref_dk, tol, row_keys=kk, relative=rel)
        assert_close("dV (all keys)", f32(dv[:, kvh_t]), ref_dv, tol, row_keys=kk)
        # rows with zero cotangent get exactly zero dQ
        other = torch.ones(p.rows, dtype=torch.bool, device="cuda")
        other[rows_t] = False
        assert float(dq_all[other].abs().max()) == 0.0
        del dq_all, dk, dv, dqm, dqb, d_o, guards
        if ws is not None:
            ws.outs = ws.grads = None
    del g_o, g_lse, o, lse
    if closed_forms:
        check_closed_forms(ba, plan, p, t, cp, ws=ws)
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


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_config4_full_size(ba, oracle, fused):
    p = W.config4()
    check_sampled(ba, oracle, p, cp=0, groups=[2, 5], n_rows=512, seed=2, edges=tile_edges(p), fused=fused)


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_varlen_ttt_full_size(ba, oracle, fused):
    """The paper's packed variable-length operator-benchmark shape (eight sequences, longest 20,480 tokens)."""
    p = W.varlen_ttt()
    assert p.n_main == 73728 and int(np.diff(p.cu_seqlens).max()) == 20480
    check_sampled(ba, oracle, p, cp=0, groups=[0, 7], n_rows=256, seed=5, edges=tile_edges(p), fused=fused)


def config5_edges(p):
    chunk = p.n_main // 16
    edges = [0, 1, p.n_main - 1]
    for c in range(16):
        edges += [c * chunk, (c + 1) * chunk - 1]
    return edges


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_config5_full_size_zigzag(ba, oracle, fused):
    """256K tokens through the emulated 8-way zigzag layout: partial forward +
    lse_merge, partial backward with fp32 accumulation (dQ kernel + dK/dV kernel, or
    the one-kernel backward that bench.py times)."""
    p = W.config5()
    # the benchmarked form (one-kernel backward) gets the larger sample and the closed forms over all rows
    check_sampled(ba, oracle, p, cp=8, groups=[0, 3, 7] if fused else [3, 7], n_rows=384 if fused else 256, seed=3,
                  edges=config5_edges(p), fused=fused, closed_forms=fused)


def test_config5_full_size_sharp_scores(ba, oracle):
    """Queries scaled by 8 (score spread 2, the running maximum moves and the lazy
    rescale path of the forward is taken) at 256K tokens, benchmark configuration."""
    p = W.config5()
    check_sampled(ba, oracle, p, cp=8, groups=[5], n_rows=128, seed=21, edges=config5_edges(p), fused=True,
                  q_scale=8.0, closed_forms=False)


@pytest.mark.parametrize("fused", [False, True], ids=["split_bwd", "fused_bwd"])
def test_zigzag_equals_monolithic_small(ba, fused):
    """Self-consistency of the two launch configurations on the GPU."""
    p = W.config5(shrink=16)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 4)
    o1, l1 = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])
    o2, l2, _ = zigzag.forward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], 8)
    assert_close("O zigzag vs monolithic", f32(o2), f32(o1).astype(np.float64), 2e-2)
    assert float((l1 - l2).abs().max()) <= 1e-5
    g1 = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o1, l1, t["d_o"])
    g2 = zigzag.backward(ba, plan, t["q_main"], t["q_branch"], t["k"], t["v"], o1, l1, t["d_o"], 8, fused=fused)
    for name, a, b in zip(("dQm", "dQb", "dK", "dV"), g1, g2[:4]):
        assert_close(name + " zigzag vs monolithic", f32(b), f32(a).astype(np.float64), 2e-2)
    plan.check()


def test_config3_full_size_dense_cotangent_one_group(ba, oracle):
    """Dense dO at full size: every gradient of one KV-head group of the
    32,768-token DFlash batch against the oracle (all rows, all keys)."""
    p = W.config3()
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 11)
    n = p.n_main
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
    nk, kk = visible_counts(p), key_viewer_counts(p)
    assert_close("O", f32(o[:, qh_t]), ref_o, tol, row_keys=nk)
    assert_lse_close(f32(lse[:, qh_t]), ref_lse)
    assert_close("dQ", f32(torch.cat([dqm, dqb], 0)[:, qh_t]), ref_dq, tol, row_keys=nk)
    assert_close("dK", f32(dk[:, 4:5]), ref_dk, tol, row_keys=kk)
    assert_close("dV", f32(dv[:, 4:5]), ref_dv, tol, row_keys=kk)
    # the one-kernel backward on the same dense cotangent (fp32 accumulators, dQ by atomic adds)
    del dqm, dqb, dk, dv
    fq, fb, fk, fv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"],
                                        accumulate=True, stages=ba.STAGE_ALL_FUSED)
    plan.check()
    assert_close("dQ fused", f32(torch.cat([fq, fb], 0)[:, qh_t]), ref_dq, tol, row_keys=nk)
    assert_close("dK fused", f32(fk[:, 4:5]), ref_dk, tol, row_keys=kk)
    assert_close("dV fused", f32(fv[:, 4:5]), ref_dv, tol, row_keys=kk)


def test_long_chain_dense_cotangent_fused_backward(ba, oracle):
    """One 16,384-token sequence with a depth-3 chain at every position, one KV group,
    dense dO: in the one-kernel backward 128 key tiles add into every late dQ row with
    atomic adds, and all of them are compared (every row, every key)."""
    n = 16384
    p = W.Problem(W.cu_from_lengths([n]), np.arange(n, dtype=np.int32), W.uniform_branch_offsets(n, 3), W.CHAIN, None,
                  2, 1, 128, name="long_chain_16k_one_group")
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    t = device_inputs(p, 17)
    o, lse = ba.branch_attn_fwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"])
    fq, fb, fk, fv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"],
                                        accumulate=True, stages=ba.STAGE_ALL_FUSED)
    gq, gb, gk, gv = ba.branch_attn_bwd(plan, t["q_main"], t["q_branch"], t["k"], t["v"], o, lse, t["d_o"],
                                        stages=ba.STAGE_ALL_FUSED)
    plan.check()
    q_all = np.concatenate([f32(t["q_main"]), f32(t["q_branch"])], 0)
    k_h, v_h = f32(t["k"]), f32(t["v"])
    ref_o, ref_lse = oracle.forward(p, q_all, k_h, v_h)
    ref_dq, ref_dk, ref_dv = oracle.backward(p, q_all, k_h, v_h, f32(t["d_o"]))
    tol = TOL["bf16"]
    nk, kk = visible_counts(p), key_viewer_counts(p)
    assert_close("O", f32(o), ref_o, tol, row_keys=nk)
    assert_lse_close(f32(lse), ref_lse)
    assert_close("dQ fused fp32", f32(torch.cat([fq, fb], 0)), ref_dq, tol, row_keys=nk)
    assert_close("dK fused fp32", f32(fk), ref_dk, tol, row_keys=kk)
    assert_close("dV fused fp32", f32(fv), ref_dv, tol, row_keys=kk)
    assert_close("dQ fused bf16", f32(torch.cat([gq, gb], 0)), ref_dq, tol, row_keys=nk)
    assert_close("dK fused bf16", f32(gk), ref_dk, tol, row_keys=kk)
    assert_close("dV fused bf16", f32(gv), ref_dv, tol, row_keys=kk)


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

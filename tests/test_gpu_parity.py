"""GPU parity: the CUDA library (through its C ABI / ctypes binding) against
the fp64 CPU oracle, element by element on the same seeded inputs."""
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


def impls_for(ba, p):
    out = [ba.IMPL_SIMT]
    if p.dtype == "bf16" and p.head_dim == 128:
        out.append(ba.IMPL_TC)
    return out


def check_full(ba, oracle, p, seed=0, std=1.0, impl=None, backward=True, groups=None, q_main=True,
               mutate=None, relative_grads=True):
    """Monolithic forward (+ backward) against the oracle on all rows.
    `relative_grads=False`: inputs with near one-hot softmax rows, where dS = P (dP - delta)
    is a cancellation and only the absolute bound applies to dQ and dK."""
    t = W.make_tensors(p, seed=seed, std=std)
    if mutate:
        mutate(t)
    d = to_dev(p, t)
    plan = ba.Plan(p, impl=impl if impl is not None else ba.IMPL_AUTO)
    assert plan.pairs == W.useful_pairs(p)
    n = p.n_main
    qm = d["q_main"] if q_main else None
    o, lse = ba.branch_attn_fwd(plan, qm, d["q_branch"], d["k"], d["v"])
    plan.check()
    ref = oracle_fwd_bwd(oracle, p, t, groups=groups, backward=backward)
    qh, kvh = ref["q_heads"], ref["kv_heads"]
    tol = TOL[p.dtype]
    lo = 0 if q_main else n
    assert_close("O", f32(o)[lo:, qh], ref["o"][lo:], tol)
    assert_lse_close(f32(lse)[lo:, qh], ref["lse"][lo:])
    if not backward:
        return
    if not q_main:
        # gradients of the branch rows only: cotangent of main rows is zero
        t["d_o"][:n] = 0
        d["d_o"][:n] = 0
        # the forward left main rows of O/LSE unwritten; the backward must not read them
        ref = oracle_fwd_bwd(oracle, p, t, groups=groups)
    dqm, dqb, dk, dv = ba.branch_attn_bwd(plan, qm, d["q_branch"], d["k"], d["v"], o, lse, d["d_o"])
    nk, kk = visible_counts(p), key_viewer_counts(p)
    if q_main:
        assert_close("dQ_main", f32(dqm)[:, qh], ref["dq"][:n], tol, row_keys=nk[:n], relative=relative_grads)
    assert_close("dQ_branch", f32(dqb)[:, qh], ref["dq"][n:], tol, row_keys=nk[n:], relative=relative_grads)
    assert_close("dK", f32(dk)[:, kvh], ref["dk"], tol, row_keys=kk, relative=relative_grads)
    assert_close("dV", f32(dv)[:, kvh], ref["dv"], tol, row_keys=kk)
    plan.check()


# ------------------------------------------------------------------ metadata

def test_plan_counts_pairs_and_rejects_bad_metadata(ba):
    for kind in (W.CHAIN, W.BLOCK, W.TREE):
        p = W.odd_shapes(kind)
        assert ba.Plan(p).pairs == W.useful_pairs(p)
    p = W.config1()
    assert ba.Plan(p).pairs == 126184

    def expect_meta_error(q):
        with pytest.raises(ba.BranchAttnError) as e:
            ba.Plan(q)
        assert e.value.code == -4, e.value

    import copy
    q = copy.copy(W.odd_shapes(W.CHAIN)); q.anchor_idx = q.anchor_idx.copy(); q.anchor_idx[3] = 0
    expect_meta_error(q)                                      # anchors not sorted
    q = copy.copy(W.odd_shapes(W.CHAIN)); q.anchor_idx = q.anchor_idx.copy(); q.anchor_idx[-1] = 405
    expect_meta_error(q)                                      # anchor == N
    q = copy.copy(W.odd_shapes(W.TREE)); q.parent = q.parent.copy(); q.parent[5] = 7
    expect_meta_error(q)                                      # parent[i] >= i
    q = copy.copy(W.odd_shapes(W.CHAIN)); q.cu_seqlens = q.cu_seqlens.copy(); q.cu_seqlens[2] = 0
    expect_meta_error(q)                                      # cu_seqlens decreasing
    q = copy.copy(W.odd_shapes(W.BLOCK))
    q.branch_offsets = np.array([0, 70] + [70 + 3 * i for i in range(1, 12)], dtype=np.int32)
    expect_meta_error(q)                                      # a branch of 70 tokens
    torch.cuda.synchronize()


def test_noop_cases_through_the_raw_c_abi(ba):
    """A = 0 with NULL branch arrays and N = 0 are valid problems: the plan is built without
    touching the absent arrays and every data call is a no-op that returns BA_OK.  Called
    through ctypes directly (the Plan class would hide the NULL pointers)."""
    import ctypes as C
    lib = ba._lib()

    def create(**kw):
        prob = ba._Problem(h_q=4, h_kv=2, head_dim=128, dtype=ba.BA_BF16, softmax_scale=0.0, impl=ba.IMPL_AUTO,
                           uniform_len=0, anchor_idx=None, branch_offsets=None, parent=None, **kw)
        nbytes = lib.ba_plan_bytes(C.byref(prob))
        assert nbytes > 0
        mem = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        handle = C.c_void_p()
        rc = lib.ba_plan_create(C.byref(prob), ba._p(mem), nbytes, ba._stream(), C.byref(handle))
        return rc, handle, mem

    cu = torch.tensor([0, 100, 300], dtype=torch.int32, device="cuda")
    for kind in (W.CHAIN, W.BLOCK, W.TREE):
        rc, handle, mem = create(n_main=300, n_branch=0, num_seqs=2, num_branches=0, mask_kind=kind,
                                 cu_seqlens=cu.data_ptr())
        assert rc == 0, rc
        assert lib.ba_plan_pairs(handle) == 100 * 101 // 2 + 200 * 201 // 2
        # q = 0 forward with q_branch = NULL: LSE = log(position in the sequence + 1)
        q = torch.zeros((300, 4, 128), dtype=torch.bfloat16, device="cuda")
        kv = torch.randn((300, 2, 128), device="cuda").to(torch.bfloat16)
        o = torch.empty_like(q)
        lse = torch.empty((300, 4), dtype=torch.float32, device="cuda")
        rc = lib.branch_attn_fwd(handle, ba._p(q), None, ba._p(kv), ba._p(kv), ba._p(o), ba._p(lse), None, 0, ba._stream())
        assert rc == 0, rc
        assert lib.ba_plan_check(handle, ba._stream()) == 0
        want = np.log(np.concatenate([np.arange(1, 101), np.arange(1, 201)]).astype(np.float64))
        assert np.abs(f32(lse) - want[:, None]).max() < 1e-5
        # backward with dQ_branch = NULL
        ws_bytes = lib.ba_workspace_bytes(handle, ba.OP_BWD)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
        g = [torch.empty_like(q), torch.empty_like(kv), torch.empty_like(kv)]
        rc = lib.branch_attn_bwd(handle, ba._p(q), None, ba._p(kv), ba._p(kv), ba._p(o), ba._p(lse), ba._p(q),
                                 0, 300, 0, 0, 0, 300, ba.PART_ALL, 0, ba._p(g[0]), None, ba._p(g[1]), ba._p(g[2]),
                                 ba._p(ws), ws_bytes, ba._stream())
        assert rc == 0, rc
        assert lib.ba_plan_check(handle, ba._stream()) == 0
        assert float(g[0].abs().max()) == 0.0 and float(g[2].abs().max()) == 0.0     # dO = 0
        lib.ba_plan_destroy(handle)

    # N = 0: one empty sequence, or no sequence at all (cu_seqlens NULL)
    cu0 = torch.zeros(2, dtype=torch.int32, device="cuda")
    for kw in (dict(num_seqs=1, cu_seqlens=cu0.data_ptr()), dict(num_seqs=0, cu_seqlens=None)):
        rc, handle, mem = create(n_main=0, n_branch=0, num_branches=0, mask_kind=W.CHAIN, **kw)
        assert rc == 0, rc
        assert lib.ba_plan_pairs(handle) == 0
        assert lib.branch_attn_fwd(handle, None, None, None, None, None, None, None, 0, ba._stream()) == 0
        assert lib.branch_attn_fwd_partial(handle, None, None, None, None, 0, 0, 0, 0, 0, 0, ba.PART_ALL, None, None,
                                           None, 0, ba._stream()) == 0
        assert lib.branch_attn_bwd(handle, None, None, None, None, None, None, None, 0, 0, 0, 0, 0, 0, ba.PART_ALL, 0,
                                   None, None, None, None, None, 0, ba._stream()) == 0
        assert lib.ba_plan_check(handle, ba._stream()) == 0
        lib.ba_plan_destroy(handle)
    # branches declared but their arrays missing: refused on the host
    rc, handle, mem = create(n_main=300, n_branch=3, num_seqs=2, num_branches=1, mask_kind=W.CHAIN,
                             cu_seqlens=cu.data_ptr())
    assert rc == -1
    torch.cuda.synchronize()


def test_bounded_wait_runs_out_and_the_library_carries_on(ba, oracle):
    """A wait on a barrier nobody signals gives up after its cycle limit: the kernel returns,
    ba_plan_check reports BA_ETIMEOUT once and clears it, and the next calls are correct."""
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16")
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    plan.check()
    plan.selftest_bounded_wait(100000)
    with pytest.raises(ba.BranchAttnError) as e:
        plan.check()
    assert e.value.code == -6          # BA_ETIMEOUT
    plan.check()                       # cleared by the check that reported it
    lib = ba._lib()
    assert lib.ba_selftest_bounded_wait(plan.handle, 0, ba._stream()) == -1           # limits outside (0, 1e8] refused
    assert lib.ba_selftest_bounded_wait(plan.handle, 10**9, ba._stream()) == -1
    check_full(ba, oracle, p, seed=3, std=0.5, impl=ba.IMPL_TC)                        # the context is intact


def test_binding_refuses_tensors_the_kernels_could_not_address(ba):
    """The library sees raw pointers: a strided view, a wrong dtype, shape or device must be
    stopped in the binding, before any kernel could read or write outside an allocation."""
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16")
    d = to_dev(p, W.make_tensors(p, seed=2, std=0.5))
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
    wide = torch.zeros((p.rows, 2 * p.h_kv, p.head_dim), dtype=torch.bfloat16, device="cuda")
    cases = [
        dict(k=wide[:, ::2]),                                   # strided view of the right shape
        dict(k=d["k"].float()),                                 # wrong dtype
        dict(k=d["k"][:-1]),                                    # one row short
        dict(q_branch=d["q_branch"].cpu()),                     # wrong device
        dict(v=None),                                           # missing
    ]
    for bad in cases:
        args = dict(q_main=d["q_main"], q_branch=d["q_branch"], k=d["k"], v=d["v"])
        args.update(bad)
        with pytest.raises(ValueError):
            ba.branch_attn_fwd(plan, args["q_main"], args["q_branch"], args["k"], args["v"])
        with pytest.raises(ValueError):
            ba.branch_attn_bwd(plan, args["q_main"], args["q_branch"], args["k"], args["v"], o, lse, d["d_o"])
    with pytest.raises(ValueError):                              # outputs are checked too
        ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"], out=o[:, :, :64])
    with pytest.raises(ValueError):
        ba.branch_attn_bwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse[:, :2], d["d_o"])
    with pytest.raises(ValueError):
        ba.ba_finalize_grads(torch.zeros((4, 8), device="cuda")[:, ::2])
    plan.check()


# --------------------------------------------------------------------- merge

def test_lse_merge_matches_oracle(ba, oracle):
    rng = np.random.default_rng(0)
    rows, h, d = 1000, 3, 128
    oa, ob = rng.standard_normal((2, rows, h, d)).astype(np.float32)
    la, lb = (rng.standard_normal((2, rows, h)) * 5).astype(np.float32)
    la[::7] = -np.inf
    lb[::5] = -np.inf                                        # rows 0, 35, ... have both empty
    lb[3] = la[3] + 60.0
    want_o, want_l = oracle.lse_merge(oa, la, ob, lb)
    toa, tob, tla, tlb = (torch.from_numpy(x).cuda() for x in (oa, ob, la, lb))
    o, l = ba.lse_merge(toa, tla, tob, tlb)
    assert_close("O", f32(o), want_o, 1e-5)
    assert_lse_close(f32(l), want_l)
    assert np.abs(f32(l)[~np.isneginf(want_l)] - want_l[~np.isneginf(want_l)]).max() < 1e-5
    ob16, _ = ba.lse_merge(toa, tla, tob, tlb, out_dtype=torch.bfloat16)
    assert_close("O bf16", f32(ob16), want_o, 2e-2)
    # in place into (o_a, lse_a); d = 64 variant
    oa64, ob64 = toa[..., :64].contiguous(), tob[..., :64].contiguous()
    w_o, w_l = oracle.lse_merge(oa[..., :64], la, ob[..., :64], lb)
    la_c = tla.clone()
    ba.lse_merge(oa64, la_c, ob64, tlb, out=oa64, lse_out=la_c)
    assert_close("O in place", f32(oa64), w_o, 1e-5)
    assert_lse_close(f32(la_c), w_l)


# ----------------------------------------------------------- the five configs

def test_config1_tiny_fp32_full(ba, oracle):
    check_full(ba, oracle, W.config1(), seed=0, std=1.0)


@pytest.mark.parametrize("kind", [W.CHAIN, W.BLOCK, W.TREE])
@pytest.mark.parametrize("dtype,d", [("fp32", 64), ("fp32", 128), ("bf16", 64), ("bf16", 128)])
def test_odd_shapes_all_masks(ba, oracle, kind, dtype, d):
    p = W.odd_shapes(kind, head_dim=d, dtype=dtype)
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=3, std=1.0 if dtype == "fp32" else 0.5, impl=impl)


@pytest.mark.parametrize("kind", [W.CHAIN, W.TREE])
def test_branch_queries_only(ba, oracle, kind):
    p = W.odd_shapes(kind, head_dim=128, dtype="bf16")
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=4, std=0.5, impl=impl, q_main=False)


@pytest.mark.parametrize("cfg,shrink", [(2, 8), (3, 16), (4, 16), (5, 128), (6, 64)])
def test_shrunken_configs_bf16(ba, oracle, cfg, shrink):
    p = W.CONFIGS[cfg](shrink)
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=0, std=0.5, impl=impl, backward=(cfg != 2), groups=[0, p.h_kv - 1])


@pytest.mark.parametrize("h_q,h_kv", [(2, 2), (3, 1), (5, 1), (6, 2)])
def test_head_group_sizes(ba, oracle, h_q, h_kv):
    """Query heads per KV head 1, 3, 5 (an odd head is left over in the head-pair
    work split of the tensor-core kernels) and 3 again with two KV heads."""
    p = W.odd_shapes(W.BLOCK, head_dim=128, dtype="bf16", h_q=h_q, h_kv=h_kv)
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=8, std=0.5, impl=impl)


def test_branch_part_as_its_own_partial_merged_last(ba, oracle):
    """The paper's literal order: main-sequence partials over key chunks first,
    the locally computed branch component merged at the end (Eq. lse-merge)."""
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16")
    t = W.make_tensors(p, seed=9, std=0.5)
    d = to_dev(p, t)
    n, a = p.n_main, p.num_branches
    for impl in impls_for(ba, p):
        plan = ba.Plan(p, impl=impl)
        o_full, lse_full = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
        acc = None
        for kv, parts in (((0, 200), ba.PART_MAIN), ((200, n), ba.PART_MAIN), ((0, 0), ba.PART_BRANCH)):
            part = ba.branch_attn_fwd_partial(plan, d["q_main"], d["q_branch"], d["k"], d["v"], (0, n), (0, a), kv, parts)
            acc = part if acc is None else ba.lse_merge(acc[0], acc[1], part[0], part[1])
        assert_close("merged O", f32(acc[0]), f32(o_full).astype(np.float64), TOL["bf16"])
        assert_lse_close(f32(acc[1]), f32(lse_full).astype(np.float64))
        ref = oracle_fwd_bwd(oracle, p, t, backward=False)
        assert_close("merged O vs oracle", f32(acc[0]), ref["o"], TOL["bf16"])
        plan.check()


def test_no_branches(ba, oracle):
    cu = W.cu_from_lengths([100, 300, 29])
    p = W.Problem(cu, np.zeros(0, np.int32), np.zeros(1, np.int32), W.CHAIN, None, 4, 2, 128, dtype="bf16")
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=5, std=0.5, impl=impl)


# ----------------------------------------------------------------- stress

def _sharp(t):
    t["q_main"] *= 8
    t["q_branch"] *= 8


def _offset(t):
    rng = np.random.default_rng(99)
    c = W.round_to_bf16(rng.standard_normal(t["k"].shape[-1]).astype(np.float32) * 4)
    t["k"] += c
    t["k"][:] = W.round_to_bf16(t["k"])


def _late_outlier(t):
    t["k"][400] = W.round_to_bf16(t["q_main"][404, 0] * 3)   # one key aligned with a late query


@pytest.mark.parametrize("mutate", [_sharp, _offset, _late_outlier])
def test_stress_inputs(ba, oracle, mutate):
    p = W.odd_shapes(W.CHAIN, head_dim=128, dtype="bf16", h_q=4, h_kv=2)
    for impl in impls_for(ba, p):
        check_full(ba, oracle, p, seed=6, std=0.5, impl=impl, mutate=mutate,
                   relative_grads=False)


# ------------------------------------------------------- partial mode + merge

@pytest.mark.parametrize("dtype,d", [("fp32", 64), ("bf16", 128)])
def test_partial_chunks_merge_to_monolithic(ba, oracle, dtype, d):
    p = W.odd_shapes(W.TREE, head_dim=d, dtype=dtype)
    t = W.make_tensors(p, seed=7, std=0.5)
    dv_ = to_dev(p, t)
    n, a = p.n_main, p.num_branches
    tol = TOL[dtype]
    for impl in impls_for(ba, p):
        plan = ba.Plan(p, impl=impl)
        o_full, lse_full = ba.branch_attn_fwd(plan, dv_["q_main"], dv_["q_branch"], dv_["k"], dv_["v"])
        # query block: main rows [10, 300), branches [2, 11); key chunks with ragged edges
        qm, br = (10, 300), (2, 11)
        t0, t1 = plan.token_range(*br)
        rows = np.concatenate([np.arange(*qm), n + np.arange(t0, t1)])
        chunks = [(0, 17), (17, 18), (18, 150), (150, 150), (150, n)]
        acc = None
        for i, kv in enumerate(chunks):
            parts = ba.PART_MAIN | (ba.PART_BRANCH if i == 2 else 0)
            o_p, l_p = ba.branch_attn_fwd_partial(plan, dv_["q_main"], dv_["q_branch"], dv_["k"], dv_["v"],
                                                  qm, br, kv, parts)
            ref = oracle_fwd_bwd(oracle, p, t, rows=rows, backward=False, parts=parts, kv_range=kv)
            assert_close(f"O_part{i}", f32(o_p), ref["o"], tol)
            assert_lse_close(f32(l_p), ref["lse"])
            acc = (o_p, l_p) if acc is None else ba.lse_merge(acc[0], acc[1], o_p, l_p, out=acc[0], lse_out=acc[1])
        rows_t = torch.from_numpy(rows).cuda()
        assert_close("merged O", f32(acc[0]), f32(o_full[rows_t]).astype(np.float64), tol)
        assert_lse_close(f32(acc[1]), f32(lse_full[rows_t]).astype(np.float64))

        # backward: per-chunk accumulation equals the monolithic gradient
        mono = ba.branch_attn_bwd(plan, dv_["q_main"], dv_["q_branch"], dv_["k"], dv_["v"], o_full, lse_full,
                                  dv_["d_o"])
        grads = None
        for i, kv in enumerate(chunks):
            parts = ba.PART_MAIN | (ba.PART_BRANCH if i == 2 else 0)
            for qmr, brr in (((0, 100), (0, 5)), ((100, n), (5, a))):
                grads = ba.branch_attn_bwd(plan, dv_["q_main"], dv_["q_branch"], dv_["k"], dv_["v"], o_full,
                                           lse_full, dv_["d_o"], qm_range=qmr, br_range=brr, kv_range=kv,
                                           parts=parts, accumulate=True, grads=grads)
        ref = oracle_fwd_bwd(oracle, p, t)
        want = (ref["dq"][:n], ref["dq"][n:], ref["dk"], ref["dv"])
        nk, kk = visible_counts(p), key_viewer_counts(p)
        for name, g_acc, g_mono, w, rk in zip(("dQm", "dQb", "dK", "dV"), grads, mono, want, (nk[:n], nk[n:], kk, kk)):
            assert_close(name + " accumulated", f32(g_acc), w, tol, row_keys=rk)
            fin = ba.ba_finalize_grads(g_acc, dtype=plan.torch_dtype)
            assert_close(name + " finalized", f32(fin), w, tol, row_keys=rk)
            assert_close(name + " monolithic", f32(g_mono), w, tol, row_keys=rk)
    torch.cuda.synchronize()


def test_partial_forward_merged_in_the_epilogue(ba, oracle):
    """Ring steps whose (O, LSE) are merged into the running result inside the kernel
    (Eq. lse-merge in the epilogue) against the oracle's monolithic forward, on chunks
    that leave rows without any visible key, then give them some."""
    p = W.odd_shapes(W.TREE, head_dim=128, dtype="bf16")
    t = W.make_tensors(p, seed=13, std=0.5)
    d = to_dev(p, t)
    n, a = p.n_main, p.num_branches
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    ref = oracle_fwd_bwd(oracle, p, t, backward=False)
    for qm, br in (((0, n), (0, a)), ((37, 300), (2, a - 1))):
        t0, t1 = plan.token_range(*br)
        rows = np.concatenate([np.arange(qm[0], qm[1]), n + np.arange(t0, t1)])
        acc = None
        # the branch part first or last, an empty chunk, one-key chunks
        for order in (0, 1):
            chunks = [(150, n), (0, 17), (17, 18), (150, 150), (18, 150)]
            acc = None
            for i, kv in enumerate(chunks):
                parts = ba.PART_MAIN | (ba.PART_BRANCH if i == (0 if order == 0 else 4) else 0)
                if acc is None:
                    acc = ba.branch_attn_fwd_partial(plan, d["q_main"], d["q_branch"], d["k"], d["v"], qm, br, kv, parts)
                else:
                    ba.branch_attn_fwd_partial_merge(plan, d["q_main"], d["q_branch"], d["k"], d["v"], qm, br, kv,
                                                     parts, acc[0], acc[1])
            plan.check()
            assert_close(f"merged O (order {order})", f32(acc[0]), ref["o"][rows], TOL["bf16"])
            assert_lse_close(f32(acc[1]), ref["lse"][rows])
    # a key set that no selected row sees at all: -inf and zeros, and merging into it works
    acc = ba.branch_attn_fwd_partial(plan, d["q_main"], d["q_branch"], d["k"], d["v"], (0, 10), (0, 0), (200, n), ba.PART_MAIN)
    assert torch.isneginf(acc[1]).all() and float(acc[0].abs().max()) == 0.0
    ba.branch_attn_fwd_partial_merge(plan, d["q_main"], d["q_branch"], d["k"], d["v"], (0, 10), (0, 0), (0, 200),
                                     ba.PART_MAIN, acc[0], acc[1])
    plan.check()
    assert_close("merge into an empty result", f32(acc[0]), ref["o"][:10], TOL["bf16"])
    assert_lse_close(f32(acc[1]), ref["lse"][:10])
    simt = ba.Plan(p, impl=ba.IMPL_SIMT)
    with pytest.raises(ba.BranchAttnError) as e:
        ba.branch_attn_fwd_partial_merge(simt, d["q_main"], d["q_branch"], d["k"], d["v"], (0, 10), (0, 0), (0, 200),
                                         ba.PART_MAIN, acc[0], acc[1])
    assert e.value.code == -2   # BA_EUNSUPPORTED

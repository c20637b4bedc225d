"""CPU-only checks: workload generators, the zigzag schedule, and that the
C-ABI library loads and exports every symbol its header declares."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_07108_b200 import workloads as W
from paper_2609_07108_b200 import zigzag

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_named_configs_have_the_stated_shapes():
    p1 = W.config1()
    assert (p1.n_main, p1.num_branches, p1.n_branch, p1.h_q, p1.h_kv, p1.head_dim) == (640, 40, 120, 4, 4, 64)
    assert W.useful_pairs(p1) == 126184
    p2 = W.config2()
    assert p2.n_main == 8192 and p2.num_seqs == 8 and p2.n_branch == 3 * 8192 and p2.kind == W.CHAIN
    p3 = W.config3()
    assert p3.n_main == 32768 and p3.num_seqs == 16 and p3.num_branches == 512 and p3.n_branch == 8192
    assert len(np.unique(p3.anchor_idx)) == 512 and (np.diff(p3.anchor_idx) > 0).all()
    p4 = W.config4()
    assert p4.n_main == 65536 and p4.num_branches == 1024 and p4.n_branch == 31 * 1024
    par = p4.parent.reshape(1024, 31)
    assert (par[:, 0] == -1).all() and (par[:, 1:] < np.arange(1, 31)[None]).all() and (par[:, 1:] >= 0).all()
    depth = np.ones((1024, 31), dtype=int)
    for i in range(1, 31):
        depth[:, i] = depth[np.arange(1024), par[:, i]] + 1
    assert depth.max() == 6
    p5 = W.config5()
    assert p5.n_main == 262144 and p5.rows == 1048576
    assert W.useful_pairs(p5) == 137441050624
    for p in (p2, p3, p4):
        lens = np.diff(p.cu_seqlens)
        assert lens.min() >= 16 and lens.sum() == p.n_main
    # the shape of the paper's packed variable-length operator benchmark (Section 4.4):
    # longest sequence 20,480 tokens, padded-to-longest size about 2.25x the real size
    pv = W.varlen_ttt()
    lens = np.diff(pv.cu_seqlens)
    assert lens.max() == 20480 and pv.n_main == 73728 and pv.n_branch == 3 * 73728 and pv.kind == W.CHAIN
    assert 2.1 < len(lens) * lens.max() / lens.sum() < 2.3
    assert W.useful_pairs(pv) == 1871249408


def test_generators_are_seeded_and_bf16_exact():
    p = W.config2(shrink=32)
    a, b = W.make_tensors(p, seed=3, std=0.5), W.make_tensors(p, seed=3, std=0.5)
    for k in a:
        assert np.array_equal(a[k], b[k])
        assert np.array_equal(W.round_to_bf16(a[k]), a[k])            # already bf16 values
        assert np.array_equal(W.bf16_bits_to_f32(W.bf16_bits(a[k])), a[k])
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0e-40, 65504.0], dtype=np.float32)
    r = W.round_to_bf16(x)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.015625)  # ties to even, both ways


def test_zigzag_schedule_is_balanced_and_complete():
    p = W.config5(shrink=64)
    cp = 8
    blocks = zigzag.schedule(p, cp)
    nc = 2 * cp
    # every (q chunk, kv chunk <= q chunk) pair exactly once
    seen = sorted((b.q_chunk, b.kv_chunk) for b in blocks)
    assert seen == sorted((q, k) for q in range(nc) for k in range(q + 1))
    # each rank: 15 full blocks + 2 diagonal blocks ("load-balanced zigzag")
    for r in range(cp):
        mine = [b for b in blocks if b.rank == r]
        assert sum(b.diagonal for b in mine) == 2 and len(mine) == nc - 1 + 2
        assert {b.q_chunk for b in mine} == set(zigzag.rank_chunks(r, cp))
    # the branch-local part is computed exactly once per q chunk, in the local step
    for q in range(nc):
        bp = [b for b in blocks if b.q_chunk == q and b.branch_part]
        assert len(bp) == 1 and bp[0].step == 0 and bp[0].kv_chunk == q
    # ring step s of rank r reads only the chunks of rank (r - s) mod C
    for b in blocks:
        assert b.kv_chunk in zigzag.rank_chunks((b.rank - b.step) % cp, cp)
    # useful pairs per rank: equal up to the in-chunk (diagonal) remainder
    per = zigzag.pairs_per_rank(p, cp)
    assert sum(per) + 6 * p.n_main == W.useful_pairs(p)               # + branch-local pairs (1+2+3)
    assert max(per) - min(per) == 0 or (max(per) - min(per)) / max(per) < 1e-2


def test_library_exports_every_declared_symbol():
    from paper_2609_07108_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    header = open(os.path.join(ROOT, "include", "branch_attn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    header = re.sub(r"^\s*#.*$", "", header, flags=re.M)      # preprocessor lines declare no symbols
    names = re.findall(r"\b([A-Za-z_][A-Za-z0-9_]*)\s*\([^;{]*\)\s*;", header)
    assert {"branch_attn_fwd", "branch_attn_fwd_partial", "lse_merge", "branch_attn_bwd",
            "ba_plan_create", "ba_plan_bytes", "ba_finalize_grads"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in the header but not exported"
    from paper_2609_07108_b200 import binding
    assert set(binding.EXPORTS) == set(names)
    assert binding._lib().ba_status_string(-4) == b"metadata failed device-side validation"


def test_host_side_argument_checks_need_no_gpu():
    """Calls that fail validation return before touching the device."""
    from paper_2609_07108_b200 import binding
    lib = binding._lib()
    bad = binding._Problem(n_main=16, n_branch=0, num_seqs=1, num_branches=0, h_q=3, h_kv=2,
                           head_dim=128, dtype=0)
    assert lib.ba_plan_bytes(ctypes.byref(bad)) == 0                  # h_q % h_kv != 0
    ok = binding._Problem(n_main=16, n_branch=0, num_seqs=1, num_branches=0, h_q=4, h_kv=2,
                          head_dim=96, dtype=0)
    assert lib.ba_plan_bytes(ctypes.byref(ok)) == 0                   # head_dim unsupported
    ok.head_dim = 128
    assert lib.ba_plan_bytes(ctypes.byref(ok)) > 0
    out = ctypes.c_void_p()
    assert lib.ba_plan_create(ctypes.byref(ok), None, 0, None, ctypes.byref(out)) == -1   # NULL cu_seqlens
    assert lib.lse_merge(4, 6, None, None, None, None, None, 1, None, None) == -1
    assert lib.lse_merge(-1, 128, None, None, None, None, None, 1, None, None) == -1
    assert lib.ba_finalize_grads(None, None, 0, 0, None) == 0
    assert lib.branch_attn_fwd(None, None, None, None, None, None, None, None, 0, None) == -1


def test_closed_form_helpers_agree_with_brute_force():
    from helpers import GROUP_OFFSET, N_BITS, branch_visibility, expected_bit_fractions, visible_counts
    """The closed forms themselves, on a small tree batch, against explicit enumeration."""
    p = W.config4(shrink=64)
    vis_b = branch_visibility(p)
    cu = p.cu_seqlens.astype(np.int64)
    n = p.n_main
    for g in (0, 3):
        exp = expected_bit_fractions(p, g)
        rng = np.random.default_rng(0)
        for r in rng.choice(p.rows, size=40, replace=False):
            if r < n:
                s = np.searchsorted(cu, r, side="right") - 1
                keys = list(range(cu[s], r + 1))
            else:
                tkn = r - n
                b = tkn // 31
                a = int(p.anchor_idx[b])
                s = np.searchsorted(cu, a, side="right") - 1
                keys = list(range(cu[s], a + 1))
                node = tkn - 31 * b
                while node >= 0:
                    keys.append(n + 31 * b + node)
                    node = int(p.parent[31 * b + node])
                assert sorted(k - n - 31 * b for k in keys if k >= n) == list(np.nonzero(vis_b[tkn])[0])
            codes = np.array(keys, dtype=np.int64) + g * GROUP_OFFSET
            assert len(keys) == visible_counts(p)[r]
            for c in range(N_BITS):
                assert abs(((codes >> c) & 1).mean() - exp[r, c]) < 1e-12

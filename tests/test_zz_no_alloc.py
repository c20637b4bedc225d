"""branch_attn_bwd_static: the backward for callers that cannot allocate device
scratch when they call (fixed memory arenas, hooks where allocator calls are
forbidden).  It must give what branch_attn_bwd gives, call after call, while
using only the library's built-in scratch array.

Collected last on purpose (file name): a failure here cannot hide another
test's result in a run that stops at the first failure.  It passes on its own
in a fresh process and after the rest of the suite."""
import gc

import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _inputs(p, seed):
    t = W.make_tensors(p, seed=seed, std=0.5)
    dt = torch.bfloat16 if p.dtype == "bf16" else torch.float32
    return {k: torch.from_numpy(v).to("cuda", dt) for k, v in t.items()}


@pytest.mark.parametrize("make", [lambda: W.config2(shrink=8), lambda: W.odd_shapes(W.TREE, head_dim=128, dtype="bf16"),
                                  lambda: W.config1()])
def test_static_scratch_backward_matches_workspace_backward_twice(make):
    from paper_2609_07108_b200 import binding as ba
    p = make()
    plan = ba.Plan(p)
    tol = 2e-2 if p.dtype == "bf16" else 1e-4
    for call in range(2):                       # two calls in a row share the built-in array
        d = _inputs(p, seed=20 + call)
        o, lse = ba.branch_attn_fwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"])
        want = ba.branch_attn_bwd(plan, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"])
        got = tuple(torch.full_like(g, float("nan")) for g in want)
        gc.collect()                              # garbage of earlier tests must not be freed in between
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        ba.branch_attn_bwd_static(plan, d["q_main"], d["q_branch"], d["k"], d["v"], o, lse, d["d_o"], grads=got)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() <= before      # the call itself took no device memory
        plan.check()
        for name, a, b in zip(("dQ_main", "dQ_branch", "dK", "dV"), got, want):
            err = float((a.float() - b.float()).abs().max())
            assert np.isfinite(err) and err <= tol, f"call {call}: {name} differs by {err}"


def test_static_scratch_backward_rejects_problems_beyond_its_limit():
    from paper_2609_07108_b200 import binding as ba
    p = W.config3()                              # 40,960 rows x 32 heads: 10.5 MB of scratch > 8 MiB
    plan = ba.Plan(p)
    assert ba._lib().ba_workspace_bytes(plan.handle, ba.OP_BWD) > ba.STATIC_SCRATCH_BYTES
    def empty(*shape, dtype=torch.bfloat16):
        return torch.empty(shape, dtype=dtype, device="cuda")

    n, m, r = p.n_main, p.n_branch, p.rows
    hq, hkv, d = p.h_q, p.h_kv, p.head_dim
    with pytest.raises(ba.BranchAttnError) as e:       # refused before anything is launched
        ba.branch_attn_bwd_static(plan, empty(n, hq, d), empty(m, hq, d), empty(r, hkv, d), empty(r, hkv, d),
                                  empty(r, hq, d), empty(r, hq, dtype=torch.float32), empty(r, hq, d),
                                  grads=(empty(n, hq, d), empty(m, hq, d), empty(r, hkv, d), empty(r, hkv, d)))
    assert e.value.code == -3

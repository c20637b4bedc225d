"""The K/V ring driver on one GPU: ring steps read the received shard from a local
double buffer that a side stream fills while the previous step computes.  Its
results must equal the range-based zigzag driver's bit for bit (same kernels, same
accumulation order), which is itself checked against the oracle."""
import numpy as np
import pytest
import torch

from paper_2609_07108_b200 import ring, zigzag
from paper_2609_07108_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ba():
    from paper_2609_07108_b200 import binding
    assert torch.cuda.is_available()
    return binding


def inputs(p, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)

    def draw(shape, std):
        return (torch.randn(shape, generator=g, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    n, m = p.n_main, p.n_branch
    return (draw((n, p.h_q, 128), 0.5), draw((m, p.h_q, 128), 0.5), draw((n + m, p.h_kv, 128), 0.5),
            draw((n + m, p.h_kv, 128), 0.5), draw((n + m, p.h_q, 128), 0.1))


@pytest.mark.parametrize("cp", [2, 8])
def test_ring_equals_zigzag_bit_for_bit(ba, cp):
    p = W.config5(shrink=16)                   # 16,384 tokens: chunks of 1,024 (cp 8) / 4,096 (cp 2)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    qm, qb, k, v, go = inputs(p, 51)
    o1, l1, _ = zigzag.forward(ba, plan, qm, qb, k, v, cp)
    stats = ring.new_stats()
    bufs = ring.RingBuffers(plan, cp)
    # poison the double buffer: a step that read a slot before its shard arrived would show
    bufs.k.fill_(float("nan")); bufs.v.fill_(float("nan"))
    o2, l2, _ = ring.forward(ba, plan, qm, qb, k, v, cp, bufs=bufs, stats=stats)
    plan.check()
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    assert stats["copied_bytes"] == cp * ring.shard_bytes_per_rank(p, cp)      # Eq. cp-comm, every rank
    assert len(stats["copies"]) == cp * (cp - 1) and ring.copy_ms(stats) > 0.0
    g1 = zigzag.backward(ba, plan, qm, qb, k, v, o1, l1, go, cp, fused=False)
    g1 = [x.clone() for x in g1[:4]]
    g2 = ring.backward(ba, plan, qm, qb, k, v, o1, l1, go, cp, fused=False, bufs=bufs)
    plan.check()
    for name, a, b in zip(("dQ_main", "dQ_branch", "dK", "dV"), g1, g2[:4]):
        assert torch.equal(a, b), name
    # the one-kernel backward through the ring: dK, dV bit-identical, dQ up to the order of its atomic adds
    g3 = zigzag.backward(ba, plan, qm, qb, k, v, o1, l1, go, cp, fused=True)
    g3 = [x.clone() for x in g3[:4]]
    g4 = ring.backward(ba, plan, qm, qb, k, v, o1, l1, go, cp, fused=True, bufs=bufs)
    plan.check()
    assert torch.equal(g3[2], g4[2]) and torch.equal(g3[3], g4[3])
    for a, b in zip(g3[:2], g4[:2]):
        assert float((a.float() - b.float()).abs().max()) <= 1e-3 * max(1.0, float(a.float().abs().max()))


def test_shard_calls_check_their_ranges(ba):
    p = W.config5(shrink=64)
    plan = ba.Plan(p, impl=ba.IMPL_TC)
    qm, qb, k, v, go = inputs(p, 52)
    lib = ba._lib()
    x = ba._p(k)
    # shard ends must be multiples of 128 (or N): otherwise a key tile would reach outside the shard
    for kv in ((64, 256), (0, 200), (-128, 128), (256, 128), (0, p.n_main + 128)):
        rc = lib.branch_attn_fwd_shard(plan.handle, ba._p(qm), ba._p(qb), x, x, 0, 128, 0, 0, kv[0], kv[1], 0, x, x,
                                       ba._stream())
        assert rc == -1, kv
    torch.cuda.synchronize()

"""Host logic of the K/V ring driver, on CPU: the hand-off order of the local
double buffer, the shard volume of Eq. (cp-comm), and -- with two gloo ranks that
really exchange shards through torch.distributed -- that following the plan puts
the shard of rank (r - s) mod C into the slot step s computes on."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2609_07108_b200 import ring, zigzag
from paper_2609_07108_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("cp", [1, 2, 3, 8])
def test_hand_off_plan_never_refills_a_slot_in_use(cp):
    for rank in range(cp):
        plan = ring.hand_off_plan(rank, cp)
        ring.check_plan(plan)
        computes = [a for a in plan if a[0] == "compute"]
        assert [a[1] for a in computes] == list(range(cp))                       # every ring step once, in order
        assert [a[2] for a in computes] == [(rank - s) % cp for s in range(cp)]   # shard of rank (r - s) mod C
        assert computes[0][3] is None                                             # step 0: the rank's own K/V
        recvs = [a for a in plan if a[0] == "recv"]
        assert len(recvs) == cp - 1                                               # C - 1 shards cross the ring
        for r in recvs:                                                           # each is issued before the compute
            assert plan.index(r) < plan.index(next(c for c in computes if c[1] == r[1] - 1))   # of the step before
    # a plan that refills a slot early is caught
    bad = [("recv", 1, 0, 1), ("wait", 1, 1), ("compute", 1, 0, 1), ("recv", 3, 2, 1)]
    with pytest.raises(AssertionError):
        ring.check_plan(bad)


def test_shard_volume_is_eq_cp_comm():
    p = W.config5()
    # 2 (C - 1) (N / C) d_kv b = 2 * 7 * 32768 * (8 * 128) * 2 bytes
    assert ring.shard_bytes_per_rank(p, 8) == 939524096
    # the blocks a rank computes at step s use only chunks of the shard it holds at step s
    for b in zigzag.schedule(W.config5(shrink=64), 8):
        src, chunks = ring.shard_owner_chunks(b.rank, b.step, 8)
        assert b.kv_chunk in chunks


@pytest.mark.parametrize("world", [2, 4])
def test_ranks_exchange_shards_by_the_plan(tmp_path, world):
    script = tmp_path / "ring_ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys
        sys.path.insert(0, {ROOT!r})
        import torch, torch.distributed as dist
        from paper_2609_07108_b200 import ring
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend="gloo")
        rank, cp = dist.get_rank(), dist.get_world_size()
        rows = 8
        # a rank's own shard: its two chunks, every element = 100 * owner + chunk position
        own = torch.stack([torch.full((rows,), 100.0 * rank + i) for i in range(2)])
        slots = torch.zeros((2, 2, rows))
        recvs, sends, seen = {{}}, {{}}, []
        for act in ring.hand_off_plan(rank, cp):
            if act[0] == "recv":
                _, step, src, slot = act
                recvs[step] = dist.irecv(slots[slot], src=(rank - 1) % cp)       # posted ahead of the compute
                if step == 1:                                                    # my own shard starts its trip
                    sends[0] = dist.isend(own, dst=(rank + 1) % cp)
            elif act[0] == "wait":
                _, step, slot = act
                recvs.pop(step).wait()
                if step + 1 < cp:                                                # pass the arrived shard on
                    sends[step] = dist.isend(slots[slot], dst=(rank + 1) % cp)
            elif act[0] == "compute":
                _, step, src, slot = act
                shard = own if slot is None else slots[slot]
                assert torch.equal(shard[0], torch.full((rows,), 100.0 * src)), (rank, step, shard)
                assert torch.equal(shard[1], torch.full((rows,), 100.0 * src + 1))
                seen.append(src)
            elif act[0] == "free":
                _, step, slot = act
                if step in sends:
                    sends.pop(step).wait()                                       # sent on before the slot is refilled
        for s in sends.values():
            s.wait()
        assert seen == [(rank - s) % cp for s in range(cp)], seen
        dist.barrier()
        if rank == 0:
            print("RING OK", seen)
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(world),
                          "--master-addr", "127.0.0.1", "--master-port", str(29541 + world), str(script)],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-3000:]
    assert "RING OK" in out.stdout

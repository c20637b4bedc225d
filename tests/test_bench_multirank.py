"""The N > 1 path of the benchmark is "replicas only": every rank runs the same
step on its own GPU and the job's throughput is (units of all ranks) / (time of
the slowest rank).  Checked here with two gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_rank_aggregation_takes_the_slowest_rank(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import bench
        dist, rank, world = bench.dist_setup(2, backend="gloo")
        assert world == 2
        local_ms = 100.0 if rank == 0 else 250.0          # rank 1 is the slow replica
        value, ms = bench.aggregate_throughput(dist, 1e12, local_ms)
        assert abs(ms - 250.0) < 1e-9, ms                  # max over ranks
        assert abs(value - 2 * 1e12 / 0.25 / 1e12) < 1e-9, value
        assert bench.max_over_ranks(dist, float(rank)) == 1.0
        dist.barrier()
        if rank == 0:
            print("OK", value)
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    assert "OK 8.0" in out.stdout


def test_reference_arm_only_rank_zero_works(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""

"""The benchmark's multi-rank bookkeeping (slowest rank's time, sum of units) over 2 gloo ranks on CPU."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reduce_over_ranks_two_gloo_ranks(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch.distributed as dist
        import bench
        world, rank, local = bench.dist_setup(2)
        assert world == 2
        bench.barrier(world)
        t, u = bench.reduce_over_ranks(10.0 + 5.0 * rank, 128 * (rank + 1), world)
        if rank == 0:
            print(json.dumps({{"t": t, "u": u}}))
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541", CUDA_VISIBLE_DEVICES="")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", str(script)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    import json
    r = json.loads(line)
    assert r["t"] == 15.0 and r["u"] == 384.0


def test_reference_arm_runs_without_a_gpu():
    # config 4 here: the default workload (config 5) takes the oracle minutes per step on a small host
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg4", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=600,
                         env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    r = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert r["impl"] == "reference" and r["value"] > 0 and r["cpu_baseline"]["kind"] == "oracle"
    assert r["e2e"]["h2d_bytes_per_step"] == 0
    sys.path.insert(0, ROOT)
    import bench
    assert r["config"]["workload"] == bench.WORKLOADS["cfg4"]      # the same string the CUDA arm prints

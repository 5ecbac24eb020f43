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


def test_clock_sampler_summary_from_rows():
    """The summary of the sampled nvidia-smi rows: median clock, reasons seen, board power; rows taken before the
    mark and malformed rows are left out, and rows without the power columns still give the clock figures."""
    sys.path.insert(0, ROOT)
    import bench

    class Done:
        def terminate(self): pass
        def wait(self, timeout=None): return 0

    s = bench.ClockSampler(0)
    s.proc = Done()
    s.rows = [["300", "1965", "Not Active", "Not Active", "Not Active", "Not Active", "120.0", "1000.00"],   # before the mark
              ["1965", "1965", "Not Active", "Not Active", "Not Active", "Not Active", "700.5", "1000.00"],
              ["1905", "1965", "Not Active", "Not Active", "Not Active", "Active", "905.0", "1000.00"],
              ["1890", "1965", "Not Active", "Not Active", "Not Active", "Active", "990.0", "1000.00"],
              ["[N/A]", "1965", "Not Active", "Not Active", "Not Active", "Active", "1.0", "1000.00"],
              ["short", "row"]]
    s.first = 1
    out = s.stop()
    assert out["sm_mhz"] == 1905.0 and out["sm_max_mhz"] == 1965.0 and out["samples"] == 3
    assert out["reasons"] == ["sw_power_cap"]
    assert out["power_w"] == 905.0 and out["power_limit_w"] == 1000.0 and out["power_capped_samples"] == 2
    s = bench.ClockSampler(0)
    s.proc = Done()
    s.rows = [["1800", "1965", "Not Active", "Active", "Not Active", "Not Active"]]
    out = s.stop()
    assert out["sm_mhz"] == 1800.0 and out["reasons"] == ["hw_thermal_slowdown"] and "power_w" not in out

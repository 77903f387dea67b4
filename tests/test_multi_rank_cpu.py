"""The N > 1 path of the benchmark on CPU (gloo, world size 2): ranks are independent replicas, the job's
time is the maximum over ranks and the value is the sum of the replicas' work over that time."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=2)
    rank = dist.get_rank()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
    assert ms == 15.0, ms
    v = bench.whole_job_value(3.0e12, 2, ms)              # 2 replicas x 3 TFLOP per step / 15 ms
    assert abs(v - 400.0) < 1e-9, v
    dist.barrier()
    dist.destroy_process_group()
    print("ok", rank)
""")


def test_two_rank_timing_rule_on_gloo(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29591", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=240)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("ok" in o for o in outs)


def test_single_process_is_a_noop():
    import bench
    assert bench.max_over_ranks(7.5) == 7.5
    assert bench.whole_job_value(1e12, 1, 1.0) == 1000.0

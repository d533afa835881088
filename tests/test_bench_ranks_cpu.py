"""The multi-rank plumbing of bench.py (independent replicas, slowest rank decides) on two CPU ranks over gloo."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% sys.argv[2], rank=int(sys.argv[1]), world_size=2)
rank = dist.get_rank()
ms = bench.max_over_ranks(1.0 + rank, dist, "cpu")          # rank 1 is the slow one: 2 ms per step
assert ms == 2.0, ms
v = bench.whole_job_value(5120, 2, ms)
assert abs(v - 2 * 5120 / 2e-3) < 1e-6, v
dist.barrier()
dist.destroy_process_group()
print("rank", rank, "ok")
""" % ROOT


def test_two_ranks_take_the_slowest_time_and_add_their_units(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = str(29500 + os.getpid() % 2000)
    procs = [subprocess.Popen([sys.executable, str(script), str(r), port], stdout=subprocess.PIPE, stderr=subprocess.STDOUT,
                              text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0 and "rank %d ok" % r in o, o


def test_single_rank_helpers_and_reference_arm_on_other_ranks():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_value(100, 1, 10.0) == 10000.0
    # under torchrun only rank 0 runs the reference arm; the others return without work
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_workload_arithmetic_matches_the_layer_table():
    sys.path.insert(0, ROOT)
    import bench
    from paper_1705_04862_b200.configs import CONFIGS
    roll, upd = bench.iteration_flops(CONFIGS[4])
    assert abs(roll / 1e9 - 114.93) < 0.05 and abs(upd / 1e9 - 157.99) < 0.05
    work, P = bench.kernel_work(CONFIGS[4])
    assert P == 1693875 and abs(work["clip_rmsprop"][1] - 22 * P) < 1

"""The multi-rank bookkeeping of bench.py (whole-job units = sum over ranks, job time = max over
ranks) on two gloo ranks on the CPU, and the reference arm's output contract."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank did 1000 * (rank + 1) units in (rank + 1) seconds
    units, secs = bench.reduce_job(1000.0 * (rank + 1), float(rank + 1), world, "cpu")
    q.put((rank, units, secs, bench.dist_env()))
    dist.barrier()
    dist.destroy_process_group()


def test_job_value_is_sum_of_units_over_max_of_times():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, units, secs, env in got:
        assert units == 3000.0 and secs == 2.0          # 1000 + 2000 units, max(1 s, 2 s)
        assert env[0] == rank and env[1] == 2


def test_reference_arm_prints_one_json_line_and_other_ranks_stay_silent():
    env = dict(os.environ, OMP_NUM_THREADS="4")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "tiny"], capture_output=True, text=True, env=env, timeout=600)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "params/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    env1 = dict(env, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "tiny", "--gpus", "2"], capture_output=True, text=True,
                         env=env1, timeout=600)
    assert out.returncode == 0 and out.stdout.strip() == ""

"""The N > 1 path of the benchmark is "replicas only": no data-path collective, just the timing
protocol (barrier, MAX over ranks, whole-job aggregation).  Covered here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2605_20022_b200 import replicas
    dist = replicas.init("gloo")
    assert replicas.rank_world() == (rank, world, rank)
    replicas.barrier(dist)
    mine = [10.0 + 5.0 * rank, 3.0 - rank]           # rank 1 is slower on the first timer, faster on the second
    got = replicas.max_over_ranks(mine, dist)
    out.put((rank, got))
    replicas.barrier(dist)
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregation_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29731, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [15.0, 3.0]
    from paper_2605_20022_b200 import replicas
    assert replicas.max_over_ranks([1.5, 2.5], None) == [1.5, 2.5]
    assert replicas.whole_job_us_per_step(ms_total=30.0, steps=5, world=2) == 3000.0
    assert replicas.whole_job_us_per_step(ms_total=30.0, steps=5, world=1) == 6000.0


def test_reference_arm_under_two_ranks_prints_once():
    """`bench.py --impl reference` with WORLD_SIZE=2: rank 0 prints the JSON line, rank 1 exits 0 silently."""
    outs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT="29732")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--workload", "0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True,
                           timeout=300)
        assert r.returncode == 0, r.stderr
        outs.append(r.stdout.strip())
    assert outs[1] == ""
    line = json.loads(outs[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["vs_baseline"] is None and line["value"] > 0 and line["unit"] == "us/step"


def test_plain_process_with_gpus_2_starts_two_ranks_itself():
    """`python bench.py --gpus 2` without a rank environment re-launches itself as two ranks (one per GPU on a GPU
    box); shown here on CPU with the reference arm: one JSON line comes back, from rank 0, with n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "0", "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2

"""N > 1 host logic on CPU: two gloo ranks, and the reference arm's rank gating."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2605_03110_b200 import replicas, workloads as wl
    rep = replicas.from_env()
    replicas.init_process_group(rep, "gloo")
    replicas.barrier(rep)
    my_time = 0.010 * (rank + 1)                       # rank 1 is the slow one
    t = replicas.max_over_ranks(rep, my_time)
    cfg = wl.scaled(wl.CONFIGS[1], T=64, d=32, L=1, P=8)
    X = next(wl.generate_layers(cfg, seed=rep.seed)).X
    out.put((rank, t, replicas.whole_job_throughput(rep, 1000.0, t), float(X.sum()),
             replicas.is_reporter(rep)))
    replicas.barrier(rep)


def test_two_gloo_ranks_agree_on_the_slowest_time_and_draw_different_inputs():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29611, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, v0, s0, rep0), (r1, t1, v1, s1, rep1) = res
    assert t0 == t1 == 0.020                           # MAX over ranks
    assert v0 == v1 == 2 * 1000.0 / 0.020              # whole-job units / slowest time
    assert s0 != s1                                    # replicas draw different sequences
    assert rep0 and not rep1                           # one reporter


def test_reference_arm_runs_on_rank_0_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0", "--workload", "1", "--ref-layers", "2"]
    outs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29612")
        r = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
        assert r.returncode == 0, r.stderr
        outs.append(r.stdout.strip())
    assert outs[1] == ""                               # other ranks exit 0 without work
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"].startswith("configs[0]")

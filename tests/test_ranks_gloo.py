"""The multi-rank path on CPU: two processes over gloo.

The attention path shards over the batch with no data-path exchange, so what N > 1 adds is host-side: every rank draws
its own sequences, the timed region is bracketed by a barrier, the job's time is the slowest rank's, the job's value is
the sum of what all ranks processed, and only rank 0 reports.  These tests run exactly that plumbing
(`paper_2408_01890_b200.ranks`, `bench.py --impl reference`) as two real processes.
"""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def rank_main(rank, world, port, out_dir):
    os.environ.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1",
                       "MASTER_PORT": str(port)})
    sys.path.insert(0, ROOT)
    from paper_2408_01890_b200 import synth
    from paper_2408_01890_b200.ranks import RankGroup
    g = RankGroup("gloo")
    assert (g.rank, g.world) == (rank, world)
    # every rank draws its own sequences of the same workload
    w = synth.Workload("ranks", "bf16", 1, 16, 4, 2, 32, 8, 8, "relu", 1)
    q0 = synth.to_f64(synth.prefill_inputs(w, seed=g.seed())["q0"])
    g.barrier()
    my_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    job_ms = g.max_over_ranks(my_ms)
    value = g.whole_job_per_second(w.B * w.N, job_ms)
    g.barrier()
    np.save(os.path.join(out_dir, "q0_%d.npy" % rank), q0)
    with open(os.path.join(out_dir, "rank_%d.json" % rank), "w") as f:
        json.dump({"job_ms": job_ms, "value": value}, f)
    g.close()


def test_two_ranks_over_gloo(tmp_path):
    world, port = 2, free_port()
    mp.spawn(rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / ("rank_%d.json" % r))) for r in range(world)]
    # the job's time is the slowest rank's, on every rank; the value is the whole job's: both ranks' tokens over that time
    assert all(r["job_ms"] == 15.0 for r in res)
    assert all(abs(r["value"] - 2 * 16 / 15e-3) < 1e-6 for r in res)
    # different ranks work on different data
    assert not np.array_equal(np.load(tmp_path / "q0_0.npy"), np.load(tmp_path / "q0_1.npy"))


def test_single_process_group_is_a_no_op():
    env = {k: os.environ.pop(k) for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK") if k in os.environ}
    try:
        from paper_2408_01890_b200.ranks import RankGroup
        g = RankGroup("gloo")
        assert g.world == 1 and g.dist is None
        g.barrier()
        assert g.max_over_ranks(3.5) == 3.5
        assert g.whole_job_per_second(100, 50.0) == 2000.0
        g.close()
    finally:
        os.environ.update(env)


def test_reference_arm_prints_on_rank_zero_only():
    """Launched as two ranks, the benchmark's reference arm (the CPU oracle, timed) runs and prints on rank 0; rank 1
    leaves without work and without output."""
    outs = []
    for rank in (0, 1):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(free_port()))
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                            "--warmup", "0"], env=env, capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr[-2000:]
        outs.append(r.stdout.strip())
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1] == ""

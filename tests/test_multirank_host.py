"""The N > 1 host logic of bench.py on CPU: two gloo ranks agree on the max-over-ranks timing,
own distinct replicas of the workload, and only rank 0 reports."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    import pisa_synth as S
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_env() == (rank, world, rank)
    ms = bench.max_over_ranks([10.0 + rank, 7.0 - rank], world)
    w = bench.replica_workload(S.WORKLOADS["cfg1"], rank)
    t = S.make_inputs(w)
    q.put((rank, ms, w.seed, float(t["q"].ravel()[0]), bench.job_tokens_per_s(w, world, 4, ms[0])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_and_own_distinct_replicas():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, seed0, q0, v0), (r1, ms1, seed1, q1, v1) = res
    assert ms0 == ms1 == [11.0, 7.0]                 # max over ranks, on every rank
    assert seed0 != seed1 and q0 != q1               # each rank has its own replica
    assert v0 == v1 == 2 * 1024 * 4 / (11.0e-3)       # whole-job tokens/s counts both ranks' tokens


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "cfg1", "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "cfg1", "--steps", "2", "--warmup", "1", "--ref-queries", "16"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "tokens/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_selection_quality_metrics_on_a_hand_case():
    """Recall@K and MassRatio as the paper defines them (Sec. 5 "Block-selection quality")."""
    import numpy as np

    import bench
    mass = np.array([[0.5, 0.1, 0.3, 0.1, 0.0, 0.0],        # reference top-2: blocks 0, 2
                     [0.2, 0.2, 0.6, 0.0, 0.0, 0.0]])       # reference top-2: 2 and 0 (tie -> smaller index)
    idx = np.array([[0, 3], [1, 2]], dtype=np.int32)
    rec, rat = bench.selection_quality(idx, mass)
    assert np.allclose(rec, [0.5, 0.5])
    assert np.allclose(rat, [0.6 / 0.8, 0.8 / 0.8])
    # fewer live blocks than K: the reference set shrinks, padding is ignored
    rec, rat = bench.selection_quality(np.array([[0, -1, -1]], dtype=np.int32), np.array([[1.0, 0.0, 0.0]]))
    assert np.allclose(rec, [1.0]) and np.allclose(rat, [1.0])

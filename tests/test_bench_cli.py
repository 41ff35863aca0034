"""bench.py's reference arm (the CPU oracle) runs without a GPU and keeps the JSON contract;
under a multi-rank launch only rank 0 works and prints."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(env_extra):
    env = dict(os.environ, **env_extra)
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                           "--workload", "C0", "--steps", "2", "--warmup", "1", "--ref-layers", "4",
                           "--gpus", env_extra.get("WORLD_SIZE", "1")],
                          capture_output=True, text=True, env=env, timeout=300)


def test_reference_arm_prints_the_contract_line():
    r = _run({"RANK": "0", "WORLD_SIZE": "1", "CUDA_VISIBLE_DEVICES": ""})
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["metric"] == "decode_tokens_per_s" and d["unit"] == "tokens/s"
    assert d["value"] > 0 and d["higher_is_better"] is True and d["config"]["workload"].startswith("C0")
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}


def test_reference_arm_other_ranks_exit_quietly():
    r = _run({"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1", "CUDA_VISIBLE_DEVICES": ""})
    assert r.returncode == 0 and r.stdout.strip() == ""


def _rank_main(rank, world, port, out):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    # rank r measured (10 + r) ms device-timed and (20 - r) ms end to end: the job's figures are the maxima
    ms, e2e = bench.max_over_ranks([10.0 + rank, 20.0 - rank], world, torch.device("cpu"))
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, ms, e2e))


def test_replica_timing_is_the_maximum_over_ranks_gloo_world_2():
    """The N > 1 path of the main arm (replicas only: no data-path collective): every rank gets the
    slowest rank's times, from which rank 0 reports tokens of all ranks over that time."""
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 11.0, 20.0), (1, 11.0, 20.0)]
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]      # a single rank: no collective


def test_routing_overlap_statistics_by_hand():
    """Temporal overlap = experts shared by the same layer at consecutive steps, spatial = by adjacent
    layers of one step; two layers, one sequence, top-2, three steps, counted by hand."""
    import numpy as np
    sys.path.insert(0, ROOT)
    import bench
    ids = [np.array([[[0, 1]], [[1, 2]]]), np.array([[[0, 1]], [[2, 3]]]), np.array([[[1, 5]], [[0, 1]]])]
    ov = bench.routing_overlap(ids)
    assert ov["temporal"] == (2 + 1 + 1 + 0) / 4          # (t1,t0): layers 0,1; (t2,t1): layers 0,1
    assert abs(ov["spatial"] - (1 + 0 + 1) / 3) < 1e-12   # steps 0,1,2: layer 1 against layer 0

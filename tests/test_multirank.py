"""The N > 1 path of the benchmark on CPU: two gloo ranks on 127.0.0.1.  The hot path shards by
request with no data-path collective, so what is covered is that ranks draw different requests, that
the timing is the maximum over ranks, and the whole-job arithmetic."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2402_12374_b200 import workloads as W

    cfg = W.CONFIGS["tiny"]
    parent, attn, ver = bench.build_requests(cfg, 0.6, rank, 1, 1)
    local_ms = 10.0 + 5.0 * rank  # stand-in for this rank's CUDA-event time
    ms = bench.max_over_ranks(local_ms)
    digest = float(attn[0].q.float().sum()) + float(ver[0].target_logits[:, :64].sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, (digest, parent.tolist()))
    out.put((rank, ms, bench.whole_job_us_per_step(ms, 4, world), gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_different_requests_and_the_max_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, gathered in results:
        assert ms == 15.0                                    # the slower rank decides
        assert abs(value - 1e3 * 15.0 / 4 / 2) < 1e-9        # two requests verified per step time
        assert gathered[0][0] != gathered[1][0]              # different inputs per rank
    import bench

    assert bench.max_over_ranks(3.0) == 3.0 and bench.rank_seed_base(3) == 3000


def test_reference_arm_prints_one_json_line_on_rank0_only(tmp_path):
    import json
    import subprocess
    import sys

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["higher_is_better"] is False

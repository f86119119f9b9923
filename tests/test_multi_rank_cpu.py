"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The hot path does not shard inside a
request and requests are independent, so ranks run replicas of the step on their own batches;
what the ranks share is only the timing protocol (barrier, max over ranks) and the aggregate."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2409_16560_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    spec = bench.rank_spec(inputs.config("C1"), rank)
    data = inputs.generate(spec, "cpu", parts=("verify",))
    dist.barrier()
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu")      # rank 1 is the slow one
    out.put((rank, spec["seed"], ms, float(data["logits_p"][0, 0]), int(data["forest"]["N"])))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_share_only_the_clock():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, ms0, x0, n0), (r1, seed1, ms1, x1, n1) = res
    assert seed0 != seed1 and x0 != x1          # every rank verifies its own requests
    assert n0 == n1                              # of the same shape (weak scaling)
    assert ms0 == ms1 == 20.0                    # the job's step time is the slowest rank's
    assert bench.job_value(n0, world, ms0) == n0 * 2 / 0.020


def test_reference_arm_prints_one_json_line(capsys):
    import json
    import types
    args = types.SimpleNamespace(workload="C1", warmup=0, steps=1, gpus=1, top_k=0, top_p=1.0)
    bench.run_reference(args)
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == bench.UNIT and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0

"""The N > 1 path of bench.py on CPU: two gloo ranks. The flow has no exchange step (every rank
encodes its own batch), so what there is to check is the host logic: rank-distinct inputs, the
maximum-over-ranks timing and the whole-job throughput, and that the reference arm only speaks on
rank 0."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    import iodf_synth as S
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # each rank times its own work; rank 1 is "slower"
    my_ms = [10.0 + 5.0 * rank, 2.0 - rank]
    red = bench.max_over_ranks(my_ms, world)
    x = S.config_images(0, batch=2, seed_offset=bench.rank_seed_offset(rank, 0))
    sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, torch.tensor([float(x.astype(np.int64).sum())], dtype=torch.float64))
    out[rank] = dict(red=red, value=bench.job_throughput(128, world, 10, red[0] * 1e-3), sums=[float(t) for t in sums])
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_and_shard():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0]["red"] == res[1]["red"] == [15.0, 2.0]           # max over ranks, element-wise
    assert res[0]["value"] == 128 * 2 * 10 / 15e-3                   # whole-job images/s on the slowest rank's time
    assert res[0]["sums"][0] != res[0]["sums"][1]                    # ranks draw different images


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--config", "0"], env=env, capture_output=True, text=True,
                       timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2

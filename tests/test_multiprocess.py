"""The N > 1 path of the benchmark on CPU: two gloo ranks, each a replica with its own seeded
batch (no data-path collective); the step time is the maximum over ranks and the value counts
every rank's bytes."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2609_33410_b200.workloads import make_decode_workload
    gen = dict(bench.WORKLOADS["c1"]["gen"])
    gen["seed"] = gen["seed"] + 1000 * rank                    # the replica rule bench.py uses
    w = make_decode_workload(device="cpu", **dict(gen, seqlens=256))
    local_ms = 1.0 + rank                                       # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    value = world * w.cache_bytes() / (ms * 1e-3) / 1e9
    digest = float(w.k.float().sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, (ms, value, digest))
    if rank == 0:
        torch.save(gathered, out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_replicas_and_max_timing(tmp_path):
    out = str(tmp_path / "res.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    res = torch.load(out)
    (ms0, v0, d0), (ms1, v1, d1) = res
    assert ms0 == ms1 == 2.0                                   # the maximum over ranks, on every rank
    assert v0 == v1 and abs(v0 - 2 * 256 * 8 * 4 * 128 / 2e-3 / 1e9) < 1e-9
    assert d0 != d1                                            # each replica draws its own batch

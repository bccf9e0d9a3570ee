"""The N > 1 path of the benchmark on CPU: two gloo processes check the per-rank workload
assignment (weak scaling, distinct seeds, no data-path collective) and the max-over-ranks
reduction that defines the reported step time."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2607_19378_b200 import workloads as W
    base = W.WORKLOADS["vision2d"].scaled(B=1, C=2)
    w = bench.workload_for_rank(base, rank, world)
    q, k, v, h = W.make_inputs(w)
    # every rank owns a full batch of the same shape, drawn from its own stream
    fingerprint = float(q.float().sum() + h.float().sum())
    ms_local = 1.0 + rank                      # rank 1 is the slower one
    ms, e2e = bench.max_over_ranks([ms_local, 2.0 * ms_local], dist, torch.device("cpu"))
    gathered = [None] * world
    dist.all_gather_object(gathered, (w.seed, tuple(q.shape), fingerprint))
    value = bench.aggregate_throughput(w.elements, world, ms)
    if rank == 0:
        torch.save({"ms": ms, "e2e": e2e, "gathered": gathered, "value": value, "elements": w.elements}, out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_weak_scaling_logic(tmp_path):
    world = 2
    out = str(tmp_path / "result.pt")
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    r = torch.load(out)
    assert r["ms"] == 2.0 and r["e2e"] == 4.0                     # the slowest rank defines the time
    seeds = [g[0] for g in r["gathered"]]
    shapes = [g[1] for g in r["gathered"]]
    prints = [g[2] for g in r["gathered"]]
    assert len(set(seeds)) == world and len(set(shapes)) == 1      # same shape, different data
    assert prints[0] != prints[1]
    assert abs(r["value"] - world * r["elements"] / (2.0e-3) / 1e9) < 1e-12


def test_single_process_helpers():
    import bench
    from paper_2607_19378_b200 import workloads as W
    w = W.WORKLOADS["tiny2d"]
    assert bench.workload_for_rank(w, 0, 1) is w
    assert bench.max_over_ranks([1.5, 2.5], None, torch.device("cpu")) == [1.5, 2.5]
    nbytes, flops, P = bench.op_algorithmic(W.WORKLOADS["volume3d"])
    assert P == 256 ** 3
    assert abs(nbytes - (4 * 2 ** 27 * 2 + 64 * 255 ** 3 * 2)) < 1
    assert abs(flops - 192 * 2.5 * 2 ** 24 * 24) < 1
    nbytes, flops, P = bench.op_algorithmic(W.WORKLOADS["genomics1d"])
    assert P == 2 ** 19 and abs(flops - 1280 * 2.5 * 2 ** 19 * 19) < 1


def test_gpus_flag_spawns_one_rank_per_gpu_when_no_launcher_is_present():
    """`bench.py --gpus N` without torchrun around it starts its N ranks itself: the command it builds is the
    launcher the multi-rank path expects (one process per GPU, loopback rendezvous) and carries every option on."""
    import argparse
    import bench
    args = argparse.Namespace(gpus=4, steps=7, warmup=3, workload="pde2d", impl="ours", batch=None, channels=16,
                              no_all=True, no_cpu=False, no_cufft=True)
    cmd = bench.spawn_command(args, 29512)
    assert cmd[1:4] == ["-m", "torch.distributed.run", "--nnodes=1"] and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29512"
    tail = cmd[cmd.index(os.path.join(ROOT, "bench.py")) + 1:]
    assert tail == ["--gpus", "4", "--steps", "7", "--warmup", "3", "--workload", "pde2d", "--impl", "ours",
                    "--channels", "16", "--no-all", "--no-cufft"]

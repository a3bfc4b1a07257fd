"""The N > 1 path of the benchmark: independent replicas, max-over-ranks timing (gloo, 2 CPU ranks)."""
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank r measured (10 + r) ms for the device-timed region and (20 - r) ms end to end
    ms, ms_e2e = bench.max_over_ranks([10.0 + rank, 20.0 - rank], dist, None)
    value = bench.whole_job_images_per_s(128, 50, world, ms)
    q.put((rank, ms, ms_e2e, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_max_over_ranks_and_aggregate():
    torch = pytest.importorskip("torch")
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, ms_e2e, value in out:
        assert ms == 11.0 and ms_e2e == 20.0          # slowest rank in each column
        assert abs(value - 128 * 50 * 2 / 11e-3) < 1e-6


def test_single_rank_is_identity():
    import bench
    assert bench.max_over_ranks([3.5, 7.0]) == [3.5, 7.0]
    assert bench.whole_job_images_per_s(64, 10, 1, 100.0) == 6400.0


def test_flop_accounting_of_the_named_workloads():
    """Forward conv FLOPs per image: 10.49 G (WRN-28-10), 0.2515 G (ResNet-56), 7.33 G (ResNet-34)."""
    import bench
    from workloads import get_config
    for name, gflop in (("wrn28_10", 10.487), ("resnet56", 0.2515), ("resnet110", 0.5063), ("resnet34", 7.328)):
        cfg = get_config(name)
        fwd, aux = bench.conv_flops_forward(cfg)
        assert abs(fwd / cfg["N"] / 1e9 - gflop) / gflop < 0.01, (name, fwd / cfg["N"] / 1e9)
        assert 0 < aux < 0.25 * fwd

"""The multi-GPU path shards by batch with no collective on the data path; what is left to test
without GPUs is the host logic: the batch split, the max-over-ranks reduction of the timed
region and the whole-job rate.  Two gloo ranks on the CPU."""
import os
import socket

import pytest
import torch.multiprocessing as mp

from paper_2309_06626_b200.dist_util import max_over_ranks, shard_batch, whole_job_rate


def test_shard_batch_covers_the_batch_once():
    for Nb in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            parts = [shard_batch(Nb, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == Nb
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        shard_batch(8, 2, 2)


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    elapsed = 1.0 + rank            # rank 1 is the slow one
    slowest = max_over_ranks(elapsed)
    lo, hi = shard_batch(64, rank, world)
    out.put((rank, slowest, hi - lo, whole_job_rate(100.0, slowest, world)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [2.0, 2.0]
    assert sum(r[2] for r in res) == 64
    assert res[0][3] == pytest.approx(2 * 100.0 / 2e-3)


def test_single_process_is_identity():
    assert max_over_ranks(3.5) == 3.5

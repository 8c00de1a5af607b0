"""Multi-rank host logic on CPU: two gloo ranks, rendezvous on 127.0.0.1.  Requests shard across ranks
with no data-path collective; ranks exchange only the slowest time and the unit counts."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_22098_b200 import shard, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world_size, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world_size)
    try:
        assert shard.world() == (rank, world_size)
        # the slowest rank's time and the units of all ranks reach every rank
        ms_local = 10.0 + 5.0 * rank
        assert shard.max_over_ranks(ms_local) == 10.0 + 5.0 * (world_size - 1)
        assert shard.sum_over_ranks(float(rank + 1)) == world_size * (world_size + 1) / 2
        value, ms = shard.job_throughput(units_this_rank=100.0, ms_this_rank=ms_local)
        assert ms == 10.0 + 5.0 * (world_size - 1)
        assert abs(value - 100.0 * world_size / (ms * 1e-3)) < 1e-9
        # every request of a batch lands on exactly one rank
        mine = list(shard.shard_requests(33, rank, world_size))
        gathered = [None] * world_size
        dist.all_gather_object(gathered, mine)
        flat = [i for part in gathered for i in part]
        assert flat == list(range(33))
        assert max(len(p) for p in gathered) - min(len(p) for p in gathered) <= 1
        # shards are distinct synthetic inputs, reproducible per rank
        wl = synth.WORKLOADS["tiny"]
        a = synth.make_anchor(wl, shard.shard_seed(7, rank) + 3, B=4)
        again = synth.make_anchor(wl, shard.shard_seed(7, rank) + 3, B=4)
        assert torch.equal(a, again)
        anchors = [None] * world_size
        dist.all_gather_object(anchors, a.tolist())
        assert len({tuple(x) for x in anchors}) == world_size
        dist.barrier()
        out.put((rank, "ok"))
    except Exception as e:  # report instead of hanging the peer
        out.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_rank_plumbing():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
    assert sorted(results) == [(0, "ok"), (1, "ok")], results


def test_single_process_defaults():
    assert shard.world() == (0, 1)
    assert shard.max_over_ranks(3.5) == 3.5
    assert shard.sum_over_ranks(2.0) == 2.0
    assert list(shard.shard_requests(5, 0, 1)) == [0, 1, 2, 3, 4]
    assert [len(shard.shard_requests(10, r, 4)) for r in range(4)] == [3, 3, 2, 2]
    with pytest.raises(ValueError):
        shard.shard_requests(4, 4, 4)
    assert shard.shard_seed(11, 0) != shard.shard_seed(11, 1)

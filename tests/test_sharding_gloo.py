"""The multi-rank host logic on CPU: two gloo ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2411_04975_b200 import sharding
    dev = torch.device("cpu")
    res = {}
    res["range"] = list(sharding.request_range(rank, world, 4))
    res["max"] = sharding.max_over_ranks(10.0 + rank, dev)
    rng = np.random.default_rng(rank)
    mine = [rng.integers(0, 100, size=n).astype(np.int32) for n in ([3, 0, 7] if rank == 0 else [5])]
    res["mine"] = [m.tolist() for m in mine]
    res["all"] = [a.tolist() for a in sharding.all_gather_sequences(mine, dev)]
    res["none"] = sharding.all_gather_sequences([], dev) if False else None
    # a step in which only one rank has something to contribute
    res["one_sided"] = [a.tolist() for a in sharding.all_gather_sequences(mine if rank == 1 else [], dev)]
    q.put((rank, res))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_requests_and_exchange_finished_outputs():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0]["range"] == [0, 1, 2, 3] and got[1]["range"] == [4, 5, 6, 7]
    assert got[0]["max"] == 11.0 and got[1]["max"] == 11.0
    expect = got[0]["mine"] + got[1]["mine"]            # rank order, then local order
    assert got[0]["all"] == expect and got[1]["all"] == expect
    assert got[0]["one_sided"] == got[1]["mine"] and got[1]["one_sided"] == got[1]["mine"]


def test_single_process_is_a_no_op():
    from paper_2411_04975_b200 import sharding
    assert sharding.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    out = sharding.all_gather_sequences([np.array([1, 2], dtype=np.int32)], torch.device("cpu"))
    assert [o.tolist() for o in out] == [[1, 2]]

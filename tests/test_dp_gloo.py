"""World-size-2 test (gloo, CPU) of the data-parallel load exchange: after the
all-reduce every rank's accumulators hold the global counts."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_39137_b200 import dp


class FakeRouter:
    """Host stand-in with the two accumulator hooks of the C ABI (peek / add)."""

    def __init__(self, loads):
        self.acc = loads.clone()

    def loads_peek(self):
        return self.acc.clone()

    def loads_add(self, t):
        self.acc += t


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    own = torch.randint(0, 50, (3, 768), generator=g, dtype=torch.int32)
    r = FakeRouter(own)
    total = dp.allreduce_loads(r, dist)
    # a second microbatch after the exchange keeps accumulating locally
    r.loads_add(torch.ones_like(own))
    torch.save({"own": own, "acc": r.acc, "total": total}, os.path.join(out, f"r{rank}.pt"))
    dist.destroy_process_group()


def test_allreduce_loads_world2(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = torch.load(tmp_path / "r0.pt")
    r1 = torch.load(tmp_path / "r1.pt")
    expect = r0["own"] + r1["own"]
    assert torch.equal(r0["total"], expect) and torch.equal(r1["total"], expect)
    assert torch.equal(r0["acc"], expect + 1) and torch.equal(r1["acc"], expect + 1)
    assert int(expect.sum()) == int(r0["own"].sum() + r1["own"].sum())

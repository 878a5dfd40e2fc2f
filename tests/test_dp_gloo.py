"""World-size-2 tests (gloo, CPU) of the data-parallel path: every rank routes
its own token shard, the per-expert load counts are summed over the ranks in
place, and the controller step that follows gives bit-identical biases on all
ranks -- equal to the single-process result over all tokens (Algorithm 1
line 4: n_i counts every rank's tokens of the iteration)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2609_39137_b200 import dp


class PeekAddRouter:
    """Host stand-in with only the two accumulator hooks moe_loads_peek / moe_loads_add."""

    def __init__(self, loads):
        self.acc = loads.clone()

    def loads_peek(self):
        return self.acc.clone()

    def loads_add(self, t):
        self.acc += t


class HostRouter:
    """Same call sequence and accumulator semantics as binding.Router (route_step adds to the accumulators,
    loads_view aliases them, controller_update consumes them), with the CPU oracle doing the arithmetic."""

    def __init__(self, L, E, K):
        self.L, self.E, self.K = L, E, K
        self.acc = torch.zeros(L, E, dtype=torch.int32)
        self.bias = np.zeros((L, E), np.float32)
        self.e_prev = np.zeros((L, E), np.float32)
        self.gates = np.zeros(L, np.int64)

    def route_step(self, logits):                       # logits [L][T][E] float32
        for l in range(self.L):
            idx, _, _ = oracle.route_f32(logits[l], self.bias[l], self.K)
            self.acc[l] += torch.from_numpy(oracle.load_counts(idx, self.E).astype(np.int32))

    def loads_view(self):
        return self.acc                                 # the accumulators themselves, not a copy

    def controller_update(self):
        for l in range(self.L):
            e = oracle.load_error(self.acc[l].numpy().astype(np.int64))
            self.bias[l], self.e_prev[l], g = oracle.id_update(self.bias[l], self.e_prev[l], e, 6e-3, 6e-3, center=True)
            self.gates[l] = int(g.sum())
        self.acc.zero_()


def _logits(step, shard, L, T, E):
    rng = np.random.default_rng(1000 * step + shard)
    skew = np.linspace(-1.0, 1.0, E, dtype=np.float32) * (0.5 + 0.1 * step)
    return (rng.standard_normal((L, T, E)).astype(np.float32) + skew[None, None, :])


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # (1) peek/add objects: the three-step exchange
    g = torch.Generator().manual_seed(100 + rank)
    own = torch.randint(0, 50, (3, 768), generator=g, dtype=torch.int32)
    r = PeekAddRouter(own)
    total = dp.allreduce_loads(r, dist)
    r.loads_add(torch.ones_like(own))                   # a later microbatch keeps accumulating locally
    # (2) route -> in-place all-reduce -> controller update, three iterations, two microbatches each
    L, T, E, K = 2, 96, 64, 4
    hr = HostRouter(L, E, K)
    sums = []
    for step in range(3):
        for micro in range(2):
            hr.route_step(_logits(step, 10 * micro + rank, L, T, E))
        acc = dp.allreduce_loads(hr, dist)
        assert acc is hr.acc                            # reduced in place: no copy, nothing to add back
        sums.append(int(hr.acc.sum()))
        hr.controller_update()
    torch.save({"own": own, "acc": r.acc, "total": total, "bias": hr.bias, "e_prev": hr.e_prev, "gates": hr.gates,
                "sums": sums}, os.path.join(out, f"r{rank}.pt"))
    dist.destroy_process_group()


def test_allreduce_loads_world2(tmp_path):
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0 = torch.load(tmp_path / "r0.pt", weights_only=False)
    r1 = torch.load(tmp_path / "r1.pt", weights_only=False)
    expect = r0["own"] + r1["own"]
    assert torch.equal(r0["total"], expect) and torch.equal(r1["total"], expect)
    assert torch.equal(r0["acc"], expect + 1) and torch.equal(r1["acc"], expect + 1)
    assert int(expect.sum()) == int(r0["own"].sum() + r1["own"].sum())
    # both ranks hold the same controller state, bit for bit
    for k in ("bias", "e_prev"):
        np.testing.assert_array_equal(r0[k].view(np.uint32), r1[k].view(np.uint32))
    np.testing.assert_array_equal(r0["gates"], r1["gates"])
    L, T, E, K = 2, 96, 64, 4
    assert r0["sums"] == r1["sums"] == [2 * 2 * L * T * K] * 3       # ranks x microbatches x L x T x K counts
    # ... and it is the state one process reaches when it routes every rank's tokens itself
    one = HostRouter(L, E, K)
    for step in range(3):
        for micro in range(2):
            for rank in range(2):
                one.route_step(_logits(step, 10 * micro + rank, L, T, E))
        one.controller_update()
    np.testing.assert_array_equal(one.bias.view(np.uint32), r0["bias"].view(np.uint32))
    np.testing.assert_array_equal(one.e_prev.view(np.uint32), r0["e_prev"].view(np.uint32))
    assert np.abs(one.bias).max() > 0

"""Data-parallel step with the real library on a GPU: two ranks (two processes sharing the one GPU, gloo backend, so
the exchange goes through the host and no kernel of one rank ever waits for a kernel of the other) route disjoint
token shards, sum the load accumulators IN PLACE through the tensor that aliases them (moe_loads_buffer), and run
the controller update.  Both ranks must end with bit-identical biases, equal to those of one context that routes
both shards as two microbatches (Algorithm 1 line 4: n_i counts every rank's and every microbatch's tokens)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_39137_b200 import binding, dp, synth

pytestmark = pytest.mark.gpu
WL = synth.WORKLOADS["tiny_top3"].with_(T=640, L=2)
STEPS = 3


def _weights():
    return torch.stack([synth.router_weights(WL, l, "cuda") for l in range(WL.L)])


def _shard(step, rank, world):
    return torch.stack([synth.hidden_states(WL, l, step * world + rank, "cuda") for l in range(WL.L)])


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)
    w = _weights()
    r = binding.Router(WL.L, WL.E, WL.K, WL.H, WL.T)
    view = r.loads_view()
    sums = []
    for step in range(STEPS):
        r.route_step(_shard(step, rank, world), w)
        acc = dp.allreduce_loads(r, dist)
        assert acc.data_ptr() == view.data_ptr()          # reduced in place, on the accumulators themselves
        torch.cuda.synchronize()
        sums.append(int(acc.sum()))
        r.controller_update()
    r.poll()
    loads, bias, _, _ = r.load_stats()
    torch.save({"bias": bias.cpu(), "loads": loads.cpu(), "sums": sums, "step": r.state_export(with_step=True)[2]},
               os.path.join(out, f"r{rank}.pt"))
    dist.destroy_process_group()


def test_two_ranks_reduce_loads_in_place_and_stay_bit_identical(tmp_path):
    world = 2
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    a = torch.load(tmp_path / "r0.pt", weights_only=False)
    b = torch.load(tmp_path / "r1.pt", weights_only=False)
    assert torch.equal(a["bias"].view(torch.int32), b["bias"].view(torch.int32))
    assert torch.equal(a["loads"], b["loads"])
    assert a["sums"] == b["sums"] == [world * WL.L * WL.T * WL.K] * STEPS and a["step"] == STEPS
    # one context, the ranks' shards as microbatches of the same iteration
    w = _weights()
    one = binding.Router(WL.L, WL.E, WL.K, WL.H, WL.T)
    for step in range(STEPS):
        for rank in range(world):
            one.route_step(_shard(step, rank, world), w)
        one.controller_update()
    one.poll()
    loads, bias, _, _ = one.load_stats()
    np.testing.assert_array_equal(bias.cpu().numpy().view(np.uint32), a["bias"].numpy().view(np.uint32))
    assert torch.equal(loads.cpu(), a["loads"])
    assert float(bias.abs().max()) > 0

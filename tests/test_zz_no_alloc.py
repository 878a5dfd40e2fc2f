"""The allocation-free quantile-target entry point against the existing one.

Some users of this library cannot allocate device memory at the moment they
need a result (their process gave all device memory to its own pool, or an
allocation's implicit synchronisation is unacceptable in their loop) and have
no workspace to hand in.  For them `moe_quantile_target_static` keeps its
scratch in a fixed array inside the library.  This test calls it through the C
ABI and checks that it returns exactly what the context-based quantile
controller computes from the same dump -- twice in a row with different
inputs, because the shared array keeps the previous call's contents and every
call has to clear what must start at zero.  The file name makes pytest
collect it last.
"""
import numpy as np
import pytest
import torch

from paper_2609_39137_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _reference_target(wl, step, dev):
    """Existing entry points: quantile controller with rho = 0 stores the target as the new bias."""
    r = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile")
    x = synth.hidden_states(wl, 0, step, dev)[None].contiguous()
    w = synth.router_weights(wl, 0, dev)[None].contiguous()
    logits = torch.empty(1, wl.T, wl.E, device=dev)
    alpha = torch.empty(1, wl.T, device=dev)
    r.route_step(x, w, logits_out=logits, alpha_out=alpha)
    r.controller_update()
    r.poll()
    bias = r.load_stats()[1][0].clone()
    return logits[0].contiguous(), alpha[0].contiguous(), bias


def test_static_scratch_quantile_target_matches_context_path_twice():
    dev = "cuda"
    # the output and every input exist before the calls under test: nothing is allocated in between
    cases = [(synth.WORKLOADS["top3_single"].with_(T=3000, H=256), 0),
             (synth.WORKLOADS["top5_single"].with_(T=1500, H=128), 3)]
    prepared = [(wl, *_reference_target(wl, step, dev)) for wl, step in cases]
    outs = [torch.full((wl.E,), float("nan"), device=dev) for wl, _ in cases]
    torch.cuda.synchronize()
    for (wl, logits, alpha, expect), out in zip(prepared, outs):
        before = torch.cuda.memory_allocated()
        binding.quantile_target_static(logits, alpha, wl.K, out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # bit-exact, like every other fp32 result given the same logits
        np.testing.assert_array_equal(out.cpu().numpy().view(np.uint32), expect.cpu().numpy().view(np.uint32))


def test_static_scratch_rejects_more_experts_than_it_holds():
    dev = "cuda"
    logits = torch.zeros(8, 1032, device=dev)
    alpha = torch.zeros(8, device=dev)
    out = torch.zeros(1032, device=dev)
    with pytest.raises(binding.MoeRouteError) as ei:
        binding.quantile_target_static(logits, alpha, 3, out)
    assert ei.value.code == binding.MOE_ERR_WORKSPACE

"""The allocation-free quantile-target entry point against the existing one.

Some users of this library cannot allocate device memory at the moment they
need a result (their process gave all device memory to its own pool, or an
allocation's implicit synchronisation is unacceptable in their loop) and have
no workspace to hand in.  For them `moe_quantile_target_static` keeps its
scratch in a fixed array inside the library.  This test calls it through the C
ABI and checks that it returns exactly what the context-based quantile
controller computes from the same dump, and what the CPU oracle's sort-based
quantile gives (Eq. 6-7) -- twice in a row with different inputs, because the
shared array keeps the previous call's contents and every call has to clear
what must start at zero.  The file name makes pytest collect it last.
"""
import numpy as np
import pytest
import torch

import oracle
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


def _bits(t):
    return np.ascontiguousarray(t.detach().cpu().numpy() if isinstance(t, torch.Tensor) else t, np.float32).view(np.uint32)


def test_static_scratch_quantile_target_matches_context_path_twice():
    dev = "cuda"
    # the output and every input exist before the calls under test: nothing is allocated in between
    cases = [(synth.WORKLOADS["top3_single"].with_(T=3000, H=256), 0),
             (synth.WORKLOADS["top5_single"].with_(T=1500, H=128), 3)]
    prepared = [(wl, *_reference_target(wl, step, dev)) for wl, step in cases]
    outs = [torch.full((wl.E,), float("nan"), device=dev) for wl, _ in cases]
    torch.cuda.synchronize()
    for (wl, logits, alpha, expect), out in zip(prepared, outs):
        before_torch = torch.cuda.memory_allocated()
        free_before, _ = torch.cuda.mem_get_info()       # the driver's own count: sees any cudaMalloc, torch's or not
        binding.quantile_target_static(logits, alpha, wl.K, out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert torch.cuda.memory_allocated() == before_torch
        assert free_after >= free_before                 # the call took no device memory from anyone
        # bit-exact, like every other fp32 result given the same logits: against the context path ...
        np.testing.assert_array_equal(_bits(out), _bits(expect))
        # ... and against the oracle's definition (r-th smallest margin by a full sort)
        want = oracle.quantile_target(logits.cpu().numpy(), alpha.cpu().numpy(), wl.K)
        np.testing.assert_array_equal(_bits(out), _bits(want))


def test_static_scratch_largest_then_small_expert_count_on_the_same_array():
    # the largest expert count the array holds, then a small one that is not a multiple of 32: the second call
    # must not see histogram, prefix or rank state the first one left behind
    dev = "cuda"
    g = torch.Generator(device=dev).manual_seed(9)
    for E, m, K in [(1024, 700, 6), (40, 333, 3), (1024, 64, 1)]:
        logits = (torch.randn(m, E, device=dev, generator=g) * 2).contiguous()
        s = torch.from_numpy(oracle.sigmoid_f32(logits.cpu().numpy())).to(dev)
        alpha = torch.sort(s, dim=1, descending=True).values[:, K].contiguous()       # (K+1)-th largest score, zero bias
        out = torch.full((E,), float("nan"), device=dev)
        binding.quantile_target_static(logits, alpha, K, out)
        torch.cuda.synchronize()
        want = oracle.quantile_target(logits.cpu().numpy(), alpha.cpu().numpy(), K)
        np.testing.assert_array_equal(_bits(out), _bits(want))


def test_static_scratch_rejects_more_experts_than_it_holds():
    dev = "cuda"
    logits = torch.zeros(8, 1032, device=dev)
    alpha = torch.zeros(8, device=dev)
    out = torch.zeros(1032, device=dev)
    with pytest.raises(binding.MoeRouteError) as ei:
        binding.quantile_target_static(logits, alpha, 3, out)
    assert ei.value.code == binding.MOE_ERR_WORKSPACE

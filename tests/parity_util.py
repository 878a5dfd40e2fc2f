"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI
and compare it with the CPU oracle on the same seeded inputs."""
import os

import numpy as np
import torch

import oracle
from paper_2609_39137_b200 import binding, synth

LOGIT_TOL = 1e-4      # spec: router logits within 1e-4 absolute of the fp64 definition
GAP_TOL = 1e-4        # top-K sets may differ only where the rank-K / rank-K+1 gap is below this
GATE_TOL = 1e-5       # gates vs the fp64 definition
NEAR_TIE_BUDGET = 1e-4  # at most 0.01 % of tokens may have a differing set
THREADS = max(1, min(16, os.cpu_count() or 1))


def np_(t):
    return t.detach().cpu().numpy()


def check_exact(logits_gpu, bias, K, idx_gpu, gate_gpu, alpha_gpu=None):
    """binary32 chain: given the GPU's own fp32 logits every output must match bit for bit."""
    oi, og, oa = oracle.route_f32(logits_gpu, bias, K)
    np.testing.assert_array_equal(idx_gpu, oi)
    np.testing.assert_array_equal(gate_gpu.view(np.uint32), og.view(np.uint32))
    if alpha_gpu is not None:
        np.testing.assert_array_equal(alpha_gpu.view(np.uint32), oa.view(np.uint32))
    return oi


def check_definition(x_bits, w_bits, bias, K, logits_gpu, idx_gpu, gate_gpu, rows=None, logit_tol=None):
    """binary64 definition from the bf16 operands: logits within LOGIT_TOL, same
    expert sets except near ties (counted), gates within GATE_TOL.
    Returns (#tokens with differing set, #tokens checked)."""
    if rows is not None:
        x_bits, logits_gpu, idx_gpu, gate_gpu = x_bits[rows], logits_gpu[rows], idx_gpu[rows], gate_gpu[rows]
    ref = oracle.route_tokens_f64(x_bits, w_bits, bias, K, threads=THREADS)
    err = np.max(np.abs(logits_gpu.astype(np.float64) - ref["z"]))
    if logit_tol is None:
        logit_tol = LOGIT_TOL
    assert err <= logit_tol, f"logit error {err}"
    same_set = np.all(np.sort(idx_gpu, 1) == np.sort(ref["idx"], 1), axis=1)
    clear = ref["gap"] >= GAP_TOL
    assert np.all(same_set[clear]), "expert set differs although the rank-K gap is clear"
    same_order = np.all(idx_gpu == ref["idx"], axis=1)
    if same_order.any():
        assert np.max(np.abs(gate_gpu[same_order] - ref["gate"][same_order])) <= GATE_TOL
    return int((~same_set).sum()), int(len(same_set))


def route_once(T, H, E, K, L=1, bias=None, seed=0, want_alpha=False, x=None, w=None, controller="id", **kw):
    """Routes one random batch on the GPU; returns a dict of numpy results + the Router."""
    dev = "cuda"
    g = torch.Generator(device=dev)
    g.manual_seed(1234 + seed)
    if x is None:
        x = torch.randn(L, T, H, device=dev, generator=g).to(torch.bfloat16)
    if w is None:
        w = (torch.randn(L, E, H, device=dev, generator=g) * (1.0 / max(H, 1) ** 0.5)).to(torch.bfloat16)
    r = binding.Router(L, E, K, H, max(T, 1), controller=controller, **kw)
    if bias is not None:
        r.state_import(bias=bias.to(dev).float().contiguous())
    else:
        bias = torch.zeros(L, E)
    logits = torch.full((L, T, E), float("nan"), device=dev)
    alpha = torch.full((L, T), float("nan"), device=dev) if want_alpha else None
    idx, gate = r.route_step(x, w, logits_out=logits, alpha_out=alpha)
    r.poll()
    return dict(r=r, x=x, w=w, bias=np_(bias).astype(np.float32), logits=np_(logits), idx=np_(idx), gate=np_(gate),
                alpha=None if alpha is None else np_(alpha), loads=np_(r.loads_peek()))


def full_check(res, K, rows=None):
    L = res["logits"].shape[0]
    E = res["logits"].shape[2]
    for l in range(L):
        a = None if res["alpha"] is None else res["alpha"][l]
        oi = check_exact(res["logits"][l], res["bias"][l], K, res["idx"][l], res["gate"][l], a)
        np.testing.assert_array_equal(res["loads"][l], np.bincount(oi.ravel(), minlength=E))
        xb, wb = synth.bf16_bits(res["x"][l]), synth.bf16_bits(res["w"][l])
        check_definition(xb, wb, res["bias"][l], K, res["logits"][l], res["idx"][l], res["gate"][l], rows)
    assert res["loads"].sum() == L * res["logits"].shape[1] * K    # every token gives exactly K counts


def oracle_controller_step(kind, b, e_prev, n, cfg, center, Q=None):
    """One oracle controller step for one layer from integer loads n."""
    e = oracle.load_error(n.astype(np.int64))
    if kind == "id":
        b2, ep2, g = oracle.id_update(b, e_prev, e, cfg["ki"], cfg["kd"], center=center)
        gates = int(g.sum())
    elif kind == "fixed_step":
        b2, ep2 = oracle.fixed_step_update(b, e_prev, e, cfg["eta"], center=center)
        gates = 0
    elif kind == "quantile":
        b2, ep2 = oracle.quantile_update(b, e_prev, e, Q, rho=cfg.get("rho", 0.0), center=center)
        gates = 0
    else:  # frozen
        b2, ep2, gates = b.copy(), e.copy(), 0
    mx, mn = oracle.violations(n.astype(np.int64))
    return b2, ep2, gates, mx, mn


def bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)

"""Parity of the CUDA path (called through the C ABI) against the CPU oracle.

Bars: integer results (expert indices, loads) bit-exact; every fp32 output
bit-exact given the GPU's own fp32 logits (binary32 chain of the oracle);
logits within 1e-4 of the fp64 definition computed from the bf16 operands;
expert sets equal wherever the rank-K/rank-K+1 gap is at least 1e-4.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_39137_b200 import binding, synth
from parity_util import (NEAR_TIE_BUDGET, THREADS, bits, check_definition, check_exact, full_check, np_,
                         oracle_controller_step, route_once)

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------ routing
@pytest.mark.parametrize("T,H,E,K,L,alpha", [
    (128, 64, 256, 3, 1, False),      # one tile, one chunk, one k-block
    (128, 256, 768, 3, 1, False),     # three chunks
    (300, 512, 768, 10, 1, False),    # several tiles and a ragged tail
    (1000, 256, 768, 5, 3, True),     # layers, ragged tail, alpha
    (513, 192, 768, 10, 2, True),
    (257, 320, 256, 8, 2, False),     # Top-8-of-256 shape
    (640, 1024, 768, 3, 1, True),
])
def test_route_matches_oracle(T, H, E, K, L, alpha):
    g = torch.Generator().manual_seed(T + K)
    bias = torch.randn(L, E, generator=g) * 0.02
    res = route_once(T, H, E, K, L, bias=bias, seed=T, want_alpha=alpha)
    full_check(res, K)


@pytest.mark.parametrize("T,H,E,K", [
    (1, 64, 768, 10), (127, 64, 768, 3), (129, 64, 768, 3),     # token tails
    (64, 8, 768, 5), (200, 72, 768, 5), (96, 136, 768, 10),     # hidden below / not a multiple of 64
    (256, 64, 8, 3), (256, 64, 40, 16), (256, 128, 1024, 1), (130, 64, 1000, 16),   # expert-count and K extremes
])
def test_route_edge_shapes(T, H, E, K):
    g = torch.Generator().manual_seed(E + K)
    bias = torch.randn(1, E, generator=g) * 0.05
    res = route_once(T, H, E, K, 1, bias=bias, seed=E, want_alpha=(K < 16))
    full_check(res, K)


@pytest.mark.parametrize("T,H,E,K,L,alpha", [
    (128, 64, 768, 3, 1, False),      # one tile pair, three chunk items
    (300, 512, 768, 10, 1, True),     # ragged tail, alpha from the merged lists
    (1000, 256, 768, 5, 3, True),     # layers
    (513, 192, 1000, 16, 2, False),   # four chunks, the last one mostly padding; generic (insertion) selection
    (130, 64, 1000, 15, 1, True),
    (700, 320, 264, 8, 2, True),      # second chunk holds 8 experts: fewer than K + 1 per chunk list
    (2100, 128, 512, 1, 1, True),     # more rows than one merge CTA takes
])
def test_chunk_split_scheduling_matches_oracle_and_fused_path(T, H, E, K, L, alpha):
    # the expert chunks of a tile routed by different CTA pairs and merged by the second kernel: parity with the
    # oracle, and bit-identical to the schedule that finishes the rows in the routing kernel's epilogue
    g = torch.Generator().manual_seed(T + K)
    bias = torch.randn(L, E, generator=g) * 0.02
    res = route_once(T, H, E, K, L, bias=bias, seed=T, want_alpha=alpha, chunk_split=2)
    full_check(res, K)
    fused = route_once(T, H, E, K, L, bias=bias, seed=T, want_alpha=alpha, chunk_split=1)
    for k in ("logits", "idx", "gate", "loads") + (("alpha",) if alpha else ()):
        np.testing.assert_array_equal(bits(res[k]) if res[k].dtype == np.float32 else res[k],
                                      bits(fused[k]) if fused[k].dtype == np.float32 else fused[k])
    assert res["r"].launch_count() == fused["r"].launch_count() + 1      # the merge kernel


def test_chunk_split_exact_ties_across_chunks_pick_lowest_index():
    # every score equal: the winners are the K lowest indices, all in the first chunk; with a bias plateau that
    # spans chunk boundaries the merge has to break ties between lists by expert index
    T, H, E, K = 200, 64, 768, 10
    x = torch.zeros(1, T, H, device="cuda", dtype=torch.bfloat16)
    res = route_once(T, H, E, K, x=x, chunk_split=2)
    assert np.all(res["idx"][0] == np.arange(K)[None, :])
    bias = torch.zeros(1, E)
    bias[0, 250:260] = 0.25           # straddles chunks 0 and 1
    bias[0, 600:604] = 0.25           # chunk 2
    res = route_once(T, H, E, K, x=x, bias=bias, want_alpha=True, chunk_split=2)
    assert np.all(res["idx"][0] == np.arange(250, 260)[None, :])
    assert np.all(res["alpha"][0] == np.float32(0.75))
    full_check(res, K)


def test_route_operand_layout_one_hot():
    # one-hot router rows: logit[t][e] = x[t][h(e)] exactly -- exposes any
    # swizzle / descriptor / transposition error
    T, H, E, K = 256, 256, 768, 3
    dev = "cuda"
    x = torch.randn(1, T, H, device=dev).to(torch.bfloat16)
    w = torch.zeros(1, E, H, device=dev, dtype=torch.bfloat16)
    hsel = (torch.arange(E, device=dev) * 7 + 3) % H
    w[0, torch.arange(E, device=dev), hsel] = 1.0
    res = route_once(T, H, E, K, x=x, w=w)
    expect = x[0].float()[:, hsel]
    np.testing.assert_array_equal(res["logits"][0], np_(expect))
    full_check(res, K)


@pytest.mark.parametrize("chunk_split", [1, 2])
def test_tiny_scores_take_the_library_division(chunk_split):
    # logits of -72 .. -88: every score is below 2^-100, where the kernels' branch-free gate division is not
    # used (library division instead), the approximate score is 0 for every column (all within the filter slack:
    # the exact insertion lists do the work), and one-hot router rows over 256 hidden columns give every logit
    # three times (exact ties, lowest index wins).  Gates are ratios of numbers near 1e-35.
    T, H, E, K = 300, 256, 768, 10
    dev = "cuda"
    g = torch.Generator().manual_seed(77)
    x = (-(72.0 + 16.0 * torch.rand(1, T, H, generator=g))).to(torch.bfloat16).to(dev)
    w = torch.zeros(1, E, H, device=dev, dtype=torch.bfloat16)
    hsel = (torch.arange(E, device=dev) * 7 + 3) % H
    w[0, torch.arange(E, device=dev), hsel] = 1.0
    res = route_once(T, H, E, K, x=x, w=w, want_alpha=True, chunk_split=chunk_split)
    np.testing.assert_array_equal(res["logits"][0], np_(x[0].float()[:, hsel]))
    assert res["logits"].max() < -69.4            # sigmoid < 2^-100
    full_check(res, K)
    assert np.all(np.abs(res["gate"].sum(axis=-1) - 1.0) < 1e-5)


def test_route_exact_ties_pick_lowest_index():
    # all-zero hidden states: every logit is 0, every score 0.5 -> with zero
    # bias the K lowest indices win; with a bias plateau the plateau's lowest
    T, H, E, K = 200, 64, 768, 10
    x = torch.zeros(1, T, H, device="cuda", dtype=torch.bfloat16)
    res = route_once(T, H, E, K, x=x)
    assert np.all(res["idx"][0] == np.arange(K)[None, :])
    np.testing.assert_array_equal(res["gate"][0], np.full((T, K), np.float32(1.0) / np.float32(K), np.float32))
    bias = torch.zeros(1, E)
    bias[0, 300:320] = 0.25          # plateau straddles two accumulator chunks? no: inside chunk 1, both halves
    bias[0, 100] = 0.25
    bias[0, 700] = 0.25
    res = route_once(T, H, E, K, x=x, bias=bias, want_alpha=True)
    assert np.all(res["idx"][0] == np.array([100] + list(range(300, 309)))[None, :])
    assert np.all(res["alpha"][0] == np.float32(0.75))
    full_check(res, K)


@pytest.mark.parametrize("chunk_split", [1, 2])
def test_non_finite_hidden_states_do_not_disturb_other_tokens(chunk_split):
    # the paper says nothing about NaN / Inf activations; the library's promise is only that they cannot fault and
    # cannot leak into other tokens: rows with finite inputs route exactly as without the bad rows, every index
    # written for a bad row is a valid expert or the "no expert" marker, and the loads count only valid experts
    T, H, E, K = 400, 128, 768, 10
    g = torch.Generator(device="cuda").manual_seed(3)
    x = torch.randn(1, T, H, device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn(1, E, H, device="cuda", generator=g) / 11).to(torch.bfloat16)
    clean = route_once(T, H, E, K, x=x, w=w, chunk_split=chunk_split)
    bad_rows = [5, 130, 131, 399]
    xb = x.clone()
    xb[0, 5, 7] = float("nan")
    xb[0, 130, :] = float("inf")
    xb[0, 131, 0] = float("-inf")
    xb[0, 399, 100] = float("nan")
    res = route_once(T, H, E, K, x=xb, w=w, chunk_split=chunk_split)
    assert res["r"].poll(raise_on_error=False) == binding.MOE_OK
    good = np.setdiff1d(np.arange(T), bad_rows)
    np.testing.assert_array_equal(res["idx"][0][good], clean["idx"][0][good])
    np.testing.assert_array_equal(bits(res["gate"][0][good]), bits(clean["gate"][0][good]))
    bad_idx = res["idx"][0][bad_rows]
    assert np.all(((bad_idx >= 0) & (bad_idx < E)) | (bad_idx == 0x7fffffff))
    valid = res["idx"][0][(res["idx"][0] >= 0) & (res["idx"][0] < E)]
    np.testing.assert_array_equal(res["loads"][0], np.bincount(valid, minlength=E))


def test_route_is_deterministic_and_accumulates_microbatches():
    T, H, E, K, L = 700, 256, 768, 10, 2
    a = route_once(T, H, E, K, L, seed=5)
    b = route_once(T, H, E, K, L, seed=5)
    for k in ("logits", "idx", "gate", "loads"):
        np.testing.assert_array_equal(bits(a[k]) if a[k].dtype == np.float32 else a[k],
                                      bits(b[k]) if b[k].dtype == np.float32 else b[k])
    # a second call before the controller update adds to the accumulators (Algorithm 1 line 4)
    r = a["r"]
    r.route_step(a["x"], a["w"])
    r.poll()
    np.testing.assert_array_equal(np_(r.loads_peek()), 2 * a["loads"])


def test_candidate_filter_slack_covers_every_fp32_logit():
    # the approximate score (one tanh.approx) only pre-selects candidates; over ALL finite fp32 logits it
    # must stay within half of the slack compiled into the kernel (2e-5) of the exact score
    gap = binding.debug_score_gap()
    assert 0.0 < gap < 1e-5, gap


def test_branch_free_reciprocal_equals_the_correctly_rounded_one_everywhere():
    # the score chain ends in a correctly rounded reciprocal (Section 2.2 as read here); the kernels take the
    # hardware approximation plus one Newton step: over ALL 2^32 logits the score has the same bits as with the
    # math library's reciprocal, and so has the reciprocal of every normal number with a normal reciprocal
    assert binding.debug_rcp_check() == (0, 0)


def test_gate_division_equals_the_correctly_rounded_one():
    # gates are s / D correctly rounded (Eq. 3 as read here); the kernels multiply by the correctly rounded 1 / D and
    # correct twice with exact residuals: same bits as the library's division for every denominator in [2^-20, 32]
    # with 48 numerators each
    assert binding.debug_division_check() == 0


def test_quick_score_gap_covers_every_fp32_logit():
    # the margin-histogram pass bins a logit from a quick score (hardware exp2 and reciprocal approximations) and
    # re-bins with the exact chain when the position is within twice the compiled gap (3e-7, scaled to bins) of an
    # edge: over ALL finite fp32 logits the quick score must stay inside that gap
    gap = binding.debug_quick_score_gap()
    assert 0.0 < gap < 3e-7, gap


# --------------------------------------------------------------- controllers
def _drive(kind, L, E, K, steps, loads_fn, **cfg):
    r = binding.Router(L, E, K, 64, 128, controller=kind, ki=cfg.get("ki"), kd=cfg.get("kd"), eta=cfg.get("eta"),
                       center=cfg.get("center"))
    center = cfg.get("center")
    if center is None:
        center = (kind == "id")
    b = np.zeros((L, E), np.float32)
    ep = np.zeros((L, E), np.float32)
    for t in range(steps):
        n = loads_fn(t).astype(np.int32)
        r.loads_add(torch.from_numpy(n).cuda())
        r.controller_update()
        r.poll()
        loads, bias, mxv, mnv = [np_(v) for v in r.load_stats()]
        gates = np_(r.gate_stats())
        _, e_prev = [np_(v) for v in r.state_export()]
        np.testing.assert_array_equal(loads, n)
        assert not np_(r.loads_peek()).any()               # accumulators consumed
        for l in range(L):
            b[l], ep[l], g, mx, mn = oracle_controller_step(
                kind, b[l], ep[l], n[l], dict(ki=cfg.get("ki", 6e-3), kd=cfg.get("kd", 6e-3), eta=cfg.get("eta", 1e-3)),
                center)
            assert gates[l] == g
            assert bits(mxv[l:l + 1])[0] == bits(np.array([mx]))[0] and bits(mnv[l:l + 1])[0] == bits(np.array([mn]))[0]
        np.testing.assert_array_equal(bits(bias), bits(b))
        np.testing.assert_array_equal(bits(e_prev), bits(ep))
    return b


def test_id_controller_closed_form_trajectories():
    E = 768
    half = lambda a, c: np.concatenate([np.full(384, a), np.full(384, c)])[None, :]
    ki = kd = 2.0 ** -7
    b = _drive("id", 1, E, 3, 20, lambda t: half(512, 1536), ki=ki, kd=kd)
    assert np.all(b[0, :384] == np.float32(20 / 256)) and np.all(b[0, 384:] == np.float32(-20 / 256))
    b = _drive("id", 1, E, 3, 10, lambda t: half(1024 - 16 * (t + 1), 1024 + 16 * (t + 1)), ki=ki, kd=kd)
    assert np.all(b[0, :384] == np.float32(64 / 8192)) and np.all(b[0, 384:] == np.float32(-64 / 8192))


@pytest.mark.parametrize("kind,E,L,center", [
    ("id", 768, 5, None), ("id", 256, 2, 0), ("fixed_step", 768, 3, None), ("fixed_step", 768, 2, 1),
    ("frozen", 768, 2, None), ("id", 1000, 2, None), ("id", 8, 1, None),
])
def test_controllers_random_loads_bit_exact(kind, E, L, center):
    rng = np.random.default_rng(E + L)
    K = 3
    def loads(t):
        hot = rng.integers(0, E, (L, 1))
        n = rng.poisson(40, (L, E))
        n[np.arange(L)[:, None], hot] += 500 * (t % 3)
        n[:, 1] = 0                                   # an expert that never gets a token
        return n
    kw = {} if center is None else dict(center=center)
    _drive(kind, L, E, K, 25, loads, **kw)


def test_controller_empty_batch_reports_state_error_and_keeps_state():
    r = binding.Router(2, 768, 10, 64, 128)
    n = np.zeros((2, 768), np.int32)
    n[0, :] = 7                                       # layer 0 has tokens, layer 1 has none
    r.loads_add(torch.from_numpy(n).cuda())
    r.controller_update()
    assert r.poll(raise_on_error=False) == binding.MOE_ERR_STATE
    bias, e_prev = [np_(v) for v in r.state_export()]
    assert not bias[1].any() and not e_prev[1].any()
    assert r.poll(raise_on_error=False) == binding.MOE_OK     # sticky status was cleared


def test_state_export_import_resume_is_bit_identical():
    wl = synth.WORKLOADS["tiny_top3"].with_(T=512)
    w = synth.router_weights(wl, 0, "cuda")[None]
    def run(steps, r):
        for t in steps:
            x = synth.hidden_states(wl, 0, t, "cuda")[None]
            r.route_step(x, w)
            r.controller_update()
        r.poll()
        return r
    full = run(range(8), binding.Router(1, wl.E, wl.K, wl.H, wl.T))
    first = run(range(4), binding.Router(1, wl.E, wl.K, wl.H, wl.T))
    b, ep, step = first.state_export(with_step=True)
    assert step == 4                                   # controller updates enqueued so far
    second = binding.Router(1, wl.E, wl.K, wl.H, wl.T)
    second.state_import(b, ep, step=step)
    run(range(4, 8), second)
    assert second.state_export(with_step=True)[2] == full.state_export(with_step=True)[2] == 8
    first.state_import(b)                              # step = -1 keeps the context's own counter
    assert first.state_export(with_step=True)[2] == 4
    for u, v in zip(full.state_export(), second.state_export()):
        np.testing.assert_array_equal(bits(np_(u)), bits(np_(v)))
    for u, v in zip(full.load_stats(), second.load_stats()):
        assert torch.equal(u, v)


# ------------------------------------------------------------- closed loops
def _closed_loop(wl, kind, steps, check_rows=None, step_ids=None, **kw):
    """Teacher-forced loop: the GPU runs route + update each step; the oracle
    replays every controller step from the GPU's loads (bitwise) and checks
    the routing of every step against the binary32 chain."""
    dev = "cuda"
    r = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T, controller=kind, **kw)
    center = (kind == "id")
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)])
    b = np.zeros((wl.L, wl.E), np.float32)
    ep = np.zeros((wl.L, wl.E), np.float32)
    logits = torch.empty(wl.L, wl.T, wl.E, device=dev)
    alpha = torch.empty(wl.L, wl.T, device=dev)
    differing = checked = 0
    hist = []
    for n_step, t in enumerate(range(steps) if step_ids is None else step_ids):
        x = torch.stack([synth.hidden_states(wl, l, t, dev) for l in range(wl.L)])
        idx, gate = r.route_step(x, w, logits_out=logits, alpha_out=alpha)
        r.controller_update()
        r.poll()
        loads, bias, mxv, mnv = [np_(v) for v in r.load_stats()]
        gates_gpu = np_(r.gate_stats())
        lg, ix, gt, al = np_(logits), np_(idx), np_(gate), np_(alpha)
        for l in range(wl.L):
            oi = check_exact(lg[l], b[l], wl.K, ix[l], gt[l], al[l])
            np.testing.assert_array_equal(loads[l], np.bincount(oi.ravel(), minlength=wl.E))
            if check_rows is not None and n_step % 5 == 0:
                d, c = check_definition(synth.bf16_bits(x[l]), synth.bf16_bits(w[l]), b[l], wl.K, lg[l], ix[l], gt[l],
                                        rows=check_rows)
                differing += d
                checked += c
            Q = oracle.quantile_target(lg[l], al[l], wl.K) if kind == "quantile" else None
            b[l], ep[l], g, mx, mn = oracle_controller_step(
                kind, b[l], ep[l], loads[l], dict(ki=kw.get("ki", 6e-3), kd=kw.get("kd", 6e-3), eta=kw.get("eta", 1e-3), rho=kw.get("qb_ema_rho", 0.0)),
                center, Q)
            assert bits(mxv[l:l + 1])[0] == bits(np.array([mx]))[0]
            assert gates_gpu[l] == g                   # open derivative gates (Eq. 11) counted like the oracle
        np.testing.assert_array_equal(bits(bias), bits(b))
        hist.append((float(mxv.max()), float(mnv.max()), int(gates_gpu.sum())))
    if checked:
        assert differing <= max(1, NEAR_TIE_BUDGET * checked)
    return hist


def test_closed_loop_tiny_top3_id():
    # config "Tiny Top-3-of-768": 20 controller steps, fresh batch per step
    wl = synth.WORKLOADS["tiny_top3"]
    hist = _closed_loop(wl, "id", 20, check_rows=np.arange(0, wl.T, 4))
    assert max(h[2] for h in hist) > 0                 # the derivative gate opened on routed data at some step
    assert hist[-1][0] < hist[0][0]                    # the controller reduces the overload it started with


@pytest.mark.parametrize("kind,K", [("id", 3), ("fixed_step", 3), ("quantile", 3), ("quantile", 5), ("id", 5)])
def test_closed_loop_three_controllers_reduced(kind, K):
    # the Top-3 / Top-5 single-layer comparison at a reduced token count
    wl = synth.WORKLOADS["top3_single"].with_(T=2048, H=512, K=K)
    hist = _closed_loop(wl, kind, 6)
    assert all(0 <= mx <= wl.E / K - 1 + 1e-4 and 0 <= mn <= 1 for mx, mn, _ in hist)


@pytest.mark.parametrize("rho", [0.5, 0.9])
def test_closed_loop_quantile_with_ema(rho):
    # Quantile Balancing with the exponential moving average of Section 3: b = rho b + (1 - rho) Q, bit for bit
    wl = synth.WORKLOADS["top3_single"].with_(T=1024, H=256, K=3)
    hist = _closed_loop(wl, "quantile", 5, qb_ema_rho=rho)
    assert all(0 <= mx <= wl.E / wl.K - 1 + 1e-4 and 0 <= mn <= 1 for mx, mn, _ in hist)


def test_closed_loop_quantile_two_layers():
    # Eq. 7 per layer: every layer gets its own target from its own slice of the dump
    wl = synth.WORKLOADS["top3_single"].with_(T=1024, H=256, K=5, L=2)
    hist = _closed_loop(wl, "quantile", 4)
    assert all(0 <= mx <= wl.E / wl.K - 1 + 1e-4 and 0 <= mn <= 1 for mx, mn, _ in hist)


@pytest.mark.parametrize("K", [3, 5])
def test_quantile_controller_at_full_single_layer_size(K):
    # the Top-3 / Top-5 single-layer configuration at its own size (T = 16384, H = 2048): one Quantile Balancing
    # update, target and bias bit-exact against the oracle's sort-based quantile (Eq. 6-7)
    wl = synth.WORKLOADS["top3_single"].with_(K=K)
    hist = _closed_loop(wl, "quantile", 1)
    assert 0 <= hist[0][0] <= wl.E / K - 1 + 1e-4


def test_quantile_target_with_a_large_common_bias_offset():
    # Quantile Balancing is not centred, so its bias drifts as a whole; with every bias near -1.5 the margins lie
    # in [1, 2): sign, exponent and leading mantissa bits are common, and the keys that share the 16-bit prefix of
    # an expert's quantile are far more than the 1024 a list holds.  The selection then takes a third digit pass;
    # target and bias must still be those of the oracle's sort, bit for bit.
    wl = synth.WORKLOADS["top3_single"].with_(H=512)
    dev = "cuda"
    g = torch.Generator().manual_seed(3)
    b0 = (-1.5 + 0.002 * torch.randn(1, wl.E, generator=g)).float()
    r = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile")
    r.state_import(bias=b0.to(dev).contiguous())
    w = torch.stack([synth.router_weights(wl, 0, dev)])
    x = (torch.stack([synth.hidden_states(wl, 0, 0, dev)]).float() * 0.02).to(torch.bfloat16)   # scores close together
    logits = torch.empty(1, wl.T, wl.E, device=dev)
    alpha = torch.empty(1, wl.T, device=dev)
    idx, gate = r.route_step(x, w, logits_out=logits, alpha_out=alpha)
    r.controller_update()
    r.poll()
    loads, bias, _, _ = [np_(v) for v in r.load_stats()]
    lg, al = np_(logits)[0], np_(alpha)[0]
    oi = check_exact(lg, np_(b0)[0], wl.K, np_(idx)[0], np_(gate)[0], al)
    np.testing.assert_array_equal(loads[0], np.bincount(oi.ravel(), minlength=wl.E))
    Q = oracle.quantile_target(lg, al, wl.K)
    want, _, _, _, _ = oracle_controller_step("quantile", np_(b0)[0], np.zeros(wl.E, np.float32), loads[0], dict(rho=0.0), False, Q)
    np.testing.assert_array_equal(bits(bias[0]), bits(want))
    # the premise: for some expert more than 1024 margins share the 16-bit key prefix of its quantile
    d = (oracle.sigmoid_f32(lg[:, :8]) - al[:, None]).astype(np.float32)
    u = (d + np.float32(0.0)).view(np.uint32)
    keys = np.where(u & 0x80000000, ~u, u | 0x80000000).astype(np.uint32)
    rank = wl.T - (wl.T * wl.K) // wl.E
    most = 0
    for j in range(8):
        ans = np.sort(keys[:, j])[rank - 1]
        most = max(most, int(((keys[:, j] >> 16) == (ans >> 16)).sum()))
        assert np.float32(-(d[:, j][np.argsort(keys[:, j], kind="stable")[rank - 1]])) == Q[j]
    assert most > 1024, most


@pytest.mark.parametrize("bins,value_range,T,L", [(1024, 1.0, 3000, 1), (64, 0.5, 700, 2), (2048, 2.0, 16384, 1)])
def test_quantile_controller_with_margin_histogram_estimate(bins, value_range, T, L):
    # footnote to Eq. 7: the target estimated from a per-expert margin histogram (this library's bin rule).
    # Integer counts and a fixed binary64 interpolation: bit-exact against the oracle's estimate on the GPU's own
    # dump, and within one bin width of the exact target wherever that lies inside the range
    wl = synth.WORKLOADS["top3_single"].with_(T=T, H=256, L=L)
    dev = "cuda"
    r = binding.Router(L, wl.E, wl.K, wl.H, wl.T, controller="quantile", qb_hist_bins=bins, qb_hist_range=value_range)
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(L)])
    logits = torch.empty(L, wl.T, wl.E, device=dev)
    alpha = torch.empty(L, wl.T, device=dev)
    for step in range(2):                      # the second update starts from a histogram the first one cleared
        x = torch.stack([synth.hidden_states(wl, l, step, dev) for l in range(L)])
        r.route_step(x, w, logits_out=logits, alpha_out=alpha)
        r.controller_update()
        r.poll()
        bias = np_(r.load_stats()[1])
        for l in range(L):
            lg, al = np_(logits)[l], np_(alpha)[l]
            want = oracle.quantile_target_hist(lg, al, wl.K, bins, value_range)
            np.testing.assert_array_equal(bits(bias[l]), bits(want))
            exact = oracle.quantile_target(lg, al, wl.K)
            h = 2.0 * value_range / bins
            inside = np.abs(exact) < value_range - h
            assert inside.sum() > wl.E // 2
            assert np.max(np.abs(bias[l][inside].astype(np.float64) - exact[inside])) < h * (1 + 1e-6)


def test_margin_histogram_estimate_with_exponential_moving_average():
    # the EMA diagnostic of Section 3 on top of the histogram estimate: b = rho b + (1 - rho) Q_hist, three updates
    # in a closed loop, bit for bit against the oracle's estimate and update
    wl = synth.WORKLOADS["top3_single"].with_(T=1500, H=128, K=5)
    dev, bins, value_range, rho = "cuda", 256, 1.0, 0.5
    r = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile", qb_hist_bins=bins, qb_hist_range=value_range,
                       qb_ema_rho=rho)
    w = synth.router_weights(wl, 0, dev)[None].contiguous()
    logits = torch.empty(1, wl.T, wl.E, device=dev)
    alpha = torch.empty(1, wl.T, device=dev)
    b = np.zeros(wl.E, np.float32)
    ep = np.zeros(wl.E, np.float32)
    for step in range(3):
        x = synth.hidden_states(wl, 0, step, dev)[None].contiguous()
        idx, gate = r.route_step(x, w, logits_out=logits, alpha_out=alpha)
        r.controller_update()
        r.poll()
        loads, bias, _, _ = [np_(v) for v in r.load_stats()]
        check_exact(np_(logits)[0], b, wl.K, np_(idx)[0], np_(gate)[0], np_(alpha)[0])
        Q = oracle.quantile_target_hist(np_(logits)[0], np_(alpha)[0], wl.K, bins, value_range)
        b, ep = oracle.quantile_update(b, ep, oracle.load_error(loads[0].astype(np.int64)), Q, rho=rho)
        np.testing.assert_array_equal(bits(bias[0]), bits(b))


def test_closed_loop_drifting_deep_stack_opens_the_derivative_gate():
    # deep-stack configuration at a reduced token count: the cluster means drift linearly over the 500 steps of
    # the workload, so consecutive controller steps taken from steps spread over the drift see the imbalance of
    # some experts grow -- the derivative gate of Algorithm 1 line 9 opens on routed data, and the number of
    # open gates per layer equals the oracle's
    wl = synth.WORKLOADS["top10_deep"].with_(L=6, T=2048)
    ids = [0, 40, 90, 150, 220, 300, 380, 450, 499]
    hist = _closed_loop(wl, "id", len(ids), step_ids=ids)
    assert hist[0][2] == 0                       # first step: previous error is zero, every gate closed
    assert max(h[2] for h in hist[1:]) > 0       # later steps: gates open somewhere


@pytest.mark.parametrize("tie_rows,T", [(3000, 3000), (2600, 4000), (700, 4000)])
def test_quantile_target_with_long_runs_of_equal_margins(tie_rows, T):
    # tokens with all-zero hidden states have the same score 0.5 for every expert and the same cutoff, so their
    # margins are exactly equal: more equal margins than the gathered lists hold (1024) send those experts down
    # the path that walks the key scratch itself; fewer stay on the gather path.  Target bit-exact either way.
    wl = synth.WORKLOADS["top3_single"].with_(T=T, H=128)
    dev = "cuda"
    x = synth.hidden_states(wl, 0, 0, dev)[None].contiguous()
    x[0, :tie_rows] = 0
    w = synth.router_weights(wl, 0, dev)[None].contiguous()
    r = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile")
    logits = torch.empty(1, T, wl.E, device=dev)
    alpha = torch.empty(1, T, device=dev)
    r.route_step(x, w, logits_out=logits, alpha_out=alpha)
    r.controller_update()
    r.poll()
    bias = np_(r.load_stats()[1])[0]
    want = oracle.quantile_target(np_(logits)[0], np_(alpha)[0], wl.K)
    np.testing.assert_array_equal(bits(bias), bits(want))


def test_quantile_target_count_property_on_gpu_result():
    # Section 2.3: with the cutoffs held fixed the new bias puts floor(mK/E)
    # (or, with ties at the cutoff, at most that many) margins strictly above zero
    wl = synth.WORKLOADS["top3_single"].with_(T=4096, H=256)
    dev = "cuda"
    r = binding.Router(1, wl.E, wl.K, wl.H, wl.T, controller="quantile")
    x = synth.hidden_states(wl, 0, 0, dev)[None]
    w = synth.router_weights(wl, 0, dev)[None]
    logits = torch.empty(1, wl.T, wl.E, device=dev)
    alpha = torch.empty(1, wl.T, device=dev)
    r.route_step(x, w, logits_out=logits, alpha_out=alpha)
    r.controller_update()
    r.poll()
    bias = np_(r.load_stats()[1])[0]
    S = oracle.sigmoid_f32(np_(logits)[0])
    margin = S - np_(alpha)[0][:, None]
    q = (wl.T * wl.K) // wl.E
    above = (margin > -bias[None, :]).sum(0)
    at_or_above = (margin >= -bias[None, :]).sum(0)
    assert np.all(above <= q) and np.all(at_or_above >= q + 1)
    with pytest.raises(binding.MoeRouteError):          # needs a fresh dump per update
        r.controller_update()


@pytest.mark.parametrize("chunk_split", [1, 2])
def test_host_buffer_step_matches_device_step(chunk_split):
    T, H, E, K, L = 900, 256, 768, 10, 2
    res = route_once(T, H, E, K, L, seed=9, chunk_split=chunk_split)
    r = binding.Router(L, E, K, H, T, host_staging=True, chunk_split=chunk_split)
    xh, wh = res["x"].cpu().pin_memory(), res["w"].cpu().pin_memory()
    ih = torch.empty(L, T, K, dtype=torch.int32).pin_memory()
    gh = torch.empty(L, T, K, dtype=torch.float32).pin_memory()
    r.route_step_host(xh, wh, ih, gh)
    r.poll()
    np.testing.assert_array_equal(ih.numpy(), res["idx"])
    np.testing.assert_array_equal(bits(gh.numpy()), bits(res["gate"]))
    np.testing.assert_array_equal(np_(r.loads_peek()), res["loads"])


def test_argument_errors_are_reported_not_raised_by_cuda():
    r = binding.Router(1, 768, 10, 64, 128)
    x = torch.zeros(1, 256, 64, device="cuda", dtype=torch.bfloat16)
    w = torch.zeros(1, 768, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(binding.MoeRouteError) as ei:
        r.route_step(x, w)                               # more tokens than max_tokens
    assert ei.value.code == binding.MOE_ERR_INVALID_ARG
    rq = binding.Router(1, 768, 3, 64, 128, controller="quantile")
    with pytest.raises(binding.MoeRouteError):
        rq.route_step(x[:, :128].contiguous(), w)        # quantile controller without the dump buffers
    # misaligned output buffers are refused on the host (the dump is written with 16-byte stores)
    x1 = x[:, :128].contiguous()
    n0 = r.launch_count()
    buf = torch.empty(128 * 768 + 8, device="cuda")
    for off in (1, 2, 3):
        with pytest.raises(binding.MoeRouteError) as ei:
            r.route_step(x1, w, logits_out=buf[off:off + 128 * 768])
        assert ei.value.code == binding.MOE_ERR_INVALID_ARG
    raw = torch.empty(128 * 10 * 4 + 8, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.MoeRouteError) as ei:
        r.route_step(x1, w, topk_idx=raw[2:2 + 128 * 10 * 4])      # byte tensor: only its address is used
    assert ei.value.code == binding.MOE_ERR_INVALID_ARG
    assert r.launch_count() == n0                        # nothing was launched
    r.route_step(x1, w, logits_out=buf[4:4 + 128 * 768])  # 16-byte aligned offset is fine
    assert r.poll(raise_on_error=False) == binding.MOE_OK


def test_diagnostics_match_oracle():
    # the paper's load-control diagnostics after an ID update, and the gate entropy of a routing step
    wl = synth.WORKLOADS["tiny_top3"].with_(T=1536, L=2)
    dev = "cuda"
    r = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T)
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)])
    b_old = np.zeros((wl.L, wl.E), np.float32)
    ep = np.zeros((wl.L, wl.E), np.float32)
    for t in range(4):
        x = torch.stack([synth.hidden_states(wl, l, t, dev) for l in range(wl.L)])
        idx, gate = r.route_step(x, w)
        r.controller_update()
        r.poll()
        loads, bias, _, _ = [np_(v) for v in r.load_stats()]
        diag = np_(r.load_diagnostics())
        ent = np_(r.gate_entropy(gate))
        for l in range(wl.L):
            e = oracle.load_error(loads[l].astype(np.int64))
            b_new, ep[l], g = oracle.id_update(b_old[l], ep[l], e, 6e-3, 6e-3, center=True)
            np.testing.assert_array_equal(bits(b_new), bits(bias[l]))
            want = oracle.load_diagnostics(loads[l].astype(np.int64), g, b_old[l], b_new)
            np.testing.assert_array_equal(bits(diag[l, :3]), bits(want[:3]))      # integer ratios: exact
            np.testing.assert_allclose(diag[l, 3], want[3], rtol=1e-6)            # fp64 sum, other order
            np.testing.assert_allclose(ent[l], oracle.gate_entropy_mean(np_(gate)[l]), rtol=1e-6)
            assert 0 < ent[l] <= np.log(wl.K) + 1e-6
            b_old[l] = b_new
    assert diag[:, 1].min() > 0.1            # imbalanced synthetic loads: the busiest 10 % hold more than 10 %


@pytest.mark.parametrize("L,T,H,E,K", [(1, 1500, 256, 768, 10), (3, 700, 128, 256, 8), (2, 333, 128, 1024, 5), (1, 40, 64, 72, 3)])
def test_score_stats_match_oracle(L, T, H, E, K):
    # full-pool entropies (Section 4.3) and the forward statistics of the auxiliary loss (Eq. 8) against the
    # binary64 definition on the GPU's own logit dump; fp32 per-token arithmetic -> relative tolerance 1e-5
    g = torch.Generator().manual_seed(5)
    bias = (torch.randn(L, E, generator=g) * 0.2)          # large enough that some biased scores clamp at zero
    res = route_once(T, H, E, K, L=L, bias=bias, seed=17)
    r = res["r"]
    loads = r.loads_peek()
    st = r.score_stats(torch.from_numpy(res["logits"]).cuda(), loads)
    r.poll()
    for l in range(L):
        z = res["logits"][l]
        hb = oracle.full_pool_entropy_mean(z, res["bias"][l], "biased_sigmoid")
        hs = oracle.full_pool_entropy_mean(z, None, "softmax")
        f, P, aux = oracle.aux_loss_stats(z, res["loads"][l].astype(np.int64))
        assert abs(float(st["entropy_biased"][l]) - hb) <= 1e-5 * hb
        assert abs(float(st["entropy_softmax"][l]) - hs) <= 1e-5 * hs
        np.testing.assert_allclose(np_(st["mean_prob"][l]), P, rtol=1e-5, atol=1e-9)
        assert abs(float(st["aux"][l]) - aux) <= 1e-5 * aux
    assert ((1.0 / (1.0 + np.exp(-res["logits"].astype(np.float64))) + res["bias"][:, None, :]) < 0).any()   # clamp exercised
    # deterministic: same call, same bits; outputs are optional
    st2 = r.score_stats(torch.from_numpy(res["logits"]).cuda(), loads)
    for k in st:
        np.testing.assert_array_equal(bits(np_(st[k])), bits(np_(st2[k])))
    only = r.score_stats(torch.from_numpy(res["logits"]).cuda())
    assert "aux" not in only
    np.testing.assert_array_equal(bits(np_(only["mean_prob"])), bits(np_(st["mean_prob"])))


def test_score_stats_wide_logit_range():
    # rows whose largest logit lies beyond +-40 take the kernel's direct sigmoid form, the others the shared-
    # exponential form; both against the binary64 definition on a synthetic dump with row offsets up to +-70
    L, T, E, K = 2, 900, 768, 10
    rng = np.random.default_rng(23)
    z = (rng.standard_normal((L, T, E)) * 3.0 + rng.uniform(-70.0, 70.0, size=(L, T, 1))).astype(np.float32)
    assert (np.abs(z.max(axis=2)) > 40).mean() > 0.2 and (np.abs(z.max(axis=2)) <= 40).mean() > 0.2
    bias = (rng.standard_normal((L, E)) * 0.2).astype(np.float32)
    r = binding.Router(L, E, K, 64, T)
    r.state_import(torch.from_numpy(bias).cuda(), torch.zeros(L, E, device="cuda"))
    st = r.score_stats(torch.from_numpy(z).cuda())
    r.poll()
    for l in range(L):
        hb = oracle.full_pool_entropy_mean(z[l], bias[l], "biased_sigmoid")
        hs = oracle.full_pool_entropy_mean(z[l], None, "softmax")
        _, P, _ = oracle.aux_loss_stats(z[l], np.zeros(E, dtype=np.int64))
        assert abs(float(st["entropy_biased"][l]) - hb) <= 1e-5 * hb
        assert abs(float(st["entropy_softmax"][l]) - hs) <= 1e-5 * hs
        np.testing.assert_allclose(np_(st["mean_prob"][l]), P, rtol=1e-5, atol=1e-9)
    raw = torch.zeros(L * T * E + 4, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.MoeRouteError):                   # rows are read as 16-byte words
        r.score_stats(raw[1:1 + L * T * E].view(L, T, E))


def _fuzz_case(seed):
    rng = np.random.default_rng(seed)
    E = int(rng.choice([8, 16, 40, 64, 128, 256, 264, 512, 768, 776, 1000, 1024]))
    K = int(rng.integers(1, min(16, E - 1) + 1))
    H = int(rng.choice([8, 16, 64, 72, 128, 200, 256, 320, 512]))
    T = int(rng.integers(1, 700))
    L = int(rng.integers(1, 4))
    bias_scale = float(rng.choice([0.0, 1e-3, 1e-2, 0.3, 2.0]))
    logit_scale = float(rng.choice([0.05, 1.0, 4.0]))
    quantise = bool(rng.integers(0, 3) == 0)          # coarse inputs: many exactly equal scores
    return T, H, E, K, L, bias_scale, logit_scale, quantise


@pytest.mark.parametrize("seed", range(24))
def test_route_random_shapes_bit_exact(seed):
    # seeded random shapes, bias magnitudes, logit spreads and tie densities: the binary32 chain must match the
    # oracle bit for bit on the GPU's own logits (indices, gates, alpha), and the loads must be the recount
    T, H, E, K, L, bias_scale, logit_scale, quantise = _fuzz_case(1000 + seed)
    g = torch.Generator().manual_seed(seed)
    bias = torch.randn(L, E, generator=g) * bias_scale
    x = torch.randn(L, T, H, generator=g)
    w = torch.randn(L, E, H, generator=g) * (logit_scale / max(H, 1) ** 0.5)
    if quantise:
        x, w, bias = torch.round(x), torch.round(w * 4) / 4, torch.round(bias * 8) / 8
    res = route_once(T, H, E, K, L=L, bias=bias, want_alpha=(K < 16), x=x.cuda().to(torch.bfloat16),
                     w=w.cuda().to(torch.bfloat16), chunk_split=1 + seed % 2)
    for l in range(L):
        a = None if res["alpha"] is None else res["alpha"][l]
        oi = check_exact(res["logits"][l], res["bias"][l], K, res["idx"][l], res["gate"][l], a)
        np.testing.assert_array_equal(res["loads"][l], np.bincount(oi.ravel(), minlength=E))


@pytest.mark.parametrize("T,H,E,K,L", [(300, 192, 768, 10, 2), (130, 72, 40, 3, 1), (257, 320, 256, 8, 3)])
def test_expert_contiguous_weight_layout(T, H, E, K, L):
    # weights handed over as [L][H][E]: same results, bit for bit, as with the paper's [L][E][H], and parity with the oracle
    res = route_once(T, H, E, K, L=L, seed=5)
    full_check(res, K, rows=np.arange(0, T, 7))
    wt = res["w"].transpose(1, 2).contiguous()                  # [L][H][E]
    r = binding.Router(L, E, K, H, T, w_layout=1)
    logits = torch.empty(L, T, E, device="cuda")
    idx, gate = r.route_step(res["x"], wt, logits_out=logits)
    r.poll()
    np.testing.assert_array_equal(np_(idx), res["idx"])
    np.testing.assert_array_equal(bits(np_(gate)), bits(res["gate"]))
    np.testing.assert_array_equal(bits(np_(logits)), bits(res["logits"]))
    np.testing.assert_array_equal(np_(r.loads_peek()), res["loads"])
    # host-buffer step with the same layout
    rh = binding.Router(L, E, K, H, T, w_layout=1, host_staging=True)
    ih = torch.empty(L, T, K, dtype=torch.int32).pin_memory()
    gh = torch.empty(L, T, K, dtype=torch.float32).pin_memory()
    rh.route_step_host(res["x"].cpu().pin_memory(), wt.cpu().pin_memory(), ih, gh)
    rh.poll()
    np.testing.assert_array_equal(ih.numpy(), res["idx"])


@pytest.mark.parametrize("chunk_split", [1, 2])
def test_step_replays_from_a_cuda_graph(chunk_split):
    # routing (+ the merge kernel under chunk-split scheduling) + controller update captured once into a CUDA graph
    # (all launches use programmatic stream serialisation) and replayed: state and outputs evolve exactly as with
    # eager launches
    T, H, E, K, L = 640, 256, 768, 10, 2
    g = torch.Generator(device="cuda").manual_seed(77)
    x = torch.randn(L, T, H, device="cuda", generator=g).to(torch.bfloat16)
    w = (torch.randn(L, E, H, device="cuda", generator=g) / 16).to(torch.bfloat16)
    eager = binding.Router(L, E, K, H, T, chunk_split=chunk_split)
    graphed = binding.Router(L, E, K, H, T, chunk_split=chunk_split)
    idx_e = torch.empty(L, T, K, dtype=torch.int32, device="cuda")
    gate_e = torch.empty(L, T, K, device="cuda")
    idx_g, gate_g = torch.empty_like(idx_e), torch.empty_like(gate_e)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        graphed.route_step(x, w, idx_g, gate_g)
        graphed.controller_update()
    for step in range(4):
        graph.replay()
        eager.route_step(x, w, idx_e, gate_e)
        eager.controller_update()
        torch.cuda.synchronize()
        np.testing.assert_array_equal(np_(idx_g), np_(idx_e))
        np.testing.assert_array_equal(bits(np_(gate_g)), bits(np_(gate_e)))
        for a, b in zip(graphed.load_stats(), eager.load_stats()):
            np.testing.assert_array_equal(bits(np_(a).astype(np.float32)) if a.dtype.is_floating_point else np_(a),
                                          bits(np_(b).astype(np.float32)) if b.dtype.is_floating_point else np_(b))
    graphed.poll()
    eager.poll()
    assert float(eager.load_stats()[1].abs().max()) > 0          # the bias moved: the replays really updated state


def test_bounded_wait_gives_up_and_reports_timeout():
    # a wait that nothing satisfies runs out after its iteration bound: the kernel returns, the status
    # word says MOE_ERR_TIMEOUT, and the same context keeps working afterwards
    T, H, E, K = 256, 128, 768, 10
    res = route_once(T, H, E, K, seed=3)
    r = res["r"]
    r.debug_wait_timeout(spin_limit=2000)
    assert r.poll(raise_on_error=False) == binding.MOE_ERR_TIMEOUT
    assert r.poll(raise_on_error=False) == binding.MOE_OK          # sticky status cleared by the poll
    assert not np_(r.loads_peek()).any()                           # a timed-out iteration is void: counts dropped
    idx, gate = r.route_step(res["x"], res["w"])
    r.poll()
    np.testing.assert_array_equal(np_(idx), res["idx"])
    np.testing.assert_array_equal(np_(r.loads_peek()), res["loads"])


@pytest.mark.parametrize("chunk_split,after", [(1, 2), (2, 3)])
def test_routing_kernel_gives_up_cleanly_when_its_waits_run_out(chunk_split, after):
    # the producers of ONE routing launch stop issuing loads after a few pipeline stages (nothing is left in
    # flight, no fault, no endless loop): the MMA warp's bounded wait for the next stage runs out, every role of
    # every CTA leaves its loop, tensor memory is released and the kernel returns; the host sees
    # MOE_ERR_TIMEOUT, the void step's counts are dropped, the controller state is untouched, and the same
    # context routes the same batch correctly afterwards
    T, H, E, K, L = 700, 256, 768, 10, 2
    good = route_once(T, H, E, K, L=L, seed=11, chunk_split=chunk_split)
    r = binding.Router(L, E, K, H, T, spin_limit=4000, chunk_split=chunk_split)
    r.debug_route_stall(after_loads=after)
    r.route_step(good["x"], good["w"])
    assert r.poll(raise_on_error=False) == binding.MOE_ERR_TIMEOUT
    assert "wait" in r.lib.moe_last_error(r.h).decode()
    assert not np_(r.loads_peek()).any()                         # partial histogram dropped
    assert r.poll(raise_on_error=False) == binding.MOE_OK        # sticky status cleared
    bias, e_prev = [np_(v) for v in r.state_export()]
    assert not bias.any() and not e_prev.any()                   # controller state untouched
    idx, gate = r.route_step(good["x"], good["w"])               # the stall applied to one launch only
    r.poll()
    np.testing.assert_array_equal(np_(idx), good["idx"])
    np.testing.assert_array_equal(bits(np_(gate)), bits(good["gate"]))
    np.testing.assert_array_equal(np_(r.loads_peek()), good["loads"])


@pytest.mark.parametrize("name,L,T", [("top10_deep", 48, 700), ("top10_large", 60, 700)])
def test_all_layers_of_the_deep_configurations_in_one_launch(name, L, T):
    # every layer of the 48- and 60-layer configurations in ONE routing call, at their own hidden size and a
    # reduced, ragged token count (three tile pairs per layer: 144 / 180 work items walked by the persistent
    # grid across layer changes): all tokens of all layers against the binary32 chain, per-layer loads, and a
    # row sample against the fp64 definition
    wl = synth.WORKLOADS[name].with_(T=T)
    assert wl.L == L
    dev = "cuda"
    g = torch.Generator().manual_seed(L)
    bias = torch.randn(L, wl.E, generator=g) * 0.01
    x = torch.stack([synth.hidden_states(wl, l, 1, dev) for l in range(L)])
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(L)])
    res = route_once(T, wl.H, wl.E, wl.K, L=L, bias=bias, want_alpha=True, x=x, w=w)
    full_check(res, wl.K, rows=np.arange(3, T, 16))
    # the same call without the dump (the timed configuration) gives the same selections
    r = binding.Router(L, wl.E, wl.K, wl.H, T)
    r.state_import(bias=bias.cuda().contiguous())
    idx, gate = r.route_step(x, w)
    r.poll()
    np.testing.assert_array_equal(np_(idx), res["idx"])
    np.testing.assert_array_equal(bits(np_(gate)), bits(res["gate"]))
    np.testing.assert_array_equal(np_(r.loads_peek()), res["loads"])


# ------------------------------------------------ full-size configurations
def _full_size(wl, layers, steps=1, sample=192):
    """Full T and H of a configuration (a few layers of it), in the launch
    configuration the benchmark times.  All tokens against the binary32
    chain; a seeded token sample against the fp64 definition."""
    dev = "cuda"
    wl = wl.with_(L=layers)
    r = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T)
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)])
    b = np.zeros((wl.L, wl.E), np.float32)
    rng = np.random.default_rng(wl.wid)
    differing = checked = 0
    for t in range(steps):
        x = torch.stack([synth.hidden_states(wl, l, t, dev) for l in range(wl.L)])
        idx, gate = r.route_step(x, w)                  # the timed configuration: no dump
        r.poll()
        loads = np_(r.loads_peek())
        ix, gt = np_(idx), np_(gate)
        assert loads.sum() == wl.L * wl.T * wl.K
        for l in range(wl.L):
            np.testing.assert_array_equal(loads[l], np.bincount(ix[l].ravel(), minlength=wl.E))
        # same inputs once more with the dump, one layer at a time, for the element-wise checks
        r2 = binding.Router(1, wl.E, wl.K, wl.H, wl.T)
        for l in range(wl.L):
            r2.state_import(bias=torch.from_numpy(b[l:l + 1]).cuda())
            logits = torch.empty(1, wl.T, wl.E, device=dev)
            i2, g2 = r2.route_step(x[l:l + 1].contiguous(), w[l:l + 1].contiguous(), logits_out=logits)
            r2.poll()
            np.testing.assert_array_equal(np_(i2)[0], ix[l])        # dump on/off changes nothing
            np.testing.assert_array_equal(bits(np_(g2)[0]), bits(gt[l]))
            lg = np_(logits)[0]
            check_exact(lg, b[l], wl.K, ix[l], gt[l])
            rows = np.sort(rng.choice(wl.T, sample, replace=False))
            d, c = check_definition(synth.bf16_bits(x[l]), synth.bf16_bits(w[l]), b[l], wl.K, lg, ix[l], gt[l], rows)
            differing += d
            checked += c
        r.controller_update()
        r.poll()
        b = np_(r.load_stats()[1])
    assert differing <= max(1, NEAR_TIE_BUDGET * checked)


def test_full_size_top10_single_layer():
    _full_size(synth.WORKLOADS["top10_single"], layers=1, steps=2)


def test_full_size_top3_and_top5_single_layer():
    _full_size(synth.WORKLOADS["top3_single"], layers=1)
    _full_size(synth.WORKLOADS["top5_single"], layers=1)


def test_full_size_deep_stack_layers():
    _full_size(synth.WORKLOADS["top10_deep"], layers=3, steps=2, sample=96)


def test_full_size_large_scale_layers():
    _full_size(synth.WORKLOADS["top10_large"], layers=2, sample=256)


@pytest.mark.parametrize("name", ["top10_deep", "top10_large"])
def test_bench_launch_configuration_at_full_size(name):
    # the whole configuration -- every layer at its full token count -- in ONE routing call without the dump, as
    # the benchmark launches it (top10_large: 60 layers x 65536 tokens x hidden 4096 under chunk-split scheduling,
    # 32 GB of hidden states): every token contributes exactly K counts, per-layer loads are the recount of the
    # indices, indices are valid and distinct per token, gates sum to one, and a seeded row sample of every layer
    # agrees with the fp64 definition (sets wherever the rank-K gap is clear, gates within 1e-5)
    wl = synth.WORKLOADS[name]
    dev = "cuda"
    g = torch.Generator().manual_seed(wl.wid)
    bias = (torch.randn(wl.L, wl.E, generator=g) * 0.01).contiguous()
    x = torch.empty(wl.L, wl.T, wl.H, dtype=torch.bfloat16, device=dev)
    for l in range(wl.L):
        x[l] = synth.hidden_states(wl, l, 2, dev)
    w = torch.stack([synth.router_weights(wl, l, dev) for l in range(wl.L)])
    r = binding.Router(wl.L, wl.E, wl.K, wl.H, wl.T)
    r.state_import(bias=bias.cuda())
    idx, gate = r.route_step(x, w)
    r.poll()
    loads = np_(r.loads_peek())
    assert loads.sum() == wl.L * wl.T * wl.K
    ix, gt = np_(idx), np_(gate)
    assert ix.min() >= 0 and ix.max() < wl.E
    rng = np.random.default_rng(wl.wid)
    differing = checked = 0
    for l in range(wl.L):
        np.testing.assert_array_equal(loads[l], np.bincount(ix[l].ravel(), minlength=wl.E))
        srt = np.sort(ix[l], axis=1)
        assert np.all(srt[:, 1:] != srt[:, :-1])                       # K distinct experts per token
        np.testing.assert_allclose(gt[l].sum(axis=1), 1.0, atol=2e-6)
        rows = np.sort(rng.choice(wl.T, 48, replace=False))
        ref = oracle.route_tokens_f64(synth.bf16_bits(x[l][torch.from_numpy(rows).cuda()]), synth.bf16_bits(w[l]),
                                      np_(bias[l]), wl.K, threads=THREADS)
        same_set = np.all(np.sort(ix[l][rows], 1) == np.sort(ref["idx"], 1), axis=1)
        assert np.all(same_set[ref["gap"] >= 1e-4])
        same_order = np.all(ix[l][rows] == ref["idx"], axis=1)
        assert np.max(np.abs(gt[l][rows][same_order] - ref["gate"][same_order])) <= 1e-5
        differing += int((~same_set).sum())
        checked += len(rows)
    assert differing <= max(1, NEAR_TIE_BUDGET * checked)

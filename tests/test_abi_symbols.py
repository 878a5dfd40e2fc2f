"""Host-only checks of the C-ABI library: it loads, exports every symbol the
header declares, and validates configurations without touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2609_39137_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "moe_route.h")).read()
    declared = set(re.findall(r"\b(moe_[a-z_]+)\s*\(", header))
    assert declared == set(binding.SYMBOLS), declared ^ set(binding.SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_config_struct_matches_header(lib):
    cfg = binding.default_config(2, 768, 10, 2048, 16384)
    assert cfg.struct_size == C.sizeof(binding.MoeRouteConfig) == 18 * 4
    # paper defaults: Ki = Kd = 6e-3 (Section 4), eta = 1e-3 (Section 4.1), no EMA
    assert abs(cfg.ki - 6e-3) < 1e-9 and abs(cfg.kd - 6e-3) < 1e-9 and abs(cfg.eta - 1e-3) < 1e-9
    assert cfg.qb_ema_rho == 0 and cfg.center == -1 and cfg.controller == binding.MOE_CTRL_ID


def test_workspace_bytes_and_config_validation(lib):
    cfg = binding.default_config(48, 768, 10, 2048, 16384)
    n = lib.moe_route_workspace_bytes(C.byref(cfg))
    assert n >= 4 * 48 * 768 * 4 and n % 256 == 0
    cfg.host_staging = 1
    assert lib.moe_route_workspace_bytes(C.byref(cfg)) > n + 48 * 16384 * 2048 * 2
    bad = [dict(num_experts=770), dict(num_experts=2048), dict(top_k=0), dict(top_k=17), dict(hidden=100),
           dict(num_layers=0), dict(max_tokens=0), dict(controller=7), dict(qb_ema_rho=1.0), dict(ki=-1.0),
           dict(struct_size=8), dict(w_layout=2), dict(chunk_split=3), dict(qb_hist_bins=48),
           dict(qb_hist_bins=4096), dict(qb_hist_bins=64, qb_hist_range=0.0)]
    for kw in bad:
        c = binding.default_config(48, 768, 10, 2048, 16384)
        for k, v in kw.items():
            setattr(c, k, v)
        assert lib.moe_route_workspace_bytes(C.byref(c)) == 0, kw
    # the quantile controller adds its radix-select scratch (histogram + one key per margin of a layer)
    cq = binding.default_config(48, 768, 10, 2048, 16384)
    cq.controller = binding.MOE_CTRL_QUANTILE
    assert lib.moe_route_workspace_bytes(C.byref(cq)) >= n + 16384 * 768 * 4 + 768 * 256 * 4
    # chunk-split scheduling reserves the per-chunk candidate lists; left to the library it is chosen for long
    # hidden sizes and for launches with at most 64 (tile pair, chunk) items, and not otherwise
    def ws(L, T, H, split):
        c = binding.default_config(L, 768, 10, H, T)
        c.chunk_split = split
        return lib.moe_route_workspace_bytes(C.byref(c))
    lists = lambda L, T: L * 3 * T * 11 * 8
    assert ws(1, 1024, 256, 2) >= ws(1, 1024, 256, 1) + lists(1, 1024)
    assert ws(1, 1024, 256, 0) == ws(1, 1024, 256, 2)            # 4 tile pairs x 3 chunks
    assert ws(1, 16384, 2048, 0) == ws(1, 16384, 2048, 1)        # 64 tile pairs x 3 chunks, hidden 2048
    assert ws(2, 4096, 4096, 0) == ws(2, 4096, 4096, 2)          # hidden 4096
    h = C.c_void_p()
    c = binding.default_config(1, 768, 10, 2048, 128)
    assert lib.moe_route_init(C.byref(c), None, 0, C.byref(h)) == binding.MOE_ERR_WORKSPACE
    c.top_k = 0
    assert lib.moe_route_init(C.byref(c), None, 0, C.byref(h)) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_route_poll(None) == binding.MOE_ERR_INVALID_ARG
    assert lib.moe_controller_update(None, None) == binding.MOE_ERR_INVALID_ARG

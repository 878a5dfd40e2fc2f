"""ctypes binding of include/moe_route.h (same names, argument marshalling only).

PyTorch appears only as the owner of device memory and streams: tensors are
passed as raw device pointers.  There is no CPU fallback: if the CUDA library
is missing, loading fails with an error.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MOE_ROUTE_LIB selects another build of the same library (the -DMOE_DEBUG one, libmoe_route_b200_debug.so)
LIB_PATH = os.environ.get("MOE_ROUTE_LIB") or os.path.join(_HERE, "libmoe_route_b200.so")

(MOE_OK, MOE_ERR_INVALID_ARG, MOE_ERR_UNSUPPORTED, MOE_ERR_CUDA, MOE_ERR_STATE, MOE_ERR_WORKSPACE, MOE_ERR_TIMEOUT,
 MOE_ERR_INTERNAL) = range(8)
MOE_CTRL_ID, MOE_CTRL_FIXED_STEP, MOE_CTRL_QUANTILE, MOE_CTRL_FROZEN = range(4)
CONTROLLERS = {"id": MOE_CTRL_ID, "fixed_step": MOE_CTRL_FIXED_STEP, "quantile": MOE_CTRL_QUANTILE,
               "frozen": MOE_CTRL_FROZEN}

# every symbol include/moe_route.h declares
SYMBOLS = ["moe_route_default_config", "moe_route_workspace_bytes", "moe_route_init", "moe_route_step",
           "moe_route_step_host", "moe_controller_update", "moe_load_stats", "moe_gate_stats", "moe_loads_peek",
           "moe_loads_add", "moe_loads_buffer", "moe_state_export", "moe_state_import", "moe_route_poll", "moe_route_launch_count",
           "moe_last_error", "moe_route_destroy", "moe_debug_score_gap", "moe_debug_quick_score_gap", "moe_debug_rcp_check", "moe_debug_division_check", "moe_quantile_target_static",
           "moe_load_diagnostics", "moe_gate_entropy", "moe_debug_wait_timeout", "moe_score_stats", "moe_debug_route_stall", "moe_debug_build"]


class MoeRouteConfig(C.Structure):
    _fields_ = [("struct_size", C.c_int32), ("num_layers", C.c_int32), ("num_experts", C.c_int32),
                ("top_k", C.c_int32), ("hidden", C.c_int32), ("max_tokens", C.c_int32), ("controller", C.c_int32),
                ("ki", C.c_float), ("kd", C.c_float), ("eta", C.c_float), ("qb_ema_rho", C.c_float),
                ("center", C.c_int32), ("spin_limit", C.c_int32), ("host_staging", C.c_int32),
                ("w_layout", C.c_int32), ("chunk_split", C.c_int32),
                ("qb_hist_bins", C.c_int32), ("qb_hist_range", C.c_float)]


class MoeRouteError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"moe_route error {code}: {msg}")
        self.code = code


_lib = None


def load():
    """Loads libmoe_route_b200.so (built in-tree by `build.py`); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not found: build it with `python -m paper_2609_39137_b200.build` "
                                "(there is no fallback path)")
    L = C.CDLL(LIB_PATH)
    vp, i32, cfgp = C.c_void_p, C.c_int32, C.POINTER(MoeRouteConfig)
    L.moe_route_default_config.argtypes = [cfgp, i32, i32, i32, i32, i32]
    L.moe_route_default_config.restype = None
    L.moe_route_workspace_bytes.argtypes = [cfgp]
    L.moe_route_workspace_bytes.restype = C.c_size_t
    L.moe_route_init.argtypes = [cfgp, vp, C.c_size_t, C.POINTER(vp)]
    L.moe_route_step.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp]
    L.moe_route_step_host.argtypes = [vp, vp, vp, i32, vp, vp, vp]
    L.moe_controller_update.argtypes = [vp, vp]
    L.moe_load_stats.argtypes = [vp, vp, vp, vp, vp, vp]
    L.moe_gate_stats.argtypes = [vp, vp, vp]
    L.moe_load_diagnostics.argtypes = [vp, vp, vp]
    L.moe_gate_entropy.argtypes = [vp, vp, i32, vp, vp]
    L.moe_loads_peek.argtypes = [vp, vp, vp]
    L.moe_loads_add.argtypes = [vp, vp, vp]
    L.moe_loads_buffer.argtypes = [vp, C.POINTER(vp)]
    L.moe_state_export.argtypes = [vp, vp, vp, C.POINTER(C.c_int64), vp]
    L.moe_state_import.argtypes = [vp, vp, vp, C.c_int64, vp]
    L.moe_route_poll.argtypes = [vp]
    L.moe_route_launch_count.argtypes = [vp]
    L.moe_route_launch_count.restype = C.c_int64
    L.moe_last_error.argtypes = [vp]
    L.moe_last_error.restype = C.c_char_p
    L.moe_route_destroy.argtypes = [vp]
    L.moe_debug_score_gap.argtypes = [vp, vp]
    L.moe_debug_quick_score_gap.argtypes = [vp, vp]
    L.moe_debug_rcp_check.argtypes = [vp, vp]
    L.moe_debug_division_check.argtypes = [vp, vp]
    L.moe_debug_wait_timeout.argtypes = [vp, i32, vp]
    L.moe_debug_route_stall.argtypes = [vp, i32]
    L.moe_debug_build.argtypes = []
    L.moe_score_stats.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.moe_quantile_target_static.argtypes = [vp, vp, i32, i32, i32, vp, vp]
    _lib = L
    return L


def default_config(num_layers, num_experts, top_k, hidden, max_tokens) -> MoeRouteConfig:
    cfg = MoeRouteConfig()
    load().moe_route_default_config(C.byref(cfg), num_layers, num_experts, top_k, hidden, max_tokens)
    return cfg


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def debug_score_gap(device="cuda") -> float:
    """Largest |approximate score - exact score| over all finite fp32 logits (runs on the GPU)."""
    out = torch.zeros(1, dtype=torch.float32, device=device)
    rc = load().moe_debug_score_gap(_ptr(out), _stream())
    if rc != MOE_OK:
        raise MoeRouteError(rc, "moe_debug_score_gap failed")
    return float(out.item())


def debug_rcp_check(device="cuda"):
    """(scores, reciprocals) that differ between the kernels' branch-free reciprocal and the library's correctly
    rounded one, over all 2^32 fp32 bit patterns (runs on the GPU); both must be 0."""
    out = torch.zeros(2, dtype=torch.int32, device=device)
    rc = load().moe_debug_rcp_check(_ptr(out), _stream())
    if rc != MOE_OK:
        raise MoeRouteError(rc, "moe_debug_rcp_check failed")
    a, b = out.tolist()
    return a, b


def debug_division_check(device="cuda") -> int:
    """Pairs (numerator, denominator) for which the kernels' gate division differs from the library's correctly
    rounded division, over every fp32 denominator in [2^-20, 32] with 48 numerators each; must be 0."""
    out = torch.zeros(1, dtype=torch.int32, device=device)
    rc = load().moe_debug_division_check(_ptr(out), _stream())
    if rc != MOE_OK:
        raise MoeRouteError(rc, "moe_debug_division_check failed")
    return int(out.item())


def debug_quick_score_gap(device="cuda") -> float:
    """Largest |quick score - exact score| over all finite fp32 logits (the margin-histogram pass's first guess)."""
    out = torch.zeros(1, dtype=torch.float32, device=device)
    rc = load().moe_debug_quick_score_gap(_ptr(out), _stream())
    if rc != MOE_OK:
        raise MoeRouteError(rc, "moe_debug_quick_score_gap failed")
    return float(out.item())


def quantile_target_static(logits, alpha, top_k, target_out):
    """moe_quantile_target_static: Q_j for one layer from a logits dump, using only the scratch array built
    into the library (no allocation happens in the call; `target_out` is the caller's [E] float32 tensor).
    Calls that may overlap on the GPU must not be issued concurrently: they share the one scratch array."""
    m, E = logits.shape
    assert logits.dtype == torch.float32 and alpha.dtype == torch.float32 and target_out.dtype == torch.float32
    assert logits.is_contiguous() and alpha.numel() == m and target_out.numel() == E
    rc = load().moe_quantile_target_static(_ptr(logits), _ptr(alpha), m, E, top_k, _ptr(target_out), _stream())
    if rc != MOE_OK:
        raise MoeRouteError(rc, "moe_quantile_target_static failed"
                            + (": more experts than the built-in scratch holds (1024)" if rc == MOE_ERR_WORKSPACE else ""))
    return target_out


class Router:
    """One routing + load-control context (L layers).  Methods mirror the C entry points."""

    def __init__(self, num_layers, num_experts, top_k, hidden, max_tokens, controller="id", ki=None, kd=None,
                 eta=None, qb_ema_rho=None, center=None, spin_limit=0, host_staging=False, w_layout=0,
                 chunk_split=0, qb_hist_bins=0, qb_hist_range=None, device="cuda"):
        self.lib = load()
        cfg = default_config(num_layers, num_experts, top_k, hidden, max_tokens)
        cfg.controller = CONTROLLERS[controller] if isinstance(controller, str) else int(controller)
        if ki is not None: cfg.ki = ki
        if kd is not None: cfg.kd = kd
        if eta is not None: cfg.eta = eta
        if qb_ema_rho is not None: cfg.qb_ema_rho = qb_ema_rho
        if center is not None: cfg.center = int(center)
        cfg.spin_limit = spin_limit
        cfg.host_staging = int(bool(host_staging))
        cfg.w_layout = int(w_layout)
        cfg.chunk_split = int(chunk_split)
        cfg.qb_hist_bins = int(qb_hist_bins)
        if qb_hist_range is not None: cfg.qb_hist_range = float(qb_hist_range)
        self.cfg = cfg
        self.L, self.E, self.K, self.H, self.max_tokens = num_layers, num_experts, top_k, hidden, max_tokens
        self.device = torch.device(device)
        nbytes = self.lib.moe_route_workspace_bytes(C.byref(cfg))
        if nbytes == 0:
            raise MoeRouteError(MOE_ERR_INVALID_ARG, "invalid configuration")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = self.lib.moe_route_init(C.byref(cfg), _ptr(self.workspace), nbytes, C.byref(h))
        if rc != MOE_OK:
            raise MoeRouteError(rc, "moe_route_init failed")
        self.h = h

    def _check(self, rc):
        if rc != MOE_OK:
            raise MoeRouteError(rc, self.lib.moe_last_error(self.h).decode())

    # -- moe_route_step
    def route_step(self, x, w, topk_idx=None, topk_gate=None, logits_out=None, alpha_out=None):
        """x [L][T][H] bf16, w [L][E][H] bf16 (device). Returns (topk_idx, topk_gate)."""
        T = x.shape[-2]
        assert x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16 and x.is_contiguous() and w.is_contiguous()
        assert x.numel() == self.L * T * self.H and w.numel() == self.L * self.E * self.H
        if topk_idx is None:
            topk_idx = torch.empty(self.L, T, self.K, dtype=torch.int32, device=x.device)
        if topk_gate is None:
            topk_gate = torch.empty(self.L, T, self.K, dtype=torch.float32, device=x.device)
        self._check(self.lib.moe_route_step(self.h, _ptr(x), _ptr(w), T, _ptr(topk_idx), _ptr(topk_gate),
                                            _ptr(logits_out), _ptr(alpha_out), _stream()))
        return topk_idx, topk_gate

    # -- moe_route_step_host
    def route_step_host(self, x_host, w_host, topk_idx_host, topk_gate_host):
        T = x_host.shape[-2]
        self._check(self.lib.moe_route_step_host(self.h, _ptr(x_host), _ptr(w_host), T, _ptr(topk_idx_host),
                                                 _ptr(topk_gate_host), _stream()))

    # -- moe_controller_update
    def controller_update(self):
        self._check(self.lib.moe_controller_update(self.h, _stream()))

    # -- moe_load_stats
    def load_stats(self):
        dev = self.device
        loads = torch.empty(self.L, self.E, dtype=torch.int32, device=dev)
        bias = torch.empty(self.L, self.E, dtype=torch.float32, device=dev)
        maxvio = torch.empty(self.L, dtype=torch.float32, device=dev)
        minvio = torch.empty(self.L, dtype=torch.float32, device=dev)
        self._check(self.lib.moe_load_stats(self.h, _ptr(loads), _ptr(bias), _ptr(maxvio), _ptr(minvio), _stream()))
        return loads, bias, maxvio, minvio

    def gate_stats(self):
        g = torch.empty(self.L, dtype=torch.int32, device=self.device)
        self._check(self.lib.moe_gate_stats(self.h, _ptr(g), _stream()))
        return g

    def load_diagnostics(self):
        """[L][4]: open-gate fraction, busiest-10 % share, inactive-expert ratio, mean |bias change|."""
        d = torch.empty(self.L, 4, dtype=torch.float32, device=self.device)
        self._check(self.lib.moe_load_diagnostics(self.h, _ptr(d), _stream()))
        return d

    def gate_entropy(self, topk_gate):
        """[L]: mean top-K gate entropy (nats) of the given routing step's gates [L][T][K]."""
        T = topk_gate.shape[-2]
        assert topk_gate.dtype == torch.float32 and topk_gate.is_contiguous() and topk_gate.numel() == self.L * T * self.K
        h = torch.empty(self.L, dtype=torch.float32, device=self.device)
        self._check(self.lib.moe_gate_entropy(self.h, _ptr(topk_gate), T, _ptr(h), _stream()))
        return h

    def score_stats(self, logits, loads=None):
        """Score-distribution statistics of a dumped logit tensor [L][T][E]: dict of entropy_biased [L],
        entropy_softmax [L], mean_prob [L][E] and, when `loads` ([L][E] int32 of the same tokens) is given, aux [L]."""
        T = logits.shape[-2]
        assert logits.dtype == torch.float32 and logits.is_contiguous() and logits.numel() == self.L * T * self.E
        if loads is not None:
            assert loads.dtype == torch.int32 and loads.is_contiguous() and loads.numel() == self.L * self.E
        out = dict(entropy_biased=torch.empty(self.L, dtype=torch.float32, device=self.device),
                   entropy_softmax=torch.empty(self.L, dtype=torch.float32, device=self.device),
                   mean_prob=torch.empty(self.L, self.E, dtype=torch.float32, device=self.device))
        if loads is not None:
            out["aux"] = torch.empty(self.L, dtype=torch.float32, device=self.device)
        self._check(self.lib.moe_score_stats(self.h, _ptr(logits), T, _ptr(loads) if loads is not None else None,
                                             _ptr(out["entropy_biased"]), _ptr(out["entropy_softmax"]),
                                             _ptr(out["mean_prob"]), _ptr(out["aux"]) if loads is not None else None,
                                             _stream()))
        return out

    def loads_peek(self):
        loads = torch.empty(self.L, self.E, dtype=torch.int32, device=self.device)
        self._check(self.lib.moe_loads_peek(self.h, _ptr(loads), _stream()))
        return loads

    def loads_add(self, loads):
        assert loads.dtype == torch.int32 and loads.is_contiguous() and loads.numel() == self.L * self.E
        self._check(self.lib.moe_loads_add(self.h, _ptr(loads), _stream()))

    def loads_view(self):
        """int32 [L][E] tensor that aliases the load accumulators inside the workspace (moe_loads_buffer):
        an in-place all-reduce on it, on the current stream, is the data-parallel exchange."""
        p = C.c_void_p()
        self._check(self.lib.moe_loads_buffer(self.h, C.byref(p)))
        off = p.value - self.workspace.data_ptr()
        n = self.L * self.E * 4
        assert 0 <= off and off + n <= self.workspace.numel() and off % 4 == 0
        return self.workspace[off:off + n].view(torch.int32).view(self.L, self.E)

    def state_export(self, with_step=False):
        """(bias, e_prev) [L][E] float32; with_step=True adds the controller-update counter."""
        bias = torch.empty(self.L, self.E, dtype=torch.float32, device=self.device)
        e_prev = torch.empty(self.L, self.E, dtype=torch.float32, device=self.device)
        step = C.c_int64(-1)
        self._check(self.lib.moe_state_export(self.h, _ptr(bias), _ptr(e_prev), C.byref(step), _stream()))
        return (bias, e_prev, int(step.value)) if with_step else (bias, e_prev)

    def state_import(self, bias=None, e_prev=None, step=-1):
        for t in (bias, e_prev):
            assert t is None or (t.dtype == torch.float32 and t.is_contiguous() and t.numel() == self.L * self.E)
        self._check(self.lib.moe_state_import(self.h, _ptr(bias), _ptr(e_prev), int(step), _stream()))

    def poll(self, raise_on_error=True):
        rc = self.lib.moe_route_poll(self.h)
        if rc != MOE_OK and raise_on_error:
            raise MoeRouteError(rc, self.lib.moe_last_error(self.h).decode())
        return rc

    def debug_wait_timeout(self, spin_limit=2000):
        """Launches the bounded-wait probe (a wait nothing satisfies); poll() then reports MOE_ERR_TIMEOUT."""
        self._check(self.lib.moe_debug_wait_timeout(self.h, spin_limit, _stream()))

    def debug_route_stall(self, after_loads=2):
        """The next route_step's producers stop after `after_loads` pipeline stages (validation of the give-up path)."""
        self._check(self.lib.moe_debug_route_stall(self.h, int(after_loads)))

    def launch_count(self):
        return int(self.lib.moe_route_launch_count(self.h))

    def close(self):
        if getattr(self, "h", None):
            self.lib.moe_route_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

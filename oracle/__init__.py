"""CPU oracle for the ID Balancing routing + load-control path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports or calls it and
shares no code with it.

The arithmetic lives in ``id_balancing_oracle.c`` (plain scalar C); this module
only compiles it with gcc, loads it with ctypes and marshals numpy arrays.
Functions keep the paper's notation: x hidden states, W_r router weights,
z logits, s scores, b bias, n loads, e error.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "id_balancing_oracle.c")
_LIB = os.path.join(_HERE, "libid_balancing_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction, no fast-math)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


_i64, _i32p, _f32p, _f64p = C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_double)
_u16p, _i64p = C.POINTER(C.c_uint16), C.POINTER(C.c_int64)


def lib():
    global _lib
    with _lock:
        if _lib is None:
            build()
            L = C.CDLL(_LIB)
            L.oracle_router_logits_f64.argtypes = [_u16p, _u16p, _i64, _i64, _i64, _f64p]
            L.oracle_router_logits_f64.restype = None
            L.oracle_sigmoid_f64.argtypes = [C.c_double]
            L.oracle_sigmoid_f64.restype = C.c_double
            L.oracle_route_f64.argtypes = [_f64p, _f32p, _i64, _i64, _i64, _i32p, _f64p, _f64p, _f64p]
            L.oracle_sigmoid_f32.argtypes = [C.c_float]
            L.oracle_sigmoid_f32.restype = C.c_float
            L.oracle_sigmoid_f32_array.argtypes = [_f32p, _i64, _f32p]
            L.oracle_sigmoid_f32_array.restype = None
            L.oracle_route_f32.argtypes = [_f32p, _f32p, _i64, _i64, _i64, _i32p, _f32p, _f32p]
            L.oracle_load_counts.argtypes = [_i32p, _i64, _i64, _i64, _i64p]
            L.oracle_load_error.argtypes = [_i64p, _i64, _f32p]
            L.oracle_center.argtypes = [_f32p, _i64]
            L.oracle_id_update.argtypes = [_f32p, _f32p, _f32p, _i64, C.c_float, C.c_float, C.c_int, _i32p]
            L.oracle_fixed_step_update.argtypes = [_f32p, _f32p, _f32p, _i64, C.c_float, C.c_int]
            L.oracle_quantile_target.argtypes = [_f32p, _f32p, _i64, _i64, _i64, _f32p]
            L.oracle_quantile_target_hist.argtypes = [_f32p, _f32p, _i64, _i64, _i64, _i64, C.c_float, _f32p, _i64p]
            L.oracle_quantile_update.argtypes = [_f32p, _f32p, _f32p, _f32p, _i64, C.c_float, C.c_int]
            L.oracle_violations.argtypes = [_i64p, _i64, _f32p, _f32p]
            L.oracle_load_diagnostics.argtypes = [_i64p, _i32p, _f32p, _f32p, _i64, _f32p]
            L.oracle_gate_entropy_mean.argtypes = [_f32p, _i64, _i64]
            L.oracle_gate_entropy_mean.restype = C.c_double
            L.oracle_full_pool_entropy_mean.argtypes = [_f32p, _f32p, _i64, _i64, C.c_int]
            L.oracle_full_pool_entropy_mean.restype = C.c_double
            L.oracle_aux_loss_stats.argtypes = [_f32p, _i64, _i64, _i64p, _f64p, _f64p, _f64p]
            L.oracle_route_tokens_f64.argtypes = [_u16p, _u16p, _f32p, _i64, _i64, _i64, _i64,
                                                  _f64p, _i32p, _f64p, _f64p, _f64p, _i64p]
            _lib = L
    return _lib


def _p(a, ty):
    return a.ctypes.data_as(ty)


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


# ---------------------------------------------------------------- definition
def router_logits_f64(x_bf16_bits, w_bf16_bits):
    """z = W_r x (Section 2.2). x: [T][H] uint16 bf16 bits, w: [E][H] -> [T][E] f64."""
    x = _arr(x_bf16_bits, np.uint16)
    w = _arr(w_bf16_bits, np.uint16)
    T, H = x.shape
    E, H2 = w.shape
    assert H == H2
    z = np.empty((T, E), np.float64)
    lib().oracle_router_logits_f64(_p(x, _u16p), _p(w, _u16p), T, H, E, _p(z, _f64p))
    return z


def sigmoid_f64(z: float) -> float:
    return float(lib().oracle_sigmoid_f64(float(z)))


def route_f64(z, b, K):
    """Biased top-K + gates in binary64 (Eq. 2). Returns idx, gate, alpha, gap."""
    z = _arr(z, np.float64)
    b = _arr(b, np.float32)
    T, E = z.shape
    idx = np.empty((T, K), np.int32)
    gate = np.empty((T, K), np.float64)
    alpha = np.empty(T, np.float64)
    gap = np.empty(T, np.float64)
    rc = lib().oracle_route_f64(_p(z, _f64p), _p(b, _f32p), T, E, K, _p(idx, _i32p),
                                _p(gate, _f64p), _p(alpha, _f64p), _p(gap, _f64p))
    if rc:
        raise ValueError("oracle_route_f64: bad arguments")
    return idx, gate, alpha, gap


def route_tokens_f64(x_bits, w_bits, b, K, threads: int = 1):
    """Whole definition pass over tokens: logits, scores, top-K, gates, loads.

    ``threads`` > 1 splits the tokens over Python threads (the C call releases
    the GIL); the arithmetic per token is unchanged.
    Returns dict(z, idx, gate, alpha, gap, n).
    """
    x = _arr(x_bits, np.uint16)
    w = _arr(w_bits, np.uint16)
    b = _arr(b, np.float32)
    T, H = x.shape
    E = w.shape[0]
    z = np.empty((T, E), np.float64)
    idx = np.empty((T, K), np.int32)
    gate = np.empty((T, K), np.float64)
    alpha = np.empty(T, np.float64)
    gap = np.empty(T, np.float64)
    threads = max(1, min(int(threads), T))
    bounds = np.linspace(0, T, threads + 1).astype(np.int64)
    partial = [np.zeros(E, np.int64) for _ in range(threads)]
    L = lib()

    def run(i):
        lo, hi = int(bounds[i]), int(bounds[i + 1])
        if hi <= lo:
            return 0
        return L.oracle_route_tokens_f64(
            _p(x[lo:hi], _u16p), _p(w, _u16p), _p(b, _f32p), hi - lo, H, E, K,
            _p(z[lo:hi], _f64p), _p(idx[lo:hi], _i32p), _p(gate[lo:hi], _f64p),
            _p(alpha[lo:hi], _f64p), _p(gap[lo:hi], _f64p), _p(partial[i], _i64p))

    if threads == 1:
        rcs = [run(0)]
    else:
        with ThreadPoolExecutor(threads) as ex:
            rcs = list(ex.map(run, range(threads)))
    if any(rcs):
        raise ValueError("oracle_route_tokens_f64 failed")
    n = np.sum(partial, axis=0).astype(np.int64)
    return dict(z=z, idx=idx, gate=gate, alpha=alpha, gap=gap, n=n)


# ------------------------------------------------------------ binary32 chain
def sigmoid_f32(z):
    z = _arr(z, np.float32)
    s = np.empty_like(z)
    lib().oracle_sigmoid_f32_array(_p(z, _f32p), z.size, _p(s, _f32p))
    return s


def route_f32(z, b, K):
    """Biased top-K + gates in binary32 from fp32 logits. Returns idx, gate, alpha."""
    z = _arr(z, np.float32)
    b = _arr(b, np.float32)
    T, E = z.shape
    idx = np.empty((T, K), np.int32)
    gate = np.empty((T, K), np.float32)
    alpha = np.empty(T, np.float32)
    rc = lib().oracle_route_f32(_p(z, _f32p), _p(b, _f32p), T, E, K, _p(idx, _i32p),
                                _p(gate, _f32p), _p(alpha, _f32p))
    if rc:
        raise ValueError("oracle_route_f32: bad arguments")
    return idx, gate, alpha


def load_counts(idx, E, n=None):
    """n_i += #tokens assigned to expert i (Algorithm 1 line 4)."""
    idx = _arr(idx, np.int32)
    T, K = idx.shape
    if n is None:
        n = np.zeros(E, np.int64)
    assert n.dtype == np.int64 and n.flags.c_contiguous
    if lib().oracle_load_counts(_p(idx, _i32p), T, K, E, _p(n, _i64p)):
        raise ValueError("expert index out of range")
    return n


def load_error(n):
    """e_i = (nbar - n_i)/nbar (Eq. 3)."""
    n = _arr(n, np.int64)
    e = np.empty(n.shape[0], np.float32)
    if lib().oracle_load_error(_p(n, _i64p), n.shape[0], _p(e, _f32p)):
        raise ValueError("empty batch: sum of loads is zero")
    return e


def center(b):
    b = _arr(b, np.float32).copy()
    if lib().oracle_center(_p(b, _f32p), b.shape[0]):
        raise ValueError("E must be in [1, 1024]")
    return b


def id_update(b, e_prev, e, ki, kd, center=True):
    """Algorithm 1 lines 8-13. Returns (b_new, e_prev_new, gate)."""
    b = _arr(b, np.float32).copy()
    e_prev = _arr(e_prev, np.float32).copy()
    e = _arr(e, np.float32)
    g = np.empty(b.shape[0], np.int32)
    if lib().oracle_id_update(_p(b, _f32p), _p(e_prev, _f32p), _p(e, _f32p), b.shape[0],
                              ki, kd, int(bool(center)), _p(g, _i32p)):
        raise ValueError("oracle_id_update failed")
    return b, e_prev, g


def fixed_step_update(b, e_prev, e, eta, center=False):
    """Eq. 5. Returns (b_new, e_prev_new)."""
    b = _arr(b, np.float32).copy()
    e_prev = _arr(e_prev, np.float32).copy()
    e = _arr(e, np.float32)
    if lib().oracle_fixed_step_update(_p(b, _f32p), _p(e_prev, _f32p), _p(e, _f32p),
                                      b.shape[0], eta, int(bool(center))):
        raise ValueError("oracle_fixed_step_update failed")
    return b, e_prev


def quantile_target(z32, alpha, K):
    """Eq. 7: Q_j = -quantile_{1-K/E}({S_ij - alpha_i}_i)."""
    z32 = _arr(z32, np.float32)
    alpha = _arr(alpha, np.float32)
    m, E = z32.shape
    Q = np.empty(E, np.float32)
    if lib().oracle_quantile_target(_p(z32, _f32p), _p(alpha, _f32p), m, E, K, _p(Q, _f32p)):
        raise ValueError("oracle_quantile_target failed")
    return Q


def quantile_target_hist(z32, alpha, K, bins, value_range, return_hist=False):
    """Footnote to Eq. 7: Q_j estimated from a per-expert margin histogram (`bins` uniform bins over
    [-value_range, value_range), linear interpolation inside the bin; this build's reading)."""
    z32 = _arr(z32, np.float32)
    alpha = _arr(alpha, np.float32)
    m, E = z32.shape
    Q = np.empty(E, np.float32)
    hist = np.zeros((E, bins), np.int64) if return_hist else None
    rc = lib().oracle_quantile_target_hist(_p(z32, _f32p), _p(alpha, _f32p), m, E, K, bins, float(value_range),
                                           _p(Q, _f32p), _p(hist, _i64p) if return_hist else None)
    if rc:
        raise ValueError("oracle_quantile_target_hist failed")
    return (Q, hist) if return_hist else Q


def quantile_update(b, e_prev, e, Q, rho=0.0, center=False):
    b = _arr(b, np.float32).copy()
    e_prev = _arr(e_prev, np.float32).copy()
    e = _arr(e, np.float32)
    Q = _arr(Q, np.float32)
    if lib().oracle_quantile_update(_p(b, _f32p), _p(e_prev, _f32p), _p(e, _f32p), _p(Q, _f32p),
                                    b.shape[0], rho, int(bool(center))):
        raise ValueError("oracle_quantile_update failed")
    return b, e_prev


def violations(n):
    """Eq. 13. Returns (MaxVio, MinVio) as binary32 values."""
    n = _arr(n, np.int64)
    mx, mn = C.c_float(), C.c_float()
    if lib().oracle_violations(_p(n, _i64p), n.shape[0], C.byref(mx), C.byref(mn)):
        raise ValueError("empty batch: sum of loads is zero")
    return np.float32(mx.value), np.float32(mn.value)


def load_diagnostics(n, gate, b_old, b_new):
    """(gate fraction, busiest-10 % share, inactive-expert ratio, mean |delta b|) as binary32 values."""
    n = _arr(n, np.int64)
    gate = _arr(gate, np.int32)
    b_old = _arr(b_old, np.float32)
    b_new = _arr(b_new, np.float32)
    out = np.empty(4, np.float32)
    if lib().oracle_load_diagnostics(_p(n, _i64p), _p(gate, _i32p), _p(b_old, _f32p), _p(b_new, _f32p),
                                     n.shape[0], _p(out, _f32p)):
        raise ValueError("empty batch: sum of loads is zero")
    return out


def full_pool_entropy_mean(logits, bias=None, kind="biased_sigmoid"):
    """Mean over tokens of the full-pool selection-score entropy (nats), Section 4.3.
    kind "biased_sigmoid": p = clamp(sigmoid(z) + b, 0) normalised; kind "softmax": p = softmax(z)."""
    logits = _arr(logits, np.float32)
    T, E = logits.shape
    bias = np.zeros(E, np.float32) if bias is None else _arr(bias, np.float32)
    k = {"biased_sigmoid": 0, "softmax": 1}[kind]
    return float(lib().oracle_full_pool_entropy_mean(_p(logits, _f32p), _p(bias, _f32p), T, E, k))


def aux_loss_stats(logits, loads):
    """Eq. 8 forward statistics: (f [E], P [E], sum_i f_i P_i) from logits [T][E] and the loads of the same tokens."""
    logits = _arr(logits, np.float32)
    T, E = logits.shape
    n = _arr(loads, np.int64)
    f = np.zeros(E, np.float64)
    P = np.zeros(E, np.float64)
    aux = np.zeros(1, np.float64)
    lib().oracle_aux_loss_stats(_p(logits, _f32p), T, E, _p(n, _i64p), _p(f, _f64p), _p(P, _f64p), _p(aux, _f64p))
    return f, P, float(aux[0])


def gate_entropy_mean(gate):
    """Mean over tokens of H = -sum_k w_k ln w_k (nats), Section 4.3."""
    gate = _arr(gate, np.float32)
    T, K = gate.shape
    return float(lib().oracle_gate_entropy_mean(_p(gate, _f32p), T, K))

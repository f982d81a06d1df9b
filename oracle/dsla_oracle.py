"""ctypes front end of the fp64 token-by-token DSLA checker (``dsla_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Nothing in the CUDA package imports this module and
this module imports nothing from it.  All arrays are numpy float64; reduced
precision inputs are widened exactly by the caller.

    S^i_t = g^i_t * S^i_{t-1} + k_t^T v_t,   o_t = scale * q_t (gamma S^1_t + (1-gamma) S^2_t)
(Sec. 4.1: the dual-state recurrence and its blended readout.)
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dsla_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker with gcc -O2 (no fast-math, so fp64 semantics are IEEE)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-pthread", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.dsla_oracle_run.argtypes = [dp, dp, dp, dp, dp, ctypes.c_int, dp, ip, ip,
                                        ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_double, dp, dp, ctypes.c_int]
        lib.dsla_oracle_run.restype = ctypes.c_int
        lib.dsla_oracle_run_n.argtypes = [dp, dp, dp, ctypes.POINTER(dp), ctypes.c_int, ctypes.c_int, dp, ip, ip,
                                          ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_double, dp, dp, ctypes.c_int]
        lib.dsla_oracle_run_n.restype = ctypes.c_int
        _lib = lib
    return _lib


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ip(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)) if a is not None else None


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def prefill(q, k, v, g_hist, g_rec, gamma, cu_seqlens=None, *, scale=1.0, state=None, slots=None,
            nthreads=None):
    """Token-by-token run of packed sequences.

    q, k: [T, H, dk]; v: [T, H, dv]; g_*: [T, H] (scalar gates) or [T, H, dk]
    (per-key-channel gates); gamma: [H].  cu_seqlens int32 [N+1] (default: one
    sequence).  ``state`` [num_slots, 2, H, dk, dv] is updated in place when
    given (sequence n uses slot slots[n], default n); otherwise zeros are used.
    Returns (o [T, H, dv], state).
    """
    c = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    q, k, v, g_hist, g_rec, gamma = map(c, (q, k, v, g_hist, g_rec, gamma))
    T, H, dk = q.shape
    dv = v.shape[2]
    assert k.shape == (T, H, dk) and v.shape == (T, H, dv) and gamma.shape == (H,)
    per_channel = g_hist.ndim == 3
    assert g_hist.shape == g_rec.shape == ((T, H, dk) if per_channel else (T, H))
    if cu_seqlens is None:
        cu_seqlens = np.array([0, T], dtype=np.int32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    N = cu.size - 1
    assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    sl = None if slots is None else np.ascontiguousarray(slots, dtype=np.int32)
    if state is None:
        nslots = N if sl is None else int(sl.max()) + 1
        state = np.zeros((nslots, 2, H, dk, dv), dtype=np.float64)
    assert state.dtype == np.float64 and state.flags.c_contiguous and state.shape[1:] == (2, H, dk, dv)
    if sl is not None:
        live = sl[sl >= 0]
        assert live.size == np.unique(live).size and (live.size == 0 or live.max() < state.shape[0])
    else:
        assert state.shape[0] >= N
    o = np.zeros((T, H, dv), dtype=np.float64)
    rc = _load().dsla_oracle_run(_dp(q), _dp(k), _dp(v), _dp(g_hist), _dp(g_rec), int(per_channel),
                                 _dp(gamma), _ip(cu), _ip(sl), N, H, dk, dv, float(scale),
                                 _dp(state), _dp(o), int(nthreads or default_threads()))
    if rc != 0:
        raise ValueError("dsla_oracle_run rejected its arguments")
    return o, state


def decode_step(q, k, v, g_hist, g_rec, gamma, state, slots=None, *, scale=1.0, nthreads=None):
    """One recurrence step for B rows: q, k: [B, H, dk]; v: [B, H, dv]; gates [B, H] (or
    [B, H, dk]).  Row b updates slot slots[b] (default b) in place; -1 skips the row (its output is 0).
    This is the same loop as ``prefill`` with every sequence one token long."""
    B = np.asarray(q).shape[0]
    cu = np.arange(B + 1, dtype=np.int32)
    o, _ = prefill(q, k, v, g_hist, g_rec, gamma, cu, scale=scale, state=state, slots=slots, nthreads=nthreads)
    return o


def prefill_n(q, k, v, gates, weights, cu_seqlens=None, *, scale=1.0, state=None, slots=None, nthreads=None):
    """n-state form (Sec. 4.2 / the number-of-states ablation of Sec. 5.5):
        S^i_t = g^i_t * S^i_{t-1} + k_t^T v_t,   o_t = scale * q_t sum_i w_i S^i_t.
    gates: [n, T, H] (or [n, T, H, dk]); weights: [H, n]; state [num_slots, n, H, dk, dv].  Returns (o, state)."""
    c = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    q, k, v, gates, weights = map(c, (q, k, v, gates, weights))
    T, H, dk = q.shape
    dv = v.shape[2]
    n = gates.shape[0]
    per_channel = gates.ndim == 4
    assert gates.shape[1:] == ((T, H, dk) if per_channel else (T, H)) and weights.shape == (H, n)
    if cu_seqlens is None:
        cu_seqlens = np.array([0, T], dtype=np.int32)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    N = cu.size - 1
    assert cu[0] == 0 and cu[-1] == T and np.all(np.diff(cu) >= 0)
    sl = None if slots is None else np.ascontiguousarray(slots, dtype=np.int32)
    if state is None:
        nslots = N if sl is None else int(sl.max()) + 1
        state = np.zeros((nslots, n, H, dk, dv), dtype=np.float64)
    assert state.dtype == np.float64 and state.flags.c_contiguous and state.shape[1:] == (n, H, dk, dv)
    o = np.zeros((T, H, dv), dtype=np.float64)
    dp = ctypes.POINTER(ctypes.c_double)
    gp = (dp * n)(*[_dp(gates[i]) for i in range(n)])
    rc = _load().dsla_oracle_run_n(_dp(q), _dp(k), _dp(v), gp, n, int(per_channel), _dp(weights), _ip(cu), _ip(sl),
                                   N, H, dk, dv, float(scale), _dp(state), _dp(o), int(nthreads or default_threads()))
    if rc != 0:
        raise ValueError("dsla_oracle_run_n rejected its arguments")
    return o, state


def decode_step_n(q, k, v, gates, weights, state, slots=None, *, scale=1.0, nthreads=None):
    """One recurrence step for B rows of the n-state form; gates [n, B, H] (or [n, B, H, dk])."""
    B = np.asarray(q).shape[0]
    cu = np.arange(B + 1, dtype=np.int32)
    o, _ = prefill_n(q, k, v, gates, weights, cu, scale=scale, state=state, slots=slots, nthreads=nthreads)
    return o


def gate_project(x, w, bias=None):
    """Gate producer (Sec. 5.3: the gates come from single linear layers; App. B: zero bias at initialisation):
    g = logistic(x W + b) in fp64.  x: [T, D_model], w: [D_model, n_out], bias: [n_out] or None.  Plain numpy."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    z = x @ w
    if bias is not None:
        z = z + np.asarray(bias, dtype=np.float64)
    return 1.0 / (1.0 + np.exp(-z))

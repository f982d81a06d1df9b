"""ctypes binding of ``libdsla.so``: argument marshalling only.

Every function here has the name of the C entry point it forwards to (see
``include/dsla.h``).  Tensors are torch tensors (torch supplies device memory and
streams); nothing is computed in Python.  The shared library must exist: there is
no CPU fallback and importing this module raises if it cannot be loaded.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_float, c_int, c_int32, c_size_t, c_uint64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdsla.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2506_09316_b200.build` "
                      "(there is no fallback path)")
_lib = ctypes.CDLL(LIB_PATH)

DSLA_OK, DSLA_ERR_INVALID_ARG, DSLA_ERR_UNSUPPORTED, DSLA_ERR_CUDA, DSLA_ERR_OOM, DSLA_ERR_TIMEOUT = range(6)
DSLA_ERR_SCRATCH_LIMIT = 6
DSLA_STATIC_SCRATCH_BYTES = 18 << 20
DSLA_F32, DSLA_BF16 = 0, 1
DSLA_GATE_SCALAR, DSLA_GATE_PER_KEY_CHANNEL = 0, 1
DSLA_IMPL_AUTO, DSLA_IMPL_SIMT, DSLA_IMPL_TENSOR, DSLA_IMPL_TENSOR_PAIR = 0, 1, 2, 3
_DTYPES = {torch.float32: DSLA_F32, torch.bfloat16: DSLA_BF16}
_IMPLS = {"auto": DSLA_IMPL_AUTO, "simt": DSLA_IMPL_SIMT, "tensor": DSLA_IMPL_TENSOR, "pair": DSLA_IMPL_TENSOR_PAIR}


class dsla_prefill_args(Structure):
    _fields_ = [("q", c_void_p), ("k", c_void_p), ("v", c_void_p), ("o", c_void_p),
                ("g_hist", c_void_p), ("g_rec", c_void_p), ("gamma", c_void_p),
                ("cu_seqlens", c_void_p), ("slots", c_void_p),
                ("N", c_int), ("T", c_int), ("T_total", c_int), ("max_seqlen", c_int),
                ("H", c_int), ("d_k", c_int), ("d_v", c_int), ("chunk", c_int),
                ("dtype", c_int), ("scale", c_float), ("use_initial_state", c_int), ("impl", c_int),
                ("workspace", c_void_p), ("workspace_bytes", c_size_t), ("gate_layout", c_int)]


class dsla_decode_args(Structure):
    _fields_ = [("q", c_void_p), ("k", c_void_p), ("v", c_void_p), ("o", c_void_p),
                ("g_hist", c_void_p), ("g_rec", c_void_p), ("gamma", c_void_p), ("slots", c_void_p),
                ("B", c_int), ("H", c_int), ("d_k", c_int), ("d_v", c_int),
                ("dtype", c_int), ("scale", c_float), ("gate_layout", c_int), ("row_mask", c_void_p)]


class dsla_gate_project_args(Structure):
    _fields_ = [("x", c_void_p), ("w", c_void_p), ("bias", c_void_p), ("g_hist", c_void_p), ("g_rec", c_void_p),
                ("T", c_int), ("H", c_int), ("D_model", c_int)]


class dsla_nstate_decode_args(Structure):
    _fields_ = [("q", c_void_p), ("k", c_void_p), ("v", c_void_p), ("o", c_void_p),
                ("gates", c_void_p), ("weights", c_void_p), ("slots", c_void_p), ("row_mask", c_void_p),
                ("B", c_int), ("H", c_int), ("d_k", c_int), ("d_v", c_int), ("n_states", c_int),
                ("dtype", c_int), ("scale", c_float), ("gate_layout", c_int)]


class dsla_nstate_prefill_args(Structure):
    _fields_ = [("q", c_void_p), ("k", c_void_p), ("v", c_void_p), ("o", c_void_p),
                ("gates", c_void_p), ("weights", c_void_p), ("cu_seqlens", c_void_p), ("slots", c_void_p),
                ("N", c_int), ("T", c_int), ("T_total", c_int), ("H", c_int), ("d_k", c_int), ("d_v", c_int),
                ("n_states", c_int), ("dtype", c_int), ("scale", c_float), ("use_initial_state", c_int),
                ("gate_layout", c_int), ("max_seqlen", c_int), ("impl", c_int), ("workspace", c_void_p),
                ("workspace_bytes", c_size_t)]


_lib.dsla_status_string.argtypes = [c_int]
_lib.dsla_status_string.restype = ctypes.c_char_p
_lib.dsla_launch_count.argtypes = []
_lib.dsla_launch_count.restype = c_uint64
_lib.dsla_state_bytes.argtypes = [c_int, c_int, c_int, c_int]
_lib.dsla_state_bytes.restype = c_size_t
_lib.dsla_state_alloc.argtypes = [POINTER(c_void_p), c_int, c_int, c_int, c_int, c_void_p, c_size_t]
_lib.dsla_state_alloc.restype = c_int
_lib.dsla_state_bytes_n.argtypes = [c_int, c_int, c_int, c_int, c_int]
_lib.dsla_state_bytes_n.restype = c_size_t
_lib.dsla_state_alloc_n.argtypes = [POINTER(c_void_p), c_int, c_int, c_int, c_int, c_int, c_void_p, c_size_t]
_lib.dsla_state_alloc_n.restype = c_int
_lib.dsla_nstate_decode_step.argtypes = [POINTER(dsla_nstate_decode_args), c_void_p, c_void_p]
_lib.dsla_nstate_decode_step.restype = c_int
_lib.dsla_nstate_prefill.argtypes = [POINTER(dsla_nstate_prefill_args), c_void_p, c_void_p]
_lib.dsla_nstate_prefill.restype = c_int
_lib.dsla_nstate_prefill_workspace_bytes.argtypes = [POINTER(dsla_nstate_prefill_args)]
_lib.dsla_nstate_prefill_workspace_bytes.restype = c_size_t
_lib.dsla_gate_project.argtypes = [POINTER(dsla_gate_project_args), c_void_p]
_lib.dsla_gate_project.restype = c_int
_lib.dsla_gate_project_last_error.argtypes = []
_lib.dsla_gate_project_last_error.restype = c_int
_lib.dsla_state_free.argtypes = [c_void_p]
_lib.dsla_state_free.restype = c_int
_lib.dsla_state_data.argtypes = [c_void_p]
_lib.dsla_state_data.restype = c_void_p
_lib.dsla_state_zero.argtypes = [c_void_p, c_void_p, c_int, c_void_p]
_lib.dsla_state_zero.restype = c_int
_lib.dsla_state_last_error.argtypes = [c_void_p]
_lib.dsla_state_last_error.restype = c_int
_lib.dsla_selftest_bounded_wait.argtypes = [c_void_p, ctypes.c_uint, c_void_p]
_lib.dsla_selftest_bounded_wait.restype = c_int
_lib.dsla_prefill_workspace_bytes.argtypes = [POINTER(dsla_prefill_args)]
_lib.dsla_prefill_workspace_bytes.restype = c_size_t
_lib.dsla_prefill.argtypes = [POINTER(dsla_prefill_args), c_void_p, c_void_p]
_lib.dsla_prefill.restype = c_int
_lib.dsla_prefill_static_ws.argtypes = [POINTER(dsla_prefill_args), c_void_p, c_void_p]
_lib.dsla_prefill_static_ws.restype = c_int
_lib.dsla_decode_step.argtypes = [POINTER(dsla_decode_args), c_void_p, c_void_p]
_lib.dsla_decode_step.restype = c_int
_lib.dsla_prefill_staging_bytes.argtypes = [POINTER(dsla_prefill_args)]
_lib.dsla_prefill_staging_bytes.restype = c_size_t
_lib.dsla_prefill_host.argtypes = [POINTER(dsla_prefill_args), c_void_p, c_void_p, c_size_t, c_void_p]
_lib.dsla_prefill_host.restype = c_int
_lib.dsla_decode_staging_bytes.argtypes = [POINTER(dsla_decode_args)]
_lib.dsla_decode_staging_bytes.restype = c_size_t
_lib.dsla_decode_step_host.argtypes = [POINTER(dsla_decode_args), c_void_p, c_void_p, c_size_t, c_void_p]
_lib.dsla_decode_step_host.restype = c_int


class DslaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {dsla_status_string(status)}")


def dsla_status_string(status: int) -> str:
    return _lib.dsla_status_string(int(status)).decode()


def dsla_launch_count() -> int:
    return int(_lib.dsla_launch_count())


def dsla_state_bytes(num_slots: int, H: int, d_k: int, d_v: int) -> int:
    return int(_lib.dsla_state_bytes(num_slots, H, d_k, d_v))


def _check(rc: int, where: str):
    if rc != DSLA_OK:
        raise DslaError(rc, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


class DslaState:
    """Handle of a dual-state store; ``tensor`` is a torch view [num_slots, 2, H, d_k, d_v] fp32."""

    def __init__(self, handle, tensor, num_slots, H, d_k, d_v):
        self.handle, self.tensor = handle, tensor
        self.num_slots, self.H, self.d_k, self.d_v = num_slots, H, d_k, d_v

    def __del__(self):
        try:
            dsla_state_free(self)
        except Exception:
            pass


def dsla_state_alloc(num_slots: int, H: int, d_k: int, d_v: int, device="cuda", buffer=None) -> DslaState:
    """The store borrows a torch allocation, so the library itself calls no cudaMalloc for it.  ``buffer`` may be a
    contiguous fp32 tensor of the store's size that the caller owns (e.g. a view into a larger allocation)."""
    n = dsla_state_bytes(num_slots, H, d_k, d_v)
    if buffer is not None:
        buf = buffer.view(num_slots, 2, H, d_k, d_v)
    else:
        buf = torch.empty((num_slots, 2, H, d_k, d_v), dtype=torch.float32, device=device) if n else None
    h = c_void_p()
    with torch.cuda.device(buf.device if buf is not None else device):
        rc = _lib.dsla_state_alloc(byref(h), num_slots, H, d_k, d_v, _ptr(buf), n)
    _check(rc, "dsla_state_alloc")
    return DslaState(h, buf, num_slots, H, d_k, d_v)


def dsla_state_bytes_n(num_slots: int, n_states: int, H: int, d_k: int, d_v: int) -> int:
    return int(_lib.dsla_state_bytes_n(num_slots, n_states, H, d_k, d_v))


def dsla_state_alloc_n(num_slots: int, n_states: int, H: int, d_k: int, d_v: int, device="cuda") -> DslaState:
    """Store of the n-state form; ``tensor`` is [num_slots, n_states, H, d_k, d_v] fp32."""
    n = dsla_state_bytes_n(num_slots, n_states, H, d_k, d_v)
    buf = torch.empty((num_slots, n_states, H, d_k, d_v), dtype=torch.float32, device=device) if n else None
    h = c_void_p()
    with torch.cuda.device(buf.device if buf is not None else device):
        rc = _lib.dsla_state_alloc_n(byref(h), num_slots, n_states, H, d_k, d_v, _ptr(buf), n)
    _check(rc, "dsla_state_alloc_n")
    st = DslaState(h, buf, num_slots, H, d_k, d_v)
    st.n_states = n_states
    return st


def dsla_state_free(st: DslaState):
    if st.handle is not None and st.handle.value:
        h, st.handle = st.handle, None
        _check(_lib.dsla_state_free(h), "dsla_state_free")


def dsla_state_data(st: DslaState) -> int:
    return int(_lib.dsla_state_data(st.handle) or 0)


def dsla_state_zero(st: DslaState, slots=None, stream=None):
    n = 0 if slots is None else int(slots.numel())
    _check(_lib.dsla_state_zero(st.handle, _ptr(slots), n, _stream(stream)), "dsla_state_zero")


def dsla_state_last_error(st: DslaState) -> int:
    return int(_lib.dsla_state_last_error(st.handle))


def dsla_selftest_bounded_wait(st: DslaState, max_polls: int = 2000, stream=None):
    _check(_lib.dsla_selftest_bounded_wait(st.handle, int(max_polls), _stream(stream)), "dsla_selftest_bounded_wait")


def _prefill_args(q, k, v, o, g_hist, g_rec, gamma, cu_seqlens, slots, N, T, max_seqlen, chunk, scale,
                  use_initial_state, impl, workspace):
    T_total, H, d_k = q.shape
    a = dsla_prefill_args()
    a.q, a.k, a.v, a.o = _ptr(q), _ptr(k), _ptr(v), _ptr(o)
    a.g_hist, a.g_rec, a.gamma = _ptr(g_hist), _ptr(g_rec), _ptr(gamma)
    a.cu_seqlens, a.slots = _ptr(cu_seqlens), _ptr(slots)
    a.N, a.T, a.T_total, a.max_seqlen = int(N), int(T), int(T_total), int(max_seqlen)
    a.H, a.d_k, a.d_v, a.chunk = int(H), int(d_k), int(v.shape[2]), int(chunk)
    a.dtype = _DTYPES[q.dtype]
    a.scale = float(scale)
    a.use_initial_state = int(bool(use_initial_state))
    a.impl = _IMPLS[impl] if isinstance(impl, str) else int(impl)
    a.workspace = _ptr(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    a.gate_layout = DSLA_GATE_PER_KEY_CHANNEL if (g_hist is not None and g_hist.dim() == 3) else DSLA_GATE_SCALAR
    return a


def dsla_prefill_workspace_bytes(T_total, N, max_seqlen, H, d, dtype=torch.bfloat16, chunk=64, impl="auto",
                                 dense_T=None) -> int:
    a = dsla_prefill_args()
    a.N, a.T, a.T_total, a.max_seqlen = int(N), int(dense_T or 0), int(T_total), int(max_seqlen)
    a.H, a.d_k, a.d_v, a.chunk = int(H), int(d), int(d), int(chunk)
    a.dtype = _DTYPES[dtype]
    a.impl = _IMPLS[impl]
    a.scale = 1.0
    if dense_T is None:
        a.cu_seqlens = c_void_p(8)  # only tested for NULL, never dereferenced
    return int(_lib.dsla_prefill_workspace_bytes(byref(a)))


def dsla_prefill(q, k, v, g_hist, g_rec, gamma, st: DslaState, *, o=None, cu_seqlens=None, slots=None,
                 max_seqlen=None, chunk=64, scale=1.0, use_initial_state=False, impl="auto", workspace=None,
                 stream=None):
    """q, k, v: [T_total, H, d] device tensors (fp32 or bf16).  Dense batches pass ``cu_seqlens=None``
    with q shaped [B*T, H, d] and ``max_seqlen=T``.  Returns o; final states land in ``st``."""
    T_total = q.shape[0]
    if cu_seqlens is None:
        T = int(max_seqlen) if max_seqlen is not None else T_total
        N = T_total // T if T > 0 else 0
        max_seqlen = T
    else:
        N, T = cu_seqlens.numel() - 1, 0
        if max_seqlen is None:
            raise ValueError("max_seqlen is required with cu_seqlens")
    if o is None:
        o = torch.empty_like(v)
    if workspace is None:
        need = dsla_prefill_workspace_bytes(T_total, N, max_seqlen, q.shape[1], q.shape[2], q.dtype, chunk,
                                            impl if isinstance(impl, str) else "auto",
                                            dense_T=T if cu_seqlens is None else None)
        if need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    a = _prefill_args(q, k, v, o, g_hist, g_rec, gamma, cu_seqlens, slots, N, T, max_seqlen, chunk, scale,
                      use_initial_state, impl, workspace)
    _check(_lib.dsla_prefill(byref(a), st.handle, _stream(stream)), "dsla_prefill")
    return o


def dsla_prefill_static_ws(q, k, v, g_hist, g_rec, gamma, st: DslaState, *, o=None, cu_seqlens=None, slots=None,
                           max_seqlen=None, chunk=64, scale=1.0, use_initial_state=False, impl="auto", stream=None):
    """Same as ``dsla_prefill`` but the scratch for the segment summaries is the fixed array inside the
    library, so neither the caller nor the library allocates anything for the call (``o`` must then be
    passed in by callers that cannot allocate).  Raises DslaError(DSLA_ERR_SCRATCH_LIMIT) when the sizes
    need more than DSLA_STATIC_SCRATCH_BYTES.  Calls that overlap on the GPU race on the shared array."""
    T_total = q.shape[0]
    if cu_seqlens is None:
        T = int(max_seqlen) if max_seqlen is not None else T_total
        N = T_total // T if T > 0 else 0
        max_seqlen = T
    else:
        N, T = cu_seqlens.numel() - 1, 0
        if max_seqlen is None:
            raise ValueError("max_seqlen is required with cu_seqlens")
    if o is None:
        o = torch.empty_like(v)
    a = _prefill_args(q, k, v, o, g_hist, g_rec, gamma, cu_seqlens, slots, N, T, max_seqlen, chunk, scale,
                      use_initial_state, impl, None)
    _check(_lib.dsla_prefill_static_ws(byref(a), st.handle, _stream(stream)), "dsla_prefill_static_ws")
    return o


def _decode_args(q, k, v, o, g_hist, g_rec, gamma, slots, scale, row_mask=None):
    B, H, d_k = q.shape
    a = dsla_decode_args()
    a.q, a.k, a.v, a.o = _ptr(q), _ptr(k), _ptr(v), _ptr(o)
    a.g_hist, a.g_rec, a.gamma, a.slots = _ptr(g_hist), _ptr(g_rec), _ptr(gamma), _ptr(slots)
    a.B, a.H, a.d_k, a.d_v = int(B), int(H), int(d_k), int(v.shape[2])
    a.dtype = _DTYPES[q.dtype]
    a.scale = float(scale)
    a.gate_layout = DSLA_GATE_PER_KEY_CHANNEL if g_hist.dim() == 3 else DSLA_GATE_SCALAR
    a.row_mask = _ptr(row_mask)
    return a


def dsla_decode_step(q, k, v, g_hist, g_rec, gamma, st: DslaState, *, o=None, slots=None, scale=1.0, row_mask=None,
                     stream=None):
    """q, k, v: [B, H, d] device tensors; updates the rows' slots in place and returns o [B, H, d].  Gates [B, H], or
    [B, H, d] per key channel.  ``row_mask`` (uint8 [B]): rows with 0 are not touched (state and o)."""
    if o is None:
        o = torch.empty_like(v)
    a = _decode_args(q, k, v, o, g_hist, g_rec, gamma, slots, scale, row_mask)
    _check(_lib.dsla_decode_step(byref(a), st.handle, _stream(stream)), "dsla_decode_step")
    return o


def dsla_prefill_host(q, k, v, g_hist, g_rec, gamma, st: DslaState, o, staging, *, cu_seqlens=None, slots=None,
                      max_seqlen=None, chunk=64, scale=1.0, use_initial_state=False, impl="auto", workspace=None,
                      stream=None):
    """Host-buffer variant: q, k, v, g_hist, g_rec, o are (pinned) host tensors; gamma, cu_seqlens,
    slots, staging and workspace are device tensors.  Copies run on ``stream``."""
    T_total = q.shape[0]
    if cu_seqlens is None:
        T = int(max_seqlen) if max_seqlen is not None else T_total
        N = T_total // T if T > 0 else 0
        max_seqlen = T
    else:
        N, T = cu_seqlens.numel() - 1, 0
    a = _prefill_args(q, k, v, o, g_hist, g_rec, gamma, cu_seqlens, slots, N, T, max_seqlen, chunk, scale,
                      use_initial_state, impl, workspace)
    _check(_lib.dsla_prefill_host(byref(a), st.handle, _ptr(staging), staging.numel() * staging.element_size(),
                                  _stream(stream)), "dsla_prefill_host")
    return o


def dsla_prefill_staging_bytes(T_total, N, max_seqlen, H, d, dtype=torch.bfloat16, dense_T=None) -> int:
    a = dsla_prefill_args()
    a.N, a.T, a.T_total, a.max_seqlen = int(N), int(dense_T or 0), int(T_total), int(max_seqlen)
    a.H, a.d_k, a.d_v, a.chunk = int(H), int(d), int(d), 64
    a.dtype = _DTYPES[dtype]
    a.scale = 1.0
    if dense_T is None:
        a.cu_seqlens = c_void_p(8)
    return int(_lib.dsla_prefill_staging_bytes(byref(a)))


def dsla_decode_staging_bytes(B, H, d, dtype=torch.bfloat16) -> int:
    a = dsla_decode_args()
    a.B, a.H, a.d_k, a.d_v = int(B), int(H), int(d), int(d)
    a.dtype = _DTYPES[dtype]
    return int(_lib.dsla_decode_staging_bytes(byref(a)))


def dsla_decode_step_host(q, k, v, g_hist, g_rec, gamma, st: DslaState, o, staging, *, slots=None, scale=1.0,
                          stream=None):
    a = _decode_args(q, k, v, o, g_hist, g_rec, gamma, slots, scale)
    _check(_lib.dsla_decode_step_host(byref(a), st.handle, _ptr(staging), staging.numel() * staging.element_size(),
                                      _stream(stream)), "dsla_decode_step_host")
    return o


def dsla_nstate_decode_step(q, k, v, gates, weights, st: DslaState, *, o=None, slots=None, scale=1.0, row_mask=None,
                            stream=None):
    """n-state decode step: gates [n, B, H] (or [n, B, H, d] per key channel) fp32, weights [H, n] fp32."""
    if o is None:
        o = torch.empty_like(v)
    B, H, d_k = q.shape
    a = dsla_nstate_decode_args()
    a.q, a.k, a.v, a.o = _ptr(q), _ptr(k), _ptr(v), _ptr(o)
    a.gates, a.weights, a.slots, a.row_mask = _ptr(gates), _ptr(weights), _ptr(slots), _ptr(row_mask)
    a.B, a.H, a.d_k, a.d_v, a.n_states = int(B), int(H), int(d_k), int(v.shape[2]), int(gates.shape[0])
    a.dtype = _DTYPES[q.dtype]
    a.scale = float(scale)
    a.gate_layout = DSLA_GATE_PER_KEY_CHANNEL if gates.dim() == 4 else DSLA_GATE_SCALAR
    _check(_lib.dsla_nstate_decode_step(byref(a), st.handle, _stream(stream)), "dsla_nstate_decode_step")
    return o


def _nstate_prefill_args(q, k, v, o, gates, weights, cu_seqlens, slots, max_seqlen, scale, use_initial_state, impl):
    T_total, H, d_k = q.shape
    if cu_seqlens is None:
        T = int(max_seqlen) if max_seqlen is not None else T_total
        N = T_total // T if T > 0 else 0
        max_seqlen = T
    else:
        N, T = cu_seqlens.numel() - 1, 0
        if max_seqlen is None:
            max_seqlen = T_total      # an upper bound is valid (the tighter the bound, the better the segment plan)
    a = dsla_nstate_prefill_args()
    a.q, a.k, a.v, a.o = _ptr(q), _ptr(k), _ptr(v), _ptr(o)
    a.gates, a.weights, a.cu_seqlens, a.slots = _ptr(gates), _ptr(weights), _ptr(cu_seqlens), _ptr(slots)
    a.N, a.T, a.T_total, a.H, a.d_k, a.d_v = int(N), int(T), int(T_total), int(H), int(d_k), int(v.shape[2])
    a.n_states = int(gates.shape[0])
    a.dtype = _DTYPES[q.dtype]
    a.scale = float(scale)
    a.use_initial_state = int(bool(use_initial_state))
    a.gate_layout = DSLA_GATE_PER_KEY_CHANNEL if gates.dim() == 4 else DSLA_GATE_SCALAR
    a.max_seqlen = int(max_seqlen)
    a.impl = _IMPLS[impl]
    return a


def dsla_nstate_prefill_workspace_bytes(q, k, v, gates, weights, *, cu_seqlens=None, max_seqlen=None, impl="auto") -> int:
    """Scratch bytes ``dsla_nstate_prefill`` needs for these tensors (0 for the token-by-token kernel)."""
    a = _nstate_prefill_args(q, k, v, v, gates, weights, cu_seqlens, None, max_seqlen, 1.0, False, impl)
    return int(_lib.dsla_nstate_prefill_workspace_bytes(byref(a)))


def dsla_nstate_prefill(q, k, v, gates, weights, st: DslaState, *, o=None, cu_seqlens=None, slots=None, max_seqlen=None,
                        scale=1.0, use_initial_state=False, impl="auto", workspace=None, stream=None):
    """n-state prefill: gates [n, T_total, H] (or [n, T_total, H, d] per key channel), weights [H, n].  bf16, d = 128
    with scalar gates runs on the chunkwise tensor-core kernel, one pass per pair of states (``impl="simt"`` forces the
    token-by-token CUDA-core kernel, which serves everything else)."""
    if o is None:
        o = torch.empty_like(v)
    a = _nstate_prefill_args(q, k, v, o, gates, weights, cu_seqlens, slots, max_seqlen, scale, use_initial_state, impl)
    if workspace is None:
        need = int(_lib.dsla_nstate_prefill_workspace_bytes(byref(a)))
        if need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    a.workspace = _ptr(workspace)
    a.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.dsla_nstate_prefill(byref(a), st.handle, _stream(stream)), "dsla_nstate_prefill")
    return o


def dsla_gate_project(x, w, bias=None, *, g_hist=None, g_rec=None, stream=None):
    """logistic(x W^T + bias) on the tensor cores: x [T, D_model] bf16, w [2 H, D_model] bf16, bias [2 H] fp32 or None.
    Returns (g_hist, g_rec), both [T, H] fp32."""
    T, D_model = x.shape
    H = w.shape[0] // 2
    if g_hist is None:
        g_hist = torch.empty((T, H), dtype=torch.float32, device=x.device)
    if g_rec is None:
        g_rec = torch.empty((T, H), dtype=torch.float32, device=x.device)
    a = dsla_gate_project_args()
    a.x, a.w, a.bias, a.g_hist, a.g_rec = _ptr(x), _ptr(w), _ptr(bias), _ptr(g_hist), _ptr(g_rec)
    a.T, a.H, a.D_model = int(T), int(H), int(D_model)
    _check(_lib.dsla_gate_project(byref(a), _stream(stream)), "dsla_gate_project")
    return g_hist, g_rec


def dsla_gate_project_last_error() -> int:
    return int(_lib.dsla_gate_project_last_error())

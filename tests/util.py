"""Helpers shared by the parity tests: run the CUDA path, run the CPU checker, compare."""
import numpy as np
import torch

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}   # max relative error per tensor (inf-norm relative)


def rel_err(x, ref):
    """max|x - ref| / max|ref| over the whole tensor (the error measure used for every parity claim)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.max(np.abs(ref)) if ref.size else 0.0
    num = np.max(np.abs(x - ref)) if ref.size else 0.0
    if not np.isfinite(num):
        return float("inf")
    return float(num / den) if den > 0 else float(num)


def elementwise_err(x, ref):
    """Element-wise diagnostic next to rel_err: |x - ref| / (|ref| + 1e-3 rms(ref)); returns (max, 99.9th percentile)."""
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    if ref.size == 0:
        return 0.0, 0.0
    e = np.abs(x - ref) / (np.abs(ref) + 1e-3 * np.sqrt(np.mean(ref * ref)))
    return float(e.max()), float(np.quantile(e, 0.999))


def large_element_err(x, ref):
    """max |x - ref| / |ref| over the elements whose magnitude is at least the tensor's rms."""
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    big = np.abs(ref) >= np.sqrt(np.mean(ref * ref))
    return float(np.max(np.abs(x - ref)[big] / np.abs(ref)[big])) if big.any() else 0.0


def oracle_prefill(inp, state0=None, slots=None, scale=1.0, nthreads=None):
    from oracle import dsla_oracle as orc
    f = inp.as_f64()
    st = None if state0 is None else np.ascontiguousarray(state0, dtype=np.float64).copy()
    return orc.prefill(f["q"], f["k"], f["v"], f["g_hist"], f["g_rec"], f["gamma"], f["cu_seqlens"],
                       scale=scale, state=st, slots=slots, nthreads=nthreads)


GUARD = 4096          # elements of sentinel before and after every buffer the kernels write
SENTINEL = 12345.0


class Guarded:
    """A device buffer with a band of sentinel values before and after it.  The kernels only ever get the middle
    part; `check()` fails when anything was written outside it (stands in for a memory checker)."""

    def __init__(self, numel, dtype, dev="cuda"):
        self.full = torch.full((numel + 2 * GUARD,), SENTINEL, dtype=dtype, device=dev)
        self.mid = self.full[GUARD:GUARD + numel]

    def check(self, what):
        lo, hi = self.full[:GUARD], self.full[GUARD + self.mid.numel():]
        assert bool((lo == SENTINEL).all()) and bool((hi == SENTINEL).all()), f"write outside {what}"


def gpu_prefill(inp, *, num_slots=None, state0=None, slots=None, chunk=64, impl="auto", scale=1.0, dense=False):
    """Runs dsla_prefill on cuda:0; returns (o, states) as fp64 numpy.  The output tensor and the state store sit
    between sentinel bands that must come back untouched."""
    import paper_2506_09316_b200 as dsla
    dev = "cuda"
    d = inp.to(dev)
    N = inp.N
    num_slots = num_slots or max(N, 1)
    gs = Guarded(num_slots * 2 * inp.H * inp.d * inp.d, torch.float32, dev)
    st = dsla.dsla_state_alloc(num_slots, inp.H, inp.d, inp.d, buffer=gs.mid)
    if state0 is not None:
        st.tensor.copy_(torch.as_tensor(np.asarray(state0), dtype=torch.float32))
    else:
        st.tensor.fill_(float("nan"))        # a start from zeros must not read the slot
    go = Guarded(d.v.numel(), d.v.dtype, dev)
    o = go.mid.view(d.v.shape)
    o.fill_(float("nan"))
    sl = None if slots is None else torch.as_tensor(np.asarray(slots), dtype=torch.int32, device=dev)
    lens = inp.seqlens
    kw = dict(chunk=chunk, impl=impl, scale=scale, use_initial_state=state0 is not None, slots=sl)
    if dense:
        assert len(set(lens)) == 1
        dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, o=o, max_seqlen=lens[0], **kw)
    else:
        dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, o=o, cu_seqlens=d.cu_seqlens,
                          max_seqlen=max(lens) if lens else 0, **kw)
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    gs.check("the state store")
    go.check("the output tensor")
    return o.double().cpu().numpy(), st.tensor.double().cpu().numpy()

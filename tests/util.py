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


def oracle_prefill(inp, state0=None, slots=None, scale=1.0, nthreads=None):
    from oracle import dsla_oracle as orc
    f = inp.as_f64()
    st = None if state0 is None else np.ascontiguousarray(state0, dtype=np.float64).copy()
    return orc.prefill(f["q"], f["k"], f["v"], f["g_hist"], f["g_rec"], f["gamma"], f["cu_seqlens"],
                       scale=scale, state=st, slots=slots, nthreads=nthreads)


def gpu_prefill(inp, *, num_slots=None, state0=None, slots=None, chunk=64, impl="auto", scale=1.0, dense=False):
    """Runs dsla_prefill on cuda:0; returns (o, states) as fp64 numpy."""
    import paper_2506_09316_b200 as dsla
    dev = "cuda"
    d = inp.to(dev)
    N = inp.N
    num_slots = num_slots or max(N, 1)
    st = dsla.dsla_state_alloc(num_slots, inp.H, inp.d, inp.d)
    if state0 is not None:
        st.tensor.copy_(torch.as_tensor(np.asarray(state0), dtype=torch.float32))
    else:
        st.tensor.fill_(float("nan"))        # a start from zeros must not read the slot
    sl = None if slots is None else torch.as_tensor(np.asarray(slots), dtype=torch.int32, device=dev)
    lens = inp.seqlens
    kw = dict(chunk=chunk, impl=impl, scale=scale, use_initial_state=state0 is not None, slots=sl)
    if dense:
        assert len(set(lens)) == 1
        o = dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, max_seqlen=lens[0], **kw)
    else:
        o = dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, cu_seqlens=d.cu_seqlens,
                              max_seqlen=max(lens) if lens else 0, **kw)
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    return o.double().cpu().numpy(), st.tensor.double().cpu().numpy()

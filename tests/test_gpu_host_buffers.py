"""The host-buffer entry points (pinned host tensors in, host tensor out, copies inside the call) give exactly
what the device-pointer entry points give, for a packed prefill followed by decode steps."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen
from util import TOL, oracle_prefill, rel_err

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def _pin(t):
    return t.contiguous().pin_memory()


@pytest.mark.parametrize("lens,H,dense", [([700, 33, 0, 129], 3, False), ([2000], 2, False), ([5000], 2, True)])
def test_prefill_and_decode_through_host_buffers(lens, H, dense):
    """dense=True with one long sequence takes the sliced pipeline (copies of slice i+1 and i-1 overlap the kernels of
    slice i, which continue from the states of slice i-1): same result up to summation order."""
    import paper_2506_09316_b200 as dsla
    d, dev = 128, "cuda"
    inp = gen.make_packed(9500 + len(lens), lens, H, d, BF)
    N, T_total, max_len = len(lens), sum(lens), max(lens)
    dv = inp.to(dev)
    ws_bytes = dsla.binding.dsla_prefill_workspace_bytes(T_total, N, max_len, H, d, BF, 64, "auto")
    ws = torch.empty(max(ws_bytes, 1), dtype=torch.uint8, device=dev)

    # device-pointer path
    st_a = dsla.dsla_state_alloc(N, H, d, d)
    cu = None if dense else dv.cu_seqlens
    o_a = dsla.dsla_prefill(dv.q, dv.k, dv.v, dv.g_hist, dv.g_rec, dv.gamma, st_a, cu_seqlens=cu, max_seqlen=max_len, workspace=ws)
    # host-buffer path
    st_b = dsla.dsla_state_alloc(N, H, d, d)
    stg = torch.empty(dsla.binding.dsla_prefill_staging_bytes(T_total, N, max_len, H, d, BF), dtype=torch.uint8, device=dev)
    ho = _pin(torch.empty(T_total, H, d, dtype=BF))
    dsla.dsla_prefill_host(_pin(inp.q), _pin(inp.k), _pin(inp.v), _pin(inp.g_hist), _pin(inp.g_rec), dv.gamma, st_b, ho, stg,
                           cu_seqlens=cu, max_seqlen=max_len, workspace=ws)
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st_a) == dsla.DSLA_OK and dsla.dsla_state_last_error(st_b) == dsla.DSLA_OK
    live = [n for n, L in enumerate(lens) if L > 0]
    if dense:
        assert rel_err(ho.double().numpy(), o_a.double().cpu().numpy()) <= TOL[BF]
        assert rel_err(st_b.tensor[live].double().cpu().numpy(), st_a.tensor[live].double().cpu().numpy()) <= TOL[BF]
    else:
        assert torch.equal(o_a.cpu(), ho)
        assert torch.equal(st_a.tensor[live].cpu(), st_b.tensor[live].cpu())
    o_ref, S_ref = oracle_prefill(inp)
    assert rel_err(ho.double().numpy(), o_ref) <= TOL[BF]
    for n in live:
        for i in range(2):
            assert rel_err(st_b.tensor[n, i].double().cpu().numpy(), S_ref[n, i]) <= TOL[BF]

    # two decode steps on top, rows = sequences
    stg2 = torch.empty(dsla.binding.dsla_decode_staging_bytes(N, H, d, BF), dtype=torch.uint8, device=dev)
    for step in range(2):
        dec = gen.make_dense(9600 + step, N, 1, H, d, BF)
        q, k, v = (x.reshape(N, H, d) for x in (dec.q, dec.k, dec.v))
        g1, g2 = dec.g_hist.reshape(N, H), dec.g_rec.reshape(N, H)
        o_dev = dsla.dsla_decode_step(q.to(dev), k.to(dev), v.to(dev), g1.to(dev), g2.to(dev), dv.gamma, st_a)
        o_host = _pin(torch.empty(N, H, d, dtype=BF))
        dsla.dsla_decode_step_host(_pin(q), _pin(k), _pin(v), _pin(g1), _pin(g2), dv.gamma, st_b, o_host, stg2)
        torch.cuda.synchronize()
        if dense:
            assert rel_err(o_host.double().numpy(), o_dev.double().cpu().numpy()) <= TOL[BF]
        else:
            assert torch.equal(o_dev.cpu(), o_host)
    if not dense:
        assert torch.equal(st_a.tensor.cpu()[live], st_b.tensor.cpu()[live])

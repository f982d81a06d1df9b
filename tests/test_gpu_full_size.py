"""Parity at the full sizes of the named workloads, in the launch configuration the benchmark times.
The CPU checker cannot run these in full, so sampled independent units (sequence, head[, layer]) are
compared one by one; a unit is exact evidence for itself because units do not interact."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen
from util import rel_err

pytestmark = pytest.mark.gpu
TOL = 2e-2


def oracle_unit(dev_inp, t0, t1, h, state0=None):
    """Token-by-token fp64 run of tokens [t0, t1) of head h, copied from the device tensors."""
    from oracle import dsla_oracle as orc
    f = lambda t: t[t0:t1, h:h + 1].double().cpu().numpy()
    gam = dev_inp.gamma[h:h + 1].double().cpu().numpy()
    st = None if state0 is None else np.ascontiguousarray(state0, dtype=np.float64).copy()
    return orc.prefill(f(dev_inp.q), f(dev_inp.k), f(dev_inp.v), f(dev_inp.g_hist), f(dev_inp.g_rec), gam,
                       state=st, nthreads=1)


def test_cfg3_long_context_prefill_sampled_heads():
    """Workload 3: B=1, H=32, d=128, T=65536, bf16: heads 0, 13, 31 in full (outputs and final states)."""
    import paper_2506_09316_b200 as dsla
    c = gen.CONFIGS["cfg3"]
    T, H, d = c["T"], c["H"], c["d"]
    inp = gen.make_packed_device(c["seed"], [T], H, d, torch.bfloat16)
    st = dsla.dsla_state_alloc(1, H, d, d)
    st.tensor.fill_(float("nan"))
    o = dsla.dsla_prefill(inp.q, inp.k, inp.v, inp.g_hist, inp.g_rec, inp.gamma, st, max_seqlen=T, chunk=c["chunk"])
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    for h in (0, 13, 31):
        o_ref, S_ref = oracle_unit(inp, 0, T, h)
        assert rel_err(o[:, h].float().cpu().numpy(), o_ref[:, 0]) <= TOL
        S = st.tensor[0, :, h].double().cpu().numpy()
        assert rel_err(S[0], S_ref[0, 0, 0]) <= TOL and rel_err(S[1], S_ref[0, 1, 0]) <= TOL


def test_cfg4_batched_decode_sampled_units():
    """Workload 4: B=128, H=32, d=128, 32 independent layers (17.2 GB of fp32 states), 3 steps; sampled
    (layer, row, head) units against the recurrence, every other slot of one layer checked for bookkeeping."""
    import paper_2506_09316_b200 as dsla
    from oracle import dsla_oracle as orc
    c = gen.CONFIGS["cfg4"]
    B, H, d, L = c["B"], c["H"], c["d"], c["layers"]
    steps = 3
    states = [dsla.dsla_state_alloc(B, H, d, d) for _ in range(L)]
    g = torch.Generator(device="cuda")
    g.manual_seed(c["seed"])
    for s in states:
        s.tensor.normal_(0.0, c["state_std"], generator=g)
    units = [(0, 0, 0), (0, 127, 31), (17, 64, 5), (31, 0, 31), (31, 127, 0)]
    S_ref = {u: states[u[0]].tensor[u[1], :, u[2]].double().cpu().numpy()[None, :, None].copy() for u in units}
    ring = gen.make_packed_device(c["seed"] + 1, [1] * (L * steps * B), H, d, torch.bfloat16)
    view = lambda t: t.view(L, steps, B, *t.shape[1:])
    q, k, v, g1, g2 = map(view, (ring.q, ring.k, ring.v, ring.g_hist, ring.g_rec))
    o = torch.empty_like(v)
    for s_ in range(steps):
        for l in range(L):
            dsla.dsla_decode_step(q[l, s_], k[l, s_], v[l, s_], g1[l, s_], g2[l, s_], ring.gamma, states[l], o=o[l, s_])
    torch.cuda.synchronize()
    worst = 0.0
    for (l, b, h) in units:
        for s_ in range(steps):
            f = lambda t: t[l, s_, b:b + 1, h:h + 1].double().cpu().numpy()
            o_ref = orc.decode_step(f(q), f(k), f(v), f(g1), f(g2), ring.gamma[h:h + 1].double().cpu().numpy(),
                                    S_ref[(l, b, h)], nthreads=1)
            worst = max(worst, rel_err(o[l, s_, b, h].float().cpu().numpy(), o_ref[0, 0]))
        S = states[l].tensor[b, :, h].double().cpu().numpy()
        worst = max(worst, rel_err(S, S_ref[(l, b, h)][0, :, 0]))
    assert worst <= TOL, worst


def test_cfg5_ragged_prefill_then_decode_sampled_units():
    """Workload 5: 64 prompts, lengths log-uniform in [1K, 64K] (about 1M tokens), packed varlen prefill into
    64 slots, then continuous batched decode on the same slots with finished rows marked -1."""
    import paper_2506_09316_b200 as dsla
    from oracle import dsla_oracle as orc
    c = gen.CONFIGS["cfg5"]
    H, d = c["H"], c["d"]
    lens = gen.ragged_lengths(c["seed"], c["N"], c["lo"], c["hi"])
    N, total = len(lens), int(sum(lens))
    assert 700_000 < total < 1_400_000
    inp = gen.make_packed_device(c["seed"], lens, H, d, torch.bfloat16)
    cu = inp.cu_seqlens.cpu().numpy()
    slots = torch.randperm(N, generator=torch.Generator().manual_seed(7)).to(torch.int32)
    st = dsla.dsla_state_alloc(N, H, d, d)
    st.tensor.fill_(float("nan"))
    o = dsla.dsla_prefill(inp.q, inp.k, inp.v, inp.g_hist, inp.g_rec, inp.gamma, st, cu_seqlens=inp.cu_seqlens,
                          slots=slots.cuda(), max_seqlen=max(lens))
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    order = np.argsort(lens)
    picks = [(int(order[0]), 0), (int(order[-1]), 31), (0, 7), (N - 1, 31)]     # shortest, longest, first, last
    refs = {}
    for (n, h) in picks:
        o_ref, S_ref = oracle_unit(inp, int(cu[n]), int(cu[n + 1]), h)
        assert rel_err(o[cu[n]:cu[n + 1], h].float().cpu().numpy(), o_ref[:, 0]) <= TOL, (n, h)
        S = st.tensor[int(slots[n]), :, h].double().cpu().numpy()
        assert rel_err(S[0], S_ref[0, 0, 0]) <= TOL and rel_err(S[1], S_ref[0, 1, 0]) <= TOL, (n, h)
        refs[(n, h)] = S_ref[:, :, 0:1].copy()
    # continuous batched decode on the same slots; the second half of the steps runs with a quarter of the rows finished
    steps = 8
    dec_slots = slots.clone()
    finished = torch.arange(0, N, 4)
    for s_ in range(steps):
        if s_ == steps // 2:
            dec_slots[finished] = -1
        di = gen.make_packed_device(c["seed"] + 100 + s_, [1] * N, H, d, torch.bfloat16)
        od = dsla.dsla_decode_step(di.q, di.k, di.v, di.g_hist, di.g_rec, inp.gamma, st, slots=dec_slots.cuda())
        torch.cuda.synchronize()
        for (n, h) in picks:
            if dec_slots[n] < 0:
                assert not od[n].float().abs().max().item() > 0
                continue
            f = lambda t: t[n:n + 1, h:h + 1].double().cpu().numpy()
            o_ref = orc.decode_step(f(di.q), f(di.k), f(di.v), f(di.g_hist), f(di.g_rec),
                                    inp.gamma[h:h + 1].double().cpu().numpy(), refs[(n, h)], nthreads=1)
            assert rel_err(od[n, h].float().cpu().numpy(), o_ref[0, 0]) <= TOL
    for (n, h) in picks:
        S = st.tensor[int(slots[n]), :, h].double().cpu().numpy()
        assert rel_err(S, refs[(n, h)][0, :, 0]) <= TOL

"""Parity of the wider forms of the layer against the fp64 CPU checker: gates per key channel (the gated-linear-attention
parameterisation of Sec. 2), n states with one blend weight each (Sec. 4.2, Sec. 5.5), and decode batches in which only some
rows belong to a DSLA layer (Sec. 4.5, App. D).  Tolerances are those of the dual-state path."""
import numpy as np
import pytest
import torch

from oracle import dsla_oracle as orc
from paper_2506_09316_b200 import inputs as gen
from util import TOL, rel_err

pytestmark = pytest.mark.gpu
F32, BF = torch.float32, torch.bfloat16


def _f64(t):
    return t.detach().to("cpu", torch.float64).numpy()


def _channel_gates(rng, shape, pattern="mix"):
    """Activated gates in [0, 1] per key channel: a slow and a fast family, exact zeros and ones sprinkled in."""
    g = 1.0 / (1.0 + np.exp(-rng.normal(3.0, 2.0, size=shape)))
    if pattern == "mix":
        u = rng.uniform(size=shape)
        g[u < 0.02] = 0.0
        g[u > 0.98] = 1.0
    elif pattern == "zeros":
        g[:] = 0.0
    elif pattern == "ones":
        g[:] = 1.0
    return g.astype(np.float32)


# ------------------------------------------------------------------------------------------ decode
@pytest.mark.parametrize("dtype", [F32, BF])
@pytest.mark.parametrize("d", [64, 128])
def test_decode_per_key_channel_gates(dtype, d):
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3100 + d)
    B, H = 5, 3
    inp = gen.make_dense(3101 + d, B, 1, H, d, dtype)
    g1, g2 = _channel_gates(rng, (B, H, d)), _channel_gates(rng, (B, H, d))
    st0 = gen.make_states(3102, B + 1, H, d, d, std=0.5)
    slots = np.array([3, 0, 5, 1, 4], dtype=np.int32)
    st = dsla.dsla_state_alloc(B + 1, H, d, d)
    st.tensor.copy_(st0)
    ref_state = st0.double().numpy().copy()
    dv = inp.to("cuda")
    for step in range(3):          # repeated calls on the same slots
        o = dsla.dsla_decode_step(dv.q, dv.k, dv.v, torch.from_numpy(g1).cuda(), torch.from_numpy(g2).cuda(), dv.gamma, st,
                                  slots=torch.from_numpy(slots).cuda(), scale=0.7)
        f = inp.as_f64()
        o_ref = orc.decode_step(f["q"], f["k"], f["v"], g1, g2, f["gamma"], ref_state, slots, scale=0.7)
        torch.cuda.synchronize()
        assert rel_err(_f64(o), o_ref) <= TOL[dtype]
        assert rel_err(_f64(st.tensor), ref_state) <= TOL[dtype]
    assert np.array_equal(_f64(st.tensor)[2], st0.double().numpy()[2])      # the slot no row uses


def test_decode_row_mask_leaves_masked_rows_alone():
    import paper_2506_09316_b200 as dsla
    B, H, d = 8, 4, 128
    inp = gen.make_dense(3200, B, 1, H, d, BF)
    st0 = gen.make_states(3201, B, H, d, d, std=0.3)
    st = dsla.dsla_state_alloc(B, H, d, d)
    st.tensor.copy_(st0)
    dv = inp.to("cuda")
    mask = np.array([1, 0, 1, 1, 0, 0, 1, 0], dtype=np.uint8)
    o = torch.full_like(dv.v, 7.0)          # rows of other layer types keep what their own kernel wrote
    dsla.dsla_decode_step(dv.q, dv.k, dv.v, dv.g_hist, dv.g_rec, dv.gamma, st, o=o, row_mask=torch.from_numpy(mask).cuda())
    torch.cuda.synchronize()
    f = inp.as_f64()
    ref_state = st0.double().numpy().copy()
    slots = np.where(mask == 1, np.arange(B), -1).astype(np.int32)
    o_ref = orc.decode_step(f["q"], f["k"], f["v"], f["g_hist"], f["g_rec"], f["gamma"], ref_state, slots)
    on, Sn = _f64(o), _f64(st.tensor)
    live = mask == 1
    assert rel_err(on[live], o_ref[live]) <= TOL[BF] and rel_err(Sn[live], ref_state[live]) <= TOL[BF]
    assert np.all(on[~live] == 7.0), "a masked row's output was written"
    assert np.array_equal(Sn[~live], st0.double().numpy()[~live]), "a masked row's state was written"


@pytest.mark.parametrize("n", [1, 2, 4, 8])
@pytest.mark.parametrize("vec", [False, True])
def test_nstate_decode(n, vec):
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3300 + n)
    B, H, d = 4, 3, 128
    inp = gen.make_dense(3301 + n, B, 1, H, d, BF)
    gates = _channel_gates(rng, (n, B, H, d)) if vec else _channel_gates(rng, (n, B, H))
    w = rng.normal(size=(H, n)).astype(np.float32)
    st0 = (rng.normal(size=(B, n, H, d, d)) * 0.3).astype(np.float32)
    st = dsla.dsla_state_alloc_n(B, n, H, d, d)
    st.tensor.copy_(torch.from_numpy(st0))
    ref_state = st0.astype(np.float64)
    dv = inp.to("cuda")
    f = inp.as_f64()
    mask = np.array([1, 1, 0, 1], dtype=np.uint8)
    slots = np.where(mask == 1, np.arange(B), -1).astype(np.int32)
    for step in range(2):
        o = torch.full_like(dv.v, 5.0)
        dsla.dsla_nstate_decode_step(dv.q, dv.k, dv.v, torch.from_numpy(gates).cuda(), torch.from_numpy(w).cuda(), st, o=o,
                                     scale=0.9, row_mask=torch.from_numpy(mask).cuda())
        torch.cuda.synchronize()
        o_ref = orc.decode_step_n(f["q"], f["k"], f["v"], gates, w, ref_state, slots, scale=0.9)
        live = mask == 1
        assert rel_err(_f64(o)[live], o_ref[live]) <= TOL[BF]
        assert rel_err(_f64(st.tensor), ref_state) <= TOL[BF]
        assert np.all(_f64(o)[~live] == 5.0)


def test_two_state_nstate_decode_equals_the_dual_state_step():
    """n = 2 with w = (gamma, 1 - gamma) is the dual-state layer: same kernel instantiation, same results."""
    import paper_2506_09316_b200 as dsla
    B, H, d = 6, 2, 64
    inp = gen.make_dense(3400, B, 1, H, d, F32)
    st0 = gen.make_states(3401, B, H, d, d, std=0.4)
    dv = inp.to("cuda")
    a, b = dsla.dsla_state_alloc(B, H, d, d), dsla.dsla_state_alloc_n(B, 2, H, d, d)
    a.tensor.copy_(st0); b.tensor.copy_(st0)
    o1 = dsla.dsla_decode_step(dv.q, dv.k, dv.v, dv.g_hist, dv.g_rec, dv.gamma, a)
    w = torch.stack([dv.gamma, 1.0 - dv.gamma], dim=1).contiguous()
    o2 = dsla.dsla_nstate_decode_step(dv.q, dv.k, dv.v, torch.stack([dv.g_hist, dv.g_rec]).contiguous(), w, b)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2) and torch.equal(a.tensor, b.tensor)


# ------------------------------------------------------------------------------------------ prefill
@pytest.mark.parametrize("dtype,d", [(F32, 64), (BF, 128), (F32, 128)])
@pytest.mark.parametrize("pattern", ["mix", "zeros", "ones"])
def test_prefill_per_key_channel_gates(dtype, d, pattern):
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3500 + d)
    lens = [5, 1, 0, 130, 67]
    H = 2
    inp = gen.make_packed(3501 + d, lens, H, d, dtype)
    T = inp.T_total
    g1, g2 = _channel_gates(rng, (T, H, d), pattern), _channel_gates(rng, (T, H, d), pattern)
    slots = np.array([4, 2, 0, 6, 3], dtype=np.int32)
    for use_init in (False, True):
        st0 = gen.make_states(3502, 7, H, d, d, std=0.5)
        st = dsla.dsla_state_alloc(7, H, d, d)
        st.tensor.copy_(st0)
        dv = inp.to("cuda")
        o = dsla.dsla_prefill(dv.q, dv.k, dv.v, torch.from_numpy(g1).cuda(), torch.from_numpy(g2).cuda(), dv.gamma, st,
                              cu_seqlens=dv.cu_seqlens, slots=torch.from_numpy(slots).cuda(), max_seqlen=max(lens), scale=0.5,
                              use_initial_state=use_init)
        torch.cuda.synchronize()
        assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
        f = inp.as_f64()
        ref_state = st0.double().numpy().copy() if use_init else np.zeros((7, 2, H, d, d))
        o_ref, S_ref = orc.prefill(f["q"], f["k"], f["v"], g1, g2, f["gamma"], f["cu_seqlens"], scale=0.5, state=ref_state,
                                   slots=slots)
        assert rel_err(_f64(o), o_ref) <= TOL[dtype]
        Sn = _f64(st.tensor)
        for s_idx, L in zip(slots, lens):
            if L > 0 or use_init:
                assert rel_err(Sn[s_idx], S_ref[s_idx]) <= TOL[dtype] or not np.any(S_ref[s_idx])
            if not np.any(S_ref[s_idx]):
                assert not np.any(Sn[s_idx])


def test_tensor_kernels_refuse_per_key_channel_gates():
    import paper_2506_09316_b200 as dsla
    inp = gen.make_dense(3600, 1, 70, 2, 128, BF).to("cuda")
    g = torch.ones(70, 2, 128, device="cuda")
    st = dsla.dsla_state_alloc(1, 2, 128, 128)
    for impl in ("tensor", "pair"):
        with pytest.raises(dsla.DslaError) as e:
            dsla.dsla_prefill(inp.q, inp.k, inp.v, g, g, inp.gamma, st, max_seqlen=70, impl=impl)
        assert e.value.status == dsla.DSLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("n", [1, 2, 4, 8])
@pytest.mark.parametrize("dtype,d,vec,impl", [(F32, 64, False, "auto"), (BF, 128, False, "auto"), (BF, 128, False, "simt"), (BF, 128, True, "auto"),
                                               (F32, 64, True, "auto")])
def test_nstate_prefill(n, dtype, d, vec, impl):
    """bf16, d = 128, scalar gates: AUTO runs the chunkwise tensor-core kernel once per pair of states (n = 1: a pair whose
    second state has weight 0 and never touches the slot); everything else (and impl="simt") the token-by-token kernel."""
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3700 + n + d)
    lens = [33, 0, 150, 1]
    H = 2
    inp = gen.make_packed(3701 + n, lens, H, d, dtype)
    T = inp.T_total
    gates = _channel_gates(rng, (n, T, H, d)) if vec else _channel_gates(rng, (n, T, H))
    w = rng.normal(size=(H, n)).astype(np.float32)
    slots = np.array([2, 0, 3, 1], dtype=np.int32)
    st0 = (rng.normal(size=(4, n, H, d, d)) * 0.3).astype(np.float32)
    st = dsla.dsla_state_alloc_n(4, n, H, d, d)
    st.tensor.copy_(torch.from_numpy(st0))
    dv = inp.to("cuda")
    o = dsla.dsla_nstate_prefill(dv.q, dv.k, dv.v, torch.from_numpy(gates).cuda(), torch.from_numpy(w).cuda(), st,
                                 cu_seqlens=dv.cu_seqlens, slots=torch.from_numpy(slots).cuda(), scale=0.8,
                                 use_initial_state=True, impl=impl, max_seqlen=max(lens))
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    f = inp.as_f64()
    ref_state = st0.astype(np.float64)
    o_ref, S_ref = orc.prefill_n(f["q"], f["k"], f["v"], gates, w, f["cu_seqlens"], scale=0.8, state=ref_state, slots=slots)
    # with more than one group of states the output is rounded to dtype once per group
    tol = TOL[dtype] * (1.5 if (dtype == BF and n == 8) else 1.0)
    assert rel_err(_f64(o), o_ref) <= tol
    assert rel_err(_f64(st.tensor), S_ref) <= TOL[dtype]


@pytest.mark.parametrize("n,use_init", [(1, True), (1, False), (2, False), (4, True), (8, False)])
def test_nstate_prefill_tensor_path_with_split_sequences(n, use_init):
    """Few (sequence, head) pairs and long sequences: every pair of states runs the summary pass, the fold and (on a
    resume) the snapshot of its own two states; pairs after the first add to the output."""
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3750 + n)
    lens = [1500, 64, 777]
    H, d = 2, 128
    inp = gen.make_packed(3751 + n, lens, H, d, BF)
    T = inp.T_total
    gates = (1.0 / (1.0 + np.exp(-rng.normal(3.0, 1.5, size=(n, T, H))))).astype(np.float32)
    gates[:, 100, :] = 0.0
    gates[:, 900:910, 0] = 1.0
    w = rng.normal(size=(H, n)).astype(np.float32)
    st0 = (rng.normal(size=(3, n, H, d, d)) * 0.3).astype(np.float32)
    st = dsla.dsla_state_alloc_n(3, n, H, d, d)
    st.tensor.copy_(torch.from_numpy(st0))
    dv = inp.to("cuda")
    o = dsla.dsla_nstate_prefill(dv.q, dv.k, dv.v, torch.from_numpy(gates).cuda(), torch.from_numpy(w).cuda(), st,
                                 cu_seqlens=dv.cu_seqlens, max_seqlen=max(lens), use_initial_state=use_init, impl="tensor")
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    f = inp.as_f64()
    ref_state = st0.astype(np.float64) if use_init else np.zeros_like(st0, dtype=np.float64)
    o_ref, S_ref = orc.prefill_n(f["q"], f["k"], f["v"], gates, w, f["cu_seqlens"], state=ref_state)
    assert rel_err(_f64(o), o_ref) <= TOL[BF] * (1.5 if n == 8 else 1.0)
    assert rel_err(_f64(st.tensor), S_ref) <= TOL[BF]
    # the tensor path is refused where it does not apply
    with pytest.raises(dsla.DslaError) as e:        # gates per key channel
        dsla.dsla_nstate_prefill(dv.q, dv.k, dv.v, torch.ones(n, T, H, d, device="cuda"), torch.from_numpy(w).cuda(), st,
                                 cu_seqlens=dv.cu_seqlens, max_seqlen=max(lens), impl="tensor")
    assert e.value.status == dsla.DSLA_ERR_UNSUPPORTED


def test_nstate_entry_points_check_the_store():
    import paper_2506_09316_b200 as dsla
    inp = gen.make_dense(3800, 2, 1, 2, 64, F32).to("cuda")
    st2 = dsla.dsla_state_alloc(2, 2, 64, 64)
    gates = torch.ones(4, 2, 2, device="cuda")
    w = torch.ones(2, 4, device="cuda")
    with pytest.raises(dsla.DslaError) as e:            # a two-state store handed to a four-state call
        dsla.dsla_nstate_decode_step(inp.q, inp.k, inp.v, gates, w, st2)
    assert e.value.status == dsla.DSLA_ERR_INVALID_ARG
    st4 = dsla.dsla_state_alloc_n(2, 4, 2, 64, 64)
    with pytest.raises(dsla.DslaError) as e:            # a four-state store handed to the dual-state call
        dsla.dsla_decode_step(inp.q, inp.k, inp.v, inp.g_hist, inp.g_rec, inp.gamma, st4)
    assert e.value.status == dsla.DSLA_ERR_INVALID_ARG
    with pytest.raises(dsla.DslaError) as e:            # three states: no kernel
        dsla.dsla_state_alloc_n(2, 3, 2, 64, 64)
    assert e.value.status == dsla.DSLA_ERR_UNSUPPORTED


# ------------------------------------------------------------------------------------------ gate producer
@pytest.mark.parametrize("T,H,D_model,with_bias", [(1, 8, 64, False), (130, 32, 512, True), (4096, 32, 4096, False),
                                                   (300, 16, 1024, True), (257, 128, 256, True)])
def test_gate_project(T, H, D_model, with_bias):
    """logistic(x W^T + b) against the fp64 checker (bf16 inputs widened exactly; products are exact in fp32, so only the
    summation order, the fp32 accumulator and the approximate exponential differ), then straight into a prefill."""
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3900 + T)
    x = torch.from_numpy(rng.normal(size=(T, D_model)).astype(np.float32)).to(BF)
    w = torch.from_numpy((rng.normal(size=(2 * H, D_model)) * (2.0 / np.sqrt(D_model))).astype(np.float32)).to(BF)
    b = torch.from_numpy(rng.normal(size=2 * H).astype(np.float32) * 2.0) if with_bias else None
    gh = torch.full((T, H), float("nan"), device="cuda")
    gr = torch.full((T, H), float("nan"), device="cuda")
    dsla.dsla_gate_project(x.cuda(), w.cuda(), None if b is None else b.cuda(), g_hist=gh, g_rec=gr)
    torch.cuda.synchronize()
    assert dsla.dsla_gate_project_last_error() == dsla.DSLA_OK
    ref = orc.gate_project(x.double().numpy(), w.double().numpy().T, None if b is None else b.double().numpy())
    got = np.concatenate([_f64(gh), _f64(gr)], axis=1)
    assert np.max(np.abs(got - ref)) <= 2e-5, np.max(np.abs(got - ref))
    assert got.min() >= 0.0 and got.max() <= 1.0


def test_gate_project_feeds_the_prefill():
    import paper_2506_09316_b200 as dsla
    rng = np.random.default_rng(3950)
    T, H, d, D_model = 300, 8, 128, 256
    inp = gen.make_dense(3951, 1, T, H, d, BF)
    x = torch.from_numpy(rng.normal(size=(T, D_model)).astype(np.float32)).to(BF)
    w = torch.from_numpy((rng.normal(size=(2 * H, D_model)) / np.sqrt(D_model)).astype(np.float32)).to(BF)
    b = torch.from_numpy(np.concatenate([np.full(H, 5.0), np.full(H, 1.0)]).astype(np.float32))
    gh, gr = dsla.dsla_gate_project(x.cuda(), w.cuda(), b.cuda())
    dv = inp.to("cuda")
    st = dsla.dsla_state_alloc(1, H, d, d)
    o = dsla.dsla_prefill(dv.q, dv.k, dv.v, gh, gr, dv.gamma, st, max_seqlen=T)
    torch.cuda.synchronize()
    g = orc.gate_project(x.double().numpy(), w.double().numpy().T, b.double().numpy())
    f = inp.as_f64()
    o_ref, S_ref = orc.prefill(f["q"], f["k"], f["v"], g[:, :H], g[:, H:], f["gamma"])
    assert rel_err(_f64(o), o_ref) <= TOL[BF] and rel_err(_f64(st.tensor), S_ref) <= TOL[BF]


def test_gate_project_rejects_unsupported_shapes():
    import paper_2506_09316_b200 as dsla
    x = torch.zeros(4, 100, dtype=BF, device="cuda")
    w = torch.zeros(16, 100, dtype=BF, device="cuda")
    with pytest.raises(dsla.DslaError) as e:
        dsla.dsla_gate_project(x, w)                       # D_model not a multiple of 64
    assert e.value.status == dsla.DSLA_ERR_UNSUPPORTED
    with pytest.raises(dsla.DslaError) as e:
        dsla.dsla_gate_project(torch.zeros(4, 128, dtype=BF, device="cuda"), torch.zeros(12, 128, dtype=BF, device="cuda"))   # H = 6
    assert e.value.status == dsla.DSLA_ERR_UNSUPPORTED

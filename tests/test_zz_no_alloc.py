"""dsla_prefill_static_ws: the prefill entry point for callers that cannot allocate device memory (a frozen
allocator, a plug-in that only receives its tensors, a latency path that must not touch cudaMalloc).
Its scratch is a fixed array inside the library, shared by every call, so the checks here are: same
results as dsla_prefill on the same inputs, twice in a row with different inputs (stale scratch from
the first call must not leak into the second), and a clear refusal above the built-in size."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def _run(entry, d, st, max_seqlen):
    import paper_2506_09316_b200 as dsla
    st.tensor.fill_(float("nan"))
    o = torch.full_like(d.v, float("nan"))
    entry(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, o=o, max_seqlen=max_seqlen, impl="tensor")
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    return o.float().cpu().numpy(), st.tensor.cpu().numpy().copy()


def test_static_scratch_matches_workspace_entry_twice_in_a_row():
    import paper_2506_09316_b200 as dsla
    from util import rel_err
    H, d, T = 4, 128, 1500                     # few heads: the sequence is split into segments, scratch is used
    need = dsla.binding.dsla_prefill_workspace_bytes(T, 1, T, H, d, torch.bfloat16, 64, "tensor", dense_T=T)
    assert 0 < need <= dsla.DSLA_STATIC_SCRATCH_BYTES
    st = dsla.dsla_state_alloc(1, H, d, d)
    for seed in (9101, 9102):                  # two calls in a row, different data
        dev = gen.make_dense(seed, 1, T, H, d, torch.bfloat16).to("cuda")
        o_ref, S_ref = _run(dsla.dsla_prefill, dev, st, T)
        o_new, S_new = _run(dsla.dsla_prefill_static_ws, dev, st, T)
        assert rel_err(o_new, o_ref) <= 2e-2 and rel_err(S_new, S_ref) <= 2e-2
        assert np.isfinite(o_new).all() and np.isfinite(S_new).all()


def test_static_scratch_refuses_sizes_beyond_the_array():
    import paper_2506_09316_b200 as dsla
    H, d, T, N = 37, 128, 2048, 1              # 37 heads x 4 segments of summaries: just over the built-in size
    need = dsla.binding.dsla_prefill_workspace_bytes(N * T, N, T, H, d, torch.bfloat16, 64, "tensor", dense_T=T)
    if need <= dsla.DSLA_STATIC_SCRATCH_BYTES:
        pytest.skip("this shape fits the built-in scratch")
    dev = gen.make_packed_device(9103, [T] * N, H, d, torch.bfloat16)
    st = dsla.dsla_state_alloc(N, H, d, d)
    with pytest.raises(dsla.DslaError) as e:
        dsla.dsla_prefill_static_ws(dev.q, dev.k, dev.v, dev.g_hist, dev.g_rec, dev.gamma, st, max_seqlen=T,
                                    impl="tensor")
    assert e.value.status == dsla.DSLA_ERR_SCRATCH_LIMIT

"""Failure reporting of the device side, exercised without hanging or faulting anything: the give-up path of the
bounded waits, and the check that a packed sequence fits the max_seqlen the segments were sized for."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen
from util import TOL, gpu_prefill, oracle_prefill, rel_err

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


def test_bounded_wait_gives_up_and_the_device_stays_usable():
    import paper_2506_09316_b200 as dsla
    st = dsla.dsla_state_alloc(1, 2, 128, 128)
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    dsla.dsla_selftest_bounded_wait(st, 3000)          # one warp, one barrier nobody arrives at, 3000 polls
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_ERR_TIMEOUT     # the kernel returned and said why
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK              # reading clears the word
    # an ordinary prefill afterwards is still right
    inp = gen.make_dense(9901, 1, 300, 2, 128, BF)
    o, S = gpu_prefill(inp, impl="tensor")
    o_ref, S_ref = oracle_prefill(inp)
    assert rel_err(o, o_ref) <= TOL[BF] and rel_err(S, S_ref) <= TOL[BF]


def test_selftest_rejects_unbounded_limits():
    import paper_2506_09316_b200 as dsla
    st = dsla.dsla_state_alloc(1, 2, 128, 128)
    for bad in (0, 2_000_000):
        with pytest.raises(dsla.DslaError) as e:
            dsla.dsla_selftest_bounded_wait(st, bad)
        assert e.value.status == dsla.DSLA_ERR_INVALID_ARG


@pytest.mark.parametrize("H", [2, 40])     # split into segments / one segment per sequence
def test_sequence_longer_than_max_seqlen_is_reported(H):
    """cu_seqlens lives on the device, so the host cannot check max_seqlen; the kernel does and raises the status word
    instead of silently dropping the tail of the long sequence."""
    import paper_2506_09316_b200 as dsla
    lens = [900, 130]
    inp = gen.make_packed(9902, lens, H, 128, BF)
    d = inp.to("cuda")
    st = dsla.dsla_state_alloc(2, H, 128, 128)
    dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, cu_seqlens=d.cu_seqlens, max_seqlen=256,
                      impl="tensor")
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_ERR_INVALID_ARG
    # with the right bound the same call is clean and correct
    o = dsla.dsla_prefill(d.q, d.k, d.v, d.g_hist, d.g_rec, d.gamma, st, cu_seqlens=d.cu_seqlens, max_seqlen=900,
                          impl="tensor")
    torch.cuda.synchronize()
    assert dsla.dsla_state_last_error(st) == dsla.DSLA_OK
    o_ref, _ = oracle_prefill(inp)
    assert rel_err(o.double().cpu().numpy(), o_ref) <= TOL[BF]


def test_split_prefill_with_initial_state_next_to_a_busy_stream(tc_impl):
    """A sequence split into segments that resumes from a stored state: the CTA of the last segment overwrites the slot
    that CTAs of earlier segments read as their initial state.  They read a snapshot taken beforehand, so the result must
    not depend on how the CTAs get scheduled -- here a second stream keeps part of the GPU busy with ordinary matmuls."""
    import paper_2506_09316_b200 as dsla
    inp = gen.make_dense(9903, 1, 64 * 48, 2, 128, BF)
    st0 = gen.make_states(9904, 1, 2, 128, 128, std=0.4).numpy()
    o_ref, S_ref = oracle_prefill(inp, state0=st0)
    side = torch.cuda.Stream()
    a = torch.randn(4096, 4096, device="cuda", dtype=torch.bfloat16)
    for attempt in range(3):
        with torch.cuda.stream(side):
            for _ in range(6):
                a @ a                                  # bounded, ordinary work that occupies SMs for a while
        o, S = gpu_prefill(inp, state0=st0, impl=tc_impl)
        side.synchronize()
        assert rel_err(o, o_ref) <= TOL[BF] and rel_err(S, S_ref) <= TOL[BF], f"attempt {attempt}"

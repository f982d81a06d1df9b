"""Seeded random shapes for the tensor-core prefill: packed batches of mixed lengths, head counts on both sides of
the SM count (with and without the split into segments), four gate regimes, permuted slots, optional initial
states; every case is also run twice and must reproduce bit for bit."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen
from util import TOL, gpu_prefill, oracle_prefill, rel_err

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


@pytest.mark.parametrize("case", range(12))
def test_tensor_prefill_random_case(case, tc_impl):
    rng = np.random.default_rng(9100 + case)
    H = int(rng.choice([1, 2, 3, 5, 8, 40]))
    N = int(rng.integers(1, 5 if H == 40 else 7))
    hi = 400 if H == 40 else int(rng.choice([70, 300, 1500, 3000]))
    lens = [int(x) for x in rng.integers(0, hi, size=N)]
    if sum(lens) == 0:
        lens[0] = 65
    T = sum(lens)
    inp = gen.make_packed(9200 + case, lens, H, 128, BF)
    regime = case % 4
    if regime == 1:      # strong decay with exact zeros
        g = rng.uniform(0, 1, size=(T, H)).astype(np.float32)
        g[rng.uniform(size=(T, H)) < 0.05] = 0.0
        inp.g_rec = torch.from_numpy(g)
    elif regime == 2:    # no decay at all
        inp.g_hist = torch.ones(T, H)
        inp.g_rec = torch.ones(T, H)
    elif regime == 3:    # tiny gates
        inp.g_hist = torch.full((T, H), 1e-4)
        inp.g_rec = torch.from_numpy(rng.uniform(0, 1e-2, size=(T, H)).astype(np.float32))
    use_init = bool(rng.integers(0, 2))
    slots = [int(x) for x in rng.permutation(N + 2)[:N]]
    st0 = gen.make_states(9300 + case, N + 2, H, 128, 128, std=0.3).numpy() if use_init else None
    kw = dict(state0=st0, slots=slots, num_slots=N + 2, impl=tc_impl, scale=0.7)
    o, S = gpu_prefill(inp, **kw)
    o2, S2 = gpu_prefill(inp, **kw)
    assert np.array_equal(o, o2) and all(np.array_equal(S[s], S2[s]) for s in slots), "not reproducible"
    o_ref, S_ref = oracle_prefill(inp, state0=st0, slots=slots, scale=0.7)
    assert rel_err(o, o_ref) <= TOL[BF]
    for s, L in zip(slots, lens):
        if L > 0 or use_init:
            for i in range(2):
                assert rel_err(S[s, i], S_ref[s, i]) <= TOL[BF]

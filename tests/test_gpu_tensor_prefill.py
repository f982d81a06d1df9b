"""Parity of the tensor-core (tcgen05) prefill kernel against the fp64 CPU checker."""
import numpy as np
import pytest
import torch

from paper_2506_09316_b200 import inputs as gen
from test_gpu_parity import _with_gates, check_prefill

pytestmark = pytest.mark.gpu
BF = torch.bfloat16


@pytest.mark.parametrize("T", [1, 2, 63, 64, 65, 131, 513, 1100])
def test_tensor_prefill_lengths(T, tc_impl):
    H = 3 if T < 600 else 2          # few (sequence, head) pairs: long inputs are split into segments
    check_prefill(gen.make_dense(8000 + T, 1, T, H, 128, BF), impl=tc_impl)


def test_tensor_prefill_many_heads_single_segment(tc_impl):
    check_prefill(gen.make_dense(8100, 5, 200, 32, 128, BF), impl=tc_impl, dense=True)


def test_tensor_prefill_ragged_slots_initial_state(tc_impl):
    lens = [5, 1, 0, 130, 67, 700]
    inp = gen.make_packed(8200, lens, 2, 128, BF)
    check_prefill(inp, impl=tc_impl)
    slots = [4, 2, 0, 6, 3, 1]
    st0 = gen.make_states(8201, 8, 2, 128, 128, std=0.5).numpy()
    check_prefill(inp, state0=st0, slots=slots, num_slots=8, impl=tc_impl, scale=0.5)


def test_tensor_prefill_packed_batch_longest_first(tc_impl):
    """More (sequence, head) pairs than SMs: no split, blocks visit the sequences by descending length (ties,
    empty sequences and a ragged last chunk included); slots are permuted so a wrong sequence index shows."""
    rng = np.random.default_rng(8600)
    lens = [int(x) for x in rng.integers(1, 400, size=38)] + [0, 257, 257, 64]
    inp = gen.make_packed(8601, lens, 4, 128, BF)
    slots = [int(x) for x in rng.permutation(len(lens))]
    check_prefill(inp, slots=slots, num_slots=len(lens), impl=tc_impl)


def test_tensor_prefill_ragged_batch_split_into_segments(tc_impl):
    """Few pairs with very different lengths: every sequence is cut with the longest one's segment plan, so short
    sequences leave later segments empty; summaries, their fold into the initial state and the order array all run."""
    inp = gen.make_packed(8700, [3000, 700, 65, 0, 1], 2, 128, BF)
    check_prefill(inp, impl=tc_impl)
    st0 = gen.make_states(8701, 5, 2, 128, 128, std=0.3).numpy()
    check_prefill(inp, state0=st0, impl=tc_impl)


@pytest.mark.parametrize("T", [64 * 40, 64 * 200 + 17])
def test_tensor_prefill_single_head_sixteen_segments(T, tc_impl):
    """One (sequence, head) pair: the deepest split (up to 16 segments, later ones shorter than earlier ones)."""
    check_prefill(gen.make_dense(8800 + T % 97, 1, T, 1, 128, BF), impl=tc_impl)


@pytest.mark.parametrize("pattern", ["ones", "zeros", "single_zero", "alternating", "swapped", "tiny"])
def test_tensor_prefill_gate_patterns(pattern, tc_impl):
    T, H, d = 600, 2, 128
    inp = gen.make_dense(8300, 1, T, H, d, BF)
    t = np.arange(T)[:, None]
    if pattern == "ones":
        _with_gates(inp, 1.0, 1.0)
    elif pattern == "zeros":
        _with_gates(inp, 0.0, 0.0)
    elif pattern == "single_zero":
        g1 = inp.g_hist.numpy().copy(); g1[70] = 0.0; g1[400] = 0.0
        _with_gates(inp, g1, inp.g_rec.numpy())
    elif pattern == "alternating":
        _with_gates(inp, np.where(t % 2 == 0, 1.0, 0.5), np.where(t % 2 == 0, 0.5, 1.0))
    elif pattern == "swapped":
        _with_gates(inp, inp.g_rec.numpy().copy(), inp.g_hist.numpy().copy())
    elif pattern == "tiny":
        _with_gates(inp, 1e-3, np.where(t % 7 == 0, 0.0, 1e-2))
    st0 = gen.make_states(8301, 1, H, d, d, std=0.3).numpy()
    check_prefill(inp, impl=tc_impl)
    check_prefill(inp, state0=st0, impl=tc_impl)


@pytest.mark.parametrize("gamma", [0.0, 1.0, -0.3, 1.7])
def test_tensor_prefill_gamma_values(gamma, tc_impl):
    inp = gen.make_dense(8400, 1, 300, 2, 128, BF)
    inp.gamma = torch.full((2,), gamma, dtype=torch.float32)
    check_prefill(inp, impl=tc_impl)


def test_tensor_matches_cuda_core_kernel_closely(tc_impl):
    """Both kernels see the same bf16 inputs; they differ only by bf16 operand rounding."""
    from util import gpu_prefill, rel_err
    inp = gen.make_dense(8500, 1, 1000, 4, 128, BF)
    o_t, S_t = gpu_prefill(inp, impl=tc_impl)
    o_s, S_s = gpu_prefill(inp, impl="simt")
    assert rel_err(o_t, o_s) <= 2e-2 and rel_err(S_t, S_s) <= 2e-2

"""Pins of the n-state checker and of the gate producer's checker (CPU only).

n states (Sec. 4.2 discusses why two suffice, Sec. 5.5 runs 1, 2, 4 and 8): every state recurs on itself with
its own gate, the output blends them with one weight per state.  Pinned by the unrolled score form written out
with explicit gate products, by the two-state function (bit for bit) and by a plain single-state loop.
Gate producer (Sec. 5.3, App. B): logistic of a linear layer; pinned by hand values and brute-force loops."""
import math

import numpy as np

from oracle import dsla_oracle as orc


def _rand(seed, T, H, dk, dv, n):
    r = np.random.default_rng(seed)
    q, k = r.normal(size=(T, H, dk)) / np.sqrt(dk), r.normal(size=(T, H, dk)) / np.sqrt(dk)
    v = r.normal(size=(T, H, dv))
    gates = r.uniform(0.3, 1.0, size=(n, T, H))
    w = r.normal(size=(H, n))
    return q, k, v, gates, w


def _unrolled(q, k, v, gates, w, scale=1.0):
    """o_T = scale * sum_t sum_i w_i (q_T . k_t) (prod_{tau = t+1..T} g^i_tau) v_t, by explicit loops."""
    T, H, dk = q.shape
    n = gates.shape[0]
    o = np.zeros((T, H, v.shape[2]))
    for h in range(H):
        for Tt in range(T):
            for t in range(Tt + 1):
                qk = float(q[Tt, h] @ k[t, h])
                for i in range(n):
                    prod = 1.0
                    for tau in range(t + 1, Tt + 1):
                        prod *= gates[i, tau, h]
                    o[Tt, h] += scale * w[h, i] * qk * prod * v[t, h]
    return o


def test_n_states_match_unrolled_score_form():
    for n in (1, 3, 4):
        q, k, v, gates, w = _rand(100 + n, 13, 2, 3, 5, n)
        o, S = orc.prefill_n(q, k, v, gates, w, scale=0.7)
        assert np.allclose(o, _unrolled(q, k, v, gates, w, 0.7), rtol=1e-12, atol=1e-13)
        # final state of every state: sum_t (prod of later gates) k_t^T v_t
        for i in range(n):
            for h in range(2):
                ref = np.zeros((3, 5))
                for t in range(13):
                    ref += np.prod(gates[i, t + 1:, h]) * np.outer(k[t, h], v[t, h])
                assert np.allclose(S[0, i, h], ref, rtol=1e-12, atol=1e-13)


def test_two_states_reproduce_the_dual_state_checker_bit_for_bit():
    q, k, v, gates, _ = _rand(7, 40, 3, 4, 4, 2)
    gamma = np.array([0.3, 1.7, -0.2])
    w = np.stack([gamma, 1.0 - gamma], axis=1)
    o2, S2 = orc.prefill(q, k, v, gates[0], gates[1], gamma, scale=1.0)
    on, Sn = orc.prefill_n(q, k, v, gates, w, scale=1.0)
    assert np.array_equal(S2, Sn)
    # the blend is summed in a different order (q (g S1 + (1-g) S2) vs sum_i q w_i S_i): equal to rounding
    assert np.allclose(o2, on, rtol=1e-13, atol=1e-15)


def test_one_state_is_the_plain_gated_loop():
    q, k, v, gates, w = _rand(9, 25, 2, 4, 6, 1)
    o, S = orc.prefill_n(q, k, v, gates, w)
    for h in range(2):
        St = np.zeros((4, 6))
        for t in range(25):
            St = gates[0, t, h] * St + np.outer(k[t, h], v[t, h])      # Sec. 3: S_t = G_t (.) S_{t-1} + k_t^T v_t
            assert np.allclose(o[t, h], w[h, 0] * (q[t, h] @ St), rtol=1e-12, atol=1e-14)
        assert np.allclose(S[0, 0, h], St, rtol=1e-12)


def test_n_state_per_channel_gates_packing_slots_and_decode():
    r = np.random.default_rng(11)
    T, H, dk, dv, n = 17, 2, 3, 4, 4
    q, k, v, _, w = _rand(12, T, H, dk, dv, n)
    gates = r.uniform(0.2, 1.0, size=(n, T, H, dk))
    cu = np.array([0, 5, 5, 17], dtype=np.int32)
    slots = np.array([2, 0, 1], dtype=np.int32)
    st = r.normal(size=(3, n, H, dk, dv))
    st0 = st.copy()
    o, S = orc.prefill_n(q, k, v, gates, w, cu, state=st, slots=slots)
    # every sequence alone, token by token through decode_step_n, from its own slot
    for s_idx, (a, b) in enumerate(zip(cu[:-1], cu[1:])):
        cur = st0[slots[s_idx]][None].copy()
        for t in range(a, b):
            ot = orc.decode_step_n(q[t:t + 1], k[t:t + 1], v[t:t + 1], gates[:, t:t + 1], w, cur)
            assert np.allclose(ot[0], o[t], rtol=1e-12, atol=1e-14)
        assert np.allclose(cur[0], S[slots[s_idx]], rtol=1e-12, atol=1e-14)
    # brute force for one head of the last sequence, per-channel products
    h, a, b = 1, 5, 17
    for i in range(n):
        ref = np.zeros((dk, dv))
        for c in range(dk):
            ref[c] = st0[1, i, h, c] * np.prod(gates[i, a:b, h, c])
            for t in range(a, b):
                ref[c] += np.prod(gates[i, t + 1:b, h, c]) * k[t, h, c] * v[t, h]
        assert np.allclose(S[1, i, h], ref, rtol=1e-11, atol=1e-13)


def test_gate_project_hand_values_and_brute_force():
    # hand values: logistic(0) = 1/2, logistic(ln 3) = 3/4, logistic(-ln 3) = 1/4
    x = np.array([[0.0, 0.0], [1.0, 0.0], [0.0, 1.0]])
    w = np.array([[math.log(3.0), 0.0], [-math.log(3.0), 2.0]])
    g = orc.gate_project(x, w)
    assert np.allclose(g[0], [0.5, 0.5]) and np.allclose(g[1], [0.75, 0.5]) and np.allclose(g[2, 0], 0.25)
    assert np.isclose(g[2, 1], 1.0 / (1.0 + math.exp(-2.0)))
    # bias shifts the pre-activation; zero bias (the initialisation of App. B) changes nothing
    assert np.allclose(orc.gate_project(x, w, np.zeros(2)), g)
    assert np.isclose(orc.gate_project(x[:1], w, np.array([math.log(3.0), 0.0]))[0, 0], 0.75)
    # brute force
    r = np.random.default_rng(5)
    x, w, b = r.normal(size=(7, 9)), r.normal(size=(9, 4)), r.normal(size=4)
    g = orc.gate_project(x, w, b)
    for t in range(7):
        for j in range(4):
            z = sum(x[t, c] * w[c, j] for c in range(9)) + b[j]
            assert math.isclose(g[t, j], 1.0 / (1.0 + math.exp(-z)), rel_tol=1e-12)
    # logistic(-z) = 1 - logistic(z)
    assert np.allclose(orc.gate_project(-x, w), 1.0 - orc.gate_project(x, w))

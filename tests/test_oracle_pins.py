"""Pins for the fp64 CPU checker: every check here compares it with something that is
not itself -- hand-worked numbers, closed forms, brute-force sums written from the
unrolled score form, textbook special cases.  No GPU needed."""
import os

import numpy as np
import pytest

from oracle import dsla_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rand_case(seed, T, H, dk, dv, lo=0.05, hi=1.0, per_channel=False):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((T, H, dk))
    k = rng.standard_normal((T, H, dk))
    v = rng.standard_normal((T, H, dv))
    gs = (T, H, dk) if per_channel else (T, H)
    g1 = rng.uniform(lo, hi, gs)
    g2 = rng.uniform(lo, hi, gs)
    gam = rng.uniform(-0.3, 1.3, H)
    return q, k, v, g1, g2, gam


# ---------------------------------------------------------------- brute force restatements
def decay_product(g, s, t):
    """prod_{tau=s+1..t} g_tau, written as an explicit loop (empty product = 1)."""
    p = np.ones_like(g[0])
    for tau in range(s + 1, t + 1):
        p = p * g[tau]
    return p


def brute_quadratic(q, k, v, g1, g2, gam, scale=1.0):
    """o_T = sum_{t<=T} (gamma sigma^1_t + (1-gamma) sigma^2_t) v_t with sigma^i_t built from
    (q_T (.) k_t) times the explicit product of gates t+1..T (the unrolled score form)."""
    T, H, dk = q.shape
    dv = v.shape[2]
    o = np.zeros((T, H, dv))
    for h in range(H):
        for tq in range(T):
            for t in range(tq + 1):
                d1 = decay_product(g1[:, h], t, tq)   # scalar or [dk]
                d2 = decay_product(g2[:, h], t, tq)
                s1 = np.sum(q[tq, h] * k[t, h] * d1)
                s2 = np.sum(q[tq, h] * k[t, h] * d2)
                o[tq, h] += (gam[h] * s1 + (1 - gam[h]) * s2) * v[t, h]
    return scale * o


def brute_final_state(k, v, g):
    """S_T = sum_t (prod_{tau>t} g_tau) k_t^T v_t, explicit loops."""
    T, H, dk = k.shape
    dv = v.shape[2]
    S = np.zeros((H, dk, dv))
    for h in range(H):
        for t in range(T):
            d = decay_product(g[:, h], t, T - 1)
            S[h] += np.outer(k[t, h] * d, v[t, h])
    return S


def chunked_restatement(q, k, v, g1, g2, gam, C, S0=None):
    """Chunkwise form derived from the recurrence: within a chunk the masked quadratic form,
    across chunks a decayed carry.  b_j = inclusive cumulative log-gate inside the chunk."""
    T, H, dk = q.shape
    dv = v.shape[2]
    o = np.zeros((T, H, dv))
    S = np.zeros((2, H, dk, dv)) if S0 is None else S0.copy()
    for h in range(H):
        for c0 in range(0, T, C):
            c1 = min(T, c0 + C)
            Q, K, V = q[c0:c1, h], k[c0:c1, h], v[c0:c1, h]
            P = Q @ K.T
            out = np.zeros((c1 - c0, dv))
            for i, (g, w) in enumerate(((g1, gam[h]), (g2, 1 - gam[h]))):
                with np.errstate(divide="ignore"):
                    b = np.cumsum(np.log(g[c0:c1, h]))
                D = np.tril(np.exp(b[:, None] - b[None, :]))
                out += w * ((P * D) @ V + np.exp(b)[:, None] * (Q @ S[i, h]))
                S[i, h] = np.exp(b[-1]) * S[i, h] + (K * np.exp(b[-1] - b)[:, None]).T @ V
            o[c0:c1, h] = out
    return o, S


# ---------------------------------------------------------------- hand-worked numbers
def _rows(path):
    return [list(map(float, l.split())) for l in open(path) if l.strip() and not l.startswith("#")]


def test_hand_example_d1():
    rows = _rows(os.path.join(GOLD, "hand_example_d1.txt"))
    T = len(rows)
    one = np.ones((T, 1, 1))
    for n in range(1, T + 1):
        o, S = orc.prefill(one[:n], one[:n], one[:n], np.full((n, 1), 0.5), np.full((n, 1), 0.25), np.array([0.5]))
        assert o[-1, 0, 0] == rows[n - 1][3]
        assert S[0, 0, 0, 0, 0] == rows[n - 1][1] and S[0, 1, 0, 0, 0] == rows[n - 1][2]


def test_hand_example_d2():
    r = _rows(os.path.join(GOLD, "hand_example_d2.txt"))
    q = np.array([[[1.0, 2.0]], [[1.0, 1.0]]])
    k = np.array([[[1.0, 0.0]], [[0.0, 2.0]]])
    v = np.array([[[2.0, 3.0]], [[1.0, -1.0]]])
    o, S = orc.prefill(q, k, v, np.full((2, 1), 0.5), np.zeros((2, 1)), np.array([0.25]))
    assert o[0, 0].tolist() == r[0] and o[1, 0].tolist() == r[1]
    assert S[0, 0, 0].ravel().tolist() == r[2] and S[0, 1, 0].ravel().tolist() == r[3]
    # asymmetric k, v make a transposed outer product (v^T k) fail here
    assert not np.allclose(S[0, 0, 0], S[0, 0, 0].T)


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("T,H,dk,dv", [(1, 1, 3, 2), (7, 2, 4, 5), (33, 1, 8, 3)])
def test_matches_unrolled_score_form(T, H, dk, dv):
    q, k, v, g1, g2, gam = rand_case(T, T, H, dk, dv)
    o, S = orc.prefill(q, k, v, g1, g2, gam, scale=0.7)
    ref = brute_quadratic(q, k, v, g1, g2, gam, scale=0.7)
    assert np.max(np.abs(o - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    assert np.allclose(S[0, 0], brute_final_state(k, v, g1), rtol=0, atol=1e-12)
    assert np.allclose(S[0, 1], brute_final_state(k, v, g2), rtol=0, atol=1e-12)


def test_per_channel_gates_match_brute_force():
    q, k, v, g1, g2, gam = rand_case(5, 19, 2, 6, 4, per_channel=True)
    o, S = orc.prefill(q, k, v, g1, g2, gam)
    ref = brute_quadratic(q, k, v, g1, g2, gam)
    assert np.max(np.abs(o - ref)) <= 1e-12
    assert np.allclose(S[0, 1], brute_final_state(k, v, g2), rtol=0, atol=1e-12)
    # scalar gates are the per-channel form with a constant vector
    gs1, gs2 = g1[:, :, 0], g2[:, :, 0]
    o_s, _ = orc.prefill(q, k, v, gs1, gs2, gam)
    o_c, _ = orc.prefill(q, k, v, np.repeat(gs1[:, :, None], 6, 2), np.repeat(gs2[:, :, None], 6, 2), gam)
    assert np.array_equal(o_s, o_c)


# ---------------------------------------------------------------- reductions / closed forms
def single_state_gla(q, k, v, g):
    """Single-state gated linear attention (Sec. 3 recurrence), plain numpy, one head."""
    T, dk = q.shape
    S = np.zeros((dk, v.shape[1]))
    o = np.zeros((T, v.shape[1]))
    for t in range(T):
        S = g[t] * S + np.outer(k[t], v[t])
        o[t] = q[t] @ S
    return o, S


def test_gla_reduction():
    q, k, v, g1, g2, gam = rand_case(11, 23, 2, 5, 4)
    for gval, gsel in ((1.0, g1), (0.0, g2)):
        o, S = orc.prefill(q, k, v, g1, g2, np.full(2, gval))
        for h in range(2):
            ro, rS = single_state_gla(q[:, h], k[:, h], v[:, h], gsel[:, h])
            assert np.allclose(o[:, h], ro, rtol=0, atol=1e-12)
    # equal gates: output does not depend on gamma and both states coincide
    oa, Sa = orc.prefill(q, k, v, g1, g1, np.array([0.1, 0.9]))
    ob, Sb = orc.prefill(q, k, v, g1, g1, np.array([1.7, -0.3]))
    assert np.allclose(oa, ob, rtol=0, atol=1e-12) and np.array_equal(Sa[0, 0], Sa[0, 1])


def test_decay_one_is_causal_linear_attention():
    q, k, v, _, _, gam = rand_case(3, 40, 2, 6, 5)
    ones = np.ones((40, 2))
    o, S = orc.prefill(q, k, v, ones, ones, gam)
    kv = np.cumsum(np.einsum("tha,thb->thab", k, v), axis=0)      # running sum of k^T v
    ref = np.einsum("tha,thab->thb", q, kv)
    assert np.allclose(o, ref, rtol=0, atol=1e-11)
    assert np.allclose(S[0, 0], kv[-1], rtol=0, atol=1e-11) and np.allclose(S[0, 1], kv[-1], rtol=0, atol=1e-11)


def test_decay_zero_keeps_only_current_token():
    q, k, v, _, _, gam = rand_case(4, 17, 3, 4, 6)
    z = np.zeros((17, 3))
    S0 = np.random.default_rng(9).standard_normal((1, 2, 3, 4, 6))     # a non-zero start must be wiped too
    o, S = orc.prefill(q, k, v, z, z, gam, state=S0.copy())
    ref = np.einsum("tha,tha->th", q, k)[:, :, None] * v
    assert np.allclose(o, ref, rtol=0, atol=1e-13)
    assert np.allclose(S[0, 0], np.einsum("ha,hb->hab", k[-1], v[-1]), rtol=0, atol=1e-13)


def test_geometric_series_closed_form():
    T, dk, dv = 50, 4, 3
    g1, g2, gam = 0.9, 0.3, 0.35
    e0 = np.zeros((T, 1, dk)); e0[:, 0, 0] = 1.0
    vv = np.tile(np.array([1.0, -2.0, 0.5]), (T, 1, 1))
    o, _ = orc.prefill(e0, e0, vv, np.full((T, 1), g1), np.full((T, 1), g2), np.array([gam]))
    t = np.arange(T)
    coef = gam * (1 - g1 ** (t + 1)) / (1 - g1) + (1 - gam) * (1 - g2 ** (t + 1)) / (1 - g2)
    assert np.allclose(o[:, 0], coef[:, None] * vv[:, 0], rtol=1e-13, atol=0)


def test_mixed_zero_gate_inside_sequence():
    # a single zero gate cuts the history exactly at that token for that state only
    q, k, v, g1, g2, gam = rand_case(6, 20, 1, 4, 4)
    g1[9] = 0.0
    o, S = orc.prefill(q, k, v, g1, g2, np.array([1.0]))
    o_tail, S_tail = orc.prefill(q[9:], k[9:], v[9:], g1[9:], g2[9:], np.array([1.0]))
    assert np.allclose(o[9:], o_tail, rtol=0, atol=1e-13) and np.allclose(S[0, 0], S_tail[0, 0], atol=1e-13)
    assert not np.allclose(S[0, 1], S_tail[0, 1])


# ---------------------------------------------------------------- composition / invariance
def test_composition_prefill_decode():
    T = 29
    q, k, v, g1, g2, gam = rand_case(21, T + 1, 2, 5, 4)
    o_full, S_full = orc.prefill(q, k, v, g1, g2, gam)
    o_a, S_a = orc.prefill(q[:T], k[:T], v[:T], g1[:T], g2[:T], gam)
    o_b = orc.decode_step(q[T:], k[T:], v[T:], g1[T:], g2[T:], gam, S_a)
    assert np.allclose(o_full[:T], o_a, rtol=0, atol=1e-13)
    assert np.allclose(o_full[T:], o_b, rtol=0, atol=1e-13) and np.allclose(S_full, S_a, rtol=0, atol=1e-13)
    # split prefill with carried state, and n decode steps from a state = prefill of n tokens
    o1, S1 = orc.prefill(q[:10], k[:10], v[:10], g1[:10], g2[:10], gam)
    o2, S2 = orc.prefill(q[10:], k[10:], v[10:], g1[10:], g2[10:], gam, state=S1)
    assert np.allclose(np.concatenate([o1, o2]), o_full, rtol=0, atol=1e-13) and np.allclose(S2, S_full, atol=1e-13)
    S = np.zeros_like(S_full)
    outs = [orc.decode_step(q[t:t + 1], k[t:t + 1], v[t:t + 1], g1[t:t + 1], g2[t:t + 1], gam, S) for t in range(T + 1)]
    assert np.allclose(np.concatenate(outs), o_full, rtol=0, atol=1e-13)


@pytest.mark.parametrize("C", [1, 16, 64, 128, 150])
def test_chunk_size_invariance(C):
    T = 150
    q, k, v, g1, g2, gam = rand_case(31, T, 2, 8, 6, lo=0.3)
    o, S = orc.prefill(q, k, v, g1, g2, gam)
    S0 = np.random.default_rng(1).standard_normal((2, 2, 8, 6))
    oc, Sc = chunked_restatement(q, k, v, g1, g2, gam, C)
    assert np.max(np.abs(o - oc)) <= 1e-10 and np.max(np.abs(S[0] - Sc)) <= 1e-10
    o2, S2 = orc.prefill(q, k, v, g1, g2, gam, state=S0[None].copy())
    oc2, Sc2 = chunked_restatement(q, k, v, g1, g2, gam, C, S0)
    assert np.max(np.abs(o2 - oc2)) <= 1e-10 and np.max(np.abs(S2[0] - Sc2)) <= 1e-10


def test_linearity_and_affinity():
    q, k, v, g1, g2, gam = rand_case(41, 25, 2, 4, 4)
    v2 = np.random.default_rng(2).standard_normal(v.shape)
    f = lambda vv, gg=gam, S=None: orc.prefill(q, k, vv, g1, g2, gg, state=None if S is None else S.copy())[0]
    assert np.allclose(f(2.0 * v - 3.0 * v2), 2.0 * f(v) - 3.0 * f(v2), rtol=0, atol=1e-11)
    ga, gb = np.array([0.2, 0.4]), np.array([0.9, -0.5])
    assert np.allclose(f(v, 0.25 * ga + 0.75 * gb), 0.25 * f(v, ga) + 0.75 * f(v, gb), rtol=0, atol=1e-12)
    S0 = np.random.default_rng(3).standard_normal((1, 2, 2, 4, 4))
    zero = np.zeros_like(v)
    # o(v, S0) = o(v, 0) + o(0, S0): linear in the initial state
    assert np.allclose(f(v, gam, S0), f(v) + f(zero, gam, S0), rtol=0, atol=1e-12)


def test_heads_sequences_and_slots_are_independent():
    lens = [5, 1, 0, 12, 7]
    T = sum(lens)
    q, k, v, g1, g2, gam = rand_case(51, T, 3, 4, 5)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    o, S = orc.prefill(q, k, v, g1, g2, gam, cu)
    for n, L in enumerate(lens):
        sl = slice(cu[n], cu[n + 1])
        if L == 0:
            assert not S[n].any()
            continue
        o1, S1 = orc.prefill(q[sl], k[sl], v[sl], g1[sl], g2[sl], gam)
        assert np.array_equal(o[sl], o1) and np.array_equal(S[n], S1[0])
    perm = np.array([2, 0, 1])
    op, Sp = orc.prefill(q[:, perm], k[:, perm], v[:, perm], g1[:, perm], g2[:, perm], gam[perm], cu)
    assert np.array_equal(op, o[:, perm]) and np.array_equal(Sp, S[:, :, perm])
    # slots: permuted placement, an empty sequence leaves its slot untouched, -1 rows are skipped
    slots = np.array([4, 2, 0, 1, 3], dtype=np.int32)
    st = np.full((5, 2, 3, 4, 5), 0.0)
    st[0] = 7.0
    o_s, st = orc.prefill(q, k, v, g1, g2, gam, cu, state=st, slots=slots)
    assert np.all(st[0] == 7.0)                      # empty sequence n=2 -> slot 0 unchanged
    assert np.array_equal(st[4], S[0]) and np.array_equal(st[1], S[3])
    B = 4
    qd, kd, vd, gd1, gd2, _ = rand_case(52, B, 3, 4, 5)
    st2 = np.random.default_rng(5).standard_normal((6, 2, 3, 4, 5))
    keep = st2.copy()
    od = orc.decode_step(qd, kd, vd, gd1, gd2, gam, st2, np.array([5, -1, 0, 3], dtype=np.int32))
    assert not od[1].any() and np.array_equal(st2[[1, 2, 4]], keep[[1, 2, 4]])
    assert not np.array_equal(st2[5], keep[5])


def test_threads_do_not_change_results():
    q, k, v, g1, g2, gam = rand_case(61, 64, 4, 8, 8)
    cu = np.array([0, 10, 40, 64], dtype=np.int32)
    a = orc.prefill(q, k, v, g1, g2, gam, cu, nthreads=1)
    b = orc.prefill(q, k, v, g1, g2, gam, cu, nthreads=7)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])

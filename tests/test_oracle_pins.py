"""Pins for the fp64 oracle: what the paper and the mathematics fix, not the oracle itself.

Each test evaluates a closed form, an invariant, a library routine or an exact
rational brute force that a correct implementation of the gated delta rule
(paper, subsection "Gated Delta Net")

    S_t = S_{t-1} alpha_t (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,   o_t = scale S_t q_t

must satisfy, and compares the oracle against it.  A dropped term, a wrong sign,
a transposed state, a pre- instead of post-update output or a wrong head map
fails at least one of them.  CPU only.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
from scipy.linalg import hadamard

import oracle
from paper_2607_17979_b200 import inputs as I
from chunked_ref import chunked_prefill


# ----------------------------------------------------------------------------- helpers
def q_bf16(x):
    """Quantise fp64 -> bf16; return (bits, exact fp64 values of those bits)."""
    bits = I.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    return bits, I.bf16_bits_to_f64(bits)


def rand_problem(rs, T, Hqk, Hv, dk, dv, alpha_lo=0.5, unit_k=False):
    qb, q = q_bf16(rs.standard_normal((T, Hqk, dk)))
    kk = rs.standard_normal((T, Hqk, dk))
    if unit_k:
        kk /= np.linalg.norm(kk, axis=-1, keepdims=True)
    kb, k = q_bf16(kk)
    vb, v = q_bf16(rs.standard_normal((T, Hv, dv)))
    g = np.log(rs.uniform(alpha_lo, 1.0, (T, Hv))).astype(np.float32)
    beta = rs.uniform(0.0, 1.0, (T, Hv)).astype(np.float32)
    return dict(qb=qb, kb=kb, vb=vb, q=q, k=k, v=v, g=g, beta=beta)


def run_single(p, S0=None, scale=1.0, cu=None):
    T = p["qb"].shape[0]
    cu = np.array([0, T], dtype=np.int32) if cu is None else cu
    return oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu,
                          init_state=S0, scale=scale)[:2]


# ----------------------------------------------------------------------------- closed forms
def test_one_token_closed_form_uses_updated_state():
    # S_0 = 0  =>  S_1 = beta v k^T,  o_1 = scale * beta (k.q) v.   A pre-update output would be 0.
    rs = np.random.default_rng(1)
    p = rand_problem(rs, 1, 1, 1, 5, 3)
    o, S = run_single(p, scale=0.37)
    beta = float(p["beta"][0, 0])
    k, q, v = p["k"][0, 0], p["q"][0, 0], p["v"][0, 0]
    np.testing.assert_allclose(S[0, 0], beta * np.outer(v, k), rtol=1e-14, atol=0)
    np.testing.assert_allclose(o[0, 0], 0.37 * beta * (k @ q) * v, rtol=1e-13, atol=1e-300)
    assert np.abs(o).max() > 0


def test_two_token_closed_form_decay_inside_bracket():
    # S_2 = alpha_2 beta_1 v_1 k_1^T (I - beta_2 k_2 k_2^T) + beta_2 v_2 k_2^T
    rs = np.random.default_rng(2)
    p = rand_problem(rs, 2, 1, 1, 4, 6)
    o, S = run_single(p)
    a2 = math.exp(float(p["g"][1, 0]))
    b1, b2 = float(p["beta"][0, 0]), float(p["beta"][1, 0])
    k1, k2 = p["k"][0, 0], p["k"][1, 0]
    v1, v2 = p["v"][0, 0], p["v"][1, 0]
    S2 = a2 * b1 * np.outer(v1, k1) @ (np.eye(4) - b2 * np.outer(k2, k2)) + b2 * np.outer(v2, k2)
    np.testing.assert_allclose(S[0, 0], S2, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(o[1, 0], S2 @ p["q"][1, 0], rtol=1e-12, atol=1e-15)


def test_rank_one_orientation_dv_rows_dk_columns():
    # v = e_3 (dv index), k = e_5 (dk index): only S[3][5] is non-zero.
    dk, dv = 8, 6
    k = np.zeros((1, 1, dk)); k[0, 0, 5] = 1.0
    v = np.zeros((1, 1, dv)); v[0, 0, 3] = 1.0
    q = np.ones((1, 1, dk))
    g = np.zeros((1, 1), np.float32); beta = np.ones((1, 1), np.float32)
    o, S = oracle.prefill(q_bf16(q)[0], q_bf16(k)[0], q_bf16(v)[0], g, beta,
                          np.array([0, 1], np.int32))[:2]
    expect = np.zeros((dv, dk)); expect[3, 5] = 1.0
    assert np.array_equal(S[0, 0], expect)
    assert np.array_equal(o[0, 0], expect @ np.ones(dk))


def test_beta_zero_is_pure_decay():
    # beta = 0  =>  S_T = exp(sum g) S_0,  o_t = scale exp(sum_{<=t} g) S_0 q_t
    rs = np.random.default_rng(3)
    T, dk, dv = 17, 7, 5
    p = rand_problem(rs, T, 1, 1, dk, dv)
    p["beta"][:] = 0
    S0 = rs.standard_normal((1, 1, dv, dk))
    o, S = run_single(p, S0=S0.copy(), scale=0.5)
    csum = np.cumsum(p["g"][:, 0].astype(np.float64))
    np.testing.assert_allclose(S[0, 0], np.exp(csum[-1]) * S0[0, 0], rtol=1e-13)
    for t in range(T):
        np.testing.assert_allclose(o[t, 0], 0.5 * np.exp(csum[t]) * (S0[0, 0] @ p["q"][t, 0]),
                                   rtol=1e-12, atol=1e-15)


def test_unit_key_beta_one_stores_value_exactly():
    # ||k|| = 1, beta = 1  =>  S_t k_t = v_t for any alpha (to 1e-12).
    # keys +-1/8 on 64 of 128 coordinates are exactly unit-norm in bf16.
    rs = np.random.default_rng(4)
    T, dk, dv = 9, 128, 16
    k = np.zeros((T, 1, dk))
    for t in range(T):
        idx = rs.permutation(dk)[:64]
        k[t, 0, idx] = rs.choice([-0.125, 0.125], 64)
    p = rand_problem(rs, T, 1, 1, dk, dv)
    p["kb"], p["k"] = q_bf16(k)
    assert np.all(np.abs(np.linalg.norm(p["k"], axis=-1) - 1) == 0)
    p["beta"][:] = 1
    S0 = rs.standard_normal((1, 1, dv, dk))
    for t in range(1, T + 1):
        sub = {n: a[:t] for n, a in p.items()}
        _, S = run_single(sub, S0=S0.copy())
        assert np.abs(S[0, 0] @ p["k"][t - 1, 0] - p["v"][t - 1, 0]).max() < 1e-12


def test_general_key_readout_identity():
    # S_t k_t = alpha (1 - beta |k|^2) S_{t-1} k_t + beta |k|^2 v_t   for any k.
    rs = np.random.default_rng(5)
    T, dk, dv = 6, 9, 4
    p = rand_problem(rs, T, 1, 1, dk, dv)
    S0 = rs.standard_normal((1, 1, dv, dk))
    prev = S0[0, 0]
    for t in range(1, T + 1):
        sub = {n: a[:t] for n, a in p.items()}
        _, S = run_single(sub, S0=S0.copy())
        kt, vt = p["k"][t - 1, 0], p["v"][t - 1, 0]
        a = math.exp(float(p["g"][t - 1, 0])); b = float(p["beta"][t - 1, 0]); n2 = kt @ kt
        np.testing.assert_allclose(S[0, 0] @ kt, a * (1 - b * n2) * (prev @ kt) + b * n2 * vt,
                                   rtol=1e-11, atol=1e-13)
        prev = S[0, 0]


def test_orthonormal_keys_reduce_to_linear_attention():
    # alpha = 1, beta = 1, orthonormal keys  =>  S_T = sum_i v_i k_i^T (the plain linear-attention
    # state) and perfect recall S_T k_i = v_i.  Hadamard rows / 8 are exact in bf16.
    dk, dv, T = 64, 10, 64
    H = hadamard(dk).astype(np.float64) / 8.0
    rs = np.random.default_rng(6)
    p = rand_problem(rs, T, 1, 1, dk, dv)
    p["kb"], p["k"] = q_bf16(H[:, None, :])
    p["g"][:] = 0; p["beta"][:] = 1
    o, S = run_single(p)
    lin = np.einsum("tj,tc->jc", p["v"][:, 0], p["k"][:, 0])
    np.testing.assert_allclose(S[0, 0], lin, rtol=0, atol=1e-13)
    np.testing.assert_allclose(S[0, 0] @ p["k"][:, 0].T, p["v"][:, 0].T, atol=1e-13)
    # outputs equal causal linear attention o_t = sum_{i<=t} (k_i.q_t) v_i
    causal = np.tril(p["q"][:, 0] @ p["k"][:, 0].T)
    np.testing.assert_allclose(o[:, 0], causal @ p["v"][:, 0], atol=1e-12)


def test_alpha_one_is_deltanet_literal_matrix_form():
    # g = 0: S_t = S_{t-1}(I - beta k k^T) + beta v k^T, evaluated as explicit matrix products.
    rs = np.random.default_rng(7)
    T, dk, dv = 11, 6, 5
    p = rand_problem(rs, T, 1, 1, dk, dv)
    p["g"][:] = 0
    S0 = rs.standard_normal((1, 1, dv, dk))
    o, S = run_single(p, S0=S0.copy())
    M = S0[0, 0].copy()
    for t in range(T):
        kt, vt, b = p["k"][t, 0], p["v"][t, 0], float(p["beta"][t, 0])
        M = M @ (np.eye(dk) - b * np.outer(kt, kt)) + b * np.outer(vt, kt)
        np.testing.assert_allclose(o[t, 0], M @ p["q"][t, 0], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(S[0, 0], M, rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("d", [2, 3, 4, 128])
def test_literal_bracket_formula(d):
    # S_t = S_{t-1} (alpha (I - beta k k^T)) + beta v k^T with explicit matrices, gates on.
    rs = np.random.default_rng(70 + d)
    T = 5
    p = rand_problem(rs, T, 1, 1, d, d, unit_k=(d == 128))
    S0 = rs.standard_normal((1, 1, d, d))
    _, S = run_single(p, S0=S0.copy())
    M = S0[0, 0].copy()
    for t in range(T):
        kt, vt = p["k"][t, 0], p["v"][t, 0]
        a, b = math.exp(float(p["g"][t, 0])), float(p["beta"][t, 0])
        M = M @ (a * (np.eye(d) - b * np.outer(kt, kt))) + b * np.outer(vt, kt)
    np.testing.assert_allclose(S[0, 0], M, rtol=1e-12, atol=1e-14)


def test_exact_rational_brute_force_tiny():
    # d = 2, T = 3, every input a small dyadic rational; the recurrence is expanded in exact
    # rational arithmetic (alpha_t = the double exp(g_t) taken as an exact rational).
    F = Fraction
    q = [[F(1, 2), F(-3, 4)], [F(5, 8), F(1, 4)], [F(-1, 2), F(1, 1)]]
    k = [[F(3, 4), F(1, 2)], [F(-1, 4), F(7, 8)], [F(1, 2), F(1, 2)]]
    v = [[F(1, 1), F(-2, 1)], [F(3, 2), F(1, 2)], [F(-1, 4), F(3, 1)]]
    g32 = np.array([-0.25, -0.0625, -0.5], np.float32)
    be32 = np.array([0.5, 0.75, 0.25], np.float32)
    S = [[F(1, 4), F(-1, 2)], [F(3, 4), F(1, 8)]]
    scale = F(1, 2)
    outs = []
    for t in range(3):
        a = F(math.exp(float(g32[t]))); b = F(float(be32[t]))
        kt, vt, qt = k[t], v[t], q[t]
        # M = alpha (I - beta k k^T)
        M = [[a * ((1 if r == c else 0) - b * kt[r] * kt[c]) for c in range(2)] for r in range(2)]
        S = [[sum(S[j][r] * M[r][c] for r in range(2)) + b * vt[j] * kt[c] for c in range(2)]
             for j in range(2)]
        outs.append([scale * sum(S[j][c] * qt[c] for c in range(2)) for j in range(2)])
    tof = lambda rows: np.array([[float(x) for x in r] for r in rows])
    S0 = tof([[F(1, 4), F(-1, 2)], [F(3, 4), F(1, 8)]])[None, None]
    o, Sf = oracle.prefill(q_bf16(tof(q)[:, None, :])[0], q_bf16(tof(k)[:, None, :])[0],
                           q_bf16(tof(v)[:, None, :])[0], g32[:, None], be32[:, None],
                           np.array([0, 3], np.int32), init_state=S0, scale=0.5)[:2]
    np.testing.assert_allclose(Sf[0, 0], tof(S), rtol=1e-15, atol=1e-16)
    np.testing.assert_allclose(o[:, 0], tof(outs), rtol=1e-15, atol=1e-16)


# ----------------------------------------------------------------------------- invariants
def test_linearity_in_state_and_values():
    rs = np.random.default_rng(8)
    T, dk, dv = 12, 8, 6
    p = rand_problem(rs, T, 1, 1, dk, dv)
    # values on a coarse dyadic grid so that a*x + c*y stays exactly representable in bf16
    grid = lambda: np.round(rs.uniform(-2, 2, (T, 1, dv)) * 4) / 4
    vx, vy = grid(), grid()
    X0, Y0 = rs.standard_normal((2, 1, 1, dv, dk))
    a, c = 2.0, -0.5
    def run(vv, S0):
        pp = dict(p); pp["vb"], pp["v"] = q_bf16(vv)
        assert np.array_equal(pp["v"], vv)
        return run_single(pp, S0=S0.copy(), scale=0.7)
    ox, Sx = run(vx, X0); oy, Sy = run(vy, Y0); oz, Sz = run(a * vx + c * vy, a * X0 + c * Y0)
    np.testing.assert_allclose(oz, a * ox + c * oy, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(Sz, a * Sx + c * Sy, rtol=1e-11, atol=1e-12)


def test_scale_is_linear_and_scale_one_is_the_papers_formula():
    rs = np.random.default_rng(9)
    p = rand_problem(rs, 7, 1, 1, 8, 8)
    o1, S1 = run_single(p, scale=1.0)
    o2, S2 = run_single(p, scale=0.125)
    assert np.array_equal(S1, S2)
    np.testing.assert_allclose(o2, 0.125 * o1, rtol=1e-15)


def test_rows_of_state_evolve_independently():
    rs = np.random.default_rng(10)
    T, dk, dv = 9, 8, 7
    p = rand_problem(rs, T, 1, 1, dk, dv)
    S0 = rs.standard_normal((1, 1, dv, dk))
    perm = rs.permutation(dv)
    o, S = run_single(p, S0=S0.copy())
    pp = dict(p); pp["vb"] = p["vb"][:, :, perm]
    o2, S2 = run_single(pp, S0=S0[:, :, perm].copy())
    assert np.array_equal(o2, o[:, :, perm])
    assert np.array_equal(S2, S[:, :, perm])


def test_contraction_bound_unit_keys():
    # |k| = 1, beta in [0,1]  =>  |S_t|_F <= alpha_t |S_{t-1}|_F + beta_t |v_t|
    rs = np.random.default_rng(11)
    T, dk, dv = 40, 128, 8
    k = np.zeros((T, 1, dk))
    for t in range(T):
        k[t, 0, rs.permutation(dk)[:64]] = rs.choice([-0.125, 0.125], 64)
    p = rand_problem(rs, T, 1, 1, dk, dv)
    p["kb"], p["k"] = q_bf16(k)
    S0 = rs.standard_normal((1, 1, dv, dk))
    prev = np.linalg.norm(S0)
    for t in range(1, T + 1):
        sub = {n: a[:t] for n, a in p.items()}
        _, S = run_single(sub, S0=S0.copy())
        a, b = math.exp(float(p["g"][t - 1, 0])), float(p["beta"][t - 1, 0])
        cur = np.linalg.norm(S)
        assert cur <= a * prev + b * np.linalg.norm(p["v"][t - 1, 0]) + 1e-12
        prev = cur


# ----------------------------------------------------------------------------- independent derivation
@pytest.mark.parametrize("chunk", [1, 7, 16, 64])
def test_chunked_wy_form_with_library_triangular_solve(chunk):
    rs = np.random.default_rng(12)
    lens = [200, 0, 37, 64]
    T = sum(lens); Hqk, Hv, dk, dv = 2, 4, 16, 12
    p = rand_problem(rs, T, Hqk, Hv, dk, dv, alpha_lo=0.8, unit_k=True)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    S0 = rs.standard_normal((len(lens), Hv, dv, dk))
    o, S, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu,
                             init_state=S0.copy(), scale=0.3)
    o2, S2 = chunked_prefill(p["q"], p["k"], p["v"], p["g"].astype(np.float64),
                             p["beta"].astype(np.float64), cu, S0, 0.3, chunk)
    np.testing.assert_allclose(o, o2, rtol=0, atol=1e-10)
    np.testing.assert_allclose(S, S2, rtol=0, atol=1e-10)
    assert np.array_equal(S[1], S0[1])          # empty sequence: state passes through


# ----------------------------------------------------------------------------- composition, packing, heads, slots
def test_prefill_equals_repeated_decode_and_split_prefill():
    rs = np.random.default_rng(13)
    L, Hqk, Hv, dk, dv = 23, 2, 4, 8, 6
    p = rand_problem(rs, L, Hqk, Hv, dk, dv)
    S0 = rs.standard_normal((1, Hv, dv, dk))
    cu = np.array([0, L], np.int32)
    o, S, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu, S0.copy(), scale=0.4)
    pool = S0.copy()
    for t in range(L):
        ot, _ = oracle.decode(p["qb"][t:t + 1], p["kb"][t:t + 1], p["vb"][t:t + 1],
                              p["g"][t:t + 1], p["beta"][t:t + 1], pool, None, 0.4)
        assert np.array_equal(ot[0], o[t])
    assert np.array_equal(pool, S)
    L1 = 9
    a = {n: x[:L1] for n, x in p.items()}; b = {n: x[L1:] for n, x in p.items()}
    o1, S1, _ = oracle.prefill(a["qb"], a["kb"], a["vb"], a["g"], a["beta"],
                               np.array([0, L1], np.int32), S0.copy(), scale=0.4)
    o2, S2, _ = oracle.prefill(b["qb"], b["kb"], b["vb"], b["g"], b["beta"],
                               np.array([0, L - L1], np.int32), S1, scale=0.4)
    assert np.array_equal(np.concatenate([o1, o2]), o) and np.array_equal(S2, S)


def test_packed_batch_equals_each_sequence_alone():
    rs = np.random.default_rng(14)
    lens = [5, 0, 11, 1]
    T = sum(lens); Hqk, Hv, dk, dv = 1, 2, 8, 8
    p = rand_problem(rs, T, Hqk, Hv, dk, dv)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    S0 = rs.standard_normal((4, Hv, dv, dk))
    o, S, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu, S0.copy())
    for n in range(4):
        sl = slice(cu[n], cu[n + 1])
        on, Sn, _ = oracle.prefill(p["qb"][sl], p["kb"][sl], p["vb"][sl], p["g"][sl], p["beta"][sl],
                                   np.array([0, lens[n]], np.int32), S0[n:n + 1].copy())
        assert np.array_equal(on, o[sl]) and np.array_equal(Sn[0], S[n])


def test_grouped_head_map_consecutive_v_heads_share_a_qk_head():
    rs = np.random.default_rng(15)
    T, Hqk, Hv, dk, dv = 6, 2, 6, 8, 5          # G = 3: v-heads 0,1,2 -> qk 0; 3,4,5 -> qk 1
    p = rand_problem(rs, T, Hqk, Hv, dk, dv)
    for a in ("vb", "g", "beta"):
        p[a][:, :] = p[a][:, :1]                # identical per-v-head inputs
    S0 = np.repeat(rs.standard_normal((1, 1, dv, dk)), Hv, axis=1)
    o, S, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"],
                             np.array([0, T], np.int32), S0.copy())
    for h in (1, 2):
        assert np.array_equal(o[:, h], o[:, 0]) and np.array_equal(S[0, h], S[0, 0])
    for h in (4, 5):
        assert np.array_equal(o[:, h], o[:, 3])
    assert not np.allclose(o[:, 3], o[:, 0])
    # and each v-head equals a single-head run with its own q/k head
    for h in (0, 4):
        oh, Sh, _ = oracle.prefill(p["qb"][:, h // 3:h // 3 + 1], p["kb"][:, h // 3:h // 3 + 1],
                                   p["vb"][:, h:h + 1], p["g"][:, h:h + 1], p["beta"][:, h:h + 1],
                                   np.array([0, T], np.int32), S0[:, h:h + 1].copy())
        assert np.array_equal(oh[:, 0], o[:, h]) and np.array_equal(Sh[0, 0], S[0, h])


def test_decode_slot_semantics_exact():
    rs = np.random.default_rng(16)
    B, Hqk, Hv, d, slots = 5, 1, 2, 8, 9
    p = rand_problem(rs, B, Hqk, Hv, d, d)
    pool0 = rs.standard_normal((slots, Hv, d, d))
    idx = np.array([7, 2, -1, 0, 12], np.int32)          # -1 = padding, 12 = out of range
    pool = pool0.copy()
    o, bad = oracle.decode(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], pool, idx, 0.5)
    assert bad == Hv                              # counted per (entry, v-head) unit
    assert np.array_equal(o[2], np.zeros((Hv, d))) and np.array_equal(o[4], np.zeros((Hv, d)))
    untouched = [s for s in range(slots) if s not in (7, 2, 0)]
    assert np.array_equal(pool[untouched], pool0[untouched])
    for i, s in [(0, 7), (1, 2), (3, 0)]:
        one = pool0[s:s + 1].copy()
        oi, _ = oracle.decode(p["qb"][i:i + 1], p["kb"][i:i + 1], p["vb"][i:i + 1],
                              p["g"][i:i + 1], p["beta"][i:i + 1], one, None, 0.5)
        assert np.array_equal(oi[0], o[i]) and np.array_equal(one[0], pool[s])


def test_prefill_slots_and_alias():
    rs = np.random.default_rng(17)
    lens = [4, 3]; Hqk, Hv, d = 1, 1, 4
    p = rand_problem(rs, 7, Hqk, Hv, d, d)
    cu = np.array([0, 4, 7], np.int32)
    pool0 = rs.standard_normal((5, Hv, d, d))
    idx = np.array([3, 1], np.int32)
    pool = pool0.copy()
    o, S, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu, init_state=pool,
                             slot_idx=idx, final_state=pool)          # aliased in/out
    assert S is pool
    assert np.array_equal(pool[[0, 2, 4]], pool0[[0, 2, 4]])
    o2, S2, _ = oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu,
                               init_state=pool0[[3, 1]].copy())
    assert np.array_equal(o, o2) and np.array_equal(S2[0], pool[3]) and np.array_equal(S2[1], pool[1])


def test_bad_cu_seqlens_rejected():
    rs = np.random.default_rng(18)
    p = rand_problem(rs, 4, 1, 1, 4, 4)
    with pytest.raises(ValueError):
        oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], np.array([0, 3, 2, 4], np.int32))
    with pytest.raises(ValueError):
        oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], np.array([0, 3], np.int32))


def test_thread_count_never_changes_a_bit():
    """Threads only split the independent (sequence, v-head) units among themselves: one thread,
    three threads and the default count must give identical bits for prefill and for decode."""
    rs = np.random.default_rng(19)
    lens = [9, 0, 14, 3, 21]
    T = sum(lens); Hqk, Hv, dk, dv = 2, 6, 8, 5
    p = rand_problem(rs, T, Hqk, Hv, dk, dv)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    S0 = rs.standard_normal((5, Hv, dv, dk))
    runs = [oracle.prefill(p["qb"], p["kb"], p["vb"], p["g"], p["beta"], cu, S0.copy(), scale=0.7,
                           n_threads=n) for n in (1, 3, 0)]
    for o, S, _ in runs[1:]:
        assert np.array_equal(o, runs[0][0]) and np.array_equal(S, runs[0][1])
    B = 7
    d = rand_problem(rs, B, Hqk, Hv, dk, dv)
    pool0 = rs.standard_normal((B, Hv, dv, dk))
    outs = []
    for n in (1, 3, 0):
        pool = pool0.copy()
        o, _ = oracle.decode(d["qb"], d["kb"], d["vb"], d["g"], d["beta"], pool, None, 0.7, n_threads=n)
        outs.append((o, pool))
    for o, pool in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(pool, outs[0][1])

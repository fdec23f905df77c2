"""Pins of the oracle's gate helper (g = -exp(A_log) softplus(a + dt_bias), beta = sigmoid(b)):
closed forms and identities of softplus and the logistic function, and the link to the
recurrence's pure-decay closed form.  CPU only."""
import math

import numpy as np

import oracle
from paper_2607_17979_b200 import inputs as I


def bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, np.float32))


def test_softplus_closed_forms():
    a = bits([[0.0, 0.0, 0.0]])
    # a + dt_bias = 0  ->  softplus = ln 2;  A_log = 0, ln 3, -ln 2
    g, _ = oracle.gate(a, a, [0.0, math.log(3.0), -math.log(2.0)], [0.0, 0.0, 0.0])
    assert np.allclose(g[0], [-math.log(2.0), -3 * math.log(2.0), -0.5 * math.log(2.0)], rtol=1e-15)
    # the bias is added before the softplus: a = 1, bias = -1 is the same zero argument
    g, _ = oracle.gate(bits([[1.0]]), bits([[0.0]]), [0.0], [-1.0])
    assert math.isclose(g[0, 0], -math.log(2.0), rel_tol=1e-15)
    # softplus(x) = ln(1 + e^x) written out, moderate x (bf16-exact values)
    xs = np.array([[-4.0, -1.5, -0.25, 0.5, 2.0, 7.0]], np.float32)
    g, _ = oracle.gate(bits(xs), bits(xs), np.zeros(6), np.zeros(6))
    assert np.allclose(-g, np.log(1.0 + np.exp(xs.astype(np.float64))), rtol=1e-14)


def test_softplus_tails_and_identity():
    xs = np.array([[-64.0, -40.0, 40.0, 64.0]], np.float32)
    g, _ = oracle.gate(bits(xs), bits(xs), np.zeros(4), np.zeros(4))
    sp = -g[0]
    assert sp[0] == math.exp(-64.0) or math.isclose(sp[0], math.exp(-64.0), rel_tol=1e-12)
    assert math.isclose(sp[1], math.exp(-40.0), rel_tol=1e-12)
    assert math.isclose(sp[2], 40.0, rel_tol=1e-15) and math.isclose(sp[3], 64.0, rel_tol=1e-15)
    # softplus(x) - softplus(-x) = x
    x = I.bf16_bits_to_f64(I.gate_inputs(50, 4, seed=3)["a"])
    gp, _ = oracle.gate(bits(x), bits(x), np.zeros(4), np.zeros(4))
    gm, _ = oracle.gate(bits(-x), bits(x), np.zeros(4), np.zeros(4))
    assert np.allclose((-gp) - (-gm), x, rtol=0, atol=1e-14)


def test_gate_is_nonpositive_monotone_and_scaled_by_the_head_rate():
    d = I.gate_inputs(200, 8, seed=5)
    g, beta = oracle.gate(d["a"], d["b"], d["A_log"], d["dt_bias"])
    assert (g < 0).all() and (beta > 0).all() and (beta < 1).all()
    # larger a -> stronger decay (more negative g), per head
    a = I.bf16_bits_to_f64(d["a"])
    for h in range(8):
        order = np.argsort(a[:, h])
        assert (np.diff(g[order, h]) <= 0).all()
    # doubling exp(A_log) doubles g
    g2, _ = oracle.gate(d["a"], d["b"], d["A_log"] + np.float32(math.log(2.0)), d["dt_bias"])
    assert np.allclose(g2, 2 * g, rtol=1e-6)     # A_log is rounded to fp32 before the call


def test_logistic_identities():
    d = I.gate_inputs(100, 4, seed=6)
    b = I.bf16_bits_to_f64(d["b"])
    _, beta = oracle.gate(d["a"], d["b"], d["A_log"], d["dt_bias"])
    _, beta_neg = oracle.gate(d["a"], bits(-b), d["A_log"], d["dt_bias"])
    assert np.allclose(beta + beta_neg, 1.0, rtol=0, atol=1e-15)
    assert np.allclose(np.log(beta / (1 - beta)), b, rtol=0, atol=1e-12)      # logit inverts it
    _, half = oracle.gate(bits([[0.0]]), bits([[0.0]]), [0.0], [0.0])
    assert half[0, 0] == 0.5


def test_gate_output_drives_the_pure_decay_closed_form():
    """With beta forced to 0 the recurrence only decays: S_T = exp(sum g) S_0; the helper's g
    (negative) must give a shrinking state through the oracle's prefill."""
    T, Hv = 9, 2
    d = I.gate_inputs(T, Hv, seed=8)
    g, _ = oracle.gate(d["a"], d["b"], d["A_log"], d["dt_bias"])
    p = I.prefill_inputs([T], 1, Hv, seed=9, init="normal")
    g32 = g.astype(np.float32)
    S0 = p["init_state"].astype(np.float64)
    _, S, _ = oracle.prefill(p["q"], p["k"], p["v"], g32, np.zeros((T, Hv), np.float32),
                             p["cu_seqlens"], S0, None, 1.0)
    decay = np.exp(g32.astype(np.float64).sum(axis=0))
    assert (decay < 1).all()
    assert np.allclose(S[0], decay[:, None, None] * S0[0], rtol=1e-13)

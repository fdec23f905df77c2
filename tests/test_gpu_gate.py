"""GPU parity: gdn_gate against the fp64 oracle, and the helper feeding gdn_prefill."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U

pytestmark = pytest.mark.gpu


def run_gate(d):
    from paper_2607_17979_b200 import api
    T, Hv = d["T"], d["Hv"]
    g = torch.full((T, Hv), float("nan"), device="cuda")
    beta = torch.full((T, Hv), float("nan"), device="cuda")
    api.gdn_gate(U.dev_bf16(d["a"]), U.dev_bf16(d["b"]), U.dev(d["A_log"]), U.dev(d["dt_bias"]), g, beta)
    torch.cuda.synchronize()
    return g, beta


@pytest.mark.parametrize("T,Hv", [(1, 1), (7, 3), (1000, 32), (8192, 32)])
def test_gate_matches_oracle(T, Hv):
    d = I.gate_inputs(T, Hv, seed=40 + T)
    g, beta = run_gate(d)
    g_ref, beta_ref = oracle.gate(d["a"], d["b"], d["A_log"], d["dt_bias"])
    # fp32 exp/log1p: a few ulps
    assert np.abs(g.cpu().numpy() / g_ref - 1).max() < 2e-6
    assert np.abs(beta.cpu().numpy() / beta_ref - 1).max() < 1e-6


def test_gate_extreme_arguments_stay_finite():
    d = I.gate_inputs(4, 2, seed=1)
    d["a"] = I.f32_to_bf16_bits(np.array([[-200.0, 200.0], [-30.0, 30.0], [0.0, 0.0], [88.0, -88.0]], np.float32))
    d["b"] = d["a"].copy()
    g, beta = run_gate(d)
    g_ref, beta_ref = oracle.gate(d["a"], d["b"], d["A_log"], d["dt_bias"])
    gh, bh = g.cpu().numpy().astype(np.float64), beta.cpu().numpy().astype(np.float64)
    assert np.isfinite(gh).all() and np.isfinite(bh).all() and (gh <= 0).all()
    assert np.allclose(gh, g_ref, rtol=1e-5, atol=1e-30)
    assert np.allclose(bh, beta_ref, rtol=1e-5, atol=1e-30)


def test_gate_output_feeds_prefill():
    from paper_2607_17979_b200 import api
    p = I.prefill_inputs([150, 90], 2, 4, seed=60, init="normal")
    T, N = p["T"], p["N"]
    d = I.gate_inputs(T, 4, seed=61)
    d["A_log"] = (d["A_log"] - 3.0).astype(np.float32)        # mild decay: alpha around 0.9
    g, beta = run_gate(d)
    o = torch.empty((T, 4, 128), dtype=torch.bfloat16, device="cuda")
    final = torch.empty((N, 4, 128, 128), dtype=torch.float32, device="cuda")
    ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, 2, 4), dtype=torch.uint8, device="cuda")
    api.gdn_prefill(U.dev_bf16(p["q"]), U.dev_bf16(p["k"]), U.dev_bf16(p["v"]), g, beta,
                    U.dev(p["cu_seqlens"]), U.dev(p["init_state"]), final, None, o, p["scale"], ws)
    torch.cuda.synchronize()
    # the oracle takes the SAME fp32 g, beta the device produced (the helper's own parity is above)
    o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], g.cpu().numpy(), beta.cpu().numpy(),
                                     p["cu_seqlens"], p["init_state"].astype(np.float64), None, p["scale"])
    U.check_o(U.host_f64_from_bf16(o), o_ref, U.O_REL_L2_PREFILL)
    U.check_state(final.cpu().numpy().astype(np.float64), S_ref, U.STATE_REL_L2_PREFILL)

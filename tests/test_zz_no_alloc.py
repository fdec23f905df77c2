"""gdn_prefill_static, the prefill entry point for callers that may not allocate device memory
(they cannot hand gdn_prefill a workspace of their own), against gdn_prefill on the same inputs.

The scratch array inside the library is shared by every call and keeps the previous call's
contents, so the check runs two calls in a row, the second on a smaller and differently shaped
batch, and each must reproduce gdn_prefill's result exactly (same kernels, same arithmetic order).
Collected last on purpose (file name), so an -x run has already exercised everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U

pytestmark = pytest.mark.gpu


def _run(p, static):
    from paper_2607_17979_b200 import api
    N, Hv, T = p["N"], p["Hv"], p["T"]
    final = torch.full((N, Hv, 128, 128), float("nan"), dtype=torch.float32, device="cuda")
    o = torch.full((T, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (U.dev_bf16(p["q"]), U.dev_bf16(p["k"]), U.dev_bf16(p["v"]), U.dev(p["g"]),
            U.dev(p["beta"]), U.dev(p["cu_seqlens"]), U.dev(p["init_state"]), final, None, o,
            p["scale"])
    if static:
        api.gdn_prefill_static(*args, dev_status=status)
    else:
        ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, p["Hqk"], Hv), dtype=torch.uint8,
                         device="cuda")
        api.gdn_prefill(*args, ws, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return U.host_f64_from_bf16(o), final.cpu().numpy()


def test_static_workspace_entry_point_matches_gdn_prefill_on_two_calls_in_a_row():
    from paper_2607_17979_b200 import api
    assert api.gdn_prefill_static_workspace_bytes() == 32 << 20
    first = I.prefill_inputs([200, 64, 0, 129], 2, 4, seed=4100, init="normal")
    second = I.prefill_inputs([70, 33], 1, 2, seed=4101, init="zero")      # fewer, other shapes
    for p in (first, second):
        assert api.gdn_prefill_workspace_bytes(p["T"], p["N"], p["Hqk"], p["Hv"]) <= 32 << 20
        o_s, S_s = _run(p, static=True)
        o_r, S_r = _run(p, static=False)
        assert np.abs(o_s - o_r).max() <= U.O_MAX_ABS and U.rel_l2(o_s, o_r) <= U.O_REL_L2_PREFILL
        assert U.rel_l2(S_s.astype(np.float64), S_r.astype(np.float64)) <= U.STATE_REL_L2_PREFILL
        assert np.array_equal(o_s, o_r) and np.array_equal(S_s, S_r)
        # and against the fp64 oracle, like every other entry point
        o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], p["g"], p["beta"], p["cu_seqlens"],
                                         None if p["init_state"] is None
                                         else p["init_state"].astype(np.float64), None, p["scale"])
        U.check_o(o_s, o_ref, U.O_REL_L2_PREFILL)
        U.check_state(S_s.astype(np.float64), S_ref, U.STATE_REL_L2_PREFILL)


def test_static_workspace_entry_point_at_the_edge_of_its_array():
    """With 32 v-heads and two sequences: the largest batch whose scratch still fits the array runs
    and reproduces gdn_prefill; one more chunk is refused with GDN_ERR_LIMIT and writes nothing."""
    from paper_2607_17979_b200 import api
    limit = api.gdn_prefill_static_workspace_bytes()
    chunks = 1
    while api.gdn_prefill_workspace_bytes(64 * (chunks + 1), 2, 16, 32) <= limit:
        chunks += 1
    T_fit = 64 * chunks                       # floor(T/64) + N = chunks + 2 chunk slots
    assert api.gdn_prefill_workspace_bytes(T_fit, 2, 16, 32) <= limit
    assert api.gdn_prefill_workspace_bytes(T_fit + 64, 2, 16, 32) > limit
    assert chunks + 2 == api.STATIC_MAX_CHUNK_SLOTS_HV32      # the figure the header states
    fit = I.prefill_inputs([T_fit - 100, 100], 16, 32, seed=4103, init="normal")
    o_s, S_s = _run(fit, static=True)
    o_r, S_r = _run(fit, static=False)
    assert np.array_equal(o_s, o_r) and np.array_equal(S_s, S_r)
    over = I.prefill_inputs([T_fit - 100 + 64, 100], 16, 32, seed=4104, init="zero")
    final = torch.zeros((2, 32, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.zeros((over["T"], 32, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.GdnError) as e:
        api.gdn_prefill_static(U.dev_bf16(over["q"]), U.dev_bf16(over["k"]), U.dev_bf16(over["v"]),
                               U.dev(over["g"]), U.dev(over["beta"]), U.dev(over["cu_seqlens"]), None,
                               final, None, o, over["scale"])
    assert e.value.code == -7
    torch.cuda.synchronize()
    assert float(final.abs().max()) == 0 and float(o.float().abs().max()) == 0


def test_static_workspace_entry_point_rejects_batches_beyond_its_array():
    from paper_2607_17979_b200 import api
    p = I.prefill_inputs([64] * 20, 16, 32, seed=4102, init="zero")       # 40 chunk slots x 32 heads
    assert api.gdn_prefill_workspace_bytes(p["T"], p["N"], 16, 32) > 32 << 20
    final = torch.zeros((20, 32, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.zeros((p["T"], 32, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(api.GdnError) as e:
        api.gdn_prefill_static(U.dev_bf16(p["q"]), U.dev_bf16(p["k"]), U.dev_bf16(p["v"]),
                               U.dev(p["g"]), U.dev(p["beta"]), U.dev(p["cu_seqlens"]), None, final,
                               None, o, p["scale"])
    assert e.value.code == -7
    torch.cuda.synchronize()
    assert float(final.abs().max()) == 0 and float(o.float().abs().max()) == 0

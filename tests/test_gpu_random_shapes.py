"""GPU parity on randomly drawn shapes: many small trials per route, each against the fp64 oracle.

The fixed cases of the other files pin the shapes one can think of; this file draws the ones one
does not: head counts and groupings, batch sizes, ragged lengths around the chunk size (with empty
sequences), initial states or none, slot tables with padding entries and spare slots, wide and
narrow gate ranges.  Every trial is seeded, so a failure names its recipe.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U
from test_gpu_prefill import run_prefill, oracle_prefill

pytestmark = pytest.mark.gpu

PREFILL_ROUTES = ["auto", "stream", "fused", "overlap", "recurrent"]
TRIALS = 12


def _draw_prefill(rs, route):
    Hqk = int(rs.choice([1, 2, 4, 8, 16]))
    Hv = Hqk * int(rs.choice([1, 2, 4])) if Hqk <= 8 else Hqk * int(rs.choice([1, 2]))
    N = int(rs.integers(1, 7))
    top = 40 if route == "recurrent" else 330
    lens = []
    for _ in range(N):
        kind = rs.integers(0, 5)
        if kind == 0:
            lens.append(0)
        elif kind == 1:
            lens.append(64 * int(rs.integers(1, 5)))               # whole chunks
        elif kind == 2:
            lens.append(64 * int(rs.integers(1, 5)) + int(rs.choice([-1, 1])))
        else:
            lens.append(int(rs.integers(1, top)))
    if route == "recurrent":
        lens = [min(x, top) for x in lens]
    if sum(lens) == 0:
        lens[0] = 70 if route != "recurrent" else 9
    return Hqk, Hv, lens


@pytest.mark.parametrize("route", PREFILL_ROUTES)
@pytest.mark.parametrize("trial", range(TRIALS))
def test_prefill_random_shapes(route, trial):
    seed = 7000 + 100 * PREFILL_ROUTES.index(route) + trial
    rs = np.random.default_rng(seed)
    Hqk, Hv, lens = _draw_prefill(rs, route)
    init = "normal" if rs.integers(0, 3) else "zero"
    alpha_lo = float(rs.choice([0.5, 0.9, 0.99]))
    p = I.prefill_inputs(lens, Hqk, Hv, seed=seed, alpha_lo=alpha_lo, init=init)
    N = p["N"]
    use_slots = bool(rs.integers(0, 2))
    if use_slots:
        num_slots = N + int(rs.integers(0, 4))
        idx = rs.permutation(num_slots)[:N].astype(np.int32)
        pad = rs.random(N) < 0.2
        idx[pad] = -1
        pool = (rs.standard_normal((num_slots, Hv, 128, 128)) * 0.02).astype(np.float32)
        o, S, status = run_prefill(p, route, slot_idx=idx, num_slots=num_slots, init=pool, alias=True)
        o_ref, S_ref, bad = oracle_prefill(p, slot_idx=idx, num_slots=num_slots, init=pool)
        assert status == 0 and bad == 0, (seed, lens, idx)
        live = [int(s) for s in idx if s >= 0]
        untouched = [s for s in range(num_slots) if s not in live]
        assert np.array_equal(S[untouched], pool[untouched]), (seed, lens, idx)
        cu = p["cu_seqlens"]
        for n in range(N):
            if idx[n] < 0 and cu[n + 1] > cu[n]:
                assert np.abs(o[cu[n]:cu[n + 1]]).max() == 0, (seed, lens, idx)
        S, S_ref = S[live], S_ref[live]
    else:
        o, S, status = run_prefill(p, route)
        o_ref, S_ref, _ = oracle_prefill(p)
        assert status == 0, (seed, lens)
    assert np.isfinite(o).all() and np.isfinite(S).all(), (seed, lens)
    if p["T"] > 0 and np.abs(o_ref).max() > 0:
        err = np.abs(o - o_ref).max()
        assert err <= U.O_MAX_ABS, (seed, lens, err)
        assert U.rel_l2(o, o_ref) <= 2 * U.O_REL_L2_PREFILL, (seed, lens, U.rel_l2(o, o_ref))
    if S.size:
        assert U.rel_l2(S.astype(np.float64), S_ref) <= U.STATE_REL_L2_PREFILL, (seed, lens)


@pytest.mark.parametrize("trial", range(TRIALS))
def test_decode_random_shapes(trial):
    from paper_2607_17979_b200 import api
    seed = 7900 + trial
    rs = np.random.default_rng(seed)
    Hqk = int(rs.choice([1, 2, 4, 8, 16]))
    Hv = Hqk * int(rs.choice([1, 2, 4])) if Hqk <= 8 else Hqk * int(rs.choice([1, 2]))
    B = int(rs.integers(1, 40))
    num_slots = B + int(rs.integers(0, 9))
    d = I.decode_inputs(B, Hqk, Hv, 128, num_slots, seed=seed, slots="perm" if num_slots > B else "identity",
                        alpha_lo=float(rs.choice([0.5, 0.9, 0.99])))
    idx = np.arange(B, dtype=np.int32) if d["slot_idx"] is None else d["slot_idx"].copy()
    idx[rs.random(B) < 0.15] = -1
    pool = U.dev(d["state"])
    o = torch.full((B, Hv, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.gdn_decode(U.dev_bf16(d["q"]), U.dev_bf16(d["k"]), U.dev_bf16(d["v"]), U.dev(d["g"]), U.dev(d["beta"]),
                   pool, U.dev(idx), o, d["scale"], dev_status=status)
    torch.cuda.synchronize()
    S_ref = d["state"].astype(np.float64)
    o_ref, bad = oracle.decode(d["q"], d["k"], d["v"], d["g"], d["beta"], S_ref, idx, d["scale"])
    assert int(status.item()) == 0 and bad == 0
    o_gpu = U.host_f64_from_bf16(o)
    S_gpu = pool.cpu().numpy()
    live = [int(s) for s in idx if s >= 0]
    untouched = [s for s in range(num_slots) if s not in live]
    assert np.array_equal(S_gpu[untouched], d["state"][untouched]), (seed, idx)
    assert np.abs(o_gpu[idx < 0]).max(initial=0.0) == 0
    if live:
        U.check_o(o_gpu[idx >= 0], o_ref[idx >= 0], U.O_REL_L2_DECODE)
        U.check_state(S_gpu[live].astype(np.float64), S_ref[live], U.STATE_REL_L2_DECODE)

"""GPU parity on randomly drawn small batches: every prefill route (three launches, fused,
persistent state pass, token by token, and the length-routed entry point) against the fp64 oracle,
with random head groupings, slot permutations, padding slots, empty sequences and gate ranges."""
import numpy as np
import pytest

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U
from test_gpu_prefill import run_prefill

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(12))
def test_random_batch_all_routes(seed):
    rng = np.random.default_rng(9000 + seed)
    N = int(rng.integers(1, 14))
    longest = [40, 200, 700][seed % 3]
    lens = [int(x) for x in rng.integers(0, longest, size=N)]
    if sum(lens) == 0:
        lens[0] = 5
    Hqk = int(rng.choice([1, 2, 4]))
    Hv = Hqk * int(rng.choice([1, 2, 4]))
    p = I.prefill_inputs(lens, Hqk, Hv, seed=int(rng.integers(1, 1 << 30)), init="normal",
                         alpha_lo=float(rng.choice([0.5, 0.9, 0.99])))
    num_slots = N + int(rng.integers(0, 3))
    slots = rng.permutation(num_slots)[:N].astype(np.int32)
    if seed % 2:
        slots[int(rng.integers(0, N))] = -1
    init = np.zeros((num_slots, Hv, 128, 128), np.float32)
    for n in range(N):
        if slots[n] >= 0:
            init[slots[n]] = p["init_state"][n]
    o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], p["g"], p["beta"], p["cu_seqlens"],
                                     init.astype(np.float64), slots, p["scale"], num_slots=num_slots)
    keep = slots[slots >= 0]
    for impl in ("chunked", "fused", "stream", "recurrent", "auto"):
        o, S, status = run_prefill(p, impl, slot_idx=slots, num_slots=num_slots, init=init,
                                   pool_fill=0.0)
        assert status == 0, impl
        U.check_o(o, o_ref, U.O_REL_L2_PREFILL)
        if len(keep):
            U.check_state(S[keep].astype(np.float64), S_ref[keep], U.STATE_REL_L2_PREFILL)

"""GPU parity of gdn_prefill_overlap (the intra-chunk work in two parts around the state pass).
Its state pass waits for records of a later launch, so these tests run after every other
prefill test: the generic prefill cases once more through this entry point, then its own."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U
import test_gpu_prefill as P
from test_gpu_prefill import run_prefill, oracle_prefill

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("L", [1, 2, 63, 64, 65, 127, 128, 129, 200])
def test_single_sequence_lengths(L):
    P.test_single_sequence_lengths("overlap", L)


@pytest.mark.parametrize("Hqk,Hv", [(1, 1), (1, 2), (2, 4), (4, 8), (16, 32)])
def test_packed_ragged_batch_with_empty_sequence(Hqk, Hv):
    P.test_packed_ragged_batch_with_empty_sequence("overlap", Hqk, Hv)


def test_slots_padding_alias_and_untouched_slots():
    P.test_slots_padding_alias_and_untouched_slots("overlap")


@pytest.mark.parametrize("case", ["beta0", "beta1", "g0", "alpha09", "v0", "same_keys"])
def test_degenerate_values(case):
    P.test_degenerate_values("overlap", case)


def test_bad_cu_seqlens_sets_status_and_skips():
    P.test_bad_cu_seqlens_sets_status_and_skips("overlap")


def test_deterministic_and_split_prefill_hand_off():
    P.test_deterministic_and_split_prefill_hand_off("overlap")


def test_batches_that_are_all_padding_or_all_empty():
    P.test_batches_that_are_all_padding_or_all_empty("overlap")


def test_repeatable_under_load_many_ctas():
    P.test_chunked_repeatable_under_load_many_ctas("overlap")


def test_many_short_sequences_far_more_units_than_sms():
    P.test_many_short_sequences_stream_across_unit_boundaries("overlap")


@pytest.mark.parametrize("config", [3, 4])
def test_benchmark_prefill_configs(config):
    """The varlen batch and the 32768-token sequence in full, every v-head against the oracle."""
    p = I.make_config(config, 1)
    o_ref, S_ref, _ = oracle_prefill(p)
    if config == 3:
        o, S, status = run_prefill(p, "overlap")
        assert status == 0
        U.check_o(o, o_ref, U.O_REL_L2_PREFILL)
        U.check_state(S.astype(np.float64), S_ref, U.STATE_REL_L2_PREFILL)
        return
    P.check_long_context(p, o_ref, S_ref, "overlap")


@pytest.mark.parametrize("split", [-1, 0, 150, 400, 1000])
def test_two_part_production_at_any_cut(split):
    """gdn_prefill_overlap produces the records before the cut ahead of the state pass and the
    others beside it, behind flags: every cut (none, some, all of the items up front, or the
    library's own choice) must give the oracle's result, with sequences of very unequal length,
    an empty one, a padding slot and a ragged tail in the batch."""
    lens = [1500, 64, 0, 333, 700, 1]
    p = I.prefill_inputs(lens, 2, 4, seed=77, init="normal")
    num_slots = 8
    slots = np.array([5, 0, 3, -1, 7, 2], np.int32)
    init = np.zeros((num_slots, 4, 128, 128), np.float32)
    for n in range(len(lens)):
        if slots[n] >= 0:
            init[slots[n]] = p["init_state"][n]
    o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], p["g"], p["beta"], p["cu_seqlens"],
                                     init.astype(np.float64), slots, p["scale"], num_slots=num_slots)
    o, S, status = run_prefill(p, "overlap", slot_idx=slots, num_slots=num_slots, init=init,
                               pool_fill=0.0, split_permille=split)
    assert status == 0
    U.check_o(o, o_ref, U.O_REL_L2_PREFILL)
    keep = slots[slots >= 0]
    U.check_state(S[keep].astype(np.float64), S_ref[keep], U.STATE_REL_L2_PREFILL)
    untouched = [s for s in range(num_slots) if s not in keep]
    assert np.array_equal(S[untouched], init[untouched])


def test_two_part_production_matches_the_three_launches_bit_for_bit():
    """Same kernels' arithmetic in another schedule: on the varlen benchmark shape the overlapped
    route and the persistent state pass must agree exactly, whatever the cut."""
    p = I.prefill_inputs([512, 1024, 2048, 4096], 16, 32, seed=5, init="zero")
    o_s, S_s, st_s = run_prefill(p, "stream", init=None)
    for split in (-1, 300):
        o_o, S_o, st_o = run_prefill(p, "overlap", init=None, split_permille=split)
        assert st_s == 0 and st_o == 0
        assert np.array_equal(o_s, o_o) and np.array_equal(S_s, S_o)


def test_two_part_production_replayed_from_a_cuda_graph():
    """The four launches are programmatic dependents of one another and the last does not wait for
    the one before it; captured into a CUDA graph and replayed they must still give the eager
    result (the flags and the queue are cleared by the first launch of every call)."""
    from paper_2607_17979_b200 import api
    p = I.prefill_inputs([2600, 700, 65], 2, 4, seed=9, init="zero")
    T, N = p["T"], p["N"]
    ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, 2, 4), dtype=torch.uint8, device="cuda")
    args = (U.dev_bf16(p["q"]), U.dev_bf16(p["k"]), U.dev_bf16(p["v"]), U.dev(p["g"]),
            U.dev(p["beta"]), U.dev(p["cu_seqlens"]))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def outs():
        return (torch.zeros((N, 4, 128, 128), dtype=torch.float32, device="cuda"),
                torch.zeros((T, 4, 128), dtype=torch.bfloat16, device="cuda"))

    f0, o0 = outs()
    api.gdn_prefill(*args, None, f0, None, o0, p["scale"], ws, route="overlap", split_permille=300,
                    dev_status=status)
    torch.cuda.synchronize()
    f1, o1 = outs()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(2):
                api.gdn_prefill(*args, None, f1, None, o1, p["scale"], ws, route="overlap",
                                split_permille=300, dev_status=status)
    for _ in range(3):
        f1.zero_()
        o1.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(f0, f1) and torch.equal(o0, o1)
    assert int(status.item()) == 0
    o_ref, S_ref, _ = oracle_prefill(p, init=None)
    U.check_o(U.host_f64_from_bf16(o1), o_ref, U.O_REL_L2_PREFILL)
    U.check_state(f1.cpu().numpy().astype(np.float64), S_ref, U.STATE_REL_L2_PREFILL)



@pytest.mark.parametrize("lens,slots", [([1500, 64, 0, 333, 700, 1], [5, 0, 3, -1, 7, 2]),
                                        ([1309, 1478, 993, 1452], [0, 1, 2, 3]),
                                        ([1849, 67, 1043, 2012, 1319, 475, 1702], [7, 0, 5, 6, 4, 2, 3])])
def test_serialised_launches_cost_time_not_results(lens, slots):
    """split_permille = -2 launches the producers of the second part as an ordinary successor of
    the state pass, which is what a tool that serialises launches would do: the state pass's waits
    for their records run out (soon, and without an error), it marks what it finished, and the
    last launch runs the other units once the records exist.  Same results, status clean."""
    p = I.prefill_inputs(lens, 2, 4, seed=78, init="normal")
    num_slots = 8
    slots = np.array(slots, np.int32)
    init = np.zeros((num_slots, 4, 128, 128), np.float32)
    for n in range(len(lens)):
        if slots[n] >= 0:
            init[slots[n]] = p["init_state"][n]
    o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], p["g"], p["beta"], p["cu_seqlens"],
                                     init.astype(np.float64), slots, p["scale"], num_slots=num_slots)
    o_par, S_par, st_par = run_prefill(p, "overlap", slot_idx=slots, num_slots=num_slots, init=init,
                                       pool_fill=0.0, split_permille=-1)
    for alias in (False, True):
        kw = dict(alias=True) if alias else dict(pool_fill=0.0)
        o, S, status = run_prefill(p, "overlap", slot_idx=slots, num_slots=num_slots, init=init.copy(),
                                   split_permille=-2, **kw)
        assert status == 0 and st_par == 0
        assert np.array_equal(o, o_par)
        keep = slots[slots >= 0]
        assert np.array_equal(S[keep], S_par[keep])
        U.check_o(o, o_ref, U.O_REL_L2_PREFILL)
        U.check_state(S[keep].astype(np.float64), S_ref[keep], U.STATE_REL_L2_PREFILL)


def test_host_buffer_prefill_behind_the_two_part_route():
    """gdn_prefill_host on a batch that gdn_prefill sends to the two-part production: the copy of o
    back to the host follows the last launch.  Five calls in a row, each compared bit for bit with
    the device entry point."""
    from paper_2607_17979_b200 import api
    lens = [2700, 2600]
    p = I.prefill_inputs(lens, 16, 32, seed=21, init="zero")
    T, N = p["T"], p["N"]
    assert api.gdn_prefill_route(T, N, max(lens), 32) == "overlap"
    ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, 16, 32), dtype=torch.uint8, device="cuda")
    o_dev, S_dev, st = run_prefill(p, "overlap", init=None)
    assert st == 0
    host = {n: U.dev_bf16(p[n]).cpu().pin_memory() for n in ("q", "k", "v")}
    host.update({n: torch.from_numpy(p[n]).pin_memory() for n in ("g", "beta", "cu_seqlens")})
    stage = torch.empty(api.gdn_prefill_host_staging_bytes(T, N, 16, 32), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(5):
        h_o = torch.zeros((T, 32, 128), dtype=torch.bfloat16).pin_memory()
        final = torch.zeros((N, 32, 128, 128), dtype=torch.float32, device="cuda")
        api.gdn_prefill_host(host["q"], host["k"], host["v"], host["g"], host["beta"],
                             host["cu_seqlens"], None, final, None, h_o, p["scale"], stage, ws,
                             max_seqlen_hint=max(lens), dev_status=status)
        torch.cuda.synchronize()
        assert np.array_equal(U.host_f64_from_bf16(h_o), o_dev)
        assert np.array_equal(final.cpu().numpy(), S_dev)
    assert int(status.item()) == 0

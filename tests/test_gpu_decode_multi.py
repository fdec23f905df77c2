"""GPU parity: gdn_decode_multi (L new tokens per sequence, either state orientation) against
the fp64 oracle applied token by token."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_17979_b200 import inputs as I
import gpu_util as U

pytestmark = pytest.mark.gpu

VK, KV = 0, 1


def run_multi(d, layout, slot_idx="from_inputs"):
    from paper_2607_17979_b200 import api
    slot = d["slot_idx"] if isinstance(slot_idx, str) else slot_idx
    state = d["state"] if layout == VK else np.ascontiguousarray(d["state"].transpose(0, 1, 3, 2))
    pool = U.dev(state)
    o = torch.full((d["B"], d["L"], d["Hv"], 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.gdn_decode_multi(U.dev_bf16(d["q"]), U.dev_bf16(d["k"]), U.dev_bf16(d["v"]), U.dev(d["g"]),
                         U.dev(d["beta"]), pool, U.dev(slot), o, d["scale"], layout, status)
    torch.cuda.synchronize()
    got = pool.cpu().numpy()
    if layout == KV:
        got = np.ascontiguousarray(got.transpose(0, 1, 3, 2))
    return U.host_f64_from_bf16(o), got, int(status.item())


def oracle_multi(d, slot_idx="from_inputs"):
    """L successive one-token oracle steps on an fp64 pool (tiles [dv][dk])."""
    slot = d["slot_idx"] if isinstance(slot_idx, str) else slot_idx
    pool = d["state"].astype(np.float64)
    o = np.zeros((d["B"], d["L"], d["Hv"], 128))
    bad = 0
    for t in range(d["L"]):
        c = lambda a: np.ascontiguousarray(a[:, t])
        o[:, t], bad = oracle.decode(c(d["q"]), c(d["k"]), c(d["v"]), c(d["g"]), c(d["beta"]),
                                     pool, slot, d["scale"])
    return o, pool, bad


@pytest.mark.parametrize("layout", [VK, KV])
@pytest.mark.parametrize("B,L,Hqk,Hv,slots", [(1, 1, 1, 1, 1), (2, 2, 1, 2, 3), (3, 5, 2, 4, 5),
                                              (7, 8, 4, 8, 7), (5, 16, 2, 4, 9), (80, 3, 2, 4, 96),
                                              (12, 4, 16, 32, 12)])
def test_decode_multi_matches_token_by_token_oracle(layout, B, L, Hqk, Hv, slots):
    d = I.decode_multi_inputs(B, L, Hqk, Hv, 128, slots, seed=300 + B + L,
                              slots="perm" if slots > B else "identity")
    o, pool, status = run_multi(d, layout)
    o_ref, pool_ref, _ = oracle_multi(d)
    assert status == 0
    U.check_o(o, o_ref, U.O_REL_L2_DECODE)
    touched = np.arange(B) if d["slot_idx"] is None else d["slot_idx"]
    U.check_state(pool[touched].astype(np.float64), pool_ref[touched], U.STATE_REL_L2_DECODE)
    assert U.rel_l2(pool[touched].astype(np.float64), pool_ref[touched]) < 1e-5
    untouched = np.setdiff1d(np.arange(slots), touched)
    assert np.array_equal(pool[untouched], d["state"][untouched])


@pytest.mark.parametrize("layout", [VK, KV])
def test_decode_multi_with_one_token_tracks_gdn_decode(layout):
    """L = 1 is the one-token kernel's result up to the order of the fp32 sums."""
    from paper_2607_17979_b200 import api
    for B in (3, 40):
        d = I.decode_multi_inputs(B, 1, 2, 4, 128, B, seed=321)
        o, pool, _ = run_multi(d, layout)
        pool1 = U.dev(d["state"])
        o1 = torch.empty((B, 4, 128), dtype=torch.bfloat16, device="cuda")
        api.gdn_decode(U.dev_bf16(d["q"][:, 0]), U.dev_bf16(d["k"][:, 0]), U.dev_bf16(d["v"][:, 0]),
                       U.dev(d["g"][:, 0]), U.dev(d["beta"][:, 0]), pool1, None, o1, d["scale"])
        torch.cuda.synchronize()
        assert U.rel_l2(pool.astype(np.float64), pool1.cpu().numpy().astype(np.float64)) < 1e-6
        assert U.rel_l2(o[:, 0], U.host_f64_from_bf16(o1)) < 2e-3   # a few bf16 ulps flip


@pytest.mark.parametrize("layout", [VK, KV])
def test_decode_multi_padding_and_out_of_range_slots(layout):
    d = I.decode_multi_inputs(6, 3, 2, 4, 128, 8, seed=7)
    idx = np.array([5, -1, 0, 9, 3, -7], np.int32)
    o, pool, status = run_multi(d, layout, idx)
    o_ref, pool_ref, _ = oracle_multi(d, idx)
    assert status == 1
    assert np.array_equal(o[[1, 3, 5]], np.zeros((3, 3, 4, 128)))
    U.check_o(o, o_ref, U.O_REL_L2_DECODE)
    assert np.array_equal(pool[[1, 2, 4, 6, 7]], d["state"][[1, 2, 4, 6, 7]])
    U.check_state(pool[[5, 0, 3]].astype(np.float64), pool_ref[[5, 0, 3]], U.STATE_REL_L2_DECODE)


@pytest.mark.parametrize("layout", [VK, KV])
def test_decode_multi_equals_prefill_oracle_on_equal_length_sequences(layout):
    """The same call seen as a packed prefill of B sequences of L tokens each (the oracle's
    prefill keeps fp64 across the tokens, the decode oracle too: they must agree, and the GPU
    with both)."""
    d = I.decode_multi_inputs(4, 6, 2, 4, 128, 4, seed=55)
    B, L = 4, 6
    flat = lambda a: np.ascontiguousarray(a.reshape((B * L,) + a.shape[2:]))
    cu = np.arange(B + 1, dtype=np.int32) * L
    o_p, S_p, _ = oracle.prefill(flat(d["q"]), flat(d["k"]), flat(d["v"]), flat(d["g"]),
                                 flat(d["beta"]), cu, d["state"].astype(np.float64), None,
                                 d["scale"])
    o_ref, pool_ref, _ = oracle_multi(d)
    assert np.allclose(o_p.reshape(o_ref.shape), o_ref, rtol=0, atol=1e-12)
    assert np.allclose(S_p, pool_ref, rtol=0, atol=1e-12)
    o, pool, _ = run_multi(d, layout)
    U.check_o(o, o_ref, U.O_REL_L2_DECODE)
    U.check_state(pool.astype(np.float64), pool_ref, U.STATE_REL_L2_DECODE)


def test_decode_multi_full_size_batch():
    """B = 64, Hv = 32 (the benchmark's decode shape) with 4 tokens per sequence, both
    orientations, every tile against the oracle."""
    d = I.decode_multi_inputs(64, 4, 16, 32, 128, 64, seed=I.config_seed(1, 0))
    o_ref, pool_ref, _ = oracle_multi(d)
    for layout in (VK, KV):
        o, pool, status = run_multi(d, layout)
        assert status == 0
        U.check_o(o, o_ref, U.O_REL_L2_DECODE)
        U.check_state(pool.astype(np.float64), pool_ref, U.STATE_REL_L2_DECODE)


def test_decode_multi_rejects_bad_arguments():
    from paper_2607_17979_b200 import api
    d = I.decode_multi_inputs(2, 17, 1, 2, 128, 2, seed=1)
    args = lambda: (U.dev_bf16(d["q"]), U.dev_bf16(d["k"]), U.dev_bf16(d["v"]), U.dev(d["g"]),
                    U.dev(d["beta"]), U.dev(d["state"]), None,
                    torch.empty((2, 17, 2, 128), dtype=torch.bfloat16, device="cuda"), d["scale"])
    with pytest.raises(api.GdnError) as e:
        api.gdn_decode_multi(*args())
    assert e.value.code == -7
    d = I.decode_multi_inputs(2, 2, 1, 2, 128, 2, seed=1)
    with pytest.raises(api.GdnError) as e:
        api.gdn_decode_multi(U.dev_bf16(d["q"]), U.dev_bf16(d["k"]), U.dev_bf16(d["v"]),
                             U.dev(d["g"]), U.dev(d["beta"]), U.dev(d["state"]), None,
                             torch.empty((2, 2, 2, 128), dtype=torch.bfloat16, device="cuda"),
                             d["scale"], 2)
    assert e.value.code == -3


def test_state_transpose_in_place_and_prefill_into_a_transposed_pool():
    """gdn_state_transpose is bit-exact, skips unlisted slots, and brackets gdn_prefill so that a
    pool kept as [dk][dv] tiles can be prefilled and then decoded in that orientation."""
    from paper_2607_17979_b200 import api
    rng = np.random.default_rng(5)
    pool_h = rng.standard_normal((6, 4, 128, 128)).astype(np.float32)
    pool = U.dev(pool_h)
    idx = np.array([4, -1, 1, 7], np.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    api.gdn_state_transpose(pool, U.dev(idx), dev_status=status)
    torch.cuda.synchronize()
    want = pool_h.copy()
    want[[4, 1]] = pool_h[[4, 1]].transpose(0, 1, 3, 2)
    assert np.array_equal(pool.cpu().numpy(), want) and int(status.item()) == 1
    api.gdn_state_transpose(pool)            # every slot
    torch.cuda.synchronize()
    want = want.transpose(0, 1, 3, 2)
    assert np.array_equal(pool.cpu().numpy(), want)

    # prefill into a [dk][dv] pool, then one multi-token decode in that orientation
    p = I.prefill_inputs([70, 130], 2, 4, seed=91, init="normal")
    T, N = p["T"], p["N"]
    kv_pool = U.dev(np.ascontiguousarray(p["init_state"].transpose(0, 1, 3, 2)))
    o = torch.empty((T, 4, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, 2, 4), dtype=torch.uint8, device="cuda")
    api.gdn_state_transpose(kv_pool)
    api.gdn_prefill(U.dev_bf16(p["q"]), U.dev_bf16(p["k"]), U.dev_bf16(p["v"]), U.dev(p["g"]),
                    U.dev(p["beta"]), U.dev(p["cu_seqlens"]), kv_pool, kv_pool, None, o, p["scale"], ws)
    api.gdn_state_transpose(kv_pool)
    d = I.decode_multi_inputs(N, 3, 2, 4, 128, N, seed=92)
    o2 = torch.empty((N, 3, 4, 128), dtype=torch.bfloat16, device="cuda")
    api.gdn_decode_multi(U.dev_bf16(d["q"]), U.dev_bf16(d["k"]), U.dev_bf16(d["v"]), U.dev(d["g"]),
                         U.dev(d["beta"]), kv_pool, None, o2, d["scale"], KV)
    torch.cuda.synchronize()
    o_ref, S_ref, _ = oracle.prefill(p["q"], p["k"], p["v"], p["g"], p["beta"], p["cu_seqlens"],
                                     p["init_state"].astype(np.float64), None, p["scale"])
    U.check_o(U.host_f64_from_bf16(o), o_ref, U.O_REL_L2_PREFILL)
    d["state"] = S_ref
    o2_ref, S2_ref, _ = oracle_multi(d)
    U.check_o(U.host_f64_from_bf16(o2), o2_ref, U.O_REL_L2_PREFILL)
    got = kv_pool.cpu().numpy().transpose(0, 1, 3, 2).astype(np.float64)
    U.check_state(got, S2_ref, U.STATE_REL_L2_PREFILL)

"""The seeded input generator: layout, value recipe, and its bf16 rounding against torch's."""
import numpy as np
import torch

from paper_2607_17979_b200 import inputs as I


def test_bf16_rounding_matches_library_conversion():
    rs = np.random.default_rng(0)
    x = np.concatenate([rs.standard_normal(20000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.001953125, 1.005859375, 3.4e38,
                                  1e-40, -2.5], np.float32)])
    mine = I.f32_to_bf16_bits(x)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, lib)
    back = I.bf16_bits_to_f32(mine)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_decode_inputs_recipe_and_determinism():
    a = I.decode_inputs(8, 2, 4, 128, num_slots=16, seed=5, slots="perm")
    b = I.decode_inputs(8, 2, 4, 128, num_slots=16, seed=5, slots="perm")
    for n in ("q", "k", "v", "g", "beta", "state", "slot_idx"):
        assert np.array_equal(a[n], b[n])
    assert a["q"].dtype == np.uint16 and a["q"].shape == (8, 2, 128)
    assert a["v"].shape == (8, 4, 128) and a["state"].shape == (16, 4, 128, 128)
    assert a["state"].dtype == np.float32 and a["g"].dtype == np.float32
    for n in ("q", "k"):
        nrm = np.linalg.norm(I.bf16_bits_to_f64(a[n]), axis=-1)
        assert np.abs(nrm - 1).max() < 4e-3
    alpha = np.exp(a["g"].astype(np.float64))
    assert alpha.min() >= 0.9 - 1e-6 and alpha.max() < 1.0
    assert a["beta"].min() > 0 and a["beta"].max() < 1
    assert abs(a["state"].std() - 0.02) < 5e-4
    assert sorted(a["slot_idx"].tolist()) == sorted(set(a["slot_idx"].tolist()))
    assert a["slot_idx"].dtype == np.int32 and a["slot_idx"].max() < 16
    c = I.decode_inputs(8, 2, 4, 128, num_slots=16, seed=6, slots="perm")
    assert not np.array_equal(a["q"], c["q"])
    assert abs(a["scale"] - 1 / np.sqrt(128)) < 1e-8


def test_prefill_inputs_layout():
    p = I.prefill_inputs([5, 0, 70], 2, 4, 128, seed=3, init="normal")
    assert p["cu_seqlens"].tolist() == [0, 5, 5, 75] and p["cu_seqlens"].dtype == np.int32
    assert p["q"].shape == (75, 2, 128) and p["v"].shape == (75, 4, 128)
    assert p["g"].shape == (75, 4) and p["init_state"].shape == (3, 4, 128, 128)
    assert I.prefill_inputs([4], 1, 1, init="zero")["init_state"] is None


def test_config_table_matches_the_five_benchmark_configurations():
    kinds = [c["kind"] for c in I.CONFIGS]
    assert kinds == ["decode"] * 3 + ["prefill"] * 2
    assert I.CONFIGS[3]["seq_lens"] == [512, 1024, 2048, 4096] and sum(I.CONFIGS[3]["seq_lens"]) == 7680
    assert I.CONFIGS[4]["seq_lens"] == [32768] and I.CONFIGS[4]["alpha_lo"] == 0.95
    c0 = I.make_config(0)
    assert c0["state"].shape == (1, 8, 128, 128) and c0["q"].shape == (1, 4, 128)

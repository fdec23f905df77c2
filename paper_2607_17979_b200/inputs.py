"""Seeded synthetic inputs for the gated-delta-rule decode and prefill paths.

This module only draws numbers and lays them out; it holds none of the
operator's arithmetic.  Both the CPU oracle's tests and the CUDA library's
tests and benchmark take their inputs from here, so the two see identical
bytes.  Every tensor comes from numpy's counter-based Philox generator keyed by
(seed, tensor tag), so a tensor's values do not depend on which other tensors
were drawn before it.

Value recipe (the five benchmark configurations):
  q, k   N(0,1) per element in fp64, L2-normalised per (token, head) vector in
         fp64, rounded fp64 -> fp32 -> bf16 (round to nearest even)
  v      N(0,1) -> bf16
  g      log(alpha), alpha ~ U[alpha_lo, 1), stored fp32, per (token, v-head)
  beta   sigmoid(N(0,1)), stored fp32, per (token, v-head)
  state  N(0, std 0.02) fp32, or zeros
  scale  1/sqrt(dk) as fp32
bf16 tensors are returned as uint16 bit patterns.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 20260717

_TAGS = {"q": 1, "k": 2, "v": 3, "alpha": 4, "beta": 5, "state": 6, "slots": 7,
         "gate_a": 8, "gate_b": 9, "A_log": 10, "dt_bias": 11}


def rng(seed: int, tag: str) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed) & (2**64 - 1), _TAGS[tag]]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


def _unit_vectors_bf16(gen: np.random.Generator, shape) -> np.ndarray:
    x = gen.standard_normal(shape, dtype=np.float64)
    x /= np.linalg.norm(x, axis=-1, keepdims=True)
    return f32_to_bf16_bits(x.astype(np.float32))


def _normal_bf16(gen: np.random.Generator, shape) -> np.ndarray:
    # drawn in blocks so very large tensors do not need an fp64 temporary of full size
    return f32_to_bf16_bits(gen.standard_normal(shape, dtype=np.float32))


def _gates(seed: int, shape, alpha_lo: float):
    alpha = rng(seed, "alpha").uniform(alpha_lo, 1.0, size=shape)
    g = np.log(alpha).astype(np.float32)
    z = rng(seed, "beta").standard_normal(shape, dtype=np.float64)
    beta = (1.0 / (1.0 + np.exp(-z))).astype(np.float32)
    return g, beta


def _state(seed: int, shape, kind: str) -> np.ndarray:
    if kind == "zero":
        return np.zeros(shape, dtype=np.float32)
    gen = rng(seed, "state")
    out = np.empty(shape, dtype=np.float32)
    flat = out.reshape(-1)
    step = 1 << 24
    for s in range(0, flat.size, step):
        e = min(flat.size, s + step)
        flat[s:e] = gen.standard_normal(e - s, dtype=np.float32) * np.float32(0.02)
    return out


def decode_inputs(B: int, Hqk: int, Hv: int, d: int = 128, num_slots: int | None = None,
                  seed: int = BASE_SEED, alpha_lo: float = 0.9, slots: str = "identity",
                  state: str = "normal") -> dict:
    """One decode step's inputs.

    slots: "identity" (slot_idx None, slot i = sequence i) or "perm" (the first B
    entries of a seeded permutation of range(num_slots), int32).
    """
    num_slots = B if num_slots is None else num_slots
    q = _unit_vectors_bf16(rng(seed, "q"), (B, Hqk, d))
    k = _unit_vectors_bf16(rng(seed, "k"), (B, Hqk, d))
    v = _normal_bf16(rng(seed, "v"), (B, Hv, d))
    g, beta = _gates(seed, (B, Hv), alpha_lo)
    pool = _state(seed, (num_slots, Hv, d, d), state)
    slot_idx = None
    if slots == "perm":
        slot_idx = rng(seed, "slots").permutation(num_slots)[:B].astype(np.int32)
    elif slots != "identity":
        raise ValueError(slots)
    return dict(q=q, k=k, v=v, g=g, beta=beta, state=pool, slot_idx=slot_idx,
                scale=float(np.float32(1.0 / np.sqrt(d))),
                B=B, Hqk=Hqk, Hv=Hv, dk=d, dv=d, num_slots=num_slots)


def decode_multi_inputs(B: int, L: int, Hqk: int, Hv: int, d: int = 128,
                        num_slots: int | None = None, seed: int = BASE_SEED,
                        alpha_lo: float = 0.9, slots: str = "identity",
                        state: str = "normal") -> dict:
    """Inputs of one multi-token decode call: L new tokens for each of B sequences
    (q, k [B, L, Hqk, d]; v [B, L, Hv, d]; g, beta [B, L, Hv]); pool and slots as in
    decode_inputs.  ``state`` holds tiles [dv][dk]."""
    num_slots = B if num_slots is None else num_slots
    q = _unit_vectors_bf16(rng(seed, "q"), (B, L, Hqk, d))
    k = _unit_vectors_bf16(rng(seed, "k"), (B, L, Hqk, d))
    v = _normal_bf16(rng(seed, "v"), (B, L, Hv, d))
    g, beta = _gates(seed, (B, L, Hv), alpha_lo)
    pool = _state(seed, (num_slots, Hv, d, d), state)
    slot_idx = None
    if slots == "perm":
        slot_idx = rng(seed, "slots").permutation(num_slots)[:B].astype(np.int32)
    elif slots != "identity":
        raise ValueError(slots)
    return dict(q=q, k=k, v=v, g=g, beta=beta, state=pool, slot_idx=slot_idx,
                scale=float(np.float32(1.0 / np.sqrt(d))),
                B=B, L=L, Hqk=Hqk, Hv=Hv, dk=d, dv=d, num_slots=num_slots)


def gate_inputs(T: int, Hv: int, seed: int = BASE_SEED) -> dict:
    """Raw inputs of the gate helper: a, b ~ N(0,1) as bf16 bits [T, Hv]; A_log = ln U[1,16) and
    dt_bias ~ N(0,1), fp32 [Hv]."""
    a = _normal_bf16(rng(seed, "gate_a"), (T, Hv))
    b = _normal_bf16(rng(seed, "gate_b"), (T, Hv))
    A_log = np.log(rng(seed, "A_log").uniform(1.0, 16.0, size=Hv)).astype(np.float32)
    dt_bias = rng(seed, "dt_bias").standard_normal(Hv).astype(np.float32)
    return dict(a=a, b=b, A_log=A_log, dt_bias=dt_bias, T=T, Hv=Hv)


def prefill_inputs(seq_lens, Hqk: int, Hv: int, d: int = 128, seed: int = BASE_SEED,
                   alpha_lo: float = 0.9, init: str = "zero") -> dict:
    """A packed variable-length prefill batch.

    init: "zero" (init_state None) or "normal" (N(0, 0.02) fp32 per sequence).
    """
    seq_lens = [int(x) for x in seq_lens]
    N = len(seq_lens)
    cu = np.zeros(N + 1, dtype=np.int32)
    cu[1:] = np.cumsum(seq_lens)
    T = int(cu[-1])
    q = _unit_vectors_bf16(rng(seed, "q"), (T, Hqk, d))
    k = _unit_vectors_bf16(rng(seed, "k"), (T, Hqk, d))
    v = _normal_bf16(rng(seed, "v"), (T, Hv, d))
    g, beta = _gates(seed, (T, Hv), alpha_lo)
    init_state = None if init == "zero" else _state(seed, (N, Hv, d, d), "normal")
    return dict(q=q, k=k, v=v, g=g, beta=beta, cu_seqlens=cu, init_state=init_state,
                scale=float(np.float32(1.0 / np.sqrt(d))),
                T=T, N=N, Hqk=Hqk, Hv=Hv, dk=d, dv=d, seq_lens=seq_lens)


# The five benchmark configurations (index = configuration number).
CONFIGS = [
    dict(kind="decode", name="decode_B1", B=1, Hqk=4, Hv=8, num_slots=1, slots="identity",
         alpha_lo=0.9),
    dict(kind="decode", name="decode_B64", B=64, Hqk=16, Hv=32, num_slots=64, slots="identity",
         alpha_lo=0.9),
    dict(kind="decode", name="decode_B256_of_512", B=256, Hqk=16, Hv=32, num_slots=512,
         slots="perm", alpha_lo=0.9),
    dict(kind="prefill", name="prefill_varlen_7680", seq_lens=[512, 1024, 2048, 4096], Hqk=16,
         Hv=32, alpha_lo=0.9, init="zero"),
    dict(kind="prefill", name="prefill_long_32768", seq_lens=[32768], Hqk=16, Hv=32,
         alpha_lo=0.95, init="normal"),
]


def config_seed(config: int, trial: int = 0) -> int:
    return BASE_SEED + 1000 * config + trial


def make_config(config: int, trial: int = 0) -> dict:
    c = CONFIGS[config]
    seed = config_seed(config, trial)
    if c["kind"] == "decode":
        return decode_inputs(c["B"], c["Hqk"], c["Hv"], 128, c["num_slots"], seed,
                             c["alpha_lo"], c["slots"])
    return prefill_inputs(c["seq_lens"], c["Hqk"], c["Hv"], 128, seed, c["alpha_lo"], c["init"])

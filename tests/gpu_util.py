"""Helpers for the GPU parity tests: move generator output to the device, call the C-ABI
binding, run the fp64 oracle on the same bytes, and compute the error metrics."""
import numpy as np
import torch

import oracle
from paper_2607_17979_b200 import inputs as I

# Acceptance bounds.  The first of each pair is the stated gate; the relative bound beside it
# is there because |o| is ~1e-2 on these inputs, so an absolute 2e-2 alone would pass o = 0.
O_MAX_ABS = 2e-2
O_REL_L2_DECODE = 5e-3
O_REL_L2_PREFILL = 1e-2
STATE_REL_L2_DECODE = 1e-3
STATE_REL_L2_PREFILL = 5e-3


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def host_f64_from_bf16(t):
    return I.bf16_bits_to_f64(t.detach().cpu().view(torch.int16).numpy().view(np.uint16))


def dev(x, dtype=None):
    if x is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    return t if dtype is None else t.to(dtype)


def rel_l2(a, b):
    den = np.linalg.norm(b.ravel())
    num = np.linalg.norm((a - b).ravel())
    return num / den if den > 0 else num


def worst_tile_rel_l2(a, b):
    """a, b: [..., dv, dk]; worst relative Frobenius error over the leading tiles."""
    d = np.linalg.norm((a - b).reshape(-1, a.shape[-2] * a.shape[-1]), axis=1)
    n = np.linalg.norm(b.reshape(-1, a.shape[-2] * a.shape[-1]), axis=1)
    ok = n > 0
    return float(np.max(d[ok] / n[ok])) if ok.any() else float(d.max(initial=0.0))


def check_o(o_gpu, o_ref, rel_bound):
    err = np.abs(o_gpu - o_ref).max(initial=0.0)
    rel = rel_l2(o_gpu, o_ref)
    assert err <= O_MAX_ABS, f"o max-abs {err:.3e}"
    assert rel <= rel_bound, f"o rel-L2 {rel:.3e}"
    nr, ng = np.linalg.norm(o_ref), np.linalg.norm(o_gpu)
    assert abs(ng - nr) <= 0.01 * nr + 1e-12, f"|o| {ng:.4e} vs {nr:.4e}"
    return err, rel


def check_state(S_gpu, S_ref, bound):
    rel = rel_l2(S_gpu, S_ref)
    worst = worst_tile_rel_l2(S_gpu, S_ref)
    assert rel <= bound, f"state rel-L2 {rel:.3e}"
    assert worst <= 2 * bound, f"worst tile rel-L2 {worst:.3e}"
    return rel, worst

"""Thin binding over the C-ABI library (``include/gdn.h``): argument marshalling only.

Every function takes torch CUDA tensors, checks dtype / contiguity / device,
and passes raw device pointers and the current CUDA stream to the entry point
of the same name.  Nothing is computed here, and there is no fallback: if the
compiled library is missing the import fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgdn_b200.so")

EXPORTS = ("gdn_decode", "gdn_prefill_workspace_bytes", "gdn_prefill", "gdn_prefill_chunked",
           "gdn_prefill_fused", "gdn_prefill_stream", "gdn_prefill_overlap", "gdn_prefill_route", "gdn_decode_multi", "gdn_gate",
           "gdn_state_transpose", "gdn_decode_host", "gdn_decode_host_staging_bytes",
           "gdn_prefill_host", "gdn_prefill_host_staging_bytes",
           "gdn_prefill_recurrent",
           "gdn_prefill_static", "gdn_prefill_static_workspace_bytes",
           "gdn_host_us_per_decode_call", "gdn_host_us_per_prefill_call", "gdn_status_string",
           "gdn_last_cuda_error_string", "gdn_version")

# kernels one call enqueues (for the benchmark's launch count)
LAUNCHES_PER_DECODE = 1
LAUNCHES_PER_PREFILL = 3
LAUNCHES_PER_STEP = LAUNCHES_PER_DECODE + LAUNCHES_PER_PREFILL

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2607_17979_b200.build` "
        "(nvcc, sm_100a). There is no CPU or PyTorch fallback for the gated delta rule kernels.")

_lib = ctypes.CDLL(LIB_PATH)
_P, _I, _F, _Z = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float, ctypes.c_size_t
_lib.gdn_decode.restype = ctypes.c_int
_lib.gdn_decode.argtypes = [_P] * 8 + [_I] * 6 + [_F, _P, _P]
_lib.gdn_prefill_workspace_bytes.restype = _Z
_lib.gdn_decode_multi.restype = ctypes.c_int
_lib.gdn_decode_multi.argtypes = [_P] * 8 + [_I] * 7 + [_F, _I, _P, _P]
_lib.gdn_gate.restype = ctypes.c_int
_lib.gdn_gate.argtypes = [_P] * 6 + [_I, _I, _P]
_lib.gdn_state_transpose.restype = ctypes.c_int
_lib.gdn_state_transpose.argtypes = [_P, _P] + [_I] * 5 + [_P, _P]
_lib.gdn_prefill_workspace_bytes.argtypes = [_I] * 7
_lib.gdn_prefill.restype = ctypes.c_int
_lib.gdn_prefill.argtypes = [_P] * 10 + [_I] * 9 + [_F, _P, _Z, _P, _P]
_lib.gdn_prefill_chunked.restype = ctypes.c_int
_lib.gdn_prefill_chunked.argtypes = _lib.gdn_prefill.argtypes
_lib.gdn_prefill_fused.restype = ctypes.c_int
_lib.gdn_prefill_fused.argtypes = _lib.gdn_prefill.argtypes
_lib.gdn_prefill_route.restype = ctypes.c_int
_lib.gdn_prefill_route.argtypes = [_I] * 6
_lib.gdn_prefill_stream.restype = ctypes.c_int
_lib.gdn_prefill_stream.argtypes = _lib.gdn_prefill.argtypes
_lib.gdn_prefill_overlap.restype = ctypes.c_int
_lib.gdn_prefill_overlap.argtypes = _lib.gdn_prefill.argtypes + [_I]
_lib.gdn_prefill_recurrent.restype = ctypes.c_int
_lib.gdn_prefill_recurrent.argtypes = [_P] * 10 + [_I] * 7 + [_F, _P, _P]
_lib.gdn_prefill_static.restype = ctypes.c_int
_lib.gdn_prefill_static.argtypes = [_P] * 10 + [_I] * 9 + [_F, _P, _P]
_lib.gdn_prefill_static_workspace_bytes.restype = _Z
_lib.gdn_prefill_static_workspace_bytes.argtypes = []
_lib.gdn_decode_host_staging_bytes.restype = _Z
_lib.gdn_decode_host_staging_bytes.argtypes = [_I] * 3
_lib.gdn_decode_host.restype = ctypes.c_int
_lib.gdn_decode_host.argtypes = [_P] * 8 + [_I] * 6 + [_F, _P, _Z, _P, _P]
_lib.gdn_prefill_host_staging_bytes.restype = _Z
_lib.gdn_prefill_host_staging_bytes.argtypes = [_I] * 4
_lib.gdn_prefill_host.restype = ctypes.c_int
_lib.gdn_prefill_host.argtypes = [_P] * 10 + [_I] * 9 + [_F, _P, _Z, _P, _Z, _P, _P]
_lib.gdn_host_us_per_decode_call.restype = ctypes.c_double
_lib.gdn_host_us_per_decode_call.argtypes = [_P] * 8 + [_I] * 6 + [_F, _P, _I]
_lib.gdn_host_us_per_prefill_call.restype = ctypes.c_double
_lib.gdn_host_us_per_prefill_call.argtypes = [_P] * 10 + [_I] * 9 + [_F, _P, _Z, _P, _I]
_lib.gdn_status_string.restype = ctypes.c_char_p
_lib.gdn_status_string.argtypes = [ctypes.c_int]
_lib.gdn_last_cuda_error_string.restype = ctypes.c_char_p
_lib.gdn_version.restype = ctypes.c_int


class GdnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = f" [{_lib.gdn_last_cuda_error_string().decode()}]" if code == -6 else ""
        super().__init__(f"{where}: {status_string(code)} ({code}){detail}")


def status_string(code: int) -> str:
    return _lib.gdn_status_string(int(code)).decode()


def version() -> int:
    return int(_lib.gdn_version())


def _dev(t, dtype, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise TypeError(f"{name} is required")
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def gdn_decode(q, k, v, g, beta, state_pool, slot_idx, o, scale, dev_status=None):
    """One decode step, state_pool updated in place, o written.  Shapes as in gdn.h."""
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    rc = _lib.gdn_decode(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(state_pool, torch.float32, "state_pool"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        B, Hqk, Hv, dk, dv, state_pool.shape[0], float(scale),
        _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_decode")


DECODE_MAX_TOKENS = 16
STATE_VK, STATE_KV = 0, 1


def gdn_decode_multi(q, k, v, g, beta, state_pool, slot_idx, o, scale, state_layout=STATE_VK,
                     dev_status=None):
    """L new tokens per sequence in one call (q [B,L,Hqk,128], v/o [B,L,Hv,128], g/beta [B,L,Hv]);
    ``state_layout`` STATE_VK = tiles [dv][dk], STATE_KV = tiles [dk][dv]."""
    B, L, Hqk, dk = q.shape
    _, _, Hv, dv = v.shape
    rc = _lib.gdn_decode_multi(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(state_pool, torch.float32, "state_pool"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        B, L, Hqk, Hv, dk, dv, state_pool.shape[0], float(scale), int(state_layout),
        _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_decode_multi")


def gdn_gate(a, b, A_log, dt_bias, g, beta):
    """g = -exp(A_log) * softplus(a + dt_bias), beta = sigmoid(b); a, b bf16 [T, Hv]."""
    T, Hv = a.shape
    rc = _lib.gdn_gate(_dev(a, torch.bfloat16, "a"), _dev(b, torch.bfloat16, "b"),
                       _dev(A_log, torch.float32, "A_log"), _dev(dt_bias, torch.float32, "dt_bias"),
                       _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"), T, Hv,
                       _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_gate")


def gdn_state_transpose(state_pool, slot_idx=None, n=None, dev_status=None):
    """Transpose in place the tiles of ``n`` entries (default: every slot) of a
    [num_slots, Hv, 128, 128] fp32 CUDA pool."""
    num_slots, Hv, dv, dk = state_pool.shape
    if n is None:
        n = slot_idx.shape[0] if slot_idx is not None else num_slots
    rc = _lib.gdn_state_transpose(
        _dev(state_pool, torch.float32, "state_pool"), _dev(slot_idx, torch.int32, "slot_idx", True),
        int(n), Hv, dk, dv, num_slots, _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_state_transpose")


ROUTES = {0: "none", 1: "recurrent", 2: "chunked", 3: "fused", 4: "stream", 5: "overlap"}


def gdn_prefill_route(T, N, max_seqlen_hint, Hv, sm_count=148, cooperative_launch=True) -> str:
    """Which route gdn_prefill takes for a batch of this shape on a device with sm_count SMs."""
    return ROUTES[int(_lib.gdn_prefill_route(T, N, int(max_seqlen_hint), Hv, sm_count,
                                             1 if cooperative_launch else 0))]


def gdn_prefill_workspace_bytes(T, N, Hqk, Hv, dk=128, dv=128, chunk=64) -> int:
    return int(_lib.gdn_prefill_workspace_bytes(T, N, Hqk, Hv, dk, dv, chunk))


def gdn_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, scale,
                workspace, max_seqlen_hint=0, chunk=64, dev_status=None, route="auto",
                split_permille=-1):
    """Prefill over packed sequences.  ``workspace`` is a uint8 CUDA tensor.  ``route`` picks the
    entry point: "auto" = gdn_prefill (routes by length), "chunked" = gdn_prefill_chunked (three
    launches), "fused" = gdn_prefill_fused (one cooperative launch), "stream" = gdn_prefill_stream
    (three launches, persistent state pass), "overlap" = gdn_prefill_overlap (the intra-chunk work
    in two parts around the state pass; ``split_permille`` is its last argument)."""
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    fn = {"auto": _lib.gdn_prefill, "chunked": _lib.gdn_prefill_chunked,
          "fused": _lib.gdn_prefill_fused, "stream": _lib.gdn_prefill_stream,
          "overlap": _lib.gdn_prefill_overlap}[route]
    extra = (int(split_permille),) if route == "overlap" else ()
    rc = fn(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(cu_seqlens, torch.int32, "cu_seqlens"),
        _dev(init_state, torch.float32, "init_state", True),
        _dev(final_state, torch.float32, "final_state"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        T, N, int(max_seqlen_hint), Hqk, Hv, dk, dv, int(chunk), final_state.shape[0],
        float(scale), _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
        _dev(dev_status, torch.int32, "dev_status", True), _stream(), *extra)
    if rc != 0:
        raise GdnError(rc, "gdn_prefill")


def gdn_prefill_recurrent(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o,
                          scale, dev_status=None):
    """Token-by-token prefill on the CUDA cores; same arguments as gdn_prefill, no workspace."""
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    rc = _lib.gdn_prefill_recurrent(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(cu_seqlens, torch.int32, "cu_seqlens"),
        _dev(init_state, torch.float32, "init_state", True),
        _dev(final_state, torch.float32, "final_state"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        T, N, Hqk, Hv, dk, dv, final_state.shape[0], float(scale),
        _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_prefill_recurrent")


# chunk slots (floor(T/64) + N) the built-in array of gdn_prefill_static covers at 32 v-heads
STATIC_MAX_CHUNK_SLOTS_HV32 = 14


def gdn_prefill_static_workspace_bytes() -> int:
    """Size of the scratch array built into the library (the limit gdn_prefill_static enforces)."""
    return int(_lib.gdn_prefill_static_workspace_bytes())


def gdn_prefill_static(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, scale,
                       max_seqlen_hint=0, chunk=64, dev_status=None):
    """gdn_prefill without a caller-supplied workspace, for callers that may not allocate device
    memory: the scratch is a fixed array inside the library.  Raises GdnError(-7) when the batch
    needs more scratch than that array holds.  Calls sharing a device must not overlap."""
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    rc = _lib.gdn_prefill_static(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(cu_seqlens, torch.int32, "cu_seqlens"),
        _dev(init_state, torch.float32, "init_state", True),
        _dev(final_state, torch.float32, "final_state"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        T, N, int(max_seqlen_hint), Hqk, Hv, dk, dv, int(chunk), final_state.shape[0],
        float(scale), _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_prefill_static")


def gdn_host_us_per_decode_call(q, k, v, g, beta, state_pool, slot_idx, o, scale, reps=100) -> float:
    """Mean host microseconds inside one gdn_decode call (a C++ loop of ``reps`` calls; see gdn.h)."""
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    us = _lib.gdn_host_us_per_decode_call(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(state_pool, torch.float32, "state_pool"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        B, Hqk, Hv, dk, dv, state_pool.shape[0], float(scale), _stream(), int(reps))
    if us < 0:
        raise GdnError(int(us), "gdn_host_us_per_decode_call")
    return float(us)


def gdn_host_us_per_prefill_call(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o,
                                 scale, workspace, max_seqlen_hint=0, chunk=64, reps=50) -> float:
    """Mean host microseconds inside one gdn_prefill call (a C++ loop of ``reps`` calls)."""
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    us = _lib.gdn_host_us_per_prefill_call(
        _dev(q, torch.bfloat16, "q"), _dev(k, torch.bfloat16, "k"), _dev(v, torch.bfloat16, "v"),
        _dev(g, torch.float32, "g"), _dev(beta, torch.float32, "beta"),
        _dev(cu_seqlens, torch.int32, "cu_seqlens"),
        _dev(init_state, torch.float32, "init_state", True),
        _dev(final_state, torch.float32, "final_state"),
        _dev(slot_idx, torch.int32, "slot_idx", True), _dev(o, torch.bfloat16, "o"),
        T, N, int(max_seqlen_hint), Hqk, Hv, dk, dv, int(chunk), final_state.shape[0],
        float(scale), _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(),
        int(reps))
    if us < 0:
        raise GdnError(int(us), "gdn_host_us_per_prefill_call")
    return float(us)


def _host(t, dtype, name, allow_none=False):
    if t is None:
        if allow_none:
            return None
        raise TypeError(f"{name} is required")
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous host tensor of dtype {dtype}")
    return ctypes.c_void_p(t.data_ptr())


def gdn_decode_host_staging_bytes(B, Hqk, Hv) -> int:
    return int(_lib.gdn_decode_host_staging_bytes(B, Hqk, Hv))


def gdn_decode_host(q, k, v, g, beta, state_pool, slot_idx, o, scale, staging, dev_status=None):
    """gdn_decode with host (pinned) q, k, v, g, beta, slot_idx and o; the state pool, the uint8
    staging tensor and dev_status are CUDA tensors.  o is valid after a stream synchronise."""
    B, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    rc = _lib.gdn_decode_host(
        _host(q, torch.bfloat16, "q"), _host(k, torch.bfloat16, "k"), _host(v, torch.bfloat16, "v"),
        _host(g, torch.float32, "g"), _host(beta, torch.float32, "beta"),
        _dev(state_pool, torch.float32, "state_pool"),
        _host(slot_idx, torch.int32, "slot_idx", True), _host(o, torch.bfloat16, "o"),
        B, Hqk, Hv, dk, dv, state_pool.shape[0], float(scale),
        _dev(staging, torch.uint8, "staging"), staging.numel(),
        _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_decode_host")


def gdn_prefill_host_staging_bytes(T, N, Hqk, Hv) -> int:
    return int(_lib.gdn_prefill_host_staging_bytes(T, N, Hqk, Hv))


def gdn_prefill_host(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, scale,
                     staging, workspace, max_seqlen_hint=0, chunk=64, dev_status=None):
    """gdn_prefill with host (pinned) q, k, v, g, beta, cu_seqlens, slot_idx and o."""
    T, Hqk, dk = q.shape
    _, Hv, dv = v.shape
    N = cu_seqlens.shape[0] - 1
    rc = _lib.gdn_prefill_host(
        _host(q, torch.bfloat16, "q"), _host(k, torch.bfloat16, "k"), _host(v, torch.bfloat16, "v"),
        _host(g, torch.float32, "g"), _host(beta, torch.float32, "beta"),
        _host(cu_seqlens, torch.int32, "cu_seqlens"),
        _dev(init_state, torch.float32, "init_state", True),
        _dev(final_state, torch.float32, "final_state"),
        _host(slot_idx, torch.int32, "slot_idx", True), _host(o, torch.bfloat16, "o"),
        T, N, int(max_seqlen_hint), Hqk, Hv, dk, dv, int(chunk), final_state.shape[0],
        float(scale), _dev(staging, torch.uint8, "staging"), staging.numel(),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
        _dev(dev_status, torch.int32, "dev_status", True), _stream())
    if rc != 0:
        raise GdnError(rc, "gdn_prefill_host")

"""Latency sweep over the short-prompt / small-batch regime (decode B = 1..64, prefill from a few
tokens to 8192 tokens in up to 57 sequences): the shape distribution of the paper's per-workload
GDN tables, on seeded synthetic inputs.  Prints one JSON object per shape and a summary line.

    python sweep.py [--reps 200]
    python sweep.py --lens 144x56,128 --route stream   # one prefill shape
    python sweep.py --lens 512,1024,2048,4096 --route overlap --split-permille 1000
    python sweep.py --decode-multi 64x4                # one multi-token shape
    python sweep.py --decode 256 --slots 512 --reps 40 # one decode shape
    python sweep.py --gate 8192 | --transpose 64       # the gate helper / the tile transpose

Each shape's call is captured `GRAPH_CALLS` times into one CUDA graph, and the graph is replayed
and timed with CUDA events: the number is device time per call including kernel launch gaps but
not the Python binding's host overhead (about 15 us per call, which would otherwise hide every
kernel shorter than that).  Inputs stay L2-resident, as they are in a serving loop at these sizes.
Beside it, `host_us` is the time the HOST spends inside one eager call of the C entry point
(argument checks, tensor maps, launches), measured by a C++ loop inside the library.
`bench.py` imports `run()` for the "sweep" key of its JSON line.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from paper_2607_17979_b200 import api, inputs as I

DECODE_BATCHES = [1, 4, 8, 16, 32, 48, 64]
MULTI_SHAPES = [(1, 2), (1, 8), (8, 4), (32, 4), (64, 1), (64, 2), (64, 4), (64, 8)]
PREFILL_SHAPES = [[6], [12], [35], [100], [256], [512], [1024], [300, 700], [2855, 2854],
                  [410] * 20, [144] * 56 + [128]]
# the (batch, tokens) grid on which the host time per eager call is reported
HOST_DECODE_BATCHES = [1, 8, 64]
HOST_PREFILL_TOKENS = [6, 100, 1024]


def _bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _dev(x):
    return None if x is None else torch.from_numpy(x).cuda()


GRAPH_CALLS = 20


def _time(fn, reps):
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(3):          # warm-up outside capture (also resolves lazy set-up)
            fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(GRAPH_CALLS):
            fn()
    replays = max(2, reps // GRAPH_CALLS)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * GRAPH_CALLS) * 1e3          # microseconds


def _multi_rows(B, L, reps):
    d = I.decode_multi_inputs(B, L, 16, 32, 128, B, seed=I.BASE_SEED + 7 * B + L)
    t = {n: _bf16(d[n]) for n in "qkv"}
    g, beta, pool = _dev(d["g"]), _dev(d["beta"]), _dev(d["state"])
    o = torch.empty((B, L, 32, 128), dtype=torch.bfloat16, device="cuda")
    out = []
    for layout, name in ((api.STATE_VK, "vk"), (api.STATE_KV, "kv")):
        us = _time(lambda: api.gdn_decode_multi(t["q"], t["k"], t["v"], g, beta, pool, None, o,
                                                d["scale"], layout), reps)
        out.append({"op": "decode_multi", "B": B, "L": L, "layout": name, "us": us,
                    "tokens_per_s": B * L / us * 1e6})
    return out


def _decode_row(B, reps, slots=None, host=False):
    slots = B if slots is None else slots
    d = I.decode_inputs(B, 16, 32, 128, slots, seed=I.BASE_SEED + B,
                        slots="perm" if slots > B else "identity")
    t = {n: _bf16(d[n]) for n in "qkv"}
    g, beta, pool, idx = _dev(d["g"]), _dev(d["beta"]), _dev(d["state"]), _dev(d["slot_idx"])
    o = torch.empty((B, 32, 128), dtype=torch.bfloat16, device="cuda")
    us = _time(lambda: api.gdn_decode(t["q"], t["k"], t["v"], g, beta, pool, idx, o, d["scale"]), reps)
    row = {"op": "decode", "B": B, "Hqk": 16, "Hv": 32, "us": us,
           "state_GBps": 2 * B * 32 * 65536 / us / 1e3}
    if host:
        row["host_us"] = api.gdn_host_us_per_decode_call(t["q"], t["k"], t["v"], g, beta, pool, idx, o,
                                                         d["scale"], reps=200)
    return row


def _gate_row(T, reps):
    d = I.gate_inputs(T, 32, seed=I.BASE_SEED + T)
    a, b = _bf16(d["a"]), _bf16(d["b"])
    A_log, dt_bias = _dev(d["A_log"]), _dev(d["dt_bias"])
    g = torch.empty((T, 32), dtype=torch.float32, device="cuda")
    beta = torch.empty_like(g)
    us = _time(lambda: api.gdn_gate(a, b, A_log, dt_bias, g, beta), reps)
    return {"op": "gate", "T": T, "Hv": 32, "us": us}


def _transpose_row(n, reps):
    pool = torch.randn((n, 32, 128, 128), dtype=torch.float32, device="cuda")
    us = _time(lambda: api.gdn_state_transpose(pool), reps)
    return {"op": "state_transpose", "slots": n, "Hv": 32, "us": us,
            "GBps": 2 * n * 32 * 65536 / us / 1e3}


def _prefill_row(lens, route, reps, split_permille=-1, host=False):
    p = I.prefill_inputs(lens, 16, 32, 128, seed=I.BASE_SEED + sum(lens), init="zero")
    t = {n: _bf16(p[n]) for n in "qkv"}
    g, beta, cu = _dev(p["g"]), _dev(p["beta"]), _dev(p["cu_seqlens"])
    final = torch.empty((p["N"], 32, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.empty((p["T"], 32, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(api.gdn_prefill_workspace_bytes(p["T"], p["N"], 16, 32), dtype=torch.uint8,
                     device="cuda")
    us = _time(lambda: api.gdn_prefill(t["q"], t["k"], t["v"], g, beta, cu, None, final, None, o,
                                       p["scale"], ws, max_seqlen_hint=max(lens), route=route,
                                       split_permille=split_permille), reps)
    row = {"op": "prefill", "route": route, "tokens": p["T"], "seqs": p["N"], "longest": max(lens),
           "us": us, "tokens_per_s": p["T"] / us * 1e6}
    if route == "auto":
        row["route_taken"] = api.gdn_prefill_route(p["T"], p["N"], max(lens), 32)
    if host:
        row["host_us"] = api.gdn_host_us_per_prefill_call(t["q"], t["k"], t["v"], g, beta, cu, None,
                                                          final, None, o, p["scale"], ws,
                                                          max_seqlen_hint=max(lens), reps=50)
    return row


def run(reps=200, multi=True):
    """The whole sweep; returns (rows, summary)."""
    rows = []
    for B in DECODE_BATCHES:
        rows.append(_decode_row(B, reps, host=B in HOST_DECODE_BATCHES))
    if multi:   # multi-token decode (L new tokens per sequence in one call), both state orientations
        for B, L in MULTI_SHAPES:
            rows += _multi_rows(B, L, reps)
    for lens in PREFILL_SHAPES:
        rows.append(_prefill_row(lens, "auto", max(10, reps // 4),
                                 host=len(lens) == 1 and lens[0] in HOST_PREFILL_TOKENS))
    dec = [r["us"] for r in rows if r["op"] == "decode"]
    pre = [r["us"] for r in rows if r["op"] == "prefill"]
    summary = {"summary": "mean latency over the sweep (CUDA-graph replay, device time per call)",
               "decode_mean_us": float(np.mean(dec)), "prefill_mean_us": float(np.mean(pre)),
               "decode_batches": DECODE_BATCHES,
               "prefill_shapes": [f"{len(l)}x{l[0]}" if len(set(l)) == 1 else
                                  (f"{len(l)} seqs, {sum(l)} tokens" if len(l) > 4 else "+".join(map(str, l)))
                                  for l in PREFILL_SHAPES],
               "host_us_per_eager_call": {
                   "decode": {str(r["B"]): r["host_us"] for r in rows
                              if r["op"] == "decode" and "host_us" in r},
                   "prefill": {str(r["tokens"]): r["host_us"] for r in rows
                               if r["op"] == "prefill" and "host_us" in r}}}
    return rows, summary


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=200)
    ap.add_argument("--lens", default="", help="time one prefill shape only: comma-separated "
                    "sequence lengths, LENxCOUNT for repeats (e.g. 144x56,128)")
    ap.add_argument("--route", default="auto", choices=["auto", "chunked", "fused", "stream", "overlap"])
    ap.add_argument("--split-permille", type=int, default=-1, help="last argument of the overlap route")
    ap.add_argument("--decode-multi", default="", help="time one multi-token decode shape only: "
                    "BxL (both state orientations)")
    ap.add_argument("--decode", type=int, default=0, help="time one decode batch size only")
    ap.add_argument("--slots", type=int, default=0, help="pool slots for --decode (default: B)")
    ap.add_argument("--gate", type=int, default=0, help="time the gate helper on this many tokens only")
    ap.add_argument("--transpose", type=int, default=0, help="time the in-place tile transpose on "
                    "this many slots only")
    args = ap.parse_args()
    if args.decode_multi:
        B, _, L = args.decode_multi.partition("x")
        for r in _multi_rows(int(B), int(L), args.reps):
            print(json.dumps(r))
        return
    if args.gate:
        print(json.dumps(_gate_row(args.gate, args.reps)))
        return
    if args.transpose:
        print(json.dumps(_transpose_row(args.transpose, args.reps)))
        return
    if args.decode:
        print(json.dumps(_decode_row(args.decode, args.reps, slots=args.slots or None, host=True)))
        return
    if args.lens:
        lens = []
        for part in args.lens.split(","):
            n, _, c = part.partition("x")
            lens += [int(n)] * (int(c) if c else 1)
        print(json.dumps(_prefill_row(lens, args.route, max(10, args.reps // 4),
                                      split_permille=args.split_permille, host=True)))
        return
    rows, summary = run(args.reps)
    for r in rows:
        print(json.dumps(r))
    print(json.dumps(summary))


if __name__ == "__main__":
    main()

"""Latency sweep over the short-prompt / small-batch regime (decode B = 1..64, prefill from a few
tokens to 8192 tokens in up to 57 sequences): the shape distribution of the paper's per-workload
GDN tables, on seeded synthetic inputs.  Prints one JSON object per shape and a summary line.

    python -m paper_2607_17979_b200.sweep [--reps 200]
    python -m paper_2607_17979_b200.sweep --lens 144x56,128 --route stream   # one prefill shape
    python -m paper_2607_17979_b200.sweep --decode-multi 64x4                # one multi-token shape

Each shape's call is captured `GRAPH_CALLS` times into one CUDA graph, and the graph is replayed
and timed with CUDA events: the number is device time per call including kernel launch gaps but
not the Python binding's host overhead (about 15 us per call, which would otherwise hide every
kernel shorter than that).  Inputs stay L2-resident, as they are in a serving loop at these sizes.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import api, inputs as I

DECODE_BATCHES = [1, 4, 8, 16, 32, 48, 64]
MULTI_SHAPES = [(1, 2), (1, 8), (8, 4), (32, 4), (64, 1), (64, 2), (64, 4), (64, 8)]
PREFILL_SHAPES = [[6], [12], [35], [100], [256], [512], [1024], [300, 700], [2855, 2854],
                  [410] * 20, [144] * 56 + [128]]


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


def _prefill_row(lens, route, reps):
    p = I.prefill_inputs(lens, 16, 32, 128, seed=I.BASE_SEED + sum(lens), init="zero")
    t = {n: _bf16(p[n]) for n in "qkv"}
    g, beta, cu = _dev(p["g"]), _dev(p["beta"]), _dev(p["cu_seqlens"])
    final = torch.empty((p["N"], 32, 128, 128), dtype=torch.float32, device="cuda")
    o = torch.empty((p["T"], 32, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(api.gdn_prefill_workspace_bytes(p["T"], p["N"], 16, 32), dtype=torch.uint8,
                     device="cuda")
    us = _time(lambda: api.gdn_prefill(t["q"], t["k"], t["v"], g, beta, cu, None, final, None, o,
                                       p["scale"], ws, max_seqlen_hint=max(lens), route=route), reps)
    return {"op": "prefill", "route": route, "tokens": p["T"], "seqs": p["N"], "longest": max(lens),
            "us": us, "tokens_per_s": p["T"] / us * 1e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=200)
    ap.add_argument("--lens", default="", help="time one prefill shape only: comma-separated "
                    "sequence lengths, LENxCOUNT for repeats (e.g. 144x56,128)")
    ap.add_argument("--route", default="auto", choices=["auto", "chunked", "fused", "stream", "overlap"])
    ap.add_argument("--decode-multi", default="", help="time one multi-token decode shape only: "
                    "BxL (both state orientations)")
    args = ap.parse_args()
    rows = []
    if args.decode_multi:
        B, _, L = args.decode_multi.partition("x")
        for r in _multi_rows(int(B), int(L), args.reps):
            print(json.dumps(r))
        return
    if args.lens:
        lens = []
        for part in args.lens.split(","):
            n, _, c = part.partition("x")
            lens += [int(n)] * (int(c) if c else 1)
        print(json.dumps(_prefill_row(lens, args.route, max(10, args.reps // 4))))
        return
    for B in DECODE_BATCHES:
        d = I.decode_inputs(B, 16, 32, 128, B, seed=I.BASE_SEED + B)
        t = {n: _bf16(d[n]) for n in "qkv"}
        g, beta, pool = _dev(d["g"]), _dev(d["beta"]), _dev(d["state"])
        o = torch.empty((B, 32, 128), dtype=torch.bfloat16, device="cuda")
        us = _time(lambda: api.gdn_decode(t["q"], t["k"], t["v"], g, beta, pool, None, o, d["scale"]),
                   args.reps)
        rows.append({"op": "decode", "B": B, "Hqk": 16, "Hv": 32, "us": us,
                     "state_GBps": 2 * B * 32 * 65536 / us / 1e3})
    # multi-token decode (L new tokens per sequence in one call), both state orientations
    for B, L in MULTI_SHAPES:
        rows += _multi_rows(B, L, args.reps)
    for lens in PREFILL_SHAPES:
        rows.append(_prefill_row(lens, "auto", max(10, args.reps // 4)))
    for r in rows:
        print(json.dumps(r))
    dec = [r["us"] for r in rows if r["op"] == "decode"]
    pre = [r["us"] for r in rows if r["op"] == "prefill"]
    print(json.dumps({"summary": "mean latency over the sweep", "decode_mean_us": float(np.mean(dec)),
                      "prefill_mean_us": float(np.mean(pre))}))


if __name__ == "__main__":
    main()

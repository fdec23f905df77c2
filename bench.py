#!/usr/bin/env python
"""Benchmark of the gated delta rule hot path on B200: decode state-GB/s and prefill tokens/s.

One step = one decode call on the B=64 configuration (64 sequences x 32 v-heads, a 128 MiB fp32
state pool updated in place) followed by one chunked prefill call on the packed variable-length
configuration (4 sequences, 7680 tokens).  Both are timed separately with CUDA events on the
launching stream, on inputs that rotate through more memory than L2 holds.  The headline `value` is decode state-GB/s; the prefill
leg's tokens/s and roofline are reported in the same JSON line under "prefill".

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Outside that timed step, rank 0 of a 1-GPU run also times the other three configurations and two
measurement workloads, a few calls each, and adds them to the same JSON line: "decode_b1"
(B=1 latency), "decode_paged" (B=256 of 512 slots, 1 GiB pool), "prefill_long" (one sequence of
32768 tokens), "chain_bound" (the dependent chunk step of this run, from two single-sequence
calls of 8192 and 16384 tokens) and "sweep" (mean latency over the short-prompt / small-batch
shapes under CUDA-graph replay, with the host time per eager call).

With N > 1 (launched by torch.distributed.run) every rank runs the same per-GPU workload on its
own GPU (independent sequences, no data-path collective: weak scaling); the timed region is
bracketed by a barrier and the per-step times are the max over ranks.
`--impl reference` times the fp64 CPU oracle on the host cores on the same metric.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_17979_b200 import inputs as I  # noqa: E402

DECODE_CFG, PREFILL_CFG = 1, 3
DEC_POOLS, PRE_SETS = 8, 3
TILE_BYTES = 128 * 128 * 4
WORKLOAD = ("step = gdn_decode B=64 Hqk=16 Hv=32 d=128, 128 MiB fp32 state pool in place (configs[1]) "
            "+ gdn_prefill 4 seqs {512,1024,2048,4096} = 7680 tokens, chunk 64 (configs[3])")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# single-sequence shapes whose time difference gives the dependent chunk step of this run
CHAIN_SHORT, CHAIN_LONG = 8192, 16384
EXTRA_REPS = 20          # timed calls of each workload outside the main step


def ncu_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per call from the committed ncu captures:
    profiles/traffic.json is rewritten whenever a summary under profiles/ is refreshed."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            return json.load(f)
    except (OSError, ValueError):
        return {}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def decode_bytes(B, Hqk, Hv, with_idx):
    """Algorithmic bytes of one decode call: state read + written, q, k, v, o, g, beta (+ slots)."""
    state = 2 * B * Hv * TILE_BYTES
    other = B * (2 * Hqk * 128 * 2 + 2 * Hv * 128 * 2 + 2 * Hv * 4 + (4 if with_idx else 0))
    return state, state + other


def prefill_bytes_flops(T, N, Hqk, Hv, with_init):
    """Algorithmic bytes / flops of one prefill call (triangular products at half, Gram products
    once per q/k head): 24832 B and 4194304 flop per token at Hqk=16, Hv=32."""
    per_tok = 2 * Hqk * 128 * 2 + 2 * Hv * 128 * 2 + 2 * Hv * 4
    nbytes = T * per_tok + N * Hv * TILE_BYTES * (2 if with_init else 1) + 4 * (N + 1)
    flops = T * (Hqk * 16384 + Hv * 122880)
    return nbytes, flops


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", "20"], stdout=open(self.path, "w"),
                stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


def oracle_sample(dec, pre, decode_reps=5):
    """Time the fp64 oracle, as it stands, on the host cores: the whole decode configuration
    (`decode_reps` consecutive steps on its pool) and the whole prefill configuration once."""
    import oracle
    oracle.build()
    cores = min(oracle.default_threads(), len(os.sched_getaffinity(0)))
    pool = dec["state"].astype(np.float64)
    t0 = time.perf_counter()
    for _ in range(decode_reps):
        oracle.decode(dec["q"], dec["k"], dec["v"], dec["g"], dec["beta"], pool, dec["slot_idx"],
                      dec["scale"], n_threads=cores)
    t_dec = (time.perf_counter() - t0) / decode_reps
    t0 = time.perf_counter()
    oracle.prefill(pre["q"], pre["k"], pre["v"], pre["g"], pre["beta"], pre["cu_seqlens"], None, None,
                   pre["scale"], n_threads=cores)
    t_pre = time.perf_counter() - t0
    state_bytes, _ = decode_bytes(dec["B"], dec["Hqk"], dec["Hv"], dec["slot_idx"] is not None)
    return dict(cores=cores, decode_s=t_dec, decode_state_gbs=state_bytes / t_dec / 1e9,
                prefill_s=t_pre, prefill_tokens=pre["T"], prefill_tok_s=pre["T"] / t_pre,
                sample=(f"decode: the whole B={dec['B']} step, mean of {decode_reps} consecutive "
                        f"steps ({t_dec * 1e3:.1f} ms each; state bytes counted as fp32); prefill: "
                        f"the whole varlen batch ({pre['T']} tokens, {pre['Hv']} v-heads, "
                        f"{t_pre:.2f} s)"))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dec = I.make_config(DECODE_CFG)
    pre = I.make_config(PREFILL_CFG)
    for _ in range(args.warmup):
        r = oracle_sample(dec, pre)
    times, gbs, last = [], [], None
    for _ in range(args.steps):
        last = oracle_sample(dec, pre)
        times.append(last["decode_s"] + last["prefill_s"])
        gbs.append(last["decode_state_gbs"])
    dec_gbs = float(np.mean(gbs))
    line = {
        "impl": "reference", "metric": "gdn_decode_state_GBps", "value": dec_gbs, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * float(np.mean(times)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": "host run: the fp64 oracle on the host cores"},
        "cpu_baseline": {"value": dec_gbs, "unit": "GB/s", "cores": last["cores"], "kind": "oracle",
                         "sample": last["sample"]},
        "prefill": {"metric": "gdn_prefill_tokens_per_s", "value": last["prefill_tok_s"],
                    "unit": "tokens/s"},
        "e2e": {"value": dec_gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args):
    import torch
    from paper_2607_17979_b200 import api, dist as D

    rank, world, local = D.world()
    torch.cuda.set_device(local)
    D.init("nccl", torch.device("cuda", local))

    def bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    def dev(x):
        return None if x is None else torch.from_numpy(x).cuda()

    # every rank owns its own sequences (different seeds): weak scaling, no exchange
    dec = I.make_config(DECODE_CFG, trial=rank)
    pre = I.make_config(PREFILL_CFG, trial=rank)
    B, Hqk, Hv = dec["B"], dec["Hqk"], dec["Hv"]
    T, N = pre["T"], pre["N"]

    d_in = {n: (bf16(dec[n]) if n in "qkv" else dev(dec[n])) for n in ("q", "k", "v", "g", "beta")}
    # decode rotates over DEC_POOLS distinct 128 MiB pools (1 GiB > 126 MB L2) and prefill over
    # PRE_SETS distinct input sets, so no call finds its inputs in L2 from the previous step
    pools = [dev(dec["state"]) for _ in range(DEC_POOLS)]
    d_o = torch.empty((B, Hv, 128), dtype=torch.bfloat16, device="cuda")
    p_sets = [{n: (bf16(pre[n]) if n in "qkv" else dev(pre[n])) for n in ("q", "k", "v", "g", "beta")}
              for _ in range(PRE_SETS)]
    p_in = p_sets[0]
    cu = dev(pre["cu_seqlens"])
    p_final = torch.empty((N, Hv, 128, 128), dtype=torch.float32, device="cuda")
    p_o = torch.empty((T, Hv, 128), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(max(api.gdn_prefill_workspace_bytes(T, N, Hqk, Hv), 256), dtype=torch.uint8,
                     device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    counter = {"step": 0}

    # pinned host buffers + device staging for the end-to-end leg (host-buffer entry points)
    h_dec = {n: t.cpu().pin_memory() for n, t in d_in.items()}
    h_do = torch.empty_like(d_o, device="cpu").pin_memory()
    h_pre = {n: t.cpu().pin_memory() for n, t in p_in.items()}
    h_cu = cu.cpu().pin_memory()
    h_po = torch.empty_like(p_o, device="cpu").pin_memory()
    stage_d = torch.empty(api.gdn_decode_host_staging_bytes(B, Hqk, Hv), dtype=torch.uint8, device="cuda")
    stage_p = torch.empty(api.gdn_prefill_host_staging_bytes(T, N, Hqk, Hv), dtype=torch.uint8,
                          device="cuda")

    def decode_call():
        pool = pools[counter["step"] % DEC_POOLS]
        api.gdn_decode(d_in["q"], d_in["k"], d_in["v"], d_in["g"], d_in["beta"], pool, None, d_o,
                       dec["scale"], status)

    def prefill_call(src=None):
        x = p_sets[counter["step"] % PRE_SETS] if src is None else src
        api.gdn_prefill(x["q"], x["k"], x["v"], x["g"], x["beta"], cu, None, p_final,
                        None, p_o, pre["scale"], ws, max_seqlen_hint=max(pre["seq_lens"]),
                        dev_status=status)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def step(timed):
        counter["step"] += 1
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record(); decode_call(); e1.record()
        e2.record(); prefill_call(); e3.record()
        if timed is not None:
            timed.append((e0, e1, e2, e3))

    def e2e_step(timed):
        counter["step"] += 1
        e0, e1, e2, e3 = ev(), ev(), ev(), ev()
        e0.record()
        api.gdn_decode_host(h_dec["q"], h_dec["k"], h_dec["v"], h_dec["g"], h_dec["beta"],
                            pools[counter["step"] % DEC_POOLS], None, h_do, dec["scale"], stage_d,
                            dev_status=status)
        e1.record()
        e2.record()
        api.gdn_prefill_host(h_pre["q"], h_pre["k"], h_pre["v"], h_pre["g"], h_pre["beta"], h_cu,
                             None, p_final, None, h_po, pre["scale"], stage_p, ws,
                             max_seqlen_hint=max(pre["seq_lens"]), dev_status=status)
        e3.record()
        if timed is not None:
            timed.append((e0, e1, e2, e3))

    def barrier():
        D.barrier()
        torch.cuda.synchronize()

    def timed_region(fn):
        for _ in range(args.warmup):
            fn(None)
        barrier()
        evs = []
        for _ in range(args.steps):
            fn(evs)
        barrier()
        dec_ms = np.array([a.elapsed_time(b) for a, b, _, _ in evs])
        pre_ms = np.array([c.elapsed_time(d) for _, _, c, d in evs])
        slowest = D.max_over_ranks([dec_ms.mean(), pre_ms.mean()], device="cuda")
        spread = {"decode_ms_median": float(np.median(dec_ms)), "decode_ms_min": float(dec_ms.min()),
                  "prefill_ms_median": float(np.median(pre_ms)), "prefill_ms_min": float(pre_ms.min())}
        return slowest[0], slowest[1], spread

    # clocks are sampled from before the warm-up to after the timed steps (the GPU is under the
    # same load throughout; the timed steps alone can be shorter than one sampling period)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    dec_ms, pre_ms, spread = timed_region(step)
    e2e_dec_ms, e2e_pre_ms, _ = timed_region(e2e_step)
    assert int(status.item()) == 0, "device status flagged during the benchmark"
    extra = None
    if rank == 0 and world == 1 and not args.no_extra:
        # free the step's buffers first: the long-context workload alone needs 2 GB
        del pools[1:], p_sets[1:], h_pre, h_po, stage_p, stage_d
        torch.cuda.empty_cache()
        extra = extra_workloads(api, torch, status, pre)
    clocks = sampler.stop() if rank == 0 else None
    assert int(status.item()) == 0, "device status flagged during the benchmark"

    if rank == 0:
        pk, pk_kind = peaks()
        traffic = ncu_traffic()
        state_b, dec_b = decode_bytes(B, Hqk, Hv, False)
        pre_b, pre_f = prefill_bytes_flops(T, N, Hqk, Hv, False)
        dec_gbs = world * state_b / (dec_ms * 1e-3) / 1e9
        dec_ach = dec_b / (dec_ms * 1e-3) / 1e9
        pre_tok = world * T / (pre_ms * 1e-3)
        cpu = oracle_sample(dec, pre)
        h2d = sum(t.numel() * t.element_size() for t in h_dec.values())
        h2d_p = 2 * T * Hqk * 256 + T * Hv * 256 + 2 * T * Hv * 4 + (N + 1) * 4
        pre_roof = prefill_roofline(pre_b, pre_f, pre_ms, pk, pk_kind, traffic.get("prefill_config3"))
        dec_roof = {"kernel": "gdn decode (decode_kernel, one launch)", "bound": "hbm",
                    "achieved": dec_ach, "peak": pk["hbm_gbs"], "unit": "GB/s",
                    "frac": dec_ach / pk["hbm_gbs"], "peak_kind": pk_kind,
                    "frac_of_nominal_8TBps": dec_ach / 8000.0, "algorithmic_bytes": dec_b,
                    "traffic": traffic.get("decode_config1")}
        depth = -(-max(pre["seq_lens"]) // 64)
        step_us = extra["chain_bound"]["chunk_step_us"] if extra else None
        line = {
            "metric": "gdn_decode_state_GBps", "value": dec_gbs, "unit": "GB/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dec_ms + pre_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "per_gpu": True,
                       "l2": f"inputs larger than L2: decode rotates over {DEC_POOLS} distinct 128 MiB "
                             f"state pools (1 GiB), prefill over {PRE_SETS} distinct input sets "
                             "(3 x 190 MB) plus its workspace",
                       "decode_ms": dec_ms, "prefill_ms": pre_ms,
                       "this_rank_spread": spread},
            # the dominant part of the step by time is the prefill call (all its launches)
            "roofline": pre_roof,
            "decode": {"metric": "gdn_decode_state_GBps", "value": dec_gbs, "unit": "GB/s",
                       "ms": dec_ms, "roofline": dec_roof},
            "prefill": {"metric": "gdn_prefill_tokens_per_s", "value": pre_tok, "unit": "tokens/s",
                        "ms": pre_ms, "dtype": "bf16 operands, f32 accumulate and state",
                        "route": api.gdn_prefill_route(T, N, max(pre["seq_lens"]), Hv),
                        "roofline": pre_roof,
                        # the serial part: the longest sequence's chunks, one dependent chunk step
                        # each, the step measured in this run (see "chain_bound")
                        "chain_bound": {"depth_chunks": depth, "chunk_step_us": step_us,
                                        "ms": None if step_us is None else depth * step_us * 1e-3},
                        "e2e": {"value": world * T / (e2e_pre_ms * 1e-3), "unit": "tokens/s",
                                "h2d_bytes_per_step": h2d_p,
                                "d2h_bytes_per_step": T * Hv * 256},
                        "cpu_baseline": {"value": cpu["prefill_tok_s"], "unit": "tokens/s"}},
            "cpu_baseline": {"value": cpu["decode_state_gbs"], "unit": "GB/s", "cores": cpu["cores"],
                             "kind": "oracle", "sample": cpu["sample"]},
            "e2e": {"value": world * state_b / (e2e_dec_ms * 1e-3) / 1e9, "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": h_do.numel() * 2,
                    "note": "gdn_decode_host / gdn_prefill_host: q,k,v,g,beta(,cu_seqlens) from pinned "
                            "host memory and o back every step; the state pool is the resident "
                            "recurrent cache and stays in HBM"},
            "gpu_launches": args.steps * api.LAUNCHES_PER_STEP,
            "clocks": clocks,
        }
        if extra:
            for name in ("decode_b1", "decode_paged", "prefill_long", "chain_bound", "sweep"):
                line[name] = extra[name]
            for name, key in (("decode_paged", "decode_config2"), ("prefill_long", "prefill_config4")):
                roof = line[name]["roofline"]
                roof["peak"], roof["peak_kind"] = pk["hbm_gbs"], pk_kind
                roof["frac"] = roof["achieved"] / pk["hbm_gbs"]
                roof["traffic"] = traffic.get(key)
            pl = line["prefill_long"]
            roof_ms = max(pl["roofline"]["algorithmic_bytes"] / (pk["hbm_gbs"] * 1e9),
                          pl["roofline"]["algorithmic_flops"] / (pk["bf16_tflops_sustained"] * 1e12)) * 1e3
            pl["roofline"]["roofline_ms"] = roof_ms
            pl["roofline"]["frac_of_roofline_time"] = roof_ms / pl["ms"]
            pl["chain_bound"] = {"depth_chunks": 512, "chunk_step_us": step_us,
                                 "ms": 512 * step_us * 1e-3}
        print(json.dumps(line))
    D.finish()


def prefill_roofline(nbytes, flops, ms, pk, pk_kind, traffic):
    roof_ms = max(nbytes / (pk["hbm_gbs"] * 1e9), flops / (pk["bf16_tflops_sustained"] * 1e12)) * 1e3
    ach = nbytes / (ms * 1e-3) / 1e9
    return {"kernel": "gdn prefill (all launches of one call)", "bound": "hbm", "achieved": ach,
            "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"], "peak_kind": pk_kind,
            "roofline_ms": roof_ms, "frac_of_roofline_time": roof_ms / ms,
            "algorithmic_bytes": nbytes, "algorithmic_flops": flops, "traffic": traffic}


def extra_workloads(api, torch, status, pre3):
    """The configurations the main step does not time, plus the measured chunk step and the
    small-shape sweep; EXTRA_REPS eager calls each, CUDA events, after 3 warm-up calls."""
    import sweep as SW

    def bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    def dev(x):
        return None if x is None else torch.from_numpy(x).cuda()

    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timed(fn, reps=EXTRA_REPS, flush=False):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        ts = []
        for i in range(reps):
            if flush:
                flush_buf.fill_(i & 255)        # 256 MB written: nothing of the workload stays in L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(i); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return float(np.mean(ts)), float(np.median(ts)), float(np.min(ts))

    out = {}
    # ---- configs[0]: decode B=1 (latency; about 1 MB moved, launch-bound: no fraction target)
    d0 = I.make_config(0)
    t0 = {n: (bf16(d0[n]) if n in "qkv" else dev(d0[n])) for n in ("q", "k", "v", "g", "beta")}
    pool0 = dev(d0["state"])
    o0 = torch.empty((1, d0["Hv"], 128), dtype=torch.bfloat16, device="cuda")
    call0 = lambda i: api.gdn_decode(t0["q"], t0["k"], t0["v"], t0["g"], t0["beta"], pool0, None, o0,
                                     d0["scale"], status)
    cold = timed(call0, flush=True)
    hot = timed(call0)
    graph_us = SW._time(lambda: call0(0), 200)
    _, b0 = decode_bytes(1, d0["Hqk"], d0["Hv"], False)
    out["decode_b1"] = {"workload": "configs[0]: gdn_decode B=1 Hqk=4 Hv=8", "unit": "us",
                        "value": cold[1] * 1e3, "us_cold_l2_median": cold[1] * 1e3,
                        "us_hot_l2_median": hot[1] * 1e3, "us_graph_replay": graph_us,
                        "algorithmic_bytes": b0,
                        "note": "eager CUDA-event times of one tiny launch include the launch itself; "
                                "graph replay is device time per call, L2-resident"}
    del pool0

    # ---- configs[2]: decode B=256 of 512 slots, rotating over 2 pools of 1 GiB
    d2 = I.make_config(2)
    t2 = {n: (bf16(d2[n]) if n in "qkv" else dev(d2[n])) for n in ("q", "k", "v", "g", "beta")}
    idx2 = dev(d2["slot_idx"])
    pools2 = [dev(d2["state"]) for _ in range(2)]
    o2 = torch.empty((256, 32, 128), dtype=torch.bfloat16, device="cuda")
    call2 = lambda i: api.gdn_decode(t2["q"], t2["k"], t2["v"], t2["g"], t2["beta"], pools2[i & 1],
                                     idx2, o2, d2["scale"], status)
    m2 = timed(call2)
    sb2, b2 = decode_bytes(256, 16, 32, True)
    out["decode_paged"] = {"workload": "configs[2]: gdn_decode B=256 of 512 slots, 1 GiB fp32 pool, "
                                       "int32 slot indices, 2 pools in rotation",
                           "metric": "gdn_decode_state_GBps", "unit": "GB/s",
                           "value": sb2 / (m2[0] * 1e-3) / 1e9, "ms": m2[0], "ms_median": m2[1],
                           "roofline": {"kernel": "gdn decode (decode_kernel, one launch)",
                                        "bound": "hbm", "achieved": b2 / (m2[0] * 1e-3) / 1e9,
                                        "unit": "GB/s", "algorithmic_bytes": b2,
                                        "frac_of_nominal_8TBps": b2 / (m2[0] * 1e-3) / 1e9 / 8000.0}}
    del pools2, d2, t2

    # ---- a prefill call on given lengths (16 / 32 heads), mean ms
    def prefill_ms(p, reps):
        T, N, Hv = p["T"], p["N"], p["Hv"]
        t = {n: (bf16(p[n]) if n in "qkv" else dev(p[n])) for n in ("q", "k", "v", "g", "beta")}
        cu, init = dev(p["cu_seqlens"]), dev(p["init_state"])
        final = torch.empty((N, Hv, 128, 128), dtype=torch.float32, device="cuda")
        o = torch.empty((T, Hv, 128), dtype=torch.bfloat16, device="cuda")
        ws = torch.empty(api.gdn_prefill_workspace_bytes(T, N, p["Hqk"], Hv), dtype=torch.uint8,
                         device="cuda")
        hint = max(p["seq_lens"])
        return timed(lambda i: api.gdn_prefill(t["q"], t["k"], t["v"], t["g"], t["beta"], cu, init,
                                               final, None, o, p["scale"], ws, max_seqlen_hint=hint,
                                               dev_status=status), reps)

    # ---- configs[4]: one sequence of 32768 tokens (inputs 0.8 GB + workspace: larger than L2)
    p4 = I.make_config(4)
    m4 = prefill_ms(p4, max(5, EXTRA_REPS // 2))
    b4, f4 = prefill_bytes_flops(p4["T"], 1, 16, 32, True)
    out["prefill_long"] = {"workload": "configs[4]: gdn_prefill 1 sequence of 32768 tokens, Hqk=16 "
                                       "Hv=32, alpha in [0.95,1), fp32 initial state",
                           "metric": "gdn_prefill_tokens_per_s", "unit": "tokens/s",
                           "value": p4["T"] / (m4[0] * 1e-3), "ms": m4[0], "ms_median": m4[1],
                           "route": api.gdn_prefill_route(p4["T"], 1, p4["T"], 32),
                           "roofline": {"kernel": "gdn prefill (all launches of one call)",
                                        "bound": "hbm", "achieved": b4 / (m4[0] * 1e-3) / 1e9,
                                        "unit": "GB/s", "algorithmic_bytes": b4,
                                        "algorithmic_flops": f4}}
    del p4
    torch.cuda.empty_cache()

    # ---- the dependent chunk step: two single sequences whose lengths differ by 128 chunks
    ms_s = prefill_ms(I.prefill_inputs([CHAIN_SHORT], 16, 32, seed=I.BASE_SEED + 1), EXTRA_REPS)
    ms_l = prefill_ms(I.prefill_inputs([CHAIN_LONG], 16, 32, seed=I.BASE_SEED + 2), EXTRA_REPS)
    dchunks = (CHAIN_LONG - CHAIN_SHORT) // 64
    out["chain_bound"] = {"chunk_step_us": (ms_l[1] - ms_s[1]) * 1e3 / dchunks,
                          "how": f"(median ms of 1 x {CHAIN_LONG} tokens - median ms of 1 x "
                                 f"{CHAIN_SHORT} tokens) / {dchunks} chunks, Hv=32, this run",
                          "ms_short": ms_s[1], "ms_long": ms_l[1],
                          "route": api.gdn_prefill_route(CHAIN_LONG, 1, CHAIN_LONG, 32)}
    torch.cuda.empty_cache()

    # ---- small-shape sweep (CUDA-graph replay) and host time per eager call (C++ loop)
    _, summary = SW.run(reps=100, multi=False)
    out["sweep"] = summary
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true",
                    help="time the main step only (skip the other configurations and the sweep)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

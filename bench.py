#!/usr/bin/env python
"""Benchmark of the mapper-construction hot path on synthetic Qwen3-14B->32B-shaped traces.

One step = one whole 500-sequence build: the weighted statistics are accumulated chunk by chunk (the 218 GB of
traces do not fit in HBM, so each chunk is generated on the device outside the timed region and is resident
when its timed region starts), then the split reduction and the batched ridge solve at three lambdas.
The step time is the sum of the CUDA-event-timed regions (accumulate calls, reduce, solve).

Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "calib_tokens_per_s_weighted_stat_build"
WORKLOAD = "qwen14b_32b_500"
ALG_BYTES_PER_TOKEN = 2 * 40 * 8 * 128 * 2 + 2 * 64 * 8 * 128 * 2 + 2 * 64 * 8 * 4   # 430,080: every source, target element and weight once
ALG_FLOPS_PER_TOKEN = 1024 * 2 * 129 * 257                                           # dense p x (2d+1) contraction per map


def algorithmic_work(wl):
    """(bytes, flops) per calibration token: every source element, target element and weight once; the dense
    (d+1) x (2d+1) contraction per map."""
    b = 2 * wl.Ls * wl.Hs * wl.d * 2 + 2 * wl.Lt * wl.Ht * wl.d * 2 + 2 * wl.Lt * wl.Ht * 4
    f = wl.n_maps * 2 * (wl.d + 1) * (2 * wl.d + 1)
    return b, f


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, interval_ms: int = 200):
        self.index = index
        self.interval_ms = interval_ms
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", str(self.interval_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            try:
                pw.append(float(parts[2]))
            except ValueError:
                pass
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "power_w": statistics.median(pw) if pw else None}


def sustained_loop(torch, index, launch, seconds=2.5, warm=20):
    """Back-to-back launches of one call on resident inputs for at least `seconds`: the board settles at its power
    limit, which a step made of isolated 4 ms launches never reaches.  CUDA events around the whole loop; SM clock and
    power sampled with nvidia-smi inside that window only.  Returns ms per launch and the clock record."""
    for _ in range(warm):
        launch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(10):
        launch()
    e1.record()
    e1.synchronize()
    n = max(50, int(seconds * 1e3 / (e0.elapsed_time(e1) / 10)) + 1)
    sampler = ClockSampler(index, interval_ms=100)
    sampler.start()
    time.sleep(0.15)                     # the sampler's first line
    e0.record()
    for _ in range(n):
        launch()
    e1.record()
    e1.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / n
    mhz = clocks.get("sm_mhz")
    return {"ms_per_launch": ms, "launches": n, "seconds": ms * n / 1e3, "sm_mhz": mhz,
            "power_w": clocks.get("power_w"), "ms_x_mhz": (ms * mhz) if mhz else None,
            "clock_samples": clocks.get("samples"), "reasons": clocks.get("reasons")}


def oracle_sample(n_tokens: int, seed_chunk: int = 0):
    """Times the oracle's statistics + solve on a 64-map, n_tokens sample with the workload's trace law
    (4 target layers x 8 heads x K/V); maps are independent and equal-cost, so tokens/s of the whole
    1024-map workload = (sample token-maps / 1024) / seconds."""
    import numpy as np
    import oracle
    from paper_2609_00891_b200 import synth

    full = synth.workload(WORKLOAD)
    wl = synth.Workload("oracle_sample", full.index, 3, full.Hs, 4, full.Ht, full.d, (n_tokens,) * (seed_chunk + 1), 1,
                        full.lambdas, full.kind, full.noise)
    sl, sh = oracle.head_map(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, seed_chunk, sl, sh, device="cpu")

    def bits(t):
        return t.contiguous().view(__import__("torch").int16).numpy().view(np.uint16)

    a = {k: bits(v) for k, v in ch.items() if k[:3] in ("src", "tgt")}
    t0 = time.perf_counter()
    G, C = oracle.stats_traces(a["src_k"], a["src_v"], a["tgt_k"], a["tgt_v"], ch["w_k"].numpy(), ch["w_v"].numpy(), sl, sh)
    for lam in wl.lambdas:
        oracle.ridge_solve(G, C, n_tokens, lam)
    dt = time.perf_counter() - t0
    token_maps = n_tokens * wl.n_maps
    return dt, token_maps, (token_maps / full.n_maps) / dt


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on the host cores, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    n_tok = 4096
    for _ in range(args.warmup):
        oracle_sample(256)
    times, rates = [], []
    for s in range(args.steps):
        dt, token_maps, rate = oracle_sample(n_tok, s)
        times.append(dt)
        rates.append(rate)
    value = statistics.mean(rates)
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(times),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": WORKLOAD, "note": "oracle on a bounded sample per step, extrapolated over maps"},
           "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": oracle.n_threads(), "kind": "oracle",
                            "sample": "64 maps x %d tokens per step (statistics + 3 solves), tokens/s = token-maps/1024/s" % n_tok},
           "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


TRAFFIC_DRAM_BYTES_PER_TOKEN = 437400        # dram__bytes_read + dram__bytes_write per token, k_accum_ts, 14B->32B shapes
TRAFFIC_DRAM_BYTES_PER_SPLIT = 270600000     # partial-slot read-modify-write per token split (1,024 maps)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--chunks", type=int, default=0, help="limit the number of chunks per step (profiling only; marks the line as partial)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the 2.5 s back-to-back loops (accumulate, apply)")
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--splits", type=int, default=0)
    ap.add_argument("--workload", default=WORKLOAD,
                    help="synthetic workload (default: the 500-sequence 14B->32B build the metric is quoted on; "
                         "qwen8b_14b and ragged_long are the other head-local configurations)")
    ap.add_argument("--fullhead", type=int, default=0, metavar="CHUNKS",
                    help="time the full-head contrast statistics (config 3 shapes: 4 source layers x 8 heads per target "
                         "layer) on this many 50-sequence chunks and print its own JSON line")
    ap.add_argument("--multilayer", type=int, default=0, metavar="K",
                    help="time the head-local build over K selected layers per target layer (the paper's operating point is "
                         "K = 8) on one 50-sequence chunk plus the wide ridge solve, and print its own JSON line")
    ap.add_argument("--rope", action="store_true",
                    help="fit the key maps in content coordinates: rotary embedding (base 1e6, positions restart every "
                         "1024 tokens) removed inside the accumulate kernel; the JSON line says so in config")
    ap.add_argument("--selector", type=int, default=0, metavar="SETS",
                    help="time this many probe sets of the layer selector (one candidate source layer per target layer "
                         "each) on one 50-sequence chunk and print its own JSON line")
    ap.add_argument("--two-pass", action="store_true",
                    help="time the two-pass centred construction (means pass, centred accumulation, reduce, centred solve) "
                         "on the selected workload and print its own JSON line")
    ap.add_argument("--solve-case", action="store_true",
                    help="stand-alone ridge solve: 1024 synthetic systems of 129 x 129 with 128 right-hand sides at the three "
                         "lambdas (no traces resident); prints timings, no JSON line (profiling case)")
    ap.add_argument("--profile-tokens", type=int, default=0,
                    help="profiling case: run only the accumulate kernel (3 launches) and the apply kernel on this many "
                         "tokens of the same shapes, print timings, no JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_00891_b200 import binding as cb, parallel, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    wl = synth.workload(args.workload)
    alg_bytes, alg_flops = algorithmic_work(wl)
    n_chunks = args.chunks if args.chunks > 0 else wl.n_chunks
    sl, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    if args.solve_case:
        solve_case(cb, torch, wl, dev)
        return
    if args.profile_tokens > 0 and (args.fullhead > 0 or args.multilayer > 0):
        import dataclasses                      # small case of the wide-regressor kernels for ncu
        T = args.profile_tokens
        wl = dataclasses.replace(wl, seq_lens=(1024,) * (T // 1024) + ((T % 1024,) if T % 1024 else ()), seqs_per_chunk=10 ** 6)
    elif args.profile_tokens > 0:
        profile_case(args, cb, synth, torch, wl, sl, sh, dev)
        return
    if args.fullhead > 0:
        fullhead_case(args, cb, synth, torch, wl, sl, sh, dev)
        return
    if args.multilayer > 0:
        multilayer_case(args, cb, synth, torch, wl, sl, sh, dev)
        return
    if args.selector > 0:
        selector_case(args, cb, synth, torch, wl, dev)
        return
    if args.two_pass and args.profile_tokens <= 0:
        two_pass_case(args, cb, synth, torch, wl, sl, sh, dev)
        return
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=args.flags, n_splits=args.splits)
    ctx = cb.cb_create(prob, device=dev)
    law = synth.map_law(wl, dev)
    p, d, nl = wl.d + 1, wl.d, len(wl.lambdas)
    G = torch.empty(wl.n_maps, p, p, device=dev)
    C = torch.empty(wl.n_maps, p, d, device=dev)
    m0, m1 = parallel.shard_range(wl.n_maps, rank, world)
    Wb = torch.empty(nl, m1 - m0, p, d, device=dev)
    info = torch.empty(nl, m1 - m0, dtype=torch.int32, device=dev)

    # Weak scaling: every rank streams its own 500-sequence set (chunk seeds offset by rank); one exchange sums
    # the statistics; the maps are solved in per-rank slices and gathered.
    def ev():
        return torch.cuda.Event(enable_timing=True)

    def one_step():
        """Returns (accumulate ms list, reduce ms, exchange+solve ms) for one full build."""
        cb.cb_stats_reset(ctx)
        acc_ev = []
        for c in range(n_chunks):
            ch = synth.make_chunk(wl, c + 1000 * rank, sl, sh, device=dev, law=law)      # untimed: trace collection
            e0, e1 = ev(), ev()
            pos = (torch.arange(ch["n_tokens"], dtype=torch.int32, device=dev) % 1024) if args.rope else None
            e0.record()
            if args.rope:
                cb.cb_stats_accumulate_rope(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"],
                                            pos, 1e6, 1e6)
            else:
                cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
            e1.record()
            acc_ev.append((e0, e1))
            e1.synchronize()
            del ch
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        n = cb.cb_stats_reduce(ctx, G, C)
        e1.record()
        n = parallel.exchange_statistics(G, C, n)
        cb.cb_ridge_solve(G[m0:m1], C[m0:m1], n, wl.lambdas, 0, Wb, info)
        full = parallel.gather_maps(Wb, wl.n_maps)
        e2.record()
        e2.synchronize()
        return [a.elapsed_time(b) for a, b in acc_ev], e0.elapsed_time(e1), e1.elapsed_time(e2), full

    for _ in range(args.warmup):
        one_step()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = cb.cb_launch_count()
    acc_ms, red_ms, sol_ms, step_ms = [], [], [], []
    for _ in range(args.steps):
        a, r, s, full = one_step()
        acc_ms.extend(a)
        red_ms.append(r)
        sol_ms.append(s)
        step_ms.append(sum(a) + r + s)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    launches = cb.cb_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    cb.cb_device_status(ctx)
    cb.cb_check_info(info)

    total_ms = torch.tensor([sum(step_ms)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    tokens_per_step = sum(wl.chunk_tokens(c) for c in range(n_chunks))
    value = world * tokens_per_step * args.steps / (total_ms / 1e3)

    # ---- online apply (reported beside the build, not part of the step) ----
    apply_info = None
    sustained = None
    if rank == 0:
        T = wl.apply_tokens or 32768
        src = synth.make_source_cache(wl, T, dev, law)
        out_k = torch.empty(wl.Lt, T, wl.Ht, d, dtype=torch.bfloat16, device=dev)
        out_v = torch.empty_like(out_k)
        Wfull = full[min(1, nl - 1)].contiguous()
        apos = torch.arange(T, dtype=torch.int32, device=dev)

        def do_apply():
            if args.rope:
                cb.cb_apply_rope(prob, Wfull, src[0], src[1], out_k, out_v, apos, 1e6, 1e6)
            else:
                cb.cb_apply(prob, Wfull, src[0], src[1], out_k, out_v)

        for _ in range(3):
            do_apply()
        ts = []
        for _ in range(5):
            e0, e1 = ev(), ev()
            e0.record()
            do_apply()
            e1.record()
            e1.synchronize()
            ts.append(e0.elapsed_time(e1))
        abytes = 2 * (wl.Ls * wl.Hs + wl.Lt * wl.Ht) * T * d * 2
        apply_info = {"tokens": T, "ms": statistics.median(ts), "tokens_per_s": T / (statistics.median(ts) / 1e3),
                      "algorithmic_gb": abytes / 1e9, "gbs": abytes / 1e9 / (statistics.median(ts) / 1e3)}
        apply_info["frac"] = apply_info["gbs"] / measured_peaks()["hbm_gbs"]
        # the sustained loops come after both burst figures: they leave the board hot and its clock low
        # ---- sustained figure of the dominant kernel: one resident chunk, back-to-back launches for >= 2.5 s ----
        sustained = None
        if not args.no_sustained:
            ch = synth.make_chunk(wl, 0, sl, sh, device=dev, law=law)
            spos = (torch.arange(ch["n_tokens"], dtype=torch.int32, device=dev) % 1024) if args.rope else None
            cb.cb_stats_reset(ctx)

            def acc_launch():
                if args.rope:
                    cb.cb_stats_accumulate_rope(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"],
                                                spos, 1e6, 1e6)
                else:
                    cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])

            sustained = sustained_loop(torch, local, acc_launch)
            sustained["tokens_per_launch"] = int(ch["n_tokens"])
            cb.cb_device_status(ctx)
            del ch
        if not args.no_sustained:
            sa = sustained_loop(torch, local, do_apply)
            sa["gbs"] = abytes / 1e9 / (sa["ms_per_launch"] / 1e3)
            sa["frac"] = sa["gbs"] / measured_peaks()["hbm_gbs"]
            apply_info["sustained"] = sa
        cb.cb_last_device_status()
        del src, out_k, out_v

    # ---- end to end through the host-buffer entry point: H2D copies inside the timed region ----
    # every rank feeds its own GPU from its own pinned buffer; the job's figure is all ranks' tokens over the slowest rank
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, cb, synth, torch, wl, prob, ctx, sl, sh, law, dev, G, C, n_chunks)
        if world > 1:
            t_ms = torch.tensor([e2e["ms_per_step"]], dtype=torch.float64, device=dev)
            dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
            e2e["ms_per_step"] = float(t_ms.item())
            e2e["value"] = world * tokens_per_step / (e2e["ms_per_step"] / 1e3)
            e2e["h2d_bytes_per_step"] *= world
            e2e["d2h_bytes_per_step"] *= world
            e2e["note"] += "; all %d ranks at once, slowest rank's time" % world
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    peaks = measured_peaks()
    acc_avg = statistics.mean(acc_ms)
    tok_launch = tokens_per_step / n_chunks
    achieved = alg_bytes * tok_launch / 1e9 / (acc_avg / 1e3)
    roof = {"bound": "hbm", "kernel": "k_accum_ts<plain>", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"], "traffic": None,
            "ms_per_launch": acc_avg, "algorithmic_gb_per_launch": alg_bytes * tok_launch / 1e9,
            "tflops": alg_flops * tok_launch / 1e12 / (acc_avg / 1e3),
            "tensor_frac_of_burst": alg_flops * tok_launch / 1e12 / (acc_avg / 1e3) / peaks["bf16_tflops"]}
    if args.workload == WORKLOAD:
        # DRAM traffic of one launch from the ncu capture of an 8,192-token launch of the same shapes (summarised
        # under profiles/), scaled: the per-token part x tokens + the read-modify-write of
        # the partial slots per split, which does not grow with tokens
        n_splits = cb.cb_token_splits(prob)
        roof["traffic"] = TRAFFIC_DRAM_BYTES_PER_TOKEN * tok_launch + TRAFFIC_DRAM_BYTES_PER_SPLIT * n_splits
    if sustained is not None:
        # the same kernel at the board's power limit: algorithmic bytes of one launch / its time inside the loop
        sustained["achieved"] = alg_bytes * sustained["tokens_per_launch"] / 1e9 / (sustained["ms_per_launch"] / 1e3)
        sustained["frac"] = sustained["achieved"] / peaks["hbm_gbs"]
        sustained["note"] = ("back-to-back launches on one resident chunk; 'frac' above is the burst figure of the step "
                             "(each launch starts on an idle board because the next chunk is generated in between)")
        roof["sustained"] = sustained
    t_roof = max(alg_bytes * tokens_per_step / (peaks["hbm_gbs"] * 1e9),
                 alg_flops * tokens_per_step / (peaks["bf16_tflops"] * 1e12))
    ms_step = total_ms / args.steps
    cpu = None
    if not args.no_cpu and world == 1:          # the oracle is timed beside the one-GPU run only
        import oracle
        dt, token_maps, rate = oracle_sample(262144)
        cpu = {"value": rate, "unit": "tokens/s", "cores": oracle.n_threads(), "kind": "oracle",
               "sample": "64 maps x 262144 tokens of the same trace law (statistics + 3 solves) in %.1f s; "
                         "tokens/s = token-maps / 1024 maps / s" % dt}
    out = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": args.workload + (": %d seq, %d tokens, %d->%d layers x %d KV heads x %d, %d maps, lambda in %s"
                                                   % (len(wl.seq_lens), wl.n_tokens, wl.Ls, wl.Lt, wl.Ht, wl.d, wl.n_maps, list(wl.lambdas))
                                                   if n_chunks == wl.n_chunks else " PARTIAL (%d of %d chunks)" % (n_chunks, wl.n_chunks)),
                      "chunks_per_step": n_chunks, "tokens_per_chunk": int(tok_launch), "flags": args.flags,
                      "rope": bool(args.rope),
                      "l2": "inputs larger than L2 (%.1f GB per launch)" % (alg_bytes * tok_launch / 1e9),
                      "timed": "sum of CUDA-event regions: accumulate calls + reduce + exchange/solve; chunk generation untimed"},
           "s_per_500seq_build": ms_step / 1e3 * (wl.n_chunks / n_chunks) * (500.0 / len(wl.seq_lens)),
           "frac_of_roofline_whole_build": t_roof * 1e3 / ms_step,
           "breakdown_ms": {"accumulate": statistics.mean(acc_ms) * n_chunks, "reduce": statistics.mean(red_ms),
                            "solve_3_lambdas": statistics.mean(sol_ms)},
           "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "apply": apply_info,
           "gpu_launches": launches, "clocks": clocks}
    print(json.dumps(out))


def selector_case(args, cb, synth, torch, wl, dev):
    """Layer selector: probe sets with rotated layer pairing on one chunk (statistics, OLS fit, R^2, scores)."""
    import numpy as np
    sl0, sh = cb.cb_head_map_nearest(wl.Ls, wl.Hs, wl.Lt, wl.Ht)
    ch = synth.make_chunk(wl, 0, sl0, sh, device=dev)
    T, d, p = ch["n_tokens"], wl.d, wl.d + 1
    scores = torch.zeros(wl.Lt, wl.Ls, device=dev)
    G = torch.empty(wl.n_maps, p, p, device=dev)
    C = torch.empty(wl.n_maps, p, d, device=dev)
    Wb = torch.empty(1, wl.n_maps, p, d, device=dev)
    info = torch.empty(1, wl.n_maps, dtype=torch.int32, device=dev)
    r2 = torch.empty(wl.n_maps, device=dev)
    syy = torch.empty(wl.n_maps, d, device=dev)
    times = {"energy": None, "accumulate": [], "reduce_solve_r2": []}

    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1)

    for r in range(args.selector):
        sl = np.array([(int(sl0[l]) + r) % wl.Ls for l in range(wl.Lt)], np.int32)
        prob = cb.Problem(wl.Ls, wl.Hs, d, wl.Lt, wl.Ht, d, sl, sh)
        ctx = cb.cb_create(prob, device=dev)
        if r == 0:
            ws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=dev)
            cb.cb_means_reset(ctx, ws)

            def energy():
                cb.cb_means_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], ws)
                cb.cb_means_energy(ctx, ws, syy)
            times["energy"] = timed(energy)
        times["accumulate"].append(timed(lambda: cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"],
                                                                        ch["w_k"], ch["w_v"])))

        def rest():
            n = cb.cb_stats_reduce(ctx, G, C)
            cb.cb_ridge_solve(G, C, n, [0.0], 0, Wb, info)
            cb.cb_probe_r2(G, C, Wb[0], syy, n, 0.0, 0, r2)
            cb.cb_probe_scores(r2, wl.Lt, wl.Ht, sl, wl.Ls, scores)
        times["reduce_solve_r2"].append(timed(rest))
        cb.cb_device_status(ctx)
        del ctx
    cb.cb_check_info(info)
    sets = cb.cb_rank_layers(scores.cpu().numpy(), 1)
    acc, rest_ms = statistics.mean(times["accumulate"][1:] or times["accumulate"]), statistics.mean(times["reduce_solve_r2"])
    print(json.dumps({"workload": "layer selector, %s shapes, %d probe sets on one chunk of %d tokens" % (args.workload, args.selector, T),
                      "ms": {"target_energy_pass": times["energy"], "accumulate_per_set": acc, "reduce_solve_r2_per_set": rest_ms},
                      "s_all_layer_pairs_per_chunk": (times["energy"] + wl.Ls * (acc + rest_ms)) / 1e3,
                      "nearest_depth_ranked_first_for_layers": int(sum(int(sets[l][0]) == int(sl0[l]) for l in range(wl.Lt))),
                      "n_target_layers": wl.Lt}))


def two_pass_case(args, cb, synth, torch, wl, sl, sh, dev):
    """Two-pass centred construction: every chunk is read twice (means, then centred statistics)."""
    alg_bytes, alg_flops = algorithmic_work(wl)
    n_chunks = args.chunks if args.chunks > 0 else wl.n_chunks
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=args.flags, n_splits=args.splits)
    ctx = cb.cb_create(prob, device=dev)
    law = synth.map_law(wl, dev)
    d, nl = wl.d, len(wl.lambdas)
    ws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=dev)
    mu = torch.empty(wl.n_maps, 2 * d + 1, device=dev)
    A = torch.empty(wl.n_maps, d, d, device=dev)
    B = torch.empty(wl.n_maps, d, d, device=dev)
    Wb = torch.empty(nl, wl.n_maps, d + 1, d, device=dev)
    info = torch.empty(nl, wl.n_maps, dtype=torch.int32, device=dev)

    def timed(fn):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r = fn()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1), r

    def one_step():
        cb.cb_means_reset(ctx, ws)
        cb.cb_stats_reset(ctx)
        t = {"means": [], "accumulate": []}
        for c in range(n_chunks):
            ch = synth.make_chunk(wl, c, sl, sh, device=dev, law=law)
            if args.rope:
                pos = torch.arange(ch["n_tokens"], dtype=torch.int32, device=dev) % 1024
                t["means"].append(timed(lambda: cb.cb_means_accumulate_rope(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"],
                                                                            ch["tgt_v"], ch["w_k"], ch["w_v"], ws, pos,
                                                                            1e6, 1e6))[0])
            else:
                t["means"].append(timed(lambda: cb.cb_means_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"],
                                                                       ch["tgt_v"], ch["w_k"], ch["w_v"], ws))[0])
            del ch
        t["finalize"] = timed(lambda: cb.cb_means_finalize(ctx, ws, mu))[0]
        for c in range(n_chunks):
            ch = synth.make_chunk(wl, c, sl, sh, device=dev, law=law)
            if args.rope:
                pos = torch.arange(ch["n_tokens"], dtype=torch.int32, device=dev) % 1024
                t["accumulate"].append(timed(lambda: cb.cb_stats_accumulate_centered_rope(
                    ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], mu, pos, 1e6, 1e6))[0])
            else:
                t["accumulate"].append(timed(lambda: cb.cb_stats_accumulate_centered(
                    ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], mu))[0])
            del ch
        t["reduce"], n = timed(lambda: cb.cb_stats_reduce_centered(ctx, mu, A, B))
        t["solve"] = timed(lambda: cb.cb_ridge_solve_centered(A, B, mu, n, wl.lambdas, 0, Wb, info))[0]
        return t

    for _ in range(args.warmup):
        one_step()
    runs = [one_step() for _ in range(args.steps)]
    cb.cb_device_status(ctx)
    cb.cb_check_info(info)
    peaks = measured_peaks()
    tok_launch = sum(wl.chunk_tokens(c) for c in range(n_chunks)) / n_chunks
    means_ms = statistics.mean([x for r in runs for x in r["means"]])
    acc_ms = statistics.mean([x for r in runs for x in r["accumulate"]])
    step_ms = statistics.mean([sum(r["means"]) + r["finalize"] + sum(r["accumulate"]) + r["reduce"] + r["solve"] for r in runs])
    gb = alg_bytes * tok_launch / 1e9
    print(json.dumps({"workload": "two-pass centred construction%s, %s, %d chunks of %d tokens"
                      % (" with the rotary boundary" if args.rope else "", args.workload, n_chunks, tok_launch),
                      "ms_per_build": step_ms, "tokens_per_s": tok_launch * n_chunks / (step_ms / 1e3),
                      "breakdown_ms": {"means_per_chunk": means_ms, "finalize": statistics.mean([r["finalize"] for r in runs]),
                                       "accumulate_per_chunk": acc_ms, "reduce": statistics.mean([r["reduce"] for r in runs]),
                                       "solve": statistics.mean([r["solve"] for r in runs])},
                      "roofline_means": {"bound": "hbm", "kernel": "k_means", "achieved": gb / (means_ms / 1e3),
                                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gb / (means_ms / 1e3) / peaks["hbm_gbs"]},
                      "roofline_accumulate": {"bound": "hbm", "kernel": "k_accum_ts<centred>", "achieved": gb / (acc_ms / 1e3),
                                              "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gb / (acc_ms / 1e3) / peaks["hbm_gbs"]},
                      "frac_of_roofline_whole_build": 2 * alg_bytes * tok_launch * n_chunks / (peaks["hbm_gbs"] * 1e9) / (step_ms / 1e3)}))


def fullhead_case(args, cb, synth, torch, wl, sl, sh, dev):
    """Full-head contrast: statistics for the 4097-wide regressor on the same traces (compute-bound contrast)."""
    sets = cb.cb_fullhead_layer_sets(wl.Ls, wl.Lt, 4)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sets)
    pf, d = prob.pf, wl.d
    G = torch.zeros(2, wl.Lt, pf, pf, device=dev)
    C = torch.zeros(2, wl.Lt, wl.Ht, pf, d, device=dev)
    law = synth.map_law(wl, dev)
    ms = []
    for c in range(args.fullhead):
        ch = synth.make_chunk(wl, c, sl, sh, device=dev, law=law)
        wk, wv = ch["w_k"][:, 0].contiguous(), ch["w_v"][:, 0].contiguous()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_fullhead_stats_accumulate(prob, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], wk, wv, G, C)
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
        T = ch["n_tokens"]
        del ch
    peaks = measured_peaks()
    F = 32
    flops_dense = 2.0 * (2 * wl.Lt) * T * (pf * pf + wl.Ht * pf * d)              # definition: full G and every C
    fp, hpn = (F + 1) // 2, (wl.Ht + 1) // 2                                          # 2 x 2 blocked units: four products each
    units = fp * (fp + 1) // 2 + fp * hpn
    flops_issued = 2.0 * (2 * wl.Lt) * units * T * 4 * 128 * 128
    t = min(ms) / 1e3
    print(json.dumps({"workload": "full-head contrast, 14B->32B shapes, %d tokens per chunk" % T, "ms_per_chunk": ms,
                      "tokens_per_s": T / t, "dense_tflops": flops_dense / t / 1e12,
                      "issued_mma_tflops": flops_issued / t / 1e12,
                      "frac_of_bf16_peak_dense": flops_dense / t / 1e12 / peaks["bf16_tflops"],
                      "s_per_200_sequences": 4 * statistics.mean(ms) / 1e3}))


def multilayer_case(args, cb, synth, torch, wl, sl, sh, dev):
    """Head-local support over K selected layers (regressor width K*128 + 1): statistics of one chunk and the solve."""
    k = args.multilayer
    sets = cb.cb_fullhead_layer_sets(wl.Ls, wl.Lt, k)
    prob = cb.FullHeadProblem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sets)
    d = wl.d
    P = k * d + 1
    G = torch.zeros(wl.n_maps, P, P, device=dev)
    C = torch.zeros(wl.n_maps, P, d, device=dev)
    ch = synth.make_chunk(wl, 0, sl, sh, device=dev)
    T = ch["n_tokens"]
    ms = []
    for _ in range(2):
        G.zero_(); C.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_multilayer_stats_accumulate(prob, sh, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], G, C)
        e1.record()
        e1.synchronize()
        ms.append(e0.elapsed_time(e1))
    del ch
    if args.profile_tokens > 0:
        # profiling case: no solve (random maps of the right scale), the apply on the same number of tokens
        Wr = torch.randn(wl.n_maps, P, d, device=dev) / (P ** 0.5)
        src = synth.make_source_cache(wl, T, dev, synth.map_law(wl, dev))
        out_k = torch.empty(wl.Lt, T, wl.Ht, d, dtype=torch.bfloat16, device=dev)
        out_v = torch.empty_like(out_k)
        tt = []
        for i in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cb.cb_apply_multilayer(prob, sh, Wr, src[0], src[1], out_k, out_v)
            e1.record()
            e1.synchronize()
            tt.append(e0.elapsed_time(e1))
        cb.cb_last_device_status()
        print("profile case k=%d, %d tokens: statistics ms %s, apply ms %s" % (k, T, ms, tt), file=sys.stderr)
        return
    lams = list(wl.lambdas)
    nsys = len(lams) * wl.n_maps
    ws = torch.empty(cb.cb_ridge_solve_large_workspace_bytes(P, d, min(nsys, 3072)), dtype=torch.uint8, device=dev)
    Wb = torch.empty(len(lams), wl.n_maps, P, d, device=dev)
    info = torch.empty(len(lams), wl.n_maps, dtype=torch.int32, device=dev)
    ts = []
    for _ in range(2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_ridge_solve_large(G, C, T, lams, 0, Wb, info, ws)
        e1.record()
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    cb.cb_check_info(info)
    # online apply latency at the paper's prefix lengths (and a long cache)
    apply_ms = {}
    law = synth.map_law(wl, dev)
    for Tp in (128, 512, 1024, 32768):
        src = synth.make_source_cache(wl, Tp, dev, law)
        out_k = torch.empty(wl.Lt, Tp, wl.Ht, d, dtype=torch.bfloat16, device=dev)
        out_v = torch.empty_like(out_k)
        tt = []
        for i in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cb.cb_apply_multilayer(prob, sh, Wb[1], src[0], src[1], out_k, out_v)
            e1.record()
            e1.synchronize()
            if i >= 2:
                tt.append(e0.elapsed_time(e1))
        apply_ms[str(Tp)] = statistics.median(tt)
        del src, out_k, out_v
    fp = (k + 1) // 2                       # 2 x 2 blocked G units (four products) and C units (two rows x one target head)
    products = 4 * (fp * (fp + 1) // 2) + 2 * fp
    dense = 2.0 * wl.n_maps * T * (P * P + P * d)
    print(json.dumps({"apply_ms_by_prefix_tokens": apply_ms, "workload": "head-local over k=%d layers, 14B->32B shapes, P=%d, %d tokens" % (k, P, T),
                      "stats_ms_per_chunk": ms, "stats_tokens_per_s": T / (min(ms) / 1e3),
                      "issued_mma_tflops": 2.0 * wl.n_maps * products * T * 128 * 128 / (min(ms) / 1e3) / 1e12,
                      "dense_tflops": dense / (min(ms) / 1e3) / 1e12,
                      "frac_of_bf16_peak_dense": dense / (min(ms) / 1e3) / 1e12 / measured_peaks()["bf16_tflops"],
                      "solve_ms_%d_systems" % nsys: ts,
                      "solve_fp64_tflops": nsys * (P ** 3 / 3.0 + 2.0 * P * P * d) * 2 / (min(ts) / 1e3) / 1e12,
                      "s_per_128000_positions": 2.5 * min(ms) / 1e3 + min(ts) / 1e3}))


def solve_case(cb, torch, wl, dev):
    """The batched ridge solve alone on synthetic positive definite systems of the benchmark's shape."""
    g = torch.Generator(device=dev).manual_seed(7)
    p, d, n = wl.d + 1, wl.d, 4096
    X = torch.randn(wl.n_maps, 512, p, device=dev, generator=g)
    X[:, :, d] = 1.0
    G = (X.transpose(1, 2) @ X).contiguous()
    C = torch.randn(wl.n_maps, p, d, device=dev, generator=g)
    lams = list(wl.lambdas)
    Wb = torch.empty(len(lams), wl.n_maps, p, d, device=dev)
    info = torch.empty(len(lams), wl.n_maps, dtype=torch.int32, device=dev)
    ts = []
    for _ in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_ridge_solve(G, C, n, lams, 0, Wb, info)
        e1.record()
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    cb.cb_check_info(info)
    print("solve case: %d systems of order %d, %d right-hand sides: ms %s" % (len(lams) * wl.n_maps, p, d, ["%.3f" % t for t in ts]),
          file=sys.stderr)


def profile_case(args, cb, synth, torch, wl, sl, sh, dev):
    """A small case of the same kernels for ncu: same shapes and trace law, fewer tokens (inputs still > L2)."""
    import dataclasses
    T = args.profile_tokens
    small = dataclasses.replace(wl, seq_lens=(1024,) * (T // 1024) + ((T % 1024,) if T % 1024 else ()), seqs_per_chunk=10 ** 6)
    prob = cb.Problem(wl.Ls, wl.Hs, wl.d, wl.Lt, wl.Ht, wl.d, sl, sh, flags=args.flags, n_splits=args.splits)
    ctx = cb.cb_create(prob, device=dev)
    ch = synth.make_chunk(small, 0, sl, sh, device=dev)
    ts = []
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
        e1.record()
        e1.synchronize()
        ts.append(e0.elapsed_time(e1))
    cb.cb_device_status(ctx)
    p, d = wl.d + 1, wl.d
    if args.two_pass or args.rope:
        # the other accumulate variants on the same small case (two launches each), for ncu -k
        ws = torch.empty(cb.cb_means_workspace_bytes(prob), dtype=torch.uint8, device=dev)
        mu = torch.empty(wl.n_maps, 2 * d + 1, device=dev)
        pos = torch.arange(T, dtype=torch.int32, device=dev) % 1024
        tm, tc, tr = [], [], []
        cb.cb_means_reset(ctx, ws)
        for _ in range(2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cb.cb_means_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"], ws)
            e1.record()
            e1.synchronize()
            tm.append(e0.elapsed_time(e1))
        cb.cb_means_finalize(ctx, ws, mu)
        for fn, acc in ((lambda: cb.cb_stats_accumulate_centered(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"],
                                                                 ch["w_k"], ch["w_v"], mu), tc),
                        (lambda: cb.cb_stats_accumulate_rope(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"],
                                                             ch["w_k"], ch["w_v"], pos, 1e6, 1e6), tr)):
            cb.cb_stats_reset(ctx)
            for _ in range(2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                e1.synchronize()
                acc.append(e0.elapsed_time(e1))
        cb.cb_device_status(ctx)
        print("profile case: %d tokens, means ms %s, centred accumulate ms %s, rope accumulate ms %s" % (
            T, ["%.3f" % t for t in tm], ["%.3f" % t for t in tc], ["%.3f" % t for t in tr]))
        cb.cb_stats_reset(ctx)
        cb.cb_stats_accumulate(ctx, ch["src_k"], ch["src_v"], ch["tgt_k"], ch["tgt_v"], ch["w_k"], ch["w_v"])
    G = torch.empty(wl.n_maps, p, p, device=dev)
    C = torch.empty(wl.n_maps, p, d, device=dev)
    n = cb.cb_stats_reduce(ctx, G, C)
    Wb = torch.empty(1, wl.n_maps, p, d, device=dev)
    info = torch.empty(1, wl.n_maps, dtype=torch.int32, device=dev)
    cb.cb_ridge_solve(G, C, n, [1e-2], 0, Wb, info)
    out_k = torch.empty(wl.Lt, T, wl.Ht, d, dtype=torch.bfloat16, device=dev)
    out_v = torch.empty_like(out_k)
    ta = []
    for _ in range(2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        cb.cb_apply(prob, Wb[0], ch["src_k"], ch["src_v"], out_k, out_v)
        e1.record()
        e1.synchronize()
        ta.append(e0.elapsed_time(e1))
    if args.rope:
        pos = torch.arange(T, dtype=torch.int32, device=dev) % 4096
        tr = []
        for _ in range(2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cb.cb_apply_rope(prob, Wb[0], ch["src_k"], ch["src_v"], out_k, out_v, pos, 1e6, 1e6)
            e1.record()
            e1.synchronize()
            tr.append(e0.elapsed_time(e1))
        print("profile case: rope apply ms %s" % ["%.3f" % t for t in tr])
    torch.cuda.synchronize()
    print("profile case: %d tokens, accumulate ms %s (%.0f GB/s algorithmic), apply ms %s" % (
        T, ["%.3f" % t for t in ts], ALG_BYTES_PER_TOKEN * T / 1e9 / (min(ts) / 1e3), ["%.3f" % t for t in ta]))


def run_e2e(args, cb, synth, torch, wl, prob, ctx, sl, sh, law, dev, G, C, n_chunks):
    """The same build through cb_stats_accumulate_host: every chunk is copied from pinned host memory inside the
    timed region, and the fitted maps are read back.  One pinned chunk is reused for all chunk slots (same bytes
    moved per step as the full set; the machine's host memory need not hold 218 GB)."""
    ch = synth.make_chunk(wl, 0, sl, sh, device=dev, law=law)
    host = {k: v.cpu().pin_memory() for k, v in ch.items() if torch.is_tensor(v)}
    T = ch["n_tokens"]
    del ch
    torch.cuda.empty_cache()
    staging = torch.empty(cb.cb_staging_bytes(prob, T), dtype=torch.uint8, device=dev)
    p, d, nl = wl.d + 1, wl.d, len(wl.lambdas)
    Wb = torch.empty(nl, wl.n_maps, p, d, device=dev)
    info = torch.empty(nl, wl.n_maps, dtype=torch.int32, device=dev)
    Wb_host = torch.empty(Wb.shape, dtype=Wb.dtype).pin_memory()
    h2d = sum(host[k].numel() * host[k].element_size() for k in host) * n_chunks
    d2h = Wb.numel() * 4

    def step():
        cb.cb_stats_reset(ctx)
        for _ in range(n_chunks):
            cb.cb_stats_accumulate_host(ctx, host["src_k"], host["src_v"], host["tgt_k"], host["tgt_v"],
                                        host["w_k"], host["w_v"], staging)
        n = cb.cb_stats_reduce(ctx, G, C)
        cb.cb_ridge_solve(G, C, n, wl.lambdas, 0, Wb, info)
        Wb_host.copy_(Wb, non_blocking=True)

    step()
    torch.cuda.synchronize()
    k = max(1, min(args.steps, 2))
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(k):
        step()
    e1.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    ms = e0.elapsed_time(e1)
    return {"value": T * n_chunks * k / (ms / 1e3), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms / k, "wall_s": wall, "steps": k,
            "note": "one pinned 50-sequence chunk reused for every chunk slot; PCIe-bound"}


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the IndexMem decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Workload (N = 1): the 32-layer Llama-3-8B-shaped KV stack, batch 32, 16K-token context ingested in
eight 2048-token chunks with eviction to the budget B = 2048 after each, then decode steps with a
compression every token (tau = 1).  One "step" is one decode token for all 32 sequences through all
32 layers: projections, indexer scores, top-B selection, memory write, compaction, attention over
the retained entries and the gated memory readout.  Inputs and weights are seeded synthetic draws
(paper_2605_25475_b200/synth.py).

With N > 1 (torchrun) every rank runs its own replica on its own 32 sequences (the path has no
exchange step, so this is weak scaling without a data-path collective); time is the max over ranks.

One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_25475_b200 import synth

METRIC = "decode_step_tokens_per_s"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


# ----------------------------------------------------------------------------------------------
# algorithmic bytes: what one decode step has to touch in HBM (K/V cache, memory state, indexer keys, weights, inputs and outputs)
def algorithmic_bytes(wl: synth.Workload):
    # entries a step reads, averaged over the phases of a compression interval: B + 1 + p in phase p (tau = 1: B + 1)
    n = wl.B + (wl.tau + 1) / 2
    weights = 2 * (wl.HI * wl.dI * wl.D + wl.dI * wl.D + wl.HI * wl.D + wl.dM * wl.D + wl.D) + 4 * wl.dM * wl.Dkv
    kv = n * 2 * wl.Dkv * 2
    state = 4 * wl.dM * wl.Dkv + 4 * wl.dM
    kidx = n * wl.dI * 2
    io = (5 * wl.D + 4 * wl.Dkv) * 2
    evict = 4 * wl.dM + 2 * wl.Dkv + 4 * wl.Dkv
    per_seq = kv + state + kidx + io + evict
    per_layer = weights + wl.n_seq * per_seq
    # the attention kernel streams the entries cached before the call: B at tau = 1, B + p in phase p otherwise
    # (B again in the phase that compresses, where it runs after the compaction)
    attn = wl.n_seq * (wl.B + (wl.tau - 1) * (wl.tau - 2) / (2 * wl.tau)) * 2 * wl.Dkv * 2
    return {"step": wl.n_layers * per_layer, "attn_launch": attn, "readout_launch": wl.n_seq * state,
            "per_seq": per_seq, "weights": weights}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons.  Started before the warm-up (the tool needs a few hundred
    milliseconds to come up); `stop(t0, t1)` keeps the samples whose time stamp falls into the timed region."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx, self.proc, self.path = gpu_index, None, f"/tmp/indexmem_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.idx), "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0=None, t1=None):
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]), [nm for nm, val in zip(names, parts[5:9]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        try:
            os.remove(self.path)
        except OSError:
            pass
        inside = [r for r in rows if t0 is not None and t0 <= r[0] <= t1]
        out["samples_total"] = len(rows)
        if not inside and rows and t0 is not None:
            # the region was shorter than the sampling interval: the samples nearest to it
            inside = sorted(rows, key=lambda r: min(abs(r[0] - t0), abs(r[0] - t1)))[:2]
            out["note"] = "no sample fell into the timed region; the two nearest are reported"
        if t0 is None:
            inside = rows
        if inside:
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside), samples=len(inside))
        out["reasons"] = sorted({nm for r in inside for nm in r[3]})
        return out


# ----------------------------------------------------------------------------------------------
def build_context(wl: synth.Workload, device, ingest=True, log=lambda *a: None, chunk_outputs=0, score_share=0, pending_slots=0):
    from paper_2605_25475_b200 import binding as im
    g = im.IndexMem(im.Config(n_layers=wl.n_layers, max_seqs=wl.n_seq, n_q_heads=wl.H, n_kv_heads=wl.Hkv,
                              head_dim=wl.d, budget=wl.B, compress_interval=wl.tau, max_chunk=wl.chunk,
                              n_sink=wl.n_sink, chunk_outputs=chunk_outputs, score_share=score_share,
                              pending_slots=pending_slots), device)
    ids = list(range(wl.n_seq))
    for layer in range(wl.n_layers):
        g.set_weights(layer, {k: v.cpu() for k, v in synth.make_weights(wl, layer, device).items()})
    if ingest:
        t0 = time.time()
        for c in range(wl.ctx // wl.chunk):
            for layer in range(wl.n_layers):
                X, Qp, _, K, V = synth.prefill_inputs(wl, layer, c, device)
                g.prefill_chunk(layer, ids, X, Qp, K, V)
            torch.cuda.synchronize()
            log(f"ingested chunk {c + 1}/{wl.ctx // wl.chunk} ({time.time() - t0:.1f}s)")
        assert g.status() == 0
    return g, ids


def decode_inputs_all(wl, n_steps, device):
    """[n_steps][5] tensors stacked over layers: x [L, n, D], q_pre, q [L, n, H, d], k, v [L, n, Hkv, d]."""
    steps = []
    for s in range(n_steps):
        parts = [synth.decode_inputs(wl, layer, s, device) for layer in range(wl.n_layers)]
        steps.append(tuple(torch.stack([p[i] for p in parts]).contiguous() for i in range(5)))
    return steps


def pick_workload(args):
    wl = synth.CONFIGS[args.workload]
    if args.layers or args.context:
        wl = wl.replace(n_layers=args.layers or wl.n_layers, ctx=args.context or wl.ctx)
    if getattr(args, "tau", 0):
        wl = wl.replace(tau=args.tau)
    return wl


def measure_decode(wl, device, steps, warmup, graph=True, rank=0, world=1, log=lambda *a: None, opts=None,
                   profile=True, e2e_args=None, score_share=0, steps_per_graph=1, stack_call=False, pending_slots=0):
    """Ingests the workload's context, then times `steps` decode steps (all layers, all sequences per step) replayed
    from CUDA graphs, inputs resident.  Returns the raw measurements; the context is closed before returning."""
    from paper_2605_25475_b200 import binding as im
    g, ids = build_context(wl, device, log=log, score_share=score_share, pending_slots=pending_slots)
    for opt, val in (opts or {}).items():
        im.im_set_option(g.ctx, opt, val)
    L = wl.n_layers
    n_in = min(8, steps + warmup)                                # distinct input sets, cycled
    inputs = decode_inputs_all(wl, n_in, device)
    out = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=device)

    all_layers = list(range(L))

    def one_step(k, stack=stack_call):
        x, qp, q, kk, v = inputs[k % n_in]
        if stack:        # the step's layers in one call (im_decode_stack): their inputs are all there, the layers overlap
            g.decode_stack(all_layers, ids, x, qp, q, kk, v, out)
            return
        for layer in range(L):
            g.decode_step(layer, ids, x[layer], qp[layer], q[layer], kk[layer], v[layer], out[layer])

    stream = torch.cuda.Stream(device)
    graphs = None
    tau = wl.tau
    n_graphs = n_in * tau // math.gcd(n_in, tau)                 # every (input set, phase of the interval) pair that occurs
    spg = steps_per_graph if (graph and tau == 1 and n_in % steps_per_graph == 0) else 1
    # (spg consecutive steps per captured graph: a one-layer workload stands for a model whose step holds many layer
    # calls in one graph, so the cost of a graph's boundary is spread as it would be there)
    res = {}
    sampler = ClockSampler(torch.cuda.current_device() if device.index is None else device.index)
    if rank == 0:
        sampler.start()                                          # before the warm-up: the tool takes a while to come up
    with torch.cuda.stream(stream):
        c0 = g.launch_count()
        for k in range(tau):                                     # one whole interval, eagerly: ends with n = B, phase 0
            one_step(k)
        res["launches_per_step"] = (g.launch_count() - c0) / tau
        stream.synchronize()
        if graph:
            # one captured step per input set and phase: the graph reads the resident inputs where they are; which
            # kernels a step launches depends on its phase (the last step of an interval compresses)
            graphs = []
            for k in range(0, n_graphs, spg):
                gk = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gk, stream=stream):
                    for j in range(spg):
                        one_step(k + j)
                graphs.append(gk)
        if graphs is not None and spg > 1:
            assert steps % spg == 0 and warmup % spg == 0
            step_fn = lambda k: graphs[(k // spg) % len(graphs)].replay() if k % spg == 0 else None
        else:
            step_fn = (lambda k: graphs[k % n_graphs].replay()) if graphs is not None else one_step
        for w in range(warmup):
            step_fn(w)
        stream.synchronize()
        barrier(world)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        rec0 = im.im_event_count(g.ctx, im.IM_COUNT_MERGE_RECOMPUTE)
        t_wall0 = time.time()
        ev0.record(stream)
        for s in range(steps):
            step_fn(warmup + s)
        ev1.record(stream)
        torch.cuda.synchronize()
        t_wall1 = time.time()
        barrier(world)
        ms = ev0.elapsed_time(ev1)
        res["recomputes"] = im.im_event_count(g.ctx, im.IM_COUNT_MERGE_RECOMPUTE) - rec0
        res["clocks"] = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
        assert g.status() == 0
        res["ms"] = max_over_ranks(ms, world, device)
        done = warmup + steps
        while done % tau:                                        # finish the interval (phase 0 again)
            step_fn(done)
            done += 1
        res["cuda_graph"] = graphs is not None
        res["steps_per_graph"] = spg

        if profile:
            # per-launch time of the dominant kernel: the same steps again, un-graphed, with the library recording
            # CUDA events around the attention launch on this stream - once in the concurrent schedule the timed steps
            # ran (the kernel next to the readout kernel and the chain of small kernels, on the SMs the schedule
            # leaves it), once with the side streams off (the kernel alone on all SMs, against the burst peak)
            # (with a stack call per step the first pass makes stack calls: the events then sit on the stream that
            # carries the attention kernels of all layers back to back)
            prof_steps = -(-min(steps, 32) // tau) * tau            # whole intervals
            for name, conc in (("in_step", 1), ("alone", 0)):
                im.im_set_option(g.ctx, im.IM_OPT_CONCURRENCY, conc)
                im.im_profile_begin(g.ctx, prof_steps * L)
                for s in range(prof_steps):
                    one_step(s, stack=stack_call and conc == 1)
                k_ms, k_n = im.im_profile_end(g.ctx)
                res["attn_ms_" + name], res["attn_n_" + name] = k_ms, k_n
            im.im_set_option(g.ctx, im.IM_OPT_CONCURRENCY, 1)
        if stack_call and graph and tau == 1:
            # the same steps as one im_decode_step call per layer (what a model whose layers depend on one another
            # would run), replayed from graphs of their own, for comparison in the same process
            lgraphs = []
            for k in range(n_in):
                gk = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gk, stream=stream):
                    one_step(k, stack=False)
                lgraphs.append(gk)
            n_cmp = min(steps, 64)
            for k in range(3):
                lgraphs[k % n_in].replay()
            stream.synchronize()
            ev0.record(stream)
            for k in range(n_cmp):
                lgraphs[k % n_in].replay()
            ev1.record(stream)
            stream.synchronize()
            res["layer_calls_ms"] = max_over_ranks(ev0.elapsed_time(ev1), world, device) / n_cmp
            res["layer_calls_steps"] = n_cmp
            del lgraphs
            assert g.status() == 0
        if e2e_args is not None:
            # end to end: host buffers in, host buffer out, copies inside the timed region
            res["e2e"] = run_e2e(e2e_args, wl, g, ids, inputs, stream, world, device, stack_call=stack_call)
    del graphs
    g.close()
    return res


def run_ours(args, rank, world, device):
    from paper_2605_25475_b200 import binding as im
    wl = pick_workload(args)
    log = (lambda *a: print("[bench]", *a, file=sys.stderr, flush=True)) if rank == 0 else (lambda *a: None)
    opts = {}
    if args.decode_tensor >= 0:
        opts[im.IM_OPT_DECODE_TENSOR] = args.decode_tensor
    if args.readout_stages >= 0:
        opts[im.IM_OPT_READOUT_STAGES] = args.readout_stages
    if args.stack_reserved >= 0:
        opts[im.IM_OPT_STACK_RESERVED] = args.stack_reserved
    m = measure_decode(wl, device, args.steps, args.warmup, graph=bool(args.graph), rank=rank, world=world, log=log,
                       opts=opts, e2e_args=args, score_share=args.score_share, stack_call=bool(args.stack_call),
                       pending_slots=args.pending_slots)
    ms = m["ms"]
    tokens = wl.n_seq * args.steps * world
    ab = algorithmic_bytes(wl)
    peaks = measured_peaks()
    kernel = "k_attn_stream_tc" if opts.get(im.IM_OPT_DECODE_TENSOR, 0) else "k_attn_stream"

    def rate(k_ms, k_n):
        sec = k_ms / max(k_n, 1) * 1e-3
        return {"us_per_launch": sec * 1e6, "achieved": ab["attn_launch"] / sec / 1e9,
                "frac": ab["attn_launch"] / sec / 1e9 / peaks["hbm_gbs"]}
    alone, in_step = rate(m["attn_ms_alone"], m["attn_n_alone"]), rate(m["attn_ms_in_step"], m["attn_n_in_step"])
    if bool(args.stack_call) and wl.n_layers >= 2 and m["cuda_graph"]:
        # In the replayed step the attention kernels of the layers follow one another on one stream, so a launch takes at
        # most a layer's share of the step; the eager figure above carries the host's launch overheads on top.
        us = ms / args.steps / wl.n_layers * 1e3
        in_step["replayed_us_per_launch_at_most"] = us
        in_step["replayed_frac_at_least"] = ab["attn_launch"] / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]
    full = wl.name == "llama8b_stack" and not args.tau and not args.layers and not args.context
    stack = bool(args.stack_call) and wl.n_layers >= 2 and not args.score_share
    res = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name + ("" if not (args.layers or args.context) else " (reduced for profiling)")
                               + ("" if not args.tau else " (compression interval %d instead of the headline workload's)" % args.tau),
                   "layers": wl.n_layers, "batch_per_gpu": wl.n_seq, "q_heads": wl.H,
                   "kv_heads": wl.Hkv, "head_dim": wl.d, "context": wl.ctx, "budget": wl.B, "tau": wl.tau,
                   "cuda_graph": m["cuda_graph"], "score_share": args.score_share,
                   "pending_slots": args.pending_slots or 32,
                   "call": ("one im_decode_stack call per step: the inputs of all layers are resident when the step starts "
                            "(a stack driven from synthetic activations), so the call overlaps the layers"
                            if stack else "one im_decode_step call per layer"),
                   "l2": "inputs larger than L2 (each step streams %.1f GB)" % (ab["step"] / 1e9)},
        "hbm_gbs_step": ab["step"] / (ms / args.steps * 1e-3) / 1e9,
        "hbm_frac_step": ab["step"] / (ms / args.steps * 1e-3) / 1e9 / peaks["hbm_gbs"],
        "hbm_frac_step_nominal_8tbs": ab["step"] / (ms / args.steps * 1e-3) / 1e9 / 8000.0,
        "roofline": {"bound": "hbm", "kernel": kernel, "achieved": alone["achieved"], "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": alone["frac"], "peak_source": peaks["source"],
                     "schedule": "in order, the kernel alone on all SMs (side streams off, un-graphed, CUDA events around the launch)",
                     "traffic": args.traffic if full else None,
                     "traffic_source": ("profiles/k_attn_stream_llama8b_stack_2layers_ctx4096.md (ncu dram__bytes_read.sum + "
                                        "dram__bytes_write.sum of one launch of this size; a constant, not measured in this run)") if full else None,
                     "bytes_per_launch": ab["attn_launch"], "us_per_launch": alone["us_per_launch"],
                     "in_step": dict(in_step, schedule=(
                         "schedule of the timed steps: the attention kernels of the step's layers back to back on one stream, "
                         "next to the readout kernels and the small kernels of the layers in flight (un-graphed, CUDA events "
                         "around each launch on that stream)" if stack else
                         "concurrent schedule of the timed steps: the kernel on the SMs left by the front kernel, next to the "
                         "readout kernel (un-graphed, CUDA events around the launch)"))},
        "merge_recomputes_per_step": m["recomputes"] / args.steps,
        "layer_calls": ({"ms_per_step": m["layer_calls_ms"], "tokens_per_s": wl.n_seq * world / (m["layer_calls_ms"] * 1e-3),
                         "steps": m["layer_calls_steps"],
                         "note": "the same steps as one im_decode_step call per layer (layers in sequence, as in a model "
                                 "whose layers depend on one another), graph replay, same process"}
                        if "layer_calls_ms" in m else None),
        "e2e": m["e2e"], "gpu_launches": int(round(m["launches_per_step"] * args.steps)), "clocks": m["clocks"],
    }
    return res, wl


# ----------------------------------------------------------------------------------------------
# Secondary measurements: the other configurations, short runs, one entry each in the default line
def secondary_block(args, device, log):
    """Configurations 2-4 and the paper's compression interval on the headline stack, each a short run with its own
    oracle baseline.  None of them has a bandwidth target: 2 and 3 are bound by the latency of a call's kernel chain."""
    from paper_2605_25475_b200 import binding as im
    peaks = measured_peaks()
    out = {}
    for name, steps in (("llama8b_b1", 64), ("qwen7b_b8", 64)):
        wl = synth.CONFIGS[name]
        m = measure_decode(wl, device, steps, 8, log=log, profile=False, steps_per_graph=8)
        ab = algorithmic_bytes(wl)
        sec = m["ms"] / steps * 1e-3
        cpu, _ = oracle_sample(wl.replace(chunk=min(wl.chunk, 2048)), min(len(os.sched_getaffinity(0)), wl.n_seq), 48, log=log)
        out[name] = {"us_per_step": sec * 1e6, "tokens_per_s": wl.n_seq / sec, "steps": steps, "bytes_per_step": ab["step"],
                     "hbm_gbs": ab["step"] / sec / 1e9, "hbm_frac": ab["step"] / sec / 1e9 / peaks["hbm_gbs"],
                     "bound": "latency of the call's kernel chain (no bandwidth target)",
                     "config": {"layers": 1, "batch": wl.n_seq, "context": wl.ctx, "budget": wl.B, "tau": 1, "cuda_graph": True,
                                "steps_per_graph": m["steps_per_graph"]},
                     "cpu_baseline": cpu}
        log(f"secondary {name}: {sec * 1e6:.1f} us/step")
    # configuration 4: chunked prefill
    pre_args = argparse.Namespace(**vars(args))
    pre_args.steps, pre_args.warmup, pre_args.context = 8, 3, 0
    pf = run_prefill(pre_args, device)
    wl4 = synth.CONFIGS["mistral7b_prefill"]
    out["mistral7b_prefill"] = {
        "ms_per_prompt": pf["scoring"]["tensor_cores"]["ms_per_prompt"], "tokens_per_s": pf["scoring"]["tensor_cores"]["tokens_per_s"],
        "ms_per_prompt_with_outputs": pf["with_outputs"]["ms_per_prompt"],
        "scoring_kernel": {"name": "k_prefill_score_tc", "us_per_launch": pf["scoring"]["tensor_cores"]["us_per_launch"],
                           "tensor_pipe_active_pct": 10.0,
                           "tensor_pipe_source": "profiles/k_prefill_score_tc_mistral7b_prefill_ctx8192.md (ncu, not measured in this run)"},
        "config": {"layers": 1, "batch": 1, "prompt": wl4.ctx, "chunk": wl4.chunk, "budget": wl4.B},
        "cpu_baseline": oracle_prefill_sample(wl4, log)}
    log(f"secondary mistral7b_prefill: {out['mistral7b_prefill']['ms_per_prompt']:.2f} ms per prompt")
    # the paper's compression interval on the headline stack
    wl = synth.CONFIGS["llama8b_stack"].replace(tau=128)
    m = measure_decode(wl, device, 128, 128, log=log, profile=False, stack_call=True)
    ab = algorithmic_bytes(wl)
    sec = m["ms"] / 128 * 1e-3
    out["llama8b_stack_tau128"] = {
        "ms_per_step": sec * 1e3, "tokens_per_s": wl.n_seq / sec, "steps": 128, "bytes_per_step": ab["step"],
        "hbm_gbs": ab["step"] / sec / 1e9, "hbm_frac": ab["step"] / sec / 1e9 / peaks["hbm_gbs"],
        "config": {"layers": wl.n_layers, "batch": wl.n_seq, "context": wl.ctx, "budget": wl.B, "tau": 128, "cuda_graph": True,
                   "note": "one whole interval: 127 steps attend over B + p entries, one selects 128 entries per sequence"},
        "cpu_baseline": "as the headline line's (an oracle step costs the same per cached entry; the interval changes how many are cached)"}
    log(f"secondary tau=128: {sec * 1e3:.3f} ms/step")
    # reuse of one layer's indexer scores by the three layers that follow it (App. B of the paper)
    wl = synth.CONFIGS["llama8b_stack"]
    m = measure_decode(wl, device, 64, 4, log=log, profile=False, score_share=4)
    sec = m["ms"] / 64 * 1e-3
    out["llama8b_stack_score_share4"] = {
        "ms_per_step": sec * 1e3, "tokens_per_s": wl.n_seq / sec, "steps": 64,
        "config": {"layers": wl.n_layers, "batch": wl.n_seq, "context": wl.ctx, "budget": wl.B, "tau": 1, "cuda_graph": True,
                   "score_share": 4,
                   "note": "layers 4k+1 .. 4k+3 make layer 4k's selection: no indexer projections, keys or scoring in 24 of 32 layers"}}
    log(f"secondary score_share=4: {sec * 1e3:.3f} ms/step")
    return out


def oracle_prefill_sample(wl, log):
    """The oracle on two 2048-token chunks of the prefill configuration (the second one at the steady-state size: 4096
    cached keys scored by 2048 queries, 2048 evictions)."""
    from oracle import indexmem_oracle as orc
    o = orc.OracleLayer(orc.OracleConfig(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, n_sink=wl.n_sink), 1)
    o.set_weights({k: synth.f32(v) for k, v in synth.make_weights(wl, 0).items()})
    ins = [tuple(synth.f32(t[0]) for t in synth.prefill_inputs(wl, 0, c)) for c in range(2)]
    o.prefill_chunk(0, ins[0][0], ins[0][1], ins[0][3], ins[0][4])
    t0 = time.time()
    o.prefill_chunk(0, ins[1][0], ins[1][1], ins[1][3], ins[1][4])
    dt = time.time() - t0
    return {"value": wl.chunk / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
            "sample": f"one steady-state chunk ({wl.chunk} tokens against {2 * wl.chunk} cached keys, {wl.chunk} evictions); {dt:.1f}s of CPU time on 1 thread"}


def run_prefill(args, device):
    """Profiling aid, not the headline metric: chunked prefill of the Mistral-shaped configuration
    (one layer, chunks of 2048 tokens into a budget of 2048), with the scoring kernel timed by the
    library's own CUDA events for both of its implementations (tensor cores / CUDA cores)."""
    from paper_2605_25475_b200 import binding as im
    wl = synth.CONFIGS["mistral7b_prefill"]
    if args.context:
        wl = wl.replace(ctx=args.context)
    g, ids = build_context(wl, device, ingest=False, chunk_outputs=1)
    if getattr(args, "prefill_pipeline", -1) >= 0:
        im.im_set_option(g.ctx, im.IM_OPT_PREFILL_PIPELINE, args.prefill_pipeline)
    n_chunks = wl.ctx // wl.chunk
    chunks = [synth.prefill_inputs(wl, 0, c, device) for c in range(min(n_chunks, 4))]
    stream = torch.cuda.Stream(device)
    HI, dI = max(1, wl.H // 4), wl.d // 8
    res = {"mode": "prefill", "metric": "prefill_tokens_per_s", "unit": "tokens/s", "n_gpus": 1,
           "steps": args.steps, "warmup": args.warmup, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": wl.name, "prompt": wl.ctx, "chunk": wl.chunk, "budget": wl.B, "layers": 1,
                      "n_seq": wl.n_seq}, "scoring": {}}
    with torch.cuda.stream(stream):
        for name, tensor in (("tensor_cores", 1), ("cuda_cores", 0)):
            im.im_set_option(g.ctx, im.IM_OPT_PREFILL_TENSOR, tensor)
            im.im_set_option(g.ctx, im.IM_OPT_PROFILE_TARGET, 1)

            def one_pass():
                g.reset()
                for c in range(n_chunks):
                    X, Qp, _, K, V = chunks[c % len(chunks)]
                    g.prefill_chunk(0, ids, X, Qp, K, V)

            for _ in range(args.warmup):
                one_pass()
            stream.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(stream)
            for _ in range(args.steps):
                one_pass()
            assert g.status() == 0       # (also joins what the last call left running on the library's own streams)
            ev1.record(stream)
            stream.synchronize()
            ms = ev0.elapsed_time(ev1) / args.steps
            im.im_profile_begin(g.ctx, n_chunks)
            one_pass()
            k_ms, k_n = im.im_profile_end(g.ctx)
            assert g.status() == 0
            # steady-state chunk: B old keys that every query sees + the chunk's own keys under the causal mask
            pairs = wl.n_seq * (wl.B * wl.chunk + wl.chunk * (wl.chunk + 1) // 2)
            flops = 2.0 * pairs * HI * dI
            res["scoring"][name] = {"us_per_launch": k_ms / max(k_n, 1) * 1e3, "launches": k_n,
                                    "algorithmic_gflop_per_steady_launch": flops / 1e9,
                                    "ms_per_prompt": ms, "tokens_per_s": wl.n_seq * wl.ctx / (ms * 1e-3)}
        im.im_set_option(g.ctx, im.IM_OPT_PROFILE_TARGET, 0)
        # the same prompt with the layer outputs of every chunk's own queries (im_prefill_chunk_attend)
        im.im_set_option(g.ctx, im.IM_OPT_PREFILL_TENSOR, 1)
        out = torch.empty((wl.n_seq, wl.chunk, wl.H, wl.d), dtype=torch.bfloat16, device=device)

        def attend_pass():
            g.reset()
            for c in range(n_chunks):
                X, Qp, Q, K, V = chunks[c % len(chunks)]
                g.prefill_chunk_attend(0, ids, X, Qp, Q, K, V, out)

        for _ in range(args.warmup):
            attend_pass()
        stream.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(args.steps):
            attend_pass()
        ev1.record(stream)
        stream.synchronize()
        assert g.status() == 0
        ms_att = ev0.elapsed_time(ev1) / args.steps
        # attention flops of the prompt: query s of chunk c sees min(c * chunk, B) retained entries + s + 1 tokens
        pairs = sum(wl.chunk * min(c * wl.chunk, wl.B) + wl.chunk * (wl.chunk + 1) // 2 for c in range(n_chunks))
        res["with_outputs"] = {"ms_per_prompt": ms_att, "tokens_per_s": wl.n_seq * wl.ctx / (ms_att * 1e-3),
                               "attention_tflop_per_prompt": 4.0 * pairs * wl.H * wl.d * wl.n_seq / 1e12}
    res["value"] = res["scoring"]["tensor_cores"]["tokens_per_s"]
    res["ms_per_step"] = res["scoring"]["tensor_cores"]["ms_per_prompt"]
    return res


# dram__bytes_read.sum + dram__bytes_write.sum of one k_attn_stream launch (32 sequences, n = 2049 keys,
# 8 KV heads of 128), from the ncu capture summarised under profiles/; a launch has this size whatever
# the number of layers or the ingested context, so the figure needs no scaling.
ATTN_TRAFFIC_NCU = 272.0e6


def run_e2e(args, wl, g, ids, inputs, stream, world, device, stack_call=False):
    L = wl.n_layers
    n_in = len(inputs)
    # one pinned host buffer and one device buffer per input set / step: [L][x | q_pre | q | k | v] (bf16), so that a
    # layer's inputs travel in a single copy
    sizes = [t[0].numel() for t in inputs[0]]                     # elements per layer of x, q_pre, q, k, v
    per_layer = sum(sizes)
    host = []
    for inp in inputs:
        hb = torch.empty((L, per_layer), dtype=torch.bfloat16).pin_memory()
        off = 0
        for t, n in zip(inp, sizes):
            hb[:, off:off + n].copy_(t.reshape(L, n).cpu())
            off += n
        host.append(hb)
    dbuf = torch.empty((L, per_layer), dtype=torch.bfloat16, device=device)
    views, off = [], 0
    for t, n in zip(inputs[0], sizes):
        views.append([dbuf[layer, off:off + n].view(t.shape[1:]) for layer in range(L)])
        off += n
    dx, dqp, dq, dk, dv = views
    dout = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16, device=device)
    hout = torch.empty((L, wl.n_seq, wl.H, wl.d), dtype=torch.bfloat16).pin_memory()
    h2d = host[0].numel() * host[0].element_size()
    d2h = hout.numel() * hout.element_size()

    cs, ds = torch.cuda.Stream(device), torch.cuda.Stream(device)   # host-to-device / device-to-host copies
    tick = torch.zeros(L, device=device)
    ev_in = [torch.cuda.Event() for _ in range(L)]
    ev_out = [torch.cuda.Event() for _ in range(L)]
    ev_fork, ev_join = torch.cuda.Event(), torch.cuda.Event()

    # groups of consecutive layers, one stack call each: a short first group (its copy is the only one nothing hides)
    bounds = ([0, 2, 8] + list(range(16, L + 1, 8))) if (stack_call and L % 8 == 0 and L >= 16) else []
    if stack_call and getattr(args, "e2e_groups", ""):
        bounds = [int(b) for b in args.e2e_groups.split(",")]
        assert bounds[0] == 0 and bounds[-1] == L and all(b > a for a, b in zip(bounds, bounds[1:]))
    n_groups = max(len(bounds) - 1, 0)

    use_events = bool(stack_call and not getattr(args, "e2e_groups", "") and L >= 2)
    ev_done = [torch.cuda.Event() for _ in range(L)]
    if use_events:
        for e in ev_in + ev_done:
            e.record(stream)                             # (an event has a handle once it has been recorded)
        stream.synchronize()

    def enqueue_events(k):
        """One step made of ONE im_decode_stack_events call: every layer's inputs are copied in on the copy stream with
        an event behind them that the call makes the layer's kernels wait for, and every layer's output is copied out
        behind the event the call records for it, while the later layers run."""
        hb = host[k]
        ev_fork.record(stream)
        cs.wait_event(ev_fork)
        ds.wait_event(ev_fork)
        with torch.cuda.stream(cs):
            for layer in range(L):
                dbuf[layer].copy_(hb[layer], non_blocking=True)
                tick[layer:layer + 1].fill_(1.0)         # (see below: the calls depend on a kernel, not on the copy node)
                ev_in[layer].record(cs)
        g.decode_stack(list(range(L)), ids, dx, dqp, dq, dk, dv, dout, ready_events=ev_in, done_events=ev_done)
        with torch.cuda.stream(ds):
            for layer in range(L):
                ds.wait_event(ev_done[layer])
                hout[layer].copy_(dout[layer], non_blocking=True)
            ev_join.record(ds)
        ev_cs = ev_out[0]
        ev_cs.record(cs)
        stream.wait_event(ev_cs)
        stream.wait_event(ev_join)

    def enqueue_groups(k):
        """One step made of stack calls over groups of consecutive layers: the inputs of group g + 1 are copied in and
        the outputs of group g - 1 copied out while the stack call of group g runs."""
        hb = host[k]
        ev_fork.record(stream)
        cs.wait_event(ev_fork)
        ds.wait_event(ev_fork)
        for gi in range(n_groups):
            a, b = bounds[gi], bounds[gi + 1]
            with torch.cuda.stream(cs):
                dbuf[a:b].copy_(hb[a:b], non_blocking=True)
                tick[gi:gi + 1].fill_(1.0)           # (see below: the calls depend on a kernel, not on the copy node)
                ev_in[gi].record(cs)
            stream.wait_event(ev_in[gi])
            g.decode_stack(list(range(a, b)), ids, dx[a:b], dqp[a:b], dq[a:b], dk[a:b], dv[a:b], dout[a:b])
            ev_out[gi].record(stream)
            ds.wait_event(ev_out[gi])
            with torch.cuda.stream(ds):
                hout[a:b].copy_(dout[a:b], non_blocking=True)
        ev_join.record(ds)
        stream.wait_event(ev_join)

    def enqueue(k):
        """One step: the copies of layer l + 1's inputs and of layer l - 1's outputs run next to layer l's
        kernels (three streams, forked from and joined back into `stream`, so that it can be captured)."""
        if use_events:
            return enqueue_events(k)
        if n_groups:
            return enqueue_groups(k)
        hb = host[k]
        ev_fork.record(stream)
        cs.wait_event(ev_fork)
        ds.wait_event(ev_fork)
        for layer in range(L):
            with torch.cuda.stream(cs):
                dbuf[layer].copy_(hb[layer], non_blocking=True)
                # a one-element kernel behind the copy: the layer's kernels then depend on a kernel of the copy
                # stream, not on the copy-engine node itself (in a captured graph a kernel that depends directly
                # on a copy node starts about 10 us late, per layer, even when the copy ended long before)
                tick[layer:layer + 1].fill_(1.0)
                ev_in[layer].record(cs)
            stream.wait_event(ev_in[layer])
            g.decode_step(layer, ids, dx[layer], dqp[layer], dq[layer], dk[layer], dv[layer], dout[layer])
            ev_out[layer].record(stream)
            ds.wait_event(ev_out[layer])
            with torch.cuda.stream(ds):
                hout[layer].copy_(dout[layer], non_blocking=True)
        ev_join.record(ds)
        stream.wait_event(ev_join)

    # The step as a user would run it in a serving loop: host-to-device copies, the 32 layer calls and the
    # device-to-host copy of the outputs, captured once per input set into a CUDA graph (the pinned host
    # buffers are the graph's sources and destination) and replayed; without --graph the same work is enqueued
    # call by call.
    tau = wl.tau
    n_graphs = n_in * tau // math.gcd(n_in, tau)                 # one per (input set, phase of the interval) pair
    graphs = None
    if args.graph:
        for k in range(tau):                                     # one whole interval eagerly before capturing
            enqueue(k % n_in)
        stream.synchronize()
        graphs = []
        for k in range(n_graphs):
            gk = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gk, stream=stream):
                enqueue(k % n_in)
            graphs.append(gk)

    def step(s):
        if graphs is not None:
            graphs[s % n_graphs].replay()
        else:
            enqueue(s % n_in)
        stream.synchronize()                                     # the caller has the step's result on the host

    n_warm = min(3, args.warmup)
    for s in range(n_warm):
        step(s)
    barrier(world)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for s in range(args.steps):
        step(n_warm + s)
    ev1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    ms = max_over_ranks(ev0.elapsed_time(ev1), world, device)
    return {"value": wl.n_seq * args.steps * world / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms / args.steps, "cuda_graph": graphs is not None,
            "calls_per_step": ("one im_decode_stack_events call: a ready event per layer behind its input copy, a done event per layer "
                               "ahead of its output copy") if use_events else
                              ("%d im_decode_stack calls over %s layers" % (n_groups, ", ".join(str(bounds[i + 1] - bounds[i]) for i in range(n_groups))))
                              if n_groups else "%d im_decode_step calls" % L}


# ----------------------------------------------------------------------------------------------
def oracle_sample(wl, n_units, n_steps, log=lambda *a: None):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: n_units sequences of
    layer 0, cache brought to the budget by ingesting two chunks (a decode step's cost depends on
    B and the widths, not on how much context was ingested before), n_steps decode steps timed."""
    from oracle import indexmem_oracle as orc
    sub = wl.replace(n_seq=n_units)
    o = orc.OracleLayer(orc.OracleConfig(H=wl.H, Hkv=wl.Hkv, d=wl.d, B=wl.B, tau=wl.tau, n_sink=wl.n_sink), n_units)
    o.set_weights({k: synth.f32(v) for k, v in synth.make_weights(wl, 0).items()})
    ids = list(range(n_units))
    t0 = time.time()
    for c in range(2 if wl.ctx // wl.chunk >= 2 else 1):
        X, Qp, _, K, V = synth.prefill_inputs(sub, 0, c)
        o.prefill_batch(ids, synth.f32(X), synth.f32(Qp), synth.f32(K), synth.f32(V))
    log(f"oracle sample set up in {time.time() - t0:.1f}s")
    ins = [tuple(synth.f32(t) for t in synth.decode_inputs(sub, 0, s)) for s in range(n_steps)]
    t0 = time.time()
    for s in range(n_steps):
        x, qp, q, k, v = ins[s]
        o.decode_batch(ids, x, qp, q, k, v)
    dt = time.time() - t0
    cores = min(n_units, len(os.sched_getaffinity(0)))
    unit_steps = n_units * n_steps
    # one unit-step = one token of one sequence through one layer; a full token crosses n_layers layers
    tok_s = unit_steps / wl.n_layers / dt
    return {"value": tok_s, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n_units} sequences x 1 layer x {n_steps} decode steps at n=B={wl.B} "
                      f"(cache filled by two {wl.chunk}-token chunks), scaled by 1/{wl.n_layers} layers to whole tokens; "
                      f"{dt:.1f}s of CPU time on {cores} threads"}, dt


def run_reference(args, rank, world):
    wl = pick_workload(args)
    if rank != 0:
        return None
    from oracle import indexmem_oracle as orc
    orc.build()
    n_units = min(len(os.sched_getaffinity(0)), wl.n_seq, 8)
    # each "step" of this arm is one decode step of the sample; keep the whole run to a few minutes
    steps = max(1, min(args.steps, 64))
    base, dt = oracle_sample(wl, n_units, steps,
                             log=lambda *a: print("[bench]", *a, file=sys.stderr, flush=True))
    ab = algorithmic_bytes(wl)
    return {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * wl.n_seq / base["value"],
            "extrapolated": True,
            "extrapolation": (f"timed: {n_units} sequences x 1 layer x {steps} decode steps ({dt:.1f} s on the host cores); value and "
                              f"ms_per_step are that rate scaled to {wl.n_seq} sequences x {wl.n_layers} layers (units are independent)"),
            "timed_seconds": dt,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name + ("" if not (args.layers or args.context) else " (reduced for profiling)")
                                   + ("" if not args.tau else " (compression interval %d instead of the headline workload's)" % args.tau),
                       "layers": wl.n_layers, "batch_per_gpu": wl.n_seq, "q_heads": wl.H, "kv_heads": wl.Hkv, "head_dim": wl.d,
                       "context": wl.ctx, "budget": wl.B, "tau": wl.tau, "cuda_graph": False, "score_share": args.score_share,
                       "call": "the CPU oracle's decode step, one (layer, sequence) unit after the other on the host cores",
                       "l2": "inputs larger than L2 (each step streams %.1f GB)" % (ab["step"] / 1e9)},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


# ----------------------------------------------------------------------------------------------
_dist = None


def barrier(world):
    if world > 1:
        _dist.barrier()


def max_over_ranks(ms, world, device):
    if world == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    _dist.all_reduce(t, op=_dist.ReduceOp.MAX)
    return float(t.item())


def main():
    global _dist
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_stack", choices=sorted(synth.CONFIGS))
    ap.add_argument("--mode", default="decode", choices=["decode", "prefill"],
                    help="prefill: profiling aid that times the chunked prefill and its scoring kernel (1 GPU)")
    ap.add_argument("--graph", type=int, default=1, help="replay the step from a CUDA graph")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the short runs of the other configurations that the default line carries in `secondary`")
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: run only this many layers (not the headline workload)")
    ap.add_argument("--context", type=int, default=0, help="profiling aid: ingest only this many context tokens")
    ap.add_argument("--tau", type=int, default=0,
                    help="decode with this compression interval (the paper reports 128) instead of the workload's; "
                         "one CUDA graph per phase of the interval is captured")
    ap.add_argument("--decode-tensor", type=int, default=-1,
                    help="1 / 0: decode attention on the tcgen05 kernel / the mma.sync kernel (default: the library's choice)")
    ap.add_argument("--score-share", type=int, default=0,
                    help="g >= 2: layers l with l %% g != 0 reuse the indexer scores of layer l - l %% g (the paper's appendix uses 4)")
    ap.add_argument("--readout-stages", type=int, default=-1,
                    help="0: readout on plain loads; k >= 1: on a ring of k 32 KB bulk copies per CTA (default: the library's choice)")
    ap.add_argument("--stack-call", type=int, default=1,
                    help="1: a step is one im_decode_stack call over all layers (the layers overlap); 0: one im_decode_step call per layer")
    ap.add_argument("--prefill-pipeline", type=int, default=-1,
                    help="--mode prefill: 0 = a chunk call leaves only its state update running when it returns; 1 (the library's "
                         "default) = everything behind its append kernel, so that the next chunk's projections run next to it")
    ap.add_argument("--pending-slots", type=int, default=0,
                    help="length F of the list of rank-one writes folded lazily into M (0: the library's default, 32)")
    ap.add_argument("--e2e-groups", default="",
                    help="end-to-end step: layer boundaries of its im_decode_stack calls, e.g. 0,2,8,16,24,32 (the default for 32 layers)")
    ap.add_argument("--stack-reserved", type=int, default=-1,
                    help="SMs a pipelined stack call keeps free of streaming blocks (default: the library's choice)")
    ap.add_argument("--traffic", type=float, default=ATTN_TRAFFIC_NCU,
                    help="DRAM bytes per launch of the dominant kernel from an ncu capture (reported as is)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        res = run_reference(args, rank, world)
        if res is not None:
            print(json.dumps(res), flush=True)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    if world > 1:
        import torch.distributed as dist
        _dist = dist
        dist.init_process_group("nccl", device_id=device)
    if args.mode == "prefill":
        if rank == 0:
            print(json.dumps(run_prefill(args, device)), flush=True)
        return
    res, wl = run_ours(args, rank, world, device)
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            from oracle import indexmem_oracle as orc
            orc.build()
            n_units = min(len(os.sched_getaffinity(0)), wl.n_seq, 8)
            res["cpu_baseline"], _ = oracle_sample(wl, n_units, 384,
                                                   log=lambda *a: print("[bench]", *a, file=sys.stderr, flush=True))
        else:
            res["cpu_baseline"] = None
        default_run = (world == 1 and args.workload == "llama8b_stack" and not (args.layers or args.context or args.tau)
                       and args.decode_tensor < 0 and args.readout_stages < 0 and not args.score_share)
        if default_run and not args.no_secondary:
            res["secondary"] = secondary_block(args, device, lambda *a: print("[bench]", *a, file=sys.stderr, flush=True))
        print(json.dumps(res), flush=True)
    if world > 1:
        _dist.destroy_process_group()


if __name__ == "__main__":
    main()

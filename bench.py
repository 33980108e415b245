#!/usr/bin/env python
"""Benchmark of the prune-and-rebatch hot path on B200.

A step is one pass of the whole path over one batch of synthetic input shaped like a GRPO/DAPO run:
  arrol_score_partial -> arrol_select -> arrol_compact (token ids + hidden rows) -> arrol_token_logprob.
`value` = survivor tokens processed per second over the whole step, inputs resident in HBM.
`e2e`   = the same metric through arrol_prune_rebatch_host: inputs in pinned host memory, results read back.
The headline workload is the largest one (Qwen-3-8B DAPO-shaped); `per_workload` carries the same figures for the
other four at a reduced step count.  `--impl reference` times the CPU oracle (the plain fp64 program the GPU path is
checked against) on host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "survivor_logprob_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "qwen3-8b-dapo"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic of one token_logprob launch per survivor token, by (d, V, vocabulary splits), from single-launch
# profiler captures on the small cases of the same d and V (the Llama-shaped and the DAPO-shaped one): (bytes read +
# bytes written) / tokens of the launch.  At fixed d, V and split count the traffic grows in proportion to the tokens
# of the launch.
LOGPROB_DRAM_BYTES_PER_TOKEN = {(2048, 128256, 2): 60090.0, (4096, 151936, 2): 155108.0}
# DRAM bytes per scored row of score_linear_kernel streamed over consecutive rows (same kind of capture)
SCORE_LINEAR_DRAM_BYTES_PER_ROW = {(2048, 2): 4129.8}


def logprob_traffic(w, T, splits, sm_count):
    """DRAM bytes of one token_logprob launch: the profiler capture scaled by tokens where one exists for this
    (d, V, splits), else the model the captures confirmed: every wave of resident blocks streams its W_vocab split
    once and every token tile is read once per split."""
    per_tok = LOGPROB_DRAM_BYTES_PER_TOKEN.get((w.d, w.V, splits))
    if per_tok is not None:
        return per_tok * T, "profiler capture on a small case of the same d, V and split count, scaled by tokens"
    return 2.0 * w.d * (splits + w.V * splits / (sm_count * 128.0)) * T, "model 2d(splits + V*splits/(SMs*128)) per token"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
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
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [v for v in sm if v >= 0.5 * max(sm)] or sm
        return {"sm_mhz": float(np.median(busy)), "sm_max_mhz": float(max(smax)), "reasons": sorted(reasons),
                "samples": len(sm)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def auto_prompt_chunks(w):
    """Smallest number of prompt chunks (a power of two) whose packed hidden rows, next to the resident source rows,
    stay under ~60 GB per chunk of source + packed rows."""
    from paper_2603_24840_b200 import synth
    ell = synth.lengths(w).astype(np.int64)
    rows = float(ell.sum()) * 1.6            # source rows + packed survivors (roughly 0.6 of the source)
    gb = rows * w.d * 2 / 1e9
    c = 1
    while gb / c > 60.0 and c < w.P:
        c *= 2
    while w.P % c != 0:
        c += 1
    return c


def config_of(w, C):
    """Static description of the workload: the same for the GPU arm and the reference arm."""
    from paper_2603_24840_b200 import synth
    T_src = int(synth.lengths(w).astype(np.int64).sum())
    esz = 4 if w.dtype == "f32" else 2
    big = T_src * w.d * esz > 126e6
    return {"workload": w.name, "prompt_chunks": C,
            "chunking": ("none" if C == 1 else
                         "all %d prompts' source rows are resident; a step runs %d chunks of %d consecutive prompts, each "
                         "chunk different prompts, back to back through one set of packed buffers (groups and tokens "
                         "are independent, so times add)" % (w.P, C, w.P // C)),
            "P": w.P, "G": w.G, "K": w.K, "cutoff": w.cutoff, "d": w.d, "V": w.V, "head_h": w.h,
            "source_rows": T_src,
            "l2": ("inputs larger than L2 (hidden rows %.2f GB, W_vocab %.2f GB)" if big else
                   "inputs SMALLER than L2 (hidden rows %.4f GB, W_vocab %.4f GB), L2 not flushed: a latency-bound "
                   "case, no roofline figure of it is meaningful") % (T_src * w.d * esz / 1e9, w.V * w.d * esz / 1e9)}


# ------------------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and the --impl reference arm)
# ------------------------------------------------------------------------------------------------------------
def scored_rows_of(w):
    """The N hidden rows at the detection length as the GPU arm sees them: the source rows are drawn by a seeded
    generator on the device that holds them, so they are regenerated there and the N rows copied back (generation
    only; nothing of the method runs on the device).  Without a CUDA device the rows are drawn on the host instead."""
    import torch
    from paper_2603_24840_b200 import synth
    ell = synth.lengths(w)
    off = synth.src_offsets(ell)
    ridx = torch.from_numpy(off[:-1] + (w.cutoff - 1))
    if torch.cuda.is_available():
        local = dist_env()[2]
        dev = torch.device("cuda", local)
        src = synth.hidden_states(w, int(off[-1]), device=dev)
        x = src[ridx.to(dev)].cpu()
        del src
        torch.cuda.empty_cache()
        return x, "the rows the GPU arm scores"
    return synth.hidden_states(w, w.N, stream=21), "rows drawn on the host (no CUDA device to regenerate the GPU arm's)"


_ORACLE_INPUTS = {}


def oracle_inputs(w):
    """Host-side inputs of the oracle for a workload (drawn once per process: the vocabulary weights alone take seconds)."""
    import torch
    from paper_2603_24840_b200 import synth
    if w.name not in _ORACLE_INPUTS:
        ell = synth.lengths(w)
        off = synth.src_offsets(ell)
        hist_s, hist_y = synth.calib_history(w)
        _ORACLE_INPUTS[w.name] = dict(
            ell=ell, off=off, rew=synth.rewards(w), head=synth.head_weights(w), tokens=synth.token_ids(w, int(off[-1])),
            hist_s=hist_s, hist_y=hist_y, Wv=synth.as_oracle_array(synth.vocab_weights(w, dtype=torch.bfloat16)))
    return _ORACLE_INPUTS[w.name]


def oracle_step_rate(w, budget_s: float, x_cut=None, logp_rows=None):
    """Times the oracle on the workload: head scoring, probability map, selection, scan, token gather and
    advantages at full size on the given cutoff rows; the fp64 log-softmax gather on a bounded sample of survivor
    tokens.  Returns (tokens_per_s for the whole path, description, cores, T)."""
    import torch
    import oracle
    from paper_2603_24840_b200 import synth

    inp = oracle_inputs(w)
    ell, off, rew, head, tokens = inp["ell"], inp["off"], inp["rew"], inp["head"], inp["tokens"]
    hist_s, hist_y, Wv = inp["hist_s"], inp["hist_y"], inp["Wv"]
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    if x_cut is None:
        x_cut = synth.hidden_states(w, w.N, stream=21)
    cores = oracle.num_threads()

    t0 = time.perf_counter()
    s = oracle.head_score(oa(x_cut), oa(head["W1"]), oa(head["b1"]), oa(head["w2"]), oa(head["b2"]), h=w.h)
    _, lut = oracle.build_q_lut(*oracle.calib_counts(hist_s, hist_y, w.B), 1.0)
    _, _, q = oracle.prob_map(s, lut)
    keep = oracle.select(q.astype(np.float32), w.P, w.G, w.K, w.rho)
    idx, cu, S, T = oracle.survivor_scan(keep, ell)
    dst_tokens, _, _ = oracle.gather(idx, cu, off[:-1], tokens)
    oracle.advantages(rew, keep, w.G)
    t_prune = time.perf_counter() - t0

    # log-prob sample: calibrate on one row per core, then size the sample to the budget
    probe = max(cores, 1)
    H = oa(synth.hidden_states(w, max(probe, 1), stream=22).to(torch.bfloat16))
    t0 = time.perf_counter()
    oracle.token_logprob(H, Wv, dst_tokens[:probe])
    t_probe = time.perf_counter() - t0
    per_row = t_probe / probe
    n = int(max(probe, min(T, (budget_s - t_probe) / max(per_row, 1e-9))))
    if logp_rows is not None:
        n = min(n, logp_rows)
    n = max(probe, (n // probe) * probe)
    H = oa(synth.hidden_states(w, n, stream=23).to(torch.bfloat16))
    t0 = time.perf_counter()
    oracle.token_logprob(H, Wv, dst_tokens[:n])
    t_logp = time.perf_counter() - t0
    per_tok = t_logp / n
    tokens_per_s = T / (t_prune + per_tok * T)
    sample = ("scoring/selection/scan/token-gather/advantages at full size (%.3f s); fp64 log-softmax gather on %d of "
              "%d survivor tokens (%.1f s), extrapolated per token" % (t_prune, n, T, t_logp))
    return tokens_per_s, sample, cores, int(T)


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    if world > 1:
        # torchrun exports OMP_NUM_THREADS=1 to every rank; the other ranks have exited, so rank 0 times the oracle on
        # all host cores, as the single-process run does
        try:
            import ctypes
            ctypes.CDLL("libgomp.so.1").omp_set_num_threads(len(os.sched_getaffinity(0)))
        except OSError:
            pass
    C = args.prompt_chunks if args.prompt_chunks > 0 else auto_prompt_chunks(w)
    x_cut, rows_note = scored_rows_of(w)
    vals, walls = [], []
    budget = max(2.0, min(30.0, 120.0 / max(1, args.steps + args.warmup)))
    sample, cores, T = "", 0, 0
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        v, sample, cores, T = oracle_step_rate(w, budget, x_cut=x_cut)
        if i >= args.warmup:
            vals.append(v)
            walls.append(time.perf_counter() - t0)
    value = float(np.mean(vals))
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(walls)) * 1e3,
        "ms_per_step_note": "wall time of one bounded-sample step; the whole workload would take survivor_tokens / value "
                            "seconds per step",
        "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, C),
        "counts": {"survivor_tokens": T},
        "note": "CPU oracle on host cores; each step a bounded sample; scored rows: " + rows_note,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------------------
def measure(w, C, K, W, local, barrier, rank, full, args):
    """All figures of one workload on this rank.  `full`: the headline workload (update and aux legs too)."""
    import torch
    from paper_2603_24840_b200 import binding as B
    from paper_2603_24840_b200.pipeline import PruneRebatch

    if C == 1:
        pr_full = PruneRebatch(w, device=local, with_rows=True)
        views = [pr_full]
    else:
        pr_full = PruneRebatch(w, device=local, with_rows=False)
        views = PruneRebatch.chunk_views(pr_full, C)
    ctx = pr_full.ctx
    stream = torch.cuda.current_stream()
    props = torch.cuda.get_device_properties(local)
    sm_count = props.multi_processor_count

    # ---- scoring kernel on its own, before any tensor-core work: a kernel timed alone, at the clocks a short kernel
    # gets (for about a second after a log-prob launch the SM clock stays where the power cap put it, and this
    # clock-sensitive streaming kernel measures 22 % less: 5.5 against 7.05 TB/s on the Llama-shaped source) ----
    torch.cuda.synchronize()
    time.sleep(1.0)
    views[0].prune_step(with_rows=False)
    score = score_times(views[0], pr_full, w, B, torch, stream, K)

    for _ in range(W):
        for v in views:
            v.step()
    barrier()
    counts = [v.counts() for v in views]
    S = sum(c[0] for c in counts)
    T = sum(c[1] for c in counts)
    B.arrol_poll_status(ctx)

    # ---- timed region: device-resident inputs, K steps of C chunk passes ----
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K * C)]
    # time stamps of the log-prob kernel's work items (last launch of the region): SM cycles per nanosecond
    max_items = max(((v.cap + 127) // 128) * B.arrol_token_logprob_splits(ctx, v.cap, w.d, w.V) for v in views)
    stamps = torch.zeros(max_items * 4, dtype=torch.int64, device=pr_full.dev)
    B.arrol_test_hook(ctx, B.HOOK_LOGPROB_TIMING_BUFFER, stamps.data_ptr())
    B.arrol_test_hook(ctx, B.HOOK_LOGPROB_TIMING_ITEMS, max_items)
    sampler = ClockSampler(local)
    launches0 = B.arrol_launch_count(ctx)
    if rank == 0:
        sampler.start()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(K):
        for c, v in enumerate(views):
            e = ev[k * C + c]
            e[0].record(stream)
            v.score_partial()
            e[1].record(stream)
            v.select()
            e[2].record(stream)
            v.compact()
            e[3].record(stream)
            v.token_logprob()
            e[4].record(stream)
    t_end.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    launches = B.arrol_launch_count(ctx) - launches0
    total_ms = t_start.elapsed_time(t_end)
    B.arrol_test_hook(ctx, B.HOOK_LOGPROB_TIMING_BUFFER, 0)
    B.arrol_poll_status(ctx)
    seg = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in ev])  # ms, per chunk pass
    seg_step = seg.reshape(K, C, 4).sum(1).mean(0)                                # ms per step, per call

    # effective SM clock inside the last log-prob launch, and the tensor-pipe fraction at that clock
    T_last = counts[-1][1]
    splits = B.arrol_token_logprob_splits(ctx, views[-1].cap, w.d, w.V)
    tiles_last = (T_last + 127) // 128
    st = stamps.cpu().numpy().reshape(-1, 4)
    st = st[st[:, 1] > st[:, 0]]                 # the work items of the last launch that left a stamp
    in_kernel = None
    if len(st) > 0:
        # the kernel runs as pairs of blocks on 256-row tiles (one stamp per pair) or as single blocks
        blocks_per_item = 2 if len(st) <= ((tiles_last + 1) // 2) * splits else 1
        ns = (st[:, 1] - st[:, 0]).astype(np.float64)
        cyc = (st[:, 3] - st[:, 2]).astype(np.float64) * blocks_per_item
        span_ns = float(st[:, 1].max() - st[:, 0].min())
        mhz = float(cyc.sum() / ns.sum() * 1e3) / blocks_per_item
        flops_last = 2.0 * T_last * w.d * w.V
        in_kernel = {
            "sm_mhz": mhz, "what": "sum of SM cycles / sum of nanoseconds over the work items of the region's last "
                                   "log-prob launch (clock64 and globaltimer read by the kernel; no clock control touched)",
            "blocks_per_work_item": blocks_per_item,
            "busy_cycles_per_sm": float(cyc.sum() / sm_count), "span_ms": span_ns / 1e6,
            "tensor_frac_at_clock": flops_last / (sm_count * 8192.0 * (span_ns * mhz * 1e-3)),
            "tensor_frac_of_busy_cycles": flops_last / (8192.0 * cyc.sum()),
            "note": "8192 dense bf16 flop per SM per cycle; at_clock uses the launch's whole span, of_busy_cycles only "
                    "the cycles between a work item's first and last accumulator"}
    del stamps

    # ---- the same step without any packed copy of the hidden rows (token-only compaction + gathered log-prob) ----
    K_in = max(1, min(K, 3))
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def in_place_step():
        pr_full.prune_step(with_rows=False)
        pr_full.token_logprob_gathered()

    in_place_step()
    barrier()
    T_in = pr_full.counts()[1]
    a.record(stream)
    for _ in range(K_in):
        in_place_step()
    b.record(stream)
    barrier()
    in_place_ms = a.elapsed_time(b) / K_in
    in_place = {"what": "score -> select -> compact (token ids, per-token outputs) -> arrol_token_logprob_gathered over "
                        "all %d prompts in one pass: the survivors' hidden rows are read in place, no [T, d] copy "
                        "exists" % w.P,
                "value": T_in / (in_place_ms * 1e-3), "unit": UNIT, "ms_per_step": in_place_ms, "steps": K_in,
                "survivor_tokens": T_in, "packed_rows_bytes_avoided": int(T_in) * w.d * 2}

    # ---- prune step on its own (one library call; token ids only / with hidden rows / replayed from a CUDA graph) ----
    prune_us = prune_step_times(views[0], B, torch, stream, K)
    if C > 1:
        prune_us["all_prompts"] = prune_step_times(pr_full, B, torch, stream, K, rows_too=False)
        prune_us["note"] = "per chunk of %d prompts; all_prompts: one call over all %d prompts" % (w.P // C, w.P)

    update = aux = None
    if full and not args.skip_update:
        try:
            update = run_update(views[0], views[0].w, B, torch, K)
            update["tokens"] = counts[0][1]
        except (RuntimeError, MemoryError) as exc:
            print("update leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)
        torch.cuda.empty_cache()
    if full and not args.skip_aux:
        try:
            views[0].step()
            aux = run_aux(views[0], views[0].w, B, torch, K)
        except (RuntimeError, MemoryError) as exc:
            print("aux leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)
        torch.cuda.empty_cache()

    # ---- e2e: host buffers through arrol_prune_rebatch_host, the same number of steps ----
    e2e = {"ms_per_step": float("nan"), "h2d": 0, "d2h": 0, "tokens": 0}
    if not args.skip_e2e:
        try:
            e2e = run_e2e(views, pr_full, w, C, K, B, torch, barrier)
        except (RuntimeError, MemoryError) as exc:   # e.g. the pinned host copy of the inputs does not fit
            print("e2e leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)

    # ---- the log-prob call with the kernel's OTHER form.  The library runs the kernel as pairs of blocks on 256-row
    # tiles (tcgen05 cta_group::2) where pairs need no more vocabulary splits than single blocks, else as one block per
    # 128-row tile (see include/arrol.h, ARROL_HOOK_LOGPROB_PAIR); this leg forces the form the step did not use ----
    other_kernel = None
    kernel_form = int(B.arrol_token_logprob_form(ctx, views[0].cap, w.d, w.V))
    try:
        if args.skip_pair:
            raise RuntimeError("left out on request")
        v = views[0]
        v.step()
        default_splits = B.arrol_token_logprob_splits(ctx, v.cap, w.d, w.V)
        B.arrol_test_hook(ctx, B.HOOK_LOGPROB_PAIR, 0 if kernel_form == 2 else 1)
        ws_alt = torch.empty(B.arrol_token_logprob_workspace(ctx, v.cap, w.d, w.V), dtype=torch.uint8, device=v.dev)
        lp_alt = torch.empty(v.cap, dtype=torch.float32, device=v.dev)
        call = lambda: B.arrol_token_logprob(ctx, v.dst_rows, v.W_vocab, v.dst_tokens, v.cap, w.d, w.V, lp_alt, ws_alt,
                                             d_T=v.d_num[1:])
        call()
        barrier()
        a.record(stream)
        for _ in range(K_in):
            call()
        b.record(stream)
        barrier()
        ms = a.elapsed_time(b) / K_in
        T_v = v.counts()[1]
        other_kernel = {"what": "arrol_token_logprob on %s with the kernel forced to its other form: %s" % (
                            "the step's survivors" if C == 1 else "one chunk's survivors",
                            "one block per 128-row tile (tcgen05 cta_group::1)" if kernel_form == 2 else
                            "pairs of blocks on 256-row tiles (tcgen05 cta_group::2)"),
                        "launch_ms": ms, "achieved": 2.0 * T_v * w.d * w.V / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                        "vocab_splits": int(B.arrol_token_logprob_splits(ctx, v.cap, w.d, w.V)),
                        # bit-equal whenever both forms use the same number of vocabulary splits (the split count
                        # fixes the order of the log-sum-exp merge); with other counts the difference is rounding
                        "default_kernel_vocab_splits": int(default_splits),
                        "bit_equal_to_default_kernel": bool(torch.equal(lp_alt[:T_v], v.logp[:T_v])),
                        "max_abs_diff_to_default_kernel": float((lp_alt[:T_v] - v.logp[:T_v]).abs().max()),
                        "note": "a short leg at the end of the run: compare it with the figures of other short legs, not "
                                "with the long timed region (the power cap settles lower over seconds)"}
        del ws_alt, lp_alt
    except (RuntimeError, B.ArrolError) as exc:
        print("other-form leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)
    finally:
        B.arrol_test_hook(ctx, B.HOOK_LOGPROB_PAIR, 2)

    res = {"w": w, "C": C, "S": S, "T": T, "K": K, "total_ms": total_ms, "seg_step": seg_step,
           "clocks": clocks, "launches": int(launches), "in_kernel": in_kernel, "in_place": in_place,
           "other_kernel": other_kernel, "kernel_form": kernel_form,
           "prune_us": prune_us, "score": score, "update": update, "aux": aux, "e2e": e2e, "splits": int(splits),
           "sm_count": sm_count, "T_src": pr_full.T_src, "N_chunk": views[0].w.N,
           "T_chunks": [c[1] for c in counts]}
    del views, pr_full, v
    gc.collect()
    torch.cuda.empty_cache()
    ctx.close()
    return res


def prune_step_times(pr, B, torch, stream, K, rows_too=True):
    """Device time of arrol_prune_step per call, in microseconds."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out = {}
    cases = (("tokens_only", False), ("with_hidden_rows", True)) if rows_too else (("tokens_only", False),)
    for label, rows in cases:
        step_args = pr.prune_step_args(with_rows=rows)
        for _ in range(3):
            B.arrol_prune_step(pr.ctx, step_args)
        torch.cuda.synchronize()
        reps = max(K, 20)
        a.record(stream)
        for _ in range(reps):
            B.arrol_prune_step(pr.ctx, step_args)
        b.record(stream)
        torch.cuda.synchronize()
        out[label] = a.elapsed_time(b) / reps * 1e3
    # the same token-only step replayed from a captured CUDA graph: the launches cost the host one call, so this is
    # the device-side duration of the chain (the eager figure above includes host launch time)
    try:
        step_args = pr.prune_step_args(with_rows=False)
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            B.arrol_prune_step(pr.ctx, step_args)              # warm-up on the capture stream
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            B.arrol_prune_step(pr.ctx, step_args)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        reps = max(K, 20)
        a.record(stream)
        for _ in range(reps):
            graph.replay()
        b.record(stream)
        torch.cuda.synchronize()
        out["tokens_only_graph"] = a.elapsed_time(b) / reps * 1e3
        # and with L2 flushed before every replay (a 256 MB fill), one replay per measurement: the step as it runs
        # after other work has displaced its inputs (cold rows, lengths, rewards and head weights)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=pr.dev)
        cold = []
        for _ in range(reps):
            flush.fill_(1)
            a.record(stream)
            graph.replay()
            b.record(stream)
            torch.cuda.synchronize()
            cold.append(a.elapsed_time(b) * 1e3)
        out["tokens_only_graph_l2_flushed"] = float(np.median(cold))
        del graph, flush
    except RuntimeError as exc:
        print("graph replay of the prune step skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)
    return out


def score_times(pr, pr_full, w, B, torch, stream, K):
    """The scoring kernel on its own: the linear head streamed over every source row (HBM-bound: d*e bytes per row);
    the MLP head on the chunk's own N rollouts (2*d*h flops per row, on the tensor cores for bf16 heads)."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    N = pr.w.N
    n_score = min(pr_full.T_src, 1 << 20) if w.h == 0 else N
    so = [torch.empty(n_score, dtype=torch.float32, device=pr.dev) for _ in range(3)]
    ridx = None if w.h == 0 else pr.row_index
    call = lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_score, so[0], so[1], so[2], row_index=ridx,
                                         q_lut=pr.q_lut)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    reps_score = max(K, 20)
    if w.h:                    # a call of tens of microseconds: queue it behind device work so that the host's
        for _ in range(2):     # launch time does not show
            pr.compact()
    a.record(stream)
    for _ in range(reps_score):
        call()
    b.record(stream)
    torch.cuda.synchronize()
    out = {"ms": a.elapsed_time(b) / reps_score, "rows": int(n_score), "step_call": None}
    del so
    # the step's own scoring call (N rows) next to a copy of the same number of bytes: at this size both sit on the
    # launch floor, which is the achievable roof there
    if w.h == 0:
        so = [torch.empty(N, dtype=torch.float32, device=pr.dev) for _ in range(3)]
        src = torch.empty((N, w.d), dtype=pr.hidden_score.dtype, device=pr.dev)
        dst = torch.empty_like(src)
        reps = max(K, 50)
        big = [torch.empty(n_score, dtype=torch.float32, device=pr.dev) for _ in range(3)]
        filler = lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_score, big[0], big[1], big[2],
                                               q_lut=pr.q_lut)

        def timed_us(fn):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            for _ in range(8):            # device-side filler, so that the timed calls are queued behind it and the
                filler()                  # host's launch time does not show
            a.record(stream)
            for _ in range(reps):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps * 1e3

        us_score = timed_us(lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, N, so[0], so[1], so[2],
                                                          row_index=pr.row_index, q_lut=pr.q_lut))
        us_copy = timed_us(lambda: dst.copy_(src))
        out["step_call"] = {"rows": int(N), "bytes": int(N * w.d * src.element_size()), "us": us_score,
                            "size_matched_copy_us": us_copy,
                            "note": "device time of queued calls; the copy moves the same bytes once (read + write)"}
        del so, src, dst, big
    return out


def run_update(pr, w, B, torch, K):
    """Times the policy-update calls on the survivors the step produced: loss + gradient, then the lm_head backward."""
    from paper_2603_24840_b200 import update as U
    dev, cap = pr.dev, pr.cap
    pr.step()
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 77)
    logp_old = pr.logp[:cap] + 0.05 * torch.randn(cap, generator=gen, device=dev)
    grad = torch.empty(cap, dtype=torch.float32, device=dev)
    loss = torch.zeros(1, dtype=torch.float64, device=dev)
    dH = torch.empty((cap, w.d), dtype=torch.float32, device=dev)
    dW = torch.empty((w.V, w.d), dtype=torch.float32, device=dev)
    ws_bytes = U.arrol_lm_head_backward_workspace(pr.ctx, cap, w.d, w.V)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def once():
        U.arrol_policy_loss(pr.ctx, pr.logp, logp_old, pr.tok_adv, pr.tok_seq, pr.cu_seqlens, pr.d_num, cap, grad, loss,
                            eps_low=0.2, eps_high=0.28)
        mid.record(stream)
        U.arrol_lm_head_backward(pr.ctx, pr.dst_rows, pr.W_vocab, pr.dst_tokens, grad, pr.lse, cap, w.d, w.V, dH, dW, ws,
                                 d_T=pr.d_num[1:])

    a, mid, b = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    once()
    torch.cuda.synchronize()
    n = max(1, min(K, 2))
    tot = loss_ms = 0.0
    for _ in range(n):
        a.record(stream)
        once()
        b.record(stream)
        torch.cuda.synchronize()
        tot += a.elapsed_time(b)
        loss_ms += a.elapsed_time(mid)
    B.arrol_poll_status(pr.ctx)
    return {"ms": tot / n, "loss_ms": loss_ms / n, "ws_gb": ws_bytes / 1e9}


def run_aux(pr, w, B, torch, K):
    """Times the calls around the step on the workload's shapes: calibrator update + stochastic survival rule
    (Appendix A.4), head training step, rank-weighted vote (Section 4.4), confidence variant of the log-prob call."""
    from paper_2603_24840_b200 import calibrator as CAL, confidence as CF, headtrain as HT, voting as VT
    dev, N = pr.dev, w.N
    stream = torch.cuda.current_stream()
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 99)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3          # us

    out = {}
    reps = max(K, 20)
    # calibrator: push the step's N (bin, reward) pairs, rebuild the table and delta; then the stochastic rule
    cal = CAL.Calibrator(pr.ctx, w.B, 8192)
    sp = CAL.survival(w.K / w.G, 0.5, w.rho, 0.05, 0.95)
    u = torch.rand(N, generator=gen, device=dev)
    keep2 = torch.empty(N, dtype=torch.uint8, device=dev)
    out["calib_update_us"] = timed(lambda: cal.update(pr.bin, pr.rewards, sp), reps)
    out["select_stochastic_us"] = timed(lambda: CAL.arrol_select_stochastic(pr.ctx, pr.q, u, keep2, sp, d_delta=cal.delta), reps)
    # head training step on the N scored rows (labels = the rollouts' rewards)
    hh = max(w.h, 1)
    grads = {"W1": torch.empty((hh, w.d), device=dev), "b1": torch.empty(hh, device=dev)}
    if w.h:
        grads["w2"] = torch.empty(w.h, device=dev)
        grads["b2"] = torch.empty(1, device=dev)
    hloss = torch.zeros(1, dtype=torch.float64, device=dev)
    hws = torch.empty(max(HT.arrol_head_grad_workspace(pr.ctx, N, w.d, w.h), 1), dtype=torch.uint8, device=dev)
    out["head_grad_us"] = timed(lambda: HT.arrol_head_grad(pr.ctx, pr.hidden_score, pr.head, N, pr.rewards, grads, hloss, hws,
                                                           row_index=pr.row_index), reps)
    if w.h:
        out["head_grad_tflops"] = 4.0 * N * w.d * w.h / (out["head_grad_us"] * 1e-6) / 1e12   # forward + dW1
    # test-time vote: P groups of G scored rollouts with synthetic answers
    answers = torch.randint(0, 6, (N,), generator=gen, device=dev, dtype=torch.int32)
    vw = torch.empty(N, device=dev)
    win = torch.empty(w.P, dtype=torch.int32, device=dev)
    ww = torch.empty(w.P, device=dev)
    if w.G <= 32:
        out["rank_vote_us"] = timed(lambda: VT.arrol_rank_vote(pr.ctx, pr.score, answers, w.P, w.G, vw, win, ww), reps)
    # log-prob call that also emits the per-token confidence, then the per-rollout reductions
    conf = torch.empty(pr.cap, device=dev)
    tconf = torch.empty(N, device=dev)
    n = max(1, min(K, 2))
    out["token_logprob_conf_ms"] = timed(lambda: CF.arrol_token_logprob_conf(
        pr.ctx, pr.dst_rows, pr.W_vocab, pr.dst_tokens, pr.cap, w.d, w.V, pr.logp, conf, pr.workspace, lse=pr.lse,
        d_T=pr.d_num[1:]), n) / 1e3
    out["trace_confidence_us"] = timed(lambda: CF.arrol_trace_confidence(pr.ctx, conf, pr.cu_seqlens, pr.d_num, N, tconf,
                                                                          window=2048, mode=1), reps)
    out["trace_confidence_bottom_tenth_us"] = timed(lambda: CF.arrol_trace_confidence(
        pr.ctx, conf, pr.cu_seqlens, pr.d_num, N, tconf, window=2048, mode=2), reps)
    B.arrol_poll_status(pr.ctx)
    return out


def run_e2e(views, pr_full, w, C, K, B, torch, barrier):
    """Same step through the host-buffer entry point: every step copies the inputs from pinned host memory and
    reads the results back.  With C chunks a step is C calls, each with its chunk's own lengths, rewards and offsets."""
    cap = max(v.cap for v in views)
    Nc = views[0].w.N
    # rows of every chunk in the source, rebased to the chunk's first row
    spans = []
    for v in views:
        off = v.host["src_tok_off"]
        spans.append((int(off[0]), int(off[-1])))
    max_rows = max(e - s for s, e in spans)
    # one pinned block of source rows sized for the largest chunk.  With one chunk it is the workload's source; with
    # several, pinning every chunk's rows would take most of the host's memory, so the calls read their hidden rows
    # (random by construction) from this block at their own chunk's offsets.
    h_hidden = pr_full.src_rows[spans[0][0]:spans[0][0] + max_rows].cpu().pin_memory()
    steps = []
    keepalive = []
    v0 = views[0]
    h_out = {
        "h_logp": torch.empty(cap, dtype=torch.float32).pin_memory(),
        "h_adv": torch.empty(Nc, dtype=torch.float32).pin_memory(),
        "h_cu_seqlens": torch.empty(Nc + 1, dtype=torch.int64).pin_memory(),
        "h_survivor_idx": torch.empty(Nc, dtype=torch.int32).pin_memory(),
        "h_num": torch.empty(2, dtype=torch.int64).pin_memory(),
    }
    dv = {
        "W_vocab": v0.W_vocab, "d_hidden": torch.empty((Nc, w.d), dtype=torch.bfloat16, device=v0.dev),
        "d_lengths": torch.empty_like(v0.lengths), "d_src_tok_off": torch.empty_like(v0.src_tok_off),
        "d_rewards": torch.empty_like(v0.rewards),
        "d_score": v0.score, "d_prob": v0.prob, "d_q": v0.q, "d_keep": v0.keep, "d_survivor_idx": v0.survivor_idx,
        "d_cu_seqlens": v0.cu_seqlens, "d_adv": v0.adv, "d_num": v0.d_num, "d_dst_tokens": v0.dst_tokens,
        "d_dst_rows": v0.dst_rows, "d_logp": v0.logp, "d_workspace": v0.workspace,
    }
    head = dict(v0.head)
    if v0.hidden_score.dtype != torch.bfloat16:   # fp32 workload: the host-step entry takes bf16 state
        head = {k: (t.to(torch.bfloat16) if torch.is_tensor(t) else t) for k, t in head.items()}
    pin = lambda t: t.cpu().pin_memory()
    for v, (s0, e0) in zip(views, spans):
        h = dict(h_out)
        h["h_hidden"] = h_hidden
        h["h_src_tokens"] = pin(v.src_tokens[s0:e0])
        h["h_lengths"] = pin(v.lengths)
        h["h_src_tok_off"] = pin(v.src_tok_off - s0)
        h["h_rewards"] = pin(v.rewards)
        scal = dict(P=v.w.P, G=w.G, K=w.K, cutoff=w.cutoff, d=w.d, V=w.V, ddof=0, rho=w.rho, eps=1e-6,
                    inv_temperature=1.0, T_src=e0 - s0, dst_capacity_tokens=v.cap)
        tensors = dict(h)
        tensors.update(dv)
        steps.append(B.make_host_step(scal, head, v0.q_lut, tensors))
        keepalive.append(tensors)
    ctx = v0.ctx
    stream = torch.cuda.current_stream()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # warm-up step; it also gives the bytes a step moves: the small per-rollout arrays, the N hidden rows at the
    # detection length, then only the survivors' hidden rows and token ids (uploaded straight into their packed
    # positions); results: logp[T] + per-rollout arrays
    row_bytes = w.d * 2
    T_e2e = h2d = d2h = 0
    for st in steps:
        B.arrol_prune_rebatch_host(ctx, st)
        T_now = int(h_out["h_num"][1])
        T_e2e += T_now
        h2d += Nc * (4 + 8 + 4) + (Nc + T_now) * row_bytes + 4 * T_now
        d2h += Nc * (4 + 4) + (Nc + 1) * 8 + 16 + 4 * T_now + Nc
    barrier()
    a.record(stream)
    for _ in range(K):
        for st in steps:
            B.arrol_prune_rebatch_host(ctx, st)       # synchronous: returns with results in host memory
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / K
    del keepalive
    return {"ms_per_step": ms, "h2d": int(h2d), "d2h": int(d2h), "tokens": T_e2e, "steps": K}


def report(res, peaks, tokens_all, ms_per_step, e2e_ms, world):
    """The JSON fields of one measured workload (value, rooflines, break-down, prune step, e2e)."""
    w, C, T, K = res["w"], res["C"], res["T"], res["K"]
    value = tokens_all / (ms_per_step * 1e-3)
    seg = res["seg_step"]
    logp_ms_step = float(seg[3])                       # all log-prob launches of a step
    logp_ms_launch = logp_ms_step / C
    flops_step = 2.0 * T * w.d * w.V
    achieved = flops_step / (logp_ms_step * 1e-3) / 1e12
    peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    traffic, traffic_src = logprob_traffic(w, T / C, res["splits"], res["sm_count"])
    roofline = {
        "kernel": "token_logprob_kernel, %s (+ combine_splits_kernel)" % (
            "pairs of blocks on 256-row tiles, tcgen05 cta_group::2" if res["kernel_form"] == 2 else
            "one block per 128-row tile, tcgen05 cta_group::1"), "bound": "tensor", "achieved": achieved, "peak": peak,
        "unit": "TFLOP/s", "frac": achieved / peak,
        "peak_source": "%s bf16 sustained (kernel timed inside a long step)" % peaks["source"],
        "frac_of_burst": achieved / float(peaks["bf16_tflops"]), "frac_of_nominal_2250": achieved / 2250.0,
        "traffic": traffic, "traffic_source": traffic_src, "vocab_splits": res["splits"],
        "algorithmic_flops_per_launch": flops_step / C, "launch_ms": logp_ms_launch, "launches_per_step": C,
        "in_kernel_clock": res["in_kernel"],
    }
    gather_bytes = 2.0 * T * w.d * 2 + 8.0 * T
    compact_gbs = gather_bytes / (float(seg[2]) * 1e-3) / 1e9
    e2e = res["e2e"]
    e2e_ok = e2e_ms == e2e_ms and e2e_ms > 0
    out = {
        "value": value, "ms_per_step": ms_per_step, "steps": K,
        "counts": {"survivors": res["S"], "survivor_tokens": T, "source_rows": res["T_src"],
                   "survivor_tokens_per_chunk": res["T_chunks"]},
        "clocks": res["clocks"],
        "e2e": {"value": (e2e["tokens"] * world) / (e2e_ms * 1e-3) if e2e_ok else None,
                "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                "ms_per_step": e2e_ms if e2e_ok else None, "steps": e2e.get("steps", 0),
                "survivor_tokens": e2e["tokens"]},
        "gpu_launches": res["launches"],
        "roofline": roofline,
        "breakdown_ms": {"score_partial": float(seg[0]), "select": float(seg[1]), "compact": float(seg[2]),
                         "token_logprob": logp_ms_step},
        "logprob_tokens_per_s": T / (logp_ms_step * 1e-3),
        "prune_step_us": res["prune_us"],
        "compact_roofline": {"kernel": "gather_rows_bulk_kernel (+ scan_adv_kernel, gather_tokens_kernel)", "bound": "hbm",
                             "achieved": compact_gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                             "frac": compact_gbs / float(peaks["hbm_gbs"]), "frac_of_nominal_8000": compact_gbs / 8000.0,
                             "algorithmic_bytes_per_launch": gather_bytes / C},
        "in_place": res["in_place"],
    }
    if res["other_kernel"] is not None:
        pk = dict(res["other_kernel"])
        pk["frac"] = pk["achieved"] / peak
        out["roofline"]["other_form"] = pk
    sc = res["score"]
    esz = 4 if w.dtype == "f32" else 2
    if w.h == 0:
        gbs = sc["rows"] * w.d * esz / (sc["ms"] * 1e-3) / 1e9
        per_row = SCORE_LINEAR_DRAM_BYTES_PER_ROW.get((w.d, esz))
        out["score_roofline"] = {"kernel": "score_linear_kernel", "bound": "hbm", "rows": sc["rows"],
                                 "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                                 "frac": gbs / float(peaks["hbm_gbs"]), "frac_of_nominal_8000": gbs / 8000.0,
                                 "launch_ms": sc["ms"],
                                 "traffic": None if per_row is None else per_row * sc["rows"],
                                 "note": "linear head streamed over consecutive source rows; the step itself "
                                         "scores only N = %d rows (launch-latency bound)" % res["N_chunk"],
                                 "step_call": sc["step_call"]}
    else:
        tfs = 2.0 * sc["rows"] * w.d * w.h / (sc["ms"] * 1e-3) / 1e12
        tc_peak = float(peaks["bf16_tflops"])
        out["score_roofline"] = {"kernel": "score_mlp_tc_kernel (+ row packing)", "bound": "tensor",
                                 "rows": sc["rows"], "achieved": tfs, "peak": tc_peak, "unit": "TFLOP/s",
                                 "frac": tfs / tc_peak, "launch_ms": sc["ms"],
                                 "note": "2*N*d*h flops of the head's first layer over the whole call (row packing, "
                                         "contraction, GELU, probability map): a few GFLOP, bound by launch and "
                                         "pipeline latency, not by the tensor pipe"}
    if res["update"] is not None:
        u = res["update"]
        upd_flops = 6.0 * u["tokens"] * w.d * w.V
        out["update"] = {"what": "arrol_policy_loss + arrol_lm_head_backward on the survivors of %s "
                                 "(recompute + dH + dW = 6 T d V flop)" % ("the step" if C == 1 else "one chunk"),
                         "ms": u["ms"], "loss_ms": u["loss_ms"], "tokens": u["tokens"],
                         "tokens_per_s": u["tokens"] / (u["ms"] * 1e-3),
                         "achieved": upd_flops / (u["ms"] * 1e-3) / 1e12, "unit": "TFLOP/s",
                         "frac": upd_flops / (u["ms"] * 1e-3) / 1e12 / peak, "bound": "tensor",
                         "workspace_gb": u["ws_gb"]}
    if res["aux"] is not None:
        aux = dict(res["aux"])
        aux["what"] = ("calibrator update + stochastic rule on N rollouts, head training step on the N scored rows, "
                       "rank-weighted vote over P groups, log-prob call with per-token confidence and its "
                       "per-rollout reductions (%s)" % ("the step's" if C == 1 else "one chunk's"))
        out["aux"] = aux
    return out


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2603_24840_b200 import dist_util, synth

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # weak scaling: every rank prunes and re-batches its own prompts (different seed per rank), no exchange
    C = args.prompt_chunks if args.prompt_chunks > 0 else auto_prompt_chunks(w)
    while w.P % C != 0:
        C += 1
    w_rank = dist_util.shard_workload(w, rank, world)
    K = args.steps
    res = measure(w_rank, C, K, args.warmup, local, barrier, rank, True, args)

    total_ms_max, e2e_ms_max, tokens_all = dist_util.reduce_timings(res["total_ms"], res["e2e"]["ms_per_step"],
                                                                    float(res["T"]), "cuda")
    peaks = load_peaks()
    out = None
    if rank == 0:
        body = report(res, peaks, tokens_all, total_ms_max / K, e2e_ms_max, world)
        out = {"metric": METRIC, "value": body.pop("value"), "unit": UNIT, "n_gpus": world, "steps": K,
               "warmup": args.warmup, "ms_per_step": body.pop("ms_per_step"), "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
               "config": config_of(w, C)}
        body.pop("steps")
        out.update(body)

    # ---- the other workloads, same figures at a reduced step count (single-GPU runs only) ----
    if world == 1 and not args.no_per_workload:
        per = {}
        Kp = max(1, min(K, 3))
        for name in synth.WORKLOAD_ORDER:
            if name == w.name:
                continue
            wo = synth.WORKLOADS[name]
            Co = auto_prompt_chunks(wo)
            try:
                r = measure(wo, Co, Kp, 3, local, barrier, rank, False, args)
                b = report(r, peaks, float(r["T"]), r["total_ms"] / Kp, r["e2e"]["ms_per_step"], 1)
                b["warmup"] = 3
                b["config"] = config_of(wo, Co)
                per[name] = b
            except (RuntimeError, MemoryError) as exc:
                per[name] = {"skipped": str(exc).splitlines()[0]}
                torch.cuda.empty_cache()
        out["per_workload"] = per
    elif rank == 0:
        out["per_workload"] = None

    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            x_cut, rows_note = scored_rows_of(w)
            v, sample, cores, T_cpu = oracle_step_rate(w, args.cpu_budget, x_cut=x_cut)
            T_gpu = out["counts"]["survivor_tokens"]
            note = "" if T_cpu == T_gpu else (
                "; the oracle keeps %d survivor tokens on these inputs, the GPU arm %d: a few rollouts whose fp32 / "
                "fp64 scores fall on different sides of a calibration-bin edge (inside the 1e-3 score tolerance) change "
                "which rollouts of their groups survive" % (T_cpu, T_gpu))
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": sample + "; scored rows: " + rows_note + note,
                                   "survivor_tokens": T_cpu, "gpu_arm_survivor_tokens": T_gpu}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_profile_leg(args, w):
    """One call of the path a few times on a small workload, for single-kernel profiler captures: the state is built
    and a whole step run twice, then the named call three times.  Prints how the call was made."""
    import torch
    from paper_2603_24840_b200 import binding as B
    from paper_2603_24840_b200.pipeline import PruneRebatch
    pr = PruneRebatch(w, device=0, with_rows=True)
    for _ in range(2):
        pr.step()
    torch.cuda.synchronize()
    n_stream = min(pr.T_src, 1 << 20)
    so = [torch.empty(n_stream, dtype=torch.float32, device=pr.dev) for _ in range(3)]
    step_args = pr.prune_step_args(with_rows=False)
    legs = {
        "score_stream": lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_stream, so[0], so[1], so[2],
                                                      q_lut=pr.q_lut),
        "score": pr.score_partial,
        "select": pr.select,
        "compact": pr.compact,
        "compact_tokens": lambda: pr.compact(False),
        "logprob": pr.token_logprob,
        "logprob_gathered": pr.token_logprob_gathered,
        "prune_step": lambda: B.arrol_prune_step(pr.ctx, step_args),
    }
    fn = legs[args.profile_leg]
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    S, T = pr.counts()
    B.arrol_poll_status(pr.ctx)
    print(json.dumps({"profile_leg": args.profile_leg, "workload": w.name, "calls": 3, "N": w.N, "survivors": S,
                      "survivor_tokens": T, "source_rows": pr.T_src, "streamed_rows": n_stream, "d": w.d, "V": w.V}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true", help="leave out the per_workload block")
    ap.add_argument("--prompt-chunks", type=int, default=0, help="0 = choose from the memory footprint")
    ap.add_argument("--skip-update", action="store_true", help="leave out the policy-update leg")
    ap.add_argument("--skip-aux", action="store_true", help="leave out the timings of the calls around the step")
    ap.add_argument("--skip-e2e", action="store_true", help="leave out the host-buffer leg (profiler captures)")
    ap.add_argument("--skip-pair", action="store_true", help="leave out the leg that times the log-prob kernel's "
                    "other form")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle log-prob work to time")
    ap.add_argument("--profile-leg", default=None, help="run one call of the path three times (for profiler captures): "
                    "score_stream, score, select, compact, compact_tokens, logprob, logprob_gathered, prune_step")
    args = ap.parse_args()
    from paper_2603_24840_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.profile_leg:
        run_profile_leg(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_ours(args, w)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the prune-and-rebatch hot path on B200.

A step is one pass of the whole path over one batch of synthetic input shaped like a GRPO/DAPO run:
  arrol_score_partial -> arrol_select -> arrol_compact (token ids + hidden rows) -> arrol_token_logprob.
`value` = survivor tokens processed per second over the whole step, inputs resident in HBM.
`e2e`   = the same metric through arrol_prune_rebatch_host: inputs in pinned host memory, results read back.
`--impl reference` times the CPU oracle (the plain fp64 program the GPU path is checked against) on host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
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
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM traffic of one token_logprob launch per survivor token at d = 2048, V = 128256 (one vocabulary split), from
# the ncu capture summarised in profiles/token_logprob_kernel_profile-small.md: (2.433 GB read + 5.4 MB written) /
# 75,382 tokens.  At fixed d, V and split count the traffic grows in proportion to the tokens of the launch.
LOGPROB_DRAM_BYTES_PER_TOKEN = {(2048, 128256): 32340.0}


def logprob_traffic(w, T, splits, sm_count):
    """DRAM bytes of one token_logprob launch: the ncu capture scaled by tokens where one exists for this (d, V),
    else the model the capture confirmed: every wave of resident blocks streams its W_vocab split once."""
    per_tok = LOGPROB_DRAM_BYTES_PER_TOKEN.get((w.d, w.V))
    if per_tok is not None:
        return per_tok * T, "ncu capture on profile-small scaled by tokens"
    return 2.0 * w.d * (1.0 + w.V * splits / (sm_count * 128.0)) * T, "model 2d(1 + V*splits/(SMs*128)) per token"


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


# ------------------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and the --impl reference arm)
# ------------------------------------------------------------------------------------------------------------
def oracle_step_rate(w, budget_s: float, logp_rows=None):
    """Times the oracle on the workload: head scoring, probability map, selection, scan, token gather and
    advantages at full size; the fp64 log-softmax gather on a bounded sample of survivor tokens.  Returns
    (tokens_per_s for the whole path, description, cores, seconds spent)."""
    import torch
    import oracle
    from paper_2603_24840_b200 import synth

    t_begin = time.perf_counter()
    ell = synth.lengths(w)
    off = synth.src_offsets(ell)
    rew = synth.rewards(w)
    head = synth.head_weights(w)
    tokens = synth.token_ids(w, int(off[-1]))
    hist_s, hist_y = synth.calib_history(w)
    oa = lambda t: None if t is None else synth.as_oracle_array(t)
    x_cut = synth.hidden_states(w, w.N, stream=21)           # hidden rows at the detection length
    Wv = oa(synth.vocab_weights(w, dtype=torch.bfloat16))
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
    return tokens_per_s, sample, cores, time.perf_counter() - t_begin


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
    vals = []
    budget = max(2.0, min(30.0, 120.0 / max(1, args.steps + args.warmup)))
    sample = ""
    cores = 0
    for i in range(args.warmup + args.steps):
        v, sample, cores, _ = oracle_step_rate(w, budget)
        if i >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    ell_T = value
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": None, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "note": "CPU oracle on host cores; each step a bounded sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    del ell_T
    print(json.dumps(out), flush=True)


# ------------------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------------------
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2603_24840_b200 import binding as B
    from paper_2603_24840_b200 import dist_util, synth
    from paper_2603_24840_b200.pipeline import PruneRebatch

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    # weak scaling: every rank prunes and re-batches its own prompts (different seed per rank), no exchange
    C = args.prompt_chunks if args.prompt_chunks > 0 else auto_prompt_chunks(w)
    while w.P % C != 0:
        C += 1
    w_rank = dist_util.shard_workload(w, rank, world, prompt_chunks=C)

    pr = PruneRebatch(w_rank, device=local, with_rows=True)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        pr.step()
    barrier()
    S, T = pr.counts()
    B.arrol_poll_status(pr.ctx)

    # ---- timed region: device-resident inputs ----
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(K * C)]
    sampler = ClockSampler(local)
    launches0 = B.arrol_launch_count(pr.ctx)
    if rank == 0:
        sampler.start()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for k in range(K * C):             # a step = C prompt chunks through the same buffers
        ev[k][0].record(stream)
        pr.score_partial()
        ev[k][1].record(stream)
        pr.select()
        ev[k][2].record(stream)
        pr.compact()
        ev[k][3].record(stream)
        pr.token_logprob()
        ev[k][4].record(stream)
    t_end.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    launches = B.arrol_launch_count(pr.ctx) - launches0
    total_ms = t_start.elapsed_time(t_end)
    B.arrol_poll_status(pr.ctx)
    seg = np.array([[ev[k][i].elapsed_time(ev[k][i + 1]) for i in range(4)] for k in range(K * C)])  # ms
    seg_mean = seg.mean(0)             # per chunk

    # prune step without the hidden-row plane (token ids only), timed separately
    # (one library call, arrol_prune_step: the launches are issued back to back without Python in between)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    prune_us = {}
    for label, rows in (("tokens_only", False), ("with_hidden_rows", True)):
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
        prune_us[label] = a.elapsed_time(b) / reps * 1e3
    # the same token-only step replayed from a captured CUDA graph: the four to five launches cost the host one call,
    # so this is the device-side duration of the chain (the eager figure above includes host launch time)
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
        prune_us["tokens_only_graph"] = a.elapsed_time(b) / reps * 1e3
        del graph
    except RuntimeError as exc:
        print("graph replay of the prune step skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)

    # scoring kernel on its own: the linear head streamed over every source row (HBM-bound: d*e bytes per row);
    # the MLP head on the workload's own N rollouts (2*d*h flops per row, on the tensor cores for bf16 heads)
    n_score = min(pr.T_src, 1 << 20) if w.h == 0 else w_rank.N
    so = [torch.empty(n_score, dtype=torch.float32, device=pr.dev) for _ in range(3)]
    ridx = None if w.h == 0 else pr.row_index
    for _ in range(3):
        B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_score, so[0], so[1], so[2], row_index=ridx,
                              q_lut=pr.q_lut)
    torch.cuda.synchronize()
    reps_score = K if w.h == 0 else max(K, 20)
    if w.h:                    # a call of tens of microseconds: queue it behind device work so that the host's
        for _ in range(2):     # launch time does not show
            pr.compact()
    a.record(stream)
    for _ in range(reps_score):
        B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_score, so[0], so[1], so[2], row_index=ridx,
                              q_lut=pr.q_lut)
    b.record(stream)
    torch.cuda.synchronize()
    score_ms = a.elapsed_time(b) / reps_score
    del so
    # the step's own scoring call (N rows) next to a copy of the same number of bytes: at this size both sit on the
    # launch floor, which is the achievable roof there
    step_score = None
    if w.h == 0:
        N_step = w_rank.N
        so = [torch.empty(N_step, dtype=torch.float32, device=pr.dev) for _ in range(3)]
        src = torch.empty((N_step, w.d), dtype=pr.hidden_score.dtype, device=pr.dev)
        dst = torch.empty_like(src)
        reps = max(K, 50)

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

        big = [torch.empty(n_score, dtype=torch.float32, device=pr.dev) for _ in range(3)]
        filler = lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, n_score, big[0], big[1], big[2],
                                               q_lut=pr.q_lut)
        us_score = timed_us(lambda: B.arrol_score_partial(pr.ctx, pr.hidden_score, pr.head, N_step, so[0], so[1], so[2],
                                                          row_index=pr.row_index, q_lut=pr.q_lut))
        us_copy = timed_us(lambda: dst.copy_(src))
        step_score = {"rows": int(N_step), "bytes": int(N_step * w.d * src.element_size()), "us": us_score,
                      "size_matched_copy_us": us_copy,
                      "note": "device time of queued calls; the copy moves the same bytes once (read + write)"}
        del so, src, dst, big

    # ---- policy update on the same survivors (reported separately; not part of `value`) ----
    update = None
    if not args.skip_update:
        try:
            update = run_update(pr, w_rank, B, torch, K)
        except (RuntimeError, MemoryError) as exc:
            print("update leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)

    # ---- the calls around the step (reported separately; not part of `value`) ----
    aux = None
    if not args.skip_aux:
        try:
            aux = run_aux(pr, w_rank, B, torch, K)
        except (RuntimeError, MemoryError) as exc:
            print("aux leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)

    # ---- e2e: host buffers through arrol_prune_rebatch_host ----
    if args.skip_e2e:
        e2e = {"ms_per_step": float("nan"), "h2d": 0, "d2h": 0}
    else:
        try:
            e2e = run_e2e(args, w_rank, pr, B, torch, world, barrier)
        except (RuntimeError, MemoryError) as exc:   # e.g. the pinned host copy of the inputs does not fit
            print("e2e leg skipped: %s" % str(exc).splitlines()[0], file=sys.stderr)
            e2e = {"ms_per_step": float("nan"), "h2d": 0, "d2h": 0}

    # ---- reduce over ranks ----
    total_ms_max, e2e_ms_max, tokens_all = dist_util.reduce_timings(total_ms, e2e["ms_per_step"], float(T) * C, "cuda")
    e2e_ms_max *= C                      # the host-buffer leg runs one chunk per call

    if rank == 0:
        peaks = load_peaks()
        ms_per_step = total_ms_max / K
        value = tokens_all / (ms_per_step * 1e-3)
        logp_ms = float(seg_mean[3])
        flops = 2.0 * T * w.d * w.V
        achieved = flops / (logp_ms * 1e-3) / 1e12
        peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
        gather_bytes = 2.0 * T * w.d * 2 + 8.0 * T
        splits = B.arrol_token_logprob_splits(pr.ctx, pr.cap, w.d, w.V)
        traffic, traffic_src = logprob_traffic(w, T, splits, torch.cuda.get_device_properties(local).multi_processor_count)
        roofline = {
            "kernel": "token_logprob_kernel", "bound": "tensor", "achieved": achieved, "peak": peak,
            "unit": "TFLOP/s", "frac": achieved / peak,
            "peak_source": "%s bf16 sustained (kernel timed inside a long step)" % peaks["source"],
            "frac_of_burst": achieved / float(peaks["bf16_tflops"]), "frac_of_nominal_2250": achieved / 2250.0,
            "traffic": traffic, "traffic_source": traffic_src, "vocab_splits": int(splits),
            "algorithmic_flops_per_launch": flops,
            "launch_ms": logp_ms,
        }
        compact_gbs = gather_bytes / (float(seg_mean[2]) * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "prompt_chunks": C,
                       "chunking": ("none" if C == 1 else "a step runs %d chunks of %d prompts back to back through the "
                                    "same buffers (one chunk's inputs reused; groups and tokens are independent, so "
                                    "times add); survivors/survivor_tokens/source_rows are per chunk" % (C, w.P // C)),
                       "P": w.P, "G": w.G, "K": w.K, "cutoff": w.cutoff, "d": w.d, "V": w.V,
                       "head_h": w.h, "survivors": S, "survivor_tokens": T, "source_rows": pr.T_src,
                       "l2": "inputs larger than L2 (hidden rows %.2f GB, W_vocab %.2f GB)" % (
                           pr.T_src * w.d * 2 / 1e9, w.V * w.d * 2 / 1e9)},
            "clocks": clocks,
            "e2e": {"value": tokens_all / (e2e_ms_max * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": e2e["h2d"] * C, "d2h_bytes_per_step": e2e["d2h"] * C,
                    "ms_per_step": e2e_ms_max},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "breakdown_ms": {"score_partial": float(seg_mean[0]), "select": float(seg_mean[1]),
                             "compact": float(seg_mean[2]), "token_logprob": logp_ms},
            "logprob_tokens_per_s": T / (logp_ms * 1e-3),
            "prune_step_us": prune_us,
            "compact_roofline": {"bound": "hbm", "achieved": compact_gbs, "peak": float(peaks["hbm_gbs"]),
                                 "unit": "GB/s", "frac": compact_gbs / float(peaks["hbm_gbs"]),
                                 "frac_of_nominal_8000": compact_gbs / 8000.0,
                                 "algorithmic_bytes_per_launch": gather_bytes},
        }
        esz = pr.hidden_score.element_size()
        if w.h == 0:
            gbs = n_score * w.d * esz / (score_ms * 1e-3) / 1e9
            out["score_roofline"] = {"kernel": "score_linear_kernel", "bound": "hbm", "rows": int(n_score),
                                     "achieved": gbs, "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                                     "frac": gbs / float(peaks["hbm_gbs"]), "frac_of_nominal_8000": gbs / 8000.0,
                                     "launch_ms": score_ms,
                                     "note": "linear head streamed over consecutive source rows; the step itself "
                                             "scores only N = %d rows (launch-latency bound)" % w_rank.N,
                                     "step_call": step_score}
        else:
            tfs = 2.0 * n_score * w.d * w.h / (score_ms * 1e-3) / 1e12
            tc_peak = float(peaks["bf16_tflops"])
            out["score_roofline"] = {"kernel": "pack_rows_kernel + score_mlp_tc_kernel", "bound": "tensor",
                                     "rows": int(n_score), "achieved": tfs, "peak": tc_peak, "unit": "TFLOP/s",
                                     "frac": tfs / tc_peak, "launch_ms": score_ms,
                                     "note": "2*N*d*h flops of the head's first layer over the whole call (row packing, "
                                             "contraction, GELU, probability map); a few GFLOP on %d blocks: bound by "
                                             "launch and pipeline latency, not by the tensor pipe"
                                             % (((n_score + 127) // 128) * ((w.h + 63) // 64))}
        if update is not None:
            upd_flops = 6.0 * T * w.d * w.V
            out["update"] = {"what": "arrol_policy_loss + arrol_lm_head_backward on the step's survivors "
                                     "(recompute + dH + dW = 6 T d V flop)",
                             "ms": update["ms"], "loss_ms": update["loss_ms"], "tokens_per_s": T / (update["ms"] * 1e-3),
                             "achieved": upd_flops / (update["ms"] * 1e-3) / 1e12, "unit": "TFLOP/s",
                             "frac": upd_flops / (update["ms"] * 1e-3) / 1e12 / peak, "bound": "tensor",
                             "workspace_gb": update["ws_gb"]}
        if aux is not None:
            aux["what"] = ("calibrator update + stochastic rule on N rollouts, head training step on the N scored rows, "
                           "rank-weighted vote over P groups, log-prob call with per-token confidence and its "
                           "per-rollout reduction")
            out["aux"] = aux
        if not args.no_cpu_baseline and world == 1:
            v, sample, cores, _ = oracle_step_rate(w, args.cpu_budget)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_update(pr, w, B, torch, K):
    """Times the policy-update calls on the survivors the step produced: loss + gradient, then the lm_head backward."""
    from paper_2603_24840_b200 import update as U
    dev, cap = pr.dev, pr.cap
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 77)
    logp_old = pr.logp + 0.05 * torch.randn(cap, generator=gen, device=dev)
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
    n = max(1, min(K, 3))
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
    # log-prob call that also emits the per-token confidence, then the per-rollout reduction
    conf = torch.empty(pr.cap, device=dev)
    tconf = torch.empty(N, device=dev)
    n = max(1, min(K, 3))
    out["token_logprob_conf_ms"] = timed(lambda: CF.arrol_token_logprob_conf(
        pr.ctx, pr.dst_rows, pr.W_vocab, pr.dst_tokens, pr.cap, w.d, w.V, pr.logp, conf, pr.workspace, lse=pr.lse,
        d_T=pr.d_num[1:]), n) / 1e3
    out["trace_confidence_us"] = timed(lambda: CF.arrol_trace_confidence(pr.ctx, conf, pr.cu_seqlens, pr.d_num, N, tconf,
                                                                          window=2048, mode=1), reps)
    B.arrol_poll_status(pr.ctx)
    return out


def auto_prompt_chunks(w):
    """Smallest number of prompt chunks whose source + packed hidden rows stay under ~60 GB."""
    from paper_2603_24840_b200 import synth
    ell = synth.lengths(w).astype(np.int64)
    rows = float(ell.sum()) * 1.6            # source rows + packed survivors (roughly 0.6 of the source)
    gb = rows * w.d * 2 / 1e9
    c = 1
    while gb / c > 60.0 and c < w.P:
        c *= 2
    return c


def run_e2e(args, w, pr, B, torch, world, barrier):
    """Same step through the host-buffer entry point: every step copies the inputs from pinned host memory and
    reads the results back."""
    N, cap = w.N, pr.cap
    pin = lambda t: t.cpu().pin_memory()
    h = {
        "h_hidden": pin(pr.src_rows), "h_src_tokens": pin(pr.src_tokens), "h_lengths": pin(pr.lengths),
        "h_src_tok_off": pin(pr.src_tok_off), "h_rewards": pin(pr.rewards),
        "h_logp": torch.empty(cap, dtype=torch.float32).pin_memory(),
        "h_adv": torch.empty(N, dtype=torch.float32).pin_memory(),
        "h_cu_seqlens": torch.empty(N + 1, dtype=torch.int64).pin_memory(),
        "h_survivor_idx": torch.empty(N, dtype=torch.int32).pin_memory(),
        "h_num": torch.empty(2, dtype=torch.int64).pin_memory(),
    }
    dv = {
        "W_vocab": pr.W_vocab, "d_hidden": torch.empty((N, w.d), dtype=torch.bfloat16, device=pr.dev),
        "d_lengths": torch.empty_like(pr.lengths), "d_src_tok_off": torch.empty_like(pr.src_tok_off),
        "d_rewards": torch.empty_like(pr.rewards),
        "d_score": pr.score, "d_prob": pr.prob, "d_q": pr.q, "d_keep": pr.keep, "d_survivor_idx": pr.survivor_idx,
        "d_cu_seqlens": pr.cu_seqlens, "d_adv": pr.adv, "d_num": pr.d_num, "d_dst_tokens": pr.dst_tokens,
        "d_dst_rows": pr.dst_rows, "d_logp": pr.logp, "d_workspace": pr.workspace,
    }
    scal = dict(P=w.P, G=w.G, K=w.K, cutoff=w.cutoff, d=w.d, V=w.V, ddof=0, rho=w.rho, eps=1e-6,
                inv_temperature=1.0, T_src=pr.T_src, dst_capacity_tokens=cap)
    head = dict(pr.head)
    if pr.hidden_score.dtype != torch.bfloat16:   # fp32 workload: the host-step entry takes bf16 state
        head = {k: (v.to(torch.bfloat16) if torch.is_tensor(v) else v) for k, v in head.items()}
    tensors = dict(h)
    tensors.update(dv)
    step = B.make_host_step(scal, head, pr.q_lut, tensors)
    # bytes the call moves per step: the small per-rollout arrays, the N hidden rows at the detection length, then only
    # the survivors' hidden rows and token ids (uploaded straight into their packed positions); results: logp[T] +
    # per-rollout arrays
    _, T_now = pr.counts()
    row_bytes = w.d * 2
    h2d = sum(h[k].numel() * h[k].element_size() for k in ("h_lengths", "h_src_tok_off", "h_rewards"))
    h2d += (N + T_now) * row_bytes + 4 * T_now
    d2h = sum(h[k].numel() * h[k].element_size() for k in ("h_adv", "h_cu_seqlens", "h_survivor_idx", "h_num")) + 4 * T_now + N
    n_e2e = max(1, min(args.steps, 5))
    for _ in range(2):
        B.arrol_prune_rebatch_host(pr.ctx, step)
    barrier()
    stream = torch.cuda.current_stream()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(n_e2e):
        B.arrol_prune_rebatch_host(pr.ctx, step)       # synchronous: returns with results in host memory
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / n_e2e
    assert int(h["h_num"][1]) == pr.counts()[1]
    return {"ms_per_step": ms, "h2d": int(h2d), "d2h": int(d2h)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama-3.2-1b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--prompt-chunks", type=int, default=0, help="0 = choose from the memory footprint")
    ap.add_argument("--skip-update", action="store_true", help="leave out the policy-update leg")
    ap.add_argument("--skip-aux", action="store_true", help="leave out the timings of the calls around the step")
    ap.add_argument("--skip-e2e", action="store_true", help="leave out the host-buffer leg (profiler captures)")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of oracle log-prob work to time")
    args = ap.parse_args()
    from paper_2603_24840_b200 import synth
    w = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_ours(args, w)


if __name__ == "__main__":
    main()

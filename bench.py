#!/usr/bin/env python
"""Decode-throughput bench of the GPT decode step: batch 1, 16 and 128 in one invocation.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workloads 2,3,4,5,5w4,5k8] [--impl ours|reference]

A step is one tts_gpt_decode_step over the workload's batch of streams (the whole hot path: page
allocation, embed, 24 blocks, final LayerNorm, LM head, sampling).  The first workload of the list is
the headline of the JSON line (default: workload 2 = the 24-layer bf16 decoder, batch 1, prefix 400,
decoding from context 400; K = 500 steps reproduces 400 -> 900); every workload of the list, the
headline included, appears in the `workloads` array with its own value, roofline and end-to-end rate.
K steps are repeated (streams re-opened outside the timing) until the timed region covers at least
`--min-seconds`.  N > 1 runs independent replicas, one process per GPU, with no collective on the data
path: started from a plain `python bench.py --gpus N` by re-executing under torch.distributed.run, or
by the caller's own torchrun; timing is the max over ranks.  `--impl reference` times the fp64 CPU
oracle instead.  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_21042_b200 import cases as C  # noqa: E402

METRIC = "GPT decode tokens/s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0          # the "about 8 TB/s" the target statement quotes
TARGET_FRAC = 0.70                # of the HBM roofline at batch 1-16
# key -> (workload, weight format override, KV cache format)
WORKLOAD_KEYS = {"1": (1, None, C.KV_BF16), "2": (2, None, C.KV_BF16), "3": (3, None, C.KV_BF16), "4": (4, None, C.KV_BF16),
                 "5": (5, None, C.KV_BF16), "5w8": (5, C.W_INT8_PC, C.KV_BF16), "5w4": (5, C.W_INT4_G128, C.KV_BF16),
                 "4k8": (4, None, C.KV_FP8_E4M3), "5k8": (5, None, C.KV_FP8_E4M3), "5w4k8": (5, C.W_INT4_G128, C.KV_FP8_E4M3)}
DTYPE = {C.W_BF16: "bf16", C.W_INT8_PC: "bf16 activations x int8 weights (fp32 accumulate)",
         C.W_INT4_G128: "bf16 activations x int4 weights (fp32 accumulate)"}


def linear_weight_count(cfg: C.GPTConfig):
    d, F = cfg.d_model, cfg.d_ff
    return 3 * d * d + d * d + 2 * d * F


def algorithmic_bytes_per_step(cfg: C.GPTConfig, ctx_before):
    """Bytes the step must move: every weight byte once, every cached K/V byte of every active
    stream once plus the new K/V, the logits once.  ctx_before: context lengths before the step."""
    d, F, V, L = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_layer
    n_lin = linear_weight_count(cfg)
    if cfg.wfmt == C.W_BF16:
        w = n_lin * 2
    elif cfg.wfmt == C.W_INT8_PC:
        w = n_lin + (3 * d + d + F + d) * 2
    else:
        w = n_lin // 2 + n_lin // 128 * 2
    small = (3 * d + d + F + d) * 2 + 4 * d * 2           # biases + LN per layer
    weights = L * (w + small) + V * d * 2 + 2 * d * 2
    # per cached token: K and V rows of every layer, bf16, or e4m3 codes with one fp32 scale per head
    kv_per_tok = (2 * d * 2 * L) if cfg.kv_fmt == C.KV_BF16 else (2 * cfg.n_head * (cfg.head_dim + 4) * L)
    kv = sum((c + 1) * kv_per_tok for c in ctx_before)
    return weights + kv + len(ctx_before) * V * 4


def linear_flops_per_step(cfg: C.GPTConfig, n_rows):
    """2 x weights x rows over the block linears and the LM head."""
    return 2.0 * (cfg.n_layer * linear_weight_count(cfg) + cfg.vocab * cfg.d_model) * n_rows


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed regions run."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz, self.ok = [], set(), None, False
        self._stop = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "sw_power_cap": 0x4, "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.ok:
            self.t.start()

    def stop(self):
        self._stop.set()
        if self.ok:
            self.t.join(timeout=1)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, source) from the generated file, else the machine's fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1400.0, "fallback"


class WeightCache:
    """The full-size bf16 draw is made once per process; the quantized sets are derived from it."""

    def __init__(self):
        self._bf16 = {}

    def get(self, cfg: C.GPTConfig, seed: int):
        key = (cfg.n_layer, cfg.d_model, cfg.d_ff, cfg.vocab, cfg.max_pos, cfg.emb_rows, seed)
        if key not in self._bf16:
            self._bf16.clear()
            self._bf16[key] = C.make_weights(C.GPTConfig(**{**cfg.as_dict(), "wfmt": C.W_BF16}), seed=seed)
        return C.quantize_weights(self._bf16[key], cfg.wfmt)


def make_prefix_tensors(wl, device):
    import torch
    out = []
    for p in C.make_prefixes(wl.cfg, wl.prefix_lens, seed=wl.seed):
        out.append(torch.from_numpy(p.view(np.int16)).to(device))
    return out


def run_workload(key, args, wcache, device, local, world, peaks):
    """Times one workload on this rank's GPU; returns its entry of the `workloads` array (identical on
    every rank: the cross-rank reductions are inside)."""
    import torch
    import torch.distributed as dist
    from paper_2607_21042_b200 import binding as B
    from paper_2607_21042_b200 import replicas as R

    idx, wfmt, kv_fmt = WORKLOAD_KEYS[key]
    wl = C.workload(idx, wfmt=wfmt, kv_fmt=kv_fmt)
    cfg = wl.cfg
    S = wl.n_streams
    W = max(args.warmup, 3)
    max_dec = max(wl.decode_lens)
    K = min(args.steps, max_dec)
    eng = B.TtsGpt(cfg, wcache.get(cfg, wl.seed), device)
    prefixes = make_prefix_tensors(wl, device)
    V, d = cfg.vocab, cfg.d_model
    uni = None
    if wl.top_k > 1:
        uni = torch.from_numpy(C.make_uniforms(max(K, W) + 2, S, seed=wl.seed)).to(device)
    toks = torch.zeros((2, S), dtype=torch.int32, device=device)
    logits = torch.zeros((S, V), dtype=torch.float32, device=device)
    hidden = torch.zeros((S, d), dtype=torch.int16, device=device)
    torch.cuda.synchronize()

    def active_at(step, ids):
        # stream i takes decode_lens[i] steps, then is released ("drain")
        return [(i, s) for i, s in enumerate(ids) if wl.decode_lens[i] >= step]

    def open_all():
        ids, _ = eng.prefill(prefixes, top_k=wl.top_k, temperature=wl.temperature,
                             uniforms=None if uni is None else uni[0], out_tokens=toks[0])
        return ids

    def decode_run(ids, n_steps):
        """Queue n_steps steps back to back (tokens fed back on the device, no host sync); streams are
        released when their length is reached.  Returns (tokens, algorithmic bytes, steps taken)."""
        ctx = list(wl.prefix_lens)
        tokens = nbytes = steps = 0
        released = set()
        for k in range(1, n_steps + 1):
            act = active_at(k, ids)
            if not act:
                break
            for i, s in enumerate(ids):
                if wl.decode_lens[i] < k and i not in released:
                    eng.release_stream(s)
                    released.add(i)
            sids = [s for _, s in act]
            n = len(sids)
            eng.decode_step(sids, toks[1, :n], top_k=wl.top_k, temperature=wl.temperature,
                            uniforms=None if uni is None else uni[k, :n],
                            out_logits=logits[:n], out_hidden=hidden[:n])
            nbytes += algorithmic_bytes_per_step(cfg, [ctx[i] for i, _ in act])
            for i, _ in act:
                ctx[i] += 1
            tokens += n
            steps += 1
        for i, s in enumerate(ids):
            if i not in released:
                eng.release_stream(s)
        return tokens, nbytes, steps

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(n_steps, min_seconds, max_reps):
        """Repeats `n_steps` steps from freshly opened streams until the summed device time reaches
        min_seconds.  Device time = CUDA events on the engine's stream around the queued steps."""
        tot_ms = 0.0
        tot_tokens = tot_bytes = tot_steps = reps = tot_launches = 0
        while True:
            if args.profiler_range == "all":
                torch.cuda.profiler.start()     # the prefill call that opens the streams, then the decode steps
            ids = open_all()
            eng.sync()
            if args.profiler_range == "decode":
                torch.cuda.profiler.start()     # the decode steps only
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            with torch.cuda.stream(eng.stream):
                e0.record()
            l_before = eng.kernel_launches()
            tokens, nbytes, steps = decode_run(ids, n_steps)
            tot_launches += eng.kernel_launches() - l_before     # kernels of the timed steps only
            with torch.cuda.stream(eng.stream):
                e1.record()
            eng.sync()
            if args.profiler_range:
                torch.cuda.profiler.stop()
            tot_ms += e0.elapsed_time(e1)
            tot_tokens += tokens; tot_bytes += nbytes; tot_steps += steps
            reps += 1
            # every rank takes the same number of repetitions: the decision is the slowest rank's
            if R.max_over_ranks(tot_ms, device) >= min_seconds * 1e3 or reps >= max_reps:
                break
        return tot_ms, tot_tokens, tot_bytes, tot_steps, reps, tot_launches

    # warm-up: open, W steps (captures the step graph of this batch size), close
    ids = open_all()
    decode_run(ids, W)
    eng.sync()

    # ---- prefill time of one call over all prefixes (outside the decode metric) ----
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(eng.stream):
        p0.record()
    ids = open_all()
    with torch.cuda.stream(eng.stream):
        p1.record()
    eng.sync()
    prefill_ms = R.max_over_ranks(p0.elapsed_time(p1), device)
    for s in ids:
        eng.release_stream(s)
    eng.sync()
    prefill_rows = int(sum(wl.prefix_lens))

    # ---- timed region: K steps x repetitions, device-resident inputs ----
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ms, tokens, nbytes, steps_done, reps, launches = timed(K, args.min_seconds, args.max_reps)
    barrier()
    total_tokens = R.sum_over_ranks(tokens, device)     # replicas: every rank decodes its own copy of the workload
    ms = R.max_over_ranks(ms, device)
    value = total_tokens / (ms * 1e-3)

    hbm_peak, tc_peak, peak_kind = peaks
    gbs = nbytes / (ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak,
                "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS, "traffic": None, "peak_source": peak_kind,
                "kernel": "whole decode step (%d kernel launches per step)" % round(launches / max(steps_done, 1)),
                "algorithmic_bytes_per_step": nbytes / max(steps_done, 1)}
    cap = captured_traffic(wl.name)
    if cap is not None:
        # DRAM bytes of one step from the committed ncu launch list of this workload (not measured in this run:
        # a number taken under a profiler is not a bench value, so the capture is a separate, recorded run)
        roofline["traffic"] = cap["dram_bytes_per_step"]
        roofline["traffic_source"] = ("ncu dram__bytes_read.sum + dram__bytes_write.sum over the launches of one step, "
                                      "profiles/decode_step_dram_traffic.json; algorithmic bytes of the captured steps: %d"
                                      % cap["algorithmic_bytes_per_step"])
    if S <= 16:
        roofline["target_frac"] = TARGET_FRAC
        roofline["target_met"] = bool(gbs / hbm_peak >= TARGET_FRAC)

    entry = {
        "workload": wl.name, "batch": S, "weights": C.WFMT_NAMES[cfg.wfmt], "kv_cache": C.KV_NAMES[cfg.kv_fmt],
        "dtype": DTYPE[cfg.wfmt],
        "value": value, "unit": UNIT, "ms_per_step": ms / max(steps_done, 1),
        "steps": K, "repetitions": reps, "timed_steps": steps_done, "timed_ms": ms, "tokens": tokens,
        "gpu_launches": int(launches), "roofline": roofline,
        "prefix": [min(wl.prefix_lens), max(wl.prefix_lens)],
        "sampling": "greedy" if wl.top_k <= 1 else "top-k %d" % wl.top_k,
        "prefill": {"rows": prefill_rows, "streams": S, "ms": prefill_ms,
                    "rows_per_s": world * prefill_rows / (prefill_ms * 1e-3),
                    "note": "one prefill call over all prefixes (device resident), first token sampled; outside the timed region"},
    }
    # the block linears' flops over the whole call (attention, LayerNorm and the heads are inside the time, not the flops)
    pf_tf = 2.0 * linear_weight_count(cfg) * cfg.n_layer * prefill_rows / (prefill_ms * 1e-3) / 1e12
    entry["prefill"]["roofline_tensor"] = {"bound": "tensor", "achieved": pf_tf, "peak": tc_peak, "unit": "TFLOP/s",
                                           "frac": pf_tf / tc_peak, "peak_source": peak_kind + " (sustained bf16)",
                                           "kernel": "whole prefill call: flops of the four block linears / time of the call"}

    # ---- batch 128: the window in which every stream is still active, and the tensor-pipe fraction ----
    if S > 16:
        win = min(64, min(wl.decode_lens))
        wms, wtok, wbytes, wsteps, wreps, _ = timed(win, args.min_seconds / 2, args.max_reps)
        wms = R.max_over_ranks(wms, device)
        wg = wbytes / (wms * 1e-3) / 1e9
        entry["full_batch_window"] = {
            "steps": win, "repetitions": wreps, "value": R.sum_over_ranks(wtok, device) / (wms * 1e-3), "unit": UNIT,
            "ms_per_step": wms / max(wsteps, 1),
            "roofline": {"bound": "hbm", "achieved": wg, "peak": hbm_peak, "unit": "GB/s", "frac": wg / hbm_peak,
                         "frac_of_nominal_8tbs": wg / NOMINAL_HBM_GBS, "peak_source": peak_kind}}

    # ---- end to end over the same steps: host buffers in, host buffers out, one C-ABI call per step ----
    h_in = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_tok = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_log = torch.zeros((S, V), dtype=torch.float32).pin_memory()
    h_hid = torch.zeros((S, d), dtype=torch.int16).pin_memory()
    h_uni = None if uni is None else uni.cpu().pin_memory()
    e2e_s = 0.0
    e2e_tokens = e2e_steps = e2e_reps = 0
    d2h_bytes = 0
    while True:
        ids = open_all()
        eng.sync()
        h_in.copy_(toks[0].cpu())
        all_ids = (ctypes.c_int32 * S)(*ids)      # marshalled once for the steps in which every stream is active
        released = set()
        barrier()
        t0 = time.perf_counter()
        for k in range(1, K + 1):
            act = active_at(k, ids)
            if not act:
                break
            for i, s in enumerate(ids):
                if wl.decode_lens[i] < k and i not in released:
                    eng.release_stream(s)
                    released.add(i)
            n = len(act)
            sids = all_ids if n == S else [s for _, s in act]
            eng.decode_step_host(sids, h_tok, in_tokens=h_in, top_k=wl.top_k, temperature=wl.temperature,
                                 uniforms=None if h_uni is None else h_uni[k], out_logits=h_log, out_hidden=h_hid)
            h_in[:n].copy_(h_tok[:n])
            e2e_tokens += n
            e2e_steps += 1
            d2h_bytes = max(d2h_bytes, n * (4 + 4 * V + 2 * d))
        torch.cuda.synchronize()
        e2e_s += time.perf_counter() - t0
        for i, s in enumerate(ids):
            if i not in released:
                eng.release_stream(s)
        eng.sync()
        e2e_reps += 1
        if R.max_over_ranks(e2e_s, device) >= args.min_seconds / 2 or e2e_reps >= args.max_reps:
            break
    e2e_s = R.max_over_ranks(e2e_s, device)
    entry["e2e"] = {"value": R.sum_over_ranks(e2e_tokens, device) / e2e_s, "unit": UNIT,
                    "h2d_bytes_per_step": 4 * S + (4 * S if wl.top_k > 1 else 0), "d2h_bytes_per_step": int(d2h_bytes),
                    "steps": K, "repetitions": e2e_reps, "ms_per_step": e2e_s * 1e3 / max(e2e_steps, 1),
                    "note": "one tts_gpt_decode_step_host call per step over the same steps as `value`: tokens "
                            "(and uniforms) in from pinned host memory; tokens, logits and hidden rows back, valid on return"}
    entry["clocks"] = sampler.stop()
    if S > 16:      # last: tracing drops the captured step graphs
        entry["roofline_tensor"] = tensor_roofline(eng, wl, open_all, toks, S, tc_peak, peak_kind, device)
    eng.destroy()
    del eng, prefixes
    torch.cuda.empty_cache()
    return entry, wl


def captured_traffic(workload_name):
    """The recorded ncu DRAM traffic of one decode step of this workload, if profiles/ holds one."""
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "profiles", "decode_step_dram_traffic.json")
    try:
        with open(path) as f:
            return json.load(f).get(workload_name)
    except (OSError, ValueError):
        return None


def tensor_roofline(eng, wl, open_all, toks, S, tc_peak, peak_kind, device):
    """Tensor-pipe fraction of the linear phases at the full batch: one traced step gives, for every
    kernel of the chain, the instant its dependency wait was released; a linear's share of the step
    is the interval to the release of the kernel behind it.  flops of the linears / that time / the
    sustained bf16 peak."""
    import torch
    cfg = wl.cfg
    L = cfg.n_layer
    tr = torch.zeros(8 * (7 * L + 8), dtype=torch.int64, device=device)
    ids = open_all()
    eng.sync()
    per = eng.set_trace(tr)
    for _ in range(4):
        eng.decode_step(ids, toks[1, :S])
    eng.sync()
    eng.set_trace(None)
    for s in ids:
        eng.release_stream(s)
    eng.sync()
    n_k = 7 * L + 1                           # ln1 qkv attn o ln2 fc1 fc2 per layer, then the final LayerNorm
    t = tr.cpu().numpy().reshape(-1, 8)[:n_k].astype(np.float64)
    rel = t[:, 1]
    if per < n_k or not np.all(rel > 0):
        return None
    slot = np.diff(rel)                      # kernel i: release(i+1) - release(i), ns
    lin = [i for i in range(7 * L) if i % 7 in (1, 3, 5, 6)]
    lin_ns = float(np.sum(slot[lin]))
    flops = 2.0 * linear_weight_count(cfg) * S * L
    tf = flops / (lin_ns * 1e-9) / 1e12
    return {"bound": "tensor", "achieved": tf, "peak": tc_peak, "unit": "TFLOP/s", "frac": tf / tc_peak,
            "peak_source": peak_kind + " (sustained bf16)", "rows": S,
            "linear_us_per_layer": lin_ns / 1e3 / L,
            "kernel": "the four block linears (tcgen05) of one traced step, %d launches" % len(lin),
            "note": "time inside the linear phases from the timeline trace (release of a kernel's dependency wait to the release of its successor's)"}


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    peaks = measured_peaks()
    wcache = WeightCache()
    keys = [k.strip() for k in args.workloads.split(",") if k.strip()]
    entries = []
    head_wl = None
    t_start = time.time()
    for k in keys:
        e, wl = run_workload(k, args, wcache, device, local, world, peaks)
        e["wall_s"] = time.time() - t_start
        t_start = time.time()
        entries.append(e)
        if head_wl is None:
            head_wl = wl
    head = entries[0]
    out = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
        "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic",
        "config": {"workload": head["workload"], "batch": head["batch"], "weights": head["weights"],
                   "prefix": head["prefix"], "decode_steps": head["steps"], "repetitions": head["repetitions"],
                   "sampling": head["sampling"],
                   "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
                   "l2": "inputs larger than L2: %.0f MB of weights + KV stream per step" % (
                       head["roofline"]["algorithmic_bytes_per_step"] / 1e6),
                   "timed_region": "%d steps x %d repetitions = %.0f ms (streams re-opened outside the timing)" % (
                       head["steps"], head["repetitions"], head["timed_ms"])},
        "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "roofline": head["roofline"],
        "clocks": head["clocks"], "prefill": head["prefill"], "workloads": entries,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(head_wl, wcache)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


# ---------------------------------------------------------------------------------------------
# the oracle, as it stands, timed on the host cores
# ---------------------------------------------------------------------------------------------
def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_decode_rate(wl, weights, steps, context, threads=None):
    """Times `steps` cached decode steps of one stream of the workload's model in the oracle, at the
    given context.  The oracle's per-layer K/V lists are filled with `context` seeded random rows first
    (its step cost does not depend on the cached values), so that reaching the context costs no
    prefill.  threads: cap of the BLAS pool (None = as numpy starts it).  Returns (tokens/s, seconds)."""
    from oracle import gpt_oracle as O
    import contextlib
    model = O.OracleModel(wl.cfg, weights)
    st = O.OracleStream(model)
    rng = C.rng_for(wl.seed, 99)
    for l in range(model.n_layer):
        kv = rng.standard_normal(size=(2, context, model.d))
        st.k[l] = [kv[0, i] for i in range(context)]
        st.v[l] = [kv[1, i] for i in range(context)]
    st.ctx = context
    limit = contextlib.nullcontext()
    if threads is not None:
        from threadpoolctl import threadpool_limits
        limit = threadpool_limits(limits=threads, user_api="blas")
    tok = 1
    with limit:
        lg, _ = st.step(model.token_row(tok, 0))            # one untimed step
        tok = O.sample_greedy(lg)
        t0 = time.perf_counter()
        for k in range(steps):
            lg, _ = st.step(model.token_row(tok, (1 + k) % wl.cfg.max_pos))
            tok = O.sample_greedy(lg)
        dt = time.perf_counter() - t0
    return steps / dt, dt


def mid_context(wl):
    return int(np.mean(wl.prefix_lens)) + int(np.mean(wl.decode_lens)) // 2


def cpu_baseline(wl, wcache, steps=36):
    w = wcache.get(wl.cfg, wl.seed)
    ctx = mid_context(wl)
    all_rate, all_dt = oracle_decode_rate(wl, w, steps, ctx, None)
    cores = _blas_threads()
    one_rate, one_dt = oracle_decode_rate(wl, w, steps, ctx, 1)
    return {"value": all_rate, "unit": UNIT, "cores": cores, "kind": "oracle",
            "single_thread": {"value": one_rate, "unit": UNIT, "cores": 1},
            "sample": "%d consecutive single-stream decode steps of the %s model at context %d (the workload's "
                      "mid-run context; cache pre-filled with seeded random rows), once on all BLAS threads "
                      "(%.1f s) and once on one thread (%.1f s)" % (steps, C.WFMT_NAMES[wl.cfg.wfmt], ctx, all_dt, one_dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    key = [k.strip() for k in args.workloads.split(",") if k.strip()][0]
    idx, wfmt, kv_fmt = WORKLOAD_KEYS[key]
    wl = C.workload(idx, wfmt=wfmt, kv_fmt=kv_fmt)
    steps = max(1, min(args.steps, 400))
    w = C.make_weights(wl.cfg, seed=wl.seed)
    ctx = mid_context(wl)
    rate, dt = oracle_decode_rate(wl, w, steps, ctx, None)
    cores = _blas_threads()
    desc = "%d single-stream decode steps of the %s model at context %d (cache pre-filled with seeded random rows)" % (
        steps, C.WFMT_NAMES[wl.cfg.wfmt], ctx)
    out = {
        "impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": 1,
        "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.n_streams, "weights": C.WFMT_NAMES[wl.cfg.wfmt],
                   "note": "fp64 numpy oracle on the host cores; each step is one single-stream decode step"},
        "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def run_dry(args):
    """No GPU work: every rank joins a gloo group and the line is assembled from stand-in numbers
    through the same cross-rank reductions.  Checks the launcher and the reductions on a CPU machine."""
    import torch.distributed as dist
    from paper_2607_21042_b200 import replicas as R
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = 10.0 + rank
    tokens = 100
    value = R.whole_job_throughput(tokens, ms)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "dry_run": True,
                          "scaling": "weak", "config": {"workload": "none (launcher check)"}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workloads", default="2,3,4,5,5w4,5k8",
                    help="comma list of 1,2,3,4,5,5w8,5w4 and, on the 8-bit KV cache, 4k8,5k8,5w4k8; the first is the "
                         "headline of the JSON line")
    ap.add_argument("--workload", default=None, help="shorthand for --workloads with one entry")
    ap.add_argument("--min-seconds", type=float, default=0.5, help="lower bound of each workload's timed region")
    ap.add_argument("--max-reps", type=int, default=200)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run", action="store_true", help="launcher and reduction check without a GPU (gloo)")
    ap.add_argument("--profiler-range", nargs="?", const="decode", default=None, choices=["decode", "all"],
                    help="bracket the timed decode steps (or, with 'all', also the prefill call in front of them) with "
                         "cudaProfilerStart/Stop, for ncu --profile-from-start off")
    args = ap.parse_args()
    if args.workload is not None:
        args.workloads = str(args.workload)
    for k in args.workloads.split(","):
        if k.strip() not in WORKLOAD_KEYS:
            ap.error("unknown workload %r" % k)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: become N ranks, one per GPU
        from paper_2607_21042_b200 import replicas as R
        sys.exit(R.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

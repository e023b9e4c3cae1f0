#!/usr/bin/env python
"""Decode-throughput bench of the GPT decode step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2|3|4|5] [--impl ours|reference]

A step is one tts_gpt_decode_step over the workload's batch of streams (the whole hot path: embed,
24 blocks, final LayerNorm, LM head, sampling, page allocation).  Default workload: the 24-layer
bf16 decoder, batch 1, prefix 400, decode from context 400 (K = 500 steps reproduces 400 -> 900).
Prints ONE JSON line.  N > 1 runs independent replicas (one engine per GPU, no collective);
timing is the max over ranks.  `--impl reference` times the fp64 CPU oracle instead.
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


def algorithmic_bytes_per_step(cfg: C.GPTConfig, ctx_before):
    """Bytes the step must move: every weight byte once, every cached K/V byte of every active
    stream once plus the new K/V, the logits once.  ctx_before: context lengths before the step."""
    d, F, V, L = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_layer
    n_lin = 3 * d * d + d * d + 2 * d * F
    if cfg.wfmt == C.W_BF16:
        w = n_lin * 2
    elif cfg.wfmt == C.W_INT8_PC:
        w = n_lin + (3 * d + d + F + d) * 2
    else:
        w = n_lin // 2 + n_lin // 128 * 2
    small = (3 * d + d + F + d) * 2 + 4 * d * 2           # biases + LN per layer
    weights = L * (w + small) + V * d * 2 + 2 * d * 2
    kv_per_tok = 2 * d * 2 * L
    kv = sum((c + 1) * kv_per_tok for c in ctx_before)
    return weights + kv + len(ctx_before) * V * 4


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

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
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def make_prefix_tensors(wl, device):
    import torch
    out = []
    for p in C.make_prefixes(wl.cfg, wl.prefix_lens, seed=wl.seed):
        out.append(torch.from_numpy(p.view(np.int16)).to(device))
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2607_21042_b200 import binding as B
    from paper_2607_21042_b200 import replicas as R

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)

    wl = C.workload(args.workload, wfmt=args.wfmt)
    cfg = wl.cfg
    S = wl.n_streams
    K, W = args.steps, args.warmup
    max_dec = max(wl.decode_lens)
    if K > max_dec:
        K = max_dec
    weights = C.make_weights(cfg, seed=wl.seed)
    eng = B.TtsGpt(cfg, weights, device)
    del weights
    prefixes = make_prefix_tensors(wl, device)
    V, d = cfg.vocab, cfg.d_model
    uni = None
    if wl.top_k > 1:
        uni = torch.from_numpy(C.make_uniforms(K + W + 2, S, seed=wl.seed)).to(device)
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

    def decode_run(ids, n_steps, timed):
        """Queue n_steps steps back to back (tokens fed back on the device, no host sync)."""
        ctx = list(wl.prefix_lens)
        tokens = 0
        nbytes = 0
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
        for i, s in enumerate(ids):
            if i not in released:
                eng.release_stream(s)
        return tokens, nbytes

    # warm-up: open, W steps (captures the step graph), close
    ids = open_all()
    decode_run(ids, max(W, 3), False)
    eng.sync()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K steps, device-resident inputs ----
    ids = open_all()
    eng.sync()
    sampler = ClockSampler(local)
    l0 = eng.kernel_launches()
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if args.profiler_range:
        torch.cuda.profiler.start()
    with torch.cuda.stream(eng.stream):
        e0.record()
    tokens, nbytes = decode_run(ids, K, True)
    with torch.cuda.stream(eng.stream):
        e1.record()
    barrier()
    if args.profiler_range:
        torch.cuda.profiler.stop()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    launches = eng.kernel_launches() - l0
    total_tokens = R.sum_over_ranks(tokens, device)     # replicas: every rank decodes its own copy of the workload
    ms = R.max_over_ranks(ms, device)
    steps_done = min(K, max_dec)
    value = total_tokens / (ms * 1e-3)

    # ---- end to end: host buffers in, host buffers out, every step ----
    # (the prefix pass that opens the streams is timed on the way: prefix rows resident, first token out)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(eng.stream):
        p0.record()
    ids = open_all()
    with torch.cuda.stream(eng.stream):
        p1.record()
    eng.sync()
    prefill_ms = R.max_over_ranks(p0.elapsed_time(p1), device)
    prefill_rows = int(sum(wl.prefix_lens))
    n_e2e = min(K, 200)
    # One C-ABI call per step with HOST buffers (tts_gpt_decode_step_host): it copies the input tokens
    # in from page-locked memory, runs the step, copies token, logits and hidden rows back and returns
    # when they are valid.
    h_in = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_tok = torch.zeros(S, dtype=torch.int32).pin_memory()
    h_log = torch.zeros((S, V), dtype=torch.float32).pin_memory()
    h_hid = torch.zeros((S, d), dtype=torch.int16).pin_memory()
    h_uni = None if uni is None else uni.cpu().pin_memory()
    h_in.copy_(toks[0].cpu())
    d2h_bytes = 0
    all_ids = (ctypes.c_int32 * S)(*ids)      # marshalled once for the steps in which every stream is active
    barrier()
    t0 = time.perf_counter()
    e2e_tokens = 0
    for k in range(1, n_e2e + 1):
        act = active_at(k, ids)
        if not act:
            break
        n = len(act)
        sids = all_ids if n == S else [s for _, s in act]
        eng.decode_step_host(sids, h_tok, in_tokens=h_in, top_k=wl.top_k, temperature=wl.temperature,
                             uniforms=None if h_uni is None else h_uni[k], out_logits=h_log, out_hidden=h_hid)
        h_in[:n].copy_(h_tok[:n])
        e2e_tokens += n
        d2h_bytes = max(d2h_bytes, n * (4 + 4 * V + 2 * d))
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_total = R.sum_over_ranks(e2e_tokens, device)
    e2e_s = R.max_over_ranks(e2e_s, device)
    for s in ids:
        eng.release_stream(s)
    eng.sync()
    e2e = {"value": e2e_total / e2e_s, "unit": UNIT,
           "h2d_bytes_per_step": 4 * S, "d2h_bytes_per_step": int(d2h_bytes),
           "steps": n_e2e, "note": "one tts_gpt_decode_step_host call per step: tokens in from pinned host memory; tokens, logits and hidden rows back, valid on return"}

    peak, peak_kind = measured_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    # DRAM bytes per step from ncu captures of one decode step (dram__bytes_read.sum + dram__bytes_write.sum
    # over its launches; the summaries sit with the other profiles of this repository).  Workload 2:
    # 1022.7 MB read+written for a step whose algorithmic bytes are 1015.1 MB (context 405).  Workload 5,
    # bf16: 12155.3 MB for a step of 11930.8 MB.  Traffic grows with the same KV term as the algorithmic
    # bytes, so the measured ratio is applied to this run's bytes per step.
    traffic = None
    if args.workload == 2:
        traffic = (nbytes / max(steps_done, 1)) * (1022.7 / 1015.1)
    elif args.workload == 5 and cfg.wfmt == 0:
        traffic = (nbytes / max(steps_done, 1)) * (12155.3 / 11930.8)
    roofline = {"bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s", "frac": gbs / peak,
                "traffic": traffic, "peak_source": peak_kind,
                "kernel": "whole decode step (CUDA graph of %d kernels)" % (launches // max(steps_done, 1) - 1),
                "algorithmic_bytes_per_step": nbytes / max(steps_done, 1)}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps_done, "warmup": max(W, 3),
        "ms_per_step": ms / max(steps_done, 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "batch": S, "weights": C.WFMT_NAMES[cfg.wfmt],
                   "prefix": [min(wl.prefix_lens), max(wl.prefix_lens)], "decode_steps": steps_done,
                   "sampling": "greedy" if wl.top_k <= 1 else "top-k %d" % wl.top_k,
                   "parallelism": "replicas x%d" % world if world > 1 else "single GPU",
                   "l2": "inputs larger than L2: %.0f MB of weights + KV stream per step" % (nbytes / max(steps_done, 1) / 1e6)},
        "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "clocks": clocks,
        "tokens": tokens, "launches_before_timed_region": int(l0),
        "prefill": {"rows": prefill_rows, "streams": S, "ms": prefill_ms,
                    "rows_per_s": world * prefill_rows / (prefill_ms * 1e-3),
                    "note": "one prefill call over all prefixes (device resident), first token sampled; outside the timed region"},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, budget_steps=args.cpu_steps)
    eng.destroy()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def _oracle_setup(wl):
    from oracle import gpt_oracle as O
    cfg = wl.cfg
    w = C.make_weights(cfg, seed=wl.seed)
    model = O.OracleModel(cfg, w)
    del w
    return O, model


def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_decode_rate(wl, warm, steps, prefix_rows=64):
    """Times the oracle, as it stands, on `steps` cached decode steps per stream of the workload's
    model after a short prefix (its step cost is dominated by the fp64 weight matrices, so a short
    context is representative).  Returns (tokens/s, seconds, description)."""
    O, model = _oracle_setup(wl)
    P = O.bf16_to_f64(C.make_prefixes(wl.cfg, [prefix_rows], seed=wl.seed)[0])
    st = O.OracleStream(model)
    lg = None
    for r in range(prefix_rows):
        lg, _ = st.step(P[r])
    tok = O.sample_greedy(lg)
    for k in range(warm):
        lg, _ = st.step(model.token_row(tok, k))
        tok = O.sample_greedy(lg)
    t0 = time.perf_counter()
    for k in range(steps):
        lg, _ = st.step(model.token_row(tok, (warm + k) % wl.cfg.max_pos))
        tok = O.sample_greedy(lg)
    dt = time.perf_counter() - t0
    desc = "%d single-stream decode steps of the %s model at context %d..%d after a %d-row prefix" % (
        steps, C.WFMT_NAMES[wl.cfg.wfmt], prefix_rows + warm, prefix_rows + warm + steps, prefix_rows)
    return steps / dt, dt, desc


def cpu_baseline(wl, budget_steps=150):
    rate, dt, desc = oracle_decode_rate(wl, warm=2, steps=budget_steps)
    return {"value": rate, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
            "sample": desc + " (%.1f s)" % dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = C.workload(args.workload, wfmt=args.wfmt)
    steps = min(args.steps, 2000)
    rate, dt, desc = oracle_decode_rate(wl, warm=max(args.warmup, 1), steps=steps)
    cores = _blas_threads()
    out = {
        "impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": steps, "warmup": max(args.warmup, 1),
        "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.n_streams, "weights": C.WFMT_NAMES[wl.cfg.wfmt],
                   "note": "fp64 numpy oracle on the host cores; each step is one single-stream decode step"},
        "cpu_baseline": {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--wfmt", type=int, default=None, help="weight format override for workload 5")
    ap.add_argument("--cpu-steps", type=int, default=150)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profiler-range", action="store_true",
                    help="bracket the timed region with cudaProfilerStart/Stop (for ncu --profile-from-start off)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

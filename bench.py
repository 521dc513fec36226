#!/usr/bin/env python
"""Benchmark of the IPPD decode-attention hot path (question-tokens/s and roofline fractions).

A "step" is one IPPD decode step of a workload: for every layer, RoPE + append of the step's K/V and the decode
attention over the shared context and the private branches, for all questions still active (one ippd_decode_step call
over all layers by default).  Inputs are seeded and synthetic (workloads.py).  Before anything is timed, the K/V of
EVERY step of the schedule is written into the cache (a token's slot depends only on its question and step index), so
the K timed steps are spread evenly over the whole schedule instead of being its first K.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config C4] [--also C2,C3,C5] [--impl ours|reference]

Prints ONE JSON line.  The headline workload is C4 (the largest Llama-3-8B-geometry configuration that fits one GPU);
`per_config` carries the same measurements for the other configurations (C2, C3, C5 and the second family S1, S2, S3).  With N > 1 (launched by torchrun) every rank
runs an independent replica of the workload on its own GPU: the path is never sharded, there is no data-path
collective.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "IPPD decode-attn question-tokens/s"
UNIT = "question-tokens/s"
HEADLINE = "C4"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic byte of the attention kernel, from ncu
# captures of two launches each (summaries under profiles/: tcgen05_path_C2_attn_full_set.md and
# tcgen05_path_dram_traffic_C3_C4_C5_S3.md; C4 and S3 captured with fewer layers, traffic per launch grows in proportion
# to the layers); the traffic of an average launch is that ratio times its algorithmic bytes.  C5's ratio depends on
# how many 128-row blocks a prompt still has (2.5 .. 4.8 over its schedule): no single figure, reported as null.
NCU_TRAFFIC_RATIO = {"C2": 1.040, "C3": 1.009, "C4": 1.238, "S3": 2.031}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 1400.0)),
                    "kind": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops_sustained": 1400.0, "kind": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr:
            self._thr.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_sample_items(wl):
    """Inputs of the timed oracle sample: all questions of prompt 0 (at most 16) at the first, middle and last step,
    layer 0, KV head 0, assembled by the oracle's own tuple_inputs.  Generated once, outside every timed region."""
    from oracle import ippd_oracle as orc
    steps = sorted({0, wl.n_steps // 2, wl.n_steps - 1})
    items, ctx_cache = [], {}
    for s in steps:
        for k in [k for k in wl.active(s) if wl.prompt_of[k] == 0][:16]:
            items.append(orc.tuple_inputs(wl, 0, int(k), s, 0, 0, ctx_cache))
    return items, steps


def oracle_sample_rate(wl, budget_s: float, sample=None):
    """Times the fp64 oracle (as it stands) on a bounded sample of the workload on the host cores.

    One question-token = the oracle evaluated for every layer and KV head of one (question, step).  The sample is
    cycled through until the time budget is spent; the rate is an EXTRAPOLATION from those calls.
    Returns (q-tokens/s, calls, text)."""
    from oracle import ippd_oracle as orc
    g = wl.geom
    items, steps = sample if sample is not None else oracle_sample_items(wl)
    calls, t0, el = 0, time.perf_counter(), 0.0
    while el < budget_s or calls < 8:
        kk, vv, qq = items[(calls * 7) % len(items)]  # 7 is coprime to the sample size: the steps alternate
        orc.standalone_attend(kk, vv, qq, g.rope_theta)
        calls += 1
        el = time.perf_counter() - t0
    per_token = g.n_layers * g.n_kv_heads
    rate = calls / per_token / el
    text = (f"{calls} oracle calls (one (question, step, layer, KV head) each; steps {steps} of prompt 0, layer 0, "
            f"head 0) in {el:.1f} s, extrapolated by {per_token} calls per question-token")
    return rate, calls, text


def blas_threads():
    """(threads the BLAS pool may use, how the number was obtained)."""
    try:
        from threadpoolctl import threadpool_info
        pools = [i.get("num_threads", 1) for i in threadpool_info()]
        n = max(pools + [1])
        how = "largest BLAS pool reported by threadpoolctl, capped by the CPU affinity mask"
    except Exception:
        n, how = 1, "threadpoolctl unavailable: 1 assumed"
    return min(n, len(os.sched_getaffinity(0))), how


def cpu_baseline(wl, budget_s):
    sample = oracle_sample_items(wl)
    rate, calls, text = oracle_sample_rate(wl, budget_s * 0.7, sample)
    cores, how = blas_threads()
    single = None
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            single, c1, _ = oracle_sample_rate(wl, budget_s * 0.3, sample)
    except Exception:
        pass
    return {"value": rate, "unit": UNIT, "cores": cores, "cores_how": how, "kind": "oracle", "sample": text,
            "extrapolated": True, "oracle_calls_timed": calls, "single_thread_value": single}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # the whole run stays within about two minutes whatever K is: each step gets its share of that time
    per_step = max(0.03, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    sample = oracle_sample_items(wl)
    for _ in range(args.warmup):
        oracle_sample_rate(wl, per_step / 4, sample)
    rates, n_calls, t0 = [], 0, time.perf_counter()
    text = ""
    for _ in range(args.steps):
        r, calls, text = oracle_sample_rate(wl, per_step, sample)
        rates.append(r)
        n_calls += calls
    el = time.perf_counter() - t0
    value = float(np.mean(rates))
    cores, how = blas_threads()
    toks_per_step = wl.question_tokens() / wl.n_steps
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * toks_per_step / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "extrapolated": True, "oracle_calls_timed": n_calls,
            "config": {"workload": wl.name, "note": "CPU fp64 oracle; each step is a bounded sample of the workload and "
                       "ms_per_step is extrapolated from the sampled calls, not timed"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "cores_how": how, "kind": "oracle",
                             "sample": text, "extrapolated": True, "oracle_calls_timed": n_calls},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "wall_s": el}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- CUDA arm
def spread_steps(n_steps: int, count: int):
    """`count` step indices spread evenly over a schedule of n_steps steps (cycling when count > n_steps)."""
    if count >= n_steps:
        return [i % n_steps for i in range(count)]
    return [int((i + 0.5) * n_steps / count) for i in range(count)]


class ConfigBench:
    """One workload resident on the device, every step's K/V already in the cache."""

    def __init__(self, name, dev, kernel, max_resident_bytes=24e9, n_layers=0):
        import torch
        from paper_2609_05707_b200 import binding as B
        from paper_2609_05707_b200 import workloads as W
        from paper_2609_05707_b200.runner import Runner
        self.torch = torch
        base, _, kv = name.partition("/")  # "C3/e4m3": workload C3 on the 8-bit cache variant
        if kv not in ("", "e4m3"):
            raise SystemExit(f"unknown cache variant in {name!r}")
        self.kv_elem_bytes = 1 if kv == "e4m3" else 2
        self.wl = wl = W.make_workload(base, n_layers or None)
        self.g = g = wl.geom
        self.dev = dev
        self.run = Runner(wl, dev, kernel=kernel, layers_per_call=g.n_layers,
                          kv_dtype=B.KV_E4M3 if kv == "e4m3" else B.KV_BF16)
        self.run.load_header()
        self.run.append_all_steps()
        self.run.check()
        self.max_resident_bytes = max_resident_bytes
        self.inputs = {}

    def close(self):
        self.inputs.clear()
        del self.run
        self.torch.cuda.empty_cache()

    def prepare(self, steps):
        """Raw q/k/v of the given steps resident in HBM (bounded: the caller's step list may be cut)."""
        wl, g = self.wl, self.g
        per_tok = g.n_layers * (g.n_q_heads * 2 + g.n_kv_heads * 2) * g.head_dim * 2  # q, k, v and out, bf16
        used, keep = 0, []
        for s in steps:
            need = 0 if s in self.inputs or s in keep else len(wl.active(s)) * per_tok
            if used + need > self.max_resident_bytes:
                break
            used += need
            keep.append(s)
        for s in dict.fromkeys(keep):
            if s not in self.inputs:
                act = wl.active(s)
                q, k, v = self.run.step_inputs(s, act)
                out = self.torch.empty((g.n_layers, len(act), g.n_q_heads, g.head_dim), dtype=self.torch.bfloat16,
                                       device=self.dev)
                self.inputs[s] = (act, np.full(len(act), s, dtype=np.int32), q, k, v, out)
        return keep

    def step(self, s):
        act, idx, q, k, v, out = self.inputs[s]
        self.run.decode_step(act, idx, q, k, v, out)

    def timed(self, warm, steps, sync):
        """Device time (ms) of `steps`, CUDA events on the launching stream, after `warm` untimed steps."""
        torch = self.torch
        for s in warm:
            self.step(s)
        self.run.check()
        sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in steps:
            self.step(s)
        e1.record()
        sync()
        return e0.elapsed_time(e1)

    def profile(self, steps):
        """Every launch of `steps` bracketed by CUDA events (a pass of its own: the brackets slow the stream)."""
        from paper_2609_05707_b200 import binding as B
        lay = self.run.layout
        lay.profile_read()
        lay.set_option(B.OPT_PROFILE, 1)
        for s in steps:
            self.step(s)
        prof = lay.profile_read()
        lay.set_option(B.OPT_PROFILE, 0)
        return prof

    def prefill(self, peaks, layers=2, reps=2):
        """ippd_prefill_attention over the first `layers` layers of the stacked header: device time per layer and the
        fraction of the sustained bf16 tensor peak (the prefill is a dense contraction: every 128-row block of header
        tokens streams all key tiles up to its own position)."""
        from paper_2609_05707_b200 import binding as B
        torch = self.torch
        run, wl, g = self.run, self.wl, self.g
        layers = min(layers, g.n_layers)
        qkv = [run.header_inputs(l) for l in range(layers)]
        q = torch.stack([t[0] for t in qkv]).contiguous()
        k = torch.stack([t[1] for t in qkv]).contiguous()
        v = torch.stack([t[2] for t in qkv]).contiguous()
        del qkv
        n_hdr = q.shape[1]
        out = torch.empty((layers, n_hdr, g.n_q_heads, g.head_dim), dtype=torch.bfloat16, device=self.dev)
        ws = torch.empty(run.layout.workspace_bytes(layers), dtype=torch.uint8, device=self.dev)
        lay = run.layout
        lay.prefill_attention(0, layers, q, k, v, out, ws, run.stream)  # untimed
        torch.cuda.synchronize()
        lay.profile_read()
        lay.set_option(B.OPT_PROFILE, 1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            lay.prefill_attention(0, layers, q, k, v, out, ws, run.stream)
        e1.record()
        torch.cuda.synchronize()
        prof = lay.profile_read()
        lay.set_option(B.OPT_PROFILE, 0)
        run.check()
        # keys every header row sees: instruction and context rows up to themselves, question rows the instruction,
        # their context and their question's prefix
        P = wl.shared_len
        keys = P * (P + 1) // 2
        for b in range(wl.n_prompts):
            L = int(wl.ctx_len[b])
            keys += L * P + L * (L + 1) // 2
            for kq in range(int(wl.q_begin[b]), int(wl.q_begin[b + 1])):
                n = int(wl.q_len[kq])
                keys += n * (P + L) + n * (n + 1) // 2
        flops = 4 * g.head_dim * g.n_q_heads * keys * layers * reps
        att_ms = prof["attention_ms"] + prof["merge_ms"]
        tflops = flops / (att_ms * 1e-3) / 1e12 if att_ms > 0 else 0.0
        return {"header_tokens": int(n_hdr), "layers_per_call": layers, "calls_timed": reps,
                "ms_per_layer_whole_call": e0.elapsed_time(e1) / (layers * reps),
                "attention_ms_per_layer": att_ms / (layers * reps), "tflops": tflops,
                "roofline": {"bound": "tensor", "achieved": tflops, "peak": peaks["bf16_tflops_sustained"],
                             "unit": "TFLOP/s", "frac": tflops / peaks["bf16_tflops_sustained"],
                             "peak_kind": peaks["kind"] + " sustained cuBLAS bf16"},
                "api": "ippd_prefill_attention (header K/V append + attention of every header token)"}

    def read_probe(self, steps):
        """GB/s of the tile stream alone (the attention kernel's copies without its arithmetic) over `steps`."""
        torch = self.torch
        lay, g = self.run.layout, self.g
        tot_ms, tot_bytes = 0.0, 0
        for i, s in enumerate(steps):
            act, idx = self.inputs[s][0], self.inputs[s][1]
            if len(act) == 0:
                continue
            lay.begin_step(act, idx, self.run.stream)
            lay.read_probe(0, g.n_layers, self.run.stream)  # untimed: uploads the descriptor, warms the path
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            lay.read_probe(0, g.n_layers, self.run.stream)
            e1.record()
            torch.cuda.synchronize()
            b = self.wl.step_bytes(s, self.kv_elem_bytes)
            tot_ms += e0.elapsed_time(e1)
            tot_bytes += b["context"] + b["branch"]
        self.run.check()
        return tot_bytes / (tot_ms * 1e-3) / 1e9 if tot_ms > 0 else None


def measure_config(name, args, dev, peaks, sync, want_layer_modes, rank_world):
    """All device-resident measurements of one configuration; returns (entry dict, ConfigBench)."""
    cb = ConfigBench(name, dev, args.kernel, n_layers=args.layers)
    wl, g = cb.wl, cb.g
    timed = cb.prepare(spread_steps(wl.n_steps, args.steps))
    warm = cb.prepare(spread_steps(wl.n_steps, args.warmup))
    if len(timed) < args.steps:  # memory bound on the resident inputs: cycle through those that fit
        timed = [timed[i % len(timed)] for i in range(args.steps)]
    if not warm:
        warm = timed[:args.warmup]
    warm = [warm[i % len(warm)] for i in range(args.warmup)]
    ms = cb.timed(warm, timed, sync)
    tokens = sum(len(wl.active(s)) for s in timed)
    # kernel times: a separate pass with every launch bracketed, at least 16 launches
    prof_steps = [timed[i % len(timed)] for i in range(max(16, len(timed)))]
    prof = cb.profile(prof_steps)
    n_att = max(1, prof["n_attention"])
    kvb = cb.kv_elem_bytes
    bytes_total = sum(wl.step_bytes(s, kvb)["total"] for s in prof_steps)
    flops_total = sum(wl.step_flops(s) for s in prof_steps)
    call_ms = prof["attention_ms"] + prof["merge_ms"]  # the ippd_decode_attention / ippd_decode_step time
    achieved = bytes_total / (call_ms * 1e-3) / 1e9 if call_ms > 0 else 0.0
    kernel_gbs = bytes_total / (prof["attention_ms"] * 1e-3) / 1e9 if prof["attention_ms"] > 0 else 0.0
    tflops = flops_total / (call_ms * 1e-3) / 1e12 if call_ms > 0 else 0.0
    tensor_bound = name.startswith("C5")  # R = 2048 query rows per KV head: 580 flop per byte, above the ridge
    ratio = NCU_TRAFFIC_RATIO.get(name) if args.kernel in (0, 2) else None
    roof = {"bound": "tensor" if tensor_bound else "hbm",
            "achieved": tflops if tensor_bound else achieved,
            "peak": peaks["bf16_tflops_sustained"] if tensor_bound else peaks["hbm_gbs"],
            "unit": "TFLOP/s" if tensor_bound else "GB/s",
            "traffic": ratio * bytes_total / n_att if ratio else None,
            "peak_kind": peaks["kind"] + (" sustained cuBLAS bf16" if tensor_bound else " copy bandwidth"),
            "timed_kernels": "attention kernel (RoPE + append of the step's tokens inside) + merge kernel",
            "launches": n_att, "avg_call_us": 1e3 * call_ms / n_att,
            "algorithmic_bytes_per_launch": bytes_total / n_att, "algorithmic_flops_per_launch": flops_total / n_att,
            "hbm_gbs": achieved, "frac_of_8TBs": achieved / 8000.0, "tflops": tflops,
            "attention_kernel_only": {"avg_launch_us": 1e3 * prof["attention_ms"] / n_att, "hbm_gbs": kernel_gbs,
                                      "frac": kernel_gbs / peaks["hbm_gbs"], "frac_of_8TBs": kernel_gbs / 8000.0},
            "merge_us_per_call": 1e3 * prof["merge_ms"] / n_att, "append_us_per_call": 1e3 * prof["append_ms"] / n_att}
    roof["frac"] = roof["achieved"] / roof["peak"]
    probe = cb.read_probe(timed[:: max(1, len(timed) // 8)][:8]) if args.kernel in (0, 2) else None
    entry = {"value": rank_world * tokens / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms / len(timed),
             "steps": len(timed), "question_tokens": tokens, "schedule_steps_timed": sorted(set(timed)),
             "layers_per_call": g.n_layers, "roofline": roof, "read_probe_gbs": probe,
             "shape": {"prompts": wl.n_prompts, "questions": wl.n_questions, "layers": g.n_layers,
                       "q_heads": g.n_q_heads, "kv_heads": g.n_kv_heads, "head_dim": g.head_dim,
                       "decode_steps_in_schedule": wl.n_steps, "kv_cache_mb": cb.run.cache.numel() / 1e6,
                       "mb_streamed_per_step_min_mean_max": [round(x / 1e6, 1) for x in (
                           min(wl.step_bytes(s, kvb)["total"] for s in range(wl.n_steps)),
                           float(np.mean([wl.step_bytes(s, kvb)["total"] for s in range(wl.n_steps)])),
                           max(wl.step_bytes(s, kvb)["total"] for s in range(wl.n_steps)))]}}
    if kvb == 1:
        entry["kv_cache"] = ("e4m3: rotated keys and values stored as 8-bit numbers; the byte figures count one byte per "
                             "cache element, question-tokens/s compares directly with the bf16 entry of the workload")
    if want_layer_modes and args.kernel in (0, 2):
        entry["prefill"] = cb.prefill(peaks)
    if want_layer_modes:
        modes = {}
        for lpc in (1, 4, 8):
            if lpc >= g.n_layers:
                continue
            cb.run.set_layers_per_call(lpc)
            n0 = cb.run.layout.launch_count()
            m = cb.timed(warm[:3], timed, sync)
            n1 = cb.run.layout.launch_count()
            pm = cb.profile(timed[: max(1, 16 // max(1, g.n_layers // lpc)) + 1])  # every launch bracketed
            calls = max(1, pm["n_attention"])
            modes[str(lpc)] = {"layers_per_call": lpc, "ms_per_step": m / len(timed),
                               "value": rank_world * tokens / (m * 1e-3),
                               "launches_per_step": (n1 - n0) / (len(timed) + 3),
                               "us_per_call": 1e3 * m / len(timed) / -(-g.n_layers // lpc),
                               "bracketed_attention_us_per_call": 1e3 * pm["attention_ms"] / calls,
                               "bracketed_merge_us_per_call": 1e3 * pm["merge_ms"] / calls}
        cb.run.set_layers_per_call(g.n_layers)
        entry["per_layer_mode"] = modes.get("1")
        entry["layer_group_modes"] = modes
        entry["note_layer_modes"] = ("all layers in one launch needs every layer's q/k/v before layer 0 runs, which "
                                     "only independent synthetic layers can supply: an upper bound; layers_per_call = 1 "
                                     "is the launch pattern of a real model (its own work between the launches left out)")
    return entry, cb, (ms, tokens, timed, warm)


def measure_e2e(cb, args, timed, warm, sync, world):
    """The same steps through ippd_decode_step_host_async with pinned host buffers (copies inside the timed region)."""
    import torch
    from paper_2609_05707_b200 import replicas
    run, wl = cb.run, cb.wl
    uniq = list(dict.fromkeys(timed))[:8]  # pinned copies of at most eight distinct steps
    host_in = {s: tuple(t.cpu().pin_memory() for t in cb.inputs[s][2:5]) for s in uniq}
    host_out = {s: torch.empty(cb.inputs[s][5].shape, dtype=torch.bfloat16).pin_memory() for s in uniq}
    amax = max(len(cb.inputs[s][0]) for s in uniq)
    stage = torch.empty(2 * run.layout.step_stage_bytes(amax), dtype=torch.uint8, device=cb.dev)

    def e2e_step(s):
        act, idx = cb.inputs[s][0], cb.inputs[s][1]
        hq, hk, hv = host_in[s]
        run.layout.decode_step_host_async(act, idx, hq, hk, hv, host_out[s], stage, run.workspace, run.stream)

    order = [uniq[i % len(uniq)] for i in range(len(timed))]
    for i in range(min(args.warmup, 8)):
        e2e_step(order[i % len(order)])
    run.layout.host_steps_wait(run.stream)
    sync()
    run.layout.host_time_read()
    # host clock around the loop and the final wait: the last copy-out runs on the library's copy stream, which an
    # event on the compute stream would not cover
    t0 = time.perf_counter()
    for s in order:
        e2e_step(s)
    t_enq = time.perf_counter()
    run.layout.host_steps_wait(run.stream)
    ems = 1e3 * (time.perf_counter() - t0)
    sync()
    host = run.layout.host_time_read()
    ems = replicas.max_over_ranks(ems, cb.dev)
    tokens = sum(len(cb.inputs[s][0]) for s in order)
    h2d = sum(sum(t.numel() * t.element_size() for t in host_in[s]) for s in order) / len(order)
    d2h = sum(host_out[s].numel() * 2 for s in order) / len(order)
    run.check()
    return {"value": world * tokens / (ems * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": len(order), "ms_per_step": ems / len(order),
            "api": "ippd_decode_step_host_async + ippd_host_steps_wait",
            "timer": "host clock around the calls and the final wait",
            "host_us_per_step": 1e6 * (t_enq - t0) / len(order),
            "host_begin_step_us_per_step": host["begin_step_us"] / max(1, host["steps"]),
            "pcie_gbs": (h2d + d2h) * len(order) / (ems * 1e-3) / 1e9,
            "note": "host_us_per_step = host time to enqueue a step (planning, staging, launches, copies); the step "
                    "is PCIe-bound when pcie_gbs sits at the link's rate and host-bound when host_us_per_step equals "
                    "ms_per_step"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default=HEADLINE, help="headline workload")
    ap.add_argument("--also", default=None, help="comma-separated other workloads for per_config ('' = none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-layer-modes", action="store_true", help="skip the per-layer launch modes and the prefill")
    ap.add_argument("--kv-dtype", default="bf16", choices=["bf16", "e4m3"],
                    help="cache element type of --config and of the --sweep table (a name in --also takes /e4m3)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiler captures)")
    ap.add_argument("--sweep", action="store_true",
                    help="questions-per-context x context-length table (the SWEEP-L*-Q* workloads) instead of the headline line")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2609_05707_b200 import workloads as W
    if args.impl == "reference":
        run_reference(args, W.make_workload(args.config))
        return

    import torch
    import torch.distributed as dist
    from paper_2609_05707_b200 import build as ippd_build
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the IPPD library has no CPU fallback")
    if rank == 0 or world == 1:
        ippd_build.build()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2609_05707_b200 import replicas

    dev = f"cuda:{local_rank}"
    peaks = load_peaks()
    also = args.also
    if also is None:
        also = ",".join(c for c in ("C2", "C3", "C5", "S1", "S2", "S3", "C2/e4m3", "C3/e4m3") if c != args.config) \
            if (args.config == HEADLINE and world == 1) else ""
    others = [c for c in also.split(",") if c]

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    kv_suffix = "/e4m3" if args.kv_dtype == "e4m3" else ""
    if args.sweep:
        # the axes of the paper's ablations: one JSON line holding the whole table
        from paper_2609_05707_b200 import workloads as W2
        args.no_layer_modes = True
        rows = []
        for L in W2.SWEEP_CONTEXTS:
            for Q in W2.SWEEP_QUESTIONS:
                e, c, _ = measure_config(f"SWEEP-L{L}-Q{Q}" + kv_suffix, args, dev, peaks, sync_all, False, 1)
                c.close()
                r = e["roofline"]
                rows.append({"context": L, "questions": Q, "ms_per_step": e["ms_per_step"], "value": e["value"],
                             "call_us": r["avg_call_us"], "hbm_gbs": r["hbm_gbs"], "frac_of_8TBs": r["frac_of_8TBs"],
                             "frac": r["frac"], "read_probe_gbs": e["read_probe_gbs"]})
        if rank == 0:
            print(json.dumps({"metric": METRIC, "unit": UNIT, "kv_cache": args.kv_dtype, "sweep": rows, "steps": args.steps, "warmup": args.warmup,
                              "peak": peaks}), flush=True)
        return

    # ---- headline configuration ----
    t_wall0 = time.perf_counter()
    entry, cb, (ms, tokens, timed, warm) = measure_config(args.config + kv_suffix, args, dev, peaks, sync_all,
                                                          not args.no_layer_modes, 1)
    # headline figure: the timed region once more, clocks sampled while it runs
    sampler = ClockSampler(local_rank)
    for s in warm:
        cb.step(s)
    sampler.start()
    launches0 = cb.run.layout.launch_count()
    ms = cb.timed([], timed, sync_all)
    launches = cb.run.layout.launch_count() - launches0
    clocks = sampler.stop()
    value = replicas.whole_job_rate(tokens, ms, dev)  # N independent replicas; the slowest rank sets the time
    ms = replicas.max_over_ranks(ms, dev)
    e2e = None if args.no_e2e else measure_e2e(cb, args, timed, warm, sync_all, world)
    wl, g = cb.wl, cb.g
    cache_mb = cb.run.cache.numel() / 1e6
    cb.close()

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wl, 14.0)

    per_config = {args.config + kv_suffix: entry}
    for name in others:
        e, c, _ = measure_config(name, args, dev, peaks, sync_all, name == "C2" and not args.no_layer_modes, 1)
        c.close()
        per_config[name] = e

    if rank == 0:
        sb = entry["shape"]["mb_streamed_per_step_min_mean_max"]
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / len(timed), "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if not kv_suffix else "bf16 inputs and outputs, e4m3 cache",
                "data": "synthetic",
                "config": {"workload": wl.name, "prompts": wl.n_prompts, "questions": wl.n_questions,
                           "layers": g.n_layers, "q_heads": g.n_q_heads, "kv_heads": g.n_kv_heads,
                           "head_dim": g.head_dim, "decode_steps_in_schedule": wl.n_steps,
                           "layers_per_call": g.n_layers, "schedule_steps_timed": entry["schedule_steps_timed"],
                           "parallelism": f"replicas x{world}" if world > 1 else "1 gpu",
                           "l2": f"no flush: a step streams {sb[0]:.0f}..{sb[2]:.0f} MB (mean {sb[1]:.0f}) of a "
                                 f"{cache_mb:.0f} MB K/V cache, larger than the 126 MB L2"},
                "roofline": entry["roofline"], "read_probe_gbs": entry["read_probe_gbs"],
                "per_layer_mode": entry.get("per_layer_mode"), "layer_group_modes": entry.get("layer_group_modes"),
                "prefill": entry.get("prefill"),
                "per_config": per_config, "e2e": e2e, "cpu_baseline": cpu, "gpu_launches": int(launches),
                "clocks": clocks, "question_tokens": tokens, "wall_s": time.perf_counter() - t_wall0}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

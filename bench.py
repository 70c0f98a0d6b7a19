#!/usr/bin/env python
"""Benchmark of the AMS compression step (score + segment + select + compact).

One "step" is one `ams_compress` call over the whole layer stack of a workload.

Headline (`value`, `ms_per_step`, `roofline`, `e2e`, `cpu_baseline`): the largest of the five
benchmark configurations that fits one GPU, configuration 4 (Llama-3.1-70B-shaped stack: 80 layers,
64 q / 8 KV heads, one sequence of 131072 cached bf16 tokens in 16-token pages compressed to 8192,
observation window 64, 32 mass quantiles), first event.  `per_config` then carries all five
configurations, each timed in the same process on freshly generated inputs: first event, and for
the two multi-event configurations (2: 20 events with 128 appended tokens; 4: 8 events with 512)
the steady-state events 2..N run as real successive events with the EMA state carried.
Configuration 3 (309 GB of K/V) does not fit: four of its 36 layers are resident and one launch
covers those four; its figures are per such launch.

With N > 1 every rank runs its own replica of the workload (the units of the path are independent:
no collective on the data path; weak scaling).  `--gpus N` without a launcher spawns the N ranks
itself; under torchrun it must agree with WORLD_SIZE.

Prints ONE JSON line (rank 0).  `value` = whole-job steps/s with the cache resident in HBM, timed
with CUDA events on the launching stream.  `e2e` = the same through the C ABI with the step's
inputs (observation queries, block table, lengths, replacement pages) copied from pinned host
memory and its results (block table, lengths) read back and checked inside the timed region; the
paged K/V pool is the persistent device state the step operates on and is not copied.
"""
from __future__ import annotations

import argparse
import gc
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "ams_compress_steps_per_s"
UNIT = "steps/s"
HEADLINE_CFG = 4
L2_BYTES = 126 << 20
MUFU_PER_CLK_PER_SM = 16          # special-function results per clock and SM (exp2)
N_SM = 148


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", 1590.0)),
                "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "kind": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0, "kind": "fallback"}


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch from ncu captures summarised under
# profiles/ (workload -> kernel slot -> bytes per launch).  A kernel or workload without a capture of the
# current code reports null.
NCU_TRAFFIC_BYTES: dict = {
    # two-layer capture (profiles/tc_scorer_cfg4_2layers_ncu_full.md) x 40: the 80-layer launch holds 50 GB, too much to
    # capture under full counters; units are independent and each is read once per pass, so traffic grows with the layers
    "cfg4_llama70b_L80_T131072_k8192_w64": {"score_phase1": 40 * (540_616_448 + 6_414_080),
                                            "score_phase2": 40 * (542_741_760 + 11_199_488)},
    # captured at the timed size (profiles/tc_scorer_cfg1_32layers_ncu_full.md, profiles/gather_cfg1_cfg2_ncu_full.md)
    "cfg1_llama8b_L32_T16384_k2048_w32": {"score_phase1": 1_089_513_472 + 14_958_336,
                                          "score_phase2": 1_090_619_136 + 20_133_632,
                                          "gather": 270_614_528 + 219_303_168},
    # one-layer capture x 4 resident layers (profiles/keydiff_cfg3_1layer_ncu_full.md)
    "cfg3_qwen3_8b_L36_B64_T32768_k2048_keydiff": {"score_phase1": 4 * (4_295_511_552 + 7_466_752),
                                                   "score_phase2": 4 * (4_296_070_144 + 16_274_688)},
    # four-layer capture x 8 (profiles/expected_attention_cfg5_4layers_ncu_full.md)
    "cfg5_llama8b_L32_T16384_k2048_expected": {"score_phase1": 8 * (138_547_456 + 6_842_624),
                                               "score_phase2": 8 * (142_662_656 + 4_295_936)},
}


def config_dict(wl) -> dict:
    """What defines the workload of a line (the same for both arms)."""
    why = ("largest of the five configurations that fits one GPU (configuration 3 needs 309 GB)" if wl.cfg_id == HEADLINE_CFG
           else "chosen with --config")
    return {"workload": wl.name, "layers": wl.n_layers, "layers_resident": wl.layers_resident, "q_heads": wl.n_q_heads,
            "kv_heads": wl.n_kv_heads, "batch_per_gpu": wl.batch, "cache_tokens": wl.seq_len_max, "budget": wl.budget,
            "window": wl.window, "n_segments": wl.n_segments, "scorer": SCORER_NAMES[wl.scorer_id],
            "event": "first event (cache at full length); steady-state events are under per_config",
            "why_this_workload": why}


def algorithmic_bytes(wl, lens) -> tuple[int, int]:
    """(K bytes read once for scoring, kept K/V bytes read + written) per step."""
    units = wl.layers_resident * wl.n_kv_heads
    live = [int(t) for t in lens if int(t) > wl.budget]
    k_read = units * sum(live) * (512 if wl.scorer_id == 3 else 256)   # the expected-attention scorer also reads V (value norms)
    moved = units * len(live) * wl.budget * 2 * 256 * 2
    return k_read, moved


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read-only) while timing runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {getattr(nv, n): n for n in dir(nv) if n.startswith("nvmlClocksEventReason") or n.startswith("nvmlClocksThrottleReason")}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if isinstance(bit, int) and bit and mask & bit and bin(bit).count("1") == 1:
                        self.reasons.add(name.replace("nvmlClocksEventReason", "").replace("nvmlClocksThrottleReason", ""))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        rs = sorted({r for r in self.reasons if r not in ("None", "GpuIdle", "All")})
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": float(self.max_mhz) if self.max_mhz else None, "reasons": rs,
                "samples": len(self.samples)}


def max_over_ranks(ms: float, device=None) -> float:
    """Max of a per-rank duration over the job (identity without torch.distributed)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


class Bench:
    """One workload instance on one device: cache, compressor and the pieces the timing loops need."""

    def __init__(self, cfg_id, dev, layers=0):
        from paper_2605_23200_b200 import binding, inputs
        self.inputs, self.binding = inputs, binding
        wl = inputs.CONFIGS[cfg_id]
        if layers:
            wl = wl.scaled(n_layers=layers, resident_layers=0, name=wl.name + f"_REDUCED_to_{layers}_layers")
        self.wl, self.dev = wl, dev
        self.cache = inputs.make_cache(wl, dev)
        self.comp = binding.AmsCompressor(binding.config_for(wl), dev)
        self.stream = torch.cuda.current_stream(dev)
        self.dst_np = inputs.alloc_dst_pages(self.cache)
        self.dst = torch.from_numpy(self.dst_np).to(dev)
        self.table0, self.lens0 = self.cache.block_table.clone(), self.cache.seq_lens.clone()
        self.q = self.cache.obs_queries if wl.scorer_id == inputs.SCORER_TOVA else None
        self.stats = None
        if wl.scorer_id == inputs.SCORER_EXPECTED:
            self.stats = inputs.make_query_stats(self.cache)
            self.comp.set_query_stats(self.stats[0], self.stats[1], 1e-2)
        k_read, moved = algorithmic_bytes(wl, self.lens0.cpu().numpy())
        self.k_read, self.moved = k_read, moved
        # inputs smaller than twice the L2 are flushed out of it between timed steps
        self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if k_read < 2 * L2_BYTES else None

    def restore(self):
        self.cache.block_table.copy_(self.table0)
        self.cache.seq_lens.copy_(self.lens0)
        self.comp.ema_state.zero_()
        if self.flush is not None:
            self.flush.fill_(1)

    def step(self):
        wl, c = self.wl, self.cache
        self.comp.compress(c.k_pages, c.v_pages, c.block_table, c.seq_lens, self.q, wl.budget, wl.n_segments,
                           wl.scorer_id, self.dst)

    def timed(self, n, body):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in evs:
            self.restore()
            a.record(self.stream)
            body()
            b.record(self.stream)
        torch.cuda.synchronize(self.dev)
        return [a.elapsed_time(b) for a, b in evs]

    def warm(self, n):
        for _ in range(max(n, 3)):
            self.restore()
            self.step()
        self.comp.status()
        torch.cuda.synchronize(self.dev)

    def kernel_times(self, n):
        self.comp.set_profiling(True)
        acc = {}
        for _ in range(n):
            self.restore()
            self.step()
            for k, v in self.comp.kernel_times_ms().items():
                acc[k] = acc.get(k, 0.0) + v
        self.comp.set_profiling(False)
        return {k: v / n for k, v in acc.items() if v > 0.0}      # a slot no kernel of this path used stays out

    def close(self):
        self.comp.close()
        for name in ("cache", "comp", "dst", "table0", "lens0", "q", "flush", "stats"):
            setattr(self, name, None)
        gc.collect()
        torch.cuda.empty_cache()


SCORER_NAMES = {0: "tova", 1: "keydiff", 2: "external", 3: "expected_attention"}
SCORE_SLOTS = ("score_phase1", "score_combine", "score_phase2")
SELECT_SLOTS = ("segment_select", "segments_quotas", "select_compact")


def roofline_of(wl, kern_ms, k_read, moved, lens, peaks, traffic=None):
    """Roofline object of the dominant kernel that has an algorithmic byte (or operation) count: the scorer
    passes (K bytes; exponentials and tensor flops when the query block is wide) and the gather (kept rows).
    The selection kernels read no K/V byte; if one of them is the longest kernel the note says so."""
    if not kern_ms:
        return None
    overall = max(kern_ms, key=kern_ms.get)
    cands = {k: v for k, v in kern_ms.items() if k in ("score_phase1", "score_phase2", "gather")}
    dom = max(cands, key=cands.get)
    ms = cands[dom]
    rows = wl.group * max(wl.window, 1)
    note = []
    if overall != dom:
        note.append(f"longest kernel of the step is {overall} ({kern_ms[overall]:.4f} ms), which moves no K/V byte; the roofline is "
                    f"quoted for the longest kernel that does")
    if dom == "gather":
        bytes_launch, bound = moved, "hbm"
    elif wl.scorer_id == 3 and dom == "score_phase1":
        # K once (the V pass is the other scorer kernel); 2 * 128 * 128 flops per (query head, token) on the tensor pipe
        bytes_launch, bound = k_read // 2, "tensor"
    elif wl.scorer_id == 3:
        bytes_launch, bound = k_read // 2, "hbm"
    else:
        bytes_launch = k_read
        # wide query blocks: two passes with one exponential and one multiply-add per (row, token, d) each; the
        # special-function unit is the ceiling that binds first from about 75 rows, the tensor pipe next
        bound = "alu" if (wl.scorer_id == 0 and rows >= 256) else "hbm"
    out = {"kernel": dom, "bound": bound, "peak_kind": peaks["kind"], "algorithmic_bytes_per_launch": bytes_launch,
           "traffic": (traffic or {}).get(dom)}
    hbm_achieved = bytes_launch / (ms * 1e-3) / 1e9
    if bound == "hbm":
        out.update(achieved=hbm_achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=hbm_achieved / peaks["hbm_gbs"])
        note.append("achieved = algorithmic bytes of the launch / mean CUDA-event duration of that kernel; frac is of the measured copy bandwidth")
    elif bound == "tensor":
        token_heads = wl.layers_resident * wl.n_kv_heads * sum(int(t) for t in lens if int(t) > wl.budget)
        flops = token_heads * wl.group * 2 * 128 * 128
        achieved = flops / (ms * 1e-3) / 1e12
        out.update(achieved=achieved, peak=peaks["bf16_tflops"], unit="TFLOP/s", frac=achieved / peaks["bf16_tflops"],
                   operations_per_launch=flops,
                   also={"hbm_gbs": hbm_achieved, "hbm_frac": hbm_achieved / peaks["hbm_gbs"]})
        note.append("one 128 x 128 matrix-vector product per (query head, token) on the tensor pipe (K tile x covariance), bf16 in, "
                    "fp32 accumulate; frac is of the measured cuBLAS bf16 rate (burst); the K stream of the same launch is under 'also'")
    else:
        token_heads = wl.layers_resident * wl.n_kv_heads * sum(int(t) for t in lens if int(t) > wl.budget)
        exps = token_heads * rows
        flops = exps * 2 * 128
        mufu_peak = N_SM * MUFU_PER_CLK_PER_SM * peaks["sm_max_mhz"] * 1e6 / 1e9        # G results / s
        achieved = exps / (ms * 1e-3) / 1e9
        out.update(achieved=achieved, peak=mufu_peak, unit="Gexp/s", frac=achieved / mufu_peak,
                   operations_per_launch=exps,
                   also={"hbm_gbs": hbm_achieved, "hbm_frac": hbm_achieved / peaks["hbm_gbs"],
                         "tensor_tflops": flops / (ms * 1e-3) / 1e12,
                         "tensor_frac": flops / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"]})
        note.append("512 query rows per KV head: the pass takes one exp2 per (row, token) on the special-function unit "
                    "(16 results per clock and SM x 148 SMs x the maximum SM clock = peak) and is bound by it before HBM; "
                    "hbm and tensor fractions of the same launch are under 'also'")
    out["note"] = "; ".join(note)
    return out


def steady_state(b: Bench):
    """Events 2..N of a multi-event configuration, run as real successive events: the first event compresses
    the long cache, then `append_per_step` tokens are appended and the cache is compressed again, the EMA
    credit carried in the compressor's state.  Returns per-event times and the kernel split of the last."""
    wl, cache, comp, inputs = b.wl, b.cache, b.comp, b.inputs
    b.restore()
    dst_np = b.dst_np
    times = []
    kern = {}
    for ev in range(wl.steps):
        if ev > 0:
            inputs.append_tokens(cache, wl.append_per_step)
            dst_np = inputs.alloc_dst_pages(cache)
        dst = torch.from_numpy(dst_np).to(b.dev)
        q = cache.obs_queries if wl.scorer_id == inputs.SCORER_TOVA else None
        last = ev == wl.steps - 1
        if last:
            comp.set_profiling(True)
        if b.flush is not None:
            b.flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(b.stream)
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, q, wl.budget, wl.n_segments,
                      wl.scorer_id, dst)
        e1.record(b.stream)
        torch.cuda.synchronize(b.dev)
        times.append(e0.elapsed_time(e1))
        if last:
            kern = {k: v for k, v in comp.kernel_times_ms().items() if v > 0.0}
            comp.set_profiling(False)
        comp.status()
        assert bool((cache.seq_lens == wl.budget).all())
        inputs.after_compress(cache, dst_np)
    T = wl.budget + wl.append_per_step
    units = wl.layers_resident * wl.batch * wl.n_kv_heads
    bytes_ss = units * (T * 256 + wl.budget * 1024)
    ss = times[1:]
    ms = float(np.mean(ss))
    return {"events": wl.steps, "appended_per_event": wl.append_per_step, "cache_tokens": T,
            "first_event_ms": times[0], "steady_state_ms": ms, "steady_state_ms_min": float(np.min(ss)),
            "algorithmic_bytes_per_step": bytes_ss, "effective_hbm_gbs": bytes_ss / (ms * 1e-3) / 1e9,
            "effective_hbm_frac_of_8tbs": bytes_ss / (ms * 1e-3) / 8e12, "kernels_ms_last_event": kern}


def measure_config(cfg_id, dev, steps, warmup, peaks, layers=0, with_steady=True):
    """First-event timing (and steady state where the configuration has one) of one configuration."""
    b = Bench(cfg_id, dev, layers)
    wl = b.wl
    b.warm(warmup)
    per_step = b.timed(steps, b.step)
    b.comp.status()
    kern_ms = b.kernel_times(min(steps, 10))
    ms = float(np.mean(per_step))
    lens = b.lens0.cpu().numpy()
    total = b.k_read + b.moved
    entry = {
        "workload": wl.name, "layers_resident": wl.layers_resident, "layers_total": wl.n_layers, "batch": wl.batch,
        "kv_heads": wl.n_kv_heads, "query_rows_per_kv_head": wl.group * max(wl.window, 1),
        "cache_tokens": [int(lens.min()), int(lens.max())], "budget": wl.budget, "n_segments": wl.n_segments,
        "scorer": SCORER_NAMES[wl.scorer_id], "steps": steps,
        "ms_per_step": ms, "ms_per_step_min": float(np.min(per_step)), "steps_per_s": 1e3 / ms,
        "algorithmic_bytes_per_step": total, "effective_hbm_gbs": total / (ms * 1e-3) / 1e9,
        "effective_hbm_frac_of_8tbs": total / (ms * 1e-3) / 8e12,
        "effective_hbm_frac_of_measured": total / (ms * 1e-3) / (peaks["hbm_gbs"] * 1e9),
        "l2": "L2 flushed between timed steps (256 MB written)" if b.flush is not None else "inputs larger than L2",
        "launches_per_step": b.comp.last_launch_count, "kernels_ms": kern_ms,
        "roofline": roofline_of(wl, kern_ms, b.k_read, b.moved, lens, peaks, NCU_TRAFFIC_BYTES.get(wl.name)),
    }
    if wl.layers_resident != wl.n_layers:
        entry["note"] = (f"{wl.layers_resident} of {wl.n_layers} layers resident (the whole stack's K/V does not fit one GPU): "
                         f"all figures are per launch over the resident layers; the full stack is {wl.n_layers // wl.layers_resident} such launches")
    if with_steady and wl.steps > 1:
        entry["steady_state"] = steady_state(b)
    return b, entry, per_step


def e2e_loop(b: Bench, n_e2e):
    """The step through the C ABI with its inputs uploaded from pinned host memory and its results read back
    and checked every step; the upload of step i + 1 and the read-back of step i - 1 overlap the kernels of
    step i (three buffer sets, three streams, at most two steps in flight)."""
    wl, cache, comp, dev, stream = b.wl, b.cache, b.comp, b.dev, b.stream
    q, dst = b.q, b.dst
    b.restore()
    host_q = q.cpu().pin_memory() if q is not None else None
    host_table, host_lens, host_dst = b.table0.cpu().pin_memory(), b.lens0.cpu().pin_memory(), dst.cpu().pin_memory()
    out_table, out_lens = torch.empty_like(host_table).pin_memory(), torch.empty_like(host_lens).pin_memory()
    host_stats = [t.cpu().pin_memory() for t in b.stats] if b.stats is not None else None   # query statistics of this event
    h2d = sum(t.numel() * t.element_size() for t in (host_q, host_table, host_lens, host_dst, *(host_stats or [])) if t is not None)
    d2h = out_table.numel() * 4 + out_lens.numel() * 4 + 16
    NB = 3
    sets = [(q, cache.block_table, cache.seq_lens, dst)] + [
        (None if q is None else torch.empty_like(q), torch.empty_like(cache.block_table), torch.empty_like(cache.seq_lens),
         torch.empty_like(dst)) for _ in range(NB - 1)]
    stat_sets = None if b.stats is None else [b.stats] + [tuple(torch.empty_like(t) for t in b.stats) for _ in range(NB - 1)]
    copy_stream, read_stream = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    uploaded = [torch.cuda.Event() for _ in range(NB)]
    computed = [torch.cuda.Event() for _ in range(NB)]
    read_back = [torch.cuda.Event() for _ in range(NB)]
    outs = [(out_table, out_lens)] + [(torch.empty_like(out_table).pin_memory(), torch.empty_like(out_lens).pin_memory())
                                      for _ in range(NB - 1)]

    def upload(i):
        qi, ti, li, di = sets[i % NB]
        with torch.cuda.stream(copy_stream):
            if host_q is not None:
                qi.copy_(host_q, non_blocking=True)
            ti.copy_(host_table, non_blocking=True)
            li.copy_(host_lens, non_blocking=True)
            di.copy_(host_dst, non_blocking=True)
            if stat_sets is not None:
                for dev_t, host_t in zip(stat_sets[i % NB], host_stats):
                    dev_t.copy_(host_t, non_blocking=True)
            uploaded[i % NB].record(copy_stream)

    def check(i):                           # results of step i: wait for their read-back and look at them
        read_back[i % NB].synchronize()
        assert int(outs[i % NB][1][0]) == wl.budget

    def e2e_step(i):
        qi, ti, li, di = sets[i % NB]
        if i >= 2:
            check(i - 2)                    # also releases the buffer set that upload(i + 1) is about to fill
        upload(i + 1)                       # overlaps the kernels of steps i - 1 and i
        stream.wait_event(uploaded[i % NB])
        comp.ema_state.zero_()
        if stat_sets is not None:
            comp.set_query_stats(stat_sets[i % NB][0], stat_sets[i % NB][1], 1e-2)
        comp.compress(cache.k_pages, cache.v_pages, ti, li, qi, wl.budget, wl.n_segments, wl.scorer_id, di)
        computed[i % NB].record(stream)
        with torch.cuda.stream(read_stream):  # block table and lengths of this step back to pinned host memory
            read_stream.wait_event(computed[i % NB])
            outs[i % NB][0].copy_(ti, non_blocking=True)
            outs[i % NB][1].copy_(li, non_blocking=True)
            read_back[i % NB].record(read_stream)

    torch.cuda.synchronize(dev)
    upload(0)
    for i in range(3):
        e2e_step(i)
    check(1)
    check(2)
    comp.status()
    barrier()
    t0 = time.perf_counter()
    for i in range(3, 3 + n_e2e):
        e2e_step(i)
    check(1 + n_e2e)
    check(2 + n_e2e)
    comp.status()  # device status word of the whole run; synchronises the stream
    torch.cuda.synchronize(dev)
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3, dev)
    return e2e_ms, h2d, d2h


def run_ours(args, rank, world, local_rank):
    from paper_2605_23200_b200 import binding, build
    import torch.distributed as dist

    if rank == 0:
        build.build()
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        barrier()
    binding.lib()
    peaks = _peaks()
    head_cfg = args.config if args.config is not None else HEADLINE_CFG
    warmup = max(args.warmup, 3)

    # ---- headline: first event of the headline configuration
    b = Bench(head_cfg, dev, args.layers)
    wl = b.wl
    b.warm(warmup)
    step = b.step
    if args.graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            b.step()
        step = graph.replay
        b.stream = torch.cuda.current_stream(dev)
        for _ in range(3):
            b.restore()
            step()
        b.comp.status()
        torch.cuda.synchronize(dev)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    per_step = b.timed(args.steps, step)
    barrier()
    clocks = sampler.stop()
    b.comp.status()
    total_ms = max_over_ranks(float(sum(per_step)), dev)
    launches = b.comp.last_launch_count * args.steps
    kern_ms = b.kernel_times(min(args.steps, 10))
    lens = b.lens0.cpu().numpy()
    e2e = None
    if not args.no_e2e:
        n_e2e = min(args.steps, 50)
        e2e_ms, h2d, d2h = e2e_loop(b, n_e2e)
        e2e = {"value": world * n_e2e / (e2e_ms / 1e3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "steps": n_e2e,
               "note": "uploads of step i+1 and the read-back of step i-1 overlap the kernels of step i (three buffer sets, three "
                       "streams, at most two steps in flight); every step uploads all its inputs and its block table and lengths "
                       "are read back and checked"}
    ms_per_step = total_ms / args.steps
    total_bytes = b.k_read + b.moved
    out = {
        "metric": METRIC, "value": world * args.steps / (total_ms / 1e3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "dtype_detail": "bf16 K/V and queries, fp32 accumulation and scores, u64 fixed-point decisions",
        "data": "synthetic",
        "config": config_dict(wl),
        "run": {"l2": "inputs larger than L2 (K read per step %.2f GB)" % (b.k_read / 1e9) if b.flush is None
                      else "L2 flushed between timed steps (256 MB written)",
                "parallelism": f"replica x{world}" if world > 1 else "single GPU",
                "launch": "one CUDA graph per step" if args.graph else "direct kernel launches"},
        "effective_hbm_gbs": total_bytes / (ms_per_step * 1e-3) / 1e9,
        "effective_hbm_frac_of_8tbs": total_bytes / (ms_per_step * 1e-3) / 8e12,
        "effective_hbm_frac_of_measured": total_bytes / (ms_per_step * 1e-3) / (peaks["hbm_gbs"] * 1e9),
        "algorithmic_bytes_per_step": total_bytes,
        "gpu_launches": launches,
        "kernels_ms": kern_ms,
        "roofline": roofline_of(wl, kern_ms, b.k_read, b.moved, lens, peaks, NCU_TRAFFIC_BYTES.get(wl.name)),
        "e2e": e2e,
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, b.cache, b.dst_np, b.table0, b.lens0, budget_s=20.0)
    steady_head = None
    if not args.no_per_config and wl.steps > 1 and not args.layers:
        steady_head = steady_state(b)
    b.close()

    # ---- all five configurations (rank 0's replica; every rank runs them so that the ranks stay in step)
    if not args.no_per_config and args.config is None and not args.layers:
        per = {}
        for cid in range(5):
            if cid == head_cfg:
                e = {"workload": wl.name, "ms_per_step": ms_per_step, "steps_per_s": 1e3 / ms_per_step,
                     "algorithmic_bytes_per_step": total_bytes, "effective_hbm_gbs": out["effective_hbm_gbs"],
                     "effective_hbm_frac_of_8tbs": out["effective_hbm_frac_of_8tbs"], "kernels_ms": kern_ms,
                     "roofline": out["roofline"], "launches_per_step": launches // args.steps, "note": "the headline measurement above"}
                if steady_head:
                    e["steady_state"] = steady_head
                per[f"cfg{cid}"] = e
                continue
            bb, entry, _ = measure_config(cid, dev, min(args.steps, 10), 3, peaks)
            bb.close()
            per[f"cfg{cid}"] = entry
        out["per_config"] = per
        # beyond the five benchmark configurations: the expected-attention scorer on the geometry of configuration 1
        bb, entry, _ = measure_config(5, dev, min(args.steps, 10), 3, peaks)
        bb.close()
        entry["note"] = "extension, not one of the five benchmark configurations: expected-attention scorer (tensor-core kernel over K, then a pass over V)"
        out["extensions"] = {"cfg5": entry}
    elif steady_head:
        out["steady_state"] = steady_head
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def _oracle_sample(wl, cache, dst_np, table0, lens0, units):
    """Host copies of what the oracle needs for `units` and a callable that runs them."""
    import oracle
    from paper_2605_23200_b200 import inputs

    layers = sorted({u[0] for u in units})
    remap = {l: i for i, l in enumerate(layers)}
    idx = torch.tensor(layers, device=cache.k_pages.device)
    k = inputs.as_u16(cache.k_pages.index_select(0, idx))
    v = inputs.as_u16(cache.v_pages.index_select(0, idx))
    q = inputs.as_u16(cache.obs_queries.index_select(0, idx)) if cache.obs_queries is not None else None
    table, lens = table0.cpu().numpy(), lens0.cpu().numpy()
    stats = {}
    if wl.scorer_id == inputs.SCORER_EXPECTED:
        mean, cov = inputs.make_query_stats(cache)
        stats = dict(q_mean=mean.index_select(0, idx).cpu().numpy(), q_cov=inputs.as_u16(cov.index_select(0, idx)), score_eps=1e-2)
    prm = oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda, wl.ema_beta, wl.eps)
    local_units = [(remap[l], b, h) for (l, b, h) in units]
    oracle.lib()

    def run(threads):
        credit = np.zeros((len(layers), wl.batch, wl.n_kv_heads, wl.max_seq_len), np.float32)
        oracle.compress(k, v, table.copy(), lens.copy(), q, credit, wl.budget, prm, wl.scorer_id, dst_np,
                        n_q_heads=wl.n_q_heads, units=local_units, threads=threads, **stats)
    return run


def _all_units(wl):
    return [(l, b, h) for l in range(wl.layers_resident) for b in range(wl.batch) for h in range(wl.n_kv_heads)]


def cpu_baseline(wl, cache, dst_np, table0, lens0, budget_s):
    """The oracle as it stands, on the host cores, over a bounded sample of the workload's units."""
    cores = os.cpu_count() or 1
    units = _all_units(wl)
    probe = _oracle_sample(wl, cache, dst_np, table0, lens0, units[:1])
    t0 = time.perf_counter()
    probe(1)
    unit_s = time.perf_counter() - t0
    n = int(max(1, min(len(units), budget_s * cores / max(unit_s, 1e-6))))
    if n >= cores:
        n = n // cores * cores          # whole rounds of one unit per core
    sample = units[:n]
    run = _oracle_sample(wl, cache, dst_np, table0, lens0, sample)
    t0 = time.perf_counter()
    run(min(cores, n))
    dt = time.perf_counter() - t0
    return {"value": (n / len(units)) / dt, "unit": UNIT, "cores": min(cores, n), "kind": "oracle",
            "sample": f"first {n} of {len(units)} (layer, sequence, KV head) units, scaled by units; {dt:.1f} s wall "
                      f"(one unit alone: {unit_s:.1f} s on one core)"}


def run_reference(args, rank, world):
    """Reference arm: the CPU oracle, as it stands, on the host cores, same metric and workload.  One step is
    a bounded sample of the workload's units (whole units: a unit is the smallest independent piece of the
    path), scaled by units; a unit of the headline workload takes the oracle some twenty seconds on one core, so
    the sample is one unit per core, the warm-up one step, and the number of timed steps is bounded."""
    if rank != 0:
        return
    from paper_2605_23200_b200 import inputs
    cfg_id = args.config if args.config is not None else HEADLINE_CFG
    wl = inputs.CONFIGS[cfg_id]
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    # only the sampled units' layers are needed on the host: build the cache with as few layers as the sample spans
    cores = os.cpu_count() or 1
    per_layer = wl.batch * wl.n_kv_heads
    layers_needed = max(1, min(wl.layers_resident, -(-cores // per_layer)))
    wl_small = wl.scaled(n_layers=layers_needed, resident_layers=0) if layers_needed < wl.layers_resident else wl
    cache = inputs.make_cache(wl_small, dev)
    dst_np = inputs.alloc_dst_pages(cache)
    table0, lens0 = cache.block_table.clone(), cache.seq_lens.clone()
    units_all = len(_all_units(wl))
    units = _all_units(wl_small)
    probe = _oracle_sample(wl_small, cache, dst_np, table0, lens0, units[:1])
    t0 = time.perf_counter(); probe(1); unit_s = time.perf_counter() - t0
    # A unit is the smallest independent piece of the path, so a step cannot be shorter than one unit's time on
    # one core; the run is kept to a few minutes by timing at most as many steps as fit 200 s (never fewer than 3)
    # after one warm-up step, and the line says how many were timed.
    warmup = min(args.warmup, 1)
    n = int(max(1, min(len(units), cores)))
    steps = int(max(3, min(args.steps, 200.0 / max(unit_s, 1e-6))))
    run = _oracle_sample(wl_small, cache, dst_np, table0, lens0, units[:n])
    for _ in range(warmup):
        run(min(cores, n))
    t0 = time.perf_counter()
    for _ in range(steps):
        run(min(cores, n))
    dt = time.perf_counter() - t0
    value = steps * (n / units_all) / dt
    sample = (f"each step = first {n} of {units_all} units (whole units, one per core), scaled by units; one unit alone takes "
              f"{unit_s:.1f} s on one core; {steps} of the {args.steps} requested steps timed after {warmup} warm-up step(s) "
              f"so that the run ends within a few minutes")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "steps_requested": args.steps, "warmup": warmup, "ms_per_step": dt / steps * 1e3 * (units_all / n), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, n), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_plumbing(args, rank, world):
    """CPU check of the multi-rank harness (no kernels, no GPU): gloo ranks meet at the barrier, each reports a
    known duration, the maximum over ranks is taken and rank 0 prints the line.  Used by the tests."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
    barrier()
    ms = 10.0 * (rank + 1)
    total = max_over_ranks(ms)
    barrier()
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"impl": "plumbing", "n_gpus": world, "ms_max_over_ranks": total, "scaling": "weak",
                          "value": world * args.steps / (total / 1e3)}))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n):
    """`--gpus N` without a launcher: run this script as N ranks under torch.distributed.run and pass its
    output through."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "plumbing"])
    ap.add_argument("--config", type=int, default=None, help="time this configuration only (default: headline + all five)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--graph", action="store_true", help="time the step replayed from a CUDA graph")
    ap.add_argument("--layers", type=int, default=0, help="profiling only: run a reduced layer count")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    if args.impl == "plumbing":
        run_plumbing(args, rank, world)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the AMS compression step (score + segment + select + compact).

One "step" is one `ams_compress` call over the whole layer stack of the workload.
At N = 1 the workload is benchmark configuration 1 (Llama-3.1-8B-shaped stack:
32 layers, 32 q / 8 KV heads, d = 128, one sequence of 16384 cached bf16 tokens in
16-token pages, compressed to 2048; observation window 32, TOVA-style scorer).
With N > 1 every rank runs its own replica of that workload (the units of the path
are independent: no collective on the data path; weak scaling).

Prints ONE JSON line (rank 0).  `value` = whole-job steps/s with the cache resident in
HBM, timed with CUDA events on the launching stream.  `e2e` = the same through the
C ABI with the step's inputs (observation queries, block table, lengths,
replacement pages) copied from pinned host memory and its results (block table,
lengths) read back and checked inside the timed region; the upload of the next
step's inputs and the read-back of the previous step's results overlap the current
step's kernels (three buffer sets, at most two steps in flight), as a serving loop
would do; the paged K/V pool is the persistent device
state the step operates on and is not copied.
"""
from __future__ import annotations

import argparse
import json
import os
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


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the scorer passes on the
# default workload, from the ncu capture summarised in profiles/kernels_cfg1_8layers_ncu_full.md: taken on
# the 8-layer reduction of the workload and scaled x4 to the 32-layer launch (units are independent and each
# is read once per pass).  Valid for that workload and the kernels as profiled; anything else reports null.
NCU_TRAFFIC_BYTES = {
    "cfg1_llama8b_L32_T16384_k2048_w32": {"score_phase1": 4 * (271_291_904 + 9_388_288),
                                          "score_phase2": 4 * (271_763_712 + 7_136_256),
                                          "gather": None},
}


def algorithmic_bytes(wl, lens) -> tuple[int, int]:
    """(K bytes read once for scoring, kept K/V bytes read + written) per step."""
    units = wl.layers_resident * wl.n_kv_heads
    live = [int(t) for t in lens if int(t) > wl.budget]
    k_read = units * sum(live) * 256
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


def run_ours(args, rank, world, local_rank):
    from paper_2605_23200_b200 import binding, build, inputs
    import torch.distributed as dist

    if rank == 0:
        build.build()
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        barrier()
    binding.lib()
    wl = inputs.CONFIGS[args.config]
    if args.layers:
        wl = wl.scaled(n_layers=args.layers, resident_layers=0, name=wl.name + f"_REDUCED_to_{args.layers}_layers")
    cache = inputs.make_cache(wl, dev)
    comp = binding.AmsCompressor(binding.config_for(wl), dev)
    stream = torch.cuda.current_stream(dev)
    dst_np = inputs.alloc_dst_pages(cache)
    dst = torch.from_numpy(dst_np).to(dev)
    table0, lens0 = cache.block_table.clone(), cache.seq_lens.clone()
    q = cache.obs_queries if wl.scorer_id == inputs.SCORER_TOVA else None

    def restore():
        cache.block_table.copy_(table0)
        cache.seq_lens.copy_(lens0)
        comp.ema_state.zero_()

    def step():
        comp.compress(cache.k_pages, cache.v_pages, cache.block_table, cache.seq_lens, q, wl.budget, wl.n_segments,
                      wl.scorer_id, dst)

    def timed(n, body):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in evs:
            restore()
            a.record(stream)
            body()
            b.record(stream)
        torch.cuda.synchronize(dev)
        return [a.elapsed_time(b) for a, b in evs]

    for _ in range(max(args.warmup, 3)):
        restore()
        step()
    comp.status()
    torch.cuda.synchronize(dev)
    direct_step = step
    if args.graph:
        # the whole step as one CUDA graph launch (pays off where the step is launch-bound)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            direct_step()
        restore()
        step = graph.replay
        stream = torch.cuda.current_stream(dev)
        for _ in range(3):
            restore()
            step()
        comp.status()
        torch.cuda.synchronize(dev)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    per_step = timed(args.steps, step)
    barrier()
    clocks = sampler.stop()
    comp.status()
    total_ms = max_over_ranks(float(sum(per_step)), dev)
    launches = comp.last_launch_count * args.steps

    # per-kernel durations (CUDA events recorded by the library after each launch, same stream)
    comp.set_profiling(True)
    n_prof = min(args.steps, 50)
    acc = {}
    for _ in range(n_prof):
        restore()
        direct_step()
        for k, v in comp.kernel_times_ms().items():
            acc[k] = acc.get(k, 0.0) + v
    comp.set_profiling(False)
    kern_ms = {k: v / n_prof for k, v in acc.items() if v > 0.0}      # a slot no kernel of this path used stays out

    # end to end: per-step inputs from pinned host memory, results read back
    host_q = q.cpu().pin_memory() if q is not None else None
    host_table, host_lens, host_dst = table0.cpu().pin_memory(), lens0.cpu().pin_memory(), dst.cpu().pin_memory()
    out_table, out_lens = torch.empty_like(host_table).pin_memory(), torch.empty_like(host_lens).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (host_q, host_table, host_lens, host_dst) if t is not None)
    d2h = out_table.numel() * 4 + out_lens.numel() * 4 + 16

    # Two sets of device input buffers: while step i computes, the inputs of step i + 1 are uploaded on a second
    # stream (what a serving loop does); every step still uploads all its inputs from pinned host memory, and
    # its results (block table, lengths, device status) are read back and waited for before the next launch.
    NB = 3  # buffer sets: one being uploaded, one computing, one being read back
    sets = [(q, cache.block_table, cache.seq_lens, dst)] + [
        (None if q is None else torch.empty_like(q), torch.empty_like(cache.block_table), torch.empty_like(cache.seq_lens),
         torch.empty_like(dst)) for _ in range(NB - 1)]
    copy_stream = torch.cuda.Stream(dev)
    uploaded = [torch.cuda.Event() for _ in range(NB)]

    def upload(i):
        qi, ti, li, di = sets[i % NB]
        with torch.cuda.stream(copy_stream):
            if host_q is not None:
                qi.copy_(host_q, non_blocking=True)
            ti.copy_(host_table, non_blocking=True)
            li.copy_(host_lens, non_blocking=True)
            di.copy_(host_dst, non_blocking=True)
            uploaded[i % NB].record(copy_stream)

    read_stream = torch.cuda.Stream(dev)
    computed = [torch.cuda.Event() for _ in range(NB)]
    read_back = [torch.cuda.Event() for _ in range(NB)]
    outs = [(out_table, out_lens)] + [(torch.empty_like(out_table).pin_memory(), torch.empty_like(out_lens).pin_memory())
                                      for _ in range(NB - 1)]

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
        comp.compress(cache.k_pages, cache.v_pages, ti, li, qi, wl.budget, wl.n_segments, wl.scorer_id, di)
        computed[i % NB].record(stream)
        with torch.cuda.stream(read_stream):  # block table and lengths of this step back to pinned host memory
            read_stream.wait_event(computed[i % NB])
            outs[i % NB][0].copy_(ti, non_blocking=True)
            outs[i % NB][1].copy_(li, non_blocking=True)
            read_back[i % NB].record(read_stream)

    n_e2e = min(args.steps, 50)
    e2e_ms = None
    if not args.no_e2e:
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

    k_read, moved = algorithmic_bytes(wl, lens0.cpu().numpy())
    peak, peak_kind = _peaks()
    ms_per_step = total_ms / args.steps
    dominant = max(kern_ms, key=kern_ms.get)
    dom_bytes = moved if dominant == "gather" else k_read
    dom_ms = kern_ms[dominant]
    out = {
        "metric": METRIC, "value": world * args.steps / (total_ms / 1e3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "dtype_detail": "bf16 K/V and queries, fp32 accumulation and scores, u64 fixed-point decisions",
        "data": "synthetic",
        "config": {"workload": wl.name, "layers": wl.n_layers, "q_heads": wl.n_q_heads, "kv_heads": wl.n_kv_heads,
                   "batch_per_gpu": wl.batch, "cache_tokens": wl.seq_len_max, "budget": wl.budget, "window": wl.window,
                   "n_segments": wl.n_segments, "scorer": "tova" if wl.scorer_id == 0 else "keydiff",
                   "l2": "inputs larger than L2 (K read per step %.2f GB)" % (k_read / 1e9),
                   "parallelism": f"replica x{world}" if world > 1 else "single GPU",
                   "launch": "one CUDA graph per step" if args.graph else "direct kernel launches"},
        "effective_hbm_gbs": (k_read + moved) / (ms_per_step * 1e-3) / 1e9,
        "effective_hbm_frac_of_8tbs": (k_read + moved) / (ms_per_step * 1e-3) / 8e12,
        "effective_hbm_frac_of_measured": (k_read + moved) / (ms_per_step * 1e-3) / (peak * 1e9),
        "algorithmic_bytes_per_step": k_read + moved,
        "gpu_launches": launches,
        "kernels_ms": kern_ms,
        "roofline": {"kernel": dominant, "bound": "hbm", "achieved": dom_bytes / (dom_ms * 1e-3) / 1e9, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": dom_bytes / (dom_ms * 1e-3) / 1e9 / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(wl.name, {}).get(dominant), "algorithmic_bytes_per_launch": dom_bytes,
                     "note": "achieved = algorithmic bytes of the launch / mean CUDA-event duration of that kernel; "
                             "frac is of the measured copy bandwidth"},
        "e2e": None if e2e_ms is None else {"value": world * n_e2e / (e2e_ms / 1e3), "unit": UNIT,
                                            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
                                            "note": "uploads of step i+1 and the read-back of step i-1 overlap the kernels of step i (three buffer sets, three streams, at most two steps in flight); every step uploads all its inputs and its block table and lengths are read back and checked"},
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(wl, cache, dst_np, table0, lens0, budget_s=20.0)
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
    prm = oracle.Params(wl.n_segments, wl.l_min, wl.l_max, wl.q_min, wl.n_sink, wl.n_last, wl.ema_lambda, wl.ema_beta, wl.eps)
    local_units = [(remap[l], b, h) for (l, b, h) in units]
    oracle.lib()

    def run(threads):
        credit = np.zeros((len(layers), wl.batch, wl.n_kv_heads, wl.max_seq_len), np.float32)
        oracle.compress(k, v, table.copy(), lens.copy(), q, credit, wl.budget, prm, wl.scorer_id, dst_np,
                        n_q_heads=wl.n_q_heads, units=local_units, threads=threads)
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
    n = int(max(cores, min(len(units), budget_s * cores / max(unit_s, 1e-6))))
    n = max(1, min(n, len(units)))
    sample = units[:n]
    run = _oracle_sample(wl, cache, dst_np, table0, lens0, sample)
    t0 = time.perf_counter()
    run(cores)
    dt = time.perf_counter() - t0
    return {"value": (n / len(units)) / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} of {len(units)} (layer, sequence, KV head) units, scaled by units; {dt:.1f} s wall"}


def run_reference(args, rank, world):
    """Reference arm: the CPU oracle, unmodified, on the host cores, same metric and workload."""
    if rank != 0:
        return
    from paper_2605_23200_b200 import inputs
    wl = inputs.CONFIGS[args.config]
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    cache = inputs.make_cache(wl, dev)
    dst_np = inputs.alloc_dst_pages(cache)
    table0, lens0 = cache.block_table.clone(), cache.seq_lens.clone()
    cores = os.cpu_count() or 1
    units = _all_units(wl)
    probe = _oracle_sample(wl, cache, dst_np, table0, lens0, units[:1])
    t0 = time.perf_counter(); probe(1); unit_s = time.perf_counter() - t0
    total_steps = args.steps + args.warmup
    per_step_budget = 150.0 / max(total_steps, 1)
    n = int(max(1, min(len(units), per_step_budget * cores / max(unit_s, 1e-6))))
    run = _oracle_sample(wl, cache, dst_np, table0, lens0, units[:n])
    for _ in range(args.warmup):
        run(cores)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run(cores)
    dt = time.perf_counter() - t0
    value = args.steps * (n / len(units)) / dt
    sample = f"each step = first {n} of {len(units)} units, scaled by units"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3 * (len(units) / n), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--graph", action="store_true", help="time the step replayed from a CUDA graph")
    ap.add_argument("--layers", type=int, default=0, help="profiling only: run a reduced layer count")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if args.steps > 20:
            args.steps = 20 if "--steps" not in " ".join(sys.argv) else args.steps
        run_reference(args, rank, world)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression path has no CPU fallback")
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of adapter-over-cache training (PAC+ phase 2) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path over one minibatch: gather of the cached
states, adapter forward, head and loss, adapter-only backward, AdamW.  `value` is
samples/s with the cache, the shuffled ids and the losses resident in HBM (one
pac_train_epoch_dev call over K*B ids); `e2e` is the same metric through
pac_train_step_async with host ids in and the host loss out every step.
Prints ONE JSON line (rank 0).
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

import pac_inputs as pi  # noqa: E402

METRIC = "adapter_epoch_samples_per_sec"
UNIT = "samples/s"
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from the ncu
# capture summarised under profiles/ (None until a capture of the current kernel exists).
NCU_TRAFFIC_BYTES = {"t5_base": {"tensor+fused_forward": {"down_projection": 80818176, "dw_down": 84011520},
                                 "tensor": {"dw_down": 84011520}}}


def ncu_traffic(spec, kernel_path, kernel):
    """DRAM bytes per launch from the committed ncu capture (profiles/); None for kernels it does
    not cover."""
    return ((NCU_TRAFFIC_BYTES.get(spec.name.split("[")[0]) or {}).get(kernel_path) or {}).get(kernel)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


def workload_name(spec: pi.CacheSpec) -> str:
    return (f"{spec.name}: cache N={spec.N} L={spec.L} S={spec.S} d={spec.d} {spec.dtype}, r={spec.r}, "
            f"{'C' if spec.head == 'cls' else 'V'}={spec.n_out}, B={spec.B}, shuffled epochs")


def epoch_ids(spec: pi.CacheSpec, steps: int) -> np.ndarray:
    """K*B ids: consecutive seeded permutations of 0..N-1 (one per epoch), cut at K steps."""
    out, e = [], 0
    while sum(len(x) for x in out) < steps * spec.B:
        perm = pi.epoch_permutation(spec.N, 2, epoch=e)
        out.append(perm[:(spec.N // spec.B) * spec.B])
        e += 1
    return np.concatenate(out)[:steps * spec.B].astype(np.int32)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.max_mhz = period_s, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception as e:  # NVML missing: report that clocks were not sampled
            self.err = repr(e)

    def run(self):
        while self.ok and not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                mask = self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=1.0)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "clocks not sampled"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": float(self.max_mhz),
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_baseline(spec: pi.CacheSpec, budget_s: float, max_steps: int):
    """Times the CPU oracle as it stands on a bounded sample: whole train steps (B samples each)
    on freshly generated slabs until about budget_s of oracle time is spent."""
    from oracle import pac_oracle as po
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    perm = pi.epoch_permutation(spec.N, 2)
    P = po.unflatten(pi.random_params(spec, 3), spec.L, spec.d, spec.r, spec.n_out if spec.head == "cls" else None)
    labels_all = pi.labels(spec, 0).numpy().astype(np.int64)
    W_lm = pi.lm_head(spec, 0).float().numpy() if spec.head == "lm" else None
    spent, steps = 0.0, 0
    while steps < max_steps and (steps == 0 or spent < budget_s):
        ids = perm[steps * spec.B:(steps + 1) * spec.B].tolist()
        cache = pi.cache_samples(spec, 0, ids).float().numpy()
        tr = po.Trainer(cache, labels_all[ids], P, W_lm=W_lm) if steps == 0 else tr
        tr.cache, tr.labels = cache, labels_all[ids]
        t0 = time.perf_counter()
        tr.train_step(list(range(spec.B)))
        tr.adam_step()
        spent += time.perf_counter() - t0
        steps += 1
    return {"value": steps * spec.B / spent, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{steps} whole train steps (B={spec.B}) of {spec.name} in fp32, {spent:.1f} s of oracle time; "
                      "slab generation not timed"}


def run_reference(args, spec):
    """The reference arm: the CPU oracle as it stands, K timed steps after W warm-up steps,
    each step a bounded sample (B' <= B samples) so the run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import pac_oracle as po
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    P = po.unflatten(pi.random_params(spec, 3), spec.L, spec.d, spec.r, spec.n_out if spec.head == "cls" else None)
    labels_all = pi.labels(spec, 0).numpy().astype(np.int64)
    W_lm = pi.lm_head(spec, 0).float().numpy() if spec.head == "lm" else None
    perm = pi.epoch_permutation(spec.N, 2)
    pool_ids = perm[:spec.B].tolist()
    cache = pi.cache_samples(spec, 0, pool_ids).float().numpy()
    tr = po.Trainer(cache, labels_all[pool_ids], P, W_lm=W_lm)
    t0 = time.perf_counter()
    tr.train_step(list(range(spec.B)))
    tr.adam_step()
    t_full = time.perf_counter() - t0
    total = args.steps + args.warmup
    Bp = spec.B if t_full * total <= 150 else max(1, int(spec.B * 150 / (t_full * total)))
    sub = list(range(Bp))
    for _ in range(args.warmup):
        tr.train_step(sub); tr.adam_step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        tr.train_step(sub); tr.adam_step()
    dt = time.perf_counter() - t0
    value = args.steps * Bp / dt
    sample = (f"{args.steps} oracle train steps of {Bp} samples each (of B={spec.B}) drawn from one generated "
              f"minibatch of {spec.name}, fp32")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(spec), "note": "CPU oracle on host cores"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": int(cores), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_data_parallel(args, spec, ctx, dist, stream, ids_host, dev, rank, world):
    """N > 1 with a real exchange step: every rank trains on its own cache shard and local
    minibatch of B samples; the gradient buffers are summed with one NCCL all-reduce per step
    (enqueued behind the step, no host wait), the optimizer kernel applies 1/world, and the losses
    of the timed region are reduced and read once at its end (global minibatch world*B)."""
    import torch
    import paper_2408_10746_b200 as pac
    from paper_2408_10746_b200.data_parallel import DataParallel, PacLocalTrainer
    K, W, B = args.steps, args.warmup, spec.B
    hp = pac.AdamW()
    dp = DataParallel(PacLocalTrainer(ctx, stream), loss_slots=max(K, W) + 8)
    for i in range(W):
        dp.train_step(ids_host[(i % K) * B:(i % K + 1) * B]); dp.adam_step(hp)
    dp.epoch_losses()
    sampler = ClockSampler(torch.cuda.current_device())
    l0 = ctx.launch_count()
    dist.barrier(); torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
    for i in range(K):
        dp.train_step(ids_host[i * B:(i + 1) * B]); dp.adam_step(hp)
    with torch.cuda.stream(stream):
        e1.record(stream)
    dist.barrier(); torch.cuda.synchronize()
    clocks = sampler.finish()
    losses = dp.epoch_losses()
    if not np.isfinite(losses).all():
        raise SystemExit("non-finite loss in the timed region")
    t = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    value = world * K * B / (ms * 1e-3)
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms / K,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if spec.dtype == "bf16" else "f32",
           "data": "synthetic",
           "config": {"workload": workload_name(spec), "kernel_path": ctx.kernel_path(), "parallelism": f"dp{world}",
                      "global_batch": world * B, "comm": dp.comm + "; no host wait per step, losses reduced once per region"},
           "clocks": clocks, "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 4 * B, "d2h_bytes_per_step": 0, "steps": K,
                                     "note": "host ids in every step; losses read once at the end of the region"},
           "gpu_launches": int(ctx.launch_count() - l0), "roofline": None, "cpu_baseline": None, "final_loss": float(losses[-1])}
    ctx.close()
    dist.barrier()
    dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def run_codec(args):
    """Streaming throughput of pac_quantize_absmax / pac_dequantize_absmax on 2^28 fp32 values
    (1 GiB in, far above L2), against the measured copy bandwidth; 5 algorithmic bytes per element."""
    import torch
    import paper_2408_10746_b200 as pac
    n = 1 << 28
    x = torch.randn(n, device="cuda")
    peaks = load_peaks()
    res = {}
    for block in (64, 4096):
        q, c = pac.quantize_absmax(x, block)
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for _ in range(3):
            q, c = pac.quantize_absmax(x, block)
            out = pac.dequantize_absmax(q, c, block)
        torch.cuda.synchronize()
        tq, td = [], []
        for _ in range(5):
            e[0].record(); q, c = pac.quantize_absmax(x, block)
            e[1].record(); out = pac.dequantize_absmax(q, c, block)
            e[2].record(); torch.cuda.synchronize()
            tq.append(e[0].elapsed_time(e[1])); td.append(e[1].elapsed_time(e[2]))
        gq, gd = 5 * n / (np.median(tq) * 1e-3) / 1e9, 5 * n / (np.median(td) * 1e-3) / 1e9
        res[f"block{block}"] = {"quantize_gbs": gq, "quantize_frac": gq / peaks["hbm_gbs"], "dequantize_gbs": gd,
                                "dequantize_frac": gd / peaks["hbm_gbs"]}
    print(json.dumps({"metric": "absmax_int8_codec_stream", "unit": "GB/s", "n_elements": n, "dtype": "f32->i8",
                      "data": "synthetic", "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "results": res}))


def run_host_cache(args, spec):
    """The cache in page-locked host memory, reloaded per minibatch (paper Section V-B, storage cost
    analysis): whole epochs through pac_train_epoch with host ids in and host losses out.  The reload
    is bound by the host link, so the roofline is the measured host-to-device copy bandwidth."""
    import torch
    import paper_2408_10746_b200 as pac
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    h_cache = torch.empty((spec.N, spec.L, spec.S, spec.d), dtype=torch.bfloat16 if spec.dtype == "bf16" else torch.float32,
                          pin_memory=True)
    chunk = max(1, min(spec.N, (1 << 30) // max(1, spec.cache_bytes // spec.N)))
    for n0 in range(0, spec.N, chunk):                       # generated on the device, kept on the host only
        ids = list(range(n0, min(spec.N, n0 + chunk)))
        h_cache[n0:n0 + len(ids)].copy_(pi.cache_samples(spec, 0, ids, dev))
    h_labels = pi.labels(spec, 0, "cpu").pin_memory()
    # host-to-device copy bandwidth of this machine: 1 GiB page-locked -> device, best of 5
    src = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
    best = 1e9
    for _ in range(6):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); dst.copy_(src, non_blocking=True); e1.record(); torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    h2d_gbs = (1 << 30) / (best * 1e-3) / 1e9
    del src, dst
    stream = torch.cuda.Stream(device=dev)
    ctx = pac.PacContext(0, stream.cuda_stream)
    ctx.cache_register_host(h_cache, h_labels)
    ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B)
    hp = pac.AdamW()
    K, W, B = args.steps, args.warmup, spec.B
    ids_host = epoch_ids(spec, K)
    ctx.train_epoch(epoch_ids(spec, W), B, hp, want_losses=False)
    sampler = ClockSampler(0)
    launches0 = ctx.launch_count()
    torch.cuda.synchronize()
    sampler.start()
    t0 = time.perf_counter()
    losses = ctx.train_epoch(ids_host, B, hp)
    torch.cuda.synchronize()
    ms = 1e3 * (time.perf_counter() - t0)
    clocks = sampler.finish()
    if not np.isfinite(losses).all():
        raise SystemExit("non-finite loss in the timed region")
    pass_bytes = B * spec.L * spec.S * spec.d * spec.elem_bytes
    ach = pass_bytes / (ms * 1e-3 / K) / 1e9
    value = K * B / (ms * 1e-3)
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": ms / K,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if spec.dtype == "bf16" else "f32",
           "data": "synthetic",
           "config": {"workload": workload_name(spec), "cache": "page-locked host memory, reloaded per minibatch into two device "
                      "staging slots (one copy per sample on a copy stream, overlapped with the previous step)",
                      "kernel_path": ctx.kernel_path(), "parallelism": "1 GPU"},
           "clocks": clocks,
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": pass_bytes + 4 * B * (spec.S if spec.head == "lm" else 1),
                   "d2h_bytes_per_step": 4, "steps": K},
           "gpu_launches": int(ctx.launch_count() - launches0),
           "roofline": {"bound": "host_link", "achieved": ach, "peak": h2d_gbs, "unit": "GB/s", "frac": ach / h2d_gbs,
                        "peak_source": "1 GiB page-locked host-to-device copy timed in this run", "traffic": None,
                        "algorithmic_bytes_per_step": pass_bytes},
           "final_loss": float(losses[-1]), "cpu_baseline": None}
    ctx.close()
    print(json.dumps(out))


def measure_aux_workload(spec, dev, stream, peaks, K=64, W=8, R=5):
    """A second shape beside the headline one: the same per-step shapes as the named workload on a
    cache cut to fewer samples (still far larger than L2).  Median of R timed K-step regions plus the
    event-bracketed kernels and the device-timed stream phases."""
    import torch
    import paper_2408_10746_b200 as pac
    from paper_2408_10746_b200 import binding
    cache = pi.cache_full(spec, 0, dev)
    labels = pi.labels(spec, 0, dev)
    ctx = pac.PacContext(dev.index, stream.cuda_stream)
    ctx.cache_register(cache, labels)
    ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B)
    hp = pac.AdamW()
    B = spec.B
    d_ids = torch.from_numpy(epoch_ids(spec, K)).to(dev)
    ctx.train_epoch_dev(d_ids[:W * B], B, hp, None)
    ctx.sync()
    regions = []
    for _ in range(R):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            a.record(stream)
            ctx.train_epoch_dev(d_ids, B, hp, None)
            b.record(stream)
        torch.cuda.synchronize()
        regions.append(a.elapsed_time(b))
    ms = float(np.median(regions))
    pass_bytes = B * spec.L * spec.S * spec.d * spec.elem_bytes
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 1)
    ctx.kernel_times()
    ctx.train_epoch_dev(d_ids[:min(K, 32) * B], B, hp, None)
    kt = ctx.kernel_times()
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 2)
    ctx.train_epoch_dev(d_ids[:min(K, 32) * B], B, hp, None)
    pt = ctx.stream_phase_times()
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 0)
    stream_gbs = 2 * pass_bytes / (ms * 1e-3 / K) / 1e9
    out = {"workload": workload_name(spec), "kernel_path": ctx.kernel_path(), "steps": K, "repeats": R,
           "ms_per_step": ms / K, "samples_per_s": K * B / (ms * 1e-3),
           "cache_stream": {"gbs_two_reads": stream_gbs, "frac_of_peak": stream_gbs / peaks["hbm_gbs"]},
           "kernels": {n: {"avg_ms": t / c, **({"gbs": pass_bytes / (t / c * 1e-3) / 1e9,
                                                 "frac": pass_bytes / (t / c * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                                                if n in ("down_projection", "dw_down") else {})}
                       for n, (t, c) in kt.items() if c},
           "stream_phase": {n: {"avg_ms": t / c, "frac": pass_bytes / (t / c * 1e-3) / 1e9 / peaks["hbm_gbs"]}
                            for n, (t, c) in pt.items() if c}}
    ctx.close()
    del cache, labels
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2560)
    ap.add_argument("--warmup", type=int, default=128)
    ap.add_argument("--config", default="t5_base", choices=sorted(pi.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for cpu_baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--force-simt", action="store_true", help="use the plain fp32-FMA kernels")
    ap.add_argument("--forward", choices=["auto", "split", "one-kernel"], default="auto",
                    help="tensor-core path: down-projections and head phase as one kernel or two (default: library's choice)")
    ap.add_argument("--parallelism", default="replicas", choices=["replicas", "dp"],
                    help="N > 1: independent replicas (default) or data parallel with a per-step all-reduce of "
                         "the adapter gradients (paper Section V-B)")
    ap.add_argument("--codec", action="store_true",
                    help="measure the block-wise absmax INT8 codec (paper Eq. 1-2) instead of the train step")
    ap.add_argument("--cache", choices=["device", "host"], default="device",
                    help="host: keep the cache in page-locked host memory and reload every minibatch (N defaults to 1024)")
    ap.add_argument("--repeats", type=int, default=0,
                    help="how many times the K-step region is timed (median reported); default: at least 5, more "
                         "for short regions")
    ap.add_argument("--no-aux-workloads", action="store_true",
                    help="skip the reduced-N BART-Large / T5-Large entries of aux.workloads")
    ap.add_argument("--n-samples", type=int, default=0,
                    help="profiling aid: shrink the cache to this many samples (same per-step shapes); "
                         "the JSON line then names the reduced workload")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    spec = pi.CONFIGS[args.config]
    if args.n_samples:
        spec = spec.scaled(N=args.n_samples, name=f"{spec.name}[N={args.n_samples}]")
    if args.impl == "reference":
        return run_reference(args, spec)
    if args.codec:
        return run_codec(args)
    if args.cache == "host":
        if not args.n_samples:
            spec = spec.scaled(N=min(spec.N, 1024), name=f"{spec.name}[N={min(spec.N, 1024)}]")
        if args.steps == 2560:
            args.steps, args.warmup = 256, 16
        return run_host_cache(args, spec)

    import torch
    import paper_2408_10746_b200 as pac
    from paper_2408_10746_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1 or args.parallelism == "dp":
        import torch.distributed as dist
        if world == 1:                       # a one-rank group: the data-parallel path itself, without an exchange partner
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29531")
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", local))
        else:
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # the cache must fit: keep 8 GB of headroom, halve N otherwise (and say so)
    note = []
    free, _ = torch.cuda.mem_get_info()
    while spec.cache_bytes + (8 << 30) > free and spec.N > spec.B:
        spec = spec.scaled(N=spec.N // 2)
        note.append(f"N halved to {spec.N} to fit device memory")

    dev = torch.device("cuda", local)
    seed = rank                                   # each rank trains its own replica on its own cache
    cache = pi.cache_full(spec, seed, dev)
    labels = pi.labels(spec, seed, dev)
    lm = pi.lm_head(spec, seed, dev) if spec.head == "lm" else None
    stream = torch.cuda.Stream(device=dev)
    ctx = pac.PacContext(local, stream.cuda_stream)
    if args.force_simt:
        ctx.set_option(binding.PAC_OPT_KERNEL_PATH, 1)
    elif args.forward != "auto":
        ctx.set_option(binding.PAC_OPT_KERNEL_PATH, 3 if args.forward == "one-kernel" else 2)
    ctx.cache_register(cache, labels)
    ctx.adapter_init(r=spec.r, n_out=spec.n_out, max_batch=spec.B,
                     head=pac.PAC_HEAD_FROZEN_LM if spec.head == "lm" else pac.PAC_HEAD_MEANPOOL_CLS, lm_head=lm)
    hp = pac.AdamW()
    K, W, B = args.steps, args.warmup, spec.B
    ids_host = epoch_ids(spec, K)
    d_ids = torch.from_numpy(ids_host).to(dev)
    d_warm = torch.from_numpy(epoch_ids(spec, W)).to(dev)
    d_losses = torch.zeros(K, dtype=torch.float32, device=dev)
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    if args.parallelism == "dp":
        return run_data_parallel(args, spec, ctx, dist, stream, ids_host, dev, rank, world)

    # ---------------- device-resident timing (value) ----------------
    # The K-step region is timed R >= 5 times (each bracketed by a barrier and a device synchronisation
    # on both sides, CUDA events on the context's stream); the line reports the median region.  R grows
    # for short regions so that the clock sampler, which runs across all repeats, sees enough samples.
    ctx.train_epoch_dev(d_warm, B, hp, None)
    ctx.sync()
    probe0, probe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        probe0.record(stream)
        ctx.train_epoch_dev(d_ids, B, hp, None)
        probe1.record(stream)
    ctx.sync()
    region_est_ms = max(1e-3, probe0.elapsed_time(probe1))
    R = args.repeats if args.repeats > 0 else int(min(100, max(5, np.ceil(150.0 / region_est_ms))))
    if dist is not None:
        rt = torch.tensor([R], dtype=torch.int64, device=dev)
        dist.all_reduce(rt, op=dist.ReduceOp.MAX)
        R = int(rt.item())
    sampler = ClockSampler(local, period_s=0.002)
    launches0 = ctx.launch_count()
    region_ms, t_enq = [], 0.0
    barrier()
    sampler.start()
    for rep in range(R):
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(stream):
            start.record(stream)
            t0 = time.perf_counter()
            ctx.train_epoch_dev(d_ids, B, hp, d_losses)
            t_enq += time.perf_counter() - t0               # the call returns once everything is enqueued
            end.record(stream)
        barrier()
        region_ms.append(start.elapsed_time(end))
    clocks = sampler.finish()
    t_enq /= R
    launches = (ctx.launch_count() - launches0) // R        # launches of ONE K-step region
    ctx.sync()
    if dist is not None:
        t = torch.tensor(region_ms, dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)            # per repeat, the slowest rank
        region_ms = t.tolist()
    ms = float(np.median(region_ms))
    losses = d_losses.cpu().numpy()
    if not np.isfinite(losses).all():
        raise SystemExit("non-finite loss in the timed region")

    # ---------------- end to end through the public per-step call ----------------
    # every step: B ids from page-locked host memory in (H2D), the step's loss out to page-locked
    # host memory (D2H); one wait at the end, then every loss is checked on the host
    Ke = K
    h_ids = torch.from_numpy(ids_host[:Ke * B].copy()).pin_memory()
    h_losses = torch.zeros(Ke, dtype=torch.float32).pin_memory()
    ids_view, loss_ptr = h_ids.numpy(), h_losses.data_ptr()
    for i in range(3):
        ctx.train_step_async(ids_view[i * B:(i + 1) * B], hp, loss_ptr + 4 * i)
    ctx.sync()
    e2e_regions, enqueue_ms = [], 0.0
    for rep in range(R):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0 = time.perf_counter()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for i in range(Ke):
                ctx.train_step_async(ids_view[i * B:(i + 1) * B], hp, loss_ptr + 4 * i)
            e1.record(stream)
        enqueue_ms += 1e3 * (time.perf_counter() - t0)      # host time to enqueue the Ke steps
        ctx.sync()
        barrier()
        wall_ms = 1e3 * (time.perf_counter() - t0)
        e2e_regions.append(max(e0.elapsed_time(e1), wall_ms))
        if not np.isfinite(h_losses.numpy()).all():
            raise SystemExit("non-finite loss in the end-to-end region")
    enqueue_ms /= R
    e2e_ms = float(np.median(e2e_regions))

    # ---------------- per-kernel times of the two cache-stream kernels ----------------
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 1)
    ctx.kernel_times()
    Kt = min(K, 256)
    ctx.train_epoch_dev(d_ids[:Kt * B], B, hp, None)
    kt = ctx.kernel_times()
    # the same steps once more with device-side timestamps of the passes' stream phases; no event
    # brackets, so the kernels overlap as in the timed region
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 2)
    ctx.train_epoch_dev(d_ids[:Kt * B], B, hp, None)
    pt = ctx.stream_phase_times()
    ctx.set_option(binding.PAC_OPT_KERNEL_TIMING, 0)

    # ---------------- the two smaller calls of the boundary: stand-alone gather and evaluation ----------------
    aux = {}
    if rank == 0 and spec.head == "cls":
        n_aux = min(64, K)
        g_out = torch.empty((spec.L, B, spec.S, spec.d), dtype=cache.dtype, device=dev)
        ev_out = torch.empty((B, spec.n_out), dtype=torch.float32, device=dev)
        for name, call in (("gather", lambda i: ctx.gather(ids_host[i * B:(i + 1) * B], g_out)),
                           ("eval_logits", lambda i: ctx.eval_logits(ids_host[i * B:(i + 1) * B], ev_out))):
            for i in range(3):
                call(i)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ctx.sync()
            with torch.cuda.stream(stream):
                a0.record(stream)
                for i in range(n_aux):
                    call(i)
                a1.record(stream)
            ctx.sync()
            per_ms = a0.elapsed_time(a1) / n_aux
            aux[name] = {"ms_per_call": per_ms, "samples_per_s": B / (per_ms * 1e-3), "calls": n_aux}
        pass_b = B * spec.L * spec.S * spec.d * spec.elem_bytes
        aux["gather"]["gbs_read_plus_write"] = 2 * pass_b / (aux["gather"]["ms_per_call"] * 1e-3) / 1e9
        aux["gather"]["frac_of_peak"] = aux["gather"]["gbs_read_plus_write"] / load_peaks()["hbm_gbs"]
        aux["eval_logits"]["gbs_cache_read"] = pass_b / (aux["eval_logits"]["ms_per_call"] * 1e-3) / 1e9
        aux["note"] = "host ids per call (H2D of B ids inside the timed region), events on the context's stream"

    if dist is not None:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())

    peaks = load_peaks()
    pass_bytes = B * spec.L * spec.S * spec.d * spec.elem_bytes          # one read of the minibatch's slabs
    kern = {}
    for name, (tot_ms, cnt) in kt.items():
        if cnt:
            avg = tot_ms / cnt
            kern[name] = {"avg_ms": avg, "launches": cnt}
            if name in ("down_projection", "dw_down"):      # the two passes over the cached activations
                kern[name]["gbs"] = pass_bytes / (avg * 1e-3) / 1e9
    phases = {}
    for name, (tot_ms, cnt) in pt.items():
        if cnt:
            avg = tot_ms / cnt
            phases[name] = {"avg_ms": avg, "launches": cnt, "gbs": pass_bytes / (avg * 1e-3) / 1e9,
                            "frac": pass_bytes / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    if spec.head == "lm":
        # the two dense contractions of the frozen LM head: tensor-core bound
        gemm_flop = 2.0 * B * spec.S * spec.n_out * spec.d
        for old, new in (("chain_head", "lm_logits_gemm"), ("finalize", "lm_dy_gemm")):
            if old in kern:
                kern[new] = kern.pop(old)
                kern[new]["tflops"] = gemm_flop / (kern[new]["avg_ms"] * 1e-3) / 1e12
    stream_k = [k for k in kern if "gbs" in kern[k]]
    dominant = max(stream_k, key=lambda k: kern[k]["avg_ms"]) if stream_k else None
    roofline = None
    if dominant:
        a = kern[dominant]["gbs"]
        roofline = {"bound": "hbm", "kernel": dominant, "achieved": a, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": a / peaks["hbm_gbs"], "peak_source": peaks["source"],
                    "traffic": ncu_traffic(spec, ctx.kernel_path(), dominant), "algorithmic_bytes_per_launch": pass_bytes,
                    "kernels": kern,
                    # first cache copy issued -> last accumulator complete, over all CTAs of a launch (device
                    # timestamps): the part of each pass that streams the minibatch's slabs
                    "stream_phase": phases}
    gemm_k = [k for k in kern if "tflops" in kern[k]]
    if gemm_k and max(kern[k]["avg_ms"] for k in gemm_k) > (kern[dominant]["avg_ms"] if dominant else 0.0):
        # the dominant kernel is a dense contraction: report it against the measured bf16 GEMM peak
        # (the sustained figure: the kernel runs inside a long step)
        gk = max(gemm_k, key=lambda k: kern[k]["avg_ms"])
        tf_peak, tf_src = 1400.0, "fallback"
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                tf_peak, tf_src = float(json.load(f)["bf16_tflops_sustained"]), "measured (sustained)"
        except Exception:
            pass
        roofline = {"bound": "tensor", "kernel": gk, "achieved": kern[gk]["tflops"], "peak": tf_peak, "unit": "TFLOP/s",
                    "frac": kern[gk]["tflops"] / tf_peak, "peak_source": tf_src, "traffic": None,
                    "flop_per_launch": 2.0 * B * spec.S * spec.n_out * spec.d, "kernels": kern, "stream_phase": phases}
    step_s = ms * 1e-3 / K
    stream_gbs = 2 * pass_bytes / step_s / 1e9

    out = {
        "metric": METRIC, "value": world * K * B / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if spec.dtype == "bf16" else "f32", "data": "synthetic",
        "repeats": {"n": R, "statistic": "median", "region_ms_min": float(np.min(region_ms)), "region_ms_median": ms,
                    "region_ms_max": float(np.max(region_ms))},
        "config": {"workload": workload_name(spec), "kernel_path": ctx.kernel_path(),
                   "l2": "each step gathers a different minibatch from a cache far larger than L2 "
                         f"({spec.cache_bytes / 1e9:.2f} GB)", "parallelism": "replicas" if world > 1 else "1 GPU",
                   "notes": note},
        "clocks": clocks,
        "e2e": {"value": world * Ke * B / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": 4 * B,
                "d2h_bytes_per_step": 4, "steps": Ke, "host_enqueue_us_per_step": 1e3 * enqueue_ms / Ke},
        "gpu_launches": int(launches),
        "host_enqueue_us_per_step": 1e6 * t_enq / K,
        "roofline": roofline,
        "cache_stream": {"gbs_two_reads": stream_gbs, "frac_of_peak": stream_gbs / peaks["hbm_gbs"],
                         "gbs_one_read": stream_gbs / 2, "peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
                         "frac_of_8000_nominal": stream_gbs / 8000.0},
        "final_loss": float(losses[-1]),
        "aux": aux,
    }
    if rank == 0 and world == 1 and args.config == "t5_base" and not args.n_samples and not args.no_aux_workloads \
            and not args.force_simt:
        # two more shapes beside the headline one, each named as a reduced-N entry
        ctx.close()
        del cache, d_ids, d_warm
        torch.cuda.empty_cache()
        out["aux"]["workloads"] = []
        for name in ("bart_large", "t5_large"):
            big = pi.CONFIGS[name]
            out["aux"]["workloads"].append(measure_aux_workload(big.scaled(N=512, name=f"{name}[N=512]"), dev, stream, peaks))
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = oracle_baseline(spec, args.cpu_budget, 256)
    elif rank == 0:
        out["cpu_baseline"] = None
    ctx.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


if __name__ == "__main__":
    main()

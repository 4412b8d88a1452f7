#!/usr/bin/env python
"""Benchmark of the gradient-quantization hot path on B200.

One step = the whole path over one batch of synthetic gradients: for each of the K simulated
workers, level solver + quantize + bit-pack of that worker's bucket, then one unpack + dequantize
+ sum over the K packed buffers.  The metric is GB/s of fp32 gradient consumed by
levels + quantize + pack (4 bytes x elements x K per step) over the step time.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # times the CPU oracle on a bounded sample

Prints one JSON line (rank 0).
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import ogq_workloads as wl  # noqa: E402

METRIC = "fp32-gradient GB/s through levels+quantize+pack; % of B200 HBM roofline"
UNIT = "GB/s"

SCHEMES = {
    # name: (scheme id, levels s, lloyd iterations)
    "orq3": (2, 3, 0), "orq5": (2, 5, 0), "orq9": (2, 9, 0), "orq17": (2, 17, 0),
    "bingrad_b": (1, 2, 0), "bingrad_pb": (0, 2, 0),
}


def make_bucket(workload: str, worker: int) -> wl.Bucket:
    if workload == "vgg19":
        return wl.vgg19_bucket(worker)
    if workload == "resnet50":
        return wl.resnet50_bucket(worker)
    if workload == "c2":
        return wl.config2(2 + worker)
    if workload == "c1":
        return wl.config1(worker)
    if workload.startswith("sweep"):
        return wl.sweep_tensor(int(workload[5:]), 7 + worker)
    raise SystemExit(f"unknown workload {workload}")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            p = [x.strip() for x in ln.split(",")]
            if len(p) < 6:
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for nm, val in zip(names, p[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- CPU oracle arm


def oracle_sample(workload: str, scheme_name: str, seconds: float = 15.0):
    """Times the CPU oracle (levels + quantize + pack) on a bounded sample of worker 0's bucket:
    a prefix of its largest tensor sized for about `seconds` of single-threaded work."""
    import oracle

    scheme, s, lloyd = SCHEMES[scheme_name]
    b = make_bucket(workload, 0)
    sizes = np.diff(b.offsets)
    t_big = int(np.argmax(sizes))
    big = b.tensor(t_big)

    def run(v):
        t0 = time.perf_counter()
        off = np.array([0, v.size], np.int64)
        if scheme == 2:
            lv, _ = oracle.bucket_levels_orq(v, off, s)
            oracle.bucket_quantize_pack(v, off, oracle.ORQ, s, lv, None, 1, 0)
        else:
            lv, th, _ = oracle.bucket_levels_bingrad(v, off, scheme, lloyd)
            oracle.bucket_quantize_pack(v, off, scheme, 2, lv, th, 1, 0)
        return time.perf_counter() - t0

    probe = min(big.size, 1 << 17)
    rate = probe / max(run(big[:probe]), 1e-9)  # elements per second
    m = int(min(big.size, max(probe, rate * seconds)))
    return big[:m], run, f"first {m} elements of the largest tensor ({sizes[t_big]} elements) of worker 0"


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    budget = 150.0 / (steps + warmup)
    v, run, what = oracle_sample(args.workload, args.scheme, seconds=min(15.0, budget))
    for _ in range(warmup):
        run(v)
    t0 = time.perf_counter()
    for _ in range(steps):
        run(v)
    dt = (time.perf_counter() - t0) / steps
    value = 4.0 * v.size / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "scheme": args.scheme, "sample": what},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm


def run_ours(args):
    import torch

    import paper_2002_11082_b200 as ogq
    from paper_2002_11082_b200.sharding import aggregate_throughput, max_over_ranks, worker_ids

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    scheme, s, lloyd = SCHEMES[args.scheme]
    K = args.workers
    bits = ogq.ogq_bits_for_levels(s)

    # ---- inputs: K workers' buckets, generated on the host and made resident in HBM
    host = [make_bucket(args.workload, w) for w in worker_ids(rank, K)]
    h_off = host[0].offsets
    T, N = host[0].num_tensors, host[0].total
    off = torch.from_numpy(h_off).to(dev)
    h_po = ogq.ogq_packed_layout(h_off, bits)
    po = torch.from_numpy(h_po).to(dev)
    grads = [torch.from_numpy(h.values).to(dev) for h in host]
    levels = [torch.zeros((T, s), device=dev) for _ in range(K)]
    thresh = [torch.zeros((T,), device=dev) for _ in range(K)]
    status = [torch.zeros((T,), dtype=torch.int32, device=dev) for _ in range(K)]
    packed = [torch.zeros((int(h_po[-1]),), dtype=torch.int32, device=dev) for _ in range(K)]
    ws_bytes = ogq.ogq_workspace_bytes(T, N, max(s, 3))
    # workers alternate between `args.streams` CUDA streams, each with its own scratch, so that the
    # short single-CTA solver tails of one worker overlap the streaming kernels of the next
    n_streams = max(1, min(args.streams, K))
    wss = [torch.empty(ws_bytes, dtype=torch.uint8, device=dev) for _ in range(n_streams)]
    side = [torch.cuda.Stream(device=dev) for _ in range(n_streams)] if n_streams > 1 else []
    out = torch.empty(N, device=dev)
    pk_ptrs = ogq.device_pointer_array(packed)
    lv_ptrs = ogq.device_pointer_array(levels)

    def lqp(k, stream=None):
        ws = wss[k % n_streams]
        if scheme == ogq.OGQ_ORQ:
            ogq.ogq_levels_orq(grads[k], off, T, N, s, levels[k], status[k], ws, ws_bytes, stream)
            ogq.ogq_quantize_pack(grads[k], off, T, N, scheme, s, levels[k], None, args.seed, k, po, packed[k], stream)
        else:
            ogq.ogq_levels_bingrad(grads[k], off, T, N, scheme, lloyd, levels[k], thresh[k], status[k], ws, ws_bytes,
                                   stream)
            ogq.ogq_quantize_pack(grads[k], off, T, N, scheme, 2, levels[k], thresh[k], args.seed, k, po, packed[k],
                                  stream)

    def unpack():
        ogq.ogq_unpack_sum(pk_ptrs, lv_ptrs, K, off, po, T, N, s, 1.0 / K, out)

    def lqp_all(before=None):
        """levels + quantize + pack of all K workers; `before(k)` runs on worker k's stream first."""
        if n_streams == 1:
            for k in range(K):
                if before is not None:
                    before(k)
                lqp(k)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        for st in side:
            st.wait_event(fork)
        for k in range(K):
            with torch.cuda.stream(side[k % n_streams]):
                if before is not None:
                    before(k)
                lqp(k, side[k % n_streams])
        for st in side:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def step():
        lqp_all()
        unpack()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # L2 hygiene: the large buckets cycle through far more than the 126 MB L2 per step; for the small
    # workloads a buffer larger than L2 is overwritten before every timed step, outside the timed events
    need_flush = 4 * N * K <= 2 * 126e6
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if need_flush else None

    def timed(fn, reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        if not need_flush:
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            barrier()
            return max_over_ranks(a.elapsed_time(b), dist, dev)
        total = 0.0
        for _ in range(reps):
            flush_buf.fill_(1)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            total += a.elapsed_time(b)
        barrier()
        return max_over_ranks(total, dist, dev)

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    bad = [int(st.bitwise_and(16 | 8).count_nonzero().item()) for st in status]
    if any(bad):
        raise SystemExit(f"solver reported unresolved tensors: {bad}")

    # ---- the timed region: exactly `steps` steps
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ogq.ogq_launch_count()
    ms_total = timed(step, steps)
    launches = ogq.ogq_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_step = ms_total / steps
    grad_bytes = 4.0 * N * K  # fp32 gradient consumed per step and rank
    value = aggregate_throughput(grad_bytes, ms_step, world)

    # ---- per-stage and per-kernel times (separate instrumented passes, not part of `value`)
    ms_lqp = timed(lqp_all, steps) / steps
    ms_unp = timed(unpack, steps) / steps
    ogq.ogq_profile_enable(True)  # per-kernel times: one stream, so that no two kernels overlap
    torch.cuda.synchronize()
    for _ in range(steps):
        for k in range(K):
            lqp(k)
        unpack()
    torch.cuda.synchronize()
    recs = ogq.ogq_profile_collect()
    ogq.ogq_profile_enable(False)
    per_kernel = {}
    for name, ms in recs:
        tot, cnt = per_kernel.get(name, (0.0, 0))
        per_kernel[name] = (tot + ms, cnt + 1)
    alg_bytes = {  # algorithmic bytes of one launch, per the accounting in the design notes
        "k_sel_round1": 4.0 * N, "k_sel_round2": 4.0 * N, "k_sel_round3": 0.0, "k_bb_pass": 4.0 * N,
        "k_quantize_pack_random": (4.0 + bits / 8.0) * N, "k_quantize_pack_threshold": (4.0 + 1 / 8.0) * N,
        "k_unpack_sum": (K * bits / 8.0 + 4.0) * N,
    }
    peak, peak_src = measured_peaks()
    kernels = {}
    total_ms = max(sum(v[0] for v in per_kernel.values()), 1e-12)
    for name, (tot, cnt) in per_kernel.items():
        avg = tot / cnt
        gbs = alg_bytes.get(name, 0.0) / (avg * 1e-3) / 1e9 if avg > 0 else 0.0
        kernels[name] = {"launches_per_step": cnt / steps, "avg_ms": avg, "share": tot / total_ms, "alg_gbs": gbs}
    dom = max(per_kernel, key=lambda k: per_kernel[k][0])
    # DRAM bytes per element (dram__bytes_read.sum + dram__bytes_write.sum) of one launch, from one ncu
    # capture of the current kernels on a 2^26-element tensor with s = 9; traffic grows in proportion to
    # the elements streamed, so a full launch is this figure times N.  Other schemes: not captured.
    ncu_dram_bytes_per_element = {"k_sel_round1": 4.461, "k_sel_round2": 4.232, "k_quantize_pack_random": 4.397}
    traffic = None
    if args.scheme == "orq9" and dom in ncu_dram_bytes_per_element:
        traffic = ncu_dram_bytes_per_element[dom] * N
    roofline = {
        "bound": "hbm", "kernel": dom, "achieved": kernels[dom]["alg_gbs"], "peak": peak, "unit": "GB/s",
        "frac": kernels[dom]["alg_gbs"] / peak, "traffic": traffic, "peak_source": peak_src,
        "alg_bytes_per_launch": alg_bytes.get(dom, 0.0),
    }

    # ---- end to end through the C ABI with host buffers (H2D of every worker's bucket, D2H of the result)
    e2e = None
    if not args.no_e2e:
        pinned = [torch.from_numpy(h.values).pin_memory() for h in host]
        h_out = torch.empty(N, dtype=torch.float32).pin_memory()

        def e2e_step():
            lqp_all(before=lambda k: grads[k].copy_(pinned[k], non_blocking=True))
            unpack()
            h_out.copy_(out, non_blocking=True)

        e2e_steps = min(steps, 5)
        e2e_step()
        ms_e2e = timed(e2e_step, e2e_steps) / e2e_steps
        e2e = {"value": aggregate_throughput(grad_bytes, ms_e2e, world), "unit": UNIT,
               "h2d_bytes_per_step": int(4 * N * K), "d2h_bytes_per_step": int(4 * N),
               "ms_per_step": ms_e2e, "steps": e2e_steps}

    # ---- CPU oracle on a bounded sample (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        v, run, what = oracle_sample(args.workload, args.scheme, seconds=args.cpu_seconds)
        dt = run(v)
        cpu = {"value": 4.0 * v.size / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": what,
               "seconds": dt}

    if rank == 0:
        alg_lqp = (8.0 + bits / 8.0) * N * K
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "scheme": args.scheme, "levels": s, "bits": bits,
                       "workers_per_gpu": K, "tensors": T, "elements": N, "streams": n_streams,
                       "l2": "256 MB written between timed steps (flush)" if need_flush else "inputs larger than L2 (no flush)"},
            "stages": {
                "levels_quantize_pack": {"ms": ms_lqp, "grad_gbs": grad_bytes / (ms_lqp * 1e-3) / 1e9,
                                         "alg_bytes_per_elem": 8.0 + bits / 8.0,
                                         "frac_of_hbm_peak": alg_lqp / (ms_lqp * 1e-3) / 1e9 / peak,
                                         "frac_of_nominal_8tbs": alg_lqp / (ms_lqp * 1e-3) / 1e9 / 8000.0},
                "unpack_sum": {"ms": ms_unp, "alg_gbs": (K * bits / 8.0 + 4.0) * N / (ms_unp * 1e-3) / 1e9},
            },
            "kernels": kernels, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vgg19")
    ap.add_argument("--scheme", default="orq9", choices=sorted(SCHEMES))
    ap.add_argument("--workers", type=int, default=8)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--streams", type=int, default=8)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

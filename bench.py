#!/usr/bin/env python
"""Benchmark of the gradient-quantization hot path on B200.

One step = the whole path over one batch of synthetic gradients: for each of the K simulated
workers, level solver + quantize + bit-pack of that worker's bucket, then one unpack + dequantize
+ sum over the K packed buffers.  The metric is GB/s of fp32 gradient consumed by
levels + quantize + pack (4 bytes x elements x K per step) over the step time.

    python bench.py --gpus 1 --steps 10 --warmup 3
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # times the CPU oracle on a bounded sample
    python bench.py --workload resnet50 --bucket-len 512   # fixed-length bucket mode

Prints one JSON line (rank 0).  Besides the headline (K workers on K streams) the line carries the
same stage with all workers on one stream (`single_stream`) and, for the default configuration,
short runs of the other headline workloads and schemes (`secondary`).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import multiprocessing
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


def _oracle_task(task):
    """levels + quantize + pack of one tensor by the oracle (runs in a worker process)."""
    v, scheme, s, lloyd = task
    import oracle

    off = np.array([0, v.size], np.int64)
    if scheme == 2:
        lv, _ = oracle.bucket_levels_orq(v, off, s)
        oracle.bucket_quantize_pack(v, off, oracle.ORQ, s, lv, None, 1, 0)
    else:
        lv, th, _ = oracle.bucket_levels_bingrad(v, off, scheme, lloyd)
        oracle.bucket_quantize_pack(v, off, scheme, 2, lv, th, 1, 0)
    return v.size


class OraclePool:
    """The machine's host cores as oracle workers (spawned, so that no CUDA state is inherited)."""

    def __init__(self, cores=None):
        self.cores = cores or os.cpu_count() or 1
        self.pool = multiprocessing.get_context("spawn").Pool(self.cores)
        self.pool.map(_oracle_task, [(np.zeros(64, np.float32), 2, 3, 0)] * self.cores)  # load the library

    def close(self):
        self.pool.close()
        self.pool.join()

    def sample(self, workload: str, scheme_name: str, seconds: float):
        """A bounded sample of worker 0's bucket, sized for about `seconds` on all cores: whole tensors
        where they are small enough, the first kCap elements of the larger ones (the sort-based oracle
        grows faster than linearly), largest pieces dropped first when the estimate is still too long."""
        kCap = 1 << 22
        scheme, s, lloyd = SCHEMES[scheme_name]
        b = make_bucket(workload, 0)
        sizes = np.diff(b.offsets)
        probe = b.tensor(int(np.argmax(sizes)))[: 1 << 18]
        t0 = time.perf_counter()
        _oracle_task((probe, scheme, s, lloyd))
        unit = (time.perf_counter() - t0) / (probe.size * np.log2(probe.size))  # seconds per n log2 n
        pieces = [b.tensor(t)[:kCap] for t in range(b.num_tensors) if sizes[t] > 0]
        pieces.sort(key=lambda v: v.size)
        cost = lambda v: unit * v.size * max(1.0, np.log2(max(v.size, 2)))
        while len(pieces) > self.cores and sum(cost(v) for v in pieces) / self.cores > seconds:
            pieces.pop()
        used = int(sum(v.size for v in pieces))
        capped = int(sum(1 for v in pieces if v.size == kCap))
        if used == b.total:
            what = f"whole bucket of worker 0 ({b.num_tensors} tensors, {b.total} elements)"
        else:
            what = (f"{len(pieces)} of the {b.num_tensors} tensors of worker 0's bucket, smallest first, {capped} of them "
                    f"cut to their first {kCap} elements ({used} of {b.total} elements)")
        tasks = [(v, scheme, s, lloyd) for v in reversed(pieces)]
        return tasks, used, what

    def run(self, tasks) -> float:
        t0 = time.perf_counter()
        self.pool.map(_oracle_task, tasks, chunksize=1)
        return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    budget = 150.0 / (steps + warmup)
    pool = OraclePool()
    tasks, used, what = pool.sample(args.workload, args.scheme, seconds=min(12.0, budget))
    for _ in range(warmup):
        pool.run(tasks)
    t0 = time.perf_counter()
    for _ in range(steps):
        pool.run(tasks)
    dt = (time.perf_counter() - t0) / steps
    pool.close()
    value = 4.0 * used / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "scheme": args.scheme, "sample": what},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": pool.cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- CUDA arm


def kernel_sources_hash() -> str:
    """sha256 over the kernel sources and the header: the key of the stored DRAM-traffic figures."""
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2002_11082_b200", "csrc")
    for name in sorted(os.listdir(csrc)) + ["../../include/ogq.h"]:
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()


def stored_traffic(kernel: str, scheme: str):
    """DRAM bytes per element of `kernel` from the committed ncu summary, or None when the kernels have
    changed since it was taken (the file records the hash of the sources it was measured on)."""
    path = os.path.join(ROOT, "profiles", "dram_bytes_per_element.json")
    try:
        rec = json.load(open(path))
        if rec.get("sources_sha256") != kernel_sources_hash():
            return None
        return rec["entries"].get(f"{kernel}|{scheme}")
    except Exception:
        return None


class Setup:
    """One workload x scheme resident in HBM: K workers' buckets, outputs, scratch, streams."""

    def __init__(self, torch, ogq, dev, workload, scheme_name, K, seed, rank, bucket_len=0, share=None, dense=False):
        from paper_2002_11082_b200.sharding import worker_ids

        self.torch, self.ogq, self.dev = torch, ogq, dev
        self.workload, self.scheme_name, self.K, self.seed = workload, scheme_name, K, seed
        self.scheme, self.s, self.lloyd = SCHEMES[scheme_name]
        self.bits = ogq.ogq_bits_for_levels(self.s)
        self.bucket_len = bucket_len
        self.clip_c = 0.0
        self.dense = bool(dense) and self.scheme == 2
        if share is not None and share.workload == workload:
            self.host, self.grads = share.host, share.grads
        else:
            self.host = [make_bucket(workload, w) for w in worker_ids(rank, K)]
            self.grads = [torch.from_numpy(h.values).to(dev) for h in self.host]
        self.N = self.host[0].total
        if bucket_len:
            nb = (self.N + bucket_len - 1) // bucket_len
            self.h_off = np.minimum(np.arange(nb + 1, dtype=np.int64) * bucket_len, self.N)
        else:
            self.h_off = self.host[0].offsets
        self.T = self.h_off.size - 1
        T, s = self.T, self.s
        self.off = torch.from_numpy(self.h_off).to(dev)
        self.h_po = ogq.ogq_dense_layout(self.h_off, self.s) if self.dense else ogq.ogq_packed_layout(self.h_off, self.bits)
        self.code_bits = 32.0 / ogq.ogq_dense_digits(self.s) if self.dense else float(self.bits)
        self.po = torch.from_numpy(self.h_po).to(dev)
        self.levels = [torch.zeros((T, s), device=dev) for _ in range(K)]
        self.thresh = [torch.zeros((T,), device=dev) for _ in range(K)]
        self.status = [torch.zeros((T,), dtype=torch.int32, device=dev) for _ in range(K)]
        self.packed = [torch.zeros((int(self.h_po[-1]),), dtype=torch.int32, device=dev) for _ in range(K)]
        self.ws_bytes = 256 if bucket_len else ogq.ogq_workspace_bytes(T, self.N, max(s, 3))
        self.wss = [torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev) for _ in range(K)]
        self.side = [torch.cuda.Stream(device=dev) for _ in range(K)]
        self.out = torch.empty(self.N, device=dev)
        self.pk_ptrs = ogq.device_pointer_array(self.packed)
        self.lv_ptrs = ogq.device_pointer_array(self.levels)
        self.grad_bytes = 4.0 * self.N * K
        self.alg_lqp = (8.0 + self.code_bits / 8.0) * self.N * K

    def lqp(self, k, stream=None, slot=None):
        """levels + quantize + pack of worker k (scratch slot = the stream's own)."""
        ogq, s = self.ogq, self.s
        ws = self.wss[k if slot is None else slot]
        if self.bucket_len:
            ogq.ogq_bucket_encode(self.grads[k], self.N, self.bucket_len, self.scheme, s, 0, self.clip_c, self.seed, k,
                                  self.levels[k], self.thresh[k], self.status[k], self.packed[k], stream)
        elif self.scheme == ogq.OGQ_ORQ:
            ogq.ogq_levels_orq(self.grads[k], self.off, self.T, self.N, s, self.levels[k], self.status[k], ws,
                               self.ws_bytes, stream)
            if self.dense:
                ogq.ogq_quantize_pack_dense(self.grads[k], self.off, self.T, self.N, s, self.levels[k], self.seed, k,
                                            self.po, self.packed[k], stream)
            else:
                ogq.ogq_quantize_pack(self.grads[k], self.off, self.T, self.N, self.scheme, s, self.levels[k], None,
                                      self.seed, k, self.po, self.packed[k], stream)
        else:
            ogq.ogq_levels_bingrad(self.grads[k], self.off, self.T, self.N, self.scheme, self.lloyd, self.levels[k],
                                   self.thresh[k], self.status[k], ws, self.ws_bytes, stream)
            ogq.ogq_quantize_pack(self.grads[k], self.off, self.T, self.N, self.scheme, 2, self.levels[k],
                                  self.thresh[k], self.seed, k, self.po, self.packed[k], stream)

    def unpack(self):
        if self.bucket_len:
            self.ogq.ogq_bucket_decode_sum(self.pk_ptrs, self.lv_ptrs, self.K, self.N, self.bucket_len, self.s,
                                           1.0 / self.K, self.out)
            return
        if self.dense:
            self.ogq.ogq_unpack_sum_dense(self.pk_ptrs, self.lv_ptrs, self.K, self.off, self.po, self.T, self.N, self.s,
                                          1.0 / self.K, self.out)
            return
        self.ogq.ogq_unpack_sum(self.pk_ptrs, self.lv_ptrs, self.K, self.off, self.po, self.T, self.N, self.s,
                                1.0 / self.K, self.out)

    def lqp_all(self, n_streams, before=None):
        """levels + quantize + pack of all K workers, worker k on stream k mod n_streams;
        `before(k)` runs on worker k's stream first."""
        torch, K = self.torch, self.K
        if n_streams <= 1:
            for k in range(K):
                if before is not None:
                    before(k)
                self.lqp(k, None, 0)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        for st in self.side[:n_streams]:
            st.wait_event(fork)
        for k in range(K):
            st = self.side[k % n_streams]
            with torch.cuda.stream(st):
                if before is not None:
                    before(k)
                self.lqp(k, st, k % n_streams)
        for st in self.side[:n_streams]:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    def check_status(self):
        bad = [int(st.bitwise_and(16 | 8).count_nonzero().item()) for st in self.status]
        if any(bad):
            raise SystemExit(f"solver reported unresolved tensors: {bad}")


def run_ours(args):
    # the oracle's worker processes are started before the first CUDA call
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    pool = OraclePool() if (rank == 0 and world == 1 and not args.no_cpu) else None

    import torch

    import paper_2002_11082_b200 as ogq
    from paper_2002_11082_b200.sharding import aggregate_throughput, max_over_ranks

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    K = args.workers
    n_streams = max(1, min(args.streams, K))
    peak, peak_src = measured_peaks()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, reps, need_flush):
        """Device time of `reps` calls of fn (CUDA events on the current stream, max over ranks).
        Small workloads: a buffer larger than L2 is overwritten before every call, outside the events."""
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

    S = Setup(torch, ogq, dev, args.workload, args.scheme, K, args.seed, rank, args.bucket_len, dense=args.dense)
    N, T, bits, s = S.N, S.T, S.code_bits, S.s
    # L2 hygiene: the large buckets cycle through far more than the 126 MB L2 per step
    need_flush = 4 * N * K <= 2 * 126e6

    def step():
        S.lqp_all(n_streams)
        S.unpack()

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    S.check_status()

    # ---- the timed region: exactly `steps` steps
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ogq.ogq_launch_count()
    ms_total = timed(step, steps, need_flush)
    launches = ogq.ogq_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_step = ms_total / steps
    value = aggregate_throughput(S.grad_bytes, ms_step, world)

    def stage_block(setup, streams, reps, flush):
        ms = timed(lambda: setup.lqp_all(streams), reps, flush) / reps
        gbs = setup.alg_lqp / (ms * 1e-3) / 1e9
        return {"streams": streams, "ms": ms, "grad_gbs": setup.grad_bytes / (ms * 1e-3) / 1e9,
                "alg_bytes_per_elem": 8.0 + setup.code_bits / 8.0, "frac_of_hbm_peak": gbs / peak,
                "frac_of_nominal_8tbs": gbs / 8000.0}

    # ---- per-stage and per-kernel times (separate instrumented passes, not part of `value`)
    st_multi = stage_block(S, n_streams, steps, need_flush)
    st_single = stage_block(S, 1, steps, need_flush)
    ms_unp = timed(S.unpack, steps, need_flush) / steps
    ogq.ogq_profile_enable(True)  # per-kernel times: one stream, so that no two kernels overlap
    torch.cuda.synchronize()
    for _ in range(steps):
        S.lqp_all(1)
        S.unpack()
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
        "k_unpack_sum": (K * bits / 8.0 + 4.0) * N, "k_bucket_encode": (4.0 + bits / 8.0) * N,
        "k_bucket_decode_sum": (K * bits / 8.0 + 4.0) * N,
        "k_quantize_pack_dense": (4.0 + bits / 8.0) * N, "k_unpack_sum_dense": (K * bits / 8.0 + 4.0) * N,
    }
    kernels = {}
    total_ms = max(sum(v[0] for v in per_kernel.values()), 1e-12)
    for name, (tot, cnt) in per_kernel.items():
        avg = tot / cnt
        gbs = alg_bytes.get(name, 0.0) / (avg * 1e-3) / 1e9 if avg > 0 else 0.0
        kernels[name] = {"launches_per_step": cnt / steps, "avg_ms": avg, "share": tot / total_ms, "alg_gbs": gbs}
    dom = max(per_kernel, key=lambda k: per_kernel[k][0])
    per_elem = stored_traffic(dom, args.scheme if not args.bucket_len else f"{args.scheme}_d{args.bucket_len}")
    roofline = {
        "bound": "hbm", "kernel": dom, "achieved": kernels[dom]["alg_gbs"], "peak": peak, "unit": "GB/s",
        "frac": kernels[dom]["alg_gbs"] / peak, "traffic": per_elem * N if per_elem is not None else None,
        "peak_source": peak_src, "alg_bytes_per_launch": alg_bytes.get(dom, 0.0),
    }

    # ---- end to end through the C ABI with host buffers (H2D of every worker's bucket, D2H of the result)
    e2e = None
    if not args.no_e2e:
        pinned = [torch.from_numpy(h.values).pin_memory() for h in S.host]
        h_out = torch.empty(N, dtype=torch.float32).pin_memory()

        def e2e_step():
            S.lqp_all(n_streams, before=lambda k: S.grads[k].copy_(pinned[k], non_blocking=True))
            S.unpack()
            h_out.copy_(S.out, non_blocking=True)

        e2e_steps = min(steps, 5)
        e2e_step()
        ms_e2e = timed(e2e_step, e2e_steps, need_flush) / e2e_steps
        e2e = {"value": aggregate_throughput(S.grad_bytes, ms_e2e, world), "unit": UNIT,
               "h2d_bytes_per_step": int(4 * N * K), "d2h_bytes_per_step": int(4 * N),
               "ms_per_step": ms_e2e, "steps": e2e_steps}
        del pinned, h_out

    # ---- the other headline workloads and schemes, short runs (default configuration only)
    secondary = None
    if world == 1 and not args.no_secondary and args.workload == "vgg19" and args.scheme == "orq9" and not args.bucket_len:
        secondary = {}
        for wk, sch, blen in (("vgg19", "bingrad_b", 0), ("resnet50", "orq9", 0), ("resnet50", "orq3", 0),
                              ("resnet50", "bingrad_b", 0), ("resnet50", "orq9", 512)):
            X = Setup(torch, ogq, dev, wk, sch, K, args.seed, rank, blen, share=S)
            flush = 4 * X.N * K <= 2 * 126e6
            for _ in range(3):
                X.lqp_all(n_streams)
            torch.cuda.synchronize()
            X.check_status()
            key = f"{wk}_{sch}" + (f"_d{blen}" if blen else "")
            secondary[key] = {"streams_K": stage_block(X, n_streams, 5, flush), "single_stream": stage_block(X, 1, 5, flush)}
            del X
            torch.cuda.empty_cache()

    # ---- CPU oracle on a bounded sample, on all host cores (rank 0, single GPU runs only)
    cpu = None
    if pool is not None:
        tasks, used, what = pool.sample(args.workload, args.scheme, seconds=args.cpu_seconds)
        dt = pool.run(tasks)
        cpu = {"value": 4.0 * used / dt / 1e9, "unit": UNIT, "cores": pool.cores, "kind": "oracle", "sample": what,
               "seconds": dt}
        pool.close()

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": args.workload, "scheme": args.scheme, "levels": s, "bits": bits,
                       "workers_per_gpu": K, "tensors": T, "elements": N, "streams": n_streams,
                       "bucket_len": args.bucket_len or None, "packing": "base-s words" if S.dense else "bit stream",
                       "l2": "256 MB written between timed steps (flush)" if need_flush else "inputs larger than L2 (no flush)"},
            "stages": {
                "levels_quantize_pack": st_multi,
                "unpack_sum": {"ms": ms_unp, "alg_gbs": (K * bits / 8.0 + 4.0) * N / (ms_unp * 1e-3) / 1e9},
            },
            "single_stream": st_single, "secondary": secondary,
            "kernels": kernels, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e,
            "gpu_launches": int(launches), "clocks": clocks,
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_dp(args):
    """Data parallelism as in Algorithm 2: every rank is one worker.  A step = levels + quantize + pack
    of the rank's own bucket, all-gather of the packed codes and level tables (NCCL) into the rank's own
    memory, unpack + dequantize + sum over all workers from there."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    import torch

    import paper_2002_11082_b200 as ogq
    from paper_2002_11082_b200.sharding import CodeExchange, aggregate_throughput, max_over_ranks

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod
    peak, peak_src = measured_peaks()
    S = Setup(torch, ogq, dev, args.workload, args.scheme, 1, args.seed, rank)  # worker id = rank
    ex = CodeExchange(world, int(S.h_po[-1]), S.T, S.s, device=dev)
    pk_rows, lv_rows = ex.pointer_rows()
    pk_ptrs = torch.tensor(pk_rows, dtype=torch.int64, device=dev)
    lv_ptrs = torch.tensor(lv_rows, dtype=torch.int64, device=dev)

    def step():
        S.lqp(0, None, 0)
        ex.gather(dist, S.packed[0], S.levels[0])
        ogq.ogq_unpack_sum(pk_ptrs, lv_ptrs, world, S.off, S.po, S.T, S.N, S.s, 1.0 / world, S.out)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    for _ in range(warmup):
        step()
    barrier()
    S.check_status()
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    need_flush = 4 * S.N <= 2 * 126e6
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = ogq.ogq_launch_count()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0.0
    for _ in range(steps):
        if need_flush:
            flush_buf.fill_(1)
        barrier()
        a.record()
        step()
        b.record()
        torch.cuda.synchronize()
        total += a.elapsed_time(b)
    ms_step = max_over_ranks(total / steps, dist, dev)
    launches = ogq.ogq_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        line = {
            "metric": METRIC, "value": aggregate_throughput(4.0 * S.N, ms_step, world), "unit": UNIT, "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "mode": "dp",
            "config": {"workload": args.workload, "scheme": args.scheme, "levels": S.s, "bits": S.bits,
                       "workers": world, "tensors": S.T, "elements": S.N,
                       "exchange": "all-gather of packed codes and level tables, then local unpack+sum",
                       "recv_bytes_per_rank_and_step": ex.recv_bytes},
            "gpu_launches": int(launches), "clocks": clocks, "peak_source": peak_src,
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
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-secondary", action="store_true")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "dp"],
                    help="replicas: K simulated workers per GPU (default); dp: one worker per rank, codes all-gathered")
    ap.add_argument("--dense", action="store_true", help="ORQ codes in the base-s (entropy-dense) wire format")
    ap.add_argument("--bucket-len", type=int, default=0,
                    help="fixed-length bucket mode: quantize buckets of this many elements (ogq_bucket_encode)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "dp":
        run_dp(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

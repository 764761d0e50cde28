#!/usr/bin/env python
"""Benchmark of the CSER / M-CSER optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

One "step" = one pass of the whole hot path (GRBS block select + streaming kernel +
selected-block kernel) over one [n, d] batch of synthetic gradients.  The headline
workload is the largest single-GPU configuration, the BERT-large-sized one
(d = 335,141,888, n = 8, R1 = R2 = 64, H = 8, beta = 0.9: 43 GB of g/x/e/m); the other
four configurations are timed briefly in the same run and reported under "per_config".
Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank owns one column slab
of that size with global block ids and no data is exchanged ("weak" scaling); the
worker-sharded step (one all-reduce of the packed selected blocks per iteration) is
timed beside it and reported under "worker_sharded".
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "cser_steps_per_sec"
UNIT = "steps/s"
PEAK_NOMINAL_GBS = 8000.0

# dram__bytes_read.sum + dram__bytes_write.sum per step of the streaming kernel plus the selected-block
# kernel, from ncu captures of the same workloads cut to d = 8,388,608 and scaled by d (every byte is
# touched once, so traffic is proportional to d).
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"cfg2_wrn40x8_n8_R32_H8": 1.7983e9 * 35_748_708 / 8_388_608,
                                "cfg5_bertlarge_n8_R64_H8": 1.8013e9 * 335_141_888 / 8_388_608}
HEADLINE_CONFIG = 5


NO_ERROR_ARRAY = False   # --impl2: implementation II of Appendix A.4 (no e array)
EXACT_COUNT = False      # --exact-count: every mask selects exactly round(B/R) blocks
L2_RESIDENT = False      # ask the library to keep a small state in L2 (CSER_FLAG_L2_RESIDENT)
THREE_KERNELS = False    # --three-kernels: never the single-launch kernel for small problems (CSER_FLAG_THREE_KERNELS)
STAGED = False           # --staged: selected blocks through the shared-memory staged kernel (CSER_FLAG_STAGED_SELECTED)


def algorithmic_bytes(w, frac_e_touched):
    """Bytes one step must move: g read; x, (m) read+write; e read+write where touched."""
    per = 4 + 8 + (8 if w.beta != 0 else 0) + (0 if NO_ERROR_ARRAY else 8 * frac_e_touched)
    return w.n_workers * w.d * per


def expected_e_fraction(w, is_reset):
    sel = 1.0 / w.R1 if w.R1 else 0.0
    f = 1.0 - sel
    if is_reset:
        f = 1.0 - sel * (1.0 - 1.0 / w.R2)
    return f


def mean_algorithmic_bytes(w, t_first, k):
    tot = 0.0
    for t in range(t_first, t_first + k):
        tot += algorithmic_bytes(w, expected_e_fraction(w, t % w.H == 0))
    return tot / k


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, device_index):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv, self.h = pynvml, pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as ex:  # NVML not reachable: report that instead of numbers
            self.nv, self.err = None, repr(ex)

    def _poll(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self.nv:
            self._thr = threading.Thread(target=self._poll, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        if not self.nv:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable: " + self.err]}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


ORACLE_SAMPLE_ELEM_WORKERS = 1 << 25      # about 2.5 s of oracle time per step on one host core


def oracle_sample_cols(w):
    """Columns of the contiguous slab of whole blocks the oracle is timed on: the whole vector when it is
    small (workload 1 runs real full-d steps), else 2^25 element-workers' worth of it: float64 [n, cols]
    arrays of 268 MB each, far larger than the host's caches, and a few seconds of oracle time per step."""
    if w.n_workers * w.d <= ORACLE_SAMPLE_ELEM_WORKERS:
        return w.d
    return max(w.block_size, ORACLE_SAMPLE_ELEM_WORKERS // w.n_workers // w.block_size * w.block_size)


class OracleSample:
    """The CPU oracle, as it stands, on the first `cols` columns of workload w (columns are independent
    given the masks, and the masks are those of the whole vector)."""

    def __init__(self, w, cols, n_grads=3):
        import numpy as np
        from oracle import CSEROracle
        from paper_2007_13221_b200 import synth
        self.w, self.cols = w, cols
        ws = w.scaled(cols)
        self.ref = CSEROracle(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                              dtype=np.float64, cols=np.arange(cols))
        self.ref.set_x0(synth.x0(ws, "cpu").numpy())
        self.grads = [synth.gradients(ws, t, "cpu").numpy() for t in range(1, n_grads + 1)]
        self.k = 0

    def step(self):
        """One oracle step; returns its wall time in seconds."""
        t0 = time.perf_counter()
        self.ref.step(self.grads[self.k % len(self.grads)])
        self.k += 1
        return time.perf_counter() - t0


def oracle_sample_rate(w, target_seconds=15.0):
    """Time the oracle on a bounded sample of workload w.  Returns a dict: measured slab, wall time,
    steps, and the rate scaled to the full vector (work is proportional to the columns)."""
    cols = oracle_sample_cols(w)
    smp = OracleSample(w, cols)
    smp.step()                                            # warm-up (page faults, imports)
    walls = []
    while sum(walls) < target_seconds and len(walls) < 400:
        walls.append(smp.step())
    wall = sum(walls)
    rate_slab = len(walls) / wall
    return {"value": rate_slab * (cols / w.d), "unit": UNIT, "cores": 1, "kind": "oracle",
            "extrapolated": cols != w.d, "measured_cols": cols, "measured_steps": len(walls),
            "measured_wall_s": wall, "measured_steps_per_s_on_slab": rate_slab,
            "sample": (f"{len(walls)} steps of the float64 NumPy oracle on the first {cols} of {w.d} columns x "
                       f"{w.n_workers} workers of {w.name} ({8 * w.n_workers * cols / 1e6:.0f} MB per float64 array)"
                       + ("" if cols == w.d else f"; rate scaled by {cols}/{w.d} to the full vector"))}


ALL_CORES_SLAB_COLS = 1 << 20     # per process: 67 MB per float64 [8, cols] array, beyond any cache level


def all_cores_slab_cols(w, cores):
    cols = min(ALL_CORES_SLAB_COLS, max(w.block_size, w.d // cores))
    return max(w.block_size, cols // w.block_size * w.block_size)


def oracle_all_cores(w, seconds=10.0):
    """The same oracle with the columns split over all host cores: one process per core, each timing its
    own slab of whole blocks at the same moment.  Returns a dict like oracle_sample_rate's."""
    import subprocess
    cores = min(os.cpu_count() or 1, 32)       # one Python process per core; keep the memory bounded
    procs = [subprocess.Popen([sys.executable, os.path.abspath(__file__), "--config", str(w_index(w)),
                               "--oracle-slab", str(k), "--oracle-cores", str(cores),
                               "--oracle-seconds", str(seconds)] +
                              (["--d", str(w.d)] if w.d != base_config(w).d else []),
                              stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True,
                              env={**os.environ, "OMP_NUM_THREADS": "1", "MKL_NUM_THREADS": "1",
                                   "CUDA_VISIBLE_DEVICES": ""})
             for k in range(cores)]
    total, ok = 0.0, 0
    for p in procs:
        out, _ = p.communicate(timeout=600)
        try:
            total += float(json.loads(out.strip().splitlines()[-1])["rate"])
            ok += 1
        except Exception:
            pass
    cols = all_cores_slab_cols(w, cores)
    return {"value": total, "unit": UNIT, "cores": ok, "extrapolated": True, "measured_cols": cols * ok,
            "sample": (f"{ok} processes, one per core, each stepping the float64 NumPy oracle on its own {cols}-column "
                       f"slab of {w.name} for {seconds:.0f} s at the same time; rates (scaled to the full vector) added")}


def base_config(w):
    from paper_2007_13221_b200 import synth
    return synth.CONFIGS[w_index(w)]


def w_index(w):
    from paper_2007_13221_b200 import synth
    for k, c in synth.CONFIGS.items():
        if w.name.startswith(c.name):
            return k
    raise ValueError(w.name)


def oracle_slab_worker(w, slab, cores, seconds):
    """Child of oracle_all_cores: times the oracle on its own slab of whole blocks."""
    import numpy as np
    from oracle import CSEROracle
    from paper_2007_13221_b200 import synth
    width = all_cores_slab_cols(w, cores)
    c0 = min(slab * width, max(0, (w.d - width) // w.block_size * w.block_size))
    cols = np.arange(c0, min(c0 + width, w.d))
    ws = w.scaled(cols.size)
    ref = CSEROracle(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                     dtype=np.float64, cols=cols)
    ref.set_x0(synth.x0(ws, "cpu").numpy())
    grads = [synth.gradients(ws, t, "cpu").numpy() for t in range(1, 4)]
    ref.step(grads[0])
    n_steps, t0 = 0, time.perf_counter()
    while time.perf_counter() - t0 < seconds:
        ref.step(grads[n_steps % 3])
        n_steps += 1
    el = time.perf_counter() - t0
    print(json.dumps({"rate": n_steps / el * (cols.size / w.d)}))


def config_of(w, world):
    """The `config` object of the JSON line: the same in both arms (it depends on the workload only)."""
    per = 12 + (8 if w.beta != 0 else 0) + 8
    return {"workload": w.name, "d": w.d, "n_workers": w.n_workers, "block_size": w.block_size,
            "R1": w.R1, "R2": w.R2, "H": w.H, "eta": w.eta, "beta": w.beta,
            "parallelism": f"column slabs x{world}, no collective",
            "l2": f"inputs larger than L2: about {w.n_workers * w.d * per / 1e9:.2f} GB touched per step, "
                  "gradient buffers cycled"}


def run_reference(args, w):
    """--impl reference: the oracle, timed on the host cores, same metric and workload.  Each timed
    step is one oracle step on a bounded slab (the whole vector for workload 1); `ms_per_step` is the
    wall time of that measured step and `value` its rate scaled to the full vector."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cols = oracle_sample_cols(w)
    smp = OracleSample(w, cols)
    t_all0 = time.perf_counter()
    walls = []
    for k in range(args.warmup + args.steps):
        dt = smp.step()
        if k >= args.warmup:
            walls.append(dt)
        if time.perf_counter() - t_all0 > 170 and walls:
            break
    wall = sum(walls)
    rate_slab = len(walls) / wall
    value = rate_slab * (cols / w.d)
    sample = (f"each timed step = one step of the float64 NumPy oracle on the first {cols} of {w.d} columns x "
              f"{w.n_workers} workers ({8 * w.n_workers * cols / 1e6:.0f} MB per float64 array)"
              + ("" if cols == w.d else f"; value = measured rate x {cols}/{w.d}"))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(walls), "warmup": args.warmup, "ms_per_step": 1e3 * wall / len(walls),
        "ms_per_step_is": "wall time of one measured oracle step on the slab" if cols != w.d else "wall time of one oracle step",
        "extrapolated": cols != w.d, "measured_cols": cols, "measured_wall_s": wall,
        "measured_steps_per_s_on_slab": rate_slab, "full_vector_ms_per_step_estimate": 1e3 / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, max(1, args.gpus)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_workload(w, K, W, dev, rank, world, ring_n=0, with_e2e=True, flush_l2=False):
    """Time K steps of workload w on this rank's slab; returns the measured pieces."""
    import torch
    import torch.distributed as dist
    from paper_2007_13221_b200 import binding as b, synth

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            tt = torch.tensor([ms], device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            return float(tt.item())
        return ms

    # each rank owns one slab of the workload's size, with global block ids
    opt = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                 block_begin=0 if EXACT_COUNT else rank * w.n_blocks,
                 flags=(b.FLAG_NO_ERROR_ARRAY if NO_ERROR_ARRAY else 0) | (b.FLAG_EXACT_COUNT if EXACT_COUNT else 0)
                 | (b.FLAG_L2_RESIDENT if L2_RESIDENT else 0) | (b.FLAG_STAGED_SELECTED if STAGED else 0) | (b.FLAG_THREE_KERNELS if THREE_KERNELS else 0))
    opt.set_x0(synth.x0(w, dev))
    g_bytes = w.n_workers * w.d * 4
    ring_n = ring_n or max(2, min(4, int(6e9 // g_bytes)))
    ring = [synth.gradients(w, 1 + k, dev) for k in range(ring_n)]
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    for k in range(W):
        opt.step(ring[k % ring_n])
    barrier()
    launches0 = b.cser_launch_count(opt.h)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_first = opt.t + 1
    with ClockSampler(torch.cuda.current_device()) as clocks:
        ev0.record(stream)
        for k in range(K):
            opt.step(ring[k % ring_n])
        ev1.record(stream)
        barrier()
    total_ms = max_over_ranks(ev0.elapsed_time(ev1))
    out = {"launches": b.cser_launch_count(opt.h) - launches0, "ms_per_step": total_ms / K,
           "value": world * K / (total_ms * 1e-3), "alg_bytes": mean_algorithmic_bytes(w, t_first, K),
           "clocks": clocks.summary(), "ring_n": ring_n, "g_bytes": g_bytes}

    # per-kernel durations (CUDA events the library records on the launching stream): the
    # select kernel, then the streaming kernel with the selected-block kernel beside it
    b.cser_set_timing(opt.h, True)
    k_ms, k_bytes, mask_ms, k_reset = [], [], [], []
    n_prof = min(K, 4 * w.H if w.H > 1 else 16)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if flush_l2 else None
    for k in range(n_prof):
        if flush is not None:
            flush.fill_(k & 0xFF)                     # evict the 126 MB L2 between timed steps
        opt.step(ring[k % ring_n])
        a_ms, s_ms = b.cser_last_kernel_ms(opt.h)
        mask_ms.append(a_ms), k_ms.append(s_ms)
        k_bytes.append(algorithmic_bytes(w, expected_e_fraction(w, opt.t % w.H == 0)))
        k_reset.append(opt.t % w.H == 0)
    b.cser_set_timing(opt.h, False)

    def stats(sel):
        v = sorted(ms for ms, r in zip(k_ms, k_reset) if r == sel)
        by = [bb for bb, r in zip(k_bytes, k_reset) if r == sel]
        if not v:
            return None
        return {"launches": len(v), "ms_mean": sum(v) / len(v), "ms_median": v[len(v) // 2], "ms_min": v[0],
                "gbs_mean": sum(by) / (sum(v) * 1e-3) / 1e9}
    peak, peak_src = measured_peaks()
    achieved = sum(k_bytes) / (sum(k_ms) * 1e-3) / 1e9
    out["roofline"] = {
        "bound": "hbm", "kernel": "cser_stream_kernel (cser_selected_kernel runs beside it)",
        "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_source": peak_src, "frac_of_nominal_8TBs": achieved / PEAK_NOMINAL_GBS,
        "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(w.name),
        "algorithmic_bytes_per_launch": sum(k_bytes) / len(k_bytes),
        "kernel_ms_avg": sum(k_ms) / len(k_ms), "select_kernel_ms_avg": sum(mask_ms) / len(mask_ms),
        "launches_timed": len(k_ms), "l2_flushed_between_launches": bool(flush_l2),
        "plain_steps": stats(False), "reset_steps": stats(True),
    }
    del flush

    # end to end: gradients start in pinned host memory every step; a result is read back
    out["e2e"] = None
    if with_e2e:
        # two pinned host buffers, alternated; one when a buffer is several GB (every rank pins its own)
        host_ring = [torch.empty((w.n_workers, w.d), dtype=torch.float32).pin_memory()
                     for _ in range(1 if g_bytes > 4e9 else 2)]
        for hb, gb in zip(host_ring, ring):
            hb.copy_(gb)
        if len(host_ring) == 1:
            host_ring.append(host_ring[0])
        mask_host = torch.empty(w.n_blocks, dtype=torch.uint8).pin_memory()
        ke = max(3, min(K, 12))
        for k in range(2):
            opt.step_host(host_ring[k % 2])
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for k in range(ke):
            opt.step_host(host_ring[k % 2])
            b.cser_read_state(opt.h, b.STATE_MASK_G, mask_host)
            stream.synchronize()                      # the caller consumes the result every step
            _ = opt.t
        e1.record(stream)
        barrier()
        e_ms = max_over_ranks(e0.elapsed_time(e1))
        out["e2e"] = {"value": world * ke / (e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": g_bytes,
                      "d2h_bytes_per_step": w.n_blocks + 8, "steps": ke,
                      "note": "cser_step_host from pinned host gradients + read-back of the step's mask and t"}
        del host_ring
    opt.close()
    del ring
    torch.cuda.empty_cache()
    return out


def run_worker_sharded(w, K, W, dev, group, world, rank):
    """The worker-sharded step: this rank holds n / world of the workload's workers (all d columns), packs
    the sum over them of the selected blocks, the message is all-reduced over the ranks (NCCL, through
    torch.distributed; nothing to reduce when world == 1) and applied.  Timed on the device, max over ranks."""
    import torch
    import torch.distributed as dist
    from paper_2007_13221_b200 import binding as b, synth
    from paper_2007_13221_b200.shard import workers_of_rank
    first, n_local = workers_of_rank(w.n_workers, rank, world)
    opt = b.WorkerShardedCSER(w.d, n_local, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                              group=group)
    opt.set_x0(synth.x0(w, dev))
    wl = w if world == 1 else __import__("dataclasses").replace(w, n_workers=n_local, seed=w.seed + 1000 * rank)
    ring = [synth.gradients(wl, 1 + k, dev) for k in range(3)]
    for k in range(W):
        opt.step(ring[k % 3])
    if world > 1:
        dist.barrier(group=group)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for k in range(K):
        opt.step(ring[k % 3])
    ev1.record()
    if world > 1:
        dist.barrier(group=group)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / K
    if world > 1:
        tt = torch.tensor([ms], device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX, group=group)
        ms = float(tt.item())
    out = {"workload": w.name, "ranks": world, "workers_per_rank": n_local,
           "steps_per_s": 1e3 / ms, "ms_per_step": ms, "steps": K, "scaling": "strong",
           "collective": "none (one rank)" if world == 1 else "NCCL all-reduce (sum) of the packed message, fp32",
           "message_bytes_plain_step": 4 * b.cser_wshard_message_elems(opt.h, False),
           "message_bytes_reset_step": 4 * b.cser_wshard_message_elems(opt.h, True)}
    opt.close()
    del ring
    torch.cuda.empty_cache()
    return out


def run_graph_replay(w, K, dev, steps_per_graph=1):
    """`steps_per_graph` replayable steps captured in one CUDA graph (torch is the plumbing for the capture),
    replayed K / steps_per_graph times: every replay is that many more iterations."""
    import torch
    from paper_2007_13221_b200 import binding as b, synth
    opt = b.CSER(w.d, w.n_workers, w.block_size, w.R1, w.R2, w.H, w.eta, w.beta, w.seed,
                 flags=b.FLAG_THREE_KERNELS if THREE_KERNELS else 0)
    opt.set_x0(synth.x0(w, dev))
    g = synth.gradients(w, 1, dev)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b.cser_replay_begin(opt.h)
        for _ in range(3):
            b.cser_step_replayable(opt.h, g)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
        for _ in range(steps_per_graph):
            b.cser_step_replayable(opt.h, g)
    for _ in range(5):
        graph.replay()
    torch.cuda.synchronize()
    n_replays = max(1, K // steps_per_graph)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(n_replays):
        graph.replay()
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / (n_replays * steps_per_graph)
    t_end = opt.t
    b.cser_replay_end(opt.h)
    alg = mean_algorithmic_bytes(w, 1, w.H)
    out = {"steps_per_s": 1e3 / ms, "ms_per_step": ms, "steps": n_replays * steps_per_graph,
           "steps_per_graph": steps_per_graph, "iterations_done": t_end,
           "hbm_gbs_step": alg / (ms * 1e-3) / 1e9, "hbm_frac_of_8TBs": alg / (ms * 1e-3) / 1e9 / PEAK_NOMINAL_GBS}
    opt.close()
    del g, graph
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--config", type=int, default=0,
                    help="workload 1..5 (default: 5, the largest; 2 if the GPU has too little free memory)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--ring", type=int, default=0, help="distinct gradient buffers cycled through")
    ap.add_argument("--d", type=int, default=0, help="override the vector length (small profiling cases)")
    ap.add_argument("--impl2", action="store_true", help="implementation II (no error array) as the main run")
    ap.add_argument("--exact-count", action="store_true", help="exact-count GRBS masks as the main run")
    ap.add_argument("--R1", type=int, default=-1, help="override the update compressor's ratio")
    ap.add_argument("--R2", type=int, default=-1, help="override the reset compressor's ratio")
    ap.add_argument("--H", type=int, default=-1, help="override the reset interval")
    ap.add_argument("--three-kernels", action="store_true",
                    help="small problems through the three-kernel step instead of the single-launch kernel")
    ap.add_argument("--staged", action="store_true",
                    help="selected blocks through the shared-memory staged kernel instead of the register-walking one")
    ap.add_argument("--flush-l2", action="store_true", help="per-kernel figures with L2 flushed between launches")
    ap.add_argument("--ceilings", action="store_true",
                    help="measure the bandwidth ceilings and traversal / staging alternatives with the probe library")
    ap.add_argument("--oracle-slab", type=int, default=-1, help=argparse.SUPPRESS)
    ap.add_argument("--oracle-seconds", type=float, default=10.0, help=argparse.SUPPRESS)
    ap.add_argument("--oracle-cores", type=int, default=1, help=argparse.SUPPRESS)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    global NO_ERROR_ARRAY, EXACT_COUNT, STAGED, THREE_KERNELS
    NO_ERROR_ARRAY = bool(args.impl2)
    EXACT_COUNT = bool(args.exact_count)
    STAGED = bool(args.staged)
    THREE_KERNELS = bool(args.three_kernels)

    from paper_2007_13221_b200 import synth
    default_run = args.config == 0 and not args.d and args.R1 < 0 and args.R2 < 0 and args.H < 0
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    gpu_arm = args.impl == "ours" and args.oracle_slab < 0 and not args.ceilings
    if gpu_arm:
        import torch
        import torch.distributed as dist
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
        torch.cuda.set_device(local)
        if world > 1:
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    if args.config == 0:
        args.config = HEADLINE_CONFIG
        if gpu_arm:
            # the largest workload needs 53 GB per GPU; every rank must make the same choice
            need = synth.CONFIGS[HEADLINE_CONFIG].n_workers * synth.CONFIGS[HEADLINE_CONFIG].d * 4 * 5.3
            fits = torch.tensor([1 if torch.cuda.mem_get_info()[0] >= need else 0], device=f"cuda:{local}")
            if world > 1:
                dist.all_reduce(fits, op=dist.ReduceOp.MIN)
            if int(fits.item()) == 0:
                args.config = 2
    w = synth.CONFIGS[args.config]
    if args.d:
        w = w.scaled(args.d)
    if args.R1 >= 0 or args.R2 >= 0 or args.H >= 0:
        from dataclasses import replace
        w = replace(w, R1=args.R1 if args.R1 >= 0 else w.R1, R2=args.R2 if args.R2 >= 0 else w.R2,
                    H=args.H if args.H >= 0 else w.H)
        w = replace(w, name=f"{w.name}@R1={w.R1},R2={w.R2},H={w.H}")
    if args.oracle_slab >= 0:
        oracle_slab_worker(w, args.oracle_slab, args.oracle_cores, args.oracle_seconds)
        return
    if args.impl == "reference":
        run_reference(args, w)
        return
    if args.ceilings:
        run_ceilings(args)
        return

    dev = f"cuda:{local}"
    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if world > 1:
        dist.barrier()

    K, W = args.steps, args.warmup
    big = w.n_workers * w.d * 4 > 8e9           # one [n, d] array above 8 GB: two gradient buffers, one host buffer
    r = run_workload(w, K, W, dev, rank, world, ring_n=args.ring or (2 if big else 0), with_e2e=not args.no_e2e,
                     flush_l2=args.flush_l2)
    alg_bytes = r["alg_bytes"]

    def brief(ro, steps):
        """A few numbers per extra run, so that the whole line stays short."""
        gbs = ro["alg_bytes"] / (ro["ms_per_step"] * 1e-3) / 1e9
        rf = ro["roofline"]
        out = {"steps_per_s": round(ro["value"], 2), "ms_per_step": round(ro["ms_per_step"], 5), "steps": steps,
               "hbm_gbs_step": round(gbs, 1), "frac_of_8TBs": round(gbs / PEAK_NOMINAL_GBS, 4),
               "roofline": {"bound": "hbm", "achieved": round(rf["achieved"], 1), "peak": rf["peak"], "unit": "GB/s",
                            "frac": round(rf["frac"], 4), "l2_flushed": rf["l2_flushed_between_launches"],
                            "traffic": rf["traffic"]},
               "plain_ms": rf["plain_steps"] and round(rf["plain_steps"]["ms_mean"], 5),
               "reset_ms": rf["reset_steps"] and round(rf["reset_steps"]["ms_mean"], 5),
               "sm_mhz": ro["clocks"]["sm_mhz"]}
        return out

    # the other workloads and variants, briefly (single GPU, default invocation only); a failure
    # here is recorded and never costs the headline line
    per_config = None
    if world == 1 and default_run and not args.no_others and not args.impl2 and not args.exact_count \
            and not args.staged and not args.three_kernels:
        per_config = {}

        def guarded(name, fn):
            try:
                per_config[name] = fn()
            except Exception as ex:  # noqa: BLE001
                per_config[name] = "failed: " + repr(ex)[:200]
            torch.cuda.empty_cache()

        def variant(wv, flag_name, steps=50):
            global NO_ERROR_ARRAY, EXACT_COUNT, THREE_KERNELS, L2_RESIDENT
            try:
                NO_ERROR_ARRAY, EXACT_COUNT = flag_name == "impl2", flag_name == "exact"
                THREE_KERNELS, L2_RESIDENT = flag_name == "three_kernels", flag_name == "l2"
                return brief(run_workload(wv, steps, 5, dev, rank, world, with_e2e=False,
                                          flush_l2=wv is synth.CONFIGS[1]), steps)
            finally:
                NO_ERROR_ARRAY = EXACT_COUNT = THREE_KERNELS = L2_RESIDENT = False

        def other_workload(wo):
            free, _ = torch.cuda.mem_get_info()
            if free < wo.n_workers * wo.d * 4 * 6.5:
                return "skipped: not enough free device memory"
            ko = 400 if wo is synth.CONFIGS[1] else 50
            # workload 1 (67 MB of state) fits the 126 MB L2: steps/s is back to back; the roofline figure
            # is taken with L2 flushed between launches
            return brief(run_workload(wo, ko, 5, dev, rank, world, with_e2e=False,
                                      flush_l2=wo is synth.CONFIGS[1]), ko)

        w2 = synth.CONFIGS[2]
        for c in (1, 2, 3, 4):
            if synth.CONFIGS[c] is not w:
                guarded(synth.CONFIGS[c].name, lambda c=c: other_workload(synth.CONFIGS[c]))
        guarded(w2.name + " implementation II (no error array)", lambda: variant(w2, "impl2"))
        guarded(w2.name + " exact-count GRBS", lambda: variant(w2, "exact"))
        guarded(synth.CONFIGS[1].name + " three kernels instead of one launch",
                lambda: variant(synth.CONFIGS[1], "three_kernels", 400))
        guarded(w2.name + " worker-sharded entry points, one rank holding all workers",
                lambda: run_worker_sharded(w2, 50, 5, dev, None, 1, 0))
        for R in (1, 2, 4, 8):                      # small ratios: a large share of the blocks is selected
            wr = replace_ratios(w2, R, R)
            guarded(wr.name, lambda wr=wr: other_workload(wr))
        for rc, wt in synth.PAPER_TUNED.items():     # the paper's tuned (R_C2, R_C1, H) per overall ratio
            guarded(wt.name, lambda wt=wt: other_workload(wt))
        guarded(w2.name + " step captured in a CUDA graph and replayed", lambda: run_graph_replay(w2, 100, dev))
        guarded(synth.CONFIGS[1].name + " 16 steps captured in one CUDA graph and replayed (one kernel per step)",
                lambda: run_graph_replay(synth.CONFIGS[1], 4000, dev, steps_per_graph=16))

    # worker-sharded deployment (the paper's own setting): the workload's n workers split over the ranks,
    # one NCCL all-reduce of the packed selected blocks per step.  The column-slab number above stays the
    # headline; this entry is there so that a multi-GPU run measures both shardings.
    wshard = None
    if world > 1 and not args.no_others:
        try:
            ws_w = synth.CONFIGS[2]
            if ws_w.n_workers % world == 0:
                wshard = run_worker_sharded(ws_w, min(K, 50), 5, dev, dist.group.WORLD, world, rank)
            else:
                wshard = f"skipped: {ws_w.n_workers} workers do not split evenly over {world} ranks"
        except Exception as ex:  # noqa: BLE001
            wshard = "failed: " + repr(ex)[:200]

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = oracle_sample_rate(w)
        cpu["all_cores"] = oracle_all_cores(w)

    if rank == 0:
        cfg = config_of(w, world)
        if args.impl2 or args.exact_count:
            cfg["workload"] += (" implementation II" if args.impl2 else "") + (" exact-count GRBS" if args.exact_count else "")
        line = {
            "per_config": per_config, "worker_sharded": wshard,
            "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": r["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": cfg,
            "workload_notes": {"overall_compression_ratio": w.overall_ratio,
                               "deployment_bytes_per_worker_step": w.comm_bytes_per_worker_step,
                               "gradient_buffers_cycled": r["ring_n"]},
            "hbm_gbs_step": alg_bytes / (r["ms_per_step"] * 1e-3) / 1e9,
            "hbm_frac_of_8TBs": alg_bytes / (r["ms_per_step"] * 1e-3) / 1e9 / PEAK_NOMINAL_GBS,
            "algorithmic_bytes_per_step": alg_bytes,
            "roofline": r["roofline"], "cpu_baseline": cpu, "e2e": r["e2e"],
            "gpu_launches": r["launches"], "clocks": r["clocks"], "library": __graft_entry__.library_record(),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_ceilings(args):
    """--ceilings: what bounds the step kernels, re-measured with the probe library (plain kernels moving
    the bytes of one M-CSER step over the WRN-40-8-sized arrays in different orders and through different
    paths; see csrc/membw_probe.cu).  Prints one JSON object."""
    import ctypes
    import torch
    import __graft_entry__
    from paper_2007_13221_b200 import synth
    __graft_entry__.build()
    L = ctypes.CDLL(os.path.join(ROOT, "paper_2007_13221_b200", "libcser_probe.so"))
    L.cser_probe_run.argtypes = [ctypes.c_int, ctypes.c_int] + [ctypes.c_void_p] * 4 + \
        [ctypes.c_longlong, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_float), ctypes.c_void_p]
    w = synth.CONFIGS[2] if not args.d else synth.CONFIGS[2].scaled(args.d)
    n, d = w.n_workers, w.d
    torch.cuda.set_device(0)
    arrs = [torch.randn((n, d), device="cuda:0") * 0.01 for _ in range(4)]
    elems = n * d
    cases = [("read g, m, x, e (rows)", 0, 0, 16), ("write m, x, e (rows)", 1, 0, 12), ("copy g -> x (rows)", 2, 0, 8),
             ("step mix 4 read + 3 written, row after row, plain 128-bit accesses", 3, 0, 28)]
    cases += [(f"step mix, thread per column walking all workers, {u} workers in flight", 4, u, 28) for u in (1, 2, 4, 8)]
    cases += [(f"step mix, row after row, bulk copies into shared memory, {kb} KB tiles", 5, kb, 28) for kb in (2, 4, 8)]
    out = {"workload_shape": f"{n} x {d} fp32 per array ({elems * 4 / 1e9:.2f} GB)", "reps": args.steps, "patterns": []}
    with ClockSampler(0) as clocks:
        for name, pattern, variant, bytes_per in cases:
            ms = ctypes.c_float()
            rc = L.cser_probe_run(pattern, variant, *[a.data_ptr() for a in arrs], d, n, args.steps, ctypes.byref(ms), None)
            out["patterns"].append({"pattern": name, "ms": round(ms.value, 4) if rc == 0 else None,
                                    "GB_per_s": round(elems * bytes_per / (ms.value * 1e-3) / 1e9, 1) if rc == 0 else None,
                                    "rc": rc})
    out["clocks"] = clocks.summary()
    print(json.dumps(out))


def replace_ratios(w, R1, R2):
    from dataclasses import replace
    return replace(w, R1=R1, R2=R2, name=f"{w.name}@R1={R1},R2={R2}")


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the C-Coll hot path on B200.

A step = one pass of the whole hot path over one batch: the 512x512x256 smooth field with 20 % constant
blocks (67,108,864 fp32 values, error bound 1e-4 x range) goes through all five entry points of the C ABI:
  1. ccoll_compress            the field
  2. ccoll_decompress          the stream from 1
  3. ccoll_reduce_step         stream from 1 + a second seeded field as the local chunk (with sum_out)
  4. ccoll_allreduce_sim       the field viewed as P = 8 virtual ranks of n/8 values
  5. ccoll_bcast_sim (scatter) the field scattered to P = 8 virtual ranks
`value` = fp32 bytes presented to the entry points (5 x 4n per step, all ranks) / time, inputs resident in
HBM.  `e2e` = the same with the inputs coming from pinned host memory and the results read back, inside the
timed region.  Multi-GPU runs are independent replicas (the path has no exchange step): weak scaling.

`--impl reference` times the CPU oracle (test infrastructure, single thread) on a bounded sample instead.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD = "C2: 512x512x256 fp32 smooth Gaussian field (sigma 8), 20% constant blocks, eb=1e-4*range, block_len 128"
SHAPE = (512, 512, 256)
SIGMA = 8.0
P_SIM = 8
METRIC = "compress / decompress / fused reduce-step GB/s (fp32 input) and % of B200 HBM peak"
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from one ncu capture of each kernel on the
# 256x512x256 field of the same recipe (33,554,432 values; profiles/kernels_256x512x256.md),
# expressed per value: DRAM traffic grows in proportion to the values processed, so a full-size launch is
# this figure times its value count.  (Writes that are still in L2 when the kernel ends are not in it.)
NCU_DRAM_BYTES_PER_VALUE = {
    "ccoll_compress_kernel": (134.30e6 + 7.25e6) / 33554432,
    "ccoll_decode_kernel": (58.74e6 + 79.48e6) / 33554432,
    "ccoll_reduce_kernel": (193.68e6 + 158.67e6) / 33554432,
}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def max_over_ranks(value, dist, device="cuda"):
    """The slowest rank sets the time of a multi-rank measurement."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(world, bytes_per_rank, ms):
    """GB/s over all ranks: replicas do the same work each, so the job's bytes are world x the rank's."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


class ClockSampler:
    """Samples SM clock and throttle reasons (read-only NVML queries) while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


def run_reference(args, rank):
    """The oracle as it stands, single thread, on a bounded sample of the workload (first 2^22 values)."""
    if rank != 0:
        return
    import numpy as np
    from oracle import ccz
    from paper_2304_03890_b200 import fields
    sample_n = 1 << 22
    cfg = fields.config2(device="cpu", shape=(128, 128, 256), sigma=SIGMA)
    x = cfg["x"].numpy()[:sample_n]
    x2 = np.roll(x, 4096 * 7)
    eb = float(np.float32(cfg["eb"]))
    n = x.size

    def step():
        s = ccz.compress(x, eb)
        ccz.decompress(s, n)
        ccz.reduce_step(s, x2, eb, want_sum=True)
        ccz.allreduce_sim(x.reshape(P_SIM, n // P_SIM), eb)
        ccz.bcast_sim(x, P_SIM, eb, mode=1)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = 5 * 4 * n / dt / 1e9
    sample = f"first {n} values of a 128x128x256 field built by the same recipe; 1 thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(x_cpu, x2_cpu, eb):
    """Oracle, single thread, on the first 2^23 values of the very field the GPU gets (one warm-up pass, best of 2)."""
    import numpy as np
    from oracle import ccz
    n = min(1 << 23, x_cpu.size // (P_SIM * 128) * (P_SIM * 128))
    x = np.ascontiguousarray(x_cpu[:n])
    x2 = np.ascontiguousarray(x2_cpu[:n])
    best = None
    for it in range(3):
        t0 = time.perf_counter()
        s = ccz.compress(x, eb)
        ccz.decompress(s, n)
        ccz.reduce_step(s, x2, eb, want_sum=True)
        ccz.allreduce_sim(x.reshape(P_SIM, n // P_SIM), eb)
        ccz.bcast_sim(x, P_SIM, eb, mode=1)
        dt = time.perf_counter() - t0
        if it and (best is None or dt < best):
            best = dt
    return {"value": 5 * 4 * n / best / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
            "sample": f"first {n} of the {x_cpu.size} values of this run's field, all five entry points, best of 2"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--small", action="store_true", help="1/64-size field (for profiler captures and quick checks)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--field", default=None, help="AxBxC: another field shape of the same recipe (profiler captures)")
    ap.add_argument("--only", default=None, choices=["compress", "decompress", "reduce_step"],
                    help="run just one entry point per step and print a short line (profiler captures)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2304_03890_b200 import binding as B
    from paper_2304_03890_b200 import fields

    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    shape = (128, 128, 64) if args.small else SHAPE
    if args.field:
        shape = tuple(int(v) for v in args.field.split("x"))
    cfg = fields.config2(device="cuda", shape=shape, sigma=SIGMA)
    x, eb = cfg["x"], float(cfg["eb"])
    # local chunk of the reduce step: an independent field of the same recipe (another seed)
    x2 = fields.smooth_field(shape, SIGMA, -100.0, 100.0, fields.seed_for(2, 100 + rank), "cuda")
    n = x.numel()
    P = P_SIM
    B.ensure_workspace(n, P)
    bound = B.ccoll_compress_bound(n)
    s1 = torch.empty(bound, dtype=torch.uint8, device="cuda")
    s2 = torch.empty(bound, dtype=torch.uint8, device="cuda")
    nb1 = torch.zeros(1, dtype=torch.int64, device="cuda")
    nb2 = torch.zeros(1, dtype=torch.int64, device="cuda")
    dec = torch.empty(n, dtype=torch.float32, device="cuda")
    ssum = torch.empty(n, dtype=torch.float32, device="cuda")
    ar_out = torch.empty(n, dtype=torch.float32, device="cuda")
    moved = torch.zeros(1, dtype=torch.int64, device="cuda")
    C = B.ccoll_chunk_len(n, P)
    sc_out = torch.empty(P * C, dtype=torch.float32, device="cuda")
    cb = torch.zeros(P, dtype=torch.int64, device="cuda")
    xr = x.view(P, n // P)

    # the first compress tells the stream length the later calls pass as in_bytes
    B.ccoll_compress(x, eb, s1, nb1)
    assert B.ccoll_get_status() == B.OK
    in_bytes = int(nb1.item())

    def step(ev=None):
        def mark(i):
            if ev is not None:
                ev[i].record()
        mark(0)
        B.ccoll_compress(x, eb, s1, nb1)
        mark(1)
        B.ccoll_decompress(s1, in_bytes, n, dec)
        mark(2)
        B.ccoll_reduce_step(s1, in_bytes, x2, eb, s2, nb2, ssum)
        mark(3)
        B.ccoll_allreduce_sim(xr, ar_out.view(P, n // P), eb, moved)
        mark(4)
        B.ccoll_bcast_sim(x, sc_out, C, P, eb, B.SCATTER, cb)
        mark(5)

    launches_per_step = 3 + (1 + (P - 1) + 1) + (1 + 1)

    if args.only:
        # one entry point only: a small, short run for ncu captures; prints its event-timed duration
        call = {"compress": lambda: B.ccoll_compress(x, eb, s1, nb1),
                "decompress": lambda: B.ccoll_decompress(s1, in_bytes, n, dec),
                "reduce_step": lambda: B.ccoll_reduce_step(s1, in_bytes, x2, eb, s2, nb2, ssum)}[args.only]
        for _ in range(args.warmup):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        assert B.ccoll_get_status() == B.OK
        print(json.dumps({"only": args.only, "n_values": n, "ms_per_call": e0.elapsed_time(e1) / args.steps,
                          "stream_bytes": in_bytes}))
        return

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sync_all()
    assert B.ccoll_get_status() == B.OK

    # ---- device-resident timing: K steps between two events, per-call events inside ----
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    sync_all()
    t_begin.record()
    for k in range(args.steps):
        step(evs[k])
    t_end.record()
    sync_all()
    clocks = sampler.stop()
    assert B.ccoll_get_status() == B.OK
    total_ms = max_over_ranks(t_begin.elapsed_time(t_end), dist)
    ms_per_step = total_ms / args.steps
    call_ms = [statistics.mean(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) for i in range(5)]
    bytes_per_step = 5 * 4 * n
    value = whole_job_throughput(world, bytes_per_step, ms_per_step)

    # ---- rooflines of the three kernels (each of calls 1-3 is exactly one launch) ----
    peak, peak_kind = measured_peaks()
    S1, S2 = int(nb1.item()), int(nb2.item())
    alg = {
        "ccoll_compress_kernel": 4 * n + S1,
        "ccoll_decode_kernel": S1 + 4 * n,
        "ccoll_reduce_kernel": S1 + 4 * n + S2 + 4 * n,   # stream in + local in + stream out + sum_out
    }
    roofs = {}
    for name, ms in zip(("ccoll_compress_kernel", "ccoll_decode_kernel", "ccoll_reduce_kernel"), call_ms[:3]):
        ach = alg[name] / (ms * 1e-3) / 1e9
        roofs[name] = {"bound": "hbm", "achieved": ach, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                       "frac": ach / peak, "traffic": NCU_DRAM_BYTES_PER_VALUE[name] * n,
                       "traffic_source": "ncu capture at 33.5M values, scaled by value count",
                       "algorithmic_bytes": alg[name], "ms": ms,
                       "input_GBps": 4 * n / (ms * 1e-3) / 1e9}
    dominant = "ccoll_reduce_kernel"
    roofline = dict(roofs[dominant], kernel=dominant)

    # ---- end to end: inputs from pinned host memory, results read back, all inside the timed region ----
    hx = x.cpu().pin_memory()
    hx2 = x2.cpu().pin_memory()
    h_s1 = torch.empty(bound, dtype=torch.uint8).pin_memory()
    h_dec = torch.empty(n, dtype=torch.float32).pin_memory()
    h_sum = torch.empty(n, dtype=torch.float32).pin_memory()
    h_ar = torch.empty(n, dtype=torch.float32).pin_memory()
    h_nb = torch.zeros(1, dtype=torch.int64).pin_memory()
    e2e_steps = max(2, min(args.steps, 10))
    d2h = 0

    # The copies run on streams of their own, ordered against the calls by events: x2 goes up while compress and
    # decompress run, and every result starts down as soon as its call has finished (PCIe carries both ways).
    # Steps alternate between two sets of device buffers, as a caller that feeds one buffer after another would
    # run them: while the results of a step go down, the inputs of the next one come up and its calls run.  A
    # set is written again only when the step that used it before has been read out.
    s_in, s_out, s_len, cur = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    first = dict(x=x, x2=x2, s1=s1, nb1=nb1, dec=dec, s2=s2, nb2=nb2, ssum=ssum, ar=ar_out)
    sets = [first, {k: torch.empty_like(v) for k, v in first.items()}]
    for d in sets:
        d["ev"] = [torch.cuda.Event() for _ in range(6)]
        d["calls_done"], d["read_out"], d["used"] = torch.cuda.Event(), torch.cuda.Event(), False
    step_no = 0

    def e2e_step():
        nonlocal d2h, step_no
        d = sets[step_no % 2]
        step_no += 1
        ev = d["ev"]
        with torch.cuda.stream(s_in):
            if d["used"]:
                s_in.wait_event(d["calls_done"])   # the calls that read these inputs two steps ago
            d["x"].copy_(hx, non_blocking=True)
            ev[0].record(s_in)
            d["x2"].copy_(hx2, non_blocking=True)
            ev[1].record(s_in)
        if d["used"]:
            cur.wait_event(d["read_out"])          # the results these calls overwrite have gone down
        cur.wait_event(ev[0])
        B.ccoll_compress(d["x"], eb, d["s1"], d["nb1"])
        ev[2].record(cur)
        B.ccoll_decompress(d["s1"], in_bytes, n, d["dec"])
        ev[3].record(cur)
        cur.wait_event(ev[1])
        B.ccoll_reduce_step(d["s1"], in_bytes, d["x2"], eb, d["s2"], d["nb2"], d["ssum"])
        ev[4].record(cur)
        B.ccoll_allreduce_sim(d["x"].view(P, n // P), d["ar"].view(P, n // P), eb, moved)
        ev[5].record(cur)
        B.ccoll_bcast_sim(d["x"], sc_out, C, P, eb, B.SCATTER, cb)
        d["calls_done"].record(cur)
        with torch.cuda.stream(s_len):             # the stream's length, on a stream that carries nothing else
            s_len.wait_event(ev[2])
            h_nb.copy_(d["nb1"], non_blocking=True)
        s_len.synchronize()
        sb = int(h_nb.item())
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev[2])
            h_s1[:sb].copy_(d["s1"][:sb], non_blocking=True)
            s_out.wait_event(ev[3])
            h_dec.copy_(d["dec"], non_blocking=True)
            s_out.wait_event(ev[4])
            h_sum.copy_(d["ssum"], non_blocking=True)
            s_out.wait_event(ev[5])
            h_ar.copy_(d["ar"], non_blocking=True)
            d["read_out"].record(s_out)
        d["used"] = True
        d2h = sb + 3 * 4 * n + 8

    e2e_step()
    e2e_step()
    sync_all()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    sync_all()
    e2e_s = max_over_ranks((time.perf_counter() - t0) / e2e_steps, dist)
    e2e = {"value": whole_job_throughput(world, bytes_per_step, e2e_s * 1e3), "unit": "GB/s", "h2d_bytes_per_step": 2 * 4 * n,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_s * 1e3}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD if not args.small else "C2 recipe at 128x128x64 (quick check)",
                       "n_values": n, "block_len": 128, "eb": eb, "P_sim": P, "parallelism": f"replicas x{world}",
                       "l2": "inputs (256 MiB per buffer) larger than the 126 MB L2",
                       "step": "compress + decompress + reduce_step + allreduce_sim(P=8) + scatter_sim(P=8)"},
            "per_call_ms": dict(zip(("compress", "decompress", "reduce_step", "allreduce_sim", "scatter_sim"), call_ms)),
            "compression_ratio": 4 * n / S1,
            "roofline": roofline, "rooflines": roofs, "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(hx.numpy(), hx2.numpy(), eb)
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Benchmark of the quantized recurrent hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic input: for the recurrent
workloads one full sequence (all timesteps: on-line quantization of [x;h], binary product, fused gate
epilogue, every step), for the projection workload one bulk row-wise weight quantization plus one
activation quantization and one binary product.  The headline value is LSTM/GRU timesteps per second
(timesteps x concurrent sequences / time), summed over all GPUs; with N > 1 every rank runs its own
independent sequences (weak scaling, no data-path collective).

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle on the host cores instead.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1802_00150_b200 import synth  # noqa: E402

DEFAULT_WORKLOAD = "lstm1024_b1"
METRIC = "quantized LSTM/GRU timesteps per second (timesteps x concurrent sequences / s)"
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes per launch of the dominant kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by workload; the summaries are under profiles/.  None = not captured for the
# kernel as it stands.
NCU_TRAFFIC_BYTES = {"lstm1024_b1": 2422016 + 51968}    # rnn_persistent_kernel, profiles/rnn_persistent_kernel_lstm1024_b1.txt
# the batched workloads time a chain of kernels; for their dominant kernel (the tensor-core product) the cold-cache ncu
# captures under profiles/ give these DRAM bytes per launch (inside a sequence the packed weights stay in L2)
NCU_TRAFFIC_DOMINANT_KERNEL = {
    "lstm1024_b64": {"kernel": "bgemm_tc_kernel", "bytes": 3586816, "summary": "profiles/bgemm_tc_kernel_lstm1024_b64.txt"},
    "gru2048_b256": {"kernel": "bgemm_tc_persistent_kernel", "bytes": 8923136,
                     "summary": "profiles/bgemm_tc_persistent_kernel_gru2048_b256.txt"},
    "proj32768_b512": {"kernel": "bgemm_tc_persistent_kernel", "bytes": 13188352 + 10061568,
                       "summary": "profiles/bgemm_tc_persistent_kernel_proj32768_b512.txt"},
}
# the same for the cold matrix-vector kernel on 131072 x 8192 at 2/2 bits (profiles/bgemv_kernel_131072x8192_k2k2.txt)
NCU_TRAFFIC_GEMV_COLD_BYTES = 269500000


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the cold-GEMV bandwidth lines and the batched-regime lines")
    ap.add_argument("--phase-timing", action="store_true",
                    help="build the library with per-phase clock counters in the batch-1 sequence kernel, run the workload "
                         "with it and print the per-phase table instead of the benchmark line (not a benchmark value)")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes_per_timestep(wl):
    """What the method itself must move per timestep (all sequences of the batch): packed weight planes
    once, the row coefficients, the fp32 activation [x;h] in, and the fp32 state in/out."""
    words = (wl.n + 31) // 32
    w_bytes = wl.k_w * wl.m * words * 4 + 4 * wl.k_w * wl.m
    act = 4 * wl.n * wl.batch
    state = (3 if wl.cell == "lstm" else 2) * 4 * wl.H * wl.batch
    return w_bytes + act + state


def units_per_step(wl):
    return wl.steps * wl.batch if wl.cell != "proj" else 1


# ---- reference arm: the CPU oracle, as it stands, on the host cores ------------------------------------

def oracle_setup(wl, rows_limit=None):
    import oracle
    W = synth.weights(wl, rows=rows_limit).astype(np.float64)
    Wc, Wa = oracle.quantize_rows(W, wl.k_w, wl.T)
    return Wc, Wa


def oracle_step(wl, Wc, Wa, ins, batch_limit=None, timestep_limit=None):
    """One benchmark step on the oracle; returns the number of units (timesteps x sequences) it covered."""
    import oracle
    if wl.cell == "proj":
        acts = ins["acts"][:batch_limit].astype(np.float64)
        Xc, Xb = oracle.quantize_rows(acts, wl.k_a, wl.T)
        oracle.binary_gemm(Wc, Wa, Xc, Xb, wl.n)
        return acts.shape[0] / wl.batch * (Wc.shape[0] / wl.m)
    b = wl.batch if batch_limit is None else min(batch_limit, wl.batch)
    ts = wl.steps if timestep_limit is None else max(1, min(timestep_limit, wl.steps))
    xs, h0, c0 = ins["x_seq"][:ts, :b], ins["h0"][:b], ins["c0"][:b]
    if wl.cell == "lstm":
        oracle.lstm_sequence(Wc, Wa, None, wl.I, wl.H, xs, h0, c0, wl.k_a, wl.T)
    else:
        oracle.gru_sequence(Wc, Wa, None, wl.I, wl.H, xs, h0, wl.k_a, wl.T)
    return ts * b


def oracle_sample_plan(wl):
    """Bounded sample of the workload for the CPU legs: (rows_limit, batch_limit, description)."""
    if wl.cell == "proj":
        return 2048, 32, "first 2048 of %d weight rows x first 32 of %d activation vectors (scaled by work)" % (wl.m, wl.batch)
    if wl.batch > 2:
        return None, 2, "all %d timesteps for the first 2 of %d sequences" % (wl.steps, wl.batch)
    return None, None, "the full workload (%d timesteps, batch %d)" % (wl.steps, wl.batch)


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows_limit, batch_limit, desc = oracle_sample_plan(wl)
    Wc, Wa = oracle_setup(wl, rows_limit)
    ins = synth.inputs(wl)
    # keep the whole run within a few minutes: if K full samples would not fit, each step covers only the
    # first timesteps of the sequence (the sample is described in the output)
    t0 = time.perf_counter()
    oracle_step(wl, Wc, Wa, ins, batch_limit)
    t_one = time.perf_counter() - t0
    ts_limit = None
    budget_s = 150.0
    if wl.cell != "proj" and (args.steps + args.warmup) * t_one > budget_s:
        ts_limit = max(1, int(wl.steps * budget_s / ((args.steps + args.warmup) * t_one)))
        desc += "; first %d of %d timesteps per step (time budget)" % (min(ts_limit, wl.steps), wl.steps)
    for _ in range(args.warmup):
        oracle_step(wl, Wc, Wa, ins, batch_limit, ts_limit)
    units = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        units += oracle_step(wl, Wc, Wa, ins, batch_limit, ts_limit)
    dt = time.perf_counter() - t0
    value = units / dt if wl.cell != "proj" else units / dt
    unit = "timesteps/s" if wl.cell != "proj" else "passes/s"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, "n/a (CPU)"),
        "cpu_baseline": {"value": value, "unit": unit, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def workload_config(wl, l2_note):
    return {
        "workload": wl.name, "cell": wl.cell, "input": wl.I, "hidden": wl.H, "rows": wl.m, "cols": wl.n,
        "k_w": wl.k_w, "k_a": wl.k_a, "T": wl.T, "batch": wl.batch, "timesteps": wl.steps,
        "weights": "N(0,%g^2)" % wl.w_std, "inputs": wl.x_dist, "seed": wl.seed, "l2": l2_note,
        "parallelism": "independent sequences per GPU (replicas)",
    }


# ---- clocks ----------------------------------------------------------------------------------------------

class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid, self.proc, self.lines = uuid, None, []
        self.nvml, self.samples, self.stop_flag = None, [], False

    def _nvml_loop(self):
        nv = self.nvml
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
        while not self.stop_flag:
            try:
                sm = nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                self.samples.append((sm, [k for k, bit in names.items() if mask & bit]))
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(self.uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(self.uuid)
            self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.QUERY, "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            sm = [s for s, _ in self.samples]
            reasons = sorted({r for _, rs in self.samples for r in rs})
            return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": float(self.max_sm),
                    "reasons": reasons, "samples": len(sm), "source": "nvml, ~5 ms period, during the timed regions (device-resident steps and end-to-end steps)"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ---- replicas: what differs between ranks, and how their measurements are combined ----------------------

def rank_workload(wl, rank):
    """Every rank runs its own sequences (seed offset by rank) through the same model (weights are not offset)."""
    return synth.scaled(wl, seed=wl.seed + 1000 * rank) if rank else wl


def combine_over_ranks(dist, device, total_ms, e2e_total_ms, launches):
    """Slowest rank's times (MAX) and the launches of all ranks (SUM); no data-path collective exists."""
    import torch
    t = torch.tensor([total_ms, e2e_total_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    lt = torch.tensor([launches], device=device, dtype=torch.int64)
    dist.all_reduce(lt, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(lt[0])


def whole_job_value(world, units, steps, total_ms):
    """Units all ranks processed / the slowest rank's time."""
    return world * units * steps / (total_ms * 1e-3)


# ---- our arm ---------------------------------------------------------------------------------------------

def run_ours(args, wl):
    import torch
    from paper_1802_00150_b200 import amq

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    stream = torch.cuda.current_stream()

    # inputs: every rank draws its own sequences (seed offset by rank); weights are the same model
    wl_rank = rank_workload(wl, rank)
    ins = synth.inputs(wl_rank)
    W = torch.from_numpy(synth.weights(wl)).to(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)        # 256 MiB > L2 (126 MB)

    if wl.cell == "proj":
        acts = torch.from_numpy(ins["acts"]).to(dev)
        Wcodes = torch.empty((wl.m, wl.k_w, amq.words_per_row(wl.n)), dtype=torch.int32, device=dev)
        Walpha = torch.empty((wl.m, wl.k_w), dtype=torch.float32, device=dev)
        y = torch.empty((wl.batch, wl.m), dtype=torch.float32, device=dev)

        def step():
            amq.quantize(W, wl.k_w, wl.T, codes=Wcodes, coeffs=Walpha)
            xc, xb = amq.quantize(acts, wl.k_a, wl.T)
            amq.binary_gemm(Wcodes, Walpha, xc, xb, wl.n, y=y)

        h2d = acts.numel() * 4
        d2h = 4 * wl.batch
        acts_host = torch.from_numpy(ins["acts"]).pin_memory()
        y_host = torch.empty((wl.batch,), dtype=torch.float32).pin_memory()

        def step_e2e():
            acts.copy_(acts_host, non_blocking=True)
            step()
            y_host.copy_(y[:, 0], non_blocking=True)
            torch.cuda.current_stream().synchronize()
    else:
        Wcodes, Walpha = amq.quantize(W, wl.k_w, wl.T)
        del W
        x_seq = torch.from_numpy(ins["x_seq"]).to(dev)
        h0, c0 = torch.from_numpy(ins["h0"]).to(dev), torch.from_numpy(ins["c0"]).to(dev)
        ws = amq.new_workspace(wl.I, wl.H, wl.batch, wl.k_a)
        staging = amq.new_host_staging(wl.I, wl.H, wl.batch, wl.steps)
        h_last, c_last = torch.empty_like(h0), torch.empty_like(c0)
        xs_host = torch.from_numpy(ins["x_seq"]).pin_memory()
        h0_host, c0_host = torch.from_numpy(ins["h0"]).pin_memory(), torch.from_numpy(ins["c0"]).pin_memory()
        hl_host, cl_host = torch.empty_like(h0_host).pin_memory(), torch.empty_like(c0_host).pin_memory()
        if wl.cell == "lstm":
            def step():
                amq.lstm_sequence(Wcodes, Walpha, None, wl.I, wl.H, x_seq, h0, c0, wl.k_a, wl.T, ws,
                                  h_last=h_last, c_last=c_last)

            def step_e2e():
                amq.lstm_sequence_host(Wcodes, Walpha, None, wl.I, wl.H, xs_host, h0_host, c0_host, wl.k_a, wl.T,
                                       ws, staging, hl_host, cl_host)
            h2d = (xs_host.numel() + 2 * h0_host.numel()) * 4
            d2h = 2 * h0_host.numel() * 4
        else:
            def step():
                amq.gru_sequence(Wcodes, Walpha, None, wl.I, wl.H, x_seq, h0, wl.k_a, wl.T, ws, h_last=h_last)

            def step_e2e():
                amq.gru_sequence_host(Wcodes, Walpha, None, wl.I, wl.H, xs_host, h0_host, wl.k_a, wl.T,
                                      ws, staging, hl_host)
            h2d = (xs_host.numel() + h0_host.numel()) * 4
            d2h = h0_host.numel() * 4

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, iters, warmup):
        """Per-iteration CUDA events on the launching stream; L2 flushed (untimed) before each iteration."""
        for _ in range(warmup):
            fn()
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(iters)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(iters)]
        barrier()
        launches0 = amq.kernel_launches()
        for i in range(iters):
            flush.fill_(i & 0xFF)
            starts[i].record(stream)
            fn()
            stops[i].record(stream)
        barrier()
        launches = amq.kernel_launches() - launches0
        ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
        return ms, launches

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    if rank == 0:
        sampler.start()
    ms, launches = timed(step, args.steps, max(args.warmup, 3))
    total_ms = float(sum(ms))
    ms_e2e, _ = timed(step_e2e, max(3, min(args.steps, 20)), 3)
    clocks = sampler.stop() if rank == 0 else None
    e2e_total_ms = float(sum(ms_e2e))
    e2e_iters = len(ms_e2e)
    if dist is not None:
        total_ms, e2e_total_ms, launches = combine_over_ranks(dist, dev, total_ms, e2e_total_ms, launches)
    assert amq.workspace_status(ws) == 0 if wl.cell != "proj" else True

    units = units_per_step(wl)
    unit = "timesteps/s" if wl.cell != "proj" else "passes/s"
    value = whole_job_value(world, units, args.steps, total_ms)
    e2e_value = whole_job_value(world, units, e2e_iters, e2e_total_ms)
    peak, peak_kind = measured_peaks()

    line = None
    if rank == 0:
        step_ms = total_ms / args.steps
        if wl.cell == "proj":
            alg_bytes = wl.m * wl.n * 4 + wl.k_w * wl.m * ((wl.n + 31) // 32) * 4 * 2 + wl.batch * wl.m * 4
            kernel_name = "bulk quantize + binary GEMM (whole step)"
        else:
            alg_bytes = algorithmic_bytes_per_timestep(wl) * wl.steps
            kernel_name = ("rnn_persistent_kernel (one launch = the whole sequence)" if wl.batch == 1
                           else "chain of quantize_kernel + bgemm_tc_kernel per timestep")
        achieved = alg_bytes / (step_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "ms_per_step_median": float(np.median(ms)),
            "ms_per_step_min": float(np.min(ms)), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32 popcount + f32", "data": "synthetic",
            "config": workload_config(wl, "flushed before every step by an untimed 256 MiB write; inside a step "
                                          "the packed weights are re-read from L2 by design"),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": "of " + peak_kind,
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "algorithmic_bytes_per_launch": int(alg_bytes),
                         "traffic": NCU_TRAFFIC_BYTES.get(wl.name)},
            "us_per_timestep": 1e3 * step_ms / max(wl.steps, 1) if wl.cell != "proj" else None,
        }
        if wl.name in NCU_TRAFFIC_DOMINANT_KERNEL:
            line["roofline"]["traffic_dominant_kernel"] = NCU_TRAFFIC_DOMINANT_KERNEL[wl.name]
        if not args.no_extras and world == 1:
            line["gemv_cold"] = cold_gemv(amq, torch, dev, flush, peak, peak_kind)
            # the second half of the metric (binary matrix-vector product against the HBM peak) beside the first
            first = line["gemv_cold"][0]
            line["roofline"]["gemv_cold"] = {k: first[k] for k in ("workload", "ms", "ms_min", "achieved", "unit", "peak", "frac",
                                                                   "peak_kind", "frac_of_nominal_8000", "algorithmic_bytes")}
            line["roofline"]["gemv_cold"]["traffic"] = NCU_TRAFFIC_GEMV_COLD_BYTES
            line["gemv_rotated"] = rotated_gemv(amq, torch, dev, peak, peak_kind)
            line["batched"] = batched_lines(amq, torch, dev, flush, peak, peak_kind)
            assert amq.device_status() == 0
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(wl, unit)
            if not args.no_extras:
                line["cpu_baseline_table6"] = cpu_baseline_table6()
                line["cpu_baseline_batched"] = cpu_baseline_all_cores()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line))


def _event_ms(torch, fn, flush, iters, want_min=False):
    """Median device time of fn (one launch chain) with the L2 flushed, untimed, before every run."""
    times = []
    for i in range(iters):
        flush.fill_(i & 0xFF)
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        fn()
        e.record()
        torch.cuda.synchronize()
        times.append(s.elapsed_time(e))
    if want_min:
        return float(np.median(times)), float(np.min(times))
    return float(np.median(times))


def _burst_ms(torch, fn, iters):
    """Device time per call over `iters` calls enqueued back to back (for kernels shorter than a launch)."""
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s.record()
    for _ in range(iters):
        fn()
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e) / iters


def cold_gemv(amq, torch, dev, flush, peak, peak_kind):
    """Batch-1 binary GEMV on packed planes far larger than L2 (HBM-bound): achieved GB/s of packed weights."""
    out = []
    for m, n, k_w, k_a in ((131072, 8192, 2, 2), (262144, 8192, 2, 2), (131072, 8192, 3, 3), (1048576, 1024, 2, 2)):
        wpr = amq.words_per_row(n)
        g = torch.Generator(device=dev)
        g.manual_seed(0)
        Wcodes = torch.randint(-2 ** 31, 2 ** 31 - 1, (m, k_w, wpr), dtype=torch.int32, device=dev, generator=g)
        Walpha = torch.rand((m, k_w), device=dev, generator=g) * 0.02
        x = torch.from_numpy(synth.uniform((1, n), -1, 1, 0, 9)).to(dev)
        xc, xb = amq.quantize(x, k_a, 2)
        y = torch.empty((1, m), device=dev)
        for _ in range(3):
            amq.binary_gemm(Wcodes, Walpha, xc, xb, n, y=y)
        ms, ms_min = _event_ms(torch, lambda: amq.binary_gemm(Wcodes, Walpha, xc, xb, n, y=y), flush, 20, want_min=True)
        alg = Wcodes.numel() * 4 + Walpha.numel() * 4 + m * 4 + xc.numel() * 4
        gbs = alg / (ms * 1e-3) / 1e9
        out.append({"workload": "batch-1 binary GEMV %dx%d, k_w=%d, k_a=%d, packed planes %d MiB (random bits), cold" % (
                        m, n, k_w, k_a, Wcodes.numel() * 4 >> 20),
                    "ms": ms, "ms_min": ms_min, "bound": "hbm", "achieved": gbs, "unit": "GB/s", "peak": peak, "frac": gbs / peak,
                    "peak_kind": "of " + peak_kind, "frac_of_nominal_8000": gbs / 8000.0, "algorithmic_bytes": int(alg)})
        del Wcodes, Walpha, y
    return out


def rotated_gemv(amq, torch, dev, peak, peak_kind):
    """The small matrix-vector shapes (the two of Table 6 and 32768 x 1024) kept cold by rotating over distinct weight
    copies that together exceed twice the L2: one launch per copy, the whole rotation replayed from a CUDA graph so that
    the gaps between the launches are those of the device.  GB/s of packed weights over the rotation."""
    out = []
    for m, n, k in ((4096, 1024, 2), (42000, 1024, 2), (32768, 1024, 2), (42000, 1024, 3)):
        wpr = amq.words_per_row(n)
        bytes_one = m * k * wpr * 4 + m * k * 4 + m * 4
        copies = max(2, min(400, -(-(300 << 20) // bytes_one)))
        g = torch.Generator(device=dev)
        g.manual_seed(6)
        W = torch.randint(-2 ** 31, 2 ** 31 - 1, (copies, m, k, wpr), dtype=torch.int32, device=dev, generator=g)
        Wa = torch.rand((copies, m, k), device=dev, generator=g) * 0.02
        x = torch.rand((1, n), device=dev, generator=g) * 2 - 1
        xc, xb = amq.quantize(x, k, 2)
        y = torch.empty((copies, 1, m), device=dev)

        def rotation():
            for c in range(copies):
                amq.binary_gemm(W[c], Wa[c], xc, xb, n, y=y[c])

        line = {"workload": "batch-1 binary GEMV %d x %d, %d/%d bits, rotated over %d weight copies (%d MiB in all)" % (
                    m, n, k, k, copies, copies * bytes_one >> 20), "bound": "hbm", "unit": "GB/s", "peak": peak,
                "peak_kind": "of " + peak_kind, "algorithmic_bytes": int(copies * bytes_one)}
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                rotation()
                with torch.cuda.graph(graph, stream=side):
                    rotation()
            torch.cuda.current_stream().wait_stream(side)
            ms = _burst_ms(torch, graph.replay, 5)
            line.update({"ms": ms, "us_per_launch": 1e3 * ms / copies, "achieved": copies * bytes_one / (ms * 1e-3) / 1e9})
            line["frac"] = line["achieved"] / peak
        except Exception as exc:
            line["graph_replay_error"] = str(exc)[:120]
        out.append(line)
        del W, Wa, y
    return out


def batched_lines(amq, torch, dev, flush, hbm_peak, peak_kind):
    """The batched (binary GEMM) regime and the bulk quantizer, one line per benchmark shape.  The tensor-core
    product is held against the int8 peak = 2 x the measured dense bf16 figure (nominal int8 : bf16 ratio)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        bf16 = float(json.load(open(path))["bf16_tflops"])
        tkind = "of measured bf16 x 2"
    except Exception:
        bf16, tkind = 1590.0, "of fallback bf16 x 2"
    int8_tops = 2.0 * bf16
    int8_measured = measured_int8_tops(torch, dev)
    out = [{"workload": "dense int8 peak: torch._int_mm 8192 x 8192 x 8192 (library kernel), best of 10, CUDA events",
            "bound": "tensor", "achieved": int8_measured, "unit": "TOP/s (int8)", "assumed_peak_2x_bf16": int8_tops}]
    for name in ("lstm1024_b64", "gru2048_b256", "proj32768_b512"):
        wl = synth.WORKLOADS[name]
        wpr = amq.words_per_row(wl.n)
        g = torch.Generator(device=dev)
        g.manual_seed(1)
        W = torch.randn((wl.m, wl.n), device=dev, generator=g) * wl.w_std
        Wcodes, Walpha = amq.quantize(W, wl.k_w, wl.T)
        acts = torch.randn((wl.batch, wl.n), device=dev, generator=g)
        xc, xb = amq.quantize(acts, wl.k_a, wl.T)
        y = torch.empty((wl.batch, wl.m), device=dev)
        ms = _burst_ms(torch, lambda: amq.binary_gemm(Wcodes, Walpha, xc, xb, wl.n, y=y), 20)
        mac = wl.m * wl.k_w * wl.batch * wl.k_a * wpr * 32
        tops = 2.0 * mac / (ms * 1e-3) / 1e12
        out.append({"workload": "binary GEMM of %s: stacked M=%d, N=%d, K=%d bit positions" % (
                        name, wl.m * wl.k_w, wl.batch * wl.k_a, wpr * 32),
                    "ms": ms, "bound": "tensor", "achieved": tops, "unit": "TOP/s (int8, 2 per bit-MAC)", "peak": int8_tops,
                    "frac": tops / int8_tops, "peak_kind": tkind, "bit_mac_per_s": mac / (ms * 1e-3),
                    "peak_int8_measured": int8_measured,
                    "frac_of_int8_measured": (tops / int8_measured) if int8_measured else None})
        msq = _burst_ms(torch, lambda: amq.quantize(acts, wl.k_a, wl.T, codes=xc, coeffs=xb), 20)
        out.append({"workload": "on-line quantizer of %s: %d vectors of %d, k=%d, T=%d" % (name, wl.batch, wl.n, wl.k_a, wl.T),
                    "ms": msq, "bound": "latency"})
        if name == "proj32768_b512":
            msb = _event_ms(torch, lambda: amq.quantize(W, wl.k_w, wl.T, codes=Wcodes, coeffs=Walpha), flush, 10)
            alg = W.numel() * 4 + Wcodes.numel() * 4 + Walpha.numel() * 4
            gbs = alg / (msb * 1e-3) / 1e9
            out.append({"workload": "bulk row-wise quantization %dx%d, k=%d, T=%d, cold" % (wl.m, wl.n, wl.k_w, wl.T),
                        "ms": msb, "bound": "hbm", "achieved": gbs, "unit": "GB/s", "peak": hbm_peak, "frac": gbs / hbm_peak,
                        "peak_kind": "of " + peak_kind, "algorithmic_bytes": int(alg)})
        del W, Wcodes, Walpha, acts, xc, xb, y
    out.append(paper_form_line(amq, torch, dev))
    out.append(gru_forms_line(amq, torch, dev))
    out.append(greedy_decoding_line(amq, torch, dev))
    out.extend(table6_lines(amq, torch, dev, flush))
    out.append(quality_line(amq, torch, dev))
    return out


def measured_int8_tops(torch, dev):
    """Dense int8 throughput of this GPU as the library's own int8 matrix product reaches it (2 N^3 operations, best of
    10): the denominator for the tensor-core lines next to the nominal 2 x bf16 figure.  None if the routine is missing."""
    try:
        n = 8192
        a = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=dev)
        b = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=dev)
        for _ in range(3):
            torch._int_mm(a, b)
        best = 1e30
        for _ in range(10):
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record()
            torch._int_mm(a, b)
            e.record()
            torch.cuda.synchronize()
            best = min(best, s.elapsed_time(e))
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    except Exception:
        return None


def paper_form_line(amq, torch, dev):
    """The hidden-1024 LSTM in the paper's own form (separate W_i / W_h, inputs = rows of a quantized embedding,
    only h quantized on-line), 3/3/3 bits, 64 sequences, 35 timesteps: input projections of all timesteps in
    one batched product, then quantize(h) + product with W_h per timestep."""
    I = H = 1024
    k_w = k_e = k_a = 3
    batch, steps, vocab = 64, 35, 4096
    g = torch.Generator(device=dev)
    g.manual_seed(2)
    Wic, Wia = amq.quantize(torch.randn((4 * H, I), device=dev, generator=g) * 0.03, k_w, 2)
    Whc, Wha = amq.quantize(torch.randn((4 * H, H), device=dev, generator=g) * 0.03, k_w, 2)
    Wec, Wea = amq.quantize(torch.randn((vocab, I), device=dev, generator=g) * 0.5, k_e, 2)
    tokens = torch.randint(0, vocab, (steps, batch), dtype=torch.int32, device=dev, generator=g)
    h0 = torch.zeros((batch, H), device=dev)
    c0 = torch.zeros((batch, H), device=dev)
    h_last, c_last = torch.empty_like(h0), torch.empty_like(c0)
    ws = amq.new_paper_workspace(H, batch, steps, k_a)

    def run():
        xc, xb = amq.embedding_rows(Wec, Wea, I, tokens)
        amq.lstm_sequence_paper(Wic, Wia, Whc, Wha, None, I, H, xc, xb, h0, c0, k_a, 2, ws, h_last=h_last, c_last=c_last)

    ms = _burst_ms(torch, run, 10)
    return {"workload": "paper-form LSTM sequence, I=H=1024, 3/3/3 bits, %d sequences x %d timesteps (embedding gather + "
                        "one batched input projection + per-step quantize(h) and W_h product)" % (batch, steps),
            "ms": ms, "bound": "tensor+latency", "us_per_timestep": 1e3 * ms / steps,
            "timesteps_per_s": batch * steps / (ms * 1e-3)}


def gru_forms_line(amq, torch, dev):
    """One GRU timestep at the C4 shape (I = H = 2048, 2/3 bits, 256 sequences) in the two forms: the default one (reset
    gate after the product: one quantization, one product) and the original one of Cho et al. (reset gate before the
    candidate's product: two quantizations, two products)."""
    wl = synth.WORKLOADS["gru2048_b256"]
    g = torch.Generator(device=dev)
    g.manual_seed(8)
    Wc, Wa = amq.quantize(torch.randn((wl.m, wl.n), device=dev, generator=g) * wl.w_std, wl.k_w, wl.T)
    x = torch.randn((wl.batch, wl.I), device=dev, generator=g)
    h = torch.rand((wl.batch, wl.H), device=dev, generator=g) * 2 - 1
    ws = amq.new_workspace(wl.I, wl.H, wl.batch, wl.k_a)
    h1, h2 = torch.empty_like(h), torch.empty_like(h)
    ms_default = _burst_ms(torch, lambda: amq.gru_step(Wc, Wa, None, wl.I, wl.H, x, h, wl.k_a, wl.T, ws, h_out=h1), 20)
    ows = torch.empty((amq._lib.amq_gru_original_workspace_bytes(wl.I, wl.H, wl.batch, wl.k_a),), dtype=torch.uint8, device=dev)
    ms_original = _burst_ms(torch, lambda: amq.gru_step_original(Wc, Wa, None, wl.I, wl.H, x, h, wl.k_a, wl.T, ows, h_out=h2), 20)
    return {"workload": "one GRU timestep, I = H = 2048, 2/3 bits, 256 sequences: default form / original form (Cho et al.)",
            "ms": ms_default, "ms_original_form": ms_original, "bound": "tensor+latency"}


def table6_lines(amq, torch, dev, flush):
    """The two matrix-vector shapes the paper times on one CPU core (Table 6): on-line quantization of the
    1024-vector h plus the binary product, 4096 x 1024 (W_h h) and 42000 x 1024 (W_s h), at 2/2 and 3/3 bits.
    Cold = L2 flushed before every run; warm = back to back.  The paper's CPU times are quoted for context only."""
    paper_ms = {}          # the paper's single-core CPU times, kept as a fixture: rows, bits, total ms
    for ln in open(os.path.join(ROOT, "tests", "golden", "table6_cpu_ms.txt")):
        f = ln.split()
        if len(f) >= 6 and f[0].isdigit() and f[2].isdigit():
            paper_ms[(int(f[0]), int(f[2]))] = float(f[4])
    out = []
    for m in (4096, 42000):
        for k in (2, 3):
            n = 1024
            g = torch.Generator(device=dev)
            g.manual_seed(4)
            Wc, Wa = amq.quantize(torch.randn((m, n), device=dev, generator=g) * 0.05, k, 2)
            hvec = torch.rand((1, n), device=dev, generator=g) * 2 - 1
            hc, hb = amq.quantize(hvec, k, 2)
            y = torch.empty((1, m), device=dev)

            def run():
                amq.quantize(hvec, k, 2, codes=hc, coeffs=hb)
                amq.binary_gemm(Wc, Wa, hc, hb, n, y=y)

            def run_fused():
                amq.quantized_gemv(Wc, Wa, hvec, k, 2, y=y[0])

            for _ in range(3):
                run()
                run_fused()
            cold = _event_ms(torch, run, flush, 10)
            warm = _burst_ms(torch, run, 50)
            line = {"workload": "Table 6 shape: quantize(h) + binary product %d x %d, %d/%d bits, batch 1" % (m, n, k, k),
                    "ms_cold": cold, "ms_warm": warm, "bound": "latency",
                    "ms_cold_one_launch": _event_ms(torch, run_fused, flush, 10),
                    "ms_warm_one_launch": _burst_ms(torch, run_fused, 50),
                    "note": "ms_cold / ms_warm: two launches (amq_quantize, amq_binary_gemm); *_one_launch: amq_quantized_gemv",
                    "paper_cpu_ms_one_xeon_core": paper_ms[(m, k)]}
            try:
                # the same two launches replayed from a CUDA graph: device time without the cost of the Python calls
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    run()
                    with torch.cuda.graph(graph, stream=side):
                        run()
                torch.cuda.current_stream().wait_stream(side)
                line["ms_warm_graph_replay"] = _burst_ms(torch, graph.replay, 50)
                graph1 = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph1, stream=side):
                        run_fused()
                torch.cuda.current_stream().wait_stream(side)
                line["ms_warm_graph_replay_one_launch"] = _burst_ms(torch, graph1.replay, 50)
            except Exception as exc:                                  # the line stays without the replay figure
                line["graph_replay_error"] = str(exc)[:120]
            out.append(line)
            del Wc, Wa
    return out


def quality_line(amq, torch, dev):
    """Relative mean squared error ||w - w_hat||^2 / ||w||^2 of the quantization methods compared in Sec. 2 / Tables 1-2
    (greedy, refined greedy, alternating with T = 2, and alternating followed by a last coefficient refit), on
    synthetic rows (256 x 1024): Gaussian, and heavy-tailed (cube of a Gaussian).  A quality report, not a timing."""
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    base = torch.randn((256, 1024), device=dev, generator=g)
    out = {"workload": "relative MSE of the quantization methods, 256 rows x 1024, computed with the library",
           "bound": "none (quality report)"}
    for name, w in (("gaussian", base * 0.03), ("heavy_tailed", base ** 3)):
        norm = (w.double() ** 2).sum()
        table = {}
        for k in (2, 3, 4):
            row = {}
            for label, T, method, final in (("greedy", 0, amq.METHOD_ALTERNATING, False),
                                            ("refined_greedy", 0, amq.METHOD_REFINED_GREEDY, False),
                                            ("alternating_T2", 2, amq.METHOD_ALTERNATING, False),
                                            ("alternating_T2_final_refit", 2, amq.METHOD_ALTERNATING, True)):
                codes, coeffs = amq.quantize_variant(w, k, T, method, final)
                w_hat = amq.unpack(codes, coeffs, 1024)
                row[label] = float(((w.double() - w_hat.double()) ** 2).sum() / norm)
            table["k=%d" % k] = row
        out[name] = table
    return out


def greedy_decoding_line(amq, torch, dev):
    """Language-model decoding at the scale of the paper's largest vocabulary (42000 words, hidden 1024, 2/2 bits),
    one sequence, the arg-max fed back on the device: amq_lm_greedy_decode enqueues, per token, embedding row ->
    paper-form cell -> output product with the on-line quantizer of h inside -> log-softmax / arg-max (six launches)."""
    I = H = 1024
    V, k, ntok = 42000, 2, 64
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    Wic, Wia = amq.quantize(torch.randn((4 * H, I), device=dev, generator=g) * 0.03, k, 2)
    Whc, Wha = amq.quantize(torch.randn((4 * H, H), device=dev, generator=g) * 0.03, k, 2)
    Wec, Wea = amq.quantize(torch.randn((V, I), device=dev, generator=g) * 0.5, k, 2)
    Wsc, Wsa = amq.quantize(torch.randn((V, H), device=dev, generator=g) * 0.05, k, 2)
    bs = torch.randn((V,), device=dev, generator=g) * 0.1
    ws = amq.new_decode_workspace(V, I, H, k, k)
    tokens = torch.zeros((ntok + 1,), dtype=torch.int32, device=dev)
    h, c = torch.zeros((1, H), device=dev), torch.zeros((1, H), device=dev)

    first = torch.tensor([17], dtype=torch.int32, device=dev)

    def run():
        tokens[0:1].copy_(first)
        amq.lm_greedy_decode(Wec, Wea, Wic, Wia, Whc, Wha, None, Wsc, Wsa, bs, I, H, k, 2, tokens, h, c, ws)

    ms = _burst_ms(torch, run, 5)
    extra = {}
    try:
        # the same chain (7 launches per token) captured once in a CUDA graph and replayed
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            run()
            with torch.cuda.graph(graph, stream=side):
                run()
        torch.cuda.current_stream().wait_stream(side)
        gms = _burst_ms(torch, graph.replay, 5)
        extra = {"us_per_token_graph_replay": 1e3 * gms / ntok, "tokens_per_s_graph_replay": ntok * 1e3 / gms}
    except Exception as exc:
        extra = {"graph_replay_error": str(exc)[:120]}
    return {**extra, "workload": "greedy decoding, vocabulary %d, I=H=%d, 2/2 bits, one sequence, %d tokens per call (embedding row, "
                        "paper-form cell, quantize(h), output product, log-softmax/arg-max; token fed back on the device)" % (
                            V, H, ntok),
            "ms": ms, "bound": "latency", "us_per_token": 1e3 * ms / ntok, "tokens_per_s": ntok * 1e3 / ms,
            "distinct_tokens": int(torch.unique(tokens).numel())}


def cpu_baseline_table6():
    """The oracle, as it stands, on one host core, on the operations the paper times in Table 6 (on-line quantization of
    the 1024-vector h plus the binary product; weights quantized beforehand, not timed): the same kind of measurement as
    the paper's, on this machine's CPU and with a plain, untuned program."""
    import oracle
    out = []
    h = synth.uniform((1, 1024), -1, 1, 11, 1).astype(np.float64)
    for m, k in ((4096, 2), (4096, 3), (42000, 2), (42000, 3)):
        rows = min(m, 4096)                                          # quantize a block of rows and tile it: only the product is timed
        Wc, Wa = oracle.quantize_rows(synth.normal((rows, 1024), 0.05, 11, 2).astype(np.float64), k, 2)
        reps = -(-m // rows)
        Wc, Wa = np.tile(Wc, (reps, 1, 1))[:m], np.tile(Wa, (reps, 1))[:m]
        best_q, best_p = 1e30, 1e30
        for _ in range(3):
            t0 = time.perf_counter()
            hc, hb = oracle.quantize_rows(h, k, 2)
            t1 = time.perf_counter()
            oracle.binary_gemm(Wc, Wa, hc, hb, 1024)
            t2 = time.perf_counter()
            best_q, best_p = min(best_q, t1 - t0), min(best_p, t2 - t1)
        out.append({"workload": "Table 6 shape %d x 1024, %d/%d bits, batch 1: oracle on one host core" % (m, k, k),
                    "quantize_ms": 1e3 * best_q, "product_ms": 1e3 * best_p, "total_ms": 1e3 * (best_q + best_p),
                    "cores": 1, "kind": "oracle", "sample": "best of 3; weights quantized beforehand"})
    return out


def _oracle_worker(job):
    """One process of the all-cores oracle runs: its share of the sequences (or of the weight rows)."""
    name, lo, hi = job
    import oracle
    wl = synth.WORKLOADS[name]
    ins = synth.inputs(wl)
    if wl.cell == "proj":
        W = synth.weights(wl, rows=hi)[lo:hi].astype(np.float64)
        t0 = time.perf_counter()
        Wc, Wa = oracle.quantize_rows(W, wl.k_w, wl.T)                      # the bulk quantization is part of this pass
        Xc, Xb = oracle.quantize_rows(ins["acts"][:32].astype(np.float64), wl.k_a, wl.T)
        oracle.binary_gemm(Wc, Wa, Xc, Xb, wl.n)
        return time.perf_counter() - t0
    Wc, Wa = oracle_setup(wl)
    xs, h0, c0 = ins["x_seq"][:, lo:hi], ins["h0"][lo:hi], ins["c0"][lo:hi]
    t0 = time.perf_counter()
    if wl.cell == "lstm":
        oracle.lstm_sequence(Wc, Wa, None, wl.I, wl.H, xs, h0, c0, wl.k_a, wl.T)
    else:
        oracle.gru_sequence(Wc, Wa, None, wl.I, wl.H, xs, h0, wl.k_a, wl.T)
    return time.perf_counter() - t0


def cpu_baseline_all_cores():
    """The oracle, as it stands, on ALL host cores for the batched workloads: independent sequences (weight rows for
    the projection pass) are dealt out to one process per core; the time is that of the slowest process.  Bounded
    samples: one sequence per core; for the projection 64 weight rows per core and 32 of the 512 activation vectors
    (scaled to the whole pass by work)."""
    import multiprocessing as mp
    cores = os.cpu_count() or 1
    out = []
    ctx = mp.get_context("fork")
    for name in ("lstm1024_b64", "gru2048_b256", "proj32768_b512"):
        wl = synth.WORKLOADS[name]
        per = 64 if wl.cell == "proj" else 1
        jobs = [(name, c * per, (c + 1) * per) for c in range(cores)]
        try:
            with ctx.Pool(cores) as pool:
                times = pool.map(_oracle_worker, jobs)
        except Exception as exc:
            out.append({"workload": name, "error": str(exc)[:120]})
            continue
        dt = max(times)
        if wl.cell == "proj":
            fraction = (cores * per / wl.m) * (32.0 / wl.batch)
            out.append({"workload": name, "value": fraction / dt, "unit": "passes/s", "cores": cores, "kind": "oracle",
                        "sample": "%d weight rows per core (quantized and multiplied), 32 of %d activation vectors; scaled by work"
                                  % (per, wl.batch)})
        else:
            out.append({"workload": name, "value": cores * per * wl.steps / dt, "unit": "timesteps/s", "cores": cores,
                        "kind": "oracle", "sample": "one full sequence (%d timesteps) per core; weight quantization not timed" % wl.steps})
    return out


def cpu_baseline(wl, unit):
    """The oracle, as it stands, on one host core, on a bounded sample of the same workload (~10-30 s)."""
    rows_limit, batch_limit, desc = oracle_sample_plan(wl)
    Wc, Wa = oracle_setup(wl, rows_limit)
    ins = synth.inputs(wl)
    units, t0 = 0.0, time.perf_counter()
    reps = 0
    while True:
        units += oracle_step(wl, Wc, Wa, ins, batch_limit)
        reps += 1
        if time.perf_counter() - t0 > 10.0 or reps >= 200:
            break
    dt = time.perf_counter() - t0
    return {"value": units / dt, "unit": unit, "cores": 1, "kind": "oracle",
            "sample": "%d x %s; fp64, single thread; weight quantization not timed" % (reps, desc)}


def run_phase_timing(args, wl):
    """Per-phase SM clocks per timestep of the batch-1 sequence kernel (first and last CTA), from a build of the library
    with AMQ_PHASE_TIMING defined: phases = gather (x loads + waiting for the other CTAs' h), on-line quantizer,
    packing + barrier, product + gates + publish (thread 0, whose warp owns the CTA's first hidden unit)."""
    from paper_1802_00150_b200 import build
    lib = build.build(defines=["AMQ_PHASE_TIMING"], lib_name="libamq_b200_phase.so")
    os.environ["AMQ_B200_LIBRARY"] = lib
    import torch
    from paper_1802_00150_b200 import amq
    assert wl.batch == 1 and wl.cell in ("lstm", "gru"), "the phase counters are in the batch-1 sequence kernel"
    if wl.steps == 1:
        wl = synth.scaled(wl, steps=35)
    dev = torch.device("cuda", 0)
    Wcodes, Walpha = amq.quantize(torch.from_numpy(synth.weights(wl)).to(dev), wl.k_w, wl.T)
    ins = synth.inputs(wl)
    x_seq = torch.from_numpy(ins["x_seq"]).to(dev)
    h0, c0 = torch.from_numpy(ins["h0"]).to(dev), torch.from_numpy(ins["c0"]).to(dev)
    ws = amq.new_workspace(wl.I, wl.H, 1, wl.k_a)
    for _ in range(max(args.warmup, 3)):
        if wl.cell == "lstm":
            amq.lstm_sequence(Wcodes, Walpha, None, wl.I, wl.H, x_seq, h0, c0, wl.k_a, wl.T, ws)
        else:
            amq.gru_sequence(Wcodes, Walpha, None, wl.I, wl.H, x_seq, h0, wl.k_a, wl.T, ws)
    torch.cuda.synchronize()
    words = ws.cpu().numpy().view(np.uint32)
    names = ["gather", "quantize", "pack", "product_gates_publish"]
    print(json.dumps({"workload": wl.name, "timesteps": wl.steps, "unit": "SM clocks per timestep, thread 0",
                      "first_cta": dict(zip(names, (int(v) for v in words[8:12]))),
                      "last_cta": dict(zip(names, (int(v) for v in words[16:20]))),
                      "sum_first_cta": int(words[8:12].sum())}))


def main():
    args = parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.phase_timing:
        run_phase_timing(args, wl)
        return
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the ROCKET transform hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one hard transform (PPV + max) of the paper-scale batch: 60 examples x 20 channels x
50,000 steps through 10,000 random kernels, the workload the metric is quoted on.  The same run
also times the soft forward and the soft backward on the training-pass shape (32 examples) and
reports them under "passes".  Prints ONE JSON line on rank 0.

Multi-GPU: (example, kernel) pairs are independent, so ranks each transform their own batch of
60 examples (weak scaling, no data-path collective); torch.distributed is used for the barrier
and the max-over-ranks of the timings only.
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

METRIC = "ROCKET transform examples/s at 20ch x 50k, 10k kernels; % of FP32 FMA peak"
UNIT = "examples/s"
WORKLOAD = dict(N=60, C=20, L=50000, K=10000)        # paper-scale inference batch
TRAIN = dict(N=32, C=20, L=50000, K=10000)           # soft forward + backward shape
PARAM_SEED, DATA_SEED, GRAD_SEED = 8527, 2301, 527
LAMBDA, SHIFT = 10.0, 3.0

MINI_FEATURES = 9996          # MINIROCKET's default 10,000 rounded down to a multiple of its 84 kernels
# DRAM bytes (read + write) of one launch of either fused kernel, from the committed ncu capture (profiles/),
# per launch = one chunk of 12 examples.  The figures belong to one state of the kernel sources: they are
# reported only while the digest of those sources still equals NCU_SOURCES_DIGEST, and as null otherwise.
NCU_DRAM_BYTES_PER_LAUNCH = {"fast_s_forward": 55.9e6, "fast_t_forward": 311.5e6}
NCU_SOURCES_DIGEST = "7353b8ccfa8d2918"
KERNEL_SOURCES = ("rocket_fast_fwd.cu", "rocket_fast.h", "rocket_fast_geom.h", "rocket_plan.cpp")


def kernel_sources_digest():
    """Digest of the sources that decide what the fused kernels read and write."""
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2301_08527_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_fma_peak():
    """FMA rate of dependent register chains on this device (scalar and packed two-wide fp32, packed fp16),
    measured with the benchmark-only helper library; None when it cannot run."""
    import ctypes
    try:
        from paper_2301_08527_b200.build import build_bench_helper
        lib = ctypes.CDLL(build_bench_helper())
        a, b = ctypes.c_double(0.0), ctypes.c_double(0.0)
        if lib.fma_peak_measure(ctypes.byref(a), ctypes.byref(b)) != 0:
            return None
        res = {"scalar_fma_tflops": a.value, "packed_fma_tflops": b.value}
        h = ctypes.c_double(0.0)
        if lib.fma_peak_measure_f16x2(ctypes.byref(h)) == 0:
            res["packed_f16_fma_tflops"] = h.value      # fma.rn.f16x2: what a half-precision inner loop could reach
        return res
    except Exception:
        return None


def run_gemm_probe():
    """The transform of one dilation as a GEMM: Z[kernels][positions] = W'[kernels][K] X_d[K][positions] with the
    weights of every kernel laid out on a common grid of 11 centred taps x 24 channel slots (K = 264), of which a
    kernel fills 31.6 on average.  Times the library GEMM (fp32, tf32, bf16 inputs) for bucket sizes M and reports
    dense and useful TFLOP/s; an upper bound for a tensor-core form, which would also have to build X_d (every
    channel row 11 times, shifted) and pool the outputs."""
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device")
    K, N = 264, 600000                       # 12 examples x 50,000 positions
    useful = 31.6 / K
    rows = []
    for M in (64, 128, 256, 768):
        for name, dtype, tf32 in (("fp32", torch.float32, False), ("tf32", torch.float32, True), ("bf16", torch.bfloat16, False)):
            torch.backends.cuda.matmul.allow_tf32 = tf32
            A = torch.randn(M, K, device="cuda", dtype=dtype)
            B = torch.randn(K, N, device="cuda", dtype=dtype)
            C = torch.empty(M, N, device="cuda", dtype=dtype)
            for _ in range(3):
                torch.matmul(A, B, out=C)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(10):
                torch.matmul(A, B, out=C)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 10
            dense = 2.0 * M * N * K / ms / 1e9
            rows.append({"M": M, "inputs": name, "ms": ms, "dense_tflops": dense, "useful_tflops": dense * useful,
                         "useful_tflops_three_products": dense * useful / 3})
            del A, B, C
    torch.backends.cuda.matmul.allow_tf32 = False
    print(json.dumps({"probe": "library GEMM, zero-padded dense-channel formulation", "K": K, "N": N,
                      "useful_share_of_K": useful, "rows": rows}))


def fp32_peak_tflops(sm_count, sm_mhz):
    """FP32 FMA peak: SMs x 128 lanes x 2 flop x clock."""
    return sm_count * 128 * 2 * sm_mhz * 1e6 / 1e12


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.thread.join(timeout=2)
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value, world, device="cuda"):
    """Max of a python float over the ranks of the default process group (identity for one rank)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(examples_per_rank, steps, seconds_max_over_ranks, world):
    """Whole-job throughput: every rank transforms its own batch (weak scaling), the slowest rank sets the time."""
    return world * examples_per_rank * steps / seconds_max_over_ranks


def run_reference(args, rank):
    """The CPU oracle, as it stands, on the machine's host cores: a bounded sample of the workload per step."""
    if rank != 0:
        return
    import oracle
    from rocket_inputs import ar1_spike_series, generate_kernels
    w = WORKLOAD
    kp = generate_kernels(PARAM_SEED, w["K"], w["C"], w["L"])
    X = ar1_spike_series(DATA_SEED, 1, w["C"], w["L"])
    ks = np.sort(np.random.default_rng(1).choice(w["K"], args.ref_kernels, replace=False)).astype(np.int32)
    pn = np.zeros(len(ks), np.int32)
    # an example costs sum_k flops(k); the sample's share of that cost scales its time to one example
    flops_k = 2.0 * kp.length * kp.num_channels * kp.out_len
    share = flops_k[ks].sum() / flops_k.sum()
    oracle.forward_pairs(kp, X, pn[:8], ks[:8])
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oracle.forward_pairs(kp, X, pn, ks)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    per_example = float(np.mean(times)) / share
    value = 1.0 / per_example
    cores = oracle.num_threads()
    sample = "1 example x %d of %d kernels per step (%.2f%% of an example's conv flop), scaled by flop share" % (
        len(ks), w["K"], 100 * share)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "N=60 x C=20 x L=50000, K=10000 multivariate kernels, hard PPV + max (config 2)",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(kp, X, seconds_budget=15.0):
    """Times the oracle on a bounded sample of the workload (rank 0, N=1 only): whole examples,
    every kernel, as many examples as fit the time budget."""
    import oracle
    K = kp.K
    ks = np.arange(K, dtype=np.int32)
    t0 = time.perf_counter()
    oracle.forward_pairs(kp, X[:1], np.zeros(K, np.int32), ks)
    t1 = time.perf_counter() - t0
    E = int(np.clip(round(seconds_budget / max(t1, 1e-3)), 1, X.shape[0]))
    pn = np.repeat(np.arange(E, dtype=np.int32), K)
    pk = np.tile(ks, E)
    t0 = time.perf_counter()
    oracle.forward_pairs(kp, X[:E], pn, pk)
    dt = time.perf_counter() - t0
    return {"value": E / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "%d whole examples x all %d kernels in %.1f s (fp64 definition, OpenMP over pairs)" % (E, K, dt)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--ref-kernels", type=int, default=2000, help="kernels per step of the reference arm's sample")
    ap.add_argument("--skip-passes", action="store_true", help="skip the soft forward / backward timings")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="time the whole throughput sweep (config 4: 24 points, three timed "
                    "calls each) on rank 0 instead of its time-boxed default (12 points, one timed call each)")
    ap.add_argument("--skip-sweep", action="store_true", help="skip the throughput sweep")
    ap.add_argument("--small", action="store_true", help="profiling case: N=12 examples, one launch of either fused kernel")
    ap.add_argument("--profile-pass", choices=["soft", "backward", "minirocket", "f16"], default=None,
                    help="profiling case: run only that pass (config 3's soft forward or backward, the MINIROCKET "
                         "transform with 9,996 features, or the hard transform in half precision) on 12 examples, "
                         "three times, and exit")
    ap.add_argument("--gemm-probe", action="store_true",
                    help="measure what a library GEMM makes of the zero-padded dense-channel formulation of the transform "
                         "(a reference measurement for the design notes: the transform itself never calls a GEMM) and exit")
    args = ap.parse_args()

    if args.gemm_probe:
        run_gemm_probe()
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2301_08527_b200 as rk
    from paper_2301_08527_b200 import binding
    from rocket_inputs import ar1_spike_series, generate_kernels, normal_array

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the transform has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over(v):
        return max_over_ranks(v, world)

    w = dict(WORKLOAD)
    if args.small:
        w["N"] = 12
    props = torch.cuda.get_device_properties(local_rank)
    params = rk.RocketParams.generate(PARAM_SEED, w["K"], w["C"], w["L"])
    flops_ex, outputs_ex = params.work()

    # each rank owns its own batch (weak scaling): different data seed per rank
    X_host = torch.from_numpy(ar1_spike_series(DATA_SEED + 1000 * rank, w["N"], w["C"], w["L"])).pin_memory()
    X = X_host.cuda()
    feat = torch.empty((w["N"], 2 * w["K"]), dtype=torch.float32, device="cuda")
    feat_host = torch.empty((w["N"], 2 * w["K"]), dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()

    if args.profile_pass:
        # one launch of either fused kernel per call: the case the ncu captures of the soft forward and
        # of the backward use
        Xs = X[:12].contiguous()
        if args.profile_pass == "minirocket":
            mr = rk.MiniRocket.create(PARAM_SEED, w["C"], w["L"], MINI_FEATURES)
            mr.fit(X_host[:12].numpy())
            mfeat = mr.transform(Xs)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(2):
                mr.transform(Xs, out=mfeat)
            e1.record()
            torch.cuda.synchronize()
            print(json.dumps({"pass": "minirocket", "shape": "N=12 x C=%d x L=%d, %d features" % (w["C"], w["L"], MINI_FEATURES),
                              "ms": e0.elapsed_time(e1) / 2}))
            return
        if args.profile_pass == "f16":
            hfeat = rk.rocket_transform_f16(params, Xs)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(2):
                rk.rocket_transform_f16(params, Xs, out=hfeat)
            e1.record()
            torch.cuda.synchronize()
            print(json.dumps({"pass": "f16", "shape": "N=12 x C=%d x L=%d, K=%d" % (w["C"], w["L"], w["K"]),
                              "ms": e0.elapsed_time(e1) / 2}))
            return
        sfeat, arg = rk.rocket_transform_soft(params, Xs, LAMBDA, SHIFT)
        g = torch.from_numpy(normal_array(GRAD_SEED, (12, 2 * w["K"]))).cuda()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(3):
            if i == 2:
                e0.record()
            if args.profile_pass == "soft":
                rk.rocket_transform_soft(params, Xs, LAMBDA, SHIFT, out=sfeat, argmax_out=arg)
            else:
                rk.rocket_transform_soft_backward(params, Xs, LAMBDA, SHIFT, g, arg)
        e1.record()
        torch.cuda.synchronize()
        print(json.dumps({"pass": args.profile_pass, "shape": "N=12 x C=%d x L=%d, K=%d" % (w["C"], w["L"], w["K"]),
                          "ms": e0.elapsed_time(e1)}))
        return

    def time_steps(fn, steps, warmup, after_step=None):
        """CUDA-event time of `steps` calls on the launching stream, after `warmup` calls; seconds."""
        for _ in range(warmup):
            fn()
        barrier()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        evs[0].record(stream)
        for i in range(steps):
            fn()
            evs[i + 1].record(stream)
            if after_step:
                after_step()
        barrier()
        per = [evs[i].elapsed_time(evs[i + 1]) * 1e-3 for i in range(steps)]
        return evs[0].elapsed_time(evs[-1]) * 1e-3, per

    fma_peak = measured_fma_peak() if rank == 0 else None
    sampler = ClockSampler(local_rank) if rank == 0 else None
    launches0 = rk.kernel_launch_count()
    if sampler:
        sampler.start()
    # the library records events on this stream around its two fused kernels; read them after every step
    params.set_profiling(True)
    kernel_ms = []
    total_s, per_step = time_steps(lambda: rk.rocket_transform(params, X, out=feat), args.steps, args.warmup,
                                   after_step=lambda: kernel_ms.append(params.last_profile()))
    params.set_profiling(False)
    clocks = sampler.stop() if sampler else None
    launches = rk.kernel_launch_count() - launches0
    launches_timed = launches * args.steps // (args.steps + args.warmup)
    # one transform = init + per chunk of the batch (shifted copies, small-dilation kernel, large-dilation
    # kernel) + finalise: the number of launches of either fused kernel per step follows from the count
    chunk_launches = max(1, (launches // (args.steps + args.warmup) - 2) // 3)
    total_s = max_over(total_s)
    ms_per_step = 1e3 * total_s / args.steps
    value = whole_job_value(w["N"], args.steps, total_s, world)

    # end to end through the host-buffer entry point: H2D of X and D2H of the features inside the timing
    def e2e_step():
        binding.rocket_transform_host(params, X_host, feat_host)
    for _ in range(2):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    e2e_steps = max(3, args.steps // 2)
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = max_over(time.perf_counter() - t0)
    e2e = {"value": world * w["N"] * e2e_steps / e2e_s, "unit": UNIT,
           "h2d_bytes_per_step": X_host.numel() * 4, "d2h_bytes_per_step": feat_host.numel() * 4,
           "steps": e2e_steps, "api": "rocket_transform_host (pinned host buffers)"}

    # roofline of the dominant kernel (the one of the two fused kernels that takes longer): its own
    # algorithmic flop (2*len*channels*L_out over the kernels it serves, times the batch) over its own
    # launch duration, both from the library's events on the launching stream during the timed steps
    ms_s = float(np.mean([k["ms_small_dilations"] for k in kernel_ms]))
    ms_t = float(np.mean([k["ms_large_dilations"] for k in kernel_ms]))
    fl_s, fl_t = kernel_ms[-1]["flops_small_dilations"], kernel_ms[-1]["flops_large_dilations"]
    dom = "fast_t_forward (dilations >= 64)" if ms_t >= ms_s else "fast_s_forward (dilations < 64)"
    dom_ms, dom_fl = (ms_t, fl_t) if ms_t >= ms_s else (ms_s, fl_s)
    achieved = dom_fl * w["N"] / (dom_ms * 1e-3) / 1e12 if dom_ms > 0 else 0.0
    step_tflops = flops_ex * w["N"] / float(np.mean(per_step)) / 1e12
    peaks = measured_peaks()
    sm_max = (peaks or {}).get("sm_max_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
    peak = fp32_peak_tflops(props.multi_processor_count, sm_max)
    traffic_valid = kernel_sources_digest() == NCU_SOURCES_DIGEST
    roofline = {"bound": "alu", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak,
                "traffic": NCU_DRAM_BYTES_PER_LAUNCH.get(dom.split()[0]) if traffic_valid else None,
                "launch_ms": dom_ms, "launches_per_step": chunk_launches,
                "traffic_note": ("ncu, cold cache, one launch = one chunk of 12 examples (48 MB of input)" if traffic_valid else
                                 "null: the kernel sources changed since the committed ncu capture"),
                "peak_source": "derived: %d SMs x 128 FP32 lanes x 2 flop x %.0f MHz (max SM clock from %s)" % (
                                   props.multi_processor_count, sm_max,
                                   "MEASURED_PEAKS.json" if peaks else "nvidia-smi / nominal"),
                "flop_count": "2*len*channels*L_out per kernel per example; whole path %.4g flop/example, "
                              "this kernel %.4g" % (flops_ex, dom_fl),
                "kernels": {"fast_s_forward": {"ms": ms_s, "tflops": fl_s * w["N"] / (ms_s * 1e-3) / 1e12 if ms_s else None},
                            "fast_t_forward": {"ms": ms_t, "tflops": fl_t * w["N"] / (ms_t * 1e-3) / 1e12 if ms_t else None}},
                "whole_step_tflops": step_tflops, "whole_step_frac": step_tflops / peak,
                "pooling_ops_per_example": 2.0 * outputs_ex}
    # the three denominators: lanes x maximum clock (peak / frac above), lanes x the clock observed during the timed
    # steps, and the FMA rate a register-only chain microbenchmark reaches on this device in this run
    if clocks and clocks.get("sm_mhz"):
        roofline["frac_at_observed_clock"] = achieved / fp32_peak_tflops(props.multi_processor_count, clocks["sm_mhz"])
    if fma_peak:
        roofline["fma_microbenchmark"] = fma_peak
        if fma_peak["packed_fma_tflops"] > 0:
            roofline["frac_of_packed_fma_microbenchmark"] = achieved / fma_peak["packed_fma_tflops"]
            roofline["whole_step_frac_of_packed_fma_microbenchmark"] = step_tflops / fma_peak["packed_fma_tflops"]

    passes = None
    if not args.skip_passes and not args.small:
        t = TRAIN
        Xt = X[: t["N"]]
        g = torch.from_numpy(normal_array(GRAD_SEED, (t["N"], 2 * t["K"]))).cuda()
        sfeat = torch.empty((t["N"], 2 * t["K"]), dtype=torch.float32, device="cuda")
        arg = torch.empty((t["N"], t["K"]), dtype=torch.int32, device="cuda")
        dW = torch.empty((params.n_weights,), dtype=torch.float32, device="cuda")
        db = torch.empty((t["K"],), dtype=torch.float32, device="cuda")
        psteps = max(2, args.steps // 3)
        soft_by_lambda = {}
        for lam in (1.0, 10.0, 100.0):     # config 3 sweeps the temperature; LAMBDA is the one quoted below
            sl, _ = time_steps(lambda: rk.rocket_transform_soft(params, Xt, lam, SHIFT, out=sfeat, argmax_out=arg), psteps, 3)
            soft_by_lambda[lam] = max_over(sl) / psteps
        s_soft, _ = time_steps(lambda: rk.rocket_transform_soft(params, Xt, LAMBDA, SHIFT, out=sfeat, argmax_out=arg),
                               psteps, 3)
        s_bwd, _ = time_steps(lambda: rk.rocket_transform_soft_backward(params, Xt, LAMBDA, SHIFT, g, arg, dW, db),
                              psteps, 3)
        s_soft, s_bwd = max_over(s_soft) / psteps, max_over(s_bwd) / psteps
        # the hard transform from raw 8-bit intensities (per-channel scaling fused into the staging copy):
        # headline shape, device-resident bytes, and end to end from pinned host bytes
        from rocket_inputs import channel_statistics, intensity_series_u8
        X8_host = torch.from_numpy(intensity_series_u8(DATA_SEED + 1 + 1000 * rank, w["N"], w["C"], w["L"])).pin_memory()
        mean8, istd8 = channel_statistics(X8_host.numpy()[:4])
        X8 = X8_host.cuda()
        s_u8, _ = time_steps(lambda: rk.rocket_transform_u8(params, X8, mean8, istd8, out=feat), psteps, 3)
        s_u8 = max_over(s_u8) / psteps
        for _ in range(2):
            binding.rocket_transform_u8_host(params, X8_host, mean8, istd8, feat_host)
        barrier()
        t0 = time.perf_counter()
        for _ in range(psteps):
            binding.rocket_transform_u8_host(params, X8_host, mean8, istd8, feat_host)
        barrier()
        s_u8_e2e = max_over(time.perf_counter() - t0) / psteps
        del X8
        # the regressor on the features (Section 3.3): fit at the size of the paper's training set, predict on
        # the features of the timed batch
        rngr = np.random.default_rng(GRAD_SEED)
        Fr = torch.from_numpy(rngr.random((677, 2 * w["K"]), dtype=np.float32)).cuda()
        yr = torch.from_numpy((0.6 + 1.2 * rngr.random(677)).astype(np.float32)).cuda()
        rk.rocket_ridge_fit(Fr, yr, 1.0)
        torch.cuda.synchronize()
        s_fit = float("inf")
        for _ in range(2):
            t0 = time.perf_counter()
            wr, br = rk.rocket_ridge_fit(Fr, yr, 1.0)     # returns after its work has finished
            s_fit = min(s_fit, time.perf_counter() - t0)
        yhat = torch.empty((w["N"],), dtype=torch.float32, device="cuda")
        s_pred, _ = time_steps(lambda: rk.rocket_ridge_predict(feat, wr, br, out=yhat), 5, 3)
        s_pred /= 5
        del Fr
        # the hard transform in half precision (Section 5: FP16 compute), device-resident input
        s_f16, _ = time_steps(lambda: rk.rocket_transform_f16(params, X, out=feat), psteps, 3)
        s_f16 = max_over(s_f16) / psteps
        # MINIROCKET on the same batch (Section 2; Section 6, last sentence): host fit, then the fused transform
        mr = rk.MiniRocket.create(PARAM_SEED, w["C"], w["L"], MINI_FEATURES)
        t0 = time.perf_counter()
        mr.fit(X_host.numpy()[:16])
        s_mfit = time.perf_counter() - t0
        mfeat = mr.transform(X)
        s_mini, _ = time_steps(lambda: mr.transform(X, out=mfeat), psteps, 3)
        s_mini = max_over(s_mini) / psteps
        mr.close()
        del mfeat
        passes = {
            "hard_f16": {"shape": "N=%d x C=%d x L=%d, K=%d, binary16 arithmetic" % (w["N"], w["C"], w["L"], w["K"]),
                         "examples_per_s": world * w["N"] / s_f16, "ms": 1e3 * s_f16,
                         "conv_tflops": flops_ex * w["N"] / s_f16 / 1e12},
            "minirocket": {"shape": "N=%d x C=%d x L=%d, %d features" % (w["N"], w["C"], w["L"], MINI_FEATURES),
                           "examples_per_s": world * w["N"] / s_mini, "ms": 1e3 * s_mini, "host_fit_s": s_mfit},
            "ridge": {"fit_ms": 1e3 * s_fit, "fit_shape": "677 examples x %d features, alpha=1" % (2 * w["K"]),
                      "predict_ms": 1e3 * s_pred, "predict_shape": "%d examples x %d features" % (w["N"], 2 * w["K"])},
            "hard_u8": {"shape": "N=%d x C=%d x L=%d uint8, K=%d" % (w["N"], w["C"], w["L"], w["K"]),
                        "examples_per_s": world * w["N"] / s_u8, "ms": 1e3 * s_u8,
                        "e2e_examples_per_s": world * w["N"] / s_u8_e2e, "h2d_bytes_per_step": X8_host.numel()},
            "shape": "N=32 x C=20 x L=50000, K=10000 (config 3), lambda=%g, shift=%g" % (LAMBDA, SHIFT),
            "soft_forward": {"examples_per_s": world * t["N"] / s_soft, "ms": 1e3 * s_soft,
                             "conv_tflops": flops_ex * t["N"] / s_soft / 1e12,
                             "by_lambda": {"%g" % lam: {"ms": 1e3 * v, "examples_per_s": world * t["N"] / v,
                                                        "conv_tflops": flops_ex * t["N"] / v / 1e12}
                                           for lam, v in soft_by_lambda.items()}},
            "soft_backward": {"examples_per_s": world * t["N"] / s_bwd, "ms": 1e3 * s_bwd,
                              "conv_tflops": 2 * flops_ex * t["N"] / s_bwd / 1e12,
                              "flop_count": "4*len*channels*L_out (recompute z + dW)"},
        }

    sweep = None
    if rank == 0 and not args.skip_sweep and not args.small:
        # config 4: hard transform, N in {1, 8, 60, 256} x L in {10k, 50k, 200k} x K in {10k, 50k}; N = 1 is the
        # streaming latency.  Inputs: eight generated examples per L, repeated up to N.  By default a time-boxed
        # subset (N in {1, 60}, one timed call after one warm-up); --sweep times every point three times.
        sweep = []
        batch_sizes, timed, warm = ((1, 8, 60, 256), 3, 2) if args.sweep else ((1, 60), 1, 1)
        for L4 in (10000, 50000, 200000):
            X8 = torch.from_numpy(ar1_spike_series(DATA_SEED, 8, 20, L4)).cuda()
            for K4 in (10000, 50000):
                p4 = rk.RocketParams.generate(PARAM_SEED, K4, 20, L4)
                fl4, _ = p4.work()
                for N4 in batch_sizes:
                    X4 = X8.repeat((N4 + 7) // 8, 1, 1)[:N4].contiguous()
                    f4 = torch.empty((N4, 2 * K4), dtype=torch.float32, device="cuda")
                    t4, _ = time_steps(lambda: rk.rocket_transform(p4, X4, out=f4), timed, warm)
                    t4 /= timed
                    sweep.append({"N": N4, "L": L4, "K": K4, "ms": 1e3 * t4, "examples_per_s": N4 / t4,
                                  "conv_tflops": fl4 * N4 / t4 / 1e12, "timed_calls": timed})
                    del X4, f4
                p4.close()
            del X8

    cpu = None
    if rank == 0 and world == 1 and not args.skip_cpu_baseline:
        kp = generate_kernels(PARAM_SEED, w["K"], w["C"], w["L"])
        cpu = cpu_baseline(kp, X_host.numpy())

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "N=%d x C=%d x L=%d fp32, K=%d multivariate kernels, hard PPV + max (config 2)%s" % (
                           w["N"], w["C"], w["L"], w["K"], " [reduced N for profiling]" if args.small else ""),
                       "examples_per_gpu": w["N"], "l2": "inputs larger than L2 (%.0f MB per batch)" % (
                           X_host.numel() * 4 / 1e6), "timing": "CUDA events on the launching stream",
                       "seeds": {"params": PARAM_SEED, "data": DATA_SEED}},
            "conv_tflops": step_tflops, "pct_fp32_peak": 100 * step_tflops / peak,
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_timed,
            "clocks": clocks, "passes": passes,
        }
        if sweep is not None:
            line["sweep"] = sweep
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

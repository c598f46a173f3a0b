#!/usr/bin/env python
"""Benchmark of the low-bit tensor-parallel synchronisation hot path on B200.

One "step" = one synchronisation of the Llama-2-13B-shaped prefill workload
(BASELINE config 2): N = 4 simulated tensor-parallel shards, 2048 tokens x 5120
features of BF16 partial sums each; the 4 shards are quantised and packed
(tpq_quantize_pack_batch: one launch, the SMs divided among the shards; the
per-shard tpq_quantize_pack is timed too, under "extra"), then one
tpq_dequant_reduce (BF16 output) over the 4 payloads.  The static parameters
(calibration + feature selection) are computed once before the timed region,
as in the method (they never change at inference time); their throughput is
reported separately under "extra".

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Metric: GB/s of BF16 input processed (N*T*E*2 bytes per step), whole job.
N > 1 GPUs (torchrun): every rank runs the same workload on its own batch, no
data-path collective (replicas of the single-GPU simulation): weak scaling.

--impl reference times the CPU oracle (oracle/, scalar C + OpenMP) on the host
cores on the same workload; there is no other reference implementation.
"""
from __future__ import annotations

import argparse
import dataclasses
import ctypes
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

METRIC = "quantize_pack + dequant_reduce GB/s (BF16 input)"
UNIT = "GB/s"
WORKLOAD = "llama13b_prefill"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (None until a capture exists for the current kernel).
NCU_TRAFFIC_BYTES = {
    "quantize_tiled": {"bytes": 21025024, "capture": "profiles/dram_traffic_llama13b_prefill.md"},
    "quantize_tiled_batch": {"bytes": 84600000, "capture": "profiles/dram_traffic_llama13b_prefill.md"},
    "dequant_rows": {"bytes": 22106624, "capture": "profiles/dram_traffic_llama13b_prefill.md"},
}


# ------------------------------------------------------------------ helpers
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Dense BF16 TFLOP/s of the library GEMM on this machine (burst figure: the fused layer is timed alone)."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["bf16_tflops"]), "measured"
    except Exception:
        return 1590.0, "fallback"


def payload_bytes(T, E, k, bits=4):
    nbits = T * (E - k) * bits
    return ((nbits + 7) // 8 + 15) // 16 * 16 + 2 * T * k


def algorithmic_bytes(N, T, E, k, bits=4):
    """Bytes the method itself must move per launch (tables are O(N*E) and cache resident)."""
    P = payload_bytes(T, E, k, bits)
    return {"quantize_pack": 2 * T * E + P, "dequant_reduce": N * P + 2 * T * E}


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for ts, r in self.rows if ts >= t0 - 0.05]      # timed region and the per-kernel loops after it
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        region = []
        for ts, r in self.rows:
            if t0 <= ts <= t1:
                try:
                    region.append(float(r.split(",")[1]))
                except (ValueError, IndexError):
                    pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "sm_mhz_in_timed_region": statistics.median(region) if region else None,
                "power_w_max": max(power) if power else None, "samples": len(sm),
                "samples_in_timed_region": len(region), "reasons": sorted(reasons)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate_over_ranks(local_ms: float, local_units: float, dist=None):
    """max over ranks of the step time, sum over ranks of the units one step processes."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return local_ms, local_units
    import torch

    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([local_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([local_units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


# ------------------------------------------------------------------ the CPU oracle leg
def oracle_leg(w, steps: int, warmup: int):
    """Times the oracle as it stands on one full-size step; returns (GB/s, ms_per_step, cores, sample)."""
    import oracle
    from paper_2411_07942_b200 import synth

    orc = oracle.c()
    N, T, E = w.n_shards, w.tokens, w.features
    scale = synth.column_scales(w)
    cal = [synth.calibration_np(w, i, n_seq=2, tokens=256, scale=scale) for i in range(N)]
    ms, Ms = [], []
    for i in range(N):
        m, M, _ = orc.calibrate(None, None, 0, cal[i], 0.01)
        ms.append(m)
        Ms.append(M)
    R, Rbar = orc.ranges(np.stack(ms), np.stack(Ms))
    hp = orc.select(Rbar, orc.default_k(E))
    s, inv = orc.params(R)
    ys = [synth.activations_np(w, i, T, scale=scale) for i in range(N)]

    def step():
        pl = [orc.quantize_pack(ys[i], hp, inv[i]) for i in range(N)]
        orc.dequant_reduce(pl, T, E, hp, s, want_chain32=True)

    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    gbs = N * T * E * 2 / dt / 1e9
    sample = f"{steps} full steps of {w.name} (N={N}, {T}x{E} BF16 per shard), scalar C oracle, OpenMP over rows"
    return gbs, dt * 1e3, orc.num_threads(), sample


# ------------------------------------------------------------------ the other configurations (extra.configs)
def other_configs(args, dev, stream, peak, time_loop, graph_loop):
    """Config 3 (decode shape: latency, plain launches and graph replay), config 5 at 8192 tokens, config 2's
    shape with 8 shards, and the calibration pass of config 4 on 32 sequences of one shard; the same kernels,
    timed the same way."""
    import torch
    from paper_2411_07942_b200 import binding, synth

    sh = stream.cuda_stream
    out = {}

    def build(wname, n_sets):
        w = wname if isinstance(wname, synth.Workload) else synth.WORKLOADS[wname]
        N, T, E = w.n_shards, w.tokens, w.features
        scale = synth.column_scales(w)
        t = binding.Tpq(N, E)
        for i in range(N):
            cal = synth.activations_torch(w, i, 2 * 64, dev, stream=1, scale=scale)
            t.calibrate_ranges(i, cal.data_ptr(), 2, 64, stream=sh)
        torch.cuda.synchronize()
        k = len(t.select_features(-1))
        P = t.payload_bytes(T)
        sets = []
        for b in range(n_sets):
            ys = [synth.activations_torch(w, i, T, dev, stream=2 + b, scale=scale) for i in range(N)]
            pls = [torch.empty(P, dtype=torch.uint8, device=dev) for _ in range(N)]
            o = torch.empty((T, E), dtype=torch.bfloat16, device=dev)
            sets.append((ys, pls, o, (ctypes.c_void_p * N)(*[y.data_ptr() for y in ys]),
                         (ctypes.c_void_p * N)(*[p_.data_ptr() for p_ in pls])))
        return w, t, k, P, sets

    def timed(wname, n_sets, with_graph):
        w, t, k, P, sets = build(wname, n_sets)
        N, T, E = w.n_shards, w.tokens, w.features
        alg = algorithmic_bytes(N, T, E, k)
        cnt = [0]

        def q_one(b, s_=None):          # one shard per call, the shards in turn
            ys, pls, _, _, _ = sets[b % n_sets]
            i = (b // n_sets) % N
            t.quantize_pack(i, ys[i].data_ptr(), T, pls[i].data_ptr(), P, stream=sh if s_ is None else s_)

        def q_all(b, s_=None):
            _, _, _, yarr, parr = sets[b % n_sets]
            t.quantize_pack_batch(0, yarr, T, parr, P, stream=sh if s_ is None else s_)

        def d_one(b, s_=None):
            _, _, o, _, parr = sets[b % n_sets]
            t.dequant_reduce(parr, T, o.data_ptr(), binding.TPQ_OUT_BF16, stream=sh if s_ is None else s_)

        def st(b, s_=None):
            q_all(b, s_)
            d_one(b, s_)

        q_all(0)
        torch.cuda.synchronize()
        r = {"shape": f"N={N} shards x {T} tokens x {E} features, k={k}", "buffer_sets": n_sets,
             "algorithmic_bytes": {"quantize_pack": alg["quantize_pack"], "dequant_reduce": alg["dequant_reduce"]}}
        for name, fn, nbytes in (("quantize_pack", q_one, alg["quantize_pack"]),
                                 ("quantize_pack_batch", q_all, N * alg["quantize_pack"]),
                                 ("dequant_reduce", d_one, alg["dequant_reduce"]), ("step", st, None)):
            ms = time_loop(fn)
            e = {"us_per_call": ms * 1e3}
            if with_graph:
                g = graph_loop(fn, n_sets * (N if fn is q_one else 1))
                e["us_per_call_graph_replay"] = None if g is None else g * 1e3
            if nbytes:
                e["hbm_GBps"] = nbytes / ms / 1e6
                e["frac_of_measured"] = nbytes / ms / 1e6 / peak
                e["frac_of_8000"] = nbytes / ms / 1e6 / NOMINAL_HBM_GBS
            r[name] = e
        assert t.device_status() == 0
        t.close()
        del sets
        torch.cuda.empty_cache()
        return r

    out["gemma27b_decode"] = timed("gemma27b_decode", 6, True)
    out["gemma27b_decode"]["note"] = "latency-bound (0.7 MB / 1.8 MB per call): microseconds per call are the figure"
    out["large_8192_tokens"] = timed("large", 2, False)
    # the paper's tensor-parallel degree (8) on config 2's shape: the row kernel's variant for 5 to 8 devices
    import dataclasses
    out["llama13b_prefill_8_devices"] = timed(dataclasses.replace(synth.WORKLOADS["llama13b_prefill"], n_shards=8,
                                                                  name="llama13b_prefill_8_devices"), 4, False)
    # config 4: the calibration pass, 32 sequences of 2048 tokens of one shard per call (two inputs in turn)
    w = synth.WORKLOADS["calibration"]
    E, S, n_seq = w.features, w.calib_tokens, 32
    scale = synth.column_scales(w)
    bufs = [synth.activations_torch(w, 0, n_seq * S, dev, stream=1 + b, scale=scale) for b in range(2)]
    tc = binding.Tpq(w.n_shards, E)

    def cal(b):
        tc.calibrate_ranges(0, bufs[b % 2].data_ptr(), n_seq, S, stream=sh)

    ms = time_loop(cal)
    nbytes = n_seq * S * E * 2
    out["calibration_32_sequences"] = {"shape": f"{n_seq} sequences x {S} tokens x {E} features, one shard per call",
                                       "ms_per_call": ms, "bytes": nbytes, "hbm_GBps": nbytes / ms / 1e6,
                                       "frac_of_measured": nbytes / ms / 1e6 / peak,
                                       "frac_of_8000": nbytes / ms / 1e6 / NOMINAL_HBM_GBS,
                                       "full_pass_512_sequences_ms_per_shard": ms * 512 / n_seq}
    tc.close()
    del bufs
    torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="tpq", choices=["tpq", "reference"])
    ap.add_argument("--sets", type=int, default=6, help="rotating buffer sets (working set must exceed L2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-time", type=float, default=0.25,
                    help="every timed region (the K steps and each per-kernel loop) is repeated until it lasts at "
                         "least this many seconds, so that clock samples fall inside it; 0 for profiler captures")
    ap.add_argument("--no-extra-configs", action="store_true",
                    help="skip the other configurations (decode shape, large shape, calibration pass) under extra.configs")
    ap.add_argument("--workload", default=WORKLOAD,
                    help="synthetic workload (default: the configuration the metric is quoted on; the others are "
                         "for profiling captures, e.g. `--workload large --tokens 1024 --sets 2`)")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's token count")
    ap.add_argument("--shards", type=int, default=0, help="override the workload's number of shards (devices)")
    ap.add_argument("--bits", type=int, default=4, help="code width (4 = the paper's Int4 and the bench's metric; "
                                                        "2..8 run on the shape-generic kernels)")
    args = ap.parse_args()
    rank, local_rank, world = dist_env()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2411_07942_b200 import synth

    w = synth.WORKLOADS[args.workload]
    if args.tokens > 0:
        w = dataclasses.replace(w, tokens=args.tokens)
    if args.shards > 0:
        w = dataclasses.replace(w, n_shards=args.shards)
    N, T, E, k = w.n_shards, w.tokens, w.features, w.k
    in_bytes = N * T * E * 2
    config = {"workload": f"{args.workload}: N={N} shards x {T} tokens x {E} features BF16, k={k} BF16 features, "
                          f"BF16 output", "n_shards": N, "tokens": T, "features": E, "k": k}
    set_bytes = in_bytes + N * payload_bytes(T, E, k, args.bits) + 2 * T * E
    # (the same text in both arms: the GPU arm rotates its buffer sets; the CPU arm's caches are far smaller than one set)
    config["l2"] = (f"rotating {args.sets} buffer sets, {args.sets * set_bytes / 1e6:.0f} MB touched between "
                    f"reuses (> 126 MB L2)")

    if args.impl == "reference":
        if rank != 0:
            return 0
        steps = max(1, min(args.steps, 10))
        gbs, ms, cores, sample = oracle_leg(w, steps, min(args.warmup, 1))
        line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": 0, "steps": steps,
                "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
                "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    import torch
    import torch.distributed as dist

    from paper_2411_07942_b200 import binding, build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product has no CPU path")
    build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    peak, peak_kind = measured_peak()
    scale = synth.column_scales(w)
    stream = torch.cuda.current_stream()
    sh = stream.cuda_stream

    # ---- static parameters: calibration (timed separately) + selection
    t = binding.Tpq(N, E, bits=args.bits)
    cal_seqs, cal_S = 8, w.calib_tokens
    cal_bufs = [synth.activations_torch(w, i, cal_seqs * cal_S, dev, stream=1, scale=scale) for i in range(N)]
    for i in range(N):
        t.calibrate_ranges(i, cal_bufs[i].data_ptr(), cal_seqs, cal_S, stream=sh)
    torch.cuda.synchronize()
    # calibration throughput (not part of the step): a second context folds the same set a few times
    tc = binding.Tpq(N, E)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(N):
        tc.calibrate_ranges(i, cal_bufs[i].data_ptr(), cal_seqs, cal_S, stream=sh)
    torch.cuda.synchronize()
    e0.record(stream)
    cal_reps = 3
    for _ in range(cal_reps):
        for i in range(N):
            tc.calibrate_ranges(i, cal_bufs[i].data_ptr(), cal_seqs, cal_S, stream=sh)
    e1.record(stream)
    torch.cuda.synchronize()
    cal_ms = e0.elapsed_time(e1) / cal_reps
    cal_bytes = N * cal_seqs * cal_S * E * 2
    tc.close()
    ts0 = time.perf_counter()
    hp = t.select_features(-1)
    select_ms = (time.perf_counter() - ts0) * 1e3
    assert len(hp) == k
    del cal_bufs
    P = t.payload_bytes(T)
    comm = t.comm_bytes(T)
    alg = algorithmic_bytes(N, T, E, k, args.bits)

    # ---- rotating buffer sets (inputs resident in HBM; working set > L2)
    sets = []
    for b in range(args.sets):
        ys = [synth.activations_torch(w, i, T, dev, stream=2 + b, scale=scale) for i in range(N)]
        pls = [torch.empty(P, dtype=torch.uint8, device=dev) for _ in range(N)]
        out = torch.empty((T, E), dtype=torch.bfloat16, device=dev)
        yarr = (ctypes.c_void_p * N)(*[y.data_ptr() for y in ys])
        parr = (ctypes.c_void_p * N)(*[p_.data_ptr() for p_ in pls])
        sets.append((ys, pls, out, yarr, parr))

    # One step: the N simulated ranks' quantize_pack (one batched launch: the SMs are divided among the
    # N shards, as N devices would work side by side), then the local dequantise + reduce.
    def step(b):
        _, _, out, yarr, parr = sets[b % args.sets]
        t.quantize_pack_batch(0, yarr, T, parr, P, stream=sh)
        t.dequant_reduce(parr, T, out.data_ptr(), binding.TPQ_OUT_BF16, stream=sh)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for b in range(args.warmup):
        step(b)
    barrier()
    # a short pilot run (untimed work, after the warm-up) tells how long a step takes
    wa, wz = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pilot = max(args.steps, 20)
    wa.record(stream)
    for b in range(pilot):
        step(b)
    wz.record(stream)
    barrier()
    # the K steps are repeated `inner` times inside the timed region so that it lasts at least --min-time
    # (the same on every rank: rank 0's estimate from the warm-up steps is broadcast)
    est_ms = max(wa.elapsed_time(wz) / pilot, 1e-3)
    inner = max(1, int(np.ceil(1.2 * args.min_time * 1e3 / (est_ms * args.steps))))
    if world > 1:
        it_ = torch.tensor([inner], dtype=torch.int64, device=dev)
        dist.broadcast(it_, 0)
        inner = int(it_.item())
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = t.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall0 = time.time()
    ev0.record(stream)
    for b in range(args.steps * inner):
        step(b)
    ev1.record(stream)
    barrier()
    wall1 = time.time()
    local_ms = ev0.elapsed_time(ev1) / (args.steps * inner)
    gpu_launches = (t.launch_count() - launches0) // inner      # launches of the K steps

    # ---- per-kernel durations, same buffers and rotation, CUDA events on the launching stream
    def time_loop(fn, reps=None):
        """Average ms per call of fn over a loop of at least --min-time seconds (CUDA events on the stream)."""
        for b in range(3):
            fn(b)
        torch.cuda.synchronize()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 20
        a.record(stream)
        for b in range(n):
            fn(b)
        z.record(stream)
        torch.cuda.synchronize()
        est = max(a.elapsed_time(z) / n, 1e-4)
        n = max(n, int(np.ceil(args.min_time * 1e3 / est))) if reps is None else reps
        a.record(stream)
        for b in range(n):
            fn(b)
        z.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(z) / n

    def graph_loop(fn, per):
        """The same calls replayed from a CUDA graph of `per` calls: what the device needs when the host's
        launch path is out of the way.  None if capture is unavailable."""
        try:
            gs = torch.cuda.Stream()
            gs.wait_stream(stream)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=gs):
                for b in range(per):
                    fn(b, gs.cuda_stream)
            with torch.cuda.stream(gs):
                for _ in range(3):
                    g.replay()
                gs.synchronize()
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(gs)
                g.replay()
                z.record(gs)
                gs.synchronize()
                est = max(a.elapsed_time(z), 1e-4)
                n = max(3, int(np.ceil(args.min_time * 1e3 / est)))
                a.record(gs)
                for _ in range(n):
                    g.replay()
                z.record(gs)
                gs.synchronize()
            return a.elapsed_time(z) / (n * per)
        except Exception:
            torch.cuda.synchronize()
            return None

    def q_only(b, s_=None):          # one launch per shard: what each rank of a real deployment calls
        ys, pls, _, _, _ = sets[b % args.sets]
        for i in range(N):
            t.quantize_pack(i, ys[i].data_ptr(), T, pls[i].data_ptr(), P, stream=sh if s_ is None else s_)

    def qb_only(b, s_=None):         # the N shards in one launch (the step's form)
        _, _, _, yarr, parr = sets[b % args.sets]
        t.quantize_pack_batch(0, yarr, T, parr, P, stream=sh if s_ is None else s_)

    def d_only(b, s_=None):
        _, _, out, _, parr = sets[b % args.sets]
        t.dequant_reduce(parr, T, out.data_ptr(), binding.TPQ_OUT_BF16, stream=sh if s_ is None else s_)

    def step_on(b, s_):
        qb_only(b, s_)
        d_only(b, s_)

    # the sampler keeps running through the per-kernel loops below (same kernels, same buffers); each loop lasts
    # at least --min-time as well
    q_ms = time_loop(q_only) / N          # per single-shard launch
    qb_ms = time_loop(qb_only)            # per batched launch (N shards)
    d_ms = time_loop(d_only)
    # the same from a CUDA graph (one pass over the rotating buffer sets per replay): the device's own pace
    qg = graph_loop(q_only, args.sets)
    q_graph_ms = None if qg is None else qg / N
    qb_graph_ms = graph_loop(qb_only, args.sets)
    d_graph_ms = graph_loop(d_only, args.sets)
    graph_ms = graph_loop(step_on, args.sets)
    bias_dev = torch.zeros(E, dtype=torch.float32, device=dev).normal_(generator=torch.Generator(device=dev).manual_seed(7))

    def db_only(b):         # the same with the layer's bias added in the kernel's store (Section 2)
        _, _, out, _, parr = sets[b % args.sets]
        t.dequant_reduce(parr, T, out.data_ptr(), binding.TPQ_OUT_BF16, stream=sh, bias_ptr=bias_dev.data_ptr())

    db_ms = time_loop(db_only)

    # the fused exchange (Section 5) on one GPU: one shard's payload stored into 1 and into N local receive slots
    # and its arrival words published; then the bounded wait ahead of the reduction (words already set)
    words = torch.zeros(2 * N, dtype=torch.int32, device=dev)
    push_epoch = [0]

    def push_fn(n_dst):
        arrs = []
        for b in range(args.sets):
            ys, pls, _, _, _ = sets[b]
            arrs.append(((ctypes.c_void_p * n_dst)(*[pls[d].data_ptr() for d in range(n_dst)]),
                         (ctypes.c_void_p * n_dst)(*[words.data_ptr() + 4 * d for d in range(n_dst)])))

        def fn(b):
            ys, _, _, _, _ = sets[b % args.sets]
            da, aa = arrs[b % args.sets]
            for i in range(N):      # N launches per pass, like the single-shard loop above
                push_epoch[0] += 1
                t.quantize_pack_push(i, ys[i].data_ptr(), T, da, aa, P, push_epoch[0], stream=sh)
        return fn

    push_max = min(N, 16)
    p1_ms = time_loop(push_fn(1)) / N
    pn_ms = time_loop(push_fn(push_max)) / N
    words.fill_(1)
    torch.cuda.synchronize()

    def wd_only(b):
        _, _, out, _, parr = sets[b % args.sets]
        t.dequant_reduce(parr, T, out.data_ptr(), binding.TPQ_OUT_BF16, stream=sh, arrived_ptr=words.data_ptr(), epoch=1,
                         timeout_ns=50_000_000)

    wd_ms = time_loop(wd_only)

    clocks = sampler.stop(wall0, wall1) if rank == 0 else None

    # ---- (after the clock sampler has stopped: this part is tensor-bound and draws far more power than the path)
    # the layer ahead of the synchronisation point fused with the compressor (Section 2): x [T][K] times the
    # device's slice of the down projection, K = 2.7 E / N rounded to 64 (Llama's 13824 / 4 at E = 5120), against
    # the library GEMM followed by quantize_pack.  Tensor-bound; an extra, not the headline path.
    fused = None
    if args.bits == 4 and E % 8 == 0 and k % 8 == 0:
        Kd = max(64, int(round(2.7 * E / N / 64)) * 64)
        gen = torch.Generator(device=dev).manual_seed(11)
        xk = torch.randn((T, Kd), device=dev, generator=gen).to(torch.bfloat16)
        wk = (torch.randn((E, Kd), device=dev, generator=gen) / Kd ** 0.5).to(torch.bfloat16)
        wslots = torch.empty_like(wk)
        t.permute_weight(wk.data_ptr(), Kd, wslots.data_ptr(), stream=sh)
        ytmp = torch.empty((T, E), dtype=torch.bfloat16, device=dev)
        pl0 = sets[0][1][0]

        def fused_fn(b):
            t.linear_quantize_pack(0, xk.data_ptr(), wslots.data_ptr(), T, Kd, pl0.data_ptr(), P, stream=sh)

        def unfused_fn(b):
            with torch.cuda.stream(stream):
                torch.matmul(xk, wk.t(), out=ytmp)
            t.quantize_pack(0, ytmp.data_ptr(), T, pl0.data_ptr(), P, stream=sh)

        def gemm_fn(b):
            with torch.cuda.stream(stream):
                torch.matmul(xk, wk.t(), out=ytmp)

        f_ms, u_ms, g_ms = time_loop(fused_fn), time_loop(unfused_fn), time_loop(gemm_fn)
        tpeak, tkind = measured_tensor_peak()
        flops = 2.0 * T * Kd * E
        fused = {"shape": f"x [{T}][{Kd}] . w [{E}][{Kd}]^T", "fused_ms": f_ms, "fused_TFLOPs": flops / f_ms / 1e9,
                 "frac_of_" + tkind + "_bf16_peak": flops / f_ms / 1e9 / tpeak, "peak_TFLOPs": tpeak,
                 "library_gemm_then_quantize_pack_ms": u_ms, "library_gemm_alone_ms": g_ms}

    configs_extra = None
    if rank == 0 and world == 1 and not args.no_extra_configs and args.workload == WORKLOAD and not args.tokens and not args.shards and args.bits == 4:
        configs_extra = other_configs(args, dev, stream, peak, time_loop, graph_loop)

    # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timed region
    ys0 = sets[0][0]
    host_in = [torch.empty((T, E), dtype=torch.bfloat16).pin_memory() for _ in range(N)]
    for i in range(N):
        host_in[i].copy_(ys0[i])
    host_out = torch.empty((T, E), dtype=torch.bfloat16).pin_memory()

    # Every step copies its inputs up from pinned host memory, runs the path and copies the result down.
    # The read-back runs on a second stream, so the download of step b overlaps the upload of step b+1
    # (PCIe is full duplex); events keep a buffer set from being reused before its read-back is done.
    down = torch.cuda.Stream()
    ev_done = [torch.cuda.Event() for _ in range(args.sets)]
    ev_read = [torch.cuda.Event() for _ in range(args.sets)]
    used = [False] * args.sets

    def e2e_step(b):
        q = b % args.sets
        ys, _, out, yarr, parr = sets[q]
        if used[q]:
            stream.wait_event(ev_read[q])
        for i in range(N):
            ys[i].copy_(host_in[i], non_blocking=True)
        t.quantize_pack_batch(0, yarr, T, parr, P, stream=sh)
        t.dequant_reduce(parr, T, out.data_ptr(), binding.TPQ_OUT_BF16, stream=sh)
        ev_done[q].record(stream)
        with torch.cuda.stream(down):
            down.wait_event(ev_done[q])
            host_out.copy_(out, non_blocking=True)
            ev_read[q].record(down)
        used[q] = True

    e2e_reps = max(5, min(args.steps, 30))
    for b in range(3):
        e2e_step(b)
    barrier()
    a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for b in range(e2e_reps):
        e2e_step(b)
    stream.wait_stream(down)   # the last read-backs are inside the timed region
    z.record(stream)
    barrier()
    e2e_local_ms = a.elapsed_time(z) / e2e_reps
    assert t.device_status() == 0

    ms, units = aggregate_over_ranks(local_ms, float(in_bytes), dist if world > 1 else None)
    e2e_ms, _ = aggregate_over_ranks(e2e_local_ms, float(in_bytes), dist if world > 1 else None)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    value = units / (ms * 1e-3) / 1e9
    if args.bits != 4:
        config["workload"] += f", {args.bits}-bit codes"
        config["bits"] = args.bits
    default_workload = args.workload == WORKLOAD and not args.tokens and not args.shards and args.bits == 4

    def kernel_entry(name, ms_, graph_, nbytes, key):
        """One kernel's roofline entry: algorithmic bytes / measured launch time against the copy bandwidth,
        the DRAM traffic ncu saw for one launch, and which limit the kernel is at."""
        cap = NCU_TRAFFIC_BYTES.get(key) if default_workload else None   # (captured for the default workload only)
        ach = nbytes / (ms_ * 1e-3) / 1e9
        e = {"kernel": name, "launch_ms": ms_, "launch_ms_graph_replay": graph_, "algorithmic_bytes_per_launch": nbytes,
             "achieved": ach, "unit": "GB/s", "frac": ach / peak, "frac_of_nominal_8000": ach / NOMINAL_HBM_GBS,
             "traffic": cap["bytes"] if cap else None, "traffic_capture": cap["capture"] if cap else None}
        if cap:
            e["dram_GBps"] = cap["bytes"] / (ms_ * 1e-3) / 1e9
            # DRAM busy at less than half the copy rate: the launch is not limited by HBM but by instruction
            # issue and by its fixed cost (ramp, drain, dependency on the kernel ahead)
            e["bound"] = "hbm" if e["dram_GBps"] >= 0.5 * peak else "issue"
        else:
            e["bound"] = "hbm"
        return e

    kernels = [kernel_entry("quantize_pack (one shard per launch)", q_ms, q_graph_ms, alg["quantize_pack"], "quantize_tiled"),
               kernel_entry("quantize_pack_batch (N shards per launch)", qb_ms, qb_graph_ms, N * alg["quantize_pack"],
                            "quantize_tiled_batch"),
               kernel_entry("dequant_reduce", d_ms, d_graph_ms, alg["dequant_reduce"], "dequant_rows")]
    # dominant kernel of the step: the longer of its two launches
    dom = kernels[1] if qb_ms >= d_ms else kernels[2]
    roofline = {"bound": dom["bound"], "kernel": dom["kernel"], "achieved": dom["achieved"], "peak": peak, "unit": "GB/s",
                "frac": dom["frac"], "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": dom["frac_of_nominal_8000"],
                "algorithmic_bytes_per_launch": dom["algorithmic_bytes_per_launch"], "launch_ms": dom["launch_ms"],
                "traffic": dom["traffic"], "kernels": kernels}
    extra = {
        "bits_per_value": comm.bits_per_value, "bits_per_value_formula": comm.bits_per_value_formula,
        "step_cuda_graph_replay_ms": graph_ms, "inner_repeats": inner,
        "configs": configs_extra,
        "dequant_reduce_bias_ms_per_launch": db_ms,
        "fused_layer": fused,
        "exchange_one_gpu": {"quantize_pack_push_1_dst_ms": p1_ms, f"quantize_pack_push_{push_max}_dst_ms": pn_ms,
                             "dequant_reduce_arrivals_ms": wd_ms,
                             "note": "destinations are local buffers; across GPUs the stores cross NVLink"},
        "payload_bytes_per_shard": int(comm.payload_bytes),
        "comm_bytes_per_rank": {"quantized_allgather": int(comm.quantized_allgather_send),
                                "bf16_allgather": int(comm.bf16_allgather_send),
                                "bf16_ring_allreduce": int(comm.bf16_ring_allreduce_send)},
        "quantize_pack_batch": {"ms_per_launch": qb_ms, "shards_per_launch": N,
                                "hbm_GBps": N * alg["quantize_pack"] / qb_ms / 1e6,
                                "frac_of_measured": N * alg["quantize_pack"] / qb_ms / 1e6 / peak,
                                "frac_of_8000": N * alg["quantize_pack"] / qb_ms / 1e6 / NOMINAL_HBM_GBS,
                                "input_GBps": in_bytes / qb_ms / 1e6},
        "quantize_pack": {"ms_per_launch": q_ms, "hbm_GBps": alg["quantize_pack"] / q_ms / 1e6,
                          "frac_of_measured": alg["quantize_pack"] / q_ms / 1e6 / peak,
                          "frac_of_8000": alg["quantize_pack"] / q_ms / 1e6 / NOMINAL_HBM_GBS,
                          "input_GBps": 2 * T * E / q_ms / 1e6},
        "dequant_reduce": {"ms_per_launch": d_ms, "hbm_GBps": alg["dequant_reduce"] / d_ms / 1e6,
                           "frac_of_measured": alg["dequant_reduce"] / d_ms / 1e6 / peak,
                           "frac_of_8000": alg["dequant_reduce"] / d_ms / 1e6 / NOMINAL_HBM_GBS,
                           "input_GBps": in_bytes / d_ms / 1e6},
        "calibrate_ranges": {"ms": cal_ms, "bytes": cal_bytes, "hbm_GBps": cal_bytes / cal_ms / 1e6,
                             "frac_of_measured": cal_bytes / cal_ms / 1e6 / peak,
                             "shape": f"{N} shards x {cal_seqs} sequences x {cal_S} tokens x {E}"},
        "select_features_ms_incl_sync": select_ms,
    }
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "inner_repeats": inner, "timed_region_s": args.steps * inner * ms * 1e-3,
            "config": config, "clocks": clocks, "gpu_launches": int(gpu_launches),
            "e2e": {"value": world * in_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": 2 * T * E, "ms_per_step": e2e_ms},
            "roofline": roofline, "extra": extra}
    if world == 1 and not args.no_cpu_baseline:
        gbs, cms, cores, sample = oracle_leg(w, 5, 1)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                                "ms_per_step": cms}
    print(json.dumps(line))
    t.close()
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

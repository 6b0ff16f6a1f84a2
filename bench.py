#!/usr/bin/env python
"""Benchmark of the QA-LoRA linear layer on B200.

One step = one pass of the whole layer path over one batch, for both LLaMA-7B
MLP shapes (4096 -> 11008 and 11008 -> 4096, INT4, group size 32, rank 64,
M = 8192 tokens): quantize + pack, forward, backward (dX, dA, dB), merge, and
the merged layer's single-token forward.  The reported value is the forward +
backward TFLOP/s (algorithmic flops of Algorithm 1 and its gradients divided
by the time of the whole step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

The adapter gradients of both shapes land in one flat bucket that one clipped
AdamW call (Section 4.1) consumes inside the step.  With N > 1 (launched by
torch.distributed.run, one rank per GPU) every rank runs the same step on its own
batch (data parallel over tokens) and the bucket is all-reduced once over NCCL.  `--impl reference` times the CPU
oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "QA-LoRA W4 linear fwd+bwd TFLOP/s (M=8192) & M=1 GB/s, % of roofline"
WORKLOAD = "cfg3_7b_mlp_int4_g32_r64_m8192"
SHAPES = ("cfg3_7b_up", "cfg3_7b_down")
SMALL_M = "cfg2_7b_attn"


# ----------------------------------------------------------- work accounting --
# DRAM traffic of ONE launch of the forward contraction kernel at the benchmark size comes
# from the record kept beside the profile summaries (written by hand from an ncu capture,
# with the SHA-256 of the kernel's sources at the time): when the sources have changed
# since, the counters no longer describe the kernel and the bench reports null.
TRAFFIC_RECORD = os.path.join(ROOT, "profiles", "qalora_tc_kernel_fwd_cfg3_up_m8192_dram_traffic.txt")
KERNEL_SOURCES = ("gemm_tc.cu", "ptx.cuh", "common.cuh", "dequant.cuh", "debug.cuh")


def kernel_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2309_14717_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def fwd_kernel_dram_traffic():
    """(bytes per launch or None, note) from the traffic record, valid only for unchanged sources."""
    try:
        rec = dict(line.split(":", 1) for line in open(TRAFFIC_RECORD).read().splitlines() if ":" in line)
        rec = {k.strip(): v.strip() for k, v in rec.items()}
        if rec.get("sources_sha256") != kernel_sources_sha256():
            return None, "kernel sources changed since the counters were taken"
        return float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"]), "profiles/" + os.path.basename(TRAFFIC_RECORD)
    except (OSError, KeyError, ValueError) as e:
        return None, f"no usable traffic record ({type(e).__name__})"


def host_threads():
    """Threads the CPU oracle can use: the affinity mask of this process and the thread
    count of the BLAS that numpy calls."""
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    blas = None
    try:
        from threadpoolctl import threadpool_info
        blas = max((int(p.get("num_threads", 0)) for p in threadpool_info() if p.get("user_api") == "blas"), default=None)
    except Exception:
        pass
    return cores, blas


def tensor_sha256(t):
    """SHA-256 of a CPU tensor's bytes (bf16 viewed as int16)."""
    import hashlib

    import torch
    t = t.contiguous()
    if t.dtype == torch.bfloat16:
        t = t.view(torch.int16)
    return hashlib.sha256(t.numpy().tobytes()).hexdigest()


def fwd_flops(M, K, N, G, r):
    return 2 * M * K * N + M * K + 2 * M * G * r + 2 * M * r * N


def bwd_flops(M, K, N, G, r):
    return 2 * M * K * N + 2 * M * N * r + 2 * M * r * G + M * K + 2 * M * r * N + 2 * M * G * r


def fwd_bytes(M, K, N, G, r, bits):
    return K * N * bits // 8 + 8 * G * N + 2 * (G * r + r * N) + 2 * M * K + 2 * M * N


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm": p["hbm_gbs"], "tensor": p["bf16_tflops_sustained"], "tensor_burst": p["bf16_tflops"],
                "source": "measured"}
    return {"hbm": 6650.0, "tensor": 1400.0, "tensor_burst": 1590.0, "source": "fallback"}


# ------------------------------------------------------------- clock sampler --
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid):
        self.uuid = gpu_uuid
        self.proc = None
        self.lines = []          # (arrival time, text)
        self.t_begin = self.t_end = None

    def start(self):
        """Starts nvidia-smi (it needs a few hundred ms before its first sample, so this is
        called before the warm-up) and waits for the first line."""
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
            deadline = time.monotonic() + 5.0
            while not self.lines and time.monotonic() < deadline and self.proc.poll() is None:
                time.sleep(0.01)
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def begin(self):
        self.t_begin = time.monotonic()

    def end(self):
        self.t_end = time.monotonic()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.03)          # let the last sample of the region arrive
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        # samples taken during the timed region (a sample is printed right after it is taken)
        t0 = self.t_begin if self.t_begin is not None else float("-inf")
        t1 = (self.t_end if self.t_end is not None else float("inf")) + 0.02
        for stamp, line in self.lines:
            if not (t0 <= stamp <= t1):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------- CPU reference --
def oracle_setup(rows, shape=None):
    """Inputs of the CPU-oracle sample: `rows` token rows of one shape (the first by default), quantized once."""
    from oracle import qalora_oracle as O
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs, to_f64

    shape = SHAPES[0] if shape is None else shape
    cfg = CONFIGS[shape].with_(tokens=rows)
    t = make_inputs(cfg)
    codes, alpha, beta = O.quantize(t["W"].numpy(), cfg.group_size, cfg.bits)
    x, A, B, dy = (to_f64(t[k]) for k in ("x", "A", "B", "dy"))
    fl = fwd_flops(rows, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank) + bwd_flops(rows, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank)
    desc = (f"fp64 numpy oracle, forward+backward on {rows} of 8192 token rows of {shape} "
            f"(each call dequantizes the full {cfg.d_in}x{cfg.d_out} weight); quantize excluded")
    return (O, cfg, codes, alpha, beta, x, A, B, dy), fl, desc


def oracle_run(state):
    O, cfg, codes, alpha, beta, x, A, B, dy = state
    t0 = time.perf_counter()
    O.forward(x, codes, alpha, beta, cfg.group_size, A, B, cfg.scale)
    O.backward(x, dy, codes, alpha, beta, cfg.group_size, A, B, cfg.scale)
    return time.perf_counter() - t0


def oracle_sample(rows=32):
    """Times the CPU oracle (as it stands) on `rows` token rows of every shape of the
    step: forward + backward.  Returns (TFLOP/s, seconds, description, threads)."""
    import torch
    fl_sum, dt_sum, descs = 0.0, 0.0, []
    for shape in SHAPES:
        state, fl, desc = oracle_setup(rows, shape)
        dt_sum += oracle_run(state)
        fl_sum += fl
        descs.append(desc)
        del state
    return fl_sum / dt_sum / 1e12, dt_sum, "; ".join(descs), host_threads()


def run_reference(args):
    """The reference arm: the CPU oracle, one bounded sample of the workload per step."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    state, fl, desc = oracle_setup(16)
    times = []
    for i in range(args.warmup + args.steps):
        dt = oracle_run(state)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * sum(times) / max(1, len(times))
    value = fl / (ms / 1e3) / 1e12
    cores, blas = host_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": desc},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "blas_threads": blas, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------ GPU arm ---
class ShapeState:
    def __init__(self, name, rank, Q, torch):
        from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs
        cfg = CONFIGS[name]
        self.cfg = cfg
        shared = make_inputs(cfg, need=("W", "A", "B"))
        batch = make_inputs(cfg.with_(seed=cfg.seed + 1000 * (rank + 1)), need=("x", "dy"))
        self.host = {"x": batch["x"].pin_memory(), "dy": batch["dy"].pin_memory()}
        self.sha256 = {k: tensor_sha256(v) for k, v in (("W", shared["W"]), ("A", shared["A"]), ("B", shared["B"]),
                                                      ("x", batch["x"]), ("dy", batch["dy"]))}
        self.W = shared["W"].cuda()
        self.A = shared["A"].cuda()
        self.B = shared["B"].cuda()
        self.x = batch["x"].cuda()
        self.dy = batch["dy"].cuda()
        M, K, N, G, r = cfg.tokens, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank
        self.d = Q.desc(K, N, cfg.group_size, cfg.bits, r, cfg.scale)
        self.d0 = Q.desc(K, N, cfg.group_size, cfg.bits, 0, cfg.scale)
        self.codes, self.qparams = Q.alloc_packed(self.d)
        self.qmerged = torch.empty_like(self.qparams)
        self.y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        self.dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        self.ws_f = Q.alloc_workspace(self.d, M, Q.OP_FORWARD)
        self.ws_t = Q.alloc_workspace(self.d, M, Q.OP_TRAIN)          # forward + backward of a step share it
        self.x1 = self.x[:1].contiguous()
        self.y1 = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
        self.ws1 = Q.alloc_workspace(self.d0, 1, Q.OP_FORWARD)
        self.host_out = {"y": torch.empty((M, N), dtype=torch.bfloat16).pin_memory(),
                         "dx": torch.empty((M, K), dtype=torch.bfloat16).pin_memory(),
                         "dA": torch.empty((G, r), dtype=torch.float32).pin_memory(),
                         "dB": torch.empty((r, N), dtype=torch.float32).pin_memory()}
        self.staging = torch.zeros(Q.qalora_step_host_bytes(self.d, M), dtype=torch.uint8, device="cuda")
        self.flops = fwd_flops(M, K, N, G, r) + bwd_flops(M, K, N, G, r)
        self.main_flops = 2 * M * K * N


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2309_14717_b200 import binding as Q
    from paper_2309_14717_b200 import build as _build
    from paper_2309_14717_b200 import dp

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if local == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    Q.load()

    shapes = [ShapeState(n, rank, Q, torch) for n in SHAPES]
    stream = torch.cuda.current_stream()
    # All trained factors of the step live in one bucket: the backward passes write dA and dB into
    # its gradient views, ONE all-reduce sums it over the ranks and ONE clipped AdamW call
    # (Section 4.1) updates every factor and the bf16 copies the next forward reads.
    bucket = dp.AdapterBucket([(s.cfg.groups, s.cfg.rank, s.cfg.d_out) for s in shapes], device="cuda")
    for i, s in enumerate(shapes):
        bucket.load(i, s.A, s.B)
    LR = 2e-5                                          # the paper's learning rate for the 7B model

    def device_step(i, s, probe=None):
        A, B = bucket.factors(i)
        dA, dB = bucket.grads(i)
        Q.qalora_quantize(s.d, s.W, s.codes, s.qparams)
        if probe is not None:                      # events around the forward contraction kernel of this call
            Q.qalora_profile_next_main_kernel(*probe)
        Q.qalora_forward_train(s.d, s.cfg.tokens, s.x, s.codes, s.qparams, A, B, s.y, s.ws_t)
        Q.qalora_backward_train(s.d, s.cfg.tokens, s.x, s.dy, s.codes, s.qparams, A, B, s.dx, dA, dB, s.ws_t)

    def deploy_step(i, s):
        A, B = bucket.factors(i)
        Q.qalora_merge(s.d, s.qparams, A, B, s.qmerged)
        Q.qalora_forward(s.d0, 1, s.x1, s.codes, s.qmerged, None, None, s.y1, s.ws1)

    probes = []                                     # one event pair per timed step (first shape's forward kernel)

    def step():
        for j, s in enumerate(shapes):
            device_step(j, s, probes.pop() if (j == 0 and probes) else None)
        bucket.reduce()                             # the step's only exchange (a no-op on one GPU)
        bucket.update(LR)
        for j, s in enumerate(shapes):
            deploy_step(j, s)

    def e2e_step():
        # the same step through the C ABI with HOST buffers: x, dy go up and y, dx, dA, dB
        # come back inside qalora_step_host; quantize, merge and the merged one-token
        # forward work on resident weights as in the device-resident step
        for j, s in enumerate(shapes):
            A, B = bucket.factors(j)
            Q.qalora_quantize(s.d, s.W, s.codes, s.qparams)
            Q.qalora_step_host(s.d, s.cfg.tokens, s.host["x"], s.host["dy"], s.codes, s.qparams, A, B,
                               s.host_out["y"], s.host_out["dx"], s.host_out["dA"], s.host_out["dB"], s.staging)
            deploy_step(j, s)

    def timed(fn, steps, sampler=None):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        if sampler:
            sampler.begin()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        if sampler:
            sampler.end()
        if world > 1:
            dist.barrier()
        clocks = sampler.stop() if sampler else None
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, clocks

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid)
    sampler.start()                                 # before the warm-up: its first sample takes a while
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()

    probe_pairs = []
    for _ in range(args.steps):
        ka, kb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ka.record(stream); kb.record(stream)        # creates the underlying CUDA events
        probe_pairs.append((ka, kb))
    probes.extend(probe_pairs)
    torch.cuda.synchronize()
    launches0 = Q.qalora_kernel_launches()
    ms_total, clocks = timed(step, args.steps, sampler)
    s0_ = shapes[0]
    Q.qalora_forward(s0_.d, s0_.cfg.tokens, s0_.x, s0_.codes, s0_.qparams, *bucket.factors(0), s0_.y, s0_.ws_f)
    kernel_name = Q.qalora_main_kernel_name()       # which kernel the library picks for this shape
    torch.cuda.synchronize()
    launches = (Q.qalora_kernel_launches() - launches0) // max(1, args.steps)
    ms_step = ms_total / args.steps
    flops_step = sum(s.flops for s in shapes) * world
    value = flops_step / (ms_step / 1e3) / 1e12

    # dominant kernel: the forward contraction of the first shape, timed live inside the
    # timed region with events the library records around that one launch on the launch stream
    s0 = shapes[0]
    kms = sum(a.elapsed_time(b) for a, b in probe_pairs) / len(probe_pairs)
    pk = peaks()
    achieved = s0.main_flops / (kms / 1e3) / 1e12
    # Which measured cuBLAS figure fits this run: the sustained one (a seconds-long loop under
    # the power cap) only when the timed region was itself seconds long AND the power cap was
    # seen active in it; a short region at full clocks is compared with the burst figure.
    sustained = (ms_total >= 2000.0) and clocks is not None and "sw_power_cap" in (clocks.get("reasons") or [])
    peak = pk["tensor"] if sustained else pk["tensor_burst"]
    traffic, traffic_note = fwd_kernel_dram_traffic()
    roofline = {"bound": "tensor", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": pk["source"] + (" (sustained bf16)" if sustained else " (burst bf16)"),
                "frac_burst": achieved / pk["tensor_burst"], "frac_sustained": achieved / pk["tensor"],
                "peak_burst": pk["tensor_burst"], "peak_sustained": pk["tensor"],
                "step_frac_burst": value / world / pk["tensor_burst"], "step_frac_sustained": value / world / pk["tensor"],
                "kernel_ms": kms, "launches_timed": len(probe_pairs), "traffic": traffic, "traffic_source": traffic_note,
                "traffic_unit": "bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum)",
                "flops_per_launch": s0.main_flops}

    # single-token forward of the merged layer: HBM-bound leg of the metric
    small = small_m_bandwidth(Q, torch, pk)
    small_65b = mid = grouped = None
    if rank == 0:
        from paper_2309_14717_b200.synthetic import CONFIGS
        small_65b = small_m_bandwidth(Q, torch, pk, shape="cfg5_65b_up", ms=(1, 16))
        for g in (64, 128):          # the group-size sweep of the 65B configuration, one token
            r_ = small_m_bandwidth(Q, torch, pk, ms=(1,), cfg=CONFIGS["cfg5_65b_up"].with_(group_size=g))
            small_65b[f"g{g}"] = {k: r_[k] for k in ("M1", "M1_merged")}
        mid = {name: mid_m_roofline(Q, torch, pk, name) for name in (SMALL_M, "cfg5_65b_up")}
        grouped = {f"M{m}": grouped_block_bandwidth(Q, torch, pk, m) for m in (1, 16)}

    adamw = adapter_update_bandwidth(Q, torch, pk) if rank == 0 else None

    e2e_ms, _ = timed(e2e_step, args.steps)
    e2e_ms /= args.steps
    h2d = sum(s.host["x"].numel() * 2 + s.host["dy"].numel() * 2 for s in shapes)
    d2h = sum(sum(t.numel() * t.element_size() for t in s.host_out.values()) for s in shapes)

    if rank == 0:
        # the CPU oracle is timed at N = 1 only (the other GPUs would be held idle meanwhile)
        cpu = None
        if world == 1:
            v, dt, desc, (cores, blas) = oracle_sample(rows=8192)
            cpu = {"value": v, "unit": "TFLOP/s", "cores": cores, "blas_threads": blas, "kind": "oracle", "sample": desc,
                   "seconds": dt}
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "shapes": list(SHAPES), "tokens_per_gpu": 8192, "bits": 4,
                       "group_size": 32, "rank": 64,
                       "step": "both shapes: quantize+forward+backward (dA, dB into one gradient bucket); one all-reduce "
                               "of the bucket (N > 1); one clipped AdamW update of all factors; both shapes: merge + "
                               "merged M=1 forward",
                       "l2": "inputs exceed L2 (x+dy+y+dx > 470 MB per shape)",
                       "parallelism": f"dp{world}" if world > 1 else "single"},
            "clocks": clocks, "gpu_launches": int(launches),
            "e2e": {"value": flops_step / (e2e_ms / 1e3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "roofline": roofline, "small_m": small, "small_m_65b": small_65b, "mid_m": mid,
            "grouped_block": grouped, "adapter_update": adamw, "cpu_baseline": cpu,
            "inputs_sha256": {s.cfg.name: s.sha256 for s in shapes}, "inputs_match_record": inputs_match_record(shapes),
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def inputs_match_record(shapes):
    """Compares the hashes of this run's synthetic inputs (rank 0's batch) with the record kept
    in tests/golden/bench_inputs_sha256.txt, written by tests/golden/make_bench_inputs_sha256.py
    from the generator alone: a torch version that drew other numbers would show here."""
    path = os.path.join(ROOT, "tests", "golden", "bench_inputs_sha256.txt")
    try:
        want = {}
        for line in open(path):
            if line.strip() and not line.startswith("#"):
                name, tensor, digest = line.split()
                want[(name, tensor)] = digest
    except OSError:
        return None
    return all(want.get((s.cfg.name, k)) == v for s in shapes for k, v in s.sha256.items())


def adapter_update_bandwidth(Q, torch, pk, reps=10):
    """Clipped AdamW (Section 4.1) over all adapter values of a LLaMA-7B sized model
    (32 blocks x 7 projections, rank 64, group size 32): one flat array of about 80 M values,
    far larger than L2.  Algorithmic bytes per value: 4 (norm pass) + 16 read + 14 written."""
    r, g, d, f = 64, 32, 4096, 11008
    per_block = 4 * (d // g * r + r * d) + 2 * (d // g * r + r * f) + (f // g * r + r * d)
    n = 32 * per_block
    grad = torch.randn(n, device="cuda") * 1e-3
    param = torch.randn(n, device="cuda") * 0.02
    m, v = torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    pb = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(Q.qalora_adamw_workspace_bytes(), dtype=torch.uint8, device="cuda")
    norm = torch.zeros(2, device="cuda")
    for t in range(1, 4):
        Q.qalora_adamw_step(Q.adamw_hyper(t, 2e-5), n, grad, param, m, v, pb, norm, ws)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for t in range(4, 4 + reps):
        Q.qalora_adamw_step(Q.adamw_hyper(t, 2e-5), n, grad, param, m, v, pb, norm, ws)
    b.record()
    torch.cuda.synchronize()
    us = a.elapsed_time(b) * 1e3 / reps
    gbs = n * 34 / (us * 1e-6) / 1e9
    return {"values": n, "us_per_step": us, "GB/s": gbs, "frac_of_hbm": gbs / pk["hbm"], "bytes_per_value": 34,
            "launches": 2}


def small_m_bandwidth(Q, torch, pk, shape=SMALL_M, ms=(1, 4, 16), cfg=None):
    """Few-token forward of one layer shape, rotating over enough weight copies
    (> 4 x L2) that the codes stream from HBM.  The rotation is captured once in
    a CUDA graph and replayed, so that the GPU and not the host's launch rate is
    timed.  Reported for the adapted layer (pool/adapter pre-kernel + main
    kernel per call) and for the merged, deployed layer (one kernel per call)."""
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs
    cfg = CONFIGS[shape] if cfg is None else cfg
    t = make_inputs(cfg.with_(tokens=max(ms)), need=("W", "x", "A", "B"))
    d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, cfg.rank, cfg.scale)
    d0 = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, 0, cfg.scale)
    W = t["W"].cuda()
    A, B = t["A"].cuda(), t["B"].cuda()
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, W, codes, qparams)
    del W
    layer_bytes = codes.numel() * 4 + qparams.numel() * 4
    ncopies = max(8, -(-5 * 126 * 2 ** 20 // layer_bytes))      # total > 4 x L2
    copies = [(codes.clone(), qparams.clone()) for _ in range(ncopies)]
    out = {}
    side = torch.cuda.Stream()
    for M in ms:
        x = t["x"][:M].contiguous().cuda()
        y = torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda")
        for name, dd, a_, b_ in (("", d, A, B), ("_merged", d0, None, None)):
            ws = Q.alloc_workspace(dd, M, Q.OP_FORWARD)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for c, q in copies[:3]:                          # warm-up (also sets kernel attributes)
                    Q.qalora_forward(dd, M, x, c, q, a_, b_, y, ws)
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for c, q in copies:
                    Q.qalora_forward(dd, M, x, c, q, a_, b_, y, ws)
            for _ in range(2):
                graph.replay()
            torch.cuda.synchronize()
            reps = 5
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (reps * ncopies)
            nbytes = fwd_bytes(M, cfg.d_in, cfg.d_out, cfg.groups, dd.rank, cfg.bits)
            gbs = nbytes / (us * 1e-6) / 1e9
            out[f"M{M}{name}"] = {"us_per_call": us, "GB/s": gbs, "frac_of_hbm": gbs / pk["hbm"], "bytes": nbytes}
            del graph
    out["shape"] = shape
    out["peak_GB/s"] = pk["hbm"]
    out["peak_source"] = pk["source"]
    out["l2"] = (f"CUDA-graph replay rotating over {ncopies} weight copies ({ncopies * layer_bytes / 1e6:.0f} MB) "
                 "so codes stream from HBM")
    return out


def mid_m_roofline(Q, torch, pk, shape, ms=(64, 128, 256, 512)):
    """Forward of one layer shape at a few hundred tokens, adapted and merged, rotating over
    weight copies like small_m_bandwidth.  Both rooflines are given: the bytes of one call at
    the measured copy bandwidth and 2 M K N flops at the measured burst bf16 rate; `frac` is
    against the slower (larger) of the two bounds."""
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs
    cfg = CONFIGS[shape]
    t = make_inputs(cfg.with_(tokens=max(ms)), need=("W", "x", "A", "B"))
    K, N, G, r = cfg.d_in, cfg.d_out, cfg.groups, cfg.rank
    d = Q.desc(K, N, cfg.group_size, cfg.bits, r, cfg.scale)
    d0 = Q.desc(K, N, cfg.group_size, cfg.bits, 0, cfg.scale)
    W = t["W"].cuda()
    A, B = t["A"].cuda(), t["B"].cuda()
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, W, codes, qparams)
    del W
    layer_bytes = codes.numel() * 4 + qparams.numel() * 4
    ncopies = max(4, -(-5 * 126 * 2 ** 20 // layer_bytes))
    copies = [(codes.clone(), qparams.clone()) for _ in range(ncopies)]
    out = {}
    side = torch.cuda.Stream()
    for M in ms:
        x = t["x"][:M].contiguous().cuda()
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        for name, dd, a_, b_ in (("", d, A, B), ("_merged", d0, None, None)):
            ws = Q.alloc_workspace(dd, M, Q.OP_FORWARD)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for c, q in copies[:3]:
                    Q.qalora_forward(dd, M, x, c, q, a_, b_, y, ws)
            side.synchronize()
            kernel = Q.qalora_main_kernel_name()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for c, q in copies:
                    Q.qalora_forward(dd, M, x, c, q, a_, b_, y, ws)
            graph.replay()
            torch.cuda.synchronize()
            reps = 3
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (reps * ncopies)
            nbytes = fwd_bytes(M, K, N, G, dd.rank, cfg.bits)
            flops = 2 * M * K * N
            t_hbm, t_tc = nbytes / (pk["hbm"] * 1e9) * 1e6, flops / (pk["tensor_burst"] * 1e12) * 1e6
            out[f"M{M}{name}"] = {"us_per_call": us, "kernel": kernel, "bytes": nbytes, "flops": flops,
                                  "hbm_bound_us": t_hbm, "tensor_bound_us": t_tc, "frac": max(t_hbm, t_tc) / us,
                                  "bound": "hbm" if t_hbm >= t_tc else "tensor"}
            del graph
    out["shape"] = shape
    out["peaks"] = {"hbm_GB/s": pk["hbm"], "bf16_burst_TFLOP/s": pk["tensor_burst"], "source": pk["source"]}
    return out


def grouped_block_bandwidth(Q, torch, pk, M=1):
    """The five projections of a LLaMA-7B block that read the block's input (q, k, v: 4096 -> 4096;
    gate, up: 4096 -> 11008; merged INT4 layers, group size 32) on M tokens: five qalora_forward
    calls against ONE qalora_forward_group call.  CUDA-graph replay over rotating weight copies
    (> 4 x L2 in total) as in small_m_bandwidth."""
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs
    shapes = [CONFIGS["cfg2_7b_attn"]] * 3 + [CONFIGS["cfg3_7b_up"]] * 2
    base = {}
    for cfg in {c.name: c for c in shapes}.values():
        t = make_inputs(cfg.with_(tokens=M), need=("W", "x"))
        d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, 0, cfg.scale)
        codes, qparams = Q.alloc_packed(d)
        Q.qalora_quantize(d, t["W"].cuda(), codes, qparams)
        base[cfg.name] = (d, codes, qparams)
    x = t["x"][:M].contiguous().cuda()                      # every projection reads the same input
    set_bytes = sum(base[c.name][1].numel() * 4 + base[c.name][2].numel() * 4 for c in shapes)
    ncopies = max(4, -(-5 * 126 * 2 ** 20 // set_bytes))
    sets = []
    for _ in range(ncopies):
        layers = []
        for c in shapes:
            d, codes, qparams = base[c.name]
            y = torch.empty((M, c.d_out), dtype=torch.bfloat16, device="cuda")
            layers.append((d, x, codes.clone(), qparams.clone(), None, None, y))
        sets.append(layers)
    ws = torch.zeros(max(Q.qalora_forward_group_workspace_bytes(sets[0], M), 16), dtype=torch.uint8, device="cuda")
    arrays = [Q.group_layers(layers) for layers in sets]

    def separate(i):
        for d, x_, c, q, _, _, y in sets[i]:
            Q.qalora_forward(d, M, x_, c, q, None, None, y, ws)

    def grouped(i):
        Q.qalora_forward_group(arrays[i], M, ws)

    nbytes = sum(fwd_bytes(M, c.d_in, c.d_out, c.groups, 0, c.bits) for c in shapes)
    out = {"layers": [f"{c.d_in}x{c.d_out}" for c in shapes], "M": M, "bytes": nbytes}
    side = torch.cuda.Stream()
    for name, fn in (("separate", separate), ("grouped", grouped)):
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn(0); fn(1)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(ncopies):
                fn(i)
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 5
        e0.record()
        for _ in range(reps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * ncopies)
        out[name] = {"us_per_block": us, "GB/s": nbytes / (us * 1e-6) / 1e9, "frac_of_hbm": nbytes / (us * 1e-6) / 1e9 / pk["hbm"],
                     "launches": 5 if name == "separate" else 1}
        del graph
    return out


def run_only(args):
    """Profiling helper: a few launches of one operation on one shape with a
    reduced token count (inputs still exceed L2), e.g. for an ncu capture:
        python bench.py --only fwd --shape cfg3_7b_up --tokens 4096"""
    import torch

    from paper_2309_14717_b200 import binding as Q
    from paper_2309_14717_b200 import build as _build
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs

    _build.build()
    if args.only == "adamw":   # the adapter update on the 7B-sized flat array (--steps timed calls inside)
        print(json.dumps({"only": "adamw", **adapter_update_bandwidth(Q, torch, peaks(), reps=max(1, args.steps))}))
        return
    cfg = CONFIGS[args.shape].with_(tokens=args.tokens)
    if args.group_size:
        cfg = cfg.with_(group_size=args.group_size)
    if args.bits:
        cfg = cfg.with_(bits=args.bits)
    t = {k: v.cuda() for k, v in make_inputs(cfg).items()}
    M, K, N, G, r = cfg.tokens, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank
    d = Q.desc(K, N, cfg.group_size, cfg.bits, r, cfg.scale)
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, t["W"], codes, qparams)
    if args.merged:                                # the deployed layer: adapter folded into the zeros, rank 0
        Q.qalora_merge(d, qparams, t["A"], t["B"], qparams)
        d = Q.desc(K, N, cfg.group_size, cfg.bits, 0, cfg.scale)
        t["A"] = t["B"] = None
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dA = torch.empty((G, r), dtype=torch.float32, device="cuda")
    dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
    wf, wb = Q.alloc_workspace(d, M, Q.OP_FORWARD), Q.alloc_workspace(d, M, Q.OP_BACKWARD)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times, ktimes = [], []
    ka, kb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ka.record(); kb.record()
    for _ in range(args.steps + 2):
        if args.only in ("fwd", "gemv", "bwd"):
            Q.qalora_profile_next_main_kernel(ka, kb)
        e0.record()
        if args.only in ("fwd", "gemv"):
            Q.qalora_forward(d, M, t["x"], codes, qparams, t["A"], t["B"], y, wf)
        elif args.only == "bwd":
            Q.qalora_backward(d, M, t["x"], t["dy"], codes, qparams, t["A"], t["B"], dx, dA, dB, wb)
        elif args.only == "quantize":
            Q.qalora_quantize(d, t["W"], codes, qparams)
        elif args.only == "merge":
            Q.qalora_merge(d, qparams, t["A"], t["B"], qparams)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
        if args.only in ("fwd", "gemv", "bwd"):
            ktimes.append(ka.elapsed_time(kb))
    print(json.dumps({"only": args.only, "shape": args.shape, "tokens": M, "ms": times[2:],
                      "main_kernel": Q.qalora_main_kernel_name(), "main_kernel_ms": ktimes[2:],
                      "status": Q.workspace_status(wb if args.only == "bwd" else wf)}))


def run_table(args):
    """Every benchmark configuration in turn (one layer at a time): forward and backward
    at the configuration's token count, and the merged one-token forward of the 65B shapes
    per group size.  Prints a markdown table; times are medians of CUDA-event timed calls."""
    import statistics

    import torch

    from paper_2309_14717_b200 import binding as Q
    from paper_2309_14717_b200 import build as _build
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs

    _build.build()
    pk = peaks()
    cases = [(CONFIGS[n], 8192) for n in ("cfg3_7b_up", "cfg3_7b_down")]
    for bits in (3, 2):
        cases += [(CONFIGS[n].with_(bits=bits), 4096) for n in ("cfg4_13b_up", "cfg4_13b_down", "cfg4_13b_attn")]
    for g in (32, 64, 128):
        cases += [(CONFIGS[n].with_(group_size=g), 8192) for n in ("cfg5_65b_up", "cfg5_65b_down", "cfg5_65b_attn")]
    print("| layer | bits | g | M | forward ms | TFLOP/s | of sustained bf16 peak | backward ms | TFLOP/s | of peak | fwd+bwd TFLOP/s | of peak |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for cfg0, M in cases:
        cfg = cfg0.with_(tokens=M)
        t = {k: v.cuda() for k, v in make_inputs(cfg).items()}
        K, N, G, r = cfg.d_in, cfg.d_out, cfg.groups, cfg.rank
        d = Q.desc(K, N, cfg.group_size, cfg.bits, r, cfg.scale)
        codes, qparams = Q.alloc_packed(d)
        Q.qalora_quantize(d, t["W"], codes, qparams)
        del t["W"]
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.empty((G, r), dtype=torch.float32, device="cuda")
        dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
        wf, wb = Q.alloc_workspace(d, M, Q.OP_FORWARD), Q.alloc_workspace(d, M, Q.OP_BACKWARD)
        res = {}
        for op in ("fwd", "bwd"):
            ts = []
            for _ in range(3 + 7):
                e0.record()
                if op == "fwd":
                    Q.qalora_forward(d, M, t["x"], codes, qparams, t["A"], t["B"], y, wf)
                else:
                    Q.qalora_backward(d, M, t["x"], t["dy"], codes, qparams, t["A"], t["B"], dx, dA, dB, wb)
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            res[op] = statistics.median(ts[3:])
        assert Q.workspace_status(wf) == 0 and Q.workspace_status(wb) == 0
        ff, fb = fwd_flops(M, K, N, G, r), bwd_flops(M, K, N, G, r)
        tf, tb = ff / res["fwd"] / 1e9, fb / res["bwd"] / 1e9
        tt = (ff + fb) / (res["fwd"] + res["bwd"]) / 1e9
        print(f"| {cfg.name} | {cfg.bits} | {cfg.group_size} | {M} | {res['fwd']:.3f} | {tf:.0f} | {tf / pk['tensor']:.2f} | "
              f"{res['bwd']:.3f} | {tb:.0f} | {tb / pk['tensor']:.2f} | {tt:.0f} | {tt / pk['tensor']:.2f} |", flush=True)
        del t, codes, qparams, y, dx, wf, wb
        torch.cuda.empty_cache()
    print()
    print("| layer | g | merged M = 1 forward us | GB/s | of measured copy bandwidth |")
    print("|---|---|---|---|---|")
    for g in (32, 64, 128):
        for n in ("cfg5_65b_up", "cfg5_65b_down", "cfg5_65b_attn"):
            rr = small_m_bandwidth(Q, torch, pk, ms=(1,), cfg=CONFIGS[n].with_(group_size=g))["M1_merged"]
            print(f"| {n} | {g} | {rr['us_per_call']:.1f} | {rr['GB/s']:.0f} | {rr['frac_of_hbm']:.2f} |", flush=True)
            torch.cuda.empty_cache()
    print()
    print(f"peaks: bf16 {pk['tensor']:.0f} TFLOP/s, HBM {pk['hbm']:.0f} GB/s ({pk['source']})")


def run_baselines(args):
    """The paper's Table 2 comparison restated on this GPU, one layer at a time: a 16-bit LoRA
    layer (library GEMMs on a bf16 weight, adapter on the un-pooled input), a QLoRA-style layer
    (dequantize the 4-bit weight to bf16, then the same GEMMs) and this library's QA-LoRA layer.
    The two baselines are written with torch.matmul (cuBLAS): they are context, not product."""
    import statistics

    import torch

    from paper_2309_14717_b200 import binding as Q
    from paper_2309_14717_b200 import build as _build
    from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs

    _build.build()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def med(fn, reps=7, warm=3):
        ts = []
        for _ in range(warm + reps):
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts[warm:])

    print("| layer | M | 16-bit LoRA fwd+bwd ms | dequantize + 16-bit fwd+bwd ms | QA-LoRA fwd+bwd ms | QA-LoRA / LoRA | QA-LoRA / dequantize-first |")
    print("|---|---|---|---|---|---|---|")
    rows1 = []
    for name in ("cfg3_7b_up", "cfg3_7b_down", "cfg5_65b_up", "cfg5_65b_down", "cfg5_65b_attn"):
        M = 8192
        cfg = CONFIGS[name].with_(tokens=M)
        t = {k: v.cuda() for k, v in make_inputs(cfg).items()}
        K, N, G, r, s = cfg.d_in, cfg.d_out, cfg.groups, cfg.rank, cfg.scale
        d = Q.desc(K, N, cfg.group_size, cfg.bits, r, s)
        codes, qparams = Q.alloc_packed(d)
        Q.qalora_quantize(d, t["W"], codes, qparams)
        del t["W"]
        x, dy, B = t["x"], t["dy"], t["B"]
        W16 = torch.empty((K, N), dtype=torch.bfloat16, device="cuda")
        Q.qalora_dequantize(d, codes, qparams, W16)
        A_full = (torch.randn(K, r, device="cuda") * 0.02).to(torch.bfloat16)      # LoRA's A spans D_in

        def lora_step(W):
            T = x @ A_full
            y = torch.addmm(x @ W, T, B, alpha=s)
            dT = (dy @ B.t()) * s
            dx = torch.addmm(dy @ W.t(), dT, A_full.t())
            dA = x.t() @ dT
            dB = (T.t() @ dy) * s
            return y, dx, dA, dB

        def qlora_step():
            Q.qalora_dequantize(d, codes, qparams, W16)      # forward
            T = x @ A_full
            y = torch.addmm(x @ W16, T, B, alpha=s)
            Q.qalora_dequantize(d, codes, qparams, W16)      # backward dequantizes again
            dT = (dy @ B.t()) * s
            dx = torch.addmm(dy @ W16.t(), dT, A_full.t())
            return y, dx, x.t() @ dT, (T.t() @ dy) * s

        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.empty((G, r), dtype=torch.float32, device="cuda")
        dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
        wf, wb = Q.alloc_workspace(d, M, Q.OP_FORWARD), Q.alloc_workspace(d, M, Q.OP_BACKWARD)

        def qalora_step():
            Q.qalora_forward(d, M, x, codes, qparams, t["A"], B, y, wf)
            Q.qalora_backward(d, M, x, dy, codes, qparams, t["A"], B, dx, dA, dB, wb)

        # one-token serving first (before the long GEMMs heat the part): merged INT4 layer against
        # a bf16 matrix-vector product
        time.sleep(1.0)
        x1 = x[:1].contiguous()
        y1 = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
        d0 = Q.desc(K, N, cfg.group_size, cfg.bits, 0, s)
        w1 = Q.alloc_workspace(d0, 1, Q.OP_FORWARD)
        copies = max(8, int(5 * 126e6 // (K * N // 2)) + 1)     # even the 4-bit copies total > 4 x L2
        W16s = [W16.clone() for _ in range(copies)]
        Cs = [(codes.clone(), qparams.clone()) for _ in range(copies)]

        def graph_us(fn):
            g = torch.cuda.CUDAGraph()
            fn(0)
            torch.cuda.synchronize()
            with torch.cuda.graph(g):
                for i in range(copies):
                    fn(i)

            def five():
                for _ in range(5):
                    g.replay()
            return med(five, reps=3, warm=1) * 1e3 / (5 * copies)

        t16 = graph_us(lambda i: torch.matmul(x1, W16s[i], out=y1))
        t4 = graph_us(lambda i: Q.qalora_forward(d0, 1, x1, Cs[i][0], Cs[i][1], None, None, y1, w1,
                                                 torch.cuda.current_stream()))
        rows1.append(f"| {name} | {t16:.1f} | {t4:.1f} | {t16 / t4:.2f} |")
        a, b, c = med(lambda: lora_step(W16)), med(qlora_step), med(qalora_step)
        del W16s, Cs
        print(f"| {name} | {M} | {a:.3f} | {b:.3f} | {c:.3f} | {c / a:.2f} | {c / b:.2f} |", flush=True)
        del t, W16, codes, qparams, y, dx, wf, wb, x, dy
        torch.cuda.empty_cache()
    print()
    print("| layer | bf16 weight, M = 1 forward us | merged INT4 QA-LoRA, M = 1 forward us | speed-up |")
    print("|---|---|---|---|")
    print("\n".join(rows1))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--baselines", action="store_true", help="16-bit LoRA and dequantize-first layers beside QA-LoRA (markdown)")
    ap.add_argument("--table", action="store_true", help="per-configuration throughput table (markdown)")
    ap.add_argument("--only", default=None, choices=("fwd", "bwd", "gemv", "quantize", "merge", "adamw"))
    ap.add_argument("--shape", default="cfg3_7b_up")
    ap.add_argument("--tokens", type=int, default=4096)
    ap.add_argument("--merged", action="store_true", help="with --only fwd/gemv: the merged (rank 0) layer")
    ap.add_argument("--group-size", type=int, default=0, help="with --only: override the shape's group size")
    ap.add_argument("--bits", type=int, default=0, help="with --only: override the shape's bit width")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    args = ap.parse_args()
    if args.table:
        run_table(args)
    elif args.baselines:
        run_baselines(args)
    elif args.only is not None:
        run_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

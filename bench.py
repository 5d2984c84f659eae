#!/usr/bin/env python
"""Benchmark of the SBW hot path on B200.

    python bench.py --gpus N --steps K --warmup W            # this library (CUDA kernels)
    python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

One "step" is one decode step of the headline workload: `sbw_bias_logits` (context-hash seeding,
gamma 0.5, delta 2.0, key 0x5EED) on a fresh [64, 128256] bf16 logits tensor with fresh context
tokens -- 256 distinct step inputs (4.2 GB) are resident and visited in turn, so no step finds its
input in L2.  `value` is bias throughput in Gelem/s (B*V logits per second, all GPUs).  The same
JSON line carries the roofline placement of the bias kernel, the end-to-end figure through the
host-buffer entry point, the oracle timed on the host cores, and (under "extra") the self-salt
bias, detection and fused-sampling workloads with their own roofline fractions.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

KEY = 0x5EED
B2, V2 = 64, 128256                 # headline workload: bf16, context scheme
GAMMA2, DELTA2 = 0.5, 2.0
POOL = 256                          # distinct step inputs kept resident
# Algorithmic work per logit (what the method itself needs, not what the kernel spends):
#   context scheme: Philox4x32-10 word 0 = 20 32x32->64 multiplies + 20 three-input xors, and one
#   compare = 41 integer operations; 2 bytes read + 2 bytes written (bf16).
INT_OPS = {"context": 41, "selfsalt": 80, "detect_context": 62, "detect_selfsalt": 100}
# INT32 ceiling of one B200: 148 SMs x 64 INT32 lanes per SM per clock (16 per scheduler; the
# probe measures 64 ops/clk/SM for integer add, logic and 32-bit multiply-add, and 32 for the
# 32x32->64 multiply) at the 1965 MHz maximum SM clock = 18.6 T integer operations per second.
SMS, LANES_PER_SM_CLK, SM_MAX_MHZ = 148, 64, 1965.0
INT_PEAK_TOPS = SMS * LANES_PER_SM_CLK * SM_MAX_MHZ * 1e6 / 1e12
# DRAM bytes per bias launch of the headline workload: dram__bytes_read.sum + dram__bytes_write.sum
# of one ncu capture of the same kernel on B=512 (131.38 MB + 91.60 MB, profiles/), divided by 8
# because a bench launch processes 1/8 of those units and the traffic grows with the units.
NCU_TRAFFIC_BYTES = (131.38e6 + 91.60e6) / 8


def measured_peaks() -> dict:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples = []
        self._stop = threading.Event()
        self._thread = None
        self.max_mhz = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                self.samples.append((time.perf_counter(), float(mhz), int(reasons)))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, t0: float, t1: float) -> dict:
        if self.nv is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        inside = [s for s in self.samples if t0 <= s[0] <= t1] or \
            sorted(self.samples, key=lambda s: min(abs(s[0] - t0), abs(s[0] - t1)))[:3]
        mhz = sorted(s[1] for s in inside)
        bits = 0
        for s in inside:
            bits |= s[2]
        names = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap",
                 0x8: "hw_slowdown", 0x10: "sync_boost", 0x20: "sw_thermal_slowdown",
                 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
                 0x100: "display_clock_setting"}
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "samples": len(inside),
                "reasons": [n for b, n in names.items() if bits & b and n != "gpu_idle"]}


def dist_env():
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def shard_rows(total_rows: int, rank: int, world: int) -> tuple[int, int]:
    """Rows [lo, hi) of a batch owned by `rank` when a batch is sharded over `world` ranks (the
    path has no cross-row dependency, so sharding needs no collective)."""
    base, rem = divmod(total_rows, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def max_over_ranks(x: float, world: int, device=None) -> float:
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------------------- reference arm
def run_reference(args) -> None:
    """Times the CPU oracle, as it stands, on the host cores: each step is one headline decode
    step (64 x 128256 bf16, context scheme).  Rank 0 only."""
    rank, _, _ = dist_env()
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2609_03844_b200 import inputs

    cores = os.cpu_count() or 1
    n_in = min(max(args.steps, 1), 4)
    xs = [inputs.as_oracle_array(inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=1000 + i))
          for i in range(n_in)]
    cs = [inputs.uniform_tokens((B2, 1), V2, seed=2000 + i).numpy() for i in range(n_in)]
    for i in range(args.warmup):
        oracle.bias_logits(xs[i % n_in], V2, cs[i % n_in], KEY, GAMMA2, DELTA2, oracle.SCHEME_CONTEXT,
                           threads=cores)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle.bias_logits(xs[i % n_in], V2, cs[i % n_in], KEY, GAMMA2, DELTA2, oracle.SCHEME_CONTEXT,
                           threads=cores)
    dt = time.perf_counter() - t0
    value = B2 * V2 * args.steps / dt / 1e9
    line = {"impl": "reference", "metric": "sbw_bias_throughput", "value": value, "unit": "Gelem/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,   # the arm's N; the oracle itself runs on host cores
            "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {**workload_config(), "l2": f"{n_in} host-resident step inputs visited in turn (CPU run)"},
            "cpu_baseline": {"value": value, "unit": "Gelem/s", "cores": cores, "kind": "oracle",
                             "sample": f"{args.steps} full decode steps of the headline workload"},
            "e2e": {"value": value, "unit": "Gelem/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config() -> dict:
    return {"workload": "config 2: sbw_bias_logits, B=64, V=128256, bf16 logits N(0,4^2), "
                        "context-hash seeding on 1 preceding token, gamma=0.5, delta=2.0, key=0x5EED",
            "B": B2, "V": V2, "scheme": "context", "gamma": GAMMA2, "delta": DELTA2,
            "l2": f"{POOL} distinct step inputs (4.2 GB) visited in turn, far larger than the 126 MB L2"}


# ------------------------------------------------------------------------------------ our arm
def time_region(fn_enqueue, stream, world, device):
    """barrier + sync, events around fn_enqueue() on `stream`, sync + barrier; max over ranks."""
    import torch
    import torch.distributed as dist
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    fn_enqueue()
    e1.record(stream)
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, device)
    return ms, t0, t1


def run_ours(args) -> None:
    import torch
    import paper_2609_03844_b200 as sbw
    from paper_2609_03844_b200 import inputs

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SBW path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    sbw.lib()
    peaks = measured_peaks()
    K, W = args.steps, args.warmup
    stream = torch.cuda.current_stream()

    # ---- headline workload: every rank holds its own POOL step inputs (weak scaling) ----
    pool = min(POOL, max(K, 16))
    logits = [inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=10_000 * rank + i, device=dev)
              for i in range(pool)]
    ctxs = [inputs.uniform_tokens((B2, 1), V2, seed=5_000_000 + 10_000 * rank + i, device=dev)
            for i in range(pool)]
    torch.cuda.synchronize()

    def step(i):
        j = i % pool
        sbw.sbw_bias_logits(logits[j], ctxs[j], KEY, GAMMA2, DELTA2, sbw.SCHEME_CONTEXT)

    for i in range(max(W, 3)):
        step(i)
    torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.02)

    launch_mode = "stream"
    graph = None
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for i in range(K):
                    step(W + i)
            launch_mode = "cuda_graph"
        except Exception as exc:    # capture unsupported: keep the plain stream launches
            graph = None
            launch_mode = f"stream (graph capture failed: {type(exc).__name__})"
    stream = torch.cuda.current_stream()
    if graph is not None:
        graph.replay()              # one untimed replay: graph upload
        ms, t0, t1 = time_region(graph.replay, stream, world, dev)
    else:
        ms, t0, t1 = time_region(lambda: [step(W + i) for i in range(K)], stream, world, dev)
    # the same K steps as plain stream launches, for the record
    ms_stream, _, _ = time_region(lambda: [step(W + i) for i in range(K)], stream, world, dev)
    time.sleep(0.01)
    sampler.stop()
    clocks = sampler.summary(t0, t1)

    elems_step = B2 * V2
    value = world * elems_step * K / (ms * 1e-3) / 1e9
    launch_s = ms * 1e-3 / K
    int_ops = INT_OPS["context"] * elems_step
    ach_tops = int_ops / launch_s / 1e12
    hbm_gbs = 4 * elems_step / launch_s / 1e9
    roofline = {"bound": "alu", "achieved": ach_tops, "peak": INT_PEAK_TOPS, "unit": "Tint-op/s",
                "frac": ach_tops / INT_PEAK_TOPS, "traffic": NCU_TRAFFIC_BYTES,
                "peak_source": "derived: 148 SMs x 64 INT32 lanes x 1965 MHz",
                "kernel": "bias_kernel<bf16, context, vector>", "avg_launch_us": launch_s * 1e6,
                "int_ops_per_elem": INT_OPS["context"],
                "hbm": {"achieved": hbm_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": hbm_gbs / peaks["hbm_gbs"], "of": peaks["source"],
                        "bytes_per_elem": 4},
                "binding": "alu" if int_ops / (INT_PEAK_TOPS * 1e12) > 4 * elems_step / (peaks["hbm_gbs"] * 1e9)
                else "hbm"}

    # ---- end to end: host buffers through the C ABI, copies inside the timed region ----
    # Steps alternate between two streams, each with its own staging buffer, so that one step's
    # device-to-host copy overlaps the next step's host-to-device copy (PCIe is full duplex).
    n_host = 4
    h_logits = [inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=77 + i).pin_memory() for i in range(n_host)]
    h_ctx = [inputs.uniform_tokens((B2, 1), V2, seed=88 + i).pin_memory() for i in range(n_host)]
    stage_bytes = sbw.sbw_bias_logits_host_staging_bytes(torch.bfloat16, B2, V2, 1)
    lanes = [(torch.cuda.Stream(), torch.empty(stage_bytes, dtype=torch.uint8, device=dev)) for _ in range(2)]
    K_e2e = max(1, min(K, 64))
    main = torch.cuda.current_stream()

    def e2e_steps():
        fork = torch.cuda.Event()
        fork.record(main)
        for st, _ in lanes:
            st.wait_event(fork)
        for i in range(K_e2e):
            st, staging = lanes[i % 2]
            sbw.sbw_bias_logits_host(h_logits[i % n_host], h_ctx[i % n_host], KEY, GAMMA2, DELTA2,
                                     sbw.SCHEME_CONTEXT, staging, stream=st)
        for st, _ in lanes:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    e2e_steps()
    ms_e2e, _, _ = time_region(e2e_steps, main, world, dev)
    e2e = {"value": world * elems_step * K_e2e / (ms_e2e * 1e-3) / 1e9, "unit": "Gelem/s",
           "h2d_bytes_per_step": elems_step * 2 + B2 * 4, "d2h_bytes_per_step": elems_step * 2,
           "steps": K_e2e, "ms_per_step": ms_e2e / K_e2e,
           "api": "sbw_bias_logits_host (pinned host logits and context tokens), steps alternating "
                  "between two streams"}
    del h_logits, lanes

    line = {"metric": "sbw_bias_throughput", "value": value, "unit": "Gelem/s", "n_gpus": world,
            "steps": K, "warmup": W, "ms_per_step": ms / K, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {**workload_config(), "launch": launch_mode, "parallelism": f"replicas x{world}",
                       "l2": f"{pool} distinct step inputs ({pool * elems_step * 2 / 1e9:.1f} GB) visited in "
                             "turn, far larger than the 126 MB L2"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": K, "roofline": roofline,
            "stream_launch": {"value": world * elems_step * K / (ms_stream * 1e-3) / 1e9,
                              "ms_per_step": ms_stream / K}}

    if rank == 0 and world == 1 and not args.no_extra:
        del logits, ctxs
        torch.cuda.empty_cache()
        line["extra"] = run_extra(sbw, inputs, dev, peaks)
        line["detect_tokens_per_s"] = line["extra"]["detect_context_N100000"]["tokens_per_s"]
        line["cpu_baseline"] = cpu_baseline()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def cpu_baseline() -> dict:
    """The oracle, untouched, on the host cores: a bounded sample of the headline workload."""
    import torch
    import oracle
    from paper_2609_03844_b200 import inputs

    cores = os.cpu_count() or 1
    x = inputs.as_oracle_array(inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=4242))
    c = inputs.uniform_tokens((B2, 1), V2, seed=4243).numpy()
    oracle.bias_logits(x, V2, c, KEY, GAMMA2, DELTA2, oracle.SCHEME_CONTEXT, threads=cores)
    t0 = time.perf_counter()
    n = 0
    while True:
        oracle.bias_logits(x, V2, c, KEY, GAMMA2, DELTA2, oracle.SCHEME_CONTEXT, threads=cores)
        n += 1
        dt = time.perf_counter() - t0
        if dt * cores > 12.0 or n >= 64:       # about 12 core-seconds of work
            break
    t1 = time.perf_counter()
    oracle.bias_logits(x[:8], V2, c[:8], KEY, GAMMA2, DELTA2, oracle.SCHEME_CONTEXT, threads=1)
    single = 8 * V2 / (time.perf_counter() - t1) / 1e9
    return {"value": B2 * V2 * n / dt / 1e9, "unit": "Gelem/s", "cores": cores, "kind": "oracle",
            "sample": f"{n} decode steps of the headline workload ({n * B2 * V2 / 1e6:.0f} M logits)",
            "single_thread_value": single}


def _time_calls(fn, n, warm=3):
    import torch
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        fn(warm + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e-3 / n


def _time_graph(fn, n, reps=10, warm=3):
    """Device time per call of `n` calls captured into one CUDA graph and replayed `reps` times
    (what a serving loop that replays its decode step sees; stream launches of calls this short
    measure the host instead)."""
    import torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i in range(warm):
            fn(i)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(n):
                fn(warm + i)
        graph.replay()
        side.synchronize()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(side)
        for _ in range(reps):
            graph.replay()
        e1.record(side)
        e1.synchronize()
    torch.cuda.current_stream().wait_stream(side)
    return e0.elapsed_time(e1) * 1e-3 / (n * reps)


def run_extra(sbw, inputs, dev, peaks) -> dict:
    """The other workloads of the hot path, each timed on its own (inputs larger than L2 or
    rotating), and the integer-throughput probe."""
    import torch
    out = {}
    hbm = peaks["hbm_gbs"]

    def place(int_ops, nbytes, seconds):
        t_alu = int_ops / (INT_PEAK_TOPS * 1e12)
        t_hbm = nbytes / (hbm * 1e9)
        return {"bound": "alu" if t_alu >= t_hbm else "hbm", "frac": max(t_alu, t_hbm) / seconds,
                "alu_frac": t_alu / seconds, "hbm_frac": t_hbm / seconds,
                "achieved_tint_ops": int_ops / seconds / 1e12, "achieved_gbs": nbytes / seconds / 1e9}

    # config 3: full-vocabulary self-salt, fp32, B=256, V=151936, gamma .25, delta 4
    B3, V3 = 256, 151936
    p3 = [inputs.add_zipf_spike_(inputs.logits_normal(B3, V3, 4.0, torch.float32, seed=300 + i, device=dev),
                                 V3, seed=310 + i) for i in range(4)]
    c3 = [inputs.uniform_tokens((B3, 1), V3, seed=320 + i, device=dev) for i in range(4)]
    for name, scheme in (("selfsalt", sbw.SCHEME_SELFSALT), ("context", sbw.SCHEME_CONTEXT)):
        s = _time_calls(lambda i: sbw.sbw_bias_logits(p3[i % 4], c3[i % 4], KEY, 0.25, 4.0, scheme), 128)
        n = B3 * V3
        out[f"bias_fp32_{name}_B256_V151936"] = {"gelem_s": n / s / 1e9, "ms": s * 1e3,
                                                 **place(INT_OPS[name] * n, 8 * n, s)}
    # the paper's SBW-ss: self-salt on the top-40 candidates of each row only (same shape)
    s = _time_calls(lambda i: sbw.sbw_bias_logits_topk(p3[i % 4], c3[i % 4], KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT, 40), 128)
    out["bias_top40_fp32_selfsalt_B256_V151936"] = {
        "gelem_s": B3 * V3 / s / 1e9, "ms": s * 1e3, "bound": "hbm",
        "achieved_gbs": 4 * B3 * V3 / s / 1e9, "frac": 4 * B3 * V3 / s / 1e9 / hbm,
        "note": "one read of the row from HBM (4 B/logit), second read from L2, 40 columns written"}
    del p3, c3
    # the same scheme on large batches (1024 rows): fp32 at V = 151936 and bf16 at V = 128256
    for tag, dt, Vk, es in (("fp32", torch.float32, V3, 4), ("bf16", torch.bfloat16, V2, 2)):
        pk = [inputs.logits_normal(1024, Vk, 4.0, dt, seed=440 + i, device=dev) for i in range(2)]
        ck = [inputs.uniform_tokens((1024, 1), Vk, seed=450 + i, device=dev) for i in range(2)]
        s = _time_calls(lambda i: sbw.sbw_bias_logits_topk(pk[i % 2], ck[i % 2], KEY, 0.25, 4.0, sbw.SCHEME_SELFSALT, 40), 32)
        out[f"bias_top40_{tag}_selfsalt_B1024_V{Vk}"] = {
            "gelem_s": 1024 * Vk / s / 1e9, "ms": s * 1e3, "bound": "hbm",
            "achieved_gbs": es * 1024 * Vk / s / 1e9, "frac": es * 1024 * Vk / s / 1e9 / hbm}
        del pk, ck
    # config 2 shape under the self-salt scheme
    p2 = [inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=400 + i, device=dev) for i in range(16)]
    c2 = [inputs.uniform_tokens((B2, 1), V2, seed=420 + i, device=dev) for i in range(16)]
    s = _time_calls(lambda i: sbw.sbw_bias_logits(p2[i % 16], c2[i % 16], KEY, 0.5, 2.0, sbw.SCHEME_SELFSALT), 256)
    out["bias_bf16_selfsalt_B64_V128256"] = {"gelem_s": B2 * V2 / s / 1e9, "ms": s * 1e3,
                                             **place(INT_OPS["selfsalt"] * B2 * V2, 4 * B2 * V2, s)}
    # the headline step on ONE buffer that stays in L2 (16.4 MB): labelled L2-warm, not a roofline input
    s = _time_graph(lambda i: sbw.sbw_bias_logits(p2[0], c2[0], KEY, 0.5, 2.0, sbw.SCHEME_CONTEXT), 64)
    out["bias_bf16_context_B64_V128256_l2_warm_single_buffer"] = {"gelem_s": B2 * V2 / s / 1e9, "ms": s * 1e3}
    del p2, c2
    # config 5 (null half shape): 100000 sequences, lengths uniform in [64, 1024], 218 MB of ids
    N = 100000
    tokens, lengths = inputs.null_token_streams(N, 64, 1024, V2, seed=500, device=dev)
    counts = torch.empty(N, dtype=torch.int32, device=dev)
    z = torch.empty(N, dtype=torch.float64, device=dev)
    ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
    ntok = tokens.numel()
    for name, scheme in (("context", sbw.SCHEME_CONTEXT), ("selfsalt", sbw.SCHEME_SELFSALT)):
        s = _time_calls(lambda i: sbw.sbw_detect(tokens, lengths, KEY, 0.25, scheme, counts, z, workspace=ws), 30)
        out[f"detect_{name}_N100000"] = {"tokens_per_s": ntok / s, "ms": s * 1e3, "tokens": ntok,
                                         **place(INT_OPS[f"detect_{name}"] * ntok, 4 * ntok + 24 * N, s)}
    # evaluation steps on the same streams: distinct-tuple scoring, then ROC-AUC of the z array
    # against alternating labels (timing only: these streams are all unmarked)
    wsu = torch.empty(sbw.sbw_detect_unique_workspace_bytes(N, ntok, 1024), dtype=torch.uint8, device=dev)
    s = _time_calls(lambda i: sbw.sbw_detect_unique(tokens, lengths, 1024, KEY, 0.25, sbw.SCHEME_CONTEXT, counts,
                                                    z, wsu), 20)
    out["detect_unique_context_N100000"] = {"tokens_per_s": ntok / s, "ms": s * 1e3, "tokens": ntok}
    labels = (torch.arange(N, device=dev) % 2).to(torch.uint8)
    auc = torch.empty(1, dtype=torch.float64, device=dev)
    wsr = torch.empty(sbw.sbw_roc_auc_workspace_bytes(N), dtype=torch.uint8, device=dev)
    s = _time_calls(lambda i: sbw.sbw_roc_auc(z, labels, auc, wsr), 20)
    out["roc_auc_N100000"] = {"ms": s * 1e3, "pairs_per_s": (N / 2) ** 2 / s}
    del tokens, wsu
    # config 4: fused sampling sweep, bf16, V=128256, tau 0.7
    for B in (1, 8, 32, 128, 512, 1024):
        x = inputs.logits_normal(B, V2, 4.0, torch.bfloat16, seed=600 + B, device=dev)
        c = inputs.uniform_tokens((B, 1), V2, seed=700 + B, device=dev)
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        wsb = torch.empty(sbw.sbw_sample_workspace_bytes(B, V2), dtype=torch.uint8, device=dev)
        zsum = torch.empty(B, dtype=torch.float32, device=dev)
        for name, scheme in (("context", sbw.SCHEME_CONTEXT), ("selfsalt", sbw.SCHEME_SELFSALT)):
            # with the softmax sum requested every logit is hashed; ids alone let the kernel screen on
            # the Gumbel words first and hash only the candidates that could win
            s = _time_calls(lambda i: sbw.sbw_bias_sample(x, c, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, i, ids, wsb,
                                                          out_sumexp=zsum), 20)
            out[f"sample_bf16_{name}_B{B}"] = {"gelem_s": B * V2 / s / 1e9, "ms": s * 1e3,
                                               "l2_resident": B * V2 * 2 < 100e6}
            s = _time_calls(lambda i: sbw.sbw_bias_sample(x, c, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, i, ids, wsb), 20)
            out[f"sample_ids_only_bf16_{name}_B{B}"] = {"gelem_s": B * V2 / s / 1e9, "ms": s * 1e3}
            if B <= 32:   # calls this short are host-bound as stream launches: device time from a graph
                s = _time_graph(lambda i: sbw.sbw_bias_sample(x, c, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, i, ids, wsb,
                                                              out_sumexp=zsum), 16)
                out[f"sample_bf16_{name}_B{B}"]["graph_ms"] = s * 1e3
                s = _time_graph(lambda i: sbw.sbw_bias_sample(x, c, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, i, ids, wsb), 16)
                out[f"sample_ids_only_bf16_{name}_B{B}"]["graph_ms"] = s * 1e3
    # Appendix F's sampling setting (temperature 0.7, top_p 0.8) and a top-k one, through the truncated sampler
    for B in (64, 1024):
        x = inputs.logits_normal(B, V2, 4.0, torch.bfloat16, seed=600 + B, device=dev)
        c = inputs.uniform_tokens((B, 1), V2, seed=700 + B, device=dev)
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        wsf = torch.empty(sbw.sbw_sample_filtered_workspace_bytes(torch.bfloat16, B, V2), dtype=torch.uint8,
                          device=dev)
        for name, top_k, top_p in (("top_p0.8", 0, 0.8), ("top_k50", 50, 1.0)):
            s = _time_calls(lambda i: sbw.sbw_bias_sample_filtered(x, c, KEY, 0.25, 2.0, sbw.SCHEME_CONTEXT, 0.7,
                                                                   top_k, top_p, 0xC4, i, ids, wsf), 20)
            out[f"sample_filtered_bf16_context_{name}_B{B}"] = {"gelem_s": B * V2 / s / 1e9, "ms": s * 1e3}
    # SBW-ss (self-salt on the top-40 candidates) at the headline shape
    xs = [inputs.logits_normal(B2, V2, 4.0, torch.bfloat16, seed=650 + i, device=dev) for i in range(16)]
    cs = [inputs.uniform_tokens((B2, 1), V2, seed=750 + i, device=dev) for i in range(16)]
    s = _time_calls(lambda i: sbw.sbw_bias_logits_topk(xs[i % 16], cs[i % 16], KEY, 0.25, 2.0, sbw.SCHEME_SELFSALT, 40),
                    256)
    out["topk40_bf16_selfsalt_B64_V128256"] = {"gelem_s": B2 * V2 / s / 1e9, "ms": s * 1e3}
    del xs, cs
    # the paper's isolated-benchmark protocol (Appendix D: fresh (B, 151936) logits, 20 warm-up + 200
    # timed calls, CUDA events, synchronise between calls, p50/p99) on its two full-vocabulary schemes
    # with context width 4 (SBW-4, SBW-ss-V); fp32 logits (the paper does not state its dtype)
    sweep = {}
    for B in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512):
        x = inputs.logits_normal(B, 151936, 4.0, torch.float32, seed=800 + B, device=dev)
        c = inputs.uniform_tokens((B, 4), 151936, seed=900 + B, device=dev)
        for name, scheme in (("sbw4", sbw.SCHEME_CONTEXT), ("sbw_ss_v", sbw.SCHEME_SELFSALT)):
            times = []
            for i in range(220):
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record()
                sbw.sbw_bias_logits(x, c, KEY, 0.25, 2.0, scheme)
                e1.record()
                torch.cuda.synchronize()
                if i >= 20:
                    times.append(e0.elapsed_time(e1))
            times.sort()
            sweep[f"{name}_B{B}"] = {"p50_ms": times[len(times) // 2], "p95_ms": times[int(len(times) * 0.95)],
                                     "p99_ms": times[int(len(times) * 0.99)],
                                     "l2_resident": B * 151936 * 4 < 100e6}
    out["paper_protocol_latency_fp32_V151936_W4"] = sweep
    # integer-throughput probe
    probes = {}
    for kind in ("mulwide", "lop3", "iadd3", "imad", "philox", "ffma"):
        r = sbw.sbw_int_probe(kind, steps=8192, blocks_per_sm=4, threads=256)
        probes[kind] = {"ops_per_clk_per_sm": r["ops_per_clk_per_sm"], "tops": r["ops_per_s"] / 1e12,
                        "sm_mhz": r["sm_mhz_implied"]}
    out["int_probe"] = probes
    return out


PROFILE_CASES = ("topk40_fp32_selfsalt", "bias_bf16_context", "bias_bf16_selfsalt", "bias_fp32_context", "bias_fp32_selfsalt",
                 "detect_context", "detect_selfsalt", "sample_bf16_context", "sample_bf16_selfsalt",
                 "detectunique_context", "filtered_bf16_context", "sampleids_bf16_context", "sampleids_bf16_selfsalt", "filteredtopk_bf16_context")


def run_profile_case(name: str, launches: int) -> None:
    """A few launches of one kernel on an input larger than L2 and small enough for a profiler
    capture (a few hundred MB): 3 warm-up launches, then `launches` more.  Prints the launch count;
    numbers printed under a profiler are never bench values."""
    import torch
    import paper_2609_03844_b200 as sbw
    from paper_2609_03844_b200 import inputs

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    kind, dt, scheme_name = (name.split("_") + [""])[:3] if not name.startswith("detect") else \
        (name.split("_")[0], "", name.split("_")[1])
    scheme = sbw.SCHEME_SELFSALT if scheme_name == "selfsalt" else sbw.SCHEME_CONTEXT
    if kind in ("detect", "detectunique"):
        N = 100000
        tokens, lengths = inputs.null_token_streams(N, 64, 1024, V2, seed=500, device=dev)
        counts = torch.empty(N, dtype=torch.int32, device=dev)
        z = torch.empty(N, dtype=torch.float64, device=dev)
        if kind == "detect":
            ws = torch.empty(sbw.sbw_detect_workspace_bytes(N), dtype=torch.uint8, device=dev)
            fn = lambda i: sbw.sbw_detect(tokens, lengths, KEY, 0.25, scheme, counts, z, workspace=ws)  # noqa: E731
        else:
            ws = torch.empty(sbw.sbw_detect_unique_workspace_bytes(N, tokens.numel(), 1024), dtype=torch.uint8,
                             device=dev)
            fn = lambda i: sbw.sbw_detect_unique(tokens, lengths, 1024, KEY, 0.25, scheme, counts, z, ws)  # noqa: E731
    elif kind in ("filtered", "filteredtopk"):
        B = 512
        x = inputs.logits_normal(B, V2, 4.0, torch.bfloat16, seed=1, device=dev)
        ctx = inputs.uniform_tokens((B, 1), V2, seed=2, device=dev)
        ids = torch.empty(B, dtype=torch.int32, device=dev)
        ws = torch.empty(sbw.sbw_sample_filtered_workspace_bytes(x.dtype, B, V2), dtype=torch.uint8, device=dev)
        top_k, top_p = (50, 0.9) if kind == "filteredtopk" else (0, 0.8)
        fn = lambda i: sbw.sbw_bias_sample_filtered(x, ctx, KEY, 0.25, 2.0, scheme, 0.7, top_k, top_p, 0xC4, i, ids, ws)  # noqa: E731
    else:
        B, V, dtype = (512, V2, torch.bfloat16) if dt == "bf16" else (256, 151936, torch.float32)
        x = inputs.logits_normal(B, V, 4.0, dtype, seed=1, device=dev)
        ctx = inputs.uniform_tokens((B, 1), V, seed=2, device=dev)
        if kind == "topk40":
            fn = lambda i: sbw.sbw_bias_logits_topk(x, ctx, KEY, 0.25, 4.0, scheme, 40)  # noqa: E731
        elif kind == "bias":
            fn = lambda i: sbw.sbw_bias_logits(x, ctx, KEY, 0.5, 2.0, scheme)  # noqa: E731
        else:
            ids = torch.empty(B, dtype=torch.int32, device=dev)
            zsum = torch.empty(B, dtype=torch.float32, device=dev) if kind == "sample" else None
            ws = torch.empty(sbw.sbw_sample_workspace_bytes(B, V), dtype=torch.uint8, device=dev)
            fn = lambda i: sbw.sbw_bias_sample(x, ctx, KEY, 0.25, 2.0, scheme, 0.7, 0xC4, i, ids, ws,  # noqa: E731
                                               out_sumexp=zsum)
    for i in range(3 + launches):
        fn(i)
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": name, "launches": 3 + launches}))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2048)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches only")
    ap.add_argument("--no-extra", action="store_true", help="skip the secondary workloads and the CPU baseline")
    ap.add_argument("--profile-case", choices=PROFILE_CASES, default=None,
                    help="run a few launches of one kernel on a small (> L2) input, for a profiler")
    ap.add_argument("--profile-launches", type=int, default=3)
    args = ap.parse_args()
    if args.profile_case:
        run_profile_case(args.profile_case, args.profile_launches)
        return
    if args.impl == "reference":
        if args.steps == 2048:
            args.steps, args.warmup = 32, 3
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

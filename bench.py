#!/usr/bin/env python
"""Benchmark of the R-Stitch routing-decision path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole hot path (LM-head contraction, entropy, greedy token, threshold
rule, ordered compaction, stitched-span lengths) over one synthetic batch.  The default workload
is the SLM head at batch 1 (d = 1536, V = 151936), the configuration the metric is quoted on.
With N > 1 (one process per GPU under torch.distributed.run) every rank decides its own
sequences against a replicated head: the path shards by rows with no data-path collective, so
scaling is weak and the value is the sum over ranks divided by the slowest rank's time.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import rstitch_inputs as gen

METRIC = "routing decisions/sec (fused head+entropy+route) and achieved HBM GB/s vs peak"
UNIT = "decisions/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0

BENCH_WORKLOADS = {
    "c2_slm_b1": ("c2_slm_b1",), "c3_llm_b1": ("c3_llm_b1",), "c3_llm_b4": ("c3_llm_b4",),
    "c3_llm_b16": ("c3_llm_b16",), "c4_slm_b64": ("c4_slm_b64",),
    "c4_batched": ("c4_slm_b64", "c4_llm_b64"), "c5_catchup": ("c5_catchup",), "c1_tiny": ("c1_tiny",),
    # one round of the batched hybrid decode loop (Algorithm 1) for 64 sequences, all on the device, two
    # launches: the SLM head on the sequences decoding on the SLM, the LLM head on the others, each applying
    # Algorithm 1's decision block in its own tail, the LLM's call also planning the next round
    "alg1_b64": ("c4_slm_b64", "c4_llm_b64"),
    # the same round with Algorithm 1's R-Stitch+ lines, three launches: the SLM head (no decision block), the
    # router on the rows above the threshold, whose last block refines the mask and runs the SLM's decision
    # block on it, and the LLM head with its decision block and the next planning
    "alg1_plus_b64": ("c4_slm_b64", "c4_llm_b64"),
    # R-Stitch+ step, two launches: SLM head on 64 sequences, then the router on the rows the entropy rule
    # routed with the compaction of its refined mask in the same kernel
    "c4_router": ("c4_slm_b64",),
}


# ------------------------------------------------------------------------------------------
# clocks: read-only NVML polling during the timed region
# ------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x100: "display_clock_setting", 0x10: "sync_boost"}

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reason_bits, self.power = [], 0, []
        self.sm_max = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self.period = period_s

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2.0)

    def summary(self) -> dict:
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["unavailable"]}
        reasons = sorted(name for bit, name in self.REASONS.items() if self.reason_bits & bit)
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def measured_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            p = json.load(open(path))
            return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                    "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS,
            "bf16_tflops_sustained": FALLBACK_BF16_TFLOPS_SUSTAINED, "source": "fallback"}


# DRAM bytes (read + write) per launch of the dominant (head) kernel, from the ncu captures summarised under
# profiles/.  Each entry names the kernel sources it was taken with (sha256 of the files under csrc/):
# once any of them has changed the counters no longer describe the kernel and the figure reads null.
NCU_TRAFFIC = {
    "c2_slm_b1":
    {"bytes": 470766592, "summary": "profiles/head_stream_kernel_c2_slm_b1.md",
     "sources": {"rstitch_gemv.cu": "46622a9ca185e4b62ecd29c125a00875a0d28e9416790789c855643721c5222e", "rstitch_kernels.cuh": "9d5e477d91dc22a265a8430f1ac19aba750e147118779e27533337225eba6f34", "rstitch_tail.cuh": "6f57211cd838c59082c6ae636fc198557d5a6c8a6a4bda2d4a48324bb8541ce6", "rstitch_alg1.cuh": "a14e9fd9944096aff664d96854f70a356e706967772dc0d918a7f7fcccc55f0f", "rstitch_stats.cuh": "e9ff9c67605d61e89d9db77ba12376630bd3a612160977946ac7e2aadd51542e", "rstitch_ptx.cuh": "3b15b917fd957debc456aa9fe0e557fa4769f476479b08233d396504eb3cdf8c", "rstitch_sample.cuh": "40e02e3cd65cde7d19108dd6ae55f59fc1d1b0ee1171efe6f0de23e5cff04f71", "rstitch_finalize.cu": "7c388069cec80e69781d2fc0a46b5d6a71aeed12db1bc249e0bc60adb9f80107"}},
    "c3_llm_b1":
    {"bytes": 1094197912, "summary": "profiles/head_stream_kernel_c3_llm_b1.md",
     "sources": {"rstitch_gemv.cu": "46622a9ca185e4b62ecd29c125a00875a0d28e9416790789c855643721c5222e", "rstitch_kernels.cuh": "9d5e477d91dc22a265a8430f1ac19aba750e147118779e27533337225eba6f34", "rstitch_tail.cuh": "6f57211cd838c59082c6ae636fc198557d5a6c8a6a4bda2d4a48324bb8541ce6", "rstitch_alg1.cuh": "a14e9fd9944096aff664d96854f70a356e706967772dc0d918a7f7fcccc55f0f", "rstitch_stats.cuh": "e9ff9c67605d61e89d9db77ba12376630bd3a612160977946ac7e2aadd51542e", "rstitch_ptx.cuh": "3b15b917fd957debc456aa9fe0e557fa4769f476479b08233d396504eb3cdf8c", "rstitch_sample.cuh": "40e02e3cd65cde7d19108dd6ae55f59fc1d1b0ee1171efe6f0de23e5cff04f71", "rstitch_finalize.cu": "7c388069cec80e69781d2fc0a46b5d6a71aeed12db1bc249e0bc60adb9f80107"}},
    "c3_llm_b16":
    {"bytes": 1094429312, "summary": "profiles/head_umma_kernel_c3_llm_b16.md",
     "sources": {"rstitch_umma.cu": "71930ba3f0ec83a8479520e7eea7171908ed223a08bfbf93968346a06c57164f", "rstitch_kernels.cuh": "9d5e477d91dc22a265a8430f1ac19aba750e147118779e27533337225eba6f34", "rstitch_tail.cuh": "6f57211cd838c59082c6ae636fc198557d5a6c8a6a4bda2d4a48324bb8541ce6", "rstitch_alg1.cuh": "a14e9fd9944096aff664d96854f70a356e706967772dc0d918a7f7fcccc55f0f", "rstitch_stats.cuh": "e9ff9c67605d61e89d9db77ba12376630bd3a612160977946ac7e2aadd51542e", "rstitch_ptx.cuh": "3b15b917fd957debc456aa9fe0e557fa4769f476479b08233d396504eb3cdf8c", "rstitch_sample.cuh": "40e02e3cd65cde7d19108dd6ae55f59fc1d1b0ee1171efe6f0de23e5cff04f71", "rstitch_finalize.cu": "7c388069cec80e69781d2fc0a46b5d6a71aeed12db1bc249e0bc60adb9f80107"}},
    "c4_slm_b64":
    {"bytes": 471256832, "summary": "profiles/head_umma_kernel_c4_slm_b64.md",
     "sources": {"rstitch_umma.cu": "71930ba3f0ec83a8479520e7eea7171908ed223a08bfbf93968346a06c57164f", "rstitch_kernels.cuh": "9d5e477d91dc22a265a8430f1ac19aba750e147118779e27533337225eba6f34", "rstitch_tail.cuh": "6f57211cd838c59082c6ae636fc198557d5a6c8a6a4bda2d4a48324bb8541ce6", "rstitch_alg1.cuh": "a14e9fd9944096aff664d96854f70a356e706967772dc0d918a7f7fcccc55f0f", "rstitch_stats.cuh": "e9ff9c67605d61e89d9db77ba12376630bd3a612160977946ac7e2aadd51542e", "rstitch_ptx.cuh": "3b15b917fd957debc456aa9fe0e557fa4769f476479b08233d396504eb3cdf8c", "rstitch_sample.cuh": "40e02e3cd65cde7d19108dd6ae55f59fc1d1b0ee1171efe6f0de23e5cff04f71", "rstitch_finalize.cu": "7c388069cec80e69781d2fc0a46b5d6a71aeed12db1bc249e0bc60adb9f80107"}},
    "c5_catchup":
    {"bytes": 1673064760, "summary": "profiles/head_umma2_kernel_c5_catchup.md",
     "sources": {"rstitch_umma.cu": "71930ba3f0ec83a8479520e7eea7171908ed223a08bfbf93968346a06c57164f", "rstitch_kernels.cuh": "9d5e477d91dc22a265a8430f1ac19aba750e147118779e27533337225eba6f34", "rstitch_tail.cuh": "6f57211cd838c59082c6ae636fc198557d5a6c8a6a4bda2d4a48324bb8541ce6", "rstitch_alg1.cuh": "a14e9fd9944096aff664d96854f70a356e706967772dc0d918a7f7fcccc55f0f", "rstitch_stats.cuh": "e9ff9c67605d61e89d9db77ba12376630bd3a612160977946ac7e2aadd51542e", "rstitch_ptx.cuh": "3b15b917fd957debc456aa9fe0e557fa4769f476479b08233d396504eb3cdf8c", "rstitch_sample.cuh": "40e02e3cd65cde7d19108dd6ae55f59fc1d1b0ee1171efe6f0de23e5cff04f71", "rstitch_finalize.cu": "7c388069cec80e69781d2fc0a46b5d6a71aeed12db1bc249e0bc60adb9f80107"}},
}


def recorded_traffic(workload: str):
    import hashlib
    ent = NCU_TRAFFIC.get(workload)
    if not ent:
        return None
    csrc = os.path.join(ROOT, "paper_2507_17307_b200", "csrc")
    try:
        for name, digest in ent["sources"].items():
            if hashlib.sha256(open(os.path.join(csrc, name), "rb").read()).hexdigest() != digest:
                return None
    except OSError:
        return None
    return ent["bytes"]


# ------------------------------------------------------------------------------------------
# workload state
# ------------------------------------------------------------------------------------------
_W_CACHE = {}


def build_batches(names, n_rot: int, rank: int):
    """Host-side synthetic inputs: per head its W bits and n_rot rotating hidden batches."""
    heads = []
    for name in names:
        w = gen.WORKLOADS[name]
        key = (w.seed, w.d, w.V, w.sigma_w)
        if key not in _W_CACHE:                 # workloads that share a head draw it once
            _W_CACHE[key] = gen.make_w_head(w)
        w_bits = _W_CACHE[key]
        batches = []
        for i in range(n_rot):
            step = rank * 100003 + i
            if w.span_max > 1:
                k = gen.make_spans(w, step)
                R = int(k.sum())
                row_seq = np.repeat(np.arange(w.B, dtype=np.int32), k)
                hid, _ = gen.make_hidden(w, w_bits, step, rows=R)
                seq_len, kv_len = gen.make_kv_state(w, step, span=k)
            else:
                R, row_seq = w.B, None
                hid, _ = gen.make_hidden(w, w_bits, step)
                seq_len, kv_len = gen.make_kv_state(w, step)
            batches.append({"hid": hid, "R": R, "row_seq": row_seq, "seq_len": seq_len, "kv_len": kv_len})
        heads.append({"w": w, "w_bits": w_bits, "batches": batches})
    return heads


def run_reference(args, names) -> dict:
    """The oracle as it stands, on the host cores, same metric / config."""
    import oracle
    oracle.build()
    heads = build_batches(names, max(2, min(4, args.steps)), 0)
    # a step is a bounded sample of the workload: at most `sample_rows` rows of each head's batch
    sample_rows = 8 if sum(h["batches"][0]["R"] for h in heads) > 16 else None

    def one_step(i):
        rows = 0
        for h in heads:
            b = h["batches"][i % len(h["batches"])]
            hid = b["hid"] if sample_rows is None else b["hid"][:sample_rows]
            oracle.route(hid, h["w_bits"], h["w"].tau_nats)
            rows += hid.shape[0]
        return rows
    for i in range(args.warmup):
        one_step(i)
    t0 = time.perf_counter()
    rows = 0
    for i in range(args.steps):
        rows += one_step(i)
    dt = time.perf_counter() - t0
    value = rows / dt
    sample = ("every row of each step" if sample_rows is None else
              "first %d rows of each head's batch per step" % sample_rows)
    w0 = heads[0]["w"]
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "B": w0.B, "d": w0.d, "V": w0.V},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def run_vocab_parallel(args, names, rank, local_rank, world) -> int:
    """The head split by vocabulary rows over the ranks: every rank runs the head kernels on its rows of
    W_head for ALL rows of the batch, one all-gather moves 20 bytes per row and rank, every rank merges
    and decides.  Total work is fixed as ranks are added ("strong")."""
    import torch
    import paper_2507_17307_b200 as rs
    from paper_2507_17307_b200 import build as rs_build, sharding
    if rank == 0:
        rs_build.build_library()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    rs.lib()
    dev = torch.device("cuda", local_rank)
    K = args.steps if args.steps is not None else 4096
    Wm = max(args.warmup if args.warmup is not None else 64, 3)
    n_rot = 8
    head = build_batches(names[:1], n_rot, 0)[0]          # every rank sees the same rows
    w = head["w"]
    v_lo, v_hi = sharding.vocab_shard(w.V, rank, world)
    w_dev = torch.from_numpy(head["w_bits"][v_lo:v_hi].view(np.int16)).to(dev).view(torch.bfloat16)
    hd = rs.Handle(max(w.B, 64), w.d, w.V)
    stream = torch.cuda.current_stream()
    hid_dev = [torch.from_numpy(b["hid"].view(np.int16)).to(dev).view(torch.bfloat16) for b in head["batches"]]
    hid_pin = [torch.from_numpy(b["hid"].view(np.int16)).view(torch.bfloat16).pin_memory() for b in head["batches"]]
    mine = torch.zeros((w.B, rs.SHARD_WORDS), dtype=torch.int32, device=dev)
    gathered = torch.zeros((world, w.B, rs.SHARD_WORDS), dtype=torch.int32, device=dev)
    outs = [rs.RouteOutputs.allocate(w.B, w.B, dev) for _ in range(n_rot)]

    def step(i, hid=None):
        j = i % n_rot
        rs.shard_stats(hd, hid_dev[j] if hid is None else hid, w_dev, v_lo, flags=args.flags, stream=stream,
                       out=mine if world > 1 else gathered[0])
        if world > 1:
            sharding.gather_shard_stats(mine, dist, out=gathered)
        rs.shard_route(hd, gathered, w.V, w.tau_nats, stream=stream, out=outs[j])

    for i in range(Wm):
        step(i)
    torch.cuda.synchronize()
    rs.last_status(hd)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    with ClockSampler(visible_gpu_index(local_rank)) as clocks:
        ev0.record(stream)
        for i in range(K):
            step(i)
        ev1.record(stream)
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    st = rs.last_status(hd)
    if st["timeouts"] or st["nan_rows"]:
        raise SystemExit("device status after the timed region: %s" % st)
    launches = st["launches"]

    # end to end: hidden from pinned host memory every step, the decision back in pinned host memory
    host_out = {k: torch.empty_like(getattr(outs[0], k), device="cpu").pin_memory()
                for k in ("tok", "ent", "mask", "llm_idx", "llm_count")}
    stage = torch.empty_like(hid_dev[0])

    def host_step(i):
        stage.copy_(hid_pin[i % n_rot], non_blocking=True)
        step(i, stage)
        for k, t in host_out.items():
            t.copy_(getattr(outs[i % n_rot], k), non_blocking=True)
        stream.synchronize()

    Ke = max(1, min(K, 1024))
    for i in range(3):
        host_step(i)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        host_step(i)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    rs.last_status(hd)
    ms, _, launches = sharding.reduce_step_stats(ms, 0.0, launches, dist, dev)
    e2e_s, _, _ = sharding.reduce_step_stats(e2e_s, 0.0, 0, dist, dev)
    if rank == 0:
        peaks = measured_peaks()
        per_step_s = ms / 1e3 / K
        shard_bytes = (v_hi - v_lo) * w.d * 2               # rank 0's shard, the largest
        achieved = shard_bytes / per_step_s / 1e9
        line = {
            "metric": METRIC, "value": w.B * K / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload + " (vocabulary-parallel)", "B": w.B, "rows_per_step": float(w.B),
                       "d": w.d, "V": w.V, "tau_nats": w.tau_nats, "heads": list(names[:1]),
                       "path": [rs.path_name(w.B, w.d, v_hi - v_lo, args.flags)],
                       "l2": "inputs larger than L2: each step streams the rank's whole W_head shard (%.0f MB); "
                             "hidden rotates over %d buffers" % (shard_bytes / 1e6, n_rot),
                       "parallelism": "tp%d (W_head rows sharded, all-gather of %d B per row and rank, every rank "
                                      "decides)" % (world, 4 * rs.SHARD_WORDS)},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                         "peak_source": "of " + peaks["source"],
                         "note": "per GPU: the rank's shard bytes over the whole step (head kernel, gather, merge)"},
            "clocks": clocks.summary(), "gpu_launches": launches,
            "algorithmic_bytes_per_step": shard_bytes,
            "e2e": {"value": w.B * Ke / e2e_s, "unit": UNIT, "h2d_bytes_per_step": w.B * w.d * 2,
                    "d2h_bytes_per_step": sum(t.numel() * t.element_size() for t in host_out.values()),
                    "steps": Ke, "note": "hidden from pinned host memory, decision back to pinned host memory, "
                                         "stream synchronised every step; the W_head shard resident"},
        }
        print(json.dumps(line), flush=True)
    hd.destroy()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def free_port() -> int:
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
        sk.bind(("127.0.0.1", 0))
        return int(sk.getsockname()[1])


def needs_spawn(gpus: int, env) -> bool:
    """--gpus N > 1 without a launcher's environment: this process starts the N ranks itself."""
    return gpus > 1 and "WORLD_SIZE" not in env and "RANK" not in env


def default_steps(workload: str):
    """(steps, warm-up, rotating buffers) when the command line leaves them open."""
    if workload == "c5_catchup":
        return 64, 3, 2
    if workload in ("c4_batched", "alg1_b64", "alg1_plus_b64"):
        return 2048, 64, 8
    return 8192, 64, 8


def read_stream_ceiling(rs, torch, dev, stream) -> dict:
    """Bandwidth of a read-only pass over 2 GiB with the streaming head kernel's own copy pipeline."""
    n = 2 << 30
    buf = torch.empty(n, dtype=torch.uint8, device=dev)
    buf.zero_()
    gave_up = torch.zeros(1, dtype=torch.int32, device=dev)
    for _ in range(3):
        rs.probe_read_stream(buf, gave_up, stream=stream)
    torch.cuda.synchronize()
    best, times = None, []
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        rs.probe_read_stream(buf, gave_up, stream=stream)
        e1.record(stream)
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    if int(gave_up.item()) != 0:
        return {"gbs": None, "note": "a bounded wait ran out: no figure"}
    del buf
    torch.cuda.empty_cache()
    ms = float(np.median(times))
    return {"gbs": n / (ms / 1e3) / 1e9, "gbs_best": n / (min(times) / 1e3) / 1e9, "bytes": n,
            "how": "rstitch_probe_read_stream: 148 blocks, bulk copies into a shared-memory ring, nothing written; "
                   "median of 10 passes, CUDA events"}


def measure(rs, torch, dist, rank, local_rank, world, args, workload: str, K: int, Wm: int, n_rot: int,
            with_e2e: bool, min_region_s: float = 0.2) -> dict:
    """Build one workload on this rank's GPU, time `repeats` regions of exactly K steps each with CUDA
    events on the launching stream, and (with_e2e) the same steps through the host-buffer entry point."""
    names = BENCH_WORKLOADS[workload]
    heads = build_batches(names, n_rot, rank)
    dev = torch.device("cuda", local_rank)

    def bf16_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    def i32_dev(a):
        return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev)

    stream = torch.cuda.current_stream()
    alg1 = workload in ("alg1_b64", "alg1_plus_b64")
    alg1_plus = workload == "alg1_plus_b64"
    state = None
    if alg1:
        B0 = gen.WORKLOADS[names[0]].B
        state = rs.Alg1State(B0, y_cap=64, device=dev)
        state.init(i32_dev(np.random.default_rng(4242 + rank).integers(16, 2048, size=B0)), stream=stream)
        # fitted coefficients printed in the paper's latency-regression appendix (SLM-1.5B, LLM-7B), ms
        lat_models = [rs.LatencyModel(0.000021, 0.000231, -0.121046, 27.090929),
                      rs.LatencyModel(0.000027, 0.000031, -0.045256, 27.040801)]
    with_router = workload == "c4_router" or alg1_plus
    router = None
    if with_router:
        d0 = gen.WORKLOADS[names[0]].d
        rw = gen.make_router_weights(d0, 32, 64, 6, seed=77)      # 0.07 M parameters at d = 1536
        router = rs.Router({k: torch.from_numpy(v).to(dev) for k, v in rw.items()})
        r_logits = torch.zeros((64, 2), dtype=torch.float32, device=dev)
        r_switch = torch.zeros(64, dtype=torch.uint8, device=dev)
        r_idx = torch.zeros(64, dtype=torch.int32, device=dev)
        r_cnt = torch.zeros(1, dtype=torch.int32, device=dev)
    alg1_tails = []
    handles, prepared = [], [[] for _ in range(n_rot)]
    prev_out = [None] * n_rot
    algo_bytes = 0
    flops = 0.0
    for hi, h in enumerate(heads):
        w = h["w"]
        Rmax = max(b["R"] for b in h["batches"])
        hd = rs.Handle(max(Rmax, 64), w.d, w.V)
        handles.append(hd)
        w_dev = bf16_dev(h["w_bits"])
        h["w_dev"] = w_dev
        algo_bytes += w.V * w.d * 2
        for i, b in enumerate(h["batches"]):
            R = b["R"]
            out = rs.RouteOutputs.allocate(R, w.B, dev, spans=True)
            kw = dict(R=R, B=w.B, seq_len=i32_dev(b["seq_len"]), kv_len=i32_dev(b["kv_len"]),
                      row_seq=i32_dev(b["row_seq"]), flags=args.flags, stream=stream)
            if alg1:
                # run entry j of the model's batch reads row j of the pool; the live count is plan's, on device;
                # the call's own tail applies the decision block, the LLM's call also plans the next round
                if len(alg1_tails) <= hi:
                    alg1_tails.append(state.tail(hi, -1, spans=False, plan_next=(hi == 1), t_max=1 << 30,
                                                 latency=lat_models))
                kw = dict(R=w.B, B=w.B, n_rows_dev=state.run_count[hi], flags=args.flags, stream=stream,
                          alg1_tail=None if (alg1_plus and hi == 0) else alg1_tails[hi])
            elif hi == 1:
                # batched step: the LLM head runs on the subset the SLM head routed, count on device
                kw.update(row_idx=prev_out[i].llm_idx, n_rows_dev=prev_out[i].llm_count)
            prepared[i].append(rs.PreparedCall(hd, bf16_dev(b["hid"]), w_dev, w.tau_nats, out, **kw))
            if hi == 0:
                prev_out[i] = out
        flops += 2.0 * np.mean([b["R"] for b in h["batches"]]) * w.d * w.V
    w0 = heads[0]["w"]
    rows_per_step = float(np.mean([b["R"] for b in heads[0]["batches"]]))

    if alg1:
        # the first round's plans; every later round is planned by the LLM call of the round before
        state.plan(0, 1 << 30, lat_models[0], stream=stream)
        state.plan(1, 1 << 30, lat_models[1], stream=stream)

    def step(i):
        calls = prepared[i % n_rot]
        for ci, call in enumerate(calls):
            st = call.launch()
            if st != 0:
                raise rs.RstitchError(st, "rstitch_route_ex")
            if alg1_plus and ci == 0:
                o = call.out
                router.route(call._keep[1], 64, o.llm_idx, o.mask, r_idx, r_cnt, n_rows_dev=o.llm_count,
                             logits=r_logits, switch=r_switch, stream=stream, alg1_tail=alg1_tails[0], tok=o.tok,
                             n_seq_dev=state.run_count[0])
        if with_router and not alg1_plus:
            o = calls[0].out
            router.route(calls[0]._keep[1], 64, o.llm_idx, o.mask, r_idx, r_cnt, n_rows_dev=o.llm_count,
                         logits=r_logits, switch=r_switch, stream=stream)

    for i in range(Wm):
        step(i)
    torch.cuda.synchronize()
    warm_launches = sum(rs.last_status(hd)["launches"] for hd in handles)     # also clears the counters
    launches_per_step = warm_launches / float(Wm) + (1 if with_router else 0)

    graph = None
    if args.graph:
        # the step loop has no host synchronisation, so a whole rotation of steps records into one graph
        K = max(n_rot, (K // n_rot) * n_rot)
        cap_stream = torch.cuda.Stream()
        cap_stream.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(cap_stream):
            for calls in prepared:
                for c in calls:
                    c._stream = int(cap_stream.cuda_stream)
            saved = stream
            stream = cap_stream
            with torch.cuda.graph(graph, stream=cap_stream):
                for i in range(n_rot):
                    step(i)
            stream = saved
            for calls in prepared:
                for c in calls:
                    c._stream = int(saved.cuda_stream) or None
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        for hd in handles:
            rs.last_status(hd)

    def region():
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(torch.cuda.current_stream())
        if graph is not None:
            for _ in range(K // n_rot):
                graph.replay()
        else:
            for i in range(K):
                step(i)
        ev1.record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        return ev0.elapsed_time(ev1)

    # every region times exactly K steps; regions are repeated until they add up to min_region_s
    # (at least three), the step time reported is the median region's
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    times = []
    with ClockSampler(visible_gpu_index(local_rank)) as clocks:
        total = 0.0
        while len(times) < 3 or (total < min_region_s * 1e3 and len(times) < 400):
            ms_r = region()
            times.append(ms_r)
            total += ms_r
    if dist is not None:
        dist.barrier()
    repeats = n_run = len(times)
    if dist is not None and world > 1:
        # every rank runs the same number of regions: the fewest any rank chose
        t = torch.tensor([repeats], dtype=torch.int64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        repeats = int(t.item())
        times = times[:repeats]
    ms = float(np.median(times))
    stats = [rs.last_status(hd) for hd in handles]
    launches_all = sum(st["launches"] for st in stats) + (n_run * K if with_router else 0)
    launches = int(round(launches_all / float(n_run))) if graph is None else int(round(K * launches_per_step))
    if any(st["timeouts"] or st["nan_rows"] for st in stats):
        raise SystemExit("device status after the timed region: %s" % stats)

    res = {"workload": workload, "names": names, "heads": heads, "K": K, "Wm": Wm, "n_rot": n_rot, "ms": ms,
           "ms_min": float(min(times)), "ms_max": float(max(times)), "repeats": repeats, "launches": launches,
           "clocks": clocks.summary(), "algo_bytes": algo_bytes, "flops": flops, "rows_per_step": rows_per_step,
           "w0": w0, "handles": handles, "dev": dev,
           "path": [rs.path_name(int(rows_per_step), h["w"].d, h["w"].V, args.flags) for h in heads]}
    if not with_e2e:
        return res

    # end to end: the same step through rstitch_route_ex_host -- every per-step input starts in pinned
    # host memory, every output lands in host memory, copies and the stream synchronisation are inside
    # the timed region.  W_head is a model weight and stays resident.
    def pin(a, dt=None):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a))
        if dt is not None:
            t = t.view(dt)
        return t.pin_memory()

    host_calls = [[] for _ in range(n_rot)]
    h2d = d2h = 0
    for hi, h in enumerate([] if alg1 else heads):
        w = h["w"]
        for i, b in enumerate(h["batches"]):
            R = b["R"]
            ho = {"tok": torch.empty(max(R, 1), dtype=torch.int32).pin_memory(),
                  "ent": torch.empty(max(R, 1), dtype=torch.float32).pin_memory(),
                  "mask": torch.empty(w.B, dtype=torch.uint8).pin_memory(),
                  "llm_idx": torch.empty(w.B, dtype=torch.int32).pin_memory(),
                  "llm_count": torch.zeros(1, dtype=torch.int32).pin_memory(),
                  "llm_span": torch.empty(w.B, dtype=torch.int32).pin_memory(),
                  "llm_row_off": torch.empty(w.B + 1, dtype=torch.int32).pin_memory()}
            kw = dict(R=R, B=w.B, seq_len=pin(b["seq_len"]), kv_len=pin(b["kv_len"]), row_seq=pin(b["row_seq"]),
                      flags=args.flags, stream=stream)
            if hi == 1:
                kw.update(row_idx=host_calls[i][0].out["llm_idx"])     # the subset the SLM head routed
            host_calls[i].append(rs.PreparedHostCall(handles[hi], pin(b["hid"].view(np.int16), torch.bfloat16),
                                                     h["w_dev"], w.tau_nats, ho, **kw))
            if i == 0:
                n_idx = (R if b["row_seq"] is not None else 0) + (R if hi == 1 else 0) + 2 * w.B
                h2d += b["hid"].shape[0] * w.d * 2 + 4 * n_idx
                d2h += 8 * R + w.B + 4 * w.B + 4 + 4 * w.B + 4 * (w.B + 1)

    if alg1:
        # host-fed variant of the same round: both hidden pools come from pinned host memory every round
        # and the per-sequence token counts go back to the host, with a stream synchronisation
        pools_host = [[pin(b["hid"].view(np.int16), torch.bfloat16) for b in h["batches"]] for h in heads]
        pools_dev = [[prepared[i][hi]._keep[1] for i in range(n_rot)] for hi in range(2)]
        n_out_host = torch.zeros(state.B, dtype=torch.int32).pin_memory()
        h2d = sum(p[0].numel() * 2 for p in pools_host)
        d2h = state.B * 4

    def host_step_alg1(i):
        for hi in range(2):
            pools_dev[hi][i % n_rot].copy_(pools_host[hi][i % n_rot], non_blocking=True)
        step(i)
        n_out_host.copy_(state.n_out[:state.B], non_blocking=True)
        stream.synchronize()

    def host_step(i):
        if alg1:
            return host_step_alg1(i)
        calls = host_calls[i % n_rot]
        st = calls[0].launch()
        if st != 0:
            raise rs.RstitchError(st, "rstitch_route_ex_host")
        if len(calls) > 1:
            cnt = int(calls[0].out["llm_count"][0])          # host-driven: the count is on the host now
            if cnt > 0:
                calls[1].set_rows(cnt)
                st = calls[1].launch()
                if st != 0:
                    raise rs.RstitchError(st, "rstitch_route_ex_host")

    Ke = max(1, min(K, 2048 if workload != "c5_catchup" else 32))
    for i in range(3):
        host_step(i)
    torch.cuda.synchronize()
    e2e_times = []
    reps_e = 3 if Ke >= 256 else max(3, min(50, int(0.1 / max(1e-6, Ke * ms / K / 1e3))))
    for _ in range(reps_e):
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(Ke):
            host_step(i)
        torch.cuda.synchronize()
        e2e_times.append(time.perf_counter() - t0)
    res["e2e"] = {"seconds": float(np.median(e2e_times)), "steps": Ke, "h2d": h2d, "d2h": d2h, "repeats": reps_e}
    for hd in handles:
        rs.last_status(hd)
    return res


def roofline_of(res: dict, peaks: dict, read_gbs) -> dict:
    per_step_s = res["ms"] / 1e3 / res["K"]
    if res["rows_per_step"] >= 256:
        achieved = res["flops"] / per_step_s / 1e12
        long_run = res["ms"] > 1000.0
        peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
        return {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "traffic": recorded_traffic(res["workload"]), "peak_source": "of " + peaks["source"] +
                (" (sustained figure: the timed region exceeds 1 s)" if long_run else " (burst figure)"),
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "hbm_gbs": res["algo_bytes"] / per_step_s / 1e9}
    achieved = res["algo_bytes"] / per_step_s / 1e9
    roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "traffic": recorded_traffic(res["workload"]),
            "peak_source": "of " + peaks["source"] + " (copy: reads + writes)",
            "frac_of_8tbs_nominal": achieved / 8000.0, "tflops": res["flops"] / per_step_s / 1e12}
    if read_gbs:
        roof["read_stream_gbs"] = read_gbs
        roof["frac_of_read_stream"] = achieved / read_gbs
    return roof


def release(res: dict, torch):
    for hd in res["handles"]:
        hd.destroy()
    for h in res["heads"]:
        h.pop("w_dev", None)
    res["heads"] = None
    torch.cuda.empty_cache()


EXTRA_WORKLOADS = ("c3_llm_b1", "c3_llm_b4", "c3_llm_b16", "c4_slm_b64", "c4_batched", "c5_catchup")


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=None, choices=sorted(BENCH_WORKLOADS),
                    help="default: c2_slm_b1 as the headline, the other configurations beside it under 'workloads'")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="only the headline workload")
    ap.add_argument("--flags", type=lambda s: int(s, 0), default=0, help="rstitch_args_t.flags (testing)")
    ap.add_argument("--graph", action="store_true",
                    help="capture one rotation of steps into a CUDA graph and time its replays")
    ap.add_argument("--vocab-parallel", action="store_true",
                    help="shard W_head by vocabulary rows over the ranks instead of the batch by rows")
    args = ap.parse_args()

    if args.impl != "reference" and needs_spawn(args.gpus, os.environ):
        # no launcher around this process: start one rank per GPU here, same command line
        from paper_2507_17307_b200 import sharding
        return sharding.spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:])

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    extras = args.workload is None and not args.no_extras and world == 1 and not args.graph and args.flags == 0
    if args.workload is None:
        args.workload = "c2_slm_b1"
    names = BENCH_WORKLOADS[args.workload]

    if args.impl == "reference":
        if rank != 0:
            return 0
        args.steps = 8 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        print(json.dumps(run_reference(args, names)), flush=True)
        return 0

    if args.vocab_parallel:
        return run_vocab_parallel(args, names, rank, local_rank, world)

    import torch
    import paper_2507_17307_b200 as rs
    from paper_2507_17307_b200 import build as rs_build, sharding
    if rank == 0:
        rs_build.build_library()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    rs.lib()
    dev = torch.device("cuda", local_rank)

    dK, dW, n_rot = default_steps(args.workload)
    K = args.steps if args.steps is not None else dK
    Wm = max(args.warmup if args.warmup is not None else dW, 3)
    res = measure(rs, torch, dist, rank, local_rank, world, args, args.workload, K, Wm, n_rot, with_e2e=True)
    K = res["K"]

    # max over ranks of the times, sums of the rest
    ms, _, launches = sharding.reduce_step_stats(res["ms"], res["rows_per_step"], res["launches"], dist, dev)
    ms_min, _, _ = sharding.reduce_step_stats(res["ms_min"], 0.0, 0, dist, dev)
    ms_max, _, _ = sharding.reduce_step_stats(res["ms_max"], 0.0, 0, dist, dev)
    e2e = res["e2e"]
    e2e["seconds"], _, _ = sharding.reduce_step_stats(e2e["seconds"], 0.0, 0, dist, dev)
    res["ms"] = ms

    if rank == 0:
        peaks = measured_peaks()
        read = read_stream_ceiling(rs, torch, dev, torch.cuda.current_stream()) if world == 1 else {"gbs": None}
        sec = ms / 1e3
        w0, alg1 = res["w0"], args.workload in ("alg1_b64", "alg1_plus_b64")
        value = world * res["rows_per_step"] * K / sec
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "B": w0.B, "rows_per_step": res["rows_per_step"], "d": w0.d,
                       "V": w0.V, "tau_nats": w0.tau_nats, "heads": list(names), "path": res["path"],
                       "l2": "inputs larger than L2: each step streams the whole W_head (%.0f MB); "
                             "hidden rotates over %d buffers" % (res["algo_bytes"] / 1e6, n_rot),
                       "parallelism": "dp%d (rows sharded, head replicated, no collective)" % world,
                       "cuda_graph": bool(args.graph)},
            "timing": {"regions": res["repeats"], "steps_per_region": K, "statistic": "median region",
                       "ms_per_step_min": ms_min / K, "ms_per_step_max": ms_max / K,
                       "note": "every region times exactly `steps` steps between two CUDA events on the launching "
                               "stream; regions repeat until they add up to 0.2 s (at least three)"},
            "roofline": roofline_of(res, peaks, read.get("gbs")), "clocks": res["clocks"], "gpu_launches": launches,
            "algorithmic_bytes_per_step": res["algo_bytes"], "flops_per_step": res["flops"],
            # `value` counts rows (every row gets a token and an entropy); with multi-row spans a sequence
            # is decided by its last row, so the sequences decided per second are fewer
            "rows_per_s": value, "sequences_per_s": world * w0.B * K / sec,
        }
        if read.get("gbs"):
            line["read_stream"] = read
        line["e2e"] = {"value": world * res["rows_per_step"] * e2e["steps"] / e2e["seconds"], "unit": UNIT,
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                       "steps": e2e["steps"], "regions": e2e["repeats"],
                       "note": ("the round's hidden pools copied from pinned host memory, per-sequence token counts "
                                "copied back, stream synchronised every round; W_head resident") if alg1 else
                               ("rstitch_route_ex_host: pinned hidden and index arrays in, tok/ent/mask/llm_idx/"
                                "llm_count/spans out, stream synchronised every step; W_head resident")}
        heads_for_cpu = res["heads"]
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            budget, t0, rows, n = 12.0, time.perf_counter(), 0, 0
            sample_rows = 8 if res["rows_per_step"] > 16 else None
            while time.perf_counter() - t0 < budget and n < 4096:
                for h in heads_for_cpu:
                    b = h["batches"][n % n_rot]
                    hid = b["hid"] if sample_rows is None else b["hid"][:sample_rows]
                    oracle.route(hid, h["w_bits"], h["w"].tau_nats)
                rows += (heads_for_cpu[0]["batches"][n % n_rot]["hid"].shape[0] if sample_rows is None else sample_rows)
                n += 1
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {"value": rows / dt, "unit": UNIT, "cores": oracle.num_threads(),
                                    "kind": "oracle",
                                    "sample": "%d steps%s of the same batches, %.1f s" % (
                                        n, "" if sample_rows is None else " (first %d rows each)" % sample_rows, dt)}
        release(res, torch)
        if extras:
            # the other configurations, each in a short timed region of its own with its own clock record
            line["workloads"] = {}
            for wl in EXTRA_WORKLOADS:
                eK, eW, e_rot = default_steps(wl)
                eK = args.steps if args.steps is not None else min(eK, 512)
                r = measure(rs, torch, None, 0, local_rank, 1, args, wl, eK, max(3, min(Wm, 8)), e_rot, with_e2e=False)
                per_step_s = r["ms"] / 1e3 / r["K"]
                line["workloads"][wl] = {
                    "ms_per_step": r["ms"] / r["K"], "ms_per_step_min": r["ms_min"] / r["K"],
                    "ms_per_step_max": r["ms_max"] / r["K"], "regions": r["repeats"], "steps_per_region": r["K"],
                    "rows_per_step": r["rows_per_step"], "rows_per_s": r["rows_per_step"] / per_step_s,
                    "d": r["w0"].d, "V": r["w0"].V, "heads": list(r["names"]), "path": r["path"],
                    "gpu_launches": r["launches"], "roofline": roofline_of(r, peaks, read.get("gbs")),
                    "clocks": r["clocks"]}
                release(r, torch)
        print(json.dumps(line), flush=True)
    else:
        release(res, torch)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

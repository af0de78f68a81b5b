#!/usr/bin/env python
"""Benchmark of the OQM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C3|C2|C5]

One step = one pass of the whole path over one synthetic stream:
    A1  quantize every frame's kv groups of every layer into the memory bank
    A2  question embedding + cosine scores over all stored groups   } one fused launch
    A3  top-K groups per layer                                      } (stom_oqm_retrieve)
    A4  dequantize-and-gather the selected groups into the active bf16 cache
After the timed steps the three retrieval kernels are also launched one by one
(stom_oqm_score_groups, stom_oqm_topk, stom_oqm_dequant_gather) for the
per-kernel figures of `roofline_all`.
Inputs are resident in HBM before the timed region; the input stream (20.6 GB
at C3) is far larger than L2 and an L2 flush (512 MB written, then 512 MB read) separates A1 from A2-A4.

Rank 0 prints ONE JSON line.  `value` is the retrieve+dequant (A2+A3+A4)
throughput in algorithmic GB/s summed over ranks; the quantize throughput in
tokens/s and the per-query latency ride along in `submetrics`.  `e2e` measures
the same thing through the host-buffer C-ABI entry points with the
host<->device copies inside the timed region.  `--impl reference` times the CPU
oracle (a deliberately plain program) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

FALLBACK_HBM_GBS = 6650.0

# dram bytes per unit of work measured with ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a reduced
# case of the same kernel and scaled by the units one launch processes; see profiles/*.md.  None = not captured.
NCU_TRAFFIC_PER_UNIT = {
    # all figures are per kv head of the unit named (the captures ran the 4-head 7B geometry)
    "quantize_kernel": 137448.0 / 4,    # bytes per (layer, frame): 3.941 GB over 28 x 1024 units
    # bytes per (layer, selected group): 186.0 MB over 28 x 64 units; of the 183.5 MB the kernel writes only
    # 125.4 MB had left L2 when it ended (the rest is written back later), so this undercounts by design
    "dequant_gather_kernel": 103805.0 / 4,
    "score_kernel": 2067.0 / 4,         # bytes per (layer, stored group): 59.26 MB over 28 x 1024 units
    "retrieve_kernel": 2188.0 / 4,      # bytes per (layer, stored group): 62.75 MB over 28 x 1024 units (Q read per cluster)
    # bytes per frame of 196 tokens x 1152 bf16 channels (not per kv head): 561.8 MB over 1200 frames
    "ctr_similarity_kernel": 468181.0,
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C3")
    ap.add_argument("--frames-per-call", type=int, default=0, help="0: the whole stream in one quantize call")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-sample-frames", type=int, default=1024)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the C5 and C4 passes that follow the default C3 line")
    ap.add_argument("--query-every", type=int, default=60, help="C4: frames between questions")
    ap.add_argument("--layers", type=int, default=0, help="override L (reduced case for profiler captures)")
    ap.add_argument("--frames", type=int, default=0, help="override T (reduced case for profiler captures)")
    ap.add_argument("--meta", default="fp32", choices=["fp32", "fp16", "bf16"],
                    help="type the bank keeps s, m and k-bar in (fp32: the default reading; 16-bit: the compact variant)")
    return ap.parse_args()


# ---------------------------------------------------------------- byte accounting (algorithmic bytes)

META_CODE = {"bf16": 0, "fp16": 1, "fp32": 2}


def meta_of(sh) -> str:
    return str(sh.extra.get("meta", "fp32"))


def meta_bytes(sh) -> int:
    """Bytes of one stored s, m or k-bar value."""
    return 4 if meta_of(sh) == "fp32" else 2


def bytes_quantize(sh, frames):
    e = 4 if sh.dtype == "fp32" else 2
    mb = meta_bytes(sh)
    per = 2 * sh.H_k * sh.G * sh.d * e + 2 * sh.H_k * sh.G * sh.d // 2 + 4 * sh.H_k * sh.d * mb + sh.H_k * sh.d * mb + sh.H_k * 4
    return per * frames * sh.L


def bytes_score(sh, groups):
    return (sh.H_k * sh.d * meta_bytes(sh) + sh.H_k * 4 + 4) * groups * sh.L + sh.L * sh.H_q * sh.T_q * sh.d * 2


def bytes_topk(sh, groups):
    return sh.L * (groups * 4 + sh.k * 4)


def bytes_gather(sh, k):
    per = 2 * sh.H_k * sh.G * sh.d // 2 + 4 * sh.H_k * sh.d * meta_bytes(sh) + 2 * sh.H_k * sh.G * sh.d * 2
    return per * k * sh.L


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag, self.max_mhz = index, [], set(), False, None
        self.ready = threading.Event()      # set once NVML is up (or has failed): its start-up can take seconds

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            }
            self.ready.set()
            while not self.stop_flag:
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
                time.sleep(0.05)
        except Exception as ex:  # pragma: no cover
            self.reasons.add(f"nvml-unavailable:{type(ex).__name__}")
            self.ready.set()

    def result(self):
        self.stop_flag = True
        self.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


def nvml_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ---------------------------------------------------------------- CPU oracle leg

def oracle_sample(sh, K_cpu, V_cpu, Q_cpu, frames, threads=0):
    """Times the oracle on `frames` frames of every layer: quantize, score, top-K, gather.  Returns seconds per stage."""
    from oracle import oqm_oracle as orc
    from paper_2510_18269_b200 import synth
    import numpy as np
    k = min(sh.k, frames)
    # all the cores this process may run on, also under a launcher that exports OMP_NUM_THREADS=1 for its children
    threads = threads or orc.host_cores()
    cfg = orc.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, frames, 4, {"bf16": 0, "fp16": 1, "fp32": 2}[sh.dtype],
                          meta_dtype=META_CODE[meta_of(sh)])
    st = orc.Store(cfg)
    kn, vn, qn = synth.as_u16(K_cpu), synth.as_u16(V_cpu), synth.as_u16(Q_cpu)
    strides = (frames * sh.H_k * sh.G * sh.d, sh.H_k * sh.G * sh.d, sh.G * sh.d, sh.d)
    t0 = time.perf_counter()
    assert orc.quantize_frame(cfg, st, 0, sh.L, 0, frames, kn, vn, strides, n_threads=threads) == 0
    t1 = time.perf_counter()
    sc = orc.score_groups(cfg, st, 0, sh.L, frames, qn, sh.T_q, (sh.H_q * sh.T_q * sh.d, sh.T_q * sh.d, sh.d),
                          n_threads=threads)
    idx, _, _ = orc.topk(sc, k)
    S = k * sh.G
    ka = np.zeros((sh.L, sh.H_k, S, sh.d), np.uint16)
    va = np.zeros_like(ka)
    assert orc.dequant_gather(cfg, st, 0, sh.L, idx, k, frames, ka, va, orc.BF16,
                              (sh.H_k * S * sh.d, S * sh.d, sh.d), 0, n_threads=threads) == 0
    t2 = time.perf_counter()
    return {"quantize_s": t1 - t0, "retrieve_s": t2 - t1, "k": k, "threads": threads,
            "cores": orc.host_cores()}


def cpu_sample_frames(args, sh):
    """Frames of the CPU sample: --cpu-sample-frames at the 7B geometry, fewer for wider models (same bytes)."""
    f = args.cpu_sample_frames * (28 * 4) // (sh.L * sh.H_k)
    return max(16, min(sh.T, f))


def cpu_inputs(sh, frames):
    """The first `frames` frames of every layer, generated on the CPU with the same recipe."""
    import dataclasses
    import torch
    from paper_2510_18269_b200 import synth
    small = dataclasses.replace(sh, T=frames)
    planted = synth.planted_groups(small, min(sh.k // 2, frames))
    K = torch.empty(sh.L, frames, sh.H_k, sh.G, sh.d, dtype=synth.DTYPES[sh.dtype])
    V = torch.empty_like(K)
    for l in range(sh.L):
        K[l], V[l] = synth.kv_chunk(small, l, 0, frames, "cpu", planted)
    return K, V, synth.queries(small)


def run_reference(args, sh):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    frames = cpu_sample_frames(args, sh)
    K, V, Q = cpu_inputs(sh, frames)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(sh, K, V, Q, min(frames, 16))
    rs, qs = [], []
    info = None
    for _ in range(args.steps):
        info = oracle_sample(sh, K, V, Q, frames)
        rs.append(info["retrieve_s"])
        qs.append(info["quantize_s"])
    k = info["k"]
    rbytes = bytes_score(sh, frames) + bytes_topk(sh, frames) + bytes_gather(sh, k)
    rt = statistics.mean(rs)
    value = rbytes / rt / 1e9
    sample = f"first {frames} frames of all {sh.L} layers (of {sh.T}); top-{k} groups gathered per layer"
    out = {
        "impl": "reference", "metric": "OQM retrieve+dequant throughput", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": min(args.warmup, 1),
        "ms_per_step": 1e3 * (statistics.mean(qs) + rt), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": sh.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": info["threads"], "kind": "oracle", "sample": sample,
                         "quantize_tokens_per_s": frames * sh.G / statistics.mean(qs)},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


# ---------------------------------------------------------------- CUDA leg

def nvtx_range(name):
    """An NVTX range around a C-ABI call, so that a timeline shows which call a kernel belongs to."""
    import torch
    return torch.cuda.nvtx.range(name)


def median_ms(ts, a, b):
    return statistics.median(t[a].elapsed_time(t[b]) for t in ts)


def measure_stream(args, sh, dev, rank, world, sdist, peak, peak_src, steps, warmup, extras=True):
    """One workload on this rank's GPU: `steps` timed passes of the whole path (quantize the stream, flush L2, one
    question through the fused retrieval call), then the retrieval kernels one by one.  Returns the figures and,
    when `extras`, the end-to-end arm through the host-buffer entry points.  Frees its tensors on return."""
    import dataclasses
    import torch
    from paper_2510_18269_b200 import oqm, synth

    # independent streams per rank (weak scaling: every GPU serves its own video stream)
    sh = dataclasses.replace(sh, seed=sh.seed + 17 * rank)
    cfg = oqm.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, sh.T, 4, oqm.dtype_code(synth.DTYPES[sh.dtype]),
                          meta_dtype=META_CODE[meta_of(sh)])
    store = oqm.Store(cfg, device=dev, zero=False)
    K, V = synth.kv_stream(sh, dev)
    Q = synth.queries(sh, dev)
    strides = (sh.T * sh.H_k * sh.G * sh.d, sh.H_k * sh.G * sh.d, sh.G * sh.d, sh.d)
    qs = (sh.H_q * sh.T_q * sh.d, sh.T_q * sh.d, sh.d)
    sys_len = 0
    S = sys_len + sh.k * sh.G
    act = (sh.H_k * S * sh.d, S * sh.d, sh.d)
    scores = torch.empty(sh.L, sh.T, dtype=torch.float32, device=dev)
    idx = torch.empty(sh.L, sh.k, dtype=torch.int32, device=dev)
    ka = torch.empty(sh.L, sh.H_k, S, sh.d, dtype=torch.bfloat16, device=dev)
    va = torch.empty_like(ka)
    ws = torch.empty(oqm.stom_oqm_retrieve_workspace_bytes(cfg, sh.L, sh.T, sh.k), dtype=torch.uint8, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(128 << 20, dtype=torch.float32, device=dev)

    def flush_l2():
        """Write 512 MB (evicts everything), then read another 512 MB: the written lines are dirty in L2, and left
        alone their write-back would run during the next kernel (it added 12 us to a 139 us retrieval)."""
        flush.fill_(1)
        flush_rd.sum()

    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    fpc = args.frames_per_call or sh.T
    n_qcalls = (sh.T + fpc - 1) // fpc

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def quantize_stream(per_call):
        with nvtx_range("stom_oqm_quantize_frame"):
            for f0 in range(0, sh.T, per_call):
                n = min(per_call, sh.T - f0)
                oqm.stom_oqm_quantize_frame(cfg, store, 0, sh.L, f0, n, K.view(-1)[f0 * strides[1]:],
                                            V.view(-1)[f0 * strides[1]:], strides, dev_flags=flags)

    def step(timers=None):
        e = [ev() for _ in range(4)] if timers is not None else None
        if e: e[0].record()
        quantize_stream(fpc)
        if e: e[1].record()
        flush_l2()                           # evict freshly written codes / keys from L2
        if e: e[2].record()
        # A2 + A3 (one fused launch) and A4
        with nvtx_range("stom_oqm_retrieve"):
            oqm.stom_oqm_retrieve(cfg, store, 0, sh.L, sh.T, Q, sh.T_q, qs, sh.k, scores, idx, ka, va, oqm.BF16, act,
                                  sys_len, ws, dev_flags=flags)
        if e: e[3].record()
        if timers is not None:
            timers.append(e)

    def stage_step(timers):
        """The three retrieval kernels launched one by one, for the per-kernel figures.  After the gather a 512 MB
        read forces the lines the gather left dirty in L2 out to DRAM; the same read is timed alone after a flush."""
        e = [ev() for _ in range(7)]
        flush_l2()
        e[0].record()
        with nvtx_range("stom_oqm_score_groups"):
            oqm.stom_oqm_score_groups(cfg, store, 0, sh.L, sh.T, Q, sh.T_q, qs, scores, ws)
        e[1].record()
        with nvtx_range("stom_oqm_topk"):
            oqm.stom_oqm_topk(scores, sh.L, sh.T, sh.T, sh.k, idx)
        e[2].record()
        with nvtx_range("stom_oqm_dequant_gather"):
            oqm.stom_oqm_dequant_gather(cfg, store, 0, sh.L, idx, sh.k, sh.T, ka, va, oqm.BF16, act, sys_len,
                                        dev_flags=flags)
        e[3].record()
        flush_rd.sum()                       # gather's dirty lines are written back while this read runs
        e[4].record()
        flush_l2()
        e[5].record()
        flush_rd.sum()                       # the same read with nothing dirty behind it
        e[6].record()
        timers.append(e)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    sdist.barrier()

    sampler = ClockSampler(nvml_index(dev.index or 0))
    sampler.start()
    sampler.ready.wait(timeout=30)         # keep NVML's start-up out of the timed region
    timers = []
    t_start, t_end = ev(), ev()
    torch.cuda.synchronize()
    t_start.record()
    for _ in range(steps):
        step(timers)
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.result()
    total_ms = sdist.max_over_ranks(t_start.elapsed_time(t_end))

    stage_timers = []
    for _ in range(warmup):
        stage_step([])
    for _ in range(steps):
        stage_step(stage_timers)
    torch.cuda.synchronize()

    q_ms, r_ms = median_ms(timers, 0, 1), median_ms(timers, 2, 3)
    sc_ms, tk_ms, ga_ms = (median_ms(stage_timers, a, a + 1) for a in (0, 1, 2))
    # the gather with its write-back: (gather + read) - (read alone)
    ga_wb_ms = statistics.median(t[2].elapsed_time(t[4]) for t in stage_timers) - median_ms(stage_timers, 5, 6)
    q_ms, sc_ms, tk_ms, ga_ms, r_ms, ga_wb_ms = (sdist.max_over_ranks(x) for x in (q_ms, sc_ms, tk_ms, ga_ms, r_ms, ga_wb_ms))
    assert int(flags.item()) == 0, "a kernel flagged a bad index or a wait that ran out"

    # the paper's encoder batch (Sec. 4.1): 32 frames per quantize call, the stream as 225 calls back to back
    q32_ms = q32_graph_ms = None
    if extras and fpc != 32:
        reps = []
        for i in range(1 + max(2, min(5, steps))):
            a, b = ev(), ev()
            a.record(); quantize_stream(32); b.record()
            torch.cuda.synchronize()
            if i:
                reps.append(a.elapsed_time(b))
        q32_ms = sdist.max_over_ranks(statistics.median(reps))
        # the same calls captured once in a CUDA graph and replayed: the device's share, without the host's per-call cost
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            quantize_stream(32)
        reps = []
        for i in range(1 + max(2, min(5, steps))):
            a, b = ev(), ev()
            a.record(); graph.replay(); b.record()
            torch.cuda.synchronize()
            if i:
                reps.append(a.elapsed_time(b))
        q32_graph_ms = sdist.max_over_ranks(statistics.median(reps))
        del graph

    # Context for the gather, whose traffic is 3/4 writes: the rate of a plain 1 GiB fill with 4-byte elements
    # (torch's fill of 1-byte elements runs at half that rate and says nothing about the memory system).
    wbuf = torch.empty(1 << 28, dtype=torch.float32, device=dev)
    w_ms = []
    for i in range(6):
        a, b = ev(), ev()
        a.record()
        wbuf.fill_(float(i))
        b.record()
        torch.cuda.synchronize()
        w_ms.append(a.elapsed_time(b))
    write_gbs = (1 << 30) / (min(w_ms[1:]) * 1e-3) / 1e9
    del wbuf

    rbytes = bytes_score(sh, sh.T) + bytes_topk(sh, sh.T) + bytes_gather(sh, sh.k)
    qbytes = bytes_quantize(sh, sh.T)

    def roof(name, nbytes, ms, launches, unit_count):
        a = nbytes / launches / (ms / launches * 1e-3) / 1e9
        tpu = NCU_TRAFFIC_PER_UNIT.get(name) if meta_of(sh) == "fp32" else None  # captured with binary32 metadata only
        return {"kernel": name, "bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                "traffic": None if tpu is None else tpu * sh.H_k * unit_count / launches, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": nbytes / launches, "ms_per_launch": ms / launches}

    roofs = [
        roof("quantize_kernel", qbytes, q_ms, n_qcalls, sh.L * sh.T),
        roof("dequant_gather_kernel", bytes_gather(sh, sh.k), ga_ms, 1, sh.L * sh.k),
        roof("score_kernel", bytes_score(sh, sh.T), sc_ms, 1, sh.L * sh.T),
    ]
    gw = 2 * sh.H_k * sh.G * sh.d * 2 * sh.k * sh.L   # bytes the gather writes
    g = roofs[1]
    g.update({
        "write_bytes_per_launch": gw, "measured_fill_GBps": write_gbs,
        # Three readings of the same launch.  `frac` divides the algorithmic bytes by the kernel's own time: part of
        # what the kernel wrote is still dirty in L2 (126 MB) when its end event fires, which flatters a launch that
        # writes little more than L2 holds.  `frac_dram_side` counts only the bytes ncu saw reach DRAM inside the
        # kernel.  `frac_with_writeback` charges the kernel the time a following 512 MB read loses to the write-back.
        "frac_dram_side": None if g["traffic"] is None else g["traffic"] / (ga_ms * 1e-3) / 1e9 / peak,
        "ms_with_writeback": ga_wb_ms,
        "frac_with_writeback": bytes_gather(sh, sh.k) / (ga_wb_ms * 1e-3) / 1e9 / peak,
        "output_over_l2": gw / 126e6,
    })
    res = {
        "sh": sh, "value": world * rbytes / (r_ms * 1e-3) / 1e9, "rbytes": rbytes, "qbytes": qbytes,
        "total_ms": total_ms, "q_ms": q_ms, "r_ms": r_ms, "sc_ms": sc_ms, "tk_ms": tk_ms, "ga_ms": ga_ms,
        "q32_ms": q32_ms, "q32_graph_ms": q32_graph_ms, "roofs": roofs, "clocks": clocks, "fpc": fpc, "n_qcalls": n_qcalls,
    }
    if extras and not args.no_e2e:
        res["e2e"] = run_e2e(args, sh, cfg, store, K, V, Q, idx, ka, va, dev, world, sdist, rbytes)
    return res


def workload_summary(res, world, peak):
    """The figures of one workload as they appear under `submetrics` (and, for the other workloads, on their own)."""
    sh = res["sh"]
    q_ms, r_ms = res["q_ms"], res["r_ms"]
    mhz = res["clocks"].get("sm_mhz")
    out = {
        "retrieve_dequant_GBps": res["value"], "retrieve_dequant_frac_of_measured_hbm": res["value"] / world / peak,
        "quantize_tokens_per_s": world * sh.T * sh.G / (q_ms * 1e-3),
        "quantize_GBps": world * res["qbytes"] / (q_ms * 1e-3) / 1e9,
        "quantize_frac_of_measured_hbm": res["qbytes"] / (q_ms * 1e-3) / 1e9 / peak,
        "query_latency_us": r_ms * 1e3,
        "stage_us": {"quantize": q_ms * 1e3, "retrieve_fused_call": r_ms * 1e3,
                     "separate_calls": {"score": res["sc_ms"] * 1e3, "topk": res["tk_ms"] * 1e3,
                                        "dequant_gather": res["ga_ms"] * 1e3},
                     "statistic": "median over the timed steps"},
        "frac_of_nominal_8TBps": {"quantize": res["qbytes"] / (q_ms * 1e-3) / 8e12,
                                  "dequant_gather": bytes_gather(sh, sh.k) / (res["ga_ms"] * 1e-3) / 8e12},
        "dequant_gather_frac_of_measured_hbm": res["roofs"][1]["frac"],
        "dequant_gather_frac_dram_side": res["roofs"][1]["frac_dram_side"],
        "dequant_gather_frac_with_writeback": res["roofs"][1]["frac_with_writeback"],
        "sm_mhz_median": mhz,
        # the quantize kernel is bound by instruction issue, so its time follows the SM clock: time x MHz is the
        # figure to compare between runs at different clocks
        "quantize_ms_x_sm_mhz": None if mhz is None else q_ms * mhz,
    }
    if res["q32_ms"] is not None:
        def fig(ms):
            return {"ms": ms, "tokens_per_s": world * sh.T * sh.G / (ms * 1e-3),
                    "GBps": world * res["qbytes"] / (ms * 1e-3) / 1e9,
                    "frac_of_measured_hbm": res["qbytes"] / (ms * 1e-3) / 1e9 / peak}
        out["quantize_32_frames_per_call"] = {
            "calls": (sh.T + 31) // 32, "issued_from_python": fig(res["q32_ms"]),
            "cuda_graph_replay": fig(res["q32_graph_ms"]),
            "note": "the paper's encoder batch (Sec. 4.1): the same stream as back-to-back calls of 32 frames"}
    return out


def run_ours(args, sh):
    import torch
    from paper_2510_18269_b200 import oqm, synth, dist as sdist

    rank, world, local = sdist.init_from_env(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    oqm.lib()
    peak, peak_src = measured_peak()

    res = measure_stream(args, sh, dev, rank, world, sdist, peak, peak_src, args.steps, args.warmup)
    sh = res["sh"]
    out = {
        "metric": "OQM retrieve+dequant throughput", "value": res["value"], "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["total_ms"] / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": sh.name, "L": sh.L, "H_q": sh.H_q, "H_k": sh.H_k, "d": sh.d, "G": sh.G, "T": sh.T,
                   "T_q": sh.T_q, "k": sh.k, "kv_dtype": sh.dtype, "meta_dtype": meta_of(sh),
                   "frames_per_quantize_call": res["fpc"],
                   "l2": "inputs >> L2 (20.6 GB at C3); between quantize and retrieve a 512 MB write then a 512 MB read (no dirty lines left)",
                   "multi_gpu": "independent stream per rank, no collective"},
        "submetrics": workload_summary(res, world, peak),
        "roofline": res["roofs"][0], "roofline_all": res["roofs"],
        "gpu_launches": res["n_qcalls"] + 2, "clocks": res["clocks"],
        "paper_context": {"hardware": "A6000 48GB FP16 (paper)", "kv_compression": 15.7, "oqm_stage_ms_64_frames":
                          {"kv_storage": 7.3, "retrieval": 6.9, "reconstruction": 28.7}},
    }
    if "e2e" in res:
        out["e2e"] = res["e2e"]
    del res
    torch.cuda.empty_cache()

    # ---- the other workloads of the benchmark definition, single-GPU runs of the default line only
    if args.config == "C3" and world == 1 and not args.no_other_workloads and not (args.layers or args.frames):
        others = {}
        c5 = synth.CONFIGS["C5"]
        need = 2 * c5.L * c5.T * c5.H_k * c5.G * c5.d * 2 * 1.45 + (2 << 30)   # K, V, the bank, the flush buffers
        if torch.cuda.mem_get_info(dev)[0] >= need:
            r5 = measure_stream(args, c5, dev, rank, world, sdist, peak, peak_src, steps=max(2, args.steps // 3),
                                warmup=3, extras=False)
            s5 = workload_summary(r5, world, peak)
            s5["clocks"] = r5["clocks"]
            s5["roofline_all"] = r5["roofs"]
            s5["steps"] = max(2, args.steps // 3)
            others["C5-72B"] = s5
            del r5
            torch.cuda.empty_cache()
        else:
            others["C5-72B"] = {"skipped": f"needs {need / 2**30:.0f} GiB of free device memory"}
        import dataclasses
        c4 = dataclasses.replace(synth.CONFIGS["C4"], T=240)
        others["C4-7B-interleave-240-frames"] = run_stream(args, c4, dev)
        out["submetrics"]["other_workloads"] = others
        torch.cuda.empty_cache()

    # ---- the oracle on this machine's host cores, rank 0 only, single-GPU runs only
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        frames = cpu_sample_frames(args, sh)
        Kc, Vc, Qc = cpu_inputs(sh, frames)
        info = oracle_sample(sh, Kc, Vc, Qc, frames)
        k = info["k"]
        cb = bytes_score(sh, frames) + bytes_topk(sh, frames) + bytes_gather(sh, k)
        out["cpu_baseline"] = {
            "value": cb / info["retrieve_s"] / 1e9, "unit": "GB/s", "cores": info["threads"], "kind": "oracle",
            "sample": f"first {frames} frames of all {sh.L} layers (of {sh.T}); top-{k} groups gathered per layer",
            "quantize_tokens_per_s": frames * sh.G / info["quantize_s"], "seconds": info["quantize_s"] + info["retrieve_s"]}
        # the same program on ONE thread, on an eighth of that sample
        f1 = max(16, frames // 8)
        one = oracle_sample(sh, Kc[:, :f1].contiguous(), Vc[:, :f1].contiguous(), Qc, f1, threads=1)
        cb1 = bytes_score(sh, f1) + bytes_topk(sh, f1) + bytes_gather(sh, one["k"])
        out["cpu_baseline"]["one_thread"] = {
            "value": cb1 / one["retrieve_s"] / 1e9, "unit": "GB/s", "cores": 1,
            "sample": f"first {f1} frames of all {sh.L} layers; top-{one['k']} groups gathered per layer",
            "quantize_tokens_per_s": f1 * sh.G / one["quantize_s"], "seconds": one["quantize_s"] + one["retrieve_s"]}
    if rank == 0:
        print(json.dumps(out))
    sdist.finish()


def run_e2e(args, sh, cfg, store, K, V, Q, idx_dev, ka_dev, va_dev, dev, world, sdist, rbytes):
    """The same path through the host-buffer entry points: the stream goes up in 64-frame chunks from pinned host
    memory, the question goes up, the indices and the reconstructed cache come back, all copies inside the timed
    intervals.  The stream lives on the device (it is generated there); each chunk is first brought to a pinned host
    buffer OUTSIDE the timed interval, then sent through stom_oqm_quantize_frame_host inside it, so the bank the
    question runs on is the real stream's.  What comes back is compared with the device arm's result."""
    import torch
    from paper_2510_18269_b200 import oqm
    chunk = 64                                   # frames per host->device chunk
    e = 2
    one = sh.L * chunk * sh.H_k * sh.G * sh.d * e
    Kh = [torch.empty(sh.L, chunk, sh.H_k, sh.G, sh.d, dtype=K.dtype).pin_memory() for _ in range(2)]
    Vh = [torch.empty(sh.L, chunk, sh.H_k, sh.G, sh.d, dtype=K.dtype).pin_memory() for _ in range(2)]
    Qh = Q.cpu().pin_memory()
    S = sh.k * sh.G
    idx_h = torch.empty(sh.L, sh.k, dtype=torch.int32).pin_memory()
    ka_h = torch.empty(sh.L, sh.H_k, S, sh.d, dtype=torch.bfloat16).pin_memory()
    va_h = torch.empty_like(ka_h).pin_memory()
    qscr = torch.empty(oqm.stom_oqm_quantize_host_scratch_bytes(cfg, sh.L, chunk), dtype=torch.uint8, device=dev)
    rscr = torch.empty(oqm.stom_oqm_retrieve_host_scratch_bytes(cfg, sh.L, sh.T, sh.T_q, sh.k, oqm.BF16) + 256,
                       dtype=torch.uint8, device=dev)
    rscr = rscr[(-rscr.data_ptr()) % 256:]
    n_chunks = sh.T // chunk                     # whole chunks; a remainder is sent as a shorter last chunk
    tail = sh.T - n_chunks * chunk
    want_idx, want_ka, want_va = idx_dev.cpu(), ka_dev.cpu(), va_dev.cpu()   # the device arm's answer to this question

    def e2e_step(record=None):
        q_ms = 0.0
        pend = []
        for ci in range(n_chunks + (1 if tail else 0)):
            f0, n = ci * chunk, (chunk if ci < n_chunks else tail)
            s = ci & 1
            kh, vh = Kh[s][:, :n], Vh[s][:, :n]
            if n != chunk:
                kh, vh = kh.contiguous().pin_memory(), vh.contiguous().pin_memory()
            kh.copy_(K[:, f0:f0 + n])            # staging, untimed: device stream -> pinned host buffer (synchronous)
            vh.copy_(V[:, f0:f0 + n])
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            with nvtx_range("stom_oqm_quantize_frame_host"):
                oqm.stom_oqm_quantize_frame_host(cfg, store, 0, sh.L, f0, n, kh, vh, qscr)
            b.record()
            pend.append((a, b, kh, vh))
        torch.cuda.synchronize()
        q_ms = sum(a.elapsed_time(b) for a, b, _, _ in pend)
        b, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b.record()
        with nvtx_range("stom_oqm_retrieve_host"):
            oqm.stom_oqm_retrieve_host(cfg, store, 0, sh.L, sh.T, Qh, sh.T_q, sh.k, idx_h, ka_h, va_h, oqm.BF16, rscr)
        c.record()
        torch.cuda.synchronize()
        if record is not None:
            record.append((q_ms, b.elapsed_time(c)))

    e2e_step()
    sdist.barrier()
    recs = []
    for _ in range(max(1, args.e2e_steps)):
        e2e_step(recs)
    # the host arm must give the device arm's answer: same bank (quantization is deterministic), same question
    checked = bool(torch.equal(idx_h, want_idx) and torch.equal(ka_h.view(torch.int16), want_ka.view(torch.int16))
                   and torch.equal(va_h.view(torch.int16), want_va.view(torch.int16)))
    assert checked, "the host-buffer arm returned other indices or another cache than the device arm"
    q_ms = sdist.max_over_ranks(statistics.median(q for q, _ in recs))
    r_ms = sdist.max_over_ranks(statistics.median(r for _, r in recs))
    return {
        "value": world * rbytes / (r_ms * 1e-3) / 1e9, "unit": "GB/s",
        "h2d_bytes_per_step": 2 * sh.L * sh.T * sh.H_k * sh.G * sh.d * e + Qh.numel() * 2,
        "d2h_bytes_per_step": 2 * ka_h.numel() * 2 + idx_h.numel() * 4,
        "query_latency_us": r_ms * 1e3, "quantize_tokens_per_s": world * sh.T * sh.G / (q_ms * 1e-3),
        "ms_per_step": q_ms + r_ms, "result_checked_against_device_arm": checked,
        "note": "the real stream, chunk by chunk (64 frames): each chunk is brought to one of two pinned host buffers "
                "outside the timed interval, then goes through stom_oqm_quantize_frame_host inside it (the intervals "
                "are summed); then Q up, indices and the reconstructed K/V cache down in one timed "
                "stom_oqm_retrieve_host call; indices and cache are compared with the device arm's and are identical",
    }


def run_stream(args, sh, dev=None):
    """The streaming interleave (C4): frames of N_in tokens arrive one at a time, G of them are kept by a seeded mask and
    quantized on arrival (all layers in one call); every `--query-every` frames a question runs retrieval over what is
    stored so far and one decode-attention step over [system tokens || selected groups].  Returns latencies."""
    import torch
    from paper_2510_18269_b200 import oqm, synth
    import dataclasses
    if dev is None:
        torch.cuda.set_device(0)
        dev = torch.device("cuda", 0)
    oqm.lib()
    cfg = oqm.make_config(sh.L, sh.H_q, sh.H_k, sh.d, sh.G, sh.T, 4, oqm.dtype_code(synth.DTYPES[sh.dtype]),
                          meta_dtype=META_CODE[meta_of(sh)])
    store = oqm.Store(cfg, device=dev, zero=False)
    pool = 32                                    # distinct synthetic frames, cycled (5.6 MB of K and of V per frame)
    psh = dataclasses.replace(sh, T=pool)
    K, V = synth.kv_stream(psh, dev)             # [L][pool][H_k][N_in][d]
    keep = synth.keep_mask(sh, 0, sh.T).to(dev)  # [T][G]
    strides = (pool * sh.H_k * sh.N_in * sh.d, sh.H_k * sh.N_in * sh.d, sh.N_in * sh.d, sh.d)
    qs = (sh.H_q * sh.T_q * sh.d, sh.T_q * sh.d, sh.d)
    sys_len = 32
    S = sys_len + sh.k * sh.G
    act = (sh.H_k * S * sh.d, S * sh.d, sh.d)
    Q = synth.queries(sh, dev)
    q_dec = torch.randn(sh.L, sh.H_q, sh.d, device=dev).to(torch.bfloat16)
    ka = torch.randn(sh.L, sh.H_k, S, sh.d, device=dev).to(torch.bfloat16)
    va = torch.randn(sh.L, sh.H_k, S, sh.d, device=dev).to(torch.bfloat16)
    scores = torch.empty(sh.L, sh.T, dtype=torch.float32, device=dev)
    idx = torch.empty(sh.L, sh.k, dtype=torch.int32, device=dev)
    out = torch.empty(sh.L, sh.H_q, sh.d, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(oqm.stom_oqm_retrieve_workspace_bytes(cfg, sh.L, sh.T, sh.k), dtype=torch.uint8, device=dev)
    aws = torch.zeros(oqm.stom_oqm_attend_workspace_bytes(cfg, sh.L, sh.k, sys_len) + 256, dtype=torch.uint8, device=dev)
    aws = aws[(-aws.data_ptr()) % 256:]
    flags = torch.zeros(1, dtype=torch.int32, device=dev)
    scale = float(sh.d) ** -0.5

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def ingest(f):
        off = (f % pool) * strides[1]
        oqm.stom_oqm_quantize_frame(cfg, store, 0, sh.L, f, 1, K.view(-1)[off:], V.view(-1)[off:], strides,
                                    token_idx=keep[f:f + 1], tokens_per_frame_in=sh.N_in, dev_flags=flags)

    def question(n):
        sc = scores.view(-1)[:sh.L * n].view(sh.L, n)
        oqm.stom_oqm_retrieve(cfg, store, 0, sh.L, n, Q, sh.T_q, qs, sh.k, sc, idx, ka, va, oqm.BF16, act, sys_len, ws,
                              dev_flags=flags)

    def decode(n, l0=0, lc=None):
        lc = sh.L if lc is None else lc
        oqm.stom_oqm_attend(cfg, store, l0, lc, idx[l0:], sh.k, n, q_dec[l0:], (sh.H_q * sh.d, sh.d), ka[l0:], va[l0:],
                            oqm.BF16, act, sys_len, scale, out[l0:], (sh.H_q * sh.d, sh.d), aws, dev_flags=flags)

    for f in range(8):                           # warm-up (slots are rewritten by the timed pass)
        ingest(f)
    question(8)
    decode(8)
    torch.cuda.synchronize()
    sampler = ClockSampler(nvml_index(dev.index or 0))
    sampler.start()
    sampler.ready.wait(timeout=30)
    ing, qry, dec, rep, graphs = [], [], [], [], []
    every = args.query_every
    t0 = time.perf_counter()
    for f in range(sh.T):
        a, b = ev(), ev()
        a.record(); ingest(f); b.record()
        ing.append((a, b))
        if (f + 1) % every == 0:
            a, b, c = ev(), ev(), ev()
            a.record(); question(f + 1); b.record(); decode(f + 1); c.record()
            qry.append((a, b)); dec.append((b, c))
            # the same question (retrieval, then one decode step) captured as a CUDA graph and replayed once
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                question(f + 1)
                decode(f + 1)
            a, b = ev(), ev()
            a.record(); g.replay(); b.record()
            rep.append((a, b)); graphs.append(g)   # a graph lives until its replay has run
        if f % 256 == 255:
            torch.cuda.synchronize()             # bounds the number of events in flight
            graphs.clear()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0

    # one decode step as a decoder would issue it: attention called layer by layer (28 calls), captured in a CUDA
    # graph and replayed; the per-layer figure is the replay time over the layer count
    n = sh.T
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for l in range(sh.L):
            decode(n, l, 1)
    lay = []
    for i in range(12):
        a, b = ev(), ev()
        a.record(); g.replay(); b.record()
        torch.cuda.synchronize()
        if i >= 2:
            lay.append(a.elapsed_time(b) * 1e3 / sh.L)
    # the same step as ONE call over all layers, captured and replayed: the device's share of that call
    g_all = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_all):
        decode(n)
    allr = []
    for i in range(12):
        a, b = ev(), ev()
        a.record()
        for _ in range(10):
            g_all.replay()
        b.record()
        torch.cuda.synchronize()
        if i >= 2:
            allr.append(a.elapsed_time(b) * 1e3 / 10)
    clocks = sampler.result()
    assert int(flags.item()) == 0

    def stats(pairs):
        v = sorted(x.elapsed_time(y) * 1e3 for x, y in pairs)
        return {"p50_us": v[len(v) // 2], "p99_us": v[min(len(v) - 1, int(0.99 * len(v)))], "mean_us": statistics.mean(v),
                "max_us": v[-1], "n": len(v)}

    i_st, q_st, d_st, r_st = stats(ing), stats(qry), stats(dec), stats(rep)
    frame_bytes = sh.L * (2 * sh.H_k * sh.G * sh.d * 2 + 2 * sh.H_k * sh.G * sh.d // 2 + 5 * sh.H_k * sh.d * 4 + sh.H_k * 4)
    return {
        "metric": "per-query OQM latency (score + top-k + dequant-gather + decode attention), streaming interleave",
        "value": q_st["p50_us"] + d_st["p50_us"], "unit": "us", "n_gpus": 1, "steps": sh.T, "warmup": 8,
        "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": sh.name, "L": sh.L, "H_q": sh.H_q, "H_k": sh.H_k, "d": sh.d, "tokens_per_frame": sh.N_in,
                   "kept_per_frame": sh.G, "frames": sh.T, "query_every": every, "T_q": sh.T_q, "k": sh.k,
                   "system_tokens": sys_len, "frame_pool": pool},
        "per_frame_ingest": dict(i_st, algorithmic_bytes=frame_bytes),
        "per_query_retrieve": q_st, "per_decode_step_attend_all_layers": d_st,
        "per_decode_step_attend_one_layer_per_call_graph_replay_us": statistics.median(lay),
        "per_decode_step_attend_all_layers_graph_replay_us": statistics.median(allr),
        "per_query_retrieve_plus_decode_step_graph_replay": r_st,
        "wall_s_including_python": wall, "clocks": clocks,
        "note": "CUDA-event times of single calls issued from Python one after the other; latencies, not bandwidths",
    }


CTR_SHAPE = {"T": 7200, "N": 196, "D": 1152, "G": 50, "tau_c": 0.9, "dtype": "bf16", "seed": 4242}
CTR_CPU_FRAMES = 1200


def bytes_ctr(T, N, D, G, elem=2):
    """Algorithmic bytes of the CTR steps over T frames: every feature row once, saliency once, similarity written
    and read once, the integer outputs written once."""
    return T * N * D * elem + T * N * 4 + 2 * T * N * 4 + T * (N + G + 2) * 4


def run_ctr(args):
    """The CTR steps (paper Sec. 3.3: temporal similarity, static/dynamic split, budget, saliency top-k_d) over a
    2-hour stream of synthetic encoder features.  `--impl reference` times the oracle on a sample of the frames."""
    c = dict(CTR_SHAPE)
    if args.frames:
        c["T"] = args.frames
    T, N, D, G = c["T"], c["N"], c["D"], c["G"]
    name = "CTR-7B-2h" if not args.frames else f"CTR-7B-reduced-T{T}"
    from paper_2510_18269_b200 import synth
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return
        from oracle import oqm_oracle as orc
        frames = min(T, CTR_CPU_FRAMES)
        F, alpha = synth.ctr_stream(frames, N, D, c["seed"], "cpu", c["dtype"])
        Fn, an = synth.as_u16(F), alpha.numpy()
        ts = []
        for _ in range(args.steps):
            t0 = time.perf_counter()
            sim = orc.ctr_similarity(Fn, orc.BF16)
            orc.ctr_select(sim, an, G, c["tau_c"])
            ts.append(time.perf_counter() - t0)
        v = bytes_ctr(frames, N, D, G) / statistics.mean(ts) / 1e9
        sample = f"first {frames} frames (of {T})"
        print(json.dumps({
            "impl": "reference", "metric": "CTR reduce throughput", "value": v, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": 0, "ms_per_step": 1e3 * statistics.mean(ts), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": name, "sample": sample},
            "cpu_baseline": {"value": v, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))
        return
    import torch
    from paper_2510_18269_b200 import oqm, dist as sdist
    rank, world, local = sdist.init_from_env(args.gpus)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    oqm.lib()
    peak, peak_src = measured_peak()
    F, alpha = synth.ctr_stream(T, N, D, c["seed"] + 17 * rank, dev, c["dtype"])
    sim = torch.empty(T, N, dtype=torch.float32, device=dev)
    ks = torch.empty(T, dtype=torch.int32, device=dev)
    kd = torch.empty_like(ks)
    si = torch.empty(T, N, dtype=torch.int32, device=dev)
    di = torch.empty(T, G, dtype=torch.int32, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(128 << 20, dtype=torch.float32, device=dev)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    ret = torch.empty(T, G, D, dtype=F.dtype, device=dev)
    rpos = torch.empty(T, G, dtype=torch.int32, device=dev)
    mflags = torch.zeros(1, dtype=torch.int32, device=dev)

    def step(timers=None):
        flush.fill_(1)       # evict everything ...
        flush_rd.sum()       # ... and leave no dirty lines whose write-back would run during the timed kernels
        e = [ev() for _ in range(4)]
        e[0].record()
        oqm.stom_ctr_similarity(F, None, T, N, D, (N * D, D), sim)
        e[1].record()
        oqm.stom_ctr_select(sim, alpha, T, N, G, c["tau_c"], ks, kd, si, di)
        e[2].record()
        oqm.stom_ctr_merge(F, T, N, D, (N * D, D), ks, kd, si, di, G, 5, ret, rpos, dev_flags=mflags)
        e[3].record()
        if timers is not None:
            timers.append(e)

    for _ in range(args.warmup):
        step()
    sampler = ClockSampler(nvml_index(local))
    sampler.start()
    sampler.ready.wait(10)
    sdist.barrier()
    torch.cuda.synchronize()
    timers = []
    for _ in range(args.steps):
        step(timers)
    torch.cuda.synchronize()
    sdist.barrier()
    if int(mflags.item()) != 0:
        raise RuntimeError(f"stom_ctr_merge raised device flags {int(mflags.item()):#x}: its timing is void")
    clocks = sampler.result()
    sim_ms = sdist.max_over_ranks(statistics.mean(t[0].elapsed_time(t[1]) for t in timers))
    sel_ms = sdist.max_over_ranks(statistics.mean(t[1].elapsed_time(t[2]) for t in timers))
    tot_ms = sdist.max_over_ranks(statistics.mean(t[0].elapsed_time(t[2]) for t in timers))
    mg_ms = sdist.max_over_ranks(statistics.median(t[2].elapsed_time(t[3]) for t in timers))
    # Merge: the Gram matrix of a frame's N tokens is a [N x D] . [D x N] contraction of which only the part on and
    # below the diagonal is needed (counted here in 16 x 16 blocks; the kernel's two 128-row tiles compute more).  Its
    # bytes: the frame's features once, the retained group written once.
    tiles = (N + 15) // 16
    mg_flops = T * (tiles * (tiles + 1) // 2) * 2 * 16 * 16 * D
    mg_bytes = T * (N * D * 2 + G * D * 2 + (N + 3 * G + 2) * 4)
    nbytes = bytes_ctr(T, N, D, G)
    sbytes = T * N * D * 2 + T * N * 4
    a = sbytes / (sim_ms * 1e-3) / 1e9
    tpu = NCU_TRAFFIC_PER_UNIT.get("ctr_similarity_kernel")
    out = {
        "metric": "CTR reduce throughput", "value": world * nbytes / (tot_ms * 1e-3) / 1e9, "unit": "GB/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": name, **{k: c[k] for k in ("T", "N", "D", "G", "tau_c", "dtype")},
                   "l2": "features 3.25 GB >> L2; a 512 MB write then a 512 MB read before every step",
                   "multi_gpu": "independent stream per rank, no collective"},
        "submetrics": {"frames_per_s": world * T / (tot_ms * 1e-3),
                       "stage_us": {"similarity": sim_ms * 1e3, "select": sel_ms * 1e3, "merge": mg_ms * 1e3},
                       "mean_k_s": float(ks.float().mean().item()),
                       "merge": {"ms": mg_ms, "frames_per_s": world * T / (mg_ms * 1e-3),
                                 "gram_TFLOPs": mg_flops / (mg_ms * 1e-3) / 1e12,
                                 "GBps": mg_bytes / (mg_ms * 1e-3) / 1e9,
                                 "frac_of_measured_hbm": mg_bytes / (mg_ms * 1e-3) / 1e9 / peak,
                                 "note": "Merge_{k_s} + retained group; the Gram matrix runs on the tensor cores (tcgen05, "
                                         "accumulators in tensor memory); flops and bytes are the algorithmic ones; not part "
                                         "of `value`, which covers similarity + select"},
                       "whole_ctr_frames_per_s": world * T / ((tot_ms + mg_ms) * 1e-3)},
        "roofline": {"kernel": "ctr_similarity_kernel", "bound": "hbm", "achieved": a, "peak": peak, "unit": "GB/s",
                     "frac": a / peak, "traffic": None if tpu is None else tpu * T, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": sbytes, "ms_per_launch": sim_ms},
        "gpu_launches": 3, "clocks": clocks,
    }
    if not args.no_e2e:
        # host buffers: features and saliency of a chunk of frames go up, the integer outputs come back; the frame
        # before a chunk is the carried state (`prev`)
        chunk = min(600, T)
        Fh = torch.empty(chunk, N, D, dtype=F.dtype).pin_memory()
        ah = torch.empty(chunk, N, dtype=torch.float32).pin_memory()
        Fh.copy_(F[:chunk])
        ah.copy_(alpha[:chunk])
        outs_h = [torch.empty(chunk, dtype=torch.int32).pin_memory(), torch.empty(chunk, dtype=torch.int32).pin_memory(),
                  torch.empty(chunk, G, dtype=torch.int32).pin_memory()]
        Fd, ad = torch.empty_like(F[:chunk]), torch.empty_like(alpha[:chunk])
        prev = torch.empty(N, D, dtype=F.dtype, device=dev)
        n_chunks = (T + chunk - 1) // chunk
        ts = []
        for it in range(args.e2e_steps + 1):
            torch.cuda.synchronize()
            a0, a1 = ev(), ev()
            a0.record()
            for cidx in range(n_chunks):
                Fd.copy_(Fh, non_blocking=True)
                ad.copy_(ah, non_blocking=True)
                oqm.stom_ctr_reduce(Fd, prev if cidx else None, chunk, N, D, (N * D, D), ad, G, c["tau_c"], sim[:chunk],
                                    ks[:chunk], kd[:chunk], si[:chunk], di[:chunk])
                prev.copy_(Fd[chunk - 1], non_blocking=True)
                outs_h[0].copy_(ks[:chunk], non_blocking=True)
                outs_h[1].copy_(kd[:chunk], non_blocking=True)
                outs_h[2].copy_(di[:chunk], non_blocking=True)
            a1.record()
            torch.cuda.synchronize()
            if it:
                ts.append(a0.elapsed_time(a1))
        e_ms = sdist.max_over_ranks(statistics.mean(ts))
        frames = n_chunks * chunk
        out["e2e"] = {"value": world * bytes_ctr(frames, N, D, G) / (e_ms * 1e-3) / 1e9, "unit": "GB/s",
                      "h2d_bytes_per_step": n_chunks * (Fh.numel() * 2 + ah.numel() * 4),
                      "d2h_bytes_per_step": n_chunks * sum(o.numel() * 4 for o in outs_h), "ms_per_step": e_ms,
                      "note": f"{n_chunks} chunks of {chunk} frames from pinned host memory, one synthetic chunk cycled"}
    if not args.no_cpu_baseline and rank == 0 and world == 1:
        from oracle import oqm_oracle as orc
        frames = min(T, CTR_CPU_FRAMES)
        Fc, ac = F[:frames].cpu(), alpha[:frames].cpu()
        t0 = time.perf_counter()
        o_sim = orc.ctr_similarity(synth.as_u16(Fc), orc.BF16)
        orc.ctr_select(o_sim, ac.numpy(), G, c["tau_c"])
        dt = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": bytes_ctr(frames, N, D, G) / dt / 1e9, "unit": "GB/s", "cores": 1,
                               "kind": "oracle", "sample": f"first {frames} frames (of {T})", "seconds": dt}
    if rank == 0:
        print(json.dumps(out))
    sdist.finish()


def main():
    args = parse()
    if args.config == "CTR":
        run_ctr(args)
        return
    from paper_2510_18269_b200 import synth
    sh = synth.CONFIGS[args.config]
    if args.meta != "fp32":
        import dataclasses
        sh = dataclasses.replace(sh, extra={**sh.extra, "meta": args.meta}, name=f"{sh.name}-meta-{args.meta}")
    if args.config == "C4" and args.impl == "ours":
        if args.frames:
            import dataclasses
            sh = dataclasses.replace(sh, T=args.frames)
        print(json.dumps(run_stream(args, sh)))
        return
    if args.layers or args.frames:
        import dataclasses
        sh = dataclasses.replace(sh, L=args.layers or sh.L, T=args.frames or sh.T,
                                 name=f"{sh.name}-reduced-L{args.layers or sh.L}-T{args.frames or sh.T}")
    if args.impl == "reference":
        run_reference(args, sh)
    else:
        run_ours(args, sh)


if __name__ == "__main__":
    main()

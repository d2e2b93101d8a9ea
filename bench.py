#!/usr/bin/env python
"""Benchmark of the packed-KV hot path on synthetic model-shaped caches.

One step = one pass of the whole path over all layers of the workload: per
layer, quantize-append one new token per sequence, one fused low-bit decode
attention over the full context, and a dequantize of the newest 128-token page.
The reported value is the packed K + V + metadata bytes the decode step has to
stream (all layers) divided by the step time, in GB/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--sweep]

N > 1: one rank per GPU (started here through torch.distributed.run when the
launcher has not already done so); the path shards by batch with no collective,
so every rank runs the same per-GPU workload (weak scaling).
`--impl reference` times the CPU oracle on a bounded sample of the workload.
`--sweep` runs every model-shaped variant once and prints one line per variant.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2502_15075_b200 import workloads as wl  # noqa: E402

METRIC = "decode-attention HBM GB/s (packed K+V+metadata bytes per decode step / time), K4V2, 32k context"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of one launch of the dominant kernel from an ncu capture (bytes), keyed by the sha256 of the
# kernel source it was taken from; reported as null once that source has changed.
NCU_TRAFFIC = {"2efc81c41ceb77b2f51a4ef4559fd4451d9eaad89bd5cdea35b5019c7e07870a": 440967424}   # dram read 436.43 MB + write 4.54 MB
DECODE_KERNEL_SOURCES = ("kvq_decode_mma.cuh", "kvq_decode_mma_kernel.cuh", "kvq_decode_mma_list.inc")

WORKLOADS = {"tiny": wl.TINY, "1b": wl.LLAMA_1B, "8b": wl.LLAMA_8B, "14b": wl.SHAPED_14B, "70b": wl.LLAMA_70B}


def workload_from_env() -> wl.Workload:
    w = WORKLOADS[os.environ.get("KVQ_BENCH_WORKLOAD", "8b")]
    if "KVQ_BENCH_LAYERS" in os.environ:
        w = w.with_(layers=int(os.environ["KVQ_BENCH_LAYERS"]))
    if "KVQ_BENCH_CONTEXT" in os.environ:
        w = w.with_(context=int(os.environ["KVQ_BENCH_CONTEXT"]))
    if "KVQ_BENCH_BITS" in os.environ:
        kb, vb = os.environ["KVQ_BENCH_BITS"].split(",")
        w = w.with_(kb=int(kb), vb=int(vb))
    return w


def decode_bytes_per_layer(w: wl.Workload, tokens=None) -> float:
    """Algorithmic bytes of one decode launch: packed K + V + metadata of every cached token (the fp16 tail of an
    incomplete channel-wise block counts as its 2 bytes per key element)."""
    T = w.context if tokens is None else tokens
    streams = w.batch * w.n_kv_heads
    if w.k_axis == 1 and T % 128:
        full, tail = T - T % 128, T % 128
        v_tok = w.head_dim * w.vb / 8 + (0.0 if w.vb == 16 else 4.0 * w.head_dim / w.gv)
        return streams * (full * wl.packed_bytes_per_token(w) + tail * (v_tok + 2.0 * w.head_dim))
    return streams * T * wl.packed_bytes_per_token(w)


def source_bytes_per_layer(w: wl.Workload, tokens=None) -> float:
    """16-bit K and V of one layer."""
    T = w.context if tokens is None else tokens
    return 2.0 * w.batch * w.n_kv_heads * T * w.head_dim * 2


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ----------------------------------------------------------------------------- multi-rank bookkeeping
def max_over_ranks(ms: float, world: int, device) -> float:
    """Every rank times its own replica; the job's time is the slowest rank's."""
    if world <= 1:
        return ms
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(bytes_per_rank_step: float, ms_per_step: float, world: int) -> float:
    """Weak scaling: every rank streams the same number of bytes per step; aggregate over the job."""
    return world * bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def respawn_under_launcher(n: int) -> None:
    """`bench.py --gpus N` started without a launcher: start N ranks of this same command (one per GPU)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """SM clock and throttle reasons sampled every few milliseconds during the timed region (NVML, read-only)."""
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period_s: float = 0.004):
        self.sm, self.reasons, self.max_mhz, self.err = [], set(), None, None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:                         # noqa: BLE001
            self.err = f"nvml unavailable: {e}"
            return
        self._period = period_s
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self.REASONS.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception as e:                     # noqa: BLE001
                self.err = str(e)
                return
            self._stop.wait(self._period)

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join(timeout=2)
        if not self.sm:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "samples": 0, "reasons": [self.err or "no samples"]}
        return {"sm_mhz": statistics.median(self.sm), "sm_min_mhz": min(self.sm), "sm_max_mhz": self.max_mhz,
                "samples": len(self.sm), "reasons": sorted(self.reasons)}


# ----------------------------------------------------------------------------- oracle legs
def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def oracle_sample_cache(w: wl.Workload, layer: int = 0):
    """One (batch, kv-head) stream of the workload at full context, built by the oracle on the CPU."""
    from oracle.cache import OracleCache
    ws = w.with_(n_kv_heads=1, n_q_heads=w.n_q_heads // w.n_kv_heads)
    T = w.context
    k, v = wl.make_kv(ws, layer=layer, tokens=T, batch=1)
    q = wl.make_q(ws, layer=layer, batch=1)
    bits = lambda t: t.contiguous().view(torch.int16).numpy().view(np.uint16)  # noqa: E731
    cap = ((T + 127) // 128) * 128 + 128
    oc = OracleCache(1, 1, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis, w.dtype, cap)
    oc.append(bits(k)[:, :, :T - 1], bits(v)[:, :, :T - 1])
    return ws, oc, bits(k)[:, :, T - 1:], bits(v)[:, :, T - 1:], bits(q)


def oracle_step(oc, k1, v1, qb, T):
    """The hot path once on the oracle's sample: append one token, decode, dequantize the newest page."""
    oc.seq_len[:] = T - 1
    oc.append(k1, v1)
    out = oc.decode(qb)
    page0 = ((T - 1) // 128) * 128
    ko = np.zeros((oc.B, oc.H, oc.capacity, oc.D), np.uint16)
    vo = np.zeros_like(ko)
    oc.dequantize(ko, vo, page0, T)
    return out


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from threadpoolctl import threadpool_limits
    w = workload_from_env()
    ws, oc, k1, v1, qb = oracle_sample_cache(w)
    sample_bytes = w.context * wl.packed_bytes_per_token(w)          # one stream, one layer
    with threadpool_limits(limits=1):
        for _ in range(args.warmup):
            oracle_step(oc, k1, v1, qb, w.context)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            oracle_step(oc, k1, v1, qb, w.context)
        dt = time.perf_counter() - t0
    ms = dt / args.steps * 1e3
    val = sample_bytes / (ms * 1e-3) / 1e9
    sample = f"1 of {w.batch * w.n_kv_heads} (batch, kv-head) streams of 1 of {w.layers} layers per step, full context"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(w),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "host_cores_available": host_cores(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(w: wl.Workload, tokens=None, ragged=False):
    T = w.context if tokens is None else tokens
    return {"workload": f"{w.name}: {w.layers} layers, batch {w.batch}, {w.n_q_heads}q/{w.n_kv_heads}kv heads, "
                        f"head_dim {w.head_dim}, context {T}{' (ragged U(T/2,T))' if ragged else ''}, {w.dtype}, "
                        f"K{w.kb}V{w.vb}, group {w.gk}/{w.gv}, k_axis {w.k_axis}",
            "step": "per layer: append 1 token/sequence, decode attention over the full context, "
                    "dequantize the newest page",
            "l2": ("inputs larger than L2 (one layer's packed cache exceeds it and layers rotate)"
                   if decode_bytes_per_layer(w, T) * w.layers > 2.5e8 else
                   "working set below L2 capacity: launch/L2-bound, not HBM-bound"),
            "parallelism": "replicas (batch-sharded, no collective)"}


def oracle_leg(kvq, w, cfg, cache, q, out_gpu, budget_s=12.0):
    """Time the oracle's decode on sampled streams of layer 0 (about 10-30 s of CPU work) and check the GPU
    output of those streams against it."""
    from threadpoolctl import threadpool_limits
    from oracle.cache import OracleCache
    B, H = w.batch, w.n_kv_heads
    G = w.n_q_heads // H
    cap = cfg.capacity_tokens
    pages = cache.pages_view()
    qb = q.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    seq = cache.seq_len.cpu().numpy()
    n_streams = B * H
    order = [(i * 37) % n_streams for i in range(min(n_streams, 48))]      # a fixed spread over the streams
    streams = [(s // H, s % H) for s in dict.fromkeys(order)]
    got_all = out_gpu.double().cpu().numpy()
    t_used, n_done, n_tok, errs = 0.0, 0, 0, []
    with threadpool_limits(limits=1):
        for (b, h) in streams:
            oc = OracleCache(1, 1, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis, w.dtype, cap)
            oc.pages = pages[b:b + 1, h:h + 1].cpu().numpy().copy()
            if oc.k_tail is not None:
                oc.k_tail = cache.tail_view()[b:b + 1, h:h + 1].cpu().view(torch.int16).numpy().view(np.uint16).copy()
            oc.seq_len[:] = seq[b]
            t0 = time.perf_counter()
            want = oc.decode(qb[b:b + 1, h * G:(h + 1) * G])
            t_used += time.perf_counter() - t0
            n_done += 1
            n_tok += int(seq[b])
            got = got_all[b:b + 1, h * G:(h + 1) * G]
            den = np.linalg.norm(want)
            errs.append((float(np.linalg.norm(got - want) / (den if den > 0 else 1.0)), float(np.abs(got - want).max())))
            if t_used > budget_s:
                break
    sample_bytes = n_tok * wl.packed_bytes_per_token(w)
    return {"baseline": {"value": sample_bytes / t_used / 1e9, "unit": UNIT, "cores": 1,
                         "host_cores_available": host_cores(), "kind": "oracle",
                         "sample": f"decode attention of {n_done} of {B * H} (batch, kv-head) streams of layer 0 at "
                                   f"full context, {t_used:.1f} s"},
            "parity": {"streams": n_done, "rel_l2_max": max(e[0] for e in errs), "max_abs_max": max(e[1] for e in errs),
                       "tolerance": {"rel_l2": 2e-3, "max_abs": 1e-2}}}


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def stats_us(ms_list):
    return {"median": statistics.median(ms_list) * 1e3, "min": min(ms_list) * 1e3,
            "mean": sum(ms_list) / len(ms_list) * 1e3, "n": len(ms_list)}


def hbm_block(kernel, bytes_per_launch, us, peak, peak_src, traffic=None, note=None):
    ach = bytes_per_launch / (us["median"] * 1e-6) / 1e9
    d = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
         "frac": ach / peak, "frac_of_8TBps_nominal": ach / NOMINAL_HBM_GBS, "us_per_launch": us["median"],
         "us_per_launch_min": us["min"], "us_per_launch_mean": us["mean"], "launches_timed": us["n"],
         "algorithmic_bytes_per_launch": bytes_per_launch, "traffic": traffic}
    if note:
        d["note"] = note
    return d


# ----------------------------------------------------------------------------- GPU arm
def run_workload(kvq, w: wl.Workload, dev, rank: int, world: int, steps: int, warmup: int, tokens=None,
                 ragged=False, append_tokens=0, oracle_budget_s=12.0, do_e2e=True):
    """Build all layers of `w` on the device, then time `steps` steps of the hot path.  Returns the result line."""
    import torch.distributed as dist
    T, B, L = (w.context if tokens is None else tokens), w.batch, w.layers
    cap = ((T + 127) // 128) * 128 + 128
    cfg = kvq.make_config(B, w.n_q_heads, w.n_kv_heads, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis,
                          w.torch_dtype, cap)
    ws_buf = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    # ---- build all layers (bulk quantize-append of T-1 tokens), timing the quantizer
    caches, qs, k1s, v1s = [], [], [], []
    quant_ms, append_ms = [], []
    bulk = T - 1 - append_tokens
    all_lens = torch.zeros((L, B), dtype=torch.int32, device=dev)     # every layer's sequence lengths, one tensor
    for layer in range(L):
        k, v = wl.make_kv(w, layer=layer + 100 * rank, device=dev, tokens=T)
        c = kvq.Cache(cfg, device=dev, seq_len=all_lens[layer])
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        kvq.kvq_quantize_append(cfg, c, k[:, :, :bulk], v[:, :, :bulk])
        e1.record()
        if append_tokens:
            kvq.kvq_quantize_append(cfg, c, k[:, :, bulk:T - 1], v[:, :, bulk:T - 1])
        e2.record()
        torch.cuda.synchronize()
        quant_ms.append(e0.elapsed_time(e1))
        if append_tokens:
            append_ms.append(e1.elapsed_time(e2))
        caches.append(c)
        k1s.append(k[:, :, T - 1:].contiguous())
        v1s.append(v[:, :, T - 1:].contiguous())
        qs.append(wl.make_q(w, layer=layer + 100 * rank, device=dev))
        del k, v
    lens = None
    if ragged:
        lens = wl.ragged_seq_lens(w, T, B).to(dev)
    q_us = stats_us(quant_ms[1:] or quant_ms)

    outs = [torch.empty((B, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
    page0 = ((T - 1) // 128) * 128
    deq_k = torch.empty((B, w.n_kv_heads, cap, w.head_dim), dtype=w.torch_dtype, device=dev)
    deq_v = torch.empty_like(deq_k)

    def reset_lens():
        # a step appends one token to every layer: put all layers back to T - 1 cached tokens, in one operation
        if lens is None:
            all_lens.fill_(T - 1)
        else:
            all_lens.copy_((lens - 1).unsqueeze(0).expand(L, B))

    def step_device(events=None):
        reset_lens()
        for i in range(L):
            c = caches[i]
            kvq.kvq_quantize_append(cfg, c, k1s[i], v1s[i])
            if events is not None:
                a, b_ = ev(), ev()
                a.record()
            kvq.kvq_decode_attention(cfg, c, qs[i], outs[i], ws_buf)
            if events is not None:
                b_.record()
                events.append((a, b_))
            kvq.kvq_dequantize(cfg, c, deq_k, deq_v, page0, T)

    # pinned host buffers for the end-to-end variant
    hk = [t.cpu().pin_memory() for t in k1s]
    hv = [t.cpu().pin_memory() for t in v1s]
    hq = [t.cpu().pin_memory() for t in qs]
    hout = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs]
    dk, dv, dq = torch.empty_like(k1s[0]), torch.empty_like(v1s[0]), torch.empty_like(qs[0])

    def step_e2e():
        reset_lens()
        for i in range(L):
            c = caches[i]
            kvq.quantize_append_host(cfg, c, hk[i], hv[i], dk, dv)
            kvq.decode_attention_host(cfg, c, hq[i], hout[i], dq, outs[i], ws_buf)
            kvq.kvq_dequantize(cfg, c, deq_k, deq_v, page0, T)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, n, events=None):
        barrier()
        s, e = ev(), ev()
        s.record()
        for _ in range(n):
            fn(events) if events is not None else fn()
        e.record()
        barrier()
        return max_over_ranks(s.elapsed_time(e), world, dev)

    for _ in range(warmup):
        step_device()
    local_rank = dev.index or 0
    sampler = ClockSampler(local_rank) if rank == 0 else None
    events = []
    total_ms = timed(step_device, steps, events)
    clocks = sampler.stop() if sampler else None
    ms_per_step = total_ms / steps
    dec_us = stats_us([a.elapsed_time(b_) for a, b_ in events])

    # ---- the same step captured once in a CUDA graph and replayed (no per-call events, no host launch gaps)
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            # thread_local: other threads (a collective library's watchdog) may call the runtime meanwhile
            with torch.cuda.graph(step_graph, stream=side, capture_error_mode="thread_local"):
                step_device()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(2):
            step_graph.replay()
        graph_ms = timed(step_graph.replay, steps) / steps
        del step_graph
    except RuntimeError as e:                      # reported, never fatal: the eager numbers above stand
        graph_ms = "capture failed: " + str(e).splitlines()[0][:120]

    e2e_ms = None
    if do_e2e:
        for _ in range(max(1, warmup // 2)):
            step_e2e()
        e2e_ms = timed(step_e2e, steps) / steps

    # ---- dequantize of whole layers (reads the packed layer, writes 16-bit K and V), layers rotating
    deq_ms = []
    for r in range(min(max(4, L), 12) + 1):
        c = caches[r % L]
        a, b_ = ev(), ev()
        a.record()
        kvq.kvq_dequantize(cfg, c, deq_k, deq_v, 0, T)
        b_.record()
        torch.cuda.synchronize()
        if r:
            deq_ms.append(a.elapsed_time(b_))
    dq_us = stats_us(deq_ms)

    # ---- the two kernels of the fast decode path side by side (decode calls only, layers rotating): the
    # warp-level integer-MMA kernel, which is the product path, and the tcgen05 / tensor-memory kernel
    variants = {}
    for label, impl in (("warp_mma", kvq.IMPL_WARP_MMA), ("tcgen05", kvq.IMPL_TCGEN05)):
        try:
            pairs = []
            for r in range(3 * max(L, 4) + 2):
                a, b_ = ev(), ev()
                a.record()
                kvq.kvq_debug_decode_impl(cfg, caches[r % L], qs[r % L], outs[r % L], ws_buf, impl)
                b_.record()
                pairs.append((a, b_))
            torch.cuda.synchronize()
            variants[label] = stats_us([a.elapsed_time(b_) for a, b_ in pairs[2:]])
            # the same launches with one pair of events around the whole batch: a kernel's launch overlaps the one
            # before it, and the event timer's ~2 us steps average out
            n_batch = 3 * max(L, 4)
            a, b_ = ev(), ev()
            a.record()
            for r in range(n_batch):
                kvq.kvq_debug_decode_impl(cfg, caches[r % L], qs[r % L], outs[r % L], ws_buf, impl)
            b_.record()
            torch.cuda.synchronize()
            variants[label]["us_per_launch_in_a_batch"] = a.elapsed_time(b_) * 1000.0 / n_batch
        except kvq.KvqError as e:
            variants[label] = {"unsupported": e.code}
    if kvq.kvq_check_status(caches[0]) != 0:
        raise RuntimeError("library reported a status error")

    n_tok = T if lens is None else float(lens.sum().item()) / B      # mean cached tokens per sequence
    bytes_layer = decode_bytes_per_layer(w, T) * (n_tok / T)
    bytes_step = bytes_layer * L
    value = whole_job_gbs(bytes_step, ms_per_step, world)
    if rank != 0:
        return None
    peak, peak_src = peak_hbm()
    hsh = hashlib.sha256()
    for name in DECODE_KERNEL_SOURCES:
        hsh.update(open(os.path.join(ROOT, "paper_2502_15075_b200", "csrc", name), "rb").read())
    traffic = NCU_TRAFFIC.get(hsh.hexdigest()) if (w.name, w.kb, w.vb, T, ragged) == (wl.LLAMA_8B.name, 4, 2, 32768, False) else None
    roofline = hbm_block("kvq_decode_attention (one fused kernel: split decode + merge)", bytes_layer, dec_us, peak,
                         peak_src, traffic)
    src_bulk = source_bytes_per_layer(w, bulk)
    packed_bulk = decode_bytes_per_layer(w, T) * bulk / T
    roof_q = hbm_block("kvq_quantize_append, bulk build of one layer (reads 16-bit K and V, writes the packed layer)",
                       src_bulk + packed_bulk, q_us, peak, peak_src)
    roof_dq = hbm_block("kvq_dequantize of one whole layer (reads the packed layer, writes 16-bit K and V)",
                        decode_bytes_per_layer(w, T) + source_bytes_per_layer(w, T), dq_us, peak, peak_src)

    cpu = oracle_leg(kvq, w, cfg, caches[0], qs[0], outs[0], oracle_budget_s)
    fast_bits = lambda b: b in (2, 4, 8)  # noqa: E731
    deq_launches = ((1 if w.head_dim == 128 and fast_bits(w.vb) else 0) +
                    (1 if w.head_dim == 128 and w.k_axis == 0 and fast_bits(w.kb) else 0))
    if deq_launches == 2:
        deq_launches = 1 if B * w.n_kv_heads <= 148 * 8 else 2     # a short range takes both sides in one launch
    else:
        deq_launches += 1                                           # the general kernel serves what is left
    # append (quantize [+ channel-wise K] + bump), decode, dequantize of the newest page
    kern_per_layer = (2 if w.k_axis == 0 else 3) + 1 + deq_launches
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32 accumulate over 8-bit operands (fp32 softmax and merge)",
            "data": "synthetic", "config": config_dict(w, T, ragged), "roofline": roofline,
            "roofline_quantize": roof_q, "roofline_dequantize": roof_dq,
            "cpu_baseline": cpu["baseline"], "parity_sample": cpu["parity"],
            "gpu_launches": L * kern_per_layer * steps,
            "quantize": {"tokens_per_s": world * B * bulk / (q_us["median"] * 1e-6), "us_per_layer_bulk": q_us,
                         "tokens_per_call": B * bulk},
            "decode_kernels_us": variants, "clocks": clocks}
    if e2e_ms is not None:
        line["e2e"] = {"value": whole_job_gbs(bytes_step, e2e_ms, world), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": L * (2 * k1s[0].numel() * 2 + qs[0].numel() * 2),
                       "d2h_bytes_per_step": L * outs[0].numel() * 4}
    if isinstance(graph_ms, float):
        line["cuda_graph"] = {"ms_per_step": graph_ms, "value": whole_job_gbs(bytes_step, graph_ms, world), "unit": UNIT,
                              "what": "the same step (all layers) captured once in a CUDA graph and replayed"}
    elif graph_ms is not None:
        line["cuda_graph"] = {"unavailable": graph_ms}
    if append_ms:
        a_us = stats_us(append_ms[1:] or append_ms)
        line["append"] = {"tokens_per_call": B * append_tokens, "us_per_call": a_us,
                          "tokens_per_s": B * append_tokens / (a_us["median"] * 1e-6)}
    return line


SWEEP = (
    # (label, workload key, overrides, tokens, ragged, append_tokens)
    ("tiny K4V2 g32", "tiny", {}, None, False, 0),
    ("1B-shaped K4V2 g64, bulk 3968 + append 128", "1b", {}, None, False, 127),
    ("8B-shaped K4V2", "8b", {}, None, False, 0),
    ("8B-shaped K2V4", "8b", {"kb": 2, "vb": 4}, None, False, 0),
    ("8B-shaped K4V4", "8b", {"kb": 4, "vb": 4}, None, False, 0),
    ("8B-shaped K8V4", "8b", {"kb": 8, "vb": 4}, None, False, 0),
    ("8B-shaped K4V2, ragged lengths", "8b", {}, None, True, 0),
    ("14B-shaped K4V2 channel-wise keys, T=16384", "14b", {}, None, False, 0),
    ("14B-shaped K4V2 channel-wise keys, T=16383 (127-token tail)", "14b", {}, 16383, False, 0),
    ("14B-shaped K8V2 channel-wise keys, T=16384", "14b", {"kb": 8}, None, False, 0),
    ("14B-shaped K8V2 channel-wise keys, T=16383 (127-token tail)", "14b", {"kb": 8}, 16383, False, 0),
    ("70B-shaped K4V2, 80 layers resident", "70b", {}, None, False, 0),
)


def main_gpu(args):
    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2502_15075_b200 import build
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    from paper_2502_15075_b200 import kvq

    if not args.sweep:
        line = run_workload(kvq, workload_from_env(), dev, rank, world, args.steps, args.warmup)
        if rank == 0:
            print(json.dumps(line))
        return
    only = os.environ.get("KVQ_BENCH_SWEEP_ONLY")
    for label, key, over, tokens, ragged, app in SWEEP:
        if only and only not in label:
            continue
        w = WORKLOADS[key].with_(**over)
        if "KVQ_BENCH_LAYERS" in os.environ:
            w = w.with_(layers=min(w.layers, int(os.environ["KVQ_BENCH_LAYERS"])))
        line = run_workload(kvq, w, dev, rank, world, args.steps, args.warmup, tokens=tokens, ragged=ragged,
                            append_tokens=app, oracle_budget_s=4.0, do_e2e=False)
        if rank == 0:
            line["sweep"] = label
            print(json.dumps(line), flush=True)
        torch.cuda.empty_cache()


def selftest_ranks(args):
    """Rank plumbing only (gloo, CPU): rendezvous, barrier, max-over-ranks and the whole-job aggregate."""
    import torch.distributed as dist
    rank, _, world = dist_env()
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = max_over_ranks(10.0 + rank, world, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"selftest": True, "n_gpus": world, "ms_per_step": ms,
                          "value": whole_job_gbs(1e9, ms, world)}))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kvq", choices=["kvq", "reference"])
    ap.add_argument("--sweep", action="store_true", help="run every model-shaped variant, one line each")
    ap.add_argument("--selftest-ranks", action="store_true", help=argparse.SUPPRESS)
    a = ap.parse_args()
    if a.gpus > 1 and "WORLD_SIZE" not in os.environ:
        respawn_under_launcher(a.gpus)
    if a.selftest_ranks:
        selftest_ranks(a)
    elif a.impl == "reference":
        run_reference(a)
    else:
        main_gpu(a)

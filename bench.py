#!/usr/bin/env python
"""Benchmark of the packed-KV hot path on synthetic model-shaped caches.

One step = one pass of the whole path over all layers of the workload: per
layer, quantize-append one new token per sequence, one fused low-bit decode
attention over the full context, and a dequantize of the newest 128-token page.
The reported value is the packed K + V + metadata bytes the decode step has to
stream (all layers) divided by the step time, in GB/s.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 runs under torchrun, one rank per GPU; the path shards by batch with no
collective, so every rank runs the same per-GPU workload (weak scaling).
`--impl reference` times the CPU oracle on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2502_15075_b200 import workloads as wl  # noqa: E402

METRIC = "decode-attention HBM GB/s (packed K+V+metadata bytes per decode step / time), K4V2, 32k context"
UNIT = "GB/s"

# DRAM traffic of one launch of the dominant kernel from an ncu capture (bytes), keyed by the sha256 of the
# kernel source it was taken from; reported as null once that file has changed.
NCU_TRAFFIC = {"ba0a2a7127d6efbb20d92d017f81aa64248ffbac0e25a1297d0c33a0fe1c0a80": 441370368}   # dram read 436.51 MB + write 4.86 MB
DECODE_KERNEL_SOURCES = ("kvq_decode_mma.cuh", "kvq_decode_mma_kernel.cuh", "kvq_decode_mma_list.inc")


def workload_from_env() -> wl.Workload:
    name = os.environ.get("KVQ_BENCH_WORKLOAD", "8b")
    table = {"tiny": wl.TINY, "1b": wl.LLAMA_1B, "8b": wl.LLAMA_8B, "14b": wl.SHAPED_14B, "70b": wl.LLAMA_70B}
    w = table[name]
    if "KVQ_BENCH_LAYERS" in os.environ:
        w = w.with_(layers=int(os.environ["KVQ_BENCH_LAYERS"]))
    if "KVQ_BENCH_CONTEXT" in os.environ:
        w = w.with_(context=int(os.environ["KVQ_BENCH_CONTEXT"]))
    if "KVQ_BENCH_BITS" in os.environ:
        kb, vb = os.environ["KVQ_BENCH_BITS"].split(",")
        w = w.with_(kb=int(kb), vb=int(vb))
    return w


def decode_bytes_per_layer(w: wl.Workload) -> float:
    return w.batch * w.n_kv_heads * w.context * wl.packed_bytes_per_token(w)


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


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- oracle legs
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
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(w: wl.Workload):
    return {"workload": f"{w.name}: {w.layers} layers, batch {w.batch}, {w.n_q_heads}q/{w.n_kv_heads}kv heads, "
                        f"head_dim {w.head_dim}, context {w.context}, {w.dtype}, K{w.kb}V{w.vb}, "
                        f"group {w.gk}/{w.gv}, k_axis {w.k_axis}",
            "step": "per layer: append 1 token/sequence, decode attention over the full context, "
                    "dequantize the newest page",
            "l2": "inputs larger than L2 (one layer's packed cache exceeds it and layers rotate)",
            "parallelism": "replicas (batch-sharded, no collective)"}


# ----------------------------------------------------------------------------- GPU arm
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

    w = workload_from_env()
    T, B, L = w.context, w.batch, w.layers
    cap = ((T + 127) // 128) * 128 + 128
    cfg = kvq.make_config(B, w.n_q_heads, w.n_kv_heads, w.head_dim, w.kb, w.vb, w.gk, w.gv, w.k_axis,
                          w.torch_dtype, cap)
    ws_buf = torch.empty(max(16, kvq.kvq_workspace_bytes(cfg)), dtype=torch.uint8, device=dev)

    # ---- build all layers (bulk quantize-append of T-1 tokens), timing the quantizer
    caches, qs, k1s, v1s = [], [], [], []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    quant_ms = []
    for layer in range(L):
        k, v = wl.make_kv(w, layer=layer + 100 * rank, device=dev)
        c = kvq.Cache(cfg, device=dev)
        e0.record()
        kvq.kvq_quantize_append(cfg, c, k[:, :, :T - 1], v[:, :, :T - 1])
        e1.record()
        torch.cuda.synchronize()
        quant_ms.append(e0.elapsed_time(e1))
        caches.append(c)
        k1s.append(k[:, :, T - 1:].contiguous())
        v1s.append(v[:, :, T - 1:].contiguous())
        qs.append(wl.make_q(w, layer=layer + 100 * rank, device=dev))
        del k, v
    quant_ms_med = statistics.median(quant_ms[1:] or quant_ms)
    quant_tokens_s = B * (T - 1) / (quant_ms_med * 1e-3)
    quant_gbs = (2 * B * w.n_kv_heads * (T - 1) * w.head_dim * 2 + decode_bytes_per_layer(w)) / (quant_ms_med * 1e-3) / 1e9

    outs = [torch.empty((B, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev) for _ in range(L)]
    page0 = ((T - 1) // 128) * 128
    deq_k = torch.empty((B, w.n_kv_heads, cap, w.head_dim), dtype=w.torch_dtype, device=dev)
    deq_v = torch.empty_like(deq_k)

    def step_device(events=None):
        for i in range(L):
            c = caches[i]
            c.seq_len.fill_(T - 1)
            kvq.kvq_quantize_append(cfg, c, k1s[i], v1s[i])
            if events is not None:
                a = torch.cuda.Event(enable_timing=True)
                b_ = torch.cuda.Event(enable_timing=True)
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
        for i in range(L):
            c = caches[i]
            c.seq_len.fill_(T - 1)
            kvq.quantize_append_host(cfg, c, hk[i], hv[i], dk, dv)
            kvq.decode_attention_host(cfg, c, hq[i], hout[i], dq, outs[i], ws_buf)
            kvq.kvq_dequantize(cfg, c, deq_k, deq_v, page0, T)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps, events=None):
        barrier()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(steps):
            fn(events) if events is not None else fn()
        e.record()
        barrier()
        return max_over_ranks(s.elapsed_time(e), world, dev)

    for _ in range(args.warmup):
        step_device()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    events = []
    total_ms = timed(step_device, args.steps, events)
    clocks = sampler.stop() if sampler else None
    ms_per_step = total_ms / args.steps
    dec_ms = [a.elapsed_time(b_) for a, b_ in events]
    dec_ms_avg = sum(dec_ms) / len(dec_ms)

    for _ in range(max(1, args.warmup // 2)):
        step_e2e()
    e2e_ms = timed(step_e2e, args.steps) / args.steps
    if kvq.kvq_check_status(caches[0]) != 0:
        raise RuntimeError("library reported a status error")

    bytes_layer = decode_bytes_per_layer(w)
    bytes_step = bytes_layer * L
    value = whole_job_gbs(bytes_step, ms_per_step, world)
    e2e_value = whole_job_gbs(bytes_step, e2e_ms, world)

    if rank != 0:
        return
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    achieved = bytes_layer / (dec_ms_avg * 1e-3) / 1e9
    hsh = hashlib.sha256()
    for name in DECODE_KERNEL_SOURCES:
        hsh.update(open(os.path.join(ROOT, "paper_2502_15075_b200", "csrc", name), "rb").read())
    sha = hsh.hexdigest()
    roofline = {"bound": "hbm", "kernel": "kvq_decode_attention (split kernel + merge)", "achieved": achieved,
                "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                "frac_of_8TBps_nominal": achieved / 8000.0, "us_per_launch": dec_ms_avg * 1e3,
                "algorithmic_bytes_per_launch": bytes_layer, "traffic": NCU_TRAFFIC.get(sha)}

    # ---- CPU oracle on a bounded sample of the same workload, with a parity check of the GPU output
    cpu = oracle_leg(kvq, w, cfg, caches[0], qs[0], outs[0])

    n_launch = L * (2 + 2 + 1 + (1 if w.k_axis == 1 else 0))   # append (quantize [+ K channel] + bump), decode + merge, dequantize
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32 accumulate over f16 operands", "data": "synthetic",
            "config": config_dict(w), "roofline": roofline, "cpu_baseline": cpu["baseline"],
            "parity_sample": cpu["parity"],
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": L * (2 * k1s[0].numel() * 2 + qs[0].numel() * 2),
                    "d2h_bytes_per_step": L * outs[0].numel() * 4},
            "gpu_launches": n_launch * args.steps,
            "quantize": {"tokens_per_s": quant_tokens_s * world, "ms_per_layer_bulk": quant_ms_med,
                         "GBps_read_plus_write": quant_gbs, "tokens_per_call": B * (T - 1)},
            "clocks": clocks}
    print(json.dumps(line))


def oracle_leg(kvq, w, cfg, cache, q, out_gpu):
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
    t_used, n_done, errs = 0.0, 0, []
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
            got = got_all[b:b + 1, h * G:(h + 1) * G]
            errs.append((float(np.linalg.norm(got - want) / np.linalg.norm(want)), float(np.abs(got - want).max())))
            if t_used > 12.0:
                break
    sample_bytes = n_done * w.context * wl.packed_bytes_per_token(w)
    return {"baseline": {"value": sample_bytes / t_used / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"decode attention of {n_done} of {B * H} (batch, kv-head) streams of layer 0 at "
                                   f"full context, {t_used:.1f} s"},
            "parity": {"streams": n_done, "rel_l2_max": max(e[0] for e in errs), "max_abs_max": max(e[1] for e in errs),
                       "tolerance": {"rel_l2": 2e-3, "max_abs": 1e-2}}}


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="kvq", choices=["kvq", "reference"])
    a = ap.parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        main_gpu(a)

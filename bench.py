#!/usr/bin/env python
"""Benchmark of the hot path: decode steps over an XQuant KV cache at 32k context.

One step = one generated token of a whole model: for each of the 32 layers,
append the token's K,V (window append; quantize-and-pack whenever a window block
fills) and run decode attention over the packed cache plus the window.  The
metric is decode-attention GB/s: the bytes the method itself must move per
layer call (packed codes, fp16 scale / zero-point, 16-bit window, q, out)
divided by time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl ours|reference]

With N > 1 (launched by torchrun) every rank runs the same workload on its own
GPU -- sequences are independent, so the path shards by batch with no
collective -- and the aggregate is reported (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode-attention GB/s at 32k ctx"
APPEND_BLOCKS = 6  # window blocks quantized per layer in the append pass, one block per call
BULK_BYTES = 256e6  # then two calls per layer of about this much 16-bit input each (a prefill-sized append):
BULK_MIN, BULK_MAX = 16, 64  # between 16 and 64 window blocks per call
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the decode kernel (ncu, same launch shape as the
# timed one; see profiles/), with the SHA-256 of the kernel's sources at the time the counters were taken: the
# figure is reported only while the sources still hash to that.
NCU_TRAFFIC = {"c2": {"bytes": 84.05e6 + 2.60e6,
                      "sources_sha256": "aafe1f3193d74c1d55e9d1a4309874d6a8a793292f0d4dcb65080bbb7dc7a849"}}
KERNEL_SOURCES = ("xq_decode_umma.cu", "xq_layout.cuh", "xq_internal.h")


def _kernel_sources_hash():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2510_11236_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _ncu_traffic(config):
    t = NCU_TRAFFIC.get(config)
    if t is None or t["sources_sha256"] != _kernel_sources_hash():
        return None
    return t["bytes"]


def _config_block(args, w):
    """What both arms print as `config`: the workload by name and its shape."""
    from paper_2510_11236_b200 import workloads
    return {"workload": f"{args.config}: {workloads.TITLES.get(args.config, 'custom')}",
            **{k: w[k] for k in ("n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "seq", "residual_len",
                                 "group_size", "kq", "vq", "km", "vm")},
            "eta1": args.eta1, "eta2": args.eta2,
            "step": "per layer: append 1 token (+ quantize-and-pack when the window block fills) and decode attention",
            "l2": "inputs larger than L2: every step streams the whole packed cache (GBs against 126 MB of L2); "
                  "owners-first layer order keeps a pair's shared codes from being re-served by L2"}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self, t_lo=None, t_hi=None):
        """Median SM clock and the throttle reasons seen.  With a window [t_lo, t_hi] (datetime, local time) the
        figures come from the samples inside it when there are any (`window`: "timed region"), else from every
        sample since the sampler started (`window`: "whole run": warm-up and all passes)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        rows = []
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                rows.append((ts, float(parts[1]), float(parts[2]), parts[5:9]))
            except ValueError:
                continue
        inside = [r for r in rows if t_lo is not None and t_lo <= r[0] <= t_hi]
        out["window"] = "timed region" if inside else "whole run"
        clocks, mx, reasons = [], [], set()
        for ts, c, m, flags in (inside or rows):
            clocks.append(c); mx.append(m)
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), flags):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if clocks:
            out["sm_mhz"] = statistics.median(clocks)
            out["sm_max_mhz"] = max(mx)
            out["samples"] = len(clocks)
        out["reasons"] = sorted(reasons)
        return out


class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the workload: decode
    attention of one layer for `n_streams` (sequence, kv head) streams at the full
    context (dequantize the stream's packed region in fp64, then attention for
    its query heads).  Building the streams' caches is set-up, not timed."""

    def __init__(self, w, n_streams, eta1, eta2):
        import numpy as np
        import torch
        from oracle import xq_oracle as O
        from paper_2510_11236_b200 import workloads as W
        from tests import util
        S = w["seq"]
        G = w["n_q_heads"] // w["n_kv_heads"]
        self.n_streams = n_streams
        k0, v0, _, _ = W.pair_tokens(dict(w, batch=1, n_kv_heads=n_streams), 0, 0, S, "cpu")
        self.caches = []
        for s in range(n_streams):
            oc = O.OracleCache(1, 1, G, 1, w["head_dim"], w["group_size"], w["residual_len"],
                               1 if w["kq"] > 0 else 0, 1 if w["vq"] > 0 else 0, 1, 1,
                               np.float32(eta1), np.float32(eta2))
            oc.append(0, util.bits_of(k0[:, s:s + 1]), util.bits_of(v0[:, s:s + 1]))
            self.caches.append(oc)
        gen = torch.Generator().manual_seed(5)
        self.q = util.bits_of(torch.randn(1, G, w["head_dim"], generator=gen).to(torch.bfloat16))
        self.bytes = n_streams * W.algorithmic_bytes(dict(w, batch=1, n_kv_heads=1, n_q_heads=G), S, 0)
        self.cores = 1

    def run(self):
        """Seconds for one pass over the sample, single-threaded."""
        try:
            from threadpoolctl import threadpool_limits
        except Exception:  # pragma: no cover
            threadpool_limits = None
        t0 = time.perf_counter()
        if threadpool_limits is not None:
            with threadpool_limits(limits=1):
                for oc in self.caches:
                    oc.decode(0, self.q)
        else:
            for oc in self.caches:
                oc.decode(0, self.q)
        return time.perf_counter() - t0


def _oracle_worker(job):
    """One process of the all-cores figure: builds one stream's oracle cache, then runs decode passes for about
    `seconds`; returns (passes, seconds spent in them, bytes per pass)."""
    w, eta1, eta2, seconds = job
    smp = OracleSample(w, 1, eta1, eta2)
    smp.run()
    dt, passes = 0.0, 0
    while dt < seconds:
        dt += smp.run()
        passes += 1
    return passes, dt, smp.bytes


def oracle_all_cores(w, eta1, eta2, seconds=6.0):
    """The oracle on every host core at once: one single-threaded process per core (at most 32), each on its own
    stream; the figure is the sum of the processes' rates."""
    import multiprocessing as mp
    n = max(1, min(os.cpu_count() or 1, 32))
    ctx = mp.get_context("spawn")
    with ctx.Pool(n) as pool:
        res = pool.map(_oracle_worker, [(w, eta1, eta2, seconds)] * n)
    return sum(p * b / dt for p, dt, b in res) / 1e9, n


def run_reference(args, w):
    """The reference arm: the CPU oracle timed on this machine's host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_streams = 2
    smp = OracleSample(w, n_streams, args.eta1, args.eta2)
    times = []
    for i in range(args.warmup + args.steps):
        dt = smp.run()
        if i >= args.warmup:
            times.append(dt)
    T = sum(times) / len(times)
    val = smp.bytes / T / 1e9
    sample = (f"decode attention of one layer for {n_streams} of {w['batch'] * w['n_kv_heads']} (sequence, kv head) "
              f"streams at S={w['seq']} per step (dequantize + attention, fp64 numpy)")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": T * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config_block(args, w),
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="c2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--eta1", type=float, default=1.0 / 6.0)
    ap.add_argument("--eta2", type=float, default=0.045)
    ap.add_argument("--kernel", type=int, default=0)
    ap.add_argument("--splits", type=int, default=None)
    ap.add_argument("--layer-order", default="owners_first", choices=["owners_first", "ascending"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=None, help="fewer layers than the workload names (profiling captures only)")
    ap.add_argument("--seq", type=int, default=None, help="another context length (profiling captures only)")
    args = ap.parse_args()

    from paper_2510_11236_b200 import workloads as W
    w = dict(W.CONFIGS[args.config])
    if args.layers:
        w["n_layers"] = args.layers
        w["kq"], w["vq"] = min(w["kq"], args.layers), min(w["vq"], args.layers)
    if args.seq:
        w["seq"] = args.seq
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    import paper_2510_11236_b200 as xq
    from paper_2510_11236_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    w = sharding.rank_workload(w, rank)  # every rank holds its own sequences

    L, B, Hq, Hkv, D, S = w["n_layers"], w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"], w["seq"]
    K, Wm = args.steps, args.warmup
    R = w["residual_len"]
    BULK_BLOCKS = int(max(BULK_MIN, min(BULK_MAX, BULK_BYTES // (2 * B * Hkv * R * D * 2))))
    n_total = Wm + 3 * K + 8 + (APPEND_BLOCKS + 1 + 2 * BULK_BLOCKS) * R  # warm-up, three timed passes, then the append pass
    cfg = W.make_xq_config(w, max_seq=S + n_total + 1, eta1=args.eta1, eta2=args.eta2, kernel=args.kernel,
                           n_splits=args.splits)
    cache = xq.Cache(cfg, dev)

    # ---- prefill to S - warmup tokens, so that the warm-up steps end at S and the first timed step
    # ---- quantizes the full window of every layer
    S0 = max(1, S - Wm)
    for pair in range(L // 2):
        for c0 in range(0, S0, W.CHUNK):
            c1 = min(S0, c0 + W.CHUNK)
            k0, v0, k1, v1 = W.pair_tokens(w, pair, c0, c1, dev)
            cache.append_kv(2 * pair, k0, v0)
            cache.append_kv(2 * pair + 1, k1, v1)
    torch.cuda.synchronize()

    # ---- per-step inputs (distinct every step), on the device and in pinned host memory
    g = torch.Generator(device=dev).manual_seed(1234 + rank)
    n_pool = min(n_total, 64)
    pool = []
    for i in range(n_pool):
        kn = torch.randn(L, B, Hkv, 1, D, generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn(L, B, Hkv, 1, D, generator=g, device=dev).to(torch.bfloat16)
        qn = torch.randn(L, B, Hq, D, generator=g, device=dev).to(torch.bfloat16)
        pool.append((kn, vn, qn))
    host_pool = [(a.cpu().pin_memory(), b.cpu().pin_memory(), c.cpu().pin_memory()) for a, b, c in pool[:8]]
    out_dev = torch.empty(L, B, Hq, D, dtype=torch.bfloat16, device=dev)
    out_host = torch.empty(L, B, Hq, D, dtype=torch.bfloat16).pin_memory()
    order = None
    if args.layer_order == "owners_first":
        order = list(range(0, L, 2)) + list(range(1, L, 2))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_no = [0]

    def device_step():
        kn, vn, qn = pool[step_no[0] % n_pool]
        step_no[0] += 1
        cache.decode_step(kn, vn, qn, out_dev, order)

    def step_bytes(first_seq, n_steps):
        tot = 0
        for i in range(n_steps):
            for l in range(L):
                tot += W.algorithmic_bytes(w, first_seq + i, l)
        return tot

    import datetime
    sampler = ClockSampler(local) if rank == 0 else None  # runs from before the warm-up to the end of pass 3
    for _ in range(Wm):
        device_step()
    barrier()

    # ---- pass 1: whole steps, inputs resident in HBM
    seq_before = cache.seq_len(0)
    launches_before = xq.xq_launch_count(cache.handle)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_lo = datetime.datetime.now()
    e0.record()
    for _ in range(K):
        device_step()
    e1.record()
    barrier()
    t_hi = datetime.datetime.now()
    ms = e0.elapsed_time(e1)
    launches = xq.xq_launch_count(cache.handle) - launches_before
    bytes_pass1 = step_bytes(seq_before + 1, K)
    ms_max = sharding.max_over_ranks(ms, dev)
    value = sharding.aggregate_rate(bytes_pass1, ms_max, world) / 1e9
    tokens_per_s = sharding.aggregate_rate(B * sum(seq_before + 1 + i for i in range(K)), ms_max, world)

    # ---- pass 2: the same steps with CUDA events around every kernel (roofline of the dominant kernel)
    xq.xq_timing_enable(cache.handle, 1)
    seq_before2 = cache.seq_len(0)
    barrier()
    for _ in range(K):
        device_step()
    barrier()
    kinds = {}
    for kind, name in enumerate(("decode_split", "merge", "quantize_pack", "window_append")):
        rc, n, tot = xq.xq_timing_read(cache.handle, kind)
        kinds[name] = {"launches": n, "total_ms": tot, "avg_us": (tot / n * 1e3) if n else None}
    xq.xq_timing_enable(cache.handle, 0)
    dec = kinds["decode_split"]
    bytes_pass2 = step_bytes(seq_before2 + 1, K)
    peak, peak_kind = _peaks()
    isolated = bytes_pass2 / (dec["total_ms"] * 1e-3) / 1e9 if dec["launches"] else 0.0
    # The decode launches of pass 1 run back to back (each starts its prologue while its predecessor drains), so
    # their average duration over that timed region is the region's time over their number; the few other kernels
    # of the region (the steps that quantize a window block) are charged to them.
    decode_launches_pass1 = K * L
    avg_launch_us = ms / decode_launches_pass1 * 1e3
    achieved = bytes_pass1 / (ms * 1e-3) / 1e9

    # ---- pass 3: end to end through the C ABI with host buffers
    seq_before3 = cache.seq_len(0)
    h2d = sum(x.numel() * 2 for x in host_pool[0])
    d2h = out_host.numel() * 2
    stream = torch.cuda.current_stream()
    barrier()
    t0 = time.perf_counter()
    e0.record()
    for i in range(K):
        kn, vn, qn = host_pool[i % len(host_pool)]
        cache.decode_step(kn, vn, qn, out_host, order, mem=xq.XQ_MEM_HOST)
        stream.synchronize()  # the host reads the step's result
    e1.record()
    barrier()
    ms3 = e0.elapsed_time(e1)
    ms3_max = sharding.max_over_ranks(ms3, dev)
    e2e_val = sharding.aggregate_rate(step_bytes(seq_before3 + 1, K), ms3_max, world) / 1e9

    clocks = sampler.stop(t_lo, t_hi) if sampler else None

    # ---- chunk attention: the last CHUNK_T tokens of a layer as queries, causal inside the chunk (a prefill
    # ---- chunk / Appendix D's prompt workload), on the first layers of the model
    CHUNK_T, chunk_layers = 16, min(L, 4)
    qc = torch.randn(CHUNK_T, B, Hq, D, generator=g, device=dev).to(torch.bfloat16)
    oc = torch.empty_like(qc)
    for l in range(chunk_layers):
        cache.attention_chunk(l, qc, oc)
    barrier()
    e0.record()
    for l in range(chunk_layers):
        cache.attention_chunk(l, qc, oc)
    e1.record()
    barrier()
    ms_chunk = sharding.max_over_ranks(e0.elapsed_time(e1), dev)
    S_now = cache.seq_len(0)
    chunk = {"n_q_tokens": CHUNK_T, "layers": chunk_layers, "context": S_now,
             "us_per_query_token_and_layer": ms_chunk * 1e3 / (CHUNK_T * chunk_layers),
             "attended_tokens_per_s": world * B * CHUNK_T * chunk_layers * (S_now - (CHUNK_T - 1) / 2.0) / (ms_chunk * 1e-3),
             "how": "one decode launch per query token with its visibility limit"}
    rc, nsq, nsw = xq.xq_split_plan(cache.handle, 0)  # the decode launches' split plan (before the appends below)

    # ---- pass 4: the quantize-and-pack path: every layer receives whole window blocks (R tokens per call), so each
    # ---- call quantizes and packs the block that filled the window (code-owning layers: codes + scale / zero-point;
    # ---- borrowing layers: scale / zero-point only)
    gk = torch.Generator(device=dev).manual_seed(99 + rank)
    blk = [torch.randn(B, Hkv, R, D, generator=gk, device=dev).to(torch.bfloat16) for _ in range(4)]
    fill = R - (cache.seq_len(0) % R)  # top the window up so that the next R tokens flush exactly one block
    for l in range(L):
        cache.append_kv(l, blk[0][:, :, :fill].contiguous(), blk[1][:, :, :fill].contiguous())
    xq.xq_timing_enable(cache.handle, 1)
    barrier()
    for i in range(APPEND_BLOCKS):
        for l in range(L):
            cache.append_kv(l, blk[(i + l) % 4], blk[(i + l + 1) % 4])
    barrier()
    _, n_pack, ms_pack = xq.xq_timing_read(cache.handle, 2)
    _, n_wapp, ms_wapp = xq.xq_timing_read(cache.handle, 3)
    xq.xq_timing_enable(cache.handle, 0)
    block_in_bytes = 2 * B * Hkv * R * D * 2  # 16-bit K and V of one block
    # the same path at prefill size: BULK_BLOCKS window blocks per call (one pack launch each)
    bulk = [torch.randn(B, Hkv, BULK_BLOCKS * R, D, generator=gk, device=dev).to(torch.bfloat16) for _ in range(3)]
    xq.xq_timing_enable(cache.handle, 1)
    barrier()
    for i in range(2):
        for l in range(L):
            cache.append_kv(l, bulk[(i + l) % 3], bulk[(i + l + 1) % 3])
    barrier()
    _, n_bulk, ms_bulk = xq.xq_timing_read(cache.handle, 2)
    xq.xq_timing_enable(cache.handle, 0)
    del bulk
    append = {"block_tokens": R, "blocks_per_layer": APPEND_BLOCKS, "pack_launches": n_pack,
              "pack_avg_us": ms_pack / n_pack * 1e3 if n_pack else None,
              "pack_input_gbs": block_in_bytes / (ms_pack / n_pack * 1e-3) / 1e9 if n_pack else None,
              "pack_frac_of_measured_hbm": (block_in_bytes / (ms_pack / n_pack * 1e-3) / 1e9 / peak) if n_pack else None,
              "window_append_avg_us": ms_wapp / n_wapp * 1e3 if n_wapp else None,
              "input_bytes_per_block": block_in_bytes,
              "bulk": {"blocks_per_call": BULK_BLOCKS, "pack_launches": n_bulk,
                       "pack_avg_us": ms_bulk / n_bulk * 1e3 if n_bulk else None,
                       "pack_input_gbs": BULK_BLOCKS * block_in_bytes / (ms_bulk / n_bulk * 1e-3) / 1e9 if n_bulk else None,
                       "pack_frac_of_measured_hbm": (BULK_BLOCKS * block_in_bytes / (ms_bulk / n_bulk * 1e-3) / 1e9 / peak)
                       if n_bulk else None}}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": Wm,
            "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8 x u8 -> s32 tensor-core products (24-bit fixed-point operands), f32 softmax, bf16 io",
            "data": "synthetic",
            "config": _config_block(args, w),
            "run": {"equiv_bits": xq.xq_equiv_bits(cfg), "layer_order": args.layer_order,
                    "bytes_streamed_per_step_gb": bytes_pass1 / K / 1e9,
                    "splits_quantized": nsq, "splits_window": nsw,
                    "algorithmic_bytes_per_layer_call": W.algorithmic_bytes(w, S, 0)},
            "frac_of_8TBps": value / world / 8000.0,
            "frac_of_measured_hbm": value / world / peak,
            "attended_tokens_per_s": tokens_per_s,
            "gpu_launches": int(launches),
            "clocks": clocks,
            "e2e": {"value": e2e_val, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms3_max / K},
            "roofline": {"bound": "hbm", "kernel": "decode split kernel", "achieved": achieved, "peak": peak,
                         "peak_source": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_8TBps": achieved / 8000.0,
                         "traffic": _ncu_traffic(args.config) if not (args.layers or args.seq or args.splits) else None,
                         "algorithmic_bytes_per_launch": bytes_pass1 / decode_launches_pass1,
                         "avg_launch_us": avg_launch_us, "launches": decode_launches_pass1,
                         "timing": "CUDA events around the timed region of back-to-back launches, divided by the decode launches in it",
                         "isolated": {"avg_launch_us": dec["avg_us"], "achieved": isolated, "frac": isolated / peak,
                                      "launches": dec["launches"],
                                      "timing": "CUDA events around every launch (no overlap of a launch's prologue with its predecessor's tail)"}},
            "chunk": chunk,
            "kernels": kinds,
            "flush_step": {"what": "the step on which every layer's window block fills: one quantize-and-pack launch for "
                                   "all layers before that step's decode launches",
                           "pack_launches": kinds["quantize_pack"]["launches"],
                           "pack_avg_us": kinds["quantize_pack"]["avg_us"],
                           "avg_step_ms_of_the_timed_region": ms_max / K},
            "append": append,
        }
        if not args.no_cpu_baseline and world == 1:
            n_streams = min(B * Hkv, 32)
            smp = OracleSample(w, n_streams, args.eta1, args.eta2)
            dt, passes = 0.0, 0
            while dt < 12.0 and passes < 16:  # about 10-30 s of CPU work
                dt += smp.run()
                passes += 1
            all_val, all_n = oracle_all_cores(w, args.eta1, args.eta2)
            line["cpu_baseline"] = {
                "value": passes * smp.bytes / dt / 1e9, "unit": "GB/s", "cores": smp.cores, "kind": "oracle",
                "host_cores": os.cpu_count(),
                "sample": f"decode attention of one layer for {n_streams} of {B * Hkv} (sequence, kv head) streams at S={S} "
                          f"(dequantize + attention, fp64 numpy), {passes} passes, {dt:.1f} s",
                "all_cores": {"value": all_val, "unit": "GB/s", "cores": all_n,
                              "sample": f"{all_n} single-threaded processes, one stream each at S={S}, ~6 s of passes each"}}
        print(json.dumps(line), flush=True)
    cache.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

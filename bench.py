#!/usr/bin/env python
"""Throughput of the CurDKV prefill-time selection path on B200.

One step = the whole hot path (score -> select -> compact) over one synthetic KV
cache.  Prints ONE JSON line (rank 0).  ``--impl reference`` times the fp64 CPU
oracle on a bounded sample of the same workload instead.
"""
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

import numpy as np
import torch

from paper_2509_15038_b200 import synth

METRIC = "kv_head_tokens_compressed_per_s"
UNIT = "head-tokens/s"
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 << 20
# dram__bytes_read.sum + dram__bytes_write.sum of one sketch-kernel launch, from the ncu
# capture summarised under profiles/ (None: not captured for the kernel as it stands)
TRAFFIC_BYTES = {"cfg2": 1.0787e9, "cfg3": 16 * 1.0787e9}   # cfg3 = cfg2's capture x 16 head-tokens
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def workload_bytes(w, seqlens):
    """Algorithmic bytes of one step: K+V read once + compacted rows written."""
    P = w.folded_batch * w.kv_heads
    if seqlens is None:
        tokens = P * w.n_max
        kept = P * min(w.budget, w.n_max)
    else:
        tokens = int(seqlens.astype(np.int64).sum()) * w.kv_heads
        kept = int(np.minimum(seqlens, w.budget).astype(np.int64).sum()) * w.kv_heads
    row_pair = 2 * w.d * 2
    return tokens, tokens * row_pair, kept * row_pair


# --------------------------------------------------------------------------- multi-rank helpers

def rank_workload(w, rank):
    """Weak scaling: every rank holds one full copy of the workload with its own data seed.
    The problems are independent, so no rank ever needs another rank's data."""
    return synth.shrink(w, data_seed=w.data_seed + 100 * rank)


def max_over_ranks(x, device, world):
    """The slowest rank's time: what the whole job waits for."""
    if world == 1:
        return float(x)
    import torch.distributed as dist

    t = torch.tensor([x], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank, world, seconds):
    """Whole-job rate: the units all ranks processed over the slowest rank's time."""
    return world * units_per_rank / seconds


# --------------------------------------------------------------------------- CUDA arm

def run_cuda(args):
    from paper_2509_15038_b200 import binding as cur

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    w = rank_workload(synth.CONFIGS[args.workload], rank)
    if args.batch > 0:                                     # the same recipe at another batch size
        w = synth.shrink(w, batch=args.batch)
    if args.layers > 0:                                    # ... or with fewer layers (small profiling cases)
        w = synth.shrink(w, layers=args.layers)
    K, V, seqlens = synth.make_kv(w, dev)
    G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=dev)
    sl = None if seqlens is None else torch.as_tensor(seqlens, device=dev)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads, seqlens=sl, whiten=int(args.whiten),
                         ridge=1e-4 if args.whiten else 0.0)
    ws = cur.alloc_workspace(desc, w.budget, w.adaptive)
    P = w.folded_batch * w.kv_heads
    scores = torch.empty((w.folded_batch, w.kv_heads, w.n_max), dtype=torch.float32, device=dev)
    sums = torch.empty((w.folded_batch, w.kv_heads), dtype=torch.float32, device=dev)
    cap = min(w.budget, w.n_max)
    if w.adaptive:
        idx = torch.empty((P * cap,), dtype=torch.int32, device=dev)
        Ko = torch.empty((P * cap, w.d), dtype=torch.bfloat16, device=dev)
    else:
        idx = torch.empty((w.folded_batch, w.kv_heads, w.budget), dtype=torch.int32, device=dev)
        Ko = torch.empty((w.folded_batch, w.kv_heads, w.budget, w.d), dtype=torch.bfloat16, device=dev)
    Vo = torch.empty_like(Ko)
    cnt = torch.empty((w.folded_batch, w.kv_heads), dtype=torch.int32, device=dev)
    off = torch.empty((P + 1,), dtype=torch.int32, device=dev)

    def step(events=None, sketch_events=None):
        if events is not None:
            events[0].record()
        if sketch_events is not None:
            cur.curdkv_profile_next_score(*sketch_events)
        if not args.three_calls:
            # the whole path in one call; for fixed budgets its first kernel scores AND selects
            cur.curdkv_compress(K, V, G, desc, w.budget, ws, num_sink=w.num_sink, window=w.window,
                                adaptive=w.adaptive, alpha=w.alpha, scores=scores, head_sums=sums, idx=idx,
                                head_counts=cnt, head_offsets=off, K_out=Ko, V_out=Vo)
            if events is not None:
                for e in events[1:]:
                    e.record()
            return
        cur.curdkv_score(K, V, G, desc, ws, scores=scores, head_sums=sums)
        if events is not None:
            events[1].record()
        cur.curdkv_select(scores, desc, w.budget, num_sink=w.num_sink, window=w.window,
                          adaptive=w.adaptive, alpha=w.alpha, workspace=ws, idx=idx,
                          head_counts=cnt, head_offsets=off)
        if events is not None:
            events[2].record()
        cur.curdkv_compact(K, V, desc, idx, cnt, off, packed=w.adaptive, K_out=Ko, V_out=Vo,
                           workspace=ws)
        if events is not None:
            events[3].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    flags = cur.curdkv_device_status(ws)
    if flags:
        raise RuntimeError(f"device status flags {flags:#x} after warm-up")

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    launches0 = cur.launch_count()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    # events the library records right around its sketch kernel (the dominant kernel); their
    # handles only exist once they have been recorded
    sk = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
    for pair in sk:
        for e in pair:
            e.record()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    # inputs that fit in the 126 MB L2 are evicted between steps by writing a larger buffer; the
    # flushes then sit between the per-step event pairs and are not timed
    small = 2 * K.numel() * K.element_size() < 2 * L2_BYTES
    flush = torch.empty((2 * L2_BYTES,), dtype=torch.uint8, device=dev) if small else None
    barrier()
    t0.record()
    for i in range(args.steps):
        if flush is not None:
            flush.zero_()
        step(ev[i], sk[i])
    t1.record()
    barrier()
    launches = cur.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if small:
        ms_step = max_over_ranks(sum(e[0].elapsed_time(e[3]) for e in ev), dev, world) / args.steps
    else:
        ms_step = max_over_ranks(t0.elapsed_time(t1), dev, world) / args.steps
    stage_ms = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in ev]).mean(0)
    per_step = np.array([e[0].elapsed_time(e[3]) for e in ev])      # this rank's steps, one by one

    tokens, read_bytes, write_bytes = workload_bytes(w, seqlens)
    pass_bytes = read_bytes                  # K + V once: what one streaming kernel reads
    if args.whiten:
        read_bytes *= 2                      # Gram pass + sketch pass
    value = job_throughput(tokens, world, ms_step * 1e-3)
    gbs = job_throughput(read_bytes + write_bytes, world, ms_step * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    sketch_ms = float(np.mean([a.elapsed_time(b) for a, b in sk]))
    sketch_gbs = pass_bytes / (sketch_ms * 1e-3) / 1e9

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": f"{w.name}: {w.layers} layers x batch {w.batch} x {w.kv_heads} KV heads "
                        f"(GQA {w.q_heads}:{w.kv_heads}), n={w.n_max}, d={w.d}, r={w.r}, "
                        f"budget {w.budget} incl. window {w.window}, sinks {w.num_sink}, "
                        + ("AdaCurDKV alpha=%.2f" % w.alpha if w.adaptive else "fixed per-head budget")
                        + (", whitened sketch (leverage scores, ridge 1e-4)" if args.whiten else "")
                        + (f", ragged lengths {w.ragged}" if w.ragged else ""),
            "head_tokens_per_step": tokens, "seq_tokens_per_step": tokens // (w.layers * w.kv_heads),
            "l2": ("inputs (%.3f GB) fit in the 126 MB L2: a 252 MB buffer is written between steps "
                   "(outside the timed event pairs)" % (read_bytes / 1e9)) if small else
                  ("inputs (%.1f GB) exceed the 126 MB L2, no flush between steps" % (read_bytes / 1e9)),
            "sharding": "independent replicas per rank, no collective",
        },
        "gb_per_s": gbs, "counted_bytes_per_step": read_bytes + write_bytes,
        "pct_of_nominal_8000": 100 * gbs / world / NOMINAL_HBM_GBS,
        "pct_of_measured_copy": 100 * gbs / world / peak,
        "seq_tokens_per_s": value / (w.layers * w.kv_heads),
        "stage_ms": {"score": float(stage_ms[0]), "select": float(stage_ms[1]),
                     "compact": float(stage_ms[2])},
        "ms_per_step_median": float(np.median(per_step)), "ms_per_step_best": float(per_step.min()),
        "clocks": clocks,
        "gpu_launches": int(launches),
        "roofline": {
            "bound": "hbm",
            "kernel": ("sketch_items_kernel" if args.whiten else "sketch_umma_kernel") + " (inside curdkv_score)",
            "achieved": sketch_gbs, "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
            "unit": "GB/s", "frac": sketch_gbs / peak,
            "traffic": None if (args.whiten or args.batch > 0 or args.layers > 0) else TRAFFIC_BYTES.get(w.name),
            "algorithmic_bytes_per_launch": pass_bytes, "ms_per_launch": sketch_ms,
            "timer": "CUDA events recorded by the library around the kernel, mean over the timed steps",
        },
    }
    if args.graph and world == 1:
        # the same step captured once into a CUDA graph and replayed: what a caller that runs the
        # three calls back to back saves in launch overhead (only visible on small workloads)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        gev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for i in range(args.steps):
            if flush is not None:
                flush.zero_()
            gev[i][0].record()
            graph.replay()
            gev[i][1].record()
        torch.cuda.synchronize()
        out["cuda_graph"] = {"ms_per_step": float(np.mean([a_.elapsed_time(b_) for a_, b_ in gev])),
                             "eager_ms_per_step": ms_step}
    out["e2e"] = run_e2e(cur, w, K, V, seqlens, value_tokens=tokens, world=world, dev=dev,
                         steps=min(args.steps, args.e2e_steps))
    if rank == 0:
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"] = cpu_baseline(w, core_seconds=20.0)
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(cur, w, K, V, seqlens, value_tokens, world, dev, steps):
    """Same metric through curdkv_compress_host: K, V start in pinned host memory, results end
    in pinned host memory; every step pays the host->device and device->host copies."""
    import ctypes

    if steps <= 0:
        return None
    Kh = torch.empty(K.shape, dtype=K.dtype, pin_memory=True)
    Vh = torch.empty(V.shape, dtype=V.dtype, pin_memory=True)
    Kh.copy_(K)
    Vh.copy_(V)
    Gh = torch.as_tensor(synth.make_G(w.d, w.r, seed=0))
    sl_host = None if seqlens is None else np.ascontiguousarray(seqlens, dtype=np.int32)
    desc = cur.make_desc(Kh, Vh, w.r, q_heads=w.q_heads)
    if sl_host is not None:
        desc.seqlens = sl_host.ctypes.data
    elem_bytes = 2 * w.kv_heads * w.n_max * w.d * 2
    chunk_batch = int(max(1, min(w.folded_batch, (512 << 20) // elem_bytes)))
    bufs = cur.HostBuffers(desc, w.budget, w.adaptive, chunk_batch, device=dev)

    def once():
        flags = cur.curdkv_compress_host(Kh, Vh, Gh, desc, w.budget, bufs, num_sink=w.num_sink,
                                         window=w.window, adaptive=w.adaptive, alpha=w.alpha)
        if flags:
            raise RuntimeError(f"device status flags {flags:#x} in the end-to-end run")

    once()
    torch.cuda.synchronize()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        once()
    torch.cuda.synchronize()
    dt = max_over_ranks((time.perf_counter() - t0) / steps, dev, world)
    h2d = Kh.numel() * 2 + Vh.numel() * 2 + (0 if sl_host is None else sl_host.nbytes)
    d2h = (bufs.idx.numel() * 4 + bufs.counts.numel() * 4 + bufs.K_out.numel() * 2
           + bufs.V_out.numel() * 2 + (bufs.offsets.numel() * 4 if w.adaptive else 0))
    return {"value": job_throughput(value_tokens, world, dt), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": dt * 1e3, "steps": steps,
            "api": "curdkv_compress_host (pinned host K, V in; pinned host idx, K', V' out)",
            "chunk_batch": chunk_batch, "timer": "host wall clock around the synchronous calls",
            "host_link_gb_per_s": (h2d + d2h) / dt / 1e9}


# --------------------------------------------------------------------------- generation phase

DECODE = dict(layers=32, batch=16, kv_heads=8, d=128, r=32, budget=2048, num_sink=4, window=64, chunk=256)


def run_decode(args):
    """Generation-phase workload (Sec. 3.2): every step appends `chunk` new rows per head to a cache
    that holds `budget` rows and compresses it back to `budget` (Alg. 1 lines 2-10 on the cache)."""
    from paper_2509_15038_b200 import binding as cur

    c = DECODE
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    LB, H, d, t, k = c["layers"] * c["batch"], c["kv_heads"], c["d"], c["chunk"], c["budget"]
    cap = k + t
    w = synth.shrink(synth.CONFIGS["cfg2"], layers=c["layers"], batch=c["batch"], n_max=t, data_seed=6)
    K_new, V_new, _ = synth.make_kv(w, dev)
    w0 = synth.shrink(w, n_max=cap, data_seed=7)
    K0, V0, _ = synth.make_kv(w0, dev)
    G = torch.as_tensor(synth.make_G(d, c["r"], seed=0), device=dev)
    caches = [cur.DeviceCache(LB, H, cap, d, dev), cur.DeviceCache(LB, H, cap, d, dev)]
    ws = cur.cache_workspace(LB, H, cap, cap, k, dev)
    cur.curdkv_cache_append(caches[0], K0, V0, G, ws)              # fill to capacity, then to budget
    cur.curdkv_cache_compress(caches[0], caches[1], k, ws, num_sink=c["num_sink"], window=c["window"])
    live = 1

    inplace = args.decode_mode == "inplace"

    def step():
        nonlocal live
        cur.curdkv_cache_append(caches[live], K_new, V_new, G, ws)
        if inplace:       # survivors stay put, at most `chunk` rows per head move into the holes
            cur.curdkv_cache_compress_inplace(caches[live], k, ws, num_sink=c["num_sink"], window=c["window"])
        else:             # ordered copy of all survivors into the other cache
            cur.curdkv_cache_compress(caches[live], caches[1 - live], k, ws, num_sink=c["num_sink"],
                                      window=c["window"])
            live = 1 - live

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if cur.curdkv_device_status(ws):
        raise RuntimeError("device status flags set after warm-up")
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.3)
    launches0 = cur.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    launches = cur.launch_count() - launches0
    clocks = sampler.stop()
    assert int(caches[live].count.min()) == k and int(caches[live].count.max()) == k
    ms = t0.elapsed_time(t1) / args.steps
    P = LB * H
    rows = P * (k + t)                       # rows the compression looks at per step
    # new rows read and stored, their scores; held scores read; then either every survivor read and
    # written (ordered) or at most `chunk` moved rows per head read and written (in place)
    counted = P * (t * 512 * 2 + (k + t) * 4 + (t if inplace else k) * 512 * 2)
    peak, peak_kind = measured_peak()
    gbs = counted / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": rows / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "decode: %(layers)d layers x batch %(batch)d x %(kv_heads)d KV heads, cache "
                               "budget %(budget)d (sinks %(num_sink)d, window %(window)d), %(chunk)d new rows "
                               "per head and step, r=%(r)d" % c
                               + (", in-place compression" if inplace else ", ordered compression into a second cache"),
                   "head_tokens_per_step": rows,
                   "l2": "caches (%.1f GB) exceed the 126 MB L2" % (2 * 2 * P * cap * d * 2 / 1e9)},
        "gb_per_s": gbs, "counted_bytes_per_step": counted,
        "clocks": clocks, "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "whole step (append + select + gather)", "achieved": gbs,
                     "peak": peak, "peak_kind": peak_kind + " copy bandwidth", "unit": "GB/s",
                     "frac": gbs / peak, "traffic": None},
    }), flush=True)


# --------------------------------------------------------------------------- eviction loss

EVICT = dict(workload="cfg2", q_rows=512)


def run_evict(args):
    """Eviction-loss workload (Lemma 1): attention output of the full and of the compressed cache
    for synthetic queries, and the relative loss of CurDKV against key-only, value-only and random
    selections of the same size.  One step = attention over the full cache + over the CurDKV cache +
    the Frobenius difference."""
    from paper_2509_15038_b200 import binding as cur

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    w = synth.CONFIGS[EVICT["workload"]]
    m = EVICT["q_rows"]
    K, V, _ = synth.make_kv(w, dev)
    LB, H, n, d = K.shape
    g = torch.Generator(device=dev).manual_seed(99)
    # queries that look like keys of the same head (same outlier channels), so that logits are not flat
    Q = (K[:, :, torch.randint(0, n, (m,), generator=g, device=dev)].float()
         + torch.randn((LB, H, m, d), generator=g, device=dev)).to(torch.bfloat16)
    scale = 1.0 / float(np.sqrt(d))
    G = torch.as_tensor(synth.make_G(d, w.r, seed=0), device=dev)
    desc = cur.make_desc(K, V, w.r, q_heads=w.q_heads)
    ws = cur.alloc_workspace(desc, w.budget)

    def select(score_mode=0, use_projection=1, random=False):
        dsc = cur.make_desc(K, V, w.r, q_heads=w.q_heads, score_mode=score_mode, use_projection=use_projection)
        scores, _ = cur.curdkv_score(K, V, G, dsc, ws)
        if random:
            scores = torch.rand(scores.shape, generator=g, device=dev)
        idx, cnt, off = cur.curdkv_select(scores, dsc, w.budget, num_sink=w.num_sink, window=w.window, workspace=ws)
        Kc, Vc = cur.curdkv_compact(K, V, dsc, idx, cnt, off, workspace=ws)
        return Kc, Vc, cnt.reshape(-1).contiguous()

    O = torch.empty((LB, H, m, d), dtype=torch.float32, device=dev)
    Oc = torch.empty_like(O)
    Kc, Vc, rows = select()
    cdesc = cur.make_desc(Kc, Vc, w.r)
    aws = torch.empty((1 << 20,), dtype=torch.uint8, device=dev)

    def step():
        cur.curdkv_attention_out(Q, K, V, desc, scale=scale, O=O, workspace=aws)
        cur.curdkv_attention_out(Q, Kc, Vc, cdesc, scale=scale, head_rows=rows, O=Oc, workspace=aws)
        return cur.curdkv_eviction_loss(O, Oc)

    for _ in range(max(args.warmup, 3)):
        loss, ref = step()
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    time.sleep(0.3)
    launches0 = cur.launch_count()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        loss, ref = step()
    t1.record()
    torch.cuda.synchronize()
    launches = cur.launch_count() - launches0
    clocks = sampler.stop()
    ms = t0.elapsed_time(t1) / args.steps
    rel = {"curdkv": float((loss / ref).mean())}
    for name, kw in (("key_only", dict(score_mode=1)), ("value_only", dict(score_mode=2)),
                     ("key_norm", dict(score_mode=1, use_projection=0)), ("random", dict(random=True))):
        Kx, Vx, rx = select(**kw)
        cur.curdkv_attention_out(Q, Kx, Vx, cur.make_desc(Kx, Vx, w.r), scale=scale, head_rows=rx, O=Oc,
                                 workspace=aws)
        lx, _ = cur.curdkv_eviction_loss(O, Oc)
        rel[name] = float((lx / ref).mean())
    P = LB * H
    kept = int(rows.sum())
    flops = 4.0 * m * d * (P * n + kept)                 # one Q K^T and one P V per cache
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, peak_kind = float(json.load(f)["bf16_tflops_sustained"]), "measured sustained bf16 cuBLAS"
    except Exception:
        peak, peak_kind = 1400.0, "fallback sustained bf16"
    tf = flops / (ms * 1e-3) / 1e12
    print(json.dumps({
        "metric": "attention_query_key_pairs_per_s", "value": m * (P * n + kept) / (ms * 1e-3),
        "unit": "query-key pairs/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"evict: {w.name} cache ({w.layers} layers x {w.kv_heads} KV heads, n={n}, "
                               f"budget {w.budget}), {m} synthetic query rows per KV head, scale 1/sqrt(d)"},
        "relative_eviction_loss": rel, "clocks": clocks, "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "attention_umma_kernel (full + compressed cache)",
                     "achieved": tf, "peak": peak, "peak_kind": peak_kind, "unit": "TFLOP/s",
                     "frac": tf / peak, "traffic": None,
                     "note": "algorithmic flops = one QK^T and one PV; the kernel issues 1.5x that "
                             "(PV for the hi and the lo half of the weights)"},
    }), flush=True)


# --------------------------------------------------------------------------- oracle arm

def oracle_sample(w, elements):
    """K, V bits of `elements` folded-batch elements of workload w, generated on the CPU."""
    Ks, Vs = [], []
    for lb in range(elements):
        k, v = synth.make_kv_element(w, lb, "cpu")
        Ks.append(synth.to_u16(k))
        Vs.append(synth.to_u16(v))
    seqlens = synth.make_seqlens(w)
    sl = None if seqlens is None else seqlens[:elements].copy()
    return np.stack(Ks), np.stack(Vs), sl


def oracle_step(w, Ku, Vu, sl, G):
    from oracle import curdkv_oracle as orc

    sc, _ = orc.score(Ku, Vu, G, seqlens=sl)
    if w.adaptive:
        idx, cnt, off = orc.select_adaptive(sc, w.budget, w.num_sink, w.window, w.alpha, seqlens=sl)
        orc.compact(Ku, Vu, idx, cnt, off)
    else:
        idx, cnt = orc.select_fixed(sc, w.budget, w.num_sink, w.window, seqlens=sl)
        orc.compact(Ku, Vu, idx, cnt)


def sample_elements(w, core_seconds):
    """Folded-batch elements whose oracle run costs about `core_seconds` of CPU work
    (the naive fp64 loops manage roughly 7e8 multiply-adds per core-second)."""
    macs_per_elem = 2.0 * w.kv_heads * w.n_max * w.d * w.r
    return int(min(max(1, round(core_seconds * 7e8 / macs_per_elem)), w.folded_batch))


def cpu_baseline(w, core_seconds=20.0):
    from oracle import curdkv_oracle as orc

    elems = sample_elements(w, core_seconds)
    Ku, Vu, sl = oracle_sample(w, elems)
    G = synth.make_G(w.d, w.r, seed=0)
    t0 = time.perf_counter()
    oracle_step(w, Ku, Vu, sl, G)
    dt = time.perf_counter() - t0
    tokens = (elems * w.n_max if sl is None else int(sl.sum())) * w.kv_heads
    return {"value": tokens / dt, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"{elems} of {w.folded_batch} (layer, sequence) groups of {w.name} "
                      f"({elems * w.kv_heads} problems, {tokens} head-tokens), {dt:.2f} s wall",
            "seconds": dt}


def run_reference(args):
    from oracle import curdkv_oracle as orc

    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = synth.CONFIGS[args.workload]
    if args.batch > 0:
        w = synth.shrink(w, batch=args.batch)
    if args.layers > 0:
        w = synth.shrink(w, layers=args.layers)
    elems = sample_elements(w, core_seconds=20.0)
    Ku, Vu, sl = oracle_sample(w, elems)
    G = synth.make_G(w.d, w.r, seed=0)
    for _ in range(args.warmup):
        oracle_step(w, Ku, Vu, sl, G)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(w, Ku, Vu, sl, G)
    dt = (time.perf_counter() - t0) / args.steps
    tokens = (elems * w.n_max if sl is None else int(sl.sum())) * w.kv_heads
    value = tokens / dt
    sample = (f"each step = {elems} of {w.folded_batch} (layer, sequence) groups of {w.name} "
              f"({tokens} head-tokens)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name + " (bounded sample)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--workload", default="cfg3", choices=sorted(synth.CONFIGS) + ["decode", "evict"])
    ap.add_argument("--batch", type=int, default=0,
                    help="sequences per layer instead of the workload's own (cfg1-cfg5 only); 0 keeps it")
    ap.add_argument("--layers", type=int, default=0,
                    help="layers instead of the workload's own (cfg1-cfg5 only); 0 keeps them")
    ap.add_argument("--graph", action="store_true",
                    help="also time the step replayed from a CUDA graph (extra 'cuda_graph' object)")
    ap.add_argument("--three-calls", action="store_true",
                    help="time curdkv_score + curdkv_select + curdkv_compact instead of curdkv_compress")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode-mode", choices=["inplace", "ordered"], default="inplace",
                    help="--workload decode: compress inside the cache (unordered) or copy in order")
    ap.add_argument("--whiten", action="store_true",
                    help="score with the whitened sketch (approximate leverage scores; reads K, V twice)")
    ap.add_argument("--e2e-steps", type=int, default=3,
                    help="steps of the host-buffer end-to-end leg (0 disables it)")
    args = ap.parse_args()
    if args.workload in ("decode", "evict"):
        if args.impl == "reference":
            raise SystemExit("the reference arm times the prefill workloads only")
        run_decode(args) if args.workload == "decode" else run_evict(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

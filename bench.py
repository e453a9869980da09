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

class Case:
    """One workload resident in HBM with its output buffers; ``step()`` runs the whole hot path once."""

    def __init__(self, cur, w, dev, whiten=False, three_calls=False, kv=None):
        self.cur, self.w, self.dev, self.whiten, self.three_calls = cur, w, dev, whiten, three_calls
        self.K, self.V, self.seqlens = kv if kv is not None else synth.make_kv(w, dev)
        self.G = torch.as_tensor(synth.make_G(w.d, w.r, seed=0), device=dev)
        self.sl = None if self.seqlens is None else torch.as_tensor(self.seqlens, device=dev)
        self.desc = cur.make_desc(self.K, self.V, w.r, q_heads=w.q_heads, seqlens=self.sl, whiten=int(whiten),
                                  ridge=1e-4 if whiten else 0.0)
        self.ws = cur.alloc_workspace(self.desc, max(w.budget, 1), w.adaptive)
        LB, H = w.folded_batch, w.kv_heads
        P, cap = LB * H, min(w.budget, w.n_max)
        self.scores = torch.empty((LB, H, w.n_max), dtype=torch.float32, device=dev)
        self.sums = torch.empty((LB, H), dtype=torch.float32, device=dev)
        if w.adaptive:
            self.idx = torch.empty((P * cap,), dtype=torch.int32, device=dev)
            self.Ko = torch.empty((P * cap, w.d), dtype=torch.bfloat16, device=dev)
        else:
            self.idx = torch.empty((LB, H, w.budget), dtype=torch.int32, device=dev)
            self.Ko = torch.empty((LB, H, w.budget, w.d), dtype=torch.bfloat16, device=dev)
        self.Vo = torch.empty_like(self.Ko)
        self.cnt = torch.empty((LB, H), dtype=torch.int32, device=dev)
        self.off = torch.empty((P + 1,), dtype=torch.int32, device=dev)
        # inputs that fit in the 126 MB L2 are evicted between steps by writing a larger buffer
        self.small = 2 * self.K.numel() * self.K.element_size() < 2 * L2_BYTES
        self.flush = torch.empty((2 * L2_BYTES,), dtype=torch.uint8, device=dev) if self.small else None

    def step(self, events=None, kernel_events=None):
        cur, w = self.cur, self.w
        if events is not None:
            events[0].record()
        if kernel_events is not None:
            cur.curdkv_profile_next_score(*kernel_events)
        if not self.three_calls:
            # the whole path in one call; for fixed budgets its first kernel scores AND selects
            cur.curdkv_compress(self.K, self.V, self.G, self.desc, w.budget, self.ws, num_sink=w.num_sink,
                                window=w.window, adaptive=w.adaptive, alpha=w.alpha, scores=self.scores,
                                head_sums=self.sums, idx=self.idx, head_counts=self.cnt,
                                head_offsets=self.off, K_out=self.Ko, V_out=self.Vo)
        else:
            cur.curdkv_score(self.K, self.V, self.G, self.desc, self.ws, scores=self.scores, head_sums=self.sums)
            if events is not None:
                events[1].record()
            cur.curdkv_select(self.scores, self.desc, w.budget, num_sink=w.num_sink, window=w.window,
                              adaptive=w.adaptive, alpha=w.alpha, workspace=self.ws, idx=self.idx,
                              head_counts=self.cnt, head_offsets=self.off)
            if events is not None:
                events[2].record()
            cur.curdkv_compact(self.K, self.V, self.desc, self.idx, self.cnt, self.off, packed=w.adaptive,
                               K_out=self.Ko, V_out=self.Vo, workspace=self.ws)
        if events is not None:
            events[3].record()

    def timed(self, steps, warmup, barrier=None, flush=True):
        """CUDA-event timing of `steps` steps after `warmup`; returns a dict of per-step figures."""
        cur = self.cur
        sync = barrier or torch.cuda.synchronize
        for _ in range(max(warmup, 3)):
            self.step()
        sync()
        flags = cur.curdkv_device_status(self.ws)
        if flags:
            raise RuntimeError(f"device status flags {flags:#x} after warm-up ({self.w.name})")
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        # events the library records right around its streaming kernel (the dominant kernel); their
        # handles only exist once they have been recorded.  Every fourth step only: an event between
        # the streaming kernel and the gather keeps the gather from starting while the last heads are
        # still being selected, so a step that is sampled this way runs ~1 % longer.
        kv = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] if i % 4 == 0 else None
              for i in range(steps)]
        kv_used = [pair for pair in kv if pair is not None]
        for pair in kv_used:
            for e in pair:
                e.record()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        use_flush = self.flush is not None and flush
        sync()
        launches0 = cur.launch_count()
        t0.record()
        for i in range(steps):
            if use_flush:
                self.flush.zero_()                 # sits between the per-step event pairs: not timed
            self.step(ev[i], kv[i])
        t1.record()
        sync()
        per_step = np.array([e[0].elapsed_time(e[3]) for e in ev])
        out = {"ms_whole": t0.elapsed_time(t1) / steps, "ms_events": float(per_step.mean()),
               "per_step": per_step, "kernel_ms": float(np.mean([a.elapsed_time(b) for a, b in kv_used])),
               "kernel_samples": len(kv_used),
               "launches": cur.launch_count() - launches0, "flushed": use_flush}
        if self.three_calls:
            st = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in ev]).mean(0)
            out["stage_ms"] = {"score": float(st[0]), "select": float(st[1]), "compact": float(st[2])}
        else:
            out["stage_ms"] = {"score+select (streaming kernel, library events)": out["kernel_ms"],
                               "rest of the call (gather; for AdaCurDKV also the selection kernel)":
                                   float(per_step.mean()) - out["kernel_ms"]}
        return out

    def free(self):
        for name in ("K", "V", "scores", "idx", "Ko", "Vo", "flush", "ws"):
            setattr(self, name, None)
        torch.cuda.empty_cache()


def workload_text(w, whiten=False):
    return (f"{w.name}: {w.layers} layers x batch {w.batch} x {w.kv_heads} KV heads "
            f"(GQA {w.q_heads}:{w.kv_heads}), n={w.n_max}, d={w.d}, r={w.r}, "
            f"budget {w.budget} incl. window {w.window}, sinks {w.num_sink}, "
            + ("AdaCurDKV alpha=%.2f" % w.alpha if w.adaptive else "fixed per-head budget")
            + (", whitened sketch (leverage scores, ridge 1e-4)" if whiten else "")
            + (f", ragged lengths {w.ragged}" if w.ragged else ""))


def kernel_traffic(kernel, tokens):
    """DRAM bytes of one launch of `kernel`, from the ncu capture summarised under profiles/ (scaled by
    head-tokens: the kernel streams every row once, so its traffic grows in proportion), or None when
    no capture of the kernel as it stands is on file."""
    try:
        with open(os.path.join(ROOT, "profiles", "streaming_kernel_traffic.json")) as f:
            rec = json.load(f)["kernels"][kernel]
        return rec["dram_bytes_per_launch"] * tokens / rec["head_tokens_per_launch"], rec["capture"]
    except Exception:
        return None, None


def streaming_kernel_name(w, whiten, three_calls):
    sms = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    if whiten:
        return "sketch_items_kernel<%d>" % (32 if w.r <= 32 else 64)
    fused = (not three_calls and not w.adaptive and w.ragged is None and w.r <= 32 and w.n_max >= 128
             and w.folded_batch * w.kv_heads >= sms)
    return "sketch_umma_kernel<%d, %s>" % (32 if w.r <= 32 else 64, "true" if fused else "false")


def case_summary(case, t, world=1):
    """Throughput and roofline figures of one timed case."""
    w = case.w
    tokens, read_bytes, write_bytes = workload_bytes(w, case.seqlens)
    ms = t["ms_events"] if t["flushed"] else t["ms_whole"]
    gbs = (read_bytes + write_bytes) / (ms * 1e-3) / 1e9
    peak, _ = measured_peak()
    return {"ms_per_step": ms, "stage_ms": t["stage_ms"], "head_tokens_per_step": tokens,
            "head_tokens_per_s": tokens / (ms * 1e-3), "gb_per_s": gbs,
            "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS, "frac_of_measured_copy": gbs / peak,
            "streaming_kernel": streaming_kernel_name(w, case.whiten, case.three_calls),
            "streaming_kernel_ms": t["kernel_ms"],
            "streaming_kernel_gb_per_s": read_bytes / (t["kernel_ms"] * 1e-3) / 1e9,
            "gpu_launches_per_step": t["launches"] / len(t["per_step"]),
            "l2": "flushed between steps" if t["flushed"] else
                  ("inputs fit in L2, not flushed" if case.small else "inputs exceed L2")}


def oracle_check(case, lb):
    """Part of the cpu-baseline leg: the fp64 oracle on ONE (layer, sequence) group of the case (all its
    heads for AdaCurDKV, the first head otherwise), timed, and compared with what the GPU produced:
    scores within 1e-3 relative, selection equal outside the 1e-4 tie band of a cut, gathered rows
    byte-identical to the source rows at the GPU's indices."""
    from oracle import curdkv_oracle as orc

    w = case.w
    heads = range(w.kv_heads) if w.adaptive else range(1)
    n = w.n_max if case.seqlens is None else int(case.seqlens[lb])
    Ku = synth.to_u16(case.K[lb, list(heads)])[None]
    Vu = synth.to_u16(case.V[lb, list(heads)])[None]
    G = synth.make_G(w.d, w.r, seed=0)
    sl = None if case.seqlens is None else np.array([n], dtype=np.int32)
    t0 = time.perf_counter()
    rs, _ = orc.score(Ku, Vu, G, seqlens=sl)
    if w.adaptive:
        ridx, rcnt, roff = orc.select_adaptive(rs, w.budget, w.num_sink, w.window, w.alpha, seqlens=sl)
    else:
        ridx, rcnt = orc.select_fixed(rs, w.budget, w.num_sink, w.window, seqlens=sl)
    dt = time.perf_counter() - t0
    got = case.scores[lb, list(heads)].cpu().numpy().astype(np.float64)[None]
    tol = 1e-3 * np.abs(rs) + 1e-6 * np.abs(rs).max(-1, keepdims=True)
    ok = bool(np.all(np.abs(got - rs) <= tol))
    H = w.kv_heads
    off = case.off.cpu().numpy()
    cnt = case.cnt.cpu().numpy()
    gi = case.idx.cpu().numpy()
    cuts, pairs = [], []
    for j, h in enumerate(heads):
        if w.adaptive:
            g = gi[off[lb * H + h]: off[lb * H + h] + cnt[lb, h]]
            r = ridx[roff[j]: roff[j + 1]]
        else:
            g, r = gi[lb, h, : cnt[lb, h]], ridx[0, j, : rcnt[0, j]]
        forced_lo = n - min(w.window, n)
        cand = [t for t in r.tolist() if w.num_sink <= t < forced_lo]
        cuts.append(min(rs[0, j][t] for t in cand) if cand else np.inf)
        pairs.append((j, h, g, r))
        ok &= bool(np.all(np.diff(g) > 0)) and (len(g) == 0 or (g.min() >= 0 and g.max() < n))
        rows = torch.as_tensor(g.astype(np.int64), device=case.K.device)
        if w.adaptive:
            base = int(off[lb * H + h])
            ok &= bool(torch.equal(case.Ko[base: base + len(g)], case.K[lb, h][rows]))
            ok &= bool(torch.equal(case.Vo[base: base + len(g)], case.V[lb, h][rows]))
        else:
            ok &= bool(torch.equal(case.Ko[lb, h, : len(g)], case.K[lb, h][rows]))
            ok &= bool(torch.equal(case.Vo[lb, h, : len(g)], case.V[lb, h][rows]))
    ok &= sum(len(g) for _, _, g, _ in pairs) == sum(len(r) for _, _, _, r in pairs)
    lo_cut = min(cuts)
    for j, h, g, r in pairs:
        if not w.adaptive:
            ok &= len(g) == len(r)
        for t in set(g.tolist()) ^ set(r.tolist()):
            rel = min(abs(rs[0, j][t] / c - 1.0) for c in (lo_cut, cuts[j]) if np.isfinite(c) and c > 0)
            ok &= bool(rel < 1e-4)
    return {"parity": bool(ok), "group": int(lb), "heads_checked": len(list(heads)), "oracle_seconds": dt,
            "oracle_head_tokens_per_s": len(list(heads)) * n / dt}


ALL_CONFIGS = ("cfg1", "cfg2", "cfg3_b1", "cfg4", "cfg5")


def run_all_configs(cur, dev, steps, check):
    """The other benchmark configurations, a few steps each, one after the other (each cache is freed
    before the next is built): cfg1 with and without an L2-evicting write between steps, cfg2, the
    headline shape at batch 1, cfg4 (AdaCurDKV, r = 64, 128K tokens) and cfg5 at three budgets."""
    out = {}
    for name in ALL_CONFIGS:
        base = synth.CONFIGS[name]
        kv = synth.make_kv(base, dev)
        budgets = (128, 512, 2048) if name == "cfg5" else (base.budget,)
        for k in budgets:
            w = synth.shrink(base, budget=k)
            case = Case(cur, w, dev, kv=kv)
            key = name if len(budgets) == 1 else f"{name}_k{k}"
            t = case.timed(steps, 3)
            entry = case_summary(case, t)
            entry["workload"] = workload_text(w)
            if check:
                entry["oracle_check"] = oracle_check(case, w.folded_batch // 2)
            out[key if name != "cfg1" else "cfg1_l2_flushed"] = entry
            if name == "cfg1":                             # the same 4 MiB cache left in L2 between steps
                hot = case_summary(case, case.timed(steps, 3, flush=False))
                hot["workload"] = entry["workload"]
                out["cfg1_l2_resident"] = hot
            case.free()
        del kv
        torch.cuda.empty_cache()
    return out


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
    case = Case(cur, w, dev, whiten=args.whiten, three_calls=args.three_calls)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    for _ in range(max(args.warmup, 3)):
        case.step()
    barrier()
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    t = case.timed(args.steps, 0, barrier=barrier)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = max_over_ranks(t["ms_events"] if t["flushed"] else t["ms_whole"], dev, world)
    per_step = t["per_step"]

    tokens, read_bytes, write_bytes = workload_bytes(w, case.seqlens)
    pass_bytes = read_bytes                  # K + V once: what one streaming kernel reads
    value = job_throughput(tokens, world, ms_step * 1e-3)
    gbs = job_throughput(read_bytes + write_bytes, world, ms_step * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    kernel = streaming_kernel_name(w, args.whiten, args.three_calls)
    kernel_gbs = pass_bytes / (t["kernel_ms"] * 1e-3) / 1e9
    traffic, capture = kernel_traffic(kernel, tokens)

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": workload_text(w, args.whiten),
            "head_tokens_per_step": tokens, "seq_tokens_per_step": tokens // (w.layers * w.kv_heads),
            "api": ("curdkv_score + curdkv_select + curdkv_compact" if args.three_calls else "curdkv_compress"),
            "l2": ("inputs (%.3f GB) fit in the 126 MB L2: a 252 MB buffer is written between steps "
                   "(outside the timed event pairs)" % (read_bytes / 1e9)) if case.small else
                  ("inputs (%.1f GB) exceed the 126 MB L2, no flush between steps" % (read_bytes / 1e9)),
            "sharding": "independent replicas per rank, no collective",
        },
        "gb_per_s": gbs, "counted_bytes_per_step": read_bytes + write_bytes,
        "pct_of_nominal_8000": 100 * gbs / world / NOMINAL_HBM_GBS,
        "pct_of_measured_copy": 100 * gbs / world / peak,
        "seq_tokens_per_s": value / (w.layers * w.kv_heads),
        "stage_ms": t["stage_ms"],
        "ms_per_step_median": float(np.median(per_step)), "ms_per_step_best": float(per_step.min()),
        "clocks": clocks,
        "gpu_launches": int(t["launches"]),
        "roofline": {
            "bound": "hbm", "kernel": kernel + " (inside " + ("curdkv_score" if args.three_calls else "curdkv_compress") + ")",
            "achieved": kernel_gbs, "peak": peak,
            "peak_kind": peak_kind + " copy bandwidth (a read+write mix; this kernel only reads, "
                                     "which is why the fraction can exceed 1)",
            "unit": "GB/s", "frac": kernel_gbs / peak, "frac_of_nominal_8000": kernel_gbs / NOMINAL_HBM_GBS,
            "traffic": traffic, "traffic_source": capture,
            "algorithmic_bytes_per_launch": pass_bytes, "ms_per_launch": t["kernel_ms"],
            "timer": "CUDA events recorded by the library around the kernel, mean over every fourth timed "
                     "step (%d launches)" % t["kernel_samples"],
        },
    }
    if args.graph and world == 1:
        # the same step captured once into a CUDA graph and replayed: what a caller that runs the
        # calls back to back saves in launch overhead (only visible on small workloads)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            case.step()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            case.step()
        gev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for i in range(args.steps):
            if case.flush is not None:
                case.flush.zero_()
            gev[i][0].record()
            graph.replay()
            gev[i][1].record()
        torch.cuda.synchronize()
        out["cuda_graph"] = {"ms_per_step": float(np.mean([a_.elapsed_time(b_) for a_, b_ in gev])),
                             "eager_ms_per_step": ms_step}
    if not args.three_calls and world == 1 and not args.no_all_configs:
        # the separate calls on the same cache, for the stage split and the comparison
        ref = Case(cur, w, dev, whiten=args.whiten, three_calls=True, kv=(case.K, case.V, case.seqlens))
        rt = ref.timed(min(args.steps, 10), 3)
        out["three_calls"] = {"ms_per_step": rt["ms_events"] if rt["flushed"] else rt["ms_whole"],
                              "stage_ms": rt["stage_ms"], "streaming_kernel_ms": rt["kernel_ms"]}
        ref.K = ref.V = None
        ref.free()
    out["e2e"] = run_e2e(cur, w, case.K, case.V, case.seqlens, value_tokens=tokens, world=world, dev=dev,
                         steps=min(args.steps, args.e2e_steps))
    if rank == 0 and world == 1:
        if not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(w, core_seconds=20.0)
            out["cpu_baseline"]["headline_check"] = oracle_check(case, w.folded_batch // 2)
        case.free()
        if not args.no_all_configs and args.workload == "cfg3" and args.batch == 0 and args.layers == 0:
            out["all_configs"] = run_all_configs(cur, dev, steps=min(args.steps, 10),
                                                 check=not args.no_cpu_baseline)
    if rank == 0:
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
    that holds `budget` rows and compresses it back to `budget` (Alg. 1 (all steps) on the cache)."""
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
        if inplace:       # one call: new rows copied and heads selected in one launch, survivors stay
            cur.curdkv_cache_step(caches[live], K_new, V_new, G, k, ws, num_sink=c["num_sink"],
                                  window=c["window"])                    # put, at most `chunk` rows move
            return
        cur.curdkv_cache_append(caches[live], K_new, V_new, G, ws)
        if False:
            pass
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
    # What a step has to move.  In place: the new rows read once for their scores, the scores of all
    # rows looked at, and each surviving new row stored once (counted as all `chunk` of them: an upper
    # bound; evicted new rows are never stored).  Ordered: new rows read and stored, scores, and every
    # survivor read and written into the other cache.
    counted = P * ((t * 512 + (k + t) * 4 + t * 512) if inplace else (t * 512 * 2 + (k + t) * 4 + k * 512 * 2))
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
        "roofline": {"bound": "hbm", "kernel": "whole step (score the new rows, select, place the survivors)",
                     "achieved": gbs, "peak": peak, "peak_kind": peak_kind + " copy bandwidth", "unit": "GB/s",
                     "frac": gbs / peak, "traffic": None,
                     "note": "algorithmic bytes: every new row read once and stored at most once; the kernels "
                             "read the surviving new rows a second time when they place them"},
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

    split = not args.single_bf16_weights

    def step():
        cur.curdkv_attention_out(Q, K, V, desc, scale=scale, O=O, workspace=aws, weight_split=split)
        cur.curdkv_attention_out(Q, Kc, Vc, cdesc, scale=scale, head_rows=rows, O=Oc, workspace=aws,
                                 weight_split=split)
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
                                 workspace=aws, weight_split=split)
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
                     "note": ("algorithmic flops = one QK^T and one PV; the kernel issues 1.5x that "
                              "(PV for the hi and the lo half of the weights)") if split else
                             "algorithmic flops = one QK^T and one PV, issued once (single bf16 weights)"},
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


def run_dry(args):
    """Host logic of the N-rank run without a GPU (gloo): every rank takes its own replica of the
    workload description, "times" a fake step of 1 + rank/10 ms, the slowest rank's time is agreed
    on and rank 0 prints the line.  What the real run does around its kernels, and nothing else."""
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    w = rank_workload(synth.CONFIGS[args.workload], rank)
    tokens, read_bytes, write_bytes = workload_bytes(w, synth.make_seqlens(w))
    ms_step = max_over_ranks(1.0 + rank / 10.0, torch.device("cpu"), world)
    seeds = [None] * world
    if world > 1:
        dist.all_gather_object(seeds, w.data_seed)
        dist.barrier()
    else:
        seeds = [w.data_seed]
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": job_throughput(tokens, world, ms_step * 1e-3), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step,
                          "higher_is_better": True, "scaling": "weak", "data": "none (dry run of the host logic)",
                          "config": {"workload": workload_text(w), "head_tokens_per_step": tokens,
                                     "data_seeds": seeds}}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n):
    """`bench.py --gpus N` started by hand: re-launch this command as N ranks, one per GPU, the way
    the driver does (torch.distributed.run on 127.0.0.1); rank 0 prints the one line."""
    import socket

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


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
    ap.add_argument("--no-all-configs", action="store_true",
                    help="skip the other configurations (all_configs) and the three-call comparison")
    ap.add_argument("--dry-run", action="store_true",
                    help="host logic of the multi-rank path only (gloo, no CUDA): for tests on a CPU box")
    ap.add_argument("--single-bf16-weights", action="store_true",
                    help="--workload evict: softmax weights as single bf16 values (2e-3 instead of 1e-5 accuracy)")
    ap.add_argument("--decode-mode", choices=["inplace", "ordered"], default="inplace",
                    help="--workload decode: compress inside the cache (unordered) or copy in order")
    ap.add_argument("--whiten", action="store_true",
                    help="score with the whitened sketch (approximate leverage scores; reads K, V twice)")
    ap.add_argument("--e2e-steps", type=int, default=3,
                    help="steps of the host-buffer end-to-end leg (0 disables it)")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.dry_run:
        run_dry(args)
    elif args.workload in ("decode", "evict"):
        if args.impl == "reference":
            raise SystemExit("the reference arm times the prefill workloads only")
        run_decode(args) if args.workload == "decode" else run_evict(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

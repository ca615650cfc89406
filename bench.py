#!/usr/bin/env python
"""Benchmark of the sparse decode step (and, beside it, the prefill cache build).

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload NAME]

One "step" is one rq_decode_step (state update + append, page scoring, top-k,
sparse attention, combine) for every sequence of the batch at the workload's
context length and budget.  The default workload is the one the headline
metric is quoted on: batch 1, 32 heads x 128 dims, 128K context, page 16,
budget 1/16 (512 pages per head), bf16 I/O with fp32 state and accumulation.

Timing: CUDA events on the launching stream around exactly K steps after W
warm-up steps, barrier + synchronize on both sides, max over ranks.  Several
independent caches are rotated so that every step streams data that is not in
L2 (their total is many times the L2 size), and every step uses a fresh query
and token.  Prints ONE JSON line.

With --gpus N > 1 the path does not shard (heads are independent and there is
no exchange step): every rank runs an independent replica of the workload and
`value` is the per-step time divided by N.
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

METRIC = "sparse decode us/step at 128K ctx, 1/16 budget"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu captures
# (profiles/*_96k_b1.md: captured on a 96K-context case, scaled by 4/3 to the launches of the
# default workload, traffic being proportional to the pages processed): kernel -> bytes, or None
# when the kernel has changed since the capture.
NCU_TRAFFIC = {"score": 4 / 3 * (100.83e6 + 4.78e6), "attend": 4 / 3 * (100.81e6 + 3.64e6), "step": 4 / 3 * (201.73e6 + 5.97e6)}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def pick_workload(name):
    from paper_2605_28640_b200 import workloads as wl
    import dataclasses
    table = {"metric": wl.METRIC, "cfg1": wl.CONFIGS[1], "cfg2": wl.CONFIGS[2], "cfg4": wl.CONFIGS[4],
             "cfg4-1/8": dataclasses.replace(wl.CONFIGS[4], budget_den=8),
             "cfg4-1/4": dataclasses.replace(wl.CONFIGS[4], budget_den=4),
             "half": dataclasses.replace(wl.METRIC, name="decode-64k-b1", T=65536),
             "page64": dataclasses.replace(wl.METRIC, name="decode-128k-b1-page64", S=64),
             "small": dataclasses.replace(wl.CONFIGS[1], name="small-16k"),
             # the paper's own Quest settings (App. A.1): 4K context, block 64 with 16 kept pages; block 16 with 4
             "paper4k": dataclasses.replace(wl.CONFIGS[1], name="quest-4k-block64-k16", T=4096, S=64, budget_den=4),
             "paper4k-b16": dataclasses.replace(wl.CONFIGS[1], name="quest-4k-block16-k4", T=4096, S=16, budget_den=64)}
    return table[name]


def step_bytes(w, T):
    """Algorithmic bytes one decode step must touch: all page bounds + the selected K/V pages."""
    es = 2 if str(w.dtype).endswith("bfloat16") else 4
    P, K = w.pages(T), w.budget_pages(T)
    meta = w.B * w.H * P * 2 * w.D * es
    kvb = w.B * w.H * min(K, P) * w.S * w.D * es * 2
    return meta, kvb


# ------------------------------------------------------------------------- oracle arm
class OracleSample:
    """The fp64 oracle, as it stands, on `n_heads` heads of batch item 0 of the workload:
    prefill (untimed), then decode steps (append one token, score, select, attend) timed
    per call.  Heads run on a thread pool (the C code releases the GIL)."""

    def __init__(self, w, k, v, g, q, kt, vt, gt, n_heads, threads, max_steps):
        import concurrent.futures as cf
        import oracle
        import torch
        odt = oracle.BF16 if w.dtype == torch.bfloat16 else oracle.F32
        T0 = k.shape[1]
        self.K = w.budget_pages(T0 + 1)
        self.scale = w.D ** -0.5
        self.threads = threads
        self.pool = cf.ThreadPoolExecutor(threads)

        def f64(t):
            return t.detach().to(torch.float64).cpu().numpy()

        self.items = []
        for h in range(n_heads):
            hd = oracle.Head(w.D, w.S, T0 + max_steps + 1, odt)
            self.items.append((hd, f64(q[0, h]), f64(kt[0, h]), f64(vt[0, h]), f64(gt[0, h])))
        pre = [(self.items[h][0], f64(k[0, :, h]), f64(v[0, :, h]), f64(g[0, :, h])) for h in range(n_heads)]
        list(self.pool.map(lambda it: it[0].append(it[1], it[2], it[3]), pre))

    def _one(self, item):
        hd, q, a, b, c = item
        hd.append(a, b, c)
        hd.query(q, self.K, self.scale)

    def step(self):
        """One decode step of every sampled head; returns wall seconds."""
        t0 = time.perf_counter()
        list(self.pool.map(self._one, self.items))
        return time.perf_counter() - t0


def oracle_sample_for(w, dev, n_heads, threads, max_steps, inputs=None):
    import dataclasses
    from paper_2605_28640_b200 import workloads as wl
    ws = dataclasses.replace(w, B=1, H=n_heads, needles=0, resets=False)
    if inputs is None:
        k, v, g = wl.make_prefill(ws, dev, w.T - 1)
    else:
        k, v, g = inputs
    q = wl.make_query(ws, dev)
    kt, vt, gt = wl.make_token(ws, dev)
    return OracleSample(ws, k, v, g, q, kt, vt, gt, n_heads, threads, max_steps)


def run_reference(args, w):
    """--impl reference: the CPU oracle timed on the host cores on a bounded sample."""
    import torch
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    threads = n_heads = min(cores, 8, w.H)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    smp = oracle_sample_for(w, dev, n_heads, threads, args.warmup + args.steps)
    for _ in range(args.warmup):
        smp.step()
    dt = sum(smp.step() for _ in range(args.steps)) / max(args.steps, 1)
    rounds = -(-(w.B * w.H) // threads)          # a whole step = B*H heads, `threads` at a time
    us = dt * rounds * 1e6
    sample = (f"{n_heads} heads of batch item 0 at full context ({w.T} tokens), one decode step of each per "
              f"timed step on {threads} threads; scaled by ceil(B*H/threads) = {rounds} to the whole step")
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": "us/step", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w), "l2": "not applicable: CPU oracle on a sample of heads",
            "cpu_baseline": {"value": us, "unit": "us/step", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": "us/step", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def max_over_ranks(ms, world, device):
    """The slowest rank's time: what a job of `world` replicas takes."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.item()


def whole_job_us_per_step(max_ms, steps, world):
    """Replicas only: `world` GPUs each take a step in max_ms / steps, so the job takes that time per `world` steps."""
    return max_ms / steps * 1e3 / world


def selftest_ranks():
    """The rank plumbing on CPU (gloo): every rank contributes a time, rank 0 prints what the job would report."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = max_over_ranks(10.0 * (rank + 1), world, "cpu")
    if rank == 0:
        print(json.dumps({"max_ms": ms, "world": world, "us_per_step": whole_job_us_per_step(ms, 5, world)}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def workload_config(w):
    return {"workload": w.name, "batch": w.B, "heads": w.H, "head_dim": w.D, "context": w.T,
            "page_size": w.S, "budget": f"{w.budget_num}/{w.budget_den}", "budget_pages": w.budget_pages(),
            "io_dtype": str(w.dtype).replace("torch.", ""), "state_dtype": "float32"}


def event_ms(fn, stream=None):
    """Device time of fn() between two events on the current stream, synchronised on both sides."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def parity_block(w, cache, sample_inputs, q, tok, K, T0, dev, recall_cache=None, recall_w=None):
    """One decode step of the timed configuration checked against the fp64 oracle on a sample of
    heads (states, stored cache, page bounds, scores, page list, attention output), and the recall
    of the planted pages over all heads for the three budgets.  Runs before the timed region."""
    import math
    import torch
    import paper_2605_28640_b200 as rq
    from paper_2605_28640_b200 import workloads as wl
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import parity
    k_s, v_s, g_s = sample_inputs
    nh = k_s.shape[2]
    heads = sorted({0, nh // 3, nh - 1})
    out = {"sampled_heads": [[0, h] for h in heads], "checked": "state, stored cache, page bounds, scores, page list, attention"}
    try:
        ohs = {h: parity.oracle_head(w, k_s, v_s, g_s, 0, h, T0 + 8) for h in heads}
        kt, vt, gt = tok
        o = torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=dev)
        idx = torch.full((w.B, w.H, K), -7, dtype=torch.int32, device=dev)
        rq.rq_decode_step(cache.handle, q, kt, vt, gt, K, 0.0, o, idx)
        P = w.pages(T0 + 1)
        scores = torch.empty(w.B, w.H, P, dtype=torch.float32, device=dev)
        idx2 = torch.empty_like(idx)
        rq.rq_select_pages(cache.handle, q, K, scores, idx2)
        torch.cuda.synchronize()
        assert torch.equal(idx, idx2), "the decode step and the stage export select different pages"
        assert rq.rq_device_status(cache.handle) == rq.RQ_OK
        stats = {}
        parity.OBSERVED.clear()
        for h, hd in ohs.items():
            hd.append(parity.f64(kt[0, h]), parity.f64(vt[0, h]), parity.f64(gt[0, h]))
            d = parity.check_cache_level(cache, hd, 0, h, w.dtype)
            parity.check_query_level(d, hd, cache, 0, h, q, K, w.D ** -0.5, o, idx, scores, w.dtype, stats)
        out.update({"passed": True, "near_tie_heads": stats.get("near_tie", 0),
                    "near_tie_mismatches": stats.get("near_tie_mismatch", 0),
                    "pages_shared_with_the_oracles_own_chain": stats.get("e2e_overlap", 0.0) / max(stats.get("heads", 1), 1),
                    "state_abs_err_over_rms": parity.OBSERVED.get("state_abs_err_over_rms"),
                    "stored_fraction_one_step_off": parity.OBSERVED.get("stored_fraction_one_step_off"),
                    "attention_max_abs_err": stats.get("att_max"), "attention_mean_abs_err": stats.get("att_mean")})
    except AssertionError as e:
        out.update({"passed": False, "failure": str(e)[:300]})
    if w.needles and recall_cache is not None:
        # pages planted to align with this query, in a cache of the metric's own recipe (copy 0 also
        # carries the state resets of the prefill case, whose short averages outscore everything)
        planted = wl.needle_pages(recall_w, T0)
        P = w.pages(len(recall_cache))
        rec = {"cache": "copy 1 (no resets), %d tokens" % len(recall_cache)}
        for den in (4, 8, 16):
            Kd = max(1, math.ceil(P / den))
            if Kd > recall_cache.cfg.max_budget_pages:
                continue
            idd = torch.empty(w.B, w.H, Kd, dtype=torch.int32, device=dev)
            rq.rq_select_pages(recall_cache.handle, q, Kd, None, idd)
            sel = idd.cpu().numpy()
            hit = sum(len(set(planted[b, h].tolist()) & set(sel[b, h].tolist())) for b in range(w.B) for h in range(w.H))
            rec[f"1/{den}"] = hit / (w.B * w.H * w.needles)
        out["planted_page_recall"] = rec
    return out


def snapkv_block(w, cache, dev, peak):
    """Times of the SnapKV-style reduction (App. A.1) of one of the timed caches, after the decode steps: window of
    64 queries, 1/16 of the entries retained; median of five event-timed calls after two warm-up calls."""
    import torch
    import paper_2605_28640_b200 as rq
    T = len(cache)
    W, keep = 64, max(64, T // 16)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed + 99)
    qw = torch.randn(w.B, W, w.H, w.D, generator=g, device=dev, dtype=torch.float32).to(w.dtype)
    idx = torch.empty(w.B, w.H, keep, dtype=torch.int32, device=dev)
    scratch = torch.empty(rq.rq_snapkv_scratch_bytes(cache.handle), dtype=torch.uint8, device=dev)
    small = rq.Cache(w.B, w.H, w.D, w.S, keep + 64, w.dtype, w.gdtype, device=dev)
    sel = sorted(event_ms(lambda: rq.rq_snapkv_select(cache.handle, qw, W, keep, 0.0, idx, None, scratch)) for _ in range(7))[:5]
    cmp_ = sorted(event_ms(lambda: rq.rq_snapkv_compact(cache.handle, idx, keep, small.handle)) for _ in range(7))[:5]
    es = 2 if w.dtype == torch.bfloat16 else 4
    key_bytes = 2 * w.B * w.H * T * w.D * es                   # the keys are read twice (statistics, then weights)
    flops = 2 * 2.0 * W * w.D * T * w.B * w.H
    move = 2 * 2 * w.B * w.H * keep * w.D * es                 # retained keys and values read and written
    return {"window": W, "keep": keep, "tokens": T,
            "select_ms": sel[2], "select_ms_min": sel[0], "select_key_bytes": key_bytes,
            "select_gbs": key_bytes / (sel[2] * 1e-3) / 1e9, "select_frac_of_hbm_peak": key_bytes / (sel[2] * 1e-3) / 1e9 / peak,
            "select_tflops": flops / (sel[2] * 1e-3) / 1e12,
            "compact_ms": cmp_[2], "compact_ms_min": cmp_[0], "compact_bytes": move,
            "compact_gbs": move / (cmp_[2] * 1e-3) / 1e9,
            "status_ok": rq.rq_device_status(cache.handle) == rq.RQ_OK,
            "note": "rq_snapkv_select = importance (two passes over the keys) + selection; rq_snapkv_compact = reset of the "
                    "new cache + gather of the retained rows + page bounds + state"}


def moba_block(w, dev):
    """Times of the MoBA-style block-sparse prefill attention (App. A.1) at the paper's setting: prompts of 4096 tokens,
    block 64 and 128, budget 1/4 and 1/16, for the workload's batch, heads and head size; median of five event-timed calls."""
    import dataclasses
    import torch
    import paper_2605_28640_b200 as rq
    from paper_2605_28640_b200 import workloads as wl
    T = 4096
    wm = dataclasses.replace(w, T=T, needles=0, resets=False, name="moba-4k")
    cache = rq.Cache(wm.B, wm.H, wm.D, wm.S, T, wm.dtype, wm.gdtype, device=dev)
    k, v, g = wl.make_prefill(wm, dev, T)
    rq.rq_build_cache(cache.handle, k, v, g)
    del k, v, g
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 55)
    q = torch.randn(wm.B, T, wm.H, wm.D, generator=gen, device=dev, dtype=torch.float32).to(wm.dtype)
    o = torch.empty_like(q)
    out = {"tokens": T, "batch": wm.B, "heads": wm.H, "runs": []}
    for block, K in ((64, 16), (64, 4), (128, 8)):
        scratch = torch.empty(rq.rq_moba_scratch_bytes(cache.handle, block, K), dtype=torch.uint8, device=dev)
        ts = sorted(event_ms(lambda: rq.rq_moba_prefill(cache.handle, q, block, K, 0.0, o, None, None, scratch)) for _ in range(7))[:5]
        # attended (query, key) pairs: K blocks per query (fewer for the first K blocks of queries), the own block half on average
        nb = T // block
        pairs = sum(min(K, t // block + 1) * block - (block - 1 - t % block) for t in range(T))
        flops = 4.0 * pairs * wm.D * wm.B * wm.H
        out["runs"].append({"block": block, "blocks_per_query": K, "ms": ts[2], "ms_min": ts[0],
                            "attended_fraction": pairs / (T * (T + 1) / 2), "tflops_on_attended_pairs": flops / (ts[2] * 1e-3) / 1e12})
        del scratch
    out["status_ok"] = rq.rq_device_status(cache.handle) == rq.RQ_OK
    out["note"] = ("rq_moba_prefill = block means + routing of every query + attention over the chosen blocks "
                   "(both products of the attention on the tensor cores for bf16 caches)")
    return out


# ------------------------------------------------------------------------- own arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="rq", choices=["rq", "reference"])
    ap.add_argument("--workload", default="metric")
    ap.add_argument("--batch", type=int, default=0, help="the chosen workload at another batch size (context runs, not the metric)")
    ap.add_argument("--context", type=int, default=0, help="the chosen workload at another context length (context runs, not the metric)")
    ap.add_argument("--copies", type=int, default=0, help="independent caches to rotate (0 = auto, at least 4)")
    ap.add_argument("--path", type=int, default=0, choices=[0, 1, 2, 4, 8],
                    help="how the step is launched: 0 the library chooses, 1 separate kernels, 2/4/8 one launch with that many groups of heads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill", action="store_true")
    ap.add_argument("--no-parity", action="store_true")
    ap.add_argument("--selftest-ranks", action="store_true", help="CPU check of the multi-rank plumbing (gloo); used by the tests")
    ap.add_argument("--no-next", action="store_true", help="skip the SnapKV and MoBA timing blocks (they run by default)")
    ap.add_argument("--moba", action="store_true",
                    help="also time the MoBA-style block-sparse prefill attention at the paper's setting (4K prompts, block 64, "
                         "16 blocks per query) for the workload's batch and heads")
    ap.add_argument("--snapkv", action="store_true",
                    help="also time the SnapKV-style reduction of the first cache (window 64, 1/16 of the entries retained)")
    args = ap.parse_args()
    if args.selftest_ranks:
        selftest_ranks()
        return
    args.warmup = max(args.warmup, 3) if args.impl == "rq" else args.warmup

    import dataclasses
    w = pick_workload(args.workload)
    if args.batch or args.context:
        w = dataclasses.replace(w, name=f"{w.name}-b{args.batch or w.B}-t{args.context or w.T}", B=args.batch or w.B,
                                T=args.context or w.T)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import dataclasses
    import torch
    import torch.distributed as dist
    import paper_2605_28640_b200 as rq
    from paper_2605_28640_b200 import build, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    build.build_library()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    es = 2 if w.dtype == torch.bfloat16 else 4
    T0 = w.T - 1                      # the first timed step brings the context to w.T
    total_steps = args.warmup + args.steps
    # caches: at least four copies, and enough that their streamed bytes exceed L2 several times over
    meta_b, kv_b = step_bytes(w, w.T)
    l2 = torch.cuda.get_device_properties(local).L2_cache_size
    ncopies = args.copies or max(4, min(8, -(-(4 * l2) // (meta_b + kv_b))))
    # per copy: the parity step, the timed loop, two more passes for the clock sampler, the profiled and e2e passes
    per_copy = -(-total_steps // ncopies)
    cap = T0 + 6 * per_copy + 256
    K = w.budget_pages(w.T)
    maxK = max(w.budget_pages(cap) + 1, -(-w.pages(cap) // 4) + 1)      # room for the 1/4 budget of the recall sweep
    first = rank == 0 and world == 1

    caches, first_build_ms, rebuild_ms = [], [], []
    q0 = wl.make_query(w, dev, 0)
    sample_inputs = None
    for c in range(ncopies):
        wc = dataclasses.replace(w, seed=w.seed + 17 * c, resets=(c == 0))
        k, v, g = wl.make_prefill(wc, dev, T0, q_for_needles=q0 if w.needles else None)
        cache = rq.Cache(w.B, w.H, w.D, w.S, cap, w.dtype, w.gdtype, max_budget_pages=maxK, device=dev)
        cache.handle.reserved[2] = args.path
        first_build_ms.append(event_ms(lambda: rq.rq_build_cache(cache.handle, k, v, g)))
        if c == 0 and not args.no_prefill:
            # the prefill proper: rebuilds of the same cache on a kernel that has run before
            def rebuild():
                rq.rq_cache_reset(cache.handle)
                rq.rq_build_cache(cache.handle, k, v, g)
            for _ in range(7):
                rebuild_ms.append(event_ms(rebuild))
        caches.append(cache)
        if c == 0 and first and not (args.no_cpu_baseline and args.no_parity):
            nh = min(8, w.H)
            sample_inputs = (k[:1, :, :nh].clone(), v[:1, :, :nh].clone(), g[:1, :, :nh].clone())
        del k, v, g
    torch.cuda.empty_cache()

    # fresh inputs for every step, resident on the device before the timed region
    pool = 64
    qs = [wl.make_query(w, dev, s) for s in range(pool)]
    toks = [wl.make_token(w, dev, s) for s in range(pool)]
    outs = [torch.empty(w.B, w.H, w.D, dtype=w.dtype, device=dev) for _ in range(4)]

    parity = None
    if first and not args.no_parity:
        parity = parity_block(w, caches[0], sample_inputs, qs[0], toks[0], K, T0, dev, recall_cache=caches[1 % ncopies],
                              recall_w=dataclasses.replace(w, seed=w.seed + 17 * (1 % ncopies)))

    stream = torch.cuda.current_stream()

    def step(i):
        kt, vt, gt = toks[i % pool]
        rq.rq_decode_step(caches[i % ncopies].handle, qs[i % pool], kt, vt, gt, K, 0.0, outs[i % 4], stream=stream)

    launches_per_step = rq.rq_decode_step_launches(caches[1 % ncopies].handle, K)
    for i in range(args.warmup):
        step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        e0.record()
        for i in range(args.warmup, total_steps):
            step(i)
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        # keep the sampler running over more of the same work so that a short timed region still
        # gets clock samples under load: decode steps while the caches have room, then the same
        # selection and attention kernels without the append
        t_end = time.time() + 1.5
        j = total_steps
        idx_keep = torch.empty(w.B, w.H, K, dtype=torch.int32, device=dev)
        while time.time() < t_end:
            if j < 3 * total_steps:
                step(j)
            else:
                c = caches[j % ncopies].handle
                rq.rq_select_pages(c, qs[j % pool], K, None, idx_keep)
                rq.rq_attend_pages(c, qs[j % pool], idx_keep, K, 0.0, outs[j % 4])
            j += 1
            if j % 16 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
    ms_per_step = max_over_ranks(ms, world, dev) / args.steps
    n_launches = args.steps * launches_per_step

    # ---- per-kernel times of the step run as separate kernels (a separate pass, same rotation):
    # events between the kernels of a step
    prof = {}
    nprof = min(args.steps, 50) + 3
    for c in caches:
        c.handle.reserved[2] = 1
    for i in range(nprof):
        # a plain step on another cache goes first, so that the profiled kernels are launched
        # behind running work as in the timed loop (on an idle GPU every kernel's time would
        # include its launch latency)
        kt, vt, gt = toks[(i + 7) % pool]
        rq.rq_decode_step(caches[(i + 1) % ncopies].handle, qs[(i + 7) % pool], kt, vt, gt, K, 0.0, outs[1])
        kt, vt, gt = toks[i % pool]
        r = rq.rq_decode_step_profiled(caches[i % ncopies].handle, qs[i % pool], kt, vt, gt, K, 0.0, outs[0])
        if i >= 3:
            for name, us in r.items():
                prof.setdefault(name, []).append(us)
    for c in caches:
        c.handle.reserved[2] = args.path
    kernel_us = {n: sum(v) / len(v) for n, v in prof.items()}

    # ---- what one plain launch of the same size draws from HBM on this GPU: a read of as many
    # bytes as a step touches (and of half as many: one of its two streams), rotating over the caches
    sink = torch.zeros(64, dtype=torch.int32, device=dev)
    probe = {}
    for name, nbytes in (("step_sized", meta_b + kv_b), ("half_step_sized", (meta_b + kv_b) // 2)):
        nbytes = min(nbytes, caches[0].kv.numel())
        for i in range(3):
            rq.rq_probe_read(caches[i % ncopies].kv, nbytes, sink)
        reps = 12
        ms_p = event_ms(lambda: [rq.rq_probe_read(caches[i % ncopies].kv, nbytes, sink) for i in range(reps)])
        probe[name] = {"bytes": nbytes, "us": ms_p / reps * 1e3, "gbs": nbytes / (ms_p / reps * 1e-3) / 1e9}

    # ---- end to end through the host-buffer entry point (pinned host tensors, result read back)
    hq = [q.cpu().pin_memory() for q in qs[:8]]
    ht = [tuple(x.cpu().pin_memory() for x in tk) for tk in toks[:8]]
    ho = torch.empty(w.B, w.H, w.D, dtype=w.dtype).pin_memory()
    n_e2e = min(args.steps, 50)

    def e2e_step(i):
        kt, vt, gt = ht[i % 8]
        rq.rq_decode_step_host(caches[i % ncopies].handle, hq[i % 8], kt, vt, gt, K, 0.0, ho, stream=stream)
        stream.synchronize()                           # the caller reads the result before the next step

    for i in range(3):
        e2e_step(i)
    barrier()
    e0.record()
    for i in range(n_e2e):
        e2e_step(i)
    e1.record()
    barrier()
    e2e_us = max_over_ranks(e0.elapsed_time(e1), world, dev) / n_e2e * 1e3
    in_bytes = w.B * w.H * w.D * (3 * es + (2 if w.gdtype == torch.bfloat16 else 4))
    out_bytes = w.B * w.H * w.D * es

    if rank != 0:
        return

    peak, peak_kind = measured_peak()
    us = ms_per_step * 1e3
    step_gbs = (meta_b + kv_b) / (us * 1e-6) / 1e9
    kbytes = {"score": meta_b, "attend": kv_b}
    separate = {n: {"us": kernel_us[n], "gbs": kbytes[n] / (kernel_us[n] * 1e-6) / 1e9,
                    "frac": kbytes[n] / (kernel_us[n] * 1e-6) / 1e9 / peak} for n in kbytes if kernel_us.get(n)}
    if launches_per_step == 1:
        # the whole step is one kernel: its average launch duration is the step time of the timed region
        roof = {"bound": "hbm", "kernel": "step (update, scoring, selection, flash-decode and combine in one launch)",
                "achieved": step_gbs, "peak": peak, "unit": "GB/s", "frac": step_gbs / peak, "peak_kind": peak_kind,
                "traffic": NCU_TRAFFIC.get("step") if args.workload == "metric" else None,
                "bytes_per_launch": meta_b + kv_b, "launch_us": us}
    else:
        dom = max(kbytes, key=lambda n: kernel_us.get(n, 0.0))
        roof = {"bound": "hbm", "kernel": dom, "achieved": separate[dom]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": separate[dom]["frac"], "peak_kind": peak_kind,
                "traffic": NCU_TRAFFIC.get(dom) if args.workload == "metric" else None,
                "bytes_per_launch": kbytes[dom], "launch_us": kernel_us[dom]}
    roof["launch_sized_read_gbs"] = probe["step_sized" if launches_per_step == 1 else "half_step_sized"]["gbs"]
    roof["plain_read_probe"] = probe
    roof["as_separate_kernels_us"] = kernel_us
    roof["as_separate_kernels"] = separate
    line = {
        "metric": METRIC, "value": whole_job_us_per_step(ms_per_step * args.steps, args.steps, world), "unit": "us/step", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(w),
        "l2": f"inputs larger than L2: {ncopies} independent caches rotated, fresh q/k/v/g every step",
        "tokens_per_s": w.B * world / (us * 1e-6),
        "step_hbm": {"algorithmic_bytes": meta_b + kv_b, "gbs": step_gbs, "frac_of_peak": step_gbs / peak,
                     "frac_of_nominal_8tbs": step_gbs / 8000.0, "peak_gbs": peak, "peak_kind": peak_kind},
        "roofline": roof,
        "clocks": clocks.summary(),
        "e2e": {"value": whole_job_us_per_step(e2e_us * n_e2e / 1e3, n_e2e, world), "unit": "us/step", "h2d_bytes_per_step": in_bytes,
                "d2h_bytes_per_step": out_bytes},
        "gpu_launches": n_launches, "launches_per_step": launches_per_step,
    }
    if parity is not None:
        line["parity"] = parity
    if not args.no_prefill and rebuild_ms:
        runs = sorted(rebuild_ms[2:])                            # the first two rebuilds warm the kernel up
        pm = runs[len(runs) // 2]
        gs = 2 if w.gdtype == torch.bfloat16 else 4
        pbytes = w.B * w.H * T0 * w.D * (2 * es + gs + 2 * es) + w.B * w.H * w.pages(T0) * 2 * w.D * es
        line["prefill"] = {"ms": pm, "ms_min": runs[0], "tokens_per_s": w.B * T0 / (pm * 1e-3), "algorithmic_bytes": pbytes,
                           "gbs": pbytes / (pm * 1e-3) / 1e9, "frac_of_peak": pbytes / (pm * 1e-3) / 1e9 / peak,
                           "runs_ms": rebuild_ms[2:], "first_build_ms": first_build_ms,
                           "note": "median of five rebuilds (rq_cache_reset + rq_build_cache) after two warm-up rebuilds"}
    # the widened rows (SnapKV-style cache reduction, MoBA-style prefill attention): timed after the decode steps, outside
    # the timed region; a failure is reported in the block and leaves the line above intact
    if first and (args.snapkv or not args.no_next):
        try:
            line["snapkv"] = snapkv_block(w, caches[0], dev, peak)
        except Exception as e:                                  # noqa: BLE001
            line["snapkv"] = {"error": str(e)[:200]}
    if first and (args.moba or not args.no_next):
        try:
            line["moba"] = moba_block(w, dev)
        except Exception as e:                                  # noqa: BLE001
            line["moba"] = {"error": str(e)[:200]}
    if first and not args.no_cpu_baseline:
        nh = min(8, w.H)
        threads = min(os.cpu_count() or 1, nh)
        smp = oracle_sample_for(w, dev, nh, threads, 4096, inputs=sample_inputs)
        smp.step()
        probe_s = sum(smp.step() for _ in range(3)) / 3
        reps = int(max(10, min(4000, 12.0 / max(probe_s, 1e-6))))    # about 12 s of host work
        wall = sum(smp.step() for _ in range(reps))
        rounds_sample = -(-nh // threads)
        rounds_full = -(-(w.B * w.H) // threads)
        line["cpu_baseline"] = {
            "value": wall / reps / rounds_sample * rounds_full * 1e6, "unit": "us/step", "cores": threads,
            "kind": "oracle",
            "sample": (f"{nh} heads of batch item 0 at full context, {reps} decode steps each on {threads} "
                       f"threads ({wall:.1f} s wall); scaled to all {w.B * w.H} heads")}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

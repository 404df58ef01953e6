#!/usr/bin/env python
"""Benchmark of batched SuffixDecoding draft generation on B200.

A step is one decode step of the whole batch on the headline workload
(config "large_batch": 4M-token global corpus, 256 requests with 4,096-token
prompts): the tokens each request accepted in the previous step (a seeded
schedule, mean 4 tokens, taken from the request's hidden continuation) are
appended to its tree, then a draft tree is speculated for every request.  That is
one sd_step launch; the same work as two calls (sd_append, sd_speculate) is timed
beside it.  The global tree and the prompts are built
before the timed region.  One JSON line is printed by rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workload.generator import accept_schedule, get_workload  # noqa: E402

METRIC = "speculation trees/s at batch {B} (per step: append the accepted tokens, speculate)"
UNIT = "trees/s"
OUT_BYTES_PER_REQ = 4 * 64 * 3 + 64 * 8 + 4 * 3 + 8          # tokens, parents, positions, mask, scalars
FLUSH_BYTES = 256 << 20
APPEND_BYTES_PER_UPDATE = 32                                   # a node's 16-byte entry read and written back
STEP_KERNEL = "speculate_fused_kernel<true, 10, 2, 4> (all of sd_step)"
# dram__bytes_read + dram__bytes_write of one launch of that kernel on the full-size large_batch
# workload, from an ncu capture; it is reported only while the kernel source still has the
# digest the capture was taken at (profiles/ holds the summary), else as null
DRAM_TRAFFIC = {"bytes": 28.03e6, "speculate_cu_sha1": "7370e8a536030ddfd449f3b9c42399bd02e1033a"}


def dram_traffic():
    import hashlib
    if DRAM_TRAFFIC["bytes"] is None:
        return None
    try:
        with open(os.path.join(ROOT, "paper_2411_04975_b200", "csrc", "speculate.cu"), "rb") as f:
            same = hashlib.sha1(f.read()).hexdigest() == DRAM_TRAFFIC["speculate_cu_sha1"]
    except OSError:
        same = False
    return DRAM_TRAFFIC["bytes"] if same else None


def config_dict(c, args):
    """The workload both arms (the CUDA path and the oracle) are timed on: one dict for both."""
    return {"workload": c.name + (" (small)" if args.small else ""), "batch_per_gpu": c.batch,
            "global_tokens": int(c.n_seqs * c.seq_len), "prompt_len": c.prompt_len, "vocab": c.vocab,
            "D": c.depth_cap, "P": c.max_pattern, "alpha": c.alpha, "max_spec": c.max_spec, "tau": 0.0,
            "l2": "GPU arm: flushed between steps (256 MiB write outside the timed events)",
            "parallelism": f"replica x{args.gpus}, requests sharded" if args.gpus > 1 else "single GPU"}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="large_batch")
    ap.add_argument("--no-oracle", action="store_true", help="skip the CPU-oracle leg (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--oracle-samples", type=int, default=25)
    ap.add_argument("--small", action="store_true", help="1/16 corpus, batch 32: quick functional run")
    ap.add_argument("--sweep", action="store_true",
                    help="scalability sweep over the size of the global tree (shape of the paper's appendix table)")
    ap.add_argument("--sweep-oracle", action="store_true",
                    help="with --sweep: time the CPU oracle beside every row (one thread, a sample of the requests)")
    ap.add_argument("--closed-loop-oracle", action="store_true",
                    help="closed_loop config: run the CPU oracle in lock-step and compare every step (slow)")
    return ap.parse_args()


def make_workload(args):
    kw = {}
    if args.small:
        kw = dict(n_seqs=256, batch=32)
    return get_workload(args.config, **kw)


class StepInputs:
    """Per-step append inputs for `n_steps` steps of `B` requests."""

    def __init__(self, w, first_request, B, n_steps, prompts):
        self.sched = accept_schedule(B, n_steps, seed_index=first_request)
        total = self.sched.sum(axis=0)
        self.cont = [w.continuation(first_request + i, prompts[i], length=int(total[i]) + 1) for i in range(B)]
        self.cursor = np.zeros(B, dtype=np.int64)
        self.max_total = int(total.max())
        self.offsets, self.tokens, self.lists = [], [], []
        for k in range(n_steps):
            a = self.sched[k]
            off = np.zeros(B + 1, dtype=np.int64)
            off[1:] = np.cumsum(a)
            lists = [self.cont[i][self.cursor[i]:self.cursor[i] + a[i]] for i in range(B)]
            self.cursor += a
            self.offsets.append(off)
            self.lists.append(lists)
            self.tokens.append(np.concatenate(lists).astype(np.int32))


class ClockSampler:
    """Polls nvidia-smi (one query per call) from a thread while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.thread, self.stop_flag = index, [], None, threading.Event()

    def start(self):
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def _poll(self):
        while not self.stop_flag.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10)
                for line in out.stdout.strip().splitlines():
                    self.rows.append([x.strip() for x in line.split(",")])
            except (OSError, subprocess.SubprocessError):
                return
            self.stop_flag.wait(0.02)

    def stop(self):
        self.stop_flag.set()
        if self.thread is not None:
            self.thread.join(timeout=15)
        rows = [r for r in self.rows if len(r) >= 7]

        def num(x):
            try:
                return float(x)
            except ValueError:
                return None
        sm = [num(r[0]) for r in rows if num(r[0]) is not None]
        mx = [num(r[1]) for r in rows if num(r[1]) is not None]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for j, n in enumerate(names) if any(r[3 + j] == "Active" for r in rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def oracle_threads(B):
    return max(1, min(os.cpu_count() or 1, B))


# --------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2411_04975_b200 as sfx
    from paper_2411_04975_b200 import sharding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = make_workload(args)
    c = w.cfg
    B, K, W = c.batch, args.steps, args.warmup
    Ke = 0 if args.no_e2e else K
    We = 0 if args.no_e2e else min(W, 3)
    K2 = min(K, 30)                                   # steps timed as two calls, for the breakdown
    n_steps = W + K + 3 * (We + Ke) + K2             # the end-to-end loop runs once per transfer mode
    first = sharding.request_range(rank, world, B)[0]   # weak scaling: every rank has its own requests
    prompts = [w.prompt(first + i) for i in range(B)]
    steps = StepInputs(w, first, B, n_steps, prompts)

    corpus = torch.as_tensor(w.corpus(), device=dev)
    offsets = torch.as_tensor(w.corpus_offsets(), device=dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    store = sfx.SuffixStore(corpus, offsets, vocab=c.vocab, depth_cap=c.depth_cap, max_requests=B,
                            max_req_tokens=c.prompt_len + steps.max_total + 8, max_spec_cap=c.max_spec)
    torch.cuda.synchronize()
    build_ms = (time.perf_counter() - t0) * 1e3
    slots = torch.arange(B, dtype=torch.int32, device=dev)
    poff = np.zeros(B + 1, dtype=np.int64)
    poff[1:] = np.cumsum([len(p) for p in prompts])
    d_prompts = torch.as_tensor(np.concatenate(prompts), device=dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    store.build_requests(np.arange(B, dtype=np.int32), poff, d_prompts)      # sort-based, all prompts at once
    torch.cuda.synchronize()
    prompt_ms = (time.perf_counter() - t0) * 1e3

    d_off = [torch.as_tensor(o, device=dev) for o in steps.offsets[:W + K]]
    d_tok = [torch.as_tensor(t, device=dev) for t in steps.tokens[:W + K]]
    d_off2 = [torch.as_tensor(o, device=dev) for o in steps.offsets[W + K + 3 * (We + Ke):]]
    d_tok2 = [torch.as_tensor(t, device=dev) for t in steps.tokens[W + K + 3 * (We + Ke):]]
    out = store.alloc_outputs(B)
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def step(k):
        store.step(slots, d_off[k], d_tok[k], c.max_pattern, c.alpha, c.max_spec, 0, None, out)

    n_samp = 0 if (args.no_oracle or world > 1) else max(1, min(args.oracle_samples, K))
    sample_steps = sorted({W + (j * K) // n_samp for j in range(n_samp)}) if n_samp else []
    saved = {}

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    for k in range(W):
        flush.zero_()
        step(k)
    torch.cuda.synchronize()
    if rank == 0:                                      # let the clock sampler come up
        t_wait = time.perf_counter()
        while not sampler.rows and time.perf_counter() - t_wait < 5.0:
            time.sleep(0.05)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(K)]
    wall0 = time.perf_counter()
    for j in range(K):
        k = W + j
        flush.zero_()                                  # L2 flush, outside the per-step events
        ev[j][0].record()
        step(k)
        ev[j][1].record()
        if k in sample_steps:
            saved[k] = {n: t.clone() for n, t in out.items()}
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - wall0) * 1e3
    tot_ms = [ev[j][0].elapsed_time(ev[j][1]) for j in range(K)]
    timed_ms = sharding.max_over_ranks(float(sum(tot_ms)), dev)
    ms_per_step = timed_ms / K

    # ---- end to end: host buffers in, host buffers out, every step
    e2e = None
    e2e_other = None
    if not args.no_e2e:
        # per step: ONE pinned host buffer in (offsets, slots, tokens), ONE pinned host buffer out.
        # Ways to move them: "copies" = one cudaMemcpyAsync each way around the call; "direct" =
        # the call is given the pinned host buffers themselves and the kernel reads and writes
        # them across the bus; "direct_out" = inputs copied, drafts written by the kernel.  All
        # are timed; the fastest one is the e2e figure and the others are listed beside it.
        E = We + Ke
        max_tok = max(int(t.size) for t in steps.tokens[W + K:W + K + 3 * E])
        in_bytes = 8 * (B + 1) + 4 * B + 4 * max(max_tok, 1)
        d_in = torch.empty(in_bytes, dtype=torch.uint8, device=dev)
        h_packed = torch.empty(out["packed"].numel(), dtype=torch.uint8).pin_memory()
        h_out = store.unpack_outputs(h_packed, B)                # host views of the drafts

        def views(buf):
            return (buf[:8 * (B + 1)].view(torch.int64), buf[8 * (B + 1):8 * (B + 1) + 4 * B].view(torch.int32),
                    buf[8 * (B + 1) + 4 * B:].view(torch.int32))

        s_off, s_slots, s_tok = views(d_in)

        def run_e2e(mode, base):
            h_in, n_tok = [], []
            for k in range(E):
                o, t = steps.offsets[base + k], steps.tokens[base + k]
                hb = torch.empty(in_bytes, dtype=torch.uint8).pin_memory()
                ho, hs, ht = views(hb)
                ho.copy_(torch.as_tensor(o))
                hs.copy_(torch.arange(B, dtype=torch.int32))
                ht[:t.size].copy_(torch.as_tensor(t))
                h_in.append(hb)
                n_tok.append(int(t.size))
            moved = [0, 0]
            # the calls are bound to their buffers once (bind_step), as a serving loop would do
            if mode == "direct":
                calls = []
                for k in range(E):
                    ho, hs, ht = views(h_in[k])
                    calls.append(store.bind_step(hs, ho, ht, c.max_pattern, c.alpha, c.max_spec, 0, None, h_out))
            else:
                call = store.bind_step(s_slots, s_off, s_tok, c.max_pattern, c.alpha, c.max_spec, 0, None,
                                       out if mode == "copies" else h_out)
                calls = [call] * E

            def one(k):
                nb = 8 * (B + 1) + 4 * B + 4 * n_tok[k]
                if mode != "direct":
                    d_in[:nb].copy_(h_in[k][:nb], non_blocking=True)
                calls[k]()
                if mode == "copies":
                    h_packed.copy_(out["packed"], non_blocking=True)
                torch.cuda.synchronize()
                moved[0] += nb
                moved[1] += h_packed.numel()

            for k in range(We):
                one(k)
            moved[0] = moved[1] = 0
            if world > 1:
                dist.barrier()
            secs = 0.0
            for k in range(We, E):
                flush.zero_()
                torch.cuda.synchronize()                         # the flush is over before the step's clock starts
                t0 = time.perf_counter()
                one(k)                                           # ends with a synchronize: the drafts are on the host
                secs += time.perf_counter() - t0
            secs = sharding.max_over_ranks(secs, dev)
            return {"value": B * world * Ke / secs, "unit": UNIT, "h2d_bytes_per_step": moved[0] // Ke,
                    "d2h_bytes_per_step": moved[1] // Ke, "ms_per_step": secs / Ke * 1e3,
                    "transfer": {"copies": "one cudaMemcpyAsync each way around the call",
                                 "direct": "pinned host buffers passed to the call; the kernel reads and writes them",
                                 "direct_out": "inputs by cudaMemcpyAsync; the kernel writes the drafts to the pinned "
                                               "host buffer"}[mode]}

        runs = [run_e2e(mode, W + K + j * E) for j, mode in enumerate(("copies", "direct", "direct_out"))]
        runs.sort(key=lambda r: -r["value"])
        e2e, e2e_other = runs[0], runs[1:]

    # ---- the same work as two calls (sd_append, then sd_speculate), for the breakdown
    app_ms, spec_ms = [], []
    for k in range(K2):
        flush.zero_()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        store.append(slots, d_off2[k], d_tok2[k])
        e1.record()
        store.speculate(slots, c.max_pattern, c.alpha, c.max_spec, 0, None, out)
        e2.record()
        torch.cuda.synchronize()
        app_ms.append(e0.elapsed_time(e1)); spec_ms.append(e1.elapsed_time(e2))
    clocks = sampler.stop() if rank == 0 else None      # sampled from warm-up to the end of the e2e loop

    # ---- CPU oracle beside it (rank 0, one GPU): lock-step replay, sampled steps timed and compared
    cpu_baseline = None
    roofline = None
    extra = {}
    if n_samp:
        import oracle
        thr = oracle_threads(B)
        t0 = time.perf_counter()
        ref = oracle.SuffixOracle(c.depth_cap, B)
        ref.global_build(w.corpus(), w.corpus_offsets())
        ref.slot_append_batch(list(range(B)), prompts, n_threads=thr)
        setup_s = time.perf_counter() - t0
        o_times, desc, adds, upd, ctrees, ok = [], [], [], [], [], True
        for k in range(max(sample_steps) + 1):
            u0 = sum(ref.slot_updates(i) for i in range(B)) if k in sample_steps else 0
            t0 = time.perf_counter()
            ref.slot_append_batch(list(range(B)), steps.lists[k], n_threads=thr)
            if k in sample_steps:
                r = ref.speculate(list(range(B)), c.max_pattern, c.alpha, c.max_spec, n_threads=thr)
            if k in sample_steps:
                o_times.append(time.perf_counter() - t0)
                desc.append(int(r["visited"][:, 0].sum()))
                adds.append(int(r["visited"][:, 1].sum()))
                ctrees.append(int(r["visited"][:, 2].sum()))
                upd.append(sum(ref.slot_updates(i) for i in range(B)) - u0)
                g = {n: t.cpu().numpy() for n, t in saved[k].items()}
                for n in ("n_draft", "tokens", "parents", "positions", "chosen_tree", "chosen_p"):
                    ok = ok and np.array_equal(g[n], r[n])
                ok = ok and np.array_equal(g["mask"].view(np.uint32), r["mask"])
                ok = ok and np.array_equal(g["score"].view(np.int64), r["score"].view(np.int64))
        o_step = statistics.mean(o_times)
        cpu_baseline = {"value": B / o_step, "unit": UNIT, "cores": thr, "kind": "oracle",
                        "sample": f"{len(sample_steps)} of the {K} timed steps (all {B} requests each), "
                                  f"{sum(o_times):.1f} s wall on {thr} threads; setup {setup_s:.0f} s untimed"}
        visits = statistics.mean(d + a for d, a in zip(desc, adds))
        # necessary bytes of one launch: what the speculation must read and write (a 32-byte
        # look per node on a match walk, 64 per node added to a draft tree, the outputs) plus
        # what the append must (every node update reads and writes one 16-byte entry, every
        # token is written to the text)
        spec_bytes = statistics.mean(32 * d + 64 * a for d, a in zip(desc, adds)) + B * OUT_BYTES_PER_REQ
        app_bytes = statistics.mean(upd) * APPEND_BYTES_PER_UPDATE + 4 * float(np.mean([t.size for t in steps.tokens[W:W + K]]))
        alg_bytes = spec_bytes + app_bytes
        peak, which = measured_peak()
        step_s = statistics.mean(tot_ms) / 1e3                # the whole launch: append + speculate
        achieved = alg_bytes / step_s / 1e9
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": dram_traffic() if c.name == "large_batch" and not args.small else None,
                    "peak_source": which, "kernel": STEP_KERNEL,
                    "algorithmic_bytes_per_launch": alg_bytes,
                    "append_bytes_per_launch": app_bytes, "speculate_bytes_per_launch": spec_bytes,
                    "frac_of_nominal_8_TBs": achieved / 8000.0}
        if spec_ms:
            sp = spec_bytes / (statistics.mean(spec_ms) / 1e3) / 1e9
            roofline["speculate_only"] = {"achieved": sp, "frac": sp / peak,
                                          "note": "sd_speculate alone (two-call form), its own necessary bytes"}
        extra = {"parity_vs_oracle": "bit-exact" if ok else "MISMATCH", "parity_steps": len(sample_steps),
                 "candidate_trees_per_step": statistics.mean(ctrees),
                 "candidate_trees_per_s": statistics.mean(ctrees) * world / (ms_per_step / 1e3),
                 "nodes_visited_per_step": visits,
                 "nodes_visited_per_s": visits * world / (ms_per_step / 1e3)}
        ref.close()

    if rank == 0:
        st = store.stats()
        line = {
            "metric": METRIC.format(B=B), "value": B * world / (ms_per_step / 1e3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32 trees, f64 scores", "data": "synthetic",
            "config": config_dict(c, args),
            "step_us": {"mean": statistics.mean(tot_ms) * 1e3, "p50": statistics.median(tot_ms) * 1e3,
                        "max": max(tot_ms) * 1e3},
            "two_calls": {"steps": K2, "append_us": statistics.mean(app_ms) * 1e3 if app_ms else None,
                          "speculate_us": statistics.mean(spec_ms) * 1e3 if spec_ms else None},
            "tokens_appended_per_step": float(np.mean([t.size for t in steps.tokens[W:W + K]])),
            "build_ms": build_ms, "prompt_build_ms": prompt_ms, "global_nodes": st["global_nodes"],
            "device_bytes": st["device_bytes"], "wall_ms_timed_region": wall_ms,
            "gpu_launches": K, "e2e": e2e, "e2e_other_transfer": e2e_other, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "clocks": clocks,
        }
        line.update(extra)
        print(json.dumps(line), flush=True)
    store.free()
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
def run_sweep(args):
    """Memory, update time per token and look-up time per speculated token against the size of
    the global tree: the quantities of the paper's scalability table (appendix "Scalability and
    Memory Overhead"), on synthetic corpora of the headline workload's kind."""
    import torch

    import paper_2411_04975_b200 as sfx

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    K, W = min(args.steps, 30), 3
    rows = []
    for n_seqs in (512, 1024, 2048, 4096, 8192, 16384, 26368):     # the last row: 27.0 M tokens, the paper's first row
        w = get_workload("large_batch", n_seqs=n_seqs)
        c = w.cfg
        B = c.batch
        prompts = [w.prompt(i) for i in range(B)]
        steps = StepInputs(w, 0, B, W + K, prompts)
        corpus = torch.as_tensor(w.corpus(), device=dev)
        offsets = torch.as_tensor(w.corpus_offsets(), device=dev)
        build_ms = float("inf")
        for attempt in range(2):                                 # the first build also pays for fresh device allocations
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            store = sfx.SuffixStore(corpus, offsets, vocab=c.vocab, depth_cap=c.depth_cap, max_requests=B,
                                    max_req_tokens=c.prompt_len + steps.max_total + 8, max_spec_cap=c.max_spec)
            torch.cuda.synchronize()
            build_ms = min(build_ms, (time.perf_counter() - t0) * 1e3)
            if attempt == 0:
                store.free()
        st = store.stats()
        poff = np.zeros(B + 1, dtype=np.int64)
        poff[1:] = np.cumsum([len(p) for p in prompts])
        store.build_requests(np.arange(B, dtype=np.int32), poff, torch.as_tensor(np.concatenate(prompts), device=dev))
        slots = torch.arange(B, dtype=torch.int32, device=dev)
        out = store.alloc_outputs(B)
        flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
        d_off = [torch.as_tensor(o, device=dev) for o in steps.offsets]
        d_tok = [torch.as_tensor(t, device=dev) for t in steps.tokens]
        spec, app, drafts, toks = [], [], 0, 0
        for k in range(W + K):
            flush.zero_()
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record()
            store.speculate(slots, c.max_pattern, c.alpha, c.max_spec, 0, None, out)
            e1.record()
            store.append(slots, d_off[k], d_tok[k])
            e2.record()
            torch.cuda.synchronize()
            if k >= W:
                spec.append(e0.elapsed_time(e1)); app.append(e1.elapsed_time(e2))
                drafts += int(out["n_draft"].sum().item()); toks += int(d_tok[k].numel())
        n_tok = n_seqs * c.seq_len
        oracle_col = oracle_sweep_row(w, prompts, steps) if args.sweep_oracle else None
        rows.append({"oracle": oracle_col, "entries": n_seqs, "tokens": n_tok, "global_nodes": st["global_nodes"],
                     "global_tree_MB": st["global_pool_used"] * 16 / 1e6, "bytes_per_token": st["global_pool_used"] * 16 / n_tok,
                     "offline_build_ms": build_ms, "offline_update_us_per_token": build_ms * 1e3 / n_tok,
                     "online_update_us_per_token": sum(app) * 1e3 / toks,
                     "lookup_us_per_speculated_token": sum(spec) * 1e3 / max(drafts, 1),
                     "speculate_us_per_step": statistics.mean(spec) * 1e3, "draft_tokens_per_step": drafts / K})
        store.free()
        del corpus, offsets, flush
        torch.cuda.empty_cache()
    print(json.dumps({"metric": "scalability sweep (batch 256, 4,096-token prompts, one B200)", "rows": rows}), flush=True)


def oracle_sweep_row(w, prompts, steps, n_req=16, n_steps=3):
    """The CPU oracle on the same corpus, one thread (the paper's table is per-token CPU time):
    update time per token of the global build, look-up time per speculated token and online
    update time per token over `n_req` requests and `n_steps` decode steps."""
    import oracle
    import psutil
    c = w.cfg
    n_tok = c.n_seqs * c.seq_len
    need = 160 * 10 * n_tok                                       # about 10 nodes per token, 160 B per pointer-trie node
    if psutil.virtual_memory().available < 1.5 * need:
        return {"skipped": f"host memory: about {need / 1e9:.0f} GB needed for the pointer trie"}
    ref = oracle.SuffixOracle(c.depth_cap, n_req)
    t0 = time.perf_counter()
    ref.global_build(w.corpus(), w.corpus_offsets())
    build_s = time.perf_counter() - t0
    ref.slot_append_batch(list(range(n_req)), prompts[:n_req], n_threads=1)
    spec_s, app_s, drafts, toks = 0.0, 0.0, 0, 0
    for k in range(n_steps):
        t0 = time.perf_counter()
        r = ref.speculate(list(range(n_req)), c.max_pattern, c.alpha, c.max_spec, n_threads=1)
        t1 = time.perf_counter()
        ref.slot_append_batch(list(range(n_req)), steps.lists[k][:n_req], n_threads=1)
        t2 = time.perf_counter()
        spec_s += t1 - t0; app_s += t2 - t1
        drafts += int(r["n_draft"].sum()); toks += sum(len(x) for x in steps.lists[k][:n_req])
    ref.close()
    return {"threads": 1, "offline_update_us_per_token": build_s * 1e6 / n_tok,
            "online_update_us_per_token": app_s * 1e6 / max(toks, 1),
            "lookup_us_per_speculated_token": spec_s * 1e6 / max(drafts, 1),
            "sample": f"{n_req} requests x {n_steps} steps"}


# --------------------------------------------------------------------------------------------
def run_closed_loop(args):
    """The closed-loop workload: speculate -> simulated verification against the hidden continuation ->
    append accepted + bonus tokens; finished outputs go into the global tree, their slots are
    refilled.  Reports mean accepted length and steps/s (one GPU)."""
    import torch

    import paper_2411_04975_b200 as sfx
    from workload.closed_loop import ClosedLoop

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = make_workload(args)
    c = w.cfg
    B = c.batch
    K = args.steps if args.steps != 100 else (c.steps or 1000)
    store = sfx.SuffixStore(torch.as_tensor(w.corpus(), device=dev), torch.as_tensor(w.corpus_offsets(), device=dev),
                            vocab=c.vocab, depth_cap=c.depth_cap, max_requests=B,
                            max_req_tokens=c.prompt_len + c.out_len_hi + 8, max_spec_cap=c.max_spec)
    ref = None
    if args.closed_loop_oracle:
        import oracle
        ref = oracle.SuffixOracle(c.depth_cap, B)
        ref.global_build(w.corpus(), w.corpus_offsets())
    loop = ClosedLoop(w, B)
    slots_all = torch.arange(B, dtype=torch.int32, device=dev)
    out = store.alloc_outputs(B)

    side = torch.cuda.Stream(device=dev)

    def prepare(items):
        """Host side of an append: device tensors of the items, split into new requests (batched
        sort-based build) and everything else (sd_append).  Done before the timed events: the
        device-timed figures start with the inputs resident in HBM."""
        sl, lists, reset = items
        new = [i for i in range(len(sl)) if sl[i] >= 0 and reset[i]]
        skip = set(new)
        keep = [i for i in range(len(sl)) if i not in skip]
        prep = {"keep": None, "new": None, "items": items, "new_idx": new, "keep_idx": keep}
        if keep:
            ksl, klists, kreset = [sl[i] for i in keep], [lists[i] for i in keep], [reset[i] for i in keep]
            off = np.zeros(len(ksl) + 1, dtype=np.int64)
            off[1:] = np.cumsum([len(x) for x in klists])
            flat = np.concatenate(klists).astype(np.int32) if off[-1] else np.zeros(0, dtype=np.int32)
            prep["keep"] = (torch.as_tensor(np.asarray(ksl, dtype=np.int32), device=dev), torch.as_tensor(off, device=dev),
                            torch.as_tensor(flat, device=dev) if flat.size else torch.zeros(0, dtype=torch.int32, device=dev),
                            torch.as_tensor(np.asarray(kreset, dtype=np.uint8), device=dev))
            prep["global_tokens"] = sum(len(klists[i]) for i in range(len(ksl)) if ksl[i] < 0)
        if new:
            noff = np.zeros(len(new) + 1, dtype=np.int64)
            noff[1:] = np.cumsum([len(lists[i]) for i in new])
            toks_new = torch.as_tensor(np.concatenate([lists[i] for i in new]).astype(np.int32), device=dev)
            prep["new"] = ([sl[i] for i in new], noff, toks_new)
        return prep

    def enqueue(prep):
        """sd_append for the accepted tokens and the finished outputs; new requests are built
        meanwhile on a side stream (they touch other slots)."""
        sl, lists, reset = prep["items"]
        ev_pre = torch.cuda.Event()
        ev_pre.record()
        if prep["keep"] is not None:
            ka, kb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ka.record()
            store.append(*prep["keep"])
            kb.record()
            kernel_ev.append((ka, kb, prep["global_tokens"]))
        if prep["new"] is not None:
            nsl, noff, toks_new = prep["new"]
            ev_a, ev_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            refill_ev.append((ev_a, ev_b, int(noff[-1])))
            with torch.cuda.stream(side):
                side.wait_event(ev_pre)                          # not for the append enqueued just now
                ev_a.record()
                store.build_requests(nsl, noff, toks_new)
                ev_b.record()
            torch.cuda.current_stream().wait_stream(side)
        if ref is not None:
            for i in prep["keep_idx"]:
                if sl[i] < 0:
                    ref.global_insert(lists[i])
                elif reset[i]:
                    ref.slot_reset(sl[i])
            idx = [i for i in prep["keep_idx"] if sl[i] >= 0]
            ref.slot_append_batch([sl[i] for i in idx], [lists[i] for i in idx], n_threads=oracle_threads(B))
            for i in prep["new_idx"]:
                ref.slot_reset(sl[i])
            ref.slot_append_batch([sl[i] for i in prep["new_idx"]], [lists[i] for i in prep["new_idx"]],
                                  n_threads=oracle_threads(B))

    def append(items):
        enqueue(prepare(items))

    refill_ev, kernel_ev = [], []
    append(loop.start())
    torch.cuda.synchronize()
    refill_ev.clear()
    kernel_ev.clear()
    spec_ms, app_ms, ok = [], [], True
    Wc = max(args.warmup, 3)                                     # untimed first steps (first launches load the kernels)
    t_wall = time.perf_counter()
    for k in range(Wc + K):
        if k == Wc:
            refill_ev.clear()
            kernel_ev.clear()
            t_wall = time.perf_counter()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        store.speculate(slots_all, c.max_pattern, c.alpha, c.max_spec, 0, None, out)
        e1.record()
        host = {n: out[n].cpu().numpy() for n in ("n_draft", "tokens", "parents")}
        if ref is not None:
            r = ref.speculate(list(range(B)), c.max_pattern, c.alpha, c.max_spec, n_threads=oracle_threads(B))
            g = {n: t.cpu().numpy() for n, t in out.items()}
            for n in ("n_draft", "tokens", "parents", "positions", "chosen_tree", "chosen_p"):
                ok = ok and np.array_equal(g[n], r[n])
            ok = ok and np.array_equal(g["score"].view(np.int64), r["score"].view(np.int64))
        prep = prepare(loop.advance(host))
        e1b = torch.cuda.Event(enable_timing=True)
        e1b.record()
        enqueue(prep)
        e2.record()
        torch.cuda.synchronize()
        if k >= Wc:
            spec_ms.append(e0.elapsed_time(e1))
            app_ms.append(e1b.elapsed_time(e2))
    wall = time.perf_counter() - t_wall
    st = store.stats()
    summ = loop.summary()
    gpu_s = (sum(spec_ms) + sum(app_ms)) / 1e3
    line = {"metric": "closed-loop decode simulation: steps/s (GPU time of sd_speculate + sd_append) and mean accepted length",
            "value": K / gpu_s, "unit": "steps/s", "n_gpus": 1, "steps": K, "warmup": Wc,
            "ms_per_step": gpu_s / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32 trees, f64 scores", "data": "synthetic",
            "config": {"workload": c.name + (" (small)" if args.small else ""), "batch_per_gpu": B,
                       "global_tokens": int(c.n_seqs * c.seq_len), "prompt_len": c.prompt_len, "vocab": c.vocab,
                       "D": c.depth_cap, "P": c.max_pattern, "alpha": c.alpha, "max_spec": c.max_spec},
            "speculate_us": {"mean": statistics.mean(spec_ms) * 1e3, "p50": statistics.median(spec_ms) * 1e3,
                             "p90": float(np.percentile(spec_ms, 90)) * 1e3, "p99": float(np.percentile(spec_ms, 99)) * 1e3,
                             "max": max(spec_ms) * 1e3},
            "append_us": {"mean": statistics.mean(app_ms) * 1e3, "p50": statistics.median(app_ms) * 1e3,
                          "p90": float(np.percentile(app_ms, 90)) * 1e3, "max": max(app_ms) * 1e3},
            "wall_steps_per_s_with_host_verifier": K / wall, "gpu_launches": 2 * K,
            "global_nodes_end": st["global_nodes"], "global_tokens_end": st["global_tokens"],
            "global_status": st["global_status"]}
    if refill_ev:
        r_ms = [a.elapsed_time(b) for a, b, _ in refill_ev]
        line["refill"] = {"calls": len(r_ms), "mean_us": statistics.mean(r_ms) * 1e3, "max_us": max(r_ms) * 1e3,
                          "mean_tokens": statistics.mean(t for _, _, t in refill_ev),
                          "total_ms": sum(r_ms)}
    k_ms = [a.elapsed_time(b) for a, b, _ in kernel_ev]
    g_tok = [t for _, _, t in kernel_ev]
    line["append_kernel"] = {"mean_us": statistics.mean(k_ms) * 1e3, "p50_us": statistics.median(k_ms) * 1e3,
                             "max_us": max(k_ms) * 1e3, "global_tokens_per_call": statistics.mean(g_tok),
                             "us_per_global_token": sum(k_ms) * 1e3 / max(sum(g_tok), 1)}
    line.update(summ)
    if ref is not None:
        line["parity_vs_oracle"] = "bit-exact" if ok else "MISMATCH"
    print(json.dumps(line), flush=True)
    store.free()


# --------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle as it stands, on the host cores, same metric and config.
    Each step is a bounded sample of the workload's requests."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    w = make_workload(args)
    c = w.cfg
    B, K, W = c.batch, args.steps, args.warmup
    thr = oracle_threads(B)
    prompts = [w.prompt(i) for i in range(B)]
    steps = StepInputs(w, 0, B, W + K, prompts)
    ref = oracle.SuffixOracle(c.depth_cap, B)
    ref.global_build(w.corpus(), w.corpus_offsets())
    ref.slot_append_batch(list(range(B)), prompts, n_threads=thr)
    sample = list(range(B))
    budget_s = 150.0

    def step(k):
        ref.speculate(sample, c.max_pattern, c.alpha, c.max_spec, n_threads=thr)
        ref.slot_append_batch(sample, [steps.lists[k][i] for i in sample], n_threads=thr)

    t0 = time.perf_counter()
    step(0) if W > 0 else None
    t1 = time.perf_counter() - t0
    if W > 0 and t1 * (K + W) > budget_s:
        keep = max(8, int(B * budget_s / (t1 * (K + W))))
        sample = list(range(min(B, keep)))
    for k in range(1, W):
        step(k)
    t0 = time.perf_counter()
    for k in range(W, W + K):
        step(k)
    dt = time.perf_counter() - t0
    value = len(sample) * K / dt
    line = {"impl": "reference", "metric": METRIC.format(B=B), "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": dt / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32 trees, f64 scores", "data": "synthetic",
            "config": config_dict(c, args),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle",
                             "sample": f"{len(sample)} of {B} requests per step, {K} steps"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def spawn_ranks(args):
    """`--gpus N` without a launcher around it: start the N ranks here (one process per GPU)."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


if __name__ == "__main__":
    a = parse()
    if a.gpus > 1 and "WORLD_SIZE" not in os.environ and a.impl == "ours":
        sys.exit(spawn_ranks(a))
    if a.impl == "reference":
        run_reference(a)
    elif a.sweep:
        run_sweep(a)
    elif a.config == "closed_loop":
        run_closed_loop(a)
    else:
        run_ours(a)

#!/usr/bin/env python
"""Benchmark of the KVMem recall step (select + materialize + attend) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1m] [--impl native|reference]

One "step" is one pass of the whole hot path over one seeded query set: block scoring through
the Mean-K index, selection under the budget, execution-view assembly, GQA decode attention.
The history stays resident in HBM; the 16 query sets of the workload are cycled.  Rank 0 prints
ONE JSON line.  With N > 1 (launched by torch.distributed.run) every rank owns an independent
session replica on its own GPU (the path shards by session, no collective on the data path);
the timed region is bracketed by a barrier and the maximum over ranks is reported.

``--impl reference`` times the CPU oracle, as it stands, on the host cores, on a bounded sample
of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from kvmem_workloads import CONFIGS, kv_blocks, make_queries, page_table, select_params  # noqa: E402

METRIC = "select+materialize+attend steps/s"
UNIT = "steps/s"
KERNELS_PER_STEP = 6      # score_logits, score_finish, topk, gather, attend_split, attend_merge (5 when fused)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


def measured_tensor_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"tflops": 1590.0, "source": "fallback"}


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the dominant kernel on the 1M workload.
# These are constants taken from earlier ncu captures of the same kernels, not measured in the run that prints them
# (a bench run is never made under a profiler); the line says so in "traffic_source".
GATHER_TRAFFIC = {"1m": 2099369984, "chunk512": 2098579520}       # gather_bulk_kernel
# attend_split_kernel<1>, mean of six launches (128k: 134 MB read + 79 MB written; the rest of the view is still in L2 when the kernel ends)
FUSED_TRAFFIC = {"1m": 2099720917, "128k": 212966016, "batch8": 4250897493}
ROPE_FUSED_TRAFFIC = {"1m": 2098100000}   # attend_split_kernel<5> (in-block key layout)
ROPE_RAW_FUSED_TRAFFIC = {"1m": 2105828736}   # attend_split_kernel<6> (raw keys, one pass), mean of two launches
ROPE_GATHER_TRAFFIC = {"1m": 2270831360}  # gather_rope_kernel, mean of two launches
TRAFFIC_SOURCE = ("constant from an earlier ncu capture of this kernel on this workload (one launch, "
                  "dram__bytes_read.sum + dram__bytes_write.sum); not measured in this run")


def algorithmic_bytes(spec, k):
    """Bytes the method must move per step (per session): index read + view read/write + view read."""
    view = 2 * k * spec.block_tokens * spec.n_layers * spec.n_kv_heads * spec.head_dim * 2       # K and V, bf16
    index = spec.n_blocks * spec.n_layers * spec.n_kv_heads * spec.head_dim * 2
    return {"index": index, "gather": 2 * view, "attend": view if spec.attend else 0,
            "total": index + 2 * view + (view if spec.attend else 0)}


# ----------------------------------------------------------------------------- clocks

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index
        self.t_start = self.t_stop = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def window(self, t0, t1):
        self.t_start, self.t_stop = t0, t1

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for t, line in self.rows:
            if self.t_start is not None and not (self.t_start <= t <= self.t_stop + 0.05):
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- native arm

ROPE_THETA = 1.0e6


def rope_window(spec):
    """Positions the rotary table must cover: the native window plus the step's query tokens."""
    return spec.max_view_tokens + 64


def fill_pool(spec, device, seed_shift=0, rope=False, in_block=False, fp8_pages=False):
    from paper_2609_04852_b200 import Pool
    spec = spec.with_(seed=spec.seed + seed_shift)
    pool = Pool(spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.block_tokens,
                spec.n_sessions, spec.n_sessions * spec.n_blocks, spec.n_blocks, device.index,
                rope_window(spec) if rope else 0, ROPE_THETA if rope else 0.0, rope_in_block_keys=in_block, fp8_pages=fp8_pages)
    tables = page_table(spec)
    B = spec.block_tokens
    for s in range(spec.n_sessions):
        for b0 in range(0, spec.n_blocks, 1024):
            b1 = min(spec.n_blocks, b0 + 1024)
            K, V = kv_blocks(spec, s, b0, b1, device)
            if rope:    # the keys are taken as encoded at the positions they had inside their execution window
                pos0 = [(b * B) % (spec.max_view_tokens - B) for b in range(b0, b1)]
                pool.append_blocks_rope(s, K, V, pos0, tables[s, b0:b1].tolist())
                continue
            pool.append_blocks(s, K, V, tables[s, b0:b1].tolist())
        torch.cuda.synchronize(device)
    return pool, spec


def run_native(args):
    import torch.distributed as dist
    from paper_2609_04852_b200 import SelectParams
    from paper_2609_04852_b200.sharding import max_over_ranks, whole_job_rate

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: a run never silently uses fewer GPUs than asked for")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    for opt in args.option:
        from paper_2609_04852_b200 import set_option
        name, _, value = opt.partition("=")
        set_option(name, int(value))
    if world > 1 and not dist.is_initialized():
        # NCCL's own log stays on (on stderr: stdout carries rank 0's one JSON line): a multi-GPU run then shows its ranks,
        # transports and whether in-switch reduction was used
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=device)

    base = CONFIGS[args.workload]
    if args.blocks:      # a shrunken history of the same recipe: the small case for ncu captures
        f = args.blocks / base.n_blocks
        if base.name == "table4":     # the workspace sweep keeps the 64K view and grows only the history
            base = base.with_(name=f"{base.name}@{args.blocks}", n_blocks=args.blocks)
        else:
            base = base.with_(name=f"{base.name}@{args.blocks}", n_blocks=args.blocks,
                              n_planted=max(1, int(base.n_planted * f)), budget_blocks=max(1, int(base.budget_blocks * f)))
    pool, spec = fill_pool(base, device, seed_shift=1000 * rank, rope=args.rope, in_block=args.in_block, fp8_pages=args.fp8_pages)     # one independent replica per rank
    ns, M, B = spec.n_sessions, spec.n_q_tokens, spec.block_tokens
    prm = SelectParams(**select_params(spec))
    from paper_2609_04852_b200 import budget_blocks
    k = budget_blocks(prm, B, spec.n_blocks)
    cap = k * B
    qsets = [make_queries(spec, i) for i in range(spec.n_query_sets)]
    q_dev = [q.to(device) for q in qsets]
    q_pin = [q.pin_memory() for q in qsets]
    sel = torch.zeros(ns, k, dtype=torch.int32, device=device)
    n_sel = torch.zeros(ns, dtype=torch.int32, device=device)
    view = pool.new_view(ns, cap)
    out, lse = pool.new_outputs(ns, M)
    out_pin = torch.empty(out.shape, dtype=torch.float32).pin_memory()
    lse_pin = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device) if args.flush_l2 else None
    stream = torch.cuda.current_stream(device)
    fused = spec.attend and not args.unfused and not args.rope and not args.fp8
    if args.fp8:
        if not spec.attend:
            raise SystemExit("--fp8 is measured on the attend workloads")
        k8, v8t = pool.new_view_fp8(ns, cap)

    if args.rope:
        if not spec.attend or spec.n_sessions != 1:
            raise SystemExit("--rope is measured on the single-session attend workloads")
        H, d = spec.n_q_heads, spec.head_dim
        q_pos = torch.arange(k * B, k * B + M, dtype=torch.int32, device=device)     # the query sits right after the view
        q_raw = torch.empty_like(q_dev[0])

    def step(i, ev=None):
        q = q_dev[i % len(q_dev)]
        if args.rope:
            # the model's query carries RoPE: remove it for retrieval (Sec. 4.3), keep it for attention
            pool.rope_rotate(q.view(M, H, d), q_pos, out=q_raw.view(M, H, d), inverse=True)
            pool.select(q_raw, prm, sel, n_sel)
            if ev is not None:
                ev[0].record(stream)
            if args.paged and args.fp8_pages:       # FP8 repository of in-block-rotated keys: query rotated back per block
                pool.paged_attend_fp8_rope(q, sel, n_sel, out, lse, 0)
                if ev is not None:
                    ev[1].record(stream)
                    ev[2].record(stream)
                return
            if args.fp8:        # position-consistent FP8 view from bf16 pages: rotate, quantise, then FP8 attention
                pool.materialize_fp8_rope(sel, n_sel, k8, v8t, 0)
                if ev is not None:
                    ev[1].record(stream)
                pool.view_attend_fp8(q, k8, v8t, n_sel, out, lse)
                if ev is not None:
                    ev[2].record(stream)
                return
            if args.paged:      # copy-free: raw key tiles are RoPE'd in shared memory on their way to the tensor cores
                pool.paged_attend_rope(q, sel, n_sel, out, lse, 0)
                if ev is not None:
                    ev[1].record(stream)
                    ev[2].record(stream)
                return
            if not args.unfused:  # one pass: K rotated on its way through the SM (by block position on the in-block layout, per key on raw keys), stored and attended over
                pool.materialize_attend_rope(q, sel, n_sel, view, out, lse, 0)
                if ev is not None:
                    ev[1].record(stream)
                    ev[2].record(stream)
                return
            pool.materialize_rope(sel, n_sel, view, 0)
            if ev is not None:
                ev[1].record(stream)
            pool.view_attend(q, view, n_sel, out, lse)
            if ev is not None:
                ev[2].record(stream)
            return
        pool.select(q, prm, sel, n_sel)
        if ev is not None:
            ev[0].record(stream)
        if args.fp8_pages and args.paged:       # FP8 repository, copy-free: attention straight over the 1-byte pages
            pool.paged_attend_fp8(q, sel, n_sel, out, lse)
            if ev is not None:
                ev[1].record(stream)
                ev[2].record(stream)
            return
        if args.fp8 and not args.unfused:  # tiles (quantised on the way from bf16 pages) stored to the FP8 view while attended over, one pass
            pool.materialize_attend_fp8(q, sel, n_sel, k8, v8t, out, lse)
            if ev is not None:
                ev[1].record(stream)
                ev[2].record(stream)
            return
        if args.fp8:           # FP8 (E4M3) view: quantise while gathering (or copy the tiles of an FP8 repository), attend over half the bytes
            pool.materialize_fp8(sel, n_sel, k8, v8t)
            if ev is not None:
                ev[1].record(stream)
            pool.view_attend_fp8(q, k8, v8t, n_sel, out, lse)
            if ev is not None:
                ev[2].record(stream)
            return
        if args.paged:
            pool.paged_attend(q, sel, n_sel, out, lse)                  # copy-free view: no materialisation at all
            if ev is not None:
                ev[1].record(stream)
        elif fused:
            pool.materialize_attend(q, sel, n_sel, view, out, lse)      # one pass: view written while attended
            if ev is not None:
                ev[1].record(stream)
        else:
            pool.materialize(sel, n_sel, view)
            if ev is not None:
                ev[1].record(stream)
            if spec.attend:
                pool.view_attend(q, view, n_sel, out, lse)
        if ev is not None:
            ev[2].record(stream)

    def barrier():
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert pool.device_status() == 0, "device status word set during warm-up"
    assert int(n_sel.min()) == k, "selection did not fill the budget"

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)

    # ---- timed region: K steps, device-timed, inputs resident in HBM.  No event is recorded between the calls of a
    # step here: an event between two calls keeps the second kernel from launching programmatically behind the first
    # (about 15 us per step at 1M).  The per-stage times come from a second pass of K steps below.
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flush is not None:
        fb = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        fe = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    barrier()
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(K):
        if flush is not None:
            flush.fill_(i & 255)
            fb[i].record(stream)
        step(i)
        if flush is not None:
            fe[i].record(stream)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    total_ms = e0.elapsed_time(e1)
    if flush is not None:
        total_ms = sum(fb[i].elapsed_time(fe[i]) for i in range(K))          # the flush writes are not part of a step
    # ---- second pass of K steps with events after each call: stage times and the dominant kernel's launch duration
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    begins = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    barrier()
    for i in range(K):
        if flush is not None:
            flush.fill_(i & 255)
        begins[i].record(stream)
        step(i, marks[i])
    barrier()
    t_wall1 = time.time()
    step_ms = [begins[i].elapsed_time(marks[i][2]) for i in range(K)]
    sel_ms = [begins[i].elapsed_time(marks[i][0]) for i in range(K)]
    gat_ms = [marks[i][0].elapsed_time(marks[i][1]) for i in range(K)]
    att_ms = [marks[i][1].elapsed_time(marks[i][2]) for i in range(K)]
    sampler.window(t_wall0, t_wall1)
    assert pool.device_status() == 0, "device status word set during the timed region"

    # ---- end-to-end: query from pinned host memory, results read back to the host, every step
    Ke = min(K, 200)
    q_stage = torch.empty_like(q_dev[0])
    sel_pin = torch.empty(sel.shape, dtype=torch.int32).pin_memory()
    # the plain step goes through the library's host-buffer entry point, its arguments marshalled once as a decode loop would
    host_step = pool.host_step(q_pin[0].shape, prm, sel, n_sel, view, out_pin, lse_pin) if (spec.attend and not args.rope and not args.fp8) else None
    barrier()
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record(stream)
    for i in range(Ke):
        if args.rope:   # same position-consistent step, query from pinned host memory, results back to the host
            q_stage.copy_(q_pin[i % len(q_pin)], non_blocking=True)
            pool.rope_rotate(q_stage.view(M, H, d), q_pos, out=q_raw.view(M, H, d), inverse=True)
            pool.select(q_raw, prm, sel, n_sel)
            if args.paged and args.fp8_pages:
                pool.paged_attend_fp8_rope(q_stage, sel, n_sel, out, lse, 0)
            elif args.fp8:
                pool.materialize_fp8_rope(sel, n_sel, k8, v8t, 0)
                pool.view_attend_fp8(q_stage, k8, v8t, n_sel, out, lse)
            elif args.paged:
                pool.paged_attend_rope(q_stage, sel, n_sel, out, lse, 0)
            else:
                pool.materialize_attend_rope(q_stage, sel, n_sel, view, out, lse, 0)
            out_pin.copy_(out, non_blocking=True)
            lse_pin.copy_(lse, non_blocking=True)
            torch.cuda.synchronize(device)
        elif args.fp8:
            q_stage.copy_(q_pin[i % len(q_pin)], non_blocking=True)
            pool.select(q_stage, prm, sel, n_sel)
            if args.fp8_pages and args.paged:
                pool.paged_attend_fp8(q_stage, sel, n_sel, out, lse)
            elif not args.unfused:
                pool.materialize_attend_fp8(q_stage, sel, n_sel, k8, v8t, out, lse)
            else:
                pool.materialize_fp8(sel, n_sel, k8, v8t)
                pool.view_attend_fp8(q_stage, k8, v8t, n_sel, out, lse)
            out_pin.copy_(out, non_blocking=True)
            lse_pin.copy_(lse, non_blocking=True)
            torch.cuda.synchronize(device)
        elif spec.attend:
            host_step(q_pin[i % len(q_pin)])
        else:       # chunked scoring has no attend stage: host query in, selected ids out
            q_stage.copy_(q_pin[i % len(q_pin)], non_blocking=True)
            pool.select(q_stage, prm, sel, n_sel)
            pool.materialize(sel, n_sel, view)
            sel_pin.copy_(sel, non_blocking=True)
            torch.cuda.synchronize(device)
    ee1.record(stream)
    barrier()
    e2e_ms = ee0.elapsed_time(ee1)
    # keep sampling clocks long enough to see the load even when K is small
    if rank == 0 and (t_wall1 - t_wall0) < 0.5:
        t_wall0 = time.time()
        t_end = t_wall0 + 0.6
        i = 0
        while time.time() < t_end:
            step(i); i += 1
            if i % 50 == 0:
                torch.cuda.synchronize(device)
        torch.cuda.synchronize(device)
        sampler.window(t_wall0, time.time())
        clock_note = "timed region shorter than the sampling period: clocks sampled over an identical 0.6 s loop right after it"
    else:
        clock_note = "sampled during the timed region"

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device=device)     # slowest rank decides

    if rank == 0:
        clocks = sampler.stop()
        clocks["note"] = clock_note
        peaks = measured_peaks()
        ab = algorithmic_bytes(spec, k)
        med = statistics.median
        gather_s = (sum(gat_ms) / K) * 1e-3
        dom_bytes = ns * (ab["attend"] if args.paged else ab["gather"])    # paged: one read of the selected pages
        gather_gbs = dom_bytes / gather_s / 1e9
        # fused: every view byte is read once (from the pages) and written once; separate calls read it a second time
        one_pass = fused or (args.rope and not args.unfused and not args.paged)       # view written while attended
        step_bytes = ns * (ab["total"] - (ab["attend"] if one_pass else 0))
        if args.paged:
            step_bytes = ns * (ab["index"] + ab["attend"])
        step_gbs = world * K * step_bytes / (total_ms * 1e-3) / 1e9 / world      # per GPU
        rows = ns * M * spec.n_layers * spec.n_q_heads
        line = {
            "metric": METRIC, "value": whole_job_rate(K, world, total_ms), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded; shapes of the paper's agent workspaces)",
            "config": {"workload": f"{spec.name}: {ns} session(s) x {spec.n_blocks} blocks of {B} tokens "
                                   f"({spec.tokens} tokens history), {M} query token(s), {spec.n_q_heads}/{spec.n_kv_heads} heads, "
                                   f"d={spec.head_dim}, budget {k} blocks ({cap} view tokens)",
                       "history_tokens": spec.tokens, "view_tokens": cap, "query_sets": len(qsets),
                       "l2": "flushed between steps (256 MiB write)" if flush is not None else
                             "no flush: every step streams far more than the 126 MB L2" if step_bytes > 8 * (126 << 20) else
                             f"NO flush and {step_bytes / 1e6:.0f} MB per step against the 126 MB L2: partly L2-resident, "
                             "a warm-cache figure (--flush-l2 for the cold one)",
                       "parallelism": f"{world} independent session replica(s), one per GPU",
                       "calls": "kvmem_rope_rotate(q) + kvmem_select + kvmem_paged_attend_rope (copy-free, pages hold RoPE(k, in-block offset), "
                                "the query rotated back once per block)" if args.rope and args.paged and args.in_block else
                                "kvmem_rope_rotate(q) + kvmem_select + kvmem_paged_attend_rope (copy-free, keys RoPE'd in shared memory)"
                                if args.rope and args.paged else
                                "kvmem_rope_rotate(q) + kvmem_select + kvmem_materialize_attend_rope (one pass: K tiles rotated by their block "
                                "position in shared memory, stored and attended over)" if args.rope and args.in_block and not args.unfused else
                                "kvmem_rope_rotate(q) + kvmem_select + kvmem_materialize_attend_rope (one pass over raw keys: the attending warps rotate "
                                "their key fragments to the compact positions and hand them back for the store)" if args.rope and not args.unfused else
                                "kvmem_rope_rotate(q) + kvmem_select + kvmem_materialize_rope + kvmem_view_attend" if args.rope else
                                "kvmem_select + kvmem_paged_attend (NO materialize: copy-free view variant)" if args.paged else
                                "kvmem_select + kvmem_materialize_attend" if fused else
                                "kvmem_select + kvmem_materialize" + (" + kvmem_view_attend" if spec.attend else "")},
            "e2e": {"value": whole_job_rate(Ke, world, e2e_ms), "unit": UNIT, "steps": Ke,
                    "h2d_bytes_per_step": rows * spec.head_dim * 2,
                    "d2h_bytes_per_step": rows * spec.head_dim * 4 + rows * 4,
                    "api": "kvmem_recall_step_host through Pool.host_step (arguments marshalled once; pinned host query copied in, O and LSE written into the pinned host buffers by the step's last kernel, synchronous)"},
            "gpu_launches": K * (KERNELS_PER_STEP - (1 if one_pass or args.paged else 0) + (1 if args.rope else 0)),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "attend_split_kernel<4> + merge (kvmem_paged_attend_rope, in-block key layout)"
                                                   if args.rope and args.paged and args.in_block else
                                                   "attend_split_kernel<3> + merge (kvmem_paged_attend_rope)" if args.rope and args.paged else
                                                   "attend_split_kernel<5> + merge (kvmem_materialize_attend_rope: K rotated in shared memory, "
                                                   "view written while attended)" if args.rope and args.in_block and not args.unfused else
                                                   "attend_split_kernel<6> + merge (kvmem_materialize_attend_rope on raw keys: fragments rotated by the "
                                                   "attending warps, view written while attended)" if args.rope and not args.unfused else
                                                   "gather_rope_kernel (kvmem_materialize_rope)" if args.rope else
                                                   "attend_split_kernel<2> + merge (kvmem_paged_attend)" if args.paged else
                                                   "attend_split_kernel<1> + merge (kvmem_materialize_attend: view written while attended)"
                                                   if fused else "gather_bulk_kernel (kvmem_materialize)",
                         "achieved": gather_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gather_gbs / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                         "algorithmic_bytes_per_launch": dom_bytes, "avg_launch_ms": gather_s * 1e3,
                         "traffic": None if args.paged else ROPE_FUSED_TRAFFIC.get(base.name) if args.rope and args.in_block and not args.unfused else
                                    ROPE_RAW_FUSED_TRAFFIC.get(base.name) if args.rope and not args.unfused else
                                    ROPE_GATHER_TRAFFIC.get(base.name) if args.rope else
                                    FUSED_TRAFFIC.get(base.name) if fused else GATHER_TRAFFIC.get(base.name)},
            "step_hbm": {"algorithmic_bytes_per_step": step_bytes,
                         "accounting": "index + one read of the selected pages (copy-free view, nothing materialised)" if args.paged else
                                       "index + view read + view write (fused pass)" if one_pass else
                                       "index + gather read/write + attend read (separate calls)",
                         "bytes_if_separate_calls": ns * ab["total"], "achieved_gbs": step_gbs,
                         "frac_of_peak": step_gbs / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                         "nominal_peak_gbs": 8000.0},
            "stages_ms": {"select": med(sel_ms), "materialize": med(gat_ms), "attend": med(att_ms),
                          "step_median": med(step_ms), "step_min": min(step_ms),
                          "note": "from a second pass of the same K steps with an event after each call; value and ms_per_step "
                                  "come from the first pass, which records no event inside a step"},
        }
        if not spec.attend:
            # the chunked configuration is bounded by the tensor pipe: two passes of the 2*M*H*NB*d contraction.
            # The scoring kernels are timed alone through kvmem_score (kvmem_select adds the top-k kernel).
            flop_alg = 2.0 * ns * M * spec.n_layers * spec.n_q_heads * spec.n_blocks * spec.head_dim
            sc_buf = torch.zeros(ns, spec.n_blocks, dtype=torch.float32, device=device)
            for i in range(3):
                pool.score(q_dev[i % len(q_dev)], sc_buf)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(device)
            s0.record(stream)
            for i in range(50):
                pool.score(q_dev[i % len(q_dev)], sc_buf)
            s1.record(stream)
            torch.cuda.synchronize(device)
            sel_s = s0.elapsed_time(s1) / 50 * 1e-3
            tpeak = measured_tensor_peak()
            line["e2e"]["h2d_bytes_per_step"] = rows * spec.head_dim * 2
            line["e2e"]["d2h_bytes_per_step"] = ns * k * 4
            line["e2e"]["api"] = "pinned host query in, selected ids out, around kvmem_select + kvmem_materialize"
            line["gpu_launches"] = K * 6
            exe_tf, alg_tf = 2 * flop_alg / sel_s / 1e12, flop_alg / sel_s / 1e12
            line["roofline"] = {"bound": "tensor", "kernel": "score_chunk_rowstat_kernel + shift + score_chunk_colsum_kernel + finish (kvmem_score, timed alone over 50 calls)",
                                "achieved": exe_tf, "peak": tpeak["tflops"], "unit": "TFLOP/s",
                                "frac": exe_tf / tpeak["tflops"], "peak_source": f"of {tpeak['source']} (bf16 matmul burst)",
                                "frac_executed": exe_tf / tpeak["tflops"], "frac_algorithmic": alg_tf / tpeak["tflops"],
                                "frac_of_nominal_2250_executed": exe_tf / 2250.0, "frac_of_nominal_2250_algorithmic": alg_tf / 2250.0,
                                "compared_with_the_50_percent_target": "frac_executed: the exact softmax needs the row statistics before the column sums, so the "
                                "QK^T contraction is issued twice (2 x 2*M*H*NB*d flop) and that is the tensor-pipe work counted; on the contraction "
                                "counted once (frac_algorithmic) the target is not met",
                                "executed_flop_per_launch_pair": 2 * flop_alg, "algorithmic_flop": flop_alg,
                                "executed_tflops": exe_tf, "algorithmic_tflops": alg_tf, "avg_score_ms": sel_s * 1e3, "traffic": None}
        if not spec.attend and B != 64 and ns == 1:
            # The scaling workload has the paper's 32-token blocks.  Decode over the view it selects (4 query tokens:
            # 1 + 3 drafts) through the passes that read pages through the block table, each timed alone over 50 calls.
            spec4 = spec.with_(n_q_tokens=4)
            q4 = [make_queries(spec4, i).to(device) for i in range(4)]
            out4, lse4 = pool.new_outputs(ns, 4)
            view_bytes = ns * ab["gather"] // 2
            dec = {}
            for name, fn, nbytes in (("kvmem_materialize_attend", lambda qq: pool.materialize_attend(qq, sel, n_sel, view, out4, lse4), 2 * view_bytes),
                                     ("kvmem_paged_attend", lambda qq: pool.paged_attend(qq, sel, n_sel, out4, lse4), view_bytes)):
                for i in range(3):
                    fn(q4[i % 4])
                d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize(device)
                d0.record(stream)
                for i in range(50):
                    fn(q4[i % 4])
                d1.record(stream)
                torch.cuda.synchronize(device)
                us = d0.elapsed_time(d1) / 50 * 1e3
                dec[name] = {"us": us, "algorithmic_bytes": nbytes, "gbs": nbytes / (us * 1e-6) / 1e9,
                             "frac_of_peak": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
            assert pool.device_status() == 0
            line["decode_over_view"] = {"query_tokens": 4, "block_tokens": B, "view_tokens": cap, **dec}
        if args.host_index and spec.attend and ns == 1:
            # the memory-bounded variant: the index stays in pinned host memory and is streamed over PCIe in tiles
            idx_host = pool.index(0).cpu().contiguous().pin_memory()
            sc_buf = torch.zeros(spec.n_blocks, dtype=torch.float32, device=device)
            hres = {}
            for tile in (2048, 4096, 8192):
                for i in range(3):
                    pool.score_host_index(idx_host, spec.n_blocks, q_dev[i % len(q_dev)][0], sc_buf, tile)
                h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize(device)
                h0.record(stream)
                for i in range(20):
                    pool.score_host_index(idx_host, spec.n_blocks, q_dev[i % len(q_dev)][0], sc_buf, tile)
                h1.record(stream)
                torch.cuda.synchronize(device)
                ms = h0.elapsed_time(h1) / 20
                hres[str(tile)] = {"ms": ms, "h2d_gbs": idx_host.numel() * 2 / (ms * 1e-3) / 1e9}
            line["host_index_scoring"] = {"api": "kvmem_score_host_index", "index_bytes": idx_host.numel() * 2,
                                          "by_tile_blocks": hres}
        if args.fp8:
            # FP8 view: the gather reads the bf16 pages (2 B per element) and writes 1 B; attention reads 1 B
            g_bytes = ns * ab["gather"] * 3 // 4
            a_bytes = ns * ab["attend"] // 2
            g_s, a_s = med(gat_ms) * 1e-3, med(att_ms) * 1e-3
            line["config"]["calls"] = ("kvmem_rope_rotate(q) + kvmem_select + kvmem_materialize_fp8_rope + kvmem_view_attend_fp8 (position-consistent E4M3 view)"
                                       if args.rope else "kvmem_select + kvmem_materialize_fp8 + kvmem_view_attend_fp8 (E4M3 view, static scales 1.0)")
            line["dtype"] = "bf16 pages and query, E4M3 view, f16 tensor-core products, fp32 accumulation"
            one_pass_bf16 = not args.fp8_pages and not args.rope and not args.unfused
            if one_pass_bf16:       # bf16 pages quantised on their way to the view and to the tensor cores: no second read of the view
                a_bytes, a_s = 0, 1.0
                line["config"]["calls"] = ("kvmem_select + kvmem_materialize_attend_fp8 (bf16 repository: tiles quantised on the way, "
                                           "E4M3 view written while attended, static scales 1.0)")
            if args.fp8_pages:      # FP8 repository: the gather copies 1-byte tiles; --paged reads them in place
                g_bytes = ns * ab["gather"] // 2
                line["dtype"] = "E4M3 pages (quantised at append), bf16 query and index, f16 tensor-core products, fp32 accumulation"
                line["config"]["calls"] = ("kvmem_select + kvmem_paged_attend_fp8 (copy-free view over an FP8 repository)" if args.paged else
                                           "kvmem_select + kvmem_materialize_fp8 + kvmem_view_attend_fp8 over an FP8 repository")
                if args.paged:
                    g_bytes, a_bytes, a_s = a_bytes, 0, 1.0
                elif not args.unfused:
                    a_bytes, a_s = 0, 1.0
                    line["config"]["calls"] = "kvmem_select + kvmem_materialize_attend_fp8 (FP8 repository: view written while attended)"
            line["roofline"] = {"bound": "hbm", "kernel": "attend_fp8_split_kernel<paged> + merge (kvmem_paged_attend_fp8)" if args.fp8_pages and args.paged else
                                                           "attend_fp8_split_kernel<2> + merge (kvmem_materialize_attend_fp8)" if args.fp8_pages and not args.unfused else
                                                           "gather_fp8_pages_kernel (kvmem_materialize_fp8)" if args.fp8_pages else
                                                           "attend_fp8_split_kernel<4> + merge (kvmem_materialize_attend_fp8 over bf16 pages)" if one_pass_bf16 else
                                                           "gather_fp8_kernel (kvmem_materialize_fp8)", "achieved": g_bytes / g_s / 1e9,
                                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": g_bytes / g_s / 1e9 / peaks["hbm_gbs"],
                                "peak_source": f"of {peaks['source']}", "algorithmic_bytes_per_launch": g_bytes,
                                "avg_launch_ms": g_s * 1e3, "traffic": None}
            line["attend_roofline"] = {"kernel": "attend_fp8_split_kernel + merge (kvmem_view_attend_fp8)", "achieved_gbs": a_bytes / a_s / 1e9,
                                       "frac": a_bytes / a_s / 1e9 / peaks["hbm_gbs"], "algorithmic_bytes_per_launch": a_bytes,
                                       "avg_ms": a_s * 1e3}
            if (args.fp8_pages and (args.paged or not args.unfused)) or one_pass_bf16:
                line.pop("attend_roofline")
            fp8_step = ns * ab["index"] + g_bytes + a_bytes
            line["step_hbm"] = {"algorithmic_bytes_per_step": fp8_step, "accounting": "index + one read of the selected FP8 pages" if args.fp8_pages and args.paged else
                                "index + FP8 page read + FP8 view write (fused pass)" if args.fp8_pages and not args.unfused else
                                "index + FP8 page read + FP8 view write + FP8 view read" if args.fp8_pages else
                                "index + bf16 page read + FP8 view write (fused pass)" if one_pass_bf16 else "index + bf16 page read + FP8 view write + FP8 view read",
                                "achieved_gbs": K * fp8_step / (total_ms * 1e-3) / 1e9,
                                "frac_of_peak": K * fp8_step / (total_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                "peak_source": f"of {peaks['source']}", "nominal_peak_gbs": 8000.0}
            line["e2e"]["api"] = "pinned host query in, host O and LSE out, around the three calls of the FP8-view step"
        if args.rope and args.paged and args.fp8_pages:
            # FP8 repository of in-block-rotated keys, copy-free: one byte per element of the selected blocks is read
            a_bytes = ns * ab["attend"] // 2
            a_s = gather_s
            line["dtype"] = "E4M3 pages (codes of RoPE(k, offset in block), quantised at append), bf16 query and index, f16 tensor-core products, fp32 accumulation"
            line["config"]["calls"] = ("kvmem_rope_rotate(q) + kvmem_select + kvmem_paged_attend_fp8_rope (FP8 repository, position-consistent, "
                                       "copy-free: the query is rotated back once per block)")
            line["roofline"] = {"bound": "hbm", "kernel": "attend_fp8_split_kernel<3> + merge (kvmem_paged_attend_fp8_rope)", "achieved": a_bytes / a_s / 1e9,
                                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": a_bytes / a_s / 1e9 / peaks["hbm_gbs"],
                                "peak_source": f"of {peaks['source']}", "algorithmic_bytes_per_launch": a_bytes,
                                "avg_launch_ms": a_s * 1e3, "traffic": None}
            f8_step = ns * ab["index"] + a_bytes
            line["step_hbm"] = {"algorithmic_bytes_per_step": f8_step, "accounting": "index + one read of the selected FP8 pages",
                                "achieved_gbs": K * f8_step / (total_ms * 1e-3) / 1e9,
                                "frac_of_peak": K * f8_step / (total_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                "peak_source": f"of {peaks['source']}", "nominal_peak_gbs": 8000.0}
        if args.rope:
            line["e2e"]["api"] = "pinned host query in, host O and LSE out, around the four calls of the position-consistent step"
        if line["roofline"].get("traffic") is not None:
            line["roofline"]["traffic_source"] = TRAFFIC_SOURCE
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(base, args.cpu_sample_blocks)
        return line
    return None


# ----------------------------------------------------------------------------- execution cache (working-set reuse)

def run_cache(args):
    """Position-consistent step with the execution view kept across steps (Sec. 4.4): de-RoPE the query, select,
    update the cache as a working-set delta (bounded delta re-RoPE), attend over the cache through its page table."""
    from paper_2609_04852_b200 import SelectParams, budget_blocks, set_option
    if int(os.environ.get("WORLD_SIZE", "1")) != 1:
        raise SystemExit("--cache is a single-GPU measurement")
    device = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(device)
    for opt in args.option:
        name, _, value = opt.partition("=")
        set_option(name, int(value))
    base = CONFIGS[args.workload]
    if not base.attend or base.n_sessions != 1:
        raise SystemExit("--cache is measured on the single-session attend workloads")
    pool, spec = fill_pool(base, device, rope=True, in_block=args.in_block)
    M, B, H, d = spec.n_q_tokens, spec.block_tokens, spec.n_q_heads, spec.head_dim
    prm = SelectParams(**select_params(spec))
    k = budget_blocks(prm, B, spec.n_blocks)
    q_dev = [make_queries(spec, i, drift=args.drift).to(device) for i in range(spec.n_query_sets)]
    sel = torch.zeros(1, k, dtype=torch.int32, device=device)
    n_sel = torch.zeros(1, dtype=torch.int32, device=device)
    cache = pool.new_view_cache(k, args.max_delta, 0)
    out, lse = pool.new_outputs(1, M)
    q_pos = torch.arange(k * B, k * B + M, dtype=torch.int32, device=device)
    q_raw = torch.empty_like(q_dev[0])
    stream = torch.cuda.current_stream(device)

    def step(i, ev=None):
        q = q_dev[i % len(q_dev)]
        pool.rope_rotate(q.view(M, H, d), q_pos, out=q_raw.view(M, H, d), inverse=True)
        pool.select(q_raw, prm, sel, n_sel)
        if ev is not None:
            ev[0].record(stream)
        cache.update(0, sel[0], n_sel)
        if ev is not None:
            ev[1].record(stream)
        cache.attend(q[0], out[0], lse[0])
        if ev is not None:
            ev[2].record(stream)

    # steady-state statistics of the working-set delta (untimed pass over two rounds of the query sets)
    acc = torch.zeros(4, dtype=torch.int64, device=device)
    n_stat = 2 * len(q_dev)
    for i in range(n_stat):
        step(i)
        if i >= len(q_dev):
            acc += cache.stats
    torch.cuda.synchronize(device)
    stats = (acc.cpu().double() / (n_stat - len(q_dev))).tolist()
    for i in range(max(args.warmup, 3)):
        step(n_stat + i)
    torch.cuda.synchronize(device)
    assert pool.device_status() == 0
    sampler = ClockSampler(device.index)
    sampler.start()
    time.sleep(0.25)
    K = args.steps
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    begins = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize(device)
    t0 = time.time()
    e0.record(stream)
    for i in range(K):
        begins[i].record(stream)
        step(n_stat + 3 + i, marks[i])
    e1.record(stream)
    torch.cuda.synchronize(device)
    t1 = time.time()
    if t1 - t0 < 0.5:       # keep the load up long enough for the clock sampler
        t0 = time.time()
        i = 0
        while time.time() < t0 + 0.6:
            step(i); i += 1
            if i % 50 == 0:
                torch.cuda.synchronize(device)
        torch.cuda.synchronize(device)
        t1 = time.time()
    sampler.window(t0, t1)
    clocks = sampler.stop()
    assert pool.device_status() == 0
    total_ms = e0.elapsed_time(e1)
    med = statistics.median
    sel_ms = med([begins[i].elapsed_time(marks[i][0]) for i in range(K)])
    upd_ms = med([marks[i][0].elapsed_time(marks[i][1]) for i in range(K)])
    att_ms = med([marks[i][1].elapsed_time(marks[i][2]) for i in range(K)])
    # end to end: query from pinned host memory, O and LSE back to the host, every step
    q_pin = [make_queries(spec, i, drift=args.drift).pin_memory() for i in range(spec.n_query_sets)]
    out_pin, lse_pin = torch.empty(out.shape).pin_memory(), torch.empty(lse.shape).pin_memory()
    q_stage = torch.empty_like(q_dev[0])
    Ke = min(K, 200)
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record(stream)
    for i in range(Ke):
        q_stage.copy_(q_pin[i % len(q_pin)], non_blocking=True)
        pool.rope_rotate(q_stage.view(M, H, d), q_pos, out=q_raw.view(M, H, d), inverse=True)
        pool.select(q_raw, prm, sel, n_sel)
        cache.update(0, sel[0], n_sel)
        cache.attend(q_stage[0], out[0], lse[0])
        out_pin.copy_(out, non_blocking=True)
        lse_pin.copy_(lse, non_blocking=True)
        torch.cuda.synchronize(device)
    ee1.record(stream)
    torch.cuda.synchronize(device)
    peaks = measured_peaks()
    page_bytes = 2 * spec.n_layers * spec.n_kv_heads * B * d * 2
    # bytes the update has to move: an incoming block is read and written (K and V), a re-encoded one K only
    upd_bytes = stats[3] * 2 * page_bytes + (stats[1] + stats[2]) * page_bytes
    att_bytes = k * page_bytes
    rows = M * spec.n_layers * H
    line = {
        "metric": METRIC, "value": K / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic (seeded; shapes of the paper's agent workspaces)",
        "config": {"workload": f"{spec.name}: 1 session x {spec.n_blocks} blocks of {B} tokens, {M} query token(s), budget {k} blocks, "
                               f"execution cache of {k} slots, query drift {args.drift}, at most {args.max_delta} delta re-RoPE "
                               "operations between reconstructions",
                   "history_tokens": spec.tokens, "view_tokens": k * B, "query_sets": len(q_dev),
                   "l2": "no flush: every step streams far more than the 126 MB L2",
                   "parallelism": "1 session on 1 GPU",
                   "calls": "kvmem_rope_rotate(q) + kvmem_select + kvmem_view_cache_update + kvmem_view_cache_attend"},
        "e2e": {"value": Ke / (ee0.elapsed_time(ee1) * 1e-3), "unit": UNIT, "steps": Ke,
                "h2d_bytes_per_step": rows * d * 2, "d2h_bytes_per_step": rows * d * 4 + rows * 4,
                "api": "pinned host query in, host O and LSE out, around the four calls"},
        "gpu_launches": K * 8, "clocks": clocks,
        "cache": {"avg_blocks_per_step": {"unmoved": stats[0], "delta_roped": stats[1], "rebuilt": stats[2], "incoming": stats[3]},
                  "update_bytes_per_step": upd_bytes, "view_bytes": att_bytes},
        "roofline": {"bound": "hbm", "kernel": "attend_split_kernel<2> + merge over the cache slots (kvmem_view_cache_attend)",
                     "achieved": att_bytes / (att_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": att_bytes / (att_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                     "algorithmic_bytes_per_launch": att_bytes, "avg_launch_ms": att_ms, "traffic": None},
        "update_roofline": {"kernel": "view_cache_plan_kernel + view_cache_apply_kernel", "achieved_gbs": upd_bytes / (upd_ms * 1e-3) / 1e9,
                            "frac": upd_bytes / (upd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "avg_ms": upd_ms},
        "stages_ms": {"select": sel_ms, "cache_update": upd_ms, "attend": att_ms},
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- one session sharded by KV head

def run_head_sharded(args):
    """Strong scaling of ONE session over N GPUs: rank p holds the pages and index rows of KV heads
    [p G/N, (p+1) G/N) and the query heads that map to them.  Step: score the own heads, all-reduce the NB fp32
    block scores (NCCL; the only exchange), the same deterministic top-k on every rank, view assembly + attention
    over the own heads.  At N = 1 it is the default step without the collective."""
    import torch.distributed as dist
    from paper_2609_04852_b200 import Pool, SelectParams, budget_blocks, set_option
    from paper_2609_04852_b200.sharding import head_sharded_step, kv_heads_for_rank, max_over_ranks, query_heads_of
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: a run never silently uses fewer GPUs than asked for")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    for opt in args.option:
        name, _, value = opt.partition("=")
        set_option(name, int(value))
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=device)
    spec = CONFIGS[args.workload]
    if not spec.attend or spec.n_sessions != 1:
        raise SystemExit("--shard-heads is measured on the single-session attend workloads")
    if args.blocks:
        f = args.blocks / spec.n_blocks
        spec = spec.with_(name=f"{spec.name}@{args.blocks}", n_blocks=args.blocks, n_planted=max(1, int(spec.n_planted * f)),
                          budget_blocks=max(1, int(spec.budget_blocks * f)))
    r = spec.n_q_heads // spec.n_kv_heads
    g0, g1 = kv_heads_for_rank(spec.n_kv_heads, rank, world)
    h0, h1 = query_heads_of((g0, g1), r)
    G_loc, H_loc = g1 - g0, h1 - h0
    M, B, d = spec.n_q_tokens, spec.block_tokens, spec.head_dim
    pool = Pool(spec.n_layers, H_loc, G_loc, d, B, 1, spec.n_blocks, spec.n_blocks, device.index)
    table = page_table(spec)[0]
    for b0 in range(0, spec.n_blocks, 1024):          # every rank generates the same session and keeps its heads
        b1 = min(spec.n_blocks, b0 + 1024)
        K, V = kv_blocks(spec, 0, b0, b1, device)
        pool.append_blocks(0, K[:, :, g0:g1].contiguous(), V[:, :, g0:g1].contiguous(), table[b0:b1].tolist())
    torch.cuda.synchronize(device)
    prm = SelectParams(**select_params(spec))
    k = budget_blocks(prm, B, spec.n_blocks)
    qsets = [make_queries(spec, i)[:, :, :, h0:h1].contiguous() for i in range(spec.n_query_sets)]
    q_dev = [q.to(device) for q in qsets]
    q_pin = [q.pin_memory() for q in qsets]
    scores = torch.zeros(1, spec.n_blocks, dtype=torch.float32, device=device)
    sel = torch.zeros(1, k, dtype=torch.int32, device=device)
    n_sel = torch.zeros(1, dtype=torch.int32, device=device)
    view = pool.new_view(1, k * B)
    out, lse = pool.new_outputs(1, M)
    stream = torch.cuda.current_stream(device)

    def step(i):
        head_sharded_step(pool, q_dev[i % len(q_dev)], prm, scores, sel, n_sel, view, out, lse, world)

    def barrier():
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    assert pool.device_status() == 0 and int(n_sel[0]) == k
    if world > 1:       # every rank must hold the same selection: compare a checksum (bookkeeping, untimed)
        chk = torch.stack([sel.sum(dtype=torch.int64), (sel.to(torch.int64) * torch.arange(1, k + 1, device=device)).sum()])
        lo, hi = chk.clone(), chk.clone()
        dist.all_reduce(lo, op=dist.ReduceOp.MIN)
        dist.all_reduce(hi, op=dist.ReduceOp.MAX)
        assert torch.equal(lo, hi), "ranks disagree on the selected ids"
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    K = args.steps
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.time()
    e0.record(stream)
    for i in range(K):
        step(i)
    e1.record(stream)
    barrier()
    t1 = time.time()
    total_ms = e0.elapsed_time(e1)
    # end to end: the own heads of the query from pinned host memory, the own heads of O and LSE back
    out_pin, lse_pin = torch.empty(out.shape).pin_memory(), torch.empty(lse.shape).pin_memory()
    q_stage = torch.empty_like(q_dev[0])
    Ke = min(K, 200)
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ee0.record(stream)
    for i in range(Ke):
        q_stage.copy_(q_pin[i % len(q_pin)], non_blocking=True)
        head_sharded_step(pool, q_stage, prm, scores, sel, n_sel, view, out, lse, world)
        out_pin.copy_(out, non_blocking=True)
        lse_pin.copy_(lse, non_blocking=True)
        torch.cuda.synchronize(device)
    ee1.record(stream)
    barrier()
    e2e_ms = ee0.elapsed_time(ee1)
    if rank == 0 and t1 - t0 < 0.5:       # keep the load up long enough for the clock sampler (rank 0 alone: no collective)
        t0 = time.time()
        i = 0
        while time.time() < t0 + 0.6:
            pool.materialize_attend(q_dev[0], sel, n_sel, view, out, lse); i += 1
            if i % 50 == 0:
                torch.cuda.synchronize(device)
        torch.cuda.synchronize(device)
        t1 = time.time()
    sampler.window(t0, t1)
    assert pool.device_status() == 0
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device=device)
    if rank == 0:
        clocks = sampler.stop()
        peaks = measured_peaks()
        rank_bytes = 2 * k * 2 * spec.n_layers * G_loc * B * d * 2 + spec.n_layers * G_loc * spec.n_blocks * d * 2
        rows = M * spec.n_layers * H_loc
        line = {
            "metric": METRIC, "value": K / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded; shapes of the paper's agent workspaces)",
            "config": {"workload": f"{spec.name}: 1 session x {spec.n_blocks} blocks of {B} tokens, {M} query token(s), "
                                   f"{spec.n_q_heads}/{spec.n_kv_heads} heads, budget {k} blocks",
                       "history_tokens": spec.tokens, "view_tokens": k * B, "query_sets": len(qsets),
                       "l2": "no flush: every step streams far more than the 126 MB L2",
                       "parallelism": f"one session sharded by KV head over {world} GPU(s): {G_loc} KV / {H_loc} query heads per rank, "
                                      f"one all-reduce of {spec.n_blocks} fp32 block scores per step",
                       "calls": "kvmem_score + all-reduce(R) + kvmem_topk + kvmem_materialize_attend"},
            "e2e": {"value": Ke / (e2e_ms * 1e-3), "unit": UNIT, "steps": Ke, "h2d_bytes_per_step": rows * d * 2,
                    "d2h_bytes_per_step": rows * d * 4 + rows * 4,
                    "api": "pinned host query (own heads) in, host O and LSE (own heads) out, around the sharded step"},
            "gpu_launches": K * 5, "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "whole step on one rank (index + view read + view write of its heads)",
                         "achieved": rank_bytes / (total_ms / K * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": rank_bytes / (total_ms / K * 1e-3) / 1e9 / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
                         "algorithmic_bytes_per_launch": rank_bytes, "avg_launch_ms": total_ms / K, "traffic": None},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- oracle arm / CPU baseline

def _bits(t):
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


class OracleSample:
    """The oracle on a bounded sample of a workload: scoring and selection over the whole index,
    view assembly and attention over the first `sample_blocks` selected blocks (cost scaled to k)."""

    def __init__(self, spec, sample_blocks):
        from oracle import kvmem_oracle as orc
        self.orc, self.spec = orc, spec
        gen_dev = torch.device("cuda", 0) if torch.cuda.is_available() else "cpu"
        nb = spec.n_blocks
        self.idx = np.zeros((spec.n_layers, spec.n_kv_heads, nb, spec.head_dim), np.uint16)
        for b0 in range(0, nb, 1024):                                  # setup, untimed: the oracle's own index
            b1 = min(nb, b0 + 1024)
            K, _ = kv_blocks(spec, 0, b0, b1, gen_dev)
            orc.mean_k_index(_bits(K), spec.block_tokens, self.idx, b0)
        prm = select_params(spec)
        self.k = orc.budget_blocks(nb, spec.block_tokens, prm["budget_blocks"], prm["max_view_tokens"])
        self.sample_blocks = min(sample_blocks, self.k)
        self.prm = prm
        self.gen_dev = gen_dev
        self.repo = None

    def _repo_for(self, ids):
        """Pages of the sampled blocks only (setup, untimed)."""
        spec, orc = self.spec, self.orc
        repo = orc.Repository.empty(len(ids), spec.block_tokens, spec.n_layers, spec.n_kv_heads, spec.head_dim)
        table = np.full(spec.n_blocks, -1, np.int32)
        for j, b in enumerate(ids):
            K, V = kv_blocks(spec, 0, int(b), int(b) + 1, self.gen_dev)
            repo.place(_bits(K), _bits(V), np.array([j], np.int32))
            table[b] = j
        return repo, table

    def step(self, qset):
        """Returns (seconds for a whole step, scaled from the sample)."""
        spec, orc = self.spec, self.orc
        qb = _bits(make_queries(spec, qset))[0]
        t0 = time.perf_counter()
        R, _ = orc.block_scores(qb, self.idx, spec.n_blocks)
        sel = orc.select(R, spec.block_tokens, self.prm["budget_blocks"], self.prm["max_view_tokens"])
        t1 = time.perf_counter()
        ids = sel[: self.sample_blocks]
        repo, table = self._repo_for(ids)                               # untimed: materialise the sample's pages
        t2 = time.perf_counter()
        cap = len(ids) * spec.block_tokens
        vK, vV = orc.gather(repo, table, np.ascontiguousarray(ids), cap)
        if spec.attend:
            orc.attend(qb, vK, vV, cap)
        t3 = time.perf_counter()
        scale = len(sel) / max(len(ids), 1)
        return (t1 - t0) + (t3 - t2) * scale


def cpu_baseline(spec, sample_blocks, steps=1):
    from oracle import kvmem_oracle as orc
    smp = OracleSample(spec, sample_blocks)
    secs = [smp.step(i) for i in range(steps)]
    t = sum(secs) / len(secs)
    return {"value": 1.0 / t, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
            "sample": f"session 0: scoring + selection over all {spec.n_blocks} blocks timed in full; view assembly + "
                      f"attention timed on the first {smp.sample_blocks} of {smp.k} selected blocks and scaled by "
                      f"{smp.k / max(smp.sample_blocks, 1):.1f}x; {steps} step(s); oracle seconds per step = {t:.2f}"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import kvmem_oracle as orc
    spec = CONFIGS[args.workload]
    smp = OracleSample(spec, args.cpu_sample_blocks)
    for i in range(min(args.warmup, 1)):
        smp.step(i)
    K = max(1, min(args.steps, 3))
    secs = [smp.step(i) for i in range(K)]
    t = sum(secs) / K
    value = 1.0 / t
    sample = (f"scoring + selection over all {spec.n_blocks} blocks in full; view assembly + attention on the first "
              f"{smp.sample_blocks} of {smp.k} selected blocks, scaled by {smp.k / max(smp.sample_blocks, 1):.1f}x")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": min(args.warmup, 1), "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64 accumulation on bf16 inputs", "data": "synthetic (seeded)",
            "config": {"workload": f"{spec.name}: {spec.n_blocks} blocks of {spec.block_tokens} tokens, "
                                   f"{spec.n_q_tokens} query token(s), budget {smp.k} blocks"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- launcher and the other configurations

def launch_ranks(n, argv, script=None, extra_env=None):
    """Run this command as n ranks on this node (torch.distributed.run, rendezvous on 127.0.0.1) and return its exit
    code.  The ranks inherit stdout, so rank 0's single JSON line is the output of the whole command."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--nnodes=1", f"--nproc-per-node={n}",
           "--local-addr", "127.0.0.1", script or os.path.abspath(__file__), *argv]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")          # NCCL's own log stays on (stderr): ranks, transports and NVLS use are visible in the run's output
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    env.update(extra_env or {})
    return subprocess.call(cmd, env=env)


def launch_selfcheck(args):
    """The multi-rank plumbing of this benchmark with no GPU in it (gloo on the host cores): rendezvous, barrier,
    a stand-in "step" of known duration per rank, the maximum over ranks, and rank 0 printing ONE line that carries
    n_gpus = the number of ranks.  A plain `--gpus N --launch-selfcheck` launches its own N ranks first."""
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args.gpus, sys.argv[1:])
    import torch.distributed as dist
    from paper_2609_04852_b200.sharding import max_over_ranks, whole_job_rate
    world, rank = int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0"))
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: a run never silently uses fewer GPUs than asked for")
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    local_ms = 10.0 + 5.0 * rank                     # the stand-in for a rank's device-timed region
    slowest, = max_over_ranks([local_ms])
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"selfcheck": "launcher", "n_gpus": world, "steps": args.steps, "ms_slowest_rank": slowest,
                          "value": whole_job_rate(args.steps, world, slowest), "unit": UNIT}), flush=True)
    return 0


def plain_default(args):
    """The headline invocation: the 1M workload with no variant switch."""
    return (args.workload == "1m" and not args.no_other_workloads and not any(
        (args.blocks, args.flush_l2, args.rope, args.in_block, args.paged, args.unfused, args.option, args.fp8,
         args.fp8_pages, args.host_index)))


OTHER_WORKLOADS = (("tiny", 2000, True), ("128k", 2000, True), ("batch8", 400, False), ("chunk512", 300, False))


def other_workloads(args):
    """The other four configurations, measured in the same process right after the headline one with the same
    protocol (own warm-up, own clock samples, own end-to-end pass); only the figures the headline line also has."""
    import copy
    import gc
    out = {}
    for name, steps, flush in OTHER_WORKLOADS:
        gc.collect()
        torch.cuda.empty_cache()
        a = copy.copy(args)
        a.workload, a.steps, a.flush_l2, a.no_cpu_baseline = name, min(steps, max(args.steps, 20)), flush, True
        line = run_native(a)
        keep = ("value", "unit", "ms_per_step", "steps", "warmup", "dtype", "roofline", "e2e", "clocks", "gpu_launches", "stages_ms")
        rec = {k: line[k] for k in keep if k in line}
        rec["config"] = {k: line["config"][k] for k in ("workload", "l2", "calls")}
        rec["step_hbm"] = {k: line["step_hbm"][k] for k in ("algorithmic_bytes_per_step", "accounting", "achieved_gbs", "frac_of_peak", "peak_source")}
        if flush:
            # the headline figures of this workload flush L2 between steps (its view fits, or nearly fits, the 126 MB L2);
            # the same steps back to back, as a decode loop would issue them, for comparison
            a.flush_l2 = False
            warm = run_native(a)
            rec["without_l2_flush"] = {"value": warm["value"], "ms_per_step": warm["ms_per_step"],
                                       "step_hbm_frac_of_peak": warm["step_hbm"]["frac_of_peak"],
                                       "note": "partly L2-resident: not a DRAM-roofline figure"}
        out[name] = rec
    gc.collect()
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["native", "reference"], default="native")
    ap.add_argument("--workload", choices=sorted(CONFIGS), default="1m")
    ap.add_argument("--blocks", type=int, default=0, help="shrink the history to this many blocks (profiling)")
    ap.add_argument("--flush-l2", action="store_true", help="write 256 MiB between steps (for workloads near L2 size)")
    ap.add_argument("--rope", action="store_true",
                    help="position-consistent view: keys de-rotated at append, query de-rotated for retrieval, RoPE at the "
                         "compact position fused into the gather (kvmem_materialize_rope), then kvmem_view_attend")
    ap.add_argument("--in-block", action="store_true",
                    help="with --rope: the pages hold RoPE(k, offset inside the block); the view rotates by the block's position "
                         "alone and --paged rotates the query back once per block instead of every key")
    ap.add_argument("--paged", action="store_true",
                    help="copy-free execution view: kvmem_select + kvmem_paged_attend (no view is materialised; not the headline step)")
    ap.add_argument("--shard-heads", action="store_true",
                    help="N GPUs share ONE session, each holding a slice of the KV heads; one all-reduce of the block scores "
                         "per step (strong scaling; the default at N > 1 is one independent session replica per GPU)")
    ap.add_argument("--unfused", action="store_true", help="separate kvmem_materialize and kvmem_view_attend calls")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="kernel-variant switch passed to kvmem_set_option (e.g. chunk_poly=0)")
    ap.add_argument("--cache", action="store_true", help="position-consistent step over an execution cache kept across "
                    "steps (working-set reuse, bounded delta re-RoPE); not the headline step")
    ap.add_argument("--drift", type=float, default=1.0, help="--cache: how far consecutive queries move (1 = independent)")
    ap.add_argument("--max-delta", type=int, default=4, help="--cache: delta re-RoPE operations between reconstructions")
    ap.add_argument("--fp8-pages", action="store_true", help="FP8 repository: the pages hold E4M3 tiles quantised at append; with --paged "
                    "the copy-free kvmem_paged_attend_fp8, else materialize_fp8 (a byte copy) + view_attend_fp8 (implies --fp8)")
    ap.add_argument("--fp8", action="store_true", help="FP8 (E4M3) execution view: materialize_fp8 + view_attend_fp8 (not the headline step)")
    ap.add_argument("--host-index", action="store_true", help="also time scoring against the index kept in pinned host memory")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="the headline (1M) invocation also measures tiny, 128k, batch8 and chunk512 into the line's "
                         "\"workloads\" object; this switch leaves them out")
    ap.add_argument("--launch-selfcheck", action="store_true",
                    help="exercise only the multi-rank launch and timing plumbing, on the host cores with gloo (no GPU)")
    ap.add_argument("--cpu-sample-blocks", type=int, default=256)
    args = ap.parse_args()
    if args.fp8_pages and args.rope:
        if not args.paged:
            raise SystemExit("--fp8-pages --rope is the copy-free position-consistent step: add --paged")
        args.in_block = True           # codes cannot be re-encoded: the keys carry their in-block rotation, the query is rotated
    elif args.fp8_pages:
        args.fp8 = True
    if args.in_block and not (args.rope or args.cache):
        raise SystemExit("--in-block needs --rope or --cache")
    if args.impl == "reference":
        run_reference(args)
        return
    if args.launch_selfcheck:
        raise SystemExit(launch_selfcheck(args))
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # asked for N GPUs from a plain command line: become the launcher of N ranks of this same command
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:]))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the native arm")
    if args.cache:
        run_cache(args)
    elif args.shard_heads:
        run_head_sharded(args)
    else:
        line = run_native(args)
        world = int(os.environ.get("WORLD_SIZE", "1"))
        if line is not None and world == 1 and plain_default(args):
            line["workloads"] = other_workloads(args)
        if line is not None:
            print(json.dumps(line), flush=True)
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()

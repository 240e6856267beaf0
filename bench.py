#!/usr/bin/env python
"""Benchmark of the bounded-state restore path on B200.

One "step" is one pass of the whole hot path over one synthetic prefix: probe (chunk digests,
key chain, index lookup) -> bounded-window restore from the HOST tier (tier -> pinned W-slot
pool -> cudaMemcpyAsync -> device staging -> install kernels) -> commit.

  value     restore throughput with the request's own inputs (token ids, block tables) already in
            HBM; the tier is external by definition, so its bytes cross the host link every step.
  e2e       the same calls with every input in host memory: token ids copied in by the probe, the
            request (block tables) created and uploaded inside the step, bitmap and checksums read
            back; plus what bounds it on this host (link, fill alone, fill + copies).
  roofline  the install kernel as launched inside those timed steps, against the measured HBM
            copy bandwidth; `resident` is the same kernel over all chunks in one launch with the
            tier objects placed in HBM (an install microbenchmark, not a restore).
  cpu_baseline  the CPU oracle timed on the host cores (reported, not a target).

Usage: python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
With --gpus N > 1 and no launcher environment the script starts its N ranks itself; under
torchrun it is one of them.  Every process drives its own GPU and restores its own rank slices
(slice r of 2N lives on process r mod N: weak scaling); the only exchange is the one-word commit AND.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_17826_b200 import multi, synth  # noqa: E402

WORKLOAD = dict(name="32768-token prefix, 128 chunks x 16,408,576 B, 2 rank slices per GPU, W=32, "
                     "baseline 2-group/99-tensor layout, 64-token blocks",
                n_chunks=128, n_ranks=2, W=32)
# dram read + write bytes per payload byte, from one ncu capture of each install kernel on a
# 64-descriptor launch (traffic grows in proportion to the descriptors a launch carries); captured
# on the baseline and on the short-run registration, the others are scaled with the baseline figure
NCU_DRAM_BYTES_PER_PAYLOAD_BYTE = {("bsr_install_bulk_kernel", "baseline"): 1.955,
                                   ("bsr_install_vec_kernel", "baseline"): 1.955,
                                   ("bsr_install_bulk_kernel", "short_runs"): 1.903,
                                   ("bsr_install_vec_kernel", "short_runs"): 1.946}
METRIC, UNIT = "restore GB/s from the host tier (all rank slices; per-rank = value / rank slices)", "GB/s"
LAYOUTS = {"baseline": synth.baseline_layout, "hetero": synth.hetero_layout, "mtp_on": synth.mtp_on_layout,
           "short_runs": synth.short_run_layout}


def _config(n_chunks, layout_name="baseline", window=0):
    name = WORKLOAD["name"]
    if n_chunks != WORKLOAD["n_chunks"]:
        name = f"REDUCED to {n_chunks} chunks: " + name
    if layout_name != "baseline":
        name = f"LAYOUT {layout_name}: " + name
    if window and window != WORKLOAD["W"]:
        name = f"WINDOW W={window} instead of {WORKLOAD['W']}: " + name
    return {"workload": name, "rank_slices_per_gpu": WORKLOAD["n_ranks"], "W": window or WORKLOAD["W"],
            "l2": "every step moves 4.2 GB per GPU, far more than L2; no flush needed"}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (an earlier measurement of the same copy on a B200)"


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.t.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for k, n in enumerate(names)
                   if any(len(r) > 2 + k and r[2 + k].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": reasons, "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# CPU oracle legs (cpu_baseline of the default run, and --impl reference)
# --------------------------------------------------------------------------------------------
class OracleWorkload:
    """The benchmarked workload built for the oracle: tiers, tables, paged host arrays."""

    def __init__(self, layout, n_ranks, n_chunks, seed):
        from concurrent.futures import ThreadPoolExecutor

        from oracle import bsr_oracle as O
        self.O, self.R, self.N, self.seed = O, n_ranks, n_chunks, seed
        self.reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
        self.tok = synth.tokens(n_chunks * 256, seed=seed)
        keys = O.prefix_keys(O.chunk_digests(self.tok, seed), seed, 1)
        self.tiers = [O.Tier() for _ in range(n_ranks)]

        def make(ri):
            p = synth.chunk_payload(layout, ri[0], ri[1], seed=seed).copy()
            return ri, p, O.group_checksums(self.reg, p)

        with ThreadPoolExecutor(min(16, os.cpu_count() or 4)) as ex:   # set-up only, not timed
            for (r, i), p, ck in ex.map(make, [(r, i) for r in range(n_ranks) for i in range(n_chunks)]):
                self.tiers[r].put(keys[i], p, ck)
        pools = [synth.pool_blocks(layout, g, n_chunks) for g in range(self.reg.n_groups)]
        self.tables = [[synth.block_table(layout, r, g, n_chunks, seed=seed) for g in range(self.reg.n_groups)]
                       for r in range(n_ranks)]
        self.paged = [O.new_paged(self.reg, pools, synth.CANARY) for _ in range(n_ranks)]
        self.bytes = n_ranks * n_chunks * self.reg.chunk_bytes

    def step(self, W, workers=1):
        """One oracle pass: probe + strict-window restore + commit.  Returns seconds."""
        O = self.O
        t0 = time.perf_counter()
        k, hit, n_hit = O.probe(self.tok, self.seed, 1, self.tiers)
        req = O.Request(k[:n_hit], self.tables, self.R, self.reg.n_groups)
        status, st = O.restore(self.reg, self.tiers, req, self.paged, W, workers=workers)
        exposed = O.commit(self.reg, req, self.paged)
        dt = time.perf_counter() - t0
        assert status == O.OK and exposed == self.N
        return dt


def run_reference(args):
    """--impl reference: the oracle, as it stands, on one host core, on the benchmarked workload
    (all 128 chunks x 2 rank slices every step)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    layout = synth.baseline_layout()
    N = args.chunks or WORKLOAD["n_chunks"]
    wl = OracleWorkload(layout, WORKLOAD["n_ranks"], N, synth.MASTER_SEED)
    for _ in range(args.warmup):
        wl.step(WORKLOAD["W"])
    ts = [wl.step(WORKLOAD["W"]) for _ in range(args.steps)]
    ms = 1e3 * sum(ts) / len(ts)
    val = wl.bytes / (ms / 1e3) / 1e9
    desc = f"all {N} chunks x {WORKLOAD['n_ranks']} rank slices every step ({wl.bytes} B), one thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8 payload, u64 checksums/digests", "data": "synthetic",
        "config": _config(N),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))
    return 0


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
class Side:
    """A context with the workload registered and its tier filled, in host or device memory."""

    def __init__(self, B, torch, dev, layout, n_ranks, n_chunks, W, payload_host, location, **cfg):
        self.B, self.torch = B, torch
        rc, self.ctx = B.bsr_ctx_create(W, n_ranks, device=dev.index, time_kernels=True, **cfg)
        assert rc == B.BSR_OK, rc
        self.G = layout.n_groups
        pools = [synth.pool_blocks(layout, g, n_chunks) for g in range(self.G)]
        self.paged = []
        for r in range(n_ranks):
            per = [torch.full((pools[g], layout.block_tokens[g], e), synth.CANARY, dtype=torch.uint8,
                              device=dev) for g, e in layout.tensors]
            self.paged.append(per)
            rc = B.bsr_register(self.ctx, r, [(layout.block_tokens[g], pools[g]) for g in range(self.G)],
                                [(g, e, per[l].data_ptr()) for l, (g, e) in enumerate(layout.tensors)])
            assert rc == B.BSR_OK, B.bsr_last_error(self.ctx)
        self.tables = [synth.block_table(layout, r, g, n_chunks) for r in range(n_ranks) for g in range(self.G)]
        self.objs = payload_host if location == B.BSR_LOC_HOST else \
            {k: torch.from_numpy(v).to(dev) for k, v in payload_host.items()}
        self.location = location
        self.req = None

    def fill_tier(self, keys):
        B = self.B
        for (r, i), o in self.objs.items():
            ptr = o if self.location == B.BSR_LOC_HOST else o.data_ptr()
            n = o.size if self.location == B.BSR_LOC_HOST else o.numel()
            rc = B.bsr_tier_put(self.ctx, r, keys[i], ptr, n, None, self.location)  # store path stamps checksums
            assert rc == B.BSR_OK, B.bsr_last_error(self.ctx)

    def step(self, tok, n_tok, salt, tok_on_device, stream, fresh_request=False):
        """probe -> (request) -> restore -> commit.  fresh_request: the request object (block tables
        validated and uploaded) is created inside the step and its bitmap read back."""
        B = self.B
        rc, keys, bm, n_hit = B.bsr_probe(self.ctx, tok, n_tok, salt, tok_on_device)
        assert rc == B.BSR_OK
        if fresh_request and self.req is not None:
            B.bsr_req_release(self.ctx, self.req)
            self.req = None
        if self.req is None:
            rc, self.req = B.bsr_req_create(self.ctx, keys[:n_hit], self.tables)
            assert rc == B.BSR_OK, B.bsr_last_error(self.ctx)
        rc = B.bsr_restore(self.ctx, self.req, stream)
        assert rc == B.BSR_OK, (rc, B.bsr_last_error(self.ctx))
        rc, exposed = B.bsr_commit(self.ctx, self.req)
        assert rc == B.BSR_OK
        if fresh_request:
            rc, bitmap = B.bsr_req_bitmap(self.ctx, self.req, len(self.paged), self.G, n_hit)
            assert rc == B.BSR_OK and int(bitmap[0]) != 0
        return n_hit, exposed

    def stats(self):
        return self.B.bsr_get_stats(self.ctx)[1]

    def close(self):
        if self.req is not None:
            self.B.bsr_req_release(self.ctx, self.req)
        self.B.bsr_ctx_destroy(self.ctx)


def measure_h2d(torch, dev, piece_bytes, total_bytes=1 << 30, reps=5):
    """Pinned-host -> device copy bandwidth in pieces of one chunk, best of reps (GB/s)."""
    n = max(1, total_bytes // piece_bytes)
    src = torch.empty(n * piece_bytes, dtype=torch.uint8).pin_memory()
    dst = torch.empty(n * piece_bytes, dtype=torch.uint8, device=dev)
    src.fill_(1)
    best = 0.0
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(n):
            dst[k * piece_bytes:(k + 1) * piece_bytes].copy_(src[k * piece_bytes:(k + 1) * piece_bytes],
                                                            non_blocking=True)
        e1.record()
        torch.cuda.synchronize()
        best = max(best, n * piece_bytes / (e0.elapsed_time(e1) / 1e3) / 1e9)
    return best


def timed_steps(torch, dist, world, side, tok, n_tok, salt, tok_on_device, steps, warmup, n_chunks,
                coll_dev="cuda", fresh_request=False):
    """Returns (device ms per step, host wall ms per step, stats of the timed steps), the slowest rank's."""
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        _, exposed = side.step(tok, n_tok, salt, tok_on_device, stream.cuda_stream, fresh_request)
        if world > 1:  # the commit exchange is part of a step: warm its communicator up as well
            multi.commit_across_ranks(exposed, n_chunks, device=coll_dev)
    side.B.bsr_reset_stats(side.ctx)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record(stream)
    ok = True
    for _ in range(steps):
        n_hit, exposed = side.step(tok, n_tok, salt, tok_on_device, stream.cuda_stream, fresh_request)
        ok = ok and n_hit == n_chunks and exposed == n_chunks
        if world > 1:  # request-level commit across GPUs: one word, AND over ranks (Eq. 6)
            ok = ok and multi.commit_across_ranks(exposed, n_chunks, device=coll_dev) == n_chunks
    e1.record(stream)
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - t0) * 1e3
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    if world > 1:
        ms = multi.max_over_ranks(ms, device=coll_dev)
        wall_ms = multi.max_over_ranks(wall_ms, device=coll_dev)
    assert ok, "a step did not expose the full prefix"
    return ms / steps, wall_ms / steps, side.stats()


def place_on_host(torch, B, local, world):
    """With several processes on one host: this rank's share of the CPUs (those of its GPU's NUMA
    node where the platform names one), set as the process' affinity so that the library's fill
    threads and pinned pool inherit it.  Returns the CPU list."""
    allowed = sorted(os.sched_getaffinity(0))
    if world == 1:
        return allowed
    node_cpus = []
    for l in range(world):
        cpus = None
        try:
            p = torch.cuda.get_device_properties(l if l < torch.cuda.device_count() else 0)
            bus = f"{p.pci_domain_id:04x}:{p.pci_bus_id:02x}:{p.pci_device_id:02x}.0"
            rc, node, cpulist, _ = B.bsr_numa_of_pci("/sys", bus)
            if rc == B.BSR_OK and node >= 0 and cpulist:
                cpus = []
                for part in cpulist.split(","):
                    lo, _, hi = part.partition("-")
                    cpus += list(range(int(lo), int(hi or lo) + 1))
        except (AttributeError, AssertionError, RuntimeError, ValueError):
            cpus = None
        node_cpus.append(cpus)
    mine = multi.cpu_share(allowed, node_cpus, local)
    os.sched_setaffinity(0, mine)
    return mine


def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2608_17826_b200 import build
    build.build()
    from paper_2608_17826_b200 import binding as B  # raises if the CUDA library is missing

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the BSR path has no CPU fallback")
    if not args.dry_run_one_gpu and world > torch.cuda.device_count():
        raise SystemExit(f"--gpus {world} but only {torch.cuda.device_count()} CUDA devices are visible")
    cpus = place_on_host(torch, B, local, world)
    if args.dry_run_one_gpu:
        # plumbing check only: every rank drives GPU 0 and the commit word travels over gloo (NCCL
        # refuses two ranks on one device).  The ranks' kernels never wait on one another.
        local = 0
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    coll_dev = None if args.dry_run_one_gpu else "cuda"
    if world > 1:
        if args.dry_run_one_gpu:
            dist.init_process_group("gloo")
        else:
            dist.init_process_group("nccl", device_id=dev)

    layout = LAYOUTS[args.layout]()
    R, N, W = WORKLOAD["n_ranks"], args.chunks or WORKLOAD["n_chunks"], args.window or WORKLOAD["W"]
    chunk = layout.chunk_bytes
    # one request for the whole job: the same token ids everywhere; process p restores the rank
    # slices p, p + world, ... of the job's R * world slices
    slices = multi.slices_of(rank, world, R * world)
    seed = synth.MASTER_SEED
    salt = seed
    tok = synth.tokens(N * 256, seed=seed)
    payload = {(r, i): synth.chunk_payload(layout, slices[r], i, seed=seed).copy() for r in range(R) for i in range(N)}
    step_bytes = R * N * chunk
    d_tok = torch.from_numpy(tok).to(dev)
    if args.load_concurrency == 0:
        args.load_concurrency = max(2, min(16, len(cpus) // 2))
    sampler = ClockSampler(local)
    sampler.start()

    # ---- install microbenchmark: tier objects placed in HBM, all chunks in one launch -----------
    res = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_DEVICE, install_variant=args.variant)
    rc, keys, _, _ = B.bsr_probe(res.ctx, d_tok.data_ptr(), len(tok), salt, True)
    assert rc == B.BSR_OK
    res.fill_tier(keys)
    rc, in_use = B.bsr_install_kernel_in_use(res.ctx)
    assert rc == B.BSR_OK
    kernel_name = "bsr_install_vec_kernel" if in_use == B.BSR_INSTALL_VECTOR else "bsr_install_bulk_kernel"
    ms_res, _, st_res = timed_steps(torch, dist, world, res, d_tok.data_ptr(), len(tok), salt, True,
                                    args.steps, args.warmup, N, coll_dev)
    res_launches = int(st_res.install_launches)
    res_k_ms = st_res.install_kernel_ms / max(1, res_launches)
    res.close()
    del res
    torch.cuda.empty_cache()
    hbm_peak, peak_src = _peaks()
    res_payload = step_bytes * args.steps / max(1, res_launches)
    res_span_ms = st_res.install_span_ms / max(1, res_launches)
    resident = {"what": "install kernel alone: tier objects placed in HBM, probe + install + commit, no host link",
                "in_kernel_span_ms": res_span_ms,
                "frac_in_kernel": 2 * res_payload / (res_span_ms / 1e3) / 1e9 / hbm_peak if res_span_ms else None,
                "GBps_payload": step_bytes / (ms_res / 1e3) / 1e9, "ms_per_step": ms_res,
                "descriptors_per_launch": int(st_res.install_descriptors) / max(1, res_launches),
                "avg_launch_ms": res_k_ms, "achieved": 2 * res_payload / (res_k_ms / 1e3) / 1e9 if res_k_ms else None,
                "frac": 2 * res_payload / (res_k_ms / 1e3) / 1e9 / hbm_peak if res_k_ms else None, "unit": "GB/s"}

    if args.resident_only:  # profiling runs: only the install microbenchmark, no JSON contract line
        sampler.stop()
        if rank == 0:
            print(json.dumps({"resident_only": True, "layout": args.layout, "chunks": N, "kernel": kernel_name,
                              **resident}))
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- the restore: tier in host memory, through the pinned W-slot pool ------------------------
    h2d_gbs = measure_h2d(torch, dev, chunk)                  # the roofline: copies of one chunk each
    h2d_one_piece = measure_h2d(torch, dev, 1 << 30, reps=3)  # context: a single 1 GiB copy
    side = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_HOST,
                load_concurrency=args.load_concurrency, dev_staging_depth=args.depth,
                install_variant=args.variant, direct_install=args.direct, install_batch=args.install_batch)
    side.fill_tier(keys)
    # value: the request's inputs (token ids, block tables) already on the device
    ms_val, _, st_val = timed_steps(torch, dist, world, side, d_tok.data_ptr(), len(tok), salt, True,
                                    args.steps, args.warmup, N, coll_dev)
    # e2e: every input in host memory, request built inside the step, results read back
    e2e_steps = max(3, min(args.steps, 10))
    ms_e2e, wall_e2e, st_e2e = timed_steps(torch, dist, world, side, tok, len(tok), salt, False, e2e_steps,
                                           3, N, coll_dev, fresh_request=True)
    clocks = sampler.stop()
    # what bounds it on this host: the library's own fill alone, then fill + copies, no kernels
    cal = {}
    for name, stages in (("fill_only", B.BSR_CAL_FILL), ("fill_plus_h2d", B.BSR_CAL_FILL_H2D)):
        best = 0.0
        for _ in range(3):
            rc, sec = B.bsr_restore_calibrate(side.ctx, side.req, stages)
            assert rc == B.BSR_OK, B.bsr_last_error(side.ctx)
            best = max(best, step_bytes / sec / 1e9)
        cal[name] = multi.max_over_ranks(-best, device=coll_dev) * -1 if world > 1 else best  # slowest rank
    peak_staging = [int(st_val.peak_staging_bytes[r]) for r in range(R)]
    slot = int(st_val.slot_bytes)
    # probe alone (token ids in host memory)
    t0 = time.perf_counter()
    for _ in range(20):
        B.bsr_probe(side.ctx, tok, len(tok), salt, False)
    probe_us = (time.perf_counter() - t0) / 20 * 1e6
    numa_node = int(st_val.fill_numa_node)
    # the failure path's scrub: zero-fill of every destination block of the request (the call blocks
    # until the kernel has finished; the second call is the measured one)
    scrub_ms = None
    if side.req is not None:
        for _ in range(2):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            rc = B.bsr_invalidate(side.ctx, side.req, B.BSR_SCRUB)
            scrub_ms = (time.perf_counter() - t0) * 1e3
            assert rc == B.BSR_OK
    side.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    table_bytes = R * sum(synth.blocks_per_chunk(layout, g) * N * 4 for g in range(layout.n_groups))
    value = world * step_bytes / (ms_val / 1e3) / 1e9
    e2e_value = world * step_bytes / (ms_e2e / 1e3) / 1e9
    # the install kernel as launched inside the timed steps of `value`
    k_launches = int(st_val.install_launches)
    k_desc = int(st_val.install_descriptors)
    k_ms = st_val.install_kernel_ms / max(1, k_launches)
    k_span_ms = st_val.install_span_ms / max(1, k_launches)
    per_launch_payload = chunk * k_desc / max(1, k_launches)
    achieved = 2 * per_launch_payload / (k_ms / 1e3) / 1e9 if k_ms > 0 else None
    traffic_key = (kernel_name, args.layout if (kernel_name, args.layout) in NCU_DRAM_BYTES_PER_PAYLOAD_BYTE else "baseline")
    traffic = NCU_DRAM_BYTES_PER_PAYLOAD_BYTE[traffic_key] * per_launch_payload
    bounds = {"h2d link": h2d_gbs, "host fill alone (tier -> slot copies)": cal["fill_only"],
              "host memory system (fill and the copy engine's reads together)": cal["fill_plus_h2d"]}
    bound_name = min(bounds, key=bounds.get)
    bound = bounds[bound_name]

    # ---- CPU oracle on the host cores (rank 0 at N = 1 only) -----------------------------------
    del payload, side
    if world == 1:
        wl = OracleWorkload(layout, R, min(N, 128), seed)
        dt1 = wl.step(W)
        cores = os.cpu_count() or 1
        dtn = wl.step(W, workers=cores)
        cpu = {"value": wl.bytes / dt1 / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"all {wl.N} chunks x {R} rank slices, one pass ({dt1:.1f} s), one thread",
               "all_cores": {"value": wl.bytes / dtn / 1e9, "unit": UNIT, "cores": cores,
                             "sample": f"same pass with the chunks of each window handed to a pool of {cores} "
                                       f"threads ({dtn:.1f} s)"},
               "host_cores_available": cores}
    else:
        cpu = {"value": None, "unit": UNIT, "cores": 0, "kind": "oracle", "sample": "timed at N = 1 only"}

    cfg = _config(N, args.layout, args.window)
    out = {
        **({"dry_run_one_gpu": True} if args.dry_run_one_gpu else {}),
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_val, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8 payload, u64 checksums/digests", "data": "synthetic",
        "config": cfg,
        "path": {"value": "token ids and block tables in HBM; host tier -> pinned W-slot pool -> H2D -> install, "
                          "every step",
                 "e2e": ("token ids, block tables and tier in host memory; request created in the step; bitmap "
                         "read back; " + ("install kernel reads the slots over the link" if args.direct else
                                          "host tier -> pinned pool -> H2D -> install")),
                 "load_concurrency": args.load_concurrency, "dev_staging_depth": min(args.depth or max(16, (args.install_batch or 64) // R), 64),
                 "install_batch": args.install_batch or 64, "fill_cpus": len(cpus), "fill_numa_node": numa_node},
        "per_rank_GBps": value / (world * R),
        "restore_seconds": ms_val / 1e3,
        "frac_of_h2d_link": value / world / h2d_gbs,
        "probe_host_us": probe_us,
        "scrub": {"what": "bsr_invalidate(BSR_SCRUB) on the benchmarked request: host wall time of the call, "
                          "zero-fill of all its destination blocks (write-only HBM traffic)",
                  "ms": scrub_ms, "bytes": step_bytes,
                  "write_GBps": step_bytes / (scrub_ms / 1e3) / 1e9 if scrub_ms else None},
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "host_wall_ms_per_step": wall_e2e,
                "steps": e2e_steps,
                "h2d_bytes_per_step": step_bytes + len(tok) * 4 + table_bytes,
                "d2h_bytes_per_step": N * 8 + R * layout.n_groups * N * 12 + R * layout.n_groups * ((N + 63) // 64) * 8,
                "per_rank_GBps": e2e_value / (world * R), "restore_seconds": ms_e2e / 1e3,
                "h2d_link_GBps_measured": h2d_gbs, "h2d_link_GBps_single_1GiB_copy": h2d_one_piece,
                "frac_of_h2d_link": e2e_value / world / h2d_gbs,
                "host_fill_only_GBps": cal["fill_only"], "host_fill_plus_h2d_GBps": cal["fill_plus_h2d"],
                "bound": bound_name,
                "bound_GBps": bound, "frac_of_bound": e2e_value / world / bound,
                "install": {"descriptors_per_launch": k_desc / max(1, k_launches), "us_per_launch": 1e3 * k_ms,
                            "traffic_GBps": achieved, "frac_of_hbm_peak": achieved / hbm_peak if achieved else None,
                            "launches_per_step": k_launches / args.steps}},
        "peak_staging_bytes_per_rank": peak_staging, "staging_law_bytes": W * slot,
        "staging_residual_bytes": [p - W * slot for p in peak_staging],
        "gpu_launches": int(st_val.kernel_launches),
        "roofline": {"bound": "hbm", "kernel": kernel_name,
                     "what": "install launches inside the timed restore steps (one per group of chunks whose copies have landed)",
                     "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                     "frac": (achieved / hbm_peak) if achieved else None,
                     "traffic": traffic, "peak_source": peak_src,
                     "traffic_source": f"ncu dram bytes per payload byte of a 64-descriptor launch of this kernel "
                                       f"({traffic_key[1]} registration: {NCU_DRAM_BYTES_PER_PAYLOAD_BYTE[traffic_key]}) "
                                       f"x the payload of one launch",
                     "launches": k_launches, "avg_launch_ms": k_ms,
                     "in_kernel": {"what": "the same launches timed by the kernel itself: first CTA's start to the last "
                                           "CTA's end (%globaltimer), i.e. without launch and completion latency",
                                   "avg_span_ms": k_span_ms,
                                   "achieved": 2 * per_launch_payload / (k_span_ms / 1e3) / 1e9 if k_span_ms else None,
                                   "frac": 2 * per_launch_payload / (k_span_ms / 1e3) / 1e9 / hbm_peak if k_span_ms else None},
                     "descriptors_per_launch": k_desc / max(1, k_launches),
                     "algorithmic_bytes_per_launch": 2 * per_launch_payload},
        "resident": resident,
        "cpu_baseline": cpu,
        "clocks": clocks,
        # the paper's own figures, on its hardware: context, not a target
        "paper_context": {"hardware": "two DGX Spark nodes, TP = 2, Mooncake remote DRAM over 100 Gb/s RDMA / local SSD",
                          "peak_staging_MiB_per_rank_at_W32": 500.75,
                          "restore_ttft_s_512k_tokens_ssd_fs_concurrency_1_to_4": [43.1, 17.6],
                          "restore_ttft_s_524k_tokens_remote_dram": 16.41},
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_sweep(args):
    """--sweep: end-to-end restore GB/s vs W and vs fill concurrency on the long prefixes (the
    paper's window-law and storage-concurrency experiments: throughput moves, peak staging follows
    W x slot exactly).  The host tier is cyclic: 67 distinct objects per rank, key i -> object i mod 67."""
    import torch
    from paper_2608_17826_b200 import build
    build.build()
    from paper_2608_17826_b200 import binding as B
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    layout = synth.baseline_layout()
    R, P, seed = 2, 67, synth.MASTER_SEED
    objs = {(r, j): synth.chunk_payload(layout, r, j, seed=seed).copy() for r in range(R) for j in range(P)}
    h2d = measure_h2d(torch, dev, layout.chunk_bytes)
    plan = ([(512, W, 0, 0) for W in (2, 4, 8, 16, 32, 64)] + [(1024, W, 0, 0) for W in (8, 16, 32, 64)] +
            [(2048, 32, 0, 0)] + [(512, 32, lc, 0) for lc in (1, 2, 4, 8, 16)] +
            [(512, 8, 0, b) for b in (2, 8, 32)])
    for N, W, lc, batch in plan:
        tok = synth.tokens(N * 256, seed=seed + N)
        payload = {(r, i): objs[(r, i % P)] for r in range(R) for i in range(N)}
        side = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_HOST, load_concurrency=lc,
                    dev_staging_depth=args.depth, install_variant=args.variant, install_batch=batch)
        rc, keys, _, _ = B.bsr_probe(side.ctx, tok, len(tok), seed, False)
        # stamp checksums once per distinct object, reuse them for the other keys
        cks = {}
        for (r, i), o in payload.items():
            if (r, i % P) not in cks:
                assert B.bsr_tier_put(side.ctx, r, keys[i], o, o.size, None, B.BSR_LOC_HOST) == B.BSR_OK
                cks[(r, i % P)] = B.bsr_tier_checksums(side.ctx, r, keys[i], layout.n_groups)[1]
            else:
                assert B.bsr_tier_put(side.ctx, r, keys[i], o, o.size, cks[(r, i % P)], B.BSR_LOC_HOST) == B.BSR_OK
        ms, _, st = timed_steps(torch, None, 1, side, tok, len(tok), seed, False, 3, 3, N)
        nbytes = R * N * layout.chunk_bytes
        n_l = max(1, int(st.install_launches))
        print(json.dumps({"sweep": True, "chunks": N, "W": W, "load_concurrency": lc or "auto",
                          "install_batch": batch or "auto",
                          "restore_GBps": nbytes / ms / 1e6, "per_rank_GBps": nbytes / ms / 1e6 / R,
                          "restore_seconds": ms / 1e3, "frac_of_h2d_link": nbytes / ms / 1e6 / h2d,
                          "h2d_link_GBps_measured": h2d, "windows_per_restore": int(st.windows) // 3,
                          "descriptors_per_install_launch": int(st.install_descriptors) / n_l,
                          "install_us_per_launch": 1e3 * st.install_kernel_ms / n_l,
                          "peak_staging_bytes_per_rank": int(st.peak_staging_bytes[0]),
                          "staging_residual_bytes": int(st.peak_staging_bytes[0]) - W * int(st.slot_bytes)}),
              flush=True)
        side.close()
        del side
        torch.cuda.empty_cache()
    return 0


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start one process per GPU (rank r drives GPU r),
    rendezvous on the loopback address, let rank 0's line through, return the worst exit code."""
    from paper_2608_17826_b200 import build
    build.build()  # once, before the ranks start
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   LOCAL_WORLD_SIZE=str(args.gpus), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.setdefault("NCCL_DEBUG", "INFO")  # the communicator's own log (ranks, transport) goes to stderr
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__), *sys.argv[1:]], env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    worst = 0
    try:
        for p in procs:
            rc = p.wait()
            if rc != 0:
                worst = worst or rc
                for q in procs:       # a rank that failed leaves the others waiting at a barrier
                    if q.poll() is None:
                        q.terminate()
    finally:
        for q in procs:
            if q.poll() is None:
                q.kill()
    return worst


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--load-concurrency", type=int, default=0, help="fill threads (0 = half of this rank's CPUs)")
    ap.add_argument("--depth", type=int, default=0, help="device staging buffers per rank slice (0 = library default)")
    ap.add_argument("--install-batch", type=int, default=0, help="chunk descriptors per install launch (0 = default)")
    ap.add_argument("--variant", type=int, default=0, help="install kernel: 0 auto, 1 vector, 2 bulk copy")
    ap.add_argument("--layout", default="baseline", choices=sorted(LAYOUTS),
                    help="registration geometry (the contract line is the baseline one)")
    ap.add_argument("--window", type=int, default=0, help="window W in chunks (default: the workload's 32; the label says so)")
    ap.add_argument("--chunks", type=int, default=0, help="prefix length in chunks (default: the workload's 128)")
    ap.add_argument("--direct", action="store_true", help="staging-free install (kernel reads the pinned slots)")
    ap.add_argument("--dry-run-one-gpu", action="store_true",
                    help="with --gpus N on a single-GPU box: all ranks share GPU 0, gloo for the commit word; "
                         "checks the multi-process plumbing, the numbers mean nothing")
    ap.add_argument("--sweep", action="store_true", help="e2e GB/s vs W, fill concurrency and launch size (long prefixes)")
    ap.add_argument("--resident-only", action="store_true", help="small profiling runs: the install microbenchmark only")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.sweep:
        return run_sweep(args)
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())

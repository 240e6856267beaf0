#!/usr/bin/env python
"""Benchmark of the bounded-state restore path on B200.

One "step" is one pass of the whole hot path over one synthetic prefix: probe (chunk digests,
key chain, index lookup) -> bounded-window restore (install kernels) -> commit.

  value   restore throughput with the tier objects already resident in HBM (device tier): the
          install kernels read them in place, no host link involved.
  e2e     the same metric through the same C calls with the tier in ordinary HOST memory:
          tier -> pinned W-slot ring -> cudaMemcpyAsync -> device staging -> install, every step.
  roofline  the install kernel against the measured HBM copy bandwidth.
  cpu_baseline  the CPU oracle timed on a bounded sample (reported, not a target).

Usage: python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
Under torchrun (N > 1) every process drives its own GPU with its own copy of the workload
(rank slices are independent units: weak scaling); the only exchange is the one-word commit AND.
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
sys.path.insert(0, ROOT)

from paper_2608_17826_b200 import multi, synth  # noqa: E402

WORKLOAD = dict(name="32768-token prefix, 128 chunks x 16,408,576 B, 2 rank slices, W=32, "
                     "baseline 2-group/99-tensor layout, 64-token blocks",
                n_chunks=128, n_ranks=2, W=32)
# dram read + write bytes per payload byte from the ncu captures of the two install kernels (profiles/)
NCU_DRAM_BYTES_PER_PAYLOAD_BYTE = {"bsr_install_bulk_kernel": 1.957, "bsr_install_vec_kernel": 1.955}
METRIC, UNIT = "restore GB/s (all rank slices; per-rank = value / rank slices)", "GB/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (earlier pool measurement)"


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
def oracle_sample_step(layout, n_ranks, sample_chunks, W, seed):
    """One oracle pass (probe + strict-window restore + commit) over the first `sample_chunks`
    chunks of the workload.  Returns (seconds, bytes moved)."""
    from oracle import bsr_oracle as O
    reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
    tok = synth.tokens(sample_chunks * 256, seed=seed)
    keys = O.prefix_keys(O.chunk_digests(tok, seed), seed, 1)
    tiers = [O.Tier() for _ in range(n_ranks)]
    for r in range(n_ranks):
        for i in range(sample_chunks):
            p = synth.chunk_payload(layout, r, i, seed=seed).copy()
            tiers[r].put(keys[i], p, O.group_checksums(reg, p))
    pools = [synth.pool_blocks(layout, g, sample_chunks) for g in range(reg.n_groups)]
    tables = [[synth.block_table(layout, r, g, sample_chunks, seed=seed) for g in range(reg.n_groups)]
              for r in range(n_ranks)]
    paged = [O.new_paged(reg, pools, synth.CANARY) for _ in range(n_ranks)]
    t0 = time.perf_counter()
    k, hit, n_hit = O.probe(tok, seed, 1, tiers)
    req = O.Request(k[:n_hit], tables, n_ranks, reg.n_groups)
    status, st = O.restore(reg, tiers, req, paged, W)
    exposed = O.commit(reg, req, paged)
    dt = time.perf_counter() - t0
    assert status == O.OK and exposed == sample_chunks
    return dt, n_ranks * sample_chunks * reg.chunk_bytes


def run_reference(args):
    """--impl reference: the oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    layout = synth.baseline_layout()
    sample = 8
    for _ in range(args.warmup):
        oracle_sample_step(layout, WORKLOAD["n_ranks"], sample, WORKLOAD["W"], synth.MASTER_SEED)
    ts, nbytes = [], 0
    for _ in range(args.steps):
        dt, nbytes = oracle_sample_step(layout, WORKLOAD["n_ranks"], sample, WORKLOAD["W"], synth.MASTER_SEED)
        ts.append(dt)
    ms = 1e3 * sum(ts) / len(ts)
    val = nbytes / (ms / 1e3) / 1e9
    desc = f"first {sample} of {WORKLOAD['n_chunks']} chunks x {WORKLOAD['n_ranks']} rank slices per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8/u64", "data": "synthetic",
        "config": {"workload": WORKLOAD["name"], "sample": desc},
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

    def step(self, tok, n_tok, salt, tok_on_device, stream):
        B = self.B
        rc, keys, bm, n_hit = B.bsr_probe(self.ctx, tok, n_tok, salt, tok_on_device)
        assert rc == B.BSR_OK
        if self.req is None:
            rc, self.req = B.bsr_req_create(self.ctx, keys[:n_hit], self.tables)
            assert rc == B.BSR_OK, B.bsr_last_error(self.ctx)
        rc = B.bsr_restore(self.ctx, self.req, stream)
        assert rc == B.BSR_OK, (rc, B.bsr_last_error(self.ctx))
        rc, exposed = B.bsr_commit(self.ctx, self.req)
        assert rc == B.BSR_OK
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
                coll_dev="cuda"):
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        _, exposed = side.step(tok, n_tok, salt, tok_on_device, stream.cuda_stream)
        if world > 1:  # the commit exchange is part of a step: warm its communicator up as well
            multi.commit_across_ranks(exposed, n_chunks, device=coll_dev)
    side.B.bsr_reset_stats(side.ctx)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    ok = True
    for _ in range(steps):
        n_hit, exposed = side.step(tok, n_tok, salt, tok_on_device, stream.cuda_stream)
        ok = ok and n_hit == n_chunks and exposed == n_chunks
        if world > 1:  # request-level commit across GPUs: one word, AND over ranks (Eq. 6)
            ok = ok and multi.commit_across_ranks(exposed, n_chunks, device=coll_dev) == n_chunks
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    if world > 1:
        ms = multi.max_over_ranks(ms, device=coll_dev)
    assert ok, "a step did not expose the full prefix"
    return ms / steps, side.stats()


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

    layout = {"baseline": synth.baseline_layout, "hetero": synth.hetero_layout,
              "mtp_on": synth.mtp_on_layout}[args.layout]()
    R, N, W = WORKLOAD["n_ranks"], args.chunks or WORKLOAD["n_chunks"], WORKLOAD["W"]
    chunk = layout.chunk_bytes
    seed = synth.MASTER_SEED + rank
    salt = seed
    tok = synth.tokens(N * 256, seed=seed)
    payload = {(r, i): synth.chunk_payload(layout, r, i, seed=seed).copy() for r in range(R) for i in range(N)}
    step_bytes = R * N * chunk

    # ---- HBM-resident arm -----------------------------------------------------------------
    d_tok = torch.from_numpy(tok).to(dev)
    res = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_DEVICE, install_variant=args.variant)
    rc, keys, _, _ = B.bsr_probe(res.ctx, d_tok.data_ptr(), len(tok), salt, True)
    assert rc == B.BSR_OK
    res.fill_tier(keys)
    rc, in_use = B.bsr_install_kernel_in_use(res.ctx)
    assert rc == B.BSR_OK
    kernel_name = "bsr_install_vec_kernel" if in_use == B.BSR_INSTALL_VECTOR else "bsr_install_bulk_kernel"
    sampler = ClockSampler(local)
    sampler.start()
    ms_res, st_res = timed_steps(torch, dist, world, res, d_tok.data_ptr(), len(tok), salt, True,
                                 args.steps, args.warmup, N, coll_dev)
    launches = int(st_res.kernel_launches)
    k_launches = int(st_res.install_launches)
    k_ms = st_res.install_kernel_ms / max(1, k_launches)
    res.close()
    del res
    torch.cuda.empty_cache()

    if args.resident_only:  # profiling runs: only the HBM-resident arm, no JSON contract line
        if rank == 0:
            print(json.dumps({"resident_only": True, "chunks": N, "kernel": kernel_name, "ms_per_step": ms_res,
                              "install_launches": k_launches, "avg_launch_ms": k_ms,
                              "GBps": step_bytes / (ms_res / 1e3) / 1e9}))
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- end-to-end arm: tier in host memory, through the pinned W-slot ring ----------------
    h2d_gbs = measure_h2d(torch, dev, chunk)                  # the roofline: copies of one chunk each
    h2d_one_piece = measure_h2d(torch, dev, 1 << 30, reps=3)  # context: a single 1 GiB copy
    if args.load_concurrency == 0 and world > 1:
        # several processes share the host cores: split the library's default (half the hardware threads)
        args.load_concurrency = max(4, min(16, (os.cpu_count() or 8) // 2 // world))
    e2e = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_HOST,
               load_concurrency=args.load_concurrency, dev_staging_depth=args.depth,
               install_variant=args.variant, direct_install=args.direct)
    e2e.fill_tier(keys)
    e2e_steps = max(3, min(args.steps, 10))
    ms_e2e, st_e2e = timed_steps(torch, dist, world, e2e, tok, len(tok), salt, False, e2e_steps,
                                 max(3, min(args.warmup, 3)), N, coll_dev)
    peak_staging = [int(st_e2e.peak_staging_bytes[r]) for r in range(R)]
    slot = int(st_e2e.slot_bytes)
    e2e_install_us = 1e3 * st_e2e.install_kernel_ms / max(1, int(st_e2e.install_launches))
    clocks = sampler.stop()
    # probe alone (token ids in host memory: H2D, digest + chain kernel, D2H of the keys, index lookup)
    t0 = time.perf_counter()
    for _ in range(20):
        B.bsr_probe(e2e.ctx, tok, len(tok), salt, False)
    probe_us = (time.perf_counter() - t0) / 20 * 1e6
    e2e.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    hbm_peak, peak_src = _peaks()
    value = world * step_bytes / (ms_res / 1e3) / 1e9
    e2e_value = world * step_bytes / (ms_e2e / 1e3) / 1e9
    per_launch_payload = step_bytes * args.steps / max(1, k_launches)
    achieved = 2 * per_launch_payload / (k_ms / 1e3) / 1e9 if k_ms > 0 else None
    # dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of a smaller launch
    # (64 chunk descriptors, a quarter of the timed launch; traffic grows in proportion to the
    # descriptors processed): bulk kernel 1.0503 GB + 1.0050 GB for 1.0501 GB of payload = 1.957 B/B,
    # vector kernel 1.0502 GB + 1.0026 GB = 1.955 B/B.
    traffic = NCU_DRAM_BYTES_PER_PAYLOAD_BYTE[kernel_name] * per_launch_payload

    # ---- CPU oracle on a bounded sample -----------------------------------------------------
    del payload  # 4.2 GB of host memory the oracle leg regenerates for itself
    sample = min(N, 128)  # the whole workload: about 10-20 s of single-thread numpy work
    dt, nbytes = oracle_sample_step(layout, R, sample, W, seed)
    cpu = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": 1, "host_cores_available": os.cpu_count(),
           "kind": "oracle",
           "sample": f"first {sample} of {N} chunks x {R} rank slices, one pass ({dt:.1f} s)"}

    out = {
        **({"dry_run_one_gpu": True} if args.dry_run_one_gpu else {}),
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_res, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8 payload, u64 checksums/digests", "data": "synthetic",
        "config": {"workload": WORKLOAD["name"] if N == WORKLOAD["n_chunks"] else f"REDUCED to {N} chunks: " + WORKLOAD["name"],
                   "rank_slices_per_gpu": R, "W": W,
                   "l2": "inputs (4.2 GB per step) are larger than L2; no flush needed",
                   "value_path": "tier resident in HBM, probe+restore+commit",
                   "e2e_path": ("host tier -> pinned ring -> install kernel reads the slots over the link; " if args.direct else
                                "host tier -> pinned ring -> H2D -> install; ") + f"load_concurrency="
                               f"{args.load_concurrency}, dev_staging_depth={args.depth}"},
        "per_rank_GBps": value / (world * R),
        "restore_seconds": ms_res / 1e3,
        "probe_host_us": probe_us,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e, "steps": e2e_steps,
                "h2d_bytes_per_step": step_bytes + len(tok) * 4,
                "d2h_bytes_per_step": N * 8 + R * layout.n_groups * N * 12,
                "per_rank_GBps": e2e_value / (world * R), "restore_seconds": ms_e2e / 1e3,
                "install_us_per_chunk_launch": e2e_install_us,
                "h2d_link_GBps_measured": h2d_gbs, "h2d_link_GBps_single_1GiB_copy": h2d_one_piece,
                "frac_of_h2d_link": e2e_value / world / h2d_gbs},
        "peak_staging_bytes_per_rank": peak_staging, "staging_law_bytes": W * slot,
        "staging_residual_bytes": [p - W * slot for p in peak_staging],
        "gpu_launches": launches,
        "roofline": {"bound": "hbm",
                     "kernel": kernel_name,
                     "achieved": achieved,
                     "peak": hbm_peak, "unit": "GB/s", "frac": (achieved / hbm_peak) if achieved else None,
                     "traffic": traffic, "peak_source": peak_src,
                     "launches": k_launches, "avg_launch_ms": k_ms,
                     "algorithmic_bytes_per_launch": 2 * per_launch_payload},
        "cpu_baseline": cpu,
        "clocks": clocks,
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
    plan = ([(N, W, 0) for N in (512, 1024) for W in (8, 16, 32, 64)] + [(2048, 32, 0)] +
            [(512, 32, lc) for lc in (1, 2, 4, 8, 16)])
    for N, W, lc in plan:
        tok = synth.tokens(N * 256, seed=seed + N)
        payload = {(r, i): objs[(r, i % P)] for r in range(R) for i in range(N)}
        side = Side(B, torch, dev, layout, R, N, W, payload, B.BSR_LOC_HOST, load_concurrency=lc,
                    dev_staging_depth=args.depth, install_variant=args.variant)
        rc, keys, _, _ = B.bsr_probe(side.ctx, tok, len(tok), seed, False)
        # stamp checksums once per distinct object, reuse them for the other keys
        cks = {}
        for (r, i), o in payload.items():
            if (r, i % P) not in cks:
                assert B.bsr_tier_put(side.ctx, r, keys[i], o, o.size, None, B.BSR_LOC_HOST) == B.BSR_OK
                cks[(r, i % P)] = B.bsr_tier_checksums(side.ctx, r, keys[i], layout.n_groups)[1]
            else:
                assert B.bsr_tier_put(side.ctx, r, keys[i], o, o.size, cks[(r, i % P)], B.BSR_LOC_HOST) == B.BSR_OK
        ms, st = timed_steps(torch, None, 1, side, tok, len(tok), seed, False, 3, 3, N)
        nbytes = R * N * layout.chunk_bytes
        print(json.dumps({"sweep": True, "chunks": N, "W": W, "load_concurrency": lc or "auto",
                          "restore_GBps": nbytes / ms / 1e6, "per_rank_GBps": nbytes / ms / 1e6 / R,
                          "restore_seconds": ms / 1e3, "frac_of_h2d_link": nbytes / ms / 1e6 / h2d,
                          "h2d_link_GBps_measured": h2d, "windows_per_restore": int(st.windows) // 3,
                          "peak_staging_bytes_per_rank": int(st.peak_staging_bytes[0]),
                          "staging_residual_bytes": int(st.peak_staging_bytes[0]) - W * int(st.slot_bytes)}),
              flush=True)
        side.close()
        del side
        torch.cuda.empty_cache()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--load-concurrency", type=int, default=0, help="fill threads (0 = auto)")
    ap.add_argument("--depth", type=int, default=4)
    ap.add_argument("--variant", type=int, default=0, help="install kernel: 0 auto, 1 vector, 2 bulk copy")
    ap.add_argument("--layout", default="baseline", choices=["baseline", "hetero", "mtp_on"],
                    help="registration geometry (the contract line is the baseline one)")
    ap.add_argument("--chunks", type=int, default=0, help="prefix length in chunks (default: the workload's 128)")
    ap.add_argument("--direct", action="store_true", help="e2e arm: staging-free install (kernel reads the pinned slots)")
    ap.add_argument("--dry-run-one-gpu", action="store_true",
                    help="under torchrun on a single-GPU box: all ranks share GPU 0, gloo for the commit word; "
                         "checks the multi-process plumbing, the numbers mean nothing")
    ap.add_argument("--sweep", action="store_true", help="e2e GB/s vs W and vs fill concurrency (long prefixes)")
    ap.add_argument("--resident-only", action="store_true", help="small profiling runs: skip e2e and CPU legs")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.sweep:
        return run_sweep(args)
    return run_reference(args) if args.impl == "reference" else run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())

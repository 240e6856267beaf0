"""World-size-2 tests of the multi-process plumbing on CPU (gloo): sharding of rank slices, the
commit AND across processes, max-over-ranks timing.  The oracle plays each process's restore."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_17826_b200 import multi, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, fail_on, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import bsr_oracle as O
        layout = synth.tiny_layout()
        reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
        R_total, N, W = 4, 6, 2
        mine = multi.slices_of(rank, world, R_total)
        tok = synth.tokens(N * 256, seed=9)
        keys = O.prefix_keys(O.chunk_digests(tok, 9), 9, 1)
        tiers, tables, paged = [], [], []
        pools = [synth.pool_blocks(layout, g, N) for g in range(reg.n_groups)]
        for r in mine:
            t = O.Tier()
            for i in range(N):
                p = synth.chunk_payload(layout, r, i, seed=9).copy()
                ck = O.group_checksums(reg, p)
                if fail_on == (r, i):
                    p[100] ^= 1
                t.put(keys[i], p, ck)
            tiers.append(t)
            tables.append([synth.block_table(layout, r, g, N, seed=9) for g in range(reg.n_groups)])
            paged.append(O.new_paged(reg, pools, synth.CANARY))
        req = O.Request(keys, tables, len(mine), reg.n_groups)
        status, st = O.restore(reg, tiers, req, paged, W)
        local = O.commit(reg, req, paged)
        exposed = multi.commit_across_ranks(local, N)
        if exposed == 0:
            O.invalidate(reg, req, paged, scrub=False)
        slowest = multi.max_over_ranks(10.0 + rank)
        np.save(os.path.join(out_dir, f"r{rank}.npy"),
                np.array([len(mine), status, local, exposed, int(req.valid.any()), slowest]))
    finally:
        dist.destroy_process_group()


def _run(fail_on, tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, fail_on, str(tmp_path)), nprocs=2, join=True)
    return [np.load(tmp_path / f"r{r}.npy") for r in range(2)]


def test_slices_partition_the_ranks():
    for world in (1, 2, 3, 8):
        for n in (1, 2, 4, 8):
            got = sorted(r for p in range(world) for r in multi.slices_of(p, world, n))
            assert got == list(range(n))


def test_commit_and_across_two_processes_all_healthy(tmp_path):
    a, b = _run(None, tmp_path)
    for x in (a, b):
        assert x[0] == 2 and x[1] == 0 and x[2] == 6 and x[3] == 6 and x[4] == 1 and x[5] == 11.0


def test_one_process_fault_collapses_the_prefix_on_both(tmp_path):
    # slice 3 lives on process 1; its chunk 4 is corrupted (a fault after two good windows)
    a, b = _run((3, 4), tmp_path)
    assert a[1] == 0 and a[2] == 6          # process 0 was locally healthy ...
    assert b[1] == -3 and b[2] == 0         # ... process 1 failed its checksum
    assert a[3] == 0 and b[3] == 0          # request-level commit: zero on both
    assert a[4] == 0 and b[4] == 0          # and every validity bit is cleared everywhere


def test_single_process_needs_no_process_group():
    assert multi.commit_across_ranks(5, 5) == 5
    assert multi.commit_across_ranks(0, 5) == 0
    assert multi.max_over_ranks(3.5) == 3.5


def test_cpu_share_splits_each_numa_node_among_the_ranks_whose_gpu_hangs_off_it():
    """Eight processes on a two-socket host: every rank keeps a quarter of its GPU's node and no CPU
    is handed out twice; without node information the allowed CPUs are split evenly."""
    n0 = list(range(0, 16)) + list(range(32, 48))
    n1 = list(range(16, 32)) + list(range(48, 64))
    shares = [multi.cpu_share(list(range(64)), [n0] * 4 + [n1] * 4, l) for l in range(8)]
    assert all(len(s) == 8 for s in shares)
    assert sorted(c for s in shares for c in s) == list(range(64))
    assert all(set(s) <= set(n0) for s in shares[:4]) and all(set(s) <= set(n1) for s in shares[4:])
    # an affinity mask narrower than the node is respected
    assert multi.cpu_share(list(range(8)), [n0, n0], 1) == [4, 5, 6, 7]
    # no node known: an even split; more ranks than CPUs: everyone still gets one
    assert [multi.cpu_share(list(range(16)), [None] * 2, l) for l in range(2)] == [list(range(8)), list(range(8, 16))]
    assert [multi.cpu_share([0, 1], [None] * 4, l) for l in range(4)] == [[0], [0], [1], [1]]


def test_slices_of_a_job_are_dealt_round_robin_and_cover_the_job():
    for world in (1, 2, 4, 8):
        got = [multi.slices_of(p, world, 2 * world) for p in range(world)]
        assert sorted(r for s in got for r in s) == list(range(2 * world))
        assert all(s == [p, p + world] for p, s in enumerate(got))

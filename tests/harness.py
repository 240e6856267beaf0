"""Builds the same seeded case for the oracle and for the CUDA library, and compares them."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth


class Case:
    """Seeded inputs of one restore: payloads, keys, tables.  Payload arrays are held once and
    shared (read-only) by the oracle tier and the library's borrowed host tier."""

    def __init__(self, layout: synth.Layout, R: int, N: int, seed: int, salt: int | None = None,
                 reg_id: int = 1, present=None, tail_tokens: int = 0):
        self.layout, self.R, self.N, self.seed = layout, R, N, seed
        self.salt = seed if salt is None else salt
        self.reg_id = reg_id
        self.reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
        self.G = self.reg.n_groups
        self.tok = synth.tokens(N * 256 + tail_tokens, seed=seed)
        self.keys = O.prefix_keys(O.chunk_digests(self.tok, self.salt), self.salt, reg_id)
        self.payload: dict[tuple[int, int], np.ndarray] = {}
        self.cks: dict[tuple[int, int], list[int]] = {}
        todo = [(r, i) for r in range(R) for i in range(N) if present is None or present(r, i)]

        def make(ri):
            p = synth.chunk_payload(layout, ri[0], ri[1], seed=seed).copy()
            return ri, p, O.group_checksums(self.reg, p)

        if len(todo) * layout.chunk_bytes > (1 << 30):
            # a long prefix: draw the chunks (and stamp their stored checksums) on several threads
            with ThreadPoolExecutor(min(16, os.cpu_count() or 4)) as ex:
                made = list(ex.map(make, todo))
        else:
            made = [make(ri) for ri in todo]
        for ri, p, ck in made:
            self.payload[ri] = p
            self.cks[ri] = ck
        self.pools = [synth.pool_blocks(layout, g, N) for g in range(self.G)]
        self.tables = [[synth.block_table(layout, r, g, N, seed=seed) for g in range(self.G)]
                       for r in range(R)]

    # ---- oracle side
    def oracle_tiers(self):
        tiers = [O.Tier() for _ in range(self.R)]
        for (r, i), p in self.payload.items():
            tiers[r].put(self.keys[i], p, self.cks[(r, i)])
        return tiers

    def oracle_paged(self):
        return [O.new_paged(self.reg, self.pools, synth.CANARY) for _ in range(self.R)]

    def tables_prefix(self, n_adv: int):
        return [[t[: n_adv * self.reg.blocks_per_chunk(g)] for g, t in enumerate(tr)]
                for tr in self.tables]


class GpuSide:
    """The library's view of a Case: paged pools in device memory (torch), a context, the tier."""

    def __init__(self, case: Case, W: int, *, location=None, compute_ck=False, **cfg):
        import torch

        from paper_2608_17826_b200 import binding as B

        self.B, self.torch, self.case = B, torch, case
        self.dev = torch.device("cuda:0")
        rc, self.ctx = B.bsr_ctx_create(W, case.R, reg_id=case.reg_id, **cfg)
        assert rc == B.BSR_OK, rc
        self.paged = []
        for r in range(case.R):
            per = [torch.full((case.pools[g], case.layout.block_tokens[g], e), synth.CANARY,
                              dtype=torch.uint8, device=self.dev) for g, e in case.layout.tensors]
            self.paged.append(per)
            groups = [(case.layout.block_tokens[g], case.pools[g]) for g in range(case.G)]
            tensors = [(g, e, per[l].data_ptr()) for l, (g, e) in enumerate(case.layout.tensors)]
            rc = B.bsr_register(self.ctx, r, groups, tensors)
            assert rc == B.BSR_OK, (rc, B.bsr_last_error(self.ctx))
        self.location = B.BSR_LOC_HOST if location is None else location
        self.dev_objs = {}
        for (r, i), p in case.payload.items():
            ck = None if compute_ck else case.cks[(r, i)]
            if self.location == B.BSR_LOC_DEVICE:
                t = torch.from_numpy(p).to(self.dev)
                self.dev_objs[(r, i)] = t
                rc = B.bsr_tier_put(self.ctx, r, case.keys[i], t.data_ptr(), p.size, ck, B.BSR_LOC_DEVICE)
            else:
                rc = B.bsr_tier_put(self.ctx, r, case.keys[i], p, p.size, ck, B.BSR_LOC_HOST)
            assert rc == B.BSR_OK, (rc, B.bsr_last_error(self.ctx))
        torch.cuda.synchronize()
        self.req = None

    def probe(self, tok_on_device=False):
        B, c = self.B, self.case
        if tok_on_device:
            t = self.torch.from_numpy(c.tok).to(self.dev)
            self.torch.cuda.synchronize()
            return B.bsr_probe(self.ctx, t.data_ptr(), len(c.tok), c.salt, True)
        return B.bsr_probe(self.ctx, c.tok, len(c.tok), c.salt, False)

    def request(self, keys, n_adv):
        flat = [t for tr in self.case.tables_prefix(n_adv) for t in tr]
        rc, self.req = self.B.bsr_req_create(self.ctx, keys[:n_adv], flat)
        assert rc == self.B.BSR_OK, (rc, self.B.bsr_last_error(self.ctx))
        return self.req

    def restore(self):
        return self.B.bsr_restore(self.ctx, self.req, None)

    def commit(self):
        rc, n = self.B.bsr_commit(self.ctx, self.req)
        assert rc == self.B.BSR_OK
        return n

    def bitmap(self, n_adv):
        rc, bm = self.B.bsr_req_bitmap(self.ctx, self.req, self.case.R, self.case.G, n_adv)
        assert rc == self.B.BSR_OK
        return bm

    def stats(self):
        rc, st = self.B.bsr_get_stats(self.ctx)
        assert rc == self.B.BSR_OK
        return st

    def paged_numpy(self, r, l):
        return self.paged[r][l].cpu().numpy()

    def close(self):
        if self.req is not None:
            self.B.bsr_req_release(self.ctx, self.req)
            self.req = None
        if self.ctx is not None:
            self.B.bsr_ctx_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()


def assert_paged_equal(gpu: GpuSide, oracle_paged):
    c = gpu.case
    for r in range(c.R):
        for l in range(len(c.layout.tensors)):
            got = gpu.paged_numpy(r, l)
            if not np.array_equal(got, oracle_paged[r][l]):
                bad = np.argwhere(got != oracle_paged[r][l])
                raise AssertionError(f"paged mismatch rank {r} tensor {l}: {len(bad)} bytes, first at {bad[0]}")


def assert_paged_equal_on_device(gpu: GpuSide, oracle_paged_dev):
    """The same comparison, every byte of every paged tensor, against a copy of the oracle's image
    that already sits in device memory (long prefixes: nothing is downloaded)."""
    torch, c = gpu.torch, gpu.case
    for r in range(c.R):
        for l in range(len(c.layout.tensors)):
            if not torch.equal(gpu.paged[r][l], oracle_paged_dev[r][l]):
                bad = (gpu.paged[r][l] != oracle_paged_dev[r][l]).nonzero()
                raise AssertionError(f"paged mismatch rank {r} tensor {l}: {len(bad)} bytes, first at {bad[0].tolist()}")


def run_oracle(case: Case, W: int, n_adv: int | None = None, tiers=None, fetch_fault=None):
    """probe + restore + commit on the oracle.  Returns a dict of everything compared."""
    tiers = case.oracle_tiers() if tiers is None else tiers
    keys, hit, n_hit = O.probe(case.tok, case.salt, case.reg_id, tiers)
    n_adv = n_hit if n_adv is None else n_adv
    paged = case.oracle_paged()
    req = O.Request(keys[:n_adv], case.tables_prefix(n_adv), case.R, case.G)
    status, st = O.restore(case.reg, tiers, req, paged, W, fetch_fault=fetch_fault)
    exposed = O.commit(case.reg, req, paged)
    return dict(keys=keys, hit=hit, n_hit=n_hit, n_adv=n_adv, paged=paged, req=req, status=status,
                stats=st, exposed=exposed, tiers=tiers)

"""Request-level recovery on the GPU path against the oracle: the paper's failure table over two
tiers, lower-tier fallback, tier loss between probe and restore, and the force-local marker."""
import numpy as np
import pytest

from conftest import read_golden
from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

pytestmark = pytest.mark.gpu
R, N, W, SEED, RID = 2, 9, 3, 78, 9001


class TwoTier:
    """The same two-tier case on both sides."""

    def __init__(self, remote_has=lambda r, i: True, ssd_has=lambda r, i: True):
        import torch
        from paper_2608_17826_b200 import binding as B
        self.B, self.torch = B, torch
        self.layout = synth.tiny_layout()
        L = self.layout
        self.reg = O.Registration(list(L.block_tokens), list(L.tensors))
        self.tok = synth.tokens(N * 256, seed=SEED)
        self.keys = O.prefix_keys(O.chunk_digests(self.tok, SEED), SEED, 1)
        self.pools = [synth.pool_blocks(L, g, N) for g in range(self.reg.n_groups)]
        self.tables = [[synth.block_table(L, r, g, N, seed=SEED) for g in range(self.reg.n_groups)] for r in range(R)]
        rc, self.ctx = B.bsr_ctx_create(W, R, reg_id=1)
        assert rc == B.BSR_OK
        dev = torch.device("cuda:0")
        self.gpaged = []
        for r in range(R):
            per = [torch.full((self.pools[g], L.block_tokens[g], e), synth.CANARY, dtype=torch.uint8, device=dev)
                   for g, e in L.tensors]
            self.gpaged.append(per)
            assert B.bsr_register(self.ctx, r, [(L.block_tokens[g], self.pools[g]) for g in range(self.reg.n_groups)],
                                  [(g, e, per[l].data_ptr()) for l, (g, e) in enumerate(L.tensors)]) == B.BSR_OK
        self.eng = O.Engine([[O.Tier() for _ in range(R)] for _ in range(2)], [True, True])
        self.payload = {}
        for t, has in ((0, remote_has), (1, ssd_has)):
            for r in range(R):
                for i in range(N):
                    if not has(r, i):
                        continue
                    p = synth.chunk_payload(L, r, i, seed=SEED).copy()
                    ck = O.group_checksums(self.reg, p)
                    self.payload[(t, r, i)] = p
                    self.eng.tiers[t][r].put(self.keys[i], p, ck)
                    assert B.bsr_tier_put_at(self.ctx, t, r, self.keys[i], p, p.size, ck) == B.BSR_OK
        self.opaged = [O.new_paged(self.reg, self.pools, synth.CANARY) for _ in range(R)]
        self.req = None

    def set_available(self, tier, up):
        self.eng.available[tier] = up
        assert self.B.bsr_tier_set_available(self.ctx, tier, up) == self.B.BSR_OK

    def probe_both(self, rid=RID):
        B = self.B
        ok, ohit, on, otier = O.probe_request(self.eng, rid, self.tok, SEED, 1)
        rc, k, bm, n, tier = B.bsr_probe_request(self.ctx, rid, self.tok, len(self.tok), SEED)
        assert rc == B.BSR_OK and np.array_equal(k, ok) and np.array_equal(bm, O.pack_bits(ohit))
        assert (n, tier) == (on, otier)
        return k, n, tier

    def serve_both(self, rid=RID, inject=None, fetch_fault=None):
        """probe -> bind -> restore -> commit on both sides; returns (exposed, tier, status)."""
        B = self.B
        keys, n_hit, tier = self.probe_both(rid)
        if n_hit == 0:
            return 0, tier, None
        tabs = [[t[: n_hit * self.reg.blocks_per_chunk(g)] for g, t in enumerate(tr)] for tr in self.tables]
        oreq = O.Request(keys[:n_hit], tabs, R, self.reg.n_groups)
        ostatus, ost = O.restore_request(self.eng, rid, tier, self.reg, oreq, self.opaged, W, fetch_fault=fetch_fault)
        oexp = O.commit(self.reg, oreq, self.opaged)
        if self.req is not None:
            B.bsr_req_release(self.ctx, self.req)
        rc, self.req = B.bsr_req_create(self.ctx, keys[:n_hit], [t for tr in tabs for t in tr])
        assert rc == B.BSR_OK
        assert B.bsr_req_bind(self.ctx, self.req, rid, tier) == B.BSR_OK
        if inject:
            B.bsr_test_inject(self.ctx, *inject)
        status = B.bsr_restore(self.ctx, self.req, None)
        rc, exposed = B.bsr_commit(self.ctx, self.req)
        assert status == ostatus and exposed == oexp
        rc, bm = B.bsr_req_bitmap(self.ctx, self.req, R, self.reg.n_groups, n_hit)
        assert np.array_equal(bm, oreq.bitmap())
        assert B.bsr_request_is_force_local(self.ctx, rid) == (B.BSR_OK, rid in self.eng.force_local)
        if status == B.BSR_OK:
            for r in range(R):
                for l in range(len(self.layout.tensors)):
                    assert np.array_equal(self.gpaged[r][l].cpu().numpy(), self.opaged[r][l])
        return exposed, tier, status

    def close(self):
        if self.req is not None:
            self.B.bsr_req_release(self.ctx, self.req)
        self.B.bsr_ctx_destroy(self.ctx)


def test_failure_table_rows_on_two_tiers():
    want = {k: (N if v == "full" else 0) for k, v in read_golden("failure_table.txt").items()}
    c = TwoTier()
    try:
        B = c.B
        assert c.serve_both() == (want["remote_healthy"], 0, B.BSR_OK)
        st = B.bsr_get_stats(c.ctx)[1]
        assert st.bytes_restored_by_tier[0] == R * N * c.reg.chunk_bytes and st.bytes_restored_by_tier[1] == 0
    finally:
        c.close()
    c = TwoTier()
    try:
        B = c.B
        c.set_available(0, False)
        assert c.serve_both() == (want["remote_unavailable_ssd_healthy"], 1, B.BSR_OK)
        st = B.bsr_get_stats(c.ctx)[1]
        assert st.bytes_restored_by_tier[0] == 0 and st.bytes_restored_by_tier[1] == R * N * c.reg.chunk_bytes
        c.set_available(1, False)
        assert c.serve_both(rid=RID + 1) == (want["remote_and_ssd_absent"], -1, None)
    finally:
        c.close()
    c = TwoTier()
    try:
        B = c.B
        got = c.serve_both(inject=(B.BSR_INJECT_FILL_ERROR, 1, 0, W + 1, 0),
                           fetch_fault=lambda r, i: O.ERR_TRANSFER if (r, i) == (1, W + 1) else None)
        assert got == (want["one_rank_remote_restore_fault"], 0, B.BSR_ERR_TRANSFER)
        # marked: the next admission pass reports zero although both tiers could serve it
        assert c.serve_both() == (0, -1, None)
        assert c.probe_both(rid=RID + 7)[1:] == (N, 0)          # other requests are unaffected
        assert B.bsr_request_done(c.ctx, RID) == B.BSR_OK
        O.request_done(c.eng, RID)
        assert c.serve_both() == (N, 0, B.BSR_OK)               # after teardown / RUNNING admission
    finally:
        c.close()


def test_lower_tier_is_chosen_for_the_longer_prefix_and_tier_loss_fails_closed():
    c = TwoTier(remote_has=lambda r, i: i < 5 and not (r == 1 and i == 2))
    try:
        B = c.B
        assert c.probe_both()[1:] == (N, 1)                     # remote: 2 chunks, lower tier: all 9
        c.set_available(1, False)
        assert c.probe_both()[1:] == (2, 0)
        c.set_available(1, True)
        # the lower tier disappears between probe and restore
        keys, n_hit, tier = c.probe_both()
        assert tier == 1
        rc, c.req = B.bsr_req_create(c.ctx, keys[:n_hit], [t for tr in c.tables for t in tr])
        assert B.bsr_req_bind(c.ctx, c.req, RID, tier) == B.BSR_OK
        c.set_available(1, False)
        oreq = O.Request(keys[:n_hit], c.tables, R, c.reg.n_groups)
        assert O.restore_request(c.eng, RID, tier, c.reg, oreq, c.opaged, W)[0] == O.ERR_TRANSFER
        assert B.bsr_restore(c.ctx, c.req, None) == B.BSR_ERR_TRANSFER
        assert B.bsr_commit(c.ctx, c.req) == (B.BSR_OK, 0)
        assert B.bsr_request_is_force_local(c.ctx, RID) == (B.BSR_OK, True)
        for r in range(R):                                      # nothing was written
            for l in range(len(c.layout.tensors)):
                assert bool((c.gpaged[r][l] == synth.CANARY).all())
    finally:
        c.close()


def test_file_backed_lower_tier_through_the_fetch_adapter(tmp_path):
    """The lower tier lives in files (the paper's local-SSD tier): objects are indexed without bytes
    and a fetch function reads each piece straight into the pinned slot, several reads in flight.
    The remote tier is down, so the whole request is served from the files, bit-exactly; a read
    error on one rank fails the request closed."""
    import ctypes
    import os
    import torch
    from harness import Case, assert_paged_equal, run_oracle
    from paper_2608_17826_b200 import binding as B

    layout = synth.baseline_layout()                          # 16.4 MB chunks: two fill pieces each
    Rk, Nk, Wk = 2, 5, 2
    case = Case(layout, Rk, Nk, seed=79)
    ora = run_oracle(case, Wk)
    files = {}
    for (r, i), p in case.payload.items():
        path = tmp_path / f"r{r}_k{int(case.keys[i]):016x}.bin"
        p.tofile(path)
        files[(r, int(case.keys[i]))] = os.open(path, os.O_RDONLY)
    calls, fail_on = [], [None]

    def fetch(user, tier, rank, key, offset, length, dst):
        try:
            calls.append((tier, rank, key, offset, length))
            if fail_on[0] == (rank, key):
                return 5
            data = os.pread(files[(rank, key)], length, offset)
            if len(data) != length:
                return 1
            ctypes.memmove(dst, data, length)
            return 0
        except Exception:                                      # never let an exception read as success
            return 2

    cb = B.BSR_FETCH_FN(fetch)
    rc, ctx = B.bsr_ctx_create(Wk, Rk, reg_id=case.reg_id, load_concurrency=4)
    assert rc == B.BSR_OK
    dev = torch.device("cuda:0")
    paged = []
    try:
        for r in range(Rk):
            per = [torch.full((case.pools[g], layout.block_tokens[g], e), synth.CANARY, dtype=torch.uint8, device=dev)
                   for g, e in layout.tensors]
            paged.append(per)
            assert B.bsr_register(ctx, r, [(layout.block_tokens[g], case.pools[g]) for g in range(case.G)],
                                  [(g, e, per[l].data_ptr()) for l, (g, e) in enumerate(layout.tensors)]) == B.BSR_OK
        # an object without bytes needs an adapter on its tier
        assert B.bsr_tier_put_at(ctx, 1, 0, case.keys[0], None, layout.chunk_bytes, case.cks[(0, 0)]) == B.BSR_ERR_INVALID
        assert B.bsr_tier_set_fetch(ctx, 1, cb) == B.BSR_OK
        for (r, i) in case.payload:
            assert B.bsr_tier_put_at(ctx, 1, r, case.keys[i], None, layout.chunk_bytes, case.cks[(r, i)]) == B.BSR_OK
        assert B.bsr_tier_set_available(ctx, 0, False) == B.BSR_OK           # remote store is down
        rc, keys, bm, n_hit, tier = B.bsr_probe_request(ctx, 31, case.tok, len(case.tok), case.salt)
        assert (rc, n_hit, tier) == (B.BSR_OK, Nk, 1) and not calls        # probe fetched nothing
        flat = [t for tr in case.tables for t in tr]
        rc, req = B.bsr_req_create(ctx, keys, flat)
        assert rc == B.BSR_OK and B.bsr_req_bind(ctx, req, 31, tier) == B.BSR_OK
        assert B.bsr_restore(ctx, req, None) == B.BSR_OK, B.bsr_last_error(ctx)
        assert B.bsr_commit(ctx, req) == (B.BSR_OK, Nk)

        class _G:                                                           # adapter for assert_paged_equal
            pass
        g = _G()
        g.case, g.paged_numpy = case, (lambda r, l: paged[r][l].cpu().numpy())
        assert_paged_equal(g, ora["paged"])
        st = B.bsr_get_stats(ctx)[1]
        assert st.bytes_restored_by_tier[1] == Rk * Nk * layout.chunk_bytes and st.peak_staging_bytes[0] == Wk * layout.chunk_bytes
        # every byte of every object was requested exactly once, in pieces of at most 8 MiB
        got = {}
        for (t, r, k, off, ln) in calls:
            assert t == 1 and ln <= 8 << 20
            got.setdefault((r, k), []).append((off, ln))
        assert len(got) == Rk * Nk
        for pieces in got.values():
            pieces.sort()
            assert pieces[0][0] == 0 and sum(ln for _, ln in pieces) == layout.chunk_bytes
            assert all(a[0] + a[1] == b[0] for a, b in zip(pieces, pieces[1:]))
        # ... and exactly the pieces the library's host-only plan lists for this restore
        rc, plan = B.bsr_plan_pieces(layout.chunk_bytes, Nk, Rk, 4)
        assert rc == B.BSR_OK
        key_to_chunk = {int(k): i for i, k in enumerate(case.keys[:Nk])}
        assert sorted((key_to_chunk[k], r, off, ln) for (_, r, k, off, ln) in calls) == \
            sorted((int(q["chunk"]), int(q["rank"]), int(q["offset"]), int(q["bytes"])) for q in plan)
        # a read error on one rank: zero exposure, marker set
        fail_on[0] = (1, int(case.keys[3]))
        assert B.bsr_restore(ctx, req, None) == B.BSR_ERR_TRANSFER
        assert B.bsr_commit(ctx, req) == (B.BSR_OK, 0)
        assert B.bsr_request_is_force_local(ctx, 31) == (B.BSR_OK, True)
        B.bsr_req_release(ctx, req)
    finally:
        B.bsr_ctx_destroy(ctx)
        for fd in files.values():
            os.close(fd)

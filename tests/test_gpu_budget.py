"""Concurrent restores under one admission budget B (slots per rank shared by all restores in
flight) on the GPU path, against the oracle's synchronous-round model: same bytes, bitmaps and
exposure; aggregate peak staging never above B x slot; a failing request fails alone."""
import threading

import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

pytestmark = pytest.mark.gpu
R = 2


def _medium_layout():
    """1 MiB chunks: long enough restores to overlap, small enough for a full oracle comparison."""
    return synth.Layout("medium", [64, 16], [(0, 2048)] + [(1, 512)] * 4)


class TwoRequests:
    def __init__(self, Ns, W, B, corrupt=None, **cfg):
        import torch
        from paper_2608_17826_b200 import binding as B_
        self.B, self.torch = B_, torch
        self.layout = L = _medium_layout()
        self.reg = reg = O.Registration(list(L.block_tokens), list(L.tensors))
        self.Ns, self.W, self.budget = Ns, W, B
        total = sum(Ns)
        self.pools = [synth.pool_blocks(L, g, total) for g in range(reg.n_groups)]
        big = [[synth.block_table(L, r, g, total, seed=6) for g in range(reg.n_groups)] for r in range(R)]
        rc, self.ctx = B_.bsr_ctx_create(W, R, reg_id=1, budget_slots=B, **cfg)
        assert rc == B_.BSR_OK
        dev = torch.device("cuda:0")
        self.gpaged = []
        for r in range(R):
            per = [torch.full((self.pools[g], L.block_tokens[g], e), synth.CANARY, dtype=torch.uint8, device=dev)
                   for g, e in L.tensors]
            self.gpaged.append(per)
            assert B_.bsr_register(self.ctx, r, [(L.block_tokens[g], self.pools[g]) for g in range(reg.n_groups)],
                                   [(g, e, per[l].data_ptr()) for l, (g, e) in enumerate(L.tensors)]) == B_.BSR_OK
        self.tiers = [O.Tier() for _ in range(R)]
        self.oreqs, self.greqs, self.payload = [], [], {}
        first = 0
        for k, N in enumerate(Ns):
            tok = synth.tokens(N * 256, seed=200 + k)
            keys = O.prefix_keys(O.chunk_digests(tok, 4), 4, 1)
            for r in range(R):
                for i in range(N):
                    p = synth.chunk_payload(L, r, 10000 * k + i, seed=6).copy()
                    ck = O.group_checksums(reg, p)
                    if corrupt == (k, r, i):
                        p[12345] ^= 4
                    self.payload[(k, r, i)] = p
                    self.tiers[r].put(keys[i], p, ck)
                    assert B_.bsr_tier_put(self.ctx, r, keys[i], p, p.size, ck) == B_.BSR_OK
            tabs = [[big[r][g][first * reg.blocks_per_chunk(g):(first + N) * reg.blocks_per_chunk(g)]
                     for g in range(reg.n_groups)] for r in range(R)]
            first += N
            self.oreqs.append(O.Request(keys, tabs, R, reg.n_groups))
            rc, gq = B_.bsr_req_create(self.ctx, keys, [t for tr in tabs for t in tr])
            assert rc == B_.BSR_OK, B_.bsr_last_error(self.ctx)
            self.greqs.append(gq)
        self.opaged = [O.new_paged(reg, self.pools, synth.CANARY) for _ in range(R)]

    def run_gpu_concurrently(self):
        out = [None] * len(self.greqs)
        gate = threading.Barrier(len(self.greqs))

        def work(k):
            gate.wait()
            out[k] = self.B.bsr_restore(self.ctx, self.greqs[k], None)   # ctypes releases the GIL

        ts = [threading.Thread(target=work, args=(k,)) for k in range(len(self.greqs))]
        [t.start() for t in ts]
        [t.join() for t in ts]
        return out

    def compare(self, statuses):
        B = self.B
        ostatus, opeak, rounds = O.restore_concurrent(self.reg, self.tiers, self.oreqs, self.opaged, self.W, self.budget)
        assert statuses == ostatus
        for k, (gq, oq) in enumerate(zip(self.greqs, self.oreqs)):
            assert B.bsr_commit(self.ctx, gq) == (B.BSR_OK, O.commit(self.reg, oq, self.opaged))
            rc, bm = B.bsr_req_bitmap(self.ctx, gq, R, self.reg.n_groups, self.Ns[k])
            assert np.array_equal(bm, oq.bitmap())
        return opeak

    def close(self):
        for gq in self.greqs:
            self.B.bsr_req_release(self.ctx, gq)
        self.B.bsr_ctx_destroy(self.ctx)


@pytest.mark.parametrize("W,B", [(8, 12), (8, 16), (8, 3)])
def test_two_concurrent_restores_share_the_budget(W, B):
    c = TwoRequests([160, 140], W, B)
    try:
        statuses = c.run_gpu_concurrently()
        opeak = c.compare(statuses)
        assert statuses == [c.B.BSR_OK] * 2
        for r in range(R):                                          # every paged byte of both requests
            for l in range(len(c.layout.tensors)):
                assert np.array_equal(c.gpaged[r][l].cpu().numpy(), c.opaged[r][l])
        st = c.B.bsr_get_stats(c.ctx)[1]
        slot = c.reg.slot_bytes
        for r in range(R):
            assert st.ring_bytes_allocated[r] == B * slot
            assert st.peak_staging_bytes[r] <= B * slot            # the budget is never exceeded
            assert st.peak_staging_bytes[r] >= min(W, B) * slot     # one request alone fills its window
            assert st.peak_staging_bytes[r] == opeak[r] == min(B, 2 * W) * slot   # both overlapped
            assert st.bytes_installed[r] == (160 + 140) * c.reg.chunk_bytes
    finally:
        c.close()


def test_a_failing_request_fails_alone_under_a_budget():
    c = TwoRequests([120, 120], 8, 12, corrupt=(1, 0, 90))
    try:
        B = c.B
        statuses = c.run_gpu_concurrently()
        c.compare(statuses)
        assert statuses == [B.BSR_OK, B.BSR_ERR_CHECKSUM]
        # request 0 is complete and bit-exact; request 1 exposes nothing
        oq = c.oreqs[0]
        for r in range(R):
            for l, (g, _) in enumerate(c.layout.tensors):
                used = oq.block_tables[r][g]
                assert np.array_equal(c.gpaged[r][l].cpu().numpy()[used], c.opaged[r][l][used])
        st = B.bsr_get_stats(c.ctx)[1]
        assert max(st.peak_staging_bytes[:R]) <= 12 * c.reg.slot_bytes
        # the pool is whole again: a clean rerun of request 0 succeeds and can fill the budget
        assert B.bsr_restore(c.ctx, c.greqs[0], None) == B.BSR_OK
    finally:
        c.close()


def test_asynchronous_restores_share_the_budget_and_commit_waits_for_them():
    c = TwoRequests([150, 150], 8, 12)
    try:
        B = c.B
        assert B.bsr_restore_wait(c.ctx, c.greqs[0])[0] == B.BSR_ERR_STATE        # nothing pending
        for gq in c.greqs:
            assert B.bsr_restore_async(c.ctx, gq, None) == B.BSR_OK
        assert B.bsr_restore_async(c.ctx, c.greqs[0], None) == B.BSR_ERR_STATE     # already pending
        # commit on a request with a restore in flight waits for it instead of exposing zero
        assert B.bsr_commit(c.ctx, c.greqs[1]) == (B.BSR_OK, 150)
        statuses = [B.bsr_restore_wait(c.ctx, gq) for gq in c.greqs]
        assert statuses == [(B.BSR_OK, B.BSR_OK)] * 2
        opeak = c.compare([s for _, s in statuses])
        for r in range(R):
            for l in range(len(c.layout.tensors)):
                assert np.array_equal(c.gpaged[r][l].cpu().numpy(), c.opaged[r][l])
        st = B.bsr_get_stats(c.ctx)[1]
        assert st.peak_staging_bytes[0] == opeak[0] == 12 * c.reg.slot_bytes
    finally:
        c.close()


def test_four_concurrent_restores_one_failing():
    c = TwoRequests([70, 55, 64, 40], 4, 10, corrupt=(2, 1, 33), load_concurrency=6)
    try:
        B = c.B
        statuses = c.run_gpu_concurrently()
        c.compare(statuses)
        assert statuses == [B.BSR_OK, B.BSR_OK, B.BSR_ERR_CHECKSUM, B.BSR_OK]
        for k in (0, 1, 3):                                          # the healthy ones are bit-exact
            oq = c.oreqs[k]
            for r in range(R):
                for l, (g, _) in enumerate(c.layout.tensors):
                    used = oq.block_tables[r][g]
                    assert np.array_equal(c.gpaged[r][l].cpu().numpy()[used], c.opaged[r][l][used])
        st = B.bsr_get_stats(c.ctx)[1]
        slot = c.reg.slot_bytes
        assert 4 * slot <= max(st.peak_staging_bytes[:R]) <= 10 * slot
        # after the storm every slot is back: a single restore can again hold W and no more
        B.bsr_reset_stats(c.ctx)
        assert B.bsr_restore(c.ctx, c.greqs[0], None) == B.BSR_OK
        assert B.bsr_get_stats(c.ctx)[1].peak_staging_bytes[0] == 4 * slot
    finally:
        c.close()


def test_sequential_restores_with_a_budget_behave_like_the_locked_mode():
    c = TwoRequests([40, 30], 8, 20)
    try:
        B = c.B
        assert B.bsr_restore(c.ctx, c.greqs[0], None) == B.BSR_OK
        assert B.bsr_restore(c.ctx, c.greqs[1], None) == B.BSR_OK
        for q in c.oreqs:
            assert O.restore(c.reg, c.tiers, q, c.opaged, 8)[0] == O.OK
        for r in range(R):
            for l in range(len(c.layout.tensors)):
                assert np.array_equal(c.gpaged[r][l].cpu().numpy(), c.opaged[r][l])
        st = B.bsr_get_stats(c.ctx)[1]
        assert st.peak_staging_bytes[0] == 8 * c.reg.slot_bytes        # one at a time: W, not B
    finally:
        c.close()


def test_repeated_concurrent_rounds_with_scrubs_in_between_stay_bit_exact():
    """Six requests restored concurrently, eight rounds over: between rounds some requests are
    invalidated with a scrub (their blocks zeroed) and all are restored again, alternating the
    synchronous and the asynchronous call.  Every round ends with every status OK, every commit
    exposing the whole prefix and the pool whole; the last round is compared byte by byte."""
    Ns = [33, 20, 47, 8, 26, 40]
    c = TwoRequests(Ns, 4, 10, load_concurrency=6)
    try:
        B = c.B
        slot = c.reg.slot_bytes
        for rnd in range(8):
            if rnd % 2 == 0:
                statuses = c.run_gpu_concurrently()
            else:
                for gq in c.greqs:
                    assert B.bsr_restore_async(c.ctx, gq, None) == B.BSR_OK
                statuses = []
                for gq in c.greqs:
                    rc, st_ = B.bsr_restore_wait(c.ctx, gq)
                    assert rc == B.BSR_OK
                    statuses.append(st_)
            assert statuses == [B.BSR_OK] * len(Ns), (rnd, statuses)
            for k, gq in enumerate(c.greqs):
                assert B.bsr_commit(c.ctx, gq) == (B.BSR_OK, Ns[k])
            st = B.bsr_get_stats(c.ctx)[1]
            assert 4 * slot <= max(st.peak_staging_bytes[:R]) <= 10 * slot
            if rnd < 7:
                for k in ((rnd, (rnd + 3) % 6)):                     # two requests lose their blocks
                    assert B.bsr_invalidate(c.ctx, c.greqs[k % 6], B.BSR_SCRUB) == B.BSR_OK
                    assert B.bsr_commit(c.ctx, c.greqs[k % 6]) == (B.BSR_OK, 0)
        ostatus, _, _ = O.restore_concurrent(c.reg, c.tiers, c.oreqs, c.opaged, c.W, c.budget)
        assert ostatus == [O.OK] * len(Ns)
        for r in range(R):
            for l in range(len(c.layout.tensors)):
                assert np.array_equal(c.gpaged[r][l].cpu().numpy(), c.opaged[r][l])
        # the pool is whole: one restore alone holds exactly W slots again
        B.bsr_reset_stats(c.ctx)
        assert B.bsr_restore(c.ctx, c.greqs[2], None) == B.BSR_OK
        assert B.bsr_get_stats(c.ctx)[1].peak_staging_bytes[0] == 4 * slot
    finally:
        c.close()

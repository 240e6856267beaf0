"""Oracle pins for request-level recovery: the paper's failure table (full / zero, never partial),
lower-tier fallback, and the life cycle of the force-local marker."""
import numpy as np

from conftest import read_golden
from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

R, N, W, SEED, RID = 2, 9, 3, 77, 4242


def _engine(remote=True, ssd=True, remote_has=lambda r, i: True, ssd_has=lambda r, i: True):
    layout = synth.tiny_layout()
    reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
    tok = synth.tokens(N * 256, seed=SEED)
    keys = O.prefix_keys(O.chunk_digests(tok, SEED), SEED, 1)
    tiers = [[O.Tier() for _ in range(R)] for _ in range(2)]
    payload = {}
    for r in range(R):
        for i in range(N):
            p = synth.chunk_payload(layout, r, i, seed=SEED).copy()
            payload[(r, i)] = p
            ck = O.group_checksums(reg, p)
            if remote_has(r, i):
                tiers[0][r].put(keys[i], p, ck)
            if ssd_has(r, i):
                tiers[1][r].put(keys[i], p.copy(), ck)
    pools = [synth.pool_blocks(layout, g, N) for g in range(reg.n_groups)]
    tables = [[synth.block_table(layout, r, g, N, seed=SEED) for g in range(reg.n_groups)] for r in range(R)]
    paged = [O.new_paged(reg, pools, synth.CANARY) for _ in range(R)]
    return layout, reg, tok, keys, O.Engine(tiers, [remote, ssd]), tables, paged, payload


def _serve(eng, reg, tok, tables, paged, fetch_fault=None):
    keys, hit, n_hit, tier = O.probe_request(eng, RID, tok, SEED, 1)
    if n_hit == 0:
        return 0, tier, None
    tabs = [[t[: n_hit * reg.blocks_per_chunk(g)] for g, t in enumerate(tr)] for tr in tables]
    req = O.Request(keys[:n_hit], tabs, R, reg.n_groups)
    status, st = O.restore_request(eng, RID, tier, reg, req, paged, W, fetch_fault=fetch_fault)
    return O.commit(reg, req, paged), tier, status


def test_the_papers_failure_table():
    want = {k: (N if v == "full" else 0) for k, v in read_golden("failure_table.txt").items()}
    # remote healthy
    layout, reg, tok, keys, eng, tables, paged, _ = _engine()
    assert _serve(eng, reg, tok, tables, paged) == (want["remote_healthy"], 0, O.OK)
    assert all(t.bytes_read == 0 for t in eng.tiers[1])                       # the lower tier was not touched
    # remote unavailable, SSD healthy: full reuse from the lower tier
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote=False)
    assert _serve(eng, reg, tok, tables, paged) == (want["remote_unavailable_ssd_healthy"], 1, O.OK)
    assert all(t.bytes_read == 0 for t in eng.tiers[0])
    assert all(t.bytes_read == N * reg.chunk_bytes for t in eng.tiers[1])
    # remote and SSD absent: zero external reuse, nothing is restored
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote=False, ssd=False)
    assert _serve(eng, reg, tok, tables, paged) == (want["remote_and_ssd_absent"], -1, None)
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote_has=lambda r, i: False, ssd_has=lambda r, i: False)
    assert _serve(eng, reg, tok, tables, paged)[0] == 0
    # one-rank remote restore fault after one window: zero, although the lower tier is healthy
    layout, reg, tok, keys, eng, tables, paged, _ = _engine()
    fault = lambda r, i: O.ERR_TRANSFER if (r, i) == (1, W + 1) else None
    assert _serve(eng, reg, tok, tables, paged, fetch_fault=fault) == (want["one_rank_remote_restore_fault"], 0, O.ERR_TRANSFER)
    assert RID in eng.force_local


def test_force_local_marker_life_cycle():
    layout, reg, tok, keys, eng, tables, paged, payload = _engine()
    payload[(0, 4)][8] ^= 0x01                              # remote copy of one chunk is corrupt
    exposed, tier, status = _serve(eng, reg, tok, tables, paged)
    assert (exposed, tier, status) == (0, 0, O.ERR_CHECKSUM)
    # the next admission pass reports zero external tokens and does not consult any tier
    k2, hit, n_hit, tier = O.probe_request(eng, RID, tok, SEED, 1)
    assert n_hit == 0 and tier == -1 and not hit.any() and (k2 == keys).all()
    # another request is not affected and is served (from the healthy lower tier? no: tier 0 still
    # indexes the corrupt object; the probe cannot know) -- only the marked request is forced local
    assert O.probe_request(eng, RID + 1, tok, SEED, 1)[2:] == (N, 0)
    # RUNNING admission / teardown removes the marker
    O.request_done(eng, RID)
    assert O.probe_request(eng, RID, tok, SEED, 1)[2:] == (N, 0)
    O.request_done(eng, RID)                                 # idempotent


def test_tier_selection_longest_prefix_then_priority():
    # remote holds 5 chunks, SSD all 9: the request is served by the SSD tier alone, fully
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote_has=lambda r, i: i < 5)
    assert O.probe_request(eng, RID, tok, SEED, 1)[2:] == (N, 1)
    # equal prefixes: the higher-priority tier wins
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote_has=lambda r, i: i < 5, ssd_has=lambda r, i: i < 5)
    assert O.probe_request(eng, RID, tok, SEED, 1)[2:] == (5, 0)
    # a chunk missing on one rank of the remote tier shortens only that tier's prefix
    layout, reg, tok, keys, eng, tables, paged, _ = _engine(remote_has=lambda r, i: not (r == 1 and i == 2),
                                                            ssd_has=lambda r, i: i < 2)
    k, hit, n_hit, tier = O.probe_request(eng, RID, tok, SEED, 1)
    assert (n_hit, tier) == (2, 0) and list(hit) == [i != 2 for i in range(N)]


def test_tier_lost_between_probe_and_restore_fails_closed():
    layout, reg, tok, keys, eng, tables, paged, _ = _engine()
    k, hit, n_hit, tier = O.probe_request(eng, RID, tok, SEED, 1)
    eng.available[0] = False
    req = O.Request(k[:n_hit], tables, R, reg.n_groups)
    status, st = O.restore_request(eng, RID, tier, reg, req, paged, W)
    assert status == O.ERR_TRANSFER and O.commit(reg, req, paged) == 0 and RID in eng.force_local
    assert max(st.peak_staging_bytes) == 0


# ---------------------------------------------------------------- admission budget B
def _two_requests(N0, N1, corrupt=None):
    """Two requests with different token streams restoring into the same pools (disjoint blocks)."""
    layout = synth.tiny_layout()
    reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
    Rk = 2
    tiers = [O.Tier() for _ in range(Rk)]
    Ns = [N0, N1]
    pools = [synth.pool_blocks(layout, g, N0 + N1) for g in range(reg.n_groups)]
    big = [[synth.block_table(layout, r, g, N0 + N1, seed=5) for g in range(reg.n_groups)] for r in range(Rk)]
    reqs, payloads = [], {}
    for k, N in enumerate(Ns):
        tok = synth.tokens(N * 256, seed=100 + k)
        keys = O.prefix_keys(O.chunk_digests(tok, 3), 3, 1)
        for r in range(Rk):
            for i in range(N):
                p = synth.chunk_payload(layout, r, 1000 * k + i, seed=5).copy()
                ck = O.group_checksums(reg, p)
                if corrupt == (k, r, i):
                    p[7] ^= 2
                payloads[(k, r, i)] = p
                tiers[r].put(keys[i], p, ck)
        first = 0 if k == 0 else N0
        tabs = [[big[r][g][first * reg.blocks_per_chunk(g):(first + N) * reg.blocks_per_chunk(g)]
                 for g in range(reg.n_groups)] for r in range(Rk)]
        reqs.append(O.Request(keys, tabs, Rk, reg.n_groups))
    paged = [O.new_paged(reg, pools, synth.CANARY) for _ in range(Rk)]
    return layout, reg, tiers, reqs, paged, payloads, pools


def test_budget_bounds_aggregate_staging_and_results_equal_serial_restores():
    for (W, B, want_peak_slots) in [(4, 6, 6), (4, 8, 8), (4, 16, 8), (4, 3, 3), (4, 4, 4)]:
        layout, reg, tiers, reqs, paged, payloads, pools = _two_requests(11, 9)
        status, peak, rounds = O.restore_concurrent(reg, tiers, reqs, paged, W, B)
        assert status == [O.OK, O.OK]
        assert peak == [want_peak_slots * reg.slot_bytes] * 2          # min(B, sum of windows)
        assert [O.commit(reg, q, paged) for q in reqs] == [11, 9]
        # the same two requests restored one after the other give the same bytes
        layout, reg, tiers2, reqs2, paged2, _, _ = _two_requests(11, 9)
        for q in reqs2:
            assert O.restore(reg, tiers2, q, paged2, W)[0] == O.OK
        for r in range(2):
            for l in range(len(layout.tensors)):
                assert np.array_equal(paged[r][l], paged2[r][l])


def test_budget_one_request_fails_alone():
    layout, reg, tiers, reqs, paged, payloads, pools = _two_requests(8, 8, corrupt=(1, 0, 5))
    status, peak, rounds = O.restore_concurrent(reg, tiers, reqs, paged, 4, 6)
    assert status == [O.OK, O.ERR_CHECKSUM]
    assert O.commit(reg, reqs[0], paged) == 8 and O.commit(reg, reqs[1], paged) == 0
    assert reqs[0].valid.all() and not reqs[1].valid.any()
    assert max(peak) <= 6 * reg.slot_bytes

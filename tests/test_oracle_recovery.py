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

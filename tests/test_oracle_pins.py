"""Pins for the CPU oracle: values the paper prints, closed forms, inverses, brute force.

None of these tests calls the CUDA path.  Each is chosen so that a plausible slip in the oracle
(a dropped term, wrong shift, wrong index, transposed layout) fails at least one of them.
"""
import itertools

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from conftest import read_golden
from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

M = (1 << 64) - 1
PHI = 0x9E3779B97F4A7C15


# ---------------------------------------------------------------- mixer / digest / keys
def _unxorshift(y, s):
    x = y
    for _ in range(64 // s + 1):
        x = y ^ (x >> s)
    return x


def _unmix64(y):
    """Inverse of the mixer built from modular inverse and xor-shift inversion only."""
    inv = pow(PHI, -1, 1 << 64)
    y = _unxorshift(y, 32)
    y = _unxorshift((y * inv) & M, 29)
    y = _unxorshift((y * inv) & M, 32)
    return (y - PHI) & M


def test_mix64_golden_vectors():
    g = read_golden("spec_vectors.txt")
    for k, v in g.items():
        if k.startswith("mix64_"):
            assert O.mix64(int(k[6:], 16)) == int(v, 16)


def test_mix64_is_a_bijection_via_explicit_inverse():
    rng = np.random.default_rng(1)
    for x in [0, 1, M, 1 << 63] + [int(v) for v in rng.integers(0, 2**64, 200, dtype=np.uint64)]:
        assert _unmix64(O.mix64(x)) == x


def test_mix64_vector_form_equals_scalar_form():
    x = np.random.default_rng(2).integers(0, 2**64, 1000, dtype=np.uint64)
    assert [int(v) for v in O._mix64_vec(x)] == [O.mix64(int(v)) for v in x]


def _spec_tokens(n):
    return np.array([O.mix64(0xB5A ^ ((j * PHI) & M)) % 129280 for j in range(n)], dtype=np.int32)


def test_digest_and_key_golden_vectors():
    g = read_golden("spec_vectors.txt")
    tok = _spec_tokens(4096)
    assert [int(t) for t in tok[:8]] == [int(v) for v in g["tok_first8"]]
    d = O.chunk_digests(tok, salt=7)
    k = O.prefix_keys(d, salt=7, reg_id=1)
    assert len(d) == 16
    assert int(d[0]) == int(g["digest_0"], 16)
    assert int(k[0]) == int(g["key_0"], 16)
    assert int(k[15]) == int(g["key_15"], 16)


def test_digest_brute_force_and_tail_ignored():
    tok = synth.tokens(256 * 3 + 100, seed=5)
    salt = 0xDEADBEEF12345
    d = O.chunk_digests(tok, salt)
    assert len(d) == 3
    for i in range(3):
        s = 0
        for j in range(256):
            s += O.mix64((((int(tok[256 * i + j]) & 0xFFFFFFFF) << 32) | j) ^ salt)
        assert int(d[i]) == s & M


def test_digest_is_order_sensitive_and_chunk_local():
    tok = synth.tokens(1024, seed=6)
    d0 = O.chunk_digests(tok, 9)
    t2 = tok.copy()
    a, b = 256 + 3, 256 + 77
    assert t2[a] != t2[b]
    t2[a], t2[b] = tok[b], tok[a]
    d1 = O.chunk_digests(t2, 9)
    assert d1[1] != d0[1]
    assert d1[0] == d0[0] and d1[2] == d0[2] and d1[3] == d0[3]


def test_keys_have_prefix_semantics():
    tok = synth.tokens(2048, seed=7)
    k0 = O.prefix_keys(O.chunk_digests(tok, 11), 11, reg_id=3)
    t2 = tok.copy()
    t2[256 * 4 + 10] = (int(t2[256 * 4 + 10]) + 1) % synth.VOCAB
    k1 = O.prefix_keys(O.chunk_digests(t2, 11), 11, reg_id=3)
    assert (k1[:4] == k0[:4]).all()
    assert (k1[4:] != k0[4:]).all()
    k_salt = O.prefix_keys(O.chunk_digests(tok, 12), 12, reg_id=3)
    k_reg = O.prefix_keys(O.chunk_digests(tok, 11), 11, reg_id=4)
    assert (k_salt != k0).all() and (k_reg != k0).all()
    assert len(set(int(k) for k in k0)) == len(k0)


# ---------------------------------------------------------------- checksum
def test_checksum_golden_and_closed_forms():
    g = read_golden("spec_vectors.txt")
    assert O.checksum(np.array([1, 2, 3, 4], dtype="<u4").view(np.uint8)) == int(g["ck_1_2_3_4"])
    assert O.checksum(np.full(4, 0xFFFFFFFF, dtype="<u4").view(np.uint8)) == int(g["ck_4x_ffffffff"], 16)
    # sum of the first n odd numbers is n^2
    for n in (1, 7, 4096, 100003):
        assert O.checksum(np.ones(n, dtype="<u4").view(np.uint8)) == (n * n) & M
        assert O.checksum(np.full(n, 0xFFFFFFFF, dtype="<u4").view(np.uint8)) == (0xFFFFFFFF * n * n) & M
    # w_k = k: sum k(2k+1) = n(n-1)(4n+1)/6, large enough to wrap 2^64
    n = 3_000_000
    assert O.checksum(np.arange(n, dtype="<u4").view(np.uint8)) == (n * (n - 1) * (4 * n + 1) // 6) & M


def test_checksum_is_little_endian_and_detects_any_single_word_change():
    seg = np.array([0x01, 0x00, 0x00, 0x00, 0x00, 0x00, 0x00, 0x02], dtype=np.uint8)
    assert O.checksum(seg) == 1 * 1 + 0x02000000 * 3
    rng = np.random.default_rng(3)
    base = rng.integers(0, 256, 4096, dtype=np.uint8)
    c0 = O.checksum(base)
    for _ in range(50):
        s = base.copy()
        s.view("<u4")[rng.integers(0, 1024)] ^= np.uint32(rng.integers(1, 2**32))
        assert O.checksum(s) != c0
    # a swap of two different words is detected too (position weights differ)
    s = base.copy()
    w = s.view("<u4")
    w[[5, 900]] = w[[900, 5]]
    assert O.checksum(s) != c0


# ---------------------------------------------------------------- geometry and the staging law
def _reg(layout, **kw):
    return O.Registration(list(layout.block_tokens), list(layout.tensors), **kw)


def test_baseline_registration_matches_the_papers_coefficient():
    g = read_golden("paper_capacity.txt")
    reg = _reg(synth.baseline_layout())
    c = int(g["law_coefficient"])
    assert reg.chunk_bytes == c == reg.slot_bytes
    assert reg.segment(0) == (0, 56 * 256 * 1120)
    assert reg.segment(1) == (56 * 256 * 1120, c)
    assert 32 * reg.slot_bytes == int(g["rws_w32"])
    for W in (8, 16, 32, 64):
        assert W * reg.slot_bytes == float(g[f"rws_mib_w{W}"]) * 2**20  # Eq. 5, zero residual
    for N in (128, 512, 1024):
        assert N * reg.slot_bytes == int(g[f"whole_plan_peak_{N}"])
    # the paper's payload per object rounds up to the coefficient at 4 KiB granularity
    per_obj = int(g["external_128"]) // 128
    assert int(g["external_128"]) % 128 == 0 and -(-per_obj // 4096) * 4096 == c
    assert round(int(g["external_2047"]) / int(g["rws_w32"]), 4) == float(g["ratio_ext_to_live"])
    # MTP-on: 64,976 B/token
    assert O.Registration([64], [(0, 64976)]).slot_bytes * 32 == int(g["mtp_on_peak_w32"])
    hl = _reg(synth.hetero_layout())
    assert hl.chunk_bytes == c and len(hl.tensors) == 170 and hl.n_groups == 3
    ml = _reg(synth.mtp_on_layout())
    assert len(ml.tensors) == 170 and 32 * ml.slot_bytes == int(g["mtp_on_peak_w32"])


def test_slot_rounding_rule():
    reg = O.Registration([64], [(0, 20)], slot_align=4096)  # 5,120 B payload
    assert reg.chunk_bytes == 5120 and reg.slot_bytes == 8192


def _build_case(layout, R, N, seed, present=None):
    """tiers, keys, tables, paged pools for a small case, all from the seeded generators."""
    reg = _reg(layout)
    tok = synth.tokens(N * 256 + 17, seed=seed)
    tiers = [O.Tier() for _ in range(R)]
    keys = O.prefix_keys(O.chunk_digests(tok, seed), seed, reg_id=1)
    payload = {}
    for r in range(R):
        for i in range(N):
            if present is not None and not present(r, i):
                continue
            p = synth.chunk_payload(layout, r, i, seed=seed).copy()
            payload[(r, i)] = p
            tiers[r].put(keys[i], p, O.group_checksums(reg, p))
    pools = [synth.pool_blocks(layout, g, N) for g in range(reg.n_groups)]
    tables = [[synth.block_table(layout, r, g, N, seed=seed) for g in range(reg.n_groups)] for r in range(R)]
    paged = [O.new_paged(reg, pools, synth.CANARY) for _ in range(R)]
    return reg, tok, tiers, keys, tables, paged, payload, pools


@pytest.mark.parametrize("N,W", [(1, 1), (5, 2), (7, 7), (7, 64), (9, 4), (16, 4)])
def test_window_count_peak_and_work(N, W):
    layout = synth.tiny_layout()
    reg, tok, tiers, keys, tables, paged, _, _ = _build_case(layout, 2, N, seed=21)
    req = O.Request(keys[:N], tables, 2, reg.n_groups)
    status, st = O.restore(reg, tiers, req, paged, W)
    assert status == O.OK
    assert st.windows == -(-N // W)                                   # K = ceil(N / W)
    assert st.peak_staging_bytes == [min(N, W) * reg.slot_bytes] * 2  # Eq. 3 / Eq. 5; W >= N => whole plan
    assert st.bytes_filled == st.bytes_installed == [N * reg.chunk_bytes] * 2  # total work = |S|
    assert O.commit(reg, req, paged) == N
    assert req.valid.all()


def test_peak_is_independent_of_plan_length():
    layout = synth.tiny_layout()
    peaks = set()
    for N in (8, 16, 40):
        reg, tok, tiers, keys, tables, paged, _, _ = _build_case(layout, 1, N, seed=22)
        req = O.Request(keys[:N], tables, 1, reg.n_groups)
        status, st = O.restore(reg, tiers, req, paged, 8)
        assert status == O.OK
        peaks.add(st.peak_staging_bytes[0])
    assert peaks == {8 * reg.slot_bytes}                              # Proposition 1


def test_the_papers_scaling_table_rows():
    """Every row of the paper's W = 32 scaling table: objects = full 256-token chunks of the prefix,
    external GiB = objects x 16,406,080 B, and the oracle's window loop over that many chunks
    peaks at 32 slots (500.75 MiB with the 16,408,576-B slot) in K = ceil(objects / 32) windows."""
    g = read_golden("paper_capacity.txt")
    per_object = int(g["external_128"]) // 128
    layout = synth.Layout("narrow", [64], [(0, 16)])               # 4 KiB chunks keep 2,047 of them cheap
    for key, (objects, gib, mib) in read_golden("paper_scaling_table.txt").items():
        tokens, objects = int(key[4:]), int(objects)
        assert tokens // 256 == objects
        assert round(objects * per_object / 2**30, 3) == float(gib)
        assert 32 * int(g["law_coefficient"]) == float(mib) * 2**20
        reg, tok, tiers, keys, tables, paged, _, _ = _build_case(layout, 1, objects, seed=24)
        req = O.Request(keys[:objects], tables, 1, 1)
        status, st = O.restore(reg, tiers, req, paged, 32)
        assert status == O.OK and st.windows == -(-objects // 32)
        assert st.peak_staging_bytes == [32 * reg.slot_bytes]        # the same for every row


def test_w_zero_is_rejected():
    layout = synth.tiny_layout()
    reg, tok, tiers, keys, tables, paged, _, _ = _build_case(layout, 1, 2, seed=23)
    req = O.Request(keys[:2], tables, 1, reg.n_groups)
    assert O.restore(reg, tiers, req, paged, 0)[0] == O.ERR_INVALID


# ---------------------------------------------------------------- install == plain definition
def _brute_force_paged(layout, R, N, tables, payload, pools):
    """The plain definition, one byte at a time, with its own offset arithmetic."""
    out = []
    for r in range(R):
        per_rank = []
        for l, (g, e) in enumerate(layout.tensors):
            B = layout.block_tokens[g]
            arr = [[[synth.CANARY] * e for _ in range(B)] for _ in range(pools[g])]
            off_l = 256 * sum(ee for _, ee in layout.tensors[:l])
            for t in range(256 * N):
                i, tt = divmod(t, 256)
                blk = int(tables[r][g][t // B])
                src = payload[(r, i)]
                for x in range(e):
                    arr[blk][t % B][x] = int(src[off_l + tt * e + x])
            per_rank.append(np.array(arr, dtype=np.uint8))
        out.append(per_rank)
    return out


def test_restore_equals_bytewise_definition_on_tiny_input():
    layout = synth.tiny_layout()
    R, N, W = 2, 5, 2
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=31)
    req = O.Request(keys[:N], tables, R, reg.n_groups)
    assert O.restore(reg, tiers, req, paged, W)[0] == O.OK
    want = _brute_force_paged(layout, R, N, tables, payload, pools)
    for r in range(R):
        for l in range(len(layout.tensors)):
            assert np.array_equal(paged[r][l], want[r][l])
    # spare blocks keep the canary, every logical block is used exactly once
    for r in range(R):
        for g in range(reg.n_groups):
            t = tables[r][g]
            assert len(set(int(b) for b in t)) == len(t)
            spare = sorted(set(range(pools[g])) - set(int(b) for b in t))
            for l, (gg, _) in enumerate(layout.tensors):
                if gg == g:
                    assert (paged[r][l][spare] == synth.CANARY).all()


def test_parallel_for_over_a_window_equals_the_bytewise_definition_and_fails_alike():
    """The all-cores timing form of the oracle (a thread pool over the chunks of a window) against
    the same one-byte-at-a-time definition, and its failure report against the serial loop's."""
    layout = synth.tiny_layout()
    R, N, W = 2, 7, 3
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=33)
    req = O.Request(keys[:N], tables, R, reg.n_groups)
    status, st_par = O.restore(reg, tiers, req, paged, W, workers=4)
    assert status == O.OK and req.valid.all() and O.commit(reg, req, paged) == N
    assert st_par.windows == 3 and st_par.peak_staging_bytes == [W * reg.slot_bytes] * R
    assert st_par.bytes_installed == [N * reg.chunk_bytes] * R
    want = _brute_force_paged(layout, R, N, tables, payload, pools)
    for r in range(R):
        for l in range(len(layout.tensors)):
            assert np.array_equal(paged[r][l], want[r][l])
    # a corrupted word in the second window: same status, nothing valid, nothing exposed
    bad = payload[(1, 4)]
    bad[8] ^= 0x40
    for workers in (1, 4):
        req = O.Request(keys[:N], tables, R, reg.n_groups)
        status, _ = O.restore(reg, tiers, req, paged, W, workers=workers)
        assert status == O.ERR_CHECKSUM and not req.valid.any() and O.commit(reg, req, paged) == 0


@settings(max_examples=25, deadline=None, derandomize=True)
@given(st.data())
def test_restore_equals_bytewise_definition_on_random_registrations(data):
    """Random geometry (1-3 groups, block sizes 16...256, 1-3 tensors per group, odd multiples of
    16 bytes per token), random R, N, W: the window loop lands every byte where the plain
    definition puts it, peaks at min(N, W) slots and moves exactly N chunks per rank."""
    G = data.draw(st.integers(1, 3))
    blocks = [data.draw(st.sampled_from([16, 32, 64, 128, 256])) for _ in range(G)]
    tensors = [(g, 16 * data.draw(st.integers(1, 3))) for g in range(G)
               for _ in range(data.draw(st.integers(1, 3)))]
    layout = synth.Layout("random", blocks, tensors)
    R, N, W = data.draw(st.integers(1, 2)), data.draw(st.integers(1, 4)), data.draw(st.integers(1, 5))
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=data.draw(st.integers(1, 99)))
    req = O.Request(keys[:N], tables, R, reg.n_groups)
    status, stats = O.restore(reg, tiers, req, paged, W)
    assert status == O.OK and O.commit(reg, req, paged) == N
    want = _brute_force_paged(layout, R, N, tables, payload, pools)
    for r in range(R):
        for l in range(len(layout.tensors)):
            assert np.array_equal(paged[r][l], want[r][l])
        assert stats.peak_staging_bytes[r] == min(N, W) * reg.slot_bytes
        assert stats.bytes_installed[r] == N * reg.chunk_bytes
    assert stats.windows == -(-N // W)


def test_identity_table_single_tensor_is_a_plain_concatenation():
    layout = synth.Layout("one", [64], [(0, 48)])
    reg = _reg(layout)
    N = 6
    tier = O.Tier()
    keys = np.arange(1, N + 1, dtype=np.uint64)
    chunks = [synth.chunk_payload(layout, 0, i, seed=41).copy() for i in range(N)]
    for i in range(N):
        tier.put(keys[i], chunks[i], O.group_checksums(reg, chunks[i]))
    table = np.arange(N * 4, dtype=np.int32)
    paged = [O.new_paged(reg, [N * 4], 0)]
    req = O.Request(keys, [[table]], 1, 1)
    assert O.restore(reg, [tier], req, paged, 4)[0] == O.OK
    assert np.array_equal(paged[0][0].reshape(-1), np.concatenate(chunks))


# ---------------------------------------------------------------- probe
def test_probe_reads_no_payload_and_finds_longest_complete_prefix():
    layout = synth.tiny_layout()
    N = 12
    present = lambda r, i: i < 7 or i == 9 or (r == 0 and i == 7)  # chunk 7 only on rank 0; decoy 9
    reg, tok, tiers, keys, tables, paged, _, _ = _build_case(layout, 2, N, seed=51, present=present)
    k, hit, n_hit = O.probe(tok, 51, 1, tiers)
    assert (k == keys).all() and len(k) == N
    assert n_hit == 7
    assert list(hit) == [i < 7 or i == 9 for i in range(N)]
    assert all(t.bytes_read == 0 for t in tiers)
    words = O.pack_bits(hit)
    assert int(words[0]) == sum(1 << i for i in range(N) if hit[i])
    assert O.probe(tok, 52, 1, tiers)[2] == 0  # another salt: nothing is reusable


def test_pack_bits_crosses_word_boundaries():
    bits = np.zeros(130, dtype=bool)
    bits[[0, 63, 64, 129]] = True
    assert [int(w) for w in O.pack_bits(bits)] == [1 | 1 << 63, 1, 2]


# ---------------------------------------------------------------- commit: Eq. 6 truth table
def test_commit_truth_table_every_subset_of_failing_components():
    layout = synth.tiny_layout()
    R, N, W = 2, 2, 1
    G = layout.n_groups
    sites = list(itertools.product(range(R), range(G), range(N)))
    for mask in range(1 << len(sites)):
        reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=61)
        for bit, (r, g, i) in enumerate(sites):
            if mask >> bit & 1:
                lo, hi = reg.segment(g)
                payload[(r, i)][lo + 4 * ((mask * 7 + bit) % ((hi - lo) // 4))] ^= 0x40
        req = O.Request(keys[:N], tables, R, G)
        status, st = O.restore(reg, tiers, req, paged, W)
        exposed = O.commit(reg, req, paged)
        if mask == 0:
            assert status == O.OK and exposed == N and req.valid.all()
        else:
            assert status == O.ERR_CHECKSUM and exposed == 0          # never partial
            assert not req.valid.any()                                 # healthy components cleared too
            assert (req.bitmap() == 0).all()
            assert 0 < max(st.peak_staging_bytes) <= W * reg.slot_bytes


def test_commit_is_the_conjunction_of_eq6_on_every_bit_pattern():
    """Eq. 6 on the predicate itself: for every pattern of the q_{r,g} bits (one chunk), commit exposes
    the prefix only when all are set and a restore completed; one missing bit of any rank or group is zero."""
    layout = synth.tiny_layout()
    R, G = 2, layout.n_groups
    for mask in range(1 << (R * G)):
        reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, 1, seed=62)
        req = O.Request(keys[:1], tables, R, G)
        for bit, (r, g) in enumerate(itertools.product(range(R), range(G))):
            req.valid[r, g, 0] = bool(mask >> bit & 1)
        req.restored = True
        assert O.commit(reg, req, paged) == (1 if mask == (1 << (R * G)) - 1 else 0)
    # all bits set but no completed restore, or a failed one: nothing is exposed
    for restored, failed in ((False, False), (True, True)):
        req = O.Request(keys[:1], tables, R, G)
        req.valid[:] = True
        req.restored, req.failed = restored, failed
        assert O.commit(reg, req, paged) == 0


def test_failure_cases_are_fail_closed_and_scrub_zeroes_only_request_blocks():
    layout = synth.tiny_layout()
    R, N, W = 2, 9, 3
    # (a) missing chunk on one rank after probe
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=71)
    _, _, n_hit = O.probe(tok, 71, 1, tiers)
    assert n_hit == N
    tiers[1].remove(keys[5])
    req = O.Request(keys[:N], tables, R, reg.n_groups)
    status, st = O.restore(reg, tiers, req, paged, W)
    assert status == O.ERR_MISSING and O.commit(reg, req, paged) == 0 and not req.valid.any()
    # every destination block of the request is erroneous, also those of windows never reached
    for r in range(R):
        for g in range(reg.n_groups):
            assert np.array_equal(O.invalid_blocks(req, r, g), tables[r][g]) and len(tables[r][g]) > 0
    healthy = O.Request(keys[:3], [[t[: 3 * reg.blocks_per_chunk(g)] for g, t in enumerate(tr)] for tr in tables],
                        R, reg.n_groups)
    assert O.restore(reg, tiers, healthy, paged, W)[0] == O.OK and len(O.invalid_blocks(healthy, 0, 0)) == 0
    # the first window (chunks 0..2) was already copied: partial bytes exist, exposure is still zero
    assert np.array_equal(paged[0][0][tables[0][0][0]], payload[(0, 0)][: 16 * 48].reshape(16, 48))
    O.invalidate(reg, req, paged, scrub=True)
    for r in range(R):
        for l, (g, _) in enumerate(layout.tensors):
            used = tables[r][g]
            spare = sorted(set(range(pools[g])) - set(int(b) for b in used))
            assert (paged[r][l][used] == 0).all()
            assert (paged[r][l][spare] == synth.CANARY).all()
    assert O.commit(reg, req, paged) == 0
    # (b) fetch fault (transfer error / timeout) on one rank after one good window
    for code in (O.ERR_TRANSFER, O.ERR_TIMEOUT):
        reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=72)
        req = O.Request(keys[:N], tables, R, reg.n_groups)
        status, st = O.restore(reg, tiers, req, paged, W,
                               fetch_fault=lambda r, i: code if (r, i) == (1, 4) else None)
        assert status == code and O.commit(reg, req, paged) == 0 and not req.valid.any()
        assert st.windows == 2
    # (c) commit without a restore exposes nothing
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, R, N, seed=73)
    req = O.Request(keys[:N], tables, R, reg.n_groups)
    assert O.commit(reg, req, paged) == 0


def test_partial_hit_exposes_exactly_the_hit_prefix():
    layout = synth.tiny_layout()
    R, N = 2, 10
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(
        layout, R, N, seed=81, present=lambda r, i: i < 6 or i == 8)
    _, hit, n_hit = O.probe(tok, 81, 1, tiers)
    assert n_hit == 6
    tables6 = [[t[: 6 * reg.blocks_per_chunk(g)] for g, t in enumerate(tr)] for tr in tables]
    req = O.Request(keys[:6], tables6, R, reg.n_groups)
    status, st = O.restore(reg, tiers, req, paged, 4)
    assert status == O.OK and st.windows == 2 and O.commit(reg, req, paged) == 6
    assert st.bytes_installed == [6 * reg.chunk_bytes] * 2


def test_config1_full_size_baseline_layout():
    """The tiny single-rank configuration at its real geometry: 16 chunks, W = 4."""
    g = read_golden("paper_capacity.txt")
    layout = synth.baseline_layout()
    reg, tok, tiers, keys, tables, paged, payload, pools = _build_case(layout, 1, 16, seed=91)
    req = O.Request(keys[:16], tables, 1, 2)
    status, st = O.restore(reg, tiers, req, paged, 4)
    assert status == O.OK and st.windows == 4
    assert st.peak_staging_bytes == [4 * int(g["law_coefficient"])]
    assert st.bytes_installed == [16 * int(g["law_coefficient"])]
    # spot-check rows against the definition with independent index arithmetic
    rng = np.random.default_rng(0)
    for _ in range(200):
        l = int(rng.integers(0, 99))
        t = int(rng.integers(0, 4096))
        grp, e = layout.tensors[l]
        off_l = 256 * sum(ee for _, ee in layout.tensors[:l])
        row = payload[(0, t // 256)][off_l + (t % 256) * e: off_l + (t % 256) * e + e]
        assert np.array_equal(paged[0][l][tables[0][grp][t // 64], t % 64], row)

"""CUDA path vs CPU oracle, element by element, through the C interface (needs a B200)."""
import numpy as np
import pytest

from harness import Case, GpuSide, assert_paged_equal, run_oracle
from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

pytestmark = pytest.mark.gpu


def _check_success(case, W, gpu, ora, n_adv):
    B = gpu.B
    st = gpu.stats()
    slot = case.reg.slot_bytes
    assert gpu.commit() == ora["exposed"] == n_adv
    assert np.array_equal(gpu.bitmap(n_adv), ora["req"].bitmap())
    assert_paged_equal(gpu, ora["paged"])
    rc, cks = B.bsr_req_checksums(gpu.ctx, gpu.req, case.R, case.G, n_adv)
    assert rc == B.BSR_OK
    for r in range(case.R):
        for i in range(n_adv):
            assert [int(x) for x in cks[r, :, i]] == case.cks[(r, i)]
    assert st.windows == ora["stats"].windows == -(-n_adv // W)
    for r in range(case.R):
        assert st.bytes_installed[r] == ora["stats"].bytes_installed[r] == n_adv * case.reg.chunk_bytes
        if gpu.location == B.BSR_LOC_HOST:
            assert st.peak_staging_bytes[r] == ora["stats"].peak_staging_bytes[r] == min(n_adv, W) * slot
            assert st.bytes_filled[r] == st.bytes_h2d[r] == ora["stats"].bytes_filled[r]
            assert st.ring_bytes_allocated[r] == W * slot
        else:
            assert st.peak_staging_bytes[r] == 0 and st.bytes_h2d[r] == 0
    assert st.slot_bytes == slot
    assert st.tier_bytes_read_by_probe == 0
    rc, bad = B.bsr_req_invalid_blocks(gpu.ctx, gpu.req, 0, 0, 8)
    assert rc == B.BSR_OK and len(bad) == 0           # a healthy request has no erroneous block


# ---------------------------------------------------------------- probe
@pytest.mark.parametrize("N,tail,on_device", [(1, 0, False), (37, 100, False), (37, 100, True),
                                              (2048, 0, True), (2051, 255, False)])
def test_probe_keys_bitmap_prefix(N, tail, on_device):
    layout = synth.tiny_layout()
    present = (lambda r, i: i < 20 or i == 25 or (r == 1 and i == 20)) if N == 37 else (lambda r, i: i < 3)
    case = Case(layout, 2, N, seed=101, present=present, tail_tokens=tail)
    tiers = case.oracle_tiers()
    keys, hit, n_hit = O.probe(case.tok, case.salt, case.reg_id, tiers)
    with GpuSide(case, W=4) as gpu:
        rc, k, bm, nh = gpu.probe(tok_on_device=on_device)
        assert rc == gpu.B.BSR_OK
        assert np.array_equal(k, keys)
        assert np.array_equal(bm, O.pack_bits(hit))
        assert nh == n_hit == min(N, 20 if N == 37 else 3)
        st = gpu.stats()
        assert st.tier_bytes_read_by_probe == 0 and max(st.peak_staging_bytes) == 0
        # another salt: nothing reusable
        rc, k2, _, nh2 = gpu.B.bsr_probe(gpu.ctx, case.tok, len(case.tok), case.salt + 1)
        assert rc == gpu.B.BSR_OK and nh2 == 0 and not np.array_equal(k2, keys)


def test_probe_sixteen_million_tokens_and_scratch_regrowth():
    """65,539 chunks: many passes of the key chain through its shared-memory tile, scratch grown
    twice (a short probe first), and the boundary chunk counts of the digest grid."""
    import torch
    from paper_2608_17826_b200 import binding as B
    rc, ctx = B.bsr_ctx_create(4, 1, reg_id=77)
    assert rc == B.BSR_OK
    try:
        for n_chunks in (3, 65539, 2047):
            tok = synth.tokens(n_chunks * 256 + 5, seed=1500 + n_chunks)
            want = O.prefix_keys(O.chunk_digests(tok, 0xFEED), 0xFEED, 77)
            rc, keys, bm, n_hit = B.bsr_probe(ctx, tok, len(tok), 0xFEED, False)
            assert rc == B.BSR_OK and n_hit == 0 and np.array_equal(keys, want) and not bm.any()
            d_tok = torch.from_numpy(tok).cuda()
            torch.cuda.synchronize()
            rc, keys, bm, n_hit = B.bsr_probe(ctx, d_tok.data_ptr(), len(tok), 0xFEED, True)
            assert rc == B.BSR_OK and np.array_equal(keys, want)
    finally:
        B.bsr_ctx_destroy(ctx)


def test_probe_fewer_than_one_chunk():
    case = Case(synth.tiny_layout(), 1, 1, seed=102)
    with GpuSide(case, W=2) as gpu:
        rc, k, bm, nh = gpu.B.bsr_probe(gpu.ctx, case.tok[:200].copy(), 200, case.salt)
        assert rc == gpu.B.BSR_OK and nh == 0 and len(k) == 0


# ---------------------------------------------------------------- restore, success
@pytest.mark.parametrize("layout_name,R,N,W,cfg", [
    ("tiny", 1, 1, 1, {}),
    ("tiny", 2, 5, 2, {}),
    ("tiny", 2, 9, 4, dict(load_concurrency=1, dev_staging_depth=1)),
    ("tiny", 2, 23, 8, dict(load_concurrency=8, dev_staging_depth=2)),
    ("tiny", 3, 7, 64, {}),                      # W >= N: whole plan live at once
    ("tiny", 2, 70, 3, dict(load_concurrency=3)),
    ("hetero", 2, 6, 4, {}),
    ("baseline", 1, 16, 4, {}),                  # the tiny single-rank configuration
])
def test_restore_matches_oracle(layout_name, R, N, W, cfg):
    layout = {"tiny": synth.tiny_layout, "hetero": synth.hetero_layout,
              "baseline": synth.baseline_layout}[layout_name]()
    case = Case(layout, R, N, seed=200 + N)
    ora = run_oracle(case, W)
    assert ora["status"] == O.OK and ora["n_hit"] == N
    with GpuSide(case, W, **cfg) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        assert rc == gpu.B.BSR_OK and n_hit == N and np.array_equal(keys, ora["keys"])
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)
        # a second restore of the same request is idempotent
        gpu.B.bsr_reset_stats(gpu.ctx)
        assert gpu.restore() == gpu.B.BSR_OK
        _check_success(case, W, gpu, ora, N)


@pytest.mark.parametrize("layout_name,R,N,W", [("tiny", 2, 11, 4), ("hetero", 2, 5, 2), ("baseline", 2, 6, 4)])
def test_restore_from_device_resident_tier(layout_name, R, N, W):
    layout = {"tiny": synth.tiny_layout, "hetero": synth.hetero_layout,
              "baseline": synth.baseline_layout}[layout_name]()
    case = Case(layout, R, N, seed=300 + N)
    ora = run_oracle(case, W)
    with GpuSide(case, W, location=1, time_kernels=True) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)
        st = gpu.stats()
        assert st.install_kernel_ms > 0
        assert 0 < st.install_span_ms < st.install_kernel_ms      # the kernel's own span lies inside the event pair


@pytest.mark.parametrize("direct", [False, True])
def test_tier_with_some_objects_in_device_memory_and_some_on_the_host(direct):
    """A tier whose objects live partly in HBM and partly in host memory goes through the slot pool as a
    whole: host objects are copied tier -> slot -> device, device objects device -> device (with
    direct_install the kernel reads either in place); every paged byte as the oracle's, and only the
    host objects count as filled."""
    layout = synth.hetero_layout()
    R, N, W = 2, 21, 4
    case = Case(layout, R, N, seed=350)
    ora = run_oracle(case, W)
    with GpuSide(case, W, direct_install=direct) as gpu:
        B, torch = gpu.B, gpu.torch
        on_device = {(r, i): torch.from_numpy(case.payload[(r, i)]).to(gpu.dev)
                     for r in range(R) for i in range(N) if (i + r) % 3 == 1}
        for (r, i), t in on_device.items():     # the same key again: the index entry is replaced
            assert B.bsr_tier_put(gpu.ctx, r, case.keys[i], t.data_ptr(), t.numel(), case.cks[(r, i)],
                                  B.BSR_LOC_DEVICE) == B.BSR_OK
        torch.cuda.synchronize()
        rc, keys, bm, n_hit = gpu.probe()
        assert rc == B.BSR_OK and n_hit == N
        gpu.request(keys, n_hit)
        assert gpu.restore() == B.BSR_OK, B.bsr_last_error(gpu.ctx)
        assert gpu.commit() == ora["exposed"] == N
        assert np.array_equal(gpu.bitmap(N), ora["req"].bitmap())
        assert_paged_equal(gpu, ora["paged"])
        st = gpu.stats()
        for r in range(R):
            n_host = sum(1 for i in range(N) if (r, i) not in on_device)
            assert st.bytes_filled[r] == n_host * case.reg.chunk_bytes
            assert st.bytes_installed[r] == N * case.reg.chunk_bytes
            assert st.peak_staging_bytes[r] == W * case.reg.slot_bytes


def test_library_computed_checksums_equal_oracle():
    for layout in (synth.tiny_layout(), synth.hetero_layout()):
        case = Case(layout, 2, 3, seed=400)
        for loc in (0, 1):
            with GpuSide(case, 2, location=loc, compute_ck=True) as gpu:
                for (r, i), want in case.cks.items():
                    rc, got = gpu.B.bsr_tier_checksums(gpu.ctx, r, case.keys[i], case.G)
                    assert rc == gpu.B.BSR_OK and [int(x) for x in got] == want


def test_partial_hit_exposes_exactly_the_prefix():
    case = Case(synth.tiny_layout(), 2, 20, seed=500, present=lambda r, i: i < 13 or i == 16)
    ora = run_oracle(case, 4)
    assert ora["n_hit"] == 13 and ora["exposed"] == 13
    with GpuSide(case, 4) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        assert n_hit == 13 and np.array_equal(bm, O.pack_bits(ora["hit"]))
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK
        _check_success(case, 4, gpu, ora, 13)


# ---------------------------------------------------------------- failures: fail closed
def _check_failed(case, W, gpu, n_adv, want_rc, scrub_paged):
    B = gpu.B
    assert gpu.commit() == 0
    assert (gpu.bitmap(n_adv) == 0).all()
    for r in range(case.R):                      # all destination blocks of the request are erroneous
        for g, t in enumerate(case.tables_prefix(n_adv)[r]):
            rc, bad = B.bsr_req_invalid_blocks(gpu.ctx, gpu.req, r, g, len(t) + 4)
            assert rc == B.BSR_OK and np.array_equal(bad, t)
    st = gpu.stats()
    assert 0 < max(st.peak_staging_bytes[: case.R]) <= W * case.reg.slot_bytes
    assert B.bsr_invalidate(gpu.ctx, gpu.req, B.BSR_SCRUB) == B.BSR_OK
    assert_paged_equal(gpu, scrub_paged)          # request blocks zero, every other block untouched
    assert gpu.commit() == 0


def _scrubbed_oracle(case, W, n_adv, mutate_tiers=None, fetch_fault=None):
    tiers = case.oracle_tiers()
    if mutate_tiers:
        mutate_tiers(tiers)
    ora = run_oracle(case, W, n_adv=n_adv, tiers=tiers, fetch_fault=fetch_fault)
    assert ora["status"] != O.OK and ora["exposed"] == 0 and not ora["req"].valid.any()
    O.invalidate(case.reg, ora["req"], ora["paged"], scrub=True)
    return ora


FAILURE_KINDS = ["corrupt_tier", "missing", "rank_asymmetric", "corrupt_slot", "fill_error", "fill_stall"]


@pytest.mark.parametrize("kind", FAILURE_KINDS)
def test_failures_expose_nothing(kind):
    layout = synth.tiny_layout()
    R, N, W = 2, 24, 4
    case = Case(layout, R, N, seed=600)
    r, g, i, frac = synth.fault_site(R, case.G, W, N, case=FAILURE_KINDS.index(kind), seed=7)
    if kind == "rank_asymmetric":
        r, g = 1, 1
    cfg = dict(timeout_ms=1500) if kind == "fill_stall" else {}
    with GpuSide(case, W, **cfg) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        assert n_hit == N
        gpu.request(keys, N)
        fetch_fault = None
        mutate = None
        want = None
        if kind in ("corrupt_tier", "rank_asymmetric"):
            lo, hi = case.reg.segment(g)
            w = case.payload[(r, i)][lo:hi].view("<u4")
            w[frac % len(w)] ^= np.uint32(1 << (frac % 32))      # tier bytes are caller-owned
            want = B.BSR_ERR_CHECKSUM
        elif kind == "missing":
            assert B.bsr_tier_remove(gpu.ctx, r, case.keys[i]) == B.BSR_OK   # after probe
            mutate = lambda tiers: tiers[r].remove(case.keys[i])
            want = B.BSR_ERR_MISSING
        elif kind == "corrupt_slot":
            B.bsr_test_inject(gpu.ctx, B.BSR_INJECT_CORRUPT_SLOT, r, g, i, frac)
            lo, hi = case.reg.segment(g)
            def mutate(tiers, lo=lo, hi=hi):
                p = case.payload[(r, i)].copy()
                p[lo:hi].view("<u4")[0] ^= np.uint32(1)
                tiers[r].put(case.keys[i], p, case.cks[(r, i)])
            want = B.BSR_ERR_CHECKSUM
        elif kind == "fill_error":
            B.bsr_test_inject(gpu.ctx, B.BSR_INJECT_FILL_ERROR, r, 0, i, 0)
            fetch_fault = lambda rr, ii: O.ERR_TRANSFER if (rr, ii) == (r, i) else None
            want = B.BSR_ERR_TRANSFER
        elif kind == "fill_stall":
            B.bsr_test_inject(gpu.ctx, B.BSR_INJECT_FILL_STALL, r, 0, i, 0)
            fetch_fault = lambda rr, ii: O.ERR_TIMEOUT if (rr, ii) == (r, i) else None
            want = B.BSR_ERR_TIMEOUT
        ora = _scrubbed_oracle(case, W, N, mutate_tiers=mutate, fetch_fault=fetch_fault)
        assert ora["status"] == want
        assert gpu.restore() == want
        _check_failed(case, W, gpu, N, want, ora["paged"])
        # the injected fault was one shot, tier corruption is not: a clean retry must succeed
        if kind in ("corrupt_slot", "fill_error", "fill_stall"):
            good = run_oracle(case, W)
            gpu.B.bsr_reset_stats(gpu.ctx)
            assert gpu.restore() == B.BSR_OK
            _check_success(case, W, gpu, good, N)


def test_commit_without_restore_and_after_invalidate():
    case = Case(synth.tiny_layout(), 2, 6, seed=700)
    ora = run_oracle(case, 2)
    with GpuSide(case, 2) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.commit() == 0                          # nothing restored yet
        assert gpu.restore() == B.BSR_OK
        assert gpu.commit() == 6 and gpu.commit() == 6    # idempotent
        assert B.bsr_invalidate(gpu.ctx, gpu.req, 0) == B.BSR_OK
        assert gpu.commit() == 0 and (gpu.bitmap(6) == 0).all()
        assert_paged_equal(gpu, ora["paged"])             # invalidation without scrub moves no byte


# ---------------------------------------------------------------- argument checking / edge cases
def test_argument_errors_and_empty_request():
    import torch
    from paper_2608_17826_b200 import binding as B
    assert B.bsr_ctx_create(0, 1)[0] == B.BSR_ERR_INVALID          # W = 0: legacy whole-plan mode
    assert B.bsr_ctx_create(4, 0)[0] == B.BSR_ERR_INVALID
    assert B.bsr_ctx_create(4, 9)[0] == B.BSR_ERR_INVALID
    rc, ctx = B.bsr_ctx_create(4, 1)
    assert rc == B.BSR_OK
    buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda:0")
    p = buf.data_ptr()
    assert B.bsr_register(ctx, 0, [(64, 8)], [(0, 24, p)]) == B.BSR_ERR_ALIGN      # 24 % 16 != 0
    assert B.bsr_register(ctx, 0, [(64, 8)], [(0, 32, p + 8)]) == B.BSR_ERR_ALIGN  # misaligned base
    assert B.bsr_register(ctx, 0, [(48, 8)], [(0, 32, p)]) == B.BSR_ERR_INVALID    # 48 does not divide 256
    assert B.bsr_register(ctx, 0, [(64, 8), (64, 8)], [(1, 32, p), (0, 32, p)]) == B.BSR_ERR_INVALID
    assert B.bsr_register(ctx, 1, [(64, 8)], [(0, 32, p)]) == B.BSR_ERR_INVALID    # rank out of range
    assert B.bsr_register(ctx, 0, [(64, 8)], [(0, 32, p)]) == B.BSR_OK
    payload = np.zeros(256 * 32, dtype=np.uint8)
    assert B.bsr_tier_put(ctx, 0, 1, payload, payload.size - 16, [0]) == B.BSR_ERR_INVALID
    assert B.bsr_tier_put(ctx, 0, 1, payload, payload.size, [0]) == B.BSR_OK
    keys = np.array([1], dtype=np.uint64)
    assert B.bsr_req_create(ctx, keys, [np.array([0, 1, 2, 8], dtype=np.int32)])[0] == B.BSR_ERR_INVALID
    assert B.bsr_req_create(ctx, keys, [np.array([0, 1, 2, 2], dtype=np.int32)])[0] == B.BSR_ERR_INVALID
    assert B.bsr_req_create(ctx, keys, [np.array([0, 1, -1, 2], dtype=np.int32)])[0] == B.BSR_ERR_INVALID
    assert "table" in B.bsr_last_error(ctx)
    # an empty advertised prefix restores and commits to zero chunks
    rc, req = B.bsr_req_create(ctx, keys[:0], [np.zeros(0, dtype=np.int32)])
    assert rc == B.BSR_OK
    assert B.bsr_restore(ctx, req) == B.BSR_OK
    assert B.bsr_commit(ctx, req) == (B.BSR_OK, 0)
    assert B.bsr_req_release(ctx, req) == B.BSR_OK
    assert B.bsr_register(ctx, 0, [(64, 8)], [(0, 32, p)]) == B.BSR_ERR_STATE      # registration in use
    assert B.bsr_ctx_destroy(ctx) == B.BSR_OK


# ---------------------------------------------------------------- the bulk-copy install kernel
@pytest.mark.parametrize("layout_name,R,N,W,location", [
    ("tiny", 2, 9, 4, 0), ("tiny", 2, 70, 3, 0), ("tiny", 2, 11, 4, 1),
    ("hetero", 2, 6, 4, 0), ("hetero", 2, 5, 2, 1),
    ("baseline", 1, 16, 4, 0), ("baseline", 2, 6, 4, 1),
])
def test_bulk_install_kernel_matches_oracle(layout_name, R, N, W, location):
    layout = {"tiny": synth.tiny_layout, "hetero": synth.hetero_layout,
              "baseline": synth.baseline_layout}[layout_name]()
    case = Case(layout, R, N, seed=800 + N)
    ora = run_oracle(case, W)
    with GpuSide(case, W, location=location, install_variant=2) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)


def test_bulk_install_kernel_detects_corruption_and_computes_store_checksums():
    case = Case(synth.hetero_layout(), 2, 4, seed=900)
    with GpuSide(case, 2, install_variant=2, compute_ck=True) as gpu:
        B = gpu.B
        for (r, i), want in case.cks.items():
            rc, got = B.bsr_tier_checksums(gpu.ctx, r, case.keys[i], case.G)
            assert rc == B.BSR_OK and [int(x) for x in got] == want
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        lo, hi = case.reg.segment(2)
        case.payload[(1, 3)][lo:hi].view("<u4")[12345] ^= np.uint32(0x10)
        assert gpu.restore() == B.BSR_ERR_CHECKSUM
        assert gpu.commit() == 0 and (gpu.bitmap(4) == 0).all()


# ---------------------------------------------------------------- staging-free (direct) install
@pytest.mark.parametrize("layout_name,R,N,W", [("tiny", 2, 23, 4), ("hetero", 2, 6, 4), ("baseline", 2, 10, 4)])
def test_direct_install_from_pinned_slots_matches_oracle(layout_name, R, N, W):
    layout = {"tiny": synth.tiny_layout, "hetero": synth.hetero_layout,
              "baseline": synth.baseline_layout}[layout_name]()
    case = Case(layout, R, N, seed=1000 + N)
    ora = run_oracle(case, W)
    with GpuSide(case, W, direct_install=True) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)
        st = gpu.stats()
        assert st.h2d_copies == 0                                  # nothing went through the copy engine
        # corruption in a slot is still caught, exposure still collapses
        r, g, i, frac = synth.fault_site(R, case.G, 1, N, case=11, seed=3)
        gpu.B.bsr_test_inject(gpu.ctx, gpu.B.BSR_INJECT_CORRUPT_SLOT, r, g, i, frac)
        assert gpu.restore() == gpu.B.BSR_ERR_CHECKSUM
        assert gpu.commit() == 0 and (gpu.bitmap(N) == 0).all()


# ---------------------------------------------------------------- kernel choice by registration
def test_install_kernel_in_use_reports_the_choice():
    from paper_2608_17826_b200 import binding as B
    want = {"baseline": B.BSR_INSTALL_BULK, "hetero": B.BSR_INSTALL_BULK, "tiny": B.BSR_INSTALL_BULK,
            "short_runs": B.BSR_INSTALL_BULK}
    for name, layout in (("baseline", synth.baseline_layout()), ("hetero", synth.hetero_layout()),
                         ("tiny", synth.tiny_layout()), ("short_runs", synth.short_run_layout())):
        case = Case(layout, 1, 1, seed=1600)
        with GpuSide(case, 1) as gpu:
            assert B.bsr_install_kernel_in_use(gpu.ctx) == (B.BSR_OK, want[name])
        with GpuSide(case, 1, install_variant=B.BSR_INSTALL_BULK) as gpu:
            assert B.bsr_install_kernel_in_use(gpu.ctx) == (B.BSR_OK, B.BSR_INSTALL_BULK)
        with GpuSide(case, 1, install_variant=B.BSR_INSTALL_VECTOR) as gpu:
            assert B.bsr_install_kernel_in_use(gpu.ctx) == (B.BSR_OK, B.BSR_INSTALL_VECTOR)


# ---------------------------------------------------------------- many pipeline shapes
def test_many_pipeline_shapes_give_the_same_bytes():
    """Seeded sweep over W, fill threads, staging depth, chunks per install launch, install path and ranks
    on two small registrations (long runs; long runs mixed with spans of short ones): ordering bugs in the
    slot pool / copy / launch grouping / install pipeline would show as a byte or bitmap mismatch."""
    rng = np.random.default_rng(20260817)
    layouts = [synth.Layout("mid", [64, 16], [(0, 1024), (0, 48), (1, 256)]),
               synth.Layout("mixed", [64, 16, 32], [(0, 512)] * 2 + [(1, 16)] * 40 + [(1, 64)] * 3 + [(2, 32)] * 9 + [(2, 272)])]
    for trial in range(40):
        layout = layouts[trial % 2]
        R = int(rng.integers(1, 4))
        N = int(rng.integers(1, 40))
        W = int(rng.choice([1, 2, 3, 5, 8, 32, 64]))
        cfg = dict(load_concurrency=int(rng.choice([1, 2, 4, 8])), dev_staging_depth=int(rng.choice([0, 1, 2, 4, 7])),
                   install_variant=int(rng.choice([1, 2])), direct_install=bool(rng.integers(0, 3) == 0),
                   install_batch=int(rng.choice([0, 1, 3, 8, 64])))
        case = Case(layout, R, N, seed=1400 + trial)
        ora = run_oracle(case, W)
        with GpuSide(case, W, **cfg) as gpu:
            rc, keys, bm, n_hit = gpu.probe(tok_on_device=bool(trial % 2))
            assert rc == gpu.B.BSR_OK and n_hit == N, (trial, cfg)
            gpu.request(keys, n_hit)
            for _ in range(2):
                gpu.B.bsr_reset_stats(gpu.ctx)
                assert gpu.restore() == gpu.B.BSR_OK, (trial, cfg, gpu.B.bsr_last_error(gpu.ctx))
                _check_success(case, W, gpu, ora, N)


# ---------------------------------------------------------------- install launches take several chunks
@pytest.mark.parametrize("W,batch,depth,per_launch", [
    (32, 0, 0, 64),     # defaults: 64 descriptors = 32 chunks of each of the 2 rank slices
    (16, 0, 0, 64),     # ... whatever the window: a slot is free again once its copy has landed
    (4, 0, 0, 64),
    (1, 0, 0, 64),
    (16, 4, 0, 4),
    (16, 64, 3, 6),     # never more chunks per rank than staging buffers
    (2, 32, 16, 32),    # 16 chunks per rank per launch through a window of 2
    (16, 1, 0, 2),      # never less than one chunk of every rank slice
    (8, 256, 64, 96),   # the largest staging depth: the whole 48-chunk prefix of both slices in one launch
    (8, 256, 200, 96),  # ... which is also what a larger request is taken as
])
def test_install_launches_carry_the_configured_number_of_chunks(W, batch, depth, per_launch):
    layout = synth.Layout("mid", [64, 16], [(0, 1024), (0, 48), (1, 256)])
    R, N = 2, 48
    case = Case(layout, R, N, seed=1700)
    ora = run_oracle(case, W)
    with GpuSide(case, W, install_batch=batch, dev_staging_depth=depth) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        gpu.B.bsr_reset_stats(gpu.ctx)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)
        st = gpu.stats()
        assert st.install_descriptors == R * N
        assert st.install_launches == -(-R * N // per_launch)


def test_a_launch_group_that_cannot_grow_is_not_waited_for():
    """Two restores share a pool of 2 slots per rank while each would like 4 chunks per launch: neither
    can ever hold a full group, so a group is launched as soon as nothing else can make progress."""
    import threading
    layout = synth.Layout("mid", [64, 16], [(0, 1024), (1, 256)])
    R, N, W = 2, 12, 16
    case = Case(layout, R, N, seed=1701)
    ora = run_oracle(case, W)
    with GpuSide(case, W, budget_slots=2, timeout_ms=20000) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        reqs = []
        for k in range(2):
            flat = [t for tr in case.tables_prefix(N) for t in tr]
            rc, q = B.bsr_req_create(gpu.ctx, keys[:N], flat)
            assert rc == B.BSR_OK
            reqs.append(q)
        rcs = [None, None]

        def go(k):
            rcs[k] = B.bsr_restore(gpu.ctx, reqs[k], None)

        ts = [threading.Thread(target=go, args=(k,)) for k in range(2)]
        [t.start() for t in ts]
        [t.join() for t in ts]
        assert rcs == [B.BSR_OK, B.BSR_OK], B.bsr_last_error(gpu.ctx)
        for q in reqs:
            assert B.bsr_commit(gpu.ctx, q) == (B.BSR_OK, N)
        assert_paged_equal(gpu, ora["paged"])                    # both wrote the same bytes to the same blocks
        assert gpu.stats().peak_staging_bytes[0] == 2 * case.reg.slot_bytes
        for q in reqs:
            B.bsr_req_release(gpu.ctx, q)


# ---------------------------------------------------------------- calibration passes install nothing
def test_calibration_passes_move_the_bytes_but_install_nothing():
    layout = synth.Layout("mid", [64, 16], [(0, 1024), (0, 48), (1, 256)])
    R, N, W = 2, 20, 8
    case = Case(layout, R, N, seed=1702)
    ora = run_oracle(case, W)
    with GpuSide(case, W) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        for stages in (B.BSR_CAL_FILL, B.BSR_CAL_FILL_H2D):
            B.bsr_reset_stats(gpu.ctx)
            rc, sec = B.bsr_restore_calibrate(gpu.ctx, gpu.req, stages)
            assert rc == B.BSR_OK and sec > 0
            st = gpu.stats()
            assert st.install_launches == 0 and st.bytes_installed[0] == 0
            assert st.bytes_filled[0] == st.bytes_h2d[0] == st.h2d_copies == 0   # a calibration pass is not a restore
            assert st.peak_staging_bytes[0] == W * case.reg.slot_bytes       # the same slots were live
            assert gpu.commit() == 0 and (gpu.bitmap(N) == 0).all()          # nothing was installed ...
            for r in range(R):
                for l in range(len(layout.tensors)):
                    assert bool((gpu.paged[r][l] == synth.CANARY).all())     # ... and no paged byte written
        assert B.bsr_restore_calibrate(gpu.ctx, gpu.req, 7)[0] == B.BSR_ERR_INVALID
        with GpuSide(case, W, direct_install=True) as direct:           # no device staging to copy into
            direct.request(keys, n_hit)
            assert direct.B.bsr_restore_calibrate(direct.ctx, direct.req, B.BSR_CAL_FILL_H2D)[0] == B.BSR_ERR_STATE
            assert direct.B.bsr_restore_calibrate(direct.ctx, direct.req, B.BSR_CAL_FILL)[0] == B.BSR_OK
        # a missing chunk fails a calibration pass like it fails a restore
        assert B.bsr_tier_remove(gpu.ctx, 1, keys[5]) == B.BSR_OK
        assert B.bsr_restore_calibrate(gpu.ctx, gpu.req, B.BSR_CAL_FILL)[0] == B.BSR_ERR_MISSING
        p = case.payload[(1, 5)]
        assert B.bsr_tier_put(gpu.ctx, 1, keys[5], p, p.size, case.cks[(1, 5)]) == B.BSR_OK
        # the request is untouched: a real restore afterwards succeeds
        B.bsr_reset_stats(gpu.ctx)
        assert gpu.restore() == B.BSR_OK, B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)


def test_fill_threads_bound_to_the_gpus_numa_node_restore_the_same_bytes():
    """numa_bind = ALWAYS binds the fill threads and the thread that allocates the pinned pool to the CPUs
    of the GPU's NUMA node whenever the platform names one (on a single-node host that is every CPU the
    process may use); OFF never binds.  Either way the restore is the same and the stats say what was done."""
    import os
    layout = synth.Layout("mid", [64, 16], [(0, 1024), (0, 48), (1, 256)])
    R, N, W = 2, 20, 8
    case = Case(layout, R, N, seed=1703)
    ora = run_oracle(case, W)
    allowed = sorted(os.sched_getaffinity(0))
    for mode in ("off", "always"):
        from paper_2608_17826_b200 import binding as B
        with GpuSide(case, W, numa_bind=B.BSR_NUMA_OFF if mode == "off" else B.BSR_NUMA_ALWAYS) as gpu:
            rc, keys, bm, n_hit = gpu.probe()
            gpu.request(keys, n_hit)
            assert gpu.restore() == B.BSR_OK, B.bsr_last_error(gpu.ctx)
            _check_success(case, W, gpu, ora, N)
            node = gpu.stats().fill_numa_node
            assert node == -1 if mode == "off" else node >= -1
    assert sorted(os.sched_getaffinity(0)) == allowed            # the caller's own mask is never touched


def test_registration_with_an_empty_group_is_rejected():
    from paper_2608_17826_b200 import binding as B
    import torch
    rc, ctx = B.bsr_ctx_create(2, 1)
    assert rc == B.BSR_OK
    t = torch.zeros(64 * 16 * 4, dtype=torch.uint8, device="cuda")
    assert B.bsr_register(ctx, 0, [(64, 4), (64, 4), (64, 4)], [(0, 16, t.data_ptr()), (2, 16, t.data_ptr())]) \
        == B.BSR_ERR_INVALID
    assert "group 1 has no tensor" in B.bsr_last_error(ctx)
    B.bsr_ctx_destroy(ctx)


# ---------------------------------------------------------------- the timeline shows Eq. 3
@pytest.mark.parametrize("N,W,depth", [(40, 4, 2), (25, 8, 4), (9, 16, 1)])
def test_timeline_of_a_restore_never_has_more_than_w_live_chunks_per_rank(N, W, depth):
    layout = synth.Layout("mid", [64, 16], [(0, 1024), (1, 256)])      # 320 KiB chunks
    R = 2
    case = Case(layout, R, N, seed=1300 + N)
    with GpuSide(case, W, dev_staging_depth=depth) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == B.BSR_OK
        rc, tr = B.bsr_get_trace(gpu.ctx)
        assert rc == B.BSR_OK and len(tr) == N * R
        assert sorted((int(t["chunk"]), int(t["rank"])) for t in tr) == [(i, r) for i in range(N) for r in range(R)]
        assert (tr["t_admit_ns"] <= tr["t_filled_ns"]).all() and (tr["t_filled_ns"] <= tr["t_submit_ns"]).all()
        assert (tr["t_submit_ns"] < tr["t_done_ns"]).all() and (tr["slot"] < W).all()
        for r in range(R):
            t = tr[tr["rank"] == r]
            # sweep the admit (+1) and release (-1) instants: live slots of the rank never exceed W (Eq. 3) ...
            ev = sorted([(int(x), 1) for x in t["t_admit_ns"]] + [(int(x), -1) for x in t["t_done_ns"]],
                        key=lambda e: (e[0], e[1]))
            live = peak = 0
            for _, d in ev:
                live += d
                peak = max(peak, live)
            assert peak == min(N, W)                                    # ... and do reach it
            # no slot is handed to a second chunk while its previous chunk is still live
            for s in set(int(x) for x in t["slot"]):
                u = t[t["slot"] == s]
                u = u[np.argsort(u["t_admit_ns"])]
                assert (u["t_done_ns"][:-1] <= u["t_admit_ns"][1:]).all()
        assert gpu.stats().peak_staging_bytes[0] == min(N, W) * case.reg.slot_bytes


# ---------------------------------------------------------------- limits of the interface
def test_maximum_ranks_groups_and_extreme_block_sizes():
    """8 rank slices x 8 allocator groups (the interface maxima), block sizes from 2 tokens (128 blocks
    per chunk) to 256 tokens (one block per chunk), tensors of 16 B/token (16-byte runs split nowhere)."""
    blocks = [2, 4, 8, 16, 32, 64, 128, 256]
    tensors = [(g, e) for g, e in zip(range(8), [16, 32, 16, 48, 16, 64, 16, 80])] + [(7, 16)]
    layout = synth.Layout("limits", blocks, sorted(tensors))
    R, N, W = 8, 5, 2
    case = Case(layout, R, N, seed=1200)
    ora = run_oracle(case, W)
    assert ora["status"] == O.OK
    for cfg in (dict(), dict(install_variant=1), dict(direct_install=True), dict(location=1)):
        with GpuSide(case, W, **cfg) as gpu:
            rc, keys, bm, n_hit = gpu.probe()
            assert n_hit == N
            gpu.request(keys, n_hit)
            assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
            _check_success(case, W, gpu, ora, N)


# ---------------------------------------------------------------- a wait inside the kernel runs out
@pytest.mark.parametrize("layout_name", ["tiny", "baseline"])
def test_bounded_wait_inside_the_install_kernel_reports_timeout_and_context_survives(layout_name):
    """One tile of one launch is never loaded (host-armed hook) and the kernel's waits are bounded at
    50 ms: they expire, the kernel raises its error flag, drains its copies in flight and returns.
    Nothing faults or hangs; the restore fails closed and the next one succeeds."""
    layout = {"tiny": synth.tiny_layout, "baseline": synth.baseline_layout}[layout_name]()
    R, N, W = 2, 6, 4
    case = Case(layout, R, N, seed=1100)
    ora = run_oracle(case, W)
    with GpuSide(case, W, install_variant=2) as gpu:          # the waits live in the bulk-copy kernel
        B = gpu.B
        assert B.bsr_install_kernel_in_use(gpu.ctx) == (B.BSR_OK, B.BSR_INSTALL_BULK)
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert B.bsr_test_inject(gpu.ctx, B.BSR_INJECT_KERNEL_WAIT, 1, 0, 3, 0) == B.BSR_OK
        assert gpu.restore() == B.BSR_ERR_TIMEOUT
        assert "bounded wait" in B.bsr_last_error(gpu.ctx)
        assert gpu.commit() == 0 and (gpu.bitmap(N) == 0).all()
        B.bsr_reset_stats(gpu.ctx)
        assert gpu.restore() == B.BSR_OK                      # one shot: the context is intact
        _check_success(case, W, gpu, ora, N)


# ---------------------------------------------------------------- launch-shape corner cases
@pytest.mark.parametrize("variant,location", [(1, 0), (1, 1), (2, 0), (2, 1)])
def test_more_tiles_per_chunk_than_ctas_in_the_grid(variant, location):
    """160 tensors in 16-token blocks = 2,560 runs per chunk, more than the vector kernel's
    smallest grid: one CTA then handles tiles of the same chunk that belong to different groups
    and must keep their checksums apart."""
    layout = synth.Layout("many_runs", [16, 16], [(0, 16)] * 100 + [(1, 32)] * 60)
    R, N, W = 2, 5, 2
    case = Case(layout, R, N, seed=1500 + variant)
    ora = run_oracle(case, W)
    with GpuSide(case, W, location=location, install_variant=variant) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)


@pytest.mark.parametrize("variant,location", [(1, 0), (1, 1), (2, 0), (2, 1)])
@pytest.mark.parametrize("layout_name", ["odd_spans", "short_runs"])
def test_spans_of_several_short_runs_land_in_their_own_blocks(layout_name, variant, location):
    """Short destination runs travel in spans of several whole runs whose stores are scattered run by
    run.  `odd_spans`: 768-byte runs, 21 to a span, 16 to a tensor, so that spans begin in the middle
    of a tensor and run on into the next one (and the next family, of 256-byte runs, starts at an odd
    place); `short_runs`: the registration dominated by 256-byte runs, 64 to a span over 4 tensors."""
    layout = {"odd_spans": synth.Layout("odd_spans", [16, 64], [(0, 48)] * 5 + [(0, 16)] * 7 + [(1, 128)] * 3),
              "short_runs": synth.short_run_layout()}[layout_name]
    R, N, W = 2, 5, 2
    case = Case(layout, R, N, seed=1800 + variant)
    ora = run_oracle(case, W)
    with GpuSide(case, W, location=location, install_variant=variant) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)


def test_stores_of_long_runs_followed_by_a_long_stretch_of_short_run_spans_in_one_cta():
    """297 spans per chunk (16 pieces of long runs, then 281 spans of 256-byte runs) against a grid of
    2 x 148 CTAs: CTA b takes span (b - n) mod 297 of chunk n, so the CTAs with small b first issue a
    few bulk stores and then only spans whose stores are scattered by the sum warps.  The stages of
    those last bulk stores must be handed back although no further store follows them."""
    layout = synth.Layout("stores_then_spans", [64, 16], [(0, 512)] * 2 + [(1, 16)] * 1124)
    R, N, W = 1, 24, 32
    case = Case(layout, R, N, seed=1900)
    ora = run_oracle(case, W)
    for location in (1, 0):
        with GpuSide(case, W, location=location, install_variant=2, timeout_ms=10000) as gpu:
            rc, keys, bm, n_hit = gpu.probe()
            gpu.request(keys, n_hit)
            assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
            _check_success(case, W, gpu, ora, N)


def test_admission_stops_at_the_first_failure():
    """After the failing chunk is observed nothing more is admitted: at most the chunks of its launch
    group (up to D per rank) and those already in the window were fetched, not the remaining hundreds."""
    layout = synth.tiny_layout()
    R, N, W, bad, D = 2, 300, 4, 6, 32
    case = Case(layout, R, N, seed=1600)
    with GpuSide(case, W) as gpu:
        B = gpu.B
        rc, keys, bm, n_hit = gpu.probe()
        gpu.request(keys, n_hit)
        lo, hi = case.reg.segment(0)
        case.payload[(1, bad)][lo:hi].view("<u4")[5] ^= np.uint32(2)
        assert gpu.restore() == B.BSR_ERR_CHECKSUM
        st = gpu.stats()
        for r in range(R):
            assert st.bytes_filled[r] <= (bad + 1 + D + 2 * W) * case.reg.chunk_bytes
            assert st.bytes_h2d[r] <= (bad + 1 + D + 2 * W) * case.reg.chunk_bytes
            assert st.bytes_installed[r] <= (bad + 1 + D) * case.reg.chunk_bytes
        assert gpu.commit() == 0 and (gpu.bitmap(N) == 0).all()


def test_two_contexts_with_different_registrations_restore_at_the_same_time():
    """Two engines in one process (different geometry, W, kernel variant) restore concurrently on
    one GPU; neither sees the other: both are bit-exact and each keeps its own staging law."""
    import threading
    case_a = Case(synth.tiny_layout(), 2, 60, seed=1800)
    case_b = Case(synth.hetero_layout(), 1, 7, seed=1801, reg_id=5)
    ora_a, ora_b = run_oracle(case_a, 4), run_oracle(case_b, 2)
    with GpuSide(case_a, 4, install_variant=1) as ga, GpuSide(case_b, 2, install_variant=2) as gb:
        for g in (ga, gb):
            rc, keys, bm, n_hit = g.probe()
            assert rc == g.B.BSR_OK and n_hit == g.case.N
            g.request(keys, n_hit)
        out = {}
        gate = threading.Barrier(2)

        def work(name, g):
            gate.wait()
            out[name] = [g.restore() for _ in range(3)]

        ts = [threading.Thread(target=work, args=(n, g)) for n, g in (("a", ga), ("b", gb))]
        [t.start() for t in ts]
        [t.join() for t in ts]
        assert out == {"a": [ga.B.BSR_OK] * 3, "b": [ga.B.BSR_OK] * 3}
        for g, ora, W in ((ga, ora_a, 4), (gb, ora_b, 2)):
            assert g.commit() == g.case.N
            assert np.array_equal(g.bitmap(g.case.N), ora["req"].bitmap())
            assert_paged_equal(g, ora["paged"])
            st = g.stats()
            assert st.peak_staging_bytes[0] == W * g.case.reg.slot_bytes == st.ring_bytes_allocated[0]


@pytest.mark.parametrize("case_no", range(12))
def test_random_registrations_match_the_oracle(case_no):
    """Seeded random geometry: 1-4 groups, block sizes 16...256, 1-5 tensors per group of 16...1,120
    bytes per token, 1-3 ranks, 1-9 chunks, W 1-5, either kernel, tier in host or device memory."""
    rng = np.random.Generator(np.random.SFC64(0xB5B5 + case_no))
    G = int(rng.integers(1, 5))
    blocks = [int(rng.choice([16, 32, 64, 128, 256])) for _ in range(G)]
    tensors = [(g, 16 * int(rng.integers(1, 71))) for g in range(G) for _ in range(int(rng.integers(1, 6)))]
    layout = synth.Layout(f"random{case_no}", blocks, tensors)
    R, N, W = int(rng.integers(1, 4)), int(rng.integers(1, 10)), int(rng.integers(1, 6))
    variant, location = 1 + case_no % 2, (case_no // 2) % 2
    case = Case(layout, R, N, seed=1900 + case_no)
    ora = run_oracle(case, W)
    assert ora["status"] == O.OK
    with GpuSide(case, W, location=location, install_variant=variant) as gpu:
        rc, keys, bm, n_hit = gpu.probe()
        assert rc == gpu.B.BSR_OK and n_hit == N and np.array_equal(keys, ora["keys"])
        gpu.request(keys, n_hit)
        assert gpu.restore() == gpu.B.BSR_OK, gpu.B.bsr_last_error(gpu.ctx)
        _check_success(case, W, gpu, ora, N)

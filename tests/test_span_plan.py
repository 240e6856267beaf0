"""The span plan of the install kernels (host logic, no GPU): how a chunk of a registration is cut
into the contiguous spans that are loaded as units, checked against the oracle's layout arithmetic
(`Registration.tensor_offset`, the chunk byte layout) for every byte of a chunk."""
import numpy as np
import pytest

from oracle import bsr_oracle as O
from paper_2608_17826_b200 import synth

LAYOUTS = {
    "baseline": synth.baseline_layout, "hetero": synth.hetero_layout, "mtp_on": synth.mtp_on_layout,
    "short_runs": synth.short_run_layout, "tiny": synth.tiny_layout,
    "odd_spans": lambda: synth.Layout("odd_spans", [16, 64], [(0, 48)] * 5 + [(0, 16)] * 7 + [(1, 128)] * 3),
    "stores_then_spans": lambda: synth.Layout("stores_then_spans", [64, 16], [(0, 512)] * 2 + [(1, 16)] * 1124),
    "extremes": lambda: synth.Layout("extremes", [2, 256, 128], [(0, 16), (0, 16), (1, 16), (1, 4096), (2, 80)]),
}
STAGE, SPAN_RUN_MAX = 16384, 1024


@pytest.mark.parametrize("name", sorted(LAYOUTS))
def test_span_plan_covers_every_byte_of_a_chunk_once_and_names_its_destination(name):
    from paper_2608_17826_b200 import binding as B
    layout = LAYOUTS[name]()
    reg = O.Registration(list(layout.block_tokens), list(layout.tensors))
    rc, spans = B.bsr_plan_spans(layout.block_tokens, layout.tensors)
    assert rc == B.BSR_OK and len(spans) > 0
    # the spans tile the chunk in order, with no gap and no overlap
    assert int(spans["src_off"][0]) == 0
    assert (spans["src_off"][1:] == spans["src_off"][:-1] + spans["bytes"][:-1]).all()
    assert int(spans["src_off"][-1]) + int(spans["bytes"][-1]) == reg.chunk_bytes
    assert (spans["bytes"] <= STAGE).all() and (spans["bytes"] % 16 == 0).all() and (spans["bytes"] > 0).all()
    # every byte of the chunk: which (tensor, block, offset in the block's run) the plan sends it to,
    # against where the oracle's layout puts it
    want_tensor = np.empty(reg.chunk_bytes, dtype=np.int32)
    want_block = np.empty(reg.chunk_bytes, dtype=np.int32)
    want_within = np.empty(reg.chunk_bytes, dtype=np.int64)
    for l, (g, e) in enumerate(reg.tensors):
        run = reg.block_tokens[g] * e
        lo = reg.tensor_offset(l)
        k = np.arange(256 * e)
        want_tensor[lo: lo + 256 * e] = l
        want_block[lo: lo + 256 * e] = k // run
        want_within[lo: lo + 256 * e] = k % run
    got_tensor, got_block, got_within = np.empty_like(want_tensor), np.empty_like(want_block), np.empty_like(want_within)
    for s in spans:
        g, run, n_runs = int(s["group"]), int(s["run_bytes"]), int(s["n_runs"])
        nb = reg.blocks_per_chunk(g)
        lo, n = int(s["src_off"]), int(s["bytes"])
        assert run == reg.block_tokens[g] * reg.tensors[int(s["tensor"])][1]
        k = np.arange(n)
        if n_runs == 1:
            assert int(s["dst_off"]) + n <= run                     # a piece of one run
            got_tensor[lo: lo + n] = int(s["tensor"])
            got_block[lo: lo + n] = int(s["block"])
            got_within[lo: lo + n] = int(s["dst_off"]) + k
        else:
            assert int(s["dst_off"]) == 0 and n == n_runs * run and run <= SPAN_RUN_MAX   # whole short runs
            vb = int(s["block"]) + k // run
            got_tensor[lo: lo + n] = int(s["tensor"]) + vb // nb
            got_block[lo: lo + n] = vb % nb
            got_within[lo: lo + n] = k % run
            # all tensors a span runs over have one shape and one group
            ts = set(int(x) for x in np.unique(got_tensor[lo: lo + n]))
            assert len({reg.tensors[t] for t in ts}) == 1
    assert np.array_equal(got_tensor, want_tensor)
    assert np.array_equal(got_block, want_block)
    assert np.array_equal(got_within, want_within)
    # no run longer than the threshold is scattered by vector stores, no shorter one gets a stage to itself
    for s in spans:
        if int(s["n_runs"]) == 1 and int(s["run_bytes"]) <= SPAN_RUN_MAX:
            nb = reg.blocks_per_chunk(int(s["group"]))
            family = [t for t in range(len(reg.tensors)) if reg.tensors[t] == reg.tensors[int(s["tensor"])]]
            assert len(family) * nb == 1 or int(s["bytes"]) == int(s["run_bytes"])   # a last, lone run of a family


def test_span_plan_rejects_what_registration_rejects():
    from paper_2608_17826_b200 import binding as B
    assert B.bsr_plan_spans([64], [(0, 24)])[0] == B.BSR_ERR_ALIGN             # bytes per token not a multiple of 16
    assert B.bsr_plan_spans([48], [(0, 16)])[0] == B.BSR_ERR_INVALID           # block size does not divide the chunk
    assert B.bsr_plan_spans([64, 64], [(1, 16), (0, 16)])[0] == B.BSR_ERR_INVALID   # not group-major
    assert B.bsr_plan_spans([64], [(1, 16)])[0] == B.BSR_ERR_INVALID           # unknown group


def test_span_counts_of_the_benchmarked_registrations():
    from paper_2608_17826_b200 import binding as B
    counts = {}
    for name in ("baseline", "hetero", "short_runs"):
        layout = LAYOUTS[name]()
        rc, spans = B.bsr_plan_spans(layout.block_tokens, layout.tensors)
        counts[name] = (len(spans), int((spans["n_runs"] > 1).sum()))
    assert counts["baseline"] == (1292, 0)        # 56 x 4 runs in 5 pieces each + 43 x 4 runs of 2 KiB on their own
    assert counts["short_runs"] == (600, 400)     # 25,600 runs of 256 B, 64 to a span; 200 runs of 8 KiB
    assert counts["hetero"][1] > 0


# ---------------------------------------------------------------- fill pieces of a restore
MIB = 1 << 20


@pytest.mark.parametrize("chunk,N,R,threads", [(16_408_576, 128, 2, 8), (16_408_576, 4, 2, 8), (16_408_576, 1, 1, 8),
                                               (16_633_856, 37, 2, 3), (8_192_000, 32, 2, 16), (24_576, 300, 2, 8),
                                               (327_680, 40, 8, 4), (100 * MIB + 16, 3, 1, 2)])
def test_fill_pieces_tile_every_chunk_in_admission_order(chunk, N, R, threads):
    """Host-only plan of the pieces a restore is fetched and copied in: every (chunk, rank) item tiled exactly,
    items in admission order, piece sizes as the schedule states."""
    from paper_2608_17826_b200 import binding as B
    rc, p = B.bsr_plan_pieces(chunk, N, R, threads)
    assert rc == B.BSR_OK and len(p) > 0
    items = p["chunk"].astype(np.int64) * R + p["rank"]
    assert (np.diff(items) >= 0).all() and sorted(set(items.tolist())) == list(range(N * R))   # admission order, none missing
    for it in range(N * R):
        q = p[items == it]
        assert int(q["offset"][0]) == 0 and int(q["bytes"].sum()) == chunk                      # the chunk, exactly ...
        assert (q["offset"][1:] == np.cumsum(q["bytes"].astype(np.int64))[:-1]).all()           # ... in ascending pieces
    assert int(p["bytes"].max()) <= 8 * MIB
    assert int(p["bytes"].min()) >= min(chunk, 256 << 10)                                       # no sliver
    head = p[items < R]
    assert int(head["bytes"].max()) <= MIB + (256 << 10)                                        # first chunk of every rank: 1 MiB
    n_tail = min(N * R, -(-(-(-threads * 8 * MIB // chunk)) // R) * R)
    tail = p[items >= N * R - n_tail]
    assert int(tail["bytes"].max()) <= max(2 * MIB + (256 << 10), MIB + (256 << 10))            # last chunks: 2 MiB
    body = p[(items >= R) & (items < N * R - n_tail)]
    if len(body):
        # from 1 MiB the wanted size grows by 512 KiB per piece up to 8 MiB and stays there; a piece is
        # shorter only where its chunk ends
        want = np.minimum(8 * MIB, MIB + (512 << 10) * (1 + np.arange(len(body), dtype=np.int64)))
        ends_chunk = body["offset"].astype(np.int64) + body["bytes"] == chunk
        assert (body["bytes"] <= want + (256 << 10)).all()
        assert ((body["bytes"] == want) | ends_chunk).all()


def test_fill_piece_plan_rejects_bad_arguments():
    from paper_2608_17826_b200 import binding as B
    assert B.bsr_plan_pieces(0, 4, 2, 8)[0] == B.BSR_ERR_INVALID
    assert B.bsr_plan_pieces(1 << 32, 4, 2, 8)[0] == B.BSR_ERR_INVALID
    assert B.bsr_plan_pieces(4096, 4, 0, 8)[0] == B.BSR_ERR_INVALID
    assert B.bsr_plan_pieces(4096, 4, 9, 8)[0] == B.BSR_ERR_INVALID
    assert B.bsr_plan_pieces(4096, 4, 2, 0)[0] == B.BSR_ERR_INVALID
    rc, p = B.bsr_plan_pieces(4096, 0, 2, 8)
    assert rc == B.BSR_OK and len(p) == 0

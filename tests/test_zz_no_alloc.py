"""The allocation-free key entry point against the regular probe, through the C interface.

Collected last on purpose: a failure here cannot hide the result of any other test.  The
entry point keeps its scratch in a fixed array inside the library (for callers that cannot
cudaMalloc: an engine whose KV pool already owns the GPU's memory, or scheduler code that cannot
take cudaMalloc's device-wide synchronisation), and that array keeps the previous call's contents,
so the check is made on two calls in a row, the second one shorter than the first.
"""
import numpy as np
import pytest

from paper_2608_17826_b200 import synth

pytestmark = pytest.mark.gpu


def test_noalloc_keys_equal_probe_keys_on_two_calls_in_a_row():
    import torch
    from paper_2608_17826_b200 import binding as B

    dev = torch.device("cuda:0")
    reg_id = 0x5EED
    rc, ctx = B.bsr_ctx_create(4, 1, reg_id=reg_id)
    assert rc == B.BSR_OK
    try:
        stream = torch.cuda.current_stream().cuda_stream
        for n_chunks, tail, salt in [(300, 17, 0xABCDEF), (37, 0, 99), (300, 17, 0xABCDEF)]:
            tok = synth.tokens(n_chunks * 256 + tail, seed=1000 + n_chunks)
            d_tok = torch.from_numpy(tok).to(dev)
            rc, want, _, _ = B.bsr_probe(ctx, d_tok.data_ptr(), len(tok), salt, True)   # existing entry point
            assert rc == B.BSR_OK and len(want) == n_chunks
            d_keys = torch.zeros(n_chunks, dtype=torch.int64, device=dev)
            torch.cuda.synchronize()
            rc = B.bsr_probe_keys_noalloc(0, d_tok.data_ptr(), len(tok), salt, reg_id, d_keys.data_ptr(), stream)
            assert rc == B.BSR_OK
            torch.cuda.synchronize()
            got = d_keys.cpu().numpy().view(np.uint64)
            assert np.array_equal(got, want)                                             # bit-exact
        # beyond the fixed scratch: rejected before anything is launched
        big = (B.BSR_NOALLOC_MAX_CHUNKS + 1) * 256
        d_tok = torch.zeros(big, dtype=torch.int32, device=dev)
        d_keys = torch.zeros(B.BSR_NOALLOC_MAX_CHUNKS + 1, dtype=torch.int64, device=dev)
        assert B.bsr_probe_keys_noalloc(0, d_tok.data_ptr(), big, 1, 1, d_keys.data_ptr(), stream) == B.BSR_ERR_INVALID
        # exactly the maximum is accepted and matches
        n = B.BSR_NOALLOC_MAX_CHUNKS
        tok = synth.tokens(n * 256, seed=77)
        d_tok = torch.from_numpy(tok).to(dev)
        rc, want, _, _ = B.bsr_probe(ctx, d_tok.data_ptr(), len(tok), 5, True)
        assert rc == B.BSR_OK
        torch.cuda.synchronize()
        assert B.bsr_probe_keys_noalloc(0, d_tok.data_ptr(), len(tok), 5, reg_id, d_keys.data_ptr(), stream) == B.BSR_OK
        torch.cuda.synchronize()
        assert np.array_equal(d_keys[:n].cpu().numpy().view(np.uint64), want)
    finally:
        B.bsr_ctx_destroy(ctx)

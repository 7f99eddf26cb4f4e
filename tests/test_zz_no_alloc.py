"""blink_sample_noalloc against blink_sample, through the C ABI.

Some users of the library cannot allocate device memory while they run: a serving process
that gave all free HBM to the KV pool when it started (a later cudaMalloc may fail), or code
that cannot afford the device-wide synchronisation that cudaFree implies.  For them the
library offers the sampler with its scratch in a fixed array inside the library image.  This
test checks that the variant returns exactly the tokens of the allocating entry point (the
sampler's results are integers, so the comparison is for equality), on two calls in a row
with different sizes, because the scratch array is shared and keeps what the previous call
left in it.  The file name sorts last so that it runs after every other test.
"""
import numpy as np
import pytest
import torch

from paper_2604_07609_b200 import binding as B

pytestmark = pytest.mark.gpu


def _inputs(rows, vocab, seed):
    rng = np.random.default_rng(seed)
    logits = (rng.normal(size=(rows, vocab)) * 1.5).astype(np.float32)
    top_k = np.array([(0, 50, 7, 64)[i % 4] for i in range(rows)], dtype=np.int32)
    temp = np.where(np.arange(rows) % 2 == 0, 0.8, 1.25).astype(np.float32)
    ticket = (np.arange(rows, dtype=np.uint64) * 131 + seed).astype(np.uint64)
    gen = (np.arange(rows) * 3 % 211).astype(np.int32)
    sd = (np.arange(rows, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15)) ^ np.uint64(seed)
    dev = torch.from_numpy(logits).cuda()
    torch.cuda.synchronize()     # the entry point works on a stream of its own: the logits must be complete
    return dev, top_k, temp, ticket, gen, sd


def test_no_alloc_sampler_equals_allocating_sampler_on_two_calls_in_a_row():
    first = _inputs(96, 32000, 11)       # fills 96 rows of the shared scratch
    second = _inputs(37, 128256, 12)     # a shorter call afterwards must not see the first call's rows
    for args in (first, second):
        want = B.blink_sample(*args)
        got = B.blink_sample_noalloc(*args)
        assert got.dtype == np.int32 and got.shape == want.shape
        assert np.array_equal(got, want)
        assert (got >= 0).all() and (got < args[0].shape[1]).all()


def test_no_alloc_sampler_at_its_row_limit_uses_the_whole_scratch():
    """Exactly the maximum number of rows (small vocabulary): the last entries of every carved
    sub-array of the fixed scratch are written and read."""
    args = _inputs(B.SAMPLE_NOALLOC_MAX_ROWS, 512, 13)
    want = B.blink_sample(*args)
    got = B.blink_sample_noalloc(*args)
    assert np.array_equal(got, want)
    again = B.blink_sample_noalloc(*_inputs(5, 512, 14))      # and a short call right after it
    assert np.array_equal(again, B.blink_sample(*_inputs(5, 512, 14)))


def test_no_alloc_sampler_refuses_more_rows_than_its_scratch_holds():
    rows = B.SAMPLE_NOALLOC_MAX_ROWS + 1
    logits = torch.zeros((rows, 16), dtype=torch.float32, device="cuda")
    z = np.zeros(rows)
    rc = B.blink_sample_noalloc(logits, z, z + 1.0, z, z, z, raise_on_error=False)
    assert rc == B.BLINK_ETOOBIG
    assert b"capacity" in B.lib().blink_strerror(rc)

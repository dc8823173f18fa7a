"""The allocation-free compaction entry point (asx_compact_static).

Some users of this library cannot allocate device memory at the point where they need a
kept-row list: a serving loop where cudaMalloc would synchronise the device, code that runs
after a framework has taken all device memory into its own pool, or a plug-in that is only
handed raw buffers.  For them the library carries the scan's scratch inside its own image.
This test calls that entry point through the C ABI twice in a row (the second call finds the
first call's leftovers in the shared scratch) and checks that the kept-row list and the count
are identical, bit for bit, to what the ordinary entry point (asx_compact, caller-provided
scratch) returns for the same masks.  It runs in a file of its own, collected last.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
from paper_2309_06626_b200.binding import COMPACT_STATIC_MAX_ROWS

pytestmark = pytest.mark.gpu


def _reference(mask_dev):
    kept, count, scratch = asx.compact_mask(mask_dev)
    st = int(torch.cuda.current_stream().cuda_stream)
    assert asx.lib().asx_compact_status(scratch.data_ptr(), st) == 0
    c = int(count.item())
    return kept[:c].cpu().numpy(), c


def _static(mask_dev):
    rows = mask_dev.numel()
    kept = torch.full((max(rows, 1),), -7, dtype=torch.int32, device="cuda")
    count = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    st = int(torch.cuda.current_stream().cuda_stream)
    rc = asx.lib().asx_compact_static(mask_dev.data_ptr(), rows, kept.data_ptr(), count.data_ptr(), st)
    assert rc == 0, f"asx_compact_static returned {rc}"
    torch.cuda.synchronize()
    c = int(count.item())
    return kept[:c].cpu().numpy(), c


def test_static_compaction_matches_ordinary_entry_point_twice_in_a_row():
    rng = np.random.default_rng(20260906)
    # first a mask that spans many scan tiles, then a smaller one with a different density, so
    # that the second call starts from scratch words the first call left behind
    masks = [(rng.random(1_000_003) < 0.4).astype(np.uint8), (rng.random(70_001) < 0.9).astype(np.uint8)]
    for m in masks:
        md = torch.from_numpy(m).cuda()
        ref_kept, ref_count = _reference(md)
        got_kept, got_count = _static(md)
        assert got_count == ref_count == int(m.sum())
        assert np.array_equal(got_kept, ref_kept)
        assert np.array_equal(got_kept, oracle.kept_list(m))          # and both equal the definition


def test_static_compaction_rejects_sizes_beyond_its_scratch():
    st = int(torch.cuda.current_stream().cuda_stream)
    small = torch.zeros(16, dtype=torch.uint8, device="cuda")
    out = torch.zeros(16, dtype=torch.int32, device="cuda")
    rc = asx.lib().asx_compact_static(small.data_ptr(), COMPACT_STATIC_MAX_ROWS + 1, out.data_ptr(),
                                      out.data_ptr(), st)
    assert rc == 2                                   # ASX_ERR_UNSUPPORTED, nothing launched
    assert asx.lib().asx_compact_static(small.data_ptr(), -1, out.data_ptr(), out.data_ptr(), st) == 1
    torch.cuda.synchronize()


@pytest.mark.parametrize("rows", [0, 1, 16384, 16385, COMPACT_STATIC_MAX_ROWS])
def test_static_compaction_sizes_at_the_edges_of_its_two_forms(rows):
    """No rows, one row, the largest mask the one-block form takes, the smallest the two passes take,
    and the largest the built-in scratch holds (every word of it in use)."""
    rng = np.random.default_rng(rows + 3)
    m = (rng.random(rows) < 0.37).astype(np.uint8)
    md = torch.from_numpy(m).cuda() if rows else torch.zeros(0, dtype=torch.uint8, device="cuda")
    got_kept, got_count = _static(md)
    assert got_count == int(m.sum())
    assert np.array_equal(got_kept, oracle.kept_list(m))


@pytest.mark.parametrize("rows", [12_000, 1_600_000])
def test_two_static_calls_without_a_synchronisation_between_them(rows):
    """Two calls on one stream, different masks, no host synchronisation in between: the second starts
    while the first may still be running and finds its words in the shared scratch."""
    rng = np.random.default_rng(rows)
    ma, mb = (rng.random(rows) < 0.6).astype(np.uint8), (rng.random(rows) < 0.2).astype(np.uint8)
    da, db = torch.from_numpy(ma).cuda(), torch.from_numpy(mb).cuda()
    ka, kb = (torch.full((rows,), -7, dtype=torch.int32, device="cuda") for _ in range(2))
    ca, cb = (torch.full((1,), -7, dtype=torch.int32, device="cuda") for _ in range(2))
    st = int(torch.cuda.current_stream().cuda_stream)
    assert asx.lib().asx_compact_static(da.data_ptr(), rows, ka.data_ptr(), ca.data_ptr(), st) == 0
    assert asx.lib().asx_compact_static(db.data_ptr(), rows, kb.data_ptr(), cb.data_ptr(), st) == 0
    torch.cuda.synchronize()
    for m, k, c in ((ma, ka, ca), (mb, kb, cb)):
        n = int(c.item())
        assert n == int(m.sum()) and np.array_equal(k[:n].cpu().numpy(), oracle.kept_list(m))

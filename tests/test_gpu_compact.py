"""S1 on the GPU: the kept-row list must equal the oracle's bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx

pytestmark = pytest.mark.gpu


def _compact(mask_np, offset=0):
    buf = torch.zeros(mask_np.size + offset + 16, dtype=torch.uint8, device="cuda")
    view = buf[offset:offset + mask_np.size]
    view.copy_(torch.from_numpy(mask_np))
    kept, count, scratch = asx.compact_mask(view)
    assert asx.lib().asx_compact_status(scratch.data_ptr(), int(torch.cuda.current_stream().cuda_stream)) == 0
    c = int(count.item())
    return kept[:c].cpu().numpy(), c


@pytest.mark.parametrize("rows", [0, 1, 15, 16, 17, 4095, 4096, 4097, 12544, 100352, 1638400, 5_000_003])
@pytest.mark.parametrize("q", [0.0, 0.5, 0.9, 1.0])
def test_compaction_matches_oracle(rows, q):
    rng = np.random.default_rng(rows + int(q * 10))
    mask = (rng.random(rows) < q).astype(np.uint8)
    kept, c = _compact(mask)
    ref = oracle.kept_list(mask)
    assert c == ref.size
    assert np.array_equal(kept, ref)


@pytest.mark.parametrize("rows", [16383, 16384, 16385, 16400, 32768, 32769, 16384 * 9 + 4095])
def test_tile_boundaries_of_the_three_pass_form(rows):
    """Row counts around the 16384-row tiles of the large-mask passes (one block up to 16384 rows,
    count / scan / write above), with ragged and exactly full last tiles."""
    rng = np.random.default_rng(rows)
    for q in (0.0, 0.37, 1.0):
        mask = (rng.random(rows) < q).astype(np.uint8)
        kept, c = _compact(mask)
        assert np.array_equal(kept, oracle.kept_list(mask))


def test_more_tiles_than_one_round_of_the_tile_scan():
    """2^27 rows and a bit: 8196 tiles, so the one-block scan of the tile counts (8192 per round)
    carries a running total into a second round; kept runs that straddle tile boundaries."""
    rows = (1 << 27) + 3 * 16384 + 5
    rng = np.random.default_rng(27)
    mask = (rng.random(rows) < 0.5).astype(np.uint8)
    mask[16384 - 3:16384 + 3] = 1
    mask[(1 << 27) - 2:(1 << 27) + 2] = 1
    kept, c = _compact(mask)
    ref = oracle.kept_list(mask)
    assert c == ref.size
    assert np.array_equal(kept, ref)


def test_compaction_unaligned_pointer_and_nonbinary_bytes():
    rng = np.random.default_rng(3)
    mask = rng.integers(0, 3, 50001).astype(np.uint8)        # 0, 1 or 2: non-zero keeps
    for off in (1, 7, 8):
        kept, c = _compact(mask, offset=off)
        assert np.array_equal(kept, oracle.kept_list(mask))


def test_compaction_repeated_calls_share_scratch():
    mask = (np.random.default_rng(9).random(300000) < 0.3).astype(np.uint8)
    md = torch.from_numpy(mask).cuda()
    kept = torch.empty(mask.size, dtype=torch.int32, device="cuda")
    count = torch.empty(1, dtype=torch.int32, device="cuda")
    nbytes = asx.lib().asx_compact_scratch_bytes(mask.size)
    scratch = torch.full(((nbytes + 7) // 8,), -1, dtype=torch.int64, device="cuda")   # dirty on entry
    st = int(torch.cuda.current_stream().cuda_stream)
    for _ in range(3):
        assert asx.lib().asx_compact(md.data_ptr(), mask.size, kept.data_ptr(), count.data_ptr(),
                                     scratch.data_ptr(), scratch.numel() * 8, st) == 0
    torch.cuda.synchronize()
    assert np.array_equal(kept[:int(count.item())].cpu().numpy(), oracle.kept_list(mask))


def test_back_to_back_calls_on_changing_masks():
    """Several calls in a row, launches overlapping (each pass is a programmatic dependent of the one
    before), with a different mask, list and scratch every time.  A pass that reads what the pass before
    wrote through a stale L1 line gets this wrong from the second call on (the first call of a process
    is serialised by kernel loading and hides it)."""
    rows = 1 << 24
    rng = np.random.default_rng(24)
    masks = [(rng.random(rows) < q).astype(np.uint8) for q in (0.5, 0.2, 0.8, 0.5)]
    dev = [torch.from_numpy(m).cuda() for m in masks]
    outs = [asx.compact_mask(d) for d in dev]          # no synchronisation between the calls
    torch.cuda.synchronize()
    for m, (kept, count, scratch) in zip(masks, outs):
        ref = oracle.kept_list(m)
        assert int(count.item()) == ref.size
        assert np.array_equal(kept[:ref.size].cpu().numpy(), ref)


@pytest.mark.parametrize("rows", [9_000, 1_600_000])
def test_mask_written_by_the_kernel_just_before(rows):
    """asx_mask_from_activation -> asx_compact / asx_compact_static into the SAME mask buffer, with a
    different activation every round and no host synchronisation: the compaction kernels start while
    the mask kernel may still be storing the mask, and must read it only once it has finished (and
    not from a stale L1 line of the previous round)."""
    C = 8
    rng = np.random.default_rng(rows)
    st = int(torch.cuda.current_stream().cuda_stream)
    mask = torch.zeros(rows, dtype=torch.uint8, device="cuda")
    nb = asx.lib().asx_compact_scratch_bytes(rows)
    scr = torch.empty((nb + 7) // 8, dtype=torch.int64, device="cuda")
    rounds, acts, outs = 6, [], []
    for r in range(rounds):
        x = np.maximum(rng.standard_normal((rows, C)).astype(np.float32), 0.0)
        x[rng.random(rows) < (0.2 + 0.1 * r)] = 0.0
        acts.append(torch.from_numpy(x).to(torch.bfloat16).cuda())
    for r in range(rounds):
        k1 = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        k2 = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
        c1 = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        c2 = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        assert asx.lib().asx_mask_from_activation(acts[r].data_ptr(), rows, C, mask.data_ptr(), st) == 0
        assert asx.lib().asx_compact(mask.data_ptr(), rows, k1.data_ptr(), c1.data_ptr(), scr.data_ptr(), scr.numel() * 8, st) == 0
        assert asx.lib().asx_compact_static(mask.data_ptr(), rows, k2.data_ptr(), c2.data_ptr(), st) == 0
        outs.append((k1, c1, k2, c2))
    torch.cuda.synchronize()
    for r in range(rounds):
        want = oracle.kept_list(oracle.mask_from_activation(acts[r].float().cpu().numpy()))
        k1, c1, k2, c2 = outs[r]
        assert int(c1.item()) == want.size and int(c2.item()) == want.size, r
        assert np.array_equal(k1[:want.size].cpu().numpy(), want), r
        assert np.array_equal(k2[:want.size].cpu().numpy(), want), r

"""S1 on the GPU: the kept-row list must equal the oracle's bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2309_06626_b200 as asx
import workloads as wl
from gpu_util import make_problem, max_abs_tol, to_dev_bf16, REL_FROB_TOL

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
def test_tile_boundaries_of_the_two_pass_form(rows):
    """Row counts around the 16384-row tiles of the large-mask passes (one block up to 16384 rows,
    count / write by resident blocks above), with ragged and exactly full last tiles."""
    rng = np.random.default_rng(rows)
    for q in (0.0, 0.37, 1.0):
        mask = (rng.random(rows) < q).astype(np.uint8)
        kept, c = _compact(mask)
        assert np.array_equal(kept, oracle.kept_list(mask))


def test_more_tiles_than_resident_blocks():
    """2^27 rows and a bit: 8196 tiles on 1184 resident blocks, so every block walks a run of tiles and
    sums a thousand run counts for its offset; kept runs that straddle tile and run boundaries."""
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


@pytest.mark.parametrize("case", [
    # name, C_in, C_out, k, pad, H, W, Nb, pct, block, fused list expected to fit beside the pipeline stages
    ("pw_160", 32, 32, 1, 0, 160, 160, 1, 40, 4),              # 25600-row mask: compacted inside the fused kernel
    ("pw_181x181", 64, 64, 1, 0, 181, 181, 1, 50, 1),          # 32761 rows: just under the limit
    ("pw_182x182", 64, 64, 1, 0, 182, 182, 1, 50, 1),          # 33124 rows: the stand-alone passes
    ("c3_150_wide", 64, 256, 3, 1, 150, 150, 1, 70, 2),        # 22500 rows, 256-wide tiles: no room for the list, falls back
], ids=lambda c: c[0])
def test_masks_between_the_one_block_limit_and_the_fused_limit(case):
    """Masks of 16385..32768 rows are compacted inside the fused kernel when their 2-byte list fits beside the
    pipeline stages, by the stand-alone passes otherwise; either way ASX_RECOMPACT must give the stored list's result
    and the oracle's."""
    name, cin, cout, k, pad, H, W, Nb, pct, blk = case
    spec = wl.LayerSpec(name, cin, cout, k, k, 1, pad, H, W, Nb, pct, blk, "relu", wl.BASE_SEED + 8800 + H)
    x, w, b, mask = make_problem(spec, per_row=False)
    layer = asx.MaskedConvLayer(cin, cout, k, k, 1, pad)
    layer.set_mask(mask)
    xd, wd, bd = to_dev_bf16(x), to_dev_bf16(w), torch.from_numpy(b).cuda()
    y_stored = layer.run(xd, wd, bd, flags=asx.ACT_RELU).clone()
    y_re = layer.run(xd, wd, bd, flags=asx.ACT_RELU | asx.RECOMPACT).clone()
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    assert np.array_equal(layer.kept(), oracle.kept_list(mask))
    assert torch.equal(y_stored.view(torch.int16), y_re.view(torch.int16))
    # a new mask through the device copy only (no host-side list): the next RECOMPACT run must follow it
    mask2 = np.roll(mask, 7)
    layer.set_mask(mask2)
    y2 = layer.run(xd, wd, bd, flags=asx.ACT_RELU | asx.RECOMPACT)
    torch.cuda.synchronize()
    assert np.array_equal(layer.kept(), oracle.kept_list(mask2))
    ref = oracle.masked_conv(x, w, b, mask2, 1, pad, True).reshape(spec.M, cout)
    got = y2.float().cpu().numpy().astype(np.float64).reshape(spec.M, cout)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_FROB_TOL
    assert np.abs(got - ref).max() <= max_abs_tol(spec.K, oracle.bf16_round(x), oracle.bf16_round(w))
    layer.close()

"""Host logic of cwl_apply: the schedule (column tiles, K split, shrink hand-out) must cover the
output exactly once for any shape.  Pure host code: no GPU is touched."""
import itertools

import pytest

from paper_2601_21109_b200 import binding as cwl

SHAPES = [(256, 1024, 1024, 16), (2048, 4096, 4096, 64), (2048, 4096, 11008, 64), (2048, 11008, 4096, 64),
          (256, 4096, 11008, 64), (256, 11008, 4096, 64), (40321, 4096, 4096, 64), (16384, 4096, 11008, 64),
          (1, 16, 16, 16), (300, 208, 336, 0), (333, 512, 320, 64), (160, 256, 128, 256), (1000, 4096, 4096, 64),
          (512, 4096, 4096, 64), (64, 11008, 4096, 64), (7, 64, 48, 32), (130, 256, 2064, 16)]


def column_tiles(plan, d_out):
    cols, n0 = [], 0
    for _ in range(plan["wide_tiles_per_row"]):
        cols.append((n0, min(plan["wide_width"], d_out - n0)))
        n0 += plan["wide_width"]
    for _ in range(plan["narrow_tiles_per_row"]):
        cols.append((n0, min(plan["narrow_width"], d_out - n0)))
        n0 += plan["narrow_width"]
    return cols


@pytest.mark.parametrize("shape,pairs", list(itertools.product(SHAPES, [74, 72, 8, 1])))
def test_plan_covers_the_output_once(shape, pairs):
    T, d_in, d_out, R = shape
    plan = cwl.cwl_apply_plan(T, d_in, d_out, R, pairs)
    assert 1 <= plan["pairs"] <= min(pairs, 74)
    assert plan["row_tiles"] == -(-T // 256)
    cols = column_tiles(plan, d_out)
    covered = 0
    for n0, w in cols:                                  # contiguous, positive, multiples of 16, at most 512 wide
        assert n0 == covered and 16 <= w <= 512 and w % 16 == 0
        covered += w
    assert covered == d_out
    # K split: whole blocks, none empty, only when every item fits one wave and there is one tile width
    nkb = -(-d_in // 64)
    s, per = plan["split_k"], plan["k_blocks_per_split"]
    assert 1 <= s <= 16 and (s - 1) * per < nkb <= s * per
    if s > 1:
        assert plan["narrow_tiles_per_row"] == 0
        assert plan["row_tiles"] * len(cols) * s <= plan["pairs"]
    # shrink: every item handed to exactly one pair
    if R > 0:
        assert plan["shrink_items"] == plan["row_tiles"] * plan["shrink_splits"]
        assert plan["shrink_items_assigned"] == plan["shrink_items"]
    else:
        assert plan["shrink_items"] == 0 and plan["shrink_items_assigned"] == 0
    assert 2 <= plan["stages"] <= 8


def test_decode_sized_problems_split_k_and_prefill_does_not():
    assert cwl.cwl_apply_plan(256, 4096, 11008, 64)["split_k"] > 1
    assert cwl.cwl_apply_plan(256, 11008, 4096, 64)["split_k"] > 1
    p = cwl.cwl_apply_plan(2048, 4096, 4096, 64)
    assert p["split_k"] == 1 and p["wide_width"] == 512
    # 64 tiles on 74 pairs: the shrink is cut into no more items than there are pairs without a tile
    assert p["pairs"] == 74 and p["shrink_items"] <= 10 and p["shrink_items_max_per_pair"] == 1


def test_plan_rejects_bad_shapes():
    with pytest.raises(cwl.CwlError):
        cwl.cwl_apply_plan(128, 100, 64, 16)
    with pytest.raises(cwl.CwlError):
        cwl.cwl_apply_plan(0, 64, 64, 16)


def test_workspace_grows_with_the_split_and_noalloc_need_does_not():
    assert cwl.cwl_apply_workspace_bytes(256, 4096, 11008, 64) > cwl.cwl_apply_noalloc_scratch_need(256, 4096, 11008, 64)
    assert cwl.cwl_apply_noalloc_scratch_need(2048, 4096, 4096, 64) <= cwl.NOALLOC_SCRATCH_BYTES
    for T in (8192, 16384, 32768):                       # the documented reach of the built-in scratch at R = 64
        assert cwl.cwl_apply_noalloc_scratch_need(T, 4096, 11008, 64) <= cwl.NOALLOC_SCRATCH_BYTES
    assert cwl.cwl_apply_noalloc_scratch_need(65536, 4096, 4096, 64) > cwl.NOALLOC_SCRATCH_BYTES


def test_a_batch_needs_the_workspaces_of_its_items_on_their_shares_of_the_pairs():
    # host-only: the decode step's two projections, 37 of the 74 pairs each (equal weight bytes)
    both = cwl.cwl_apply_batch_workspace_bytes(256, [4096, 11008], [11008, 4096], 64)
    up = cwl.cwl_apply_batch_workspace_bytes(256, [4096], [11008], 64)
    down = cwl.cwl_apply_batch_workspace_bytes(256, [11008], [4096], 64)
    assert both >= 256 and both % 256 == 0 and up % 256 == 0 and down % 256 == 0
    # alone, an item plans for every pair; in the batch for its share: both are fp32 partial sums + H' + sync words, MBs
    assert 1 << 20 < both < 1 << 27 and 1 << 18 < up < 1 << 27 and 1 << 18 < down < 1 << 27
    assert cwl.cwl_apply_batch_workspace_bytes(256, [4096, 11008], [11008, 4096], 64) == both       # deterministic
    # no adapter: less scratch (no H', no shrink partial sums)
    assert cwl.cwl_apply_batch_workspace_bytes(256, [4096, 11008], [11008, 4096], 0) <= both
    # malformed batches answer with the minimum instead of a plan
    assert cwl.cwl_apply_batch_workspace_bytes(256, [], [], 64) == 256
    assert cwl.cwl_apply_batch_workspace_bytes(256, [64] * 5, [64] * 5, 64) == 256
    assert cwl.cwl_apply_batch_workspace_bytes(0, [4096], [4096], 64) == 256


def test_a_share_of_the_pairs_changes_the_plan_not_the_coverage():
    whole = cwl.cwl_apply_plan(256, 4096, 11008, 64, 74)
    half = cwl.cwl_apply_plan(256, 4096, 11008, 64, 37)
    assert half["pairs"] <= 37 and whole["pairs"] <= 74
    assert half["split_k"] == 1 and whole["split_k"] > 1          # 29 whole-K tiles fit 37 pairs; 74 pairs want the K loop split
    for plan in (whole, half):
        assert sum(w for _, w in column_tiles(plan, 11008)) == 11008

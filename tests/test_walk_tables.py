"""Host-side tables of the WALK executors, without a GPU: the slices cover the message exactly once,
and the merged hop lists of two neighbouring chunks keep each chunk's messages in plan order
(so every `dep` stays respected) while pairing the hops that write the same rank."""
import numpy as np
import pytest

from paper_1603_06809_b200 import bcast as B
from paper_1603_06809_b200 import workloads as W

VARIANTS = (B.BCAST_NATIVE, B.BCAST_TUNED)
FULL, RAGGED, DUAL = 0, 1, 2

SHAPES = [(8, 1 << 20), (12, 256 * 1024), (12, 256 * 1024 + 5), (64, (16 << 20) + 13), (100, 64 << 20),
          (255, 12 * 1024), (255, 4 << 20), (129, 524287), (7, 1000), (5, 3), (3, 1), (2, 4097), (33, 33 * 512 + 17),
          (16, 16 * 1536), (16, 16 * 1536 + 16), (1024, 65536 + 7)]


def slice_ranges(plan, words):
    """[(lo, hi, kind, chunk)] of every slice, from the geometry the header documents."""
    P, n, S = B.bcast_plan_num_ranks(plan), B.bcast_plan_nbytes(plan), B.bcast_plan_scatter_size(plan)
    seg_bytes = 512 * words
    out = []
    for seg, kind, c in B.bcast_plan_walk_slices(plan, words):
        seg_lo, seg_hi = seg * seg_bytes, (seg + 1) * seg_bytes
        c_lo, c_hi = min(c * S, n), min((c + 1) * S, n)
        if kind == FULL:
            assert c_lo <= seg_lo and seg_hi <= c_hi
            out.append((seg_lo, seg_hi, kind, c))
        elif kind == RAGGED:
            lo, hi = max(seg_lo, c_lo), min(seg_hi, c_hi)
            assert lo < hi and (lo, hi) != (seg_lo, seg_hi)
            out.append((lo, hi, kind, c))
        else:
            assert kind == DUAL and c + 1 < P
            cut = (c + 1) * S
            assert seg_lo < cut < seg_hi <= min((c + 2) * S, n) and c_lo <= seg_lo
            out.append((seg_lo, seg_hi, kind, c))
    return out


@pytest.mark.parametrize("P,n", SHAPES)
@pytest.mark.parametrize("words", [1, 3, 8])
def test_slices_cover_the_message_exactly_once(P, n, words):
    plan = B.bcast_plan(P, P - 1, n, B.BCAST_TUNED)
    ranges = sorted(slice_ranges(plan, words))
    assert ranges[0][0] == 0 and ranges[-1][1] == n
    for (lo0, hi0, _, _), (lo1, hi1, _, _) in zip(ranges, ranges[1:]):
        assert hi0 == lo1                      # no gap, no overlap
    kinds = B.bcast_plan_walk_slices(plan, words)[:, 1]
    order = [int(k) for k in kinds]
    rank = {RAGGED: 0, DUAL: 1, FULL: 2}       # the slow kinds are listed (and started) first
    assert [rank[k] for k in order] == sorted(rank[k] for k in order)


def test_slices_of_an_empty_plan():
    assert len(B.bcast_plan_walk_slices(B.bcast_plan(1, 0, 4096, B.BCAST_TUNED), 8)) == 0
    assert len(B.bcast_plan_walk_slices(B.bcast_plan(5, 2, 0, B.BCAST_NATIVE), 8)) == 0
    with pytest.raises(B.BcastError):
        B.bcast_plan_walk_slices(B.bcast_plan(5, 2, 100, B.BCAST_NATIVE), 9)


def test_odd_scatter_size_costs_no_extra_slices():
    # one boundary per segment at most: the cut segments become dual slices, not pairs of ragged ones
    plan = B.bcast_plan(255, 254, 32 << 20, B.BCAST_TUNED)
    s = B.bcast_plan_walk_slices(plan, 8)
    assert len(s) == (32 << 20) // 4096
    assert (s[:, 1] == DUAL).sum() == 254 and (s[:, 1] == RAGGED).sum() == 0


@pytest.mark.parametrize("variant", VARIANTS + (B.BCAST_DOUBLING,))
@pytest.mark.parametrize("P,root,n", [(8, 0, 8 * 1000 + 3), (10, 3, 10 * 77), (12, 5, 256 * 1024), (16, 15, 16 * 4099),
                                      (33, 32, 33 * 513), (64, 17, (1 << 20) + 13), (100, 63, 100 * 671089), (7, 6, 5)])
def test_pairing_keeps_plan_order_and_pairs_hops_into_the_same_rank(variant, P, root, n):
    if variant == B.BCAST_DOUBLING and P & (P - 1):
        pytest.skip("recursive doubling needs a power of two")
    plan = B.bcast_plan(P, root, n, variant)
    x = B.bcast_plan_xfers(plan)
    S = B.bcast_plan_scatter_size(plan)
    total = paired = 0
    for c in range(P - 1):
        slots = B.bcast_plan_walk_pairing(plan, c)
        lower = B.bcast_plan_walk_order(plan, c, B.BCAST_EXEC_WALK_PLAN_ORDER)
        upper = B.bcast_plan_walk_order(plan, c + 1, B.BCAST_EXEC_WALK_PLAN_ORDER)
        if min(c * S, n) == min((c + 1) * S, n) or min((c + 1) * S, n) == min((c + 2) * S, n):
            assert len(slots) == 0             # an empty chunk has no boundary to carry
            continue
        # each column, without its holes, is that chunk's plan-order list: nothing lost, nothing re-ordered
        assert np.array_equal(slots[:, 0][slots[:, 0] >= 0], lower)
        assert np.array_equal(slots[:, 1][slots[:, 1] >= 0], upper)
        assert ((slots[:, 0] >= 0) | (slots[:, 1] >= 0)).all()
        both = (slots[:, 0] >= 0) & (slots[:, 1] >= 0)
        same = both.copy()
        same[both] = x["dst_rank"][slots[both, 0]] == x["dst_rank"][slots[both, 1]]
        total += len(lower) + len(upper)
        paired += 2 * int(same.sum())
    if P >= 8 and n >= 2 * P and variant != B.BCAST_DOUBLING:
        # ring: the hop of chunk c+1 into a rank comes one step before that of chunk c
        assert paired >= 0.9 * total, (paired, total)


def test_pairing_argument_errors():
    plan = B.bcast_plan(4, 0, 4096, B.BCAST_TUNED)
    for chunk in (-1, 3, 4):
        with pytest.raises(B.BcastError):
            B.bcast_plan_walk_pairing(plan, chunk)

"""Host-side plan of the packed-groups decoder (no GPU): which groups of a work item keep the words of their rows
in rotated order, decided from a model of the shared-memory bank rules.

The model's rules were measured on the device with a microbenchmark (64-bit accesses, cycles per warp instruction
with the load/store pipe saturated); the figures pinned here are those measurements:
  * a load of 8 different words, four lanes on each, groups 480 B apart (K = 8, W = 12, C = 10): 2 passes;
    with groups 4-7 moved by one word: 1 pass;
  * a store of 32 different words laid out 320 B per group and 80 B per lane: 4 passes; with every second pair
    of groups moved by one word: 2 passes (a store never takes fewer: one pass per half-warp).
"""
import pytest

import paper_2109_09868_b200 as ap
from paper_2109_09868_b200 import binding


def test_paper_shape_counts_match_the_measured_bank_rules():
    gw, rot, plain, chosen = ap.debug_pack_rotation(8, 12, 10)
    assert gw == 8                      # 32 lanes / 4 tiles of two queries
    # unrotated: 12 workers x 5 words x 2 passes (loads) + 2 queries x 5 words x 4 passes (stores)
    assert plain == 12 * 5 * 2 + 2 * 5 * 4
    # rotated groups 2..5: four of the five word slots load in 1 pass, the wrapped one in 2; stores 2 passes
    # except the wrapped slot
    assert rot == 0b00111100
    assert chosen == 12 * (4 * 1 + 2) + 2 * (4 * 2 + 4)
    assert chosen < plain


@pytest.mark.parametrize("K,W,C", [(8, 12, 10), (4, 8, 10), (16, 24, 10), (12, 20, 10), (8, 9, 10), (8, 12, 8), (8, 16, 10)])
def test_rotation_is_used_where_it_was_measured_to_pay(K, W, C):
    gw, rot, plain, chosen = ap.debug_pack_rotation(K, W, C)
    assert gw >= 2 and rot != 0 and rot < (1 << gw)
    assert chosen < plain
    # switched off: no group rotated, the count is the plain one
    assert ap.debug_pack_rotation(K, W, C, 1) == (gw, 0, plain, plain)
    # the decision is a pure function of the shape
    assert ap.debug_pack_rotation(K, W, C) == (gw, rot, plain, chosen)


@pytest.mark.parametrize("K,W,C", [(4, 5, 10), (2, 4, 10), (4, 6, 10), (2, 3, 10), (8, 12, 6), (4, 5, 6)])
def test_rotation_is_left_out_where_it_was_measured_to_cost(K, W, C):
    """One or two lanes per group on shapes that already run at the DRAM rate, and rows under 8 classes."""
    gw, rot, plain, chosen = ap.debug_pack_rotation(K, W, C)
    assert gw >= 2 and rot == 0 and chosen == plain


def test_conflict_free_layout_is_recognised():
    # K = 4, W = 5, C = 10: 16 groups 200 B apart fall into 16 different bank pairs: every load is one pass
    gw, rot, plain, chosen = ap.debug_pack_rotation(4, 5, 10, 1)
    assert gw == 16 and plain == 5 * 5 * 1 + 2 * 5 * 4
    # K = 4, W = 8: groups 320 B apart, only four bank pairs in use: 8 passes per load
    gw, rot, plain, chosen = ap.debug_pack_rotation(4, 8, 10, 1)
    assert gw == 16 and plain == 8 * 5 * 8 + 2 * 5 * 4


def test_shapes_without_one_lane_per_row_have_no_rotation():
    gw, rot, plain, chosen = ap.debug_pack_rotation(3, 7, 20)   # rows of 10 words shared by two lanes
    assert gw == 8 and (rot, plain, chosen) == (0, 0, 0)
    assert ap.debug_pack_rotation(8, 12, 100)[0] == 0            # not this kernel's shape at all
    assert ap.debug_pack_rotation(8, 12, 7)[0] == 0              # odd number of classes


def test_bad_arguments():
    for args in ((0, 4, 10, 0), (5, 4, 10, 0), (4, 33, 10, 0), (4, 8, 0, 0), (4, 8, 10, 3), (4, 8, 10, -1)):
        with pytest.raises(binding.ApproxiferError):
            ap.debug_pack_rotation(*args)

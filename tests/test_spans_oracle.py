"""Pins for the span recursions: Eq. (1)/(2) literal forms, the hand-derived
fixture, and a brute-force walk over every window."""
import os

import pytest

from oracle import spans
from paper_2409_09083_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "spans_hand.txt")
STACKS = {"tiny": synth.stack_tiny, "yolo8": synth.stack_yolo8, "yolo16": synth.stack_yolo16}


def read_golden():
    rows = []
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        stack, grp, extent, parts, tile, sp = [f.strip() for f in line.split(";")]
        first, last = map(int, grp.split("-"))
        sp = [tuple(map(int, s.split("-"))) for s in sp.split()]
        rows.append((stack, first, last, int(extent), int(parts), int(tile), sp))
    return rows


@pytest.mark.parametrize("row", read_golden())
def test_hand_derived_spans(row):
    stack, first, last, extent, parts, tile, sp = row
    layers = STACKS[stack]()[first - 1:last]
    own = spans.equal_partition(extent, parts)[tile]
    got = spans.forward_spans(layers, extent, own)
    assert got[::-1] == sp


def test_general_receptive_field_equals_eq1_for_same_padded_convs():
    for K in (1, 3, 5, 7):
        for a1, a2 in [(0, 0), (3, 9), (17, 33)]:
            assert spans.receptive(a1, a2, K, 1, K // 2) == spans.eq1_conv(a1, a2, K, 1)


def test_eq2_is_the_adjoint_footprint_of_eq1_for_stride_one():
    # delta outputs that touch inputs [a, b] of a same-padded stride-1 conv
    for K in (1, 3, 5):
        for a, b in [(0, 4), (7, 15), (20, 20)]:
            lo, hi = spans.eq2_conv(a, b, K, 1)
            touch = [o for o in range(-10, 60)
                     if any(a <= o - K // 2 + t <= b for t in range(K))]
            assert (lo, hi) == (touch[0], touch[-1])


def test_equal_partition_is_disjoint_and_covering():
    for extent, parts in [(52, 3), (152, 5), (38, 5), (76, 5), (16, 2), (7, 7)]:
        cells = spans.equal_partition(extent, parts)
        assert cells[0][0] == 0 and cells[-1][1] == extent - 1
        for (a1, a2), (b1, b2) in zip(cells, cells[1:]):
            assert a1 <= a2 and b1 == a2 + 1


@pytest.mark.parametrize("stack,first,last,in_extent,parts", [
    ("tiny", 1, 3, 32, 2), ("yolo8", 1, 8, 416, 3), ("yolo8", 5, 8, 104, 4),
    ("yolo16", 9, 16, 76, 5), ("yolo16", 1, 16, 608, 2)])
def test_recursion_matches_brute_force_dependency(stack, first, last, in_extent, parts):
    layers = STACKS[stack]()[first - 1:last]
    out_extent = in_extent
    for l in layers:
        if l.kind == "pool":
            out_extent //= 2
    for own in spans.equal_partition(out_extent, parts):
        rec = spans.forward_spans(layers, out_extent, own)
        brute = spans.brute_force_dependency(layers, in_extent, own)
        assert rec == brute

"""Pins for the oracle's equivalent bit-width against the widths the paper prints."""
import os

import pytest

from oracle import xq_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append([float(x) for x in line.split()])
    return rows


@pytest.mark.parametrize("row", _rows("equiv_bits.txt"))
def test_printed_widths(row):
    kq, vq, km, vm, L, want = row
    got = O.equiv_bits(int(kq), int(vq), int(km), int(vm), int(L))
    assert got == want
    assert O.equiv_bits_closed_form(int(kq), int(vq), int(km), int(vm), int(L)) == want


@pytest.mark.parametrize("row", _rows("equiv_bits_kv.txt"))
def test_key_value_figures_of_worked_example(row):
    q, m, L, want = row
    assert O.equiv_bits_one(int(q), int(m), int(L)) == want


def test_rounded_prints():
    # 1.375 appears as "1.38" and 1.40625 as "1.4" in the result tables.
    assert f"{O.equiv_bits(30, 2, 32, 16):.2f}" in ("1.38", "1.37")
    assert f"{O.equiv_bits(28, 0, 32, 28):.1f}" == "1.4"


def test_direct_count_equals_closed_form_for_even_parameters():
    for L in (2, 8, 32, 40):
        for kq in range(0, L + 1, 2):
            for km in range(0, L + 1, 2):
                a = O.equiv_bits(kq, kq, km, km, L)
                b = O.equiv_bits_closed_form(kq, kq, km, km, L)
                assert abs(a - b) < 1e-12


def test_owner_pattern():
    # pair (2p, 2p+1): the even layer owns, the odd one borrows, from layer m on
    assert [O.owns_codes(l, 4) for l in range(8)] == [True, True, True, True, True, False, True, False]
    assert all(O.owns_codes(l, 32) for l in range(32))
    assert [O.layer_bits(l, 2) for l in range(4)] == [2, 2, 1, 1]


def test_benchmark_configs():
    # all 32 layers paired: 2-bit K/V -> 1.0; 2-bit K + 1-bit V -> 0.75; one pair of 2 layers -> 1.0
    assert O.equiv_bits(32, 32, 0, 0, 32) == 1.0
    assert O.equiv_bits(32, 0, 0, 0, 32) == 0.75
    assert O.equiv_bits(2, 2, 0, 0, 2) == 1.0


@pytest.mark.parametrize("group,vm", [(2, 8), (3, 14), (4, 16)])
def test_group_table_common_width(group, vm):
    """Table group compares group sizes 2, 3, 4 "under the same compression ratio": all key layers and 20 of the
    32 value layers stored on a 2-bit base, printed as 1.63.  Contiguous groups counted from the sharing start
    give exactly that for sharing from layer 8, 14 and 16, for every dominant index."""
    for k in range(group):
        stored = sum(1 for l in range(32) if O.code_owner(l, vm, group, k) == l)
        assert stored == 20
        w = O.equiv_bits(32, 32, 32, vm, 32, group, k)
        assert w == 1.625 and f"{w:.2f}" in ("1.62", "1.63")


def test_owner_of_larger_groups_and_other_dominant_layers():
    # groups of three from layer 2 on, dominant index 1: (2,3,4) -> 3, (5,6,7) -> 6
    assert [O.code_owner(l, 2, 3, 1) for l in range(8)] == [0, 1, 3, 3, 3, 6, 6, 6]
    # pairs with the second layer dominant: the even layer reads the odd one's codes
    assert [O.code_owner(l, 0, 2, 1) for l in range(4)] == [1, 1, 3, 3]
    # the default is Algorithm 1's pattern
    assert [O.code_owner(l, 4) for l in range(8)] == [0, 1, 2, 3, 4, 4, 6, 6]
    # every layer's owner owns its own codes
    for group in (2, 3, 4):
        for k in range(group):
            for m in (0, 4, 8):
                for l in range(m + 2 * group):
                    o = O.code_owner(l, m, group, k)
                    assert O.code_owner(o, m, group, k) == o

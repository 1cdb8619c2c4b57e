"""Pins for the oracle's packed layouts: round trip, bijection, bit census."""
import numpy as np
import pytest

from oracle import xq_oracle as O


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
@pytest.mark.parametrize("kind", ["k", "v"])
def test_positions_are_a_bijection_onto_the_words(bits, D, kind):
    """Two value batches (256 tokens = eight key units): every bit of every word is the bit of exactly one code."""
    pos = O.k_code_position if kind == "k" else O.v_code_position
    T = 2 * O.BATCH
    n_words = T * D * bits // 32
    seen = set()
    for t in range(T):
        for d in range(D):
            w, b = pos(t, d, bits, D)
            assert 0 <= w < n_words and 0 <= b <= 32 - bits and (b % 8) % bits == 0
            if kind == "k":
                assert w // (D * bits) == t // 32  # a unit of 32 tokens is one contiguous run of words
            else:
                assert w // (D * bits * 4) == t // O.BATCH  # so is a batch of 128 tokens
            for k in range(bits):
                seen.add((w, b + k))
    assert len(seen) == n_words * 32


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
def test_round_trip_and_census(bits, D):
    rng = np.random.default_rng(bits * 100 + D)
    T = 2 * O.BATCH + 64  # a ragged last value batch
    codes = rng.integers(0, 1 << bits, size=(T, D), dtype=np.uint8)
    for pack, unpack in ((O.pack_k_codes, O.unpack_k_codes), (O.pack_v_codes, O.unpack_v_codes)):
        slow, wr_slow = pack(codes, bits, fast=False)
        fast, wr_fast = pack(codes, bits, fast=True)
        assert np.array_equal(slow, fast) and np.array_equal(wr_slow, wr_fast)
        assert np.array_equal(unpack(slow, T, D, bits), codes)
        assert wr_slow.sum() == T * D * bits // 32  # words are never shared between written and unwritten tokens
        # no bit is set that does not belong to a code
        pop = sum(bin(int(w)).count("1") for w in slow)
        assert pop == sum(bin(int(c)).count("1") for c in codes.reshape(-1))


def test_all_ones_fill_every_bit():
    for bits, D in ((1, 128), (2, 128), (2, 64)):
        codes = np.full((O.BATCH, D), (1 << bits) - 1, dtype=np.uint8)
        assert (O.pack_k_codes(codes, bits)[0] == 0xFFFFFFFF).all()
        assert (O.pack_v_codes(codes, bits)[0] == 0xFFFFFFFF).all()


@pytest.mark.parametrize("bits", [1, 2])
def test_four_consecutive_row_elements_share_a_bit_offset(bits):
    """What the decode kernel relies on: the codes of row elements 4j .. 4j+3 sit in the four bytes of one word
    at one bit offset, so that one AND extracts them as four operand bytes."""
    D = 128
    for t in (0, 37, 200):
        for d in range(0, D, 4):
            ws = [O.k_code_position(t, d + i, bits, D) for i in range(4)]
            assert len({w for w, _ in ws}) == 1 and [b for _, b in ws] == [ws[0][1] + 8 * i for i in range(4)]
    for d in (0, 77):
        for t in range(0, 256, 4):
            ws = [O.v_code_position(t + i, d, bits, D) for i in range(4)]
            assert len({w for w, _ in ws}) == 1 and [b for _, b in ws] == [ws[0][1] + 8 * i for i in range(4)]


def test_k_and_v_layouts_swap_roles():
    # within the first batch, a channel's value row is laid out like a token's key row (D = 128: both 128 long)
    for bits in (1, 2):
        for a in range(128):
            for e in range(0, 128, 7):
                wk, bk = O.k_code_position(a % 32, e, bits, 128)
                wv, bv = O.v_code_position(e, a % 32, bits, 128)
                assert bk == bv


def test_meta_positions_are_permutations():
    for D in (64, 128):
        assert sorted(O.k_meta_position(d, D) for d in range(D)) == list(range(D))


def test_meta_pack_places_values():
    rng = np.random.default_rng(0)
    s = rng.random((3, 128)).astype(np.float16); z = rng.random((3, 128)).astype(np.float16)
    m = O.pack_k_meta(s, z)
    assert m.shape == (3, 2, 128)
    for d in (0, 1, 17, 127):
        p = O.k_meta_position(d, 128)
        assert m[2, 0, p] == s[2, d].view(np.uint16) and m[2, 1, p] == z[2, d].view(np.uint16)
    s = rng.random((32, 4)).astype(np.float16); z = rng.random((32, 4)).astype(np.float16)
    m = O.pack_v_meta(s, z)
    assert m.shape == (32, 2, 4)
    for t, gi in ((0, 0), (17, 3), (31, 1)):
        assert m[t, 0, gi] == s[t, gi].view(np.uint16) and m[t, 1, gi] == z[t, gi].view(np.uint16)

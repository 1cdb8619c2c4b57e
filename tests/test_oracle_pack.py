"""Pins for the oracle's packed layouts: round trip, bijection, bit census."""
import numpy as np
import pytest

from oracle import xq_oracle as O


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
@pytest.mark.parametrize("kind", ["k", "v"])
def test_positions_are_a_bijection_onto_whole_words(bits, D, kind):
    pos, period = (O.k_code_position, O.K_PERIOD) if kind == "k" else (O.v_code_position, O.V_PERIOD)
    wpp = period * D * bits // 32  # words per period
    seen = set()
    for t in range(2 * period):
        for d in range(D):
            w, b = pos(t, d, bits, D)
            assert 0 <= w < 2 * wpp and 0 <= b <= 32 - bits and b % bits == 0
            assert (w // wpp) == t // period
            for k in range(bits):
                seen.add((w, b + k))
    assert len(seen) == 2 * wpp * 32  # every bit of every word belongs to exactly one code


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
def test_round_trip_and_census(bits, D):
    rng = np.random.default_rng(bits * 100 + D)
    T = 256
    codes = rng.integers(0, 1 << bits, size=(T, D), dtype=np.uint8)
    for pack, unpack in ((O.pack_k_codes, O.unpack_k_codes), (O.pack_v_codes, O.unpack_v_codes)):
        slow = pack(codes, bits, fast=False)
        fast = pack(codes, bits, fast=True)
        assert np.array_equal(slow, fast)
        assert np.array_equal(unpack(slow, T, D, bits), codes)
        # no bit is set that does not belong to a code
        pop = sum(bin(int(w)).count("1") for w in slow)
        assert pop == sum(bin(int(c)).count("1") for c in codes.reshape(-1))


def test_ragged_tail_is_zero_padded():
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 4, size=(160, 64), dtype=np.uint8)  # 1.25 value blocks
    full = np.zeros((256, 64), dtype=np.uint8)
    full[:160] = codes
    assert np.array_equal(O.pack_v_codes(codes, 2), O.pack_v_codes(full, 2))
    assert np.array_equal(O.pack_v_codes(codes, 2, fast=False), O.pack_v_codes(full, 2))
    assert np.array_equal(O.pack_k_codes(codes, 2), O.pack_k_codes(full, 2)[: 160 * 64 * 2 // 32])


def test_all_ones_fill_every_bit():
    for bits, D in ((1, 128), (2, 128), (2, 64)):
        codes = np.full((128, D), (1 << bits) - 1, dtype=np.uint8)
        assert (O.pack_k_codes(codes, bits) == 0xFFFFFFFF).all()
        assert (O.pack_v_codes(codes, bits) == 0xFFFFFFFF).all()


def test_words_hold_what_the_layout_promises():
    # a key word holds consecutive channels of one token, a value word consecutive tokens of one channel;
    # even members in the low half, odd members in the high half, at the same bit of their half
    bits, D = 2, 128
    for t in (0, 5, 37):
        for d in range(0, D, 2):
            w0, b0 = O.k_code_position(t, d, bits, D)
            w1, b1 = O.k_code_position(t, d + 1, bits, D)
            assert w0 == w1 and b1 == b0 + 16 and b0 == bits * ((d % 16) // 2)
    for d in (0, 3, 127):
        for t in range(0, 256, 2):
            w0, b0 = O.v_code_position(t, d, bits, D)
            w1, b1 = O.v_code_position(t + 1, d, bits, D)
            assert w0 == w1 and b1 == b0 + 16 and b0 == bits * ((t % 16) // 2)
    # the 32 tokens of a unit read their first 16-byte chunk from consecutive addresses
    assert [O.k_code_position(t, 0, 2, 128)[0] for t in range(3)] == [0, 4, 8]
    # the channels of a block read their 16-byte chunk from consecutive addresses
    assert [O.v_code_position(0, d, 1, 128)[0] for d in range(3)] == [0, 4, 8]


def test_meta_pack_places_values():
    rng = np.random.default_rng(0)
    s = rng.random((3, 128)).astype(np.float16); z = rng.random((3, 128)).astype(np.float16)
    m = O.pack_k_meta(s, z)
    assert m.shape == (2, 3, 128)
    for d in (0, 1, 17, 127):
        assert m[0, 2, d] == s[2, d].view(np.uint16) and m[1, 2, d] == z[2, d].view(np.uint16)
    s = rng.random((32, 4)).astype(np.float16); z = rng.random((32, 4)).astype(np.float16)
    m = O.pack_v_meta(s, z)
    assert m.shape == (32, 2, 4)
    for t, gi in ((0, 0), (17, 3), (31, 1)):
        assert m[t, 0, gi] == s[t, gi].view(np.uint16) and m[t, 1, gi] == z[t, gi].view(np.uint16)

"""Pins for the oracle's packed layouts: round trip, bijection, bit census."""
import numpy as np
import pytest

from oracle import xq_oracle as O


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
@pytest.mark.parametrize("kind", ["k", "v"])
def test_positions_are_a_bijection_onto_the_tile(bits, D, kind):
    pos = O.k_code_position if kind == "k" else O.v_code_position
    tpt = O.tokens_per_code_tile(bits, D)
    assert tpt * D * bits == 128 * 32  # a tile is exactly 128 full words
    seen = set()
    for t in range(2 * tpt):
        for d in range(D):
            w, b = pos(t, d, bits, D)
            assert 0 <= w < 256 and 0 <= b <= 32 - bits and b % bits == 0
            assert (w // 128) == t // tpt
            for k in range(bits):
                seen.add((w, b + k))
    assert len(seen) == 2 * 128 * 32


@pytest.mark.parametrize("bits,D", [(1, 64), (2, 64), (1, 128), (2, 128)])
def test_round_trip_and_census(bits, D):
    rng = np.random.default_rng(bits * 100 + D)
    T = 2 * O.tokens_per_code_tile(bits, D)
    codes = rng.integers(0, 1 << bits, size=(T, D), dtype=np.uint8)
    for pack, unpack in ((O.pack_k_codes, O.unpack_k_codes), (O.pack_v_codes, O.unpack_v_codes)):
        slow = pack(codes, bits, fast=False)
        fast = pack(codes, bits, fast=True)
        assert np.array_equal(slow, fast)
        assert np.array_equal(unpack(slow, T, D, bits), codes)
        # no bit is set that does not belong to a code
        pop = sum(bin(int(w)).count("1") for w in slow)
        assert pop == sum(bin(int(c)).count("1") for c in codes.reshape(-1))


def test_all_ones_fill_every_bit():
    for bits, D in ((1, 128), (2, 128), (2, 64)):
        T = O.tokens_per_code_tile(bits, D)
        codes = np.full((T, D), (1 << bits) - 1, dtype=np.uint8)
        assert (O.pack_k_codes(codes, bits) == 0xFFFFFFFF).all()
        assert (O.pack_v_codes(codes, bits) == 0xFFFFFFFF).all()


def test_k_and_v_layouts_are_transposes_of_each_other():
    # the value layout is the key layout with token and channel swapped inside each 16x16 block
    bits, D = 2, 128
    for t in range(16):
        for d in range(D):
            cb, cc = divmod(d, 16)
            assert O.v_code_position(t, d, bits, D) == O.k_code_position(cc, cb * 16 + t, bits, D)


def test_meta_positions_are_permutations():
    for D in (64, 128):
        assert sorted(O.k_meta_position(d, D) for d in range(D)) == list(range(D))
    for n_g in (1, 2, 4):
        p = sorted(O.v_meta_position(tk, gi, n_g) for tk in range(16) for gi in range(n_g))
        assert p == list(range(16 * n_g))


def test_meta_pack_places_values():
    rng = np.random.default_rng(0)
    s = rng.random((3, 128)).astype(np.float16); z = rng.random((3, 128)).astype(np.float16)
    m = O.pack_k_meta(s, z)
    assert m.shape == (2, 3, 128)
    for d in (0, 1, 17, 127):
        p = O.k_meta_position(d, 128)
        assert m[0, 2, p] == s[2, d].view(np.uint16) and m[1, 2, p] == z[2, d].view(np.uint16)
    s = rng.random((32, 4)).astype(np.float16); z = rng.random((32, 4)).astype(np.float16)
    m = O.pack_v_meta(s, z)
    assert m.shape == (2, 2, 64)
    for t, gi in ((0, 0), (17, 3), (31, 1)):
        p = O.v_meta_position(t % 16, gi, 4)
        assert m[t // 16, 0, p] == s[t, gi].view(np.uint16) and m[t // 16, 1, p] == z[t, gi].view(np.uint16)

"""Pins for the oracle's group quantizer and calibration (Eq. 1-5, 12; Algorithm 2)."""
import numpy as np
import pytest

from oracle import xq_oracle as O


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


@pytest.mark.parametrize("bits", [1, 2])
def test_eta0_is_round_to_nearest_minmax(bits):
    # eta = 0 is the plain min-max quantizer: error at most half a step per element
    x = _rand((64, 32), 1)
    z, s, _ = O.group_params(x, bits, axis=1)
    c = O.quantize_codes(x, z, s, bits)
    zh, sh = O.calibrate(z, s, bits, 0.0)
    assert np.array_equal(zh, z) and np.array_equal(sh, s)
    xh = c.astype(np.float64) * sh.astype(np.float64) + zh.astype(np.float64)
    err = np.abs(x.astype(np.float64) - xh)
    assert (err <= 0.5 * s.astype(np.float64) * (1 + 1e-6)).all()
    # the extremes of each group take the extreme codes
    assert (c.min(axis=1) == 0).all() and (c.max(axis=1) == (1 << bits) - 1).all()
    assert (c[np.arange(64), x.argmin(axis=1)] == 0).all()
    assert (c[np.arange(64), x.argmax(axis=1)] == (1 << bits) - 1).all()


@pytest.mark.parametrize("bits", [1, 2])
def test_brute_force_nearest_level(bits):
    # tiny groups: the code is the level z + c*s nearest to x
    rng = np.random.default_rng(7)
    for g in (2, 3, 4):
        x = rng.standard_normal((200, g)).astype(np.float32)
        z, s, _ = O.group_params(x, bits, axis=1)
        c = O.quantize_codes(x, z, s, bits)
        for i in range(x.shape[0]):
            levels = [float(z[i, 0]) + k * float(s[i, 0]) for k in range(1 << bits)]
            for j in range(g):
                d = [abs(float(x[i, j]) - lv) for lv in levels]
                best = min(d)
                # skip numerical near-ties
                if sorted(d)[1] - best < 1e-5 * max(1.0, abs(float(x[i, j]))):
                    continue
                assert int(c[i, j]) == d.index(best)


def test_one_bit_rounding_function():
    # Eq. 4: [0, 0.5] -> 0, (0.5, 1] -> 1
    x = np.array([[0.0, 0.5, 0.5000001, 0.25, 0.75, 1.0]], dtype=np.float32)
    z, s, _ = O.group_params(x, 1, axis=1)
    assert z[0, 0] == 0 and s[0, 0] == 1
    assert O.quantize_codes(x, z, s, 1).tolist() == [[0, 0, 1, 0, 1, 1]]


def test_two_bit_ties_go_to_even():
    x = np.array([[0.0, 0.5, 1.5, 2.5, 3.0, 1.0, 2.0]], dtype=np.float32)
    z, s, _ = O.group_params(x, 2, axis=1)
    assert s[0, 0] == 1
    assert O.quantize_codes(x, z, s, 2).tolist() == [[0, 0, 2, 2, 3, 1, 2]]


def test_constant_group():
    x = np.full((3, 8), 1.5, dtype=np.float32)
    z, s, _ = O.group_params(x, 2, axis=1)
    c = O.quantize_codes(x, z, s, 2)
    zh, sh = O.calibrate(z, s, 2, 0.045)
    assert (c == 0).all() and (sh == 0).all() and (zh == 1.5).all()


@pytest.mark.parametrize("bits,eta", [(1, 1 / 6), (1, 0.25), (2, 0.045), (2, 0.09), (1, 1 / 3)])
def test_calibration_endpoints(bits, eta):
    # code 0 -> z + eta*s*qmax ; code qmax -> z + (1-eta)*s*qmax  (derivation before Eq. 12)
    x = _rand((128, 32), 3)
    qmax = (1 << bits) - 1
    z, s, rng = O.group_params(x, bits, axis=1)
    zh, sh = O.calibrate(z, s, bits, eta)
    z64, s64 = z.astype(np.float64), s.astype(np.float64)
    lo = z64 + eta * s64 * qmax
    hi = z64 + (1 - eta) * s64 * qmax
    assert np.allclose(zh, lo, rtol=1e-6, atol=1e-6)
    assert np.allclose(qmax * sh.astype(np.float64) + zh, hi, rtol=1e-6, atol=1e-6)
    # the dequantization interval shrinks symmetrically inside [min, max]
    assert (zh >= z).all() and (qmax * sh + zh <= z + rng + 1e-5).all()


@pytest.mark.parametrize("bits,eta", [(1, 1 / 6), (2, 0.045)])
def test_calibrated_error_bound(bits, eta):
    # x_hat = (z + c s) + eta s (qmax - 2c)  =>  |x - x_hat| <= s/2 + eta*s*qmax
    x = _rand((256, 32), 5)
    qmax = (1 << bits) - 1
    z, s, _ = O.group_params(x, bits, axis=1)
    c = O.quantize_codes(x, z, s, bits)
    zh, sh = O.calibrate(z, s, bits, eta)
    xh = c * sh.astype(np.float64) + zh.astype(np.float64)
    bound = s.astype(np.float64) * (0.5 + eta * qmax) * (1 + 1e-5)
    assert (np.abs(x - xh) <= bound).all()


def test_codes_do_not_depend_on_eta():
    # calibration changes only the stored parameters, never the integer codes
    x = _rand((32, 64), 9)
    ref = O.quantize_k_block(x, 2, 32, 0.0, True)[0]
    for eta in (0.045, 0.09, 0.2):
        assert np.array_equal(O.quantize_k_block(x, 2, 32, eta, True)[0], ref)


@pytest.mark.parametrize("eta,want", [(0.0, 1 / 12), (0.25, 1 / 48), (1 / 6, 1 / 36), (0.5, 1 / 12)])
def test_one_bit_mse_closed_form(eta, want):
    # X_T ~ U(0,1): E[(X_T - f(X_T, eta))^2] = eta^2 - eta/2 + 1/12
    rng = np.random.default_rng(11)
    n = 1 << 20
    x = rng.random(n).astype(np.float32)
    x[0], x[1] = 0.0, 1.0  # so that z = 0, s = 1 and X_T = X
    x = x.reshape(1, n)
    z, s, _ = O.group_params(x, 1, axis=1)
    c = O.quantize_codes(x, z, s, 1)
    zh, sh = O.calibrate(z, s, 1, eta)
    xh = c * sh.astype(np.float64) + zh.astype(np.float64)
    mse = float(np.mean((x - xh) ** 2))
    assert abs(mse - want) < 4e-4
    assert abs(want - (eta * eta - eta / 2 + 1 / 12)) < 1e-12


def test_calibration_reduces_one_bit_error_on_uniform_data():
    rng = np.random.default_rng(2)
    x = rng.random((512, 32)).astype(np.float32)

    def mse(eta):
        c, s, z = O.quantize_v_block(x, 1, 32, eta, True)
        return float(np.mean((O.dequantize_v(c, s, z, 32) - x) ** 2))

    assert mse(1 / 6) < mse(0.0) and mse(0.25) < mse(0.0)


@pytest.mark.parametrize("bits", [1, 2])
def test_pseudo_quantize_gives_the_same_parameters(bits):
    x = _rand((64, 128), 13)
    c, s, z = O.quantize_k_block(x, bits, 32, 0.045, True)
    c2, s2, z2 = O.quantize_k_block(x, bits, 32, 0.045, False)
    assert c2 is None and np.array_equal(s.view(np.uint16), s2.view(np.uint16))
    assert np.array_equal(z.view(np.uint16), z2.view(np.uint16))
    c, s, z = O.quantize_v_block(x, bits, 32, 0.045, True)
    c2, s2, z2 = O.quantize_v_block(x, bits, 32, 0.045, False)
    assert c2 is None and np.array_equal(s.view(np.uint16), s2.view(np.uint16))
    assert np.array_equal(z.view(np.uint16), z2.view(np.uint16))


def test_key_groups_run_over_tokens_and_value_groups_over_channels():
    # a key channel scaled by 100 must not change any other channel's parameters;
    # a value token scaled by 100 must not change any other token's parameters
    x = _rand((64, 64), 17)
    y = x.copy(); y[:, 5] *= 100
    _, s1, z1 = O.quantize_k_block(x, 2, 32, 0.0, True)
    _, s2, z2 = O.quantize_k_block(y, 2, 32, 0.0, True)
    keep = np.arange(64) != 5
    assert np.array_equal(s1[:, keep], s2[:, keep]) and not np.array_equal(s1[:, 5], s2[:, 5])
    assert s1.shape == (2, 64)
    y = x.copy(); y[7, :] *= 100
    _, s1, z1 = O.quantize_v_block(x, 2, 32, 0.0, True)
    _, s2, z2 = O.quantize_v_block(y, 2, 32, 0.0, True)
    keep = np.arange(64) != 7
    assert np.array_equal(s1[keep], s2[keep]) and not np.array_equal(s1[7], s2[7])
    assert s1.shape == (64, 2)


def test_group_parameters_match_definition_elementwise():
    x = _rand((32, 64), 19)
    _, s, z = O.quantize_k_block(x, 2, 32, 0.0, True)
    for d in range(64):
        col = x[:, d]
        assert z[0, d] == np.float16(col.min())
        assert s[0, d] == np.float16(np.float32(col.max() - col.min()) / np.float32(3))


def test_bf16_helpers():
    vals = np.array([0.0, 1.0, -2.5, 3.140625, 1e-3, 65280.0], dtype=np.float32)
    bits = O.f32_to_bf16_bits(vals)
    back = O.bf16_bits_to_f32(bits)
    assert np.allclose(back, vals, rtol=2 ** -8)
    # exact for values already representable, ties to even
    assert O.f32_to_bf16_bits(np.array([1.0], np.float32))[0] == 0x3F80
    assert O.f32_to_bf16_bits(np.array([1.00390625], np.float32))[0] == 0x3F80  # 1 + 2^-8: tie -> even
    assert O.f32_to_bf16_bits(np.array([1.01171875], np.float32))[0] == 0x3F82  # 1 + 3*2^-8: tie -> even


def test_weighted_merge_intervals():
    # Appendix F: six intervals of gamma0; inside each, round(gamma0*delta) is constant
    cuts = [0, 1 / 6, 1 / 4, 1 / 2, 3 / 4, 5 / 6, 1]
    table = {  # interval index -> c for delta = 1, 2, 3
        0: (0, 0, 0), 1: (0, 0, 1), 2: (0, 1, 1), 3: (1, 1, 2), 4: (1, 2, 2), 5: (1, 2, 3)}
    for k in range(6):
        for frac in (0.1, 0.5, 0.9):
            g0 = cuts[k] + frac * (cuts[k + 1] - cuts[k])
            for e1 in range(4):
                for e0 in range(e1, 4):
                    delta = e0 - e1
                    want = e1 + (table[k][delta - 1] if delta else 0)
                    got = O.merge_codes_weighted(np.array([e0]), np.array([e1]), g0)[0]
                    assert got == want, (g0, e0, e1)
    # gamma0 in (5/6, 1] is plain sharing of the first layer's codes
    e0 = np.arange(4).repeat(4); e1 = np.tile(np.arange(4), 4)
    assert np.array_equal(O.merge_codes_weighted(e0, e1, 0.9), e0)
    assert np.array_equal(O.merge_codes_weighted(e0, e1, 0.1), e1)

"""Pins for the oracle's cross-layer patterns beyond the accelerated default: weighted-average merging of a
pair's codes (Section 3.3.3, Appendix F), larger groups and other dominant layers (Section 3.3.4, Table group),
and half-precision inputs."""
import numpy as np
import pytest

from oracle import xq_oracle as O


def _tokens(rng, S, D, f16=False):
    x = rng.standard_normal((1, 1, S, D)).astype(np.float32)
    if f16:
        return x.astype(np.float16).view(np.uint16)
    return O.f32_to_bf16_bits(x)


def _cache(L=2, D=64, g=32, R=32, bits=2, **kw):
    q = L if bits == 2 else 0
    return O.OracleCache(L, 1, 2, 1, D, g, R, q, q, 0, 0, np.float32(0.0), np.float32(0.045), **kw)


# one value of gamma_0 inside each of Appendix F's six intervals, with the merged code it gives for the pairs
# (e0, e1) = (3, 0), (2, 0), (1, 0): floor(gamma_0 * delta + 1/2) by the appendix's case analysis
INTERVALS = [(0.05, (0, 0, 0)), (0.2, (1, 0, 0)), (0.4, (1, 1, 0)), (0.6, (2, 1, 1)), (0.8, (2, 2, 1)), (0.95, (3, 2, 1))]


@pytest.mark.parametrize("gamma0,want", INTERVALS)
def test_merge_intervals_through_gamma1(gamma0, want):
    e0 = np.array([3, 2, 1], dtype=np.uint8)
    e1 = np.zeros(3, dtype=np.uint8)
    got = O.merge_codes_gamma1(e0, e1, np.float32(1.0 - gamma0))
    assert tuple(got) == want
    # and mirrored: e_m = e1 + round(gamma_0 (e0 - e1)) also when e1 is the larger code
    got = O.merge_codes_gamma1(e1, e0, np.float32(gamma0))
    assert tuple(got) == want


@pytest.mark.parametrize("gamma0", [0.05, 0.4, 0.6, 0.95])
@pytest.mark.parametrize("bits", [1, 2])
def test_cache_merges_when_the_second_layer_quantizes(gamma0, bits):
    rng = np.random.default_rng(5)
    D, R, S = 64, 32, 70
    k0, v0 = _tokens(rng, S, D), _tokens(rng, S, D)
    k1, v1 = _tokens(rng, S, D), _tokens(rng, S, D)
    gamma1 = float(np.float32(1.0 - gamma0))
    oc = _cache(bits=bits, gamma1=gamma1)
    alone0, alone1 = _cache(L=1, bits=bits), _cache(L=1, bits=bits)
    oc.append(0, k0, v0)
    alone0.append(0, k0, v0)
    alone1.append(0, k1, v1)
    # until the second layer has quantized a block it holds the first layer's own codes
    assert np.array_equal(oc.codes_and_meta(0)[0], alone0.codes_and_meta(0)[0])
    oc.append(1, k1, v1)
    e0k, _, _, e0v, _, _ = alone0.codes_and_meta(0)
    e1k, s1k, z1k, e1v, s1v, z1v = alone1.codes_and_meta(0)
    for layer in (0, 1):
        ck, sk, zk, cv, sv, zv = oc.codes_and_meta(layer)
        assert np.array_equal(ck, O.merge_codes_weighted(e0k, e1k, 1.0 - gamma1))
        assert np.array_equal(cv, O.merge_codes_weighted(e0v, e1v, 1.0 - gamma1))
    # each layer keeps the scale and zero-point of its own data
    _, sk, zk, _, sv, zv = oc.codes_and_meta(1)
    assert np.array_equal(sk, s1k) and np.array_equal(zk, z1k) and np.array_equal(sv, s1v) and np.array_equal(zv, z1v)
    if gamma0 > 5 / 6:   # the accelerated scheme: the first layer's codes
        assert np.array_equal(oc.codes_and_meta(1)[0], e0k)
    if gamma0 < 1 / 6:   # its mirror image: the second layer's codes
        assert np.array_equal(oc.codes_and_meta(0)[0], e1k)


@pytest.mark.parametrize("group,k", [(3, 0), (3, 2), (4, 1), (2, 1)])
def test_groups_read_the_dominant_layers_codes(group, k):
    rng = np.random.default_rng(group * 10 + k)
    L, D, S = 2 * group, 64, 40
    oc = O.OracleCache(L, 1, 2, 1, D, 32, 32, L, L, 0, 0, np.float32(0.0), np.float32(0.0),
                       share_group=group, share_dominant=k)
    alone = {}
    for l in range(L):
        kk, vv = _tokens(rng, S, D), _tokens(rng, S, D)
        oc.append(l, kk, vv)
        alone[l] = _cache(L=1)
        alone[l].eta = oc.eta
        alone[l].append(0, kk, vv)
    for l in range(L):
        owner = (l // group) * group + k
        ck, sk, zk, cv, sv, zv = oc.codes_and_meta(l)
        assert np.array_equal(ck, alone[owner].codes_and_meta(0)[0])     # the dominant layer's codes
        assert np.array_equal(sk, alone[l].codes_and_meta(0)[1])         # its own parameters
        assert np.array_equal(zv, alone[l].codes_and_meta(0)[5])
    # decoding a layer uses those codes with its own scale and zero-point
    q = _tokens(rng, 1, D)[:, :, 0]
    q = np.repeat(q, 2, axis=1)
    l = k + 1 if k + 1 < group else 0
    kh = O.dequantize_k(alone[(l // group) * group + k].codes_and_meta(0)[0][0, 0], *[a[0, 0] for a in alone[l].codes_and_meta(0)[1:3]], 32)
    got_k, _ = oc.dequantized(l, 0, 0)
    assert np.array_equal(got_k[:32], kh)
    assert np.isfinite(oc.decode(l, q)).all()


def test_half_precision_inputs_are_widened_exactly():
    rng = np.random.default_rng(1)
    D, S = 64, 40
    x = rng.standard_normal((1, 1, S, D)).astype(np.float16)
    a = _cache(L=1, f16=True)
    a.append(0, x.view(np.uint16), x.view(np.uint16))
    # the same numbers given as fp32-exact bf16 would differ; compare with the block quantizer on the fp32 values
    codes, s, z = O.quantize_k_block(x[0, 0, :32].astype(np.float32), 2, 32, np.float32(0.045), True)
    ck, sk, zk, _, _, _ = a.codes_and_meta(0)
    assert np.array_equal(ck[0, 0], codes) and np.array_equal(sk[0, 0], s) and np.array_equal(zk[0, 0], z)
    assert np.array_equal(a.layers[0]["win_k"][0, 0], x[0, 0, 32:].astype(np.float32))


def test_delta_histogram_counts_code_differences():
    """Section 3.3.1's statistic: elements by |own code - shared code|.  Identical layers differ nowhere; the
    counts of a pair add up to the quantized elements; they equal a direct count over standalone quantizations."""
    rng = np.random.default_rng(8)
    D, S = 64, 100
    k0, v0 = _tokens(rng, S, D), _tokens(rng, S, D)
    k1, v1 = _tokens(rng, S, D), _tokens(rng, S, D)
    oc = _cache(delta_stats=True)
    oc.append(0, k0, v0); oc.append(1, k1, v1)
    a0, a1 = _cache(L=1), _cache(L=1)
    a0.append(0, k0, v0); a1.append(0, k1, v1)
    nq = oc.n_quantized(1)
    assert nq == 96 and (oc.delta[0] == 0).all()
    for kind, idx in ((0, 0), (1, 3)):
        e0, e1 = a0.codes_and_meta(0)[idx], a1.codes_and_meta(0)[idx]
        want = [int(np.count_nonzero(np.abs(e0.astype(int) - e1.astype(int)) == d)) for d in range(4)]
        assert list(oc.delta[1, kind]) == want and sum(want) == nq * D
    # the shared codes are untouched by the statistic
    assert np.array_equal(oc.codes_and_meta(1)[0], a0.codes_and_meta(0)[0])
    same = _cache(delta_stats=True)
    same.append(0, k0, v0); same.append(1, k0, v0)
    assert list(same.delta[1, 0]) == [nq * D, 0, 0, 0]

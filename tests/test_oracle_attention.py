"""Pins for the oracle's attention and for the cache procedure (Algorithm 1)."""
import math

import numpy as np
import pytest

from oracle import xq_oracle as O


def _bf16(x):
    return O.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def _brute_attention(q, k, v, scale):
    S, D = len(k), len(q)
    logits = [scale * sum(float(q[d]) * float(k[t][d]) for d in range(D)) for t in range(S)]
    m = max(logits)
    w = [math.exp(l - m) for l in logits]
    tot = sum(w)
    return [sum(w[t] * float(v[t][d]) for t in range(S)) / tot for d in range(D)]


def test_attention_against_loops():
    rng = np.random.default_rng(0)
    q = rng.standard_normal(8); k = rng.standard_normal((11, 8)); v = rng.standard_normal((11, 8))
    got = O.attention(q, k, v, 0.35)
    assert np.allclose(got, _brute_attention(q, k, v, 0.35), rtol=1e-12, atol=1e-12)


def test_attention_special_cases():
    rng = np.random.default_rng(1)
    k = rng.standard_normal((9, 4)); v = rng.standard_normal((9, 4))
    # zero query: uniform weights, the output is the mean value
    assert np.allclose(O.attention(np.zeros(4), k, v, 0.5), v.mean(axis=0))
    # one key aligned with a huge query: the output is that token's value
    k[3] *= 10.0  # largest norm, so k[3].k[3] > k[t].k[3] for every other t
    q = 1e3 * k[3]
    assert np.allclose(O.attention(q, k, v, 1.0), v[3], atol=1e-9)
    # a shift common to all logits changes nothing: add a constant key component along q
    q = rng.standard_normal(4)
    k2 = k + 5.0 * q / (q @ q)
    assert np.allclose(O.attention(q, k, v, 1.0), O.attention(q, k2, v, 1.0))
    # against a library softmax
    import torch
    p = torch.softmax(torch.tensor(0.7 * (k @ q)), dim=0).numpy()
    assert np.allclose(O.attention(q, k, v, 0.7), p @ v)


def _cache(L=2, B=1, Hq=2, Hkv=1, D=64, g=32, R=32, kq=2, vq=2, km=0, vm=0, e1=0.0, e2=0.0):
    return O.OracleCache(L, B, Hq, Hkv, D, g, R, kq, vq, km, vm, e1, e2)


def _kv(seed, B, H, n, D):
    rng = np.random.default_rng(seed)
    return _bf16(rng.standard_normal((B, H, n, D))), _bf16(rng.standard_normal((B, H, n, D)))


@pytest.mark.parametrize("S", [1, 31, 32, 33, 64, 65, 100])
def test_window_policy(S):
    c = _cache()
    k, v = _kv(0, 1, 1, S, 64)
    c.append(0, k, v)
    r = ((S - 1) % 32) + 1
    assert c.layers[0]["win_k"].shape[2] == r
    assert c.n_quantized(0) == S - r and c.layers[0]["seq"] == S


def test_empty_quantized_region_is_exact_16bit_attention():
    c = _cache()
    k, v = _kv(1, 1, 1, 32, 64)
    c.append(0, k, v)
    assert c.n_quantized(0) == 0
    q = _bf16(np.random.default_rng(2).standard_normal((1, 2, 64)))
    out = c.decode(0, q)
    kf, vf = O.bf16_bits_to_f32(k)[0, 0], O.bf16_bits_to_f32(v)[0, 0]
    for h in range(2):
        ref = _brute_attention(O.bf16_bits_to_f32(q)[0, h], kf, vf, 1 / math.sqrt(64))
        assert np.allclose(out[0, h], ref, rtol=1e-12, atol=1e-12)


def test_append_granularity_invariance():
    k, v = _kv(3, 2, 2, 75, 64)
    a = _cache(B=2, Hq=4, Hkv=2, e2=0.045)
    a.append(0, k, v)
    b = _cache(B=2, Hq=4, Hkv=2, e2=0.045)
    for lo, hi in ((0, 1), (1, 2), (2, 34), (34, 70), (70, 75)):
        b.append(0, k[:, :, lo:hi], v[:, :, lo:hi])
    for x, y in zip(a.codes_and_meta(0), b.codes_and_meta(0)):
        assert np.array_equal(x, y)
    assert np.array_equal(a.layers[0]["win_k"], b.layers[0]["win_k"])


def test_sharing_pair():
    k0, v0 = _kv(4, 1, 2, 96, 64)
    k1, v1 = _kv(5, 1, 2, 96, 64)
    c = _cache(Hq=2, Hkv=2, e2=0.045)
    c.append(0, k0, v0); c.append(1, k1, v1)
    own = c.codes_and_meta(0); sub = c.codes_and_meta(1)
    # the second layer of the pair reads the first layer's codes ...
    assert np.array_equal(own[0], sub[0]) and np.array_equal(own[3], sub[3])
    assert c.layers[1]["k_codes"][0] is None and c.layers[1]["v_codes"][0] is None
    # ... with its own scale / zero-point, equal to those of a stand-alone quantization of its tensor
    solo = _cache(L=1, Hq=2, Hkv=2, km=1, vm=1, e2=0.045)
    solo.append(0, k1, v1)
    s = solo.codes_and_meta(0)
    for i in (1, 2, 4, 5):
        assert np.array_equal(sub[i], s[i])
        assert not np.array_equal(sub[i], own[i])
    # the owner's codes do not depend on the subordinate layer's data
    c2 = _cache(Hq=2, Hkv=2, e2=0.045)
    c2.append(0, k0, v0); c2.append(1, k0, v0)
    assert np.array_equal(c2.codes_and_meta(0)[0], own[0])
    # identical tensors in both layers dequantize identically
    a, b = c2.dequantized(0, 0, 1), c2.dequantized(1, 0, 1)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_no_sharing_below_km():
    k0, v0 = _kv(6, 1, 1, 64, 64); k1, v1 = _kv(7, 1, 1, 64, 64)
    c = _cache(km=2, vm=0)
    c.append(0, k0, v0); c.append(1, k1, v1)
    assert c.layers[1]["k_codes"][0] is not None and c.layers[1]["v_codes"][0] is None
    own = c.codes_and_meta(0); sub = c.codes_and_meta(1)
    assert not np.array_equal(own[0], sub[0]) and np.array_equal(own[3], sub[3])


def test_decode_against_loops_with_quantized_region():
    c = _cache(Hq=2, Hkv=1, e2=0.045)
    k, v = _kv(8, 1, 1, 80, 64)
    c.append(0, k, v); c.append(1, k, v)
    q = _bf16(np.random.default_rng(9).standard_normal((1, 2, 64)))
    out = c.decode(1, q)
    kc, ks, kz, vc, vs, vz = c.codes_and_meta(1)
    nq = c.n_quantized(1)
    assert nq == 64
    K = [[float(kc[0, 0, t, d]) * float(ks[0, 0, t // 32, d]) + float(kz[0, 0, t // 32, d]) for d in range(64)]
         for t in range(nq)]
    V = [[float(vc[0, 0, t, d]) * float(vs[0, 0, t, d // 32]) + float(vz[0, 0, t, d // 32]) for d in range(64)]
         for t in range(nq)]
    K += O.bf16_bits_to_f32(k)[0, 0, nq:].astype(np.float64).tolist()
    V += O.bf16_bits_to_f32(v)[0, 0, nq:].astype(np.float64).tolist()
    for h in range(2):
        ref = _brute_attention(O.bf16_bits_to_f32(q)[0, h], K, V, 1 / math.sqrt(64))
        assert np.allclose(out[0, h], ref, rtol=1e-12, atol=1e-12)


def test_gqa_head_mapping():
    c = _cache(Hq=4, Hkv=2)
    k, v = _kv(10, 1, 2, 40, 64)
    c.append(0, k, v)
    q = _bf16(np.random.default_rng(11).standard_normal((1, 4, 64)))
    out = c.decode(0, q)
    for h in range(4):
        kh, vh = c.dequantized(0, 0, h // 2)
        assert np.allclose(out[0, h], O.attention(O.bf16_bits_to_f32(q)[0, h], kh, vh, 1 / 8))


def test_quantization_error_is_small_relative_to_two_bit_step():
    # dequantized keys stay within the calibrated bound of the originals
    c = _cache(e2=0.045)
    k, v = _kv(12, 1, 1, 64, 64)
    c.append(0, k, v)
    kh, vh = c.dequantized(0, 0, 0)
    kf = O.bf16_bits_to_f32(k)[0, 0].astype(np.float64)
    rng_k = kf[:32].max(axis=0) - kf[:32].min(axis=0)
    assert (np.abs(kh[:32] - kf[:32]) <= (rng_k / 3) * (0.5 + 0.045 * 3) * 1.01 + 1e-3).all()
    assert np.array_equal(kh[32:], kf[32:])


# ---- chunk attention (the last T tokens as queries, causal inside the chunk)

def test_chunk_of_one_is_decode():
    rng = np.random.default_rng(0)
    q, k, v = rng.standard_normal((1, 16)), rng.standard_normal((9, 16)), rng.standard_normal((9, 16))
    assert np.array_equal(O.attention_chunk(q, k, v, 0.25)[0], O.attention(q[0], k, v, 0.25))


def test_chunk_against_explicit_loops():
    rng = np.random.default_rng(1)
    S, T, D = 11, 4, 8
    q, k, v = rng.standard_normal((T, D)), rng.standard_normal((S, D)), rng.standard_normal((S, D))
    got = O.attention_chunk(q, k, v, 0.3)
    for j in range(T):
        n = S - T + j + 1  # tokens visible to query j
        logit = [0.3 * sum(q[j][d] * k[t][d] for d in range(D)) for t in range(n)]
        mx = max(logit)
        w = [np.exp(x - mx) for x in logit]
        for d in range(D):
            want = sum(w[t] * v[t][d] for t in range(n)) / sum(w)
            assert abs(got[j][d] - want) < 1e-12


def test_chunk_rows_ignore_later_tokens_and_the_last_row_sees_all():
    rng = np.random.default_rng(2)
    S, T, D = 20, 5, 8
    q, k, v = rng.standard_normal((T, D)), rng.standard_normal((S, D)), rng.standard_normal((S, D))
    base = O.attention_chunk(q, k, v, 0.5)
    assert np.allclose(base[T - 1], O.attention(q[T - 1], k, v, 0.5), rtol=0, atol=1e-14)
    for j in range(T - 1):
        k2, v2 = k.copy(), v.copy()
        k2[S - T + j + 1:] += 100.0  # tokens after query j's own position
        v2[S - T + j + 1:] -= 50.0
        again = O.attention_chunk(q, k2, v2, 0.5)
        assert np.array_equal(again[j], base[j])
        assert not np.allclose(again[T - 1], base[T - 1])
    # a row equals a decode call over its visible prefix
    for j in range(T):
        n = S - T + j + 1
        assert np.allclose(base[j], O.attention(q[j], k[:n], v[:n], 0.5), rtol=0, atol=1e-14)


def test_cache_chunk_matches_cache_decode_for_one_token():
    rng = np.random.default_rng(3)
    D, S = 64, 75
    oc = O.OracleCache(1, 1, 2, 1, D, 32, 32, 1, 1, 1, 1, np.float32(1 / 6), np.float32(0.045))
    x = O.f32_to_bf16_bits(rng.standard_normal((1, 1, S, D)).astype(np.float32))
    y = O.f32_to_bf16_bits(rng.standard_normal((1, 1, S, D)).astype(np.float32))
    oc.append(0, x, y)
    q = O.f32_to_bf16_bits(rng.standard_normal((1, 1, 2, D)).astype(np.float32))
    assert np.array_equal(oc.attention_chunk(0, q)[0], oc.decode(0, q[0]))
    # a chunk longer than the window reaches into the quantized region
    q = O.f32_to_bf16_bits(rng.standard_normal((40, 1, 2, D)).astype(np.float32))
    got = oc.attention_chunk(0, q)
    kh, vh = oc.dequantized(0, 0, 0)
    qf = O.bf16_bits_to_f32(q).astype(np.float64)
    for j in (0, 17, 39):
        n = S - 40 + j + 1
        assert np.allclose(got[j, 0, 1], O.attention(qf[j, 0, 1], kh[:n], vh[:n], oc.sm_scale), rtol=0, atol=1e-13)

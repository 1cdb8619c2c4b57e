"""CPU oracle for XQuant decode attention over a cross-layer 1/2-bit KV cache.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA path must compute.  It shares no code with the CUDA path, imports nothing
from the product package and is imported only by the tests, by the smoke check
and by the benchmark's CPU-baseline leg.  It is never tuned for speed.

Precision.  The quantizer arithmetic (Eq. 1, Eq. 2, Eq. 12) is fixed to IEEE
fp32 with one rounding per written operation, round-half-even for the code
(np.rint) and round-to-nearest-even to fp16 for the stored scale / zero-point,
because packed codes, scales and zero-points are compared bit for bit.
Dequantization (Eq. 3 with the calibrated parameters) and attention are fp64.

Inputs are 16-bit floats handed over as raw bit patterns (np.uint16 holding
bfloat16), so that the oracle and the CUDA path see identical values.

Parity pins (tests/test_oracle_*.py): equivalent bit-width against every width
the paper prints; the quantizer against the half-step error bound, the endpoint
identity of the calibration derivation, the 1-bit MSE closed form and brute
force on tiny groups; packing against the round-trip identity and a bit census;
attention against brute-force loops, the empty-quantized-region case and the
uniform-logit case; the gamma-interval enumeration of the weighted merge.
Parity unpinned by the paper (fixed by readings of it made here and then enforced
between the oracle and the CUDA path): the residual-window flush policy, the
fp16 storage type of scale / zero-point and the bit layout of packed words.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# 16-bit float helpers (bit-pattern in, exact fp32 out)
# --------------------------------------------------------------------------


def bf16_bits_to_f32(u16: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns exactly to fp32 (bf16 is the top half of fp32)."""
    u = np.asarray(u16, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 bit patterns, round-to-nearest-even (finite inputs)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = u + np.uint64(0x7FFF) + lsb
    return (u >> np.uint64(16)).astype(np.uint16)


# --------------------------------------------------------------------------
# Layer policy (Algorithm 1) and equivalent bit-width (Appendix C)
# --------------------------------------------------------------------------


def layer_bits(layer: int, q: int) -> int:
    """Bit-width of a layer: 2-bit for layers [0, q), 1-bit above (Appendix E)."""
    return 2 if layer < q else 1


def code_owner(layer: int, m: int, group: int = 2, dominant: int = 0) -> int:
    """The layer whose integer codes `layer` reads (itself when it keeps its own).
    Below the sharing start m every layer keeps its codes.  From m on, the layers
    form groups of `group` layers and only the group's dominant layer (index
    `dominant` within the group) stores codes (Section 3.3.4; ablation of Table
    group: contiguous groups of size G, "store and share only in the k-th layer").
    Groups of two follow Algorithm 1's dequantize loop, which tests the layer's
    parity (an odd layer reuses layer - 1: dominant 0); groups of three and four
    are counted from m, which is what gives Table group its common width (20 of
    32 value layers stored for G = 2, 3, 4 with sharing from layer 8, 14, 16)."""
    if layer < m:
        return layer
    if group == 2:
        return layer - layer % 2 + dominant
    return layer - (layer - m) % group + dominant


def owns_codes(layer: int, m: int) -> bool:
    """Algorithm 1, dequantize loop: a layer keeps its own integer codes when it
    lies below the sharing start m or is the first (even) layer of its pair;
    otherwise it reuses the codes of layer-1 (Section 3.3.4, dominant layer k=0,
    group size G=2).  The quantize loop of Algorithm 1 prints vm / vq in this
    test for keys / values; the dequantize loop and Appendix C use km / vm, which
    is the reading taken here."""
    return code_owner(layer, m) == layer


def equiv_bits_one(q: int, m: int, n_layers: int, group: int = 2, dominant: int = 0) -> float:
    """Average stored code bits per element of one cache kind, by direct count:
    every code-owning layer stores bits(l) per element, a subordinate layer stores
    none (Appendix C: codes only, scale / zero-point excluded)."""
    total = 0
    for l in range(n_layers):
        if code_owner(l, m, group, dominant) == l:
            total += layer_bits(l, q)
    return total / n_layers


def equiv_bits(kq: int, vq: int, km: int, vm: int, n_layers: int = 32, group: int = 2, dominant: int = 0) -> float:
    """Equivalent bit-width of Appendix C: mean of the key and value figures."""
    return 0.5 * (equiv_bits_one(kq, km, n_layers, group, dominant) + equiv_bits_one(vq, vm, n_layers, group, dominant))


def equiv_bits_closed_form(kq: int, vq: int, km: int, vm: int, n_layers: int = 32) -> float:
    """Closed form matching the paper's worked example (kq=30, vq=2, km=32,
    vm=16 -> 1.9375, 0.8125, mean 1.375): shared layers above max(q, m) cost half
    a bit, layers between min and max cost one, layers below min cost two.  Valid
    for even q and m (every configuration the paper lists)."""

    def one(q, m):
        hi, lo = max(q, m), min(q, m)
        return ((n_layers - hi) / 2 + (hi - lo) + 2 * lo) / n_layers

    return 0.5 * (one(kq, km) + one(vq, vm))


# --------------------------------------------------------------------------
# Group quantizer with data-free calibration (Eq. 1, 2, 12; Algorithm 2)
# --------------------------------------------------------------------------


def group_params(x: np.ndarray, bits: int, axis: int):
    """Eq. 1 in fp32: z = min X, s = (max X - min X) / (2^B - 1) over `axis`.
    Returns (z, s, rng) with the reduced axis kept (size 1)."""
    x = np.asarray(x, dtype=np.float32)
    qmax = np.float32((1 << bits) - 1)
    mn = x.min(axis=axis, keepdims=True)
    mx = x.max(axis=axis, keepdims=True)
    rng = (mx - mn).astype(np.float32)
    s = (rng / qmax).astype(np.float32)
    return mn.astype(np.float32), s, rng


def quantize_codes(x: np.ndarray, z: np.ndarray, s: np.ndarray, bits: int) -> np.ndarray:
    """Eq. 2 in fp32 with the UNcalibrated z, s: X_Q = round((X - z) / s), ties to
    even, clamped to [0, 2^B - 1].  A constant group (s == 0) gets code 0."""
    x = np.asarray(x, dtype=np.float32)
    qmax = (1 << bits) - 1
    safe = np.where(s == 0, np.float32(1), s).astype(np.float32)
    t = ((x - z).astype(np.float32) / safe).astype(np.float32)
    c = np.rint(t)
    c = np.clip(c, 0, qmax)
    c = np.where(s == 0, 0, c)
    return c.astype(np.uint8)


def calibrate(z: np.ndarray, s: np.ndarray, bits: int, eta: float):
    """Eq. 12 in fp32, in the order written: z_hat = z + (eta * s) * (2^B - 1),
    s_hat = (1 - 2 eta) * s.  (Algorithm 2 prints the zero-point update without
    the (2^B - 1) factor; Eq. 12 and the endpoint derivation before it carry it.)
    Returns fp32 values; storage rounding is separate."""
    eta = np.float32(eta)
    qmax = np.float32((1 << bits) - 1)
    z = np.asarray(z, dtype=np.float32)
    s = np.asarray(s, dtype=np.float32)
    t = (eta * s).astype(np.float32)
    t = (t * qmax).astype(np.float32)
    z_hat = (z + t).astype(np.float32)
    k = np.float32(np.float32(1) - np.float32(np.float32(2) * eta))
    s_hat = (k * s).astype(np.float32)
    return z_hat, s_hat


def store_f16(x: np.ndarray) -> np.ndarray:
    """Scale and zero-point are stored as IEEE fp16, rounded to nearest even."""
    return np.asarray(x, dtype=np.float32).astype(np.float16)


def quantize_k_block(k_f32: np.ndarray, bits: int, g: int, eta: float, with_codes: bool):
    """Keys, per-channel: one group per (channel, run of g consecutive tokens).
    k_f32: [T, D] with T a multiple of g.  Returns (codes [T, D] uint8 or None,
    s_hat [T/g, D] fp16, z_hat [T/g, D] fp16).  with_codes=False is
    PseudoQuantize of Algorithm 2: same parameters, no codes."""
    T, D = k_f32.shape
    assert T % g == 0
    x = np.asarray(k_f32, dtype=np.float32).reshape(T // g, g, D)
    z, s, _ = group_params(x, bits, axis=1)
    codes = quantize_codes(x, z, s, bits).reshape(T, D) if with_codes else None
    z_hat, s_hat = calibrate(z, s, bits, eta)
    return codes, store_f16(s_hat.reshape(T // g, D)), store_f16(z_hat.reshape(T // g, D))


def quantize_v_block(v_f32: np.ndarray, bits: int, g: int, eta: float, with_codes: bool):
    """Values, per-token: one group per (token, run of g consecutive channels).
    v_f32: [T, D] with D a multiple of g.  Returns (codes [T, D] uint8 or None,
    s_hat [T, D/g] fp16, z_hat [T, D/g] fp16)."""
    T, D = v_f32.shape
    assert D % g == 0
    x = np.asarray(v_f32, dtype=np.float32).reshape(T, D // g, g)
    z, s, _ = group_params(x, bits, axis=2)
    codes = quantize_codes(x, z, s, bits).reshape(T, D) if with_codes else None
    z_hat, s_hat = calibrate(z, s, bits, eta)
    return codes, store_f16(s_hat.reshape(T, D // g)), store_f16(z_hat.reshape(T, D // g))


def dequantize_k(codes: np.ndarray, s_hat: np.ndarray, z_hat: np.ndarray, g: int) -> np.ndarray:
    """Eq. 3 with calibrated parameters, fp64: X_hat = X_Q * s_hat + z_hat, the
    parameters being those of the reading layer and the codes those of the pair's
    code-owning layer."""
    T, D = codes.shape
    s = np.repeat(s_hat.astype(np.float64), g, axis=0)
    z = np.repeat(z_hat.astype(np.float64), g, axis=0)
    return codes.astype(np.float64) * s + z


def dequantize_v(codes: np.ndarray, s_hat: np.ndarray, z_hat: np.ndarray, g: int) -> np.ndarray:
    s = np.repeat(s_hat.astype(np.float64), g, axis=1)
    z = np.repeat(z_hat.astype(np.float64), g, axis=1)
    return codes.astype(np.float64) * s + z


def merge_codes_weighted(e0: np.ndarray, e1: np.ndarray, gamma0: float) -> np.ndarray:
    """Appendix F: merged code of a layer pair under weighted averaging,
    e_m = round(gamma0 * e0 + (1 - gamma0) * e1), round to nearest (the paper's
    intervals are open, so ties are outside its statement; ties-to-even here).
    gamma0 in (5/6, 1] reproduces e0, i.e. the accelerated sharing used on the
    hot path."""
    v = gamma0 * e0.astype(np.float64) + (1.0 - gamma0) * e1.astype(np.float64)
    return np.rint(v).astype(np.uint8)


def merge_codes_gamma1(e0: np.ndarray, e1: np.ndarray, gamma1) -> np.ndarray:
    """The same with the pair's weights stated as the library's configuration
    states them: gamma1 (a float32) is the second layer's weight and
    gamma0 = 1 - gamma1, both taken in double precision."""
    g1 = float(np.float32(gamma1))
    g0 = 1.0 - g1
    v = g0 * e0.astype(np.float64) + g1 * e1.astype(np.float64)
    return np.rint(v).astype(np.uint8)


# --------------------------------------------------------------------------
# Packed layouts (a choice made here; the paper does not discuss packing)
# --------------------------------------------------------------------------
# Words are little-endian 32-bit.  A byte of a word holds the codes of 8/bits
# row elements, the four bytes of a word hold four consecutive row elements at
# the same bit offset.  Keys: a row is one token (its D channels), rows are kept
# in units of 32 tokens, each unit as chunks of at most 16 bytes per token.
# Values: a row is one channel over a batch of 128 tokens, a batch is kept as
# chunks of 16 bytes per channel.

BATCH = 128  # tokens per value-code batch


def k_code_position(t: int, d: int, bits: int, D: int):
    """(word index, bit offset) of key code (token t, channel d) in one (batch,
    kv head) stream."""
    n = 32 // bits                     # codes per word
    word_in_row, e = divmod(d, n)      # e: element index inside the word
    byte, step = e % 4, e // 4         # four consecutive channels share a bit offset
    row_bytes = D * bits // 8
    chunk_bytes = min(16, row_bytes)
    chunk, off = divmod(4 * word_in_row, chunk_bytes)
    unit, lane = divmod(t, 32)
    addr = unit * 32 * row_bytes + chunk * 32 * chunk_bytes + lane * chunk_bytes + off
    return addr // 4, 8 * byte + bits * step


def v_code_position(t: int, d: int, bits: int, D: int):
    """(word index, bit offset) of value code (token t, channel d): the channel
    owns a row over the 128 tokens of a batch."""
    n = 32 // bits
    batch, tl = divmod(t, BATCH)
    word_in_row, e = divmod(tl, n)
    byte, step = e % 4, e // 4
    chunk, w = divmod(word_in_row, 4)
    addr = batch * D * 16 * bits + chunk * D * 16 + d * 16 + 4 * w
    return addr // 4, 8 * byte + bits * step


def k_stream_words(T: int, bits: int, D: int) -> int:
    """Words the key codes of T tokens occupy (T a multiple of 32)."""
    return T * D * bits // 32


def v_stream_words(T: int, bits: int, D: int) -> int:
    """Words of the value-code batches that T tokens touch (whole batches)."""
    return -(-T // BATCH) * D * 16 * bits // 4


def _pack(codes: np.ndarray, bits: int, pos_fn, n_words: int):
    """Returns (words, written): `written` marks the words that hold a code."""
    T, D = codes.shape
    words = np.zeros(n_words, dtype=np.uint32)
    written = np.zeros(n_words, dtype=bool)
    for t in range(T):
        for d in range(D):
            w, b = pos_fn(t, d, bits, D)
            words[w] |= np.uint32(int(codes[t, d]) << b)
            written[w] = True
    return words, written


_TABLE_CACHE: dict = {}


def _pack_fast(codes: np.ndarray, bits: int, pos_fn, n_words: int, period: int):
    """Same result as _pack.  The position function repeats with `period` tokens
    (32 for keys, 128 for values) up to a constant word offset per period; the
    (word, bit) table of one period is built by calling it for every element of
    the first period and the offset by calling it once more (tests check
    _pack_fast == _pack)."""
    T, D = codes.shape
    key = (pos_fn.__name__, bits, D)
    if key not in _TABLE_CACHE:
        w = np.empty((period, D), dtype=np.int64)
        b = np.empty((period, D), dtype=np.int64)
        for t in range(period):
            for d in range(D):
                w[t, d], b[t, d] = pos_fn(t, d, bits, D)
        stride = pos_fn(period, 0, bits, D)[0] - pos_fn(0, 0, bits, D)[0]
        _TABLE_CACHE[key] = (w, b, stride)
    w, b, stride = _TABLE_CACHE[key]
    words = np.zeros(n_words, dtype=np.uint32)
    written = np.zeros(n_words, dtype=bool)
    for p0 in range(0, T, period):
        n = min(period, T - p0)
        c = codes[p0:p0 + n].astype(np.uint32) << b[:n].astype(np.uint32)
        idx = (w[:n] + (p0 // period) * stride).reshape(-1)
        np.bitwise_or.at(words, idx, c.reshape(-1))
        written[idx] = True
    return words, written


def pack_k_codes(codes: np.ndarray, bits: int, fast: bool = True):
    T, D = codes.shape
    assert T % 32 == 0
    n = k_stream_words(T, bits, D)
    return _pack_fast(codes, bits, k_code_position, n, 32) if fast else _pack(codes, bits, k_code_position, n)


def pack_v_codes(codes: np.ndarray, bits: int, fast: bool = True):
    T, D = codes.shape
    n = v_stream_words(T, bits, D)
    return _pack_fast(codes, bits, v_code_position, n, BATCH) if fast else _pack(codes, bits, v_code_position, n)


def _unpack(words: np.ndarray, T: int, D: int, bits: int, pos_fn) -> np.ndarray:
    out = np.zeros((T, D), dtype=np.uint8)
    mask = (1 << bits) - 1
    for t in range(T):
        for d in range(D):
            w, b = pos_fn(t, d, bits, D)
            out[t, d] = (int(words[w]) >> b) & mask
    return out


def unpack_k_codes(words, T, D, bits):
    return _unpack(words, T, D, bits, k_code_position)


def unpack_v_codes(words, T, D, bits):
    return _unpack(words, T, D, bits, v_code_position)


def k_meta_position(d: int, D: int) -> int:
    """Index of channel d among the D scales (or the D zero-points) of one key
    token group: channels d, d+32, d+64, ... are neighbours."""
    return (d % 32) * (D // 32) + d // 32


def pack_k_meta(s_hat: np.ndarray, z_hat: np.ndarray) -> np.ndarray:
    """[n_groups, D] fp16 scale and zero -> uint16 [n_groups, 2, D]: per token
    group the permuted scales, then the permuted zero-points."""
    n, D = s_hat.shape
    out = np.zeros((n, 2, D), dtype=np.uint16)
    su = s_hat.astype(np.float16).view(np.uint16)
    zu = z_hat.astype(np.float16).view(np.uint16)
    for d in range(D):
        p = k_meta_position(d, D)
        out[:, 0, p] = su[:, d]
        out[:, 1, p] = zu[:, d]
    return out


def pack_v_meta(s_hat: np.ndarray, z_hat: np.ndarray) -> np.ndarray:
    """[T, n_g] fp16 scale and zero -> uint16 [T, 2, n_g]: per token its n_g
    scales, then its n_g zero-points."""
    T, n_g = s_hat.shape
    out = np.zeros((T, 2, n_g), dtype=np.uint16)
    out[:, 0, :] = s_hat.astype(np.float16).view(np.uint16)
    out[:, 1, :] = z_hat.astype(np.float16).view(np.uint16)
    return out


# --------------------------------------------------------------------------
# Attention (plain definition, fp64)
# --------------------------------------------------------------------------


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, sm_scale: float) -> np.ndarray:
    """One decode query against S cached tokens, no mask: logits = scale * K q,
    p = softmax(logits), out = p^T V.  q: [D], k, v: [S, D]; all fp64."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    logits = sm_scale * (k @ q)
    logits = logits - logits.max()
    p = np.exp(logits)
    p = p / p.sum()
    return p @ v


def attention_chunk(q: np.ndarray, k: np.ndarray, v: np.ndarray, sm_scale: float) -> np.ndarray:
    """The last T cached tokens as queries, causal inside the chunk (the prompt /
    output workload of Appendix D processed a chunk at a time): query j sees the
    tokens 0 .. S - T + j.  Plain definition: masked softmax attention in fp64.
    q: [T, D], k, v: [S, D] -> [T, D]."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, S = q.shape[0], k.shape[0]
    logits = sm_scale * (q @ k.T)
    visible = np.arange(S)[None, :] <= (S - T + np.arange(T))[:, None]
    logits = np.where(visible, logits, -np.inf)
    logits = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ v


# --------------------------------------------------------------------------
# Whole cache: Algorithm 1 with the residual window
# --------------------------------------------------------------------------


class OracleCache:
    """Per-layer KV cache following Algorithm 1 for one batch of sequences.

    Window policy (the paper only states a residual length R): tokens enter a
    16-bit window; when the window already holds R tokens and one more arrives,
    those R tokens are quantized as one block (keys and values alike) and the
    window restarts.  After S > 0 tokens the window holds ((S-1) mod R) + 1
    tokens and the first S minus that many are quantized.
    """

    def __init__(self, n_layers, batch, n_q_heads, n_kv_heads, head_dim, group_size,
                 residual_len, kq, vq, km, vm, eta1, eta2, sm_scale=None,
                 share_group=2, share_dominant=0, gamma1=0.0, f16=False, delta_stats=False):
        self.L, self.B, self.Hq, self.Hkv, self.D = n_layers, batch, n_q_heads, n_kv_heads, head_dim
        self.g, self.R = group_size, residual_len
        self.kq, self.vq, self.km, self.vm = kq, vq, km, vm
        self.eta = {1: np.float32(eta1), 2: np.float32(eta2)}
        self.sm_scale = float(sm_scale) if sm_scale else 1.0 / np.sqrt(head_dim)
        # sharing pattern: layers per group, dominant layer of a group, weight of a pair's second layer in the
        # merged codes (0: the dominant layer's codes are shared as they are); f16: inputs are IEEE half precision
        self.share_group, self.share_dominant, self.gamma1 = share_group or 2, share_dominant, gamma1
        self.f16 = f16
        # Section 3.3.1: per layer and cache kind, the number of quantized elements whose own code differs by
        # d = 0..3 from the code the layer reads from its dominant layer (layers that keep their codes: zeros)
        self.delta_stats = delta_stats
        self.delta = np.zeros((n_layers, 2, 4), dtype=np.int64)
        assert self.gamma1 == 0.0 or (self.share_group == 2 and self.share_dominant == 0)
        assert n_q_heads % n_kv_heads == 0 and residual_len % group_size == 0
        assert head_dim % group_size == 0
        self.layers = [self._empty_layer() for _ in range(n_layers)]

    def _empty_layer(self):
        B, H, D = self.B, self.Hkv, self.D
        return {
            "seq": 0,
            "win_k": np.zeros((B, H, 0, D), dtype=np.float32),
            "win_v": np.zeros((B, H, 0, D), dtype=np.float32),
            "k_codes": [], "k_s": [], "k_z": [],  # lists of per-block arrays [B,H,...]
            "v_codes": [], "v_s": [], "v_z": [],
        }

    def k_bits(self, l):
        return layer_bits(l, self.kq)

    def v_bits(self, l):
        return layer_bits(l, self.vq)

    def k_owner(self, l):
        return code_owner(l, self.km, self.share_group, self.share_dominant)

    def v_owner(self, l):
        return code_owner(l, self.vm, self.share_group, self.share_dominant)

    def _merges(self, l, m):
        """Section 3.3.3 / Appendix F with G = 2: the pair's second layer quantizes its
        own block as well and the pair's codes become the rounded weighted average.  In
        an incremental cache that happens when the second layer's block fills; until
        then the block holds the first layer's codes."""
        return self.gamma1 > 0.0 and l >= m and l % 2 == 1

    def _flush(self, l):
        st = self.layers[l]
        B, H = self.B, self.Hkv
        mrg_k, mrg_v = self._merges(l, self.km), self._merges(l, self.vm)
        cmp_k = self.delta_stats and self.k_owner(l) != l
        cmp_v = self.delta_stats and self.v_owner(l) != l
        own_k, own_v = self.k_owner(l) == l or mrg_k or cmp_k, self.v_owner(l) == l or mrg_v or cmp_v
        bk, bv = self.k_bits(l), self.v_bits(l)
        kc, ks, kz, vc, vs, vz = [], [], [], [], [], []
        for b in range(B):
            for h in range(H):
                c, s, z = quantize_k_block(st["win_k"][b, h], bk, self.g, self.eta[bk], own_k)
                kc.append(c); ks.append(s); kz.append(z)
                c, s, z = quantize_v_block(st["win_v"][b, h], bv, self.g, self.eta[bv], own_v)
                vc.append(c); vs.append(s); vz.append(z)

        def stack(xs):
            return None if xs[0] is None else np.stack(xs).reshape((B, H) + xs[0].shape)

        blk = len(st["k_s"])  # index of the block being quantized
        kcs, vcs = stack(kc), stack(vc)
        for kind, cmp, own, key, mine in ((0, cmp_k, self.k_owner(l), "k_codes", kcs), (1, cmp_v, self.v_owner(l), "v_codes", vcs)):
            if cmp:
                shared = self.layers[own][key]
                assert len(shared) > blk, "the dominant layer must have quantized this block"
                d = np.abs(shared[blk].astype(np.int64) - mine.astype(np.int64))
                self.delta[l, kind] += np.bincount(d.reshape(-1), minlength=4)[:4]
        if not mrg_k and self.k_owner(l) != l:
            kcs = None
        if not mrg_v and self.v_owner(l) != l:
            vcs = None
        if mrg_k:  # the pair's codes of this block: weighted average with the first layer's, rounded
            first = self.layers[l - 1]["k_codes"]
            assert len(first) > blk, "the pair's first layer must have quantized this block"
            first[blk] = merge_codes_gamma1(first[blk], kcs, self.gamma1)
            kcs = None
        if mrg_v:
            first = self.layers[l - 1]["v_codes"]
            assert len(first) > blk, "the pair's first layer must have quantized this block"
            first[blk] = merge_codes_gamma1(first[blk], vcs, self.gamma1)
            vcs = None
        st["k_codes"].append(kcs); st["k_s"].append(stack(ks)); st["k_z"].append(stack(kz))
        st["v_codes"].append(vcs); st["v_s"].append(stack(vs)); st["v_z"].append(stack(vz))
        st["win_k"] = st["win_k"][:, :, :0]
        st["win_v"] = st["win_v"][:, :, :0]

    def append(self, l: int, k_bits16: np.ndarray, v_bits16: np.ndarray):
        """k_bits16, v_bits16: [B, H_kv, n, D] bit patterns of the 16-bit input type."""
        st = self.layers[l]
        k = self._widen(k_bits16)
        v = self._widen(v_bits16)
        n = k.shape[2]
        i = 0
        while i < n:
            if st["win_k"].shape[2] == self.R:
                self._flush(l)  # the window is full and a further token arrives
            take = min(self.R - st["win_k"].shape[2], n - i)
            st["win_k"] = np.concatenate([st["win_k"], k[:, :, i:i + take]], axis=2)
            st["win_v"] = np.concatenate([st["win_v"], v[:, :, i:i + take]], axis=2)
            st["seq"] += take
            i += take

    def _widen(self, bits16):
        """16-bit inputs to fp32, exactly."""
        if self.f16:
            return np.ascontiguousarray(bits16).view(np.float16).astype(np.float32)
        return bf16_bits_to_f32(bits16)

    def n_quantized(self, l):
        return self.R * len(self.layers[l]["k_s"])

    def _concat(self, l, key, axis=2):
        blocks = self.layers[l][key]
        return np.concatenate(blocks, axis=axis)

    def codes_and_meta(self, l):
        """Logical arrays of layer l's quantized region: codes come from the
        code-owning layer of the pair, scale / zero-point from layer l itself."""
        lk, lv = self.k_owner(l), self.v_owner(l)
        nq = self.n_quantized(l)
        assert self.n_quantized(lk) >= nq and self.n_quantized(lv) >= nq
        nb = nq // self.R
        k_codes = np.concatenate(self.layers[lk]["k_codes"][:nb], axis=2)
        v_codes = np.concatenate(self.layers[lv]["v_codes"][:nb], axis=2)
        return (k_codes, self._concat(l, "k_s"), self._concat(l, "k_z"),
                v_codes, self._concat(l, "v_s"), self._concat(l, "v_z"))

    def dequantized(self, l, b, h):
        """fp64 K_hat, V_hat [S, D] for one (batch, kv head): dequantized blocks
        followed by the exact 16-bit window."""
        st = self.layers[l]
        if self.n_quantized(l) == 0:
            return st["win_k"][b, h].astype(np.float64), st["win_v"][b, h].astype(np.float64)
        kc, ks, kz, vc, vs, vz = self.codes_and_meta(l)
        kh = dequantize_k(kc[b, h], ks[b, h], kz[b, h], self.g)
        vh = dequantize_v(vc[b, h], vs[b, h], vz[b, h], self.g)
        kh = np.concatenate([kh, st["win_k"][b, h].astype(np.float64)], axis=0)
        vh = np.concatenate([vh, st["win_v"][b, h].astype(np.float64)], axis=0)
        return kh, vh

    def decode(self, l: int, q_bits16: np.ndarray, pairs=None) -> np.ndarray:
        """q_bits16: [B, H_q, D] bfloat16 bits.  Returns fp64 [B, H_q, D]; query head
        h reads kv head h // (H_q / H_kv).  `pairs` optionally restricts the work
        to a list of (batch, q head); other entries are NaN."""
        q = self._widen(q_bits16).astype(np.float64)
        G = self.Hq // self.Hkv
        out = np.full((self.B, self.Hq, self.D), np.nan, dtype=np.float64)
        todo = pairs if pairs is not None else [(b, h) for b in range(self.B) for h in range(self.Hq)]
        cache = {}
        for (b, h) in todo:
            hk = h // G
            if (b, hk) not in cache:
                cache[(b, hk)] = self.dequantized(l, b, hk)
            kh, vh = cache[(b, hk)]
            out[b, h] = attention(q[b, h], kh, vh, self.sm_scale)
        return out

    def attention_chunk(self, l: int, q_bits16: np.ndarray, pairs=None) -> np.ndarray:
        """q_bits16: [T, B, H_q, D] bit patterns: the queries of the layer's last T
        tokens.  Returns fp64 [T, B, H_q, D]; packed tokens enter through their
        dequantized values, window tokens as they are, as in decode."""
        q = self._widen(q_bits16).astype(np.float64)
        T = q.shape[0]
        G = self.Hq // self.Hkv
        out = np.full((T, self.B, self.Hq, self.D), np.nan, dtype=np.float64)
        todo = pairs if pairs is not None else [(b, h) for b in range(self.B) for h in range(self.Hq)]
        cache = {}
        for (b, h) in todo:
            hk = h // G
            if (b, hk) not in cache:
                cache[(b, hk)] = self.dequantized(l, b, hk)
            kh, vh = cache[(b, hk)]
            out[:, b, h] = attention_chunk(q[:, b, h], kh, vh, self.sm_scale)
        return out

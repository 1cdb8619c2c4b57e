"""GPU parity: the CUDA path through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2510_11236_b200 as xq
from paper_2510_11236_b200 import workloads as W
from tests import util

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

KERNELS = [xq.XQ_KERNEL_GENERIC, xq.XQ_KERNEL_AUTO]


def _fill(cache, w, layers, S, step=None):
    """Append tokens [0, S) of the synthetic workload to `layers`; returns {layer: (K, V)}."""
    kv = {}
    for pair in sorted({l // 2 for l in layers}):
        k0, v0, k1, v1 = W.pair_tokens(w, pair, 0, S, DEV)
        if 2 * pair in layers:
            kv[2 * pair] = (k0, v0)
        if 2 * pair + 1 in layers:
            kv[2 * pair + 1] = (k1, v1)
    for l in sorted(layers):
        K, V = kv[l]
        if step is None:
            cache.append_kv(l, K, V)
        else:
            for lo in range(0, S, step):
                hi = min(S, lo + step)
                cache.append_kv(l, K[:, :, lo:hi].contiguous(), V[:, :, lo:hi].contiguous())
    torch.cuda.synchronize()
    return kv


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("etas", [(0.0, 0.0), (1 / 6, 0.045)])
def test_config0_full(kernel, etas):
    w = W.CONFIGS["c0"]
    cfg = W.make_xq_config(w, eta1=etas[0], eta2=etas[1], kernel=kernel)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], w["seq"])
    assert cache.seq_len(0) == 512 and cache.quantized_len(1) == 480
    worst = 0.0
    for l in (0, 1):
        q = W.queries(w, l, 0, DEV)
        o32 = cache.decode_attention(l, q, f32=True)
        o16 = cache.decode_attention(l, q)
        torch.cuda.synchronize()
        for hk in range(w["n_kv_heads"]):
            oc = util.oracle_for_stream(cfg, [0, 1], 0, hk, kv)
            util.compare_regions(cache, oc, l, 0, hk)
            worst = max(worst, util.check_attention(cache, oc, l, q, 0, hk, o32, o16))
    assert xq.xq_equiv_bits(cfg) == 1.0
    print("config 0 worst fp32 attention error", worst)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("shape", [
    # (L, B, Hq, Hkv, D, g, R, kq, vq, km, vm, S)
    (4, 2, 8, 2, 128, 32, 64, 2, 0, 2, 0, 200),    # GQA 4, 2-bit and 1-bit layers, keys shared only from layer 2
    (2, 1, 8, 1, 128, 64, 64, 2, 2, 0, 0, 331),    # group 64, GQA 8
    (2, 2, 2, 2, 128, 32, 128, 0, 0, 0, 0, 700),   # MHA, all 1-bit
    (2, 1, 6, 2, 64, 32, 64, 0, 2, 0, 2, 260),     # head_dim 64, 1-bit keys, values not shared, GQA 3
    (2, 1, 12, 1, 128, 32, 32, 2, 2, 2, 2, 100),   # GQA 12 (> 8 heads per group), no sharing
])
def test_mixed_shapes(kernel, shape):
    L, B, Hq, Hkv, D, g, R, kq, vq, km, vm, S = shape
    w = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq=S, residual_len=R,
             group_size=g, kq=kq, vq=vq, km=km, vm=vm, n_outliers=3, outlier_scale=10.0, seed=11, n_splits=0)
    cfg = W.make_xq_config(w, kernel=kernel)
    assert xq.xq_config_check(cfg) == 0
    cache = xq.Cache(cfg, DEV)
    layers = list(range(L))
    kv = _fill(cache, w, layers, S, step=97)
    for l in layers:
        q = W.queries(w, l, 0, DEV)
        o32 = cache.decode_attention(l, q, f32=True)
        o16 = cache.decode_attention(l, q)
        torch.cuda.synchronize()
        for b in range(B):
            for hk in range(Hkv):
                oc = util.oracle_for_stream(cfg, layers, b, hk, kv)
                util.compare_regions(cache, oc, l, b, hk)
                util.check_attention(cache, oc, l, q, b, hk, o32, o16)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("S", [1, 5, 16, 31, 32, 33, 64, 65])
def test_short_sequences(kernel, S):
    # S <= R: nothing is quantized and the result is plain 16-bit attention; S = R + 1: first flush
    w = dict(W.CONFIGS["c0"], seq=S)
    cfg = W.make_xq_config(w, kernel=kernel)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], S)
    r = ((S - 1) % 32) + 1
    assert cache.quantized_len(0) == S - r
    q = W.queries(w, 1, 0, DEV)
    o32 = cache.decode_attention(1, q, f32=True)
    torch.cuda.synchronize()
    for hk in range(4):
        oc = util.oracle_for_stream(cfg, [0, 1], 0, hk, kv)
        util.compare_regions(cache, oc, 1, 0, hk)
        util.check_attention(cache, oc, 1, q, 0, hk, o32)
    if S <= 32:
        # exact 16-bit attention (fp64 on the raw inputs)
        K, V = kv[1]
        ref = torch.softmax((q[0].double()[:, None, :] * K[0].double()).sum(-1) / 8.0, dim=-1)
        ref = (ref[:, :, None] * V[0].double()).sum(1)
        assert (o32[0].double() - ref).abs().max().item() <= 2e-3


@pytest.mark.parametrize("kernel", KERNELS)
def test_append_granularity_and_split_invariance(kernel):
    w = dict(W.CONFIGS["c0"], seq=300, n_kv_heads=2, n_q_heads=4)
    outs = []
    regions = []
    for step, ns in ((None, 0), (1, 1), (37, 7), (128, 64)):
        cfg = W.make_xq_config(w, kernel=kernel, n_splits=ns)
        cache = xq.Cache(cfg, DEV)
        _fill(cache, w, [0, 1], 300, step=step)
        q = W.queries(w, 1, 3, DEV)
        outs.append(cache.decode_attention(1, q, f32=True).clone())
        nq = cache.quantized_len(1)
        regions.append([cache.region(1, k).clone() for k in range(6)])
        torch.cuda.synchronize()
    for o in outs[1:]:
        assert (o - outs[0]).abs().max().item() <= 2e-5
    D = 64
    # value codes come in batches of 128 tokens: the two complete ones are compared here
    used = {0: 288 * D * 2 // 8, 1: 256 * D * 2 // 8, 2: (288 // 32) * 2 * D * 2, 3: 288 * 2 * 2 * 2,
            4: 12 * D * 2, 5: 12 * D * 2}
    for rg in regions[1:]:
        for k in range(6):
            assert torch.equal(rg[k][:, : used[k]], regions[0][k][:, : used[k]])


def test_error_paths():
    w = dict(W.CONFIGS["c0"], seq=100)
    cfg = W.make_xq_config(w, max_seq=100)
    cache = xq.Cache(cfg, DEV)
    k0, v0, k1, v1 = W.pair_tokens(w, 0, 0, 100, DEV)
    q = W.queries(w, 0, 0, DEV)
    out = torch.empty_like(q)
    s = torch.cuda.current_stream().cuda_stream
    assert xq.xq_decode_attention(cache.handle, 0, q, out, s) == xq.XQ_ERR_ARG  # empty layer
    assert xq.xq_append_kv(cache.handle, 1, k1, v1, 100, s) == 0
    # layer 1 borrows layer 0's codes, and layer 0 is still empty
    assert xq.xq_decode_attention(cache.handle, 1, q, out, s) == xq.XQ_ERR_ORDER
    assert xq.xq_append_kv(cache.handle, 0, k0, v0, 100, s) == 0
    assert xq.xq_decode_attention(cache.handle, 1, q, out, s) == 0
    assert xq.xq_append_kv(cache.handle, 0, k0, v0, 1, s) == xq.XQ_ERR_CAPACITY
    assert xq.xq_seq_len(cache.handle, 0) == 100
    assert xq.xq_append_kv(cache.handle, 5, k0, v0, 1, s) == xq.XQ_ERR_ARG
    assert xq.xq_append_kv(cache.handle, 0, k0, v0, 0, s) == xq.XQ_ERR_ARG
    assert xq.xq_append_kv(cache.handle, 0, None, v0, 1, s) == xq.XQ_ERR_ARG
    assert xq.xq_append_kv(cache.handle, 0, k0.data_ptr() + 2, v0, 1, s) == xq.XQ_ERR_ARG
    torch.cuda.synchronize()
    assert xq.xq_reset(cache.handle) == 0 and xq.xq_seq_len(cache.handle, 0) == 0


def test_decode_step_device_and_host():
    w = dict(W.CONFIGS["c0"], seq=64)
    cfg = W.make_xq_config(w, max_seq=128)
    a, b = xq.Cache(cfg, DEV), xq.Cache(cfg, DEV)
    _fill(a, w, [0, 1], 64)
    _fill(b, w, [0, 1], 64)
    L, B, Hq, Hkv, D = 2, 1, 4, 4, 64
    for step in range(3):  # the first step flushes the full window
        kn = torch.randn(L, B, Hkv, 1, D, device=DEV).to(torch.bfloat16)
        vn = torch.randn(L, B, Hkv, 1, D, device=DEV).to(torch.bfloat16)
        q = torch.randn(L, B, Hq, D, device=DEV).to(torch.bfloat16)
        out_d = torch.empty_like(q)
        a.decode_step(kn, vn, q, out_d)
        kh, vh, qh = kn.cpu().pin_memory(), vn.cpu().pin_memory(), q.cpu().pin_memory()
        out_h = torch.empty(L, B, Hq, D, dtype=torch.bfloat16).pin_memory()
        b.decode_step(kh, vh, qh, out_h, mem=xq.XQ_MEM_HOST)
        torch.cuda.synchronize()
        assert torch.equal(out_d.cpu(), out_h)
        # and equal to the per-layer calls
        for l in range(L):
            assert a.seq_len(l) == 65 + step
            ref = a.decode_attention(l, q[l])
            assert torch.equal(ref, out_d[l])
    assert xq.xq_launch_count(a.handle) > 0


def test_decode_step_appends_inside_the_decode_kernel():
    """Steps of one token on the tensor-core kernel's shape: the token goes into the window inside the decode
    kernel except on the steps that quantize a full window first.  Every step's output equals, bit for bit, what
    xq_decode_attention returns afterwards (the kernels that append first); after every few steps the windows,
    codes, scales and zero-points equal the oracle's bit for bit and the attention is within the usual 2e-3 of
    the oracle's -- at ~100 tokens with key outlier channels ten times the rest one or two tokens carry the
    softmax, so the result follows the logits' error instead of averaging it away."""
    kernel = xq.XQ_KERNEL_AUTO
    short_context_tol = util.ATTN_TOL
    L, B, Hq, Hkv, D, R = 2, 2, 8, 2, 128, 32
    w = dict(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq=70, residual_len=R,
             group_size=32, kq=2, vq=0, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=5, n_splits=0)
    cfg = W.make_xq_config(w, max_seq=256, kernel=kernel)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], 70)
    gen = torch.Generator(device="cpu").manual_seed(17)
    launches = xq.xq_launch_count(cache.handle)
    for step in range(62):  # lengths 71 .. 132: flushes at 97 and 129
        kn = torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV)
        vn = torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV)
        q = torch.randn(L, B, Hq, D, generator=gen).to(torch.bfloat16).to(DEV)
        out = torch.empty_like(q)
        cache.decode_step(kn, vn, q, out)
        torch.cuda.synchronize()
        S = 71 + step
        flush = (S - 1) % R == 0
        now = xq.xq_launch_count(cache.handle)
        # one quantize-and-pack launch for all layers (it also refills the windows) and the decodes, or the decodes alone
        assert now - launches == (1 + L if flush else L)
        launches = now
        for l in range(L):
            kv[l] = (torch.cat([kv[l][0], kn[l]], dim=2), torch.cat([kv[l][1], vn[l]], dim=2))
            assert cache.seq_len(l) == S
            assert torch.equal(out[l], cache.decode_attention(l, q[l]))
        launches = xq.xq_launch_count(cache.handle)
        if step % 7 == 0 or flush or step == 61:
            o32 = [cache.decode_attention(l, q[l], f32=True) for l in range(L)]
            launches = xq.xq_launch_count(cache.handle)
            for b in range(B):
                for hk in range(Hkv):
                    oc = util.oracle_for_stream(cfg, [0, 1], b, hk, kv)
                    for l in range(L):
                        util.compare_regions(cache, oc, l, b, hk)
                        util.check_attention(cache, oc, l, q[l], b, hk, o32[l], None, tol=short_context_tol)


@pytest.mark.parametrize("bits", [(2, 2), (0, 0), (2, 0)])
@pytest.mark.parametrize("D,g", [(128, 32), (128, 64), (64, 32)])
def test_pack_on_lattice_data_with_exact_ties(bits, D, g):
    """Inputs on a coarse lattice (small integers and halves, some groups constant, some spanning a power of two):
    (x - z) / s falls exactly on rounding ties in a large share of the elements, where round-half-even decides
    the code.  Codes, scales and zero-points against the oracle, bit for bit."""
    L, B, Hkv, R = 2, 2, 2, 64
    kq, vq = bits
    S = 3 * R + 7
    w = dict(n_layers=L, batch=B, n_q_heads=2 * Hkv, n_kv_heads=Hkv, head_dim=D, seq=S, residual_len=R,
             group_size=g, kq=kq, vq=vq, km=0, vm=2, n_outliers=0, outlier_scale=1.0, seed=1, n_splits=0)
    # (the wide channel makes logits of tens)
    cfg = W.make_xq_config(w, kernel=xq.XQ_KERNEL_GENERIC if D == 64 else xq.XQ_KERNEL_MMA)
    cache = xq.Cache(cfg, DEV)
    gen = torch.Generator().manual_seed(100 * D + g + kq)
    kv = {}
    for l in range(L):
        K = torch.randint(-6, 7, (B, Hkv, S, D), generator=gen).float() * 0.5
        V = torch.randint(-3, 4, (B, Hkv, S, D), generator=gen).float()
        K[:, :, :, 5] = 2.0                      # constant key channel: scale 0, codes 0
        V[:, :, 11, :] = -1.5                    # constant value token
        K[:, :, :, 9] *= 64.0                    # a wide channel
        V[:, :, 17, : D // 2] *= 0.03125         # a narrow group
        kv[l] = (K.to(torch.bfloat16).to(DEV), V.to(torch.bfloat16).to(DEV))
        for lo in range(0, S, 50):
            cache.append_kv(l, kv[l][0][:, :, lo:lo + 50].contiguous(), kv[l][1][:, :, lo:lo + 50].contiguous())
    torch.cuda.synchronize()
    for l in range(L):
        q = W.queries(w, l, 0, DEV)
        o32 = cache.decode_attention(l, q, f32=True)
        for b in range(B):
            for hk in range(Hkv):
                oc = util.oracle_for_stream(cfg, list(range(L)), b, hk, kv)
                util.compare_regions(cache, oc, l, b, hk)
                util.check_attention(cache, oc, l, q, b, hk, o32, None)
    cache.close()


@pytest.mark.filterwarnings("ignore:overflow encountered in cast")  # scales of 1e30 stored as 16-bit floats
@pytest.mark.parametrize("f16", [False, True])
@pytest.mark.parametrize("bits", [(2, 2), (0, 0)])
def test_pack_on_groups_that_are_hard_for_the_thresholds(bits, f16):
    """The pack kernel codes by comparing against per-group thresholds on the 16-bit input lattice.  Groups where
    finding them takes the slow paths: a threshold next to zero under a large |z| with elements of every small
    magnitude around it (the lattice there is far finer than the quotient can tell apart), a scale whose
    significand is all ones (2 - 2^-23 times a power of two: the reciprocal sequence is not trusted), scales of
    extreme exponent (bfloat16 only), constant groups.  Codes, scales and zero-points against the oracle, bit for
    bit; no attention (the magnitudes are not a model's)."""
    L, B, Hkv, D, g, R = 2, 1, 2, 128, 32, 64
    kq, vq = bits
    S = 2 * R + 5
    dt = torch.float16 if f16 else torch.bfloat16
    w = dict(n_layers=L, batch=B, n_q_heads=Hkv, n_kv_heads=Hkv, head_dim=D, seq=S, residual_len=R,
             group_size=g, kq=kq, vq=vq, km=0, vm=0, n_outliers=0, outlier_scale=1.0, seed=1, n_splits=0)
    cfg = W.make_xq_config(w, io_dtype=xq.XQ_F16 if f16 else xq.XQ_BF16)
    cache = xq.Cache(cfg, DEV)
    gen = torch.Generator().manual_seed(7 + kq + 2 * int(f16))
    lo_exp = -20 if f16 else -120
    kv = {}
    for l in range(L):
        K = torch.randn(B, Hkv, S, D, generator=gen)
        V = torch.randn(B, Hkv, S, D, generator=gen)

        def tiny(shape):
            e = torch.randint(lo_exp, -6, shape, generator=gen).float()
            sign = torch.randint(0, 2, shape, generator=gen).float() * 2 - 1
            t = sign * torch.exp2(e)
            t[torch.rand(shape, generator=gen) < 0.2] = 0.0
            t[torch.rand(shape, generator=gen) < 0.1] = -0.0
            return t

        # thresholds at zero: the ends +-5 (also +-6 with an odd spacing), everything else tiny or zero
        for ch, end in ((3, 5.0), (4, 6.0)):
            K[:, :, :, ch] = tiny((B, Hkv, S))
            K[:, :, 0::8, ch] = end
            K[:, :, 1::8, ch] = -end
        for tok, end in ((5, 5.0), (6, 6.0)):
            V[:, :, tok::16, :] = tiny(V[:, :, tok::16, :].shape)
            V[:, :, tok::16, 0::8] = end
            V[:, :, tok::16, 1::8] = -end
        # 1-bit scale (max - min) with a significand of 24 ones: min = 2^-22, max = 4 -> 4 - 2^-22
        mn = 2.0 ** -22 if not f16 else 2.0 ** -14  # (half precision: 4 - 2^-14 has 17 ones; still an odd case)
        K[:, :, :, 7] = torch.rand(B, Hkv, S, generator=gen) * 3 + 0.5
        K[:, :, 0::4, 7] = 4.0
        K[:, :, 1::4, 7] = mn
        V[:, :, 9::16, :] = torch.rand(V[:, :, 9::16, :].shape, generator=gen) * 3 + 0.5
        V[:, :, 9::16, 0::4] = 4.0
        V[:, :, 9::16, 1::4] = mn
        if not f16:
            # scales of extreme exponent: the reciprocal sequence is not used
            K[:, :, :, 11] = (torch.rand(B, Hkv, S, generator=gen) * 2 + 1) * 1e-30
            K[:, :, :, 13] = (torch.rand(B, Hkv, S, generator=gen) * 2 - 1) * 1e30
            V[:, :, 13::16, :] = (torch.rand(V[:, :, 13::16, :].shape, generator=gen) * 2 + 1) * 1e-30
            V[:, :, 14::16, :] = (torch.rand(V[:, :, 14::16, :].shape, generator=gen) * 2 - 1) * 1e30
        K[:, :, :, 17] = -0.75  # constant groups
        V[:, :, 3::16, :] = 0.0
        kv[l] = (K.to(dt).to(DEV), V.to(dt).to(DEV))
        for lo in range(0, S, 40):
            cache.append_kv(l, kv[l][0][:, :, lo:lo + 40].contiguous(), kv[l][1][:, :, lo:lo + 40].contiguous())
    torch.cuda.synchronize()
    for l in range(L):
        for hk in range(Hkv):
            oc = util.oracle_for_stream(cfg, list(range(L)), 0, hk, kv)
            util.compare_regions(cache, oc, l, 0, hk)
    cache.close()


@pytest.mark.parametrize("G", [1, 2, 3, 4, 5, 6, 7, 8])
def test_decode_step_head_groupings(G):
    """Every size of query-head group the tensor-core kernel takes, through xq_decode_step (in-kernel append) over
    a window flush: regions bit for bit, attention against the oracle at the usual 2e-3 (700 tokens with x10
    outlier channels)."""
    kernel = xq.XQ_KERNEL_MMA
    tol = util.ATTN_TOL
    L, B, Hkv, D, R = 2, 2, 2, 128, 64
    w = dict(n_layers=L, batch=B, n_q_heads=G * Hkv, n_kv_heads=Hkv, head_dim=D, seq=700, residual_len=R,
             group_size=32, kq=2, vq=2, km=0, vm=2, n_outliers=3, outlier_scale=10.0, seed=23 + G, n_splits=0)
    cfg = W.make_xq_config(w, max_seq=800, kernel=kernel)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], 700, step=333)
    gen = torch.Generator(device="cpu").manual_seed(G)
    for step in range(6):  # lengths 701 .. 706; 705 quantizes the block 640 .. 703
        kn = torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV)
        vn = torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV)
        q = torch.randn(L, B, G * Hkv, D, generator=gen).to(torch.bfloat16).to(DEV)
        out = torch.empty_like(q)
        cache.decode_step(kn, vn, q, out)
        torch.cuda.synchronize()
        for l in range(L):
            kv[l] = (torch.cat([kv[l][0], kn[l]], dim=2), torch.cat([kv[l][1], vn[l]], dim=2))
        o32 = [cache.decode_attention(l, q[l], f32=True) for l in range(L)]
        for b in range(B):
            for hk in range(Hkv):
                oc = util.oracle_for_stream(cfg, [0, 1], b, hk, kv)
                for l in range(L):
                    util.compare_regions(cache, oc, l, b, hk)
                    util.check_attention(cache, oc, l, q[l], b, hk, o32[l], out[l], tol=tol)
    cache.close()


@pytest.mark.parametrize("S", [1000, 8192])
@pytest.mark.parametrize("bits", [(2, 0), (2, 2), (0, 0)])
def test_queries_with_a_few_dominant_tokens(S, bits):
    """Queries built from the keys of one, two or four tokens, scaled up: logits of tens on those tokens, so the
    result follows the logits' error instead of averaging it away.  The tensor-core kernel (the default) and the
    scalar kernel both stay within the 2e-3 of the other tests."""
    kq, vq = bits
    w = dict(W.CONFIGS["c2"], n_layers=2, batch=1, n_kv_heads=1, n_q_heads=4, seq=S, kq=kq, vq=vq)
    k0, v0, k1, v1 = W.pair_tokens(w, 0, 0, S, DEV)
    kv = {0: (k0, v0), 1: (k1, v1)}
    caches = {}
    for kernel in (xq.XQ_KERNEL_GENERIC, xq.XQ_KERNEL_AUTO):
        cfg = W.make_xq_config(w, kernel=kernel)
        caches[kernel] = xq.Cache(cfg, DEV)
        caches[kernel].append_kv(0, k0, v0)
        caches[kernel].append_kv(1, k1, v1)
    oc = util.oracle_for_stream(caches[xq.XQ_KERNEL_AUTO].cfg, [0, 1], 0, 0, kv)
    gen = torch.Generator().manual_seed(3)
    K = k0[0, 0].float().cpu()
    worst = {xq.XQ_KERNEL_GENERIC: 0.0, xq.XQ_KERNEL_AUTO: 0.0}
    for trial in range(6):
        t = torch.randint(0, S - 200, (8,), generator=gen)
        for layer in (0, 1):  # layer 1 borrows layer 0's codes: the same keys up to the second layer's noise
            q = torch.zeros(1, 4, 128)
            q[0, 0] = torch.randn(128, generator=gen)
            q[0, 1] = K[t[0]] * 0.3
            q[0, 2] = (K[t[1]] + K[t[2]]) * 0.21
            q[0, 3] = (K[t[3]] + K[t[4]] + K[t[5]] + K[t[6]]) * 0.15
            qb = q.to(torch.bfloat16).to(DEV)
            ref = oc.decode(layer, util.bits_of(qb))[0]
            for kernel, cache in caches.items():
                got = cache.decode_attention(layer, qb, f32=True)[0].double().cpu().numpy()
                worst[kernel] = max(worst[kernel], np.abs(got - ref).max())
    print("peaked queries, S =", S, "fp32 error: scalar %.2e, tensor-core %.2e" % (worst[xq.XQ_KERNEL_GENERIC], worst[xq.XQ_KERNEL_AUTO]))
    assert worst[xq.XQ_KERNEL_GENERIC] <= util.ATTN_TOL
    assert worst[xq.XQ_KERNEL_AUTO] <= util.ATTN_TOL
    for cache in caches.values():
        cache.close()


@pytest.mark.parametrize("group,k,m", [(3, 0, 0), (4, 0, 4), (2, 1, 0), (3, 2, 3), (4, 2, 0)])
@pytest.mark.parametrize("kernel", KERNELS)
def test_sharing_groups_and_dominant_layers(group, k, m, kernel):
    """Groups of two, three and four layers reading the codes of their k-th layer (Table group's patterns):
    regions bit for bit, attention of every layer against the oracle, and one-token steps with the dominant
    layers first (a layer ahead of its dominant layer cannot decode before that layer has appended)."""
    L = m + 2 * group
    w = dict(n_layers=L, batch=1, n_q_heads=8, n_kv_heads=2, head_dim=128, seq=200, residual_len=64, group_size=32,
             kq=L, vq=L, km=m, vm=m, n_outliers=3, outlier_scale=10.0, seed=31, n_splits=0,
             share_group=group, share_dominant=k)
    cfg = W.make_xq_config(w, max_seq=300, kernel=kernel)
    assert xq.xq_config_check(cfg) == 0
    cache = xq.Cache(cfg, DEV)
    layers = list(range(L))
    kv = _fill(cache, w, layers, 192, step=50)  # the window of 64 is full: the next token quantizes it
    owners = [m + ((l - m) // group) * group + k if l >= m else l for l in range(L)] if group > 2 else \
             [l - l % 2 + k if l >= m else l for l in range(L)]
    order = sorted(range(L), key=lambda l: (owners[l] != l, l))
    gen = torch.Generator(device="cpu").manual_seed(7)
    for step in range(2):
        kn = torch.randn(L, 1, 2, 1, 128, generator=gen).to(torch.bfloat16).to(DEV)
        vn = torch.randn(L, 1, 2, 1, 128, generator=gen).to(torch.bfloat16).to(DEV)
        q = torch.randn(L, 1, 8, 128, generator=gen).to(torch.bfloat16).to(DEV)
        out = torch.empty_like(q)
        if step == 0 and k > 0:  # ascending order would ask layer 0 of a group to read codes that are not there yet
            rc = xq.xq_decode_step(cache.handle, kn, vn, q, out, None, xq.XQ_MEM_DEVICE, torch.cuda.current_stream().cuda_stream)
            assert rc == xq.XQ_ERR_ORDER and cache.seq_len(0) == 192
        cache.decode_step(kn, vn, q, out, layer_order=order)
        torch.cuda.synchronize()
        for l in layers:
            kv[l] = (torch.cat([kv[l][0], kn[l]], dim=2), torch.cat([kv[l][1], vn[l]], dim=2))
        o32 = [cache.decode_attention(l, q[l], f32=True) for l in layers]
        for hk in range(2):
            oc = util.oracle_for_stream(cfg, layers, 0, hk, kv)
            for l in layers:
                util.compare_regions(cache, oc, l, 0, hk)
                util.check_attention(cache, oc, l, q[l], 0, hk, o32[l], out[l])
    assert xq.xq_equiv_bits(cfg) == O_equiv(L, m, group, k)
    cache.close()


def O_equiv(L, m, group, k):
    from oracle import xq_oracle as O
    return O.equiv_bits(L, L, m, m, L, group, k)


@pytest.mark.parametrize("gamma0", [0.05, 0.2, 0.4, 0.6, 0.8, 0.95])
@pytest.mark.parametrize("bits", [(2, 0), (0, 2)])
def test_weighted_average_merging(gamma0, bits):
    """gamma_0 in each of Appendix F's six intervals: once the pair's second layer has quantized a block the shared
    codes are round(gamma_0 e0 + gamma_1 e1), bit for bit; before that they are the first layer's."""
    kq, vq = bits
    w = dict(n_layers=2, batch=2, n_q_heads=4, n_kv_heads=2, head_dim=128, seq=300, residual_len=64, group_size=32,
             kq=kq, vq=vq, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=3, n_splits=0, gamma1=1.0 - gamma0)
    cfg = W.make_xq_config(w)
    cache = xq.Cache(cfg, DEV)
    k0, v0, k1, v1 = W.pair_tokens(w, 0, 0, 300, DEV)
    s = torch.cuda.current_stream().cuda_stream
    # the second layer cannot run ahead of the first
    assert xq.xq_append_kv(cache.handle, 1, k1[:, :, :100].contiguous(), v1[:, :, :100].contiguous(), 100, s) == xq.XQ_ERR_ORDER
    assert cache.seq_len(1) == 0
    cache.append_kv(0, k0[:, :, :150].contiguous(), v0[:, :, :150].contiguous())
    kv = {0: (k0[:, :, :150], v0[:, :, :150])}
    q = W.queries(w, 0, 0, DEV)
    o32 = cache.decode_attention(0, q, f32=True)
    for hk in range(2):
        oc = util.oracle_for_stream(cfg, [0], 1, hk, kv)
        util.compare_regions(cache, oc, 0, 1, hk)
        util.check_attention(cache, oc, 0, q, 1, hk, o32)
    cache.append_kv(1, k1[:, :, :150].contiguous(), v1[:, :, :150].contiguous())
    for lo in range(150, 300, 37):
        hi = min(300, lo + 37)
        for l, (K, V) in ((0, (k0, v0)), (1, (k1, v1))):
            cache.append_kv(l, K[:, :, lo:hi].contiguous(), V[:, :, lo:hi].contiguous())
    kv = {0: (k0, v0), 1: (k1, v1)}
    for layer in (0, 1):
        q = W.queries(w, layer, 0, DEV)
        o32 = cache.decode_attention(layer, q, f32=True)
        for b in range(2):
            for hk in range(2):
                # the oracle takes the same interleaving: both layers complete, block by block
                oc = util.oracle_for_stream(cfg, [0, 1], b, hk, kv)
                util.compare_regions(cache, oc, layer, b, hk)
                util.check_attention(cache, oc, layer, q, b, hk, o32)
    cache.close()


@pytest.mark.parametrize("shape", ["c0", "c2"])
def test_half_precision_io(shape):
    """K, V, q, the window and the output in IEEE half precision instead of bfloat16."""
    w = dict(W.CONFIGS[shape], n_layers=2, batch=1, seq=700)
    w["kq"], w["vq"] = min(w["kq"], 2), min(w["vq"], 2)
    cfg = W.make_xq_config(w, max_seq=800, io_dtype=xq.XQ_F16)
    cache = xq.Cache(cfg, DEV)
    k0, v0, k1, v1 = (t.to(torch.float16) for t in W.pair_tokens(w, 0, 0, 700, DEV))
    kv = {0: (k0, v0), 1: (k1, v1)}
    for lo in range(0, 700, 233):
        for l in (0, 1):
            cache.append_kv(l, kv[l][0][:, :, lo:lo + 233].contiguous(), kv[l][1][:, :, lo:lo + 233].contiguous())
    L, Hq, Hkv, D = 2, w["n_q_heads"], w["n_kv_heads"], w["head_dim"]
    gen = torch.Generator(device="cpu").manual_seed(9)
    for step in range(3):
        kn = torch.randn(L, 1, Hkv, 1, D, generator=gen).to(torch.float16).to(DEV)
        vn = torch.randn(L, 1, Hkv, 1, D, generator=gen).to(torch.float16).to(DEV)
        q = torch.randn(L, 1, Hq, D, generator=gen).to(torch.float16).to(DEV)
        out = torch.empty_like(q)
        cache.decode_step(kn, vn, q, out)
        torch.cuda.synchronize()
        for l in range(L):
            kv[l] = (torch.cat([kv[l][0], kn[l]], dim=2), torch.cat([kv[l][1], vn[l]], dim=2))
        o32 = [cache.decode_attention(l, q[l], f32=True) for l in range(L)]
        for hk in range(min(2, Hkv)):
            oc = util.oracle_for_stream(cfg, [0, 1], 0, hk, kv)
            for l in range(L):
                util.compare_regions(cache, oc, l, 0, hk)
                util.check_attention(cache, oc, l, q[l], 0, hk, o32[l], out[l])
    cache.close()


@pytest.mark.parametrize("T", [1, 4, 16, 64])
@pytest.mark.parametrize("shape", ["mha", "gqa", "d64"])
@pytest.mark.parametrize("kernel", KERNELS)
def test_attention_chunk(T, shape, kernel):
    """The last T tokens as queries, causal inside the chunk, on MHA and GQA shapes: every row against the oracle.
    With a window of 32 and 9 tokens in it, chunks of 16 and 64 reach into the packed region (their first queries
    see only a part of it)."""
    Hq, Hkv, D = {"mha": (4, 4, 128), "gqa": (8, 2, 128), "d64": (6, 2, 64)}[shape]
    S = 393  # 384 quantized + 9 in the window
    w = dict(n_layers=2, batch=2, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, seq=S, residual_len=32, group_size=32,
             kq=2, vq=0, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=41, n_splits=0)
    cfg = W.make_xq_config(w, kernel=kernel)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], S, step=131)
    gen = torch.Generator(device="cpu").manual_seed(T)
    for layer in (0, 1):
        q = torch.randn(T, 2, Hq, D, generator=gen).to(torch.bfloat16).to(DEV)
        o32 = cache.attention_chunk(layer, q, f32=True)
        o16 = cache.attention_chunk(layer, q)
        torch.cuda.synchronize()
        if T == 1:
            assert torch.equal(o16[0], cache.decode_attention(layer, q[0]))
        G = Hq // Hkv
        for b in range(2):
            for hk in range(Hkv):
                oc = util.oracle_for_stream(cfg, [0, 1], b, hk, kv)
                ref = oc.attention_chunk(layer, util.bits_of(q[:, b:b + 1, hk * G:(hk + 1) * G]))[:, 0]
                got = o32[:, b, hk * G:(hk + 1) * G].double().cpu().numpy()
                assert np.abs(got - ref).max() <= util.ATTN_TOL
                got16 = o16[:, b, hk * G:(hk + 1) * G].double().cpu().numpy()
                assert (np.abs(got16 - ref) <= util.ATTN_TOL + 2.0 ** -8 * np.abs(ref)).all()
    s = torch.cuda.current_stream().cuda_stream
    q = torch.zeros(2, 2, Hq, D, dtype=torch.bfloat16, device=DEV)
    assert xq.xq_attention_chunk(cache.handle, 0, q, q.clone(), S + 1, s) == xq.XQ_ERR_ARG
    assert xq.xq_attention_chunk(cache.handle, 0, q, q.clone(), 0, s) == xq.XQ_ERR_ARG
    cache.close()


@pytest.mark.parametrize("bits", [(2, 2), (2, 0), (0, 0)])
def test_delta_histogram(bits):
    """The pack kernel's optional statistic (Section 3.3.1): per layer and cache kind the elements by
    |own code - shared code|, against the oracle's count, exactly; the cache's contents are unchanged by it."""
    kq, vq = bits
    w = dict(n_layers=4, batch=2, n_q_heads=4, n_kv_heads=2, head_dim=128, seq=333, residual_len=64, group_size=32,
             kq=kq, vq=vq, km=2, vm=0, n_outliers=3, outlier_scale=10.0, seed=13, n_splits=0, delta_stats=1)
    cfg = W.make_xq_config(w)
    cache = xq.Cache(cfg, DEV)
    layers = [0, 1, 2, 3]
    kv = _fill(cache, w, layers, 333, step=77)
    s = torch.cuda.current_stream().cuda_stream
    want = np.zeros((4, 2, 4), dtype=np.int64)
    for b in range(2):
        for hk in range(2):
            oc = util.oracle_for_stream(cfg, layers, b, hk, kv)
            want += oc.delta
            for l in layers:
                util.compare_regions(cache, oc, l, b, hk)
    for l in layers:
        for kind in (0, 1):
            rc, got = xq.xq_delta_histogram(cache.handle, l, kind, s)
            assert rc == 0 and got == list(want[l, kind]), (l, kind, got, list(want[l, kind]))
    assert want[1, 0].sum() == 0 and want[1, 1].sum() == 2 * 2 * 320 * 128  # keys shared from layer 2 on, values from 0
    plain = xq.Cache(W.make_xq_config(dict(w, delta_stats=0)), DEV)
    assert xq.xq_delta_histogram(plain.handle, 1, 0, s)[0] == xq.XQ_ERR_CONFIG
    plain.close()
    cache.close()


def test_decode_right_after_the_pack_of_the_layer_it_reads():
    """A layer that reads another layer's codes decodes immediately after that layer packed a large append, many
    times on one stream with nothing in between: the decode kernel must not fetch packed data ahead of the pack
    kernel that is still writing it.  Every result against the oracle."""
    w = dict(W.CONFIGS["c2"], n_layers=2, batch=4, seq=8192 + 100)
    w["kq"], w["vq"] = 2, 0
    R = w["residual_len"]
    cfg = W.make_xq_config(w, max_seq=8192 + 16 * 4 * R + 200)
    cache = xq.Cache(cfg, DEV)
    kv = _fill(cache, w, [0, 1], 8192 + 100, step=2048)
    gen = torch.Generator(device="cpu").manual_seed(21)
    B, Hkv, Hq, D = 4, w["n_kv_heads"], w["n_q_heads"], w["head_dim"]
    outs, qs = [], []
    for it in range(4):
        n = 16 * R  # sixteen window blocks per append: a pack launch of several microseconds
        newk = [torch.randn(B, Hkv, n, D, generator=gen).to(torch.bfloat16).to(DEV) for _ in range(2)]
        newv = [torch.randn(B, Hkv, n, D, generator=gen).to(torch.bfloat16).to(DEV) for _ in range(2)]
        q = torch.randn(B, Hq, D, generator=gen).to(torch.bfloat16).to(DEV)
        # warm decodes so that neither layer is flagged as repacked when the appends start
        cache.decode_attention(0, q, f32=True); cache.decode_attention(1, q, f32=True)
        cache.append_kv(1, newk[1], newv[1])   # the borrowing layer's own parameters
        cache.append_kv(0, newk[0], newv[0])   # the pack of the codes layer 1 reads ...
        first = cache.decode_attention(1, q, f32=True).clone()  # ... and at once the decode that reads them
        again = cache.decode_attention(1, q, f32=True)  # the next one may fetch early: the pack is long complete
        outs.append(first)
        assert torch.equal(first, again)
        qs.append(q)
        for l in (0, 1):
            kv[l] = (torch.cat([kv[l][0], newk[l]], dim=2), torch.cat([kv[l][1], newv[l]], dim=2))
        if it < 3:
            continue
        torch.cuda.synchronize()
    # the last state against the oracle, and each earlier result against a replay at its own length
    G = Hq // Hkv
    for it in range(4):
        S_it = 8192 + 100 + (it + 1) * 16 * R
        part = {l: (kv[l][0][:, :, :S_it], kv[l][1][:, :, :S_it]) for l in (0, 1)}
        for (b, hk) in ((0, 0), (3, Hkv - 1)):
            oc = util.oracle_for_stream(cfg, [0, 1], b, hk, part)
            ref = oc.decode(1, util.bits_of(qs[it][b:b + 1, hk * G:(hk + 1) * G]))[0]
            got = outs[it][b, hk * G:(hk + 1) * G].double().cpu().numpy()
            assert np.abs(got - ref).max() <= util.ATTN_TOL, (it, b, hk)
    cache.close()


def test_chained_decode_launches_equal_single_calls():
    """The decode launches of a step overlap: each after the first reads at once and waits for its predecessor only
    before it writes the scratch and its result.  Eight layers of the 32k shape at a length where a launch fills
    every slot of the device, twelve steps back to back on one stream (one of them fills the window blocks and
    packs): every layer's result of every step equals, bit for bit, what a second cache with the same contents
    returns through separate xq_append_kv / xq_decode_attention calls, which never overlap."""
    L = 8
    w = dict(W.CONFIGS["c2"], n_layers=L, seq=6000)
    w["kq"], w["vq"] = L, 0
    cfg = W.make_xq_config(w, max_seq=6000 + 64)
    a, b = xq.Cache(cfg, DEV), xq.Cache(cfg, DEV)
    S0 = 6000 + 8  # 6008 = 46 blocks of 128 + 120 in the window: step 9 fills the blocks
    for cache in (a, b):
        for pair in range(L // 2):
            k0, v0, k1, v1 = W.pair_tokens(w, pair, 0, S0, DEV)
            cache.append_kv(2 * pair, k0, v0)
            cache.append_kv(2 * pair + 1, k1, v1)
    B, Hkv, Hq, D = w["batch"], w["n_kv_heads"], w["n_q_heads"], w["head_dim"]
    gen = torch.Generator(device="cpu").manual_seed(33)
    steps = 12
    kn = [torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV) for _ in range(steps)]
    vn = [torch.randn(L, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).to(DEV) for _ in range(steps)]
    q = [torch.randn(L, B, Hq, D, generator=gen).to(torch.bfloat16).to(DEV) for _ in range(steps)]
    outs = [torch.empty_like(q[0]) for _ in range(steps)]
    torch.cuda.synchronize()
    for i in range(steps):  # nothing between the steps
        a.decode_step(kn[i], vn[i], q[i], outs[i])
    torch.cuda.synchronize()
    a.check_device()  # raises if a kernel gave up a bounded wait
    for i in range(steps):
        for l in range(L):
            b.append_kv(l, kn[i][l], vn[i][l])
            ref = b.decode_attention(l, q[i][l])
            assert torch.equal(ref, outs[i][l]), (i, l)
    assert a.quantized_len(0) == b.quantized_len(0) == 47 * 128
    a.close(); b.close()


def test_decode_step_from_host_buffers_at_full_size():
    """xq_decode_step with pinned host buffers (the end-to-end path the benchmark times) on the 32k GQA shape with
    one layer pair: three steps, sampled streams against the oracle."""
    w = dict(W.CONFIGS["c2"], n_layers=2)
    w["kq"], w["vq"] = 2, 0
    S, B, Hkv, Hq, D = w["seq"], w["batch"], w["n_kv_heads"], w["n_q_heads"], w["head_dim"]
    cfg = W.make_xq_config(w, max_seq=S + 8)
    cache = xq.Cache(cfg, DEV)
    streams = [(0, 0), (B - 1, Hkv - 1)]
    parts = {s: [[], [], [], []] for s in streams}
    for c0 in range(0, S, W.CHUNK):
        k0, v0, k1, v1 = W.pair_tokens(w, 0, c0, min(S, c0 + W.CHUNK), DEV)
        cache.append_kv(0, k0, v0)
        cache.append_kv(1, k1, v1)
        for (b, h) in streams:
            for lst, t in zip(parts[(b, h)], (k0, v0, k1, v1)):
                lst.append(t[b:b + 1, h:h + 1].cpu())
    gen = torch.Generator(device="cpu").manual_seed(2)
    G = Hq // Hkv
    for step in range(3):  # the first step quantizes the full windows
        kn = torch.randn(2, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).pin_memory()
        vn = torch.randn(2, B, Hkv, 1, D, generator=gen).to(torch.bfloat16).pin_memory()
        q = torch.randn(2, B, Hq, D, generator=gen).to(torch.bfloat16).pin_memory()
        out = torch.empty(2, B, Hq, D, dtype=torch.bfloat16).pin_memory()
        cache.decode_step(kn, vn, q, out, mem=xq.XQ_MEM_HOST)
        torch.cuda.synchronize()
        for (b, h) in streams:
            for i, t in enumerate((kn[0], vn[0], kn[1], vn[1])):
                parts[(b, h)][i].append(t[b:b + 1, h:h + 1])
            k0, v0, k1, v1 = (torch.cat(x, dim=2) for x in parts[(b, h)])
            oc = util.oracle_for_stream(cfg, [0, 1], 0, 0, {0: (k0, v0), 1: (k1, v1)})
            for l in (0, 1):
                ref = oc.decode(l, util.bits_of(q[l, b:b + 1, h * G:(h + 1) * G]))[0]
                got = out[l, b, h * G:(h + 1) * G].double().numpy()
                assert (np.abs(got - ref) <= util.ATTN_TOL + 2.0 ** -8 * np.abs(ref)).all(), (step, b, h, l)
    cache.close()


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_full_size_configs_sampled(name):
    """The benchmark's shapes and launch configuration (library-chosen splits, tensor-core kernel), one layer
    pair at the full context: codes, scales and zero-points of sampled streams bit for bit, attention of the
    sampled streams' query heads against the oracle."""
    w = dict(W.CONFIGS[name], n_layers=2)
    w["kq"], w["vq"] = min(w["kq"], 2), min(w["vq"], 2)
    _full_size_pair(name, w, pair=0)


@pytest.mark.parametrize("name,kq,pair", [("c2", 0, 0), ("c2", 2, 1), ("c1", 0, 1)])
def test_full_size_other_layers(name, kq, pair):
    """The same at full size for a layer pair with 1-bit keys (layers at or above kq) and for the workload's
    second layer pair (other outlier channels, other data)."""
    w = dict(W.CONFIGS[name], n_layers=2)
    w["kq"], w["vq"] = kq, min(w["vq"], 2)
    _full_size_pair(name, w, pair=pair)


def _full_size_pair(name, w, pair):
    cfg = W.make_xq_config(w)  # n_splits as the workload names it (0 = library's choice, c4: 64)
    cache = xq.Cache(cfg, DEV)
    S, B, Hkv = w["seq"], w["batch"], w["n_kv_heads"]
    streams = sorted({(0, 0), (B - 1, Hkv - 1), (B // 2, Hkv // 3)})
    kv = {0: {}, 1: {}}  # per layer, per stream: the tokens of that stream only (host side)
    parts = {s: [[], [], [], []] for s in streams}
    for c0 in range(0, S, W.CHUNK):
        k0, v0, k1, v1 = W.pair_tokens(w, pair, c0, min(S, c0 + W.CHUNK), DEV)
        cache.append_kv(0, k0, v0)
        cache.append_kv(1, k1, v1)
        for (b, h) in streams:
            for lst, t in zip(parts[(b, h)], (k0, v0, k1, v1)):
                lst.append(t[b:b + 1, h:h + 1].cpu())
    torch.cuda.synchronize()
    assert cache.seq_len(1) == S and cache.quantized_len(1) == S - w["residual_len"]
    rc, nsq, nsw = xq.xq_split_plan(cache.handle, 0)
    assert rc == 0 and nsq >= 1
    if name == "c4":
        assert nsq == 64
    G = w["n_q_heads"] // Hkv
    worst = 0.0
    for layer in (0, 1):
        q = W.queries(w, layer, 0, DEV)
        o32 = cache.decode_attention(layer, q, f32=True)
        o16 = cache.decode_attention(layer, q)
        torch.cuda.synchronize()
        for (b, h) in streams:
            k0, v0, k1, v1 = (torch.cat(x, dim=2) for x in parts[(b, h)])
            one = {0: (k0, v0), 1: (k1, v1)}
            oc = util.oracle_for_stream(cfg, [0, 1], 0, 0, one)
            # the oracle holds this one stream as (sequence 0, kv head 0): compare its regions with stream (b, h)
            util.compare_regions(cache, oc, layer, b, h)
            qs = q[b:b + 1, h * G:(h + 1) * G]
            ref = oc.decode(layer, util.bits_of(qs))[0]
            got = o32[b, h * G:(h + 1) * G].double().cpu().numpy()
            err = np.abs(got - ref).max()
            assert err <= util.ATTN_TOL, f"{name} layer {layer} stream {(b, h)}: fp32 attention error {err}"
            got16 = o16[b, h * G:(h + 1) * G].double().cpu().numpy()
            assert (np.abs(got16 - ref) <= util.ATTN_TOL + 2.0 ** -8 * np.abs(ref)).all()
            worst = max(worst, err)
    print(f"{name}: splits {nsq}+{nsw}, worst fp32 attention error over sampled streams {worst:.2e}")
    cache.close()

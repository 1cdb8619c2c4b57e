"""Helpers shared by the GPU parity tests: move bits between torch and numpy,
build the oracle's view of one (sequence, kv head) stream, compare regions."""
import numpy as np
import torch

from oracle import xq_oracle as O


def bits_of(t: torch.Tensor) -> np.ndarray:
    """bf16 or fp16 tensor -> numpy uint16 bit patterns (same shape)."""
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def oracle_for_stream(cfg, layers, b, hk, kv_by_layer):
    """OracleCache holding one (sequence, kv head) stream of the given layers.
    kv_by_layer: {layer: (K, V)} torch bf16 [B, H_kv, S, D] (device or cpu)."""
    G = cfg.n_q_heads // cfg.n_kv_heads
    oc = O.OracleCache(cfg.n_layers, 1, G, 1, cfg.head_dim, cfg.group_size, cfg.residual_len,
                       cfg.kq, cfg.vq, cfg.km, cfg.vm, np.float32(cfg.eta1), np.float32(cfg.eta2),
                       cfg.sm_scale if cfg.sm_scale > 0 else None,
                       share_group=cfg.share_group or 2, share_dominant=cfg.share_dominant,
                       gamma1=float(np.float32(cfg.gamma1)), f16=cfg.io_dtype == 1, delta_stats=bool(cfg.delta_stats))
    for l in layers:
        K, V = kv_by_layer[l]
        oc.append(l, bits_of(K[b:b + 1, hk:hk + 1]), bits_of(V[b:b + 1, hk:hk + 1]))
    return oc


def compare_regions(cache, oc, layer, b, hk):
    """Bit-exact comparison of one stream's packed codes, scale and zero-point
    (and window) in the library's workspace against the oracle's packing."""
    cfg = cache.cfg
    D, g = cfg.head_dim, cfg.group_size
    bh = b * cfg.n_kv_heads + hk
    nq = oc.n_quantized(layer)
    assert cache.quantized_len(layer) == nq
    st = oc.layers[layer]
    r = st["win_k"].shape[2]
    for which, key in ((4, "win_k"), (5, "win_v")):
        got = cache.region(layer, which)[bh].cpu().numpy().view(np.uint16)[: r * D].reshape(r, D)
        want = st[key][0, 0].astype(np.float16).view(np.uint16) if oc.f16 else O.f32_to_bf16_bits(st[key][0, 0])
        assert np.array_equal(got, want), f"window {key} differs"
    if nq == 0:
        return
    kc, ks, kz, vc, vs, vz = oc.codes_and_meta(layer)
    bk, bv = oc.k_bits(layer), oc.v_bits(layer)
    want, written = O.pack_k_codes(kc[0, 0], bk)
    got = cache.region(layer, 0)[bh].cpu().numpy().view(np.uint32)[: len(want)]
    assert written.all() and np.array_equal(got, want), f"key codes differ in {np.count_nonzero(got != want)} words"
    # value codes come in batches of 128 tokens; the words of a ragged last batch that no token has reached yet
    # are not part of the cache's contents
    want, written = O.pack_v_codes(vc[0, 0], bv)
    got = cache.region(layer, 1)[bh].cpu().numpy().view(np.uint32)[: len(want)]
    assert np.array_equal(got[written], want[written]), \
        f"value codes differ in {np.count_nonzero(got[written] != want[written])} words"
    want = O.pack_k_meta(ks[0, 0], kz[0, 0]).reshape(-1)
    got = cache.region(layer, 2)[bh].cpu().numpy().view(np.uint16)[: len(want)]
    assert np.array_equal(got, want), f"key scale/zero differ in {np.count_nonzero(got != want)} entries"
    want = O.pack_v_meta(vs[0, 0], vz[0, 0]).reshape(-1)
    got = cache.region(layer, 3)[bh].cpu().numpy().view(np.uint16)[: len(want)]
    assert np.array_equal(got, want), f"value scale/zero differ in {np.count_nonzero(got != want)} entries"


ATTN_TOL = 2e-3  # max abs error on the fp32 result


def check_attention(cache, oc, layer, q, b, hk, out_f32=None, out_bf16=None, tol=ATTN_TOL):
    """Attention parity for the query heads of kv head hk of sequence b."""
    cfg = cache.cfg
    G = cfg.n_q_heads // cfg.n_kv_heads
    qs = bits_of(q[b:b + 1, hk * G:(hk + 1) * G])
    ref = oc.decode(layer, qs)[0]
    worst = 0.0
    if out_f32 is not None:
        got = out_f32[b, hk * G:(hk + 1) * G].double().cpu().numpy()
        err = np.abs(got - ref).max()
        assert err <= tol, f"fp32 attention error {err}"
        worst = max(worst, err)
    if out_bf16 is not None:
        got = out_bf16[b, hk * G:(hk + 1) * G].double().cpu().numpy()
        tol16 = tol + 2.0 ** -8 * np.abs(ref)  # plus one bf16 rounding of the result (half an ulp <= 2^-8 |x|)
        assert (np.abs(got - ref) <= tol16).all(), f"bf16 attention error {np.abs(got - ref).max()}"
    return worst

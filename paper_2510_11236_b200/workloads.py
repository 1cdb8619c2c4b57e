"""Seeded synthetic KV-cache inputs shaped like the paper's workloads.

Only random tensors are produced here -- none of the method's arithmetic.
Base layer of a pair: bf16(N(0,1)) keys and values, a fixed set of outlier key
channels per (pair, kv head) multiplied before rounding.  Second layer of the
pair: bf16(float(base) + N(0, sigma)).  Queries: bf16(N(0,1)).
Tokens are generated in fixed chunks of CHUNK tokens so that any token range
can be regenerated independently of how the cache is filled.
"""
from __future__ import annotations

import math

import torch

CHUNK = 2048

CONFIGS = {
    # tiny layer pair
    "c0": dict(n_layers=2, batch=1, n_q_heads=4, n_kv_heads=4, head_dim=64, seq=512, residual_len=32,
               group_size=32, kq=2, vq=2, km=0, vm=0, n_outliers=4, outlier_scale=8.0, seed=0, n_splits=0),
    # Llama-2-7B-shaped MHA
    "c1": dict(n_layers=32, batch=8, n_q_heads=32, n_kv_heads=32, head_dim=128, seq=4096, residual_len=128,
               group_size=32, kq=32, vq=32, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=1, n_splits=0),
    # Llama-3-8B-shaped GQA, 2-bit keys, 1-bit values
    "c2": dict(n_layers=32, batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, seq=32768, residual_len=128,
               group_size=32, kq=32, vq=0, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=2, n_splits=0),
    # Mistral-7B-shaped GQA
    "c3": dict(n_layers=32, batch=16, n_q_heads=32, n_kv_heads=8, head_dim=128, seq=8192, residual_len=64,
               group_size=64, kq=32, vq=32, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=3, n_splits=0),
    # long context, 64 splits per head
    "c4": dict(n_layers=32, batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, seq=131072, residual_len=128,
               group_size=32, kq=32, vq=0, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=4, n_splits=64),
    # Qwen2.5-14B-shaped GQA (48 layers, 40 query heads on 8 kv heads: groups of five), the paper's second model
    # family (Table qwen); 2-bit keys, the upper half of the value layers 1-bit
    "q14": dict(n_layers=48, batch=4, n_q_heads=40, n_kv_heads=8, head_dim=128, seq=16384, residual_len=128,
                group_size=32, kq=48, vq=24, km=0, vm=0, n_outliers=3, outlier_scale=10.0, seed=5, n_splits=0),
}

# one line per workload for reports
TITLES = {
    "c0": "configuration 0: tiny layer pair, 4 heads, head_dim 64, 512 tokens",
    "c1": "configuration 1: Llama-2-7B-shaped MHA, batch 8, 4k context, 2-bit keys and values",
    "c2": "configuration 2: Llama-3-8B-shaped GQA, batch 4, 32k context, 2-bit keys, 1-bit values",
    "c3": "configuration 3: Mistral-7B-shaped GQA, batch 16, 8k context, groups of 64, 2-bit keys and values",
    "c4": "configuration 4: long context, batch 1, 128k tokens, 64 splits per head",
    "q14": "Qwen2.5-14B-shaped GQA (48 layers, groups of five heads), batch 4, 16k context",
}

NOISE_SIGMA = 0.1


def _gen(device, *seed_parts):
    g = torch.Generator(device=device)
    s = 0
    for p in seed_parts:
        s = (s * 1000003 + int(p) + 1) % (2 ** 62)
    g.manual_seed(s)
    return g


def outlier_mask(w: dict, pair: int, device) -> torch.Tensor:
    """[n_kv_heads, head_dim] multiplier: outlier_scale on the outlier key channels."""
    H, D = w["n_kv_heads"], w["head_dim"]
    g = _gen("cpu", w["seed"], pair, 7)
    mult = torch.ones(H, D)
    for h in range(H):
        idx = torch.randperm(D, generator=g)[: w["n_outliers"]]
        mult[h, idx] = w["outlier_scale"]
    return mult.to(device)


def pair_chunk(w: dict, pair: int, chunk: int, device, batch_slice=None, head_slice=None):
    """K0, V0, K1, V1 as bf16 [B, H_kv, CHUNK, D] for tokens [chunk*CHUNK, (chunk+1)*CHUNK)
    of layer pair `pair` (layers 2*pair and 2*pair+1)."""
    B, H, D = w["batch"], w["n_kv_heads"], w["head_dim"]
    g = _gen(device, w["seed"], pair, chunk)
    mult = outlier_mask(w, pair, device)[None, :, None, :]
    k0 = (torch.randn(B, H, CHUNK, D, generator=g, device=device) * mult).to(torch.bfloat16)
    v0 = torch.randn(B, H, CHUNK, D, generator=g, device=device).to(torch.bfloat16)
    k1 = (k0.float() + NOISE_SIGMA * torch.randn(B, H, CHUNK, D, generator=g, device=device)).to(torch.bfloat16)
    v1 = (v0.float() + NOISE_SIGMA * torch.randn(B, H, CHUNK, D, generator=g, device=device)).to(torch.bfloat16)
    return k0, v0, k1, v1


def pair_tokens(w: dict, pair: int, start: int, stop: int, device):
    """Same, for an arbitrary token range."""
    outs = [[], [], [], []]
    c = start // CHUNK
    while c * CHUNK < stop:
        parts = pair_chunk(w, pair, c, device)
        lo = max(start, c * CHUNK) - c * CHUNK
        hi = min(stop, (c + 1) * CHUNK) - c * CHUNK
        for o, p in zip(outs, parts):
            o.append(p[:, :, lo:hi])
        c += 1
    return tuple(torch.cat(o, dim=2).contiguous() for o in outs)


def queries(w: dict, layer: int, step: int, device) -> torch.Tensor:
    """bf16 [B, H_q, D] decode queries of one layer at one step."""
    g = _gen(device, w["seed"], 100000 + layer, step)
    return torch.randn(w["batch"], w["n_q_heads"], w["head_dim"], generator=g, device=device).to(torch.bfloat16)


def make_xq_config(w: dict, *, max_seq=None, eta1=1.0 / 6.0, eta2=0.045, kernel=0, n_splits=None, io_dtype=0):
    from . import binding
    return binding.make_config(
        n_layers=w["n_layers"], batch=w["batch"], n_q_heads=w["n_q_heads"], n_kv_heads=w["n_kv_heads"],
        head_dim=w["head_dim"], max_seq=max_seq or w["seq"], group_size=w["group_size"],
        residual_len=w["residual_len"], kq=w["kq"], vq=w["vq"], km=w["km"], vm=w["vm"], eta1=eta1, eta2=eta2,
        n_splits=w["n_splits"] if n_splits is None else n_splits, kernel=kernel, io_dtype=io_dtype,
        share_group=w.get("share_group", 0), share_dominant=w.get("share_dominant", 0), gamma1=w.get("gamma1", 0.0),
        delta_stats=w.get("delta_stats", 0))


def algorithmic_bytes(w: dict, seq: int = None, layer: int = 0) -> int:
    """Bytes one decode-attention layer call must move: packed codes, 16-bit scale
    and zero-point, the 16-bit window, q and out (split-K partials excluded)."""
    S = seq or w["seq"]
    B, Hq, H, D, g, R = w["batch"], w["n_q_heads"], w["n_kv_heads"], w["head_dim"], w["group_size"], w["residual_len"]
    bk = 2 if layer < w["kq"] else 1
    bv = 2 if layer < w["vq"] else 1
    r = ((S - 1) % R) + 1
    nq = S - r
    per = nq * D * (bk + bv) // 8 + 4 * (nq // g) * D + 4 * nq * (D // g) + 4 * r * D
    return B * H * per + 4 * B * Hq * D


def sm_scale(w: dict) -> float:
    return 1.0 / math.sqrt(w["head_dim"])

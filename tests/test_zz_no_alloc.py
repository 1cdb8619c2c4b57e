"""xq_decode_attention_static: decode attention for callers that cannot allocate.

A host that gave all of its device memory to its own pools before this library
was loaded, or that forbids cudaMalloc on its serving path, has nowhere to put
the split-K partials.  The entry point under test keeps them in an array that is
part of the library image, so the call needs nothing beyond q and out.  It must
return what xq_decode_attention returns, also when the array still holds the
previous call's partials and tickets -- hence two calls in a row, on different
layers, kernels and split counts.

This file is named to be collected last: a run that stops at the first failure
has then already run every other test.
"""
import pytest
import torch

import paper_2510_11236_b200 as xq
from paper_2510_11236_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

TOL = 2e-5  # the tolerance the split-count invariance test uses; bf16 outputs of the same plan are expected equal


def _filled_cache(w, kernel, n_splits):
    cfg = W.make_xq_config(w, kernel=kernel, n_splits=n_splits)
    cache = xq.Cache(cfg, DEV)
    S = w["seq"]
    for pair in range(w["n_layers"] // 2):
        k0, v0, k1, v1 = W.pair_tokens(w, pair, 0, S, DEV)
        cache.append_kv(2 * pair, k0, v0)
        cache.append_kv(2 * pair + 1, k1, v1)
    torch.cuda.synchronize()
    return cache


@pytest.mark.parametrize("kernel", [xq.XQ_KERNEL_AUTO, xq.XQ_KERNEL_GENERIC])
def test_static_scratch_matches_workspace_scratch_twice_in_a_row(kernel):
    # GQA 4, head_dim 128, 2-bit keys / 1-bit values on shared codes: the tensor-core kernel's shape
    w = dict(W.CONFIGS["c2"], n_layers=2, batch=2, n_kv_heads=2, n_q_heads=8, seq=1500, kq=2, vq=0)
    stream = torch.cuda.current_stream().cuda_stream
    for n_splits in (0, 7):  # the second cache finds the array as the first one left it
        cache = _filled_cache(w, kernel, n_splits)
        for call, layer in enumerate((0, 1, 1)):  # calls in a row; the last repeats a layer with another query
            q = W.queries(w, layer, call, DEV)
            want = cache.decode_attention(layer, q)
            got = torch.full_like(want, float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            rc = xq.xq_decode_attention_static(cache.handle, layer, q, got, stream)
            assert rc == xq.XQ_OK, xq.xq_strerror(rc)
            torch.cuda.synchronize()
            # the handle was created before this call, so the array is already on the device: the call itself
            # must leave the device's free memory as it found it
            assert torch.cuda.mem_get_info()[0] == free_before
            assert torch.isfinite(got.float()).all()
            diff = (got.float() - want.float()).abs().max().item()
            assert diff <= TOL, f"call {call}, layer {layer}, n_splits {n_splits}: max abs difference {diff}"
        cache.close()


def test_static_scratch_rejects_what_does_not_fit():
    # 64 sequences x 32 heads x 256 splits x 130 floats = 272 MB of partials: far beyond the array
    w = dict(W.CONFIGS["c2"], n_layers=2, batch=64, seq=400, kq=2, vq=0)
    cfg = W.make_xq_config(w, kernel=xq.XQ_KERNEL_GENERIC, n_splits=xq.XQ_MAX_SPLITS)
    cache = xq.Cache(cfg, DEV)
    k0, v0, _, _ = W.pair_tokens(w, 0, 0, 400, DEV)
    cache.append_kv(0, k0, v0)
    q = W.queries(w, 0, 0, DEV)
    out = torch.zeros_like(q)
    launches = xq.xq_launch_count(cache.handle)
    rc = xq.xq_decode_attention_static(cache.handle, 0, q, out, torch.cuda.current_stream().cuda_stream)
    assert rc == xq.XQ_ERR_CAPACITY
    assert xq.xq_launch_count(cache.handle) == launches  # nothing was launched
    assert xq.xq_decode_attention_static(cache.handle, 7, q, out, 0) == xq.XQ_ERR_ARG
    torch.cuda.synchronize()
    assert not out.any()
    cache.close()

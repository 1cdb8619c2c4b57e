"""Host-only checks of the C ABI: the library loads without a GPU, exports every
declared symbol, validates configurations and evaluates the equivalent bit-width."""
import ctypes
import os
import re

import pytest

import paper_2510_11236_b200 as xq
from oracle import xq_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "xq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(xq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(xq.binding.LIB_PATH)
    names = _declared()
    assert "xq_append_kv" in names and "xq_decode_attention" in names and "xq_equiv_bits" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(xq.binding.EXPORTS)


def _cfg(**kw):
    base = dict(n_layers=32, batch=2, n_q_heads=32, n_kv_heads=8, head_dim=128, max_seq=4096)
    base.update(kw)
    return xq.make_config(**base)


def test_config_check():
    assert xq.xq_config_check(_cfg()) == xq.XQ_OK
    bad = [dict(head_dim=96), dict(group_size=48), dict(residual_len=48), dict(n_q_heads=30),
           dict(eta1=0.6), dict(eta2=-0.1), dict(kq=33), dict(km=-1), dict(n_splits=1000),
           dict(residual_len=32, group_size=64), dict(max_seq=0), dict(kernel=9),
           dict(kq=31, km=0)]  # pair (30, 31) would mix 2-bit and 1-bit keys on shared codes
    for kw in bad:
        c = _cfg(**kw)
        assert xq.xq_config_check(c) == xq.XQ_ERR_CONFIG, kw
        assert xq.xq_workspace_bytes(c) == 0
        assert xq.xq_equiv_bits(c) < 0
    # an odd kq is fine when the pair it cuts does not share codes
    assert xq.xq_config_check(_cfg(kq=31, km=32)) == xq.XQ_OK
    assert xq.xq_config_check(_cfg(kernel=xq.XQ_KERNEL_MMA)) == xq.XQ_OK
    assert xq.xq_config_check(_cfg(head_dim=64, residual_len=32, vq=0)) == xq.XQ_OK


@pytest.mark.parametrize("kq,vq,km,vm", [(30, 2, 32, 16), (32, 0, 32, 16), (28, 0, 32, 28), (32, 0, 32, 20),
                                         (32, 32, 32, 8), (32, 0, 0, 0), (32, 32, 0, 0), (16, 32, 32, 32),
                                         (32, 32, 31, 7)])
def test_equiv_bits_matches_oracle(kq, vq, km, vm):
    c = _cfg(kq=kq, vq=vq, km=km, vm=vm)
    if xq.xq_config_check(c) != 0:
        pytest.skip("invalid pairing")
    assert xq.xq_equiv_bits(c) == O.equiv_bits(kq, vq, km, vm, 32)


def test_equiv_bits_printed_example():
    # Appendix C worked example
    assert xq.xq_equiv_bits(_cfg(kq=30, vq=2, km=32, vm=16)) == 1.375


def test_workspace_accounting():
    c = _cfg(max_seq=4096 + 128, kq=32, vq=0, km=0, vm=0)
    n = xq.xq_workspace_bytes(c)
    B, H, D, g, R = 2, 8, 128, 32, 128
    nq = 4096
    per_layer_meta = B * H * (4 * (nq // g) * D + 4 * nq * (D // g))
    codes = 16 * B * H * nq * D * (2 + 1) // 8
    windows = 32 * 2 * B * H * R * D * 2
    assert n >= 32 * per_layer_meta + codes + windows
    assert n < 1.2 * (32 * per_layer_meta + codes + windows) + 64 * 1024 * 1024
    # no sharing doubles the codes
    c2 = _cfg(max_seq=4096 + 128, kq=32, vq=0, km=32, vm=32)
    assert xq.xq_workspace_bytes(c2) - n == codes


def test_create_rejects_bad_arguments_without_a_device():
    c = _cfg()
    rc, h = xq.xq_create(c, 0, 1 << 30)
    assert rc == xq.XQ_ERR_ARG
    rc, h = xq.xq_create(c, 256, 1024)  # far too small; the address is never dereferenced
    assert rc == xq.XQ_ERR_CAPACITY
    rc, h = xq.xq_create(c, 257, 1 << 40)
    assert rc == xq.XQ_ERR_ARG
    assert xq.xq_strerror(xq.XQ_ERR_ORDER).startswith("code-owning")


def test_host_state_machine_without_launches():
    # sequence bookkeeping is host arithmetic; exercise it through the handle without any launch
    c = _cfg(max_seq=1000)
    rc, h = xq.xq_create(c, 256, 1 << 40)
    assert rc == 0
    assert xq.xq_seq_len(h, 0) == 0 and xq.xq_quantized_len(h, 31) == 0
    assert xq.xq_seq_len(h, 32) == xq.XQ_ERR_ARG
    assert xq.xq_append_kv(h, 0, 0, 0, 1, 0) == xq.XQ_ERR_ARG
    assert xq.xq_append_kv(h, 0, 16, 16, 1001, 0) == xq.XQ_ERR_CAPACITY
    assert xq.xq_decode_attention(h, 0, 16, 16, 0) == xq.XQ_ERR_ARG  # empty layer
    rc, off0, st0 = xq.xq_region(h, 0, 0)
    rc, off1, st1 = xq.xq_region(h, 1, 0)
    assert rc == 0 and off0 == off1  # layer 1 borrows layer 0's key codes
    rc, m0, _ = xq.xq_region(h, 0, 2)
    rc, m1, _ = xq.xq_region(h, 1, 2)
    assert m0 != m1  # but has its own scale / zero-point
    assert xq.xq_destroy(h) == 0


def test_sharing_pattern_rules():
    ok = [dict(share_group=3, share_dominant=1, km=14, vm=14), dict(share_group=4, share_dominant=3, km=16, vm=32),
          dict(share_group=2, share_dominant=1), dict(gamma1=0.4), dict(gamma1=1.0), dict(io_dtype=xq.XQ_F16)]
    for kw in ok:
        assert xq.xq_config_check(_cfg(**kw)) == xq.XQ_OK, kw
    bad = [dict(share_group=5), dict(share_group=1), dict(share_group=3, share_dominant=3),
           dict(share_group=3, km=0, vm=0),             # 32 layers are not a whole number of groups of three
           dict(share_group=2, share_dominant=1, n_layers=31, kq=31, vq=31),  # layer 30 would read layer 31's codes
           dict(gamma1=0.4, share_group=3, km=14, vm=14), dict(gamma1=0.4, share_dominant=1),
           dict(gamma1=1.5), dict(gamma1=-0.1), dict(io_dtype=2),
           dict(share_group=4, km=16, vm=16, kq=18)]     # a group of four would mix 2-bit and 1-bit keys
    for kw in bad:
        assert xq.xq_config_check(_cfg(**kw)) == xq.XQ_ERR_CONFIG, kw


@pytest.mark.parametrize("group,vm", [(2, 8), (3, 14), (4, 16)])
def test_equiv_bits_of_group_table(group, vm):
    # Table group: all key layers and 20 of 32 value layers stored, printed 1.63
    for k in range(group):
        c = _cfg(kq=32, vq=32, km=32, vm=vm, share_group=group, share_dominant=k)
        assert xq.xq_equiv_bits(c) == 1.625 == O.equiv_bits(32, 32, 32, vm, 32, group, k)


def test_decode_step_refuses_before_it_touches_anything():
    """xq_decode_step checks pointers, layer order, capacity and kernel choice for every layer before its first
    copy or launch: a refused call leaves every layer's length as it was (no device is needed to see that)."""
    import ctypes as C
    c = _cfg(n_layers=4, max_seq=8)
    rc, h = xq.xq_create(c, 256, 1 << 40)
    assert rc == 0
    launches = xq.xq_launch_count(h)
    a = 1 << 20  # an aligned, never dereferenced address
    assert xq.xq_decode_step(h, a + 2, a, a, a) == xq.XQ_ERR_ARG      # misaligned K_new
    assert xq.xq_decode_step(h, a, a + 8, a, a) == xq.XQ_ERR_ARG      # misaligned V_new
    assert xq.xq_decode_step(h, a, a, a + 4, a) == xq.XQ_ERR_ARG      # misaligned q
    assert xq.xq_decode_step(h, a, a, a, a + 6) == xq.XQ_ERR_ARG      # misaligned out
    assert xq.xq_decode_step(h, a, a, a, a, [0, 1, 1, 2]) == xq.XQ_ERR_ARG    # a layer twice
    assert xq.xq_decode_step(h, a, a, a, a, [1, 0, 2, 3]) == xq.XQ_ERR_ORDER  # layer 1 reads layer 0's codes
    assert xq.xq_decode_step(h, a, a, a, a, None, 7) == xq.XQ_ERR_ARG         # unknown memory kind
    assert [xq.xq_seq_len(h, l) for l in range(4)] == [0, 0, 0, 0]
    assert xq.xq_launch_count(h) == launches
    assert xq.xq_destroy(h) == 0
    # a tensor-core-only configuration on a shape that kernel does not take is refused for every layer up front
    c = _cfg(n_layers=2, head_dim=64, kernel=xq.XQ_KERNEL_MMA)
    rc, h = xq.xq_create(c, 256, 1 << 40)
    assert rc == 0
    assert xq.xq_decode_step(h, a, a, a, a) == xq.XQ_ERR_CONFIG
    assert xq.xq_seq_len(h, 0) == 0 and xq.xq_reset(h) == 0
    assert xq.xq_destroy(h) == 0

"""ctypes binding of libxq.so: argument marshalling only.

Every function below has the name and the argument order of the C entry point
it forwards to (include/xq.h).  Device buffers are passed as torch tensors or
raw integer addresses; nothing is computed here.  Importing this module does
not need a GPU; loading fails loudly if the library has not been built.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libxq.so")

XQ_OK = 0
XQ_ERR_CONFIG, XQ_ERR_ARG, XQ_ERR_CAPACITY, XQ_ERR_ORDER, XQ_ERR_CUDA, XQ_ERR_NOMEM, XQ_ERR_DEVICE = -1, -2, -3, -4, -5, -6, -7
XQ_BF16, XQ_F16 = 0, 1
XQ_KERNEL_AUTO, XQ_KERNEL_GENERIC, XQ_KERNEL_MMA = 0, 1, 2
XQ_MEM_DEVICE, XQ_MEM_HOST = 0, 1
XQ_MAX_SPLITS = 256
XQ_STATIC_SCRATCH_BYTES = 8 << 20


class xq_config(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("max_seq", ctypes.c_int32),
        ("group_size", ctypes.c_int32), ("residual_len", ctypes.c_int32),
        ("kq", ctypes.c_int32), ("vq", ctypes.c_int32), ("km", ctypes.c_int32), ("vm", ctypes.c_int32),
        ("eta1", ctypes.c_float), ("eta2", ctypes.c_float), ("sm_scale", ctypes.c_float),
        ("n_splits", ctypes.c_int32), ("io_dtype", ctypes.c_int32), ("kernel", ctypes.c_int32),
        ("share_group", ctypes.c_int32), ("share_dominant", ctypes.c_int32), ("gamma1", ctypes.c_float),
        ("delta_stats", ctypes.c_int32),
    ]


_SIGNATURES = {
    "xq_config_check": (ctypes.c_int, [ctypes.POINTER(xq_config)]),
    "xq_workspace_bytes": (ctypes.c_size_t, [ctypes.POINTER(xq_config)]),
    "xq_create": (ctypes.c_int, [ctypes.POINTER(xq_config), ctypes.c_void_p, ctypes.c_size_t,
                                 ctypes.POINTER(ctypes.c_void_p)]),
    "xq_destroy": (ctypes.c_int, [ctypes.c_void_p]),
    "xq_reset": (ctypes.c_int, [ctypes.c_void_p]),
    "xq_append_kv": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_int, ctypes.c_void_p]),
    "xq_decode_attention": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_void_p]),
    "xq_decode_attention_f32": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                               ctypes.c_void_p]),
    "xq_decode_attention_static": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                                  ctypes.c_void_p]),
    "xq_attention_chunk": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                          ctypes.c_void_p]),
    "xq_attention_chunk_f32": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                              ctypes.c_int, ctypes.c_void_p]),
    "xq_decode_step": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int,
                                      ctypes.c_void_p]),
    "xq_check_device": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "xq_delta_histogram": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_ulonglong), ctypes.c_void_p]),
    "xq_equiv_bits": (ctypes.c_double, [ctypes.POINTER(xq_config)]),
    "xq_seq_len": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "xq_quantized_len": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "xq_split_plan": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                     ctypes.POINTER(ctypes.c_int)]),
    "xq_region": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t),
                                 ctypes.POINTER(ctypes.c_size_t)]),
    "xq_launch_count": (ctypes.c_longlong, [ctypes.c_void_p]),
    "xq_timing_enable": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "xq_timing_read": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int),
                                      ctypes.POINTER(ctypes.c_double)]),
    "xq_last_cuda_error": (ctypes.c_int, [ctypes.c_void_p]),
    "xq_strerror": (ctypes.c_char_p, [ctypes.c_int]),
}

EXPORTS = tuple(_SIGNATURES)

_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if libxq.so is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2510_11236_b200.build` "
                "(needs nvcc); this package has no CPU or PyTorch fallback")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


class XQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {xq_strerror(code)} ({code})")


def _ptr(x) -> int:
    """Address of a torch tensor's first element, or an int passed through."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if not x.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return x.data_ptr()


def xq_config_check(cfg: xq_config) -> int:
    return lib().xq_config_check(ctypes.byref(cfg))


def xq_workspace_bytes(cfg: xq_config) -> int:
    return lib().xq_workspace_bytes(ctypes.byref(cfg))


def xq_create(cfg: xq_config, dev_workspace, nbytes: int):
    h = ctypes.c_void_p()
    rc = lib().xq_create(ctypes.byref(cfg), _ptr(dev_workspace), nbytes, ctypes.byref(h))
    return rc, h


def xq_destroy(handle) -> int:
    return lib().xq_destroy(handle)


def xq_reset(handle) -> int:
    return lib().xq_reset(handle)


def xq_append_kv(handle, layer: int, K, V, n_tokens: int, stream: int = 0) -> int:
    return lib().xq_append_kv(handle, layer, _ptr(K), _ptr(V), n_tokens, stream)


def xq_decode_attention(handle, layer: int, q, out, stream: int = 0) -> int:
    return lib().xq_decode_attention(handle, layer, _ptr(q), _ptr(out), stream)


def xq_decode_attention_f32(handle, layer: int, q, out, stream: int = 0) -> int:
    return lib().xq_decode_attention_f32(handle, layer, _ptr(q), _ptr(out), stream)


def xq_decode_attention_static(handle, layer: int, q, out, stream: int = 0) -> int:
    return lib().xq_decode_attention_static(handle, layer, _ptr(q), _ptr(out), stream)


def xq_attention_chunk(handle, layer: int, q, out, n_q_tokens: int, stream: int = 0) -> int:
    return lib().xq_attention_chunk(handle, layer, _ptr(q), _ptr(out), n_q_tokens, stream)


def xq_attention_chunk_f32(handle, layer: int, q, out, n_q_tokens: int, stream: int = 0) -> int:
    return lib().xq_attention_chunk_f32(handle, layer, _ptr(q), _ptr(out), n_q_tokens, stream)


def xq_decode_step(handle, K_new, V_new, q, out, layer_order=None, mem: int = XQ_MEM_DEVICE, stream: int = 0) -> int:
    order = None
    if layer_order is not None:
        order = (ctypes.c_int32 * len(layer_order))(*layer_order)
    return lib().xq_decode_step(handle, _ptr(K_new), _ptr(V_new), _ptr(q), _ptr(out), order, mem, stream)


def xq_check_device(handle, stream: int = 0) -> int:
    return lib().xq_check_device(handle, stream)


def xq_delta_histogram(handle, layer: int, kind: int, stream: int = 0):
    counts = (ctypes.c_ulonglong * 4)()
    rc = lib().xq_delta_histogram(handle, layer, kind, counts, stream)
    return rc, [int(x) for x in counts]


def xq_equiv_bits(cfg: xq_config) -> float:
    return lib().xq_equiv_bits(ctypes.byref(cfg))


def xq_seq_len(handle, layer: int) -> int:
    return lib().xq_seq_len(handle, layer)


def xq_quantized_len(handle, layer: int) -> int:
    return lib().xq_quantized_len(handle, layer)


def xq_split_plan(handle, layer: int):
    a, b = ctypes.c_int(), ctypes.c_int()
    rc = lib().xq_split_plan(handle, layer, ctypes.byref(a), ctypes.byref(b))
    return rc, a.value, b.value


def xq_region(handle, layer: int, which: int):
    off, stride = ctypes.c_size_t(), ctypes.c_size_t()
    rc = lib().xq_region(handle, layer, which, ctypes.byref(off), ctypes.byref(stride))
    return rc, off.value, stride.value


def xq_launch_count(handle) -> int:
    return lib().xq_launch_count(handle)


def xq_timing_enable(handle, on: int) -> int:
    return lib().xq_timing_enable(handle, on)


def xq_timing_read(handle, kind: int):
    n, ms = ctypes.c_int(), ctypes.c_double()
    rc = lib().xq_timing_read(handle, kind, ctypes.byref(n), ctypes.byref(ms))
    return rc, n.value, ms.value


def xq_last_cuda_error(handle) -> int:
    return lib().xq_last_cuda_error(handle)


def xq_strerror(code: int) -> str:
    return lib().xq_strerror(code).decode()


def make_config(*, n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_seq, group_size=32, residual_len=128,
                kq=None, vq=None, km=0, vm=0, eta1=0.0, eta2=0.0, sm_scale=0.0, n_splits=0,
                kernel=XQ_KERNEL_AUTO, io_dtype=XQ_BF16, share_group=0, share_dominant=0, gamma1=0.0,
                delta_stats=0) -> xq_config:
    return xq_config(n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_seq, group_size, residual_len,
                     n_layers if kq is None else kq, n_layers if vq is None else vq, km, vm,
                     eta1, eta2, sm_scale, n_splits, io_dtype, kernel, share_group, share_dominant, gamma1,
                     delta_stats)


class Cache:
    """A cache handle plus the torch-owned workspace behind it (device memory and
    the current stream come from torch; every operation is one C call)."""

    def __init__(self, cfg: xq_config, device="cuda:0"):
        import torch
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = xq_workspace_bytes(cfg)
        if nbytes == 0:
            raise XQError(XQ_ERR_CONFIG, "xq_workspace_bytes")
        self.nbytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            assert self.workspace.data_ptr() % 256 == 0
            rc, self.handle = xq_create(cfg, self.workspace, nbytes)
        if rc != XQ_OK:
            raise XQError(rc, "xq_create")

    def _stream(self) -> int:
        import torch
        return torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        if getattr(self, "handle", None):
            xq_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        rc = xq_reset(self.handle)
        if rc:
            raise XQError(rc, "xq_reset")

    def append_kv(self, layer, K, V):
        n = K.shape[2]
        rc = xq_append_kv(self.handle, layer, K, V, n, self._stream())
        if rc:
            raise XQError(rc, "xq_append_kv")

    def decode_attention(self, layer, q, out=None, f32=False):
        import torch
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32 if f32 else q.dtype, device=q.device)
        fn = xq_decode_attention_f32 if f32 else xq_decode_attention
        rc = fn(self.handle, layer, q, out, self._stream())
        if rc:
            raise XQError(rc, "xq_decode_attention")
        return out

    def attention_chunk(self, layer, q, out=None, f32=False):
        """q: [n_q_tokens, batch, n_q_heads, head_dim]."""
        import torch
        if out is None:
            out = torch.empty(q.shape, dtype=torch.float32 if f32 else q.dtype, device=q.device)
        fn = xq_attention_chunk_f32 if f32 else xq_attention_chunk
        rc = fn(self.handle, layer, q, out, q.shape[0], self._stream())
        if rc:
            raise XQError(rc, "xq_attention_chunk")
        return out

    def decode_step(self, K_new, V_new, q, out, layer_order=None, mem=XQ_MEM_DEVICE):
        rc = xq_decode_step(self.handle, K_new, V_new, q, out, layer_order, mem, self._stream())
        if rc:
            raise XQError(rc, "xq_decode_step")
        return out

    def check_device(self):
        rc = xq_check_device(self.handle, self._stream())
        if rc:
            raise XQError(rc, "xq_check_device")

    def seq_len(self, layer):
        return xq_seq_len(self.handle, layer)

    def quantized_len(self, layer):
        return xq_quantized_len(self.handle, layer)

    def region(self, layer, which):
        """uint8 view [batch*n_kv_heads, stream_stride] of one workspace region."""
        rc, off, stride = xq_region(self.handle, layer, which)
        if rc:
            raise XQError(rc, "xq_region")
        n = self.cfg.batch * self.cfg.n_kv_heads
        return self.workspace[off:off + n * stride].view(n, stride)

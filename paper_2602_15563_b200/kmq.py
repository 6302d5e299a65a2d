"""ctypes binding of libkmq: same names as the C entry points, argument
marshalling only.  Every step of the layer runs in the CUDA library; there is
no Python or CPU implementation behind these calls, and loading fails loudly
when the shared library has not been built.

Tensor arguments are ``torch`` CUDA tensors (used for device memory only) or
raw integer device addresses; ``stream`` defaults to torch's current stream.
"""
from __future__ import annotations

import ctypes
import os

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libkmq.so")
_lib = None

KMQ_OK = 0
KMQ_ERR_NULL, KMQ_ERR_BITS, KMQ_ERR_SHAPE, KMQ_ERR_ALIGN = 1, 2, 3, 4
KMQ_ERR_WORKSPACE, KMQ_ERR_LAYOUT, KMQ_ERR_CUDA = 5, 6, 7
KMQ_ERR_SCRATCH_LIMIT = 8
KMQ_LAYOUT_CANONICAL = 0
KMQ_LAYOUT_TUNED = 1
KMQ_LAYOUT_TABLE = 2
KMQ_SCALE_DIRECT, KMQ_SCALE_DEFERRED = 0, 1
KMQ_LAMBDA_ABSMAX, KMQ_LAMBDA_ABSMEAN = 0, 1
KMQ_DEVICE_ERROR_WAIT_TIMEOUT = 1
KMQ_DEVICE_ERROR_SMEM_WINDOW = 2

_i64, _int, _ptr, _sz = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/kmq.h
SIGNATURES = {
    "kmq_version": (_int, []),
    "kmq_status_string": (ctypes.c_char_p, [_int]),
    "kmq_packed_bytes": (_sz, [_i64, _i64, _int, _int]),
    "kmq_packed_word_index": (_i64, [_i64, _i64, _i64, _i64, _int, _int]),
    "kmq_packed_field_shift": (_int, [_int, _int, _int]),
    "kmq_packed_bit_index": (_i64, [_i64, _i64, _int, _i64, _i64, _int, _int]),
    "kmq_preferred_layout": (_int, [_i64, _i64, _int, _i64]),
    "kmq_workspace_bytes": (_sz, [_i64, _i64, _int, _i64, _int]),
    "kmq_linear_num_launches": (_int, [_i64, _i64, _int, _i64, _int]),
    "kmq_linear_variant": (ctypes.c_char_p, [_i64, _i64, _int, _i64, _int]),
    "kmq_pack": (_int, [_ptr, _i64, _i64, _int, _int, _ptr, _ptr]),
    "kmq_unpack": (_int, [_ptr, _i64, _i64, _int, _int, _ptr, _ptr]),
    "kmq_linear": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _int, _ptr, _sz, _ptr]),
    "kmq_linear_host": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _int, _ptr, _ptr, _ptr, _sz, _ptr]),
    "kmq_linear_static_scratch": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _int, _ptr]),
    "kmq_static_scratch_capacity": (_sz, []),
    "kmq_linear_tcgen05": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _ptr]),
    "kmq_device_error_flags": (_int, [_ptr]),
    "kmq_dequant_to_bf16": (_int, [_ptr, _ptr, _ptr, _i64, _i64, _int, _int, _ptr]),
    "kmq_block_packed_bytes": (_sz, [_i64, _i64, _int]),
    "kmq_block_pack": (_int, [_ptr, _i64, _i64, _int, _ptr, _ptr]),
    "kmq_block_linear": (_int, [_ptr, _ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _int, _ptr]),
    "kmq_block_dequant_to_bf16": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _ptr]),
    "kmq_block_table_bytes": (_sz, [_i64, _i64, _int]),
    "kmq_block_table_index_offset": (_i64, [_i64, _i64, _i64, _i64, _int]),
    "kmq_block_table_scale_offset": (_i64, [_i64, _i64, _i64, _i64, _int]),
    "kmq_block_table_pack": (_int, [_ptr, _ptr, _i64, _i64, _int, _ptr, _ptr]),
    "kmq_block_table_unpack": (_int, [_ptr, _i64, _i64, _int, _ptr, _ptr, _ptr]),
    "kmq_block_table_workspace_bytes": (_sz, [_i64, _i64, _int]),
    "kmq_block_table_linear": (_int, [_ptr, _ptr, _ptr, _ptr, _i64, _i64, _int, _i64, _ptr, _sz, _ptr]),
    "kmq_kmeans_rows": (_int, [_ptr, _i64, _i64, _int, _int, _ptr, _ptr, _ptr]),
    "kmq_assign_pack": (_int, [_ptr, _ptr, _i64, _i64, _int, _int, _ptr, _ptr]),
    "kmq_quantize_rows": (_int, [_ptr, _i64, _i64, _int, _int, _int, _ptr, _ptr, _ptr]),
    "kmq_block_scales": (_int, [_ptr, _i64, _i64, _int, _ptr, _ptr]),
    "kmq_block_sample_count": (_i64, [_i64, _i64, _i64]),
    "kmq_block_sample": (_int, [_ptr, _ptr, _i64, _i64, _i64, _ptr, _ptr]),
    "kmq_block_assign_pack": (_int, [_ptr, _ptr, _ptr, _i64, _i64, _int, _ptr, _ptr]),
    "kmq_block_quantize": (_int, [_ptr, _i64, _i64, _int, _int, _int, _i64, _ptr, _ptr, _ptr, _ptr, _ptr]),
    "kmq_probe_launch": (_int, [_ptr]),
    "kmq_probe_read_out_bytes": (_sz, []),
    "kmq_probe_read": (_int, [_ptr, _sz, _ptr, _ptr]),
}


class KmqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load libkmq.so (once).  Raises if it is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise ImportError(
                f"{_LIB_PATH} not found: build it with "
                "`python -m paper_2602_15563_b200.build` (needs nvcc); libkmq has no CPU fallback")
        handle = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _addr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def _check(status: int, where: str) -> None:
    if status != KMQ_OK:
        raise KmqError(status, where)


def status_string(status: int) -> str:
    return lib().kmq_status_string(int(status)).decode()


def kmq_version() -> int:
    return lib().kmq_version()


def kmq_packed_bytes(N, K, bits, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_packed_bytes(N, K, bits, layout)


def kmq_packed_word_index(n, j, N, K, bits, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_packed_word_index(n, j, N, K, bits, layout)


def kmq_packed_field_shift(i, bits, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_packed_field_shift(i, bits, layout)


def kmq_packed_bit_index(n, k, plane, N, K, bits, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_packed_bit_index(n, k, plane, N, K, bits, layout)


def kmq_preferred_layout(N, K, bits, M) -> int:
    return lib().kmq_preferred_layout(N, K, bits, M)


def kmq_workspace_bytes(N, K, bits, M, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_workspace_bytes(N, K, bits, M, layout)


def kmq_linear_num_launches(N, K, bits, M, layout=KMQ_LAYOUT_CANONICAL) -> int:
    return lib().kmq_linear_num_launches(N, K, bits, M, layout)


def kmq_linear_variant(N, K, bits, M, layout=KMQ_LAYOUT_CANONICAL) -> str:
    return lib().kmq_linear_variant(N, K, bits, M, layout).decode()


def kmq_pack(idx, N, K, bits, packed, layout=KMQ_LAYOUT_CANONICAL, stream=None, check=True) -> int:
    st = lib().kmq_pack(_addr(idx), N, K, bits, layout, _addr(packed), _stream(stream))
    if check:
        _check(st, "kmq_pack")
    return st


def kmq_unpack(packed, N, K, bits, idx, layout=KMQ_LAYOUT_CANONICAL, stream=None, check=True) -> int:
    st = lib().kmq_unpack(_addr(packed), N, K, bits, layout, _addr(idx), _stream(stream))
    if check:
        _check(st, "kmq_unpack")
    return st


def kmq_linear(packed, codebooks, x, y, N, K, bits, M, workspace=None, workspace_bytes=None,
               layout=KMQ_LAYOUT_CANONICAL, stream=None, check=True) -> int:
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else workspace.numel() * workspace.element_size()
    st = lib().kmq_linear(_addr(packed), _addr(codebooks), _addr(x), _addr(y), N, K, bits, M, layout,
                          _addr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(st, "kmq_linear")
    return st


def kmq_linear_host(packed, codebooks, x_host, y_host, N, K, bits, M, x_dev, y_dev, workspace=None,
                    workspace_bytes=None, layout=KMQ_LAYOUT_CANONICAL, stream=None, check=True) -> int:
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else workspace.numel() * workspace.element_size()
    st = lib().kmq_linear_host(_addr(packed), _addr(codebooks), _addr(x_host), _addr(y_host), N, K, bits, M, layout,
                               _addr(x_dev), _addr(y_dev), _addr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(st, "kmq_linear_host")
    return st


def kmq_linear_static_scratch(packed, codebooks, x, y, N, K, bits, M, layout=KMQ_LAYOUT_CANONICAL, stream=None,
                              check=True) -> int:
    """kmq_linear for callers that may not allocate: scratch, where needed, is a fixed array inside the library."""
    st = lib().kmq_linear_static_scratch(_addr(packed), _addr(codebooks), _addr(x), _addr(y), N, K, bits, M, layout,
                                         _stream(stream))
    if check:
        _check(st, "kmq_linear_static_scratch")
    return st


def kmq_static_scratch_capacity() -> int:
    return lib().kmq_static_scratch_capacity()


def kmq_linear_tcgen05(packed, codebooks, x, y, N, K, bits, M, stream=None, check=True) -> int:
    """kmq_linear through the tcgen05 / tensor-memory kernel (tuned layout only)."""
    st = lib().kmq_linear_tcgen05(_addr(packed), _addr(codebooks), _addr(x), _addr(y), N, K, bits, M, _stream(stream))
    if check:
        _check(st, "kmq_linear_tcgen05")
    return st


def kmq_device_error_flags() -> int:
    """Synchronise the device; return and clear the error word of the kernels (0 = no bounded wait ran out)."""
    flags = ctypes.c_uint(0)
    _check(lib().kmq_device_error_flags(ctypes.addressof(flags)), "kmq_device_error_flags")
    return flags.value


def kmq_dequant_to_bf16(packed, codebooks, W, N, K, bits, layout=KMQ_LAYOUT_CANONICAL, stream=None, check=True) -> int:
    st = lib().kmq_dequant_to_bf16(_addr(packed), _addr(codebooks), _addr(W), N, K, bits, layout, _stream(stream))
    if check:
        _check(st, "kmq_dequant_to_bf16")
    return st


def kmq_probe_launch(stream=None, check=True) -> int:
    """Enqueue the do-nothing kernel (the fixed cost of a call)."""
    st = lib().kmq_probe_launch(_stream(stream))
    if check:
        _check(st, "kmq_probe_launch")
    return st


def kmq_probe_read_out_bytes() -> int:
    return lib().kmq_probe_read_out_bytes()


def kmq_probe_read(buf, nbytes, out, stream=None, check=True) -> int:
    """Read `nbytes` of `buf` once with streaming loads (the read-only bandwidth ceiling)."""
    st = lib().kmq_probe_read(_addr(buf), nbytes, _addr(out), _stream(stream))
    if check:
        _check(st, "kmq_probe_read")
    return st


def kmq_block_packed_bytes(N, K, bits) -> int:
    return lib().kmq_block_packed_bytes(N, K, bits)


def kmq_block_pack(idx, N, K, bits, wq, stream=None, check=True) -> int:
    st = lib().kmq_block_pack(_addr(idx), N, K, bits, _addr(wq), _stream(stream))
    if check:
        _check(st, "kmq_block_pack")
    return st


def kmq_block_linear(wq, scales, codebook, x, y, N, K, bits, M, scale_order=KMQ_SCALE_DEFERRED, stream=None,
                     check=True) -> int:
    """The paper's block format (shared codebook, bf16 scale per block of 64): y = x * W^T."""
    st = lib().kmq_block_linear(_addr(wq), _addr(scales), _addr(codebook), _addr(x), _addr(y), N, K, bits, M,
                                scale_order, _stream(stream))
    if check:
        _check(st, "kmq_block_linear")
    return st


def kmq_block_dequant_to_bf16(wq, scales, codebook, W, N, K, bits, stream=None, check=True) -> int:
    st = lib().kmq_block_dequant_to_bf16(_addr(wq), _addr(scales), _addr(codebook), _addr(W), N, K, bits,
                                         _stream(stream))
    if check:
        _check(st, "kmq_block_dequant_to_bf16")
    return st


def kmq_kmeans_rows(W, N, K, bits, iters, codebooks, centroids=None, stream=None, check=True) -> int:
    """Per-row 1-D Lloyd fit: W float32 [N, K] -> codebooks bf16 [N, 2^bits] (and float64 centroids if given)."""
    st = lib().kmq_kmeans_rows(_addr(W), N, K, bits, iters, _addr(codebooks), _addr(centroids), _stream(stream))
    if check:
        _check(st, "kmq_kmeans_rows")
    return st


def kmq_assign_pack(W, codebooks, N, K, bits, layout, packed, stream=None, check=True) -> int:
    """Nearest stored centroid of every weight, written as packed indices in `layout`."""
    st = lib().kmq_assign_pack(_addr(W), _addr(codebooks), N, K, bits, layout, _addr(packed), _stream(stream))
    if check:
        _check(st, "kmq_assign_pack")
    return st


def kmq_quantize_rows(W, N, K, bits, iters, layout, codebooks, packed, stream=None, check=True) -> int:
    st = lib().kmq_quantize_rows(_addr(W), N, K, bits, iters, layout, _addr(codebooks), _addr(packed),
                                 _stream(stream))
    if check:
        _check(st, "kmq_quantize_rows")
    return st


def kmq_block_scales(W, N, K, lam, scales, stream=None, check=True) -> int:
    st = lib().kmq_block_scales(_addr(W), N, K, lam, _addr(scales), _stream(stream))
    if check:
        _check(st, "kmq_block_scales")
    return st


def kmq_block_sample_count(N, K, samples) -> int:
    return lib().kmq_block_sample_count(N, K, samples)


def kmq_block_sample(W, scales, N, K, samples, out, stream=None, check=True) -> int:
    st = lib().kmq_block_sample(_addr(W), _addr(scales), N, K, samples, _addr(out), _stream(stream))
    if check:
        _check(st, "kmq_block_sample")
    return st


def kmq_block_assign_pack(W, scales, codebook, N, K, bits, wq, stream=None, check=True) -> int:
    st = lib().kmq_block_assign_pack(_addr(W), _addr(scales), _addr(codebook), N, K, bits, _addr(wq),
                                     _stream(stream))
    if check:
        _check(st, "kmq_block_assign_pack")
    return st


def kmq_block_quantize(W, N, K, bits, lam, iters, samples, scales, codebook, wq, sample_workspace, stream=None,
                       check=True) -> int:
    """Block format, all steps: scales, strided normalised sample, shared codebook fit, packed indices."""
    st = lib().kmq_block_quantize(_addr(W), N, K, bits, lam, iters, samples, _addr(scales), _addr(codebook),
                                  _addr(wq), _addr(sample_workspace), _stream(stream))
    if check:
        _check(st, "kmq_block_quantize")
    return st


def kmq_block_table_bytes(N, K, bits) -> int:
    return lib().kmq_block_table_bytes(N, K, bits)


def kmq_block_table_index_offset(n, k, N, K, bits) -> int:
    return lib().kmq_block_table_index_offset(n, k, N, K, bits)


def kmq_block_table_scale_offset(n, k, N, K, bits) -> int:
    return lib().kmq_block_table_scale_offset(n, k, N, K, bits)


def kmq_block_table_pack(wq, scales, N, K, bits, table, stream=None, check=True) -> int:
    st = lib().kmq_block_table_pack(_addr(wq), _addr(scales), N, K, bits, _addr(table), _stream(stream))
    if check:
        _check(st, "kmq_block_table_pack")
    return st


def kmq_block_table_unpack(table, N, K, bits, wq, scales, stream=None, check=True) -> int:
    st = lib().kmq_block_table_unpack(_addr(table), N, K, bits, _addr(wq), _addr(scales), _stream(stream))
    if check:
        _check(st, "kmq_block_table_unpack")
    return st


def kmq_block_table_workspace_bytes(N, K, bits) -> int:
    return lib().kmq_block_table_workspace_bytes(N, K, bits)


def kmq_block_table_linear(table, codebook, x, y, N, K, bits, M, workspace=None, workspace_bytes=0, stream=None,
                           check=True) -> int:
    """Block format through the activation table: y = x * W^T, one pass per batch row."""
    st = lib().kmq_block_table_linear(_addr(table), _addr(codebook), _addr(x), _addr(y), N, K, bits, M,
                                      _addr(workspace), workspace_bytes, _stream(stream))
    if check:
        _check(st, "kmq_block_table_linear")
    return st

"""Thin ctypes binding of ``libfastsgd_b200.so`` (same names as ``include/fastsgd.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  Loading fails loudly if the library has not
been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfastsgd_b200.so")

OK = 0
E_NULL, E_ALIGN, E_BAD_PARAM, E_BAD_N, E_CAPACITY, E_NO_WORKSPACE, E_NOT_IMPLEMENTED, E_CUDA, E_TRUNCATED = range(-1, -10, -1)
E_TOO_LARGE = -10
NOALLOC_MAX_N = 1 << 28
ST_OK, ST_NONFINITE, ST_CAPACITY, ST_TIMEOUT = 0, 1, 2, 3
ST_BAD_MAGIC, ST_BAD_VERSION, ST_BAD_STATUS, ST_N_MISMATCH, ST_PARAM_MISMATCH = 16, 17, 18, 19, 20
ST_TRUNCATED, ST_BAD_DIRECTORY, ST_BAD_KEY, ST_BAD_CODE = 21, 22, 23, 24

EXPORTS = [
    "fastsgd_compress", "fastsgd_compress_batch", "fastsgd_decompress_accumulate", "fastsgd_decompress_accumulate_batch", "fastsgd_compress_bound",
    "fastsgd_workspace_bytes", "fastsgd_set_workspace", "fastsgd_stream_info",
    "fastsgd_decode_status", "fastsgd_abs_sum", "fastsgd_host_scratch_bytes",
    "fastsgd_compress_host", "fastsgd_decompress_accumulate_host", "fastsgd_launch_count",
    "fastsgd_strerror", "fastsgd_version", "fastsgd_kernel_timing_enable", "fastsgd_kernel_timing_read", "fastsgd_abs_sum_noalloc",
    "fastsgd_sparse_adam_update_batch", "fastsgd_sparse_adam_update_packed_batch", "fastsgd_key_encode_paper", "fastsgd_key_encode_paper_bound",
    "fastsgd_compress_kv",
    "fastsgd_debug_set_wait_limits", "fastsgd_debug_layout", "fastsgd_debug_trace_compiled", "fastsgd_debug_set_grid",
]


class Params(C.Structure):
    _fields_ = [("base", C.c_double), ("tau", C.c_uint32), ("flag_bits", C.c_uint32),
                ("group_log2", C.c_uint32), ("reserved", C.c_uint32)]


class Adam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


def params(base: float, tau: int = 128, flag_bits: int = 2, group_log2: int = 14) -> Params:
    return Params(float(base), int(tau), int(flag_bits), int(group_log2), 0)


class FastSGDError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def lib():
    """The loaded C-ABI library.  Raises if it was not built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2112_04291_b200.build` "
                "(needs nvcc; there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, u64, PP = C.c_void_p, C.c_uint64, C.POINTER(Params)
        u64p, intp = C.POINTER(C.c_uint64), C.POINTER(C.c_int)
        L.fastsgd_compress.restype = C.c_int
        L.fastsgd_compress.argtypes = [vp, u64, PP, vp, u64, vp]
        L.fastsgd_decompress_accumulate.restype = C.c_int
        L.fastsgd_decompress_accumulate.argtypes = [vp, u64, u64, PP, vp, vp]
        L.fastsgd_compress_batch.restype = C.c_int
        L.fastsgd_compress_batch.argtypes = [C.POINTER(vp), u64, PP, C.POINTER(vp), u64, C.c_uint32, vp]
        L.fastsgd_decompress_accumulate_batch.restype = C.c_int
        L.fastsgd_decompress_accumulate_batch.argtypes = [C.POINTER(vp), u64p, C.c_uint32, u64, PP, vp, vp]
        L.fastsgd_compress_kv.restype = C.c_int
        L.fastsgd_compress_kv.argtypes = [vp, vp, u64, u64, PP, vp, u64, vp]
        L.fastsgd_key_encode_paper_bound.restype = C.c_uint64
        L.fastsgd_key_encode_paper_bound.argtypes = [u64, C.c_uint32]
        L.fastsgd_key_encode_paper.restype = C.c_int
        L.fastsgd_key_encode_paper.argtypes = [vp, u64, C.c_uint32, vp, u64, vp]
        L.fastsgd_sparse_adam_update_batch.restype = C.c_int
        L.fastsgd_sparse_adam_update_batch.argtypes = [C.POINTER(vp), u64p, C.c_uint32, u64, PP, C.POINTER(Adam), vp, vp, vp, vp, vp]
        L.fastsgd_sparse_adam_update_packed_batch.restype = C.c_int
        L.fastsgd_sparse_adam_update_packed_batch.argtypes = [C.POINTER(vp), u64p, C.c_uint32, u64, PP, C.POINTER(Adam), vp, vp]
        L.fastsgd_compress_bound.restype = u64
        L.fastsgd_compress_bound.argtypes = [u64, PP]
        L.fastsgd_workspace_bytes.restype = u64
        L.fastsgd_workspace_bytes.argtypes = [u64, PP]
        L.fastsgd_set_workspace.restype = C.c_int
        L.fastsgd_set_workspace.argtypes = [vp, u64, vp]
        L.fastsgd_stream_info.restype = C.c_int
        L.fastsgd_stream_info.argtypes = [vp, vp, u64p, u64p, intp]
        L.fastsgd_decode_status.restype = C.c_int
        L.fastsgd_decode_status.argtypes = [vp, intp]
        L.fastsgd_abs_sum.restype = C.c_int
        L.fastsgd_abs_sum.argtypes = [vp, u64, vp, vp]
        L.fastsgd_host_scratch_bytes.restype = u64
        L.fastsgd_host_scratch_bytes.argtypes = [u64, PP]
        L.fastsgd_compress_host.restype = C.c_int
        L.fastsgd_compress_host.argtypes = [vp, u64, PP, vp, u64, u64p, intp, vp, u64, vp]
        L.fastsgd_decompress_accumulate_host.restype = C.c_int
        L.fastsgd_decompress_accumulate_host.argtypes = [C.POINTER(vp), u64p, C.c_uint32, u64, PP, vp, C.c_int, intp, vp, u64, vp]
        L.fastsgd_launch_count.restype = u64
        L.fastsgd_launch_count.argtypes = []
        L.fastsgd_strerror.restype = C.c_char_p
        L.fastsgd_strerror.argtypes = [C.c_int]
        L.fastsgd_version.restype = C.c_int
        L.fastsgd_version.argtypes = []
        L.fastsgd_abs_sum_noalloc.restype = C.c_int
        L.fastsgd_abs_sum_noalloc.argtypes = [vp, u64, vp, vp]
        L.fastsgd_kernel_timing_enable.restype = C.c_int
        L.fastsgd_kernel_timing_enable.argtypes = [C.c_int]
        L.fastsgd_kernel_timing_read.restype = C.c_int
        L.fastsgd_kernel_timing_read.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_uint64)]
        L.fastsgd_debug_set_wait_limits.restype = C.c_int
        L.fastsgd_debug_set_wait_limits.argtypes = [C.c_uint32, C.c_uint32, C.c_uint32]
        L.fastsgd_debug_set_grid.restype = C.c_int
        L.fastsgd_debug_set_grid.argtypes = [C.c_uint32]
        L.fastsgd_debug_layout.restype = C.c_int
        L.fastsgd_debug_layout.argtypes = [u64p, C.c_uint32]
        L.fastsgd_debug_trace_compiled.restype = C.c_int
        L.fastsgd_debug_trace_compiled.argtypes = []
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().fastsgd_strerror(int(code)).decode()


def _stream_handle(stream=None) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise FastSGDError(rc, where)


def compress_bound(n: int, p: Params) -> int:
    return int(lib().fastsgd_compress_bound(n, C.byref(p)))


def workspace_bytes(n: int, p: Params) -> int:
    return int(lib().fastsgd_workspace_bytes(n, C.byref(p)))


_workspace_keepalive = None


def set_workspace(ws: torch.Tensor, stream=None) -> None:
    """Registers a uint8 CUDA tensor as the library's scratch (kept alive here)."""
    global _workspace_keepalive
    assert ws.is_cuda and ws.dtype == torch.uint8 and ws.is_contiguous()
    _check(lib().fastsgd_set_workspace(ws.data_ptr(), ws.numel(), _stream_handle(stream)), "fastsgd_set_workspace")
    _workspace_keepalive = ws


def ensure_workspace(n: int, p: Params, device="cuda") -> torch.Tensor:
    """Allocates (torch) and registers a workspace large enough for n entries, if needed."""
    need = workspace_bytes(n, p)
    ws = _workspace_keepalive
    dev = torch.device(device)
    if dev.index is None:
        dev = torch.device(dev.type, torch.cuda.current_device())
    if ws is None or ws.numel() < need or ws.device != dev:
        ws = torch.empty(max(need, 4096), dtype=torch.uint8, device=dev)
        set_workspace(ws)
    return ws


def compress(grad: torch.Tensor, p: Params, out: torch.Tensor, stream=None) -> int:
    """fastsgd_compress: enqueues the encoder; returns the host-visible return code."""
    assert grad.is_cuda and grad.dtype == torch.float32 and grad.is_contiguous()
    assert out.is_cuda and out.dtype == torch.uint8 and out.is_contiguous()
    return lib().fastsgd_compress(grad.data_ptr(), grad.numel(), C.byref(p), out.data_ptr(), out.numel(),
                                  _stream_handle(stream))


def compress_batch(grads, p: Params, outs, stream=None) -> int:
    """fastsgd_compress_batch: several workers' gradients (same length) in one launch per 8."""
    k = len(grads)
    assert k == len(outs) and k > 0
    n = grads[0].numel()
    assert all(g.is_cuda and g.dtype == torch.float32 and g.is_contiguous() and g.numel() == n for g in grads)
    cap = outs[0].numel()
    assert all(o.is_cuda and o.dtype == torch.uint8 and o.is_contiguous() and o.numel() == cap for o in outs)
    gp = (C.c_void_p * k)(*[int(g.data_ptr()) for g in grads])
    op = (C.c_void_p * k)(*[int(o.data_ptr()) for o in outs])
    return lib().fastsgd_compress_batch(gp, n, C.byref(p), op, cap, k, _stream_handle(stream))


def decompress_accumulate(stream_in: torch.Tensor, nbytes: int, n: int, p: Params, dense: torch.Tensor,
                          stream=None) -> int:
    assert stream_in.is_cuda and stream_in.dtype == torch.uint8
    assert dense.is_cuda and dense.dtype == torch.float32 and dense.is_contiguous() and dense.numel() == n
    return lib().fastsgd_decompress_accumulate(stream_in.data_ptr(), int(nbytes), int(n), C.byref(p),
                                               dense.data_ptr(), _stream_handle(stream))


def decompress_accumulate_batch(streams_in, nbytes, n: int, p: Params, dense: torch.Tensor, stream=None) -> int:
    """fastsgd_decompress_accumulate_batch: all workers' streams in one launch (per 8 streams)."""
    assert dense.is_cuda and dense.dtype == torch.float32 and dense.is_contiguous() and dense.numel() == n
    k = len(streams_in)
    assert all(s.is_cuda and s.dtype == torch.uint8 for s in streams_in) and len(nbytes) == k
    ptrs = (C.c_void_p * k)(*[int(s.data_ptr()) for s in streams_in])
    sizes = (C.c_uint64 * k)(*[int(b) for b in nbytes])
    return lib().fastsgd_decompress_accumulate_batch(ptrs, sizes, k, int(n), C.byref(p), dense.data_ptr(),
                                                     _stream_handle(stream))


def sparse_adam_update_batch(streams_in, nbytes, n: int, p: Params, hyper: Adam, grad_scratch: torch.Tensor,
                             theta: torch.Tensor, m: torch.Tensor, v: torch.Tensor, stream=None) -> int:
    """fastsgd_sparse_adam_update_batch: decode the workers' streams, one Adam step where the aggregated gradient is non-zero."""
    for a in (grad_scratch, theta, m, v):
        assert a.is_cuda and a.dtype == torch.float32 and a.is_contiguous() and a.numel() == n
    k = len(streams_in)
    assert all(s.is_cuda and s.dtype == torch.uint8 for s in streams_in) and len(nbytes) == k
    ptrs = (C.c_void_p * k)(*[int(s.data_ptr()) for s in streams_in])
    sizes = (C.c_uint64 * k)(*[int(b) for b in nbytes])
    return lib().fastsgd_sparse_adam_update_batch(ptrs, sizes, k, int(n), C.byref(p), C.byref(hyper), grad_scratch.data_ptr(),
                                                  theta.data_ptr(), m.data_ptr(), v.data_ptr(), _stream_handle(stream))


def sparse_adam_update_packed_batch(streams_in, nbytes, n: int, p: Params, hyper: Adam, state: torch.Tensor, stream=None) -> int:
    """fastsgd_sparse_adam_update_packed_batch: the same step on the state kept as (theta, m, v, g) per coordinate."""
    assert state.is_cuda and state.dtype == torch.float32 and state.is_contiguous() and state.numel() == 4 * n
    k = len(streams_in)
    assert all(s.is_cuda and s.dtype == torch.uint8 for s in streams_in) and len(nbytes) == k
    ptrs = (C.c_void_p * k)(*[int(s.data_ptr()) for s in streams_in])
    sizes = (C.c_uint64 * k)(*[int(b) for b in nbytes])
    return lib().fastsgd_sparse_adam_update_packed_batch(ptrs, sizes, k, int(n), C.byref(p), C.byref(hyper), state.data_ptr(),
                                                         _stream_handle(stream))


def compress_kv(keys: torch.Tensor, values: torch.Tensor, n: int, p: Params, out: torch.Tensor, stream=None) -> int:
    """fastsgd_compress_kv: the gradient as ascending keys (int32 tensor holding 32-bit keys) and their fp32 values."""
    assert keys.is_cuda and keys.dtype == torch.int32 and keys.is_contiguous()
    assert values.is_cuda and values.dtype == torch.float32 and values.is_contiguous() and values.numel() == keys.numel()
    assert out.is_cuda and out.dtype == torch.uint8 and out.is_contiguous()
    cnt = keys.numel()
    return lib().fastsgd_compress_kv(keys.data_ptr() if cnt else None, values.data_ptr() if cnt else None, cnt, int(n),
                                     C.byref(p), out.data_ptr(), out.numel(), _stream_handle(stream))


def key_encode_paper_bound(d: int, flag_bits: int) -> int:
    return int(lib().fastsgd_key_encode_paper_bound(int(d), int(flag_bits)))


def key_encode_paper(keys: torch.Tensor, flag_bits: int, out: torch.Tensor, stream=None) -> int:
    """fastsgd_key_encode_paper: Algorithm 2 as printed over `keys` (int32 tensor holding ascending 32-bit keys)."""
    assert keys.is_cuda and keys.dtype == torch.int32 and keys.is_contiguous()
    assert out.is_cuda and out.dtype == torch.uint8 and out.is_contiguous()
    return lib().fastsgd_key_encode_paper(keys.data_ptr() if keys.numel() else None, keys.numel(), int(flag_bits),
                                          out.data_ptr(), out.numel(), _stream_handle(stream))


def stream_info(stream_in: torch.Tensor, stream=None):
    """(total_bytes, d, status) of a stream's header; synchronises."""
    tb, d, st = C.c_uint64(0), C.c_uint64(0), C.c_int(0)
    _check(lib().fastsgd_stream_info(stream_in.data_ptr(), _stream_handle(stream), C.byref(tb), C.byref(d),
                                     C.byref(st)), "fastsgd_stream_info")
    return tb.value, d.value, st.value


def decode_status(stream=None) -> int:
    st = C.c_int(0)
    _check(lib().fastsgd_decode_status(_stream_handle(stream), C.byref(st)), "fastsgd_decode_status")
    return st.value


def abs_sum(grad: torch.Tensor, out: torch.Tensor, stream=None) -> int:
    assert grad.is_cuda and grad.dtype == torch.float32 and out.is_cuda and out.dtype == torch.float64
    return lib().fastsgd_abs_sum(grad.data_ptr(), grad.numel(), out.data_ptr(), _stream_handle(stream))


def abs_sum_noalloc(grad: torch.Tensor, out: torch.Tensor, stream=None) -> int:
    """fastsgd_abs_sum_noalloc: the same sum, with the library's built-in scratch (no workspace needed)."""
    assert grad.is_cuda and grad.dtype == torch.float32 and out.is_cuda and out.dtype == torch.float64
    return lib().fastsgd_abs_sum_noalloc(grad.data_ptr(), grad.numel(), out.data_ptr(), _stream_handle(stream))


def host_scratch_bytes(n: int, p: Params) -> int:
    return int(lib().fastsgd_host_scratch_bytes(n, C.byref(p)))


def compress_host(grad_host: torch.Tensor, p: Params, out_host: torch.Tensor, scratch: torch.Tensor, stream=None):
    """Host-buffer encoder -> (return code, produced bytes, header status)."""
    assert not grad_host.is_cuda and grad_host.dtype == torch.float32 and grad_host.is_contiguous()
    assert not out_host.is_cuda and out_host.dtype == torch.uint8 and scratch.is_cuda
    produced, st = C.c_uint64(0), C.c_int(0)
    rc = lib().fastsgd_compress_host(grad_host.data_ptr(), grad_host.numel(), C.byref(p), out_host.data_ptr(),
                                     out_host.numel(), C.byref(produced), C.byref(st), scratch.data_ptr(),
                                     scratch.numel(), _stream_handle(stream))
    return rc, produced.value, st.value


def decompress_accumulate_host(streams_host, nbytes, n: int, p: Params, dense_host: torch.Tensor,
                               scratch: torch.Tensor, accumulate: bool = False, stream=None):
    """Host-buffer decoder + aggregation of several streams -> (return code, decoder status)."""
    assert not dense_host.is_cuda and dense_host.dtype == torch.float32 and dense_host.numel() == n
    k = len(streams_host)
    ptrs = (C.c_void_p * k)(*[int(s.data_ptr()) for s in streams_host])
    sizes = (C.c_uint64 * k)(*[int(b) for b in nbytes])
    st = C.c_int(0)
    rc = lib().fastsgd_decompress_accumulate_host(ptrs, sizes, k, int(n), C.byref(p), dense_host.data_ptr(),
                                                  int(bool(accumulate)), C.byref(st), scratch.data_ptr(),
                                                  scratch.numel(), _stream_handle(stream))
    return rc, st.value


def launch_count() -> int:
    return int(lib().fastsgd_launch_count())


KERNELS = ("k_abs_sum", "k_compress", "k_decode_accumulate")


def kernel_timing_enable(on: bool) -> None:
    _check(lib().fastsgd_kernel_timing_enable(int(bool(on))), "fastsgd_kernel_timing_enable")


def kernel_timing_read():
    """{kernel name: (total ms, launches)} since the last read; synchronises."""
    ms = (C.c_double * 3)()
    cnt = (C.c_uint64 * 3)()
    _check(lib().fastsgd_kernel_timing_read(ms, cnt), "fastsgd_kernel_timing_read")
    return {k: (ms[i], int(cnt[i])) for i, k in enumerate(KERNELS)}


def debug_set_wait_limits(block_polls: int = 0, copy_tries: int = 0, queue_polls: int = 0) -> None:
    """fastsgd_debug_set_wait_limits: shorten (or, with zeros, restore) the kernels' bounded waits.  Test aid."""
    _check(lib().fastsgd_debug_set_wait_limits(int(block_polls), int(copy_tries), int(queue_polls)),
           "fastsgd_debug_set_wait_limits")


def debug_set_grid(blocks: int = 0) -> None:
    """fastsgd_debug_set_grid: cap the encoders' thread blocks (0: default).  Test aid."""
    _check(lib().fastsgd_debug_set_grid(int(blocks)), "fastsgd_debug_set_grid")


LAYOUT_FIELDS = ("bar_count", "ne_count", "error", "decoder_trace", "encoder_trace", "encoder_trace_bytes",
                 "queue_slots", "queue_counters")


def debug_layout() -> dict:
    """fastsgd_debug_layout: byte offsets of a few fields inside the registered workspace."""
    v = (C.c_uint64 * len(LAYOUT_FIELDS))()
    _check(lib().fastsgd_debug_layout(v, len(LAYOUT_FIELDS)), "fastsgd_debug_layout")
    return {k: int(v[i]) for i, k in enumerate(LAYOUT_FIELDS)}


def workspace_u32(field: str, count: int):
    """`count` 32-bit words of the registered workspace at a field of debug_layout(), as a torch view
    (reads and writes go to device memory; synchronise before relying on them)."""
    ws = _workspace_keepalive
    assert ws is not None, "no workspace registered through this module"
    off = debug_layout()[field]
    return ws[off:off + 4 * count].view(torch.int32)


def listed_tiles(jobs: int):
    """Tiles the encode pass of the last fastsgd_compress(_batch) launch read a second time, per gradient
    (the others held nothing to keep, or were still in shared memory).  Synchronises."""
    torch.cuda.synchronize()
    return [int(x) for x in workspace_u32("ne_count", 8)[:jobs].cpu().tolist()]


def debug_trace_blocks(blocks: int = 148):
    """Per-block stamps (ns, %globaltimer) of the last compress launch, shape (blocks, 8, 8): for
    each block and each gradient of the launch: start, end of the sum pass, previous gradient's
    pending tiles placed, grid barrier passed, table ready, end of the encode loop; slot 6 of
    gradient 0 holds the end of the launch's last drain.  Only a library built with -DFASTSGD_TRACE
    writes them (None otherwise); synchronises."""
    ws = _workspace_keepalive
    if ws is None or not lib().fastsgd_debug_trace_compiled():
        return None
    torch.cuda.synchronize()
    off = debug_layout()["encoder_trace"]
    return ws[off:off + 512 * blocks].cpu().numpy().view("<u8").reshape(blocks, 8, 8).astype("int64")

"""Thin Python binding of libthc's C ABI (include/thc.h): argument marshalling only.

Every step of the round runs in the library's CUDA kernels.  PyTorch is used here for
device memory and the current stream; nothing in this module computes.  If libthc.so is
missing the import of the library fails loudly -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libthc.so")
_lib = None

THC_OK, THC_EINVAL, THC_EUNSUPPORTED, THC_ECUDA, THC_EWORKSPACE = 0, -1, -2, -3, -4
THC_F32, THC_BF16 = 0, 1
THC_MAX_WORKERS = 64
STATUS_NONFINITE, STATUS_ZERO_BLOCK, STATUS_WAIT_TIMEOUT = 1, 2, 4

EXPORTS = ("thc_create", "thc_destroy", "thc_sizes", "thc_prepare", "thc_compress",
           "thc_quantize_rotated", "thc_aggregate", "thc_decompress", "thc_aggregate_decompress", "thc_prepare_noalloc",
           "thc_error_feedback", "thc_accumulate_error", "thc_prepare_compress", "thc_prepare_minmax", "thc_debug_skip_tasks", "thc_status", "thc_strerror", "thc_version")
NOALLOC_SCRATCH_BYTES = 4 << 20


class ThcError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class _Config(ctypes.Structure):
    _fields_ = [("bits", ctypes.c_uint32), ("granularity", ctypes.c_uint32),
                ("table", ctypes.c_uint16 * 256), ("t_p", ctypes.c_double),
                ("log2_block", ctypes.c_uint32), ("seed", ctypes.c_uint64),
                ("in_dtype", ctypes.c_uint32), ("workers", ctypes.c_uint32),
                ("acc_bits", ctypes.c_uint32), ("range_mode", ctypes.c_uint32)]


class _Sizes(ctypes.Structure):
    _fields_ = [("d_pad", ctypes.c_uint64), ("nblocks", ctypes.c_uint64),
                ("packed_bytes", ctypes.c_uint64), ("sum_bytes", ctypes.c_uint64),
                ("rotated_bytes", ctypes.c_uint64), ("workspace_bytes", ctypes.c_uint64),
                ("acc_bits", ctypes.c_uint32), ("fused_scales", ctypes.c_uint32),
                ("scales_count", ctypes.c_uint64)]


@dataclass(frozen=True)
class Sizes:
    d_pad: int
    nblocks: int
    packed_bytes: int
    sum_bytes: int
    rotated_bytes: int
    workspace_bytes: int
    acc_bits: int
    fused_scales: int = 0
    scales_count: int = 0


def lib():
    """Load libthc.so (built in-tree by ``python -m paper_2302_08545_b200._build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          "`python -m paper_2302_08545_b200._build`; there is no fallback")
    L = ctypes.CDLL(_LIB_PATH)
    vp, u32, u64 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64
    pp = ctypes.POINTER(ctypes.c_void_p)
    L.thc_create.argtypes = [ctypes.POINTER(_Config), pp]
    L.thc_destroy.argtypes = [vp]
    L.thc_sizes.argtypes = [vp, u64, u32, ctypes.POINTER(_Sizes)]
    L.thc_prepare.argtypes = [vp, pp, u32, u64, vp, vp, u64, vp]
    L.thc_compress.argtypes = [vp, pp, u32, u32, u64, u32, vp, pp, pp, vp, u64, vp]
    L.thc_quantize_rotated.argtypes = [vp, pp, u32, u32, u64, u32, vp, pp, vp]
    L.thc_aggregate.argtypes = [vp, pp, u32, u64, vp, vp]
    L.thc_decompress.argtypes = [vp, vp, u32, u64, u32, vp, vp, vp, u64, vp]
    L.thc_aggregate_decompress.argtypes = [vp, pp, u32, u64, u32, vp, vp, vp, vp, u64, vp]
    L.thc_prepare_noalloc.argtypes = [pp, u32, u64, u32, u32, ctypes.c_double, vp, vp, vp]
    L.thc_prepare_minmax.argtypes = [vp, pp, u32, u64, u32, vp, pp, vp, u64, vp]
    L.thc_prepare_compress.argtypes = [vp, pp, u32, u32, u64, u32, vp, pp, pp, vp, u64, vp]
    L.thc_error_feedback.argtypes = [vp, pp, pp, u32, u64, u32, vp, pp, vp, u64, vp]
    L.thc_accumulate_error.argtypes = [vp, pp, pp, u32, u64, vp]
    L.thc_debug_skip_tasks.argtypes = [vp, u32]
    L.thc_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
    for name in EXPORTS[:-2]:
        getattr(L, name).restype = ctypes.c_int
    L.thc_strerror.argtypes = [ctypes.c_int]
    L.thc_strerror.restype = ctypes.c_char_p
    L.thc_version.argtypes = []
    L.thc_version.restype = ctypes.c_char_p
    _lib = L
    return L


def strerror(code: int) -> str:
    return lib().thc_strerror(code).decode()


def version() -> str:
    return lib().thc_version().decode()


def _check(code: int, where: str):
    if code != THC_OK:
        raise ThcError(code, where)


def _ptr_array(ptrs):
    arr = (ctypes.c_void_p * len(ptrs))(*[ctypes.c_void_p(int(p)) for p in ptrs])
    return arr


def _dp(t) -> int:
    """Device (or host) address of a torch tensor / raw integer address / None."""
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


def prepare_noalloc(grads, d: int, log2_block: int, in_dtype: int, t_p: float, scales,
                    status=None, stream=None):
    """thc_prepare_noalloc: the preliminary stage for callers that may not allocate device
    memory.  No context and no workspace: the scratch is a fixed array inside the library
    (NOALLOC_SCRATCH_BYTES per GPU).  `status` is an optional device uint32 tensor the status
    bits are OR-ed into.  Raises ThcError(THC_EWORKSPACE) when the input is too large for
    the built-in scratch."""
    arr = _ptr_array([_dp(g) for g in grads])
    _check(lib().thc_prepare_noalloc(arr, len(grads), d, log2_block, in_dtype, float(t_p),
                                     _dp(scales), _dp(status), _stream(stream)),
           "thc_prepare_noalloc")


class Context:
    """Owns a ``thc_ctx``.  Methods mirror the C entry points one to one."""

    def __init__(self, bits: int, granularity: int, table, t_p: float, log2_block: int,
                 seed: int, in_dtype: int = THC_F32, workers: int = 8, acc_bits: int = 0,
                 range_mode: int = 0):
        cfg = _Config()
        cfg.bits, cfg.granularity = bits, granularity
        for i, v in enumerate(table):
            cfg.table[i] = int(v)
        cfg.t_p, cfg.log2_block, cfg.seed = float(t_p), log2_block, seed & 0xFFFFFFFFFFFFFFFF
        cfg.in_dtype, cfg.workers, cfg.acc_bits = in_dtype, workers, acc_bits
        cfg.range_mode = range_mode
        self._h = ctypes.c_void_p()
        _check(lib().thc_create(ctypes.byref(cfg), ctypes.byref(self._h)), "thc_create")
        self.bits, self.granularity, self.log2_block = bits, granularity, log2_block
        self.workers = workers

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().thc_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sizes(self, d: int, n_local: int) -> Sizes:
        s = _Sizes()
        _check(lib().thc_sizes(self._h, d, n_local, ctypes.byref(s)), "thc_sizes")
        return Sizes(s.d_pad, s.nblocks, s.packed_bytes, s.sum_bytes, s.rotated_bytes,
                     s.workspace_bytes, s.acc_bits, s.fused_scales, s.scales_count)

    def prepare(self, grads, d: int, scales, workspace, stream=None):
        arr = _ptr_array([_dp(g) for g in grads])
        _check(lib().thc_prepare(self._h, arr, len(grads), d, _dp(scales), _dp(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(stream)),
               "thc_prepare")

    def prepare_minmax(self, grads, d: int, rnd: int, scales, workspace, rotated=None, stream=None):
        arr = _ptr_array([_dp(g) for g in grads])
        ra = _ptr_array([_dp(r) for r in rotated]) if rotated is not None else None
        _check(lib().thc_prepare_minmax(self._h, arr, len(grads), d, rnd, _dp(scales), ra, _dp(workspace),
                                        workspace.numel() * workspace.element_size(), _stream(stream)),
               "thc_prepare_minmax")

    def compress(self, grads, d: int, rnd: int, scales, packed, workspace, rotated=None,
                 worker_base: int = 0, stream=None):
        n = len(grads)
        ga = _ptr_array([_dp(g) for g in grads])
        pa = _ptr_array([_dp(p) for p in packed])
        ra = _ptr_array([_dp(r) for r in rotated]) if rotated is not None else None
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib().thc_compress(self._h, ga, n, worker_base, d, rnd, _dp(scales), pa, ra,
                                  _dp(workspace), ws_bytes, _stream(stream)), "thc_compress")

    def prepare_compress(self, grads, d: int, rnd: int, scales, packed, workspace, rotated=None,
                         worker_base: int = 0, stream=None):
        n = len(grads)
        ga = _ptr_array([_dp(g) for g in grads])
        pa = _ptr_array([_dp(p) for p in packed])
        ra = _ptr_array([_dp(r) for r in rotated]) if rotated is not None else None
        _check(lib().thc_prepare_compress(self._h, ga, n, worker_base, d, rnd, _dp(scales), pa, ra,
                                          _dp(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)), "thc_prepare_compress")

    def quantize_rotated(self, rotated, d: int, rnd: int, scales, packed, worker_base: int = 0,
                         stream=None):
        ra = _ptr_array([_dp(r) for r in rotated])
        pa = _ptr_array([_dp(p) for p in packed])
        _check(lib().thc_quantize_rotated(self._h, ra, len(rotated), worker_base, d, rnd,
                                          _dp(scales), pa, _stream(stream)), "thc_quantize_rotated")

    def aggregate(self, packed, d: int, total, stream=None):
        pa = _ptr_array([_dp(p) for p in packed])
        _check(lib().thc_aggregate(self._h, pa, len(packed), d, _dp(total), _stream(stream)),
               "thc_aggregate")

    def decompress(self, total, divisor: int, d: int, rnd: int, scales, out, workspace,
                   stream=None):
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib().thc_decompress(self._h, _dp(total), divisor, d, rnd, _dp(scales), _dp(out),
                                    _dp(workspace), ws_bytes, _stream(stream)), "thc_decompress")

    def aggregate_decompress(self, packed, d: int, rnd: int, scales, out, workspace, total=None,
                             stream=None):
        pa = _ptr_array([_dp(p) for p in packed])
        ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
        _check(lib().thc_aggregate_decompress(self._h, pa, len(packed), d, rnd, _dp(scales), _dp(out),
                                              _dp(total), _dp(workspace), ws_bytes, _stream(stream)),
               "thc_aggregate_decompress")

    def error_feedback(self, grads, packed, d: int, rnd: int, scales, ef, workspace, stream=None):
        ga = _ptr_array([_dp(g) for g in grads])
        pa = _ptr_array([_dp(p) for p in packed])
        ea = _ptr_array([_dp(e) for e in ef])
        _check(lib().thc_error_feedback(self._h, ga, pa, len(grads), d, rnd, _dp(scales), ea,
                                        _dp(workspace), workspace.numel() * workspace.element_size(),
                                        _stream(stream)), "thc_error_feedback")

    def accumulate_error(self, grads, ef, d: int, stream=None):
        ga = _ptr_array([_dp(g) for g in grads])
        ea = _ptr_array([_dp(e) for e in ef])
        _check(lib().thc_accumulate_error(self._h, ga, ea, len(grads), d, _stream(stream)),
               "thc_accumulate_error")

    def debug_skip_tasks(self, count: int):
        """Test hook: the next pipeline launch starts its task queue at `count`."""
        _check(lib().thc_debug_skip_tasks(self._h, count), "thc_debug_skip_tasks")

    def status(self, stream=None) -> int:
        flags = ctypes.c_uint32(0)
        _check(lib().thc_status(self._h, ctypes.byref(flags), _stream(stream)), "thc_status")
        return flags.value

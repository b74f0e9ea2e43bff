"""ctypes front end of the THC CPU oracle (``thc_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
CPU-baseline / reference legs of ``bench.py``.  The product package never imports it, and
this module never imports the product package.

Everything here is argument marshalling; the arithmetic lives in the C file, whose header
lists the passages of the THC paper it follows and the readings it takes.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "thc_oracle.c")
_LIB = os.path.join(_HERE, "libthc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc.  -ffp-contract=off: only the written fmaf() fuse."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    u8p, u16p, u32p = (ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_uint16),
                       ctypes.POINTER(ctypes.c_uint32))
    f32p, f64p = ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_double)
    u32, u64, vp = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_void_p
    lib.thc_oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
    lib.thc_oracle_philox4x32_10.restype = None
    lib.thc_oracle_sign.argtypes = [u64, u32, u64]
    lib.thc_oracle_sign.restype = ctypes.c_int
    lib.thc_oracle_u16.argtypes = [u64, u32, u32, u64]
    lib.thc_oracle_u16.restype = u32
    lib.thc_oracle_fwht.argtypes = [f32p, u64]
    lib.thc_oracle_fwht.restype = None
    lib.thc_oracle_scales.argtypes = [f32p, u32, u64, u32, ctypes.c_double, f32p]
    lib.thc_oracle_scales.restype = None
    lib.thc_oracle_rht_forward.argtypes = [f32p, u64, u32, u64, u32, f32p]
    lib.thc_oracle_rht_forward.restype = None
    lib.thc_oracle_rht_inverse.argtypes = [f32p, u64, u32, u64, u32, f32p]
    lib.thc_oracle_rht_inverse.restype = None
    lib.thc_oracle_rht_forward_at.argtypes = [f32p, u64, u32, u64, u32, u64, f32p]
    lib.thc_oracle_rht_forward_at.restype = None
    lib.thc_oracle_rht_inverse_at.argtypes = [f32p, u64, u32, u64, u32, u64, f32p]
    lib.thc_oracle_rht_inverse_at.restype = None
    lib.thc_oracle_quantize_at.argtypes = [f32p, u64, u32, f32p, u32, u32, u16p, u64, u32, u32, u64, u8p]
    lib.thc_oracle_quantize_at.restype = None
    lib.thc_oracle_quantize.argtypes = [f32p, u64, u32, f32p, u32, u32, u16p, u64, u32, u32, u8p]
    lib.thc_oracle_quantize.restype = None
    lib.thc_oracle_pack.argtypes = [u8p, u64, u32, u8p]
    lib.thc_oracle_pack.restype = None
    lib.thc_oracle_unpack.argtypes = [u8p, u64, u32, u8p]
    lib.thc_oracle_unpack.restype = None
    lib.thc_oracle_aggregate.argtypes = [u8p, u32, u64, u32, u16p, u32, vp]
    lib.thc_oracle_aggregate.restype = None
    lib.thc_oracle_decompress.argtypes = [vp, u32, u32, u64, u32, f32p, u32, u64, u32, f32p]
    lib.thc_oracle_decompress.restype = None
    lib.thc_oracle_estimate.argtypes = [vp, u32, u32, u64, u32, f32p, u32, f32p]
    lib.thc_oracle_estimate.restype = None
    lib.thc_oracle_error_feedback.argtypes = [f32p, u8p, u64, u32, f32p, u32, u16p, u64, u32, f32p]
    lib.thc_oracle_error_feedback.restype = None
    lib.thc_oracle_dequantize.argtypes = [u8p, u64, u32, f32p, u32, u16p, f64p]
    lib.thc_oracle_dequantize.restype = None
    lib.thc_oracle_quantize_range_at.argtypes = [f32p, u64, u32, f32p, f32p, u32, u32, u16p, u64, u32, u32, u64, u8p]
    lib.thc_oracle_quantize_range_at.restype = None
    lib.thc_oracle_estimate_range.argtypes = [vp, u32, u32, u64, u32, f32p, f32p, u32, f32p]
    lib.thc_oracle_estimate_range.restype = None
    lib.thc_oracle_decompress_range.argtypes = [vp, u32, u32, u64, u32, f32p, f32p, u32, u64, u32, f32p]
    lib.thc_oracle_decompress_range.restype = None
    lib.thc_oracle_error_feedback_range.argtypes = [f32p, u8p, u64, u32, f32p, f32p, u32, u16p, u64, u32, f32p]
    lib.thc_oracle_error_feedback_range.restype = None
    lib.thc_oracle_ranges.argtypes = [f32p, u32, u64, u32, u64, u32, f32p, f32p]
    lib.thc_oracle_ranges.restype = None
    _lib = lib
    return lib


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


@dataclass(frozen=True)
class Config:
    """Parameters of Algorithm 3's input line plus the readings' free choices."""
    bits: int                 # b
    granularity: int          # g
    table: tuple              # T[0..2^b-1]
    t_p: float                # Phi^-1(1 - p/2)
    log2_block: int           # k, RHT block B = 2^k
    seed: int                 # shared by all workers

    @property
    def block(self) -> int:
        return 1 << self.log2_block

    def d_pad(self, d: int) -> int:
        return -(-d // self.block) * self.block

    def table_u16(self) -> np.ndarray:
        t = np.zeros(256, dtype=np.uint16)
        t[:len(self.table)] = self.table
        return t


def acc_bits(n: int, g: int) -> int:
    """Smallest of 8/16/32 bits that holds the largest aggregate n*g (Section 8.4 of the
    paper: the maximal aggregated value is g*n)."""
    for w in (8, 16, 32):
        if n * g <= (1 << w) - 1:
            return w
    raise ValueError("n*g does not fit 32 bits")


def bf16_to_f32(a_u16: np.ndarray) -> np.ndarray:
    """Exact upcast of bfloat16 bit patterns (uint16) to float32."""
    return (a_u16.astype(np.uint32) << 16).view(np.float32)


# ---------------------------------------------------------------------------------------
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _load().thc_oracle_philox4x32_10(_p(c, ctypes.c_uint32), _p(k, ctypes.c_uint32),
                                     _p(out, ctypes.c_uint32))
    return out


def sign(seed: int, rnd: int, j: int) -> int:
    return int(_load().thc_oracle_sign(seed, rnd, j))


def signs(seed: int, rnd: int, j0: int, count: int) -> np.ndarray:
    lib = _load()
    return np.array([lib.thc_oracle_sign(seed, rnd, j0 + t) for t in range(count)], dtype=np.int8)


def u16(seed: int, rnd: int, worker: int, j: int) -> int:
    return int(_load().thc_oracle_u16(seed, rnd, worker, j))


def fwht(v) -> np.ndarray:
    """Unnormalised H_B v (fp32, radix-2, ascending stride)."""
    a = _f32(v).copy()
    assert a.ndim == 1 and a.size & (a.size - 1) == 0
    _load().thc_oracle_fwht(_p(a, ctypes.c_float), a.size)
    return a


def scales(x, cfg: Config) -> np.ndarray:
    """M per block from the [n, d] worker gradients (Section 5.3)."""
    x = _f32(x)
    n, d = x.shape
    nb = cfg.d_pad(d) // cfg.block
    out = np.zeros(nb, dtype=np.float32)
    _load().thc_oracle_scales(_p(x, ctypes.c_float), n, d, cfg.log2_block, cfg.t_p,
                              _p(out, ctypes.c_float))
    return out


def ranges(x, cfg: Config, rnd: int):
    """Exact (lo, hi) per RHT block of the rotated coordinates over all workers (Algorithm 1's
    preliminary stage applied after the rotation).  x is [n, d]."""
    x = _f32(x)
    n, d = x.shape
    nb = cfg.d_pad(d) // cfg.block
    lo = np.zeros(nb, dtype=np.float32)
    hi = np.zeros(nb, dtype=np.float32)
    _load().thc_oracle_ranges(_p(x, ctypes.c_float), n, d, cfg.log2_block, cfg.seed, rnd,
                              _p(lo, ctypes.c_float), _p(hi, ctypes.c_float))
    return lo, hi


def rht_forward(x, cfg: Config, rnd: int, j_base: int = 0) -> np.ndarray:
    """j_base: padded coordinate of x[0] in the whole vector (a multiple of the block), for
    transforming a slice of a long vector."""
    x = _f32(x)
    d = x.size
    assert j_base % cfg.block == 0
    r = np.zeros(cfg.d_pad(d), dtype=np.float32)
    _load().thc_oracle_rht_forward_at(_p(x, ctypes.c_float), d, cfg.log2_block, cfg.seed, rnd,
                                      j_base, _p(r, ctypes.c_float))
    return r


def rht_inverse(v, d: int, cfg: Config, rnd: int, j_base: int = 0) -> np.ndarray:
    v = _f32(v).copy()
    assert v.size == cfg.d_pad(d) and j_base % cfg.block == 0
    out = np.zeros(d, dtype=np.float32)
    _load().thc_oracle_rht_inverse_at(_p(v, ctypes.c_float), d, cfg.log2_block, cfg.seed, rnd,
                                      j_base, _p(out, ctypes.c_float))
    return out


def quantize(r, scl, cfg: Config, rnd: int, worker: int, j_base: int = 0, lo=None) -> np.ndarray:
    """Rotated coordinates -> one table index per coordinate (uint8, unpacked).  With j_base,
    r is a slice starting at that padded coordinate and scl[0] is the scale of its block.
    With lo, the range of a block is [lo, scl] (Algorithm 1's exact range) instead of
    [-scl, scl]."""
    r = _f32(r)
    scl = _f32(scl)
    assert j_base % cfg.block == 0
    z = np.zeros(r.size, dtype=np.uint8)
    t = cfg.table_u16()
    if lo is not None:
        lo = _f32(lo)
        _load().thc_oracle_quantize_range_at(_p(r, ctypes.c_float), r.size, cfg.log2_block,
                                             _p(lo, ctypes.c_float), _p(scl, ctypes.c_float),
                                             cfg.bits, cfg.granularity, _p(t, ctypes.c_uint16),
                                             cfg.seed, rnd, worker, j_base, _p(z, ctypes.c_uint8))
        return z
    _load().thc_oracle_quantize_at(_p(r, ctypes.c_float), r.size, cfg.log2_block,
                                   _p(scl, ctypes.c_float), cfg.bits, cfg.granularity,
                                   _p(t, ctypes.c_uint16), cfg.seed, rnd, worker, j_base,
                                   _p(z, ctypes.c_uint8))
    return z


def pack(z, bits: int) -> np.ndarray:
    z = np.ascontiguousarray(z, dtype=np.uint8)
    out = np.zeros(z.size * bits // 8, dtype=np.uint8)
    _load().thc_oracle_pack(_p(z, ctypes.c_uint8), z.size, bits, _p(out, ctypes.c_uint8))
    return out


def unpack(packed, d_pad: int, bits: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    z = np.zeros(d_pad, dtype=np.uint8)
    _load().thc_oracle_unpack(_p(packed, ctypes.c_uint8), d_pad, bits, _p(z, ctypes.c_uint8))
    return z


def aggregate(packed, d_pad: int, cfg: Config, w: int) -> np.ndarray:
    """[n, d_pad*b/8] packed indices -> d_pad sums of table values (uint of w bits)."""
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    assert packed.shape[1] == d_pad * cfg.bits // 8
    out = np.zeros(d_pad, dtype={8: np.uint8, 16: np.uint16, 32: np.uint32}[w])
    t = cfg.table_u16()
    _load().thc_oracle_aggregate(_p(packed, ctypes.c_uint8), n, d_pad, cfg.bits,
                                 _p(t, ctypes.c_uint16), w, out.ctypes.data_as(ctypes.c_void_p))
    return out


def decompress(total, divisor: int, d: int, scl, cfg: Config, rnd: int, lo=None) -> np.ndarray:
    total = np.ascontiguousarray(total)
    w = total.dtype.itemsize * 8
    scl = _f32(scl)
    out = np.zeros(d, dtype=np.float32)
    if lo is not None:
        lo = _f32(lo)
        _load().thc_oracle_decompress_range(total.ctypes.data_as(ctypes.c_void_p), w, divisor, d,
                                            cfg.log2_block, _p(lo, ctypes.c_float),
                                            _p(scl, ctypes.c_float), cfg.granularity, cfg.seed, rnd,
                                            _p(out, ctypes.c_float))
        return out
    _load().thc_oracle_decompress(total.ctypes.data_as(ctypes.c_void_p), w, divisor, d,
                                  cfg.log2_block, _p(scl, ctypes.c_float), cfg.granularity,
                                  cfg.seed, rnd, _p(out, ctypes.c_float))
    return out


def estimate(total, divisor: int, scl, cfg: Config, lo=None) -> np.ndarray:
    """Algorithm 2's 'Estimate' line: the averaged vector, still in the rotated domain."""
    total = np.ascontiguousarray(total)
    w = total.dtype.itemsize * 8
    scl = _f32(scl)
    v = np.zeros(total.size, dtype=np.float32)
    if lo is not None:
        lo = _f32(lo)
        _load().thc_oracle_estimate_range(total.ctypes.data_as(ctypes.c_void_p), w, divisor,
                                          total.size, cfg.log2_block, _p(lo, ctypes.c_float),
                                          _p(scl, ctypes.c_float), cfg.granularity,
                                          _p(v, ctypes.c_float))
        return v
    _load().thc_oracle_estimate(total.ctypes.data_as(ctypes.c_void_p), w, divisor, total.size,
                                cfg.log2_block, _p(scl, ctypes.c_float), cfg.granularity,
                                _p(v, ctypes.c_float))
    return v


def error_feedback(x, z, scl, cfg: Config, rnd: int, lo=None) -> np.ndarray:
    """e = x - RHT^-1(X) for one worker (Algorithm 3): x has d entries, z d_pad indices."""
    x = _f32(x)
    z = np.ascontiguousarray(z, dtype=np.uint8)
    scl = _f32(scl)
    assert z.size == cfg.d_pad(x.size)
    e = np.zeros(x.size, dtype=np.float32)
    t = cfg.table_u16()
    if lo is not None:
        lo = _f32(lo)
        _load().thc_oracle_error_feedback_range(_p(x, ctypes.c_float), _p(z, ctypes.c_uint8), x.size,
                                                cfg.log2_block, _p(lo, ctypes.c_float),
                                                _p(scl, ctypes.c_float), cfg.granularity,
                                                _p(t, ctypes.c_uint16), cfg.seed, rnd,
                                                _p(e, ctypes.c_float))
        return e
    _load().thc_oracle_error_feedback(_p(x, ctypes.c_float), _p(z, ctypes.c_uint8), x.size,
                                      cfg.log2_block, _p(scl, ctypes.c_float), cfg.granularity,
                                      _p(t, ctypes.c_uint16), cfg.seed, rnd, _p(e, ctypes.c_float))
    return e


def dequantize(z, scl, cfg: Config) -> np.ndarray:
    """Real value each index stands for, before the inverse RHT (float64)."""
    z = np.ascontiguousarray(z, dtype=np.uint8)
    scl = _f32(scl)
    out = np.zeros(z.size, dtype=np.float64)
    t = cfg.table_u16()
    _load().thc_oracle_dequantize(_p(z, ctypes.c_uint8), z.size, cfg.log2_block,
                                  _p(scl, ctypes.c_float), cfg.granularity,
                                  _p(t, ctypes.c_uint16), _p(out, ctypes.c_double))
    return out


# ---------------------------------------------------------------------------------------
def compress(x, scl, cfg: Config, rnd: int, worker_base: int = 0, lo=None):
    """All of a worker's compress step for each row of x: returns (packed [n, bytes],
    rotated [n, d_pad])."""
    x = _f32(x)
    n, d = x.shape
    d_pad = cfg.d_pad(d)
    rotated = np.zeros((n, d_pad), dtype=np.float32)
    packed = np.zeros((n, d_pad * cfg.bits // 8), dtype=np.uint8)
    for i in range(n):
        rotated[i] = rht_forward(x[i], cfg, rnd)
        packed[i] = pack(quantize(rotated[i], scl, cfg, rnd, worker_base + i, lo=lo), cfg.bits)
    return packed, rotated


def thc_round(x, cfg: Config, rnd: int = 0, scl=None, exact_range: bool = False):
    """One whole round (Algorithm 3, THC lines): returns a dict with every stage.  With
    exact_range the clamp range is the exact min/max of the rotated coordinates (Algorithm 1's
    preliminary stage) instead of the norm-based [-M, M] of Section 5.3."""
    x = _f32(x)
    n, d = x.shape
    lo = None
    if exact_range:
        lo, scl = ranges(x, cfg, rnd)
    elif scl is None:
        scl = scales(x, cfg)
    packed, rotated = compress(x, scl, cfg, rnd, lo=lo)
    w = acc_bits(n, cfg.granularity)
    total = aggregate(packed, cfg.d_pad(d), cfg, w)
    out = decompress(total, n, d, scl, cfg, rnd, lo=lo)
    return {"lo": lo, "scales": scl, "rotated": rotated, "packed": packed, "sum": total, "out": out,
            "acc_bits": w}

"""CPU oracle of the TAH-Quant boundary codec: TEST INFRASTRUCTURE, not the product.

Thin ctypes face of ``tahq_oracle.c`` (plain scalar C written from the paper,
Sec. 3.1-3.4).  Only ``tests/``, the smoke check and the benchmark's CPU
baseline import this package.  The CUDA library and its Python binding never
do, and nothing here imports them.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tahq_oracle.c")
_SRC_Q = os.path.join(_HERE, "qnaive_oracle.c")
_HDR_Q = os.path.join(_HERE, "qnaive_oracle.h")
_HDR = os.path.join(_HERE, "tahq_oracle.h")
_LIB = os.path.join(_HERE, "libtahq_oracle.so")

F32, BF16 = 0, 1


class _Params(C.Structure):
    _fields_ = [
        ("dtype", C.c_uint32),
        ("tokens", C.c_uint64),
        ("hidden", C.c_uint32),
        ("group_tokens", C.c_uint32),
        ("tile", C.c_uint32),
        ("budget_millibits", C.c_uint32),
        ("tau", C.c_float),
        ("eps_l1", C.c_float),
        ("eps_log", C.c_float),
        ("eps_ratio", C.c_float),
        ("rounding", C.c_uint32),
        ("seed", C.c_uint64),
        ("alloc_tile", C.c_uint32),
    ]


class _Layout(C.Structure):
    _fields_ = [
        ("n_tiles", C.c_uint64),
        ("n_groups", C.c_uint64),
        ("tiles_per_group", C.c_uint64),
        ("k_hi", C.c_uint64),
        ("lo_bits", C.c_uint32),
        ("hi_bits", C.c_uint32),
        ("off_bitmap", C.c_uint64),
        ("off_scale_zero", C.c_uint64),
        ("off_pivot", C.c_uint64),
        ("off_payload", C.c_uint64),
        ("payload_bytes", C.c_uint64),
        ("total_bytes", C.c_uint64),
    ]


class _QParams(C.Structure):
    _fields_ = [("dtype", C.c_uint32), ("tokens", C.c_uint64), ("hidden", C.c_uint32), ("bits", C.c_uint32),
                ("per_tensor", C.c_uint32), ("prescale", C.c_float)]


class _QLayout(C.Structure):
    _fields_ = [("n_scales", C.c_uint64), ("off_scales", C.c_uint64), ("off_payload", C.c_uint64),
                ("row_bytes", C.c_uint64), ("total_bytes", C.c_uint64)]


@dataclass
class QNaiveParams:
    """Fixed-point gradient compressor of Algorithm 1 line 6 (b bits, per-token or per-tensor scale, pre-scale c)."""

    tokens: int
    hidden: int
    dtype: int = F32
    bits: int = 8
    per_tensor: int = 0
    prescale: float = 1.0

    def c(self) -> _QParams:
        return _QParams(self.dtype, self.tokens, self.hidden, self.bits, self.per_tensor, self.prescale)


@dataclass
class Params:
    """Configuration of one boundary tensor (names follow the paper: G, S, tau, ...)."""

    tokens: int
    hidden: int
    dtype: int = F32
    group_tokens: int = 0
    tile: int = 64
    budget_millibits: int = 3800
    tau: float = 2.0
    eps_l1: float = 1e-8
    eps_log: float = 1e-8
    eps_ratio: float = 1e-8
    rounding: int = 0
    seed: int = 0
    alloc_tile: int = 0          # A of Sec. 3.2 (0 = the quantisation tile)

    def c(self) -> _Params:
        return _Params(self.dtype, self.tokens, self.hidden, self.group_tokens, self.tile,
                       self.budget_millibits, self.tau, self.eps_l1, self.eps_log, self.eps_ratio,
                       self.rounding, self.seed, self.alloc_tile)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction, no fast-math); returns the library path."""
    newest = max(os.path.getmtime(f) for f in (_SRC, _HDR, _SRC_Q, _HDR_Q))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, _SRC_Q, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp = C.POINTER(C.c_float)
        L.tahqo_layout_of.argtypes = [C.POINTER(_Params), C.POINTER(_Layout)]
        L.tahqo_layout_of.restype = C.c_int
        L.tahqo_packed_bound.argtypes = [C.POINTER(_Params)]
        L.tahqo_packed_bound.restype = C.c_size_t
        L.tahqo_encode.argtypes = [C.POINTER(_Params), C.c_void_p, C.c_void_p, C.c_size_t]
        L.tahqo_encode.restype = C.c_int
        L.tahqo_decode.argtypes = [C.POINTER(_Params), C.c_void_p, C.c_size_t, C.c_void_p]
        L.tahqo_decode.restype = C.c_int
        L.tahqo_treesum.argtypes = [fp, C.c_uint32]
        L.tahqo_treesum.restype = C.c_float
        L.tahqo_lg2_array.argtypes = [fp, fp, C.c_size_t]
        L.tahqo_score.argtypes = [fp, C.c_uint32, C.c_float, C.c_float]
        L.tahqo_score.restype = C.c_float
        L.tahqo_allocate.argtypes = [fp, C.c_uint64, C.c_uint64, C.c_void_p]
        L.tahqo_pivot.argtypes = [fp, C.c_uint32, C.c_float, C.c_float,
                                  C.POINTER(C.c_uint32), C.POINTER(C.c_int)]
        L.tahqo_swap_hadamard.argtypes = [fp, C.c_uint32, C.c_uint32]
        L.tahqo_f32_to_f16.argtypes = [C.c_float]
        L.tahqo_f32_to_f16.restype = C.c_uint16
        L.tahqo_f16_to_f32.argtypes = [C.c_uint16]
        L.tahqo_f16_to_f32.restype = C.c_float
        L.tahqo_f32_to_bf16.argtypes = [C.c_float]
        L.tahqo_f32_to_bf16.restype = C.c_uint16
        L.tahqo_range.argtypes = [fp, C.c_uint32, C.c_uint32,
                                  C.POINTER(C.c_uint16), C.POINTER(C.c_uint16)]
        L.tahqo_quantise.argtypes = [fp, C.c_uint32, C.c_uint32, C.c_uint16, C.c_uint16,
                                     C.c_uint32, C.c_uint64, C.c_uint64, C.POINTER(C.c_uint32)]
        L.tahqo_philox4x32_10.argtypes = [C.POINTER(C.c_uint32)] * 3
        L.qnaiveo_layout_of.argtypes = [C.POINTER(_QParams), C.POINTER(_QLayout)]
        L.qnaiveo_layout_of.restype = C.c_int
        L.qnaiveo_packed_bound.argtypes = [C.POINTER(_QParams)]
        L.qnaiveo_packed_bound.restype = C.c_size_t
        L.qnaiveo_encode.argtypes = [C.POINTER(_QParams), C.c_void_p, C.c_void_p, C.c_size_t]
        L.qnaiveo_encode.restype = C.c_int
        L.qnaiveo_decode.argtypes = [C.POINTER(_QParams), C.c_void_p, C.c_size_t, C.c_void_p]
        L.qnaiveo_decode.restype = C.c_int
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def set_threads(n: int) -> None:
    """Number of host threads for the per-tile loops of encode/decode (OpenMP)."""
    os.environ["OMP_NUM_THREADS"] = str(n)
    try:
        C.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
    except OSError:
        pass


def layout(p: Params) -> dict:
    out = _Layout()
    pc = p.c()
    if lib().tahqo_layout_of(C.byref(pc), C.byref(out)):
        raise ValueError("invalid TAH-Quant parameters")
    return {k: int(getattr(out, k)) for k, _ in _Layout._fields_}


def packed_bound(p: Params) -> int:
    pc = p.c()
    return int(lib().tahqo_packed_bound(C.byref(pc)))


def _as_input(p: Params, x: np.ndarray) -> np.ndarray:
    """fp32 tensors as float32 arrays; bf16 tensors as uint16 arrays holding the bf16 bit patterns."""
    want = np.float32 if p.dtype == F32 else np.uint16
    x = np.ascontiguousarray(x)
    if x.dtype != want:
        raise TypeError(f"expected {want} array for dtype {p.dtype}, got {x.dtype}")
    if x.size != p.tokens * p.hidden:
        raise ValueError("array size does not match tokens x hidden")
    return x


def encode(p: Params, x: np.ndarray) -> np.ndarray:
    x = _as_input(p, x)
    n = packed_bound(p)
    if n == 0:
        raise ValueError("invalid TAH-Quant parameters")
    out = np.empty(n, dtype=np.uint8)
    pc = p.c()
    rc = lib().tahqo_encode(C.byref(pc), x.ctypes.data, out.ctypes.data, n)
    if rc:
        raise RuntimeError(f"oracle encode failed: {rc}")
    return out


def decode(p: Params, packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty(p.tokens * p.hidden, dtype=np.float32 if p.dtype == F32 else np.uint16)
    pc = p.c()
    rc = lib().tahqo_decode(C.byref(pc), packed.ctypes.data, packed.size, out.ctypes.data)
    if rc:
        raise RuntimeError(f"oracle decode failed: {rc}")
    return out.reshape(p.tokens, p.hidden)


# ---- single steps (for the pins) -------------------------------------------------

def treesum(x) -> float:
    x = _f32(x)
    return float(lib().tahqo_treesum(_fp(x), x.size))


def lg2(x) -> np.ndarray:
    x = _f32(x)
    y = np.empty_like(x)
    lib().tahqo_lg2_array(_fp(x), _fp(y), x.size)
    return y


def score(tile, eps_l1=1e-8, eps_log=1e-8) -> float:
    t = _f32(tile)
    return float(lib().tahqo_score(_fp(t), t.size, eps_l1, eps_log))


def allocate(scores, k_hi: int) -> np.ndarray:
    s = _f32(scores)
    out = np.zeros(s.size, dtype=np.uint8)
    lib().tahqo_allocate(_fp(s), s.size, k_hi, out.ctypes.data)
    return out


def pivot(tile, tau=2.0, eps_ratio=1e-8):
    t = _f32(tile)
    d, f = C.c_uint32(), C.c_int()
    lib().tahqo_pivot(_fp(t), t.size, tau, eps_ratio, C.byref(d), C.byref(f))
    return int(d.value), bool(f.value)


def swap_hadamard(tile, d: int) -> np.ndarray:
    t = _f32(tile).copy()
    lib().tahqo_swap_hadamard(_fp(t), t.size, d)
    return t


def f32_to_f16(x: float) -> int:
    return int(lib().tahqo_f32_to_f16(float(x)))


def f16_to_f32(h: int) -> float:
    return float(lib().tahqo_f16_to_f32(int(h)))


def f32_to_bf16(x: float) -> int:
    return int(lib().tahqo_f32_to_bf16(float(x)))


def tile_range(v, bits: int):
    v = _f32(v)
    s, z = C.c_uint16(), C.c_uint16()
    lib().tahqo_range(_fp(v), v.size, bits, C.byref(s), C.byref(z))
    return int(s.value), int(z.value)


def quantise(v, bits: int, s_h: int, z_h: int, rounding=0, seed=0, first_elem=0) -> np.ndarray:
    v = _f32(v)
    q = np.empty(v.size, dtype=np.uint32)
    lib().tahqo_quantise(_fp(v), v.size, bits, s_h, z_h, rounding, seed, first_elem,
                         q.ctypes.data_as(C.POINTER(C.c_uint32)))
    return q


def philox4x32_10(key, ctr) -> np.ndarray:
    k = (C.c_uint32 * 2)(*key)
    c = (C.c_uint32 * 4)(*ctr)
    o = (C.c_uint32 * 4)()
    lib().tahqo_philox4x32_10(k, c, o)
    return np.array(list(o), dtype=np.uint32)


# ---------------------------------------------------------------- fixed-point gradient compressor
def qnaive_layout(p: QNaiveParams) -> dict:
    L = _QLayout()
    if lib().qnaiveo_layout_of(C.byref(p.c()), C.byref(L)):
        raise ValueError("invalid parameters")
    return {f: getattr(L, f) for f, _ in _QLayout._fields_}


def qnaive_packed_bound(p: QNaiveParams) -> int:
    return int(lib().qnaiveo_packed_bound(C.byref(p.c())))


def qnaive_encode(p: QNaiveParams, x: np.ndarray) -> np.ndarray:
    want = np.uint16 if p.dtype == BF16 else np.float32
    x = np.ascontiguousarray(x)
    if x.dtype != want or x.size != p.tokens * p.hidden:
        raise ValueError("input does not match the parameters")
    n = qnaive_packed_bound(p)
    if n == 0:
        raise ValueError("invalid parameters")
    out = np.empty(n, dtype=np.uint8)
    rc = lib().qnaiveo_encode(C.byref(p.c()), x.ctypes.data, out.ctypes.data, n)
    if rc:
        raise RuntimeError(f"qnaiveo_encode failed: {rc}")
    return out


def qnaive_decode(p: QNaiveParams, packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.empty((p.tokens, p.hidden), dtype=np.uint16 if p.dtype == BF16 else np.float32)
    rc = lib().qnaiveo_decode(C.byref(p.c()), packed.ctypes.data, packed.size, out.ctypes.data)
    if rc:
        raise RuntimeError(f"qnaiveo_decode failed: {rc}")
    return out

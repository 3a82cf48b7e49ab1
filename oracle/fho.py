"""ctypes binding of the CPU oracle (oracle/fho.c).

Test infrastructure only: tests, the smoke check and the benchmark's CPU-baseline leg load this
module; the CUDA library never does.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fho.c")
_LIB = os.path.join(_HERE, "libfho.so")

OK, ERR_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_NONFINITE, ERR_CORRUPT = 0, -1, -2, -3, -4, -5
F32, BF16 = 0, 1
AUTO, OFF, ALL, CHANNEL, TENSOR = 0, 1, 2, 3, 4
NORMAL, SALIENT, RAW = 0, 1, 2


class Desc(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("n", C.c_int32), ("c", C.c_int32), ("h", C.c_int32),
                ("w", C.c_int32), ("tensor_id", C.c_uint64)]


class Params(C.Structure):
    _fields_ = [("bits", C.c_int32), ("salient_mode", C.c_int32), ("rho_num", C.c_int32),
                ("rho_den", C.c_int32), ("block", C.c_int32), ("tau_num", C.c_int32),
                ("tau_den", C.c_int32), ("eps", C.c_float), ("dense_bits", C.c_int32),
                ("rounding", C.c_int32), ("seed", C.c_uint64), ("entropy", C.c_int32), ("reserved", C.c_int32)]


def params(bits=2, salient_mode=AUTO, rho=(1, 32), block=8, tau=(1, 4), eps=0.0625, dense_bits=8,
           rounding=0, seed=0, entropy=0) -> Params:
    return Params(bits, salient_mode, rho[0], rho[1], block, tau[0], tau[1], eps, dense_bits,
                  rounding, seed, entropy, 0)


def desc(shape, dtype=F32, tensor_id=0) -> Desc:
    n, c, h, w = shape
    return Desc(dtype, n, c, h, w, tensor_id)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, no contraction of a*b+c, OpenMP over planes)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.fho_compressed_bytes.restype = C.c_size_t
        L.fho_compressed_bytes.argtypes = [C.POINTER(Desc), C.POINTER(Params), C.c_int]
        L.fho_compress.restype = C.c_int
        L.fho_compress.argtypes = [C.POINTER(Desc), C.POINTER(Params), C.c_void_p, C.c_void_p,
                                   C.c_size_t, C.POINTER(C.c_uint64)]
        L.fho_decompress.restype = C.c_int
        L.fho_decompress.argtypes = [C.c_void_p, C.c_size_t, C.POINTER(Desc), C.c_void_p]
        L.fho_plane_sigma.restype = None
        L.fho_plane_sigma.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_float), C.POINTER(C.c_float),
                                      C.POINTER(C.c_float), C.POINTER(C.c_int64)]
        L.fho_channel_sigma.restype = None
        L.fho_channel_sigma.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(C.c_float),
                                        C.POINTER(C.c_float), C.POINTER(C.c_float), C.POINTER(C.c_int64)]
        L.fho_plane_sums.restype = None
        L.fho_plane_sums.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                     C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.fho_quant_params.restype = None
        L.fho_quant_params.argtypes = [C.c_float, C.c_float, C.c_int, C.POINTER(C.c_float),
                                       C.POINTER(C.c_float)]
        L.fho_quant_code.restype = C.c_uint32
        L.fho_quant_code.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int]
        L.fho_dequant.restype = C.c_float
        L.fho_dequant.argtypes = [C.c_uint32, C.c_float, C.c_float]
        L.fho_philox4x32_10.restype = None
        L.fho_philox4x32_10.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.fho_quant_code_random.restype = C.c_uint32
        L.fho_quant_code_random.argtypes = [C.c_float, C.c_float, C.c_float, C.c_int, C.c_uint32]
        L.fho_huffman_lengths.restype = None
        L.fho_huffman_lengths.argtypes = [C.POINTER(C.c_uint32), C.POINTER(C.c_uint8)]
        L.fho_canonical_codes.restype = None
        L.fho_canonical_codes.argtypes = [C.POINTER(C.c_uint8), C.POINTER(C.c_uint32)]
        L.fho_set_threads.argtypes = [C.c_int]
        L.fho_max_threads.restype = C.c_int
        L.fho_get_threads.restype = C.c_int
        _lib = L
    return _lib


def set_threads(t: int) -> None:
    lib().fho_set_threads(int(t))


def max_threads() -> int:
    return int(lib().fho_max_threads())


def compressed_bytes(d: Desc, p: Params, which: int = 0) -> int:
    return int(lib().fho_compressed_bytes(C.byref(d), C.byref(p), which))


def compress(x: np.ndarray, d: Desc, p: Params, capacity: int | None = None) -> Tuple[int, np.ndarray, int]:
    """x: flat float32 (F32) or uint16 bit patterns (BF16).  Returns (status, packed bytes, total)."""
    x = np.ascontiguousarray(x)
    assert x.dtype == (np.float32 if d.dtype == F32 else np.uint16)
    assert x.size == d.n * d.c * d.h * d.w
    cap = compressed_bytes(d, p, 1) if capacity is None else capacity
    dst = np.zeros(max(cap, 1), dtype=np.uint8)
    out2 = (C.c_uint64 * 2)()
    st = lib().fho_compress(C.byref(d), C.byref(p), x.ctypes.data, dst.ctypes.data, cap, out2)
    total = int(out2[0])
    return st, (dst[:total] if st == OK else dst[:cap]), total


def decompress(packed: np.ndarray, d: Desc, nbytes: int | None = None) -> Tuple[int, np.ndarray]:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.zeros(d.n * d.c * d.h * d.w, dtype=np.float32 if d.dtype == F32 else np.uint16)
    st = lib().fho_decompress(packed.ctypes.data, packed.size if nbytes is None else nbytes,
                              C.byref(d), out.ctypes.data)
    return st, out


def plane_sigma(x: np.ndarray):
    """Three-sigma statistics of one plane: (lo, d_lo, d_hi, n_out) -- the smallest element, the two
    thresholds as fp32 distances from it, and the number of elements outside them."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    lo, dlo, dhi = C.c_float(), C.c_float(), C.c_float()
    n = C.c_int64()
    lib().fho_plane_sigma(x.ctypes.data, x.size, C.byref(lo), C.byref(dlo), C.byref(dhi), C.byref(n))
    return lo.value, dlo.value, dhi.value, n.value


def channel_sigma(x: np.ndarray):
    """x: (n_planes, hw) float32, the planes in scope (a channel over the batch, or a whole tensor).
    Returns (lo, d_lo, d_hi, n_out)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    lo, dlo, dhi = C.c_float(), C.c_float(), C.c_float()
    n = C.c_int64()
    lib().fho_channel_sigma(x.ctypes.data, x.shape[0], x.shape[1], x.shape[1], C.byref(lo), C.byref(dlo), C.byref(dhi),
                            C.byref(n))
    return lo.value, dlo.value, dhi.value, n.value


def plane_sums(x: np.ndarray):
    """Integer moment sums of a plane's distances from its minimum: (I_s, I_q, e, applies)."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    a, b = C.c_int64(), C.c_int64()
    e, ap = C.c_int32(), C.c_int32()
    lib().fho_plane_sums(x.ctypes.data, x.size, C.byref(a), C.byref(b), C.byref(e), C.byref(ap))
    return a.value, b.value, e.value, ap.value


def quant_params(lo: float, hi: float, bits: int):
    inv, scale = C.c_float(), C.c_float()
    lib().fho_quant_params(lo, hi, bits, C.byref(inv), C.byref(scale))
    return inv.value, scale.value


def quant_code(x: float, lo: float, inv: float, bits: int) -> int:
    return int(lib().fho_quant_code(x, lo, inv, bits))


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*ctr)
    k = (C.c_uint32 * 2)(*key)
    o = (C.c_uint32 * 4)()
    lib().fho_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def quant_code_random(x: float, lo: float, inv: float, bits: int, word: int) -> int:
    return int(lib().fho_quant_code_random(x, lo, inv, bits, word))


def huffman_lengths(hist):
    """Code lengths (256 uint8) of the Huffman code of a 256-bin histogram."""
    h = (C.c_uint32 * 256)(*[int(v) for v in hist])
    out = (C.c_uint8 * 256)()
    lib().fho_huffman_lengths(h, out)
    return [int(v) for v in out]


def canonical_codes(lengths):
    """Canonical code values of a list of 256 code lengths (0 where the length is 0)."""
    l = (C.c_uint8 * 256)(*[int(v) for v in lengths])
    out = (C.c_uint32 * 256)()
    lib().fho_canonical_codes(l, out)
    return [int(v) for v in out]


def dequant(q: int, lo: float, scale: float) -> float:
    return float(lib().fho_dequant(q, lo, scale))


# ---- container parsing helpers (layout knowledge for tests; reads only) ----------------------

def parse_header(buf: np.ndarray) -> dict:
    b = np.ascontiguousarray(buf[:64], dtype=np.uint8).tobytes()
    import struct
    magic, ver, dtype, bits, N, Cc, H, W, block, dense_bits, rounding, mode, rn, rd, tn, td, eps, \
        n_sal, n_raw, tid, total = struct.unpack("<IHBBIIIIBBBBHHHHfIIQQ", b)
    return dict(magic=magic, version=ver, dtype=dtype, bits=bits, n=N, c=Cc, h=H, w=W, block=block,
                dense_bits=dense_bits, rounding=rounding, salient_mode=mode, rho=(rn, rd),
                tau=(tn, td), eps=eps, n_salient=n_sal, n_raw=n_raw, tensor_id=tid,
                total_bytes=total)


def parse_table(buf: np.ndarray, P: int):
    """Returns (off16 u32[P], cls u32[P], n_out u32[P], lo f32[P], scale f32[P])."""
    t = np.ascontiguousarray(buf[64:64 + 16 * P], dtype=np.uint8).view(np.uint32).reshape(P, 4)
    return t[:, 0].copy(), t[:, 1] & 3, t[:, 1] >> 2, t[:, 2].copy().view(np.float32), \
        t[:, 3].copy().view(np.float32)

"""ctypes binding of the CPU oracle (oracle/entro_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module,
and this module never imports the product package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import NamedTuple, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "entro_oracle.c")
_SO = os.path.join(_HERE, "libentro_oracle.so")

MODE_AUTO, MODE_UNSIGNED, MODE_ASYMMETRIC = 0, 1, 2
SUB_BLOCKS = 32
ERRORS = {1: "bad argument", 2: "buffer too small", 3: "non-finite weight", 4: "code longer than 32 bits",
          5: "corrupt stream"}


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"oracle error {code}: {ERRORS.get(code, '?')}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp32 kept strict: no contraction, no fast-math)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-pthread", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


class _QParams(C.Structure):
    _fields_ = [("bits", C.c_int32), ("mode", C.c_int32), ("scale", C.c_float),
                ("zero_point", C.c_int32), ("lo", C.c_float), ("hi", C.c_float)]


class QParams(NamedTuple):
    bits: int
    mode: int
    scale: float        # exactly representable fp32 value
    zero_point: int
    lo: float
    hi: float


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, u16p, u32p, u64p = (C.POINTER(t) for t in (C.c_uint8, C.c_uint16, C.c_uint32, C.c_uint64))
        f64p = C.POINTER(C.c_double)
        L.oracle_f16_to_f32.restype = C.c_float
        L.oracle_f16_to_f32.argtypes = [C.c_uint16]
        L.oracle_f32_to_f16_rne.restype = C.c_uint16
        L.oracle_f32_to_f16_rne.argtypes = [C.c_float]
        L.oracle_f16_to_f32_array.restype = None
        L.oracle_f16_to_f32_array.argtypes = [u16p, C.c_uint64, C.POINTER(C.c_float)]
        L.oracle_f32_to_f16_array.restype = None
        L.oracle_f32_to_f16_array.argtypes = [C.POINTER(C.c_float), C.c_uint64, u16p]
        L.oracle_quant_params.argtypes = [u16p, C.c_uint64, C.c_int, C.c_int, C.POINTER(_QParams)]
        L.oracle_quantize_one.restype = C.c_uint8
        L.oracle_quantize_one.argtypes = [C.c_uint16, C.c_float, C.c_int, C.c_int]
        L.oracle_quantize_tensor.argtypes = [u16p, C.c_uint64, C.c_int, C.c_int, u8p, C.POINTER(_QParams)]
        L.oracle_quantize_blocks.argtypes = [u16p, C.c_uint64, C.c_int, C.c_int, C.c_uint64, u8p,
                                             C.POINTER(C.c_float), C.POINTER(C.c_int32)]
        L.oracle_dequant_one.restype = C.c_uint16
        L.oracle_dequant_one.argtypes = [C.c_uint8, C.c_float, C.c_int]
        L.oracle_dequant.restype = None
        L.oracle_dequant.argtypes = [u8p, C.c_uint64, C.c_float, C.c_int, u16p]
        L.oracle_histogram.argtypes = [u8p, C.c_uint64, C.c_int, u64p]
        L.oracle_huffman_lengths.argtypes = [u64p, C.c_int, u8p]
        L.oracle_length_limited_lengths.argtypes = [u64p, C.c_int, C.c_int, u8p]
        L.oracle_canonical_codes.argtypes = [u8p, C.c_int, u32p]
        L.oracle_num_chunks.restype = C.c_uint64
        L.oracle_num_chunks.argtypes = [C.c_uint64, C.c_uint32]
        L.oracle_encode.argtypes = [u8p, C.c_uint64, u8p, u32p, C.c_int, C.c_uint32, u32p, C.c_uint64,
                                    u64p, u16p, u64p]
        L.oracle_decode_dequant.argtypes = [u32p, u64p, C.c_uint64, C.c_uint32, u8p, C.c_int, C.c_float,
                                            C.c_int, u8p, u16p]
        L.oracle_decode_dequant_chunks.argtypes = [u32p, u64p, C.c_uint64, C.c_uint32, u8p, C.c_int,
                                                   C.c_float, C.c_int, u64p, C.c_uint64, u8p, u16p]
        L.oracle_decode_dequant_mt.argtypes = [u32p, u64p, C.c_uint64, C.c_uint32, u8p, C.c_int,
                                               C.c_float, C.c_int, u16p, C.c_int]
        L.oracle_gemv_f64.restype = None
        L.oracle_gemv_f64.argtypes = [u16p, C.c_uint64, C.c_uint64, u16p, f64p, f64p]
        _lib = L
    return _lib


def _ptr(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ctype))


def _check(rc: int) -> None:
    if rc:
        raise OracleError(rc)


def _as_u16(w: np.ndarray) -> np.ndarray:
    """fp16 array (or raw uint16 bit patterns) -> flat contiguous uint16 view."""
    w = np.ascontiguousarray(w)
    if w.dtype == np.float16:
        w = w.view(np.uint16)
    assert w.dtype == np.uint16
    return w.reshape(-1)


# ----------------------------------------------------------------------------- scalar helpers

def f16_to_f32(h: int) -> float:
    return float(lib().oracle_f16_to_f32(int(h)))


def f32_to_f16(f: float) -> int:
    return int(lib().oracle_f32_to_f16_rne(C.c_float(f)))


def f16_to_f32_array(h: np.ndarray) -> np.ndarray:
    h = _as_u16(h)
    f = np.empty(h.size, dtype=np.float32)
    lib().oracle_f16_to_f32_array(_ptr(h, C.c_uint16), h.size, _ptr(f, C.c_float))
    return f


def f32_to_f16_array(f: np.ndarray) -> np.ndarray:
    f = np.ascontiguousarray(f, dtype=np.float32).reshape(-1)
    h = np.empty(f.size, dtype=np.uint16)
    lib().oracle_f32_to_f16_array(_ptr(f, C.c_float), f.size, _ptr(h, C.c_uint16))
    return h


def quantize_one(w_bits: int, s: float, z: int, bits: int) -> int:
    return int(lib().oracle_quantize_one(int(w_bits), C.c_float(s), int(z), int(bits)))


def dequant_one(q: int, s: float, z: int) -> int:
    return int(lib().oracle_dequant_one(int(q), C.c_float(s), int(z)))


# ----------------------------------------------------------------------------- stages

def quant_params(w: np.ndarray, bits: int, mode: int = MODE_AUTO) -> QParams:
    w = _as_u16(w)
    qp = _QParams()
    _check(lib().oracle_quant_params(_ptr(w, C.c_uint16), w.size, bits, mode, C.byref(qp)))
    return QParams(qp.bits, qp.mode, qp.scale, qp.zero_point, qp.lo, qp.hi)


def quantize_tensor(w: np.ndarray, bits: int, mode: int = MODE_AUTO):
    """-> (q uint8 [n], QParams)"""
    w = _as_u16(w)
    q = np.empty(w.size, dtype=np.uint8)
    qp = _QParams()
    _check(lib().oracle_quantize_tensor(_ptr(w, C.c_uint16), w.size, bits, mode, _ptr(q, C.c_uint8),
                                        C.byref(qp)))
    return q, QParams(qp.bits, qp.mode, qp.scale, qp.zero_point, qp.lo, qp.hi)


def quantize_blocks(w: np.ndarray, bits: int, block: int, mode: int = MODE_AUTO):
    """Block-based quantisation, the paper's comparison grid (Section 3, Table 2 "SOTA"): every run of
    `block` weights by itself.  -> (q uint8 [n], scales float32 [blocks], zero points int32 [blocks])"""
    w = _as_u16(w)
    nb = (w.size + block - 1) // block
    q = np.empty(w.size, dtype=np.uint8)
    scales = np.empty(nb, dtype=np.float32)
    zps = np.empty(nb, dtype=np.int32)
    _check(lib().oracle_quantize_blocks(_ptr(w, C.c_uint16), w.size, bits, mode, block, _ptr(q, C.c_uint8),
                                        _ptr(scales, C.c_float), _ptr(zps, C.c_int32)))
    return q, scales, zps


def dequant(q: np.ndarray, s: float, z: int) -> np.ndarray:
    """-> fp16 bit patterns (uint16)"""
    q = np.ascontiguousarray(q, dtype=np.uint8).reshape(-1)
    out = np.empty(q.size, dtype=np.uint16)
    lib().oracle_dequant(_ptr(q, C.c_uint8), q.size, C.c_float(s), int(z), _ptr(out, C.c_uint16))
    return out


def histogram(q: np.ndarray, nsym: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8).reshape(-1)
    counts = np.zeros(nsym, dtype=np.uint64)
    _check(lib().oracle_histogram(_ptr(q, C.c_uint8), q.size, nsym, _ptr(counts, C.c_uint64)))
    return counts


def huffman_lengths(counts: Sequence[int]) -> np.ndarray:
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    ln = np.zeros(counts.size, dtype=np.uint8)
    _check(lib().oracle_huffman_lengths(_ptr(counts, C.c_uint64), counts.size, _ptr(ln, C.c_uint8)))
    return ln


def length_limited_lengths(counts: Sequence[int], max_len: int) -> np.ndarray:
    """Optimal code lengths with no code longer than max_len (package-merge)."""
    counts = np.ascontiguousarray(counts, dtype=np.uint64)
    ln = np.zeros(counts.size, dtype=np.uint8)
    _check(lib().oracle_length_limited_lengths(_ptr(counts, C.c_uint64), counts.size, int(max_len), _ptr(ln, C.c_uint8)))
    return ln


def canonical_codes(lengths: Sequence[int]) -> np.ndarray:
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    code = np.zeros(ln.size, dtype=np.uint32)
    _check(lib().oracle_canonical_codes(_ptr(ln, C.c_uint8), ln.size, _ptr(code, C.c_uint32)))
    return code


def num_chunks(n: int, chunk_symbols: int) -> int:
    return (n + chunk_symbols - 1) // chunk_symbols


class Encoded(NamedTuple):
    stream: np.ndarray      # uint32 words, zero padded
    offsets: np.ndarray     # uint64 [n_chunks + 1]
    sub_len: np.ndarray     # uint16 [n_chunks, 32]
    total_bits: int


def encode(q: np.ndarray, lengths: np.ndarray, codes: np.ndarray, chunk_symbols: int,
           slack_words: int = 8) -> Encoded:
    q = np.ascontiguousarray(q, dtype=np.uint8).reshape(-1)
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    cd = np.ascontiguousarray(codes, dtype=np.uint32)
    bits = int(ln.astype(np.int64)[q].sum()) if q.size else 0
    cap = (bits + 31) // 32 + slack_words
    stream = np.zeros(max(cap, 1), dtype=np.uint32)
    nch = num_chunks(q.size, chunk_symbols)
    offsets = np.zeros(nch + 1, dtype=np.uint64)
    sub_len = np.zeros((nch, SUB_BLOCKS), dtype=np.uint16)
    total = C.c_uint64(0)
    _check(lib().oracle_encode(_ptr(q, C.c_uint8), q.size, _ptr(ln, C.c_uint8), _ptr(cd, C.c_uint32),
                               ln.size, chunk_symbols, _ptr(stream, C.c_uint32), stream.size,
                               _ptr(offsets, C.c_uint64), _ptr(sub_len, C.c_uint16), C.byref(total)))
    return Encoded(stream, offsets, sub_len, int(total.value))


def decode_dequant(stream: np.ndarray, offsets: np.ndarray, n: int, chunk_symbols: int,
                   lengths: np.ndarray, s: float, z: int, want_q: bool = True, want_out: bool = True,
                   chunk_ids: Optional[Sequence[int]] = None, threads: int = 0):
    """Bit-serial decode + dequant.  -> (q uint8 or None, out uint16 fp16-bits or None).
    chunk_ids: decode only these chunks (others left zero).  threads > 0: the
    thread-per-segment driver (fp16 output only)."""
    stream = np.ascontiguousarray(stream, dtype=np.uint32)
    offsets = np.ascontiguousarray(offsets, dtype=np.uint64)
    ln = np.ascontiguousarray(lengths, dtype=np.uint8)
    q = np.zeros(n, dtype=np.uint8) if want_q else None
    out = np.zeros(n, dtype=np.uint16) if want_out else None
    L = lib()
    if threads > 0:
        assert out is not None and chunk_ids is None
        _check(L.oracle_decode_dequant_mt(_ptr(stream, C.c_uint32), _ptr(offsets, C.c_uint64), n,
                                          chunk_symbols, _ptr(ln, C.c_uint8), ln.size, C.c_float(s), int(z),
                                          _ptr(out, C.c_uint16), threads))
        return None, out
    if chunk_ids is None:
        _check(L.oracle_decode_dequant(_ptr(stream, C.c_uint32), _ptr(offsets, C.c_uint64), n, chunk_symbols,
                                       _ptr(ln, C.c_uint8), ln.size, C.c_float(s), int(z),
                                       _ptr(q, C.c_uint8), _ptr(out, C.c_uint16)))
    else:
        ids = np.ascontiguousarray(chunk_ids, dtype=np.uint64)
        _check(L.oracle_decode_dequant_chunks(_ptr(stream, C.c_uint32), _ptr(offsets, C.c_uint64), n,
                                              chunk_symbols, _ptr(ln, C.c_uint8), ln.size, C.c_float(s),
                                              int(z), _ptr(ids, C.c_uint64), ids.size,
                                              _ptr(q, C.c_uint8), _ptr(out, C.c_uint16)))
    return q, out


def gemv_f64(w_hat: np.ndarray, rows: int, cols: int, x: np.ndarray):
    """-> (y fp64 [rows], sum_i |w x| fp64 [rows]) over fp16 operands."""
    w_hat = _as_u16(w_hat)
    x = _as_u16(x)
    assert w_hat.size == rows * cols and x.size == cols
    y = np.zeros(rows, dtype=np.float64)
    a = np.zeros(rows, dtype=np.float64)
    lib().oracle_gemv_f64(_ptr(w_hat, C.c_uint16), rows, cols, _ptr(x, C.c_uint16), _ptr(y, C.c_double),
                          _ptr(a, C.c_double))
    return y, a


class Compressed(NamedTuple):
    qp: QParams
    q: np.ndarray
    counts: np.ndarray
    lengths: np.ndarray
    codes: np.ndarray
    enc: Encoded


def compress(w: np.ndarray, bits: int, chunk_symbols: int, mode: int = MODE_AUTO) -> Compressed:
    """The offline side in the paper's order: quantise, count, build the code, encode."""
    q, qp = quantize_tensor(w, bits, mode)
    counts = histogram(q, 1 << bits)
    lengths = huffman_lengths(counts)
    codes = canonical_codes(lengths)
    enc = encode(q, lengths, codes, chunk_symbols)
    return Compressed(qp, q, counts, lengths, codes, enc)

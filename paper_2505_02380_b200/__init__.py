"""Python binding of the entro C-ABI library (include/entro.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch is used for device memory and streams.  There is no CPU
fallback: loading fails loudly if the compiled library is missing, and every
call raises EntroError on a non-zero status.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, NamedTuple, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# The checked build (libentro_checked.so, see build.py) is loaded instead when ENTRO_LIBRARY names it.
LIB_PATH = os.environ.get("ENTRO_LIBRARY") or os.path.join(_HERE, "libentro.so")

MAX_SYMBOLS = 256
SUB_BLOCKS = 32
STREAM_SLACK_WORDS = 8
MAX_CODE_LEN = 32
MAX_CHUNK_SYMBOLS = 16384
MODE_AUTO, MODE_UNSIGNED, MODE_ASYMMETRIC = 0, 1, 2

OK, ERR_INVALID_ARG, ERR_BUFFER_TOO_SMALL, ERR_NONFINITE, ERR_CODE_TOO_LONG, ERR_CORRUPT_STREAM, ERR_CUDA, \
    ERR_UNSUPPORTED, ERR_TOO_MANY_TENSORS = range(9)
STATIC_MAX_TENSORS = 8
GEMV_MAX_BATCH = 8
DEFAULT_DECODE_CONFIG = (12, 32, 1, 1792)   # lut_bits, warps_per_cta, ctas_per_sm, chunks_per_item


class EntroError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: entro status {status} ({status_string(status)})")
        self.status = status


class QParams(C.Structure):
    _fields_ = [("bits", C.c_int32), ("mode", C.c_int32), ("scale", C.c_float), ("zero_point", C.c_int32),
                ("lo", C.c_float), ("hi", C.c_float)]


class Codebook(C.Structure):
    _fields_ = [("nsym", C.c_int32), ("max_len", C.c_int32), ("len", C.c_uint8 * MAX_SYMBOLS),
                ("code", C.c_uint32 * MAX_SYMBOLS)]

    def lengths(self) -> np.ndarray:
        return np.frombuffer(self.len, dtype=np.uint8, count=self.nsym).copy()

    def codes(self) -> np.ndarray:
        return np.frombuffer(self.code, dtype=np.uint32, count=self.nsym).copy()

    @staticmethod
    def from_lengths(lengths: Sequence[int], codes: Optional[Sequence[int]] = None) -> "Codebook":
        cb = Codebook()
        cb.nsym = len(lengths)
        cb.max_len = int(max(lengths))
        for k, l in enumerate(lengths):
            cb.len[k] = int(l)
        if codes is not None:
            for k, c in enumerate(codes):
                cb.code[k] = int(c)
        return cb


class TensorDesc(C.Structure):
    _fields_ = [("stream_dev", C.c_void_p), ("stream_words", C.c_uint64), ("index_dev", C.c_void_p),
                ("n", C.c_uint64), ("chunk_symbols", C.c_uint32), ("scale", C.c_float),
                ("zero_point", C.c_int32), ("cb", Codebook), ("out_fp16_dev", C.c_void_p)]


class GemvIO(C.Structure):
    _fields_ = [("rows", C.c_uint32), ("cols", C.c_uint32), ("x_fp16_dev", C.c_void_p), ("y_fp16_dev", C.c_void_p),
                ("batch", C.c_uint32), ("reserved", C.c_uint32)]


class QuantizeJob(C.Structure):
    _fields_ = [("w_fp16_dev", C.c_void_p), ("n", C.c_uint64), ("bits", C.c_int32), ("mode", C.c_int32),
                ("q_dev", C.c_void_p)]


class EncodeJob(C.Structure):
    _fields_ = [("q_dev", C.c_void_p), ("n", C.c_uint64), ("cb_host", C.POINTER(Codebook)), ("chunk_symbols", C.c_uint32),
                ("reserved", C.c_uint32), ("stream_dev", C.c_void_p), ("stream_cap_words", C.c_uint64),
                ("index_dev", C.c_void_p), ("index_cap_bytes", C.c_uint64)]


class HostIO(C.Structure):
    _fields_ = [("stream_host", C.c_void_p), ("index_host", C.c_void_p), ("out_fp16_host", C.c_void_p)]


_lib = None


def lib():
    """The loaded library.  Raises if it has not been built (python -m paper_2505_02380_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_02380_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(LIB_PATH)
        vp, u64, u32, i32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int
        L.entro_quantize_tensor.argtypes = [vp, u64, i32, i32, vp, C.POINTER(QParams), vp]
        L.entro_histogram.argtypes = [vp, u64, i32, C.POINTER(C.c_uint64), vp]
        L.entro_quantize_blocks.argtypes = [vp, u64, i32, i32, u32, vp, vp, vp, vp]
        L.entro_build_codebook.argtypes = [C.POINTER(C.c_uint64), i32, C.POINTER(Codebook)]
        L.entro_build_codebook_limited.argtypes = [C.POINTER(C.c_uint64), i32, i32, C.POINTER(Codebook)]
        L.entro_stream_words.restype = u64
        L.entro_stream_words.argtypes = [C.POINTER(C.c_uint64), C.POINTER(Codebook)]
        L.entro_encode_bound_words.restype = u64
        L.entro_encode_bound_words.argtypes = [u64, C.POINTER(Codebook)]
        L.entro_index_bytes.restype = u64
        L.entro_index_bytes.argtypes = [u64, u32]
        L.entro_encode.argtypes = [vp, u64, C.POINTER(Codebook), u32, vp, u64, vp, u64, C.POINTER(C.c_uint64), vp]
        L.entro_quantize_histogram_batched.argtypes = [C.POINTER(QuantizeJob), i32, C.POINTER(QParams),
                                                       C.POINTER(C.c_uint64), vp]
        L.entro_encode_batched.argtypes = [C.POINTER(EncodeJob), i32, C.POINTER(C.c_uint64), vp]
        L.entro_decode_dequant.argtypes = [vp, u64, vp, u64, u32, C.POINTER(Codebook), C.c_float, C.c_int32, vp, vp]
        L.entro_decode_dequant_batched.argtypes = [C.POINTER(TensorDesc), i32, vp]
        L.entro_decode_dequant_batched_host.argtypes = [C.POINTER(TensorDesc), C.POINTER(HostIO), i32, vp]
        L.entro_decode_symbols_batched.argtypes = [C.POINTER(TensorDesc), i32, i32, vp]
        L.entro_decode_dequant_gemv.argtypes = [C.POINTER(TensorDesc), C.POINTER(GemvIO), i32, vp]
        L.entro_gemv_prepare.argtypes = [C.POINTER(TensorDesc), C.POINTER(GemvIO), i32, vp, C.POINTER(vp)]
        L.entro_gemv_run.argtypes = [vp, vp]
        L.entro_gemv_release.argtypes = [vp]
        L.entro_gemv_fp16.argtypes = [vp, u32, u32, vp, vp, vp]
        L.entro_decode_dequant_static.argtypes = [C.POINTER(TensorDesc), i32, vp, vp]
        L.entro_last_device_status.argtypes = [vp]
        L.entro_set_decode_config.argtypes = [i32, i32, i32, i32]
        L.entro_profile_begin.argtypes = [i32]
        L.entro_profile_read.restype = i32
        L.entro_profile_read.argtypes = [C.POINTER(C.c_float), i32]
        L.entro_checked_build.restype = i32
        L.entro_checked_build.argtypes = []
        L.entro_check_violations.restype = C.c_longlong
        L.entro_check_violations.argtypes = []
        L.entro_kernel_launch_count.restype = u64
        L.entro_kernel_launch_count.argtypes = []
        L.entro_status_string.restype = C.c_char_p
        L.entro_status_string.argtypes = [i32]
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


# Every symbol include/entro.h declares.
EXPORTS = ["entro_quantize_tensor", "entro_quantize_blocks", "entro_histogram", "entro_build_codebook", "entro_build_codebook_limited", "entro_stream_words",
           "entro_encode_bound_words", "entro_index_bytes", "entro_encode", "entro_quantize_histogram_batched",
           "entro_encode_batched", "entro_decode_dequant",
           "entro_decode_dequant_batched", "entro_decode_dequant_batched_host", "entro_decode_dequant_static",
           "entro_decode_dequant_gemv", "entro_gemv_prepare", "entro_gemv_run", "entro_gemv_release", "entro_gemv_fp16", "entro_decode_symbols_batched", "entro_last_device_status",
           "entro_set_decode_config", "entro_checked_build", "entro_check_violations", "entro_profile_begin", "entro_profile_read", "entro_kernel_launch_count",
           "entro_status_string"]


def status_string(status: int) -> str:
    return lib().entro_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise EntroError(status, what)


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype) -> int:
    assert t.is_cuda and t.is_contiguous() and t.dtype == dtype, (t.device, t.dtype, dtype)
    return t.data_ptr()


# ----------------------------------------------------------------------------- thin wrappers, same names

def entro_quantize_tensor(w_fp16: torch.Tensor, bits: int, mode: int = MODE_AUTO,
                          stream: Optional[torch.cuda.Stream] = None):
    """-> (q uint8 device tensor, one symbol per byte; QParams)"""
    n = w_fp16.numel()
    q = torch.empty(n, dtype=torch.uint8, device=w_fp16.device)
    qp = QParams()
    _check(lib().entro_quantize_tensor(_dev(w_fp16, torch.float16), n, bits, mode, q.data_ptr(), C.byref(qp),
                                       _stream(stream)), "entro_quantize_tensor")
    return q, qp


def entro_quantize_blocks(w_fp16: torch.Tensor, bits: int, block: int = 32, mode: int = MODE_AUTO,
                          stream: Optional[torch.cuda.Stream] = None):
    """Block-based quantisation, the paper's comparison grid.
    -> (q uint8 device tensor, scales float32 [blocks], zero points int32 [blocks])"""
    n = w_fp16.numel()
    nb = (n + block - 1) // block
    q = torch.empty(n, dtype=torch.uint8, device=w_fp16.device)
    scales = torch.empty(nb, dtype=torch.float32, device=w_fp16.device)
    zps = torch.empty(nb, dtype=torch.int32, device=w_fp16.device)
    _check(lib().entro_quantize_blocks(_dev(w_fp16, torch.float16), n, bits, mode, block, q.data_ptr(),
                                       scales.data_ptr(), zps.data_ptr(), _stream(stream)), "entro_quantize_blocks")
    return q, scales, zps


def entro_histogram(q: torch.Tensor, bits: int, stream: Optional[torch.cuda.Stream] = None) -> np.ndarray:
    counts = (C.c_uint64 * (1 << bits))()
    _check(lib().entro_histogram(_dev(q, torch.uint8), q.numel(), bits, counts, _stream(stream)), "entro_histogram")
    return np.frombuffer(counts, dtype=np.uint64).copy()


def entro_build_codebook(counts: Sequence[int]) -> Codebook:
    arr = (C.c_uint64 * len(counts))(*[int(c) for c in counts])
    cb = Codebook()
    _check(lib().entro_build_codebook(arr, len(counts), C.byref(cb)), "entro_build_codebook")
    return cb


def entro_build_codebook_limited(counts: Sequence[int], max_len: int) -> Codebook:
    """Canonical codebook of the cheapest code with no code longer than max_len."""
    arr = (C.c_uint64 * len(counts))(*[int(c) for c in counts])
    cb = Codebook()
    _check(lib().entro_build_codebook_limited(arr, len(counts), int(max_len), C.byref(cb)), "entro_build_codebook_limited")
    return cb


def entro_index_bytes(n: int, chunk_symbols: int) -> int:
    return int(lib().entro_index_bytes(n, chunk_symbols))


def entro_stream_words(counts: Sequence[int], cb: Codebook) -> int:
    arr = (C.c_uint64 * len(counts))(*[int(c) for c in counts])
    return int(lib().entro_stream_words(arr, C.byref(cb)))


def entro_encode_bound_words(n: int, cb: Codebook) -> int:
    return int(lib().entro_encode_bound_words(n, C.byref(cb)))


class Encoded(NamedTuple):
    stream: torch.Tensor     # int32 words on the device (bit patterns of the uint32 stream)
    index: torch.Tensor      # uint8 bytes on the device: offsets then sub-block lengths
    total_bits: int
    n: int
    chunk_symbols: int

    @property
    def n_chunks(self) -> int:
        return (self.n + self.chunk_symbols - 1) // self.chunk_symbols

    def offsets(self) -> np.ndarray:
        return self.index[:8 * (self.n_chunks + 1)].cpu().numpy().view(np.uint64)

    def sub_len(self) -> np.ndarray:
        return self.index[8 * (self.n_chunks + 1):].cpu().numpy().view(np.uint16).reshape(-1, SUB_BLOCKS)

    def stream_np(self) -> np.ndarray:
        return self.stream.cpu().numpy().view(np.uint32)


def entro_encode(q: torch.Tensor, cb: Codebook, chunk_symbols: int, stream_words: Optional[int] = None,
                 stream: Optional[torch.cuda.Stream] = None) -> Encoded:
    """stream_words: capacity of the stream buffer (default: the bound for n symbols of max_len bits)."""
    n = q.numel()
    cap = stream_words if stream_words is not None else entro_encode_bound_words(n, cb)
    sbuf = torch.empty(cap, dtype=torch.int32, device=q.device)
    ibytes = entro_index_bytes(n, chunk_symbols)
    if ibytes == 0:
        raise EntroError(ERR_INVALID_ARG, "entro_index_bytes")
    ibuf = torch.empty(ibytes, dtype=torch.uint8, device=q.device)
    total = C.c_uint64(0)
    _check(lib().entro_encode(_dev(q, torch.uint8), n, C.byref(cb), chunk_symbols, sbuf.data_ptr(), cap,
                              ibuf.data_ptr(), ibytes, C.byref(total), _stream(stream)), "entro_encode")
    return Encoded(sbuf, ibuf, int(total.value), n, chunk_symbols)


def entro_quantize_histogram_batched(ws: Sequence[torch.Tensor], bits: int, mode: int = MODE_AUTO,
                                     stream: Optional[torch.cuda.Stream] = None,
                                     qs: Optional[Sequence[torch.Tensor]] = None):
    """Quantise every fp16 device tensor of ws and count its symbols, one synchronisation for all.
    qs: the uint8 device tensors that receive the symbols (new ones if not given).
    -> (qs, qps: list of QParams, counts: uint64 array [len(ws), 256])"""
    n = len(ws)
    if qs is None:
        qs = [torch.empty(w.numel(), dtype=torch.uint8, device=w.device) for w in ws]
    jobs = (QuantizeJob * n)()
    for j, (w, q) in enumerate(zip(ws, qs)):
        jobs[j] = QuantizeJob(_dev(w, torch.float16), w.numel(), bits, mode, q.data_ptr())
    qps = (QParams * n)()
    counts = np.zeros((n, MAX_SYMBOLS), dtype=np.uint64)
    _check(lib().entro_quantize_histogram_batched(jobs, n, qps, counts.ctypes.data_as(C.POINTER(C.c_uint64)),
                                                  _stream(stream)), "entro_quantize_histogram_batched")
    return qs, list(qps), counts


def entro_encode_batched(qs: Sequence[torch.Tensor], cbs: Sequence[Codebook], chunk_symbols: int,
                         stream_words: Sequence[int], stream: Optional[torch.cuda.Stream] = None,
                         bufs: Optional[Sequence] = None) -> List[Encoded]:
    """entro_encode for every (q, codebook), one synchronisation for all.  stream_words[j]: capacity
    of tensor j's stream buffer (entro_stream_words of its counts).  bufs[j] = (int32 stream tensor of
    stream_words[j] words, uint8 index tensor of entro_index_bytes bytes) if the caller brings the
    buffers (for instance slices of two large allocations)."""
    n = len(qs)
    jobs = (EncodeJob * n)()
    given = bufs is not None
    bufs = list(bufs) if given else []
    for j, (q, cb) in enumerate(zip(qs, cbs)):
        ibytes = entro_index_bytes(q.numel(), chunk_symbols)
        if ibytes == 0:
            raise EntroError(ERR_INVALID_ARG, "entro_index_bytes")
        if given:
            sbuf, ibuf = bufs[j]
            assert sbuf.numel() == int(stream_words[j]) and ibuf.numel() == ibytes
        else:
            sbuf = torch.empty(int(stream_words[j]), dtype=torch.int32, device=q.device)
            ibuf = torch.empty(ibytes, dtype=torch.uint8, device=q.device)
            bufs.append((sbuf, ibuf))
        jobs[j] = EncodeJob(_dev(q, torch.uint8), q.numel(), C.pointer(cb), chunk_symbols, 0, _dev(sbuf, torch.int32),
                            sbuf.numel(), _dev(ibuf, torch.uint8), ibytes)
    totals = (C.c_uint64 * n)()
    _check(lib().entro_encode_batched(jobs, n, totals, _stream(stream)), "entro_encode_batched")
    return [Encoded(sbuf, ibuf, int(totals[j]), qs[j].numel(), chunk_symbols) for j, (sbuf, ibuf) in enumerate(bufs)]


def entro_stream_words_np(counts_row: np.ndarray, cb: Codebook) -> int:
    """entro_stream_words on a row of the counts array of entro_quantize_histogram_batched."""
    return int(lib().entro_stream_words(counts_row.ctypes.data_as(C.POINTER(C.c_uint64)), C.byref(cb)))


def entro_build_codebook_np(counts_row: np.ndarray, nsym: int) -> Codebook:
    """entro_build_codebook on a row of that counts array (no conversion to a list)."""
    cb = Codebook()
    _check(lib().entro_build_codebook(counts_row.ctypes.data_as(C.POINTER(C.c_uint64)), nsym, C.byref(cb)),
           "entro_build_codebook")
    return cb


def entro_decode_dequant(stream_words: torch.Tensor, index: torch.Tensor, n: int, chunk_symbols: int, cb: Codebook,
                         scale: float, zero_point: int, out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Asynchronous.  -> fp16 device tensor of n values."""
    if out is None:
        out = torch.empty(n, dtype=torch.float16, device=stream_words.device)
    _check(lib().entro_decode_dequant(_dev(stream_words, torch.int32), stream_words.numel(),
                                      _dev(index, torch.uint8), n, chunk_symbols, C.byref(cb), C.c_float(scale),
                                      int(zero_point), _dev(out, torch.float16), _stream(stream)),
           "entro_decode_dequant")
    return out


def make_desc(stream_words: torch.Tensor, index: torch.Tensor, n: int, chunk_symbols: int, cb: Codebook,
              scale: float, zero_point: int, out: torch.Tensor) -> TensorDesc:
    d = TensorDesc()
    d.stream_dev = _dev(stream_words, torch.int32)
    d.stream_words = stream_words.numel()
    d.index_dev = _dev(index, torch.uint8)
    d.n = n
    d.chunk_symbols = chunk_symbols
    d.scale = scale
    d.zero_point = zero_point
    d.cb = cb
    d.out_fp16_dev = _dev(out, torch.float16)
    return d


def desc_array(descs: List[TensorDesc]):
    return (TensorDesc * len(descs))(*descs)


def entro_decode_dequant_batched(descs, stream: Optional[torch.cuda.Stream] = None) -> None:
    """descs: a ctypes array from desc_array() (or a list of TensorDesc).  Asynchronous."""
    if isinstance(descs, list):
        descs = desc_array(descs)
    _check(lib().entro_decode_dequant_batched(descs, len(descs), _stream(stream)), "entro_decode_dequant_batched")


def make_desc_bytes(stream_words: torch.Tensor, index: torch.Tensor, n: int, chunk_symbols: int, cb: Codebook,
                    out: torch.Tensor) -> TensorDesc:
    """A descriptor for entro_decode_symbols_batched: out is a uint8 device tensor."""
    d = make_desc_no_out(stream_words, index, n, chunk_symbols, cb, 1.0, 0)
    d.out_fp16_dev = _dev(out, torch.uint8)
    return d


def entro_decode_symbols_batched(descs, packed: bool = False, stream: Optional[torch.cuda.Stream] = None) -> None:
    """Decode to integer symbols (one per byte, or two 4-bit symbols per byte).  Asynchronous."""
    if isinstance(descs, list):
        descs = desc_array(descs)
    _check(lib().entro_decode_symbols_batched(descs, len(descs), 1 if packed else 0, _stream(stream)),
           "entro_decode_symbols_batched")


def entro_decode_dequant_batched_host(descs, io, stream: Optional[torch.cuda.Stream] = None) -> None:
    """descs, io: ctypes arrays of TensorDesc / HostIO of equal length.  Synchronises."""
    _check(lib().entro_decode_dequant_batched_host(descs, io, len(descs), _stream(stream)),
           "entro_decode_dequant_batched_host")


def make_desc_no_out(stream_words: torch.Tensor, index: torch.Tensor, n: int, chunk_symbols: int, cb: Codebook,
                     scale: float, zero_point: int) -> TensorDesc:
    """A descriptor for the fused matrix-vector call, which writes no fp16 weights."""
    d = TensorDesc()
    d.stream_dev = _dev(stream_words, torch.int32)
    d.stream_words = stream_words.numel()
    d.index_dev = _dev(index, torch.uint8)
    d.n = n
    d.chunk_symbols = chunk_symbols
    d.scale = scale
    d.zero_point = zero_point
    d.cb = cb
    d.out_fp16_dev = None
    return d


def _gemv_batch(x: torch.Tensor) -> int:
    return int(x.shape[0]) if x.dim() == 2 else 1


def make_gemv_io(xs: Sequence[torch.Tensor], ys: Sequence[torch.Tensor], shapes: Sequence):
    """The ctypes array entro_decode_dequant_gemv takes, for callers that repeat a call and want
    to marshal once.  shapes[i] = (rows, cols) of W_i; xs[i] holds cols fp16 values (one token)
    or [batch, cols] (a small batch), ys[i] rows or [batch, rows]."""
    n = len(xs)
    io = (GemvIO * n)()
    for i in range(n):
        io[i] = GemvIO(int(shapes[i][0]), int(shapes[i][1]), _dev(xs[i], torch.float16), _dev(ys[i], torch.float16),
                       _gemv_batch(xs[i]), 0)
    return io


def entro_decode_dequant_gemv(descs, xs: Optional[Sequence[torch.Tensor]] = None, shapes: Optional[Sequence] = None,
                              ys: Optional[List[torch.Tensor]] = None, stream: Optional[torch.cuda.Stream] = None,
                              io=None):
    """descs[i]: compressed W_i of shape shapes[i] = (rows, cols); xs[i]: fp16 vector of cols values,
    or [batch, cols] for a batch of up to GEMV_MAX_BATCH tokens.  -> fp16 y_i = W_i x_i, rows values or
    [batch, rows] (the ys given, or new ones).  Pass io = make_gemv_io(...) instead of xs / shapes / ys
    to skip the marshalling.  Asynchronous."""
    if isinstance(descs, list):
        descs = desc_array(descs)
    n = len(descs)
    if io is None:
        if ys is None:
            ys = [torch.empty((xs[i].shape[0], shapes[i][0]) if xs[i].dim() == 2 else shapes[i][0],
                              dtype=torch.float16, device=xs[i].device) for i in range(n)]
        io = make_gemv_io(xs, ys, shapes)
    _check(lib().entro_decode_dequant_gemv(descs, io, n, _stream(stream)), "entro_decode_dequant_gemv")
    return ys


class GemvPlan:
    """Handle of entro_gemv_prepare: keeps the descriptors, x and y alive for as long as the plan
    holds their device pointers."""

    def __init__(self, handle: int, keep):
        self.handle, self._keep = handle, keep

    def release(self) -> None:
        if self.handle:
            _check(lib().entro_gemv_release(self.handle), "entro_gemv_release")
            self.handle = None

    def __del__(self):
        try:
            self.release()
        except Exception:
            pass


def entro_gemv_prepare(descs, xs: Optional[Sequence[torch.Tensor]] = None, shapes: Optional[Sequence] = None,
                       ys: Optional[List[torch.Tensor]] = None, stream: Optional[torch.cuda.Stream] = None, io=None):
    """Arguments as for entro_decode_dequant_gemv.  -> (GemvPlan, ys).  Every entro_gemv_run(plan)
    reads xs (refreshed in place by the caller) and writes ys."""
    if isinstance(descs, list):
        descs = desc_array(descs)
    n = len(descs)
    if io is None:
        if ys is None:
            ys = [torch.empty((xs[i].shape[0], shapes[i][0]) if xs[i].dim() == 2 else shapes[i][0],
                              dtype=torch.float16, device=xs[i].device) for i in range(n)]
        io = make_gemv_io(xs, ys, shapes)
    handle = C.c_void_p()
    _check(lib().entro_gemv_prepare(descs, io, n, _stream(stream), C.byref(handle)), "entro_gemv_prepare")
    return GemvPlan(handle.value, (descs, xs, ys, io)), ys


def entro_gemv_run(plan: GemvPlan, stream: Optional[torch.cuda.Stream] = None) -> None:
    """One launch: decode + dequantise + multiply + round into the plan's ys.  Asynchronous."""
    _check(lib().entro_gemv_run(plan.handle, _stream(stream)), "entro_gemv_run")


def entro_gemv_release(plan: GemvPlan) -> None:
    plan.release()


def entro_gemv_fp16(w: torch.Tensor, x: torch.Tensor, y: Optional[torch.Tensor] = None,
                    stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """y = W x for an fp16 matrix W [rows, cols] on the device (fp32 accumulation).  Asynchronous."""
    rows, cols = w.shape
    if y is None:
        y = torch.empty(rows, dtype=torch.float16, device=w.device)
    _check(lib().entro_gemv_fp16(_dev(w, torch.float16), rows, cols, _dev(x, torch.float16), _dev(y, torch.float16),
                                 _stream(stream)), "entro_gemv_fp16")
    return y


def entro_decode_dequant_static(descs, status: Optional[torch.Tensor] = None,
                                stream: Optional[torch.cuda.Stream] = None) -> None:
    """The batched decode for callers that cannot allocate device memory: at most
    STATIC_MAX_TENSORS tensors, no allocator call inside the library.  status: an int32
    device tensor of one element that receives 0 (clean) or non-zero (corrupt input).
    Asynchronous."""
    if isinstance(descs, list):
        descs = desc_array(descs)
    sp = None if status is None else _dev(status, torch.int32)
    _check(lib().entro_decode_dequant_static(descs, len(descs), sp, _stream(stream)), "entro_decode_dequant_static")


def entro_last_device_status(stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(lib().entro_last_device_status(_stream(stream)))


def entro_set_decode_config(lut_bits: int = 0, warps_per_cta: int = 0, ctas_per_sm: int = 0,
                            chunks_per_item: int = 0) -> None:
    _check(lib().entro_set_decode_config(lut_bits, warps_per_cta, ctas_per_sm, chunks_per_item),
           "entro_set_decode_config")


def entro_profile_begin(max_records: int) -> None:
    _check(lib().entro_profile_begin(max_records), "entro_profile_begin")


def entro_profile_read(cap: int = 65536) -> List[float]:
    buf = (C.c_float * cap)()
    n = lib().entro_profile_read(buf, cap)
    if n < 0:
        raise EntroError(ERR_CUDA, "entro_profile_read")
    return [float(buf[i]) for i in range(n)]


def entro_checked_build() -> bool:
    return bool(lib().entro_checked_build())


def entro_check_violations() -> int:
    """Checked build: waits for the device, returns and clears the count of accesses the kernels'
    own bounds checks refused.  Always 0 in the ordinary build."""
    n = int(lib().entro_check_violations())
    if n < 0:
        raise EntroError(ERR_CUDA, "entro_check_violations")
    return n


def entro_kernel_launch_count() -> int:
    return int(lib().entro_kernel_launch_count())

"""A file of entropy-coded weights, and the way back onto the device.

What the paper is for (Section 1, Section 3): a quantised model is stored Huffman-coded, and
decoded when it is loaded.  This module only moves bytes and marshals arguments; every step
of the method runs in the library's kernels:

    compress(named fp16 tensors on the device)  ->  CompressedModel   (quantise, histogram,
                                                    codebook, encode per tensor)
    CompressedModel.save(path) / CompressedModel.load(path)           (one flat file)
    CompressedModel.to_device()                 ->  {name: fp16 tensor} (streams from pinned
                                                    host memory, decoded on the device in one
                                                    call; nothing is copied back)

File layout: 8 bytes magic, 8 bytes little-endian header length, a JSON header (per tensor:
name, shape, bits, chunk size, scale, zero point, code lengths, and offset / size of its
stream and index), then the streams and indices, each starting on a 64-byte boundary, exactly
as the decoder reads them.
"""
from __future__ import annotations

import json
import os
import struct
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

import paper_2505_02380_b200 as E

MAGIC = b"ENTROW01"
ALIGN = 64


class CompressedTensor:
    """One tensor: host copies of its stream and index, and what the decoder needs beside them."""

    def __init__(self, name: str, shape: Tuple[int, ...], bits: int, chunk_symbols: int, scale: float,
                 zero_point: int, lengths: List[int], stream: torch.Tensor, index: torch.Tensor, total_bits: int):
        self.name, self.shape, self.bits, self.chunk_symbols = name, tuple(shape), bits, chunk_symbols
        self.scale, self.zero_point, self.lengths = float(scale), int(zero_point), list(lengths)
        self.stream, self.index, self.total_bits = stream, index, int(total_bits)   # host int32 / uint8 tensors

    @property
    def numel(self) -> int:
        return int(np.prod(self.shape)) if self.shape else 1

    def codebook(self) -> "E.Codebook":
        return E.Codebook.from_lengths(self.lengths)      # the decoder reads the lengths only


def _check_entry(path: str, e: dict, stream_words: int, index_bytes: int) -> None:
    """The sizes a header entry states must agree with one another before anything is handed to
    the decoder: it sizes its reads of the index from shape and chunk size, and of the stream
    from total_bits, not from the sizes of the blobs."""
    def bad(what: str):
        raise ValueError(f"{path}: {e.get('name')!r}: {what}")

    shape, chunk, bits, lengths = e["shape"], e["chunk_symbols"], e["bits"], e["lengths"]
    if bits not in (4, 8):
        bad(f"bits = {bits}")
    if not isinstance(lengths, list) or not 1 <= len(lengths) <= (1 << bits) or \
            any(not isinstance(l, int) or l < 0 or l > E.MAX_CODE_LEN for l in lengths):
        bad("code lengths do not describe an alphabet of this width")
    if any(not isinstance(d, int) or d < 0 for d in shape):
        bad(f"shape = {shape}")
    numel = int(np.prod(shape, dtype=np.int64)) if shape else 1
    if not isinstance(chunk, int) or chunk < E.SUB_BLOCKS or chunk % E.SUB_BLOCKS or chunk > E.MAX_CHUNK_SYMBOLS:
        bad(f"chunk_symbols = {chunk}")
    if numel == 0:
        bad("empty tensor")
    n_chunks = (numel + chunk - 1) // chunk
    if index_bytes != 8 * (n_chunks + 1) + 2 * E.SUB_BLOCKS * n_chunks:
        bad(f"index of {index_bytes} bytes does not fit {numel} symbols in chunks of {chunk}")
    total_bits = e["total_bits"]
    if not isinstance(total_bits, int) or total_bits < 0 or \
            stream_words < (total_bits + 31) // 32 + E.STREAM_SLACK_WORDS:
        bad(f"stream of {stream_words} words is too short for {total_bits} bits")
    if not 0 <= e["zero_point"] < (1 << bits):
        bad(f"zero_point = {e['zero_point']}")


class CompressedModel:
    def __init__(self, tensors: List[CompressedTensor]):
        self.tensors = tensors

    # ------------------------------------------------------------------ sizes

    def coded_bytes(self) -> int:
        """Stream bits (rounded up per tensor) plus the chunk index."""
        return sum((t.total_bits + 7) // 8 + t.index.numel() for t in self.tensors)

    def report(self) -> dict:
        n = sum(t.numel for t in self.tensors)
        raw = sum(t.numel * t.bits for t in self.tensors) / 8
        return {"weights": n, "fp16_bytes": 2 * n, "quantised_bytes": int(raw), "coded_bytes": self.coded_bytes(),
                "bits_per_weight": 8.0 * sum((t.total_bits + 7) // 8 for t in self.tensors) / max(n, 1),
                "index_bits_per_weight": 8.0 * sum(t.index.numel() for t in self.tensors) / max(n, 1)}

    # ------------------------------------------------------------------ file

    def save(self, path: str) -> None:
        header, pos = [], 0
        blobs = []
        for t in self.tensors:
            entry = {"name": t.name, "shape": list(t.shape), "bits": t.bits, "chunk_symbols": t.chunk_symbols,
                     "scale_bits": int(np.float32(t.scale).view(np.uint32)), "zero_point": t.zero_point,
                     "lengths": t.lengths, "total_bits": t.total_bits}
            for key, buf in (("stream", t.stream.numpy().view(np.uint8)), ("index", t.index.numpy())):
                pos = (pos + ALIGN - 1) // ALIGN * ALIGN
                entry[key] = [pos, int(buf.size)]
                blobs.append((pos, buf))
                pos += int(buf.size)
            header.append(entry)
        head = json.dumps({"tensors": header}).encode()
        start = (16 + len(head) + ALIGN - 1) // ALIGN * ALIGN
        with open(path, "wb") as f:
            f.write(MAGIC + struct.pack("<Q", len(head)) + head)
            for off, buf in blobs:
                f.seek(start + off)
                f.write(buf.tobytes())
            f.truncate(start + pos)

    @staticmethod
    def load(path: str, pin: bool = True) -> "CompressedModel":
        """Reads the file into (pinned) host memory.  No device work."""
        with open(path, "rb") as f:
            if f.read(8) != MAGIC:
                raise ValueError(f"{path}: not a file of this format")
            (hlen,) = struct.unpack("<Q", f.read(8))
            head = json.loads(f.read(hlen).decode())
            start = (16 + hlen + ALIGN - 1) // ALIGN * ALIGN
            size = os.fstat(f.fileno()).st_size
            tensors = []
            for e in head["tensors"]:
                bufs = {}
                for key, dtype in (("stream", torch.int32), ("index", torch.uint8)):
                    off, nbytes = e[key]
                    if start + off + nbytes > size or (key == "stream" and nbytes % 4):
                        raise ValueError(f"{path}: {e['name']}: {key} lies outside the file")
                    t = torch.empty(nbytes, dtype=torch.uint8, pin_memory=pin and torch.cuda.is_available())
                    f.seek(start + off)
                    got = f.readinto(memoryview(t.numpy()))
                    if got != nbytes:
                        raise ValueError(f"{path}: {e['name']}: short read")
                    bufs[key] = t.view(dtype)
                _check_entry(path, e, bufs["stream"].numel(), bufs["index"].numel())
                scale = float(np.uint32(e["scale_bits"]).view(np.float32))
                tensors.append(CompressedTensor(e["name"], tuple(e["shape"]), e["bits"], e["chunk_symbols"], scale,
                                                e["zero_point"], e["lengths"], bufs["stream"], bufs["index"],
                                                e["total_bits"]))
        return CompressedModel(tensors)

    # ------------------------------------------------------------------ device

    def to_device(self, device: str = "cuda", stream: Optional[torch.cuda.Stream] = None) -> Dict[str, torch.Tensor]:
        """Uploads the streams and decodes them on the device (one call of the host-buffer entry point
        with the results left on the device).  -> {name: fp16 tensor of the tensor's shape}."""
        descs, io, out, keep = [], (E.HostIO * len(self.tensors))(), {}, []
        for i, t in enumerate(self.tensors):
            d_stream = torch.empty(t.stream.numel(), dtype=torch.int32, device=device)
            d_index = torch.empty(t.index.numel(), dtype=torch.uint8, device=device)
            w = torch.empty(t.shape, dtype=torch.float16, device=device)
            descs.append(E.make_desc(d_stream, d_index, t.numel, t.chunk_symbols, t.codebook(), t.scale, t.zero_point,
                                     w.view(-1)))
            io[i] = E.HostIO(t.stream.data_ptr(), t.index.data_ptr(), None)
            keep += [d_stream, d_index]
            out[t.name] = w
        E.entro_decode_dequant_batched_host(E.desc_array(descs), io, stream)
        status = E.entro_last_device_status(stream)
        if status != E.OK:
            raise E.EntroError(status, "CompressedModel.to_device")
        return out


def compress(named: Dict[str, torch.Tensor], bits: int = 8, chunk_symbols: Optional[int] = None) -> CompressedModel:
    """Quantise (one grid per tensor, Eq. 1), Huffman-code and index every fp16 device tensor."""
    if chunk_symbols is None:
        chunk_symbols = 4096 if bits == 8 else 8192
    tensors = []
    for name, w in named.items():
        flat = w.contiguous().view(-1)
        q, qp = E.entro_quantize_tensor(flat, bits)
        counts = E.entro_histogram(q, bits).tolist()
        cb = E.entro_build_codebook(counts)
        enc = E.entro_encode(q, cb, chunk_symbols, stream_words=E.entro_stream_words(counts, cb))
        tensors.append(CompressedTensor(name, tuple(w.shape), bits, chunk_symbols, qp.scale, qp.zero_point,
                                        cb.lengths().tolist(), enc.stream.cpu(), enc.index.cpu(), enc.total_bits))
    return CompressedModel(tensors)

"""An encoder for the compressed format, written from the words of include/entro.h alone
("Compressed format": stream, segments, order inside a chunk, index).

It shares nothing with the oracle or the library: plain loops over chunks, sub-blocks, groups
and symbols in exactly the order the header states.  The tests hold the oracle's encoder and
the library's encoder and decoder to it, so that the header is a contract somebody else can
implement from."""
from __future__ import annotations

import numpy as np

SUB_BLOCKS = 32          # ENTRO_SUB_BLOCKS
SLACK_WORDS = 8          # ENTRO_STREAM_SLACK_WORDS


def encode(q, lengths, codes, chunk_symbols):
    """q: symbols in row-major element order; lengths[k], codes[k]: code of symbol k, the code
    right-aligned in lengths[k] bits.  -> (stream uint32 words, offsets uint64, sub_len uint16 [n_chunks, 32])"""
    n = len(q)
    n_chunks = (n + chunk_symbols - 1) // chunk_symbols
    offsets = np.zeros(n_chunks + 1, dtype=np.uint64)
    sub_len = np.zeros((n_chunks, SUB_BLOCKS), dtype=np.uint16)
    bits = []                                                  # the stream, one entry per bit
    for c in range(n_chunks):
        e = q[c * chunk_symbols:(c + 1) * chunk_symbols]       # the chunk's symbols e[0 .. m)
        m = len(e)
        offsets[c] = len(bits)
        n_groups = (m + 7) // 8
        for l in range(SUB_BLOCKS):                            # sub-block 0 first, then 1, ... 31
            before = len(bits)
            for g in range(l, n_groups, SUB_BLOCKS):           # its groups in ascending g
                for sym in e[8 * g:8 * g + 8]:                 # a group's symbols in element order
                    length, code = int(lengths[sym]), int(codes[sym])
                    assert length > 0
                    bits.extend((code >> (length - 1 - b)) & 1 for b in range(length))   # MSB first
            sub_len[c, l] = len(bits) - before
    offsets[n_chunks] = len(bits)
    n_words = (len(bits) + 31) // 32 + SLACK_WORDS
    stream = np.zeros(n_words, dtype=np.uint32)
    for i, b in enumerate(bits):                               # stream bit i is bit (31 - i % 32) of word i / 32
        if b:
            stream[i // 32] |= np.uint32(1 << (31 - i % 32))
    return stream, offsets, sub_len


def index_bytes(offsets, sub_len):
    """offsets, then sub_len, back to back."""
    return np.concatenate([offsets.view(np.uint8), sub_len.reshape(-1).view(np.uint8)])

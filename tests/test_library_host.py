"""CPU-side checks of the CUDA library: it loads, exports everything the header declares,
and its host-only entry points agree with the oracle.  No kernel runs here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
import workloads
import paper_2505_02380_b200 as E
from paper_2505_02380_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "entro.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(entro_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    L = C.CDLL(E.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert declared == set(E.EXPORTS)


def test_golden_lengths_and_codes():
    from test_oracle_huffman import _golden_cases
    for counts, lengths in _golden_cases():
        cb = E.entro_build_codebook(counts)
        assert cb.lengths().tolist() == lengths
        assert cb.max_len == max(lengths)


def test_codebook_matches_oracle_bit_exactly():
    rng = np.random.default_rng(2024)
    for t in range(600):
        n = [16, 256, int(rng.integers(1, 257))][t % 3]
        hi = [1, 3, 60, 10**7][t % 4]
        counts = rng.integers(0, hi + 1, size=n)
        if counts.sum() == 0:
            counts[int(rng.integers(0, n))] = 1
        cb = E.entro_build_codebook(counts)
        ln = oracle.huffman_lengths(counts)
        assert np.array_equal(cb.lengths(), ln), counts
        assert np.array_equal(cb.codes(), oracle.canonical_codes(ln))
        assert cb.max_len == int(ln.max())


def test_limited_codebook_matches_oracle_bit_exactly():
    rng = np.random.default_rng(12)
    cases = [[1, 1, 2, 3, 5, 8], [5, 5, 5, 5], [1, 1, 1, 1, 1, 1, 1], [0, 3, 0, 9, 1]]
    for _ in range(40):
        n = int(rng.integers(2, 257))
        c = rng.integers(0, 1000, n)
        c[rng.integers(0, n)] = 10 ** 6          # a dominant symbol makes long tails
        cases.append(c.tolist())
    for bits in (4, 8):
        w = workloads.make_values(1 << 18, 0.02, 70 + bits).numpy()
        q, _ = oracle.quantize_tensor(w, bits)
        cases.append(oracle.histogram(q, 1 << bits).tolist())
    for counts in cases:
        used = sum(1 for c in counts if c)
        for cap in (32, 16, 12, 10, 8):
            if used > 1 and (1 << cap) < used:
                continue
            ref = oracle.length_limited_lengths(counts, cap)
            cb = E.entro_build_codebook_limited(counts, cap)
            assert cb.lengths().tolist() == ref.tolist(), (counts[:8], cap)
            assert cb.codes().tolist() == oracle.canonical_codes(ref).tolist()
            assert cb.max_len == int(ref.max())
    with pytest.raises(E.EntroError) as e:
        E.entro_build_codebook_limited([1] * 9, 3)
    assert e.value.status == E.ERR_CODE_TOO_LONG


def test_codebook_errors():
    fib = [1, 1]
    while len(fib) < 40:
        fib.append(fib[-1] + fib[-2])
    with pytest.raises(E.EntroError) as e:
        E.entro_build_codebook(fib)
    assert e.value.status == E.ERR_CODE_TOO_LONG
    with pytest.raises(E.EntroError) as e:
        E.entro_build_codebook([0, 0, 0])
    assert e.value.status == E.ERR_INVALID_ARG
    fib33 = fib[:33]        # depth 32: the longest supported code
    assert E.entro_build_codebook(fib33).max_len == 32


def test_size_helpers():
    assert E.entro_index_bytes(1 << 20, 4096) == 8 * 257 + 64 * 256
    assert E.entro_index_bytes(4097, 4096) == 8 * 3 + 64 * 2
    assert E.entro_index_bytes(100, 48) == 0          # not a multiple of 32
    assert E.entro_index_bytes(100, 32768) == 0       # above the maximum
    counts = [5, 0, 3, 9]
    cb = E.entro_build_codebook(counts)
    bits = sum(c * l for c, l in zip(counts, cb.lengths().tolist()))
    assert E.entro_stream_words(counts, cb) == (bits + 31) // 32 + E.STREAM_SLACK_WORDS
    assert E.entro_encode_bound_words(1000, cb) == (1000 * cb.max_len + 31) // 32 + E.STREAM_SLACK_WORDS
    assert E.status_string(E.ERR_CORRUPT_STREAM) and E.status_string(E.OK) == "ok"


def test_argument_errors_are_found_before_any_launch():
    """Null pointers and bad sizes are refused on the host (no device is touched)."""
    L = E.lib()
    cb = E.entro_build_codebook([1, 2, 3, 4])
    qp = E.QParams()
    assert L.entro_quantize_tensor(None, 16, 8, 0, None, C.byref(qp), None) == E.ERR_INVALID_ARG
    assert L.entro_quantize_tensor(16, 16, 5, 0, 16, C.byref(qp), None) == E.ERR_INVALID_ARG
    counts = (C.c_uint64 * 256)()
    assert L.entro_histogram(None, 16, 8, counts, None) == E.ERR_INVALID_ARG
    total = C.c_uint64()
    assert L.entro_encode(None, 16, C.byref(cb), 4096, None, 0, None, 0, C.byref(total), None) == E.ERR_INVALID_ARG
    assert L.entro_encode(16, 16, C.byref(cb), 100, 16, 64, 16, 4096, C.byref(total), None) == E.ERR_INVALID_ARG
    # symbols that do not start on a 16-byte boundary (an offset view of a tensor: q[1:]) are refused
    assert L.entro_encode(17, 16, C.byref(cb), 4096, 16, 64, 16, 4096, C.byref(total), None) == E.ERR_INVALID_ARG
    assert L.entro_decode_dequant(None, 0, None, 16, 4096, C.byref(cb), 1.0, 0, None, None) == E.ERR_INVALID_ARG
    assert L.entro_decode_dequant(16, 100, 16, 16, 4096, C.byref(cb), 1.0, 0, 24, None) == E.ERR_INVALID_ARG  # misaligned out
    bad = E.Codebook.from_lengths([1, 1, 1, 0])        # over-subscribed lengths
    assert L.entro_decode_dequant(16, 100, 16, 16, 4096, C.byref(bad), 1.0, 0, 32, None) == E.ERR_INVALID_ARG
    assert L.entro_decode_dequant_batched(None, 3, None) == E.ERR_INVALID_ARG
    assert L.entro_decode_dequant_batched(None, 0, None) == E.OK

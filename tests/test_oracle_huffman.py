"""Pins for the oracle's code construction, encoder and decoder.

What the paper fixes (Section 3): the code is an optimal prefix code built by recursive
pair merging (so: a full binary tree, Kraft sum exactly 1, average length within one bit
of the entropy, no cheaper prefix code exists), coding is lossless, and every segment
decodes on its own from its known boundary."""
import functools
from fractions import Fraction
import heapq
import itertools
import math
import os

import numpy as np
import pytest

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "huffman_tiebreak.txt")


def _golden_cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            lhs, rhs = line.split("->")
            out.append(([int(t) for t in lhs.split()], [int(t) for t in rhs.split()]))
    return out


def _cost(counts, lengths):
    return sum(int(c) * int(l) for c, l in zip(counts, lengths))


def _kraft_is_one(lengths):
    used = [int(l) for l in lengths if l]
    m = max(used)
    return sum(1 << (m - l) for l in used) == (1 << m)


# ----------------------------------------------------------------------------- lengths

@pytest.mark.parametrize("counts,lengths", _golden_cases())
def test_hand_worked_lengths(counts, lengths):
    assert oracle.huffman_lengths(counts).tolist() == lengths


@functools.lru_cache(maxsize=None)
def _best_tree_cost(weights):
    """Cheapest full binary tree over these leaf weights, trying EVERY pair at every
    step (not just the two smallest): cost = sum of internal-node weights."""
    if len(weights) == 1:
        return 0
    best = None
    for i, j in itertools.combinations(range(len(weights)), 2):
        merged = weights[i] + weights[j]
        rest = tuple(sorted(w for k, w in enumerate(weights) if k != i and k != j) + [merged])
        c = merged + _best_tree_cost(tuple(sorted(rest)))
        best = c if best is None or c < best else best
    return best


def _best_kraft_cost(counts):
    """Cheapest length vector with Kraft sum <= 1, by exhaustive enumeration."""
    n = len(counts)
    best = None
    for ls in itertools.product(range(1, n), repeat=n):
        if sum(2.0 ** -l for l in ls) <= 1.0:
            c = _cost(counts, ls)
            best = c if best is None or c < best else best
    return best


def test_optimal_against_brute_force_small_alphabets():
    rng = np.random.default_rng(123)
    for n in range(2, 9):
        for trial in range(12):
            hi = [3, 10, 1000][trial % 3]       # small ranges force many ties
            counts = rng.integers(1, hi + 1, size=n).tolist()
            ln = oracle.huffman_lengths(counts)
            assert _kraft_is_one(ln)
            assert _cost(counts, ln) == _best_tree_cost(tuple(sorted(counts))), counts
            if n <= 6:
                assert _cost(counts, ln) == _best_kraft_cost(counts), counts


def _heap_huffman_cost(counts):
    """A different construction (binary heap, arbitrary tie order): the cost is unique."""
    h = [int(c) for c in counts if c]
    heapq.heapify(h)
    cost = 0
    while len(h) > 1:
        a, b = heapq.heappop(h), heapq.heappop(h)
        cost += a + b
        heapq.heappush(h, a + b)
    return cost


@pytest.mark.parametrize("nsym", [16, 256])
def test_cost_kraft_and_entropy_bounds_on_weight_histograms(nsym):
    bits = 4 if nsym == 16 else 8
    for seed in range(4):
        w = workloads.make_values(1 << 18, 0.02, seed).numpy()
        q, _ = oracle.quantize_tensor(w, bits)
        counts = oracle.histogram(q, nsym)
        assert np.array_equal(counts, np.bincount(q, minlength=nsym).astype(np.uint64))
        ln = oracle.huffman_lengths(counts)
        assert np.all((ln > 0) == (counts > 0))
        assert _kraft_is_one(ln)
        assert _cost(counts, ln) == _heap_huffman_cost(counts)
        p = counts[counts > 0].astype(np.float64) / counts.sum()
        H = float(-(p * np.log2(p)).sum())
        Lbar = _cost(counts, ln) / int(counts.sum())
        assert H <= Lbar + 1e-12 < H + 1


def test_random_histograms_cost_and_kraft():
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(2, 257))
        counts = rng.integers(0, [2, 5, 1000, 10**9][trial % 4] + 1, size=n)
        if np.count_nonzero(counts) < 2:
            counts[:2] = 1
        ln = oracle.huffman_lengths(counts)
        assert _kraft_is_one(ln)
        assert _cost(counts, ln) == _heap_huffman_cost(counts)
        assert np.all((ln > 0) == (counts > 0))


def test_textbook_length_patterns():
    for k in range(1, 9):
        assert oracle.huffman_lengths([7] * (1 << k)).tolist() == [k] * (1 << k)
    # dyadic probabilities: length = -log2 p, average length equals the entropy
    counts = [1 << 10, 1 << 9, 1 << 8, 1 << 7, 1 << 7]
    ln = oracle.huffman_lengths(counts).tolist()
    assert ln == [1, 2, 3, 4, 4]
    total = sum(counts)
    H = -sum(c / total * math.log2(c / total) for c in counts)
    assert abs(_cost(counts, ln) / total - H) < 1e-12
    # Fibonacci counts give the deepest possible tree: max length n - 1
    fib = [1, 1]
    while len(fib) < 30:
        fib.append(fib[-1] + fib[-2])
    ln = oracle.huffman_lengths(fib)
    assert ln.max() == len(fib) - 1
    fib40 = [1, 1]
    while len(fib40) < 40:
        fib40.append(fib40[-1] + fib40[-2])
    with pytest.raises(oracle.OracleError) as e:          # depth 39 > 32: refused
        oracle.huffman_lengths(fib40)
    assert e.value.code == 4


def test_minimum_variance_rule_gives_smallest_max_length():
    """Leaf-before-internal on ties is the minimum-variance rule: among all optimal
    codes it has the smallest maximum length.  Checked by enumeration."""
    rng = np.random.default_rng(9)
    for _ in range(40):
        n = int(rng.integers(3, 7))
        counts = rng.integers(1, 4, size=n).tolist()
        ln = oracle.huffman_lengths(counts)
        best_cost = _cost(counts, ln)
        min_max = None
        for ls in itertools.product(range(1, n), repeat=n):
            if sum(2.0 ** -l for l in ls) <= 1.0 and _cost(counts, ls) == best_cost:
                min_max = max(ls) if min_max is None else min(min_max, max(ls))
        assert int(ln.max()) == min_max, counts


# ----------------------------------------------------------------------------- canonical codes

def _bitstr(code, length):
    return format(int(code), "b").zfill(int(length)) if length else ""


def test_canonical_codes_prefix_free_and_ordered():
    rng = np.random.default_rng(1)
    for trial in range(60):
        n = int(rng.integers(2, 257))
        counts = rng.integers(0, 50, size=n)
        if np.count_nonzero(counts) < 2:
            counts[:2] = 1
        ln = oracle.huffman_lengths(counts)
        cd = oracle.canonical_codes(ln)
        words = {k: _bitstr(cd[k], ln[k]) for k in range(n) if ln[k]}
        assert all(int(cd[k]) < (1 << int(ln[k])) for k in words)
        ws = sorted(words.values())
        assert len(set(ws)) == len(ws)
        for a, b in zip(ws, ws[1:]):                 # sorted: a prefix would sit right before
            assert not b.startswith(a)
        # ordered by (length, symbol); numerically consecutive within a length
        order = sorted(words, key=lambda k: (ln[k], k))
        assert words[order[0]] == "0" * int(ln[order[0]])
        for a, b in zip(order, order[1:]):
            if ln[a] == ln[b]:
                assert int(cd[b]) == int(cd[a]) + 1
            else:
                assert int(cd[b]) == (int(cd[a]) + 1) << (int(ln[b]) - int(ln[a]))
        # left-justified codes increase strictly in that order, the last is all ones
        lj = [int(cd[k]) << (32 - int(ln[k])) for k in order]
        assert all(x < y for x, y in zip(lj, lj[1:]))
        assert words[order[-1]] == "1" * int(ln[order[-1]])


def test_canonical_codes_known_example():
    # lengths 2 1 3 3: symbol 1 -> 0, symbol 0 -> 10, symbols 2, 3 -> 110, 111
    assert oracle.canonical_codes([2, 1, 3, 3]).tolist() == [0b10, 0b0, 0b110, 0b111]
    assert oracle.canonical_codes([0, 1, 0, 0]).tolist() == [0, 0, 0, 0]
    with pytest.raises(oracle.OracleError):
        oracle.canonical_codes([1, 1, 1])           # over-subscribed


# ----------------------------------------------------------------------------- stream + index

def _stream_bits(stream, nbits):
    """Bit i of the stream = bit (31 - i % 32) of word i // 32, via NumPy unpackbits."""
    by = np.ascontiguousarray(stream, dtype=">u4") if False else stream.astype(">u4")
    return np.unpackbits(by.view(np.uint8))[:nbits]


def _stored_order(n, chunk):
    """Independent statement of the storage order: element indices in the order their
    codewords appear in the stream, and the sub-block each belongs to.  Inside a chunk the
    symbols form groups of 8; group g belongs to sub-block g % 32; a sub-block holds its
    groups in increasing g; sub-blocks follow each other 0 .. 31."""
    i = np.arange(n, dtype=np.int64)
    c, r = i // chunk, i % chunk
    g = r // 8
    lane, rnd, k = g % 32, g // 32, r % 8
    order = np.lexsort((k, rnd, lane, c))          # last key is the primary one
    return order, lane


def test_stored_order_small_example_by_hand():
    """chunk = 32 * 8 * 2 = 512: lane 0 holds elements 0..7 then 256..263, lane 1 holds 8..15 then 264..271."""
    order, lane = _stored_order(512 + 20, 512)
    assert order[:16].tolist() == list(range(0, 8)) + list(range(256, 264))
    assert order[16:32].tolist() == list(range(8, 16)) + list(range(264, 272))
    assert order[496:512].tolist() == list(range(248, 256)) + list(range(504, 512))
    # ragged second chunk of 20 symbols: groups 0, 1 full, group 2 has 4 symbols, lanes 0..2
    assert order[512:].tolist() == list(range(512, 532))
    assert lane[512:].tolist() == [0] * 8 + [1] * 8 + [2] * 4


@pytest.mark.parametrize("bits,chunk", [(8, 4096), (4, 8192), (8, 64), (4, 32), (8, 512)])
def test_stream_is_concatenation_of_codewords_and_index_is_consistent(bits, chunk):
    n = 3 * chunk + chunk // 3 + 5
    w = workloads.make_values(n, 0.02, 42 + bits).numpy()
    c = oracle.compress(w, bits, chunk)
    ln, cd, enc = c.lengths, c.codes, c.enc
    order, lane = _stored_order(n, chunk)
    text = "".join(_bitstr(cd[s], ln[s]) for s in c.q[order].tolist())
    assert enc.total_bits == len(text) == int((c.counts * ln.astype(np.uint64)).sum())
    got = "".join(map(str, _stream_bits(enc.stream, enc.total_bits).tolist()))
    assert got == text
    # zero padding after the last bit
    assert not _stream_bits(enc.stream, enc.stream.size * 32)[enc.total_bits:].any()
    # index: start of chunk k is the number of bits of the k * chunk symbols before it
    per_sym = ln.astype(np.int64)[c.q]
    cum = np.concatenate([[0], np.cumsum(per_sym)])
    nch = oracle.num_chunks(n, chunk)
    assert enc.offsets.size == nch + 1
    for k in range(nch + 1):
        assert int(enc.offsets[k]) == int(cum[min(k * chunk, n)])
    # sub-block lengths: bits of the elements that belong to each sub-block
    for k in range(nch):
        a, b = k * chunk, min((k + 1) * chunk, n)
        want = np.bincount(lane[a:b], weights=per_sym[a:b], minlength=32).astype(np.int64)
        assert enc.sub_len[k].astype(np.int64).tolist() == want.tolist()
        assert int(enc.sub_len[k].sum()) == int(enc.offsets[k + 1] - enc.offsets[k])


@pytest.mark.parametrize("bits,chunk,n", [(8, 4096, 2 * 4096 + 1000), (4, 8192, 8192 + 77), (8, 512, 3 * 512 + 20),
                                          (8, 32, 100), (4, 64, 64), (8, 4096, 5)])
def test_oracle_stream_and_index_equal_an_encoder_written_from_the_public_header(bits, chunk, n):
    """tests/format_from_header.py restates the header's format text as loops; the oracle's
    stream, chunk offsets and sub-block lengths must be what those loops write."""
    import format_from_header
    w = workloads.make_values(n, 0.02, 4242 + n).numpy()
    c = oracle.compress(w, bits, chunk)
    stream, offsets, sub_len = format_from_header.encode(c.q.tolist(), c.lengths.tolist(), c.codes.tolist(), chunk)
    assert np.array_equal(stream, c.enc.stream)
    assert np.array_equal(offsets, c.enc.offsets)
    assert np.array_equal(sub_len, c.enc.sub_len)


# ----------------------------------------------------------------------------- decoder

def _dict_decode(bits_arr, start, count, table):
    """Independent decoder: grow a bit string until it is a key of {codeword: symbol}."""
    out, pos = [], start
    for _ in range(count):
        cur = ""
        while cur not in table:
            cur += str(int(bits_arr[pos]))
            pos += 1
            assert len(cur) <= 32
        out.append(table[cur])
    return out, pos


@pytest.mark.parametrize("bits,chunk", [(8, 4096), (4, 8192), (8, 128)])
def test_round_trip_and_segment_independence(bits, chunk):
    for n in (1, 31, chunk - 1, chunk, chunk + 1, 5 * chunk + 77):
        w = workloads.make_values(n, 0.03, n + bits).numpy()
        c = oracle.compress(w, bits, chunk)
        enc = c.enc
        q, out = oracle.decode_dequant(enc.stream, enc.offsets, n, chunk, c.lengths, c.qp.scale,
                                       c.qp.zero_point)
        assert np.array_equal(q, c.q)                                    # lossless
        assert np.array_equal(out, oracle.dequant(c.q, c.qp.scale, c.qp.zero_point))
        # any subset of chunks, in any order, gives the same symbols there
        nch = oracle.num_chunks(n, chunk)
        ids = list(range(nch))[::-1][::2]
        q2, _ = oracle.decode_dequant(enc.stream, enc.offsets, n, chunk, c.lengths, c.qp.scale,
                                      c.qp.zero_point, chunk_ids=ids)
        for k in ids:
            assert np.array_equal(q2[k * chunk:(k + 1) * chunk], c.q[k * chunk:(k + 1) * chunk])
        # thread-per-segment driver
        _, out3 = oracle.decode_dequant(enc.stream, enc.offsets, n, chunk, c.lengths, c.qp.scale,
                                        c.qp.zero_point, want_q=False, threads=3)
        assert np.array_equal(out3, out)


def test_decoder_against_dictionary_decoder():
    n, chunk = 3000, 1024
    w = workloads.make_values(n, 0.02, 77).numpy()
    c = oracle.compress(w, 8, chunk)
    table = {_bitstr(c.codes[s], c.lengths[s]): s for s in range(256) if c.lengths[s]}
    bits_arr = _stream_bits(c.enc.stream, c.enc.total_bits)
    order, _ = _stored_order(n, chunk)
    for k in range(oracle.num_chunks(n, chunk)):
        cnt = min(chunk, n - k * chunk)
        syms, end = _dict_decode(bits_arr, int(c.enc.offsets[k]), cnt, table)
        assert end == int(c.enc.offsets[k + 1])
        assert syms == c.q[order[k * chunk:k * chunk + cnt]].tolist()


def test_decoder_rejects_corruption():
    n, chunk = 20000, 4096
    w = workloads.make_values(n, 0.02, 5).numpy()
    c = oracle.compress(w, 8, chunk)
    enc = c.enc
    bad_off = enc.offsets.copy()
    bad_off[2] += 3                                   # wrong boundary: chunk 1 ends elsewhere
    with pytest.raises(oracle.OracleError) as e:
        oracle.decode_dequant(enc.stream, bad_off, n, chunk, c.lengths, c.qp.scale, c.qp.zero_point)
    assert e.value.code == 5
    # a single used symbol has code "0"; a 1 bit is not a codeword
    ln = np.zeros(256, dtype=np.uint8)
    ln[9] = 1
    stream = np.array([0x80000000, 0], dtype=np.uint32)
    with pytest.raises(oracle.OracleError):
        oracle.decode_dequant(stream, np.array([0, 4], dtype=np.uint64), 4, 4096, ln, 1.0, 0)
    q, _ = oracle.decode_dequant(np.zeros(2, dtype=np.uint32), np.array([0, 4], dtype=np.uint64), 4, 4096,
                                 ln, 1.0, 0)
    assert q.tolist() == [9, 9, 9, 9]


def test_long_codes_round_trip():
    """Fibonacci-like histogram: code lengths up to 30 bits survive encode -> decode."""
    fib = [1, 1]
    while len(fib) < 31:
        fib.append(fib[-1] + fib[-2])
    ln = oracle.huffman_lengths(fib + [0] * (256 - len(fib)))
    assert ln.max() == 30
    cd = oracle.canonical_codes(ln)
    rng = np.random.default_rng(3)
    q = np.concatenate([np.arange(31), rng.integers(0, 31, 5000), rng.integers(25, 31, 3000)]).astype(np.uint8)
    rng.shuffle(q)
    enc = oracle.encode(q, ln, cd, 4096)
    q2, _ = oracle.decode_dequant(enc.stream, enc.offsets, q.size, 4096, ln, 1.0, 0)
    assert np.array_equal(q2, q)


# ----------------------------------------------------------------------------- length-limited codes

def _best_limited_cost(counts, max_len):
    """Brute force: the cheapest Kraft-feasible length vector with every length <= max_len."""
    used = [c for c in counts if c]
    best = None
    for ls in itertools.product(range(1, max_len + 1), repeat=len(used)):
        if sum(2.0 ** -l for l in ls) <= 1.0 + 1e-12:
            cost = sum(c * l for c, l in zip(used, ls))
            best = cost if best is None else min(best, cost)
    return best


def test_length_limited_optimal_against_brute_force():
    rng = np.random.default_rng(5)
    for trial in range(60):
        n = int(rng.integers(2, 7))
        counts = rng.integers(1, 50, n).tolist() if trial % 3 else (2 ** rng.integers(0, 7, n)).tolist()
        lo = int(np.ceil(np.log2(n)))
        for max_len in range(max(lo, 1), 6):
            ln = oracle.length_limited_lengths(counts, max_len)
            assert ln.max() <= max_len
            assert sum(Fraction(1, 2 ** int(l)) for l in ln) == 1          # complete code
            assert int((np.array(counts) * ln).sum()) == _best_limited_cost(counts, max_len), (counts, max_len)


def test_length_limited_reduces_to_huffman_cost_and_obeys_the_cap():
    rng = np.random.default_rng(6)
    for nsym in (16, 256):
        w = workloads.make_values(1 << 18, 0.02, 900 + nsym).numpy()
        bits = 4 if nsym == 16 else 8
        q, _ = oracle.quantize_tensor(w, bits)
        counts = oracle.histogram(q, nsym)
        huff = oracle.huffman_lengths(counts)
        cost_h = int((counts * huff.astype(np.uint64)).sum())
        # a cap at or above the Huffman depth changes nothing about the cost
        ln = oracle.length_limited_lengths(counts, int(huff.max()))
        assert int((counts * ln.astype(np.uint64)).sum()) == cost_h
        prev = None
        for cap in sorted({int(huff.max()) - 1, 16, 12, 10}, reverse=True):
            if (1 << cap) < int((counts > 0).sum()):
                continue
            ln = oracle.length_limited_lengths(counts, cap)
            used = ln[counts > 0]
            assert used.min() >= 1 and used.max() <= cap and not ln[counts == 0].any()
            assert sum(Fraction(1, 2 ** int(l)) for l in used) == 1
            cost = int((counts * ln.astype(np.uint64)).sum())
            assert cost >= cost_h and (prev is None or cost >= prev)       # tighter cap, never cheaper
            prev = cost
            oracle.canonical_codes(ln)                                     # a valid canonical code exists


def test_length_limited_hand_cases():
    # cap 2 on four symbols forces the fixed-length code whatever the counts
    assert oracle.length_limited_lengths([1, 1, 2, 100], 2).tolist() == [2, 2, 2, 2]
    # Fibonacci counts a..f = 1 1 2 3 5 8 want depths 5 5 4 3 2 1; cap 4, merged by hand under the stated rule:
    #   level 4: a1 b1 c2 d3 e5 f8                         packages P1=ab(2) P2=cd(5) P3=ef(13)
    #   level 3: a1 b1 c2 P1 d3 e5 P2 f8 P3                packages Q1=ab(2) Q2=c+P1(4) Q3=de(8) Q4=P2+f(13)
    #   level 2: a1 b1 c2 Q1 d3 Q2 e5 f8 Q3 Q4             packages R1=ab(2) R2=c+Q1(4) R3=d+Q2(7) R4=ef(13) R5
    #   level 1: a b c R1 d R2 e R3 f R4 | R5              first 10 items: a b c {ab} d {cab} e {dcab} f {ef}
    #   a, b appear 4 times, c 3 times, d, e, f twice
    assert oracle.length_limited_lengths([1, 1, 2, 3, 5, 8], 4).tolist() == [4, 4, 3, 2, 2, 2]
    assert oracle.length_limited_lengths([0, 9, 0], 5).tolist() == [0, 1, 0]
    with pytest.raises(oracle.OracleError):
        oracle.length_limited_lengths([1, 1, 1, 1, 1], 2)                  # five symbols need 3 bits

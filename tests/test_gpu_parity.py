"""GPU parity: every library stage against the CPU oracle on the same seeded inputs,
called through the C ABI.  Integer results (symbols, counts, code lengths, codes, stream
words, index) must be bit-exact.  fp16 outputs must be bit-exact too: both sides compute
s * (q - z) as one fp32 product rounded once to fp16 (tolerance: 0 ulp)."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import (assert_status_ok, codebook_from_oracle, expected_out, gpu_decode_from_oracle_stream,
                     index_bytes_np, to_dev_index, to_dev_stream)

pytestmark = pytest.mark.gpu


def _values(n, sigma, seed, kind="matrix"):
    """Identical fp16 bytes for both sides: drawn on the CPU, copied to the device."""
    w = workloads.make_values(n, sigma, seed, kind)
    return w.numpy(), w.cuda()


# ----------------------------------------------------------------------------- quantiser, histogram

@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("n,kind", [(1, "matrix"), (7, "matrix"), (8, "gain"), (1000, "matrix"), (4097, "gain"),
                                    (1 << 20, "matrix"), ((1 << 20) + 13, "matrix")])
def test_quantise_matches_oracle(bits, n, kind):
    w_np, w_dev = _values(n, 0.02, 10 * bits + n % 97, kind)
    q_ref, qp_ref = oracle.quantize_tensor(w_np, bits)
    q, qp = E.entro_quantize_tensor(w_dev, bits)
    assert (qp.bits, qp.mode, qp.zero_point) == (qp_ref.bits, qp_ref.mode, qp_ref.zero_point)
    assert np.float32(qp.scale).tobytes() == np.float32(qp_ref.scale).tobytes()
    assert qp.lo == qp_ref.lo and qp.hi == qp_ref.hi
    assert np.array_equal(q.cpu().numpy(), q_ref)


@pytest.mark.parametrize("mode", [E.MODE_UNSIGNED, E.MODE_ASYMMETRIC])
def test_quantise_forced_modes_and_degenerate(mode):
    for vals in ([0.0, 0.0, 0.0], [-3.0, -3.0], [2.0, 2.0], [-1.0, 0.5, 0.25], [0.5, 1.5, 2.5, 3.5, 254.5, 255.0, 0.0]):
        w = torch.tensor(vals, dtype=torch.float16)
        q_ref, qp_ref = oracle.quantize_tensor(w.numpy(), 8, mode)
        q, qp = E.entro_quantize_tensor(w.cuda(), 8, mode)
        assert (qp.mode, qp.zero_point, qp.scale) == (qp_ref.mode, qp_ref.zero_point, qp_ref.scale)
        assert q.cpu().numpy().tolist() == q_ref.tolist()


def test_quantise_refuses_nonfinite():
    for bad in (float("inf"), float("-inf"), float("nan")):
        w = torch.full((5000,), 0.25, dtype=torch.float16)
        w[4321] = bad
        with pytest.raises(E.EntroError) as e:
            E.entro_quantize_tensor(w.cuda(), 8)
        assert e.value.status == E.ERR_NONFINITE


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("n,block", [(1, 32), (31, 32), (32, 32), (33, 32), (5000, 32), (4096, 128), (100000, 32),
                                     (777, 1000), (1 << 20, 32)])
def test_block_quantiser_matches_oracle(bits, n, block):
    """The comparison grid of Table 2: codes, scales and zero points of every block, bit for bit."""
    w_np, w = _values(n, 0.02, 13 * n + bits + block)
    q_ref, s_ref, z_ref = oracle.quantize_blocks(w_np, bits, block)
    q, scales, zps = E.entro_quantize_blocks(w, bits, block)
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(zps.cpu().numpy(), z_ref)
    for mode in (E.MODE_UNSIGNED, E.MODE_ASYMMETRIC):
        q_ref, s_ref, z_ref = oracle.quantize_blocks(w_np, bits, block, mode)
        q, scales, zps = E.entro_quantize_blocks(w, bits, block, mode)
        assert np.array_equal(q.cpu().numpy(), q_ref), mode
        assert np.array_equal(zps.cpu().numpy(), z_ref), mode


def test_block_quantiser_refuses_nonfinite():
    w = torch.zeros(256, dtype=torch.float16, device="cuda")
    w[77] = float("nan")
    with pytest.raises(E.EntroError) as e:
        E.entro_quantize_blocks(w, 8, 32)
    assert e.value.status == E.ERR_NONFINITE


@pytest.mark.parametrize("bits", [4, 8])
def test_histogram_matches_oracle(bits):
    for n in (1, 15, 16, 17, 100_003, 1 << 21):
        w_np, _ = _values(n, 0.02, n % 1000 + bits)
        q_ref, _ = oracle.quantize_tensor(w_np, bits)
        counts = E.entro_histogram(torch.from_numpy(q_ref).cuda(), bits)
        assert np.array_equal(counts, oracle.histogram(q_ref, 1 << bits))
    with pytest.raises(E.EntroError):
        E.entro_histogram(torch.full((100,), 16, dtype=torch.uint8).cuda(), 4)


# ----------------------------------------------------------------------------- encoder

@pytest.mark.parametrize("bits,chunk", [(8, 4096), (4, 8192), (8, 32), (4, 1024)])
def test_encode_matches_oracle_stream_and_index(bits, chunk):
    for n in (1, 33, chunk - 1, chunk, chunk + 1, 7 * chunk + 123, 300_000):
        w_np, _ = _values(n, 0.02, bits * 1000 + n % 1000)
        c = oracle.compress(w_np, bits, chunk)
        cb = E.entro_build_codebook(c.counts.tolist())
        assert np.array_equal(cb.lengths(), c.lengths) and np.array_equal(cb.codes(), c.codes)
        words = E.entro_stream_words(c.counts.tolist(), cb)
        assert words == c.enc.stream.size
        enc = E.entro_encode(torch.from_numpy(c.q).cuda(), cb, chunk, stream_words=words)
        assert enc.total_bits == c.enc.total_bits
        assert np.array_equal(enc.stream_np(), c.enc.stream)
        assert np.array_equal(enc.offsets(), c.enc.offsets)
        assert np.array_equal(enc.sub_len(), c.enc.sub_len)


@pytest.mark.parametrize("bits,chunk,n", [(8, 4096, 2 * 4096 + 1000), (4, 8192, 2 * 8192 + 77), (8, 512, 3 * 512 + 20),
                                          (8, 32, 100), (8, 4096, 5)])
def test_format_stated_in_the_header_is_the_format_the_library_uses(bits, chunk, n):
    """An encoder written from the words of include/entro.h alone (tests/format_from_header.py):
    the library's encoder writes the same stream and index, and the library's decoder turns
    that encoder's stream into the dequantised symbols, bit for bit."""
    import format_from_header
    w_np, w_dev = _values(n, 0.02, 777 + n)
    q, qp = E.entro_quantize_tensor(w_dev, bits)
    counts = E.entro_histogram(q, bits).tolist()
    cb = E.entro_build_codebook(counts)
    q_np = q.cpu().numpy()
    stream, offsets, sub_len = format_from_header.encode(q_np.tolist(), cb.lengths().tolist(), cb.codes().tolist(), chunk)
    enc = E.entro_encode(q, cb, chunk, stream_words=E.entro_stream_words(counts, cb))
    assert np.array_equal(enc.stream_np(), stream)
    assert np.array_equal(enc.offsets(), offsets)
    assert np.array_equal(enc.sub_len(), sub_len)
    index = torch.from_numpy(format_from_header.index_bytes(offsets, sub_len).copy()).cuda()
    out = E.entro_decode_dequant(to_dev_stream(stream), index, n, chunk, cb, qp.scale, qp.zero_point)
    torch.cuda.synchronize()
    assert_status_ok()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q_np, qp.scale, qp.zero_point))


def test_batched_offline_stages_equal_the_per_tensor_calls_and_the_oracle():
    """entro_quantize_histogram_batched / entro_encode_batched: parameters (computed on the device),
    symbols, counts, streams and indices of every tensor equal the per-tensor calls' and the oracle's."""
    specs = [(8, 300_000 + 7, "matrix"), (8, 4096, "gain"), (8, 1, "matrix"), (8, 5 * 4096, "matrix"), (8, 33, "gain")]
    for bits, chunk in ((8, 4096), (4, 8192)):
        vals = [_values(n, 0.02 + 0.003 * k, 8800 + 10 * bits + k, kind) for k, (_, n, kind) in enumerate(specs)]
        qs, qps, counts = E.entro_quantize_histogram_batched([v[1] for v in vals], bits)
        cbs, words = [], []
        for j, (w_np, w_dev) in enumerate(vals):
            c = oracle.compress(w_np, bits, chunk)
            q1, qp1 = E.entro_quantize_tensor(w_dev, bits)
            assert (np.float32(qps[j].scale).tobytes(), qps[j].zero_point, qps[j].mode) == \
                   (np.float32(c.qp.scale).tobytes(), c.qp.zero_point, c.qp.mode) == \
                   (np.float32(qp1.scale).tobytes(), qp1.zero_point, qp1.mode), j
            assert np.array_equal(qs[j].cpu().numpy(), c.q) and torch.equal(qs[j], q1), j
            assert np.array_equal(counts[j, :1 << bits], c.counts) and not counts[j, 1 << bits:].any(), j
            cb = E.entro_build_codebook_np(counts[j], 1 << bits)
            assert np.array_equal(cb.lengths(), c.lengths)
            cbs.append(cb)
            words.append(E.entro_stream_words_np(counts[j], cb))
            vals[j] = (c, w_dev)
        encs = E.entro_encode_batched(qs, cbs, chunk, words)
        for j, enc in enumerate(encs):
            c = vals[j][0]
            assert enc.total_bits == c.enc.total_bits, j
            assert np.array_equal(enc.stream_np(), c.enc.stream), j
            assert np.array_equal(enc.offsets(), c.enc.offsets) and np.array_equal(enc.sub_len(), c.enc.sub_len), j
        # a stream buffer that is too small is reported and left zeroed; the others are complete
        short = list(words)
        short[0] = E.STREAM_SLACK_WORDS + 2
        with pytest.raises(E.EntroError) as e:
            E.entro_encode_batched(qs, cbs, chunk, short)
        assert e.value.status == E.ERR_BUFFER_TOO_SMALL
    # a tensor with an infinity is reported; the other tensors of the batch are complete
    w_bad = vals[0][1].clone()
    w_bad[5] = float("inf")
    with pytest.raises(E.EntroError) as e:
        E.entro_quantize_histogram_batched([vals[3][1], w_bad], 8)
    assert e.value.status == E.ERR_NONFINITE


def test_encode_errors():
    q = torch.tensor([0, 1, 2, 3] * 100, dtype=torch.uint8).cuda()
    cb = E.entro_build_codebook([5, 5, 5, 0])              # symbol 3 has no code
    with pytest.raises(E.EntroError) as e:
        E.entro_encode(q, cb, 4096)
    assert e.value.status == E.ERR_INVALID_ARG
    cb = E.entro_build_codebook([5, 5, 5, 5])
    with pytest.raises(E.EntroError) as e:
        E.entro_encode(q, cb, 4096, stream_words=E.STREAM_SLACK_WORDS + 2)   # needs 25 words
    assert e.value.status == E.ERR_BUFFER_TOO_SMALL


# ----------------------------------------------------------------------------- decode + dequant

@pytest.mark.parametrize("bits,chunk", [(8, 4096), (4, 8192), (8, 1024), (4, 4096), (8, 32), (8, 96)])
def test_decode_of_oracle_streams_small_and_ragged(bits, chunk):
    sizes = [1, 2, 31, 32, 33, chunk // 32, chunk - 1, chunk, chunk + 1, 2 * chunk, 3 * chunk + 517, 40 * chunk + 5]
    for n in sizes:
        w_np, _ = _values(n, 0.02, 7 * n + bits)
        c = oracle.compress(w_np, bits, chunk)
        got = gpu_decode_from_oracle_stream(c, n, chunk)
        assert np.array_equal(got, expected_out(c)), (bits, chunk, n)
    assert_status_ok()


@pytest.mark.parametrize("bits,chunk", [(8, 4096), (4, 8192)])
def test_decode_flat_histograms(bits, chunk):
    """Inputs without heavy tails spread the symbols over many levels: the 8-bit path then uses
    the wider exponent-indexed table and groups of three, the 4-bit path one symbol per lookup.
    A uniform histogram (every code the same length) is resolved by no table cell at all and
    runs entirely on the symbol-by-symbol repair."""
    for n in (chunk - 1, 9 * chunk, 33 * chunk + 77):
        w_np, _ = _values(n, 0.02, 4242 + n % 100 + bits, "gauss")
        c = oracle.compress(w_np, bits, chunk)
        assert np.array_equal(gpu_decode_from_oracle_stream(c, n, chunk), expected_out(c)), (bits, n)
    nsym = 1 << bits
    q = np.random.default_rng(bits).integers(0, nsym, 20 * chunk + 5).astype(np.uint8)
    ln = oracle.huffman_lengths(np.bincount(q, minlength=nsym).tolist())
    cd = oracle.canonical_codes(ln)
    enc = oracle.encode(q, ln, cd, chunk)
    out = E.entro_decode_dequant(to_dev_stream(enc.stream), to_dev_index(enc), q.size, chunk,
                                 E.Codebook.from_lengths(ln.tolist(), cd.tolist()), 0.03125, nsym // 2)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.03125, nsym // 2))
    assert_status_ok()


@pytest.mark.parametrize("sigma_levels,foreign", [(0.6, False), (2.0, False), (6.0, False), (14.0, False), (40.0, False),
                                                  (40.0, True)])
def test_decode_every_group_size(sigma_levels, foreign):
    """The decoder picks the number of lookups per group from the code lengths and the bits
    per symbol: below 2 bit per symbol eight lookups share one view, narrow histograms take two
    fours under one check, wider ones four, three,
    and a codebook that does not fit its data (here: built for a narrow histogram, used on a
    wide one, about 14 bits per symbol) two.  Symbols are drawn directly, as rounded
    Gaussians of the given width in quantisation levels; the values check the symbols."""
    chunk, n = 4096, 21 * 4096 + 333
    rng = np.random.default_rng(int(sigma_levels * 10) + foreign)
    q = np.clip(np.rint(rng.normal(128.0, sigma_levels, n)), 0, 255).astype(np.uint8)
    counts = np.bincount(q, minlength=256)
    if foreign:
        narrow = np.clip(np.rint(rng.normal(128.0, 3.0, n)), 0, 255).astype(np.uint8)
        counts = np.bincount(narrow, minlength=256) + 1          # every symbol keeps a code
    ln = oracle.huffman_lengths(counts.tolist())
    cd = oracle.canonical_codes(ln)
    enc = oracle.encode(q, ln, cd, chunk)
    if foreign:
        assert int(enc.offsets[-1]) / n > 8.5
    out = E.entro_decode_dequant(to_dev_stream(enc.stream), to_dev_index(enc), n, chunk,
                                 E.Codebook.from_lengths(ln.tolist(), cd.tolist()), 0.0078125, 128)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.0078125, 128))
    assert_status_ok()


@pytest.mark.parametrize("sigma_levels", [0.45, 1.6, 9.0, 24.0])
def test_groups_under_one_check_are_repaired_wherever_they_fail(sigma_levels):
    """Several groups of lookups share one check; when it fails, what failed first is repaired
    and what came after it is done again (3 + 3 + 2 lookups, two fours), or everything is
    written again (sixteen or thirty-two symbols of a narrow histogram).  A million symbols at widths near
    the upper end of each mode's range make every position of a group fail hundreds of
    times: groups that need 32 bits or more, and codes beyond the table's reach."""
    chunk, n = 4096, 256 * 4096
    rng = np.random.default_rng(int(sigma_levels * 10))
    q = np.clip(np.rint(rng.normal(128.0, sigma_levels, n)), 0, 255).astype(np.uint8)
    q[rng.integers(0, n, n // 400)] = rng.integers(0, 256, n // 400).astype(np.uint8)   # rare symbols, long codes
    ln = oracle.huffman_lengths(np.bincount(q, minlength=256).tolist())
    cd = oracle.canonical_codes(ln)
    enc = oracle.encode(q, ln, cd, chunk)
    out = E.entro_decode_dequant(to_dev_stream(enc.stream), to_dev_index(enc), n, chunk,
                                 E.Codebook.from_lengths(ln.tolist(), cd.tolist()), 0.0078125, 128)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.0078125, 128))
    assert_status_ok()


@pytest.mark.parametrize("chunk", [8192, 16384])
def test_chunks_larger_than_a_warps_ring(chunk):
    """At 8 bit per symbol a chunk of 8192 or 16384 symbols does not fit the 5 KB of shared
    memory a warp has in the usual launch shape; the library then launches fewer warps with
    larger rings (and whatever still does not fit is decoded from global memory)."""
    rng = np.random.default_rng(chunk)
    tensors = []
    for n in (6 * chunk + 77, 3 * chunk):
        q = rng.integers(0, 256, n).astype(np.uint8)
        ln = oracle.huffman_lengths(np.bincount(q, minlength=256).tolist())
        cd = oracle.canonical_codes(ln)
        tensors.append((q, ln, cd, oracle.encode(q, ln, cd, chunk)))
    descs, outs, keep = [], [], []
    for q, ln, cd, enc in tensors:
        assert int(enc.offsets[1]) // 8 > 6000
        s, ix = to_dev_stream(enc.stream), to_dev_index(enc)
        out = torch.empty(q.size, dtype=torch.float16, device="cuda")
        keep += [s, ix]
        descs.append(E.make_desc(s, ix, q.size, chunk, E.Codebook.from_lengths(ln.tolist(), cd.tolist()), 0.03125, 128, out))
        outs.append(out)
    E.entro_decode_dequant_batched(descs)
    torch.cuda.synchronize()
    assert_status_ok()
    for (q, _, _, _), out in zip(tensors, outs):
        assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.03125, 128))


@pytest.mark.parametrize("sigma_levels,lo,hi", [(0.3, 1.0, 1.3), (0.5, 1.32, 1.74), (0.6, 1.32, 1.74), (1.5, 1.8, 4.0)])
def test_decode_four_bit_modes(sigma_levels, lo, hi):
    """4-bit alphabets are decoded eight symbols per lookup while eight codes usually fit
    the table's window (up to 1.31 bit per symbol) and one by one above (eight lookups on one
    32-bit view up to 2 bit per symbol).  Symbols are drawn
    directly as rounded Gaussians; the bit rate is checked so that the cases lie on both
    sides of that limit, close to it and far from it; output as fp16 values, and as packed
    nibbles (the integer sink of the same loops)."""
    chunk, n = 8192, 19 * 8192 + 4101
    rng = np.random.default_rng(int(sigma_levels * 100))
    q = np.clip(np.rint(rng.normal(8.0, sigma_levels, n)), 0, 15).astype(np.uint8)
    q[:: 997] = rng.integers(0, 16, q[:: 997].size)          # every symbol occurs, some codes are long
    ln = oracle.huffman_lengths(np.bincount(q, minlength=16).tolist())
    cd = oracle.canonical_codes(ln)
    enc = oracle.encode(q, ln, cd, chunk)
    assert lo <= int(enc.offsets[-1]) / n <= hi
    cb = E.Codebook.from_lengths(ln.tolist(), cd.tolist())
    s, ix = to_dev_stream(enc.stream), to_dev_index(enc)
    out = E.entro_decode_dequant(s, ix, n, chunk, cb, 0.0625, 8)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.0625, 8))
    packed = torch.full(((n + 1) // 2,), 0xEE, dtype=torch.uint8, device="cuda")
    E.entro_decode_symbols_batched([E.make_desc_bytes(s, ix, n, chunk, cb, packed)], True)
    torch.cuda.synchronize()
    q2 = np.concatenate([q, np.zeros(n & 1, dtype=np.uint8)])
    assert np.array_equal(packed.cpu().numpy(), (q2[0::2] | (q2[1::2] << 4)).astype(np.uint8))
    assert_status_ok()


@pytest.mark.parametrize("bits,chunk,packed", [(8, 4096, False), (4, 8192, False), (4, 8192, True), (4, 1024, True),
                                               (8, 96, False), (4, 64, True)])
def test_decode_to_integer_symbols(bits, chunk, packed):
    """The paper's decoder hands integers to the inference engine: one symbol per byte, or two
    4-bit symbols per byte.  Bit-exact against the oracle's quantised symbols."""
    keep, descs, outs, refs = [], [], [], []
    for n in (1, 2, 33, chunk - 1, chunk, 3 * chunk + 517, 40 * chunk + 5, 64 * chunk):
        w_np, _ = _values(n, 0.02, 31 * n % 1000 + bits)
        c = oracle.compress(w_np, bits, chunk)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        out = torch.full(((n + 1) // 2 if packed else n,), 0xEE, dtype=torch.uint8, device="cuda")
        keep += [s, ix]
        descs.append(E.make_desc_bytes(s, ix, n, chunk, codebook_from_oracle(c), out))
        outs.append(out)
        q = c.q
        if packed:
            q2 = np.concatenate([q, np.zeros(n & 1, dtype=np.uint8)])
            refs.append((q2[0::2] | (q2[1::2] << 4)).astype(np.uint8))
        else:
            refs.append(q)
    E.entro_decode_symbols_batched(descs, packed)
    torch.cuda.synchronize()
    assert_status_ok()
    for out, ref in zip(outs, refs):
        assert np.array_equal(out.cpu().numpy(), ref)


@pytest.mark.parametrize("bits,chunk,cap", [(8, 4096, 12), (8, 4096, 9), (4, 8192, 6)])
def test_length_limited_codes_encode_and_decode(bits, chunk, cap):
    """The optional capped code: the library's codebook equals the oracle's, the GPU encoder
    produces the oracle's stream under it, and the ordinary decode call returns the dequantised
    symbols."""
    n = 37 * chunk + 1234
    w_np, w_dev = _values(n, 0.02, 5150 + cap)
    q_ref, qp = oracle.quantize_tensor(w_np, bits)
    counts = oracle.histogram(q_ref, 1 << bits)
    ln = oracle.length_limited_lengths(counts, cap)
    cd = oracle.canonical_codes(ln)
    assert ln.max() <= cap < oracle.huffman_lengths(counts).max()       # the cap really binds
    enc_ref = oracle.encode(q_ref, ln, cd, chunk)
    cb = E.entro_build_codebook_limited(counts.tolist(), cap)
    assert np.array_equal(cb.lengths(), ln) and np.array_equal(cb.codes(), cd)
    enc = E.entro_encode(torch.from_numpy(q_ref).cuda(), cb, chunk, stream_words=E.entro_stream_words(counts.tolist(), cb))
    assert enc.total_bits == enc_ref.total_bits and np.array_equal(enc.stream_np(), enc_ref.stream)
    out = E.entro_decode_dequant(enc.stream, enc.index, n, chunk, cb, qp.scale, qp.zero_point)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q_ref, qp.scale, qp.zero_point))
    assert_status_ok()


def test_decode_config1_single_tensor():
    """1024 x 1024, sigma 0.02, seed 0, asymmetric uint8, 4096-symbol chunks."""
    wl = workloads.single_tensor()
    spec = wl.tensors[0]
    w = workloads.make_tensor(spec)
    c = oracle.compress(w.numpy(), wl.bits, wl.chunk_symbols)
    assert c.qp.mode == oracle.MODE_ASYMMETRIC
    got = gpu_decode_from_oracle_stream(c, spec.numel, wl.chunk_symbols)
    assert np.array_equal(got, expected_out(c))
    # and the whole GPU pipeline on the same bytes
    q, qp = E.entro_quantize_tensor(w.cuda().view(-1), wl.bits)
    assert np.array_equal(q.cpu().numpy(), c.q)
    counts = E.entro_histogram(q, wl.bits)
    cb = E.entro_build_codebook(counts.tolist())
    enc = E.entro_encode(q, cb, wl.chunk_symbols, stream_words=E.entro_stream_words(counts.tolist(), cb))
    assert np.array_equal(enc.stream_np(), c.enc.stream)
    out = E.entro_decode_dequant(enc.stream, enc.index, spec.numel, wl.chunk_symbols, cb, qp.scale, qp.zero_point)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint16), expected_out(c))
    assert_status_ok()


def _fib_counts(k, nsym):
    fib = [1, 1]
    while len(fib) < k:
        fib.append(fib[-1] + fib[-2])
    return fib[:k] + [0] * (nsym - k)


def test_repeated_call_on_few_tensors_reuses_what_is_in_place():
    """A batched decode of few tensors leaves descriptors and tables on the device; the same call
    again is then only the decode launch.  Repeats, other tensors in between, and another user of
    the library's device area in between (an encode) must all give the oracle's output."""
    cases = []
    for k, (bits, chunk, n) in enumerate([(8, 4096, 5 * 4096 + 77), (4, 8192, 3 * 8192), (8, 4096, 300_000)]):
        w_np, _ = _values(n, 0.02, 6100 + k)
        c = oracle.compress(w_np, bits, chunk)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        out = torch.zeros(n, dtype=torch.float16, device="cuda")
        cases.append((c, s, ix, out, E.make_desc(s, ix, n, chunk, codebook_from_oracle(c), c.qp.scale, c.qp.zero_point, out)))

    def run(which):
        descs = E.desc_array([cases[i][4] for i in which])
        for i in which:
            cases[i][3].zero_()
        E.entro_decode_dequant_batched(descs)
        torch.cuda.synchronize()
        assert_status_ok()
        for i in which:
            assert np.array_equal(cases[i][3].cpu().numpy().view(np.uint16), expected_out(cases[i][0])), (which, i)

    launches = E.entro_kernel_launch_count()
    run([0, 1])
    first = E.entro_kernel_launch_count() - launches
    run([0, 1])                                            # the repeat
    assert E.entro_kernel_launch_count() - launches == first + 1
    run([2])                                               # other tensors
    run([0, 1])
    q = torch.from_numpy(cases[0][0].q).cuda()
    E.entro_encode(q, codebook_from_oracle(cases[0][0]), 4096)       # writes the library's device area
    run([0, 1])
    run([0, 1])


@pytest.mark.parametrize("k,nsym", [(31, 256), (33, 256), (16, 16), (12, 16)])
def test_decode_long_codes(k, nsym):
    """Fibonacci histograms give code lengths up to k - 1 (32 at most): the lookup table's
    escape path must decode them, including runs of long codes next to each other."""
    counts = _fib_counts(k, nsym)
    ln = oracle.huffman_lengths(counts)
    assert ln.max() == k - 1
    cd = oracle.canonical_codes(ln)
    rng = np.random.default_rng(k)
    parts = [np.arange(k), rng.integers(0, k, 20000), rng.integers(0, min(k, 8), 3000),
             np.repeat(np.arange(k), 40), rng.integers(max(0, k - 6), k, 30000)]
    q = np.concatenate(parts).astype(np.uint8)
    rng.shuffle(q[: q.size // 2])
    for chunk in (4096, 8192, 64):
        enc = oracle.encode(q, ln, cd, chunk)
        s, z = 0.0123, 3
        cb = E.Codebook.from_lengths(ln.tolist(), cd.tolist())
        out = E.entro_decode_dequant(to_dev_stream(enc.stream), to_dev_index(enc), q.size, chunk, cb, s, z)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, s, z))
    assert_status_ok()


def test_decode_single_symbol_alphabet_and_two_symbols():
    for counts in ([0, 9, 0, 0], [4, 0, 0, 6]):
        ln = oracle.huffman_lengths(counts)
        cd = oracle.canonical_codes(ln)
        used = [k for k, c in enumerate(counts) if c]
        q = np.random.default_rng(1).choice(used, 10000).astype(np.uint8)
        enc = oracle.encode(q, ln, cd, 4096)
        cb = E.Codebook.from_lengths(ln.tolist(), cd.tolist())
        out = E.entro_decode_dequant(to_dev_stream(enc.stream), to_dev_index(enc), q.size, 4096, cb, 0.5, 1)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy().view(np.uint16), oracle.dequant(q, 0.5, 1))
    assert_status_ok()


@pytest.mark.parametrize("lut_bits,warps,ctas,per_item", [(10, 8, 2, 8), (12, 16, 1, 64), (11, 32, 1, 7),
                                                          (11, 4, 2, 1), (12, 16, 2, 64)])
def test_decode_launch_shapes(lut_bits, warps, ctas, per_item):
    """The result does not depend on table width, CTA shape or work-item size."""
    try:
        E.entro_set_decode_config(lut_bits, warps, ctas, per_item)
        for bits, chunk, n in ((8, 4096, 600_000 + 77), (4, 8192, 900_000)):
            w_np, _ = _values(n, 0.03, lut_bits + warps)
            c = oracle.compress(w_np, bits, chunk)
            assert np.array_equal(gpu_decode_from_oracle_stream(c, n, chunk), expected_out(c))
        assert_status_ok()
    finally:
        E.entro_set_decode_config(*E.DEFAULT_DECODE_CONFIG)


def test_batched_decode_mixed_tensors():
    """One launch over tensors of different widths, chunk sizes, modes and lengths."""
    specs = [(8, 4096, 300_000, "matrix"), (4, 8192, 100_000, "matrix"), (8, 4096, 2048, "gain"),
             (4, 8192, 3072, "gain"), (8, 4096, 4096 * 130 + 1, "matrix"), (8, 1024, 50_000, "matrix"),
             (4, 8192, 8192 * 9, "matrix"), (8, 4096, 1, "matrix")]
    keep, descs, outs, refs = [], [], [], []
    for i, (bits, chunk, n, kind) in enumerate(specs):
        w_np, _ = _values(n, 0.02 + 0.003 * i, 500 + i, kind)
        c = oracle.compress(w_np, bits, chunk)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        out = torch.zeros(n, dtype=torch.float16, device="cuda")
        keep += [s, ix]
        outs.append(out)
        refs.append(expected_out(c))
        descs.append(E.make_desc(s, ix, n, chunk, codebook_from_oracle(c), c.qp.scale, c.qp.zero_point, out))
    E.entro_decode_dequant_batched(descs)
    torch.cuda.synchronize()
    for out, ref in zip(outs, refs):
        assert np.array_equal(out.cpu().numpy().view(np.uint16), ref)
    assert_status_ok()


def test_host_buffer_entry_point():
    n, bits, chunk = 500_000, 8, 4096
    w_np, _ = _values(n, 0.02, 99)
    c = oracle.compress(w_np, bits, chunk)
    h_stream = torch.from_numpy(c.enc.stream.view(np.int32).copy()).pin_memory()
    h_index = torch.from_numpy(index_bytes_np(c.enc).copy()).pin_memory()
    h_out = torch.zeros(n, dtype=torch.float16).pin_memory()
    d_stream = torch.empty_like(h_stream, device="cuda")
    d_index = torch.empty_like(h_index, device="cuda")
    d_out = torch.empty(n, dtype=torch.float16, device="cuda")
    descs = E.desc_array([E.make_desc(d_stream, d_index, n, chunk, codebook_from_oracle(c), c.qp.scale,
                                      c.qp.zero_point, d_out)])
    io = (E.HostIO * 1)(E.HostIO(h_stream.data_ptr(), h_index.data_ptr(), h_out.data_ptr()))
    E.entro_decode_dequant_batched_host(descs, io)
    assert np.array_equal(h_out.numpy().view(np.uint16), expected_out(c))
    assert_status_ok()
    # without a host output buffer the result is left on the device
    d_out.zero_()
    d_stream.zero_()
    h_out.zero_()
    io = (E.HostIO * 1)(E.HostIO(h_stream.data_ptr(), h_index.data_ptr(), None))
    E.entro_decode_dequant_batched_host(descs, io)
    assert np.array_equal(d_out.cpu().numpy().view(np.uint16), expected_out(c))
    assert not h_out.any()
    assert_status_ok()


# ----------------------------------------------------------------------------- malformed input

def test_malformed_input_is_reported_not_fatal():
    n, bits, chunk = 200_000, 8, 4096
    w_np, _ = _values(n, 0.02, 31337)
    c = oracle.compress(w_np, bits, chunk)
    cb = codebook_from_oracle(c)
    good_stream, good_index = c.enc.stream, index_bytes_np(c.enc)

    def run(stream_np, index_np):
        out = E.entro_decode_dequant(to_dev_stream(stream_np), torch.from_numpy(index_np.copy()).cuda(), n, chunk,
                                     cb, c.qp.scale, c.qp.zero_point)
        st = E.entro_last_device_status()
        return out.cpu().numpy().view(np.uint16), st

    out, st = run(good_stream, good_index)
    assert st == E.OK and np.array_equal(out, expected_out(c))
    # (a) a chunk boundary moved: that chunk and its neighbour no longer match their sub-block lengths
    idx = good_index.copy()
    off = idx[: 8 * (oracle.num_chunks(n, chunk) + 1)].view(np.uint64)
    off[3] += 5
    _, st = run(good_stream, idx)
    assert st == E.ERR_CORRUPT_STREAM
    # (b) an offset far beyond the stream buffer
    idx = good_index.copy()
    off = idx[: 8 * (oracle.num_chunks(n, chunk) + 1)].view(np.uint64)
    off[5] = 1 << 40
    off[6] = (1 << 40) + 100
    _, st = run(good_stream, idx)
    assert st == E.ERR_CORRUPT_STREAM
    # (c) flipped stream bits: lanes end somewhere other than their recorded end
    bad = good_stream.copy()
    bad[100:140] ^= 0x5A5A5A5A
    out, st = run(bad, good_index)
    assert st == E.ERR_CORRUPT_STREAM
    first_bad_chunk = int(np.searchsorted(c.enc.offsets, 100 * 32, side="right")) - 1
    assert np.array_equal(out[: first_bad_chunk * chunk], expected_out(c)[: first_bad_chunk * chunk])
    # (d) the status word was cleared by the read: a good run is clean again
    out, st = run(good_stream, good_index)
    assert st == E.OK and np.array_equal(out, expected_out(c))


# ----------------------------------------------------------------------------- model-shaped workloads

def _check_workload_slice(wl, specs):
    """Full GPU pipeline vs the oracle, tensor by tensor, then one batched decode."""
    keep, descs, outs, refs = [], [], [], []
    for spec in specs:
        w = workloads.make_tensor(spec, "cuda").view(-1)
        w_np = w.cpu().numpy()
        c = oracle.compress(w_np, wl.bits, wl.chunk_symbols)
        q, qp = E.entro_quantize_tensor(w, wl.bits)
        assert (qp.mode, qp.zero_point, qp.scale) == (c.qp.mode, c.qp.zero_point, c.qp.scale), spec.name
        assert torch.equal(q.cpu(), torch.from_numpy(c.q)), spec.name
        counts = E.entro_histogram(q, wl.bits)
        assert np.array_equal(counts, c.counts)
        cb = E.entro_build_codebook(counts.tolist())
        assert np.array_equal(cb.lengths(), c.lengths) and np.array_equal(cb.codes(), c.codes), spec.name
        enc = E.entro_encode(q, cb, wl.chunk_symbols, stream_words=E.entro_stream_words(counts.tolist(), cb))
        assert torch.equal(enc.stream.cpu(), torch.from_numpy(c.enc.stream.view(np.int32))), spec.name
        assert np.array_equal(enc.offsets(), c.enc.offsets) and np.array_equal(enc.sub_len(), c.enc.sub_len)
        out = torch.zeros(spec.numel, dtype=torch.float16, device="cuda")
        keep += [enc]
        outs.append(out)
        refs.append(torch.from_numpy(expected_out(c).view(np.int16)))
        descs.append(E.make_desc(enc.stream, enc.index, spec.numel, wl.chunk_symbols, cb, qp.scale, qp.zero_point, out))
    E.entro_decode_dequant_batched(descs)
    torch.cuda.synchronize()
    for spec, out, ref in zip(specs, outs, refs):
        assert torch.equal(out.cpu().view(torch.int16), ref), spec.name
    assert_status_ok()


def test_smollm_shaped_first_layer_and_gains():
    wl = workloads.smollm_1p7b(max_layers=1)
    specs = [t for t in wl.tensors if t.name.startswith("layers.0.") or t.kind == "gain"]
    modes = set()
    for spec in specs:
        modes.add(oracle.quant_params(workloads.make_tensor(spec).numpy(), wl.bits).mode)
    assert modes == {oracle.MODE_UNSIGNED, oracle.MODE_ASYMMETRIC}       # both branches of the mixed scheme
    _check_workload_slice(wl, specs)


def test_phi3_shaped_first_layer_uint4():
    wl = workloads.phi3_mini_4k(max_layers=1)
    _check_workload_slice(wl, [t for t in wl.tensors if t.name.startswith("layers.0.") or t.kind == "gain"])


@pytest.mark.parametrize("bits", [8, 4])
def test_mistral_shaped_first_layer(bits):
    wl = workloads.mistral_7b(bits=bits, max_layers=1)
    _check_workload_slice(wl, [t for t in wl.tensors if t.name.startswith("layers.0.") or t.kind == "gain"])

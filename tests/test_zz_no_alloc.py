"""entro_decode_dequant_static: the decode entry point for host applications that cannot
let the library allocate (all device memory already in the application's own pool, or an
allocation's device-wide synchronisation not acceptable while other streams run).

Collected last on purpose.  It runs the new entry point through the C ABI on two calls in
a row and compares it, bit for bit (the tolerance of every decode test here is zero), with
the regular batched entry point and with the oracle's definition of the output.  The
second call uses fewer and different tensors, so anything the first call left in the
shared scratch array would show."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import codebook_from_oracle, expected_out, to_dev_index, to_dev_stream

pytestmark = pytest.mark.gpu


def _case(specs, seed0):
    keep, descs_a, descs_b, outs_a, outs_b, refs = [], [], [], [], [], []
    for i, (bits, chunk, n, kind) in enumerate(specs):
        w = workloads.make_values(n, 0.02 + 0.004 * i, seed0 + i, kind).numpy()
        c = oracle.compress(w, bits, chunk)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        a = torch.zeros(n, dtype=torch.float16, device="cuda")
        b = torch.zeros(n, dtype=torch.float16, device="cuda")
        cb = codebook_from_oracle(c)
        keep += [s, ix]
        descs_a.append(E.make_desc(s, ix, n, chunk, cb, c.qp.scale, c.qp.zero_point, a))
        descs_b.append(E.make_desc(s, ix, n, chunk, cb, c.qp.scale, c.qp.zero_point, b))
        outs_a.append(a)
        outs_b.append(b)
        refs.append(expected_out(c))
    return keep, descs_a, descs_b, outs_a, outs_b, refs


def _run_and_compare(specs, seed0):
    keep, descs_a, descs_b, outs_a, outs_b, refs = _case(specs, seed0)
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    E.entro_decode_dequant_batched(descs_a)
    E.entro_decode_dequant_static(descs_b, status)
    torch.cuda.synchronize()
    assert E.entro_last_device_status() == E.OK
    assert int(status.item()) == 0
    for a, b, ref in zip(outs_a, outs_b, refs):
        got_a = a.cpu().numpy().view(np.uint16)
        got_b = b.cpu().numpy().view(np.uint16)
        assert np.array_equal(got_b, got_a)      # same as the existing entry point
        assert np.array_equal(got_b, ref)        # and both are what the oracle defines


def test_static_entry_point_matches_batched_on_two_calls_in_a_row():
    first = [(8, 4096, 700_000 + 13, "matrix"), (4, 8192, 500_000, "matrix"), (8, 4096, 4096, "gain"),
             (4, 8192, 3000, "gain"), (8, 1024, 90_001, "matrix"), (8, 4096, 1, "matrix"),
             (4, 8192, 8192 * 20, "matrix"), (8, 4096, 4096 * 150, "matrix")]
    assert len(first) == E.STATIC_MAX_TENSORS
    _run_and_compare(first, 9000)
    second = [(4, 8192, 300_000 + 5, "matrix"), (8, 4096, 250_000, "matrix"), (8, 4096, 100, "gain")]
    _run_and_compare(second, 9100)


def test_static_entry_point_with_chunks_larger_than_a_warps_ring():
    """Flat 8-bit symbols in 8192-symbol chunks: a chunk is about 8 KB, more than the 5 KB of
    shared memory a warp has in the usual launch shape.  Both entry points then launch fewer
    warps with larger rings; their outputs must agree bit for bit and be the dequantised
    symbols."""
    chunk = 8192
    rng = np.random.default_rng(9400)
    keep, descs_a, descs_b, outs_a, outs_b, refs = [], [], [], [], [], []
    for n in (5 * chunk + 31, 2 * chunk):
        q = rng.integers(0, 256, n).astype(np.uint8)
        ln = oracle.huffman_lengths(np.bincount(q, minlength=256).tolist())
        cd = oracle.canonical_codes(ln)
        enc = oracle.encode(q, ln, cd, chunk)
        assert int(enc.offsets[1]) // 8 > 6000
        s, ix = to_dev_stream(enc.stream), to_dev_index(enc)
        cb = E.Codebook.from_lengths(ln.tolist(), cd.tolist())
        a = torch.zeros(n, dtype=torch.float16, device="cuda")
        b = torch.zeros(n, dtype=torch.float16, device="cuda")
        keep += [s, ix]
        descs_a.append(E.make_desc(s, ix, n, chunk, cb, 0.03125, 128, a))
        descs_b.append(E.make_desc(s, ix, n, chunk, cb, 0.03125, 128, b))
        outs_a.append(a)
        outs_b.append(b)
        refs.append(oracle.dequant(q, 0.03125, 128))
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    E.entro_decode_dequant_batched(descs_a)
    E.entro_decode_dequant_static(descs_b, status)
    torch.cuda.synchronize()
    assert E.entro_last_device_status() == E.OK and int(status.item()) == 0
    for a, b, ref in zip(outs_a, outs_b, refs):
        assert np.array_equal(b.cpu().numpy().view(np.uint16), a.cpu().numpy().view(np.uint16))
        assert np.array_equal(b.cpu().numpy().view(np.uint16), ref)


def test_static_entry_point_reports_corruption_in_the_callers_word():
    n, chunk = 150_000, 4096
    c = oracle.compress(workloads.make_values(n, 0.02, 9200).numpy(), 8, chunk)
    bad = c.enc.stream.copy()
    bad[50:80] ^= 0x3C3C3C3C
    out = torch.zeros(n, dtype=torch.float16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    desc = E.make_desc(to_dev_stream(bad), to_dev_index(c.enc), n, chunk, codebook_from_oracle(c), c.qp.scale,
                       c.qp.zero_point, out)
    E.entro_decode_dequant_static([desc], status)
    torch.cuda.synchronize()
    assert int(status.item()) != 0
    # the next call starts from a cleared status word
    good = E.make_desc(to_dev_stream(c.enc.stream), to_dev_index(c.enc), n, chunk, codebook_from_oracle(c),
                       c.qp.scale, c.qp.zero_point, out)
    E.entro_decode_dequant_static([good], status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(out.cpu().numpy().view(np.uint16), expected_out(c))


def test_static_entry_point_rejects_more_tensors_than_it_holds():
    n, chunk = 5000, 4096
    c = oracle.compress(workloads.make_values(n, 0.02, 9300).numpy(), 8, chunk)
    s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
    out = torch.zeros(n, dtype=torch.float16, device="cuda")
    descs = [E.make_desc(s, ix, n, chunk, codebook_from_oracle(c), c.qp.scale, c.qp.zero_point, out)
             for _ in range(E.STATIC_MAX_TENSORS + 1)]
    with pytest.raises(E.EntroError) as e:
        E.entro_decode_dequant_static(descs)
    assert e.value.status == E.ERR_TOO_MANY_TENSORS
    assert "static scratch" in E.status_string(E.ERR_TOO_MANY_TENSORS)

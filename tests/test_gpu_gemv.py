"""Fused decode + dequantise + matrix-vector product (one token or a small batch) against the oracle.

The weights inside the product are the bit-exact fp16 values of the decode path (checked
elsewhere); the product itself is summed in fp32 in an order that differs from the oracle's
fp64 loop, so it has a tolerance: |y - y64| <= 2^-10 |y64| + cols * 2^-23 * sum|w x| + 2^-24
(one fp16 rounding of the result, the fp32 accumulation bound, the fp16 subnormal step).
With x a unit vector the product reduces to reading a column and must be bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import assert_status_ok, codebook_from_oracle, expected_out, to_dev_index, to_dev_stream

pytestmark = pytest.mark.gpu


def _f16(bits_u16):
    return bits_u16.view(np.float16).astype(np.float64)


def _compressed(rows, cols, bits, chunk, seed, sigma=0.02):
    w = workloads.make_values(rows * cols, sigma, seed).numpy()
    c = oracle.compress(w, bits, chunk)
    s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
    desc = E.make_desc_no_out(s, ix, rows * cols, chunk, codebook_from_oracle(c), c.qp.scale, c.qp.zero_point)
    desc._keep = (s, ix)          # the descriptor holds raw pointers: keep the device buffers alive with it
    return c, desc


def _check(y_gpu_u16, w_hat_u16, rows, cols, x_u16):
    y64, asum = oracle.gemv_f64(w_hat_u16, rows, cols, x_u16)
    got = _f16(y_gpu_u16)
    bound = 2.0 ** -10 * np.abs(y64) + cols * 2.0 ** -23 * asum + 2.0 ** -24
    bad = np.abs(got - y64) > bound
    assert not bad.any(), (int(bad.sum()), float(np.abs(got - y64).max()))


@pytest.mark.parametrize("bits,chunk,rows,cols", [(4, 8192, 64, 512), (8, 4096, 64, 512), (4, 8192, 3, 1280),
                                                  (8, 4096, 37, 768), (4, 8192, 33, 4096), (4, 1024, 16, 256)])
def test_fused_gemv_small(bits, chunk, rows, cols):
    c, desc = _compressed(rows, cols, bits, chunk, 7000 + rows + cols)
    x = workloads.make_vector(cols, 11).cuda()
    (y,) = E.entro_decode_dequant_gemv([desc], [x], [(rows, cols)])
    torch.cuda.synchronize()
    assert_status_ok()
    _check(y.cpu().numpy().view(np.uint16), expected_out(c), rows, cols, x.cpu().numpy().view(np.uint16))


@pytest.mark.parametrize("bits,chunk", [(4, 8192), (8, 4096)])
def test_unit_vector_reads_a_column_bit_exactly(bits, chunk):
    rows, cols = 48, 1024
    c, desc = _compressed(rows, cols, bits, chunk, 7100 + bits)
    w_hat = expected_out(c).reshape(rows, cols)
    for j in (0, 1, 255, 256, 777, cols - 1):
        x = torch.zeros(cols, dtype=torch.float16)
        x[j] = 1.0
        (y,) = E.entro_decode_dequant_gemv([desc], [x.cuda()], [(rows, cols)])
        torch.cuda.synchronize()
        got = y.cpu().numpy().view(np.uint16)
        want = w_hat[:, j].copy()
        want[want == 0x8000] = 0            # -0 + 0 = +0
        assert np.array_equal(got, want), j
    assert_status_ok()


@pytest.mark.parametrize("bits,chunk,rows,cols,batch", [(4, 8192, 64, 512, 2), (8, 4096, 64, 512, 3), (4, 8192, 3, 1280, 4),
                                                        (8, 4096, 37, 768, 5), (4, 8192, 33, 4096, 8), (4, 1024, 16, 256, 7),
                                                        (8, 4096, 9, 14336, 2), (4, 8192, 40, 2048, 1)])
def test_fused_gemv_small_batch(bits, chunk, rows, cols, batch):
    """Every token of a batch is an independent product with the same weights: each row of
    the [batch, rows] result is checked against the oracle's product for that token."""
    c, desc = _compressed(rows, cols, bits, chunk, 7500 + rows + cols + batch)
    x = torch.stack([workloads.make_vector(cols, 300 + 17 * b) for b in range(batch)]).cuda()
    (y,) = E.entro_decode_dequant_gemv([desc], [x], [(rows, cols)])
    torch.cuda.synchronize()
    assert_status_ok()
    assert tuple(y.shape) == (batch, rows)
    y_np, x_np = y.cpu().numpy().view(np.uint16), x.cpu().numpy().view(np.uint16)
    for b in range(batch):
        _check(y_np[b], expected_out(c), rows, cols, x_np[b])


def test_batch_of_unit_vectors_reads_columns_bit_exactly():
    rows, cols, batch = 48, 1024, 6
    c, desc = _compressed(rows, cols, 4, 8192, 7600)
    w_hat = expected_out(c).reshape(rows, cols)
    picks = [0, 255, 256, 511, 777, cols - 1]
    x = torch.zeros(batch, cols, dtype=torch.float16)
    for b, j in enumerate(picks):
        x[b, j] = 1.0
    (y,) = E.entro_decode_dequant_gemv([desc], [x.cuda()], [(rows, cols)])
    torch.cuda.synchronize()
    got = y.cpu().numpy().view(np.uint16)
    for b, j in enumerate(picks):
        want = w_hat[:, j].copy()
        want[want == 0x8000] = 0            # -0 + 0 = +0
        assert np.array_equal(got[b], want), (b, j)
    assert_status_ok()


def test_one_call_with_different_batches_per_tensor():
    shapes, batches = [(32, 512), (8, 2048), (24, 256)], [3, 1, 8]
    cs, descs, xs = [], [], []
    for k, ((rows, cols), batch) in enumerate(zip(shapes, batches)):
        c, desc = _compressed(rows, cols, 4 if k != 1 else 8, 8192 if k != 1 else 4096, 7700 + k)
        cs.append(c)
        descs.append(desc)
        x = torch.stack([workloads.make_vector(cols, 900 + 10 * k + b) for b in range(batch)]).cuda()
        xs.append(x if batch > 1 else x[0].contiguous())
    ys = E.entro_decode_dequant_gemv(descs, xs, shapes)
    torch.cuda.synchronize()
    assert_status_ok()
    for c, (rows, cols), batch, x, y in zip(cs, shapes, batches, xs, ys):
        y_np = y.cpu().numpy().view(np.uint16).reshape(batch, rows)
        x_np = x.cpu().numpy().view(np.uint16).reshape(batch, cols)
        for b in range(batch):
            _check(y_np[b], expected_out(c), rows, cols, x_np[b])


def test_mistral_shaped_layer_fused_and_unfused():
    """The seven projections of one mistral-shaped layer (4-bit symbols, 8192-symbol chunks)
    in ONE fused call, against the oracle; and the plain fp16 GEMV on the decoded weights."""
    wl = workloads.mistral_layer_stack(max_layers=1)
    descs, xs, shapes, refs, keep = [], [], [], [], []
    for k, spec in enumerate(wl.tensors):
        w = workloads.make_tensor(spec, "cuda").view(-1).cpu().numpy()
        c = oracle.compress(w, wl.bits, wl.chunk_symbols)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        keep += [s, ix]
        descs.append(E.make_desc_no_out(s, ix, spec.numel, wl.chunk_symbols, codebook_from_oracle(c), c.qp.scale,
                                        c.qp.zero_point))
        xs.append(workloads.make_vector(spec.cols, 100 + k).cuda())
        shapes.append((spec.rows, spec.cols))
        refs.append(expected_out(c))
    ys = E.entro_decode_dequant_gemv(descs, xs, shapes)
    torch.cuda.synchronize()
    assert_status_ok()
    for spec, y, x, ref in zip(wl.tensors, ys, xs, refs):
        _check(y.cpu().numpy().view(np.uint16), ref, spec.rows, spec.cols, x.cpu().numpy().view(np.uint16))
        w_dev = torch.from_numpy(ref.view(np.float16).reshape(spec.rows, spec.cols)).cuda()
        y2 = E.entro_gemv_fp16(w_dev, x)
        torch.cuda.synchronize()
        _check(y2.cpu().numpy().view(np.uint16), ref, spec.rows, spec.cols, x.cpu().numpy().view(np.uint16))


def test_gemv_argument_errors():
    c, desc = _compressed(8, 512, 4, 8192, 7300)
    x = torch.zeros(512, dtype=torch.float16, device="cuda")
    with pytest.raises(E.EntroError) as e:
        E.entro_decode_dequant_gemv([desc], [x], [(16, 512)])          # rows * cols != n
    assert e.value.status == E.ERR_INVALID_ARG
    c2, desc2 = _compressed(8, 384, 4, 8192, 7301)
    with pytest.raises(E.EntroError) as e:
        E.entro_decode_dequant_gemv([desc2], [x[:384].contiguous()], [(8, 384)])   # cols not a multiple of 256
    assert e.value.status == E.ERR_UNSUPPORTED
    x9 = torch.zeros(E.GEMV_MAX_BATCH + 1, 512, dtype=torch.float16, device="cuda")
    with pytest.raises(E.EntroError) as e:
        E.entro_decode_dequant_gemv([desc], [x9], [(8, 512)])          # more tokens than the maximum
    assert e.value.status == E.ERR_INVALID_ARG
    c3, desc3 = _compressed(2, 8192, 4, 8192, 7302)
    x5 = torch.zeros(5, 8192, dtype=torch.float16, device="cuda")
    with pytest.raises(E.EntroError) as e:
        E.entro_decode_dequant_gemv([desc3], [x5], [(2, 8192)])        # batch * cols above what shared memory stages
    assert e.value.status == E.ERR_UNSUPPORTED

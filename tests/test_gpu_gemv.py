"""Fused decode + dequantise + matrix-vector product (one token or a small batch) against the oracle.

The weights inside the product are the bit-exact fp16 values of the decode path (checked
elsewhere); the product itself is summed in fp32 in an order that differs from the oracle's
fp64 loop, so for general x it has a tolerance, derived from the kernel's summation:

  a lane adds the products of its columns into one fp32 accumulator by fused multiply-adds
  (the product of two fp16 values is exact in fp32, so each step rounds once): cols / 32 steps
  when the whole row lies in one chunk, fewer per warp when it spans several; the 32 lanes
  are then added up in 5 shuffle levels; every chunk that holds a part of the row adds its
  partial sum to the row's accumulator with one atomic addition (at most cols / chunk + 2 of
  them).  A term therefore passes through at most  depth = cols / 32 + 5 + cols / chunk + 2
  roundings of relative size 2^-24, and  |sum_fp32 - sum| <= depth * 2^-24 * sum|w x|  to first
  order; the result is rounded once to fp16 (relative 2^-11, or half the subnormal step 2^-25):

      |y - y64| <= 2^-11 |y64| + depth * 2^-24 * sum|w x| + 2^-25          (x 1.01 for the second order)

  At cols = 14336 and 8192-symbol chunks depth is 457, so the sum's share of the bound is
  0.39 of one average product |w x| (sum|w x| / cols): a dropped or doubled product is seen.
  Tensors whose last chunk is ragged, and chunk sizes that are no multiple of 256, decode that
  part symbol by symbol and add every group of 8 products atomically: depth 8 + cols / 8 + 2.

Where x is chosen so that every partial sum is exact in fp32 whatever the order (few
non-zeros, each a power of two: all terms are multiples of one quantum and sum|terms| stays
below 2^24 quanta, asserted in the test), the result is unique and is compared bit for bit
with the oracle's fp64 sum rounded once to fp16.  With x a unit vector the product reduces
to reading a column."""
import functools

import numpy as np
import pytest
import torch

import oracle
import paper_2505_02380_b200 as E
import workloads
from helpers import assert_status_ok, codebook_from_oracle, expected_out, to_dev_index, to_dev_stream

pytestmark = pytest.mark.gpu


@pytest.fixture(params=["call", "plan"])
def gemv(request):
    """The fused products two ways: the one-shot call, and a plan prepared once and run twice
    (first on other vectors, then, with x refreshed in place, on the ones the test gave: the
    second run must not see anything the first one left in the plan's sums)."""
    if request.param == "call":
        return E.entro_decode_dequant_gemv

    def via_plan(descs, xs, shapes):
        xs = list(xs)
        first = [torch.roll(x, 1, dims=-1) * 0.5 for x in xs]
        bufs = [f.clone() for f in first]
        plan, ys = E.entro_gemv_prepare(descs, bufs, shapes)
        E.entro_gemv_run(plan)
        for b, x in zip(bufs, xs):
            b.copy_(x)
        E.entro_gemv_run(plan)
        torch.cuda.synchronize()
        E.entro_gemv_release(plan)
        return ys
    return via_plan


def _f16(bits_u16):
    return bits_u16.view(np.float16).astype(np.float64)


def _compressed(rows, cols, bits, chunk, seed, sigma=0.02):
    w = workloads.make_values(rows * cols, sigma, seed).numpy()
    c = oracle.compress(w, bits, chunk)
    s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
    desc = E.make_desc_no_out(s, ix, rows * cols, chunk, codebook_from_oracle(c), c.qp.scale, c.qp.zero_point)
    desc._keep = (s, ix)          # the descriptor holds raw pointers: keep the device buffers alive with it
    return c, desc


def _depth(cols, chunk, n):
    """Most roundings a product passes through on its way into y (see the module's docstring)."""
    staged = cols // 32 + 5 + cols // chunk + 2
    if n % chunk == 0 and chunk % 256 == 0:
        return staged
    return max(staged, 8 + cols // 8 + 2)


def _check(y_gpu_u16, w_hat_u16, rows, cols, x_u16, chunk):
    y64, asum = oracle.gemv_f64(w_hat_u16, rows, cols, x_u16)
    got = _f16(y_gpu_u16)
    depth = _depth(cols, chunk, rows * cols)
    bound = 1.01 * (2.0 ** -11 * np.abs(y64) + depth * 2.0 ** -24 * asum + 2.0 ** -25)
    bad = np.abs(got - y64) > bound
    assert not bad.any(), (int(bad.sum()), float(np.abs(got - y64).max()))


def _exact_x(cols, chunk, seed):
    """A vector whose product with any fp16 row sums exactly in fp32 in every order: a few
    non-zeros, each +-2^k with k in {-1, 0, 1}, at the columns where the kernel's bookkeeping
    changes: the row's first and last column, the edges of a 256-column step, and every column
    that is the last of a chunk or the first of the next one in some row of a matrix this wide."""
    picks = {0, 1, 255, 256, cols - 257, cols - 256, cols - 1}
    r = 0
    while True:                                        # chunk borders as columns: (k * chunk - r * cols) for the rows r
        first = (-r * cols) % chunk                    # of one period of the pattern
        picks.update(j for b in range(first, cols + 1, chunk) for j in (b - 1, b) if 0 <= j < cols)
        r += 1
        if (r * cols) % chunk == 0 or r >= 64:
            break
    picks = sorted(picks)
    rng = np.random.default_rng(seed)
    x = np.zeros(cols, dtype=np.float16)
    x[picks] = rng.choice(np.array([0.5, 1.0, 2.0, -0.5, -1.0, -2.0], dtype=np.float16), size=len(picks))
    return x


def _check_exact(y_gpu_u16, w_hat_u16, rows, cols, x_f16):
    """x from _exact_x: every partial sum is exact, so y is the exact sum rounded once."""
    x_u16 = x_f16.view(np.uint16)
    y64, asum = oracle.gemv_f64(w_hat_u16, rows, cols, x_u16)
    # sufficient for exactness in any order: all terms are multiples of a quantum u, and
    # sum|terms| < 2^24 u.  u: the smallest power of two that any term of the row may have
    # as its lowest bit = (smallest ulp among the row's weights that meet a non-zero of x) / 2
    cols_used = np.flatnonzero(x_f16)
    w = w_hat_u16.reshape(rows, cols)[:, cols_used].view(np.float16).astype(np.float64)
    mant, exp = np.frexp(np.abs(w))                    # |w| = mant * 2^exp, mant in [0.5, 1)
    ulp = np.where(w != 0, np.maximum(np.ldexp(1.0, exp - 11), 2.0 ** -24), np.inf)
    u = ulp.min(axis=1) / 2.0                          # |x| >= 1/2
    assert np.all(asum < 2.0 ** 24 * u), "the chosen x does not make the fp32 sums exact"
    assert np.all(y64.astype(np.float32).astype(np.float64) == y64)
    want = oracle.f32_to_f16_array(y64.astype(np.float32))
    assert np.array_equal(y_gpu_u16, want), int((y_gpu_u16 != want).sum())


@pytest.mark.parametrize("bits,chunk,rows,cols", [(4, 8192, 64, 512), (8, 4096, 64, 512), (4, 8192, 3, 1280),
                                                  (8, 4096, 37, 768), (4, 8192, 33, 4096), (4, 1024, 16, 256)])
def test_fused_gemv_small(gemv, bits, chunk, rows, cols):
    c, desc = _compressed(rows, cols, bits, chunk, 7000 + rows + cols)
    x = workloads.make_vector(cols, 11).cuda()
    (y,) = gemv([desc], [x], [(rows, cols)])
    torch.cuda.synchronize()
    assert_status_ok()
    _check(y.cpu().numpy().view(np.uint16), expected_out(c), rows, cols, x.cpu().numpy().view(np.uint16), chunk)


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
def test_fused_gemv_small_batch(gemv, bits, chunk, rows, cols, batch):
    """Every token of a batch is an independent product with the same weights: each row of
    the [batch, rows] result is checked against the oracle's product for that token."""
    c, desc = _compressed(rows, cols, bits, chunk, 7500 + rows + cols + batch)
    x = torch.stack([workloads.make_vector(cols, 300 + 17 * b) for b in range(batch)]).cuda()
    (y,) = gemv([desc], [x], [(rows, cols)])
    torch.cuda.synchronize()
    assert_status_ok()
    assert tuple(y.shape) == (batch, rows)
    y_np, x_np = y.cpu().numpy().view(np.uint16), x.cpu().numpy().view(np.uint16)
    for b in range(batch):
        _check(y_np[b], expected_out(c), rows, cols, x_np[b], chunk)


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


def test_one_call_with_different_batches_per_tensor(gemv):
    shapes, batches = [(32, 512), (8, 2048), (24, 256)], [3, 1, 8]
    cs, descs, xs = [], [], []
    for k, ((rows, cols), batch) in enumerate(zip(shapes, batches)):
        c, desc = _compressed(rows, cols, 4 if k != 1 else 8, 8192 if k != 1 else 4096, 7700 + k)
        cs.append(c)
        descs.append(desc)
        x = torch.stack([workloads.make_vector(cols, 900 + 10 * k + b) for b in range(batch)]).cuda()
        xs.append(x if batch > 1 else x[0].contiguous())
    ys = gemv(descs, xs, shapes)
    torch.cuda.synchronize()
    assert_status_ok()
    for c, (rows, cols), batch, x, y in zip(cs, shapes, batches, xs, ys):
        y_np = y.cpu().numpy().view(np.uint16).reshape(batch, rows)
        x_np = x.cpu().numpy().view(np.uint16).reshape(batch, cols)
        for b in range(batch):
            _check(y_np[b], expected_out(c), rows, cols, x_np[b], 4096 if c.qp.bits == 8 else 8192)


@functools.lru_cache(maxsize=1)
def _mistral_layer():
    """The seven projections of one mistral-shaped layer, compressed by the oracle (once for
    the tests below) and put on the device."""
    wl = workloads.mistral_layer_stack(max_layers=1)
    descs, shapes, refs, keep = [], [], [], []
    for spec in wl.tensors:
        w = workloads.make_tensor(spec, "cuda").view(-1).cpu().numpy()
        c = oracle.compress(w, wl.bits, wl.chunk_symbols)
        s, ix = to_dev_stream(c.enc.stream), to_dev_index(c.enc)
        keep += [s, ix]
        descs.append(E.make_desc_no_out(s, ix, spec.numel, wl.chunk_symbols, codebook_from_oracle(c), c.qp.scale,
                                        c.qp.zero_point))
        shapes.append((spec.rows, spec.cols))
        refs.append(expected_out(c))
    return wl, descs, shapes, refs, keep


def test_mistral_shaped_layer_fused_and_unfused(gemv):
    """The seven projections of one mistral-shaped layer (4-bit symbols, 8192-symbol chunks)
    in ONE fused call, against the oracle; and the plain fp16 GEMV on the decoded weights."""
    wl, descs, shapes, refs, _ = _mistral_layer()
    xs = [workloads.make_vector(cols, 100 + k).cuda() for k, (rows, cols) in enumerate(shapes)]
    ys = gemv(descs, xs, shapes)
    torch.cuda.synchronize()
    assert_status_ok()
    for (rows, cols), y, x, ref in zip(shapes, ys, xs, refs):
        _check(y.cpu().numpy().view(np.uint16), ref, rows, cols, x.cpu().numpy().view(np.uint16), wl.chunk_symbols)
        w_dev = torch.from_numpy(ref.view(np.float16).reshape(rows, cols)).cuda()
        y2 = E.entro_gemv_fp16(w_dev, x)
        torch.cuda.synchronize()
        _check(y2.cpu().numpy().view(np.uint16), ref, rows, cols, x.cpu().numpy().view(np.uint16), wl.chunk_symbols)


def test_mistral_shaped_layer_exact_sums_bit_for_bit(gemv):
    """Config 5 at its own shapes: the seven projections of a mistral-shaped layer (4-bit symbols,
    8192-symbol chunks; 4096 x 14336 down_proj rows span two or three chunks and are combined
    with atomics), one token and batches of 2, 4 and 8, with x chosen so that fp32 sums are exact
    in any order: y must equal the oracle's fp64 sum rounded once to fp16, bit for bit."""
    wl, descs, shapes, refs, _ = _mistral_layer()
    for batch in (1, 2, 4, 8):
        pick = [k for k, (r, cc) in enumerate(shapes) if cc * batch <= 32768]      # x of a batch must fit its staging
        if batch > 2:
            pick = pick[:2] + pick[4:5]                                          # q, k and gate: the oracle's loop is slow
        xs_np = [np.stack([_exact_x(shapes[k][1], wl.chunk_symbols, 50 * batch + 7 * k + b) for b in range(batch)])
                 for k in pick]
        xs = [torch.from_numpy(x if batch > 1 else x[0]).cuda() for x in xs_np]
        ys = gemv([descs[k] for k in pick], xs, [shapes[k] for k in pick])
        torch.cuda.synchronize()
        assert_status_ok()
        for k, x_np, y in zip(pick, xs_np, ys):
            y_np = y.cpu().numpy().view(np.uint16).reshape(batch, shapes[k][0])
            for b in range(batch):
                _check_exact(y_np[b], refs[k], shapes[k][0], shapes[k][1], x_np[b])


@pytest.mark.parametrize("bits,chunk,rows,cols,batch", [(8, 4096, 96, 14336, 1), (8, 4096, 96, 14336, 2), (8, 4096, 128, 4096, 4),
                                                        (4, 8192, 40, 2048, 8), (8, 1024, 33, 1280, 3), (4, 8192, 7, 14336, 1)])
def test_exact_sums_bit_for_bit_other_shapes(gemv, bits, chunk, rows, cols, batch):
    """The same at 8-bit symbols with 4096-symbol chunks (a 14336-column row spans four or five
    chunks), small chunks, and a tensor whose last chunk is ragged."""
    c, desc = _compressed(rows, cols, bits, chunk, 7800 + rows + cols)
    x_np = np.stack([_exact_x(cols, chunk, 900 + b) for b in range(batch)])
    x = torch.from_numpy(x_np if batch > 1 else x_np[0]).cuda()
    (y,) = gemv([desc], [x], [(rows, cols)])
    torch.cuda.synchronize()
    assert_status_ok()
    y_np = y.cpu().numpy().view(np.uint16).reshape(batch, rows)
    for b in range(batch):
        _check_exact(y_np[b], expected_out(c), rows, cols, x_np[b])


def test_plan_argument_errors_and_release():
    c, desc = _compressed(8, 512, 4, 8192, 7310)
    x = torch.zeros(512, dtype=torch.float16, device="cuda")
    with pytest.raises(E.EntroError) as e:
        E.entro_gemv_prepare([desc], [x], [(16, 512)])                 # rows * cols != n
    assert e.value.status == E.ERR_INVALID_ARG
    L = E.lib()
    assert L.entro_gemv_run(None, None) == E.ERR_INVALID_ARG
    assert L.entro_gemv_release(None) == E.OK
    plan, (y,) = E.entro_gemv_prepare([desc], [x], [(8, 512)])
    E.entro_gemv_run(plan)
    torch.cuda.synchronize()
    assert_status_ok()
    assert not y.cpu().numpy().any()                                    # W . 0 = 0
    E.entro_gemv_release(plan)
    E.entro_gemv_release(plan)                                          # a released handle is inert in the binding


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

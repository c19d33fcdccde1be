"""Pins for the oracle's floating-point parts: fp16 conversions, the quantiser (Eq. 1)
and the dequantiser.  Nothing here re-types the oracle's formulas: the checks are NumPy's
own float16, closed forms on dyadic grids, and error bounds."""
import numpy as np
import pytest

import oracle
import workloads


# ----------------------------------------------------------------------------- fp16 conversions

def test_f16_to_f32_all_patterns_match_numpy():
    h = np.arange(65536, dtype=np.uint16)
    got = oracle.f16_to_f32_array(h)
    ref = h.view(np.float16).astype(np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_f32_to_f16_roundtrip_all_patterns():
    h = np.arange(65536, dtype=np.uint16)
    f = h.view(np.float16).astype(np.float32)
    back = oracle.f32_to_f16_array(f)
    nan = np.isnan(f)
    assert np.array_equal(back[~nan], h[~nan])
    assert np.all((back[nan] & 0x7c00) == 0x7c00) and np.all((back[nan] & 0x3ff) != 0)


def test_f32_to_f16_random_and_special_match_numpy():
    rng = np.random.default_rng(7)
    parts = [
        rng.standard_normal(2_000_000).astype(np.float32),
        (rng.standard_normal(1_000_000) * 1e-6).astype(np.float32),       # subnormal range
        (rng.standard_normal(1_000_000) * 3e4).astype(np.float32),        # near overflow
        rng.integers(0, 2**32, size=4_000_000, dtype=np.uint64).astype(np.uint32).view(np.float32),
    ]
    # exact ties between neighbouring fp16 values (all of them), both signs
    h = np.arange(0, 0x7c00, dtype=np.uint16)
    a = h.view(np.float16).astype(np.float64)
    b = (h + 1).astype(np.uint16).view(np.float16).astype(np.float64)
    b[-1] = 65536.0
    mid = ((a + b) / 2).astype(np.float32)        # exact in fp32
    parts += [mid, -mid, np.nextafter(mid, np.float32(0)), np.nextafter(mid, np.float32(1e9))]
    parts += [np.array([0.0, -0.0, 65504.0, 65519.99, 65520.0, 65536.0, 1e10, -1e10, np.inf, -np.inf,
                        2.0**-24, 2.0**-25, 2.0**-25 * 1.0001, 2.0**-26, 2.0**-14, 2.0**-14 - 2.0**-25],
                       dtype=np.float32)]
    f = np.concatenate(parts)
    f = f[~np.isnan(f)]
    with np.errstate(over="ignore"):
        ref = f.astype(np.float16).view(np.uint16)
    got = oracle.f32_to_f16_array(f)
    bad = np.nonzero(got != ref)[0]
    assert bad.size == 0, (f[bad[:5]], got[bad[:5]], ref[bad[:5]])


# ----------------------------------------------------------------------------- dequantiser

@pytest.mark.parametrize("bits", [4, 8])
def test_dequant_matches_numpy_float32_product(bits):
    rng = np.random.default_rng(bits)
    q = np.arange(1 << bits, dtype=np.uint8)
    for _ in range(200):
        s = np.float32(10.0 ** rng.uniform(-6, 1))
        z = int(rng.integers(0, 1 << bits))
        ref = (s * (q.astype(np.int32) - z).astype(np.float32)).astype(np.float16).view(np.uint16)
        assert np.array_equal(oracle.dequant(q, float(s), z), ref)


def test_dequant_dyadic_closed_form():
    # s = 2^-8, z = 128: w_hat = (q - 128) / 256 exactly, every value representable in fp16
    q = np.arange(256, dtype=np.uint8)
    out = oracle.dequant(q, 2.0 ** -8, 128).view(np.float16).astype(np.float64)
    assert np.array_equal(out, (q.astype(np.float64) - 128) / 256)


# ----------------------------------------------------------------------------- quantiser

def _f16(x):
    return np.asarray(x, dtype=np.float64).astype(np.float16)


def test_quantise_dyadic_grid_is_exact_asymmetric():
    # lo = -128 * 2^-8, hi = 127 * 2^-8: s = 2^-8 exactly, z = 128, q = k + 128, w_hat = w
    k = np.arange(-128, 128)
    w = _f16(k / 256.0)
    rng = np.random.default_rng(0)
    w = np.concatenate([w, rng.choice(w, 5000)])
    q, qp = oracle.quantize_tensor(w, 8)
    assert qp.mode == oracle.MODE_ASYMMETRIC and qp.scale == 2.0 ** -8 and qp.zero_point == 128
    assert np.array_equal(q.astype(np.int64), np.rint(w.astype(np.float64) * 256).astype(np.int64) + 128)
    assert np.array_equal(oracle.dequant(q, qp.scale, qp.zero_point), w.view(np.uint16))


def test_quantise_dyadic_grid_is_exact_unsigned():
    # all weights >= 0, hi = 15 * 2^-4: unsigned branch, s = 2^-4, z = 0
    w = _f16(np.arange(16) / 16.0)
    q, qp = oracle.quantize_tensor(np.tile(w, 7), 4)
    assert qp.mode == oracle.MODE_UNSIGNED and qp.zero_point == 0 and qp.scale == 2.0 ** -4
    assert np.array_equal(q, np.tile(np.arange(16, dtype=np.uint8), 7))


def test_mode_rule_and_forced_modes():
    pos = _f16([0.0, 0.5, 1.0, 2.0])
    neg = _f16([-0.25, 0.5, 1.0])
    assert oracle.quant_params(pos, 8).mode == oracle.MODE_UNSIGNED
    assert oracle.quant_params(neg, 8).mode == oracle.MODE_ASYMMETRIC
    assert oracle.quant_params(pos, 8, oracle.MODE_ASYMMETRIC).mode == oracle.MODE_ASYMMETRIC
    qp = oracle.quant_params(_f16([-0.0, 1.0]), 8)       # -0.0 is not negative
    assert qp.mode == oracle.MODE_UNSIGNED


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_quantiser_error_bound_and_end_points(bits, seed):
    w = workloads.make_values(200_000, 0.02, seed).numpy()
    q, qp = oracle.quantize_tensor(w, bits)
    qmax = (1 << bits) - 1
    s, z = np.float64(qp.scale), qp.zero_point
    assert qp.lo == float(w.min()) and qp.hi == float(w.max())
    # s is the fp32 quotient of the range by qmax
    assert qp.scale == float((np.float32(qp.hi) - np.float32(qp.lo)) / np.float32(qmax))
    w64 = w.astype(np.float64)
    unclamped = np.rint(w64 / s) + z          # fp64 stand-in; differs from fp32 only on near-ties
    inside = (unclamped >= 0) & (unclamped <= qmax)
    err = np.abs(w64 - s * (q.astype(np.float64) - z))
    assert np.all(err[inside] <= s / 2 * (1 + 1e-5))
    assert q[np.argmin(w)] == 0                                  # q(lo) = 0
    assert q[np.argmax(w)] in (qmax - 1, qmax)                   # top end clamps by at most one step
    assert q.max() <= qmax
    # zero maps to the zero-point and back to exactly zero
    w0 = np.concatenate([w, _f16([0.0])])
    q0, qp0 = oracle.quantize_tensor(w0, bits)
    assert q0[-1] == qp0.zero_point
    assert oracle.dequant(q0[-1:], qp0.scale, qp0.zero_point)[0] == 0


@pytest.mark.parametrize("bits", [4, 8])
def test_quantiser_matches_numpy_float32_pipeline(bits):
    """Independent restatement with NumPy float32 ufuncs (true division, rint = ties-to-even)."""
    for seed, kind in [(3, "matrix"), (4, "matrix"), (5, "gain")]:
        w = workloads.make_values(1 << 18, 0.03, seed, kind).numpy()
        q, qp = oracle.quantize_tensor(w, bits)
        w32 = w.astype(np.float32)
        qmax = np.float32((1 << bits) - 1)
        lo, hi = w32.min(), w32.max()
        if lo >= 0:
            s, z = hi / qmax, 0
        else:
            s = (hi - lo) / qmax
            z = int(np.clip(np.rint(-lo / s), 0, qmax))
        assert s.dtype == np.float32
        ref = np.clip(np.rint(w32 / s).astype(np.int64) + z, 0, int(qmax)).astype(np.uint8)
        assert qp.scale == float(s) and qp.zero_point == z
        assert np.array_equal(q, ref)


def test_quantiser_ties_round_to_even():
    # s = 1 (hi = 255, lo = 0 -> unsigned): halves must go to the even neighbour
    w = _f16([0.0, 0.5, 1.5, 2.5, 3.5, 254.5, 255.0])
    q, qp = oracle.quantize_tensor(w, 8)
    assert qp.scale == 1.0 and qp.zero_point == 0
    assert q.tolist() == [0, 0, 2, 2, 4, 254, 255]


def test_quantiser_degenerate_and_nonfinite():
    q, qp = oracle.quantize_tensor(_f16([0.0, 0.0, 0.0]), 8)
    assert qp.scale == 1.0 and qp.zero_point == 0 and q.tolist() == [0, 0, 0]
    q, qp = oracle.quantize_tensor(_f16([-3.0, -3.0]), 8)
    assert qp.scale == 1.0 and qp.zero_point == 3 and q.tolist() == [0, 0]
    assert oracle.dequant(q, qp.scale, qp.zero_point).view(np.float16).tolist() == [-3.0, -3.0]
    q, qp = oracle.quantize_tensor(_f16([2.0, 2.0]), 4)
    assert qp.mode == oracle.MODE_UNSIGNED and q.tolist() == [15, 15]
    for bad in (np.inf, -np.inf, np.nan):
        with pytest.raises(oracle.OracleError) as e:
            oracle.quantize_tensor(_f16([0.1, bad, 0.2]), 8)
        assert e.value.code == 3


def test_gemv_reference_reduces_to_column_read_and_numpy():
    rng = np.random.default_rng(11)
    rows, cols = 37, 256
    w = rng.standard_normal((rows, cols)).astype(np.float16)
    for j in (0, 5, cols - 1):
        x = np.zeros(cols, dtype=np.float16)
        x[j] = 1.0
        y, a = oracle.gemv_f64(w, rows, cols, x)
        assert np.array_equal(y, w[:, j].astype(np.float64))
        assert np.array_equal(a, np.abs(w[:, j].astype(np.float64)))
    x = rng.standard_normal(cols).astype(np.float16)
    y, a = oracle.gemv_f64(w, rows, cols, x)
    ref = w.astype(np.float64) @ x.astype(np.float64)
    assert np.allclose(y, ref, rtol=0, atol=1e-12)
    assert np.allclose(a, np.abs(w.astype(np.float64) * x.astype(np.float64)).sum(1), rtol=1e-14)


# ----------------------------------------------------------------------------- block-based grid (Table 2, "SOTA")

def test_block_quantiser_is_the_tensor_quantiser_on_every_block():
    """Pinned to the per-tensor quantiser (itself pinned above): quantising in blocks is
    quantising each slice as a tensor of its own, the last one shorter; one block as long
    as the tensor is the tensor quantiser."""
    for bits in (4, 8):
        for n, block in ((1000, 32), (64, 32), (33, 32), (5, 32), (4096, 128), (777, 1000)):
            w = workloads.make_values(n, 0.03, 31 * n + bits).numpy()
            q, scales, zps = oracle.quantize_blocks(w, bits, block)
            for b, first in enumerate(range(0, n, block)):
                qs, qp = oracle.quantize_tensor(w[first:first + block], bits)
                assert np.array_equal(q[first:first + block], qs), (bits, n, block, b)
                assert scales[b] == np.float32(qp.scale) and zps[b] == qp.zero_point
            assert len(scales) == (n + block - 1) // block


def test_block_quantiser_hand_example():
    """Two blocks of four worked by hand at 4 bits.  (-1, 0, 1, 3): s = 4/15, z = rne(3.75) = 4,
    codes rne(w/s) + 4 = 0, 4, 8, 15.  (0, 1, 2, 5): no negative value, so unsigned, s = 1/3,
    codes rne(3 w) = 0, 3, 6, 15."""
    w = np.array([-1, 0, 1, 3, 0, 1, 2, 5], dtype=np.float16)
    q, scales, zps = oracle.quantize_blocks(w, 4, 4)
    assert q.tolist() == [0, 4, 8, 15, 0, 3, 6, 15]
    assert zps.tolist() == [4, 0]
    assert scales.tolist() == [np.float32(4) / np.float32(15), np.float32(5) / np.float32(15)]


def test_block_grid_flattens_the_histogram():
    """The paper's reason for quantising whole tensors (Section 3): a grid per block of 32
    spreads the codes over the levels, one grid per tensor leaves them peaked.  On heavy-tailed
    synthetic weights the block grid's symbol entropy must be the higher one, by a wide margin."""
    w = workloads.make_values(1 << 18, 0.02, 99).numpy()

    def entropy(q, nsym):
        p = np.bincount(q, minlength=nsym) / q.size
        p = p[p > 0]
        return float(-(p * np.log2(p)).sum())

    for bits in (4, 8):
        qt, _ = oracle.quantize_tensor(w, bits)
        qb, _, _ = oracle.quantize_blocks(w, bits, 32)
        assert entropy(qb, 1 << bits) > entropy(qt, 1 << bits) + 1.0

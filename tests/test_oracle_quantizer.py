"""Pins for the oracle's batch-norm fold and weight quantizer (CPU only)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import aiq_oracle as O
from exact32 import (f32_to_fraction, round_to_f32, sqrt_f32, quantize_row_exact,
                     half_rne_exact)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _hand_rows():
    rows = []
    with open(os.path.join(GOLDEN, "quantizer_hand_rows.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, vals, codes, packed = [p.strip() for p in line.split("|")]
            rows.append((int(bits), [float(v) for v in vals.split()],
                         [int(c) for c in codes.split()],
                         [int(b, 16) for b in packed.split()]))
    return rows


@pytest.mark.parametrize("bits,vals,codes,packed", _hand_rows())
def test_hand_rows(bits, vals, codes, packed):
    W = np.asarray([vals], dtype=np.float32)
    v, s = O.quantize_rows(W, bits)
    assert v.dtype == np.int8
    assert v[0].tolist() == codes
    assert s[0] == np.float32(1.0)
    p = O.pack_rows(v, bits)
    assert p.shape == (1, O.packed_row_bytes(len(vals), bits))
    assert p[0, :len(packed)].tolist() == packed
    assert not p[0, len(packed):].any()            # padding is zero
    assert O.unpack_rows(p, len(vals), bits)[0].tolist() == codes


@pytest.mark.parametrize("bits", [4, 8])
def test_codes_and_scales_match_exact_rational_arithmetic(bits):
    """s = fl(amax/qmax), code = rne(fl(w/s)) evaluated with exact rationals and explicit
    binary32 rounding; separates true division from multiply-by-reciprocal and catches a
    wrong tie rule."""
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((24, 19)) * 0.3).astype(np.float32)
    W[3] *= np.float32(1e-3)
    W[5, :] = 0.0
    W[6, 4] = 0.0
    # a deliberate near-tie: -0.25 / fl(0.5/127) is within an ulp of -63.5
    W[7, :] = 0.0
    W[7, 0], W[7, 1] = 0.5, -0.25
    v, s = O.quantize_rows(W, bits)
    for n in range(W.shape[0]):
        codes, sc = quantize_row_exact(W[n], bits)
        assert f32_to_fraction(s[n]) == sc, n
        assert v[n].tolist() == codes, n


def test_division_not_reciprocal_multiply():
    """The pinned rule is w / s.  Build rows full of near-ties (w close to (k + 1/2) s),
    where w * fl(1/s) lands on the other side often enough, and check the oracle follows
    the exactly rounded division."""
    rng = np.random.default_rng(11)
    rows = []
    for _ in range(60):
        amax = np.float32(rng.uniform(0.1, 3.0))
        s = amax / np.float32(127.0)
        k = rng.integers(-126, 126, 63).astype(np.float32) + np.float32(0.5)
        w = (k * s).astype(np.float32)
        w = np.nextafter(w, np.float32(0.0)) if rng.random() < 0.5 else w
        rows.append(np.concatenate([[amax], w]).astype(np.float32))
    W = np.stack(rows)
    v, s = O.quantize_rows(W, 8)
    recip = np.rint(W * (np.float32(1.0) / s)[:, None]).astype(np.int64)
    differ = np.argwhere(recip != v)
    assert len(differ) > 0, "sample does not separate the two rules"
    checked = set()
    for n, k in differ[:40]:
        if n not in checked:
            codes, sc = quantize_row_exact(W[n], 8)
            assert v[n].tolist() == codes
            assert f32_to_fraction(s[n]) == sc
            checked.add(n)


@pytest.mark.parametrize("bits", [4, 8])
def test_power_of_two_scale_invariance(bits):
    rng = np.random.default_rng(3)
    W = rng.standard_normal((16, 50)).astype(np.float32)
    v, s = O.quantize_rows(W, bits)
    for sh in (-9, 5):
        v2, s2 = O.quantize_rows(W * np.float32(2.0 ** sh), bits)
        assert np.array_equal(v, v2)
        assert np.array_equal(s2, s * np.float32(2.0 ** sh))


@pytest.mark.parametrize("bits", [4, 8])
def test_code_range_and_extremum(bits):
    rng = np.random.default_rng(5)
    W = rng.standard_normal((64, 100)).astype(np.float32)
    v, s = O.quantize_rows(W, bits)
    qmax = 2 ** (bits - 1) - 1
    assert v.min() >= -(2 ** (bits - 1)) and v.max() <= qmax
    k = np.argmax(np.abs(W), axis=1)
    assert np.all(np.abs(v[np.arange(64), k].astype(int)) == qmax)
    assert np.all(np.sign(v[np.arange(64), k]) == np.sign(W[np.arange(64), k]))


def test_reconstruction_error_bounds():
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((32, 200)) * 0.05).astype(np.float32)
    for bits in (4, 8):
        v, s = O.quantize_rows(W, bits)
        err = np.abs(W.astype(np.float64) - O.dequantize_rows(v, s, bits).astype(np.float64))
        bound = 0.5 * s[:, None].astype(np.float64) + 4 * np.spacing(np.abs(W)).astype(np.float64)
        assert np.all(err <= bound)
    v, s = O.quantize_rows(W, 16)
    big = np.abs(W) > 2.0 ** -14
    rel = np.abs(W.astype(np.float64) - v.astype(np.float64))[big] / np.abs(W.astype(np.float64))[big]
    assert rel.max() <= 2.0 ** -11
    v, s = O.quantize_rows(W, 32)
    assert np.array_equal(v.view(np.uint32), W.view(np.uint32))
    assert np.all(s == 1.0)


def test_half_is_round_to_nearest_even():
    vals = np.asarray([[1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 0.1, -0.3, 6.1e-5, 3.0e-6,
                        1.0 + 2.0 ** -11 + 2.0 ** -20, 1000.123]], dtype=np.float32)
    v, s = O.quantize_rows(vals, 16)
    for a, h in zip(vals[0], v[0]):
        assert Fraction(float(h)) == half_rne_exact(a)
    assert Fraction(float(v[0, 0])) == 1                       # tie -> even mantissa
    assert Fraction(float(v[0, 1])) == 1 + Fraction(4, 2 ** 11)


def test_zero_row_and_nonfinite_and_bad_bits():
    v, s = O.quantize_rows(np.zeros((2, 5), np.float32), 4)
    assert not v.any() and np.all(s == 1.0)
    bad = np.ones((2, 3), np.float32)
    bad[1, 2] = np.inf
    with pytest.raises(ValueError):
        O.quantize_rows(bad, 8)
    bad[1, 2] = np.nan
    with pytest.raises(ValueError):
        O.quantize_rows(bad, 4)
    with pytest.raises(ValueError):
        O.quantize_rows(np.ones((2, 3), np.float32), 5)


@pytest.mark.parametrize("bits", [4, 8, 16, 32])
@pytest.mark.parametrize("K", [1, 9, 27, 32, 33, 144])
def test_pack_layout(bits, K):
    rng = np.random.default_rng(K)
    W = rng.standard_normal((5, K)).astype(np.float32)
    v, _ = O.quantize_rows(W, bits)
    p = O.pack_rows(v, bits)
    kp = (K + 31) // 32 * 32
    assert p.shape == (5, kp * bits // 8) and p.dtype == np.uint8
    assert p.shape[1] % 16 == 0
    assert np.array_equal(O.unpack_rows(p, K, bits), v)
    # element-by-element statement of the layout
    for n in range(5):
        for k in range(kp):
            if bits == 4:
                nib = (int(p[n, k // 2]) >> (4 * (k % 2))) & 0xF
                val = nib - 16 if nib >= 8 else nib
                assert val == (int(v[n, k]) if k < K else 0)
            else:
                nb = bits // 8
                raw = p[n, k * nb:(k + 1) * nb].tobytes()
                want = v[n, k].tobytes() if k < K else bytes(nb)
                assert raw == want


def test_fold_matches_exact_rational_arithmetic():
    rng = np.random.default_rng(21)
    cout, K = 6, 7
    W = rng.standard_normal((cout, K)).astype(np.float32)
    gamma = rng.uniform(0.5, 1.5, cout).astype(np.float32)
    beta = (rng.standard_normal(cout) * 0.1).astype(np.float32)
    mean = (rng.standard_normal(cout) * 0.1).astype(np.float32)
    var = rng.uniform(0.5, 1.5, cout).astype(np.float32)
    Wf, bf = O.fold_bn(W, gamma, beta, mean, var)
    eps = f32_to_fraction(np.float32(1e-5))
    for n in range(cout):
        g = round_to_f32(f32_to_fraction(gamma[n]) / sqrt_f32(round_to_f32(f32_to_fraction(var[n]) + eps)))
        assert f32_to_fraction(bf[n]) == round_to_f32(
            f32_to_fraction(beta[n]) - round_to_f32(f32_to_fraction(mean[n]) * g))
        for k in range(K):
            assert f32_to_fraction(Wf[n, k]) == round_to_f32(f32_to_fraction(W[n, k]) * g)


def test_fold_identity_case():
    """gamma = sqrt(var + eps) exactly representable -> g = 1, W unchanged, b = beta - mean."""
    W = np.arange(12, dtype=np.float32).reshape(2, 6)
    var = np.asarray([1.0, 4.0], np.float32) - np.float32(1e-5)
    # (var + eps) rounds back to 1.0 and 4.0 here; check, then gamma = 1, 2
    assert np.all(var + np.float32(1e-5) == np.asarray([1.0, 4.0], np.float32))
    Wf, bf = O.fold_bn(W, np.asarray([1.0, 2.0], np.float32), np.asarray([0.5, 0.25], np.float32),
                       np.asarray([0.125, 1.0], np.float32), var)
    assert np.array_equal(Wf, W)
    assert bf.tolist() == [0.375, -0.75]


# ---------------------------------------------------------------- per-tensor-scale variant
def _per_tensor_cases():
    out = []
    with open(os.path.join(GOLDEN, "quantizer_per_tensor_hand.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, rows, scale, codes, row_codes = [p.strip() for p in line.split("|")]
            parse = lambda t, conv: [[conv(v) for v in r.split()] for r in t.split("/")]
            out.append((int(bits), parse(rows, float), float(scale), parse(codes, int), parse(row_codes, int)))
    return out


@pytest.mark.parametrize("bits,rows,scale,codes,row_codes", _per_tensor_cases())
def test_per_tensor_hand_tables(bits, rows, scale, codes, row_codes):
    W = np.asarray(rows, dtype=np.float32)
    v, s = O.quantize_rows(W, bits, per_tensor=True)
    assert v.tolist() == codes
    assert s.tolist() == [scale] * len(rows)                 # the one scale, repeated for every row
    v_row, _ = O.quantize_rows(W, bits)                      # the default granularity differs on these tensors
    assert v_row.tolist() == row_codes


@pytest.mark.parametrize("bits", [4, 8])
def test_per_tensor_matches_exact_rational_arithmetic_and_bounds(bits):
    """The tensor flattened to one long row is the per-channel rule applied once: same exact-rational
    model.  Also: equal to the per-channel result when every row has the same maximum; codes in
    range with the extremum attained somewhere; |w - s*code| <= s/2 (+ rounding of the product)."""
    rng = np.random.default_rng(21)
    W = (rng.standard_normal((9, 13)) * 0.2).astype(np.float32)
    W[4] *= np.float32(0.01)
    v, s = O.quantize_rows(W, bits, per_tensor=True)
    codes, sc = quantize_row_exact(W.reshape(-1), bits)
    assert all(f32_to_fraction(x) == sc for x in s)
    assert v.reshape(-1).tolist() == codes
    qmax = 2 ** (bits - 1) - 1
    assert np.abs(v).max() == qmax and v.min() >= -(qmax + 1) and v.max() <= qmax
    w_hat = O.dequantize_rows(v, s, bits)
    assert np.all(np.abs(W.astype(np.float64) - w_hat.astype(np.float64)) <= float(s[0]) * (0.5 + 1e-6))
    # rows with a common maximum: both granularities agree
    W2 = W.copy()
    W2[:, 0] = np.float32(3.0)
    a, sa = O.quantize_rows(W2, bits, per_tensor=True)
    b, sb = O.quantize_rows(W2, bits)
    assert np.array_equal(a, b) and np.array_equal(sa, sb)
    # 16 / 32 bits do not depend on the granularity
    for wide in (16, 32):
        a, sa = O.quantize_rows(W, wide, per_tensor=True)
        b, sb = O.quantize_rows(W, wide)
        assert np.array_equal(a, b) and np.array_equal(sa, sb)
    # an all-zero tensor keeps scale 1
    z, sz = O.quantize_rows(np.zeros((3, 5), np.float32), bits, per_tensor=True)
    assert not z.any() and sz.tolist() == [1.0, 1.0, 1.0]


def test_ai_does_not_depend_on_the_scale_granularity():
    """AI counts weight bytes by bit-width only (Section 1 (i)); per-tensor and per-channel banks of
    the same scheme have the same analytic intensity, while their accuracies may differ."""
    from aiq_workloads import resnet20, gen_model, gen_images
    arch = resnet20()
    params = gen_model(arch, 1234)
    folded = O.fold_model(arch, params)
    x = gen_images(4, 3, 32, 32, 3)
    bank_c = O.build_weight_bank(folded, (4,))
    bank_t = O.build_weight_bank(folded, (4,), per_tensor=True)
    scheme = [4] * 22
    assert not np.array_equal(O.forward_scheme(arch, bank_c, scheme, x), O.forward_scheme(arch, bank_t, scheme, x))
    assert O.scheme_ai(arch, scheme) == O.scheme_ai(arch, scheme)      # no bank argument at all: bytes follow q only

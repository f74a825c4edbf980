"""CPU pins for oracle/sketch.py: the Philox stream, the Gaussian transform, E[S S^T] = I."""
import os

import numpy as np
import pytest
from scipy import stats

from oracle import sketch as sk


def _kat(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([int(w, 16) for w in line.split()])
    return rows


def test_philox_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for row in rows:
        out = sk.philox4x32_10(*row[:6])
        assert [int(v) for v in out] == row[6:]


def test_philox_vectorised_matches_scalar(golden_dir):
    rows = np.array(_kat(golden_dir), dtype=np.uint64)
    out = sk.philox4x32_10(*(rows[:, k] for k in range(6)))
    for k in range(4):
        assert np.array_equal(out[k], rows[:, 6 + k])


def test_philox_words_are_uniform():
    # one million words: every bit set half of the time, byte histogram flat
    i = np.arange(1 << 18, dtype=np.uint64)
    words = np.concatenate(sk.philox4x32_10(i, 5, 0, 0, 123, 456))
    for b in range(32):
        frac = float(((words >> np.uint64(b)) & np.uint64(1)).mean())
        assert abs(frac - 0.5) < 4 * 0.5 / np.sqrt(words.size)
    hist = np.bincount((words & np.uint64(0xFF)).astype(np.int64), minlength=256)
    chi2 = float(((hist - words.size / 256) ** 2 / (words.size / 256)).sum())
    assert chi2 < stats.chi2.ppf(1 - 1e-6, 255)


def _reference_pair_f64(xa, xb):
    """Box-Muller of the same (u, theta) with double-precision libm."""
    xa = np.asarray(xa, dtype=np.uint64)
    xb = np.asarray(xb, dtype=np.uint64)
    u = ((xa >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23
    frac = ((xb >> np.uint64(6)) & np.uint64(0x7FFFFF)).astype(np.float64) * 2.0 ** -23
    theta = ((xb >> np.uint64(29)).astype(np.float64) + frac) * (np.pi / 4)
    rho = np.sqrt(-2.0 * np.log(u))
    return rho * np.cos(theta), rho * np.sin(theta)


def test_gaussian_pair_close_to_libm_box_muller():
    rng = np.random.default_rng(11)
    xa = rng.integers(0, 1 << 32, size=400_000, dtype=np.uint64)
    xb = rng.integers(0, 1 << 32, size=400_000, dtype=np.uint64)
    # force the corners: smallest / largest u, every octant boundary
    xa[:4] = [0, 0xFFFFFFFF, 0x1FF, 0xFFFFFE00]
    xb[:16] = [o << 29 for o in range(8)] + [(o << 29) | 0x1FFFFFFF for o in range(8)]
    z0, z1 = sk.gaussian_pair(xa, xb)
    assert z0.dtype == np.float32 and z1.dtype == np.float32
    r0, r1 = _reference_pair_f64(xa, xb)
    for z, ref in ((z0, r0), (z1, r1)):
        err = np.abs(z.astype(np.float64) - ref)
        # a few binary32 ulps of the radius (|z| <= 5.8, ulp(4) = 4.8e-7)
        assert err.max() < 2e-6
        assert (err / np.maximum(np.abs(ref), 1.0)).max() < 6e-7
        assert np.median(err / np.maximum(np.abs(ref), 1e-30)) < 1.2e-7


def test_gaussian_pair_extremes_are_finite():
    z0, z1 = sk.gaussian_pair(np.array([0, 0xFFFFFFFF], dtype=np.uint64), np.array([0, 0], dtype=np.uint64))
    # u = 2^-24 gives the largest radius sqrt(48 ln 2) = 5.768; u = 1 - 2^-24 the smallest, 3.45e-4
    assert abs(float(z0[0]) - np.sqrt(48 * np.log(2.0))) < 1e-5
    assert abs(float(z0[1]) - np.sqrt(-2 * np.log1p(-2.0 ** -24))) < 1e-9
    assert float(z1[0]) == 0.0 and float(z1[1]) == 0.0


def test_layout_counter_is_row_and_column_quad():
    seed, kind = 0x1234_5678_9ABC_DEF0, 0
    z = sk.standard_normal_block(seed, 6, 12, kind)
    for i in (0, 5):
        for q in (0, 2):
            x = sk.philox4x32_10(i, q, 0, kind, seed & 0xFFFFFFFF, seed >> 32)
            a0, a1 = _reference_pair_f64(x[0], x[1])
            b0, b1 = _reference_pair_f64(x[2], x[3])
            want = np.array([a0, a1, b0, b1]).ravel()
            assert np.allclose(z[i, 4 * q:4 * q + 4], want, atol=2e-6, rtol=0)


def test_values_depend_only_on_seed_row_column():
    a = sk.standard_normal_block(3, 40, 64)
    assert np.array_equal(a[:, :16], sk.standard_normal_block(3, 40, 16))
    assert np.array_equal(a[7:19], sk.standard_normal_block(3, 12, 64, row0=7))
    assert not np.array_equal(a, sk.standard_normal_block(4, 40, 64))
    assert not np.array_equal(a, sk.standard_normal_block(3 + (1 << 32), 40, 64))  # high key word is used
    assert not np.array_equal(a, sk.standard_normal_block(3, 40, 64, kind=1))


def test_sketch_scale_and_power_of_two_ranks():
    for r in (16, 64, 256):  # 1/sqrt(r) is a power of two: scaling is exact
        z = sk.standard_normal_block(9, 32, r)
        assert np.array_equal(sk.sketch(9, 32, r), z * np.float32(1.0 / np.sqrt(r)))
        assert np.array_equal(sk.sketch(9, 32, r).astype(np.float64) * np.sqrt(r), z.astype(np.float64))
    s = sk.sketch(9, 32, 128)
    assert s.dtype == np.float32
    assert np.array_equal(s, sk.standard_normal_block(9, 32, 128) * np.float32(0.08838834764831845))


def test_moments_and_ks():
    z = sk.standard_normal_block(2024, 4096, 2560).ravel().astype(np.float64)  # ~1.05e7 samples
    n = z.size
    assert abs(z.mean()) < 5 / np.sqrt(n)
    assert abs(z.var() - 1.0) < 5 * np.sqrt(2.0 / n)
    assert abs((z ** 3).mean()) < 5 * np.sqrt(15.0 / n)
    assert abs((z ** 4).mean() - 3.0) < 5 * np.sqrt(96.0 / n)
    ks = stats.kstest(z[:1_000_000], "norm")
    assert ks.pvalue > 1e-3
    # neighbours in a row (same Philox call) and in a column (adjacent counters) are uncorrelated
    zz = z.reshape(4096, 2560)
    for lag_prod in ((zz[:, :-1] * zz[:, 1:]), (zz[:-1] * zz[1:])):
        assert abs(lag_prod.mean()) < 5 / np.sqrt(lag_prod.size)


def test_expected_outer_product_is_identity():
    # mean_t S_t S_t^T -> I ; E||mean - I||_F^2 = d (d+1) / (r T) for iid N(0, 1/r) entries
    d, r = 48, 16
    acc = np.zeros((d, d))
    errs = {}
    for t in range(1024):
        s = sk.sketch(t, d, r).astype(np.float64)
        acc += s @ s.T
        if t + 1 in (16, 64, 256, 1024):
            errs[t + 1] = np.linalg.norm(acc / (t + 1) - np.eye(d)) ** 2
    for T, e in errs.items():
        assert 0.85 < e / (d * (d + 1) / (r * T)) < 1.15, (T, e)


def test_round_to_bf16_ties_to_even():
    def f(bits):
        return np.array([bits], dtype=np.uint32).view(np.float32)

    def bits_of(x):
        return int(sk.round_to_bf16(x).view(np.uint32)[0])

    assert bits_of(f(0x3F800000)) == 0x3F800000
    assert bits_of(f(0x3F808000)) == 0x3F800000  # tie, even stays
    assert bits_of(f(0x3F818000)) == 0x3F820000  # tie, odd goes up
    assert bits_of(f(0x3F808001)) == 0x3F810000
    assert bits_of(f(0xBF80FFFF)) == 0xBF810000
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    y = sk.round_to_bf16(x)
    assert np.all(y.view(np.uint32) & 0xFFFF == 0)
    assert np.max(np.abs(y - x) / np.abs(x)) <= 2.0 ** -8  # half an ulp of an 8-bit significand


def test_sketch_for_dtype():
    s32 = sk.sketch_for_dtype(5, 64, 32, "f32")
    sb = sk.sketch_for_dtype(5, 64, 32, "bf16")
    assert s32.dtype == np.float64 and sb.dtype == np.float64
    assert np.array_equal(s32, sk.sketch(5, 64, 32).astype(np.float64))
    assert np.array_equal(sb, sk.round_to_bf16(sk.sketch(5, 64, 32)).astype(np.float64))
    with pytest.raises(ValueError):
        sk.sketch_for_dtype(5, 64, 32, "f16")


def test_frozen_bit_patterns(golden_dir):
    """The stored bit patterns (written from this oracle by make_sketch_golden.py) still hold."""
    cache = {}
    with open(os.path.join(golden_dir, "sketch_v1_bits.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            w = line.split()
            seed, d_in, r = int(w[0], 16), int(w[1]), int(w[2])
            if (seed, d_in, r) not in cache:
                cache[(seed, d_in, r)] = sk.sketch(seed, d_in, r)
            s = cache[(seed, d_in, r)]
            if w[3] == "sum_fp32_bits_xor":
                assert int(np.bitwise_xor.reduce(s.view(np.uint32).ravel())) == int(w[5], 16)
                continue
            i, j = int(w[3]), int(w[4])
            assert int(s[i:i + 1, j].view(np.uint32)[0]) == int(w[5], 16)
            assert int(sk.round_to_bf16(s[i:i + 1, j]).view(np.uint32)[0]) >> 16 == int(w[6], 16)

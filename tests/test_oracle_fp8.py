"""Pins of the oracle's 8-bit floating point paths (Related work, "Quantization"): the E4M3 widening
against the format's definition written out with exact fractions and against torch's own conversion, the
quantised scoring functions against exact rational brute force, library compositions in fp64 and the
bf16 oracle on values both formats hold exactly, the quantised attention likewise."""
from fractions import Fraction

import numpy as np
import pytest
import torch


def _e4m3_fraction(bits):
    """The OCP E4M3 (finite) definition: sign, 4-bit exponent with bias 7, 3-bit mantissa; exponent field 0 is
    subnormal; S.1111.111 is NaN; there are no infinities."""
    sign = -1 if bits & 0x80 else 1
    e, m = (bits >> 3) & 0xF, bits & 0x7
    if e == 15 and m == 7:
        return None
    if e == 0:
        return sign * Fraction(m, 8) * Fraction(1, 2 ** 6)
    return sign * (1 + Fraction(m, 8)) * (Fraction(2) ** (e - 7))


def test_e4m3_table_matches_the_format_definition_and_torch(oracle):
    table = np.array([oracle.e4m3_to_double(b) for b in range(256)])
    for b in range(256):
        want = _e4m3_fraction(b)
        if want is None:
            assert np.isnan(table[b])
        else:
            assert Fraction(table[b]) == want, b
    assert table[0x7E] == 448.0 and table[0xFE] == -448.0 and table[0x01] == 2.0 ** -9 and table[0x08] == 2.0 ** -6
    assert table[0x00] == 0.0 and table[0x80] == 0.0 and np.signbit(table[0x80])
    assert np.isnan(table[0x7F]) and np.isnan(table[0xFF]) and np.isfinite(np.delete(table, [0x7F, 0xFF])).all()
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    np.testing.assert_array_equal(np.nan_to_num(table, nan=12345.0), np.nan_to_num(lib, nan=12345.0))


def _rand_fp8(rng, shape):
    """Random E4M3 bytes without the two NaN patterns."""
    a = rng.integers(0, 256, size=shape, dtype=np.uint8)
    a[(a & 0x7F) == 0x7F] = 0x3A
    return a


def test_score_linear_fp8_matches_exact_rational_brute_force(oracle):
    rng = np.random.default_rng(0)
    T, Dh, H = 6, 11, 3
    X8, W8 = _rand_fp8(rng, (T, Dh)), _rand_fp8(rng, (H, Dh))
    sx = np.array([0.5, 1.0, 2.0, 0.25, 1.5, 3.0], dtype=np.float32)
    sw = np.array([1.0, 0.125, 4.0], dtype=np.float32)
    b = np.array([0.25, -1.0, 8.0], dtype=np.float32)
    got = oracle.score_linear_fp8(X8, sx, W8, sw, b)
    for t in range(T):
        for h in range(H):
            acc = sum(_e4m3_fraction(int(X8[t, k])) * _e4m3_fraction(int(W8[h, k])) for k in range(Dh))
            want = Fraction(float(b[h])) + Fraction(float(sx[t])) * Fraction(float(sw[h])) * acc
            assert got[t, h] == np.float32(float(want))          # one rounding of the exact value
    # no scales, no bias: the plain dot product
    plain = oracle.score_linear_fp8(X8, None, W8, None, None)
    assert plain[2, 1] == np.float32(float(sum(_e4m3_fraction(int(X8[2, k])) * _e4m3_fraction(int(W8[1, k])) for k in range(Dh))))


def _widen(oracle, a):
    lut = np.array([oracle.e4m3_to_double(b) for b in range(256)])
    return lut[a]


def test_score_fp8_equals_torch_fp64_composition(oracle):
    rng = np.random.default_rng(1)
    T, Dh, N1, H = 17, 96, 40, 5
    X8, W18 = _rand_fp8(rng, (T, Dh)) & 0xBF, _rand_fp8(rng, (N1, Dh)) & 0xB7        # keep magnitudes moderate
    sx = rng.uniform(0.01, 0.1, T).astype(np.float32)
    sw = rng.uniform(0.01, 0.1, N1).astype(np.float32)
    b1 = rng.normal(size=N1).astype(np.float32)
    b2 = rng.normal(size=H).astype(np.float32)
    W2 = torch.randn(H, N1, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    W2b = W2.view(torch.int16).numpy().view(np.uint16)
    got = oracle.score_mlp_fp8(X8, sx, W18, sw, b1, W2b, b2)
    Xd, Wd = torch.from_numpy(_widen(oracle, X8)), torch.from_numpy(_widen(oracle, W18))
    z = (Xd @ Wd.T) * torch.from_numpy(sx.astype(np.float64))[:, None] * torch.from_numpy(sw.astype(np.float64))[None, :] \
        + torch.from_numpy(b1.astype(np.float64))
    want = torch.nn.functional.gelu(z) @ W2.to(torch.float64).T + torch.from_numpy(b2.astype(np.float64))
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-6, atol=1e-6)
    # dropping a scale or a bias changes the result
    assert np.abs(oracle.score_mlp_fp8(X8, None, W18, sw, b1, W2b, b2) - got).max() > 1e-3
    assert np.abs(oracle.score_mlp_fp8(X8, sx, W18, None, b1, W2b, b2) - got).max() > 1e-3
    assert np.abs(oracle.score_mlp_fp8(X8, sx, W18, sw, None, W2b, b2) - got).max() > 1e-3
    # the linear form against the same library product
    Wl = W18[:H]
    gl = oracle.score_linear_fp8(X8, sx, Wl, sw[:H], b2)
    wl = (Xd @ Wd[:H].T) * torch.from_numpy(sx.astype(np.float64))[:, None] * torch.from_numpy(sw[:H].astype(np.float64))[None, :] \
        + torch.from_numpy(b2.astype(np.float64))
    np.testing.assert_allclose(gl, wl.numpy(), rtol=1e-6, atol=1e-6)


def test_fp8_scoring_equals_bf16_scoring_on_values_both_formats_hold(oracle):
    """Every E4M3 value is also a bf16 value (3 mantissa bits, exponents -9..8): with unit scales the quantised
    functions must give exactly what the bf16 functions give on the same numbers."""
    rng = np.random.default_rng(2)
    T, Dh, N1, H = 9, 64, 24, 4
    X8, W18 = _rand_fp8(rng, (T, Dh)), _rand_fp8(rng, (N1, Dh))
    to_bf16 = lambda a: torch.from_numpy(_widen(oracle, a)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(torch.from_numpy(_widen(oracle, X8)).to(torch.bfloat16).to(torch.float64).numpy(), _widen(oracle, X8))
    W2 = rng.integers(0x3000, 0x4000, size=(H, N1), dtype=np.uint16)
    b1 = rng.normal(size=N1).astype(np.float32)
    np.testing.assert_array_equal(oracle.score_mlp_fp8(X8, None, W18, None, b1, W2, None),
                                  oracle.score_mlp(to_bf16(X8), to_bf16(W18), b1, W2, None))
    np.testing.assert_array_equal(oracle.score_linear_fp8(X8, None, W18[:H], None, None),
                                  oracle.score_linear(to_bf16(X8), to_bf16(W18[:H]), None))
    # a per-token scale that is a power of two scales the linear score exactly
    sx = np.full(T, 4.0, dtype=np.float32)
    np.testing.assert_array_equal(oracle.score_linear_fp8(X8, sx, W18[:H], None, None),
                                  4.0 * oracle.score_linear_fp8(X8, None, W18[:H], None, None))


def test_attention_fp8_matches_torch_fp64_and_the_bf16_attention(oracle):
    rng = np.random.default_rng(5)
    G, D, n = 4, 32, 50
    q = torch.randn(G, D, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    qb = q.view(torch.int16).numpy().view(np.uint16)
    K8, V8 = _rand_fp8(rng, (n, D)) & 0xBF, _rand_fp8(rng, (n, D)) & 0xBF
    ks = rng.uniform(0.05, 0.3, n).astype(np.float32)
    vs = rng.uniform(0.5, 2.0, n).astype(np.float32)
    scale = 1.0 / np.sqrt(D)
    got = oracle.attention_fp8(qb, K8, ks, V8, vs, scale)
    Kd = torch.from_numpy(_widen(oracle, K8)) * torch.from_numpy(ks.astype(np.float64))[:, None]
    Vd = torch.from_numpy(_widen(oracle, V8)) * torch.from_numpy(vs.astype(np.float64))[:, None]
    want = torch.softmax(q.to(torch.float64) @ Kd.T * scale, dim=-1) @ Vd
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-6, atol=1e-7)
    # unit scales: the bf16 attention on the same numbers, bit for bit
    to_bf16 = lambda a: torch.from_numpy(_widen(oracle, a)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(oracle.attention_fp8(qb, K8, None, V8, None, scale),
                                  oracle.attention(qb, to_bf16(K8), to_bf16(V8), scale))
    # K and V scales are not interchangeable, and an empty list gives zeros
    assert np.abs(oracle.attention_fp8(qb, K8, vs, V8, ks, scale) - got).max() > 1e-3
    assert (oracle.attention_fp8(qb, K8[:0], None, V8[:0], None, scale) == 0).all()
    # one row: its value row exactly (times its scale)
    one = oracle.attention_fp8(qb, K8[:1], ks[:1], V8[:1], vs[:1], scale)
    np.testing.assert_array_equal(one, np.tile((_widen(oracle, V8[:1]) * np.float64(vs[0])).astype(np.float32), (G, 1)))

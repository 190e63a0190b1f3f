"""Pins for the oracle's surrogate scoring (CPU only).

The paper prints no worked numeric example of scores, so the scoring oracle is
pinned by: exact rational brute force on tiny inputs, special cases that reduce
to a single input element, a library composition in fp64 (torch), GELU
identities and the normal CDF from scipy, and the paper's printed parameter
totals and overhead table (tests/golden/overhead_table.txt).
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from paper_2601_07891_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(a):
    """float array -> bf16 bit patterns (round to nearest even via torch)."""
    return synth.bits(torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


def _widen(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32)


def _exact_linear(Xb, Wb, b):
    X = _widen(Xb)
    W = _widen(Wb)
    T, Dh = X.shape
    H = W.shape[0]
    out = np.zeros((T, H), dtype=np.float32)
    for t in range(T):
        for h in range(H):
            acc = Fraction(float(b[h])) if b is not None else Fraction(0)
            for k in range(Dh):
                acc += Fraction(float(X[t, k])) * Fraction(float(W[h, k]))
            out[t, h] = np.float32(float(acc))
    return out


def test_linear_matches_exact_rational_brute_force(oracle):
    rng = np.random.default_rng(1)
    T, Dh, H = 7, 13, 3                     # deliberately non-square, H != Dh != T
    Xb = _bf16_bits(rng.standard_normal((T, Dh)))
    Wb = _bf16_bits(rng.standard_normal((H, Dh)) * 0.3)
    b = rng.standard_normal(H).astype(np.float32)
    got = oracle.score_linear(Xb, Wb, b)
    want = _exact_linear(Xb, Wb, b)
    assert got.shape == (T, H) and got.dtype == np.float32
    # fp64 accumulation of 13 exact products: at most one fp32 ulp from the exact sum
    np.testing.assert_allclose(got, want, rtol=2e-7, atol=1e-7)
    # no bias == zero bias
    np.testing.assert_array_equal(oracle.score_linear(Xb, Wb, None),
                                  oracle.score_linear(Xb, Wb, np.zeros(H, np.float32)))


def test_linear_one_hot_weight_selects_hidden_element(oracle):
    rng = np.random.default_rng(2)
    T, Dh, H = 9, 32, 8
    Xb = _bf16_bits(rng.standard_normal((T, Dh)))
    cols = [3, 31, 0, 7, 7, 16, 1, 30]
    W = np.zeros((H, Dh), dtype=np.float32)
    for h, k in enumerate(cols):
        W[h, k] = 1.0
    got = oracle.score_linear(Xb, _bf16_bits(W), None)
    want = _widen(Xb)[:, cols]
    np.testing.assert_array_equal(got, want)       # exact: one non-zero product


def test_linear_zero_weight_gives_bias(oracle):
    Xb = _bf16_bits(np.random.default_rng(3).standard_normal((5, 16)))
    b = np.array([0.5, -1.25, 3.0], dtype=np.float32)
    got = oracle.score_linear(Xb, np.zeros((3, 16), np.uint16), b)
    np.testing.assert_array_equal(got, np.tile(b, (5, 1)))


def test_linear_is_linear_and_position_wise(oracle):
    rng = np.random.default_rng(4)
    T, Dh, H = 6, 24, 4
    x = rng.integers(-8, 9, size=(T, Dh)).astype(np.float32)      # exact in bf16, sums exact
    y = rng.integers(-8, 9, size=(T, Dh)).astype(np.float32)
    Wb = _bf16_bits(rng.integers(-4, 5, size=(H, Dh)).astype(np.float32) / 4.0)
    b = np.array([1.0, -2.0, 0.5, 0.25], dtype=np.float32)
    fx = oracle.score_linear(_bf16_bits(x), Wb, b)
    fy = oracle.score_linear(_bf16_bits(y), Wb, b)
    fxy = oracle.score_linear(_bf16_bits(x + y), Wb, b)
    np.testing.assert_array_equal(fxy, fx + fy - b)
    # scoring a slice of positions == slicing the scores (the model acts per position)
    np.testing.assert_array_equal(oracle.score_linear(_bf16_bits(x[2:5]), Wb, b), fx[2:5])


def test_gelu_identities_and_normal_cdf(oracle):
    from scipy.stats import norm
    assert oracle.gelu(0.0) == 0.0
    for x in [0.1, 0.5, 1.0, 2.5, 4.0, 7.0]:
        assert abs((oracle.gelu(x) - oracle.gelu(-x)) - x) < 1e-15 * max(1.0, x)
        assert abs(oracle.gelu(x) - x * norm.cdf(x)) < 1e-15 * max(1.0, x)      # GELU(x) = x Phi(x)
        assert abs(oracle.gelu(-x) - (-x) * norm.cdf(-x)) < 1e-15
    assert abs(oracle.gelu(8.0) - 8.0) < 1e-13
    assert abs(oracle.gelu(-8.0)) < 1e-13
    # strictly the erf form, not the tanh approximation (they differ by ~2e-4 near x=2)
    tanh_form = 0.5 * 2.0 * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (2.0 + 0.044715 * 8.0)))
    assert abs(oracle.gelu(2.0) - tanh_form) > 1e-5


def test_mlp_selector_reduces_to_scalar_gelu(oracle):
    from scipy.stats import norm
    rng = np.random.default_rng(5)
    T, Dh, N1, H = 11, 16, 4, 2
    Xb = _bf16_bits(rng.standard_normal((T, Dh)) * 2.0)
    W1 = np.zeros((N1, Dh), np.float32)
    sel = [5, 0, 15, 9]
    for j, k in enumerate(sel):
        W1[j, k] = 1.0
    W2 = np.zeros((H, N1), np.float32)
    W2[0, 2] = 1.0          # head 0 reads hidden unit 2 -> input column 15
    W2[1, 1] = 1.0          # head 1 reads hidden unit 1 -> input column 0
    got = oracle.score_mlp(Xb, _bf16_bits(W1), None, _bf16_bits(W2), None)
    x = _widen(Xb).astype(np.float64)
    want = np.stack([x[:, 15] * norm.cdf(x[:, 15]), x[:, 0] * norm.cdf(x[:, 0])], axis=1)
    np.testing.assert_allclose(got, want.astype(np.float32), rtol=2e-7, atol=1e-7)


def test_mlp_matches_torch_fp64_library_composition(oracle):
    g = torch.Generator().manual_seed(6)
    T, Dh, N1, H = 19, 40, 24, 5            # all different: a transposed operand cannot pass
    X = torch.randn(T, Dh, generator=g).to(torch.bfloat16)
    W1 = (torch.randn(N1, Dh, generator=g) / math.sqrt(Dh)).to(torch.bfloat16)
    W2 = (torch.randn(H, N1, generator=g) / math.sqrt(N1)).to(torch.bfloat16)
    b1 = torch.randn(N1, generator=g) * 0.3
    b2 = torch.randn(H, generator=g) * 0.3
    z = torch.nn.functional.linear(X.double(), W1.double(), b1.double())
    s = torch.nn.functional.linear(torch.nn.functional.gelu(z), W2.double(), b2.double())
    got = oracle.score_mlp(synth.bits(X), synth.bits(W1), b1.numpy(), synth.bits(W2), b2.numpy())
    np.testing.assert_allclose(got, s.float().numpy(), rtol=3e-7, atol=2e-7)
    # dropping either bias must change the answer (the bias terms are really there)
    no_b1 = oracle.score_mlp(synth.bits(X), synth.bits(W1), None, synth.bits(W2), b2.numpy())
    no_b2 = oracle.score_mlp(synth.bits(X), synth.bits(W1), b1.numpy(), synth.bits(W2), None)
    assert np.abs(no_b1 - got).max() > 1e-3 and np.abs(no_b2 - got).max() > 1e-3
    np.testing.assert_allclose(no_b2 + b2.numpy(), got, rtol=1e-6, atol=1e-6)


def test_linear_matches_torch_fp64_at_model_width(oracle):
    X = synth.hidden_states(33, 4096, seed=11)
    W, _ = synth.linear_weights(4096, 8, seed=12)
    b = (torch.arange(8, dtype=torch.float32) - 3.5) / 7.0
    want = torch.nn.functional.linear(X.double(), W.double(), b.double()).float().numpy()
    got = oracle.score_linear(synth.bits(X), synth.bits(W), b.numpy())
    np.testing.assert_allclose(got, want, rtol=3e-7, atol=3e-7)
    # unit-variance scores, as the workload recipe assumes
    assert 0.7 < got.std() < 1.4


def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "overhead_table.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            p = line.split()
            rows.append(dict(model=p[0], H_Q=int(p[1]), H=int(p[2]), D=int(p[3]), Dh=int(p[4]),
                             D_int=int(p[5]), mlp_pct=float(p[6]), lin_pct=float(p[7]),
                             n_layers=int(p[8]), best=p[9], params_M=float(p[10])))
    assert len(rows) == 3
    return rows


def test_flop_closed_forms_reproduce_the_overhead_table(oracle):
    for r in _golden_rows():
        C = oracle.layer_flops(r["H_Q"], r["H"], r["D"], r["Dh"], r["D_int"])
        N1 = r["Dh"] // 8
        c_mlp = oracle.mlp_flops(r["Dh"], N1, r["H"])
        c_lin = oracle.linear_flops(r["Dh"], r["H"])
        assert c_mlp == r["Dh"] / 4 * (r["Dh"] + r["H"])          # the paper's factored form
        assert abs(100.0 * c_mlp / C - r["mlp_pct"]) <= 0.005 + 1e-12, r["model"]
        assert abs(100.0 * c_lin / C - r["lin_pct"]) <= 0.005 + 1e-12, r["model"]
    assert oracle.mlp_flops(4096, 512, 8) == 4202496
    assert oracle.mlp_flops(5120, 640, 8) == 6563840
    assert oracle.linear_flops(4096, 8) == 65536


def test_parameter_totals_match_the_summary_table(oracle):
    for r in _golden_rows():
        N1 = r["Dh"] // 8 if r["best"] == "mlp" else 0
        total = oracle.param_count(r["Dh"], N1, r["H"]) * r["n_layers"]
        assert abs(total / 1e6 - r["params_M"]) / r["params_M"] < 0.05, (r["model"], total)


def test_workload_table_matches_the_paper_shapes():
    rows = {r["model"]: r for r in _golden_rows()}
    for name, model in [("qwen3_8b_prefill_32k", "Qwen3-8B"), ("llama31_8b_prefill_4x16k", "Llama-3.1-8B-Instruct"),
                        ("qwen3_32b_prefill_128k_paged", "Qwen3-32B"), ("qwen3_8b_decode_b128", "Qwen3-8B")]:
        wl = synth.WORKLOADS[name]
        r = rows[model]
        assert (wl.d_model, wl.n_kv_heads, wl.head_dim, wl.n_layers) == (r["Dh"], r["H"], r["D"], r["n_layers"])
        if wl.surrogate == "mlp":
            assert wl.hidden == wl.d_model // 8
        assert wl.window == 128

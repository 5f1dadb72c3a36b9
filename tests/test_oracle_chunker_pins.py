"""Pins for the oracle's context chunker (row normalisation + linear map):
library routines in fp64, closed forms, invariances, brute force.  No GPU."""
import math

import numpy as np
import pytest
import torch

from paper_2512_20687_b200 import workloads as wl


def bf(x):
    return wl.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def rnd(seed, name, shape, std=1.0):
    return wl.normal_bf16(seed, name, shape, std)


def f64(b):
    return wl.bf16_bits_to_f64(b)


def test_rmsnorm_against_torch_fp64(oracle):
    x, g = rnd(1, "x", (5, 96)), rnd(1, "g", (96,))
    got = oracle.rmsnorm(x, g, eps=1e-5)
    want = torch.nn.functional.rms_norm(torch.from_numpy(f64(x)), (96,), torch.from_numpy(f64(g)), eps=1e-5)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-13, atol=1e-14)
    plain = oracle.rmsnorm(x, None, eps=0.0)
    np.testing.assert_allclose((plain ** 2).mean(axis=1), 1.0, rtol=1e-13)       # unit mean square


def test_rmsnorm_closed_forms(oracle):
    # a constant row becomes its sign times gamma; a single non-zero entry a becomes sign(a) sqrt(cols)
    g = rnd(2, "g", (8,))
    x = bf(np.stack([np.full(8, 3.0), np.full(8, -0.5)]))
    got = oracle.rmsnorm(x, g, eps=0.0)
    np.testing.assert_allclose(got, np.stack([f64(g), -f64(g)]), rtol=1e-15)
    one = np.zeros((2, 16), np.float32)
    one[0, 3], one[1, 7] = 2.5, -4.0
    got = oracle.rmsnorm(bf(one), None, eps=0.0)
    want = np.zeros((2, 16))
    want[0, 3], want[1, 7] = 4.0, -4.0
    np.testing.assert_allclose(got, want, rtol=1e-15)
    # eps enters under the root: x = 0 gives 0, tiny rows are damped
    assert not oracle.rmsnorm(bf(np.zeros((1, 4))), None, eps=1e-6).any()
    got = oracle.rmsnorm(bf(np.full((1, 4), 1.0)), None, eps=3.0)
    np.testing.assert_allclose(got, 0.5, rtol=1e-15)                              # 1 / sqrt(1 + 3)


def test_rmsnorm_ignores_positive_scaling_and_other_rows(oracle):
    x = rnd(3, "x", (4, 64))
    a = oracle.rmsnorm(x, None, eps=0.0)
    b = oracle.rmsnorm(bf(4.0 * f64(x)), None, eps=0.0)                          # exact in bf16 and in fp64
    assert np.array_equal(a, b)
    x2 = x.copy()
    x2[1:] = rnd(4, "y", (3, 64))
    assert np.array_equal(oracle.rmsnorm(x2, None, eps=0.0)[0], a[0])


@pytest.mark.parametrize("with_bias", [False, True])
def test_linear_against_numpy_and_torch(oracle, with_bias):
    B, K, N = 6, 80, 24
    x, w = rnd(5, "x", (B, K)), rnd(5, "w", (K, N), std=K ** -0.5)
    bias = rnd(5, "b", (N,)) if with_bias else None
    got = oracle.linear(x, w, bias)
    want = f64(x) @ f64(w) + (f64(bias) if with_bias else 0.0)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    tw = torch.nn.functional.linear(torch.from_numpy(f64(x)), torch.from_numpy(f64(w)).T,
                                    torch.from_numpy(f64(bias)) if with_bias else None)
    np.testing.assert_allclose(got, tw.numpy(), rtol=1e-12, atol=1e-13)
    assert np.array_equal(got, oracle.linear(x, np.ascontiguousarray(w.T), bias, w_out_major=True, n_threads=3))


def test_linear_one_hot_rows_and_pure_python(oracle):
    K, N = 12, 5
    w, bias = rnd(6, "w", (K, N)), rnd(6, "b", (N,))
    got = oracle.linear(bf(np.eye(K)), w)
    assert np.array_equal(got, f64(w))                                            # row k of W, exactly
    x = rnd(6, "x", (2, K))
    got = oracle.linear(x, w, bias)
    X, W, Bv = f64(x), f64(w), f64(bias)
    for b in range(2):
        for n in range(N):
            assert abs(got[b, n] - (sum(X[b, k] * W[k, n] for k in range(K)) + Bv[n])) < 1e-13


def test_linear_with_k_equal_d_is_the_converter(oracle):
    cfg = wl.scaled(wl.CONFIGS[0], B=3, D=32, P=2)
    c = wl.converter_inputs(cfg, with_bias=True)
    U = oracle.converter(c["x"], c["w_in_major"], c["bias"])
    y = oracle.linear(c["x"], c["w_in_major"], c["bias"])
    assert np.array_equal(U.reshape(3, -1), y)


def test_chunker_composition(oracle):
    """Normalise, round to bf16, project: against the same three steps in numpy, and
    the closed form for a one-hot input (sqrt(K) times a weight row plus the bias)."""
    cfg = wl.scaled(wl.CONFIGS[0], B=4, D=32)
    c = wl.chunker_inputs(cfg)
    xn, y = oracle.chunker(c["x"], c["gamma"], c["eps"], c["w_in_major"], c["bias"])
    X = f64(c["x"])
    want_n = X * f64(c["gamma"]) / np.sqrt((X ** 2).mean(axis=1, keepdims=True) + c["eps"])
    assert np.array_equal(xn, wl.f32_to_bf16_bits(want_n.astype(np.float32)))
    np.testing.assert_allclose(y, f64(xn) @ f64(c["w_in_major"]) + f64(c["bias"]), rtol=1e-12, atol=1e-13)
    K = c["K"]
    one = np.zeros((1, K), np.float32)
    one[0, 9] = 7.0
    _, y1 = oracle.chunker(bf(one), None, 0.0, c["w_in_major"], c["bias"])
    root = f64(bf(np.array([math.sqrt(K)])))[0]                                   # sqrt(128) rounded to bf16
    np.testing.assert_allclose(y1[0], root * f64(c["w_in_major"])[9] + f64(c["bias"]), rtol=1e-13)

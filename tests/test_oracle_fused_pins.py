"""Pins of the fused matmul + pointwise consumer oracle (CPU only): C = act(A.B + bias[n]).

The consumer is a generic op with identity maps and a broadcast bias (Sections 2.1 and 3.3 of the paper); the oracle
evaluates it the unfused way.  Pinned by closed forms, by the separately pinned matmul oracle, by brute force in exact
rational arithmetic, by NumPy in f64, and by planted mistakes."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import ref
from paper_2202_03293_b200 import inputs

SEED = inputs.BASE_SEED + 90


def test_identity_consumer_without_bias_is_the_matmul():
    a, b = inputs.uniform((23, 17), SEED, 1), inputs.uniform((17, 11), SEED, 2)
    C, S = ref.matmul_bias_act(a, b)
    C0, S0 = ref.matmul(a, b)
    assert np.array_equal(C, C0) and np.array_equal(S, S0)


def test_closed_forms():
    # A = identity: the product is B, so C = act(B + bias), exactly
    n = 9
    b = inputs.small_ints((n, 7), SEED, 3).astype(np.float32)
    bias = np.array([3, -3, 0, 1, -1, 2, -2], np.float32)
    eye = np.eye(n, dtype=np.float32)
    C, S = ref.matmul_bias_act(eye, b, bias, "none")
    assert np.array_equal(C, b.astype(np.float64) + bias)
    C, _ = ref.matmul_bias_act(eye, b, bias, "relu")
    assert np.array_equal(C, np.maximum(b.astype(np.float64) + bias, 0.0))
    assert np.array_equal(S, np.abs(b.astype(np.float64)) + np.abs(bias))
    # ones . ones + bias = K + bias[n]: the bias varies along n only (a bias indexed by m would give other values)
    M, N, K = 5, 4, 6
    bias = np.array([10, 20, 30, 40], np.float32)
    C, _ = ref.matmul_bias_act(np.ones((M, K), np.float32), np.ones((K, N), np.float32), bias)
    assert np.array_equal(C, np.tile(K + bias.astype(np.float64), (M, 1)))
    # relu clamps exactly the negative entries and leaves zero and positive ones alone
    a = np.array([[1.0], [-1.0], [0.0]], np.float32)
    C, _ = ref.matmul_bias_act(a, np.array([[2.0, -2.0]], np.float32), np.array([0.5, 0.5], np.float32), "relu")
    assert np.array_equal(C, np.array([[2.5, 0.0], [0.0, 2.5], [0.5, 0.5]]))


def test_brute_force_in_exact_arithmetic():
    rng = np.random.default_rng(SEED)
    for M, N, K in ((1, 1, 1), (3, 4, 5), (5, 2, 7), (4, 6, 1)):
        a = rng.integers(-8, 9, (M, K)).astype(np.float32) / 4
        b = rng.integers(-8, 9, (K, N)).astype(np.float32) / 8
        bias = rng.integers(-8, 9, (N,)).astype(np.float32) / 2
        for act in ("none", "relu"):
            C, S = ref.matmul_bias_act(a, b, bias, act)
            for m in range(M):
                for n in range(N):
                    acc = sum(Fraction(float(a[m, k])) * Fraction(float(b[k, n])) for k in range(K)) + Fraction(float(bias[n]))
                    if act == "relu" and acc < 0:
                        acc = Fraction(0)
                    assert Fraction(float(C[m, n])) == acc
                    s = sum(abs(Fraction(float(a[m, k])) * Fraction(float(b[k, n]))) for k in range(K)) + abs(Fraction(float(bias[n])))
                    assert Fraction(float(S[m, n])) == s


def test_against_numpy_f64_and_strided_views():
    a, b = inputs.uniform((40, 33), SEED, 4), inputs.uniform((33, 27), SEED, 5)
    bias = inputs.uniform((27,), SEED, 6)
    want = a.astype(np.float64) @ b.astype(np.float64) + bias.astype(np.float64)
    C, _ = ref.matmul_bias_act(a, b, bias, "none")
    assert np.allclose(C, want, rtol=0, atol=1e-12)
    C, _ = ref.matmul_bias_act(a, b, bias, "relu")
    assert np.allclose(C, np.maximum(want, 0.0), rtol=0, atol=1e-12)
    # transposed storage and a strided bias are the same op
    C2, _ = ref.matmul_bias_act(np.ascontiguousarray(a.T).T, np.ascontiguousarray(b.T).T, np.repeat(bias, 2)[::2], "relu")
    assert np.array_equal(C, C2)


def test_planted_mistakes_are_caught():
    a, b = inputs.uniform((6, 5), SEED, 7), inputs.uniform((5, 6), SEED, 8)
    bias = inputs.uniform((6,), SEED, 9)
    C, _ = ref.matmul_bias_act(a, b, bias, "relu")
    p = a.astype(np.float64) @ b.astype(np.float64)
    assert not np.allclose(C, np.maximum(p, 0.0) + bias)                  # consumer applied before the bias
    assert not np.allclose(C, np.maximum(p + bias[:, None], 0.0))         # bias broadcast along the wrong index
    assert not np.allclose(C, p + bias)                                   # consumer dropped
    # an unknown consumer code is rejected and nothing is written
    import ctypes
    i64, out = ctypes.c_int64, np.full((1, 1), 7.0)
    one = np.ones((1, 1), np.float32)
    rc = ref.lib().sg_ref_matmul_bias_act(i64(1), i64(1), i64(1), ctypes.c_void_p(one.ctypes.data), i64(1), i64(1),
                                          ctypes.c_void_p(one.ctypes.data), i64(1), i64(1), ctypes.c_void_p(0), i64(0), ctypes.c_int(7),
                                          ctypes.c_void_p(out.ctypes.data), i64(1), i64(1), ctypes.c_void_p(0), ctypes.c_int(1))
    assert rc == 1 and out[0, 0] == 7.0

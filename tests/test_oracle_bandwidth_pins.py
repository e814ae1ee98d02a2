"""Pins of the oracle's memory-bound 2-D kernels (Section 4.4: Copy2D, Transpose2D, ColRed2D,
RowRed2D): the figure caption that fixes the reduced index, closed forms, brute force through
the generic-op enumerator, the link to the pinned matmul (a reduction is a product with a
vector of ones), library cross-checks and planted mistakes.  CPU only."""
import os

import numpy as np
import pytest

from oracle import generic, ref
from paper_2202_03293_b200 import inputs

SEED = inputs.BASE_SEED + 70
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def vals(shape, tid, dist="uniform"):
    return inputs.make(shape, SEED, tid, dist, "f32")[1]


def test_reduced_index_follows_the_l3_figure_caption():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "l3_figure_reduction_outputs.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert rows
    for R, C, n_row, n_col in (map(int, r) for r in rows):
        A = np.ones((R, C), np.float32)
        out_r, _ = ref.rowred2d(A)
        out_c, _ = ref.colred2d(A)
        assert out_r.shape == (n_row,) and np.all(out_r == C)      # each row summed over its C entries
        assert out_c.shape == (n_col,) and np.all(out_c == R)


def test_closed_forms_on_an_index_ramp():
    # A[i,j] = i*C + j: colsum[j] = C*R(R-1)/2 + R*j, rowsum[i] = i*C*C + C(C-1)/2; square on
    # purpose, so reducing the wrong index gives the right shape and the wrong numbers
    R = C = 37
    A = (np.arange(R)[:, None] * C + np.arange(C)[None, :]).astype(np.float32)
    out_c, S_c = ref.colred2d(A)
    out_r, S_r = ref.rowred2d(A)
    assert np.array_equal(out_c, C * R * (R - 1) / 2 + R * np.arange(C, dtype=np.float64))
    assert np.array_equal(out_r, np.arange(R, dtype=np.float64) * C * C + C * (C - 1) / 2)
    assert np.array_equal(S_c, out_c) and np.array_equal(S_r, out_r)   # all entries non-negative
    assert not np.array_equal(out_c, out_r)


def test_sum_abs_is_the_sum_of_magnitudes():
    A = vals((13, 29), 1, "normal")
    for fn, axis in ((ref.colred2d, 0), (ref.rowred2d, 1)):
        out, S = fn(A)
        assert np.allclose(S, np.abs(A.astype(np.float64)).sum(axis), rtol=1e-13, atol=0)
        assert np.all(np.abs(out) <= S * (1 + 1e-15))
        _, S_neg = fn(-A)
        assert np.array_equal(S, S_neg)


@pytest.mark.parametrize("R,C", [(1, 1), (1, 9), (7, 1), (5, 6), (6, 5)])
def test_brute_force_through_the_generic_op(R, C):
    A = vals((R, C), 2, "normal")
    m_in, m_out = generic.colred2d_maps()
    assert np.allclose(ref.colred2d(A)[0], generic.evaluate_unary((R, C), m_in, m_out, A, (C,)), rtol=1e-14, atol=1e-300)
    m_in, m_out = generic.rowred2d_maps()
    assert np.allclose(ref.rowred2d(A)[0], generic.evaluate_unary((R, C), m_in, m_out, A, (R,)), rtol=1e-14, atol=1e-300)
    m_in, m_out = generic.transpose2d_maps()
    assert np.array_equal(ref.transpose2d(A), generic.evaluate_unary((R, C), m_in, m_out, A, (C, R)).astype(np.float32))
    m_in, m_out = generic.copy2d_maps()
    assert np.array_equal(ref.copy2d(A), generic.evaluate_unary((R, C), m_in, m_out, A, (R, C)).astype(np.float32))


def test_reduction_is_a_product_with_ones():
    # ColRed2D = 1^T A and RowRed2D = A 1, through the oracle's (separately pinned) matmul
    R, C = 23, 41
    A = vals((R, C), 3, "normal")
    ones_r = np.ones((1, R), np.float32)
    ones_c = np.ones((C, 1), np.float32)
    mc, ms = ref.matmul(ones_r, A)
    out_c, S_c = ref.colred2d(A)
    assert np.array_equal(out_c, mc[0]) and np.array_equal(S_c, ms[0])
    mr, ms = ref.matmul(A, ones_c)
    out_r, S_r = ref.rowred2d(A)
    assert np.array_equal(out_r, mr[:, 0]) and np.array_equal(S_r, ms[:, 0])


def test_library_cross_check_and_exactness_bound():
    # numpy's pairwise f64 sums differ from the sequential f64 sums by rounding only
    R, C = 300, 257
    A = vals((R, C), 4, "normal")
    A64 = A.astype(np.float64)
    out_c, S_c = ref.colred2d(A)
    out_r, S_r = ref.rowred2d(A)
    assert np.all(np.abs(out_c - A64.sum(0)) <= 1e-13 * S_c)
    assert np.all(np.abs(out_r - A64.sum(1)) <= 1e-13 * S_r)
    # exactly representable inputs: integers sum exactly
    Ai = np.round(A * 64).astype(np.float32)
    assert np.array_equal(ref.colred2d(Ai)[0], Ai.astype(np.int64).sum(0).astype(np.float64))
    assert np.array_equal(ref.rowred2d(Ai)[0], Ai.astype(np.int64).sum(1).astype(np.float64))


def test_rowred_is_colred_of_the_transpose():
    R, C = 19, 33
    A = vals((R, C), 5, "normal")
    At = ref.transpose2d(A)
    assert At.shape == (C, R)
    assert np.array_equal(ref.rowred2d(A)[0], ref.colred2d(At)[0])
    assert np.array_equal(ref.colred2d(A)[0], ref.rowred2d(At)[0])


def test_accumulate_mode_adds_to_the_destination():
    A = vals((9, 14), 6, "normal")
    o0 = np.linspace(-3, 3, 14)
    assert np.array_equal(ref.colred2d(A, o0)[0], o0 + ref.colred2d(A)[0])
    o1 = np.linspace(5, -5, 9)
    assert np.array_equal(ref.rowred2d(A, o1)[0], o1 + ref.rowred2d(A)[0])


@pytest.mark.parametrize("dtype", [np.float32, np.uint16, np.int32])
def test_transpose_and_copy_move_bit_patterns(dtype):
    R, C = 11, 17
    rng = np.random.default_rng(SEED)
    raw = rng.integers(0, 2 ** (8 * np.dtype(dtype).itemsize), size=(R, C), dtype=np.uint64)
    A = raw.astype(np.uint16 if np.dtype(dtype).itemsize == 2 else np.uint32).view(dtype)   # includes NaN payloads
    T = ref.transpose2d(A)
    assert T.dtype == A.dtype and T.shape == (C, R)
    for i in range(R):
        for j in range(C):
            assert T.view(np.uint8).reshape(C, R, -1)[j, i].tobytes() == A.view(np.uint8).reshape(R, C, -1)[i, j].tobytes()
    assert ref.transpose2d(T).tobytes() == np.ascontiguousarray(A).tobytes()        # involution
    assert ref.copy2d(A).tobytes() == np.ascontiguousarray(A).tobytes()
    assert ref.transpose2d(A).tobytes() == np.ascontiguousarray(A.T).tobytes()      # library routine


def test_strided_views_are_read_through_their_strides():
    base = vals((20, 30), 7, "normal")
    view = base[3:17:2, 29:1:-3]                        # row step 2, negative column step
    assert np.array_equal(ref.copy2d(view), np.ascontiguousarray(view))
    assert np.array_equal(ref.transpose2d(view), np.ascontiguousarray(view.T))
    assert np.array_equal(ref.colred2d(view)[0], ref.colred2d(np.ascontiguousarray(view))[0])
    assert np.array_equal(ref.rowred2d(base.T)[0], ref.colred2d(base)[0])           # column-major view


def test_empty_shapes():
    assert ref.copy2d(np.zeros((0, 5), np.float32)).shape == (0, 5)
    assert ref.transpose2d(np.zeros((4, 0), np.float32)).shape == (0, 4)
    out, S = ref.colred2d(np.zeros((0, 6), np.float32))
    assert out.shape == (6,) and np.all(out == 0) and np.all(S == 0)    # empty sum is the neutral value
    out, _ = ref.rowred2d(np.zeros((3, 0), np.float32), np.array([1.0, 2.0, 3.0]))
    assert np.array_equal(out, [1.0, 2.0, 3.0])


def test_planted_mistakes_are_caught():
    # the pins above must reject a reduction along the other index, a copy that forgets to
    # swap, and a sum that drops its last term
    R = C = 16
    A = (np.arange(R)[:, None] * C + np.arange(C)[None, :]).astype(np.float32)
    want_c = C * R * (R - 1) / 2 + R * np.arange(C, dtype=np.float64)
    assert not np.array_equal(ref.rowred2d(A)[0], want_c)              # wrong index
    assert not np.array_equal(ref.copy2d(A), np.ascontiguousarray(A.T))  # no swap
    assert not np.array_equal(ref.colred2d(A[:-1])[0], want_c)         # dropped term

"""Brute-force evaluator of a generic structured op (test infrastructure only).

The paper describes every named op as one configuration of a generic n-D op:
a rectangular iteration domain, one affine indexing map per operand, and a
scalar body (Section 3.3, "linalg.generic"; the contraction body is a
multiply-accumulate).  This module evaluates that description directly, with
no knowledge of matmul or convolution: it walks the flat iteration space,
decodes the multi-index, applies the indexing maps (integer matrices) and
scatter-adds the product.  It exists to pin the hand-written loop nests of
``sg_ref.c`` on tiny shapes and is far too slow for anything else.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np


def evaluate(domain, map_lhs, map_rhs, map_out, lhs, rhs, out_shape):
    """out[map_out @ i] += lhs[map_lhs @ i] * rhs[map_rhs @ i] for every i in the domain.

    ``domain``  : sizes of the iterators, e.g. (M, N, K)
    ``map_*``   : integer matrices, one row per operand dimension, one column per iterator
    Exact rational arithmetic on the (float) inputs, converted to f64 at the end.
    """
    domain = [int(d) for d in domain]
    total = 1
    for d in domain:
        total *= d
    out = {}
    for flat in range(total):
        idx = []
        rem = flat
        for d in reversed(domain):
            idx.append(rem % d)
            rem //= d
        idx.reverse()

        def apply(mat):
            return tuple(sum(int(r[j]) * idx[j] for j in range(len(idx))) for r in mat)

        a = Fraction(float(lhs[apply(map_lhs)]))
        b = Fraction(float(rhs[apply(map_rhs)]))
        key = apply(map_out)
        out[key] = out.get(key, Fraction(0)) + a * b
    res = np.zeros(out_shape, np.float64)
    for key, val in out.items():
        res[key] = float(val)
    return res


def matmul_maps():
    # iterators (m, n, k)
    return [[1, 0, 0], [0, 0, 1]], [[0, 0, 1], [0, 1, 0]], [[1, 0, 0], [0, 1, 0]]


def conv1d_maps(sw, dw):
    # iterators (n, w, f, kw, c)
    m_in = [[1, 0, 0, 0, 0], [0, sw, 0, dw, 0], [0, 0, 0, 0, 1]]
    m_k = [[0, 0, 0, 1, 0], [0, 0, 0, 0, 1], [0, 0, 1, 0, 0]]
    m_o = [[1, 0, 0, 0, 0], [0, 1, 0, 0, 0], [0, 0, 1, 0, 0]]
    return m_in, m_k, m_o


def conv2d_maps(sh, sw, dh, dw):
    # iterators (n, h, w, f, kh, kw, c)
    m_in = [[1, 0, 0, 0, 0, 0, 0], [0, sh, 0, 0, dh, 0, 0], [0, 0, sw, 0, 0, dw, 0],
            [0, 0, 0, 0, 0, 0, 1]]
    m_k = [[0, 0, 0, 0, 1, 0, 0], [0, 0, 0, 0, 0, 1, 0], [0, 0, 0, 0, 0, 0, 1],
           [0, 0, 0, 1, 0, 0, 0]]
    m_o = [[1, 0, 0, 0, 0, 0, 0], [0, 1, 0, 0, 0, 0, 0], [0, 0, 1, 0, 0, 0, 0],
           [0, 0, 0, 1, 0, 0, 0]]
    return m_in, m_k, m_o


def depthwise_conv2d_maps(sh, sw, dh, dw):
    # iterators (n, h, w, c, kh, kw): the channel iterator is parallel (Section 4.6.3)
    m_in = [[1, 0, 0, 0, 0, 0], [0, sh, 0, 0, dh, 0], [0, 0, sw, 0, 0, dw], [0, 0, 0, 1, 0, 0]]
    m_k = [[0, 0, 0, 0, 1, 0], [0, 0, 0, 0, 0, 1], [0, 0, 0, 1, 0, 0]]
    m_o = [[1, 0, 0, 0, 0, 0], [0, 1, 0, 0, 0, 0], [0, 0, 1, 0, 0, 0], [0, 0, 0, 1, 0, 0]]
    return m_in, m_k, m_o


def evaluate_unary(domain, map_in, map_out, src, out_shape):
    """out[map_out @ i] += src[map_in @ i] for every i in the domain (body: add, or a plain
    assignment where every output index is reached once).  The memory-bound kernels of
    Section 4.4 are this op with different maps.  Exact rational accumulation."""
    domain = [int(d) for d in domain]
    total = 1
    for d in domain:
        total *= d
    acc = {}
    for flat in range(total):
        idx = []
        rem = flat
        for d in reversed(domain):
            idx.append(rem % d)
            rem //= d
        idx.reverse()
        k_in = tuple(sum(int(r[j]) * idx[j] for j in range(len(idx))) for r in map_in)
        k_out = tuple(sum(int(r[j]) * idx[j] for j in range(len(idx))) for r in map_out)
        acc[k_out] = acc.get(k_out, Fraction(0)) + Fraction(float(src[k_in]))
    res = np.zeros(out_shape, np.float64)
    for key, val in acc.items():
        res[key] = float(val)
    return res


def copy2d_maps():
    # iterators (i, j)
    return [[1, 0], [0, 1]], [[1, 0], [0, 1]]


def transpose2d_maps():
    return [[1, 0], [0, 1]], [[0, 1], [1, 0]]


def colred2d_maps():
    # i is the reduction iterator: the output keeps j
    return [[1, 0], [0, 1]], [[0, 1]]


def rowred2d_maps():
    return [[1, 0], [0, 1]], [[1, 0]]

"""Pins for the CPU oracle: every check here compares it with something that is
not the oracle itself: the worked example the paper shows, closed forms,
brute force over the generic op description, library routines in f64, and
identities between the ops that the paper states."""
import os

import numpy as np
import pytest

from oracle import generic, ref
from paper_2202_03293_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SEED = inputs.BASE_SEED


def rnd(shape, tid, dist="uniform"):
    return inputs.make(shape, SEED, tid, dist)[1]


# --- P1: the paper's own example (Appendix A.4) and its conv analogues -----------------

def test_ones_matmul_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "appendix_a4_ones_matmul.txt"))
            if l.strip() and not l.startswith("#")]
    assert rows
    for M, N, K, expect in rows:
        M, N, K = int(M), int(N), int(K)
        C, S = ref.matmul(np.ones((M, K), np.float32), np.ones((K, N), np.float32),
                          C_in=np.zeros((M, N)))
        assert C.shape == (M, N)
        assert np.all(C == float(expect))
        assert np.all(S == float(expect))


def test_ones_conv_counts_reduction_size():
    O, _ = ref.conv1d_nwc_wcf(np.ones((2, 11, 5), np.float32), np.ones((3, 5, 4), np.float32))
    assert O.shape == (2, 9, 4) and np.all(O == 3 * 5)
    O, _ = ref.conv2d_nhwc_hwcf(np.ones((2, 7, 9, 3), np.float32), np.ones((2, 4, 3, 5), np.float32))
    assert O.shape == (2, 6, 6, 5) and np.all(O == 2 * 4 * 3)


# --- P2: identity ----------------------------------------------------------------------

def test_identity_matmul():
    A = rnd((6, 9), 1)
    C, _ = ref.matmul(A, np.eye(9, dtype=np.float32))
    assert np.array_equal(C, A.astype(np.float64))
    B = rnd((6, 4), 2)
    C, _ = ref.matmul(np.eye(6, dtype=np.float32), B)
    assert np.array_equal(C, B.astype(np.float64))


# --- P3: delta filter = shift ------------------------------------------------------------

@pytest.mark.parametrize("sw,dw,kw0", [(1, 1, 0), (1, 1, 2), (2, 1, 1), (1, 2, 2), (2, 3, 1), (3, 2, 2)])
def test_delta_filter_conv1d_is_shift(sw, dw, kw0):
    N, C, KW, Wo = 2, 4, 3, 5
    W_in = (Wo - 1) * sw + (KW - 1) * dw + 1
    I = rnd((N, W_in, C), 3)
    Kf = np.zeros((KW, C, C), np.float32)
    Kf[kw0] = np.eye(C)
    O, _ = ref.conv1d_nwc_wcf(I, Kf, stride=sw, dilation=dw)
    expect = I[:, kw0 * dw: kw0 * dw + (Wo - 1) * sw + 1: sw, :]
    assert np.array_equal(O, expect.astype(np.float64))


@pytest.mark.parametrize("sh,sw,dh,dw,kh0,kw0", [(1, 1, 1, 1, 0, 2), (1, 1, 1, 1, 1, 0), (2, 1, 1, 2, 1, 2),
                                                (1, 3, 2, 1, 0, 1), (2, 2, 2, 3, 1, 2)])
def test_delta_filter_conv2d_is_shift(sh, sw, dh, dw, kh0, kw0):
    N, C, KH, KW, Ho, Wo = 2, 3, 2, 3, 3, 4
    H_in = (Ho - 1) * sh + (KH - 1) * dh + 1
    W_in = (Wo - 1) * sw + (KW - 1) * dw + 1
    I = rnd((N, H_in, W_in, C), 4)
    Kf = np.zeros((KH, KW, C, C), np.float32)
    Kf[kh0, kw0] = np.eye(C)
    O, _ = ref.conv2d_nhwc_hwcf(I, Kf, stride=(sh, sw), dilation=(dh, dw))
    expect = I[:, kh0 * dh: kh0 * dh + (Ho - 1) * sh + 1: sh, kw0 * dw: kw0 * dw + (Wo - 1) * sw + 1: sw, :]
    assert np.array_equal(O, expect.astype(np.float64))


def test_delta_filter_selects_channel_not_filter_index():
    # K[kw0, c0, f0] = 1 alone: O[n,w,f0] = I[n,w+kw0,c0], all other f are zero.
    I = rnd((1, 8, 3), 5)
    Kf = np.zeros((2, 3, 4), np.float32)
    Kf[1, 2, 3] = 1.0
    O, _ = ref.conv1d_nwc_wcf(I, Kf)
    assert np.array_equal(O[0, :, 3], I[0, 1:8, 2].astype(np.float64))
    assert np.all(O[..., :3] == 0)


# --- P4: brute force over the generic op description -------------------------------------

def close(a, b, S):
    return np.all(np.abs(a - b) <= 1e-13 * (S + 1e-300) + 1e-300)


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (2, 16, 2), (3, 5, 4), (5, 2, 3)])
def test_generic_enumerator_matmul(M, N, K):
    A, B = rnd((M, K), 6), rnd((K, N), 7)
    ml, mr, mo = generic.matmul_maps()
    want = generic.evaluate((M, N, K), ml, mr, mo, A, B, (M, N))
    got, S = ref.matmul(A, B)
    assert close(got, want, S)


@pytest.mark.parametrize("N,Wo,F,KW,C,sw,dw", [(1, 1, 1, 1, 1, 1, 1), (2, 3, 4, 3, 2, 1, 1), (1, 4, 2, 2, 3, 2, 1),
                                               (2, 2, 3, 3, 2, 1, 3), (1, 3, 2, 2, 2, 3, 2)])
def test_generic_enumerator_conv1d(N, Wo, F, KW, C, sw, dw):
    W_in = (Wo - 1) * sw + (KW - 1) * dw + 1
    I, Kf = rnd((N, W_in, C), 8), rnd((KW, C, F), 9)
    ml, mr, mo = generic.conv1d_maps(sw, dw)
    want = generic.evaluate((N, Wo, F, KW, C), ml, mr, mo, I, Kf, (N, Wo, F))
    got, S = ref.conv1d_nwc_wcf(I, Kf, stride=sw, dilation=dw)
    assert close(got, want, S)


@pytest.mark.parametrize("N,Ho,Wo,F,KH,KW,C,sh,sw,dh,dw", [(1, 2, 3, 2, 2, 3, 2, 1, 1, 1, 1),
                                                           (2, 2, 2, 3, 3, 2, 2, 2, 1, 1, 2),
                                                           (1, 3, 2, 2, 2, 2, 3, 1, 3, 2, 1)])
def test_generic_enumerator_conv2d(N, Ho, Wo, F, KH, KW, C, sh, sw, dh, dw):
    H_in = (Ho - 1) * sh + (KH - 1) * dh + 1
    W_in = (Wo - 1) * sw + (KW - 1) * dw + 1
    I, Kf = rnd((N, H_in, W_in, C), 10), rnd((KH, KW, C, F), 11)
    ml, mr, mo = generic.conv2d_maps(sh, sw, dh, dw)
    want = generic.evaluate((N, Ho, Wo, F, KH, KW, C), ml, mr, mo, I, Kf, (N, Ho, Wo, F))
    got, S = ref.conv2d_nhwc_hwcf(I, Kf, stride=(sh, sw), dilation=(dh, dw))
    assert close(got, want, S)


# --- P5: identities between the ops (Section 4.6.2: 2-D with H = Kh = 1 is the 1-D op) -----

def test_conv1d_kw1_is_matmul():
    I, Kf = rnd((3, 7, 5), 12), rnd((1, 5, 6), 13)
    O, _ = ref.conv1d_nwc_wcf(I, Kf)
    C, _ = ref.matmul(I.reshape(21, 5), Kf.reshape(5, 6))
    assert np.array_equal(O.reshape(21, 6), C)


def test_conv1d_single_output_is_matmul_over_kw_c():
    I, Kf = rnd((4, 3, 5), 14), rnd((3, 5, 2), 15)
    O, _ = ref.conv1d_nwc_wcf(I, Kf)
    C, _ = ref.matmul(I.reshape(4, 15), Kf.reshape(15, 2))
    assert np.array_equal(O.reshape(4, 2), C)


def test_conv2d_h1_kh1_is_conv1d():
    I, Kf = rnd((2, 9, 4), 16), rnd((3, 4, 5), 17)
    O1, S1 = ref.conv1d_nwc_wcf(I, Kf, stride=2, dilation=1)
    O2, S2 = ref.conv2d_nhwc_hwcf(I[:, None], Kf[None], stride=(1, 2), dilation=(1, 1))
    assert np.array_equal(O2[:, 0], O1) and np.array_equal(S2[:, 0], S1)


def test_matmul_strided_views_equal_explicit_transposes():
    A, B = rnd((5, 7), 18), rnd((7, 3), 19)
    C0, _ = ref.matmul(A, B)
    At = np.ascontiguousarray(A.T)      # stored as A[k,m]
    Bt = np.ascontiguousarray(B.T)      # stored as B[n,k]
    C1, _ = ref.matmul(At.T, B)
    C2, _ = ref.matmul(A, Bt.T)
    assert np.array_equal(C0, C1) and np.array_equal(C0, C2)
    # and a transposed product is a different thing
    Csq, _ = ref.matmul(rnd((4, 4), 20), rnd((4, 4), 21))
    Csw, _ = ref.matmul(rnd((4, 4), 21), rnd((4, 4), 20))
    assert not np.array_equal(Csq, Csw)


# --- P6: the tiled op is the same op on subsets (Section 3.1) --------------------------------

def test_tiling_invariance_matmul_and_conv():
    A, B = rnd((9, 8), 22), rnd((8, 10), 23)
    C, _ = ref.matmul(A, B)
    parts = np.zeros_like(C)
    for m0 in range(0, 9, 4):
        for n0 in range(0, 10, 3):
            acc = None
            for k0 in range(0, 8, 3):   # reduction tiles accumulate into the same output tile
                acc, _ = ref.matmul(A[m0:m0 + 4, k0:k0 + 3], B[k0:k0 + 3, n0:n0 + 3], C_in=acc)
            parts[m0:m0 + 4, n0:n0 + 3] = acc
    assert np.allclose(parts, C, rtol=0, atol=1e-14)

    I, Kf = rnd((1, 12, 3), 24), rnd((3, 3, 4), 25)
    O, _ = ref.conv1d_nwc_wcf(I, Kf)
    for w0 in range(0, 10, 4):
        w1 = min(w0 + 4, 10)
        Ot, _ = ref.conv1d_nwc_wcf(I[:, w0:w1 + 2], Kf)      # input tile carries the halo KW-1
        assert np.array_equal(Ot, O[:, w0:w1])


# --- P8: library routines in f64 -------------------------------------------------------------

def test_matches_numpy_and_torch_f64():
    import torch
    import torch.nn.functional as Fn
    A, B = rnd((33, 47), 26), rnd((47, 29), 27)
    C, S = ref.matmul(A, B)
    assert np.all(np.abs(C - A.astype(np.float64) @ B.astype(np.float64)) <= 1e-14 * S)
    assert np.all(np.abs(S - np.abs(A).astype(np.float64) @ np.abs(B).astype(np.float64)) <= 1e-14 * S)

    I, Kf = rnd((2, 19, 6), 28, "normal"), rnd((3, 6, 5), 29, "normal")
    O, S = ref.conv1d_nwc_wcf(I, Kf, stride=2, dilation=3)
    t = Fn.conv1d(torch.from_numpy(I).double().permute(0, 2, 1),
                  torch.from_numpy(Kf).double().permute(2, 1, 0), stride=2, dilation=3)
    assert np.all(np.abs(O - t.permute(0, 2, 1).numpy()) <= 1e-13 * S)

    I, Kf = rnd((2, 11, 13, 4), 30, "normal"), rnd((3, 2, 4, 5), 31, "normal")
    O, S = ref.conv2d_nhwc_hwcf(I, Kf, stride=(2, 1), dilation=(1, 3))
    t = Fn.conv2d(torch.from_numpy(I).double().permute(0, 3, 1, 2),
                  torch.from_numpy(Kf).double().permute(3, 2, 0, 1), stride=(2, 1), dilation=(1, 3))
    assert np.all(np.abs(O - t.permute(0, 2, 3, 1).numpy()) <= 1e-13 * S)


# --- accumulate mode, sum-abs, point variants, argument checks -------------------------------

def test_accumulate_adds_to_existing_output():
    A, B = rnd((4, 6), 32), rnd((6, 5), 33)
    C0 = rnd((4, 5), 34).astype(np.float64)
    C, _ = ref.matmul(A, B)
    Cacc, _ = ref.matmul(A, B, C_in=C0)
    assert np.array_equal(Cacc, C0 + C)
    I, Kf = rnd((1, 5, 6, 2), 35), rnd((2, 2, 2, 3), 36)
    O0 = rnd((1, 4, 5, 3), 37).astype(np.float64)
    O, _ = ref.conv2d_nhwc_hwcf(I, Kf)
    Oacc, _ = ref.conv2d_nhwc_hwcf(I, Kf, O_in=O0)
    assert np.array_equal(Oacc, O0 + O)


def test_sum_abs_is_result_on_absolute_inputs():
    I, Kf = rnd((2, 9, 3), 38), rnd((2, 3, 4), 39)
    _, S = ref.conv1d_nwc_wcf(I, Kf)
    Oabs, _ = ref.conv1d_nwc_wcf(np.abs(I), np.abs(Kf))
    assert np.array_equal(S, Oabs)


def test_point_variants_equal_full():
    A, B = rnd((13, 21), 40), rnd((21, 17), 41)
    C, S = ref.matmul(A, B)
    pm = np.array([0, 12, 5, 7]); pn = np.array([16, 0, 3, 3])
    c, s = ref.matmul_points(A, B, pm, pn)
    assert np.array_equal(c, C[pm, pn]) and np.array_equal(s, S[pm, pn])
    I, Kf = rnd((2, 6, 7, 3), 42), rnd((2, 3, 3, 4), 43)
    O, S = ref.conv2d_nhwc_hwcf(I, Kf, stride=(1, 2), dilation=(2, 1))
    pn_, ph, pw, pf = np.array([0, 1, 1]), np.array([0, 3, 2]), np.array([1, 0, 2]), np.array([3, 0, 2])
    o, s = ref.conv2d_points(I, Kf, pn_, ph, pw, pf, stride=(1, 2), dilation=(2, 1))
    assert np.array_equal(o, O[pn_, ph, pw, pf]) and np.array_equal(s, S[pn_, ph, pw, pf])


def test_input_too_small_is_rejected_and_larger_input_is_ignored():
    I, Kf = rnd((1, 6, 2), 44), rnd((3, 2, 2), 45)
    with pytest.raises(ValueError):
        ref.conv1d_nwc_wcf(I, Kf, W_out=5)
    O4, _ = ref.conv1d_nwc_wcf(I, Kf)                # W_out = 4 uses all of I
    O3, _ = ref.conv1d_nwc_wcf(I, Kf, W_out=3)       # the excess column is simply unread
    assert np.array_equal(O3, O4[:, :3])


def test_bf16_inputs_are_exact_in_f32_products():
    # bf16 x bf16 products have at most 16 significant bits: exact in f32, so the oracle on the
    # widened values is the exact sum the bf16 path approximates only through f32 accumulation.
    bits, vals = inputs.as_bf16(inputs.uniform((64,), SEED, 46))
    assert np.array_equal(inputs.bf16_bits_to_f32(bits), vals)
    p32 = vals[:32] * vals[32:]
    p64 = vals[:32].astype(np.float64) * vals[32:].astype(np.float64)
    assert np.array_equal(p32.astype(np.float64), p64)


def test_generator_is_reproducible_and_in_range():
    a = inputs.uniform((1000,), SEED, 1)
    b = inputs.uniform((1000,), SEED, 1)
    c = inputs.uniform((1000,), SEED, 2)
    assert np.array_equal(a, b) and not np.array_equal(a, c)
    assert a.min() >= -1.0 and a.max() < 1.0 and abs(float(a.mean())) < 0.1
    z = inputs.normal((20000,), SEED, 3)
    assert abs(float(z.mean())) < 0.03 and abs(float(z.std()) - 1.0) < 0.03
    # splitmix64 reference values for the published constants: state 0 -> first outputs
    s = inputs.splitmix64(np.array([0], dtype=np.uint64))
    assert int(s[0]) == 0xE220A8397B1DCDAF

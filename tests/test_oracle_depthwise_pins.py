"""Pins of the depthwise-convolution oracle (Section 4.6.3): closed forms, brute force against the
generic-op enumerator, the reduction to a dense convolution with a diagonal filter, a library
cross-check.  CPU only."""
import numpy as np
import pytest

from oracle import generic, ref
from paper_2202_03293_b200 import inputs

SEED = inputs.BASE_SEED + 50


def vals(shape, tid, dist="uniform"):
    return inputs.make(shape, SEED, tid, dist, "f32")[1]


def test_all_ones_counts_the_window_only():
    # the channel iterator is parallel: the sum has KH*KW terms, not KH*KW*C
    I = np.ones((2, 9, 11, 5), np.float32)
    K = np.ones((3, 4, 5), np.float32)
    O, S = ref.depthwise_conv2d_nhwc_hwc(I, K)
    assert O.shape == (2, 7, 8, 5) and np.all(O == 12) and np.all(S == 12)
    O1, _ = ref.depthwise_conv1d_nwc_wc(np.ones((3, 20, 4), np.float32), np.ones((5, 4), np.float32))
    assert O1.shape == (3, 16, 4) and np.all(O1 == 5)


@pytest.mark.parametrize("sh,sw,dh,dw,kh0,kw0", [(1, 1, 1, 1, 2, 0), (2, 1, 1, 3, 0, 1), (1, 2, 2, 1, 1, 2), (3, 2, 2, 3, 2, 1)])
def test_delta_filter_is_a_per_channel_scaled_shift(sh, sw, dh, dw, kh0, kw0):
    # K[kh0,kw0,c] = g[c], zero elsewhere  =>  O[n,h,w,c] = g[c] * I[n, h*sh+kh0*dh, w*sw+kw0*dw, c]
    N, Ho, Wo, C, KH, KW = 2, 4, 5, 6, 3, 3
    Hin, Win = (Ho - 1) * sh + (KH - 1) * dh + 1, (Wo - 1) * sw + (KW - 1) * dw + 1
    I = vals((N, Hin, Win, C), 1)
    g = np.array([1, 2, 4, 0.5, -1, 0.25], np.float32)          # exact scalings
    K = np.zeros((KH, KW, C), np.float32)
    K[kh0, kw0] = g
    O, _ = ref.depthwise_conv2d_nhwc_hwc(I, K, (sh, sw), (dh, dw))
    want = I[:, kh0 * dh::sh, kw0 * dw::sw][:, :Ho, :Wo].astype(np.float64) * g
    assert np.array_equal(O, want)


@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,sh,sw,dh,dw", [(1, 2, 3, 2, 2, 3, 1, 1, 1, 1), (2, 3, 2, 3, 3, 2, 2, 1, 1, 2),
                                                          (1, 2, 2, 4, 2, 2, 3, 2, 2, 3), (2, 1, 4, 1, 1, 3, 1, 2, 1, 2)])
def test_generic_enumerator_depthwise(N, Ho, Wo, C, KH, KW, sh, sw, dh, dw):
    Hin, Win = (Ho - 1) * sh + (KH - 1) * dh + 1, (Wo - 1) * sw + (KW - 1) * dw + 1
    I = vals((N, Hin, Win, C), 2)
    K = vals((KH, KW, C), 3)
    O, _ = ref.depthwise_conv2d_nhwc_hwc(I, K, (sh, sw), (dh, dw))
    m_in, m_k, m_o = generic.depthwise_conv2d_maps(sh, sw, dh, dw)
    want = generic.evaluate((N, Ho, Wo, C, KH, KW), m_in, m_k, m_o, I, K, (N, Ho, Wo, C))
    assert np.allclose(O, want, rtol=0, atol=1e-12)


def test_depthwise_is_the_dense_convolution_with_a_diagonal_filter():
    # K_dense[kh,kw,c,f] = K[kh,kw,c] if c == f else 0: the dense op (pinned on its own) then
    # computes the depthwise one
    N, Hin, Win, C, KH, KW = 2, 9, 8, 5, 3, 2
    I = vals((N, Hin, Win, C), 4, "normal")
    K = vals((KH, KW, C), 5, "normal")
    Kd = np.zeros((KH, KW, C, C), np.float32)
    for c in range(C):
        Kd[:, :, c, c] = K[:, :, c]
    for st, dl in (((1, 1), (1, 1)), ((2, 1), (1, 2))):
        O, S = ref.depthwise_conv2d_nhwc_hwc(I, K, st, dl)
        Od, Sd = ref.conv2d_nhwc_hwcf(I, Kd, st, dl)
        assert np.array_equal(O, Od) and np.array_equal(S, Sd)


def test_one_dimensional_op_is_the_two_dimensional_one_with_h_1():
    I = vals((3, 17, 4), 6)
    K = vals((3, 4), 7)
    O1, S1 = ref.depthwise_conv1d_nwc_wc(I, K, 2, 2)
    O2, S2 = ref.depthwise_conv2d_nhwc_hwc(I[:, None], K[None], (1, 2), (1, 2))
    assert np.array_equal(O1, O2[:, 0]) and np.array_equal(S1, S2[:, 0])
    # a window of one tap is an elementwise product with a per-channel scale
    O, _ = ref.depthwise_conv1d_nwc_wc(I, K[:1])
    assert np.array_equal(O, I.astype(np.float64) * K[0].astype(np.float64))


def test_matches_torch_grouped_convolution_f64():
    torch = pytest.importorskip("torch")
    N, Hin, Win, C, KH, KW = 2, 12, 10, 6, 3, 3
    I = vals((N, Hin, Win, C), 8, "normal")
    K = vals((KH, KW, C), 9, "normal")
    for st, dl in (((1, 1), (1, 1)), ((2, 2), (1, 1)), ((1, 2), (2, 1))):
        O, _ = ref.depthwise_conv2d_nhwc_hwc(I, K, st, dl)
        x = torch.from_numpy(I).double().permute(0, 3, 1, 2)
        w = torch.from_numpy(K).double().permute(2, 0, 1)[:, None]
        y = torch.nn.functional.conv2d(x, w, stride=st, dilation=dl, groups=C).permute(0, 2, 3, 1).numpy()
        assert np.allclose(O, y, rtol=1e-12, atol=1e-12)


def test_accumulate_sum_abs_and_rejection():
    I = vals((1, 6, 7, 3), 10)
    K = vals((2, 3, 3), 11)
    O0 = vals((1, 5, 5, 3), 12)
    O, S = ref.depthwise_conv2d_nhwc_hwc(I, K, O_in=O0)
    P, _ = ref.depthwise_conv2d_nhwc_hwc(I, K)
    assert np.allclose(O, P + O0, rtol=0, atol=1e-12)
    Pa, _ = ref.depthwise_conv2d_nhwc_hwc(np.abs(I), np.abs(K))
    assert np.allclose(S, Pa, rtol=0, atol=1e-12)
    with pytest.raises(ValueError):
        ref.depthwise_conv2d_nhwc_hwc(I, K, out_hw=(6, 5))       # input too small for 6 output rows
    big, _ = ref.depthwise_conv2d_nhwc_hwc(np.pad(I, ((0, 0), (0, 2), (0, 3), (0, 0))), K, out_hw=(5, 5))
    assert np.array_equal(big, P)                                # a larger input is allowed, the excess unread

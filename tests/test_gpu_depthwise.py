"""Parity of the depthwise convolutions (Section 4.6.3) with the CPU oracle, element by element,
within |err| <= 1e-4 * sum |a*b|, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from helpers import assert_within_bound, operand
from oracle import ref
from paper_2202_03293_b200 import binding as sg
from paper_2202_03293_b200 import inputs

pytestmark = pytest.mark.gpu
SEED = inputs.BASE_SEED + 60


def run2d(N, Ho, Wo, C, KH, KW, st, dl, dtype, accumulate=False, extra=(0, 0), dist="normal"):
    Hin = (Ho - 1) * st[0] + (KH - 1) * dl[0] + 1 + extra[0]
    Win = (Wo - 1) * st[1] + (KW - 1) * dl[1] + 1 + extra[1]
    I, i = operand((N, Hin, Win, C), SEED, 1, dist, dtype)
    K, k = operand((KH, KW, C), SEED, 2, dist, dtype)
    if accumulate:
        O, o0 = operand((N, Ho, Wo, C), SEED, 3, "uniform", "f32")
        O = O.clone()
    else:
        O, o0 = torch.full((N, Ho, Wo, C), float("nan"), device="cuda"), None
    sg.sg_depthwise_conv2d_nhwc_hwc(I, K, O, st, dl, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    want, S = ref.depthwise_conv2d_nhwc_hwc(i, k, st, dl, O_in=o0, out_hw=(Ho, Wo))
    if accumulate:
        S = S + np.abs(o0)
    return O, want, S


# MobileNet-like layers at batch 1 (the paper's 2-D experiment), a batched one, odd sizes,
# windows wider than the register path, strides and dilations in every combination of 1 and 2
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,st,dl", [(1, 112, 112, 32, 3, 3, (1, 1), (1, 1)), (1, 56, 56, 128, 3, 3, (2, 2), (1, 1)),
                                                    (1, 7, 7, 1024, 3, 3, (1, 1), (1, 1)), (4, 28, 28, 256, 3, 3, (1, 1), (2, 2)),
                                                    (2, 13, 19, 36, 2, 5, (1, 2), (2, 1)), (3, 9, 10, 8, 3, 9, (1, 1), (1, 1)),
                                                    (2, 20, 21, 64, 5, 5, (2, 2), (2, 2)), (1, 1, 1, 4, 1, 1, (1, 1), (1, 1))])
def test_depthwise_conv2d(dtype, N, Ho, Wo, C, KH, KW, st, dl):
    O, want, S = run2d(N, Ho, Wo, C, KH, KW, st, dl, dtype)
    assert_within_bound(O, want, S, "depthwise conv2d")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_depthwise_conv2d_accumulate_and_oversized_input(dtype):
    O, want, S = run2d(2, 15, 17, 32, 3, 3, (1, 1), (1, 1), dtype, accumulate=True, extra=(2, 3))
    assert_within_bound(O, want, S, "accumulate, larger input")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N,Wo,C,KW,sw,dw", [(1, 1000, 32, 3, 1, 1), (2, 333, 32, 3, 2, 1), (3, 200, 64, 5, 1, 2), (1, 55, 12, 3, 2, 2)])
def test_depthwise_conv1d(dtype, N, Wo, C, KW, sw, dw):
    Win = (Wo - 1) * sw + (KW - 1) * dw + 1
    I, i = operand((N, Win, C), SEED, 4, "uniform", dtype)
    K, k = operand((KW, C), SEED, 5, "uniform", dtype)
    O = torch.full((N, Wo, C), float("nan"), device="cuda")
    sg.sg_depthwise_conv1d_nwc_wc(I, K, O, sw, dw)
    torch.cuda.synchronize()
    want, S = ref.depthwise_conv1d_nwc_wc(i, k, sw, dw)
    assert_within_bound(O, want, S, "depthwise conv1d")


def test_depthwise_generic_layouts():
    # channel counts that are no multiple of 4, channel slices (pitch != C, offset that breaks the
    # alignment), channels-first storage handed over as a permuted view: the one-element-per-thread kernel
    N, Ho, Wo, C = 2, 10, 11, 7
    Ibig, i = operand((N, Ho + 2, Wo + 2, C + 3), SEED, 6, "normal", "f32")
    K, k = operand((3, 3, C), SEED, 7, "normal", "f32")
    Obig = torch.zeros(N, Ho, Wo, C + 1, device="cuda")
    sg.sg_depthwise_conv2d_nhwc_hwc(Ibig[..., 2:C + 2], K, Obig[..., 1:])
    want, S = ref.depthwise_conv2d_nhwc_hwc(np.ascontiguousarray(i[..., 2:C + 2]), k)
    assert_within_bound(Obig[..., 1:], want, S, "channel slices")
    assert torch.all(Obig[..., 0] == 0)
    Inchw, i2 = operand((N, 8, Ho + 2, Wo + 2), SEED, 8, "normal", "bf16")
    K2, k2 = operand((3, 3, 8), SEED, 9, "normal", "bf16")
    O2 = torch.empty(N, Ho, Wo, 8, device="cuda")
    sg.sg_depthwise_conv2d_nhwc_hwc(Inchw.permute(0, 2, 3, 1), K2, O2)
    want, S = ref.depthwise_conv2d_nhwc_hwc(np.ascontiguousarray(i2.transpose(0, 2, 3, 1)), k2)
    assert_within_bound(O2, want, S, "NCHW storage through strides")


def test_depthwise_closed_forms_exactness_and_rejections():
    # integer inputs: exact; delta filter: a per-channel scaled shift of the input
    O, want, S = run2d(2, 12, 14, 16, 3, 3, (1, 1), (1, 1), "bf16", dist="ints")
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)
    I, i = operand((1, 20, 22, 8), SEED, 10, "normal", "f32")
    K = torch.zeros(3, 3, 8, device="cuda")
    K[2, 1] = torch.tensor([1, 2, 4, 0.5, -1, 0.25, 8, -2.0], device="cuda")
    O = torch.empty(1, 18, 20, 8, device="cuda")
    sg.sg_depthwise_conv2d_nhwc_hwc(I, K, O)
    torch.cuda.synchronize()
    assert torch.equal(O, I[:, 2:20, 1:21, :] * K[2, 1])
    with pytest.raises(sg.SgError):          # input too small
        sg.sg_depthwise_conv2d_nhwc_hwc(I, K, torch.empty(1, 19, 20, 8, device="cuda"))
    # empty window: overwrite writes zeros, accumulate leaves the output alone
    E = torch.full((1, 4, 2, 8), 5.0, device="cuda")
    sg.sg_depthwise_conv2d_nhwc_hwc(torch.zeros(1, 4, 4, 8, device="cuda"), torch.zeros(0, 3, 8, device="cuda"), E, mode=sg.SG_ACCUMULATE)
    torch.cuda.synchronize()
    assert torch.all(E == 5.0)
    sg.sg_depthwise_conv2d_nhwc_hwc(torch.zeros(1, 4, 4, 8, device="cuda"), torch.zeros(0, 3, 8, device="cuda"), E)
    torch.cuda.synchronize()
    assert torch.all(E == 0.0)


# 3 x 3, unit strides, enough tiles to fill the GPU: the kernels that stage whole input tiles (TMA) or walk down the rows
# with a rolling register window.  Ragged tile edges in h, w and the channel blocks, batch 1 and batched, 32- and
# 64-channel blocks, integer data (exact), accumulate mode.
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("N,Ho,Wo,C", [(8, 56, 56, 64), (5, 37, 45, 96), (16, 30, 70, 32), (1, 200, 210, 128), (3, 61, 33, 200),
                                       (2, 100, 100, 40), (16, 200, 203, 16), (32, 112, 112, 64)])   # the last: bench.py's layer
def test_depthwise_conv2d_tiled_kernels(dtype, stride, N, Ho, Wo, C):
    st = (stride, stride)
    O, want, S = run2d(N, Ho, Wo, C, 3, 3, st, (1, 1), dtype)
    assert_within_bound(O, want, S, "depthwise conv2d, tiled")
    O, want, S = run2d(N, Ho, Wo, C, 3, 3, st, (1, 1), dtype, dist="ints")
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)
    O, want, S = run2d(N, Ho, Wo, C, 3, 3, st, (1, 1), dtype, accumulate=True, extra=(1, 2))
    assert_within_bound(O, want, S, "depthwise conv2d, tiled, accumulate")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_depthwise_conv2d_tiled_channel_slice(dtype):
    # a 64-channel slice of an 80-channel tensor (pixel pitch != C) into a slice of a wider output; NaN around the slice
    # of the output must survive, and the channels outside the input slice must not leak in
    N, Ho, Wo, C = 6, 40, 48, 64
    Ibig, i = operand((N, Ho + 2, Wo + 2, 80), SEED, 20, "normal", dtype)
    K, k = operand((3, 3, C), SEED, 21, "normal", dtype)
    Obig = torch.full((N, Ho, Wo, 72), float("nan"), device="cuda")
    sg.sg_depthwise_conv2d_nhwc_hwc(Ibig[..., 8:72], K, Obig[..., 4:68])
    torch.cuda.synchronize()
    sg.sg_check()
    want, S = ref.depthwise_conv2d_nhwc_hwc(np.ascontiguousarray(i[..., 8:72]), k)
    assert_within_bound(Obig[..., 4:68], want, S, "channel slice, tiled")
    assert torch.all(torch.isnan(Obig[..., :4])) and torch.all(torch.isnan(Obig[..., 68:]))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_depthwise_kernel_selection(dtype):
    """Which of the four depthwise kernels takes a shape (sg_last_kernel_name names the exact kernel)."""
    # 3 x 3, stride 1 or 2, aligned NHWC, at least one tile per SM: whole input tiles staged by TMA
    for st in (1, 2):
        O, want, S = run2d(32, 112, 112, 64, 3, 3, (st, st), (1, 1), dtype)
        assert sg.sg_last_kernel_name() == "depthwise_tma_kernel"
        assert_within_bound(O, want, S, "tma kernel")
    # the same walk down the rows with ordinary loads, for layouts outside the TMA rules: a bf16 channel slice whose
    # base is 8-byte but not 16-byte aligned (f32 vector loads need 16 bytes themselves, so only bf16 gets here)
    if dtype == "bf16":
        N, Ho, Wo, C = 16, 100, 100, 64
        Ibig, i = operand((N, Ho + 2, Wo + 2, 72), SEED, 30, "normal", dtype)
        K, k = operand((3, 3, C), SEED, 31, "normal", dtype)
        O = torch.full((N, Ho, Wo, C), float("nan"), device="cuda")
        sg.sg_depthwise_conv2d_nhwc_hwc(Ibig[..., 4:68], K, O)       # base offset 8 bytes
        torch.cuda.synchronize()
        assert sg.sg_last_kernel_name() == "depthwise_roll_kernel"
        want, S = ref.depthwise_conv2d_nhwc_hwc(np.ascontiguousarray(i[..., 4:68]), k)
        assert_within_bound(O, want, S, "rolling-window kernel")
    # too few tiles for the tiled kernels, or a window / dilation they do not take: four channels x four columns per thread
    O, want, S = run2d(1, 7, 7, 1024, 3, 3, (1, 1), (1, 1), dtype)
    assert sg.sg_last_kernel_name() == "depthwise_vec_kernel"
    assert_within_bound(O, want, S, "vec kernel, 3x3")
    O, want, S = run2d(2, 20, 21, 64, 5, 5, (2, 2), (2, 2), dtype)
    assert sg.sg_last_kernel_name() == "depthwise_vec_kernel"
    assert_within_bound(O, want, S, "vec kernel, 5x5 dilated")
    # channels not a multiple of 4: one element per thread
    O, want, S = run2d(2, 9, 10, 7, 3, 3, (1, 1), (1, 1), dtype)
    assert sg.sg_last_kernel_name() == "depthwise_generic_kernel"
    assert_within_bound(O, want, S, "generic kernel")
    assert sg.sg_last_kernel() == sg.SG_KERNEL_FFMA

"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element,
within |err| <= 1e-4 * sum_k |a*b|, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from helpers import assert_within_bound, operand
from oracle import ref
from paper_2202_03293_b200 import binding as sg
from paper_2202_03293_b200 import inputs

pytestmark = pytest.mark.gpu
SEED = inputs.BASE_SEED
FFMA, TENSOR, STRIP = sg.SG_KERNEL_FFMA, sg.SG_KERNEL_TENSOR, sg.SG_KERNEL_CONV_STRIP


@pytest.fixture(autouse=True)
def _reset_override():
    sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    sg.sg_set_tile_override(0, 0, 0)
    yield
    sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    sg.sg_set_tile_override(0, 0, 0)
    sg.sg_check()      # no kernel of the test gave up on a bounded wait


def run_matmul(M, N, K, dtype, family=None, accumulate=False, dist="uniform", seed=SEED):
    A, a = operand((M, K), seed, 1, dist, dtype)
    B, b = operand((K, N), seed, 2, dist, dtype)
    if accumulate:
        C, c0 = operand((M, N), seed, 3, "uniform", "f32")
        C = C.clone()
    else:
        C, c0 = torch.full((M, N), float("nan"), device="cuda"), None
    if family is not None:
        sg.sg_set_kernel_override(family)
    sg.sg_matmul(A, B, C, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    want, S = ref.matmul(a, b, C_in=c0)
    if accumulate:
        S = S + np.abs(c0)          # the added term |C_in * 1| belongs to the sum of magnitudes
    return C, want, S


# ------------------------------------------------------------------ config 1: matmul 128^3 f32

# f32 inputs on the tensor-core path are three tf32 products per term (hi*hi + hi*lo + lo*hi):
# the result must stay at f32 accuracy, far inside the parity bound.
F32_TENSOR_RATIO = 4e-6


@pytest.mark.parametrize("accumulate", [False, True])
@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_c1_matmul_128_f32(accumulate, family):
    C, want, S = run_matmul(128, 128, 128, "f32", family=family, accumulate=accumulate, seed=SEED + 0)
    assert sg.sg_last_kernel() == family
    assert_within_bound(C, want, S, "matmul 128^3 f32")


def test_c1_default_selection_is_tensor_path():
    C, want, S = run_matmul(128, 128, 128, "f32", seed=SEED + 0)
    assert sg.sg_last_kernel() == TENSOR


# ------------------------------------------------------------------ matmul, both kernel families

@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (256, 256, 256), (300, 200, 136), (129, 72, 8), (1, 8, 8),
                                   (515, 264, 1000), (128, 64, 4096), (384, 520, 72)])
@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_matmul_bf16_shapes(M, N, K, family):
    C, want, S = run_matmul(M, N, K, "bf16", family=family, seed=SEED + 1)
    assert sg.sg_last_kernel() == family
    assert_within_bound(C, want, S, f"matmul bf16 {M}x{N}x{K} family {family}")


@pytest.mark.parametrize("M,N,K", [(64, 64, 64), (130, 70, 50), (257, 129, 33), (1, 1, 1), (5, 3, 2), (512, 256, 384)])
def test_matmul_f32_shapes(M, N, K):
    C, want, S = run_matmul(M, N, K, "f32", seed=SEED + 1)
    assert_within_bound(C, want, S, f"matmul f32 {M}x{N}x{K}")


@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (256, 256, 256), (300, 200, 136), (129, 72, 8), (1, 8, 8),
                                   (515, 264, 1000), (128, 64, 4096), (384, 520, 72), (1024, 768, 36)])
def test_matmul_f32_tensor_path_keeps_f32_accuracy(M, N, K):
    C, want, S = run_matmul(M, N, K, "f32", family=TENSOR, seed=SEED + 1)
    assert sg.sg_last_kernel() == TENSOR
    ratio = assert_within_bound(C, want, S, f"matmul f32 3xTF32 {M}x{N}x{K}")
    assert ratio < F32_TENSOR_RATIO, ratio
    # normal-distributed values exercise every exponent, not just [-1, 1)
    C, want, S = run_matmul(M, N, K, "f32", family=TENSOR, dist="normal", seed=SEED + 9)
    assert assert_within_bound(C, want, S, "normal inputs") < F32_TENSOR_RATIO


@pytest.mark.parametrize("bn,cg", [("64", "1"), ("128", "1"), ("256", "1"), ("128", "2"), ("256", "2")])
def test_tensor_path_every_tile_variant(bn, cg):
    # the tile variant (width, one CTA or a CTA pair) is normally chosen from the shape; exercise
    # each instantiation on shapes with ragged edges in m, n and k, several tiles per CTA, and
    # on both convolutions.  The override is read once per process, so these run in a child.
    import subprocess, sys, os
    code = (
        "import sys; sys.path.insert(0, 'tests'); sys.path.insert(0, '.');"
        "import test_gpu_parity as t;"
        "from helpers import assert_within_bound;"
        "C, want, S = t.run_matmul(400, 520, 200, 'bf16', family=t.TENSOR, seed=t.SEED + 7);"
        "assert_within_bound(C, want, S, 'ragged');"
        "C, want, S = t.run_matmul(400, 520, 200, 'bf16', family=t.TENSOR, accumulate=True, seed=t.SEED + 7);"
        "assert_within_bound(C, want, S, 'ragged acc');"
        "C, want, S = t.run_matmul(2048 + 136, 2304, 328, 'bf16', family=t.TENSOR, seed=t.SEED + 7);"
        "assert_within_bound(C, want, S, 'many tiles per CTA');"
        "O, want, S = t.run_conv2d(5, 30, 27, 72, 3, 3, 136, (1, 1), (1, 1), 'bf16', family=t.TENSOR, seed=t.SEED + 7);"
        "assert_within_bound(O, want, S, 'conv2d');"
        "O, want, S = t.run_conv1d(3, 700, 64, 3, 200, 2, 2, 'bf16', family=t.TENSOR, seed=t.SEED + 7);"
        "assert_within_bound(O, want, S, 'conv1d');"
        "C, want, S = t.run_matmul(400, 520, 200, 'f32', family=t.TENSOR, seed=t.SEED + 7);"
        "assert assert_within_bound(C, want, S, 'f32 ragged') < t.F32_TENSOR_RATIO;"
        "C, want, S = t.run_matmul(400, 520, 200, 'f32', family=t.TENSOR, accumulate=True, seed=t.SEED + 7);"
        "assert_within_bound(C, want, S, 'f32 ragged acc');"
        "C, want, S = t.run_matmul(2048 + 136, 2304, 164, 'f32', family=t.TENSOR, seed=t.SEED + 7);"
        "assert assert_within_bound(C, want, S, 'f32 many tiles per CTA') < t.F32_TENSOR_RATIO;"
        "O, want, S = t.run_conv2d(5, 30, 27, 72, 3, 3, 136, (1, 1), (1, 1), 'f32', family=t.TENSOR, seed=t.SEED + 7);"
        "assert assert_within_bound(O, want, S, 'f32 conv2d') < t.F32_TENSOR_RATIO;"
        "O, want, S = t.run_conv1d(3, 700, 64, 3, 200, 2, 2, 'f32', family=t.TENSOR, seed=t.SEED + 7);"
        "assert assert_within_bound(O, want, S, 'f32 conv1d') < t.F32_TENSOR_RATIO;"
        " t.sg.sg_check(); print('child-ok')"
    )
    env = dict(os.environ, SG_TC_BN=bn, SG_TC_CG=cg)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "child-ok" in out.stdout, out.stdout + out.stderr


# ------------------------------------------------------------------ reduction dealt out in k ranges

@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("bn,cg,splits", [(64, 1, 2), (64, 1, 5), (128, 1, 4), (128, 2, 3), (256, 2, 8), (256, 1, 16)])
@pytest.mark.parametrize("accumulate", [False, True])
def test_matmul_split_reduction(dtype, bn, cg, splits, accumulate):
    if dtype == "f32" and (bn, cg) == (256, 1):
        pytest.skip("no such f32 instantiation")
    # ragged in m, n and k; the last k range is shorter than the others
    M, N, K = 300, 328, 2000 if dtype == "bf16" else 1000
    sg.sg_set_tile_override(bn, cg, splits)
    C, want, S = run_matmul(M, N, K, dtype, family=TENSOR, accumulate=accumulate, seed=SEED + 11)
    assert sg.sg_last_tile_choice() == (bn, cg, splits)
    ratio = assert_within_bound(C, want, S, f"split {splits} of {dtype} {bn}x{cg}")
    assert ratio < F32_TENSOR_RATIO


def test_split_reduction_is_chosen_for_few_tiles_and_long_k():
    for dtype in ("bf16", "f32"):
        C, want, S = run_matmul(256, 256, 4096, dtype, seed=SEED + 12)
        assert sg.sg_last_kernel() == TENSOR and sg.sg_last_tile_choice()[2] > 1
        assert_within_bound(C, want, S, "256x256x4096")
        # integer inputs: every order of the partial sums gives the same bits
        C, want, S = run_matmul(256, 256, 4096, dtype, dist="ints", seed=SEED + 12)
        assert np.array_equal(C.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_conv_split_reduction(dtype):
    sg.sg_set_tile_override(128, 1, 3)
    O, want, S = run_conv2d(3, 20, 20, 64, 3, 3, 128, (1, 1), (1, 1), dtype, family=TENSOR, seed=SEED + 13)
    assert sg.sg_last_tile_choice() == (128, 1, 3)
    assert_within_bound(O, want, S, "conv2d split over taps")
    sg.sg_set_tile_override(64, 1, 2)
    O, want, S = run_conv1d(4, 300, 136, 3, 128, 1, 1, dtype, family=TENSOR, accumulate=True, seed=SEED + 13)
    assert sg.sg_last_tile_choice() == (64, 1, 2)
    assert_within_bound(O, want, S, "conv1d split, accumulate")


@pytest.mark.parametrize("family", [FFMA, TENSOR])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_matmul_integer_inputs_are_bit_exact(family, dtype):
    # integers in [-2,2]: every product and partial sum is exact in f32, so every summation
    # order (and the hi/lo split of the f32 tensor-core path) gives the bits of the f64 oracle.
    C, want, S = run_matmul(256, 192, 320, dtype, family=family, dist="ints", seed=SEED + 2)
    assert sg.sg_last_kernel() == family
    assert np.array_equal(C.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_matmul_accumulate_into_nonzero_output(family):
    C, want, S = run_matmul(260, 136, 200, "bf16", family=family, accumulate=True, seed=SEED + 3)
    assert sg.sg_last_kernel() == family
    assert_within_bound(C, want, S, "accumulate")


def test_matmul_paper_example_ones():
    # Appendix A.4: ones(M,K) . ones(K,N) accumulated into zeros(M,N) gives K everywhere.
    for dt, tdt in (("f32", torch.float32), ("bf16", torch.bfloat16)):
        M, N, K = 200, 136, 328
        A = torch.ones(M, K, device="cuda", dtype=tdt)
        B = torch.ones(K, N, device="cuda", dtype=tdt)
        C = torch.zeros(M, N, device="cuda")
        sg.sg_matmul(A, B, C, sg.SG_ACCUMULATE)
        torch.cuda.synchronize()
        assert torch.all(C == K)


def test_matmul_transposed_operands_through_strides():
    # Section 4.6.1: A^T B and A B^T are the same op under different strides.
    M, N, K = 150, 90, 70
    At, a_t = operand((K, M), SEED, 4, "uniform", "f32")      # stored A[k,m]
    Bt, b_t = operand((N, K), SEED, 5, "uniform", "f32")      # stored B[n,k]
    B, b = operand((K, N), SEED, 6, "uniform", "f32")
    A, a = operand((M, K), SEED, 7, "uniform", "f32")
    C = torch.empty(M, N, device="cuda")
    sg.sg_matmul(At.t(), B, C)
    want, S = ref.matmul(np.ascontiguousarray(a_t.T), b)
    assert_within_bound(C, want, S, "A^T B")
    sg.sg_matmul(A, Bt.t(), C)
    want, S = ref.matmul(a, np.ascontiguousarray(b_t.T))
    assert_within_bound(C, want, S, "A B^T")
    # column-major output view
    Ct = torch.empty(N, M, device="cuda")
    sg.sg_matmul(A, B, Ct.t())
    want, S = ref.matmul(a, b)
    assert_within_bound(Ct.t(), want, S, "column-major C")


def test_matmul_padded_rows_and_offsets():
    # non-dense pitches and an element offset that breaks 16-byte alignment: generic path
    M, N, K = 100, 60, 40
    Abig, a = operand((M, K + 3), SEED, 8, "uniform", "bf16")
    Bbig, b = operand((K, N + 5), SEED, 9, "uniform", "bf16")
    Cbig = torch.zeros(M, N + 7, device="cuda")
    A, B, C = Abig[:, 1:K + 1], Bbig[:, 3:N + 3], Cbig[:, 2:N + 2]
    sg.sg_matmul(A, B, C)
    assert sg.sg_last_kernel() == FFMA
    want, S = ref.matmul(a[:, 1:K + 1], b[:, 3:N + 3])
    assert_within_bound(C, want, S, "padded")
    assert torch.all(Cbig[:, :2] == 0) and torch.all(Cbig[:, N + 2:] == 0)     # nothing outside the view written
    # aligned pitches larger than the row: still tensor-core eligible
    M, N, K = 100, 56, 40
    Abig, a = operand((M, K + 24), SEED, 10, "uniform", "bf16")
    Cbig = torch.zeros(M, N + 4, device="cuda")
    Bd, b = operand((K, N), SEED, 11, "uniform", "bf16")
    sg.sg_matmul(Abig[:, 8:K + 8], Bd, Cbig[:, 4:])
    assert sg.sg_last_kernel() == TENSOR
    want, S = ref.matmul(a[:, 8:K + 8], b)
    assert_within_bound(Cbig[:, 4:], want, S, "pitched")
    assert torch.all(Cbig[:, :4] == 0)


def test_padded_rows_whose_extent_ends_inside_a_16_byte_unit():
    # aligned pitches, but K and N end inside a 16-byte unit: TMA would read and write the rest of that unit (the row
    # padding, NaN here), so the call must not take the tensor path; nothing outside the views may change
    M, N, K = 130, 57, 43
    for dtype in ("bf16", "f32"):
        Abig, a = operand((M, 48), SEED, 60, "uniform", dtype)
        Bbig, b = operand((K, 64), SEED, 61, "uniform", dtype)
        Abig[:, K:] = float("nan")
        Bbig[:, N:] = float("nan")
        Cbig = torch.full((M, 64), float("nan"), device="cuda")
        sg.sg_matmul(Abig[:, :K], Bbig[:, :N], Cbig[:, :N])
        torch.cuda.synchronize()
        assert sg.sg_last_kernel() == FFMA
        want, S = ref.matmul(a[:, :K], b[:, :N])
        assert_within_bound(Cbig[:, :N], want, S, "ragged extents, padded pitches")
        assert torch.all(torch.isnan(Cbig[:, N:]))


def test_degenerate_sizes():
    A = torch.ones(8, 0, device="cuda", dtype=torch.bfloat16)
    B = torch.ones(0, 8, device="cuda", dtype=torch.bfloat16)
    C = torch.full((8, 8), 5.0, device="cuda")
    sg.sg_matmul(A, B, C, sg.SG_ACCUMULATE)       # empty reduction adds nothing
    torch.cuda.synchronize()
    assert torch.all(C == 5.0)
    sg.sg_matmul(A, B, C, sg.SG_OVERWRITE)        # empty reduction: the sum is zero
    torch.cuda.synchronize()
    assert torch.all(C == 0.0)
    Cpad = torch.full((8, 12), 5.0, device="cuda")
    sg.sg_matmul(A, B, Cpad[:, 2:10], sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    assert torch.all(Cpad[:, 2:10] == 0.0) and torch.all(Cpad[:, :2] == 5.0) and torch.all(Cpad[:, 10:] == 5.0)
    E = torch.empty(0, 8, device="cuda")
    sg.sg_matmul(torch.empty(0, 4, device="cuda"), torch.empty(4, 8, device="cuda"), E)


# ------------------------------------------------------------------ convolutions

def run_conv1d(N, Wo, C, KW, F, sw, dw, dtype, family=None, accumulate=False, dist="uniform", seed=SEED, extra_w=0):
    W_in = (Wo - 1) * sw + (KW - 1) * dw + 1 + extra_w
    I, i = operand((N, W_in, C), seed, 1, dist, dtype)
    Kf, k = operand((KW, C, F), seed, 2, dist, dtype)
    if accumulate:
        O, o0 = operand((N, Wo, F), seed, 3, "uniform", "f32")
        O = O.clone()
    else:
        O, o0 = torch.full((N, Wo, F), float("nan"), device="cuda"), None
    if family is not None:
        sg.sg_set_kernel_override(family)
    sg.sg_conv1d_nwc_wcf(I, Kf, O, sw, dw, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    want, S = ref.conv1d_nwc_wcf(i, k, stride=sw, dilation=dw, O_in=o0, W_out=Wo)
    if accumulate:
        S = S + np.abs(o0)
    return O, want, S


def run_conv2d(N, Ho, Wo, C, KH, KW, F, st, dl, dtype, family=None, accumulate=False, dist="normal", seed=SEED,
               extra=(0, 0)):
    H_in = (Ho - 1) * st[0] + (KH - 1) * dl[0] + 1 + extra[0]
    W_in = (Wo - 1) * st[1] + (KW - 1) * dl[1] + 1 + extra[1]
    I, i = operand((N, H_in, W_in, C), seed, 1, dist, dtype)
    Kf, k = operand((KH, KW, C, F), seed, 2, dist, dtype)
    if accumulate:
        O, o0 = operand((N, Ho, Wo, F), seed, 3, "uniform", "f32")
        O = O.clone()
    else:
        O, o0 = torch.full((N, Ho, Wo, F), float("nan"), device="cuda"), None
    if family is not None:
        sg.sg_set_kernel_override(family)
    sg.sg_conv2d_nhwc_hwcf(I, Kf, O, st, dl, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    want, S = ref.conv2d_nhwc_hwcf(i, k, stride=st, dilation=dl, O_in=o0, out_hw=(Ho, Wo))
    if accumulate:
        S = S + np.abs(o0)
    return O, want, S


@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_c3_conv1d_f32_full(family):
    # config 3: N=32, W=1026, C=64, KW=3, F=128, stride 1, f32, uniform[-1,1)
    O, want, S = run_conv1d(32, 1024, 64, 3, 128, 1, 1, "f32", family=family, seed=SEED + 2)
    assert sg.sg_last_kernel() == family
    ratio = assert_within_bound(O, want, S, "conv1d config 3")
    assert ratio < F32_TENSOR_RATIO


def test_c4_conv2d_bf16_full():
    # config 4: N=16, H=W=58, C=64, 3x3, F=128, stride 1, bf16 in / f32 out, N(0,1)
    O, want, S = run_conv2d(16, 56, 56, 64, 3, 3, 128, (1, 1), (1, 1), "bf16", seed=SEED + 3)
    assert sg.sg_last_kernel() == STRIP
    assert_within_bound(O, want, S, "conv2d config 4")
    O, want, S = run_conv2d(16, 56, 56, 64, 3, 3, 128, (1, 1), (1, 1), "bf16", family=TENSOR, seed=SEED + 3)
    assert sg.sg_last_kernel() == TENSOR
    assert_within_bound(O, want, S, "conv2d config 4, im2col kernel")


@pytest.mark.parametrize("family", [FFMA, TENSOR])
@pytest.mark.parametrize("N,Wo,C,KW,F,sw,dw", [(4, 300, 64, 3, 128, 1, 1), (3, 333, 72, 5, 40, 1, 1),
                                               (2, 500, 64, 3, 64, 2, 1), (2, 411, 128, 3, 72, 1, 2),
                                               (5, 97, 200, 2, 136, 3, 2)])
def test_conv1d_bf16(family, N, Wo, C, KW, F, sw, dw):
    O, want, S = run_conv1d(N, Wo, C, KW, F, sw, dw, "bf16", family=family, seed=SEED + 4)
    assert sg.sg_last_kernel() == family
    assert_within_bound(O, want, S, "conv1d bf16")


@pytest.mark.parametrize("family", [FFMA, TENSOR])
@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,F,st,dl", [(3, 20, 20, 64, 3, 3, 128, (1, 1), (1, 1)),
                                                      (4, 13, 17, 72, 2, 3, 40, (1, 1), (1, 1)),
                                                      (2, 20, 19, 64, 3, 3, 64, (2, 2), (1, 1)),
                                                      (3, 21, 18, 64, 3, 2, 72, (1, 1), (2, 2)),
                                                      (1, 40, 40, 32, 3, 3, 64, (2, 1), (1, 3)),
                                                      (1, 55, 55, 32, 3, 3, 64, (2, 2), (2, 2))])
def test_conv2d_bf16(family, N, Ho, Wo, C, KH, KW, F, st, dl):
    O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, st, dl, "bf16", family=family, seed=SEED + 5)
    assert sg.sg_last_kernel() == family
    assert_within_bound(O, want, S, "conv2d bf16")


# the stride-1 kernel with a resident filter: ragged channels and columns, dilations, tiles that
# wrap over image rows and images, 1-D and 2-D, more than one column tile
@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,F,dl", [(3, 20, 20, 64, 3, 3, 128, (1, 1)), (4, 13, 17, 72, 2, 3, 40, (1, 1)),
                                                   (3, 21, 18, 64, 3, 2, 72, (2, 2)), (2, 30, 40, 136, 1, 3, 64, (1, 3)),
                                                   (5, 7, 40, 24, 3, 1, 200, (1, 1)), (1, 1, 300, 64, 1, 1, 128, (1, 1))])
@pytest.mark.parametrize("accumulate", [False, True])
def test_conv2d_strip_kernel(N, Ho, Wo, C, KH, KW, F, dl, accumulate):
    O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, (1, 1), dl, "bf16", family=STRIP, accumulate=accumulate, seed=SEED + 14)
    assert sg.sg_last_kernel() == STRIP
    assert_within_bound(O, want, S, "conv2d strip kernel")


@pytest.mark.parametrize("N,Wo,C,KW,F,dw", [(4, 300, 64, 3, 128, 1), (3, 333, 72, 5, 40, 1), (2, 411, 128, 3, 72, 2), (1, 5000, 64, 7, 64, 4)])
def test_conv1d_strip_kernel(N, Wo, C, KW, F, dw):
    O, want, S = run_conv1d(N, Wo, C, KW, F, 1, dw, "bf16", family=STRIP, seed=SEED + 15, extra_w=3)
    assert sg.sg_last_kernel() == STRIP
    assert_within_bound(O, want, S, "conv1d strip kernel")


# f32 inputs on the same kernel: the filter split once into hi and lo and kept resident, the strips split per tap into
# tensor memory.  Config 3 at full size in both modes, dilations, ragged channel blocks, 2-D windows, integer inputs.
@pytest.mark.parametrize("accumulate", [False, True])
def test_c3_conv1d_f32_strip_kernel_full(accumulate):
    O, want, S = run_conv1d(32, 1024, 64, 3, 128, 1, 1, "f32", family=STRIP, accumulate=accumulate, seed=SEED + 2)
    assert sg.sg_last_kernel_name() == "conv_strip_kernel<f32>"
    assert assert_within_bound(O, want, S, "conv1d config 3, strip kernel") < F32_TENSOR_RATIO
    O, want, S = run_conv1d(32, 1024, 64, 3, 128, 1, 1, "f32", seed=SEED + 2)      # and it is the default choice
    assert sg.sg_last_kernel_name() == "conv_strip_kernel<f32>"
    assert assert_within_bound(O, want, S, "conv1d config 3, default") < F32_TENSOR_RATIO


@pytest.mark.parametrize("N,Wo,C,KW,F,dw", [(4, 300, 64, 3, 128, 1), (3, 333, 40, 3, 64, 1), (2, 411, 64, 3, 96, 2), (1, 5000, 64, 3, 64, 4),
                                            (5, 97, 32, 2, 32, 3)])
def test_conv1d_f32_strip_kernel(N, Wo, C, KW, F, dw):
    O, want, S = run_conv1d(N, Wo, C, KW, F, 1, dw, "f32", family=STRIP, seed=SEED + 17, extra_w=3)
    assert sg.sg_last_kernel_name() == "conv_strip_kernel<f32>"
    assert assert_within_bound(O, want, S, "conv1d f32 strip kernel") < F32_TENSOR_RATIO
    O, want, S = run_conv1d(N, Wo, C, KW, F, 1, dw, "f32", family=STRIP, dist="ints", seed=SEED + 17)
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,F,dl", [(3, 20, 20, 32, 2, 2, 64, (1, 1)), (2, 30, 40, 40, 1, 3, 128, (1, 3)),
                                                   (4, 13, 17, 16, 2, 3, 32, (1, 1)), (2, 9, 150, 32, 2, 2, 64, (2, 1))])
@pytest.mark.parametrize("accumulate", [False, True])
def test_conv2d_f32_strip_kernel(N, Ho, Wo, C, KH, KW, F, dl, accumulate):
    O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, (1, 1), dl, "f32", family=STRIP, accumulate=accumulate, seed=SEED + 18)
    assert sg.sg_last_kernel_name() == "conv_strip_kernel<f32>"
    assert assert_within_bound(O, want, S, "conv2d f32 strip kernel") < F32_TENSOR_RATIO


def test_conv_strip_kernel_changes_filter_inside_a_cta():
    # two column tiles and an odd number of position tiles, more items than CTA groups: some
    # group's run of items straddles the column tiles, so it reloads its resident filter
    O, want, S = run_conv2d(2, 79, 79, 64, 3, 3, 200, (1, 1), (1, 1), "bf16", family=STRIP, seed=SEED + 16)
    assert sg.sg_last_kernel() == STRIP
    assert_within_bound(O, want, S, "two column tiles")


def test_conv_strip_kernel_exact_and_rejections():
    O, want, S = run_conv2d(2, 24, 24, 64, 3, 3, 64, (1, 1), (1, 1), "bf16", family=STRIP, dist="ints", seed=SEED + 7)
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)
    # strided convolutions and filters beyond shared memory (here also: 3 x 3 x 64 x 64 in f32, split into hi and lo) are
    # not this kernel's
    I = torch.zeros(1, 40, 40, 64, device="cuda", dtype=torch.bfloat16)
    Kf = torch.zeros(3, 3, 64, 64, device="cuda", dtype=torch.bfloat16)
    sg.sg_set_kernel_override(STRIP)
    with pytest.raises(sg.SgError):
        sg.sg_conv2d_nhwc_hwcf(I, Kf, torch.empty(1, 19, 19, 64, device="cuda"), (2, 2), (1, 1))
    with pytest.raises(sg.SgError):
        sg.sg_conv2d_nhwc_hwcf(I.float(), Kf.float(), torch.empty(1, 38, 38, 64, device="cuda"))
    big = torch.zeros(3, 3, 512, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(sg.SgError):
        sg.sg_conv2d_nhwc_hwcf(torch.zeros(1, 40, 40, 512, device="cuda", dtype=torch.bfloat16), big,
                               torch.empty(1, 38, 38, 128, device="cuda"))
    sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    sg.sg_conv2d_nhwc_hwcf(torch.zeros(1, 40, 40, 512, device="cuda", dtype=torch.bfloat16), big,
                           torch.empty(1, 38, 38, 128, device="cuda"))
    assert sg.sg_last_kernel() == TENSOR        # falls back to the im2col kernel


@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,F,st,dl", [(1, 5, 6, 3, 2, 3, 5, (1, 1), (1, 1)), (2, 9, 7, 32, 3, 3, 64, (1, 2), (2, 1)),
                                                      (1, 20, 20, 32, 3, 3, 64, (1, 1), (1, 1))])
def test_conv2d_f32(N, Ho, Wo, C, KH, KW, F, st, dl):
    O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, st, dl, "f32", seed=SEED + 6)
    assert_within_bound(O, want, S, "conv2d f32")


@pytest.mark.parametrize("N,Ho,Wo,C,KH,KW,F,st,dl", [(3, 20, 20, 64, 3, 3, 128, (1, 1), (1, 1)),
                                                      (4, 13, 17, 72, 2, 3, 40, (1, 1), (1, 1)),
                                                      (2, 20, 19, 64, 3, 3, 64, (2, 2), (1, 1)),
                                                      (1, 55, 55, 32, 3, 3, 64, (2, 2), (2, 2))])
def test_conv2d_f32_tensor_path(N, Ho, Wo, C, KH, KW, F, st, dl):
    O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, st, dl, "f32", family=TENSOR, seed=SEED + 6)
    assert sg.sg_last_kernel() == TENSOR
    assert assert_within_bound(O, want, S, "conv2d f32 3xTF32") < F32_TENSOR_RATIO


@pytest.mark.parametrize("N,Wo,C,KW,F,sw,dw", [(4, 300, 64, 3, 128, 1, 1), (3, 333, 72, 5, 40, 1, 1),
                                               (2, 500, 64, 3, 64, 2, 1), (5, 97, 200, 2, 136, 3, 2)])
def test_conv1d_f32_tensor_path(N, Wo, C, KW, F, sw, dw):
    O, want, S = run_conv1d(N, Wo, C, KW, F, sw, dw, "f32", family=TENSOR, seed=SEED + 4)
    assert sg.sg_last_kernel() == TENSOR
    assert assert_within_bound(O, want, S, "conv1d f32 3xTF32") < F32_TENSOR_RATIO


@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_conv_integer_inputs_are_bit_exact(family):
    O, want, S = run_conv2d(2, 24, 24, 64, 3, 3, 64, (1, 1), (1, 1), "bf16", family=family, dist="ints", seed=SEED + 7)
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)
    O, want, S = run_conv1d(3, 400, 64, 3, 64, 1, 1, "bf16", family=family, dist="ints", seed=SEED + 7)
    assert np.array_equal(O.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("family", [FFMA, TENSOR])
def test_conv_accumulate_and_oversized_input(family):
    O, want, S = run_conv2d(3, 18, 22, 64, 3, 3, 72, (1, 1), (1, 1), "bf16", family=family, accumulate=True,
                            seed=SEED + 8, extra=(2, 3))
    assert_within_bound(O, want, S, "conv2d accumulate, larger input")
    O, want, S = run_conv1d(3, 350, 64, 3, 64, 1, 1, "bf16", family=family, accumulate=True, seed=SEED + 8, extra_w=5)
    assert_within_bound(O, want, S, "conv1d accumulate, larger input")


def test_conv_delta_filter_is_a_shift_on_gpu():
    # closed form on the device path: K[kh0,kw0,c,f] = delta(c,f)  =>  O[n,h,w,f] = I[n,h+kh0,w+kw0,f]
    N, H, W, C = 2, 30, 34, 64
    I, i = operand((N, H, W, C), SEED, 12, "normal", "bf16")
    Kf = torch.zeros(3, 3, C, C, device="cuda", dtype=torch.bfloat16)
    Kf[2, 1] = torch.eye(C, device="cuda", dtype=torch.bfloat16)
    O = torch.empty(N, H - 2, W - 2, C, device="cuda")
    for fam in (FFMA, TENSOR, STRIP):
        sg.sg_set_kernel_override(fam)
        O.fill_(float("nan"))
        sg.sg_conv2d_nhwc_hwcf(I, Kf, O)
        assert sg.sg_last_kernel() == fam
        torch.cuda.synchronize()
        assert torch.equal(O, I[:, 2:H, 1:W - 1, :].float())


def test_conv_noncontiguous_views_use_generic_kernel():
    N, Ho, Wo, C, F = 2, 10, 12, 16, 24
    Ibig, i = operand((N, Ho + 2, Wo + 2, C + 2), SEED, 13, "normal", "bf16")
    Kf, k = operand((3, 3, C, F), SEED, 14, "normal", "bf16")
    Obig = torch.zeros(N, Ho, Wo, F + 1, device="cuda")
    sg.sg_conv2d_nhwc_hwcf(Ibig[..., 1:C + 1], Kf, Obig[..., 1:])
    assert sg.sg_last_kernel() == FFMA
    want, S = ref.conv2d_nhwc_hwcf(np.ascontiguousarray(i[..., 1:C + 1]), k)
    assert_within_bound(Obig[..., 1:], want, S, "strided views")
    assert torch.all(Obig[..., 0] == 0)


# ------------------------------------------------------------------ full-size problems, sampled outputs

def sample_points(M, N, count, seed):
    h = inputs.splitmix64(np.arange(2 * count, dtype=np.uint64) ^ np.uint64(seed))
    pm = (h[:count] % np.uint64(M)).astype(np.int64)
    pn = (h[count:] % np.uint64(N)).astype(np.int64)
    # add the corners and the tile seams, where an indexing mistake would show first
    edge_m = np.array([0, 0, M - 1, M - 1, 127 % M, 128 % M, M // 2], np.int64)
    edge_n = np.array([0, N - 1, 0, N - 1, 63 % N, 64 % N, N // 2], np.int64)
    return np.concatenate([pm, edge_m]), np.concatenate([pn, edge_n])


@pytest.mark.parametrize("M,N,K,cfg", [(4096, 4096, 4096, 1), (8192, 8192, 8192, 4), (16384, 64, 4096, 4),
                                       (4096, 256, 2048, 1), (256, 4096, 512, 1)])
def test_full_size_bf16_matmul_sampled(M, N, K, cfg):
    A, a = operand((M, K), SEED + cfg, 1, "uniform", "bf16")
    B, b = operand((K, N), SEED + cfg, 2, "uniform", "bf16")
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_matmul(A, B, C)
    torch.cuda.synchronize()
    assert sg.sg_last_kernel() == TENSOR
    pm, pn = sample_points(M, N, 4096, 99)
    want, S = ref.matmul_points(a, b, pm, pn)
    got = C[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()]
    assert_within_bound(got, want, S, f"sampled {M}x{N}x{K}")
    assert not torch.isnan(C).any()            # every element was written
    # a property that holds at any size: row sums of C equal A . (row sums of B)
    rs = (A.double() @ B.double().sum(dim=1, keepdim=True)).squeeze(1)
    assert torch.allclose(C.double().sum(dim=1), rs, rtol=1e-6, atol=1e-2 * K ** 0.5)


@pytest.mark.parametrize("M,N,K", [(1024, 1024, 1024), (4096, 4096, 4096), (256, 4096, 2048)])
def test_full_size_f32_matmul_sampled(M, N, K):
    A, a = operand((M, K), SEED + 1, 1, "uniform", "f32")
    B, b = operand((K, N), SEED + 1, 2, "uniform", "f32")
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_matmul(A, B, C)
    torch.cuda.synchronize()
    pm, pn = sample_points(M, N, 4096, 98)
    want, S = ref.matmul_points(a, b, pm, pn)
    got = C[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()]
    assert sg.sg_last_kernel() == TENSOR
    assert assert_within_bound(got, want, S, f"sampled f32 {M}x{N}x{K}") < F32_TENSOR_RATIO
    assert not torch.isnan(C).any()


def test_f32_tensor_path_special_values():
    # the hi/lo split must not turn a large finite value into infinity; an infinite or NaN input
    # gives a non-finite output (inf * lo with lo = 0 is NaN: the 3xTF32 path does not keep
    # the sign of an infinity, which the header documents)
    M, N, K = 128, 64, 32
    A = torch.zeros(M, K, device="cuda")
    B = torch.zeros(K, N, device="cuda")
    fmax = torch.finfo(torch.float32).max
    A[0, 0] = fmax                    # rounding hi up would overflow
    A[1, 0] = float("inf")
    A[2, 0] = float("nan")
    A[3, 0] = -fmax
    A[4, 0] = 1.0 + 2.0 ** -23        # lo carries the last bit
    B[0, :] = 0.25
    C = torch.empty(M, N, device="cuda")
    sg.sg_set_kernel_override(TENSOR)
    sg.sg_matmul(A, B, C)
    torch.cuda.synchronize()
    assert sg.sg_last_kernel() == TENSOR
    assert torch.all(torch.isfinite(C[0])) and torch.allclose(C[0], torch.full_like(C[0], fmax * 0.25), rtol=1e-6, atol=0)
    assert torch.allclose(C[3], torch.full_like(C[3], -fmax * 0.25), rtol=1e-6, atol=0)
    assert not torch.isfinite(C[1]).any() and not torch.isfinite(C[2]).any()
    assert torch.all(C[4] == (1.0 + 2.0 ** -23) * 0.25)
    assert torch.all(C[5:] == 0)


def test_sweep_shapes_in_the_benchmark_launch_configuration():
    # bench.py replays CUDA graphs that hold the sweep's calls on parallel branches; here a spread
    # of sweep shapes (both dtypes; split reductions, pairs, single CTAs among them) runs the same
    # way, twice, and sampled outputs of every shape are checked against the oracle
    shapes = [(256, 256, 4096), (4096, 256, 256), (1024, 512, 2048), (2048, 4096, 512), (512, 1024, 1024),
              (4096, 4096, 256), (256, 2048, 4096), (2048, 2048, 2048)]
    work = []
    for dtype in ("f32", "bf16"):
        for i, (M, N, K) in enumerate(shapes):
            A, a = operand((M, K), SEED + 20 + i, 1, "uniform", dtype)
            B, b = operand((K, N), SEED + 20 + i, 2, "uniform", dtype)
            work.append((A, B, torch.full((M, N), float("nan"), device="cuda"), a, b))
    for A, B, C, _, _ in work[:2]:
        sg.sg_matmul(A, B, C)          # first calls outside capture (driver entry points, attributes)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    lanes = [torch.cuda.Stream() for _ in range(3)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for ln in lanes:
            ln.wait_stream(side)
        for i, (A, B, C, _, _) in enumerate(work):
            if i % 4 == 0:
                sg.sg_matmul(A, B, C)
            else:
                with torch.cuda.stream(lanes[i % 4 - 1]):
                    sg.sg_matmul(A, B, C)
        for ln in lanes:
            side.wait_stream(ln)
    for _, _, C, _, _ in work:
        C.fill_(float("nan"))
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    for A, B, C, a, b in work:
        M, N = C.shape
        pm, pn = sample_points(M, N, 512, 97)
        want, S = ref.matmul_points(a, b, pm, pn)
        got = C[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()]
        assert_within_bound(got, want, S, f"graph replay {tuple(A.shape)} x {tuple(B.shape)} {A.dtype}")
        assert not torch.isnan(C).any()


# ------------------------------------------------------------------ transposed operands on the tensor-core path

def run_matmul_layout(M, N, K, a_t, b_t, accumulate=False, seed=SEED + 30, dtype="bf16"):
    """matmul with A stored [k][m] (a_t) and / or B stored [n][k] (b_t), handed over as strided views."""
    A, a = operand((K, M) if a_t else (M, K), seed, 1, "uniform", dtype)
    B, b = operand((N, K) if b_t else (K, N), seed, 2, "uniform", dtype)
    if accumulate:
        C, c0 = operand((M, N), seed, 3, "uniform", "f32")
        C = C.clone()
    else:
        C, c0 = torch.full((M, N), float("nan"), device="cuda"), None
    sg.sg_matmul(A.t() if a_t else A, B.t() if b_t else B, C, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    want, S = ref.matmul(np.ascontiguousarray(a.T) if a_t else a, np.ascontiguousarray(b.T) if b_t else b, C_in=c0)
    if accumulate:
        S = S + np.abs(c0)
    return C, want, S


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("a_t,b_t", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (320, 200, 136), (64, 72, 8), (512, 264, 1000), (1024, 768, 72)])
def test_matmul_transposed_operands_tensor_path(dtype, a_t, b_t, M, N, K):
    # Section 4.6.1: A^T B, A B^T (and both) are the same op under different strides
    sg.sg_set_kernel_override(TENSOR)
    C, want, S = run_matmul_layout(M, N, K, a_t, b_t, dtype=dtype)
    assert sg.sg_last_kernel() == TENSOR
    assert assert_within_bound(C, want, S, f"{dtype} A^T={a_t} B^T={b_t} {M}x{N}x{K}") < F32_TENSOR_RATIO


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("a_t,b_t", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("bn,cg,splits", [(64, 1, 1), (128, 1, 3), (256, 2, 1), (256, 2, 4)])
def test_matmul_transposed_operands_every_variant(dtype, a_t, b_t, bn, cg, splits):
    sg.sg_set_kernel_override(TENSOR)
    sg.sg_set_tile_override(bn, cg, splits)
    C, want, S = run_matmul_layout(448, 520, 456, a_t, b_t, accumulate=(splits == 3), dtype=dtype)
    assert sg.sg_last_tile_choice() == (bn, cg, splits)
    assert_within_bound(C, want, S, "forced variant")
    sg.sg_set_tile_override(0, 0, 0)
    # integer inputs: exact
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    A = torch.randint(-2, 3, (256, 192), device="cuda").to(tdt)       # stored [k][m] or [m][k]
    B = torch.randint(-2, 3, (192, 320), device="cuda").to(tdt)
    Aview = A.t().contiguous().t() if a_t else A                                    # same values, transposed storage
    Bview = B.t().contiguous().t() if b_t else B
    C = torch.empty(256, 320, device="cuda")
    sg.sg_matmul(Aview, Bview, C)
    torch.cuda.synchronize()
    assert sg.sg_last_kernel() == TENSOR
    assert torch.equal(C, A.float() @ B.float())


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_matmul_transposed_full_size_sampled(dtype):
    M = N = K = 4096
    At, a_t = operand((K, M), SEED + 31, 1, "uniform", dtype)
    Bt, b_t = operand((N, K), SEED + 31, 2, "uniform", dtype)
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_matmul(At.t(), Bt.t(), C)
    torch.cuda.synchronize()
    assert sg.sg_last_kernel() == TENSOR
    pm, pn = sample_points(M, N, 2048, 96)
    want, S = ref.matmul_points(np.ascontiguousarray(a_t.T), np.ascontiguousarray(b_t.T), pm, pn)
    got = C[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()]
    assert_within_bound(got, want, S, "A^T B^T 4096^3")
    assert not torch.isnan(C).any()


def test_random_shapes_layouts_and_modes():
    """Seeded sweep: matmuls of random extents (multiples of 8, so most take the tensor path; some not), either
    operand stored transposed, both dtypes, both modes; convolutions of random extents, strides and dilations."""
    rng = np.random.default_rng(SEED + 7)
    for case in range(48):
        M, N, K = (int(rng.integers(1, 90)) * 8 for _ in range(3))
        if rng.integers(0, 6) == 0:
            M, N, K = M + int(rng.integers(1, 8)), N + int(rng.integers(1, 8)), K + int(rng.integers(1, 8))
        dtype = str(rng.choice(["f32", "bf16"]))
        a_t, b_t, acc = (bool(rng.integers(0, 2)) for _ in range(3))
        A, a = operand((K, M) if a_t else (M, K), SEED, 300 + case, "uniform", dtype)
        B, b = operand((N, K) if b_t else (K, N), SEED, 400 + case, "uniform", dtype)
        if a_t:
            A, a = A.t(), a.T
        if b_t:
            B, b = B.t(), b.T
        if acc:
            C, c0 = operand((M, N), SEED, 500 + case, "uniform", "f32")
            C = C.clone()
        else:
            C, c0 = torch.full((M, N), float("nan"), device="cuda"), None
        sg.sg_matmul(A, B, C, sg.SG_ACCUMULATE if acc else sg.SG_OVERWRITE)
        torch.cuda.synchronize()
        want, S = ref.matmul(a, b, C_in=c0)
        assert_within_bound(C, want, S + (np.abs(c0) if acc else 0.0), f"random matmul {case}: {M}x{N}x{K} {dtype} a_t={a_t} b_t={b_t} acc={acc}")
    for case in range(24):
        dtype = str(rng.choice(["f32", "bf16"]))
        N, Ho, Wo = int(rng.integers(1, 5)), int(rng.integers(1, 40)), int(rng.integers(1, 40))
        C, F = int(rng.integers(1, 12)) * 8, int(rng.integers(1, 20)) * 8
        KH, KW = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        st = (int(rng.integers(1, 3)), int(rng.integers(1, 3)))
        dl = (int(rng.integers(1, 3)), int(rng.integers(1, 3)))
        acc = bool(rng.integers(0, 2))
        O, want, S = run_conv2d(N, Ho, Wo, C, KH, KW, F, st, dl, dtype, accumulate=acc, seed=SEED + case)
        assert_within_bound(O, want, S, f"random conv2d {case}: {N}x{Ho}x{Wo}x{C} {KH}x{KW} F={F} st={st} dl={dl} {dtype} acc={acc}")


# Stream-K tail: more tiles than CTAs and a partly filled last wave, so the last tiles are cut along k into equal
# runs (one per CTA or pair) whose partial sums meet by reduce-add.  Sampled rows across all tiles against the oracle.
@pytest.mark.parametrize("accumulate", [False, True])
@pytest.mark.parametrize("dtype,M,N,K,tile", [("f32", 2176, 1280, 2048, (128, 1)), ("f32", 2304, 2560, 2048, (256, 2)),
                                              ("bf16", 2176, 1280, 16384, (128, 1)), ("f32", 2090, 1300, 2048, (128, 1))])
def test_stream_k_tail(dtype, M, N, K, tile, accumulate):
    A, a = operand((M, K), SEED, 31, "uniform", dtype)
    B, b = operand((K, N), SEED, 32, "uniform", dtype)
    if accumulate:
        C, c0 = operand((M, N), SEED, 33, "uniform", "f32")
        C = C.clone()
    else:
        C, c0 = torch.full((M, N), float("nan"), device="cuda"), None
    sg.sg_set_tile_override(tile[0], tile[1], 1)
    sg.sg_matmul(A, B, C, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    sg.sg_check()
    first, run = sg.sg_last_stream_k()
    assert first > 0 and run > 0, "this shape was meant to take the stream-K tail"
    rows = np.unique(np.concatenate([np.arange(0, M, 37), np.arange(M - 130, M)]))
    want, S = ref.matmul(a[rows], b, C_in=None if c0 is None else c0[rows])
    if accumulate:
        S = S + np.abs(c0[rows])
    assert_within_bound(C[torch.from_numpy(rows).cuda()], want, S, f"stream-K tail {dtype} {M}x{N}x{K}")
    assert not torch.isnan(C).any()


def test_stream_k_tail_exact_on_integers():
    M, N, K = 2176, 1280, 2048
    A, a = operand((M, K), SEED, 34, "ints", "f32")
    B, b = operand((K, N), SEED, 35, "ints", "f32")
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_set_tile_override(128, 1, 1)
    sg.sg_matmul(A, B, C)
    torch.cuda.synchronize()
    assert sg.sg_last_stream_k()[1] > 0
    want = (a.astype(np.float64) @ b.astype(np.float64))       # small integers: every partial sum is exact
    assert np.array_equal(C.cpu().numpy().astype(np.float64), want)


def test_stream_k_tail_on_a_convolution():
    # 4 x 72 x 72 output pixels = 162 row tiles of 128 on 148 SMs, 72 k-blocks (3 x 3 taps x 256 channels, f32)
    sg.sg_set_tile_override(128, 1, 1)
    O, want, S = run_conv2d(4, 72, 72, 256, 3, 3, 128, (1, 1), (1, 1), "f32", family=TENSOR)
    assert sg.sg_last_stream_k()[1] > 0, "this shape was meant to take the stream-K tail"
    assert_within_bound(O, want, S, "stream-K tail, conv2d f32")


# ------------------------------------------------------------------ config 2: every shape of the sweep, both dtypes

SWEEP = (256, 512, 1024, 2048, 4096)
SWEEP_SHAPES = [(m, n, k) for m in SWEEP for n in SWEEP for k in SWEEP]
_sweep_cache = {}


def sweep_operands(dtype):
    """One seeded 4096 x 4096 sample per operand and dtype (as the benchmark draws them); a shape's operands are the
    leading sub-blocks, copied into dense buffers of their own."""
    if dtype not in _sweep_cache:
        _sweep_cache[dtype] = (operand((4096, 4096), SEED + 1, 1, "uniform", dtype), operand((4096, 4096), SEED + 1, 2, "uniform", dtype))
    return _sweep_cache[dtype]


def seam_points(M, N, count, seed):
    """`count` hashed points plus the corners and both sides of every 128-row / 64-column tile seam along two lines."""
    pm, pn = sample_points(M, N, count, seed)
    sm = np.array([m for t in range(128, M, 128) for m in (t - 1, t)], np.int64)
    sn = np.array([n for t in range(64, N, 64) for n in (t - 1, t)], np.int64)
    pm = np.concatenate([pm, sm, np.full(sn.size, M - 1, np.int64), np.full(sn.size, M // 3, np.int64)])
    pn = np.concatenate([pn, np.full(sm.size, N - 1, np.int64), sn, sn])
    return pm, pn


def check_sweep_point(C, a, b, M, N, K, dtype, what):
    pm, pn = seam_points(M, N, 512, 1000 + M + 2 * N + 3 * K)
    want, S = ref.matmul_points(a[:M, :K], b[:K, :N], pm, pn)
    got = C[torch.from_numpy(pm).cuda(), torch.from_numpy(pn).cuda()]
    ratio = assert_within_bound(got, want, S, f"{what} {dtype} {M}x{N}x{K}")
    assert not torch.isnan(C).any(), f"{what} {dtype} {M}x{N}x{K}: unwritten elements"
    if dtype == "f32":
        assert ratio < F32_TENSOR_RATIO, ratio


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("M", SWEEP)
def test_sweep_every_shape(dtype, M):
    """All 125 shapes {256..4096}^3 of the benchmark's sweep (25 per test case), each into a NaN-filled output:
    >= 512 sampled points plus tile seams and corners against the oracle, no element left unwritten."""
    (A, a), (B, b) = sweep_operands(dtype)
    for N in SWEEP:
        for K in SWEEP:
            Ad, Bd = A[:M, :K].contiguous(), B[:K, :N].contiguous()
            C = torch.full((M, N), float("nan"), device="cuda")
            sg.sg_matmul(Ad, Bd, C)
            torch.cuda.synchronize()
            assert sg.sg_last_kernel() == TENSOR
            check_sweep_point(C, a, b, M, N, K, dtype, "sweep")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_sweep_in_the_benchmark_launch_configuration(dtype):
    """The 64 sweep shapes without a 4096 extent, launched the way bench.py launches a step: captured once into a CUDA
    graph on four parallel branches, largest first, replayed twice; every shape checked as above."""
    (A, a), (B, b) = sweep_operands(dtype)
    shapes = sorted([s for s in SWEEP_SHAPES if 4096 not in s], key=lambda s: -s[0] * s[1] * s[2])
    work = [(A[:m, :k].contiguous(), B[:k, :n].contiguous(), torch.full((m, n), float("nan"), device="cuda")) for m, n, k in shapes]
    for Ad, Bd, C in work[:2]:
        sg.sg_matmul(Ad, Bd, C)          # first calls outside capture (driver entry points, attributes)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    lanes = [torch.cuda.Stream() for _ in range(3)]
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        for ln in lanes:
            ln.wait_stream(side)
        for i, (Ad, Bd, C) in enumerate(work):
            if i % 4 == 0:
                sg.sg_matmul(Ad, Bd, C)
            else:
                with torch.cuda.stream(lanes[i % 4 - 1]):
                    sg.sg_matmul(Ad, Bd, C)
        for ln in lanes:
            side.wait_stream(ln)
    for _, _, C in work:
        C.fill_(float("nan"))
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    sg.sg_check()
    for (m, n, k), (_, _, C) in zip(shapes, work):
        check_sweep_point(C, a, b, m, n, k, dtype, "graph replay")


# ------------------------------------------------------------------ forced k splits without a forced tile

@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("splits", [2, 3, 8, 64])
def test_forced_split_alone_never_fails(dtype, splits):
    # a forced number of k ranges with the tile left to the library is taken when every range gets at least one
    # k-block (4 k-blocks of 64 bf16, 8 of 32 f32 here) and ignored otherwise; the call succeeds either way
    M, N, K = 4096, 4096, 256
    (A, a), (B, b) = sweep_operands(dtype)
    Ad, Bd = A[:M, :K].contiguous(), B[:K, :N].contiguous()
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_set_tile_override(0, 0, splits)
    sg.sg_matmul(Ad, Bd, C)
    torch.cuda.synchronize()
    honoured = {("bf16", 2), ("f32", 2), ("f32", 3), ("f32", 8)}
    if (dtype, splits) in honoured:
        assert sg.sg_last_tile_choice()[2] == splits
    check_sweep_point(C, a, b, M, N, K, dtype, f"forced split {splits}")


def test_forced_pair_count_that_no_variant_can_honour():
    # 64 columns: only the single-CTA 64-column tile applies; asking for pairs falls back to it
    sg.sg_set_tile_override(0, 2, 0)
    C, want, S = run_matmul(512, 64, 256, "bf16", family=TENSOR, seed=SEED + 40)
    assert sg.sg_last_tile_choice()[:2] == (64, 1)
    assert_within_bound(C, want, S, "forced pairs on a 64-column problem")


# ------------------------------------------------------------------ the time-out path

def test_device_timeout_is_reported_once_and_cleared():
    """A warp that waits about a millisecond on a barrier nobody signals gives up like any pipeline wait: the status
    word is set, the kernel returns, sg_check reports SG_ERR_DEVICE_TIMEOUT exactly once, and the device stays usable."""
    sg.sg_check()
    sg.sg_selftest_wait_timeout(2_000_000)
    with pytest.raises(sg.SgError) as err:
        sg.sg_check()
    assert err.value.code == 5 and "wait expired" in str(err.value)
    sg.sg_check()                                   # cleared by the read
    C, want, S = run_matmul(256, 256, 256, "bf16", family=TENSOR, seed=SEED + 41)
    assert_within_bound(C, want, S, "after a reported time-out")
    sg.sg_check()


# ------------------------------------------------------------------ host-side state: tensor-map cache, overlapped launches

def test_tensor_map_cache_hits_and_never_serves_a_stale_map():
    A = torch.randint(-2, 3, (512, 256), device="cuda").to(torch.bfloat16)
    B = torch.randint(-2, 3, (256, 384), device="cuda").to(torch.bfloat16)
    C = torch.empty(512, 384, device="cuda")
    sg.sg_set_kernel_override(TENSOR)
    h0, m0 = sg.sg_tensor_map_cache_stats()
    sg.sg_matmul(A, B, C)
    h1, m1 = sg.sg_tensor_map_cache_stats()
    sg.sg_matmul(A, B, C)
    h2, m2 = sg.sg_tensor_map_cache_stats()
    # three maps per call: looked up, encoded when new (an earlier test may have left a map of the same address and
    # geometry behind), and found by the second call
    assert (h1 - h0) + (m1 - m0) == 3 and m1 - m0 >= 1 and m2 == m1 and h2 - h1 == 3
    torch.cuda.synchronize()
    assert torch.equal(C, A.float() @ B.float())
    # the same base pointers with another geometry: other keys, so other maps
    A2, B2, C2 = A.view(-1)[:256 * 128].view(256, 128), B.view(-1)[:128 * 192].view(128, 192), C.view(-1)[:256 * 192].view(256, 192)
    sg.sg_matmul(A2, B2, C2)
    torch.cuda.synchronize()
    assert torch.equal(C2, A2.float() @ B2.float())
    # more distinct maps than the cache holds (2048): entries are replaced, results stay right
    big = torch.randint(-2, 3, (128 + 900, 64), device="cuda").to(torch.bfloat16)
    Bs = torch.randint(-2, 3, (64, 64), device="cuda").to(torch.bfloat16)
    outs = torch.empty(900, 128 + 900, 64, device="cuda")
    for i in range(900):
        sg.sg_matmul(big[:128 + i], Bs, outs[i, :128 + i])
    sg.sg_matmul(A, B, C)                    # its maps may have been evicted meanwhile
    torch.cuda.synchronize()
    want = big.float() @ Bs.float()
    for i in (0, 1, 450, 899):
        assert torch.equal(outs[i, :128 + i], want[:128 + i])
    assert torch.equal(C, A.float() @ B.float())
    h3, m3 = sg.sg_tensor_map_cache_stats()
    assert m3 - m2 >= 1800                   # every one of those shapes needed its own input and output map


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_back_to_back_calls_that_depend_on_each_other(dtype):
    """Tensor-core launches may start while the kernel ahead of them drains; they must still see its results (a call
    that reads the previous call's output) and must not overwrite what it still reads (a call that writes the previous
    call's input).  Small integers keep every result exact; no synchronisation between the calls."""
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    M, K = 1024, 256
    A = torch.randint(-1, 2, (M, K), device="cuda").to(tdt)
    Bm = torch.randint(-1, 2, (K, K), device="cuda").to(tdt)
    P = torch.zeros(K, K, device="cuda")
    P[torch.arange(K, device="cuda"), torch.randperm(K, device="cuda")] = 1.0          # a permutation: products stay in {-1, 0, 1}
    P = P.to(tdt)
    X = torch.empty(M, K, device="cuda")              # f32 outputs; re-read as inputs only on the f32 path
    Y = torch.empty(M, K, device="cuda")
    sg.sg_set_kernel_override(TENSOR)
    if dtype == "f32":
        sg.sg_matmul(A, Bm, X)                        # X = A.B           (|x| <= 256)
        for _ in range(6):
            sg.sg_matmul(X, P, Y)                     # reads X right behind the call that wrote it
            sg.sg_matmul(Y, P, X)                     # writes X right behind the call that read it
        torch.cuda.synchronize()
        want = A.double() @ Bm.double()
        for _ in range(12):
            want = want @ P.double()
        assert torch.equal(X.double(), want)
    else:
        # bf16 inputs cannot be an f32 output; alternate two products into the same output instead: the last one wins
        B2 = torch.randint(-1, 2, (K, K), device="cuda").to(tdt)
        for _ in range(6):
            sg.sg_matmul(A, Bm, X)
            sg.sg_matmul(A, B2, X)
            sg.sg_matmul(A, Bm, X, sg.SG_ACCUMULATE)  # adds onto the call ahead of it
        torch.cuda.synchronize()
        assert torch.equal(X.double(), A.double() @ (B2.double() + Bm.double()))
    sg.sg_check()

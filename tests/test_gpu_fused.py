"""Parity of the fused matmul + pointwise consumer, C = act(A.B + bias[n]) (Sections 2.1 and 3.3 of the paper), with the
CPU oracle, element by element, within |err| <= 1e-4 * (sum_k |a*b| + |bias|), on the same seeded inputs."""
import numpy as np
import pytest
import torch

from helpers import assert_within_bound, operand
from oracle import ref
from paper_2202_03293_b200 import binding as sg
from paper_2202_03293_b200 import inputs

pytestmark = pytest.mark.gpu
SEED = inputs.BASE_SEED + 91
ACT = {"none": sg.SG_ACT_NONE, "relu": sg.SG_ACT_RELU}


@pytest.fixture(autouse=True)
def _reset_override():
    sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    sg.sg_set_tile_override(0, 0, 0)
    yield
    sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    sg.sg_set_tile_override(0, 0, 0)
    sg.sg_check()


def run(M, N, K, dtype, act, with_bias=True, dist="uniform", family=None, bias_view=None):
    A, a = operand((M, K), SEED, 1, dist, dtype)
    B, b = operand((K, N), SEED, 2, dist, dtype)
    bias = bias_h = None
    if with_bias:
        bias, bias_h = operand((N,), SEED, 3, dist, "f32")
        if bias_view is not None:
            wide = torch.zeros(2 * N + 1, device="cuda")
            wide[bias_view::2][:N] = bias
            bias = wide[bias_view::2][:N]
    C = torch.full((M, N), float("nan"), device="cuda")
    if family is not None:
        sg.sg_set_kernel_override(family)
    sg.sg_matmul_bias_act(A, B, bias, C, ACT[act])
    torch.cuda.synchronize()
    want, S = ref.matmul_bias_act(a, b, bias_h, act)
    return C, want, S


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("act", ["none", "relu"])
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (300, 200, 136), (129, 72, 8), (515, 264, 1000), (1024, 768, 72), (256, 256, 4096)])
def test_fused_matmul_on_the_tensor_path(dtype, act, M, N, K):
    C, want, S = run(M, N, K, dtype, act)
    assert sg.sg_last_kernel() == sg.SG_KERNEL_TENSOR and sg.sg_last_tile_choice()[2] == 1     # never a split reduction
    assert sg.sg_last_stream_k()[1] == 0
    assert assert_within_bound(C, want, S, f"fused {dtype} {act} {M}x{N}x{K}") < 4e-6
    if act == "relu":
        assert (C >= 0).all() and (C == 0).any() and (C > 0).any()


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("bn,cg", [(64, 1), (128, 1), (256, 1), (128, 2), (256, 2)])
def test_fused_matmul_every_tile_variant(dtype, bn, cg):
    if dtype == "f32" and (bn, cg) == (256, 1):
        pytest.skip("no such f32 instantiation")
    sg.sg_set_tile_override(bn, cg, 4)          # the forced split is dropped: the consumer is not linear
    C, want, S = run(400, 520, 200, dtype, "relu")
    assert sg.sg_last_tile_choice() == (bn, cg, 1)
    assert_within_bound(C, want, S, f"fused, tile {bn}x{cg}")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_fused_matmul_variants_of_the_consumer(dtype):
    C, want, S = run(200, 136, 72, dtype, "relu", with_bias=False)          # consumer without a bias
    assert_within_bound(C, want, S, "relu only")
    C, want, S = run(200, 136, 72, dtype, "none", with_bias=False)          # no consumer at all: the plain product
    assert_within_bound(C, want, S, "identity")
    C, want, S = run(256, 192, 320, dtype, "relu", dist="ints")             # small integers: exact
    assert np.array_equal(C.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_fused_matmul_on_the_cuda_core_kernel(dtype):
    # layouts outside the TMA rules, a strided or unaligned bias, and the forced family
    C, want, S = run(131, 57, 43, dtype, "relu")
    assert sg.sg_last_kernel_name() == "ffma_kernel"
    assert_within_bound(C, want, S, "ragged extents")
    C, want, S = run(128, 128, 64, dtype, "relu", bias_view=1)              # bias stride 2, base offset 4 bytes
    assert sg.sg_last_kernel_name() == "ffma_kernel"
    assert_within_bound(C, want, S, "strided bias")
    C, want, S = run(300, 200, 136, dtype, "none", family=sg.SG_KERNEL_FFMA)
    assert sg.sg_last_kernel_name() == "ffma_kernel"
    assert_within_bound(C, want, S, "forced family")


def test_fused_matmul_empty_reduction_and_rejections():
    # K = 0: the sum is empty, C = act(bias)
    bias = torch.tensor([1.5, -2.0, 0.0, 3.0, -0.5, 4.0, -4.0, 0.25], device="cuda")
    A = torch.empty(5, 0, device="cuda")
    B = torch.empty(0, 8, device="cuda")
    C = torch.full((5, 8), float("nan"), device="cuda")
    sg.sg_matmul_bias_act(A, B, bias, C, sg.SG_ACT_RELU)
    torch.cuda.synchronize()
    assert torch.equal(C, torch.clamp(bias, min=0).expand(5, 8))
    sg.sg_matmul_bias_act(A, B, bias, C, sg.SG_ACT_NONE)
    torch.cuda.synchronize()
    assert torch.equal(C, bias.expand(5, 8))
    L = sg.lib()
    fake = 4096
    assert L.sg_matmul_bias_act(4, 4, 4, fake, 4, 1, fake, 4, 1, None, 0, 7, fake, 4, 1, sg.SG_F32, None) == 2      # unknown consumer
    assert L.sg_matmul_bias_act(4, 4, 4, fake, 4, 1, fake, 4, 1, fake + 2, 1, 0, fake, 4, 1, sg.SG_F32, None) == 3  # misaligned bias
    assert L.sg_matmul_bias_act(4, 4, 4, fake, 4, 1, fake, 4, 1, fake, -1, 0, fake, 4, 1, sg.SG_F32, None) == 1     # negative stride
    assert L.sg_matmul_bias_act(0, 4, 4, None, 4, 1, None, 4, 1, None, 0, 0, None, 4, 1, sg.SG_F32, None) == 0      # nothing to write


def test_fused_matmul_full_size_sampled():
    M, N, K = 4096, 4096, 1024
    A, a = operand((M, K), SEED, 11, "uniform", "bf16")
    B, b = operand((K, N), SEED, 12, "uniform", "bf16")
    bias, bias_h = operand((N,), SEED, 13, "normal", "f32")
    C = torch.full((M, N), float("nan"), device="cuda")
    sg.sg_matmul_bias_act(A, B, bias, C, sg.SG_ACT_RELU)
    torch.cuda.synchronize()
    assert sg.sg_last_kernel() == sg.SG_KERNEL_TENSOR
    rows = np.unique(np.concatenate([np.arange(0, M, 257), [127, 128, 255, 256, M - 1]]))
    want, S = ref.matmul_bias_act(a[rows], b, bias_h, "relu")
    assert_within_bound(C[torch.from_numpy(rows).cuda()], want, S, "fused 4096x4096x1024, sampled rows")
    assert not torch.isnan(C).any() and (C >= 0).all()
    # a property that holds at any size: the fused result equals relu(unfused product + bias), both from this library
    P = torch.empty(M, N, device="cuda")
    sg.sg_matmul(A, B, P)
    torch.cuda.synchronize()
    assert torch.equal(C, torch.clamp(P + bias, min=0))

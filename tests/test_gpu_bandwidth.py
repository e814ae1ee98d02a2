"""Parity of the memory-bound 2-D kernels (Section 4.4: Copy2D, Transpose2D, ColRed2D, RowRed2D) with
the CPU oracle on the same seeded inputs: bit-exact for the copy and the transpose (they move bit
patterns), |err| <= 1e-4 * sum |a| per output for the reductions (a reduction is a contraction with
a vector of ones, so the contraction bound applies)."""
import numpy as np
import pytest
import torch

from helpers import assert_within_bound, operand
from oracle import ref
from paper_2202_03293_b200 import binding as sg
from paper_2202_03293_b200 import inputs

pytestmark = pytest.mark.gpu
SEED = inputs.BASE_SEED + 80
SENTINEL = {4: 0x7FC0BEEF, 2: 0x7FCB}        # NaN patterns: untouched padding must keep them


def random_bits(shape, esize, tid):
    """Every bit pattern is legal data for a move: NaN payloads, infinities and denormals included."""
    h = inputs._hash(SEED, tid, int(np.prod(shape)), stream=5)
    return (h >> np.uint64(64 - 8 * esize)).astype(np.uint32 if esize == 4 else np.uint16).reshape(shape)


def to_dev(bits):
    t = torch.from_numpy(bits.view(np.int32 if bits.itemsize == 4 else np.int16).copy()).cuda()
    return t.view(torch.float32 if bits.itemsize == 4 else torch.bfloat16)


def dev_bits(t):
    return t.view(torch.int32 if t.element_size() == 4 else torch.int16).cpu().numpy().view(
        np.uint32 if t.element_size() == 4 else np.uint16)


def padded(rows, cols, pitch, esize):
    """Device buffer of `rows` rows `pitch` elements apart, filled with the sentinel; returns (buffer, view)."""
    buf = to_dev(np.full((rows, pitch), SENTINEL[esize], np.uint32 if esize == 4 else np.uint16))
    return buf, buf[:, :cols]


def check_move(op, R, C, esize, src_pitch=None, dst_pitch=None, want_kernel=None):
    src_pitch = src_pitch or C
    n_dr, n_dc = (C, R) if op == "transpose" else (R, C)
    dst_pitch = dst_pitch or n_dc
    bits = random_bits((R, src_pitch), esize, 1)
    src = to_dev(bits)[:, :C]
    buf, dst = padded(n_dr, n_dc, dst_pitch, esize)
    (sg.sg_transpose2d if op == "transpose" else sg.sg_copy2d)(src, dst)
    torch.cuda.synchronize()
    sg.sg_check()
    if want_kernel is not None:
        assert sg.sg_last_kernel() == want_kernel
    want = (ref.transpose2d if op == "transpose" else ref.copy2d)(bits[:, :C])
    got = dev_bits(buf)
    assert np.array_equal(got[:, :n_dc], want), f"{op} {R}x{C} differs"
    assert np.all(got[:, n_dc:] == SENTINEL[esize]), "padding of the destination was written"


def up8(v):
    return (v + 7) // 8 * 8


# the paper's L3-figure size, single rows and columns, sizes spanning several tiles with ragged
# tails in both directions, dense and padded pitches; all meet the TMA rules
@pytest.mark.parametrize("esize", [4, 2])
@pytest.mark.parametrize("op", ["copy", "transpose"])
@pytest.mark.parametrize("R,C,pad", [(250, 960, 0), (1, 8, 0), (8, 1, 0), (129, 257, 8), (1000, 300, 0), (2125, 1064, 16),
                                     (64, 4096, 0), (4096, 64, 0), (513, 8, 8), (3, 700, 0)])
def test_move_tma_path(op, R, C, pad, esize):
    dst_cols = R if op == "transpose" else C
    # rows of the destination shorter than one 16-byte unit leave nothing for the TMA kernel
    want = sg.SG_KERNEL_TMA_MOVE if dst_cols * esize >= 16 else sg.SG_KERNEL_FFMA
    check_move(op, R, C, esize, up8(C) + pad, up8(dst_cols) + pad, want)


# pitches that break the 16-byte rule take the strided kernel
@pytest.mark.parametrize("esize", [4, 2])
@pytest.mark.parametrize("op", ["copy", "transpose"])
@pytest.mark.parametrize("R,C", [(1, 1), (100, 33), (33, 100), (257, 129), (5, 1001)])
def test_move_unaligned_dense(op, R, C, esize):
    dst_cols = R if op == "transpose" else C
    unaligned = (C * esize) % 16 != 0 or (dst_cols * esize) % 16 != 0
    check_move(op, R, C, esize, None, None, sg.SG_KERNEL_FFMA if unaligned else sg.SG_KERNEL_TMA_MOVE)


@pytest.mark.parametrize("esize", [4, 2])
def test_move_strided_views(esize):
    base_bits = random_bits((70, 90), esize, 2)
    base = to_dev(base_bits)
    # column step 3, row step 2; and a column-major source (a transposed view)
    for view, nview in ((base[3:63:2, 1:88:3], base_bits[3:63:2, 1:88:3]), (base.t(), base_bits.T)):
        R, C = view.shape
        dst = to_dev(np.zeros((R, C), base_bits.dtype))
        sg.sg_copy2d(view, dst)
        dst_t = to_dev(np.zeros((C, R), base_bits.dtype))
        sg.sg_transpose2d(view, dst_t)
        torch.cuda.synchronize()
        assert sg.sg_last_kernel() == sg.SG_KERNEL_FFMA
        assert np.array_equal(dev_bits(dst), ref.copy2d(nview))
        assert np.array_equal(dev_bits(dst_t), ref.transpose2d(nview))
    # a strided destination: every other column of a wider buffer
    wide = to_dev(np.full((40, 64), SENTINEL[esize], base_bits.dtype))
    src_bits = random_bits((40, 32), esize, 3)
    sg.sg_copy2d(to_dev(src_bits), wide[:, ::2])
    torch.cuda.synchronize()
    got = dev_bits(wide)
    assert np.array_equal(got[:, ::2], src_bits) and np.all(got[:, 1::2] == SENTINEL[esize])


def test_move_forced_kernels_agree():
    bits = random_bits((300, 200), 4, 4)
    src = to_dev(bits)
    outs = []
    try:
        for fam in (sg.SG_KERNEL_FFMA, sg.SG_KERNEL_TMA_MOVE):
            sg.sg_set_kernel_override(fam)
            dst = to_dev(np.zeros((200, 304), np.uint32))[:, :300]
            sg.sg_transpose2d(src, dst)
            torch.cuda.synchronize()
            assert sg.sg_last_kernel() == fam
            outs.append(dev_bits(dst.contiguous()))
        # the TMA kernel refuses a layout it cannot take instead of falling back
        with pytest.raises(sg.SgError):
            sg.sg_copy2d(src[:, ::2], to_dev(np.zeros((300, 100), np.uint32)))
    finally:
        sg.sg_set_kernel_override(sg.SG_KERNEL_AUTO)
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], ref.transpose2d(bits))


def test_move_empty_and_invalid():
    e = torch.empty((0, 7), device="cuda")
    sg.sg_copy2d(e, torch.empty((0, 7), device="cuda"))
    sg.sg_transpose2d(e, torch.empty((7, 0), device="cuda"))
    with pytest.raises(ValueError):
        sg.sg_transpose2d(torch.zeros((3, 4), device="cuda"), torch.zeros((3, 4), device="cuda"))
    L = sg.lib()
    assert L.sg_copy2d(-1, 4, None, 4, 1, None, 4, 1, sg.SG_F32, None) == 1          # invalid argument
    assert L.sg_copy2d(4, 4, None, 4, 1, None, 4, 1, sg.SG_F32, None) == 1           # null pointers
    assert L.sg_copy2d(4, 4, None, 4, 1, None, 4, 1, 7, None) == 2                   # unknown dtype
    assert L.sg_colred2d(4, 4, None, 4, 1, None, 1, sg.SG_F32, 5, None) == 2         # unknown mode


def run_reduce(op, R, C, dtype, dist="normal", accumulate=False, pitch=None, view=None):
    pitch = pitch or C
    A, a = operand((R, pitch), SEED, 10, dist, dtype)
    A, a = A[:, :C], a[:, :C]
    if view is not None:
        A, a = view(A), view(a)
    n_out = A.shape[1] if op == "col" else A.shape[0]
    if accumulate:
        out, o0 = operand((n_out,), SEED, 11, "uniform", "f32")
        out = out.clone()
    else:
        out, o0 = torch.full((n_out,), float("nan"), device="cuda"), None
    (sg.sg_colred2d if op == "col" else sg.sg_rowred2d)(A, out, sg.SG_ACCUMULATE if accumulate else sg.SG_OVERWRITE)
    torch.cuda.synchronize()
    sg.sg_check()
    want, S = (ref.colred2d if op == "col" else ref.rowred2d)(a, o0)
    if accumulate:
        S = S + np.abs(o0)
    return assert_within_bound(out, want, S, f"{op}red {R}x{C} {dtype}")


# the paper's size, degenerate vectors, tall-skinny and short-wide shapes whose reduced index is
# split across thread blocks, ragged sizes
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["col", "row"])
@pytest.mark.parametrize("R,C", [(250, 960), (1, 1), (1, 5000), (5000, 1), (3000, 2048), (200000, 8), (8, 200000),
                                 (70000, 40), (24, 100000), (1027, 513), (4, 4)])
def test_reductions(op, R, C, dtype):
    pitch = (C + 7) // 8 * 8
    run_reduce(op, R, C, dtype, pitch=pitch)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("op", ["col", "row"])
def test_reductions_accumulate_and_layouts(op, dtype):
    run_reduce(op, 777, 345, dtype, accumulate=True, pitch=352)
    run_reduce(op, 20000, 16, dtype, accumulate=True)                       # split + accumulate: no clearing
    run_reduce(op, 301, 203, dtype)                                          # dense, unaligned pitch: scalar loads
    run_reduce(op, 120, 250, dtype, view=lambda x: x[::2, 1::3])             # strided view
    run_reduce(op, 130, 90, dtype, view=lambda x: x.T if isinstance(x, np.ndarray) else x.t())   # column-major


def test_reductions_exact_on_small_integers():
    # integer data sums exactly in f32: any dropped or doubled element shows
    for op in ("col", "row"):
        assert run_reduce(op, 5000, 520, "f32", dist="ints") == 0.0
        assert run_reduce(op, 64, 30000, "bf16", dist="ints") == 0.0


def test_reductions_empty():
    out = torch.full((6,), 5.0, device="cuda")
    sg.sg_colred2d(torch.empty((0, 6), device="cuda"), out)                   # empty sum -> 0
    assert torch.all(out == 0)
    out = torch.full((3,), 5.0, device="cuda")
    sg.sg_rowred2d(torch.empty((3, 0), device="cuda"), out, sg.SG_ACCUMULATE)
    assert torch.all(out == 5.0)
    sg.sg_rowred2d(torch.empty((0, 9), device="cuda"), torch.empty((0,), device="cuda"))


def test_full_size_moves_sampled():
    """The shape bench.py times (805 MB of f32, larger than L2): rows and columns sampled against the oracle."""
    R, C = 16384, 12288
    bits = random_bits((R, C), 4, 20)
    src = to_dev(bits)
    rows = np.array([0, 1, 127, 128, 4095, 8190, 8191, 8192, 16383])
    cols = np.array([0, 31, 32, 6143, 12287])
    dst = torch.empty_like(src)
    sg.sg_copy2d(src, dst)
    dst_t = torch.empty((C, R), device="cuda")
    sg.sg_transpose2d(src, dst_t)
    torch.cuda.synchronize()
    sg.sg_check()
    assert sg.sg_last_kernel() == sg.SG_KERNEL_TMA_MOVE
    assert np.array_equal(dev_bits(dst[rows]), ref.copy2d(bits[rows]))
    assert np.array_equal(dev_bits(dst[:, cols].contiguous()), ref.copy2d(bits[:, cols]))
    assert np.array_equal(dev_bits(dst_t[:, rows].contiguous()), ref.transpose2d(bits[rows]))
    assert np.array_equal(dev_bits(dst_t[cols]), ref.transpose2d(bits[:, cols]))
    # properties that hold at any size: a copy equals its source, transposing twice returns it
    assert torch.equal(dst.view(torch.int32), src.view(torch.int32))
    back = torch.empty_like(src)
    sg.sg_transpose2d(dst_t, back)
    torch.cuda.synchronize()
    assert torch.equal(back.view(torch.int32), src.view(torch.int32))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_full_size_reductions(dtype):
    R, C = 16384, 12288        # the shape bench.py times
    A, a = operand((R, C), SEED, 21, "uniform", dtype)
    for op, fn, oracle, n_out in (("col", sg.sg_colred2d, ref.colred2d, C), ("row", sg.sg_rowred2d, ref.rowred2d, R)):
        out = torch.full((n_out,), float("nan"), device="cuda")
        fn(A, out)
        torch.cuda.synchronize()
        sg.sg_check()
        want, S = oracle(a)
        assert assert_within_bound(out, want, S, f"{op}red full size {dtype}") < 1e-5


def test_random_shapes_and_pitches():
    """Seeded sweep over small shapes, pitches (aligned and not), dtypes and modes: every kernel path and every
    hand-over between the TMA body and the strided tail gets hit many times."""
    rng = np.random.default_rng(SEED)
    for case in range(60):
        R, C = int(rng.integers(1, 420)), int(rng.integers(1, 420))
        esize = int(rng.choice([2, 4]))
        op = str(rng.choice(["copy", "transpose"]))
        dst_cols = R if op == "transpose" else C
        aligned = bool(rng.integers(0, 2))
        sp = (up8(C) + 8 * int(rng.integers(0, 3))) if aligned else C + int(rng.integers(0, 7))
        dp = (up8(dst_cols) + 8 * int(rng.integers(0, 3))) if aligned else dst_cols + int(rng.integers(0, 7))
        check_move(op, R, C, esize, sp, dp)
    for case in range(60):
        R, C = int(rng.integers(1, 700)), int(rng.integers(1, 700))
        dtype = str(rng.choice(["f32", "bf16"]))
        op = str(rng.choice(["col", "row"]))
        pitch = up8(C) if rng.integers(0, 2) else C + int(rng.integers(0, 5))
        run_reduce(op, R, C, dtype, accumulate=bool(rng.integers(0, 2)), pitch=pitch)


def test_bandwidth_kernel_selection():
    """sg_last_kernel_name names the exact kernel: TMA movers for aligned layouts, the strided mover otherwise; the
    vector or the scalar form of each reduction."""
    src = torch.zeros((256, 512), device="cuda")
    sg.sg_copy2d(src, torch.empty_like(src))
    assert sg.sg_last_kernel_name() == "copy_tma_kernel"
    sg.sg_transpose2d(src, torch.empty((512, 256), device="cuda"))
    assert sg.sg_last_kernel_name() == "transpose_tma_kernel"
    odd = torch.zeros((255, 511), device="cuda")
    sg.sg_copy2d(odd, torch.empty_like(odd))                 # pitch of 511 floats: not a multiple of 16 bytes
    assert sg.sg_last_kernel_name() == "tile_move_kernel"
    sg.sg_transpose2d(src.t(), torch.empty((256, 512), device="cuda"))     # column-major source
    assert sg.sg_last_kernel_name() == "tile_move_kernel"
    for dt in (torch.float32, torch.bfloat16):
        A = torch.ones((300, 512), device="cuda", dtype=dt)
        out_c, out_r = torch.empty(512, device="cuda"), torch.empty(300, device="cuda")
        sg.sg_colred2d(A, out_c)
        assert sg.sg_last_kernel_name() == "colred_kernel<vec>"
        sg.sg_rowred2d(A, out_r)
        assert sg.sg_last_kernel_name() == "rowred_kernel<vec>"
        torch.cuda.synchronize()
        assert torch.all(out_c == 300) and torch.all(out_r == 512)
        B = torch.ones((300, 515), device="cuda", dtype=dt)[:, 1:514]       # unaligned base and pitch
        out_c = torch.empty(513, device="cuda")
        sg.sg_colred2d(B, out_c)
        assert sg.sg_last_kernel_name() == "colred_kernel<scalar>"
        sg.sg_rowred2d(B, out_r)
        assert sg.sg_last_kernel_name() == "rowred_kernel<scalar>"
        torch.cuda.synchronize()
        assert torch.all(out_c == 300) and torch.all(out_r == 513)
    sg.sg_check()

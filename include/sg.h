/*
 * sg.h: C ABI of the structured contraction library for NVIDIA B200 (sm_100a).
 *
 * Three contractions, each defined by a rectangular iteration domain and one
 * indexing map per operand, evaluated on the GPU by hand-written CUDA kernels:
 *
 *   sg_matmul             C[m,n]     (+)= sum_k         A[m,k] * B[k,n]
 *   sg_conv1d_nwc_wcf     O[n,w,f]   (+)= sum_{kw,c}    I[n, w*sw + kw*dw, c] * K[kw,c,f]
 *   sg_conv2d_nhwc_hwcf   O[n,h,w,f] (+)= sum_{kh,kw,c} I[n, h*sh + kh*dh, w*sw + kw*dw, c] * K[kh,kw,c,f]
 *
 * and, declared further down, the memory-bound ops of the same paper: the
 * depthwise convolutions (sg_depthwise_conv1d_nwc_wc, sg_depthwise_conv2d_nhwc_hwc)
 * and the 2-D copy, transpose and row / column reductions (sg_copy2d,
 * sg_transpose2d, sg_colred2d, sg_rowred2d).
 *
 * Conventions common to all entry points (the contraction-specific ones apply
 * to the three ops above)
 *   - Every data pointer is a DEVICE pointer owned by the caller.  Inputs are
 *     read only; the output is written (SG_OVERWRITE) or read and written
 *     (SG_ACCUMULATE).  The output must not overlap an input.
 *   - Strides are in ELEMENTS of the operand's type (the strided-buffer
 *     convention of the paper's memref type, Section 2.2) and need not be
 *     dense.  Negative strides are rejected.  An input stride may be 0 (the
 *     operand is broadcast along that dimension); an output stride of 0
 *     along a dimension of extent > 1 is rejected (SG_ERR_INVALID_ARG): the
 *     output's elements must be distinct.
 *   - `in_dtype` is the element type of BOTH inputs.  The output is always
 *     f32 and products are accumulated in f32 (bf16 inputs are widened
 *     exactly; f32 inputs keep f32 accuracy).
 *   - Calls only enqueue work on `stream` and return; they never synchronise
 *     and never allocate device memory.  The first call on a device creates
 *     small host-side state (driver entry points, kernel attributes); the
 *     tensor-core paths keep a bounded, process-wide cache of encoded tensor
 *     maps keyed by pointer, extents, strides and box (sg_shutdown drops it).
 *   - The return value reports argument and launch errors.  Device-side
 *     pipeline time-outs (which indicate a library bug, not a user error) are
 *     recorded in a per-device status word that sg_check() reads.
 *   - Zero-sized parallel dimensions are a successful no-op.  A zero-sized
 *     reduction zero-fills the output in SG_OVERWRITE mode and leaves it
 *     untouched in SG_ACCUMULATE mode.
 *   - Shapes whose layout allows it (unit stride on the contiguous dimension,
 *     16-byte aligned bases and row pitches) run on the tensor-core path
 *     (TMA + tcgen05): bf16 inputs directly, f32 inputs as three tf32 products
 *     per term (each input split into hi + lo, lo*hi + hi*lo + hi*hi summed in
 *     f32), which keeps f32 accuracy for finite inputs: the error stays below
 *     1e-5 * sum_k |a*b|.  On that f32 path an infinite input gives NaN rather
 *     than a signed infinity.  Everything else runs on a strided CUDA-core
 *     FFMA kernel.  There is no CPU fallback.
 */
#ifndef SG_H_
#define SG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque stand-in for cudaStream_t so that this header needs no CUDA include. */
typedef void *sg_stream_t;

typedef enum {
    SG_OK = 0,
    SG_ERR_INVALID_ARG = 1,    /* null pointer, negative size, stride/dilation < 1, input too small */
    SG_ERR_UNSUPPORTED = 2,    /* unknown dtype or mode, sizes beyond 2^31-1 per dimension         */
    SG_ERR_ALIGNMENT = 3,      /* pointer not aligned to its element size                          */
    SG_ERR_CUDA = 4,           /* a CUDA runtime or driver call failed                             */
    SG_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait expired (reported by sg_check)        */
    SG_ERR_INTERNAL = 6
} sg_status;

typedef enum { SG_F32 = 0, SG_BF16 = 1 } sg_dtype;

enum { SG_OVERWRITE = 0, SG_ACCUMULATE = 1 };

/* Pointwise consumers that sg_matmul_bias_act can fold into the write-back. */
enum { SG_ACT_NONE = 0, SG_ACT_RELU = 1 };

/* Kernel families, for sg_set_kernel_override(). */
enum {
    SG_KERNEL_AUTO = 0,
    SG_KERNEL_FFMA = 1,        /* strided CUDA-core kernel, any layout                                   */
    SG_KERNEL_TENSOR = 2,      /* TMA + tcgen05 implicit GEMM (matmul; convolutions through TMA im2col)  */
    SG_KERNEL_CONV_STRIP = 3,  /* tcgen05 kernel for stride-1 bf16 convolutions: resident filter, each
                                  input pixel fetched once per tile                                      */
    SG_KERNEL_TMA_MOVE = 4     /* copy / transpose that move every tile with TMA loads and stores        */
};

/*
 * Matrix multiplication (paper Section 4.6.1, variant "AB"; iterators
 * (m,n,k) = (parallel, parallel, reduction), maps A:(m,k) B:(k,n) C:(m,n)).
 * The transposed variants of the same section (A^T B, A B^T) are obtained
 * through the stride arguments alone; with 16-byte aligned pitches (and M
 * a multiple of 64 for bf16, 32 for f32, when A is stored [k][m]) they run
 * on the tensor-core path like the plain layout.
 *   A  : M x K elements of in_dtype, element (m,k) at A[m*a_stride_m + k*a_stride_k]
 *   B  : K x N elements of in_dtype, element (k,n) at B[k*b_stride_k + n*b_stride_n]
 *   C  : M x N f32,                  element (m,n) at C[m*c_stride_m + n*c_stride_n]
 *   mode: SG_OVERWRITE  C = A.B ;  SG_ACCUMULATE  C = C_in + A.B  (C is the tied
 *         in/out operand of the destination-passing form, Section 3.4)
 */
sg_status sg_matmul(int64_t M, int64_t N, int64_t K,
                    const void *A, int64_t a_stride_m, int64_t a_stride_k,
                    const void *B, int64_t b_stride_k, int64_t b_stride_n,
                    float *C, int64_t c_stride_m, int64_t c_stride_n,
                    sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * Matrix multiplication with a fused pointwise consumer (the paper fuses tensor operations at the
 * tiled level, Section 2.1; a pointwise op has identity indexing maps and a lower-dimensional
 * operand is broadcast, Section 3.3 items 1 and 2):
 *     C[m,n] = act( sum_k A[m,k] * B[k,n] + bias[n] )
 * i.e. sg_matmul followed by the generic op with maps (m,n)->(m,n), (m,n)->(n), (m,n)->(m,n) and body
 * r = act(p + b), evaluated in the contraction's write-back so that the product never goes to memory.
 *   bias: N f32 values (device), element n at bias[n*bias_stride]; may be NULL (no bias)
 *   act : SG_ACT_NONE (identity) or SG_ACT_RELU (max(., 0)); other values SG_ERR_UNSUPPORTED
 * C is overwritten (there is no accumulating form: the consumer is not linear).  An empty reduction
 * (K = 0) writes act(bias[n]).  A, B, C, in_dtype, stream as for sg_matmul; the sum is accumulated in
 * f32, bias added and act applied in f32.  With a unit bias stride and a 16-byte aligned bias the call
 * takes the tensor-core path where sg_matmul would (one work item per tile: a split reduction or a
 * stream-K tail cannot apply a non-linear consumer to partial sums); otherwise the CUDA-core kernel.
 */
sg_status sg_matmul_bias_act(int64_t M, int64_t N, int64_t K,
                             const void *A, int64_t a_stride_m, int64_t a_stride_k,
                             const void *B, int64_t b_stride_k, int64_t b_stride_n,
                             const float *bias, int64_t bias_stride, int act,
                             float *C, int64_t c_stride_m, int64_t c_stride_n,
                             sg_dtype in_dtype, sg_stream_t stream);

/*
 * 1-D convolution, input layout NWC, filter layout WCF, output NWF
 * (index notation of Section 3; strided/dilated form of Section 4.6.2, "(1-D)").
 * Iteration domain 0<=n<N, 0<=w<W_out, 0<=f<F, 0<=kw<KW, 0<=c<C; the filter
 * is not flipped and nothing is padded: the call is rejected unless
 * W_in >= (W_out-1)*stride_w + (KW-1)*dilation_w + 1.  Input columns beyond
 * that are not read.
 *   I : N x W_in x C,   strides i_strides[3] = {n, w, c}
 *   Kf: KW x C x F,     strides k_strides[3] = {kw, c, f}
 *   O : N x W_out x F,  strides o_strides[3] = {n, w, f}   (f32)
 */
sg_status sg_conv1d_nwc_wcf(int64_t N, int64_t W_out, int64_t F, int64_t KW, int64_t C,
                            int64_t W_in, int64_t stride_w, int64_t dilation_w,
                            const void *I, const int64_t i_strides[3],
                            const void *Kf, const int64_t k_strides[3],
                            float *O, const int64_t o_strides[3],
                            sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * 2-D convolution, input NHWC, filter HWCF, output NHWF (Section 4.6.2, "(2-D)").
 * Iteration domain (n,h,w,f,kh,kw,c); same rules as the 1-D op in both
 * spatial dimensions.
 *   I : N x H_in x W_in x C,    strides {n, h, w, c}
 *   Kf: KH x KW x C x F,        strides {kh, kw, c, f}
 *   O : N x H_out x W_out x F,  strides {n, h, w, f}   (f32)
 */
sg_status sg_conv2d_nhwc_hwcf(int64_t N, int64_t H_out, int64_t W_out, int64_t F,
                              int64_t KH, int64_t KW, int64_t C, int64_t H_in, int64_t W_in,
                              int64_t stride_h, int64_t stride_w,
                              int64_t dilation_h, int64_t dilation_w,
                              const void *I, const int64_t i_strides[4],
                              const void *Kf, const int64_t k_strides[4],
                              float *O, const int64_t o_strides[4],
                              sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * Depthwise 2-D convolution, input NHWC, filter HWC, output NHWC (Section 4.6.3, "(2-D)"):
 *   O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*sh + kh*dh, w*sw + kw*dw, c] * K[kh,kw,c]
 * Iterators (n,h,w,c,kh,kw): the channel iterator is parallel, only the window is reduced.
 * Same rules as the dense convolutions (no padding, filter not flipped, input large enough
 * or SG_ERR_INVALID_ARG, strides in elements).  The op is bound by memory bandwidth and runs
 * on the CUDA cores: four channels per thread when channels are contiguous in all three
 * tensors, C is a multiple of 4 and pointers and pitches allow 16-byte (f32) / 8-byte (bf16)
 * accesses; one element per thread otherwise.
 *   I : N x H_in x W_in x C,    strides {n, h, w, c}
 *   Kf: KH x KW x C,            strides {kh, kw, c}
 *   O : N x H_out x W_out x C,  strides {n, h, w, c}   (f32)
 */
sg_status sg_depthwise_conv2d_nhwc_hwc(int64_t N, int64_t H_out, int64_t W_out, int64_t C, int64_t KH, int64_t KW,
                                       int64_t H_in, int64_t W_in, int64_t stride_h, int64_t stride_w,
                                       int64_t dilation_h, int64_t dilation_w,
                                       const void *I, const int64_t i_strides[4],
                                       const void *Kf, const int64_t k_strides[3],
                                       float *O, const int64_t o_strides[4],
                                       sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * Depthwise 1-D convolution, input NWC, filter WC, output NWC (Section 4.6.3, "(1-D)"):
 *   O[n,w,c] (+)= sum_kw I[n, w*sw + kw*dw, c] * K[kw,c]
 * The 2-D op with H = KH = 1.   I strides {n, w, c}; Kf strides {kw, c}; O strides {n, w, c}.
 */
sg_status sg_depthwise_conv1d_nwc_wc(int64_t N, int64_t W_out, int64_t C, int64_t KW, int64_t W_in,
                                     int64_t stride_w, int64_t dilation_w,
                                     const void *I, const int64_t i_strides[3],
                                     const void *Kf, const int64_t k_strides[2],
                                     float *O, const int64_t o_strides[3],
                                     sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * The memory-bound 2-D kernels (Section 4.4, "Benchmarks": Copy2D, Transpose2D, ColRed2D,
 * RowRed2D; measured in Section 4.5).  All operate on an R x C tensor whose element (i,j) is at
 * base[i*stride_r + j*stride_c] (strides in elements, any non-negative values); R and C up to
 * 2^31 - 2^20 (SG_ERR_UNSUPPORTED beyond).
 *
 * Copy2D:       dst[i,j] = src[i,j]        dst is R x C
 * Transpose2D:  dst[j,i] = src[i,j]        dst is C x R; dst_stride_r is the pitch of ITS rows
 *                                          (index j), dst_stride_c the step along i
 * Elements are moved as bit patterns of `dtype`'s size (4 bytes for SG_F32, 2 for SG_BF16);
 * nothing is converted.  dst must not overlap src.  With unit column strides, 16-byte aligned
 * bases and row pitches that are multiples of 16 bytes the call runs on TMA-only kernels
 * (SG_KERNEL_TMA_MOVE); any other layout runs on a strided CUDA-core kernel.
 */
sg_status sg_copy2d(int64_t R, int64_t C, const void *src, int64_t src_stride_r, int64_t src_stride_c,
                    void *dst, int64_t dst_stride_r, int64_t dst_stride_c, sg_dtype dtype, sg_stream_t stream);
sg_status sg_transpose2d(int64_t R, int64_t C, const void *src, int64_t src_stride_r, int64_t src_stride_c,
                         void *dst, int64_t dst_stride_r, int64_t dst_stride_c, sg_dtype dtype, sg_stream_t stream);

/*
 * ColRed2D:  out[j] (+)= sum_i A[i,j]   C outputs (the row index is reduced)
 * RowRed2D:  out[i] (+)= sum_j A[i,j]   R outputs (the column index is reduced)
 * The caption of the paper's L3 bandwidth figure fixes the naming: for a 250 x 960 tensor the
 * row reduction writes 250 values, the column reduction 960.  A holds `in_dtype` elements, the
 * sums are accumulated and written in f32 (bf16 inputs are widened exactly); out[k] is at
 * out[k*out_stride].  mode as for the contractions; an empty reduction writes 0 (SG_OVERWRITE)
 * or leaves out untouched (SG_ACCUMULATE).  When the shape has too few outputs to occupy the
 * GPU the reduced index is split across thread blocks whose partial sums are added into `out`
 * with float atomics, so the rounding of the last bits may differ from call to call.
 * `out` must not overlap A.
 */
sg_status sg_colred2d(int64_t R, int64_t C, const void *A, int64_t a_stride_r, int64_t a_stride_c,
                      float *out, int64_t out_stride, sg_dtype in_dtype, int mode, sg_stream_t stream);
sg_status sg_rowred2d(int64_t R, int64_t C, const void *A, int64_t a_stride_r, int64_t a_stride_c,
                      float *out, int64_t out_stride, sg_dtype in_dtype, int mode, sg_stream_t stream);

/*
 * Synchronises `stream` and returns the current device's status word:
 * SG_OK, SG_ERR_DEVICE_TIMEOUT if any kernel since the last sg_check gave up
 * on a bounded wait (its output is then undefined), or SG_ERR_CUDA if the
 * synchronisation itself failed.  Reading clears the word.
 */
sg_status sg_check(sg_stream_t stream);

/* Static, NUL-terminated description of a status code. */
const char *sg_status_string(sg_status status);

/* Library version, major*10000 + minor*100 + patch. */
int sg_version(void);

/*
 * Which kernel family the most recent successful call on this host thread
 * selected: SG_KERNEL_FFMA (any CUDA-core kernel), SG_KERNEL_TENSOR, SG_KERNEL_CONV_STRIP or
 * SG_KERNEL_TMA_MOVE (0 before any call).
 */
int sg_last_kernel(void);

/*
 * Name of the compute kernel that call launched (a static string, "" before any call; clearing
 * kernels launched ahead of it are not named): "tc_gemm_kernel<bf16>", "tc_gemm_kernel<f32>",
 * "conv_strip_kernel<bf16>", "conv_strip_kernel<f32>", "ffma_kernel", "depthwise_tma_kernel",
 * "depthwise_roll_kernel", "depthwise_vec_kernel", "depthwise_generic_kernel", "copy_tma_kernel",
 * "transpose_tma_kernel", "tile_move_kernel", "colred_kernel<vec>", "colred_kernel<scalar>",
 * "rowred_kernel<vec>", "rowred_kernel<scalar>".  For tests and benchmarks.
 */
const char *sg_last_kernel_name(void);

/*
 * Number of kernels this library has launched in this process so far
 * (monotonic, all threads).  Used by benchmarks to report launch counts.
 */
int64_t sg_launch_count(void);

/*
 * Force a kernel family for later calls on this process (testing and
 * benchmarking): SG_KERNEL_AUTO restores the default selection (the
 * convolution kernel where it applies, else the tensor-core GEMM, else the
 * CUDA-core kernel).  Forcing SG_KERNEL_TENSOR or SG_KERNEL_CONV_STRIP makes
 * calls that kernel cannot take return SG_ERR_UNSUPPORTED instead of falling
 * back.  For sg_copy2d / sg_transpose2d, SG_KERNEL_FFMA forces the strided kernel and
 * SG_KERNEL_TMA_MOVE the TMA kernel (SG_ERR_UNSUPPORTED when the layout rules it out).
 */
sg_status sg_set_kernel_override(int kernel_family);

/*
 * Tensor-core path only, for testing and benchmarking: force the output tile width (64, 128
 * or 256 columns), the number of CTAs that share a tile (1, or 2 = a CTA pair working on 256
 * rows) and the number of contiguous k ranges a tile's reduction is dealt out in (partial
 * sums then meet in the output by reduce-add; an overwriting call clears the output first).
 * 0 leaves a choice to the library's cost estimate.  A combination that does not exist (256
 * columns on one CTA with f32 inputs) or does not fit the shape falls back to that estimate.
 * Returns SG_ERR_INVALID_ARG for other values.  The environment variables SG_TC_BN, SG_TC_CG
 * and SG_TC_SPLIT, read at the first call, set the same three values.
 */
sg_status sg_set_tile_override(int tile_n, int ctas_per_tile, int k_splits);

/* {tile width, CTAs per tile, k ranges} of the most recent tensor-core launch made by this host thread. */
void sg_last_tile_choice(int out[3]);

/*
 * Stream-K tail of the most recent tensor-core launch made by this host thread: when whole tiles are dealt out and the last
 * wave of tiles would be partly filled, the tiles of that wave are cut along the reduction instead (every CTA or CTA
 * pair gets an equal run of their k-blocks; the partial sums meet in the output by reduce-add).  out[0] = index of
 * the first tile of the tail in the tile order (-1: no tail), out[1] = k-blocks per run.  SG_TC_SK=0 in the
 * environment (read at the first call) turns the tail off.
 */
void sg_last_stream_k(int out[2]);

/*
 * Tensor-map cache counters since the library was loaded: out[0] = look-ups answered from the
 * cache, out[1] = look-ups that had to encode a map.  The cache is keyed by device, base pointer,
 * element type, extents, byte strides, box and the other encode parameters, never by the
 * memory's contents; it holds at most 2048 maps (about 0.7 MB of host memory), replacing the
 * least recently used entry of a full bucket.
 */
void sg_tensor_map_cache_stats(int64_t out[2]);

/*
 * Self-test of the device-side time-out path (the paper has no counterpart): launches one warp
 * that waits `budget_cycles` SM clock cycles (1e3 .. 2e7, i.e. at most about 10 ms) on a barrier
 * that nothing signals, then gives up exactly as a pipeline wait of the kernels above would: it
 * sets the device status word and returns normally.  The next sg_check() on that device reports
 * SG_ERR_DEVICE_TIMEOUT once and clears the word.  Nothing traps and nothing spins past the budget.
 */
sg_status sg_selftest_wait_timeout(int64_t budget_cycles, sg_stream_t stream);

/*
 * Environment switches, all for testing and benchmarking, all read once at the first tensor-core
 * call of the process:
 *   SG_TC_BN, SG_TC_CG, SG_TC_SPLIT   as sg_set_tile_override
 *   SG_TC_SK        0: never cut the last wave into a stream-K tail; 2: whenever the shape allows it
 *   SG_TC_KPS       1: one k-block per pipeline stage everywhere (bf16 matmuls normally move two)
 *   SG_TC_TA        0: keep the split f32 input tile in shared memory instead of tensor memory
 *   SG_TC_PDL       0: tensor-core launches never start before the kernel ahead of them in the
 *                   stream has finished (by default they set themselves up while it drains and
 *                   wait for it before their first global read or write)
 *   SG_CONV_SINGLE  1: the stride-1 convolution kernel never uses CTA pairs
 */

/* Drops cached tensor maps and other host-side state.  Safe to call twice. */
void sg_shutdown(void);

#ifdef __cplusplus
}
#endif
#endif /* SG_H_ */

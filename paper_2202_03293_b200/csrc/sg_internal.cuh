// Shared declarations of the CUDA side of the library (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sg.h"

namespace sg {

// Every op is run as one implicit GEMM  O[m, f] (+)= sum_k  In(m, k) * Flt(k, f)  with
//   m = (n, h, w)  flattened over the output's batch and spatial iterators,
//   k = (kh, kw, c) flattened over the reduction iterators,
// and operand addresses that separate into a row part and a reduction part:
//   In (m,k) at  n*i_n + (h*sh + kh*dh)*i_h + (w*sw + kw*dw)*i_w + c*i_c
//   Flt(k,f) at  kh*k_kh + kw*k_kw + c*k_c + f*k_f
//   O  (m,f) at  n*o_n + h*o_h + w*o_w + f*o_f
// A matmul is the case Ho = KH = KW = 1, batch 1, Wo = M, C = K (a 1x1 filter).
struct Problem {
    int M, N, K;             // GEMM extents: M = batch*Ho*Wo, N = F, K = KH*KW*C
    int batch, Ho, Wo;       // decomposition of m
    int KH, KW, C;           // decomposition of k
    int Hin, Win;            // input spatial extents (bounds of the im2col box)
    int sh, sw, dh, dw;      // strides and dilations of the window
    int64_t i_n, i_h, i_w, i_c;
    int64_t k_kh, k_kw, k_c, k_f;
    int64_t o_n, o_h, o_w, o_f;
    int in_bf16;             // 1: inputs are bf16, 0: f32
    int accumulate;          // 1: O = O_in + result
    int spatial_rank;        // 0 matmul, 1 conv1d, 2 conv2d
    // fused pointwise consumer of the write-back (overwrite mode only): O = act(acc + bias[f])
    const float *bias;       // f32 vector over f (device), or null
    int64_t bias_f;          // its element stride
    int act;                 // SG_ACT_NONE or SG_ACT_RELU
};

// Launchers (each returns the cudaError_t of its launch).
cudaError_t launch_ffma(const Problem &p, const void *In, const void *Flt, float *O,
                        cudaStream_t stream);
cudaError_t launch_zero_fill(const Problem &p, float *O, cudaStream_t stream);

// Tensor-core path: returns SG_ERR_UNSUPPORTED (and launches nothing) when the layout
// does not satisfy the TMA rules.
sg_status launch_tensor(const Problem &p, const void *In, const void *Flt, float *O,
                        cudaStream_t stream);
void tensor_shutdown();
// One warp that waits `budget_cycles` on a barrier nobody signals, then reports the time-out like any pipeline wait.
cudaError_t launch_wait_timeout_selftest(long long budget_cycles, cudaStream_t stream);
// Driver entry points resolved by the tensor path, for the other tensor-core kernels: whether the
// current device is usable (and its SM count), and a tiled tensor-map encoder (interleave none,
// element strides 1, out-of-bounds elements read as zero).  Call with no library lock held.
bool tensor_driver_ready(int *num_sms);
// The current device's index and SM count plus two test switches (SG_TC_PDL, SG_CONV_SINGLE); false when the device is unusable.
bool tensor_device_info(int *device, int *num_sms, int *pdl, int *conv_single);
// Raises a kernel's dynamic shared-memory limit once per device; `slot` (144..159 for callers outside the GEMM file)
// names the kernel instantiation.
bool tensor_ensure_smem_attr(int slot, const void *kernel, int bytes);
bool tensor_encode_tiled(CUtensorMap *map, CUtensorMapDataType type, int rank, void *base, const cuuint64_t *dims,
                         const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle,
                         CUtensorMapL2promotion promotion);
// Stride-1 bf16 convolutions with a resident filter (sg_conv.cu): SG_ERR_UNSUPPORTED when the
// shape or layout does not qualify (nothing is launched then).
sg_status launch_conv_strip(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream);
sg_status conv_read_status(cudaStream_t stream);
void tensor_set_tile_override(int bn, int cg, int splits);
void tensor_last_choice(int out[3]);
void tensor_map_cache_stats(long long out[2]);     // {hits, misses} since the library was loaded
void tensor_last_stream_k(int out[2]);
// Reads and clears the current device's status word (written by kernels whose bounded
// waits expire); the caller has already synchronised the stream.
sg_status tensor_read_status(cudaStream_t stream);

// Depthwise convolution (Section 4.6.3): O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*sh+kh*dh, w*sw+kw*dw, c] * K[kh,kw,c].
struct DepthwiseProblem {
    int N, Ho, Wo, C, KH, KW;
    int sh, sw, dh, dw;
    int64_t i_n, i_h, i_w, i_c;
    int64_t k_kh, k_kw, k_c;
    int64_t o_n, o_h, o_w, o_c;
    int in_bf16, accumulate;
};
cudaError_t launch_depthwise(const DepthwiseProblem &p, const void *I, const void *Kf, float *O, cudaStream_t stream);
sg_status depthwise_read_status(cudaStream_t stream);

// The memory-bound 2-D kernels (Section 4.4).  launch_move2d: dst[i,j] = src[i,j], or dst[j,i] = src[i,j] when
// `transpose`; elements of `esize` (2 or 4) bytes, strides in elements; `force` 0 picks, 1 = strided kernel only, 2 = TMA
// kernel or SG_ERR_UNSUPPORTED; *used_tma reports whether the TMA kernels ran.
// launch_reduce2d: out[j] (+)= sum_i A[i,j] when `colred`, else out[i] (+)= sum_j A[i,j].
sg_status launch_move2d(bool transpose, int64_t R, int64_t C, const void *src, int64_t s_r, int64_t s_c, void *dst, int64_t d_r,
                        int64_t d_c, int esize, int force, int *used_tma, cudaStream_t stream);
sg_status launch_reduce2d(bool colred, int64_t R, int64_t C, const void *A, int64_t a_r, int64_t a_c, int in_bf16, float *out,
                          int64_t os, int accumulate, cudaStream_t stream);
sg_status bandwidth_read_status(cudaStream_t stream);

void count_launch(int n = 1);
// Records the name of the compute kernel a call launched (a static string), for sg_last_kernel_name().
void note_kernel(const char *name);

}  // namespace sg

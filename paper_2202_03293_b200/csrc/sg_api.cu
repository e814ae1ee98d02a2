// C ABI entry points: argument validation, the implicit-GEMM view of each op, kernel selection.
#include <atomic>
#include <limits>

#include "sg_internal.cuh"

namespace sg {
namespace {

std::atomic<int64_t> g_launches{0};
std::atomic<int> g_override{SG_KERNEL_AUTO};
thread_local int t_last_kernel = 0;
thread_local const char *t_last_kernel_name = "";

constexpr int64_t kMaxDim = std::numeric_limits<int32_t>::max();

inline bool fits(int64_t v) { return v >= 0 && v <= kMaxDim; }
constexpr int64_t kTileSlack = 1 << 20;   // head room for extents rounded up to tiles or split ranges

sg_status run(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream) {
    if (p.M == 0 || p.N == 0) return SG_OK;                       // nothing to write
    if (p.K == 0 && (p.bias != nullptr || p.act != SG_ACT_NONE)) {
        // empty reduction under a fused consumer: act(bias), written by the CUDA-core kernel's write-back
        if (launch_ffma(p, In, Flt, O, stream) != cudaSuccess) return SG_ERR_CUDA;
        t_last_kernel = SG_KERNEL_FFMA;
        return SG_OK;
    }
    if (p.K == 0) {                                               // empty reduction: the sum is 0
        if (p.accumulate) return SG_OK;
        return launch_zero_fill(p, O, stream) == cudaSuccess ? SG_OK : SG_ERR_CUDA;
    }
    const int force = g_override.load();
    if (force == SG_KERNEL_AUTO || force == SG_KERNEL_CONV_STRIP) {
        // stride-1 bf16 convolutions whose filter fits in shared memory
        sg_status st = launch_conv_strip(p, In, Flt, O, stream);
        if (st == SG_OK) { t_last_kernel = SG_KERNEL_CONV_STRIP; return SG_OK; }
        if (st != SG_ERR_UNSUPPORTED || force == SG_KERNEL_CONV_STRIP) return st;
    }
    if (force != SG_KERNEL_FFMA) {
        sg_status st = launch_tensor(p, In, Flt, O, stream);
        if (st == SG_OK) { t_last_kernel = SG_KERNEL_TENSOR; return SG_OK; }
        if (st != SG_ERR_UNSUPPORTED || force == SG_KERNEL_TENSOR) return st;
    }
    if (launch_ffma(p, In, Flt, O, stream) != cudaSuccess) return SG_ERR_CUDA;
    t_last_kernel = SG_KERNEL_FFMA;
    return SG_OK;
}

sg_status check_common(const void *a, const void *b, const void *o, sg_dtype dt, int mode) {
    if (dt != SG_F32 && dt != SG_BF16) return SG_ERR_UNSUPPORTED;
    if (mode != SG_OVERWRITE && mode != SG_ACCUMULATE) return SG_ERR_UNSUPPORTED;
    const uintptr_t es = dt == SG_BF16 ? 2 : 4;
    if (a && reinterpret_cast<uintptr_t>(a) % es) return SG_ERR_ALIGNMENT;
    if (b && reinterpret_cast<uintptr_t>(b) % es) return SG_ERR_ALIGNMENT;
    if (o && reinterpret_cast<uintptr_t>(o) % 4) return SG_ERR_ALIGNMENT;
    return SG_OK;
}

}  // namespace

void count_launch(int n) { g_launches.fetch_add(n); }
void note_kernel(const char *name) { t_last_kernel_name = name; }

}  // namespace sg

using namespace sg;

extern "C" {

sg_status sg_matmul(int64_t M, int64_t N, int64_t K, const void *A, int64_t a_stride_m, int64_t a_stride_k,
                    const void *B, int64_t b_stride_k, int64_t b_stride_n, float *C, int64_t c_stride_m,
                    int64_t c_stride_n, sg_dtype in_dtype, int mode, sg_stream_t stream) {
    if (M < 0 || N < 0 || K < 0) return SG_ERR_INVALID_ARG;
    sg_status st = check_common(A, B, C, in_dtype, mode);
    if (st != SG_OK) return st;
    if (!fits(M) || !fits(N) || !fits(K)) return SG_ERR_UNSUPPORTED;
    const bool has_out = M > 0 && N > 0;
    if (has_out && !C) return SG_ERR_INVALID_ARG;
    if (has_out && K > 0 && (!A || !B)) return SG_ERR_INVALID_ARG;
    if (a_stride_m < 0 || a_stride_k < 0 || b_stride_k < 0 || b_stride_n < 0 || c_stride_m < 0 || c_stride_n < 0)
        return SG_ERR_INVALID_ARG;
    if ((M > 1 && c_stride_m == 0) || (N > 1 && c_stride_n == 0)) return SG_ERR_INVALID_ARG;   // output elements would coincide
    Problem p{};
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.batch = 1; p.Ho = 1; p.Wo = (int)M;
    p.KH = 1; p.KW = 1; p.C = (int)K;
    p.Hin = 1; p.Win = (int)M;
    p.sh = p.sw = p.dh = p.dw = 1;
    p.i_n = 0; p.i_h = 0; p.i_w = a_stride_m; p.i_c = a_stride_k;
    p.k_kh = 0; p.k_kw = 0; p.k_c = b_stride_k; p.k_f = b_stride_n;
    p.o_n = 0; p.o_h = 0; p.o_w = c_stride_m; p.o_f = c_stride_n;
    p.in_bf16 = in_dtype == SG_BF16; p.accumulate = mode == SG_ACCUMULATE; p.spatial_rank = 0;
    return run(p, A, B, C, static_cast<cudaStream_t>(stream));
}

sg_status sg_matmul_bias_act(int64_t M, int64_t N, int64_t K, const void *A, int64_t a_stride_m, int64_t a_stride_k,
                             const void *B, int64_t b_stride_k, int64_t b_stride_n, const float *bias, int64_t bias_stride,
                             int act, float *C, int64_t c_stride_m, int64_t c_stride_n, sg_dtype in_dtype, sg_stream_t stream) {
    if (M < 0 || N < 0 || K < 0) return SG_ERR_INVALID_ARG;
    sg_status st = check_common(A, B, C, in_dtype, SG_OVERWRITE);
    if (st != SG_OK) return st;
    if (act != SG_ACT_NONE && act != SG_ACT_RELU) return SG_ERR_UNSUPPORTED;
    if (bias && reinterpret_cast<uintptr_t>(bias) % 4) return SG_ERR_ALIGNMENT;
    if (!fits(M) || !fits(N) || !fits(K)) return SG_ERR_UNSUPPORTED;
    const bool has_out = M > 0 && N > 0;
    if (has_out && !C) return SG_ERR_INVALID_ARG;
    if (has_out && K > 0 && (!A || !B)) return SG_ERR_INVALID_ARG;
    if (a_stride_m < 0 || a_stride_k < 0 || b_stride_k < 0 || b_stride_n < 0 || c_stride_m < 0 || c_stride_n < 0 || bias_stride < 0)
        return SG_ERR_INVALID_ARG;
    if ((M > 1 && c_stride_m == 0) || (N > 1 && c_stride_n == 0)) return SG_ERR_INVALID_ARG;
    Problem p{};
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.batch = 1; p.Ho = 1; p.Wo = (int)M;
    p.KH = 1; p.KW = 1; p.C = (int)K;
    p.Hin = 1; p.Win = (int)M;
    p.sh = p.sw = p.dh = p.dw = 1;
    p.i_n = 0; p.i_h = 0; p.i_w = a_stride_m; p.i_c = a_stride_k;
    p.k_kh = 0; p.k_kw = 0; p.k_c = b_stride_k; p.k_f = b_stride_n;
    p.o_n = 0; p.o_h = 0; p.o_w = c_stride_m; p.o_f = c_stride_n;
    p.in_bf16 = in_dtype == SG_BF16; p.accumulate = 0; p.spatial_rank = 0;
    p.bias = bias; p.bias_f = bias_stride; p.act = act;
    return run(p, A, B, C, static_cast<cudaStream_t>(stream));
}

sg_status sg_conv1d_nwc_wcf(int64_t N, int64_t W_out, int64_t F, int64_t KW, int64_t C, int64_t W_in,
                            int64_t stride_w, int64_t dilation_w, const void *I, const int64_t i_strides[3],
                            const void *Kf, const int64_t k_strides[3], float *O, const int64_t o_strides[3],
                            sg_dtype in_dtype, int mode, sg_stream_t stream) {
    if (N < 0 || W_out < 0 || F < 0 || KW < 0 || C < 0 || W_in < 0) return SG_ERR_INVALID_ARG;
    if (stride_w < 1 || dilation_w < 1) return SG_ERR_INVALID_ARG;
    if (!i_strides || !k_strides || !o_strides) return SG_ERR_INVALID_ARG;
    sg_status st = check_common(I, Kf, O, in_dtype, mode);
    if (st != SG_OK) return st;
    for (int i = 0; i < 3; ++i)
        if (i_strides[i] < 0 || k_strides[i] < 0 || o_strides[i] < 0) return SG_ERR_INVALID_ARG;
    if ((N > 1 && o_strides[0] == 0) || (W_out > 1 && o_strides[1] == 0) || (F > 1 && o_strides[2] == 0)) return SG_ERR_INVALID_ARG;
    if (!fits(N) || !fits(W_out) || !fits(F) || !fits(KW) || !fits(C) || !fits(W_in) || !fits(stride_w) ||
        !fits(dilation_w)) return SG_ERR_UNSUPPORTED;
    if (W_out > 0 && KW > 0 && W_in < (W_out - 1) * stride_w + (KW - 1) * dilation_w + 1) return SG_ERR_INVALID_ARG;
    if (!fits(N * W_out) || !fits(KW * C)) return SG_ERR_UNSUPPORTED;
    const bool has_out = N > 0 && W_out > 0 && F > 0;
    if (has_out && !O) return SG_ERR_INVALID_ARG;
    if (has_out && KW * C > 0 && (!I || !Kf)) return SG_ERR_INVALID_ARG;
    Problem p{};
    p.M = (int)(N * W_out); p.N = (int)F; p.K = (int)(KW * C);
    p.batch = (int)N; p.Ho = 1; p.Wo = (int)W_out;
    p.KH = 1; p.KW = (int)KW; p.C = (int)C;
    p.Hin = 1; p.Win = (int)W_in;
    p.sh = 1; p.sw = (int)stride_w; p.dh = 1; p.dw = (int)dilation_w;
    p.i_n = i_strides[0]; p.i_h = 0; p.i_w = i_strides[1]; p.i_c = i_strides[2];
    p.k_kh = 0; p.k_kw = k_strides[0]; p.k_c = k_strides[1]; p.k_f = k_strides[2];
    p.o_n = o_strides[0]; p.o_h = 0; p.o_w = o_strides[1]; p.o_f = o_strides[2];
    p.in_bf16 = in_dtype == SG_BF16; p.accumulate = mode == SG_ACCUMULATE; p.spatial_rank = 1;
    return run(p, I, Kf, O, static_cast<cudaStream_t>(stream));
}

sg_status sg_conv2d_nhwc_hwcf(int64_t N, int64_t H_out, int64_t W_out, int64_t F, int64_t KH, int64_t KW, int64_t C,
                              int64_t H_in, int64_t W_in, int64_t stride_h, int64_t stride_w, int64_t dilation_h,
                              int64_t dilation_w, const void *I, const int64_t i_strides[4], const void *Kf,
                              const int64_t k_strides[4], float *O, const int64_t o_strides[4], sg_dtype in_dtype,
                              int mode, sg_stream_t stream) {
    if (N < 0 || H_out < 0 || W_out < 0 || F < 0 || KH < 0 || KW < 0 || C < 0 || H_in < 0 || W_in < 0)
        return SG_ERR_INVALID_ARG;
    if (stride_h < 1 || stride_w < 1 || dilation_h < 1 || dilation_w < 1) return SG_ERR_INVALID_ARG;
    if (!i_strides || !k_strides || !o_strides) return SG_ERR_INVALID_ARG;
    sg_status st = check_common(I, Kf, O, in_dtype, mode);
    if (st != SG_OK) return st;
    for (int i = 0; i < 4; ++i)
        if (i_strides[i] < 0 || k_strides[i] < 0 || o_strides[i] < 0) return SG_ERR_INVALID_ARG;
    if ((N > 1 && o_strides[0] == 0) || (H_out > 1 && o_strides[1] == 0) || (W_out > 1 && o_strides[2] == 0) ||
        (F > 1 && o_strides[3] == 0)) return SG_ERR_INVALID_ARG;
    if (!fits(N) || !fits(H_out) || !fits(W_out) || !fits(F) || !fits(KH) || !fits(KW) || !fits(C) || !fits(H_in) ||
        !fits(W_in) || !fits(stride_h) || !fits(stride_w) || !fits(dilation_h) || !fits(dilation_w))
        return SG_ERR_UNSUPPORTED;
    if (H_out > 0 && KH > 0 && H_in < (H_out - 1) * stride_h + (KH - 1) * dilation_h + 1) return SG_ERR_INVALID_ARG;
    if (W_out > 0 && KW > 0 && W_in < (W_out - 1) * stride_w + (KW - 1) * dilation_w + 1) return SG_ERR_INVALID_ARG;
    if (!fits(H_out * W_out) || !fits(N * H_out * W_out) || !fits(KH * KW) || !fits(KH * KW * C))
        return SG_ERR_UNSUPPORTED;
    const bool has_out = N > 0 && H_out > 0 && W_out > 0 && F > 0;
    if (has_out && !O) return SG_ERR_INVALID_ARG;
    if (has_out && KH * KW * C > 0 && (!I || !Kf)) return SG_ERR_INVALID_ARG;
    Problem p{};
    p.M = (int)(N * H_out * W_out); p.N = (int)F; p.K = (int)(KH * KW * C);
    p.batch = (int)N; p.Ho = (int)H_out; p.Wo = (int)W_out;
    p.KH = (int)KH; p.KW = (int)KW; p.C = (int)C;
    p.Hin = (int)H_in; p.Win = (int)W_in;
    p.sh = (int)stride_h; p.sw = (int)stride_w; p.dh = (int)dilation_h; p.dw = (int)dilation_w;
    p.i_n = i_strides[0]; p.i_h = i_strides[1]; p.i_w = i_strides[2]; p.i_c = i_strides[3];
    p.k_kh = k_strides[0]; p.k_kw = k_strides[1]; p.k_c = k_strides[2]; p.k_f = k_strides[3];
    p.o_n = o_strides[0]; p.o_h = o_strides[1]; p.o_w = o_strides[2]; p.o_f = o_strides[3];
    p.in_bf16 = in_dtype == SG_BF16; p.accumulate = mode == SG_ACCUMULATE; p.spatial_rank = 2;
    return run(p, I, Kf, O, static_cast<cudaStream_t>(stream));
}

sg_status sg_depthwise_conv2d_nhwc_hwc(int64_t N, int64_t H_out, int64_t W_out, int64_t C, int64_t KH, int64_t KW,
                                       int64_t H_in, int64_t W_in, int64_t stride_h, int64_t stride_w,
                                       int64_t dilation_h, int64_t dilation_w, const void *I, const int64_t i_strides[4],
                                       const void *Kf, const int64_t k_strides[3], float *O, const int64_t o_strides[4],
                                       sg_dtype in_dtype, int mode, sg_stream_t stream) {
    if (N < 0 || H_out < 0 || W_out < 0 || C < 0 || KH < 0 || KW < 0 || H_in < 0 || W_in < 0) return SG_ERR_INVALID_ARG;
    if (stride_h < 1 || stride_w < 1 || dilation_h < 1 || dilation_w < 1) return SG_ERR_INVALID_ARG;
    if (!i_strides || !k_strides || !o_strides) return SG_ERR_INVALID_ARG;
    sg_status st = check_common(I, Kf, O, in_dtype, mode);
    if (st != SG_OK) return st;
    for (int i = 0; i < 4; ++i)
        if (i_strides[i] < 0 || o_strides[i] < 0 || (i < 3 && k_strides[i] < 0)) return SG_ERR_INVALID_ARG;
    if ((N > 1 && o_strides[0] == 0) || (H_out > 1 && o_strides[1] == 0) || (W_out > 1 && o_strides[2] == 0) ||
        (C > 1 && o_strides[3] == 0)) return SG_ERR_INVALID_ARG;
    if (!fits(N) || !fits(H_out) || !fits(W_out) || !fits(C) || !fits(KH) || !fits(KW) || !fits(H_in) || !fits(W_in) ||
        !fits(stride_h) || !fits(stride_w) || !fits(dilation_h) || !fits(dilation_w)) return SG_ERR_UNSUPPORTED;
    if (H_out > 0 && KH > 0 && H_in < (H_out - 1) * stride_h + (KH - 1) * dilation_h + 1) return SG_ERR_INVALID_ARG;
    if (W_out > 0 && KW > 0 && W_in < (W_out - 1) * stride_w + (KW - 1) * dilation_w + 1) return SG_ERR_INVALID_ARG;
    if (!fits(H_in * stride_h) || !fits(W_in * stride_w) || !fits(KH * KW)) return SG_ERR_UNSUPPORTED;
    const bool has_out = N > 0 && H_out > 0 && W_out > 0 && C > 0;
    if (!has_out) return SG_OK;
    if (!O) return SG_ERR_INVALID_ARG;
    if (KH * KW > 0 && (!I || !Kf)) return SG_ERR_INVALID_ARG;
    if (KH * KW == 0 && mode == SG_ACCUMULATE) return SG_OK;      // empty window: the sum is 0
    DepthwiseProblem p{};
    p.N = (int)N; p.Ho = (int)H_out; p.Wo = (int)W_out; p.C = (int)C; p.KH = (int)KH; p.KW = (int)KW;
    p.sh = (int)stride_h; p.sw = (int)stride_w; p.dh = (int)dilation_h; p.dw = (int)dilation_w;
    p.i_n = i_strides[0]; p.i_h = i_strides[1]; p.i_w = i_strides[2]; p.i_c = i_strides[3];
    p.k_kh = k_strides[0]; p.k_kw = k_strides[1]; p.k_c = k_strides[2];
    p.o_n = o_strides[0]; p.o_h = o_strides[1]; p.o_w = o_strides[2]; p.o_c = o_strides[3];
    p.in_bf16 = in_dtype == SG_BF16; p.accumulate = mode == SG_ACCUMULATE;
    if (launch_depthwise(p, I, Kf, O, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SG_ERR_CUDA;
    t_last_kernel = SG_KERNEL_FFMA;     // a CUDA-core kernel
    return SG_OK;
}

sg_status sg_depthwise_conv1d_nwc_wc(int64_t N, int64_t W_out, int64_t C, int64_t KW, int64_t W_in, int64_t stride_w,
                                     int64_t dilation_w, const void *I, const int64_t i_strides[3], const void *Kf,
                                     const int64_t k_strides[2], float *O, const int64_t o_strides[3], sg_dtype in_dtype,
                                     int mode, sg_stream_t stream) {
    if (!i_strides || !k_strides || !o_strides) return SG_ERR_INVALID_ARG;
    // the 1-D op is the 2-D op with H = KH = 1 (Section 4.6.3)
    const int64_t is4[4] = {i_strides[0], 0, i_strides[1], i_strides[2]};
    const int64_t ks3[3] = {0, k_strides[0], k_strides[1]};
    const int64_t os4[4] = {o_strides[0], 0, o_strides[1], o_strides[2]};
    return sg_depthwise_conv2d_nhwc_hwc(N, 1, W_out, C, 1, KW, 1, W_in, 1, stride_w, 1, dilation_w, I, is4, Kf, ks3, O, os4,
                                        in_dtype, mode, stream);
}

namespace {
sg_status move2d(bool transpose, int64_t R, int64_t C, const void *src, int64_t s_r, int64_t s_c, void *dst, int64_t d_r, int64_t d_c,
                 sg_dtype dtype, sg_stream_t stream) {
    using namespace sg;
    if (dtype != SG_F32 && dtype != SG_BF16) return SG_ERR_UNSUPPORTED;
    if (R < 0 || C < 0 || s_r < 0 || s_c < 0 || d_r < 0 || d_c < 0) return SG_ERR_INVALID_ARG;
    if (!fits(R + kTileSlack) || !fits(C + kTileSlack)) return SG_ERR_UNSUPPORTED;   // tile coordinates stay in int32
    if (R == 0 || C == 0) return SG_OK;
    if (!src || !dst) return SG_ERR_INVALID_ARG;
    // destination elements must not coincide (dst is R x C for a copy, C x R for a transpose)
    if (((transpose ? C : R) > 1 && d_r == 0) || ((transpose ? R : C) > 1 && d_c == 0)) return SG_ERR_INVALID_ARG;
    const int es = dtype == SG_BF16 ? 2 : 4;
    if (reinterpret_cast<uintptr_t>(src) % es || reinterpret_cast<uintptr_t>(dst) % es) return SG_ERR_ALIGNMENT;
    const int ov = g_override.load();
    const int force = ov == SG_KERNEL_FFMA ? 1 : (ov == SG_KERNEL_TMA_MOVE ? 2 : 0);
    int used_tma = 0;
    const sg_status st = launch_move2d(transpose, R, C, src, s_r, s_c, dst, d_r, d_c, es, force, &used_tma, static_cast<cudaStream_t>(stream));
    if (st == SG_OK) t_last_kernel = used_tma ? SG_KERNEL_TMA_MOVE : SG_KERNEL_FFMA;
    return st;
}

sg_status reduce2d(bool colred, int64_t R, int64_t C, const void *A, int64_t a_r, int64_t a_c, float *out, int64_t out_stride,
                   sg_dtype in_dtype, int mode, sg_stream_t stream) {
    using namespace sg;
    sg_status st = check_common(A, nullptr, out, in_dtype, mode);
    if (st != SG_OK) return st;
    if (R < 0 || C < 0 || a_r < 0 || a_c < 0 || out_stride < 0) return SG_ERR_INVALID_ARG;
    if (!fits(R + kTileSlack) || !fits(C + kTileSlack)) return SG_ERR_UNSUPPORTED;   // rounded-up split ranges stay in int32
    const int64_t n_out = colred ? C : R, n_red = colred ? R : C;
    if (n_out == 0) return SG_OK;
    if (!out || (n_red > 0 && !A)) return SG_ERR_INVALID_ARG;
    if (n_out > 1 && out_stride == 0) return SG_ERR_INVALID_ARG;      // output elements would coincide
    if (n_red == 0 && mode == SG_ACCUMULATE) return SG_OK;
    st = launch_reduce2d(colred, R, C, A, a_r, a_c, in_dtype == SG_BF16, out, out_stride, mode == SG_ACCUMULATE,
                         static_cast<cudaStream_t>(stream));
    if (st == SG_OK) t_last_kernel = SG_KERNEL_FFMA;     // CUDA-core kernels
    return st;
}
}  // namespace

sg_status sg_copy2d(int64_t R, int64_t C, const void *src, int64_t src_stride_r, int64_t src_stride_c, void *dst,
                    int64_t dst_stride_r, int64_t dst_stride_c, sg_dtype dtype, sg_stream_t stream) {
    return move2d(false, R, C, src, src_stride_r, src_stride_c, dst, dst_stride_r, dst_stride_c, dtype, stream);
}

sg_status sg_transpose2d(int64_t R, int64_t C, const void *src, int64_t src_stride_r, int64_t src_stride_c, void *dst,
                         int64_t dst_stride_r, int64_t dst_stride_c, sg_dtype dtype, sg_stream_t stream) {
    return move2d(true, R, C, src, src_stride_r, src_stride_c, dst, dst_stride_r, dst_stride_c, dtype, stream);
}

sg_status sg_colred2d(int64_t R, int64_t C, const void *A, int64_t a_stride_r, int64_t a_stride_c, float *out, int64_t out_stride,
                      sg_dtype in_dtype, int mode, sg_stream_t stream) {
    return reduce2d(true, R, C, A, a_stride_r, a_stride_c, out, out_stride, in_dtype, mode, stream);
}

sg_status sg_rowred2d(int64_t R, int64_t C, const void *A, int64_t a_stride_r, int64_t a_stride_c, float *out, int64_t out_stride,
                      sg_dtype in_dtype, int mode, sg_stream_t stream) {
    return reduce2d(false, R, C, A, a_stride_r, a_stride_c, out, out_stride, in_dtype, mode, stream);
}

sg_status sg_check(sg_stream_t stream) {
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return SG_ERR_CUDA;
    return tensor_read_status(s);
}

const char *sg_status_string(sg_status status) {
    switch (status) {
        case SG_OK: return "ok";
        case SG_ERR_INVALID_ARG: return "invalid argument";
        case SG_ERR_UNSUPPORTED: return "unsupported dtype, mode, size or layout";
        case SG_ERR_ALIGNMENT: return "pointer not aligned to its element size";
        case SG_ERR_CUDA: return "CUDA runtime or driver call failed";
        case SG_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case SG_ERR_INTERNAL: return "internal error";
    }
    return "unknown status";
}

int sg_version(void) { return 200; }   // 0.2.0: depthwise convolutions and the memory-bound 2-D kernels joined the three contractions

int sg_last_kernel(void) { return t_last_kernel; }

const char *sg_last_kernel_name(void) { return t_last_kernel_name; }

int64_t sg_launch_count(void) { return g_launches.load(); }

sg_status sg_set_kernel_override(int kernel_family) {
    if (kernel_family != SG_KERNEL_AUTO && kernel_family != SG_KERNEL_FFMA && kernel_family != SG_KERNEL_TENSOR &&
        kernel_family != SG_KERNEL_CONV_STRIP && kernel_family != SG_KERNEL_TMA_MOVE)
        return SG_ERR_INVALID_ARG;
    g_override.store(kernel_family);
    return SG_OK;
}

sg_status sg_set_tile_override(int tile_n, int ctas_per_tile, int k_splits) {
    if (tile_n != 0 && tile_n != 64 && tile_n != 128 && tile_n != 256) return SG_ERR_INVALID_ARG;
    if (ctas_per_tile < 0 || ctas_per_tile > 2 || k_splits < 0 || k_splits > 64) return SG_ERR_INVALID_ARG;
    tensor_set_tile_override(tile_n, ctas_per_tile, k_splits);
    return SG_OK;
}

void sg_last_tile_choice(int out[3]) {
    if (out) tensor_last_choice(out);
}

void sg_last_stream_k(int out[2]) {
    if (out) sg::tensor_last_stream_k(out);
}

void sg_tensor_map_cache_stats(int64_t out[2]) {
    if (!out) return;
    long long v[2];
    tensor_map_cache_stats(v);
    out[0] = v[0]; out[1] = v[1];
}

sg_status sg_selftest_wait_timeout(int64_t budget_cycles, sg_stream_t stream) {
    if (budget_cycles < 1000 || budget_cycles > 20000000) return SG_ERR_INVALID_ARG;    // at most ~10 ms of spinning
    return launch_wait_timeout_selftest((long long)budget_cycles, static_cast<cudaStream_t>(stream)) == cudaSuccess ? SG_OK : SG_ERR_CUDA;
}

void sg_shutdown(void) { tensor_shutdown(); }

}  // extern "C"

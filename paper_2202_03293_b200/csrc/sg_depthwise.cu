// Depthwise convolutions (Section 4.6.3): O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*Sh+kh*Dh, w*Sw+kw*Dw, c] * K[kh,kw,c].
//
// The channel iterator is parallel, only the window is reduced: KH*KW multiply-adds per output
// element against at least one element read and one written, so the op is bound by HBM
// bandwidth and runs on the CUDA cores.  The fast kernel gives each thread four consecutive
// channels (one 16-byte access; consecutive threads take consecutive channel groups, so a warp
// reads and writes whole lines) of TW consecutive output columns; for the 3 x 3 window with unit
// stride and dilation along w the input columns the TW windows share are loaded once into
// registers, otherwise every tap is loaded where it is needed and the L1 serves the repeats.  Any other layout (channel strides
// other than 1, channel counts that are not a multiple of 4, unaligned pointers or pitches)
// takes a one-output-per-thread kernel with full stride arithmetic.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sg_internal.cuh"

namespace sg {
namespace {

constexpr int TW = 4;            // output columns per thread in the fast kernel

__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p) {
    const uint2 raw = *reinterpret_cast<const uint2 *>(p);
    // bf16 -> f32 is a 16-bit shift: exact
    return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xFFFF0000u),
                       __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xFFFF0000u));
}
__device__ __forceinline__ float load1(const float *p) { return *p; }
__device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

__device__ __forceinline__ void fma4(float4 &acc, const float4 a, const float4 b) {
    acc.x = fmaf(a.x, b.x, acc.x); acc.y = fmaf(a.y, b.y, acc.y);
    acc.z = fmaf(a.z, b.z, acc.z); acc.w = fmaf(a.w, b.w, acc.w);
}

// Four channels x TW output columns per thread.  UNIT: stride 1, dilation 1 along w and KW <= MAX_KW_REG.
// K3: a 3 x 3 window with unit stride and dilation along w, known at compile time: the columns
// the TW windows of a filter row share (w0 .. w0+TW+1) are loaded once, and all 18 input loads
// of a thread are issued before the first of them is needed.  Otherwise every tap is loaded
// where it is needed and the L1 serves the repeats.
// IDX: the type the work index is decoded in (32-bit whenever the work fits: 64-bit divisions
// would cost more than the op).  One work item per thread.
template <typename T, bool K3, typename IDX>
__global__ void __launch_bounds__(256)
depthwise_vec_kernel(const DepthwiseProblem p, const T *__restrict__ I, const T *__restrict__ Kf, float *__restrict__ O) {
    const IDX c4s = (IDX)(p.C / 4);
    const IDX wts = (IDX)((p.Wo + TW - 1) / TW);
    const IDX total = (IDX)p.N * (IDX)p.Ho * wts * c4s;
    const IDX idx = (IDX)blockIdx.x * 256 + threadIdx.x;
    if (idx < total) {
        const int c = (int)(idx % c4s) * 4;
        IDX r = idx / c4s;
        const int w0 = (int)(r % wts) * TW;
        r /= wts;
        const int h = (int)(r % (IDX)p.Ho), n = (int)(r / (IDX)p.Ho);
        float4 acc[TW];
#pragma unroll
        for (int t = 0; t < TW; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        const T *in_n = I + (int64_t)n * p.i_n + c;
        if constexpr (K3) {
            float4 col[3][TW + 2];
#pragma unroll
            for (int kh = 0; kh < 3; ++kh) {
                const T *row = in_n + (int64_t)(h * p.sh + kh * p.dh) * p.i_h;
#pragma unroll
                for (int j = 0; j < TW + 2; ++j)
                    if (w0 + j < p.Wo + 2) col[kh][j] = load4(row + (int64_t)(w0 + j) * p.i_w);
            }
#pragma unroll
            for (int kh = 0; kh < 3; ++kh)
#pragma unroll
                for (int kw = 0; kw < 3; ++kw) {
                    const float4 f = load4(Kf + (int64_t)kh * p.k_kh + (int64_t)kw * p.k_kw + c);
#pragma unroll
                    for (int t = 0; t < TW; ++t)
                        if (w0 + t < p.Wo) fma4(acc[t], col[kh][t + kw], f);
                }
        } else {
            for (int kh = 0; kh < p.KH; ++kh) {
                const T *row = in_n + (int64_t)(h * p.sh + kh * p.dh) * p.i_h;
                const T *frow = Kf + (int64_t)kh * p.k_kh + c;
                for (int kw = 0; kw < p.KW; ++kw) {
                    const float4 f = load4(frow + (int64_t)kw * p.k_kw);
#pragma unroll
                    for (int t = 0; t < TW; ++t)
                        if (w0 + t < p.Wo) fma4(acc[t], load4(row + (int64_t)((w0 + t) * p.sw + kw * p.dw) * p.i_w), f);
                }
            }
        }
        float *out = O + (int64_t)n * p.o_n + (int64_t)h * p.o_h + c;
#pragma unroll
        for (int t = 0; t < TW; ++t) {
            if (w0 + t >= p.Wo) break;
            float4 *o = reinterpret_cast<float4 *>(out + (int64_t)(w0 + t) * p.o_w);
            float4 v = acc[t];
            if (p.accumulate) {
                const float4 old = *o;
                v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
            }
            *o = v;
        }
    }
}

// Any strides: one output element per thread.
template <typename T, typename IDX>
__global__ void __launch_bounds__(256)
depthwise_generic_kernel(const DepthwiseProblem p, const T *__restrict__ I, const T *__restrict__ Kf, float *__restrict__ O) {
    const IDX total = (IDX)p.N * (IDX)p.Ho * (IDX)p.Wo * (IDX)p.C;
    const IDX idx = (IDX)blockIdx.x * 256 + threadIdx.x;
    if (idx < total) {
        const int c = (int)(idx % (IDX)p.C);
        IDX r = idx / (IDX)p.C;
        const int w = (int)(r % (IDX)p.Wo);
        r /= (IDX)p.Wo;
        const int h = (int)(r % (IDX)p.Ho), n = (int)(r / (IDX)p.Ho);
        float acc = 0.f;
        for (int kh = 0; kh < p.KH; ++kh)
            for (int kw = 0; kw < p.KW; ++kw)
                acc = fmaf(load1(I + (int64_t)n * p.i_n + (int64_t)(h * p.sh + kh * p.dh) * p.i_h +
                                 (int64_t)(w * p.sw + kw * p.dw) * p.i_w + (int64_t)c * p.i_c),
                           load1(Kf + (int64_t)kh * p.k_kh + (int64_t)kw * p.k_kw + (int64_t)c * p.k_c), acc);
        float *o = O + (int64_t)n * p.o_n + (int64_t)h * p.o_h + (int64_t)w * p.o_w + (int64_t)c * p.o_c;
        *o = p.accumulate ? *o + acc : acc;
    }
}

inline bool mult4(int64_t v) { return v % 4 == 0; }

template <typename T>
cudaError_t launch_typed(const DepthwiseProblem &p, const T *I, const T *Kf, float *O, cudaStream_t stream) {
    const bool vec = p.i_c == 1 && p.k_c == 1 && p.o_c == 1 && p.C % 4 == 0 &&
                     mult4(p.i_n) && mult4(p.i_h) && mult4(p.i_w) && mult4(p.k_kh) && mult4(p.k_kw) &&
                     mult4(p.o_n) && mult4(p.o_h) && mult4(p.o_w) &&
                     reinterpret_cast<uintptr_t>(I) % (4 * sizeof(T)) == 0 && reinterpret_cast<uintptr_t>(Kf) % (4 * sizeof(T)) == 0 &&
                     reinterpret_cast<uintptr_t>(O) % 16 == 0;
    const int64_t work = vec ? (int64_t)p.N * p.Ho * ((p.Wo + TW - 1) / TW) * (p.C / 4) : (int64_t)p.N * p.Ho * p.Wo * p.C;
    const int64_t blocks64 = (work + 255) / 256;
    if (blocks64 > 0x7fffffff) return cudaErrorInvalidConfiguration;
    const unsigned blocks = (unsigned)blocks64;
    const bool small = work < ((int64_t)1 << 32) - 256;
    const bool unit3 = p.sw == 1 && p.dw == 1 && p.KW == 3 && p.KH == 3;
#define SG_DW(KERNEL) KERNEL<<<blocks, 256, 0, stream>>>(p, I, Kf, O)
    if (vec && unit3) { if (small) SG_DW((depthwise_vec_kernel<T, true, uint32_t>)); else SG_DW((depthwise_vec_kernel<T, true, uint64_t>)); }
    else if (vec) { if (small) SG_DW((depthwise_vec_kernel<T, false, uint32_t>)); else SG_DW((depthwise_vec_kernel<T, false, uint64_t>)); }
    else { if (small) SG_DW((depthwise_generic_kernel<T, uint32_t>)); else SG_DW((depthwise_generic_kernel<T, uint64_t>)); }
#undef SG_DW
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_depthwise(const DepthwiseProblem &p, const void *I, const void *Kf, float *O, cudaStream_t stream) {
    if (p.in_bf16)
        return launch_typed(p, static_cast<const __nv_bfloat16 *>(I), static_cast<const __nv_bfloat16 *>(Kf), O, stream);
    return launch_typed(p, static_cast<const float *>(I), static_cast<const float *>(Kf), O, stream);
}

}  // namespace sg

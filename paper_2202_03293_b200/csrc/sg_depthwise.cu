// Depthwise convolutions (Section 4.6.3): O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*Sh+kh*Dh, w*Sw+kw*Dw, c] * K[kh,kw,c].
//
// The channel iterator is parallel, only the window is reduced: KH*KW multiply-adds per output
// element against at least one element read and one written, so the op is bound by HBM
// bandwidth and runs on the CUDA cores.  The fast kernel gives each thread four consecutive
// channels (one 16-byte access; consecutive threads take consecutive channel groups, so a warp
// reads and writes whole lines) of TW consecutive output columns; with unit stride and dilation
// the input columns the TW windows share are loaded once into registers, otherwise every tap is
// loaded where it is needed and the L1 serves the repeats.  Any other layout (channel strides
// other than 1, channel counts that are not a multiple of 4, unaligned pointers or pitches)
// takes a one-output-per-thread kernel with full stride arithmetic.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sg_internal.cuh"

namespace sg {
namespace {

constexpr int TW = 4;            // output columns per thread in the fast kernel
constexpr int MAX_KW_REG = 7;    // widest window row kept in registers

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
template <typename T, bool UNIT>
__global__ void __launch_bounds__(256)
depthwise_vec_kernel(const DepthwiseProblem p, const T *__restrict__ I, const T *__restrict__ Kf, float *__restrict__ O) {
    const int c4s = p.C / 4;
    const int wts = (p.Wo + TW - 1) / TW;
    const int64_t total = (int64_t)p.N * p.Ho * wts * c4s;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % c4s) * 4;
        int64_t r = idx / c4s;
        const int w0 = (int)(r % wts) * TW;
        r /= wts;
        const int h = (int)(r % p.Ho), n = (int)(r / p.Ho);
        float4 acc[TW];
#pragma unroll
        for (int t = 0; t < TW; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        const T *in_n = I + (int64_t)n * p.i_n + c;
        for (int kh = 0; kh < p.KH; ++kh) {
            const T *row = in_n + (int64_t)(h * p.sh + kh * p.dh) * p.i_h;
            const T *frow = Kf + (int64_t)kh * p.k_kh + c;
            if constexpr (UNIT) {
                // the TW windows cover columns w0 .. w0+TW+KW-2: each is loaded once
                float4 col[TW + MAX_KW_REG - 1];
#pragma unroll
                for (int j = 0; j < TW + MAX_KW_REG - 1; ++j)
                    if (j < TW + p.KW - 1 && w0 + j < p.Wo + p.KW - 1) col[j] = load4(row + (int64_t)(w0 + j) * p.i_w);
#pragma unroll
                for (int kw = 0; kw < MAX_KW_REG; ++kw) {
                    if (kw < p.KW) {
                        const float4 f = load4(frow + (int64_t)kw * p.k_kw);
#pragma unroll
                        for (int t = 0; t < TW; ++t)
                            if (w0 + t < p.Wo) fma4(acc[t], col[t + kw], f);
                    }
                }
            } else {
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
template <typename T>
__global__ void __launch_bounds__(256)
depthwise_generic_kernel(const DepthwiseProblem p, const T *__restrict__ I, const T *__restrict__ Kf, float *__restrict__ O) {
    const int64_t total = (int64_t)p.N * p.Ho * p.Wo * p.C;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % p.C);
        int64_t r = idx / p.C;
        const int w = (int)(r % p.Wo);
        r /= p.Wo;
        const int h = (int)(r % p.Ho), n = (int)(r / p.Ho);
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
    const int64_t want = (work + 255) / 256;
    const int blocks = (int)(want < 148 * 32 ? want : 148 * 32);
    if (vec) {
        if (p.sw == 1 && p.dw == 1 && p.KW <= MAX_KW_REG) depthwise_vec_kernel<T, true><<<blocks, 256, 0, stream>>>(p, I, Kf, O);
        else depthwise_vec_kernel<T, false><<<blocks, 256, 0, stream>>>(p, I, Kf, O);
    } else {
        depthwise_generic_kernel<T><<<blocks, 256, 0, stream>>>(p, I, Kf, O);
    }
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

// Depthwise convolutions (Section 4.6.3): O[n,h,w,c] (+)= sum_{kh,kw} I[n, h*Sh+kh*Dh, w*Sw+kw*Dw, c] * K[kh,kw,c].
//
// The channel iterator is parallel, only the window is reduced: KH*KW multiply-adds per output
// element against at least one element read and one written, so the op is bound by HBM
// bandwidth and runs on the CUDA cores.  The fast kernel gives each thread four consecutive
// channels (one 16-byte access; consecutive threads take consecutive channel groups, so a warp
// reads and writes whole lines) of TW consecutive output columns; for the 3 x 3 window with unit
// stride and dilation along w the input columns the TW windows share are loaded once into
// registers, otherwise every tap is loaded where it is needed and the L1 serves the repeats.
// Large 3 x 3 / unit-stride problems take one of two kernels that fetch every input element about
// 1.5 times instead of 4.5: a TMA-staged tile kernel (layouts that meet the TMA rules) or a
// kernel that walks down the rows with a rolling register window.  Any other layout (channel
// strides other than 1, channel counts that are not a multiple of 4, unaligned pointers or
// pitches) takes a one-output-per-thread kernel with full stride arithmetic.
#include <algorithm>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sg_internal.cuh"
#include "sg_tc_ptx.cuh"

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

// 3 x 3 window, unit stride and dilation along w and h, large problems: a thread owns four channels of TW output
// columns and walks down ROLL_ROWS output rows, keeping the three input rows of the window in registers.  Each step loads
// ONE new input row (TW+2 sixteen-byte loads) instead of three, so an input element is fetched 1.5 (columns) x
// (ROLL_ROWS+2)/ROLL_ROWS (rows) times from L1/L2 instead of 4.5 times; the six multiply-adds per output that use the two
// rows already held run while the new row is in flight.  The row buffers rotate by role (compile-time indices), not by copy.
#ifndef SG_DW_ROLL_TW
#define SG_DW_ROLL_TW 4
#endif
#ifndef SG_DW_ROLL_BLOCK
#define SG_DW_ROLL_BLOCK 128
#endif
#ifndef SG_DW_ROLL_MINB
#define SG_DW_ROLL_MINB 3
#endif
#ifndef SG_DW_ROLL_ROWS
#define SG_DW_ROLL_ROWS 8
#endif
constexpr int ROLL_ROWS = SG_DW_ROLL_ROWS;      // output rows a thread walks down
constexpr int ROLL_TW = SG_DW_ROLL_TW;          // output columns per thread
constexpr int ROLL_BLOCK = SG_DW_ROLL_BLOCK;    // threads per block

template <typename T, int R>
__device__ __forceinline__ void roll_step(const DepthwiseProblem &p, const T *in_col, float *out_col, int h, int w0,
                                          uint32_t flt_smem, uint32_t flt_pitch, float4 (&col)[3][ROLL_TW + 2]) {
    // rows h and h+1 sit in col[R % 3] and col[(R + 1) % 3]; row h+2 goes to col[(R + 2) % 3]
    const T *row = in_col + (int64_t)(h + 2) * p.i_h;
#pragma unroll
    for (int j = 0; j < ROLL_TW + 2; ++j)
        if (w0 + j < p.Wo + 2) col[(R + 2) % 3][j] = load4(row + (int64_t)j * p.i_w);
    float4 acc[ROLL_TW];
#pragma unroll
    for (int t = 0; t < ROLL_TW; ++t) acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int kh = 0; kh < 3; ++kh)
#pragma unroll
        for (int kw = 0; kw < 3; ++kw) {
            // the thread's four filter values of this tap, from shared memory (volatile: re-read every step
            // rather than held in 36 registers for the whole walk)
            float4 f;
            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(f.x), "=f"(f.y), "=f"(f.z), "=f"(f.w)
                         : "r"(flt_smem + (uint32_t)(kh * 3 + kw) * flt_pitch));
#pragma unroll
            for (int t = 0; t < ROLL_TW; ++t) fma4(acc[t], col[(R + kh) % 3][t + kw], f);
        }
    float *out = out_col + (int64_t)h * p.o_h;
#pragma unroll
    for (int t = 0; t < ROLL_TW; ++t) {
        if (w0 + t >= p.Wo) break;
        float4 *o = reinterpret_cast<float4 *>(out + (int64_t)t * p.o_w);
        float4 v = acc[t];
        if (p.accumulate) {
            const float4 old = *o;
            v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
        }
        *o = v;
    }
}

template <typename T>
__global__ void __launch_bounds__(ROLL_BLOCK, SG_DW_ROLL_MINB)
depthwise_roll_kernel(const DepthwiseProblem p, const T *__restrict__ I, const T *__restrict__ Kf, float *__restrict__ O) {
    const uint32_t c4s = (uint32_t)(p.C / 4);
    const uint32_t wts = (uint32_t)((p.Wo + ROLL_TW - 1) / ROLL_TW);
    const uint32_t hts = (uint32_t)((p.Ho + ROLL_ROWS - 1) / ROLL_ROWS);
    const uint32_t total = (uint32_t)p.N * hts * wts * c4s;
    // the whole filter as f32 in shared memory: [tap][channel]
    extern __shared__ float4 flt_shared[];
    float *sflt = reinterpret_cast<float *>(flt_shared);
    for (int i = threadIdx.x; i < 9 * p.C; i += ROLL_BLOCK) {
        const int tap = i / p.C, ch = i - tap * p.C;
        sflt[i] = load1(Kf + (int64_t)(tap / 3) * p.k_kh + (int64_t)(tap % 3) * p.k_kw + ch);
    }
    __syncthreads();
    const uint32_t idx = blockIdx.x * (uint32_t)ROLL_BLOCK + threadIdx.x;
    if (idx >= total) return;
    const int c = (int)(idx % c4s) * 4;
    uint32_t r = idx / c4s;
    const int w0 = (int)(r % wts) * ROLL_TW;
    r /= wts;
    const int h0 = (int)(r % hts) * ROLL_ROWS, n = (int)(r / hts);
    const int h1 = min(p.Ho, h0 + ROLL_ROWS);
    const uint32_t flt_smem = (uint32_t)__cvta_generic_to_shared(sflt + c), flt_pitch = (uint32_t)p.C * 4u;
    const T *in_col = I + (int64_t)n * p.i_n + (int64_t)w0 * p.i_w + c;
    float *out_col = O + (int64_t)n * p.o_n + (int64_t)w0 * p.o_w + c;
    float4 col[3][ROLL_TW + 2];
#pragma unroll
    for (int k = 0; k < 2; ++k)
#pragma unroll
        for (int j = 0; j < ROLL_TW + 2; ++j)
            if (w0 + j < p.Wo + 2) col[k][j] = load4(in_col + (int64_t)(h0 + k) * p.i_h + (int64_t)j * p.i_w);
    int h = h0;
    for (; h + 2 < h1; h += 3) {
        roll_step<T, 0>(p, in_col, out_col, h, w0, flt_smem, flt_pitch, col);
        roll_step<T, 1>(p, in_col, out_col, h + 1, w0, flt_smem, flt_pitch, col);
        roll_step<T, 2>(p, in_col, out_col, h + 2, w0, flt_smem, flt_pitch, col);
    }
    if (h < h1) roll_step<T, 0>(p, in_col, out_col, h, w0, flt_smem, flt_pitch, col);
    if (h + 1 < h1) roll_step<T, 1>(p, in_col, out_col, h + 1, w0, flt_smem, flt_pitch, col);
}

// 3 x 3 window, unit strides and dilations, layouts that meet the TMA rules, problems of at least one tile per SM:
// the input tile of a CTA (DT_ROWS+2 rows x TWB+2 columns x CB channels, halo included) is fetched by ONE tensor load
// into a two-stage shared-memory ring, so the fetch of the next tile runs while this one is computed and an input
// element crosses L2 -> SM about 1.4 times instead of 4.5.  256 compute threads: thread (column wl, channel group cg)
// walks down the DT_ROWS output rows of its column with the 3 x 3 window of float4 in registers (three new
// shared-memory reads per output, conflict-free: a warp reads whole contiguous pixels) and stores its outputs
// straight from registers (a warp writes whole pixels).  Warp 8 is the producer.
constexpr int DT_THREADS = 256 + 32;

// S: stride along h and w (1 or 2).  A tile is ROWS output rows x TWB output columns x CB channels.
template <typename T, int CB, int S>
struct DtCfg {
    static constexpr int CG = CB / 4;                 // channel groups (threads) per pixel
    static constexpr int TWB = 256 / CG;              // output columns per tile
    static constexpr int ROWS = S == 1 ? 8 : 2;       // output rows per tile
    static constexpr int IN_W = (TWB - 1) * S + 3, IN_H = (ROWS - 1) * S + 3;
    static constexpr int PIXEL_BYTES = CB * (int)sizeof(T);
    static constexpr int BOX_BYTES = PIXEL_BYTES * IN_W * IN_H;
    static constexpr int STAGE_BYTES = (BOX_BYTES + 127) / 128 * 128;
};

__device__ __forceinline__ float4 lds4(uint32_t addr, float) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 lds4(uint32_t addr, __nv_bfloat16) {
    uint32_t a, b;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(a), "=r"(b) : "r"(addr));
    return make_float4(__uint_as_float(a << 16), __uint_as_float(a & 0xFFFF0000u), __uint_as_float(b << 16), __uint_as_float(b & 0xFFFF0000u));
}

// The grid is a multiple of c_blocks (or smaller than it never), so a CTA keeps one channel block
// for all its tiles and a thread loads its nine filter values once.
template <typename T, int CB, int S>
__global__ void __launch_bounds__(DT_THREADS)
depthwise_tma_kernel(const __grid_constant__ CUtensorMap map_in, const DepthwiseProblem p, const T *__restrict__ Kf,
                     float *__restrict__ O, int tiles_w, int tiles_h, int c_blocks, int num_tiles) {
    using C = DtCfg<T, CB, S>;
    extern __shared__ uint8_t dt_smem[];
    __shared__ uint64_t full_bar[2], empty_bar[2];
    __shared__ int abort_load, abort_compute;
    const uint32_t ring = (smem_u32(dt_smem) + 127u) & ~127u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 8); }
        abort_load = 0; abort_compute = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&map_in);
            int k = 0;
            for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
                const int s = k & 1;
                const uint32_t ph = (uint32_t)(k >> 1) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, &abort_load)) break;
                int r = t;
                const int cb = r % c_blocks; r /= c_blocks;
                const int wt = r % tiles_w; r /= tiles_w;
                const int ht = r % tiles_h, n = r / tiles_h;
                mbar_expect_tx(smem_u32(&full_bar[s]), C::BOX_BYTES);
                tma_load_4d(ring + (uint32_t)s * C::STAGE_BYTES, &map_in, smem_u32(&full_bar[s]), cb * CB, wt * C::TWB * S, ht * C::ROWS * S, n);
            }
            if (abort_load)      // gave up: let the loads already issued land before the shared memory goes away
                for (int j = (k > 2 ? k - 2 : 0); j < k; ++j)
                    for (int i = 0; i < (1 << 20) && !mbar_try_wait(smem_u32(&full_bar[j & 1]), (uint32_t)(j >> 1) & 1u); ++i) {}
        }
    } else {
        const int cg = threadIdx.x % C::CG, wl = threadIdx.x / C::CG;
        const int c = (int)(blockIdx.x % c_blocks) * CB + cg * 4;      // the same for every tile of this CTA
        float4 flt[3][3];
#pragma unroll
        for (int kh = 0; kh < 3; ++kh)
#pragma unroll
            for (int kw = 0; kw < 3; ++kw)
                flt[kh][kw] = c < p.C ? load4(Kf + (int64_t)kh * p.k_kh + (int64_t)kw * p.k_kw + c) : make_float4(0.f, 0.f, 0.f, 0.f);
        int k = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
            const int s = k & 1;
            const uint32_t ph = (uint32_t)(k >> 1) & 1u;
            int r = t / c_blocks;
            const int wt = r % tiles_w; r /= tiles_w;
            const int ht = r % tiles_h, n = r / tiles_h;
            const int w = wt * C::TWB + wl, h0 = ht * C::ROWS;
            const bool live = c < p.C && w < p.Wo;
            const bool ok = mbar_wait(smem_u32(&full_bar[s]), ph, &abort_compute);
            if (!__all_sync(0xffffffffu, ok)) break;
            // this thread's columns of the tile: pixel (row r, column S*wl + kw) of the stage; tile row r lives in win[r % 3]
            const uint32_t col_base = ring + (uint32_t)s * C::STAGE_BYTES + (uint32_t)(wl * S * CB + cg * 4) * (uint32_t)sizeof(T);
            float4 win[3][3];
#pragma unroll
            for (int rr = 0; rr < 3 - S; ++rr)
#pragma unroll
                for (int kw = 0; kw < 3; ++kw) win[rr][kw] = lds4(col_base + (uint32_t)((rr * C::IN_W + kw) * C::PIXEL_BYTES), T());
            float *out = O + (int64_t)n * p.o_n + (int64_t)w * p.o_w + c;
#pragma unroll
            for (int hh = 0; hh < C::ROWS; ++hh) {
                // the window of output row hh is tile rows S*hh .. S*hh+2; the first 3-S of them are already held
#pragma unroll
                for (int rr = S * hh + 3 - S; rr <= S * hh + 2; ++rr)
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw)
                        win[rr % 3][kw] = lds4(col_base + (uint32_t)((rr * C::IN_W + kw) * C::PIXEL_BYTES), T());
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int kh = 0; kh < 3; ++kh)
#pragma unroll
                    for (int kw = 0; kw < 3; ++kw) fma4(acc, win[(S * hh + kh) % 3][kw], flt[kh][kw]);
                if (live && h0 + hh < p.Ho) {
                    float4 *o = reinterpret_cast<float4 *>(out + (int64_t)(h0 + hh) * p.o_h);
                    if (p.accumulate) {
                        const float4 old = *o;
                        acc.x += old.x; acc.y += old.y; acc.z += old.z; acc.w += old.w;
                    }
                    *o = acc;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));       // this warp has read all it needs of the stage
        }
    }
    __syncthreads();
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

template <typename T, int CB, int S>
bool try_launch_tma(const DepthwiseProblem &p, const T *I, const T *Kf, float *O, int num_sms, cudaStream_t stream, cudaError_t *err) {
    using C = DtCfg<T, CB, S>;
    const int64_t es = sizeof(T);
    const int tiles_w = (p.Wo + C::TWB - 1) / C::TWB, tiles_h = (p.Ho + C::ROWS - 1) / C::ROWS, c_blocks = (p.C + CB - 1) / CB;
    const int64_t tiles = (int64_t)p.N * tiles_h * tiles_w * c_blocks;
    if (tiles < num_sms || tiles >= ((int64_t)1 << 31) || c_blocks > num_sms) return false;
    // the part of the input that is read: ((Ho-1)*S+3) x ((Wo-1)*S+3) pixels per image
    const int64_t h_ext = (int64_t)(p.Ho - 1) * S + 3, w_ext = (int64_t)(p.Wo - 1) * S + 3;
    const int64_t s_n = p.N > 1 ? p.i_n : h_ext * p.i_h;
    cuuint64_t dims[4] = {(cuuint64_t)p.C, (cuuint64_t)w_ext, (cuuint64_t)h_ext, (cuuint64_t)p.N};
    cuuint64_t strides[3] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)(p.i_h * es), (cuuint64_t)(s_n * es)};
    cuuint32_t box[4] = {(cuuint32_t)CB, (cuuint32_t)C::IN_W, (cuuint32_t)C::IN_H, 1};
    for (int i = 0; i < 3; ++i)
        if (strides[i] % 16 != 0 || strides[i] >= ((cuuint64_t)1 << 40)) return false;
    CUtensorMap map_in;
    if (!tensor_encode_tiled(&map_in, sizeof(T) == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                             const_cast<T *>(I), dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
        return false;
    const int smem = 2 * C::STAGE_BYTES + 128;
    static int attr_device = -1;      // the attribute is per device
    int dev = 0;
    cudaGetDevice(&dev);
    if (attr_device != dev) {
        if (cudaFuncSetAttribute(depthwise_tma_kernel<T, CB, S>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
        attr_device = dev;
    }
    // two CTAs per SM, rounded down to a multiple of the channel blocks: tile t has block t % c_blocks, so every CTA keeps one
    int64_t grid = std::min<int64_t>(tiles, 2 * (int64_t)num_sms);
    grid -= grid % c_blocks;
    depthwise_tma_kernel<T, CB, S><<<(int)grid, DT_THREADS, smem, stream>>>(map_in, p, Kf, O, tiles_w, tiles_h, c_blocks, (int)tiles);
    count_launch();
    note_kernel("depthwise_tma_kernel");
    *err = cudaGetLastError();
    return true;
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
    const bool win3 = p.KW == 3 && p.KH == 3 && p.dw == 1 && p.dh == 1;
    if (vec && win3 && p.sh == p.sw && p.sh <= 2 && reinterpret_cast<uintptr_t>(I) % 16 == 0 &&
        (p.C * (int64_t)sizeof(T)) % 16 == 0) {
        // TMA-staged tiles (TMA checks the channel bound in 16-byte units, hence the condition on C)
        int num_sms = 0;
        cudaError_t err = cudaSuccess;
        if (tensor_driver_ready(&num_sms) && p.C >= 32) {
            bool done;
            if (p.sh == 1) done = p.C >= 64 ? try_launch_tma<T, 64, 1>(p, I, Kf, O, num_sms, stream, &err) : try_launch_tma<T, 32, 1>(p, I, Kf, O, num_sms, stream, &err);
            else done = p.C >= 64 ? try_launch_tma<T, 64, 2>(p, I, Kf, O, num_sms, stream, &err) : try_launch_tma<T, 32, 2>(p, I, Kf, O, num_sms, stream, &err);
            if (done) return err;
        }
    }
    if (vec && unit3 && p.sh == 1 && p.dh == 1) {
        // enough row segments to give every SM several thread blocks: walk down the rows with a rolling window
        const int64_t items = (int64_t)p.N * ((p.Ho + ROLL_ROWS - 1) / ROLL_ROWS) * ((p.Wo + ROLL_TW - 1) / ROLL_TW) * (p.C / 4);
        if (items >= (int64_t)148 * 256 * 2 && items < ((int64_t)1 << 32) - 256 && 9 * p.C * 4 <= 48 * 1024) {
            depthwise_roll_kernel<T><<<(unsigned)((items + ROLL_BLOCK - 1) / ROLL_BLOCK), ROLL_BLOCK, 9 * p.C * 4, stream>>>(p, I, Kf, O);
            count_launch();
            note_kernel("depthwise_roll_kernel");
            return cudaGetLastError();
        }
    }
#define SG_DW(KERNEL) KERNEL<<<blocks, 256, 0, stream>>>(p, I, Kf, O)
    if (vec && unit3) { if (small) SG_DW((depthwise_vec_kernel<T, true, uint32_t>)); else SG_DW((depthwise_vec_kernel<T, true, uint64_t>)); }
    else if (vec) { if (small) SG_DW((depthwise_vec_kernel<T, false, uint32_t>)); else SG_DW((depthwise_vec_kernel<T, false, uint64_t>)); }
    else { if (small) SG_DW((depthwise_generic_kernel<T, uint32_t>)); else SG_DW((depthwise_generic_kernel<T, uint64_t>)); }
#undef SG_DW
    count_launch();
    note_kernel(vec ? "depthwise_vec_kernel" : "depthwise_generic_kernel");
    return cudaGetLastError();
}

}  // namespace

sg_status depthwise_read_status(cudaStream_t stream) { return read_status_word(stream); }

cudaError_t launch_depthwise(const DepthwiseProblem &p, const void *I, const void *Kf, float *O, cudaStream_t stream) {
    if (p.in_bf16)
        return launch_typed(p, static_cast<const __nv_bfloat16 *>(I), static_cast<const __nv_bfloat16 *>(Kf), O, stream);
    return launch_typed(p, static_cast<const float *>(I), static_cast<const float *>(Kf), O, stream);
}

}  // namespace sg

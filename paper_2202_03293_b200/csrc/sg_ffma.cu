// CUDA-core path: a register-tiled FFMA implicit GEMM that accepts any element strides.
//
// It serves (a) every f32 call, keeping full f32 accuracy (each product and each
// accumulation step is one fused multiply-add in f32), and (b) every call whose layout
// the tensor-core path cannot take (non-unit inner strides, unaligned bases or pitches).
//
// Tiling follows the decomposition of Section 3.1 of the paper: the parallel iterators
// (m = (n,h,w), f) are cut into 128 x 128 output tiles, one per CTA; the reduction
// iterators (kh,kw,c) are walked in blocks of 16; partial tiles are padded with the
// additive neutral 0 on load and predicated on store (Section 3.2).  The operand subset
// of a tile is the image of the tile under the operand's indexing map, which for these
// ops separates into a per-row offset plus a per-k offset (see Problem).
#include "sg_internal.cuh"

namespace sg {
namespace {

constexpr int BM = 128, BN = 128, BK = 16, THREADS = 256;
constexpr int LDA = BM + 4;   // padded: transposed stores of the In tile spread over banks

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(unsigned short v) { return __uint_as_float(((unsigned)v) << 16); }

__device__ __forceinline__ void load4(const float *p, float (&v)[4]) {
    float4 t = *reinterpret_cast<const float4 *>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
__device__ __forceinline__ void load4(const unsigned short *p, float (&v)[4]) {
    uint2 t = *reinterpret_cast<const uint2 *>(p);
    v[0] = __uint_as_float(t.x << 16);
    v[1] = __uint_as_float(t.x & 0xFFFF0000u);
    v[2] = __uint_as_float(t.y << 16);
    v[3] = __uint_as_float(t.y & 0xFFFF0000u);
}

// Offset of output row m in the input (its window origin) and in the output.
__device__ __forceinline__ void row_offsets(const Problem &p, int m, int64_t &in_off, int64_t &out_off) {
    int hw = p.Ho * p.Wo;
    int n = m / hw, r = m - n * hw;
    int h = r / p.Wo, w = r - h * p.Wo;
    in_off = (int64_t)n * p.i_n + (int64_t)h * p.sh * p.i_h + (int64_t)w * p.sw * p.i_w;
    out_off = (int64_t)n * p.o_n + (int64_t)h * p.o_h + (int64_t)w * p.o_w;
}

// Offset of reduction index k = (kh, kw, c) in the input window and in the filter.
__device__ __forceinline__ void k_offsets(const Problem &p, int k, int64_t &in_off, int64_t &flt_off) {
    int kwc = p.KW * p.C;
    int kh = k / kwc, r = k - kh * kwc;
    int kw = r / p.C, c = r - kw * p.C;
    in_off = (int64_t)kh * p.dh * p.i_h + (int64_t)kw * p.dw * p.i_w + (int64_t)c * p.i_c;
    flt_off = (int64_t)kh * p.k_kh + (int64_t)kw * p.k_kw + (int64_t)c * p.k_c;
}

template <typename T, bool VEC_A, bool VEC_B>
__global__ void __launch_bounds__(THREADS)
ffma_kernel(Problem p, const T *__restrict__ In, const T *__restrict__ Flt, float *__restrict__ O, int vec_c) {
    __shared__ __align__(16) float As[2][BK][LDA];   // In tile, stored k-major: As[k][m]
    __shared__ __align__(16) float Bs[2][BK][BN];    // filter tile:            Bs[k][f]

    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * BM;
    const int n0 = blockIdx.y * BN;

    // ---- what this thread fetches from global memory per k-block ----
    constexpr int A_LOADS = VEC_A ? 2 : 8;
    constexpr int B_LOADS = VEC_B ? 2 : 8;
    const int a_kl = VEC_A ? (tid & 3) * 4 : (tid & 15);   // k within the block (same for all its loads)
    int a_row[A_LOADS];
    int64_t a_rowoff[A_LOADS];
    bool a_rowok[A_LOADS];
#pragma unroll
    for (int i = 0; i < A_LOADS; ++i) {
        a_row[i] = VEC_A ? (tid >> 2) + i * 64 : (tid >> 4) + i * 16;
        int m = m0 + a_row[i];
        a_rowok[i] = m < p.M;
        int64_t dummy;
        a_rowoff[i] = 0;
        if (a_rowok[i]) row_offsets(p, m, a_rowoff[i], dummy);
    }
    const int b_nl = VEC_B ? (tid & 31) * 4 : (tid & 127);
    const bool b_nok = VEC_B ? (n0 + b_nl + 3 < p.N) : (n0 + b_nl < p.N);
    const int64_t b_noff = (int64_t)(n0 + b_nl) * p.k_f;

    float a_reg[A_LOADS][VEC_A ? 4 : 1];
    float b_reg[B_LOADS][VEC_B ? 4 : 1];

    auto fetch = [&](int kb) {
        {   // In tile
            int k = kb * BK + a_kl;
            int64_t ka = 0, kf = 0;
            bool kok = k < p.K;
            if (kok) k_offsets(p, k, ka, kf);
#pragma unroll
            for (int i = 0; i < A_LOADS; ++i) {
                if constexpr (VEC_A) {
                    if (kok && a_rowok[i]) load4(In + a_rowoff[i] + ka, a_reg[i]);
                    else { a_reg[i][0] = a_reg[i][1] = a_reg[i][2] = a_reg[i][3] = 0.f; }
                } else {
                    a_reg[i][0] = (kok && a_rowok[i]) ? to_f32(In[a_rowoff[i] + ka]) : 0.f;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < B_LOADS; ++i) {   // filter tile
            int kl = VEC_B ? (tid >> 5) + i * 8 : (tid >> 7) + i * 2;
            int k = kb * BK + kl;
            int64_t ka = 0, kf = 0;
            bool ok = (k < p.K) && b_nok;
            if (ok) k_offsets(p, k, ka, kf);
            if constexpr (VEC_B) {
                if (ok) load4(Flt + kf + b_noff, b_reg[i]);
                else { b_reg[i][0] = b_reg[i][1] = b_reg[i][2] = b_reg[i][3] = 0.f; }
            } else {
                b_reg[i][0] = ok ? to_f32(Flt[kf + b_noff]) : 0.f;
            }
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int i = 0; i < A_LOADS; ++i) {
            if constexpr (VEC_A) {
#pragma unroll
                for (int j = 0; j < 4; ++j) As[buf][a_kl + j][a_row[i]] = a_reg[i][j];
            } else {
                As[buf][a_kl][a_row[i]] = a_reg[i][0];
            }
        }
#pragma unroll
        for (int i = 0; i < B_LOADS; ++i) {
            int kl = VEC_B ? (tid >> 5) + i * 8 : (tid >> 7) + i * 2;
            if constexpr (VEC_B) {
                *reinterpret_cast<float4 *>(&Bs[buf][kl][b_nl]) =
                    make_float4(b_reg[i][0], b_reg[i][1], b_reg[i][2], b_reg[i][3]);
            } else {
                Bs[buf][kl][b_nl] = b_reg[i][0];
            }
        }
    };

    // ---- 8 x 8 register tile per thread: rows {ty*4.., 64+ty*4..}, cols {tx*4.., 64+tx*4..} ----
    const int ty = tid >> 4, tx = tid & 15;
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    const int num_kb = (p.K + BK - 1) / BK;
    if (num_kb > 0) {
        fetch(0);
        stash(0);
    }
    __syncthreads();
    for (int kb = 0; kb < num_kb; ++kb) {
        const int buf = kb & 1;
        if (kb + 1 < num_kb) fetch(kb + 1);   // global loads in flight during the FMAs below
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[8], b[8];
            float4 t;
            t = *reinterpret_cast<const float4 *>(&As[buf][k][ty * 4]);
            a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
            t = *reinterpret_cast<const float4 *>(&As[buf][k][64 + ty * 4]);
            a[4] = t.x; a[5] = t.y; a[6] = t.z; a[7] = t.w;
            t = *reinterpret_cast<const float4 *>(&Bs[buf][k][tx * 4]);
            b[0] = t.x; b[1] = t.y; b[2] = t.z; b[3] = t.w;
            t = *reinterpret_cast<const float4 *>(&Bs[buf][k][64 + tx * 4]);
            b[4] = t.x; b[5] = t.y; b[6] = t.z; b[7] = t.w;
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (kb + 1 < num_kb) stash(buf ^ 1);
        __syncthreads();
    }

    // ---- fused pointwise consumer (Sections 2.1, 3.3): r = act(acc + bias[f]), the bias broadcast along the rows ----
    if (p.bias != nullptr || p.act != SG_ACT_NONE) {
#pragma unroll
        for (int jh = 0; jh < 2; ++jh)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = n0 + jh * 64 + tx * 4 + j;
                const float b = (p.bias != nullptr && n < p.N) ? p.bias[(int64_t)n * p.bias_f] : 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float v = acc[i][jh * 4 + j] + b;
                    acc[i][jh * 4 + j] = (p.act == SG_ACT_RELU && v < 0.f) ? 0.f : v;
                }
            }
    }
    // ---- write-back: O = acc  or  O = O_in + acc ----
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        int m = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + (i - 4));
        if (m >= p.M) continue;
        int64_t in_off, out_off;
        row_offsets(p, m, in_off, out_off);
#pragma unroll
        for (int jh = 0; jh < 2; ++jh) {
            int n = n0 + jh * 64 + tx * 4;
            float *dst = O + out_off + (int64_t)n * p.o_f;
            if (vec_c && n + 3 < p.N) {
                float4 v = make_float4(acc[i][jh * 4 + 0], acc[i][jh * 4 + 1], acc[i][jh * 4 + 2], acc[i][jh * 4 + 3]);
                if (p.accumulate) {
                    float4 o = *reinterpret_cast<const float4 *>(dst);
                    v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                }
                *reinterpret_cast<float4 *>(dst) = v;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (n + j < p.N) {
                        float v = acc[i][jh * 4 + j];
                        float *d = dst + (int64_t)j * p.o_f;
                        *d = p.accumulate ? (*d + v) : v;
                    }
                }
            }
        }
    }
}

__global__ void zero_fill_kernel(Problem p, float *__restrict__ O) {
    asm volatile("griddepcontrol.launch_dependents;");   // a dependent launch waits for this grid's end where it needs the zeros
    int64_t total = (int64_t)p.M * p.N;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        int m = (int)(i / p.N), n = (int)(i - (int64_t)m * p.N);
        int64_t in_off, out_off;
        row_offsets(p, m, in_off, out_off);
        O[out_off + (int64_t)n * p.o_f] = 0.f;
    }
}

// The output as one M x N matrix of contiguous, 16-byte aligned rows `pitch` floats apart
// (what the tensor-core path requires of it): four columns per thread.
__global__ void zero_fill_rows_kernel(float *__restrict__ O, int M, int n4, int64_t pitch) {
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t total = (int64_t)M * n4;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int m = (int)(i / n4), c = (int)(i - (int64_t)m * n4);
        reinterpret_cast<float4 *>(O + (int64_t)m * pitch)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

inline bool mult_of(int64_t v, int64_t q) { return v % q == 0; }

template <typename T>
cudaError_t launch_typed(const Problem &p, const T *In, const T *Flt, float *O, cudaStream_t stream) {
    // 4 consecutive k (resp. f) may be fetched as one 8- or 16-byte load when they are
    // contiguous in memory and every address involved is a multiple of 4 elements.
    const uintptr_t vec_bytes = 4 * sizeof(T);
    bool vec_a = p.i_c == 1 && mult_of(p.C, 4) && mult_of(p.i_n, 4) && mult_of(p.i_h, 4) &&
                 mult_of(p.i_w, 4) && (reinterpret_cast<uintptr_t>(In) % vec_bytes == 0);
    bool vec_b = p.k_f == 1 && mult_of(p.N, 4) && mult_of(p.k_kh, 4) && mult_of(p.k_kw, 4) &&
                 mult_of(p.k_c, 4) && (reinterpret_cast<uintptr_t>(Flt) % vec_bytes == 0);
    int vec_c = p.o_f == 1 && mult_of(p.o_n, 4) && mult_of(p.o_h, 4) && mult_of(p.o_w, 4) &&
                (reinterpret_cast<uintptr_t>(O) % 16 == 0);
    dim3 grid((p.M + BM - 1) / BM, (p.N + BN - 1) / BN);
    if (grid.y > 65535) return cudaErrorInvalidConfiguration;
    if (vec_a && vec_b) ffma_kernel<T, true, true><<<grid, THREADS, 0, stream>>>(p, In, Flt, O, vec_c);
    else if (vec_a) ffma_kernel<T, true, false><<<grid, THREADS, 0, stream>>>(p, In, Flt, O, vec_c);
    else if (vec_b) ffma_kernel<T, false, true><<<grid, THREADS, 0, stream>>>(p, In, Flt, O, vec_c);
    else ffma_kernel<T, false, false><<<grid, THREADS, 0, stream>>>(p, In, Flt, O, vec_c);
    count_launch();
    note_kernel("ffma_kernel");
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_ffma(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream) {
    if (p.in_bf16)
        return launch_typed(p, static_cast<const unsigned short *>(In), static_cast<const unsigned short *>(Flt), O, stream);
    return launch_typed(p, static_cast<const float *>(In), static_cast<const float *>(Flt), O, stream);
}

cudaError_t launch_zero_fill(const Problem &p, float *O, cudaStream_t stream) {
    const bool uniform_rows = p.o_f == 1 && (p.Ho == 1 || p.o_h == (int64_t)p.Wo * p.o_w) &&
                              (p.batch == 1 || p.o_n == (int64_t)p.Ho * p.Wo * p.o_w);
    if (uniform_rows && p.N % 4 == 0 && p.o_w % 4 == 0 && reinterpret_cast<uintptr_t>(O) % 16 == 0) {
        const int64_t work = (int64_t)p.M * (p.N / 4);
        const int blocks = (int)((work + 255) / 256 < 148 * 8 ? (work + 255) / 256 : 148 * 8);
        zero_fill_rows_kernel<<<blocks, 256, 0, stream>>>(O, p.M, p.N / 4, p.o_w);
        count_launch();
        return cudaGetLastError();
    }
    int64_t total = (int64_t)p.M * p.N;
    int blocks = (int)((total + 255) / 256 < 148 * 8 ? (total + 255) / 256 : 148 * 8);
    zero_fill_kernel<<<blocks, 256, 0, stream>>>(p, O);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sg

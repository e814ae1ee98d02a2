// The memory-bound 2-D kernels (Section 4.4: Copy2D, Transpose2D, ColRed2D, RowRed2D).
//
//   Copy2D       dst[i,j] = src[i,j]
//   Transpose2D  dst[j,i] = src[i,j]
//   ColRed2D     out[j] (+)= sum_i A[i,j]
//   RowRed2D     out[i] (+)= sum_j A[i,j]
//
// All four are bound by HBM traffic; the kernels differ in how they keep enough bytes in flight.
//   - Copy2D and Transpose2D, when the layout meets the TMA rules (unit column stride, 16-byte
//     aligned bases and row pitches), move tiles with TMA only: a persistent CTA per SM slot runs
//     a shared-memory ring that one thread fills with tensor loads and another drains with tensor
//     stores.  The copy never touches the data with an ordinary instruction; the transpose has
//     four warps turn each 128-row tile around in shared memory between the load and the store
//     (4-byte elements: 16-byte reads of the 128-byte swizzled input tile, a register transpose
//     of a 4 x 4 block, 16-byte writes into the swizzled output tile; 2-byte elements: 8 x 8
//     blocks through ldmatrix.trans and stmatrix).  Ragged edges cost nothing: loads
//     read zeros beyond the tensor, stores are clipped.
//   - The reductions use plain 16-byte loads with four in flight per thread at full occupancy,
//     f32 accumulators, and a shared-memory / shuffle tree per CTA.  When the shape has too few
//     independent outputs to fill the chip, the reduced index is split across CTAs and the
//     partial sums meet in the output through float atomics (an overwriting call clears the
//     output first); nothing but the operands is read or written.
//   - Anything else (non-unit column strides, unaligned pitches) runs on strided 32 x 32 tile
//     kernels.
#include <algorithm>

#include "sg_internal.cuh"
#include "sg_tc_ptx.cuh"

namespace sg {
namespace {

// Bounded, flag-free wait used only while winding down after a time-out: lets copies that are
// still in flight land before the CTA gives its shared memory back.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    for (int i = 0; i < (1 << 20); ++i)
        if (mbar_try_wait(bar, parity)) return;
}

// ------------------------------------------------------------------------------ Copy2D (TMA)
#ifndef SG_CP_STAGES
#define SG_CP_STAGES 6
#endif
#ifndef SG_CP_STORES_IN_FLIGHT
#define SG_CP_STORES_IN_FLIGHT 2
#endif
#ifndef SG_CP_STAGE_BYTES
#define SG_CP_STAGE_BYTES 32768
#endif
#ifndef SG_CP_CTAS_PER_SM
#define SG_CP_CTAS_PER_SM 1
#endif
#ifndef SG_CP_BOX_X
#define SG_CP_BOX_X 256
#endif
constexpr int CP_STAGES = SG_CP_STAGES;                         // ring depth
constexpr int CP_STORES_IN_FLIGHT = SG_CP_STORES_IN_FLIGHT;     // stores whose shared-memory reads may be pending
constexpr int CP_STAGE_BYTES = SG_CP_STAGE_BYTES;
constexpr int CP_CTAS_PER_SM = SG_CP_CTAS_PER_SM;
static_assert(CP_STAGES > CP_STORES_IN_FLIGHT + 1, "the ring must leave room for loads");

// Tiles are dealt round-robin to the CTAs; warp 0 loads, warp 1 stores, one lane each.
__global__ void __launch_bounds__(64) copy_tma_kernel(const __grid_constant__ CUtensorMap map_src,
                                                       const __grid_constant__ CUtensorMap map_dst, int tiles_x, int num_tiles,
                                                       int box_x, int box_y, uint32_t box_bytes) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[CP_STAGES], empty_bar[CP_STAGES];
    __shared__ int abort_load, abort_store;
    const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < CP_STAGES; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        abort_load = 0; abort_store = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0 && lane == 0) {
        prefetch_tensormap(&map_src);
        int k = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
            const int s = k % CP_STAGES;
            const uint32_t ph = (uint32_t)(k / CP_STAGES) & 1u;
            if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, &abort_load)) break;
            mbar_expect_tx(smem_u32(&full_bar[s]), box_bytes);
            tma_load_2d(ring + (uint32_t)s * CP_STAGE_BYTES, &map_src, smem_u32(&full_bar[s]), (t % tiles_x) * box_x, (t / tiles_x) * box_y);
        }
        if (abort_load)   // gave up: let the loads already issued land
            for (int j = (k > CP_STAGES ? k - CP_STAGES : 0); j < k; ++j) mbar_drain(smem_u32(&full_bar[j % CP_STAGES]), (uint32_t)(j / CP_STAGES) & 1u);
    } else if (warp == 1 && lane == 0) {
        prefetch_tensormap(&map_dst);
        int k = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
            const int s = k % CP_STAGES;
            const uint32_t ph = (uint32_t)(k / CP_STAGES) & 1u;
            if (!mbar_wait(smem_u32(&full_bar[s]), ph, &abort_store)) break;
            tma_store_2d(&map_dst, ring + (uint32_t)s * CP_STAGE_BYTES, (t % tiles_x) * box_x, (t / tiles_x) * box_y);
            bulk_commit();
            if (k >= CP_STORES_IN_FLIGHT) {   // the store issued CP_STORES_IN_FLIGHT tiles ago has read its stage
                bulk_wait_read<CP_STORES_IN_FLIGHT>();
                mbar_arrive(smem_u32(&empty_bar[(k - CP_STORES_IN_FLIGHT) % CP_STAGES]));
            }
        }
        bulk_wait_read<0>();      // the ring must stay until the last stores have read it; the grid's end completes the writes
    }
    __syncthreads();
}

// ------------------------------------------------------------------------- Transpose2D (TMA)
// One tile = 128 input rows x 128 bytes (W = 128/ES columns).  Input stage: the tile as TMA wrote
// it with the 128-byte swizzle (16-byte chunk index XOR row mod 8).  Output staging: the W x 128
// transposed tile as 128/W blocks of [W rows][128 bytes], same swizzle, stored by four tensor
// stores of 32 rows each (one per transposer warp, which also produces exactly those rows).
#ifndef SG_TR_PANEL
#define SG_TR_PANEL 8
#endif
constexpr int TR_PANEL = SG_TR_PANEL;     // tile columns per panel of the tile order
constexpr int TR_IN_STAGES = 4;
constexpr int TR_TILE_BYTES = 16384;
constexpr int TR_THREADS = 32 + 128;

// 4 x 4 block of 4-byte elements held as four 16-byte rows: the transpose is a renaming of registers.
__device__ __forceinline__ void transpose_block(const uint4 (&v)[4], uint4 (&o)[4]) {
    o[0] = make_uint4(v[0].x, v[1].x, v[2].x, v[3].x);
    o[1] = make_uint4(v[0].y, v[1].y, v[2].y, v[3].y);
    o[2] = make_uint4(v[0].z, v[1].z, v[2].z, v[3].z);
    o[3] = make_uint4(v[0].w, v[1].w, v[2].w, v[3].w);
}

// Tile order: panels of `panel` tile columns, walked row by row inside a panel.  The tiles in flight at one time then
// cover a block of the matrix rather than a thin strip of it, so that both the reads (128 bytes per row and tile) and the
// writes (128 input rows = one run of an output row per tile) fall on runs of memory that neighbouring tiles extend.
__device__ __forceinline__ void tile_coords(int t, int tiles_c, int tiles_r, int panel, int &tr, int &tc) {
    const int per_panel = panel * tiles_r;
    const int pi = t / per_panel, within = t - pi * per_panel;
    const int start = pi * panel, width = min(panel, tiles_c - start);
    tr = within / width;
    tc = start + within - tr * width;
}

template <int ES>
__global__ void __launch_bounds__(TR_THREADS) transpose_tma_kernel(const __grid_constant__ CUtensorMap map_src,
                                                                    const __grid_constant__ CUtensorMap map_dst, int tiles_c,
                                                                    int tiles_r, int panel, int dst_cols, int dst_rows) {
    const int num_tiles = tiles_c * tiles_r;
    constexpr int E = 16 / ES;       // elements per 16-byte chunk = side of the register block
    constexpr int W = 128 / ES;      // input columns per tile = output rows per tile
    constexpr int P = 128 / E;       // row groups per tile
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[TR_IN_STAGES], empty_bar[TR_IN_STAGES];
    __shared__ int abort_load, abort_turn;
    const uint32_t in_ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t out_ring = in_ring + TR_IN_STAGES * TR_TILE_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < TR_IN_STAGES; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 4); }
        abort_load = 0; abort_turn = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&map_src);
            int k = 0;
            for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
                const int s = k % TR_IN_STAGES;
                const uint32_t ph = (uint32_t)(k / TR_IN_STAGES) & 1u;
                if (!mbar_wait(smem_u32(&empty_bar[s]), ph ^ 1u, &abort_load)) break;
                mbar_expect_tx(smem_u32(&full_bar[s]), TR_TILE_BYTES);
                int tr, tc;
                tile_coords(t, tiles_c, tiles_r, panel, tr, tc);
                tma_load_2d(in_ring + (uint32_t)s * TR_TILE_BYTES, &map_src, smem_u32(&full_bar[s]), tc * W, tr * 128);
            }
            if (abort_load)
                for (int j = (k > TR_IN_STAGES ? k - TR_IN_STAGES : 0); j < k; ++j)
                    mbar_drain(smem_u32(&full_bar[j % TR_IN_STAGES]), (uint32_t)(j / TR_IN_STAGES) & 1u);
        }
    } else {
        // Warp w owns store w of every tile: the 32 output rows x 128 bytes that sit at staging offset w * 4 KB.  What it
        // reads for them (f32: input rows 32w .. 32w+31, all 32 columns; 2-byte elements: rows 64(w/2) .. +63, columns
        // 32(w%2) .. +31) nobody else reads, so the four warps never wait for one another.
        const int w = warp - 1;
        if (lane == 0) prefetch_tensormap(&map_dst);
        // each lane turns E x E blocks (row group p, 16-byte chunk q); a quarter-warp covers two row groups x four chunks
        const int q = ES == 4 ? ((lane & 3) | ((lane >> 1) & 4)) : (4 * (w & 1) + (lane & 3));
        const int p0 = ES == 4 ? (8 * w + ((lane >> 2) & 1) + 2 * ((lane >> 4) & 1)) : (8 * (w >> 1) + (lane >> 2));
        constexpr int BLOCKS_PER_LANE = ES == 4 ? 2 : 1;
        const int b = w / (W / 32), h = w % (W / 32);
        int k = 0;
        for (int t = blockIdx.x; t < num_tiles; t += gridDim.x, ++k) {
            const int s = k % TR_IN_STAGES;
            const uint32_t ph = (uint32_t)(k / TR_IN_STAGES) & 1u;
            const bool ok = mbar_wait(smem_u32(&full_bar[s]), ph, &abort_turn);
            if (!__all_sync(0xffffffffu, ok)) break;
            if (lane == 0) bulk_wait_read<1>();                        // this warp's store from two tiles ago has read its staging
            __syncwarp();
            const uint32_t in_tile = in_ring + (uint32_t)s * TR_TILE_BYTES;
            const uint32_t out_tile = out_ring + (uint32_t)(k & 1) * TR_TILE_BYTES;
            if constexpr (ES == 2) {
                // 2-byte elements: the matrix load/store instructions do the turn.  Instruction i handles input rows
                // 8p .. 8p+7 (p = 8b + i) of the warp's four chunks: ldmatrix.trans hands every lane two consecutive
                // elements of a transposed 8 x 8 block per chunk, stmatrix writes those blocks as 16-byte rows.  In both,
                // the eight row addresses of a block fall on eight different swizzled chunks: no bank conflicts.
                const int m = lane >> 3, rr = lane & 7;           // this lane addresses row rr of block m
                const int qm = 4 * h + m;                         // chunk of block m
                const int c = 8 * qm + rr;                        // output row this lane addresses
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int row = 8 * (8 * b + i) + rr;
                    const uint32_t src_addr = in_tile + (uint32_t)row * 128u + (uint32_t)((qm ^ rr) << 4);
                    uint32_t r0, r1, r2, r3;
                    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(src_addr));
                    const uint32_t dst_addr = out_tile + (uint32_t)b * (uint32_t)(W * 128) + (uint32_t)c * 128u + (uint32_t)((i ^ (c & 7)) << 4);
                    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1, %2, %3, %4};"
                                 ::"r"(dst_addr), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
                }
            } else {
#pragma unroll
                for (int i = 0; i < BLOCKS_PER_LANE; ++i) {
                    const int p = p0 + 4 * i;
                    uint4 v[E], o[E];
#pragma unroll
                    for (int kk = 0; kk < E; ++kk) {
                        const int row = E * p + kk;
                        const uint32_t addr = in_tile + (uint32_t)row * 128u + (uint32_t)((q ^ (row & 7)) << 4);
                        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[kk].x), "=r"(v[kk].y), "=r"(v[kk].z), "=r"(v[kk].w) : "r"(addr));
                    }
                    transpose_block(v, o);
#pragma unroll
                    for (int j = 0; j < E; ++j) {
                        const int c = E * q + j;                       // output row within the tile
                        const uint32_t addr = out_tile + (uint32_t)(p >> 3) * (uint32_t)(W * 128) + (uint32_t)c * 128u +
                                              (uint32_t)(((p & 7) ^ (c & 7)) << 4);
                        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(o[j].x), "r"(o[j].y), "r"(o[j].z), "r"(o[j].w) : "memory");
                    }
                }
            }
            fence_async_smem();                                        // staging writes -> visible to the tensor store
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&empty_bar[s]));                  // this warp is done with the input stage
                int tr, tc;
                tile_coords(t, tiles_c, tiles_r, panel, tr, tc);
                const int x = tr * 128 + b * W, y = tc * W + h * 32;
                if (x < dst_cols && y < dst_rows) tma_store_2d(&map_dst, out_tile + (uint32_t)w * 4096u, x, y);
                bulk_commit();
            }
        }
        if (lane == 0) bulk_wait_read<0>();
    }
    __syncthreads();
}

// ------------------------------------------------------------------ strided 32 x 32 tile kernel
// dst[i*d_i + j*d_j] = src[i*s_i + j*s_j]; a transpose is the same call with the destination
// strides exchanged.  WRITE_BY_I: consecutive threads write consecutive i (the destination is
// contiguous along i), else consecutive j.
template <typename U, bool WRITE_BY_I>
__global__ void __launch_bounds__(256) tile_move_kernel(const U *__restrict__ src, int64_t s_i, int64_t s_j, U *__restrict__ dst,
                                                         int64_t d_i, int64_t d_j, int R, int C, int tiles_j, int64_t num_tiles) {
    __shared__ U tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int64_t t = blockIdx.x; t < num_tiles; t += gridDim.x) {
        const int i0 = (int)(t / tiles_j) * 32, j0 = (int)(t % tiles_j) * 32;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = i0 + ty + 8 * k, j = j0 + tx;
            if (i < R && j < C) tile[ty + 8 * k][tx] = src[(int64_t)i * s_i + (int64_t)j * s_j];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if constexpr (WRITE_BY_I) {
                const int i = i0 + tx, j = j0 + ty + 8 * k;
                if (i < R && j < C) dst[(int64_t)i * d_i + (int64_t)j * d_j] = tile[tx][ty + 8 * k];
            } else {
                const int i = i0 + ty + 8 * k, j = j0 + tx;
                if (i < R && j < C) dst[(int64_t)i * d_i + (int64_t)j * d_j] = tile[ty + 8 * k][tx];
            }
        }
        __syncthreads();
    }
}

// --------------------------------------------------------------------------------- reductions
inline bool aligned16(const void *p) { return reinterpret_cast<uintptr_t>(p) % 16 == 0; }

template <typename T, int VEC>
struct Chunk {
    float f[VEC];
};

__device__ __forceinline__ float widen(float x) { return x; }
__device__ __forceinline__ float widen(uint16_t bits) { return __uint_as_float((uint32_t)bits << 16); }

// Adds up to VEC consecutive elements starting at `ptr` (element stride `sc`) into acc.
// `nvalid` == VEC takes the 16-byte path (VEC > 1 implies sc == 1 and an aligned address).
// One whole chunk (VEC > 1: 16 bytes at an aligned address), added element-wise into acc.
template <typename T, int VEC>
__device__ __forceinline__ void accumulate_raw(float (&acc)[VEC], const uint4 &raw) {
    if constexpr (VEC == 4) {
        acc[0] += __uint_as_float(raw.x); acc[1] += __uint_as_float(raw.y);
        acc[2] += __uint_as_float(raw.z); acc[3] += __uint_as_float(raw.w);
    } else if constexpr (VEC == 8) {
        const uint32_t wds[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            acc[2 * w] += __uint_as_float(wds[w] << 16);
            acc[2 * w + 1] += __uint_as_float(wds[w] & 0xFFFF0000u);
        }
    }
}

template <typename T, int VEC>
__device__ __forceinline__ void add_chunk(float (&acc)[VEC], const T *ptr, int64_t sc, int nvalid) {
    if constexpr (VEC > 1) {
        if (nvalid == VEC) {
            accumulate_raw<T, VEC>(acc, __ldg(reinterpret_cast<const uint4 *>(ptr)));
            return;
        }
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v)
        if (v < nvalid) acc[v] += widen(__ldg(ptr + (int64_t)v * sc));
}

// Rows r, r+rp, ... < r1 of one chunk, eight loads in flight.  FULL: the chunk has all VEC columns (16-byte loads).
template <typename T, int VEC, bool FULL>
__device__ __forceinline__ void colred_walk(float (&acc)[VEC], const T *base, int64_t ld, int64_t sc, int64_t r, int64_t r1, int rp,
                                            int nvalid) {
    constexpr int U = 8;
    if constexpr (FULL && VEC > 1) {
        // all eight 16-byte loads are issued before the first is consumed
        for (; r + (U - 1) * rp < r1; r += U * rp) {
            uint4 raw[U];
#pragma unroll
            for (int u = 0; u < U; ++u) raw[u] = __ldg(reinterpret_cast<const uint4 *>(base + (r + u * rp) * ld));
#pragma unroll
            for (int u = 0; u < U; ++u) accumulate_raw<T, VEC>(acc, raw[u]);
        }
    } else {
        for (; r + (U - 1) * rp < r1; r += U * rp) {
            float part[U];
#pragma unroll
            for (int u = 0; u < U; ++u) part[u] = 0.f;
#pragma unroll
            for (int v = 0; v < VEC; ++v) {
                if (v < nvalid) {
#pragma unroll
                    for (int u = 0; u < U; ++u) part[u] = widen(__ldg(base + (r + u * rp) * ld + (int64_t)v * sc));
                    acc[v] += ((part[0] + part[1]) + (part[2] + part[3])) + ((part[4] + part[5]) + (part[6] + part[7]));
                }
            }
        }
    }
    for (; r < r1; r += rp) add_chunk<T, VEC>(acc, base + r * ld, sc, FULL ? VEC : nvalid);
}

// ColRed2D.  A CTA owns `cw` chunks of VEC columns and the rows [r0, r1) of its split;
// thread (g, cc) = (t / cw, t % cw) walks rows r0+g, r0+g+rp, ... of chunk cc.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) colred_kernel(const T *__restrict__ A, int64_t ld, int64_t sc, int R, int C,
                                                      float *__restrict__ out, int64_t os, int cw, int rp, int rows_per_split,
                                                      int use_atomic, int accumulate) {
    __shared__ float red[256][VEC + 1];
    const int t = threadIdx.x, g = t / cw, cc = t - g * cw;
    const int64_t col0 = ((int64_t)blockIdx.x * cw + cc) * VEC;
    const int r0 = blockIdx.y * rows_per_split;
    const int r1 = min(R, r0 + rows_per_split);
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    const bool active = g < rp && col0 < C;
    const int nvalid = active ? (int)min((int64_t)VEC, (int64_t)C - col0) : 0;
    if (active) {
        const T *base = A + col0 * sc;
        if (nvalid == VEC) colred_walk<T, VEC, true>(acc, base, ld, sc, r0 + g, r1, rp, VEC);
        else colred_walk<T, VEC, false>(acc, base, ld, sc, r0 + g, r1, rp, nvalid);
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) red[t][v] = acc[v];
    __syncthreads();
    // (after the clearing kernel of an overwriting split reduction; this grid may have started beside it)
    if (use_atomic) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (g == 0 && col0 < C) {
        for (int gg = 1; gg < rp; ++gg)
#pragma unroll
            for (int v = 0; v < VEC; ++v) acc[v] += red[gg * cw + cc][v];
        if (VEC >= 4 && use_atomic == 2 && nvalid == VEC) {
            // dense, 16-byte aligned output: four sums per atomic
#pragma unroll
            for (int v = 0; v < VEC; v += 4)
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out + col0 + v), "f"(acc[v]), "f"(acc[(v + 1) % VEC]),
                             "f"(acc[(v + 2) % VEC]), "f"(acc[(v + 3) % VEC]) : "memory");
            return;
        }
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            if (v < nvalid) {
                float *o = out + (col0 + v) * os;
                if (use_atomic) atomicAdd(o, acc[v]);
                else *o = (accumulate ? *o : 0.f) + acc[v];
            }
        }
    }
}

// RowRed2D.  `lanes` (a power of two <= 32) lanes share a row; a warp holds 32/lanes rows.
// blockIdx.y selects the column range [c0, c1) of a split (whole chunks except at the end).
template <typename T, int VEC>
__global__ void __launch_bounds__(256) rowred_kernel(const T *__restrict__ A, int64_t ld, int64_t sc, int R, int C,
                                                      float *__restrict__ out, int64_t os, int lanes, int cols_per_split,
                                                      int use_atomic, int accumulate) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int rows_per_warp = 32 / lanes;
    const int64_t row = ((int64_t)blockIdx.x * 8 + warp) * rows_per_warp + lane / lanes;
    const int sub = lane % lanes;
    const int c0 = blockIdx.y * cols_per_split;
    const int c1 = min(C, c0 + cols_per_split);
    float acc[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) acc[v] = 0.f;
    if (row < R && c0 < c1) {
        const T *base = A + row * ld;
        const int full_end = c0 + (c1 - c0) / VEC * VEC;      // whole chunks
        int64_t c = c0 + sub * VEC;
        const int64_t step = lanes * VEC;
        if constexpr (VEC > 1) {
            for (; c + 7 * step < full_end; c += 8 * step) {      // eight 16-byte loads in flight
                uint4 raw[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) raw[u] = __ldg(reinterpret_cast<const uint4 *>(base + c + u * step));
#pragma unroll
                for (int u = 0; u < 8; ++u) accumulate_raw<T, VEC>(acc, raw[u]);
            }
        } else {
            for (; c + 7 * step < full_end; c += 8 * step) {
                float part[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) part[u] = widen(__ldg(base + (c + u * step) * sc));
                acc[0] += ((part[0] + part[1]) + (part[2] + part[3])) + ((part[4] + part[5]) + (part[6] + part[7]));
            }
        }
        for (; c < full_end; c += step) add_chunk<T, VEC>(acc, base + c * sc, sc, VEC);
        if (VEC > 1 && sub == 0 && full_end < c1) {            // the ragged end of the range, element by element
            float tail = 0.f;
            for (int cc = full_end; cc < c1; ++cc) tail += widen(__ldg(base + (int64_t)cc * sc));
            acc[0] += tail;
        }
    }
    float sum = acc[0];
#pragma unroll
    for (int v = 1; v < VEC; ++v) sum += acc[v];
    for (int off = lanes >> 1; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    if (use_atomic) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (sub == 0 && row < R && (c0 < c1 || blockIdx.y == 0)) {
        float *o = out + row * os;
        if (use_atomic) atomicAdd(o, sum);
        else *o = (accumulate ? *o : 0.f) + sum;
    }
}

__global__ void zero_vector_kernel(float *__restrict__ out, int64_t n, int64_t os) {
    asm volatile("griddepcontrol.launch_dependents;");   // the reduction behind it may start; it waits before its atomics
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) out[i * os] = 0.f;
}

// Launches `kernel`; `after_clear`: a clearing kernel was just enqueued ahead of it and the launch may overlap it
// (programmatic dependent launch; the kernel waits for the clearing grid before its first atomic).
template <typename... KArgs, typename... Args>
cudaError_t launch_reduction(void (*kernel)(KArgs...), dim3 grid, bool after_clear, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(256, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_clear ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename T, int VEC>
cudaError_t launch_reduce_typed(bool colred, const T *A, int64_t ld, int64_t sc, int R, int C, float *out, int64_t os,
                                int accumulate, int num_sms, cudaStream_t stream) {
    const int target_ctas = num_sms * 8;
    if (!colred) {
        // RowRed2D: one output per row
        const int chunks = (C + VEC - 1) / VEC;
        int lanes = 1;
        while (lanes < 32 && lanes < chunks) lanes <<= 1;
        const int rows_per_cta = 8 * (32 / lanes);
        const int64_t row_ctas = ((int64_t)R + rows_per_cta - 1) / rows_per_cta;
        int splits = 1;
        const int min_chunks_per_split = lanes * 16;
        if (row_ctas < target_ctas && chunks > min_chunks_per_split)
            splits = (int)std::min<int64_t>((target_ctas + row_ctas - 1) / row_ctas, (chunks + min_chunks_per_split - 1) / min_chunks_per_split);
        int chunks_per_split = (chunks + splits - 1) / splits;
        chunks_per_split = (chunks_per_split + lanes - 1) / lanes * lanes;
        splits = (chunks + chunks_per_split - 1) / chunks_per_split;
        const int use_atomic = splits > 1;
        if (use_atomic && !accumulate) {
            zero_vector_kernel<<<(int)std::min<int64_t>(((int64_t)R + 255) / 256, 1184), 256, 0, stream>>>(out, R, os);
            count_launch();
        }
        const cudaError_t e = launch_reduction(rowred_kernel<T, VEC>, dim3((unsigned)row_ctas, (unsigned)splits), use_atomic && !accumulate, stream,
                                               A, ld, sc, R, C, out, os, lanes, chunks_per_split * VEC, use_atomic, accumulate);
        count_launch();
        note_kernel(VEC > 1 ? "rowred_kernel<vec>" : "rowred_kernel<scalar>");
        return e;
    } else {
        // ColRed2D: one output per column
        const int64_t chunks = ((int64_t)C + VEC - 1) / VEC;
        const int cw = (int)std::min<int64_t>(chunks, 256);
        const int rp = 256 / cw;
        const int64_t col_blocks = (chunks + cw - 1) / cw;
        // row ranges: as many as give every SM its full set of resident thread blocks, in one wave
        static int resident = 0;
        if (resident == 0) {
            int n = 0;
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, colred_kernel<T, VEC>, 256, 0) != cudaSuccess || n < 1) n = 2;
            resident = n;
        }
        int splits = 1;
        const int min_rows_per_split = rp * 16;
        const int64_t wave = (int64_t)num_sms * resident;
        if (col_blocks < wave && R > min_rows_per_split)
            splits = (int)std::min<int64_t>(wave / col_blocks, ((int64_t)R + min_rows_per_split - 1) / min_rows_per_split);
        int rows_per_split = (R + splits - 1) / splits;
        rows_per_split = (rows_per_split + rp - 1) / rp * rp;
        splits = (R + rows_per_split - 1) / rows_per_split;
        // 2: the output is dense and 16-byte aligned, so whole chunks may use vector atomics
        const int use_atomic = splits > 1 ? ((os == 1 && aligned16(out)) ? 2 : 1) : 0;
        if (use_atomic && !accumulate) {
            zero_vector_kernel<<<(int)std::min<int64_t>(((int64_t)C + 255) / 256, 1184), 256, 0, stream>>>(out, C, os);
            count_launch();
        }
        const cudaError_t e = launch_reduction(colred_kernel<T, VEC>, dim3((unsigned)col_blocks, (unsigned)splits), use_atomic && !accumulate, stream,
                                               A, ld, sc, R, C, out, os, cw, rp, rows_per_split, use_atomic, accumulate);
        count_launch();
        note_kernel(VEC > 1 ? "colred_kernel<vec>" : "colred_kernel<scalar>");
        return e;
    }
}

template <typename U>
cudaError_t launch_tile_move(const U *src, int64_t s_i, int64_t s_j, U *dst, int64_t d_i, int64_t d_j, int R, int C, int num_sms,
                             cudaStream_t stream, bool note = true) {
    const int tiles_j = (C + 31) / 32;
    const int64_t num_tiles = (int64_t)((R + 31) / 32) * tiles_j;
    const int grid = (int)std::min<int64_t>(num_tiles, (int64_t)num_sms * 8);
    // write along whichever destination index is closer to contiguous
    if (d_i < d_j) tile_move_kernel<U, true><<<grid, 256, 0, stream>>>(src, s_i, s_j, dst, d_i, d_j, R, C, tiles_j, num_tiles);
    else tile_move_kernel<U, false><<<grid, 256, 0, stream>>>(src, s_i, s_j, dst, d_i, d_j, R, C, tiles_j, num_tiles);
    count_launch();
    if (note) note_kernel("tile_move_kernel");
    return cudaGetLastError();
}

// device on which each kernel's shared-memory limit was last raised (the attribute is per device)
int g_attr_copy = -1, g_attr_tr4 = -1, g_attr_tr2 = -1;
inline int current_device() { int d = 0; cudaGetDevice(&d); return d; }

}  // namespace

sg_status launch_move2d(bool transpose, int64_t R, int64_t C, const void *src, int64_t s_r, int64_t s_c, void *dst, int64_t d_r,
                        int64_t d_c, int esize, int force, int *used_tma, cudaStream_t stream) {
    *used_tma = 0;
    int num_sms = 0;
    if (!tensor_driver_ready(&num_sms)) return SG_ERR_CUDA;
    const bool tma_ok = force != 1 && s_c == 1 && d_c == 1 && aligned16(src) && aligned16(dst) && (s_r * esize) % 16 == 0 &&
                        (d_r * esize) % 16 == 0 && s_r * esize < ((int64_t)1 << 40) && d_r * esize < ((int64_t)1 << 40) &&
                        (R == 1 || s_r >= C) && ((transpose ? C : R) == 1 || d_r >= (transpose ? R : C));
    const CUtensorMapDataType type = esize == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT16;
    // TMA checks the bounds of the contiguous dimension in 16-byte units, so a store would write the rest of the unit
    // in which a row of the destination ends: the TMA kernels take the part whose destination rows are whole units
    // (`body`), the strided kernel the last few columns of the destination.
    const int vec = 16 / esize;
    const int64_t inner = transpose ? R : C;             // extent of the destination's contiguous dimension
    const int64_t body = inner - inner % vec, tail = inner - body;
    if (tma_ok && body > 0 && (tail == 0 || force != 2)) {
        const int64_t Rb = transpose ? body : R, Cb = transpose ? C : body;      // the source part the TMA kernel moves
        bool launched = false;
        CUtensorMap map_src, map_dst;
        cuuint64_t st_src[1] = {(cuuint64_t)(s_r * esize)}, st_dst[1] = {(cuuint64_t)(d_r * esize)};
        if (!transpose) {
            // box: up to 256 elements wide, as many rows as fit a 32 KB stage
            const int box_x = (int)std::min<int64_t>(SG_CP_BOX_X, Cb);
            const int box_y = (int)std::min<int64_t>(std::min<int64_t>(256, CP_STAGE_BYTES / (box_x * esize)), Rb);
            cuuint64_t dims[2] = {(cuuint64_t)Cb, (cuuint64_t)Rb};
            cuuint32_t box[2] = {(cuuint32_t)box_x, (cuuint32_t)box_y};
            const int64_t tiles_x = (Cb + box_x - 1) / box_x, tiles_y = (Rb + box_y - 1) / box_y;
            if (tiles_x * tiles_y < ((int64_t)1 << 31) &&
                tensor_encode_tiled(&map_src, type, 2, const_cast<void *>(src), dims, st_src, box, CU_TENSOR_MAP_SWIZZLE_NONE,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B) &&
                tensor_encode_tiled(&map_dst, type, 2, dst, dims, st_dst, box, CU_TENSOR_MAP_SWIZZLE_NONE,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B)) {
                const int smem = CP_STAGES * CP_STAGE_BYTES + 1024;
                const int dev = current_device();
                if (g_attr_copy != dev) {
                    if (cudaFuncSetAttribute(copy_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return SG_ERR_CUDA;
                    g_attr_copy = dev;
                }
                const int num_tiles = (int)(tiles_x * tiles_y);
                copy_tma_kernel<<<std::min(num_tiles, CP_CTAS_PER_SM * num_sms), 64, smem, stream>>>(map_src, map_dst, (int)tiles_x, num_tiles, box_x, box_y,
                                                                                    (uint32_t)(box_x * box_y * esize));
                launched = true;
            }
        } else {
            const int W = 128 / esize;
            cuuint64_t dims_s[2] = {(cuuint64_t)Cb, (cuuint64_t)Rb}, dims_d[2] = {(cuuint64_t)Rb, (cuuint64_t)Cb};
            cuuint32_t box_s[2] = {(cuuint32_t)W, 128}, box_d[2] = {(cuuint32_t)W, 32};
            const int64_t tiles_c = (Cb + W - 1) / W, tiles_r = (Rb + 127) / 128;
            if (tiles_c * tiles_r < ((int64_t)1 << 31) &&
                tensor_encode_tiled(&map_src, type, 2, const_cast<void *>(src), dims_s, st_src, box_s, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B) &&
                tensor_encode_tiled(&map_dst, type, 2, dst, dims_d, st_dst, box_d, CU_TENSOR_MAP_SWIZZLE_128B,
                                    CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) {
                const int smem = (TR_IN_STAGES + 2) * TR_TILE_BYTES + 1024;
                int &attr = esize == 4 ? g_attr_tr4 : g_attr_tr2;
                const int dev = current_device();
                if (attr != dev) {
                    const cudaError_t e = esize == 4
                        ? cudaFuncSetAttribute(transpose_tma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                        : cudaFuncSetAttribute(transpose_tma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
                    if (e != cudaSuccess) return SG_ERR_CUDA;
                    attr = dev;
                }
                const int num_tiles = (int)(tiles_c * tiles_r);
                const int grid = std::min(num_tiles, 2 * num_sms);
                const int panel = (int)std::min<int64_t>(tiles_c, TR_PANEL);
                if (esize == 4) transpose_tma_kernel<4><<<grid, TR_THREADS, smem, stream>>>(map_src, map_dst, (int)tiles_c, (int)tiles_r, panel, (int)Rb, (int)Cb);
                else transpose_tma_kernel<2><<<grid, TR_THREADS, smem, stream>>>(map_src, map_dst, (int)tiles_c, (int)tiles_r, panel, (int)Rb, (int)Cb);
                launched = true;
            }
        }
        if (launched) {
            count_launch();
            note_kernel(transpose ? "transpose_tma_kernel" : "copy_tma_kernel");
            *used_tma = 1;
            if (cudaGetLastError() != cudaSuccess) return SG_ERR_CUDA;
            if (tail == 0) return SG_OK;
            // the last `tail` columns of the destination: source rows [body, R) of a transpose, columns [body, C) of a copy
            const char *s_tail = static_cast<const char *>(src) + (transpose ? body * s_r : body * s_c) * esize;
            char *d_tail = static_cast<char *>(dst) + body * d_c * esize;
            const int64_t Rt = transpose ? tail : R, Ct = transpose ? C : tail;
            const int64_t di = transpose ? d_c : d_r, dj = transpose ? d_r : d_c;
            const cudaError_t e = esize == 4
                ? launch_tile_move(reinterpret_cast<const uint32_t *>(s_tail), s_r, s_c, reinterpret_cast<uint32_t *>(d_tail), di, dj, (int)Rt, (int)Ct, num_sms, stream, false)
                : launch_tile_move(reinterpret_cast<const uint16_t *>(s_tail), s_r, s_c, reinterpret_cast<uint16_t *>(d_tail), di, dj, (int)Rt, (int)Ct, num_sms, stream, false);
            return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
        }
    }
    if (force == 2) return SG_ERR_UNSUPPORTED;
    // strided path: destination index pair (i, j) of the source element; a transpose exchanges the strides
    const int64_t di = transpose ? d_c : d_r, dj = transpose ? d_r : d_c;
    const cudaError_t e = esize == 4
        ? launch_tile_move(static_cast<const uint32_t *>(src), s_r, s_c, static_cast<uint32_t *>(dst), di, dj, (int)R, (int)C, num_sms, stream)
        : launch_tile_move(static_cast<const uint16_t *>(src), s_r, s_c, static_cast<uint16_t *>(dst), di, dj, (int)R, (int)C, num_sms, stream);
    return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
}

sg_status launch_reduce2d(bool colred, int64_t R, int64_t C, const void *A, int64_t a_r, int64_t a_c, int in_bf16, float *out,
                          int64_t os, int accumulate, cudaStream_t stream) {
    int num_sms = 0;
    if (!tensor_driver_ready(&num_sms)) return SG_ERR_CUDA;
    const int64_t n_out = colred ? C : R, n_red = colred ? R : C;
    if (n_red == 0) {      // empty sum: the neutral value
        if (!accumulate) {
            zero_vector_kernel<<<(int)std::min<int64_t>((n_out + 255) / 256, 1184), 256, 0, stream>>>(out, n_out, os);
            count_launch();
            if (cudaGetLastError() != cudaSuccess) return SG_ERR_CUDA;
        }
        return SG_OK;
    }
    const int es = in_bf16 ? 2 : 4;
    const bool vec_ok = a_c == 1 && aligned16(A) && (a_r * es) % 16 == 0;
    cudaError_t e;
    if (in_bf16) {
        const uint16_t *p = static_cast<const uint16_t *>(A);
        e = vec_ok ? launch_reduce_typed<uint16_t, 8>(colred, p, a_r, a_c, (int)R, (int)C, out, os, accumulate, num_sms, stream)
                   : launch_reduce_typed<uint16_t, 1>(colred, p, a_r, a_c, (int)R, (int)C, out, os, accumulate, num_sms, stream);
    } else {
        const float *p = static_cast<const float *>(A);
        e = vec_ok ? launch_reduce_typed<float, 4>(colred, p, a_r, a_c, (int)R, (int)C, out, os, accumulate, num_sms, stream)
                   : launch_reduce_typed<float, 1>(colred, p, a_r, a_c, (int)R, (int)C, out, os, accumulate, num_sms, stream);
    }
    return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
}

sg_status bandwidth_read_status(cudaStream_t stream) { return read_status_word(stream); }

}  // namespace sg

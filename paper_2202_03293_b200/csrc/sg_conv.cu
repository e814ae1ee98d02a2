// Stride-1 convolutions on the tensor cores with every input pixel fetched once per tile and the
// filter resident in shared memory; bf16 inputs directly, f32 inputs as three tf32 products per term.
//
// The im2col kernel fetches, for each of the KH*KW filter taps, a fresh 128-pixel input tile and
// a fresh filter tile: on conv_2d 3x3 that is nine copies of nearly the same pixels and nine
// filter tiles per output tile, and the TMA issue / L2 -> shared memory fill rate bounds it.
// Here positions are counted with the INPUT's row pitch, q = (n*H_in + h)*W_in + w, so the input
// pixel of tap (kh, kw) is row q + kh*dh*W_in + kw*dw of the input seen as a [N*H_in*W_in, C]
// matrix.  A tile is 128 consecutive q that start at the beginning of an output row:
//   * W_in <= 128: R whole image rows (R*W_in <= 128); positions with w >= W_out are computed and dropped;
//   * W_in  > 128: a segment of 128 output positions of one image row.
// Per block of channels (64 bf16 / 32 f32) ONE TMA load brings, for every filter row kh, the strip
// of 128 + (KW-1)*dw rows that the KW taps of that row need (a 3-D box over an overlapping view of
// the input whose third dimension steps by dh*W_in rows).  The filter (all taps, all channels, the
// tile's columns) is loaded once per CTA and stays in shared memory.
//   bf16: each tap's MMAs read its strip through a matrix descriptor whose start address is
//         shifted by kw*dw rows.
//   f32:  x = hi + lo with hi = x rounded to tf32.  The filter is split once per CTA (and transposed
//         to K-major, which kind::tf32 needs) into a tf32 tile of hi and a bf16 tile [hi | lo];
//         sixteen converter warps split the strip rows of each tap the same way into tensor memory
//         (the tap's shift is a row offset of their reads), and the MMA warp accumulates the
//         corrections lo*hi + hi*lo as one bf16 contraction over [lo | hi] . [hi | lo] and the main
//         term hi*hi in tf32, the A operand in tensor memory: 8 MMAs per 32 channels of a tap.
//
// Because tiles start at row beginnings, the epilogue is TMA only: TMEM -> registers -> a swizzled
// staging copy of the whole tile, laid out [image row][32-column chunk][w][32 f32] -> ONE tensor
// store (or reduce-add) per tile through a 5-D map {f in chunk, w, chunk, h, n} of the output (a
// TMA instruction costs its issuing thread about 0.3 us whatever it moves, so the number of
// instructions is what counts); the TMA unit clips w >= W_out of a last segment and h >= H_out of
// a last tile.  Outputs whose F is no multiple of 32 are stored chunk by chunk and row by row.
//
// Warp roles: warp 0 producer (TMA), warp 1 MMA issuer and TMEM owner, warps 2-5 epilogue,
// warps 6-21 converters (f32 only).  Every wait is bounded.
#include <algorithm>

#include "sg_internal.cuh"
#include "sg_tc_ptx.cuh"

namespace sg {
namespace {

constexpr int BM = 128;
constexpr int MAX_KH = 8;
constexpr int MAX_STAGES = 8;
constexpr int CONVERTER_WARPS = 16;
constexpr int A_SLOTS = 4;                   // f32: split input k-blocks in flight in tensor memory (64 columns each)
constexpr int SMEM_LIMIT = 232448 - 1024;    // opt-in maximum minus the alignment slack

struct ConvParams {
    int Q;                 // N * H_in * W_in positions of the input matrix
    int num_tiles;         // position tiles (one per CTA; a pair takes two neighbours)
    int num_pos_items;     // ceil(num_tiles / CG)
    int num_f_tiles;
    int N, Hin, Win, Hout, Wout;
    int KH, KW, kbpt;      // filter rows, taps per row, channel blocks per tap
    int dw;                // input rows between taps of a filter row
    int rows_per_tile;     // R: image rows per tile (1 when a tile is a segment of a row)
    int segs;              // segments of 128 positions per image row (1 when a tile holds whole rows)
    int tiles_per_image;
    int chunk_rows;        // staging rows of one 32-column chunk of one image row: W_out (128 for segments)
    int staging_bytes;     // the staged tile (f32: at least the raw filter, which is staged there before it is split)
    int blocked_store;     // 1: F is a multiple of 32, one 5-D store moves the tile; 0: one 4-D store per image row and chunk
    int strip_rows;        // 128 + (KW - 1) * dw
    int strip_stage_bytes; // KH strips of strip_rows x 128 B, rounded up to 1 KiB
    int stages;
    int flt_bytes;         // resident filter
    int flt_blocked;       // bf16: 1 = the filter map is blocked by 64 columns (one load per filter row and channel block)
    int F;
    int accumulate;
    int wait_prior;        // 1: launched to overlap the kernel ahead of it: wait for it before touching global memory
};

template <int BN, int CG, bool F32>
struct ConvCfg {
    static constexpr int B_COLS = BN / CG;                           // filter columns resident in this CTA
    static constexpr int BLOCK_BYTES = B_COLS * 128 * (F32 ? 2 : 1); // one (tap, channel block); f32: [hi, tf32 | hi and lo, bf16]
    static constexpr int ACC_COLS = 2 * BN;
    static constexpr int USED_COLS = ACC_COLS + (F32 ? A_SLOTS * 64 : 0);
    static constexpr int TMEM_COLS = USED_COLS <= 128 ? 128 : USED_COLS <= 256 ? 256 : 512;
    static constexpr int THREADS = 64 + 128 + (F32 ? 32 * CONVERTER_WARPS : 0);
    static_assert(USED_COLS <= 512 && B_COLS % 64 == 0, "tile width");
};

__device__ __forceinline__ void tma_store_4d(const CUtensorMap *map, uint32_t src, int x, int y, int z, int w) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_4d(const CUtensorMap *map, uint32_t src, int x, int y, int z, int w) {
    asm volatile("cp.reduce.async.bulk.tensor.4d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void tma_store_5d(const CUtensorMap *map, uint32_t src, int x, int y, int z, int w, int v) {
    asm volatile("cp.async.bulk.tensor.5d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_5d(const CUtensorMap *map, uint32_t src, int x, int y, int z, int w, int v) {
    asm volatile("cp.reduce.async.bulk.tensor.5d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4, %5, %6}], [%1];"
                 ::"l"(map), "r"(src), "r"(x), "r"(y), "r"(z), "r"(w), "r"(v) : "memory");
}
// CG = 1: one CTA computes a tile of 128 positions x BN columns.  CG = 2: a CTA pair (one cluster) computes two
// neighbouring tiles x BN columns with tcgen05.mma.cta_group::2: each CTA loads the strips of its own tile and keeps
// its own BN/2 columns of the filter, which halves the resident filter and leaves room for a deeper ring of strips.
template <int BN, int CG, bool F32>
__global__ void __launch_bounds__(ConvCfg<BN, CG, F32>::THREADS, 1)
conv_strip_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_flt,
                  const __grid_constant__ CUtensorMap map_out, const ConvParams p) {
    using C = ConvCfg<BN, CG, F32>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t flt_addr = smem_base;
    const uint32_t strips_addr = flt_addr + p.flt_bytes;
    const uint32_t ring_bytes = (uint32_t)(p.stages * p.strip_stage_bytes);
    const uint32_t staging_off = p.flt_bytes + ring_bytes;
    const uint32_t staging_addr = smem_base + staging_off;
    uint8_t *staging_gen = smem_gen + staging_off;
    const uint32_t bars_addr = staging_addr + (uint32_t)p.staging_bytes;
    uint8_t *bars_gen = staging_gen + p.staging_bytes;
    // barrier block: full[8] | empty[8] | split_full[4] | split_empty[4] | acc_full[2] | acc_empty[2] | flt_full |
    //                flt_free | (unused) | tmem_ptr | abort
    auto full_bar = [&](int s) { return bars_addr + 8u * s; };
    auto empty_bar = [&](int s) { return bars_addr + 8u * (8 + s); };
    auto split_full_bar = [&](int s) { return bars_addr + 8u * (16 + s); };
    auto split_empty_bar = [&](int s) { return bars_addr + 8u * (20 + s); };
    auto acc_full_bar = [&](int b) { return bars_addr + 8u * (24 + b); };
    auto acc_empty_bar = [&](int b) { return bars_addr + 8u * (26 + b); };
    const uint32_t flt_full_bar = bars_addr + 8u * 28;
    const uint32_t flt_free_bar = bars_addr + 8u * 29;
    volatile uint32_t *tmem_ptr_slot = reinterpret_cast<volatile uint32_t *>(bars_gen + 8 * 31);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_gen + 8 * 31 + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // a launch behind this one that asked for it may start to set itself up as our CTAs leave their SMs
    asm volatile("griddepcontrol.launch_dependents;");
    if (threadIdx.x == 0) { prefetch_tensormap(&map_in); prefetch_tensormap(&map_flt); prefetch_tensormap(&map_out); }
    // In a pair, CTA 0 (the leader) issues the MMAs and owns the barriers the bf16 loads signal.
    const uint32_t cta_rank = CG == 2 ? cluster_ctarank() : 0u;
    const int group_id = (int)blockIdx.x / CG, num_groups = (int)gridDim.x / CG;
    if (warp == 0) {
        // One barrier per lane.  full: one arrive.expect_tx by the producer.  empty: one tcgen05.commit (bf16) or one
        // arrive per converter warp of this CTA (f32).  split_full / flt_ready: one arrive per converter warp of every
        // CTA of the group.  acc_empty: one arrive per epilogue warp of every CTA of the group.
        const uint32_t count = lane < 8 ? 1u : lane < 16 ? (F32 ? CONVERTER_WARPS : 1u) : lane < 20 ? (uint32_t)(CONVERTER_WARPS * CG)
                             : lane < 26 ? 1u : lane < 28 ? (uint32_t)(4 * CG) : lane < 30 ? 1u : (uint32_t)(CONVERTER_WARPS * CG);
        if (lane < 31) mbar_init(bars_addr + 8u * lane, count);
        if (lane == 31) *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if constexpr (CG == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(const_cast<uint32_t *>(tmem_ptr_slot))), "r"((uint32_t)C::TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(const_cast<uint32_t *>(tmem_ptr_slot))), "r"((uint32_t)C::TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();   // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_slot;

    // this group's items: a contiguous, balanced run of (column tile, position item), positions fastest, so that the
    // resident filter changes as rarely as possible
    const int total_items = p.num_pos_items * p.num_f_tiles;
    const int item0 = (int)((long long)group_id * total_items / num_groups);
    const int item1 = (int)((long long)(group_id + 1) * total_items / num_groups);
    // tile -> first position, image, first row, first column
    struct Tile { int q0, n, h0, w0; bool live; };
    auto decode = [&](int pos_item) {
        Tile t;
        const int tile = pos_item * CG + (int)cta_rank;
        t.live = tile < p.num_tiles;
        t.n = tile / p.tiles_per_image;
        const int r = tile - t.n * p.tiles_per_image;
        if (p.segs == 1) { t.h0 = r * p.rows_per_tile; t.w0 = 0; }
        else { t.h0 = r / p.segs; t.w0 = (r - t.h0 * p.segs) * BM; }
        t.q0 = t.live ? (t.n * p.Hin + t.h0) * p.Win + t.w0 : p.Q;      // a dead tile reads zeros only
        return t;
    };
    const uint32_t strips_tx = (uint32_t)(p.KH * p.strip_rows) * 128u;
    // bf16 pairs count both CTAs' strip bytes on the leader's barrier, which its MMA thread waits on; f32 pairs signal
    // each CTA's own barrier (its converter warps wait there)
    constexpr bool REMOTE_FULL = CG == 2 && !F32;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            if (p.wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");    // inputs may come from the kernel ahead
            int it = 0, cur_ft = -1, epochs = 0;
            bool ok = true;
            auto load_strips = [&](int q0, int cb) {       // one load: the strips of all filter rows
                const int s = it % p.stages;
                if (!mbar_wait(empty_bar(s), ((it / p.stages) & 1) ^ 1u, abort_flag)) return false;
                if (!REMOTE_FULL || cta_rank == 0) mbar_expect_tx(full_bar(s), (REMOTE_FULL ? CG : 1) * strips_tx);
                tma_tile_3d<REMOTE_FULL>(strips_addr + s * p.strip_stage_bytes, &map_in,
                                         REMOTE_FULL ? map_to_cta(full_bar(s), 0) : full_bar(s), cb * (F32 ? 32 : 64), q0, 0);
                return true;
            };
            for (int item = item0; item < item1 && ok; ++item) {
                const int ft = item / p.num_pos_items;
                const Tile t = decode(item - ft * p.num_pos_items);
                int cb = 0;
                if (ft != cur_ft) {
                    // the MMAs of the previous column tile must have finished reading the filter
                    if (epochs > 0 && !mbar_wait(flt_free_bar, (epochs - 1) & 1, abort_flag)) { ok = false; break; }
                    cur_ft = ft;
                    ++epochs;
                    const int f0 = ft * BN + (int)cta_rank * C::B_COLS;
                    // the first tile's first strips go out ahead of the filter (each TMA instruction costs this thread ~0.3 us)
                    ok = load_strips(t.q0, 0); ++it; cb = 1;
                    // one box per channel block: {columns of a sub-tile, channels of a block, B_COLS / sub-tile columns, KW, KH}
                    const uint32_t load_bytes = (uint32_t)(p.KH * p.KW) * (uint32_t)C::B_COLS * 128u;
                    if constexpr (F32) {
                        // raw filter of this CTA's columns into the staging area, which is idle until the first epilogue
                        // (there is one column tile only: the host side sees to it); the converter warps split it
                        mbar_expect_tx(flt_full_bar, (uint32_t)p.kbpt * load_bytes);
                        for (int c2 = 0; c2 < p.kbpt; ++c2)
                            tma_tile_5d<false>(staging_addr + (uint32_t)c2 * load_bytes, &map_flt, flt_full_bar, 0, c2 * 32, f0 / 32, 0, 0);
                    } else {
                        const uint32_t fbar = CG == 2 ? map_to_cta(flt_full_bar, 0) : flt_full_bar;
                        if (cta_rank == 0) mbar_expect_tx(flt_full_bar, CG * p.kbpt * load_bytes);
                        for (int c2 = 0; c2 < p.kbpt; ++c2) {
                            const uint32_t dst = flt_addr + (uint32_t)c2 * load_bytes;
                            if (p.flt_blocked) {
                                tma_tile_5d<CG == 2>(dst, &map_flt, fbar, 0, c2 * 64, f0 / 64, 0, 0);
                            } else {
                                for (int kh = 0; kh < p.KH; ++kh)
                                    for (int kw = 0; kw < p.KW; ++kw)
#pragma unroll
                                        for (int j = 0; j < C::B_COLS / 64; ++j) {
                                            const uint32_t d2 = dst + (uint32_t)(kh * p.KW + kw) * C::BLOCK_BYTES + j * 8192;
                                            if constexpr (CG == 2) tma_load_4d_cg2(d2, &map_flt, fbar, f0 + j * 64, c2 * 64, kw, kh);
                                            else tma_load_4d(d2, &map_flt, fbar, f0 + j * 64, c2 * 64, kw, kh);
                                        }
                            }
                        }
                    }
                }
                for (; cb < p.kbpt && ok; ++cb, ++it) ok = load_strips(t.q0, cb);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA).  The
        // whole warp walks the loop so that addresses stay warp-uniform; one elected lane issues.
        if (cta_rank == 0) {
            constexpr uint32_t idesc = F32 ? make_idesc(BN, CG * BM, true, false, false)     // split tiles are K-major
                                           : make_idesc(BN, CG * BM, false, false, true);   // bf16 filter read as stored: N-major
            const bool issuer = elect_one();
            auto wait_all = [&](bool passed) { return __all_sync(0xffffffffu, passed) != 0; };
            // arrive, once the MMAs issued so far have finished, on the same barrier of every CTA of the group
            auto commit_all = [&](uint32_t bar) {
                if (!issuer) return;
                if constexpr (CG == 1) {
                    umma_commit(bar);
                } else {
                    umma_commit_cg2(map_to_cta(bar, 0));
                    umma_commit_cg2(map_to_cta(bar, 1));
                }
            };
            int it = 0, kbi = 0, tl = 0, cur_ft = -1, epochs = 0;
            bool flt_ready = false;      // this epoch's filter has landed (f32: has been split)
            bool ok = true;
            for (int item = item0; item < item1 && ok; ++item, ++tl) {
                const int ft = item / p.num_pos_items;
                if (ft != cur_ft) { cur_ft = ft; ++epochs; flt_ready = false; }
                const int buf = tl & 1;
                if (!wait_all(mbar_wait<CG == 2>(acc_empty_bar(buf), ((tl >> 1) & 1) ^ 1u, abort_flag))) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                uint32_t acc = 0;
                for (int cb = 0; cb < p.kbpt && ok; ++cb, ++it) {
                    if constexpr (F32) {
                        // (a slot's barrier also stands for the filter block its k-block uses: the converter warps split
                        // that block, during this CTA's first tile, before they signal the slot)
                        for (int kh = 0; kh < p.KH && ok; ++kh)
                            for (int kw = 0; kw < p.KW; ++kw, ++kbi) {
                                const int s = kbi & (A_SLOTS - 1);
                                if (!wait_all(mbar_wait<CG == 2>(split_full_bar(s), (kbi / A_SLOTS) & 1, abort_flag))) { ok = false; break; }
                                tc_fence_after();
                                // filter block (K-major, 8-column groups 1024 B apart): hi in tf32 | [hi, lo] in bf16; input in
                                // tensor memory, lane = position: hi in 32 columns of tf32 | [lo, hi] in 2 x 16 columns of bf16 pairs
                                constexpr uint32_t idesc16 = make_idesc(BN, CG * BM, false, false, false);
                                const uint32_t blk = flt_addr + (uint32_t)((cb * p.KH + kh) * p.KW + kw) * C::BLOCK_BYTES;
                                const uint64_t bh = make_smem_desc(blk, 16, 1024);
                                const uint64_t b16 = make_smem_desc(blk + C::B_COLS * 128, 16, 1024);
                                const uint32_t a_hi = tmem_base + (uint32_t)(C::ACC_COLS + s * 64), a16 = a_hi + 32;
                                if (issuer) {
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {      // the corrections [lo | hi] . [hi | lo] first: small terms
                                        if constexpr (CG == 1) umma_bf16_ts(d_tmem, a16 + k * 8, b16 + (uint64_t)(k * 2), idesc16, acc);
                                        else umma_bf16_ts_cg2(d_tmem, a16 + k * 8, b16 + (uint64_t)(k * 2), idesc16, acc);
                                        acc = 1u;
                                    }
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        if constexpr (CG == 1) umma_tf32_ts(d_tmem, a_hi + k * 8, bh + (uint64_t)(k * 2), idesc, 1u);
                                        else umma_tf32_ts_cg2(d_tmem, a_hi + k * 8, bh + (uint64_t)(k * 2), idesc, 1u);
                                    }
                                }
                                commit_all(split_empty_bar(s));
                            }
                    } else {
                        const int s = it % p.stages;
                        if (!wait_all(mbar_wait(full_bar(s), (it / p.stages) & 1, abort_flag))) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t strips = strips_addr + s * p.strip_stage_bytes;
                        if (!flt_ready) {
                            if (!wait_all(mbar_wait(flt_full_bar, (epochs - 1) & 1, abort_flag))) { ok = false; break; }
                            tc_fence_after();
                            flt_ready = true;
                        }
                        for (int kh = 0; kh < p.KH; ++kh) {
                            for (int kw = 0; kw < p.KW; ++kw) {
                                // the tap's 128 pixels start kw*dw rows into the strip of filter row kh: same
                                // K-major layout, start address shifted by whole rows.  The 128-byte swizzle is
                                // a function of the absolute shared-memory address, for the TMA that wrote the
                                // strips and for the tensor core alike, so the shifted descriptor (base-offset
                                // field clear) reads exactly the rows it names.
                                const uint32_t a_addr = strips + (uint32_t)(kh * p.strip_rows + kw * p.dw) * 128u;
                                const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024);
                                const uint32_t b_addr = flt_addr + ((cb * p.KH + kh) * p.KW + kw) * C::BLOCK_BYTES;
                                const uint64_t b_desc = make_smem_desc(b_addr, 8192, 1024);
                                if (issuer) {
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        if constexpr (CG == 2) umma_bf16_cg2(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 128), idesc, acc);
                                        else umma_bf16(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * 128), idesc, acc);
                                        acc = 1u;
                                    }
                                }
                            }
                        }
                        if (ok) commit_all(empty_bar(s));
                    }
                }
                if (ok) {
                    commit_all(acc_full_bar(buf));
                    const bool last_of_ft = item + 1 >= item1 || (item + 1) / p.num_pos_items != ft;
                    if (last_of_ft) commit_all(flt_free_bar);
                }
            }
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------ converters (f32 only; warps 6 to 21)
        if constexpr (F32) {
            const int cw = warp - 6;
            const int quarter = warp & 3, kpart = cw >> 2;     // TMEM lane quarter this warp may touch; its 8 of the 32 k columns
            bool ok = item0 < item1;
            // ---- the filter, once per CTA, block by block during the first tile: raw sub-tiles [32 k][32 columns] (128-byte
            // rows, as stored) -> hi and lo tiles, K-major ([column][32 k] rows of 128 B in 8-row groups, 16-byte chunk c of
            // row f at chunk c ^ (f & 7)).  A block (one tap, 32 channels, 64 columns) is sixteen units of an eighth of a
            // sub-tile (4 k), one per converter warp: lane = column reads down its column (every load one 128-byte row across
            // the warp) and writes one chunk of its row of both tiles.
            static_assert(8 * C::B_COLS / 32 == CONVERTER_WARPS, "one filter unit per converter warp");
            if (ok && !mbar_wait(flt_full_bar, 0, abort_flag)) ok = false;
            auto split_filter_block = [&](int b) {
                const int j = cw >> 3, eighth = cw & 7;
                const float *col = reinterpret_cast<const float *>(staging_gen + (size_t)b * (C::B_COLS * 128) + j * 4096) + eighth * 4 * 32 + lane;
                uint32_t x[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) x[k] = __float_as_uint(col[k * 32]);
                const int f = j * 32 + lane;
                const int rowoff = (f >> 3) * 1024 + (f & 7) * 128;
                uint4 h;
                uint2 h16, l16;
                split4_mix(make_uint4(x[0], x[1], x[2], x[3]), h, h16, l16);
                uint8_t *blk = smem_gen + (size_t)b * C::BLOCK_BYTES;
                *reinterpret_cast<uint4 *>(blk + rowoff + ((eighth ^ (f & 7)) << 4)) = h;
                // the bf16 tile's row of this column: [hi of the 32 k | lo of the 32 k], 8 bytes for these 4 k in each half
                uint8_t *r16 = blk + C::B_COLS * 128 + rowoff + (eighth & 1) * 8;
                *reinterpret_cast<uint2 *>(r16 + (((eighth >> 1) ^ (f & 7)) << 4)) = h16;
                *reinterpret_cast<uint2 *>(r16 + (((4 + (eighth >> 1)) ^ (f & 7)) << 4)) = l16;
            };
            // ---- the strips: per (channel block, tap) this warp's 32 positions x 8 channels -> tensor memory
            int it = 0, kbi = 0;
            for (int item = item0; item < item1 && ok; ++item) {
                for (int cb = 0; cb < p.kbpt && ok; ++cb, ++it) {
                    const int r = it % p.stages;
                    if (!mbar_wait(full_bar(r), (it / p.stages) & 1, abort_flag)) { ok = false; break; }
                    const uint8_t *stage = smem_gen + p.flt_bytes + (size_t)r * p.strip_stage_bytes;
                    for (int kh = 0; kh < p.KH && ok; ++kh)
                        for (int kw = 0; kw < p.KW; ++kw, ++kbi) {
                            const int s = kbi & (A_SLOTS - 1);
                            if (item == item0) {
                                // first tile: this k-block's filter block (raw in the staging area) is split on the way
                                split_filter_block((cb * p.KH + kh) * p.KW + kw);
                                fence_async_smem();       // generic-proxy writes -> visible to the tensor core's reads
                            }
                            // row of the stage that holds this lane's position under tap (kh, kw); TMA wrote the stage
                            // with the 128-byte swizzle (chunk c of row x at chunk c ^ (x & 7))
                            const int row = kh * p.strip_rows + kw * p.dw + quarter * 32 + lane;
                            const uint8_t *rp = stage + (size_t)row * 128;
                            uint4 a_raw[2];
#pragma unroll
                            for (int i = 0; i < 2; ++i)
                                a_raw[i] = *reinterpret_cast<const uint4 *>(rp + (((kpart * 2 + i) ^ (row & 7)) << 4));
                            uint32_t hi[8], lo16[4], hi16[4];
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                uint4 h;
                                uint2 a, b;
                                split4_mix(a_raw[i], h, a, b);
                                hi[4 * i] = h.x; hi[4 * i + 1] = h.y; hi[4 * i + 2] = h.z; hi[4 * i + 3] = h.w;
                                hi16[2 * i] = a.x; hi16[2 * i + 1] = a.y;
                                lo16[2 * i] = b.x; lo16[2 * i + 1] = b.y;
                            }
                            // the MMAs that read this slot's tensor-memory columns four k-blocks ago are done
                            if (!mbar_wait<CG == 2>(split_empty_bar(s), ((kbi / A_SLOTS) & 1) ^ 1u, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            // this thread's 8 k: tf32 hi in columns 8*kpart.., bf16 pairs in columns 32 + 4*kpart.. (lo) and 48 + 4*kpart.. (hi)
                            const uint32_t t_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(C::ACC_COLS + s * 64);
                            tmem_st_32x8(t_base + kpart * 8, hi);
                            tmem_st_32x4(t_base + 32 + kpart * 4, lo16);
                            tmem_st_32x4(t_base + 48 + kpart * 4, hi16);
                            tmem_st_wait();
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) {
                                if constexpr (CG == 1) mbar_arrive(split_full_bar(s));
                                else mbar_arrive_cluster(map_to_cta(split_full_bar(s), 0));
                            }
                        }
                    __syncwarp();
                    if (ok && lane == 0) mbar_arrive(empty_bar(r));          // the raw stage may be refilled
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2 to 5)
        // The four warps stage the whole tile in shared memory the way one tensor store reads it: [image row i][32-column
        // chunk j][w][32 f32], rows of 128 bytes with the 128-byte swizzle (a function of the row's absolute index, as the
        // TMA unit applies it).  Each warp writes its TMEM lane quarter's positions; one thread then issues the store.
        const int q = warp & 3;        // TMEM lane quarter this warp may access
        const bool issuer = warp == 2 && lane == 0;
        constexpr int CHUNKS = BN / 32;
        int tl = 0;
        bool ok = true;
        if (p.wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");      // the output may still be in use by the kernel ahead
        for (int item = item0; item < item1 && ok; ++item, ++tl) {
            const int ft = item / p.num_pos_items;
            const Tile t = decode(item - ft * p.num_pos_items);
            // this lane's position -> its staging row in chunk 0, or -1 when the position is no output
            const int pos = q * 32 + lane;
            int row0 = -1, rows_here = 0;
            if (t.live) {
                if (p.segs == 1) {
                    const int i = pos / p.Win, w = pos - i * p.Win;
                    rows_here = min(p.rows_per_tile, p.Hout - t.h0);
                    if (i < rows_here && w < p.Wout) row0 = i * CHUNKS * p.chunk_rows + w;
                } else {
                    rows_here = 1;
                    row0 = pos;          // (positions beyond W_out are clipped by the store)
                }
            }
            const int buf = tl & 1;
            if (!epilogue_all(mbar_wait(acc_full_bar(buf), (tl >> 1) & 1, abort_flag))) { ok = false; break; }
            tc_fence_after();
            if (issuer) bulk_wait_read<0>();          // the previous tile's store has read the staging area
            asm volatile("bar.sync 1, 128;" ::: "memory");
            // two chunks leave tensor memory per wait (64 registers in flight)
#pragma unroll 1
            for (int j = 0; j < CHUNKS; j += 2) {
                uint32_t r[2][32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + j * 32), r[0]);
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + (j + 1) * 32), r[1]);
                tmem_ld_wait();
                if (row0 >= 0) {
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj) {
                        const int row = row0 + (j + jj) * p.chunk_rows;
                        uint8_t *dst = staging_gen + (size_t)row * 128;
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            *reinterpret_cast<uint4 *>(dst + ((c ^ (row & 7)) << 4)) =
                                make_uint4(r[jj][4 * c], r[jj][4 * c + 1], r[jj][4 * c + 2], r[jj][4 * c + 3]);
                    }
                }
            }
            // every tcgen05.ld of this buffer has completed: hand it back to the MMA thread
            tc_fence_before();
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                if constexpr (CG == 1) mbar_arrive(acc_empty_bar(buf));
                else mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (issuer && rows_here > 0) {
                if (p.blocked_store) {
                    // box {32 columns, chunk_rows positions, CHUNKS column chunks, R image rows, 1}
                    if (p.accumulate) tma_reduce_add_5d(&map_out, staging_addr, 0, t.w0, ft * CHUNKS, t.h0, t.n);
                    else tma_store_5d(&map_out, staging_addr, 0, t.w0, ft * CHUNKS, t.h0, t.n);
                } else {
                    for (int i = 0; i < rows_here; ++i)
                        for (int j = 0; j < CHUNKS; ++j) {
                            const int x = ft * BN + j * 32;
                            if (x >= p.F) break;
                            const uint32_t src = staging_addr + (uint32_t)((i * CHUNKS + j) * p.chunk_rows) * 128u;
                            if (p.accumulate) tma_reduce_add_4d(&map_out, src, x, t.w0, t.h0 + i, t.n);
                            else tma_store_4d(&map_out, src, x, t.w0, t.h0 + i, t.n);
                        }
                }
                bulk_commit();
            }
        }
        // the staging area must stay until the last store has read it; the writes themselves are complete
        // when the grid is
        if (issuer) bulk_wait_read<0>();
    }

    // ---------------------------------------------------------------- teardown
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(5000);   // let TMA loads in flight land
        __syncthreads();
    }
    // a pair leaves together: the leader's MMAs read the peer's shared memory and both CTAs
    // signal barriers in each other's shared memory
    if constexpr (CG == 2) cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        if constexpr (CG == 2)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)C::TMEM_COLS) : "memory");
    }
}

inline bool mult(int64_t v, int64_t q) { return v % q == 0; }

template <int BN, int CG, bool F32>
sg_status launch_kernel(const CUtensorMap &map_in, const CUtensorMap &map_flt, const CUtensorMap &map_out, const ConvParams &cp,
                        int grid, int smem_bytes, int slot, cudaStream_t stream) {
    using C = ConvCfg<BN, CG, F32>;
    if (!tensor_ensure_smem_attr(144 + slot, reinterpret_cast<const void *>(conv_strip_kernel<BN, CG, F32>), SMEM_LIMIT + 1024))
        return SG_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(C::THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cp.wait_prior ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, conv_strip_kernel<BN, CG, F32>, map_in, map_flt, map_out, cp);
    count_launch();
    note_kernel(F32 ? "conv_strip_kernel<f32>" : "conv_strip_kernel<bf16>");
    return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
}

}  // namespace

sg_status launch_conv_strip(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream) {
    // ---- eligibility: unit conv strides, dense pixel pitch, TMA alignment rules ----
    if (p.spatial_rank == 0) return SG_ERR_UNSUPPORTED;
    if (p.sh != 1 || p.sw != 1) return SG_ERR_UNSUPPORTED;
    if (p.i_c != 1 || p.k_f != 1 || p.o_f != 1) return SG_ERR_UNSUPPORTED;
    if (p.KH > MAX_KH || p.KH < 1 || p.KW < 1 || p.KW > 256) return SG_ERR_UNSUPPORTED;
    const bool f32 = !p.in_bf16;
    const int64_t es = f32 ? 4 : 2;
    const int bkc = 128 / (int)es;                // channels per block
    // the input must be one [N*H_in*W_in, C] matrix with a uniform row pitch
    if (p.Hin > 1 && p.i_h != (int64_t)p.Win * p.i_w) return SG_ERR_UNSUPPORTED;
    if (p.batch > 1 && p.i_n != (int64_t)p.Hin * p.Win * p.i_w) return SG_ERR_UNSUPPORTED;
    if (p.i_w < p.C || p.k_c < p.N) return SG_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(In) % 16 || reinterpret_cast<uintptr_t>(Flt) % 16 || reinterpret_cast<uintptr_t>(O) % 16)
        return SG_ERR_UNSUPPORTED;
    if (!mult(p.i_w * es, 16) || !mult(p.k_c * es, 16)) return SG_ERR_UNSUPPORTED;
    if (!mult((int64_t)p.C * es, 16) || !mult((int64_t)p.N * es, 16)) return SG_ERR_UNSUPPORTED;   // TMA bounds work in 16-byte units
    if (p.KW > 1 && !mult(p.k_kw * es, 16)) return SG_ERR_UNSUPPORTED;
    if (p.KH > 1 && !mult(p.k_kh * es, 16)) return SG_ERR_UNSUPPORTED;
    // the output as a 4-D tensor {f, w, h, n} for the tensor stores
    if (!mult(p.o_w, 4) || (p.Ho > 1 && !mult(p.o_h, 4)) || (p.batch > 1 && !mult(p.o_n, 4)) || !mult(p.N, 4)) return SG_ERR_UNSUPPORTED;
    if (p.o_w < p.N) return SG_ERR_UNSUPPORTED;
    const int64_t pitch_limit = (int64_t)1 << 40;
    if (p.i_w * es >= pitch_limit || p.k_c * es >= pitch_limit) return SG_ERR_UNSUPPORTED;
    const int64_t Q = (int64_t)p.batch * p.Hin * p.Win;
    if (Q > 0x7fffffff - 4096) return SG_ERR_UNSUPPORTED;
    if (BM + (int64_t)(p.KW - 1) * p.dw > 256) return SG_ERR_UNSUPPORTED;
    const int64_t shift_rows = (int64_t)p.dh * p.Win;              // input rows between filter rows
    const int64_t q_extent = Q - (int64_t)(p.KH - 1) * shift_rows;
    if (q_extent < 1 || shift_rows * p.i_w * es >= pitch_limit) return SG_ERR_UNSUPPORTED;

    // ---- tiles: whole image rows (W_in <= 128) or segments of a row ----
    int rows_per_tile = 1, segs = 1, chunk_rows = BM;
    if (p.Win <= BM) {
        rows_per_tile = std::min(BM / p.Win, p.Ho);
        chunk_rows = p.Wo;
    } else {
        segs = (p.Wo + BM - 1) / BM;
    }
    // rows of a strip that feed outputs (the tensor core reads 128 rows per tap whatever lies behind them in shared
    // memory; what it makes of the rest lands in positions that are dropped)
    const int64_t strip_rows = (p.Win <= BM ? (int64_t)rows_per_tile * p.Win : BM) + (int64_t)(p.KW - 1) * p.dw;
    const int64_t tiles_per_image = p.Win <= BM ? (p.Ho + rows_per_tile - 1) / rows_per_tile : (int64_t)p.Ho * segs;
    const int64_t num_tiles = (int64_t)p.batch * tiles_per_image;
    if (num_tiles > 0x3fffffff) return SG_ERR_UNSUPPORTED;
    // tensor-core rows that compute outputs: below half, the im2col kernel (whose tile rows are all outputs) is the better one
    if ((double)p.M < 0.5 * (double)num_tiles * BM) return SG_ERR_UNSUPPORTED;

    int dev = 0, num_sms = 0, pdl = -1, single = 0;
    if (!tensor_device_info(&dev, &num_sms, &pdl, &single)) return SG_ERR_CUDA;

    // 128 columns on a CTA pair when there are more than 64 columns and at least two tiles (each CTA keeps 64 columns of
    // the filter); otherwise one CTA with 64 or 128 columns.  f32: the split filter (hi and lo) of the one column tile
    // must fit beside a ring whose top can stage the raw filter.
    const int BN = p.N > 64 ? 128 : 64;
    const int kbpt = (p.C + bkc - 1) / bkc;
    const int strip_stage_bytes = (int)(((int64_t)p.KH * strip_rows * 128 + 1023) / 1024) * 1024;   // KH strips per stage
    int CG = (BN == 128 && num_tiles > 1 && single == 0) ? 2 : 1;
    if (f32 && (p.N > BN || (BN == 128 && CG == 1))) return SG_ERR_UNSUPPORTED;
    int64_t flt_bytes = 0, fixed = 0, staging_bytes = 0;
    int stages = 0;
    for (;; CG = 1) {
        flt_bytes = (int64_t)p.KH * p.KW * kbpt * (BN / CG) * 128 * (f32 ? 2 : 1);
        // the staged output tile: [image row][32-column chunk][position][32 f32]; f32: the raw filter (half the size of
        // the split one) waits there to be split
        staging_bytes = (int64_t)rows_per_tile * (BN / 32) * chunk_rows * 128;
        if (f32 && staging_bytes < flt_bytes / 2) staging_bytes = flt_bytes / 2;
        staging_bytes = (staging_bytes + 1023) / 1024 * 1024;
        fixed = flt_bytes + staging_bytes + 512;
        stages = (int)((SMEM_LIMIT - fixed) / strip_stage_bytes);
        if (stages > MAX_STAGES) stages = MAX_STAGES;
        if (stages >= 2 || CG == 1 || f32) break;
    }
    if (stages < 2) return SG_ERR_UNSUPPORTED;
    const int smem_bytes = (int)(fixed + (int64_t)stages * strip_stage_bytes + 1024);

    alignas(64) CUtensorMap map_in, map_flt, map_out;
    const CUtensorMapDataType in_type = f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    {
        // overlapping 3-D view: {channel, position, filter row}; a step in the third dimension is
        // dh*W_in positions.  The position extent stops (KH-1)*dh*W_in short of the end so that no
        // coordinate reaches past the tensor: what that cuts off (read as zero) feeds only positions
        // with h >= H_out of the last image, which are not outputs.
        cuuint64_t dims[3] = {(cuuint64_t)p.C, (cuuint64_t)q_extent, (cuuint64_t)p.KH};
        cuuint64_t strides[2] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)((p.KH > 1 ? shift_rows : Q) * p.i_w * es)};
        cuuint32_t box[3] = {(cuuint32_t)bkc, (cuuint32_t)strip_rows, (cuuint32_t)p.KH};
        if (strides[1] >= ((cuuint64_t)1 << 40)) return SG_ERR_UNSUPPORTED;
        if (!tensor_encode_tiled(&map_in, in_type, 3, const_cast<void *>(In), dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return SG_ERR_UNSUPPORTED;
    }
    const int64_t s_kw = p.KW > 1 ? p.k_kw : (int64_t)p.C * p.k_c;
    const int64_t s_kh = p.KH > 1 ? p.k_kh : (int64_t)p.KW * s_kw;
    const int sub = f32 ? 32 : 64;               // filter columns per 128-byte row
    const bool flt_blocked = p.N % sub == 0;     // whole column blocks: one box per filter row and channel block
    if (f32 && !flt_blocked) return SG_ERR_UNSUPPORTED;
    if (flt_blocked) {
        // {column in block, channel, column block, kw, kh}, box {sub, channels per block, B_COLS/sub, KW, KH}; bf16 lands as
        // the tensor core reads it (128-byte swizzle), f32 as stored (the converter warps transpose it)
        cuuint64_t dims[5] = {(cuuint64_t)sub, (cuuint64_t)p.C, (cuuint64_t)(p.N / sub), (cuuint64_t)p.KW, (cuuint64_t)p.KH};
        cuuint64_t strides[4] = {(cuuint64_t)(p.k_c * es), 128, (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
        cuuint32_t box[5] = {(cuuint32_t)sub, (cuuint32_t)bkc, (cuuint32_t)(BN / CG / sub), (cuuint32_t)p.KW, (cuuint32_t)p.KH};
        if (!tensor_encode_tiled(&map_flt, in_type, 5, const_cast<void *>(Flt), dims, strides, box,
                                 f32 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B))
            return SG_ERR_UNSUPPORTED;
    } else {
        cuuint64_t dims[4] = {(cuuint64_t)p.N, (cuuint64_t)p.C, (cuuint64_t)p.KW, (cuuint64_t)p.KH};
        cuuint64_t strides[3] = {(cuuint64_t)(p.k_c * es), (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
        cuuint32_t box[4] = {64, 64, 1, 1};
        if (!tensor_encode_tiled(&map_flt, in_type, 4, const_cast<void *>(Flt), dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return SG_ERR_UNSUPPORTED;
    }
    const bool blocked_store = p.N % 32 == 0;
    {
        // A dimension of extent 1 gets the dense stride (its own is not used and may be 0).
        const int64_t s_w = p.o_w, s_h = p.Ho > 1 ? p.o_h : (int64_t)p.Wo * s_w, s_n = p.batch > 1 ? p.o_n : (int64_t)p.Ho * s_h;
        if (s_w * 4 >= pitch_limit || s_h * 4 >= pitch_limit || s_n * 4 >= pitch_limit || s_h % 4 != 0 || s_n % 4 != 0) return SG_ERR_UNSUPPORTED;
        bool ok;
        if (blocked_store) {
            // {f in chunk, w, chunk, h, n}: one box {32, positions of a row (segment), chunks of the tile, rows of the tile, 1}
            // is the whole tile
            cuuint64_t dims[5] = {32, (cuuint64_t)p.Wo, (cuuint64_t)(p.N / 32), (cuuint64_t)p.Ho, (cuuint64_t)p.batch};
            cuuint64_t strides[4] = {(cuuint64_t)(s_w * 4), 128, (cuuint64_t)(s_h * 4), (cuuint64_t)(s_n * 4)};
            cuuint32_t box[5] = {32, (cuuint32_t)chunk_rows, (cuuint32_t)(BN / 32), (cuuint32_t)rows_per_tile, 1};
            ok = tensor_encode_tiled(&map_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, O, dims, strides, box,
                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
        } else {
            // {f, w, h, n}; one store = 32 columns x the positions of one image row (or one 128-position segment)
            cuuint64_t dims[4] = {(cuuint64_t)p.N, (cuuint64_t)p.Wo, (cuuint64_t)p.Ho, (cuuint64_t)p.batch};
            cuuint64_t strides[3] = {(cuuint64_t)(s_w * 4), (cuuint64_t)(s_h * 4), (cuuint64_t)(s_n * 4)};
            cuuint32_t box[4] = {32, (cuuint32_t)chunk_rows, 1, 1};
            ok = tensor_encode_tiled(&map_out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, O, dims, strides, box,
                                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE);
        }
        if (!ok) return SG_ERR_UNSUPPORTED;
    }

    ConvParams cp{};
    cp.Q = (int)Q;
    cp.num_tiles = (int)num_tiles;
    cp.num_pos_items = (int)((num_tiles + CG - 1) / CG);
    cp.num_f_tiles = (p.N + BN - 1) / BN;
    const int total = cp.num_pos_items * cp.num_f_tiles;
    const int groups_max = num_sms / CG;
    const int groups = total < groups_max ? total : groups_max;
    const int grid = CG * groups;
    cp.N = p.batch; cp.Hin = p.Hin; cp.Win = p.Win; cp.Hout = p.Ho; cp.Wout = p.Wo;
    cp.KH = p.KH; cp.KW = p.KW; cp.kbpt = kbpt;
    cp.dw = p.dw;
    cp.rows_per_tile = rows_per_tile; cp.segs = segs; cp.tiles_per_image = (int)tiles_per_image;
    cp.chunk_rows = chunk_rows; cp.staging_bytes = (int)staging_bytes; cp.blocked_store = blocked_store ? 1 : 0;
    cp.strip_rows = (int)strip_rows; cp.strip_stage_bytes = strip_stage_bytes; cp.stages = stages;
    cp.flt_bytes = (int)flt_bytes;
    cp.flt_blocked = flt_blocked ? 1 : 0;
    cp.F = p.N; cp.accumulate = p.accumulate;
    cp.wait_prior = pdl == 0 ? 0 : 1;

    if (f32) {
        if (BN == 64) return launch_kernel<64, 1, true>(map_in, map_flt, map_out, cp, grid, smem_bytes, 3, stream);
        return launch_kernel<128, 2, true>(map_in, map_flt, map_out, cp, grid, smem_bytes, 4, stream);
    }
    if (BN == 64) return launch_kernel<64, 1, false>(map_in, map_flt, map_out, cp, grid, smem_bytes, 0, stream);
    if (CG == 2) return launch_kernel<128, 2, false>(map_in, map_flt, map_out, cp, grid, smem_bytes, 2, stream);
    return launch_kernel<128, 1, false>(map_in, map_flt, map_out, cp, grid, smem_bytes, 1, stream);
}

sg_status conv_read_status(cudaStream_t stream) { return read_status_word(stream); }

}  // namespace sg

// Stride-1 bf16 convolutions on the tensor cores with every input pixel fetched once per tile
// and the filter resident in shared memory.
//
// The im2col kernel fetches, for each of the KH*KW filter taps, a fresh 128-pixel input tile and
// a fresh filter tile: on conv_2d 3x3 that is nine copies of nearly the same pixels and nine
// filter tiles per output tile, and the TMA issue / L2 -> shared memory fill rate bounds it.
// Here the iteration space is walked in "padded" output coordinates: q = (n*H_in + h)*W_in + w
// counts output positions with the INPUT's row pitch, so the input pixel of tap (kh, kw) is row
// q + kh*dh*W_in + kw*dw of the input seen as a [N*H_in*W_in, C] matrix.  A tile is 128
// consecutive q (256 for a CTA pair).  Per block of 64 channels ONE TMA load brings, for every
// filter row kh, the strip of 128 + (KW-1)*dw rows that the KW taps of that row need (a 3-D
// box over an overlapping view of the input whose third dimension steps by dh*W_in rows), and
// each tap's MMAs read its strip through a matrix descriptor whose start address is shifted by
// kw*dw rows.  The filter (all taps, all channels, the tile's columns) is loaded once per CTA.
// Positions whose (h, w) fall outside the output (the last KH-1 rows and KW-1 columns of every
// image) are computed and dropped in the epilogue: (H_in*W_in)/(H_out*W_out) - 1 of the MMA
// work, 7 % on 58x58 -> 56x56.
//
// Warp roles: warp 0 producer (TMA), warp 1 MMA issuer and TMEM owner, warps 2-9 epilogue
// (TMEM -> registers -> shared-memory transpose -> 128-byte row segments in global memory, rows
// that are not outputs skipped).  Every wait is bounded.
#include <mutex>

#include "sg_internal.cuh"
#include "sg_tc_ptx.cuh"

namespace sg {
namespace {

constexpr int BM = 128;
constexpr int SUB_BYTES = 64 * 128;          // filter sub-tile: 64 k-rows x 64 columns of bf16
constexpr int MAX_KH = 8;
constexpr int MAX_STAGES = 8;
constexpr int EPI_WARPS = 8;                 // two per TMEM lane quarter, each takes half of the tile's columns
constexpr int STAGING_BYTES = EPI_WARPS * 4096;   // one 32 x 32 f32 chunk per epilogue warp
constexpr int CONV_THREADS = 64 + 32 * EPI_WARPS;
constexpr int SMEM_LIMIT = 232448 - 1024;    // opt-in maximum minus the alignment slack

struct ConvParams {
    int Q;                 // N * H_in * W_in padded output positions
    int num_q_tiles, num_f_tiles, items_per_group;
    int KH, KW, kbpt;      // filter rows, taps per row, 64-channel blocks per tap
    int Hin, Win, Hout, Wout;
    int dw;                // input rows between taps of a filter row
    int strip_rows;        // 128 + (KW - 1) * dw
    int strip_stage_bytes; // KH strips of strip_rows x 128 B, rounded up to 1 KiB
    int stages;
    int flt_bytes;         // resident filter: KH * kbpt * KW blocks of B_COLS x 128 B
    int flt_blocked;       // 1: the filter map is blocked by 64 columns (one load per filter row and channel block)
    int F;
    int accumulate;
    long long o_n, o_h, o_w;
    float *O;
};

// CG = 1: one CTA computes 128 positions x BN columns.  CG = 2: a CTA pair (one cluster)
// computes 256 positions x BN columns with tcgen05.mma.cta_group::2: each CTA loads the strips
// of its own 128 positions and keeps its own BN/2 columns of the filter, which halves the
// resident filter and leaves room for a deeper ring of strips.
template <int BN, int CG>
__global__ void __launch_bounds__(CONV_THREADS, 1)
conv_strip_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_flt, const ConvParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t flt_addr = smem_base;
    const uint32_t strips_addr = flt_addr + p.flt_bytes;
    const uint32_t staging_off = p.flt_bytes + p.stages * p.strip_stage_bytes;
    uint8_t *staging_gen = smem_gen + staging_off;
    const uint32_t bars_addr = smem_base + staging_off + STAGING_BYTES;
    uint8_t *bars_gen = staging_gen + STAGING_BYTES;
    // barrier block: full[8] | empty[8] | flt_full[8] | flt_free | acc_full[2] | acc_empty[2] | tmem_ptr | abort
    auto full_bar = [&](int s) { return bars_addr + 8u * s; };
    auto empty_bar = [&](int s) { return bars_addr + 8u * (8 + s); };
    auto flt_full_bar = [&](int kh) { return bars_addr + 8u * (16 + kh); };
    const uint32_t flt_free_bar = bars_addr + 8u * 24;
    auto acc_full_bar = [&](int b) { return bars_addr + 8u * (25 + b); };
    auto acc_empty_bar = [&](int b) { return bars_addr + 8u * (27 + b); };
    volatile uint32_t *tmem_ptr_slot = reinterpret_cast<volatile uint32_t *>(bars_gen + 8 * 29);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_gen + 8 * 29 + 4);
    constexpr uint32_t TMEM_COLS = 2 * BN;
    constexpr int B_COLS = BN / CG;            // filter columns resident in this CTA

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) { prefetch_tensormap(&map_in); prefetch_tensormap(&map_flt); }
    // In a pair, CTA 0 (the leader) issues the MMAs and owns the barriers the loads signal.
    const uint32_t cta_rank = CG == 2 ? cluster_ctarank() : 0u;
    const int group_id = (int)blockIdx.x / CG;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int k = 0; k < MAX_KH; ++k) mbar_init(flt_full_bar(k), 1);
        mbar_init(flt_free_bar, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), EPI_WARPS * CG); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        if constexpr (CG == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(const_cast<uint32_t *>(tmem_ptr_slot))), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32(const_cast<uint32_t *>(tmem_ptr_slot))), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (CG == 2) cluster_sync_all();   // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_slot;

    // this group's items: a contiguous run of (column tile, q tile), q fastest, so that the resident
    // filter changes as rarely as possible
    const int total_items = p.num_q_tiles * p.num_f_tiles;
    const int item0 = group_id * p.items_per_group;
    const int item1 = item0 + p.items_per_group < total_items ? item0 + p.items_per_group : total_items;
    const uint32_t flt_block_bytes = (uint32_t)B_COLS * 128u;   // one (tap, channel block): B_COLS/64 sub-tiles
    const uint32_t strips_tx = (uint32_t)(p.KH * p.strip_rows) * 128u;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            int it = 0, cur_ft = -1, epochs = 0;
            bool ok = true;
            auto load_strips = [&](int q0, int cb) {       // one load: the strips of all filter rows
                const int s = it % p.stages;
                if (!mbar_wait(empty_bar(s), ((it / p.stages) & 1) ^ 1u, abort_flag)) return false;
                // (a pair's loads all signal the leader's barriers, which the leader arms for both CTAs)
                if (cta_rank == 0) mbar_expect_tx(full_bar(s), CG * strips_tx);
                tma_tile_3d<CG == 2>(strips_addr + s * p.strip_stage_bytes, &map_in,
                                     CG == 2 ? map_to_cta(full_bar(s), 0) : full_bar(s), cb * 64, q0, 0);
                return true;
            };
            for (int item = item0; item < item1 && ok; ++item) {
                const int ft = item / p.num_q_tiles, qt = item - ft * p.num_q_tiles;
                const int q0 = (qt * CG + (int)cta_rank) * BM;
                int cb = 0;
                if (ft != cur_ft) {
                    // the MMAs of the previous column tile must have finished reading the filter
                    if (epochs > 0 && !mbar_wait(flt_free_bar, (epochs - 1) & 1, abort_flag)) { ok = false; break; }
                    cur_ft = ft;
                    ++epochs;
                    const int f0 = ft * BN + (int)cta_rank * B_COLS;
                    for (int kh = 0; kh < p.KH && ok; ++kh) {
                        const uint32_t fbar = CG == 2 ? map_to_cta(flt_full_bar(kh), 0) : flt_full_bar(kh);
                        if (cta_rank == 0) mbar_expect_tx(flt_full_bar(kh), CG * p.kbpt * p.KW * flt_block_bytes);
                        for (int c2 = 0; c2 < p.kbpt; ++c2) {
                            const uint32_t dst = flt_addr + ((kh * p.kbpt + c2) * p.KW) * flt_block_bytes;
                            if (p.flt_blocked) {
                                // box {64 columns, 64 channels, B_COLS/64 column blocks, KW taps, 1}
                                tma_tile_5d<CG == 2>(dst, &map_flt, fbar, 0, c2 * 64, f0 / 64, 0, kh);
                            } else {
                                for (int kw = 0; kw < p.KW; ++kw)
#pragma unroll
                                    for (int j = 0; j < B_COLS / 64; ++j) {
                                        if constexpr (CG == 2) tma_load_4d_cg2(dst + kw * flt_block_bytes + j * SUB_BYTES, &map_flt, fbar, f0 + j * 64, c2 * 64, kw, kh);
                                        else tma_load_4d(dst + kw * flt_block_bytes + j * SUB_BYTES, &map_flt, fbar, f0 + j * 64, c2 * 64, kw, kh);
                                    }
                            }
                        }
                        // the first tile's strips go out right behind the first filter row
                        if (kh == 0) { ok = load_strips(q0, 0); ++it; cb = 1; }
                    }
                }
                for (; cb < p.kbpt && ok; ++cb, ++it) ok = load_strips(q0, cb);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA).  The
        // whole warp walks the loop so that addresses stay warp-uniform; one elected lane issues.
        if (cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc(BN, CG * BM, false, false, true);   // filter read as stored: N-major
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
            int it = 0, tl = 0, cur_ft = -1, epochs = 0;
            unsigned flt_ready = 0;      // bit kh: this epoch's filter row kh has landed
            bool ok = true;
            for (int item = item0; item < item1 && ok; ++item, ++tl) {
                const int ft = item / p.num_q_tiles;
                if (ft != cur_ft) { cur_ft = ft; ++epochs; flt_ready = 0; }
                const int buf = tl & 1;
                if (!wait_all(mbar_wait(acc_empty_bar(buf), ((tl >> 1) & 1) ^ 1u, abort_flag))) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                uint32_t acc = 0;
                for (int cb = 0; cb < p.kbpt && ok; ++cb, ++it) {
                    const int s = it % p.stages;
                    if (!wait_all(mbar_wait(full_bar(s), (it / p.stages) & 1, abort_flag))) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t strips = strips_addr + s * p.strip_stage_bytes;
                    for (int kh = 0; kh < p.KH && ok; ++kh) {
                        if (!(flt_ready >> kh & 1u)) {
                            if (!wait_all(mbar_wait(flt_full_bar(kh), (epochs - 1) & 1, abort_flag))) { ok = false; break; }
                            tc_fence_after();
                            flt_ready |= 1u << kh;
                        }
                        for (int kw = 0; kw < p.KW; ++kw) {
                            // the tap's 128 pixels start kw*dw rows into the strip of filter row kh: same
                            // K-major layout, start address shifted by whole rows.  The 128-byte swizzle is
                            // a function of the absolute shared-memory address, for the TMA that wrote the
                            // strips and for the tensor core alike, so the shifted descriptor (base-offset
                            // field clear) reads exactly the rows it names.
                            const uint32_t a_addr = strips + (uint32_t)(kh * p.strip_rows + kw * p.dw) * 128u;
                            const uint64_t a_desc = make_smem_desc(a_addr, 16, 1024);
                            const uint32_t b_addr = flt_addr + ((kh * p.kbpt + cb) * p.KW + kw) * flt_block_bytes;
                            const uint64_t b_desc = make_smem_desc(b_addr, SUB_BYTES, 1024);
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
                if (ok) {
                    commit_all(acc_full_bar(buf));
                    const bool last_of_ft = item + 1 >= item1 || (item + 1) / p.num_q_tiles != ft;
                    if (last_of_ft) commit_all(flt_free_bar);
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int quarter = warp & 3;          // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;      // which half of the tile's columns this warp writes
        constexpr int CHUNKS = BN / 64;        // 32-column chunks per warp
        uint8_t *stg = staging_gen + (warp - 2) * 4096;
        const long long img = (long long)p.Hin * p.Win;
        int tl = 0;
        bool ok = true;
        for (int item = item0; item < item1 && ok; ++item, ++tl) {
            const int ft = item / p.num_q_tiles, qt = item - ft * p.num_q_tiles;
            // this lane's row: padded position q -> (n, h, w) -> its address in O, or null when the
            // position is not an output
            const long long q = ((long long)qt * CG + cta_rank) * BM + quarter * 32 + lane;
            float *row_ptr = nullptr;
            if (q < p.Q) {
                const int n = (int)(q / img);
                const int r = (int)(q - (long long)n * img);
                const int h = r / p.Win, w = r - h * p.Win;
                if (h < p.Hout && w < p.Wout) row_ptr = p.O + n * p.o_n + h * p.o_h + w * p.o_w;
            }
            const int buf = tl & 1;
            if (!mbar_wait(acc_full_bar(buf), (tl >> 1) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
            // all of this warp's columns leave TMEM at once; the accumulator buffer is handed back
            // before the slow part (shared-memory transpose, global stores)
            uint32_t r[CHUNKS][32];
#pragma unroll
            for (int j = 0; j < CHUNKS; ++j)
                tmem_ld_32x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + (half * CHUNKS + j) * 32), r[j]);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (CG == 1) mbar_arrive(acc_empty_bar(buf));
                else mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));
            }
#pragma unroll
            for (int j = 0; j < CHUNKS; ++j) {
                // transpose through shared memory: lane = row writes its 8 chunks rotated by its row
                // index (conflict-free), then 8 lanes read one row's 128 bytes
                uint8_t *mine = stg + lane * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4 *>(mine + (((c + lane) & 7) << 4)) =
                        make_uint4(r[j][4 * c], r[j][4 * c + 1], r[j][4 * c + 2], r[j][4 * c + 3]);
                __syncwarp();
                const int cc = lane & 7;
                const int col = ft * BN + (half * CHUNKS + j) * 32 + cc * 4;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + (lane >> 3);
                    float *dst = reinterpret_cast<float *>(__shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(row_ptr), rr));
                    float4 v = *reinterpret_cast<const float4 *>(stg + rr * 128 + (((cc + rr) & 7) << 4));
                    if (dst != nullptr && col < p.F) {
                        float4 *o = reinterpret_cast<float4 *>(dst + col);
                        if (p.accumulate) {
                            const float4 old = *o;
                            v.x += old.x; v.y += old.y; v.z += old.z; v.w += old.w;
                        }
                        *o = v;
                    }
                }
                __syncwarp();
            }
        }
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
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

std::mutex g_conv_mu;
bool g_attr_set[3] = {false, false, false};
int g_attr_device = -1;
int g_force_single = -1;       // SG_CONV_SINGLE=1 (testing): never use CTA pairs

inline bool mult(int64_t v, int64_t q) { return v % q == 0; }

}  // namespace

sg_status launch_conv_strip(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream) {
    // ---- eligibility: bf16, unit conv strides, dense pixel pitch, TMA alignment rules ----
    if (p.spatial_rank == 0 || !p.in_bf16) return SG_ERR_UNSUPPORTED;
    if (p.sh != 1 || p.sw != 1) return SG_ERR_UNSUPPORTED;
    if (p.i_c != 1 || p.k_f != 1 || p.o_f != 1) return SG_ERR_UNSUPPORTED;
    if (p.KH > MAX_KH || p.KH < 1 || p.KW < 1 || p.KW > 256) return SG_ERR_UNSUPPORTED;
    const int64_t es = 2;
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
    if (!mult(p.o_w, 4) || (p.Ho > 1 && !mult(p.o_h, 4)) || (p.batch > 1 && !mult(p.o_n, 4)) || !mult(p.N, 4)) return SG_ERR_UNSUPPORTED;
    const int64_t pitch_limit = (int64_t)1 << 40;
    if (p.i_w * es >= pitch_limit || p.k_c * es >= pitch_limit) return SG_ERR_UNSUPPORTED;
    const int64_t Q = (int64_t)p.batch * p.Hin * p.Win;
    if (Q > 0x7fffffff - 4096) return SG_ERR_UNSUPPORTED;
    const int64_t strip_rows = BM + (int64_t)(p.KW - 1) * p.dw;
    if (strip_rows > 256) return SG_ERR_UNSUPPORTED;
    const int64_t shift_rows = (int64_t)p.dh * p.Win;              // input rows between filter rows
    const int64_t q_extent = Q - (int64_t)(p.KH - 1) * shift_rows;
    if (q_extent < 1 || shift_rows * p.i_w * es >= pitch_limit) return SG_ERR_UNSUPPORTED;
    // wasted positions: the padded domain against the true one
    if ((double)Q > 1.35 * (double)p.M) return SG_ERR_UNSUPPORTED;

    if (g_force_single < 0) {
        const char *e = getenv("SG_CONV_SINGLE");
        g_force_single = e ? atoi(e) : 0;
    }
    // 128 columns on a CTA pair when there are more than 64 columns and at least two 128-position
    // tiles (each CTA keeps 64 columns of the filter); otherwise one CTA with 64 or 128 columns
    const int BN = p.N > 64 ? 128 : 64;
    const int kbpt = (p.C + 63) / 64;
    const int strip_stage_bytes = (int)(((int64_t)p.KH * strip_rows * 128 + 1023) / 1024) * 1024;   // KH strips per stage
    int CG = (BN == 128 && Q > BM && g_force_single == 0) ? 2 : 1;
    int64_t flt_bytes = 0, fixed = 0;
    int stages = 0;
    for (;; CG = 1) {
        flt_bytes = (int64_t)p.KH * p.KW * kbpt * (BN / CG) * 128;
        fixed = flt_bytes + STAGING_BYTES + 256;
        stages = (int)((SMEM_LIMIT - fixed) / strip_stage_bytes);
        if (stages > MAX_STAGES) stages = MAX_STAGES;
        if (stages >= 2 || CG == 1) break;
    }
    if (stages < 2) return SG_ERR_UNSUPPORTED;
    const int smem_bytes = (int)(fixed + (int64_t)stages * strip_stage_bytes + 1024);

    std::lock_guard<std::mutex> lock(g_conv_mu);
    int num_sms = 0;
    if (!tensor_driver_ready(&num_sms)) return SG_ERR_CUDA;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev != g_attr_device) { g_attr_set[0] = g_attr_set[1] = g_attr_set[2] = false; g_attr_device = dev; }

    alignas(64) CUtensorMap map_in, map_flt;
    {
        // overlapping 3-D view: {channel, position, filter row}; a step in the third dimension is
        // dh*W_in positions.  The position extent stops (KH-1)*dh*W_in short of the end so that no
        // coordinate reaches past the tensor: what that cuts off (read as zero) feeds only positions
        // with h >= H_out of the last image, which are not outputs.
        cuuint64_t dims[3] = {(cuuint64_t)p.C, (cuuint64_t)q_extent, (cuuint64_t)p.KH};
        cuuint64_t strides[2] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)((p.KH > 1 ? shift_rows : Q) * p.i_w * es)};
        cuuint32_t box[3] = {64, (cuuint32_t)strip_rows, (cuuint32_t)p.KH};
        if (strides[1] >= ((cuuint64_t)1 << 40)) return SG_ERR_UNSUPPORTED;
        if (!tensor_encode_tiled(&map_in, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(In), dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return SG_ERR_UNSUPPORTED;
    }
    const int64_t s_kw = p.KW > 1 ? p.k_kw : (int64_t)p.C * p.k_c;
    const int64_t s_kh = p.KH > 1 ? p.k_kh : (int64_t)p.KW * s_kw;
    const bool flt_blocked = p.N % 64 == 0;     // whole 64-column blocks: one box per filter row and channel block
    if (flt_blocked) {
        // {column in block, channel, column block, kw, kh}, box {64, 64, B_COLS/64, KW, 1}
        cuuint64_t dims[5] = {64, (cuuint64_t)p.C, (cuuint64_t)(p.N / 64), (cuuint64_t)p.KW, (cuuint64_t)p.KH};
        cuuint64_t strides[4] = {(cuuint64_t)(p.k_c * es), 128, (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
        cuuint32_t box[5] = {64, 64, (cuuint32_t)(BN / CG / 64), (cuuint32_t)p.KW, 1};
        if (!tensor_encode_tiled(&map_flt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(Flt), dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return SG_ERR_UNSUPPORTED;
    } else {
        cuuint64_t dims[4] = {(cuuint64_t)p.N, (cuuint64_t)p.C, (cuuint64_t)p.KW, (cuuint64_t)p.KH};
        cuuint64_t strides[3] = {(cuuint64_t)(p.k_c * es), (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
        cuuint32_t box[4] = {64, 64, 1, 1};
        if (!tensor_encode_tiled(&map_flt, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(Flt), dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B)) return SG_ERR_UNSUPPORTED;
    }

    ConvParams cp{};
    cp.Q = (int)Q;
    cp.num_q_tiles = (int)((Q + CG * BM - 1) / (CG * BM));
    cp.num_f_tiles = (p.N + BN - 1) / BN;
    const int total = cp.num_q_tiles * cp.num_f_tiles;
    const int groups_max = num_sms / CG;
    const int groups = total < groups_max ? total : groups_max;
    cp.items_per_group = (total + groups - 1) / groups;
    const int grid = CG * ((total + cp.items_per_group - 1) / cp.items_per_group);
    cp.KH = p.KH; cp.KW = p.KW; cp.kbpt = kbpt;
    cp.Hin = p.Hin; cp.Win = p.Win; cp.Hout = p.Ho; cp.Wout = p.Wo;
    cp.dw = p.dw;
    cp.strip_rows = (int)strip_rows; cp.strip_stage_bytes = strip_stage_bytes; cp.stages = stages;
    cp.flt_bytes = (int)flt_bytes;
    cp.flt_blocked = flt_blocked ? 1 : 0;
    cp.F = p.N; cp.accumulate = p.accumulate;
    cp.o_n = p.o_n; cp.o_h = p.o_h; cp.o_w = p.o_w; cp.O = O;

    void (*kernel)(const CUtensorMap, const CUtensorMap, const ConvParams) =
        BN == 64 ? conv_strip_kernel<64, 1> : (CG == 2 ? conv_strip_kernel<128, 2> : conv_strip_kernel<128, 1>);
    const int slot = BN == 64 ? 0 : (CG == 2 ? 2 : 1);
    if (!g_attr_set[slot]) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT + 1024) != cudaSuccess)
            return SG_ERR_CUDA;
        g_attr_set[slot] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(CONV_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, map_in, map_flt, cp);
    count_launch();
    note_kernel("conv_strip_kernel");
    return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
}

sg_status conv_read_status(cudaStream_t stream) { return read_status_word(stream); }

}  // namespace sg

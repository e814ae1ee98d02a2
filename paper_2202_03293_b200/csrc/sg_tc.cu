// Tensor-core path for sm_100a: TMA -> swizzled shared memory -> tcgen05.mma -> TMEM -> TMA store.
//
// One persistent CTA per SM (or CTA pair per two SMs) walks a static list of work items: whole
// output tiles, equal k ranges of a tile (split reduction), or its run of the stream-K tail that
// replaces a partly filled last wave of tiles.  Inside a CTA the work is split by warp role:
//
//   warp 0  producer : per k-block waits for a free stage, then issues the TMA loads of the
//                      input tile (tiled mode for matmul, im2col mode for the convolutions:
//                      the TMA unit itself gathers the sliding window, Section 3.2's
//                      "padding/packing" done in hardware) and of the filter tile.
//   warp 1  MMA      : one thread waits for a full stage and issues tcgen05.mma into one of
//                      two TMEM accumulator buffers; tcgen05.commit releases the stage and,
//                      after the last k-block, publishes the accumulator.
//   warps 2-5 epilogue: each owns one 32-lane quarter of TMEM; tcgen05.ld -> registers ->
//                      swizzled staging buffer -> TMA store (or TMA reduce-add when the op
//                      accumulates into its output), overlapping the next tile's main loop.
//
// Shared-memory operand layouts (both 128-byte swizzled, written by TMA, read by the MMA
// unit through matrix descriptors):
//   input tile   K-major : 128 rows (output pixels) x 64 bf16 (128 B per row)
//   filter tile  N-major : BN/64 sub-tiles, each 64 k-rows x 64 bf16 (128 B per row); the
//                          filter is stored [k][f] with f contiguous, so it is consumed as
//                          an MN-major operand instead of being transposed.
//
// f32 inputs run on the same pipeline with every element split as x = hi + lo, hi = x rounded to tf32: the TMA
// writes the raw f32 tiles into its ring, sixteen converter warps split them and write a second ring of two slots
// (transposing the filter tile to K-major on the way, which kind::tf32 needs; the split input tile goes to tensor
// memory), and the MMA thread accumulates lo*hi + hi*lo + hi*hi in f32: the dropped term is below 2^-21 |a*b|, so
// f32 accuracy is kept.  In the plain layout hi*hi runs in tf32 and the two corrections as one bf16 contraction over
// [lo | hi] . [hi | lo] (8 MMAs per k-block); the transposed layouts run three tf32 products (12).  Raw tiles are
// 128 rows x 32 f32 (input) and 32 k-rows x 32 f32 sub-tiles (filter), again 128 bytes per row.
//
// Every wait in this file is bounded: a wait that expires sets an abort flag in shared
// memory and a bit in the device status word, every role then leaves its loop, the CTA
// drains its copies, frees its TMEM and returns.
#include <cuda.h>

#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "sg_internal.cuh"
#include "sg_tc_ptx.cuh"

namespace sg {
namespace {

constexpr int BM = 128;           // rows of an output tile = lanes of TMEM = M of one MMA
constexpr int ROW_BYTES = 128;    // one k-block = one 128-byte swizzle row: 64 bf16 or 32 f32
constexpr int K_STEPS = 4;        // tcgen05.mma per k-block and product: 32 bytes of k each
constexpr int A_STAGE_BYTES = BM * ROW_BYTES;
constexpr int CONVERTER_THREADS = 512;        // f32 path: 16 warps splitting tiles into hi and lo (one k-block is a serial
                                              // chain of ~200 instructions per warp with 8 warps: longer than its MMAs take)
constexpr int STAGING_BYTES = 2 * 16384;      // epilogue: 2 staging tiles of 128 rows x 128 B


struct TcParams {
    int M, N;
    int num_m_tiles, num_n_tiles;
    int num_kb;          // k-blocks per tile = taps * kb_per_tap
    int splits;          // work items per tile: the k-blocks are dealt out in `splits` contiguous ranges
    int kb_per_split;    // ceil(num_kb / splits); partial sums meet in the output by reduce-add
    int kb_per_tap;      // ceil(C / 64)
    int KW;              // taps are ordered (kh, kw)
    int a_mode;          // 0: tiled 2-D (matmul), 1: im2col 3-D (conv1d), 2: im2col 4-D (conv2d)
    int Ho, Wo, sh, sw, dh, dw;
    int accumulate;
    int b_blocked;       // 1: the filter map is blocked by sub-tile columns: one TMA load fetches the whole filter tile
    int sk_first_tile;   // stream-K tail: tiles from this one on are not dealt out whole; their k-blocks, taken as one
    int sk_units;        //   sequence, are cut into equal runs of `sk_units` k-blocks, one run per CTA (or pair); 0 = no tail
    const float *bias;   // fused pointwise consumer of the write-back: O = act(acc + bias[column]); null = no bias
    int act;             // SG_ACT_NONE or SG_ACT_RELU (only with one work item per tile and in overwrite mode)
    int wait_prior;      // the launch may start before the kernel ahead of it in the stream has finished (programmatic
                         // dependent launch).  1: that kernel is this library's clearing kernel, which touches only the
                         // output: the stores wait for it (griddepcontrol.wait), the loads need not.  2: it is any
                         // kernel: loads and stores both wait.  0: an ordinary launch.
};

template <int BN, int CG, bool F32, int KPS = 1, bool TA = false>
struct Cfg {
    // CG = 1: one CTA owns a 128 x BN tile.  CG = 2: a pair of CTAs (one cluster) owns a
    // 256 x BN tile; each CTA stages its own 128 input rows and its own BN/2 filter columns,
    // and one tcgen05.mma.cta_group::2 per k-step feeds both SMs' tensor cores, so every
    // filter element is staged once per pair instead of once per CTA.
    static constexpr int ELT = F32 ? 4 : 2;                   // bytes per input element
    static constexpr int BK = ROW_BYTES / ELT;                // elements per k-block
    static constexpr int SUB_COLS = ROW_BYTES / ELT;          // filter columns per sub-tile (one 128-byte row)
    static constexpr int SUB_BYTES = BK * ROW_BYTES;          // one filter sub-tile: BK k-rows
    static constexpr int B_COLS = BN / CG;                    // filter columns staged by this CTA
    static constexpr int B_STAGE_BYTES = B_COLS * ROW_BYTES;  // = BK * B_COLS * ELT
    // KPS k-blocks travel together in one stage: [input tile of each k-block | filter tile: sub-tiles of
    // KPS*BK k-rows], fetched by ONE load per operand (a TMA instruction costs the same whatever its size)
    static constexpr int STAGE_BYTES = KPS * (A_STAGE_BYTES + B_STAGE_BYTES);   // written by TMA per stage
    // bf16: one ring of stages, TMA -> MMA.  f32: the TMA ring holds raw tiles; a second ring of
    // two slots holds what the converter warps make of them, [input hi | input lo | filter hi |
    // filter lo], the filter transposed to K-major on the way (kind::tf32 takes no N-major operand).
    // (two slots are enough: with three the kernel is no faster - a k-block is bound by shared-memory bandwidth: the raw tiles
    // written by TMA and read by the converters, the split filter written, and the MMAs' filter reads)
    static constexpr int SPLIT_SLOTS = F32 ? 2 : 0;
    // TA (f32): the split input tile lives in tensor memory (the MMA reads its A operand there), which
    // takes its writes and its three reads per k-step off the shared-memory pipe; a slot then holds
    // [filter hi | filter lo] only.
    static constexpr int SPLIT_BYTES = TA ? 2 * B_STAGE_BYTES : 2 * STAGE_BYTES;
    static constexpr int RING_BUDGET = 196608 - SPLIT_SLOTS * SPLIT_BYTES;
    static constexpr int STAGES = (RING_BUDGET / STAGE_BYTES) > 8 ? 8 : (RING_BUDGET / STAGE_BYTES);
    // warps: input producer, MMA, 4 epilogue (, 8 converter), filter producer
    static constexpr int THREADS = 192 + (F32 ? CONVERTER_THREADS : 0) + 32;
    static constexpr int FLT_WARP = THREADS / 32 - 1;
    // two accumulator buffers (one when the split input's 2 slots x 64 columns would not fit beside two)
    static constexpr int A_TMEM_COLS = TA ? SPLIT_SLOTS * 64 : 0;
    static constexpr int ACC_BUFS = 2 * BN + A_TMEM_COLS > 512 ? 1 : 2;
    static constexpr int USED_COLS = ACC_BUFS * BN + A_TMEM_COLS;
    static constexpr int TMEM_COLS = USED_COLS <= 32 ? 32 : USED_COLS <= 64 ? 64 : USED_COLS <= 128 ? 128 : USED_COLS <= 256 ? 256 : 512;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + SPLIT_SLOTS * SPLIT_BYTES + STAGING_BYTES +
                                      1024 /*alignment slack*/ + 256 /*barriers*/;
    static constexpr int B_KSTEP_DESC = 16 * ROW_BYTES / 16;   // bf16 filter tile, N-major: 16 k-rows per k-step
    static_assert(B_COLS % 64 == 0 && BN % 16 == 0 && BN <= 256, "tile width");
    static_assert(TMEM_COLS <= 512 && (TMEM_COLS & (TMEM_COLS - 1)) == 0, "TMEM columns");
    static_assert(STAGES >= 2 && STAGES <= 8, "ring depth");
    static_assert(KPS == 1 || (KPS == 2 && !F32), "k-blocks per stage");
    static_assert(!TA || F32, "tensor-memory input operand: f32 path only");
};

// Static tile order: groups of 8 tile-rows, row index fastest inside a group, so that the
// CTAs running at the same time share filter columns and a bounded set of input rows in L2.
__device__ __forceinline__ void tile_coords(int t, int num_m_tiles, int num_n_tiles, int &mt, int &nt) {
    constexpr int GM = 8;
    int per_group = GM * num_n_tiles;
    int g = t / per_group, r = t - g * per_group;
    int rows = num_m_tiles - g * GM;
    if (rows > GM) rows = GM;
    nt = r / rows;
    mt = g * GM + (r - nt * rows);
}

// LAY (bf16 matmuls, one k-block per stage): bit 0 = the input operand is stored transposed
// ([k][m], m contiguous: A^T B of Section 4.6.1) and consumed as an M-major operand; bit 1 = the
// filter operand is stored transposed ([n][k], k contiguous: A B^T) and consumed K-major.
// Clears the output tiles first_tile .. (one block per tile) ahead of a launch whose stream-K tail adds into them.
__global__ void __launch_bounds__(256) zero_tiles_kernel(float *__restrict__ O, int64_t pitch, int M, int N, int tile_rows, int tile_cols,
                                                         int num_m_tiles, int num_n_tiles, int first_tile) {
    asm volatile("griddepcontrol.launch_dependents;");     // the launch behind waits for this grid before its first store
    int mt, nt;
    tile_coords(first_tile + (int)blockIdx.x, num_m_tiles, num_n_tiles, mt, nt);
    const int m0 = mt * tile_rows, n0 = nt * tile_cols;
    const int rows = min(tile_rows, M - m0), c4 = min(tile_cols, N - n0) / 4;      // N is a multiple of 4 on this path
    for (int i = threadIdx.x; i < rows * c4; i += 256) {
        const int r = i / c4, c = i - r * c4;
        reinterpret_cast<float4 *>(O + (int64_t)(m0 + r) * pitch + n0)[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}

template <int BN, int CG, bool F32, int KPS, int LAY>
__global__ void __launch_bounds__(Cfg<BN, CG, F32, KPS, (LAY & 4) != 0>::THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_flt,
               const __grid_constant__ CUtensorMap map_out, const TcParams p) {
    constexpr bool A_MN = (LAY & 1) != 0, B_KM = (LAY & 2) != 0, TA = (LAY & 4) != 0;
    // MIX (f32, plain layout, split input in tensor memory): the correction products lo*hi + hi*lo run as bf16 MMAs
    constexpr bool MIX = (LAY & 8) != 0;
    using C = Cfg<BN, CG, F32, KPS, TA>;
    static_assert(!TA || F32, "tensor-memory input operand: f32 path only");
    static_assert(!MIX || LAY == 12, "bf16 corrections: plain layout with the split input in tensor memory");
    static_assert(LAY == 0 || KPS == 1, "transposed layouts: one k-block per stage");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t stages_addr = smem_base;
    const uint32_t split_addr = smem_base + C::STAGES * C::STAGE_BYTES;      // f32 only: hi/lo slots
    const uint32_t staging_addr = split_addr + C::SPLIT_SLOTS * C::SPLIT_BYTES;
    uint8_t *staging_gen = smem_gen + C::STAGES * C::STAGE_BYTES + C::SPLIT_SLOTS * C::SPLIT_BYTES;
    const uint32_t bars_addr = staging_addr + STAGING_BYTES;
    uint8_t *bars_gen = staging_gen + STAGING_BYTES;
    // barrier block: full[8] | empty[8] | split_full[4] | split_empty[4] | acc_full[2] | acc_empty[2] | tmem_ptr | abort
    auto full_bar = [&](int s) { return bars_addr + 8u * s; };
    auto empty_bar = [&](int s) { return bars_addr + 8u * (8 + s); };
    auto split_full_bar = [&](int s) { return bars_addr + 8u * (16 + s); };
    auto split_empty_bar = [&](int s) { return bars_addr + 8u * (20 + s); };
    auto acc_full_bar = [&](int b) { return bars_addr + 8u * (24 + b); };
    auto acc_empty_bar = [&](int b) { return bars_addr + 8u * (26 + b); };
    volatile uint32_t *tmem_ptr_slot = reinterpret_cast<volatile uint32_t *>(bars_gen + 8 * 28);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_gen + 8 * 28 + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // A launch behind this one that asked for it may start now: its CTAs take an SM as soon as one of ours leaves it
    // and set themselves up while the rest of this grid drains; they touch global memory only after this grid is done.
    asm volatile("griddepcontrol.launch_dependents;");
    if (threadIdx.x == 0) { prefetch_tensormap(&map_in); prefetch_tensormap(&map_flt); prefetch_tensormap(&map_out); }
    // In a pair, CTA 0 (the leader) issues the MMAs; both CTAs produce and both run epilogues.
    const uint32_t cta_rank = CG == 2 ? cluster_ctarank() : 0u;
    const int group_id = CG == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int num_groups = CG == 2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        // full: one arrive.expect_tx by each of the two producers.  empty: one tcgen05.commit (bf16) or one arrive per
        // converter warp of this CTA (f32).  split_full: one arrive per converter warp of every CTA
        // of the group.  split_empty / acc_full: one tcgen05.commit.  acc_empty: one arrive per
        // epilogue warp of every CTA of the group.
        for (int s = 0; s < C::STAGES; ++s) {
            mbar_init(full_bar(s), 2);
            mbar_init(empty_bar(s), F32 ? CONVERTER_THREADS / 32 : 1);
        }
        for (int s = 0; s < C::SPLIT_SLOTS; ++s) {
            mbar_init(split_full_bar(s), (CONVERTER_THREADS / 32) * CG);
            mbar_init(split_empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full_bar(b), 1); mbar_init(acc_empty_bar(b), 4 * CG); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {   // TMEM allocation is a warp-wide operation (the same warp in both CTAs of a pair)
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

    // work items: (tile of (CG*128) x BN, k range); the splits of one tile are neighbours in the
    // order, so they run at the same time and their operands meet in L2.  Every role walks the same
    // sequence: first the items dealt round-robin (whole tiles, or `splits` equal k ranges per tile), then
    // this group's run of the stream-K tail: the tiles that would make a last, partly filled wave are
    // not dealt out whole; their k-blocks, taken as one sequence, are cut into equal runs, one per group,
    // and each run is one to three (tile, k range) items whose partial sums meet in the output by reduce-add.
    const int total_tiles = p.num_m_tiles * p.num_n_tiles;
    const int dealt_items = (p.sk_units > 0 ? p.sk_first_tile : total_tiles) * p.splits;
    const int sk_total = p.sk_units > 0 ? (total_tiles - p.sk_first_tile) * p.num_kb : 0;
    const int sk_u0 = min(sk_total, group_id * p.sk_units), sk_u1 = min(sk_total, sk_u0 + p.sk_units);
    struct Cursor { int i, u; };
    auto next_item = [&](Cursor &c, int &tile, int &kb0, int &kb1, int &add) -> bool {
        const int t = group_id + c.i * num_groups;
        if (t < dealt_items) {
            tile = t / p.splits;
            kb0 = (t - tile * p.splits) * p.kb_per_split;
            kb1 = kb0 + p.kb_per_split < p.num_kb ? kb0 + p.kb_per_split : p.num_kb;
            add = p.accumulate;
            ++c.i;
            return true;
        }
        if (c.u >= sk_u1) return false;
        const int first = c.u / p.num_kb;
        tile = p.sk_first_tile + first;
        kb0 = c.u - first * p.num_kb;
        kb1 = min(p.num_kb, kb0 + (sk_u1 - c.u));
        c.u += kb1 - kb0;
        add = 1;
        return true;
    };
    // bf16 pairs count both CTAs' TMA bytes on the leader's barrier, which its MMA thread waits
    // on.  f32 pairs signal each CTA's own barrier (its converter warps wait there) and the
    // leader's MMA thread waits on the split barrier instead.
    constexpr bool REMOTE_FULL = (CG == 2) && !F32;

    if (warp == 0 || warp == C::FLT_WARP) {
        // ------------------------------------------------------------ producers: warp 0 fetches the
        // input tiles, the last warp the filter tiles; both arm the stage's barrier for their bytes
        if (lane == 0) {
            const bool input_side = warp == 0;
            // the operands may be the output of the kernel ahead of this one
            if (p.wait_prior == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
            int it = 0;   // k-block counter across all of this CTA's tiles
            bool ok = true;
            Cursor cur{0, sk_u0};
            int tile, kb0, kb1, add;
            while (ok && next_item(cur, tile, kb0, kb1, add)) {
                int mt, nt;
                tile_coords(tile, p.num_m_tiles, p.num_n_tiles, mt, nt);
                const int m0 = (mt * CG + (int)cta_rank) * BM;
                const int n0 = nt * BN + (int)cta_rank * C::B_COLS;
                int pix_n = 0, pix_h = 0, pix_w = 0;   // first output pixel of this CTA's rows
                if (p.a_mode != 0) {
                    int hw = p.Ho * p.Wo;
                    pix_n = m0 / hw;
                    int r = m0 - pix_n * hw;
                    pix_h = r / p.Wo;
                    pix_w = r - pix_h * p.Wo;
                }
                for (int kb = kb0; kb < kb1; kb += KPS, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t a_dst = stages_addr + s * C::STAGE_BYTES;
                    const uint32_t b_dst = a_dst + KPS * A_STAGE_BYTES;
                    const int tap = kb / p.kb_per_tap;
                    const int c0 = (kb - tap * p.kb_per_tap) * C::BK;
                    const int kh = tap / p.KW, kw = tap - kh * p.KW;
                    // bf16 pairs: the leader alone arms its barrier, for the pair's total (a remote arrive by
                    // the peer would order it after its own loads in flight and serialise the ring)
                    const uint32_t bar = REMOTE_FULL ? map_to_cta(full_bar(s), 0) : full_bar(s);
                    const uint32_t my_bytes = KPS * (input_side ? A_STAGE_BYTES : C::B_STAGE_BYTES);
                    if (!REMOTE_FULL || cta_rank == 0) mbar_expect_tx(full_bar(s), (REMOTE_FULL ? CG : 1) * my_bytes);
                    if (input_side) {
                        if constexpr (A_MN) {
                            // transposed input: map blocked by sub-tile rows of m (one 128-byte row: 64 bf16 or
                            // 32 f32), box {rows in block, BK k-rows, 128 / rows-in-block blocks}
                            tma_tile_3d<REMOTE_FULL>(a_dst, &map_in, bar, 0, c0, m0 / C::SUB_COLS);
                        } else if constexpr (KPS > 1) {
                            // matmul only: the input map is blocked by k-blocks, box {BK, 128 rows, KPS k-blocks}
                            tma_tile_3d<REMOTE_FULL>(a_dst, &map_in, bar, 0, m0, kb);
                        } else if constexpr (!REMOTE_FULL) {
                            if (p.a_mode == 0) {
                                tma_load_2d(a_dst, &map_in, bar, c0, m0);
                            } else if (p.a_mode == 1) {
                                tma_load_im2col_3d(a_dst, &map_in, bar, c0, pix_w * p.sw, pix_n, (unsigned short)(kw * p.dw));
                            } else {
                                tma_load_im2col_4d(a_dst, &map_in, bar, c0, pix_w * p.sw, pix_h * p.sh, pix_n,
                                                   (unsigned short)(kw * p.dw), (unsigned short)(kh * p.dh));
                            }
                        } else {
                            if (p.a_mode == 0) {
                                tma_load_2d_cg2(a_dst, &map_in, bar, c0, m0);
                            } else if (p.a_mode == 1) {
                                tma_load_im2col_3d_cg2(a_dst, &map_in, bar, c0, pix_w * p.sw, pix_n, (unsigned short)(kw * p.dw));
                            } else {
                                tma_load_im2col_4d_cg2(a_dst, &map_in, bar, c0, pix_w * p.sw, pix_h * p.sh, pix_n,
                                                       (unsigned short)(kw * p.dw), (unsigned short)(kh * p.dh));
                            }
                        }
                    } else if constexpr (B_KM) {
                        // transposed filter: rows are columns n, k contiguous; box {BK, B_COLS rows}
                        if constexpr (REMOTE_FULL) tma_load_2d_cg2(b_dst, &map_flt, bar, c0, n0);
                        else tma_load_2d(b_dst, &map_flt, bar, c0, n0);
                    } else if (p.b_blocked) {
                        // box {sub-tile columns, KPS*BK channels, B_COLS / SUB_COLS column blocks, 1, 1}
                        tma_tile_5d<REMOTE_FULL>(b_dst, &map_flt, bar, 0, c0, n0 / C::SUB_COLS, kw, kh);
                    } else {
#pragma unroll
                        for (int j = 0; j < C::B_COLS / C::SUB_COLS; ++j) {
                            if constexpr (REMOTE_FULL) tma_load_4d_cg2(b_dst + j * C::SUB_BYTES, &map_flt, bar, n0 + j * C::SUB_COLS, c0, kw, kh);
                            else tma_load_4d(b_dst + j * C::SUB_BYTES, &map_flt, bar, n0 + j * C::SUB_COLS, c0, kw, kh);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop, so that addresses and descriptors are warp-uniform values;
        // one elected lane issues the MMAs and the commits (a loop run by a single lane of a
        // diverged warp pays for moving every descriptor out of per-lane registers: measured
        // ~120 cycles per MMA, as much as a 128 x 256 x 16 MMA takes to execute).
        if (cta_rank == 0) {
            constexpr uint32_t idesc = make_idesc(BN, CG * BM, F32, A_MN && !F32, !F32 && !B_KM);   // f32: the converter warps hand over K-major tiles
            const bool issuer = elect_one();
            auto wait_all = [&](bool passed) { return __all_sync(0xffffffffu, passed) != 0; };
            auto mma = [&](uint32_t d, uint64_t ad, uint64_t bd, uint32_t acc) {
                if (!issuer) return;
                if constexpr (F32) {
                    if constexpr (CG == 1) umma_tf32(d, ad, bd, idesc, acc); else umma_tf32_cg2(d, ad, bd, idesc, acc);
                } else {
                    if constexpr (CG == 1) umma_bf16(d, ad, bd, idesc, acc); else umma_bf16_cg2(d, ad, bd, idesc, acc);
                }
            };
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
            int it = 0, tl = 0;
            bool ok = true;
            Cursor cur{0, sk_u0};
            int tile, kb0, kb1, add;
            for (; ok && next_item(cur, tile, kb0, kb1, add); ++tl) {
                const int buf = tl % C::ACC_BUFS;
                if (!wait_all(mbar_wait(acc_empty_bar(buf), ((tl / C::ACC_BUFS) & 1) ^ 1u, abort_flag))) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = kb0; kb < kb1; kb += KPS, ++it) {
                    if constexpr (F32) {
                        const int s = it % C::SPLIT_SLOTS;
                        if (!wait_all(mbar_wait<CG == 2>(split_full_bar(s), (it / C::SPLIT_SLOTS) & 1, abort_flag))) { ok = false; break; }
                        tc_fence_after();
                        if constexpr (MIX) {
                            // slot: [filter hi, tf32, K-major | filter as bf16, K-major rows of 64 k: hi then lo].  Tensor
                            // memory: input hi (32 columns of tf32) | input as bf16: lo (16 columns), hi (16 columns).
                            // The corrections [lo | hi] . [hi | lo] are four bf16 k-steps of 16, the main term four tf32
                            // k-steps of 8: 8 MMAs per k-block instead of 12.
                            constexpr uint32_t idesc16 = make_idesc(BN, CG * BM, false, false, false);
                            const uint32_t slot = split_addr + s * C::SPLIT_BYTES;
                            const uint64_t bh = make_smem_desc(slot, 16, 1024);
                            const uint64_t b16 = make_smem_desc(slot + C::B_STAGE_BYTES, 16, 1024);
                            const uint32_t a_hi = tmem_base + (uint32_t)(C::ACC_BUFS * BN + s * 64), a16 = a_hi + 32;
                            if (issuer) {
#pragma unroll
                                for (int k = 0; k < K_STEPS; ++k) {      // small terms first
                                    const uint32_t acc = (kb > kb0 || k > 0) ? 1u : 0u;
                                    if constexpr (CG == 1) umma_bf16_ts(d_tmem, a16 + k * 8, b16 + (uint64_t)(k * 2), idesc16, acc);
                                    else umma_bf16_ts_cg2(d_tmem, a16 + k * 8, b16 + (uint64_t)(k * 2), idesc16, acc);
                                }
#pragma unroll
                                for (int k = 0; k < K_STEPS; ++k) {
                                    if constexpr (CG == 1) umma_tf32_ts(d_tmem, a_hi + k * 8, bh + (uint64_t)(k * 2), idesc, 1u);
                                    else umma_tf32_ts_cg2(d_tmem, a_hi + k * 8, bh + (uint64_t)(k * 2), idesc, 1u);
                                }
                            }
                        } else if constexpr (TA) {
                            // filter hi | lo in the slot (K-major); input hi | lo in tensor memory, 32 columns
                            // (k) each, lane = row: the MMA takes its A operand from there
                            const uint32_t slot = split_addr + s * C::SPLIT_BYTES;
                            const uint64_t bh = make_smem_desc(slot, 16, 1024);
                            const uint64_t bl = make_smem_desc(slot + C::B_STAGE_BYTES, 16, 1024);
                            const uint32_t a_hi = tmem_base + (uint32_t)(C::ACC_BUFS * BN + s * 64), a_lo = a_hi + 32;
#pragma unroll
                            for (int k = 0; k < K_STEPS; ++k) {
                                const uint64_t o = (uint64_t)(k * 2);
                                const uint32_t acc = (kb > kb0 || k > 0) ? 1u : 0u;
                                if (issuer) {
                                    if constexpr (CG == 1) {
                                        umma_tf32_ts(d_tmem, a_lo + k * 8, bh + o, idesc, acc);   // small terms first
                                        umma_tf32_ts(d_tmem, a_hi + k * 8, bl + o, idesc, 1u);
                                        umma_tf32_ts(d_tmem, a_hi + k * 8, bh + o, idesc, 1u);
                                    } else {
                                        umma_tf32_ts_cg2(d_tmem, a_lo + k * 8, bh + o, idesc, acc);
                                        umma_tf32_ts_cg2(d_tmem, a_hi + k * 8, bl + o, idesc, 1u);
                                        umma_tf32_ts_cg2(d_tmem, a_hi + k * 8, bh + o, idesc, 1u);
                                    }
                                }
                            }
                        } else {
                        // slot: [input hi | input lo | filter hi | filter lo], all K-major: 8-row groups
                        // 1024 B apart, a k-step of 8 f32 is 32 B inside the swizzled 128-byte row
                        const uint32_t a_hi = split_addr + s * C::SPLIT_BYTES;
                        const uint64_t ah = make_smem_desc(a_hi, 16, 1024);
                        const uint64_t al = make_smem_desc(a_hi + A_STAGE_BYTES, 16, 1024);
                        const uint64_t bh = make_smem_desc(a_hi + 2 * A_STAGE_BYTES, 16, 1024);
                        const uint64_t bl = make_smem_desc(a_hi + 2 * A_STAGE_BYTES + C::B_STAGE_BYTES, 16, 1024);
#pragma unroll
                        for (int k = 0; k < K_STEPS; ++k) {
                            const uint64_t o = (uint64_t)(k * 2);
                            mma(d_tmem, al + o, bh + o, (kb > kb0 || k > 0) ? 1u : 0u);   // small terms first
                            mma(d_tmem, ah + o, bl + o, 1u);
                            mma(d_tmem, ah + o, bh + o, 1u);
                        }
                        }
                        commit_all(split_empty_bar(s));
                    } else {
                        const int s = it % C::STAGES;
                        const uint32_t ph = (it / C::STAGES) & 1;
                        if (!wait_all(mbar_wait(full_bar(s), ph, abort_flag))) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_addr = stages_addr + s * C::STAGE_BYTES;
                        const uint32_t b_addr = a_addr + KPS * A_STAGE_BYTES;
#pragma unroll
                        for (int kbi = 0; kbi < KPS; ++kbi) {
                            if (kb + kbi >= kb1) break;      // an odd k range ends inside its last stage
                            // input tile, K-major: 8-row groups are 1024 B apart; a k-step of 16 bf16 is 32 B
                            // inside the swizzled 128-byte row.  Stored transposed it is M-major like the
                            // filter below: two 64-row sub-tiles, a k-step 16 rows of 128 B.
                            const uint64_t a_desc = A_MN ? make_smem_desc(a_addr, C::SUB_BYTES, 1024)
                                                         : make_smem_desc(a_addr + kbi * A_STAGE_BYTES, 16, 1024);
                            // filter tile, N-major: 64-column sub-tiles of KPS*BK k-rows are KPS*SUB_BYTES apart
                            // (leading offset), 8-row k groups 1024 B apart (stride offset); a k-step of 16
                            // rows is 2048 B, a k-block BK rows.  Stored transposed it is K-major like the
                            // input tile.
                            const uint64_t b_desc = B_KM ? make_smem_desc(b_addr, 16, 1024)
                                                         : make_smem_desc(b_addr + kbi * C::SUB_BYTES, KPS * C::SUB_BYTES, 1024);
                            constexpr int A_STEP = A_MN ? C::B_KSTEP_DESC : 2, B_STEP = B_KM ? 2 : C::B_KSTEP_DESC;
#pragma unroll
                            for (int k = 0; k < K_STEPS; ++k)
                                mma(d_tmem, a_desc + (uint64_t)(k * A_STEP), b_desc + (uint64_t)(k * B_STEP),
                                    (kb + kbi > kb0 || k > 0) ? 1u : 0u);
                        }
                        // the stage is free (in every CTA of the group) once these MMAs have read it
                        commit_all(empty_bar(s));
                    }
                }
                if (ok) commit_all(acc_full_bar(buf));
            }
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------ converter (f32 only; warps 6 to 21)
        if constexpr (F32) {
            const int cw = warp - 6;                       // converter warp
            const int ct = (int)threadIdx.x - 192;         // converter thread
            // MIX: this thread's fixed share of a k-block.  Input: row (warp & 3) * 32 + lane (the TMEM lane quarter this warp
            // may touch), k columns 8 * (cw >> 2) ..: two 16-byte chunks of the swizzled raw row.  Filter: unit cw = (sub-tile of
            // 32 columns, quarter of its 32 k): lane = column f reads 8 k down its column and owns chunks of row f.
            uint32_t mx_a_off[2] = {0, 0}, mx_hi_off[2] = {0, 0}, mx_b_src = 0, mx_h16_off = 0, mx_l16_off = 0, mx_tmem = 0;
            bool mx_has_unit = false;
            if constexpr (MIX) {
                const int row = (warp & 3) * 32 + lane;
                for (int i = 0; i < 2; ++i) mx_a_off[i] = (uint32_t)(row * 128 + ((((cw >> 2) * 2 + i) ^ (row & 7)) << 4));
                const int uj = cw >> 2, uq = cw & 3, f = uj * 32 + lane;
                mx_has_unit = cw < 4 * C::B_COLS / 32;
                mx_b_src = (uint32_t)(A_STAGE_BYTES + uj * C::SUB_BYTES + (uq * 8 * 32 + lane) * 4);
                const uint32_t rowoff = (uint32_t)((f >> 3) * 1024 + (f & 7) * 128);
                mx_hi_off[0] = rowoff + (uint32_t)(((2 * uq) ^ (f & 7)) << 4);
                mx_hi_off[1] = rowoff + (uint32_t)(((2 * uq + 1) ^ (f & 7)) << 4);
                mx_h16_off = (uint32_t)C::B_STAGE_BYTES + rowoff + (uint32_t)((uq ^ (f & 7)) << 4);
                mx_l16_off = (uint32_t)C::B_STAGE_BYTES + rowoff + (uint32_t)(((4 + uq) ^ (f & 7)) << 4);
                mx_tmem = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(C::ACC_BUFS * BN);
            }
            int it = 0;
            bool ok = true;
            Cursor cur{0, sk_u0};
            int tile, kb0, kb1, add;
            while (ok && next_item(cur, tile, kb0, kb1, add)) {
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int r = it % C::STAGES, s = it % C::SPLIT_SLOTS;
                    if (!mbar_wait(full_bar(r), (it / C::STAGES) & 1, abort_flag)) { ok = false; break; }
                    if (!mbar_wait<CG == 2>(split_empty_bar(s), ((it / C::SPLIT_SLOTS) & 1) ^ 1u, abort_flag)) { ok = false; break; }
                    if constexpr (TA) tc_fence_after();     // the MMAs that read this slot's tensor-memory columns are done
                    const uint8_t *raw = smem_gen + r * C::STAGE_BYTES;
                    uint8_t *slot = smem_gen + C::STAGES * C::STAGE_BYTES + s * C::SPLIT_BYTES;
                    if constexpr (MIX) {
                        // Plain layout, corrections as bf16 MMAs.  Every address below is fixed per thread (set up ahead of
                        // the loops); the loads go out first, input rows then filter columns.
                        const uint4 a0 = *reinterpret_cast<const uint4 *>(raw + mx_a_off[0]);
                        const uint4 a1 = *reinterpret_cast<const uint4 *>(raw + mx_a_off[1]);
                        uint32_t x[8];
                        if (mx_has_unit) {
                            const float *col = reinterpret_cast<const float *>(raw + mx_b_src);
#pragma unroll
                            for (int k = 0; k < 8; ++k) x[k] = __float_as_uint(col[k * 32]);
                        }
                        // input: this thread's 8 k of its row -> tf32 hi (8 columns), bf16 pairs lo and hi (4 columns each)
                        {
                            uint4 h0, h1, h16, l16;
                            split8_mix(a0, a1, h0, h1, h16, l16);
                            const uint32_t hi[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
                            const uint32_t lo4[4] = {l16.x, l16.y, l16.z, l16.w}, hi4[4] = {h16.x, h16.y, h16.z, h16.w};
                            const uint32_t t_base = mx_tmem + (uint32_t)(s * 64);
                            tmem_st_32x8(t_base + (cw >> 2) * 8, hi);
                            tmem_st_32x4(t_base + 32 + (cw >> 2) * 4, lo4);
                            tmem_st_32x4(t_base + 48 + (cw >> 2) * 4, hi4);
                        }
                        // filter: 8 k of this lane's column -> two chunks of its row of the tf32 hi tile, one chunk each of the
                        // hi half and the lo half of its row of the bf16 tile (rows of 128 B, 128-byte swizzled)
                        if (mx_has_unit) {
                            uint4 h0, h1, h16, l16;
                            split8_mix(make_uint4(x[0], x[1], x[2], x[3]), make_uint4(x[4], x[5], x[6], x[7]), h0, h1, h16, l16);
                            *reinterpret_cast<uint4 *>(slot + mx_hi_off[0]) = h0;
                            *reinterpret_cast<uint4 *>(slot + mx_hi_off[1]) = h1;
                            *reinterpret_cast<uint4 *>(slot + mx_h16_off) = h16;
                            *reinterpret_cast<uint4 *>(slot + mx_l16_off) = l16;
                        }
                    } else {
                    // An operand tile that arrives K-major (rows of 32 k, 128-byte swizzled by the TMA) is
                    // split elementwise: the swizzled placement of the elements is kept.
                    auto split_elementwise = [&](const uint8_t *src_tile, uint8_t *hi_tile, uint8_t *lo_tile, auto bytes_tag) {
                        constexpr int BYTES = decltype(bytes_tag)::value;
                        const uint4 *src = reinterpret_cast<const uint4 *>(src_tile) + ct;
                        uint4 *hi = reinterpret_cast<uint4 *>(hi_tile) + ct;
                        uint4 *lo = reinterpret_cast<uint4 *>(lo_tile) + ct;
                        constexpr int N = BYTES / 16 / CONVERTER_THREADS;   // 16-byte chunks per thread
                        static_assert(N >= 1 && BYTES % (16 * CONVERTER_THREADS) == 0, "converter chunking");
                        uint4 v[N];
#pragma unroll
                        for (int i = 0; i < N; ++i) v[i] = src[i * CONVERTER_THREADS];
#pragma unroll
                        for (int i = 0; i < N; ++i) {
                            uint4 h, l;
                            split4(v[i], h, l);
                            hi[i * CONVERTER_THREADS] = h;
                            lo[i * CONVERTER_THREADS] = l;
                        }
                    };
                    // An operand tile that arrives MN-major (sub-tiles of [32 k][32 rows-or-columns], 128-byte
                    // rows, not swizzled) is transposed while it is split: the split tiles are K-major,
                    // [row][32 k] rows of 128 B in 8-row groups with the 128-byte swizzle (16-byte chunk c of
                    // row f sits at chunk c ^ (f & 7)).  A unit is an eighth of a sub-tile (4 k); lane = f
                    // reads a column (one 128-byte row per load across the warp) and writes one chunk of its row.
                    auto split_transpose = [&](const uint8_t *src_tile, uint8_t *hi_tile, uint8_t *lo_tile, auto cols_tag) {
                        constexpr int COLS = decltype(cols_tag)::value;
                        const float *braw = reinterpret_cast<const float *>(src_tile);
                        constexpr int UNITS = 8 * COLS / 32;
#pragma unroll
                        for (int u = cw; u < UNITS; u += CONVERTER_THREADS / 32) {
                            const int j = u >> 3, eighth = u & 7;
                            const float *col = braw + j * (C::SUB_BYTES / 4) + eighth * 4 * 32 + lane;
                            uint32_t x[4];
#pragma unroll
                            for (int k = 0; k < 4; ++k) x[k] = __float_as_uint(col[k * 32]);
                            const int f = j * 32 + lane;
                            const int off = (f >> 3) * 1024 + (f & 7) * 128 + ((eighth ^ (f & 7)) << 4);
                            uint4 h, l;
                            split4(make_uint4(x[0], x[1], x[2], x[3]), h, l);
                            *reinterpret_cast<uint4 *>(hi_tile + off) = h;
                            *reinterpret_cast<uint4 *>(lo_tile + off) = l;
                        }
                    };
                    // input: K-major as stored, M-major when stored transposed; filter: N-major as stored,
                    // K-major when stored transposed.  kind::tf32 takes K-major operands only.
                    uint8_t *b_slot = slot + (TA ? 0 : 2 * A_STAGE_BYTES);
                    // Order within a k-block: the input rows are read first, the filter part (shared memory to shared
                    // memory) runs while those loads are in flight, then the input part goes to tensor memory and the
                    // proxy fence for the filter writes overlaps the tensor-memory stores; one wait at the end.
                    uint4 a_raw[2];
                    if constexpr (TA) {
                        // input tile -> tensor memory: this warp may touch lane quarter (warp & 3); the four warps
                        // of a quarter take 8 of the 32 k columns each.  Lane = row reads its 32 bytes of the
                        // swizzled raw tile and stores 8 hi and 8 lo words.
                        if constexpr (A_MN) {
                            // stored transposed: the raw tile is four [32 k][32 rows] sub-tiles (128-byte rows, not
                            // swizzled); sub-tile (warp & 3) holds this warp's rows, lane = row reads its 8 k values
                            // down a column (every load a whole 128-byte row across the warp)
                            const float *col = reinterpret_cast<const float *>(raw) + (warp & 3) * (C::SUB_BYTES / 4) + (cw >> 2) * 8 * 32 + lane;
                            a_raw[0] = make_uint4(__float_as_uint(col[0]), __float_as_uint(col[32]), __float_as_uint(col[64]), __float_as_uint(col[96]));
                            a_raw[1] = make_uint4(__float_as_uint(col[128]), __float_as_uint(col[160]), __float_as_uint(col[192]), __float_as_uint(col[224]));
                        } else {
                            const int row = (warp & 3) * 32 + lane;
                            const uint8_t *rp = raw + row * 128;
#pragma unroll
                            for (int i = 0; i < 2; ++i)
                                a_raw[i] = *reinterpret_cast<const uint4 *>(rp + ((((cw >> 2) * 2 + i) ^ (row & 7)) << 4));
                        }
                    } else if constexpr (A_MN) {
                        split_transpose(raw, slot, slot + A_STAGE_BYTES, std::integral_constant<int, BM>{});
                    } else {
                        split_elementwise(raw, slot, slot + A_STAGE_BYTES, std::integral_constant<int, A_STAGE_BYTES>{});
                    }
                    if constexpr (B_KM)
                        split_elementwise(raw + A_STAGE_BYTES, b_slot, b_slot + C::B_STAGE_BYTES, std::integral_constant<int, C::B_STAGE_BYTES>{});
                    else
                        split_transpose(raw + A_STAGE_BYTES, b_slot, b_slot + C::B_STAGE_BYTES, std::integral_constant<int, C::B_COLS>{});
                    if constexpr (TA) {
                        const int quarter = warp & 3, kpart = cw >> 2;
                        uint32_t hi[8], lo[8];
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            uint4 h, l;
                            split4(a_raw[i], h, l);
                            hi[4 * i] = h.x; hi[4 * i + 1] = h.y; hi[4 * i + 2] = h.z; hi[4 * i + 3] = h.w;
                            lo[4 * i] = l.x; lo[4 * i + 1] = l.y; lo[4 * i + 2] = l.z; lo[4 * i + 3] = l.w;
                        }
                        const uint32_t t_hi = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(C::ACC_BUFS * BN + s * 64 + kpart * 8);
                        tmem_st_32x8(t_hi, hi);
                        tmem_st_32x8(t_hi + 32, lo);
                    }
                    }   // (!MIX)
                    fence_async_smem();     // generic-proxy writes -> visible to the tensor core's reads
                    if constexpr (TA) {
                        tmem_st_wait();
                        tc_fence_before();
                    }
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(empty_bar(r));          // the raw stage may be refilled
                        if constexpr (CG == 1) mbar_arrive(split_full_bar(s));
                        else mbar_arrive_cluster(map_to_cta(split_full_bar(s), 0));
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        // The four warps share two staging tiles of 128 rows x 32 columns (16 KB, 128-byte swizzle):
        // each writes its TMEM lane quarter's rows, then ONE TMA store (or reduce-add) moves the
        // whole 128 x 32 chunk, issued by the warps in turn: a TMA instruction costs its thread
        // about as much for 16 KB as for 4 KB.
        const int q = warp & 3;        // TMEM lane quarter this warp may access
        const int ew = warp - 2;       // 0..3: whose turn it is to issue
        auto epi_sync = [] { asm volatile("bar.sync 1, 128;" ::: "memory"); };
        int tl = 0, chunk_count = 0;
        bool ok = true;
        // This grid may have started beside the kernel ahead of it.  Behind a clearing kernel the whole first reduction
        // runs meanwhile, but the first reduce-add must see the cleared output; behind any other kernel the output may
        // still be in use (read or written) until that kernel has finished.
        if (p.wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");
        Cursor cur{0, sk_u0};
        int tile, kb0, kb1, add;
        for (; ok && next_item(cur, tile, kb0, kb1, add); ++tl) {
            int mt, nt;
            tile_coords(tile, p.num_m_tiles, p.num_n_tiles, mt, nt);
            const int m0 = (mt * CG + (int)cta_rank) * BM, n0 = nt * BN;
            const int buf = tl % C::ACC_BUFS;
            // (the four warps take the same way here and meet at every epi_sync below)
            if (!epilogue_all(mbar_wait(acc_full_bar(buf), (tl / C::ACC_BUFS) & 1, abort_flag))) { ok = false; break; }
            tc_fence_after();
#pragma unroll 1
            for (int j = 0; j < BN / 32; ++j, ++chunk_count) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + j * 32), r);
                tmem_ld_wait();
                if (p.bias != nullptr || p.act != SG_ACT_NONE) {
                    // fused pointwise consumer (Sections 2.1, 3.3): r = act(acc + bias[column]); the bias loads are
                    // warp-uniform 16-byte loads (every lane holds the same 32 columns of its own row)
                    const int x = n0 + j * 32;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (p.bias != nullptr && x + 4 * c < p.N) b = __ldg(reinterpret_cast<const float4 *>(p.bias + x) + c);
                        const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            float v = __uint_as_float(r[4 * c + e]) + bv[e];
                            r[4 * c + e] = __float_as_uint((p.act == SG_ACT_RELU && v < 0.f) ? 0.f : v);
                        }
                    }
                }
                const int sb = chunk_count & 1;
                // staging tile sb was last read by the store of two chunks ago, whose issuer waited for
                // that read before the previous chunk's epi_sync
                uint8_t *row = staging_gen + sb * 16384 + (q * 32 + lane) * 128;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint4 v = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
                    *reinterpret_cast<uint4 *>(row + ((c ^ (lane & 7)) << 4)) = v;
                }
                fence_async_smem();
                // the issuer of the previous chunk's store makes sure that store has read its tile
                if (lane == 0 && ew == ((chunk_count + 3) & 3)) bulk_wait_read<0>();
                epi_sync();
                if (lane == 0 && ew == (chunk_count & 3)) {
                    const int x = n0 + j * 32;
                    if (x < p.N && m0 < p.M) {
                        if (add) tma_reduce_add_2d(&map_out, staging_addr + sb * 16384, x, m0);
                        else tma_store_2d(&map_out, staging_addr + sb * 16384, x, m0);
                    }
                    bulk_commit();
                }
            }
            // every tcgen05.ld of this buffer has completed: hand it back to the MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if constexpr (CG == 1) mbar_arrive(acc_empty_bar(buf));
                else mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));
            }
        }
        // the staging tiles must stay until the last stores have read them; the writes themselves are complete
        // when the grid is
        if (lane == 0) bulk_wait_read<0>();
    }

    // ---------------------------------------------------------------- teardown
    __syncthreads();
    if (*abort_flag) {
        // give any TMA load still in flight time to land before the shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(5000);
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

// Self-test of the time-out path: one warp waits, with a short budget, on an mbarrier that nothing ever signals, gives
// up the way the pipelines above do (abort flag, status bit) and returns normally.
__global__ void __launch_bounds__(32) wait_timeout_selftest_kernel(long long budget_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &abort_flag, budget_cycles);
    __syncwarp();
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
typedef CUresult (*EncodeIm2colFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const int *, const int *, cuuint32_t, cuuint32_t,
                                   const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// ---- process-wide host state -----------------------------------------------------------------
// g_mu guards the driver entry points, the per-device records and the overrides; it is held for a few loads and stores,
// never across a tensor-map encode or a launch.  The tensor-map cache has a lock of its own.
constexpr int kMaxDevices = 64;
constexpr int kAttrSlots = 160;
struct DeviceState {
    bool ready = false;
    int num_sms = 0;
    bool attr_set[kAttrSlots] = {};      // shared-memory limit raised for kernel instantiation `slot` on this device
};
struct Overrides {
    bool env_read = false;
    int bn = 0;      // tile width forced by SG_TC_BN or sg_set_tile_override (0: automatic)
    int cg = 0;      // CTAs per tile (0: automatic)
    int split = 0;   // k ranges per tile (0: automatic)
    int kps = 0;     // SG_TC_KPS=1 (testing): one k-block per stage everywhere
    int sk = -1;     // SG_TC_SK (testing): 0 = never cut the last wave into a stream-K tail, 2 = whenever it is possible
    int ta = -1;     // SG_TC_TA (testing): 0 never, 1 always keep the split f32 input tile in tensor memory
    int pdl = -1;    // SG_TC_PDL (testing): 0 = launches never overlap the tail of the kernel ahead of them
    int conv_single = 0;   // SG_CONV_SINGLE=1 (testing): the stride-1 convolution kernel never uses CTA pairs
    int mix = -1;    // SG_TC_MIX (testing): 0 = f32 correction products as tf32 MMAs (three tf32 products per term) instead of bf16
};
std::mutex g_mu;
EncodeTiledFn g_encode_tiled = nullptr;
EncodeIm2colFn g_encode_im2col = nullptr;
DeviceState g_dev[kMaxDevices];
Overrides g_ov;
thread_local int t_last_sk[2] = {-1, 0};
thread_local int t_last_choice[3] = {0, 0, 0};

// The environment switches are read once per process (caller holds g_mu).
void read_env_locked() {
    if (g_ov.env_read) return;
    auto env = [](const char *name, int dflt) { const char *e = getenv(name); return e ? atoi(e) : dflt; };
    g_ov.bn = env("SG_TC_BN", 0); g_ov.cg = env("SG_TC_CG", 0); g_ov.split = env("SG_TC_SPLIT", 0);
    g_ov.kps = env("SG_TC_KPS", 0); g_ov.ta = env("SG_TC_TA", -1); g_ov.sk = env("SG_TC_SK", -1);
    g_ov.pdl = env("SG_TC_PDL", -1);
    g_ov.conv_single = env("SG_CONV_SINGLE", 0);
    g_ov.mix = env("SG_TC_MIX", -1);
    g_ov.env_read = true;
}

// The current device's record (created at the first call on that device), or nullptr when the device is unusable.
// Fills a snapshot of the overrides when asked for.
const DeviceState *device_state(int *device_out, Overrides *ov_out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_encode_tiled || !g_encode_im2col) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn) return nullptr;
        g_encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
        fn = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn) return nullptr;
        g_encode_im2col = reinterpret_cast<EncodeIm2colFn>(fn);
    }
    DeviceState &d = g_dev[dev];
    if (!d.ready) {
        int major = 0;
        if (cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess || major != 10) return nullptr;
        d.ready = true;
    }
    read_env_locked();
    if (device_out) *device_out = dev;
    if (ov_out) *ov_out = g_ov;
    return &d;
}

// Raises a kernel's dynamic shared-memory limit once per device and instantiation.
template <typename Kernel>
bool ensure_smem_attr(int dev, int slot, Kernel kernel, int bytes) {
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (g_dev[dev].attr_set[slot]) return true;
    }
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(g_mu);
    g_dev[dev].attr_set[slot] = true;
    return true;
}

// ---- tensor-map cache -------------------------------------------------------------------------
// Encoding a tensor map is a driver call of about a microsecond, and a call needs three.  A map depends only on the
// address and geometry it describes (never on the memory's contents), so encoded maps are kept in a bounded,
// process-wide table keyed by everything that goes into the encode: device, base pointer, element type, extents, byte
// strides, box, traversal strides, im2col corners, swizzle and L2 promotion.  4-way buckets, oldest entry of a full bucket
// replaced; sg_shutdown drops the table.
struct MapKey {
    uint64_t base;
    uint64_t dims[5];
    uint64_t strides[4];
    uint32_t box[5];
    uint32_t trav[5];
    int32_t lower[3], upper[3];
    uint32_t rank, type, swizzle, promotion, im2col, channels_per_pixel, pixels_per_column, device;
};
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    uint32_t used, age;
};
constexpr uint32_t kCacheBuckets = 512, kCacheWays = 4;
std::mutex g_cache_mu;
MapSlot *g_cache = nullptr;
uint32_t g_cache_clock = 0;
std::atomic<long long> g_cache_hits{0}, g_cache_misses{0};

inline uint64_t hash_key(const MapKey &k) {
    const uint64_t *w = reinterpret_cast<const uint64_t *>(&k);
    uint64_t h = 0x9E3779B97F4A7C15ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; ++i) { h ^= w[i]; h *= 0xff51afd7ed558ccdull; h ^= h >> 32; }
    return h;
}
static_assert(sizeof(MapKey) % 8 == 0, "MapKey is hashed in 64-bit words");

// Looks the key up; on a miss calls `encode` (outside the lock) and stores the result.
template <typename Encode>
bool cached_map(const MapKey &key, CUtensorMap *out, Encode encode) {
    const uint32_t bucket = (uint32_t)(hash_key(key) % kCacheBuckets) * kCacheWays;
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        if (g_cache) {
            for (uint32_t w = 0; w < kCacheWays; ++w) {
                MapSlot &sl = g_cache[bucket + w];
                if (sl.used && memcmp(&sl.key, &key, sizeof(MapKey)) == 0) {
                    *out = sl.map;
                    sl.age = ++g_cache_clock;
                    g_cache_hits.fetch_add(1, std::memory_order_relaxed);
                    return true;
                }
            }
        }
    }
    if (!encode(out)) return false;
    g_cache_misses.fetch_add(1, std::memory_order_relaxed);
    std::lock_guard<std::mutex> lock(g_cache_mu);
    if (!g_cache) {
        g_cache = static_cast<MapSlot *>(calloc((size_t)kCacheBuckets * kCacheWays, sizeof(MapSlot)));
        if (!g_cache) return true;      // no table: the map is still good
    }
    uint32_t victim = 0, oldest = 0xffffffffu;
    for (uint32_t w = 0; w < kCacheWays; ++w) {
        const MapSlot &sl = g_cache[bucket + w];
        if (!sl.used) { victim = w; break; }
        if (sl.age < oldest) { oldest = sl.age; victim = w; }
    }
    MapSlot &sl = g_cache[bucket + victim];
    sl.key = key; sl.map = *out; sl.used = 1; sl.age = ++g_cache_clock;
    return true;
}

bool encode_tiled_cached(CUtensorMap *map, int device, CUtensorMapDataType type, int rank, const void *base, const cuuint64_t *dims,
                         const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle,
                         CUtensorMapL2promotion promotion) {
    MapKey k;
    memset(&k, 0, sizeof(k));
    k.base = reinterpret_cast<uint64_t>(base);
    for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.box[i] = box[i]; k.trav[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
    k.rank = (uint32_t)rank; k.type = (uint32_t)type; k.swizzle = (uint32_t)swizzle; k.promotion = (uint32_t)promotion;
    k.device = (uint32_t)device;
    EncodeTiledFn fn = g_encode_tiled;      // set before any caller gets here (device_state)
    return cached_map(k, map, [&](CUtensorMap *m) {
        const cuuint32_t ones[5] = {1, 1, 1, 1, 1};
        return fn(m, type, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                  promotion, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

bool encode_im2col_cached(CUtensorMap *map, int device, CUtensorMapDataType type, int rank, const void *base, const cuuint64_t *dims,
                          const cuuint64_t *strides, const int *lower, const int *upper, cuuint32_t channels_per_pixel,
                          cuuint32_t pixels_per_column, const cuuint32_t *trav) {
    MapKey k;
    memset(&k, 0, sizeof(k));
    k.base = reinterpret_cast<uint64_t>(base);
    for (int i = 0; i < rank; ++i) { k.dims[i] = dims[i]; k.trav[i] = trav[i]; }
    for (int i = 0; i + 1 < rank; ++i) k.strides[i] = strides[i];
    for (int i = 0; i + 2 < rank; ++i) { k.lower[i] = lower[i]; k.upper[i] = upper[i]; }
    k.rank = (uint32_t)rank; k.type = (uint32_t)type; k.swizzle = (uint32_t)CU_TENSOR_MAP_SWIZZLE_128B;
    k.promotion = (uint32_t)CU_TENSOR_MAP_L2_PROMOTION_L2_128B; k.im2col = 1;
    k.channels_per_pixel = channels_per_pixel; k.pixels_per_column = pixels_per_column; k.device = (uint32_t)device;
    EncodeIm2colFn fn = g_encode_im2col;
    return cached_map(k, map, [&](CUtensorMap *m) {
        return fn(m, type, (cuuint32_t)rank, const_cast<void *>(base), dims, strides, lower, upper, channels_per_pixel, pixels_per_column,
                  trav, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    });
}

inline bool mult(int64_t v, int64_t q) { return v % q == 0; }

struct Variant { int bn, cg; double mma_ns, mma_ns_f32; };
// Time one CTA's tensor core (bf16) or shared memory (f32: TMA fill, hi/lo split and the operand
// reads of 12 MMAs share it) needs for one k-block of a tile, in ns.
constexpr Variant kVariants[] = {{64, 1, 100.0, 750.0}, {128, 1, 135.0, 1000.0}, {256, 1, 330.0, 1500.0},
                                 {128, 2, 135.0, 750.0}, {256, 2, 330.0, 1000.0}};
constexpr int kNumVariants = sizeof(kVariants) / sizeof(kVariants[0]);

// Estimated kernel time in ns of `tiles` tiles dealt out in `sp` k ranges each over `groups`
// CTAs or CTA pairs.  A k-block costs the slowest of: the CTA's own MMA / shared-memory
// time, the CTA's share of the L2 -> shared memory fill rate of the whole chip (what bounds
// every large problem here: 9 to 14 TB/s), and the fill rate one SM reaches alone.  The
// constants were fitted to timings of every variant and split on the 125 shapes
// {256..4096}^3 in both dtypes; the choices they lead to are within 1 % of the best
// per-shape choice in total time.
double estimate_ns(const Variant &v, bool f32, int64_t tiles, int64_t groups, int num_kb, int sp, bool accumulate) {
    const int64_t items = tiles * sp;
    const int64_t waves = (items + groups - 1) / groups;
    const int kbs = (num_kb + sp - 1) / sp;
    const double active = (double)((items < groups ? items : groups) * v.cg);
    const double stage_bytes = A_STAGE_BYTES + (double)(v.bn / v.cg) * ROW_BYTES;
    const double chip_fill = f32 ? 9000.0 : 14000.0, sm_fill = f32 ? 40.0 : 130.0;      // bytes per ns
    double kb_ns = f32 ? v.mma_ns_f32 : v.mma_ns;
    if (active * stage_bytes / chip_fill > kb_ns) kb_ns = active * stage_bytes / chip_fill;
    if (stage_bytes / sm_fill > kb_ns) kb_ns = stage_bytes / sm_fill;
    const double item_ns = 1500.0 + (double)v.bn * (f32 ? 24.0 : 12.0);                // pipeline fill + epilogue of one item
    double t = (double)waves * kbs * kb_ns + item_ns + (double)(waves - 1) * (f32 ? 0.0 : 0.3) * item_ns;
    if (v.cg == 2) t += f32 ? 800.0 : 2000.0;                                          // cluster launch, cross-CTA signalling
    if (sp > 1) t += (f32 ? 4000.0 : 2500.0) - (accumulate ? 1500.0 : 0.0);            // reduce-add traffic, the clearing launch
    return t;
}

struct LaunchCtx {
    const DeviceState *dev;
    int device;
    cudaStream_t stream;
};

template <int BN, int CG, bool F32, int KPS, int LAY = 0>
sg_status launch_variant(const CUtensorMap &mi, const CUtensorMap &mf, const CUtensorMap &mo, TcParams tp, int M, int N,
                         int slot, const LaunchCtx &ctx) {
  if constexpr ((F32 && BN == 256 && CG == 1) || (KPS == 2 && (F32 || (BN == 256 && CG == 1))) ||
                ((LAY & 3) != 0 && (KPS != 1 || (BN == 256 && CG == 1) || (BN == 128 && CG == 2))) ||
                ((LAY & 4) != 0 && !F32)) {
    return SG_ERR_INTERNAL;   // the split slots of a 128 x 256 f32 tile do not fit beside a TMA ring
  } else {
    using C = Cfg<BN, CG, F32, KPS, (LAY & 4) != 0>;
    static_assert(5 * 3 * 8 <= kAttrSlots, "attribute slots");
    if (!ensure_smem_attr(ctx.device, slot, tc_gemm_kernel<BN, CG, F32, KPS, LAY>, C::SMEM_BYTES)) return SG_ERR_CUDA;
    tp.num_m_tiles = (M + CG * BM - 1) / (CG * BM);
    tp.num_n_tiles = (N + BN - 1) / BN;
    const int tiles = tp.num_m_tiles * tp.num_n_tiles * tp.splits;
    const int groups = ctx.dev->num_sms / CG;
    // (a stream-K tail deals its runs to every group, also when there are fewer tiles than groups)
    const int grid = CG * ((tiles < groups && tp.sk_units == 0) ? tiles : groups);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(C::THREADS, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = ctx.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = tp.wait_prior ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, tc_gemm_kernel<BN, CG, F32, KPS, LAY>, mi, mf, mo, tp);
    count_launch();
    note_kernel(F32 ? "tc_gemm_kernel<f32>" : "tc_gemm_kernel<bf16>");
    return e == cudaSuccess ? SG_OK : SG_ERR_CUDA;
  }
}

}  // namespace

sg_status launch_tensor(const Problem &p, const void *In, const void *Flt, float *O, cudaStream_t stream) {
    // ---- layout rules of the TMA descriptors (bytes): unit inner stride, 16-byte aligned
    //      bases and pitches; output rows uniformly strided so that O is one 2-D matrix ----
    const bool f32 = !p.in_bf16;
    const int64_t es = f32 ? 4 : 2;
    const int BK = ROW_BYTES / (int)es;          // elements per k-block
    const CUtensorMapDataType in_type = f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    // matmuls may hand either operand transposed through its strides (Section 4.6.1, A^T B and
    // A B^T): the input [k][m] with m contiguous, the filter [n][k] with k contiguous
    const bool a_mn = p.spatial_rank == 0 && p.i_c != 1 && p.i_w == 1;
    const bool b_km = p.spatial_rank == 0 && p.k_f != 1 && p.k_c == 1;
    const int lay = (a_mn ? 1 : 0) | (b_km ? 2 : 0);
    if ((p.i_c != 1 && !a_mn) || (p.k_f != 1 && !b_km) || p.o_f != 1) return SG_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(In) % 16 || reinterpret_cast<uintptr_t>(Flt) % 16 ||
        reinterpret_cast<uintptr_t>(O) % 16) return SG_ERR_UNSUPPORTED;
    const int64_t a_pitch = a_mn ? p.i_c : p.i_w, b_pitch = b_km ? p.k_f : p.k_c;     // elements between rows as stored
    if (!mult(a_pitch * es, 16) || !mult(b_pitch * es, 16) || !mult(p.o_w * 4, 16)) return SG_ERR_UNSUPPORTED;
    // TMA checks the bounds of the contiguous dimension in 16-byte units: an extent that ends inside a unit would
    // let loads read, and stores write, the rest of that unit (row padding), so such extents are left to the CUDA-core kernel
    if (!mult((a_mn ? (int64_t)p.M : (int64_t)p.C) * es, 16) || !mult((b_km ? (int64_t)p.K : (int64_t)p.N) * es, 16) ||
        !mult((int64_t)p.N * 4, 16)) return SG_ERR_UNSUPPORTED;
    if (a_mn && (p.M % BK != 0 || a_pitch < p.M)) return SG_ERR_UNSUPPORTED;   // whole sub-tile blocks of m (64 bf16 / 32 f32 rows)
    if (b_km && b_pitch < p.K) return SG_ERR_UNSUPPORTED;
    if (p.Ho > 1 && p.o_h != (int64_t)p.Wo * p.o_w) return SG_ERR_UNSUPPORTED;
    if (p.batch > 1 && p.o_n != (int64_t)p.Ho * p.Wo * p.o_w) return SG_ERR_UNSUPPORTED;
    if (p.KW > 1 && !mult(p.k_kw * es, 16)) return SG_ERR_UNSUPPORTED;
    if (p.KH > 1 && !mult(p.k_kh * es, 16)) return SG_ERR_UNSUPPORTED;
    if ((!a_mn && p.i_w < p.C) || (!b_km && p.k_c < p.N) || p.o_w < p.N) return SG_ERR_UNSUPPORTED;   // overlapping rows
    const int64_t pitch_limit = (int64_t)1 << 40;
    if (a_pitch * es >= pitch_limit || b_pitch * es >= pitch_limit || p.o_w * 4 >= pitch_limit) return SG_ERR_UNSUPPORTED;

    // a fused consumer: unit-stride, 16-byte aligned bias (the epilogue reads it in float4); overwrite mode only
    const bool fused = p.bias != nullptr || p.act != SG_ACT_NONE;
    if (fused && (p.accumulate || p.spatial_rank != 0)) return SG_ERR_UNSUPPORTED;
    if (p.bias != nullptr && (p.bias_f != 1 || reinterpret_cast<uintptr_t>(p.bias) % 16)) return SG_ERR_UNSUPPORTED;

    LaunchCtx ctx{nullptr, 0, stream};
    Overrides ov;
    ctx.dev = device_state(&ctx.device, &ov);
    if (!ctx.dev) return SG_ERR_CUDA;
    const int num_sms = ctx.dev->num_sms;

    alignas(64) CUtensorMap map_in, map_flt, map_out;
    TcParams tp{};
    tp.M = p.M; tp.N = p.N;
    tp.KW = p.KW;
    tp.kb_per_tap = (p.C + BK - 1) / BK;
    tp.num_kb = p.KH * p.KW * tp.kb_per_tap;
    tp.Ho = p.Ho; tp.Wo = p.Wo; tp.sh = p.sh; tp.sw = p.sw; tp.dh = p.dh; tp.dw = p.dw;
    tp.accumulate = p.accumulate;
    tp.bias = p.bias; tp.act = p.act;
    if (fused) { ov.split = 1; ov.sk = 0; }      // the consumer is not linear: whole reductions only

    // ---- input operand ----
    if (p.spatial_rank == 0) {
        tp.a_mode = 0;      // the map is encoded below, once the tile variant is known
    } else {
        // im2col descriptors: the bounding box of base pixels is [0, used - (K-1)*d) per spatial
        // dimension, walked with the conv stride, which yields exactly W_out (H_out) base
        // pixels per row (column); the filter tap is added per load as an offset.
        const int64_t used_w = (int64_t)(p.Wo - 1) * p.sw + (int64_t)(p.KW - 1) * p.dw + 1;
        const int64_t used_h = (int64_t)(p.Ho - 1) * p.sh + (int64_t)(p.KH - 1) * p.dh + 1;
        const int64_t span_w = (int64_t)(p.KW - 1) * p.dw, span_h = (int64_t)(p.KH - 1) * p.dh;
        if (p.sw > 8 || p.sh > 8) return SG_ERR_UNSUPPORTED;
        // Tensors below 128 KiB are kept off the im2col path.
        int64_t in_bytes = (int64_t)p.batch * (p.spatial_rank == 2 ? used_h : 1) * used_w * p.C * es;
        if (in_bytes < 131072) return SG_ERR_UNSUPPORTED;
        bool ok;
        if (p.spatial_rank == 1) {
            if (span_w > 32767) return SG_ERR_UNSUPPORTED;
            if (p.batch > 1 && !mult(p.i_n * es, 16)) return SG_ERR_UNSUPPORTED;
            tp.a_mode = 1;
            cuuint64_t dims[3] = {(cuuint64_t)p.C, (cuuint64_t)used_w, (cuuint64_t)p.batch};
            cuuint64_t strides[2] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)((p.batch > 1 ? p.i_n : used_w * p.i_w) * es)};
            int lower[1] = {0}, upper[1] = {(int)-span_w};
            cuuint32_t trav[3] = {1, (cuuint32_t)p.sw, 1};
            ok = encode_im2col_cached(&map_in, ctx.device, in_type, 3, In, dims, strides, lower, upper, BK, BM, trav);
        } else {
            if (span_w > 127 || span_h > 127) return SG_ERR_UNSUPPORTED;
            if (!mult(p.i_h * es, 16) || (p.batch > 1 && !mult(p.i_n * es, 16))) return SG_ERR_UNSUPPORTED;
            tp.a_mode = 2;
            cuuint64_t dims[4] = {(cuuint64_t)p.C, (cuuint64_t)used_w, (cuuint64_t)used_h, (cuuint64_t)p.batch};
            cuuint64_t strides[3] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)(p.i_h * es),
                                     (cuuint64_t)((p.batch > 1 ? p.i_n : used_h * p.i_h) * es)};
            int lower[2] = {0, 0}, upper[2] = {(int)-span_w, (int)-span_h};
            cuuint32_t trav[4] = {1, (cuuint32_t)p.sw, (cuuint32_t)p.sh, 1};
            ok = encode_im2col_cached(&map_in, ctx.device, in_type, 4, In, dims, strides, lower, upper, BK, BM, trav);
        }
        if (!ok) return SG_ERR_UNSUPPORTED;
    }
    // ---- output: 2-D {f, m} f32, stored in boxes of 32 columns x 128 rows ----
    {
        cuuint64_t dims[2] = {(cuuint64_t)p.N, (cuuint64_t)p.M};
        cuuint64_t strides[1] = {(cuuint64_t)(p.o_w * 4)};
        cuuint32_t box[2] = {32, BM};     // one store moves a chunk of 128 rows x 32 columns
        if (!encode_tiled_cached(&map_out, ctx.device, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, O, dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE)) return SG_ERR_UNSUPPORTED;
    }

    // ---- tile variant and k split: lowest estimated time ----
    int pick = -1, splits = 1;
    if (ov.bn > 0) {
        for (int i = 0; i < kNumVariants; ++i)
            if (kVariants[i].bn == ov.bn && kVariants[i].cg == (ov.cg > 0 ? ov.cg : 1) &&
                !(f32 && kVariants[i].bn == 256 && kVariants[i].cg == 1) &&
                !(lay != 0 && ((kVariants[i].bn == 256 && kVariants[i].cg == 1) || (kVariants[i].bn == 128 && kVariants[i].cg == 2)))) pick = i;
    }
    auto valid_split = [&](int s) {      // every range of ceil(num_kb / s) k-blocks must be non-empty
        const int per = (tp.num_kb + s - 1) / s;
        return s >= 1 && (s - 1) * per < tp.num_kb;
    };
    if (pick >= 0) {
        splits = ov.split > 0 && valid_split(ov.split) ? ov.split : 1;
    } else {
        // A forced split is taken as given when it fits the reduction (every range non-empty), with the variant that
        // is cheapest for it; one that does not fit is ignored and the estimate chooses the split as well.
        const int forced = ov.split > 0 && valid_split(ov.split) ? ov.split : 0;
        double best = 1e300;
        // (a forced pair count that no variant can honour on this shape is dropped in a second pass)
        for (int pass = 0; pass < 2 && pick < 0; ++pass)
        for (int i = 0; i < kNumVariants; ++i) {
            // (forced == 1 for a fused consumer: one work item per tile)
            const Variant &v = kVariants[i];
            if (pass == 0 && ov.cg > 0 && v.cg != ov.cg && !(v.cg == 1 && p.M <= BM)) continue;
            if (f32 && v.bn == 256 && v.cg == 1) continue;       // not built (shared-memory budget)
            if (lay != 0 && ((v.bn == 256 && v.cg == 1) || (v.bn == 128 && v.cg == 2))) continue;   // not built for transposed operands
            if (v.bn > 64 && v.bn / 2 >= p.N) continue;          // at most half of the tile would be used
            if (v.cg == 2 && p.M <= BM) continue;                // the second CTA would have no rows
            const int64_t tiles = (int64_t)((p.M + v.cg * BM - 1) / (v.cg * BM)) * ((p.N + v.bn - 1) / v.bn);
            const int64_t groups = num_sms / v.cg;
            if (forced) {
                const double c = estimate_ns(v, f32, tiles, groups, tp.num_kb, forced, p.accumulate != 0);
                if (c < best) { best = c; pick = i; splits = forced; }
                continue;
            }
            for (int sp = 1; sp <= 32; sp *= 2) {
                if (!valid_split(sp)) break;
                if (sp > 1 && tiles * (sp / 2) >= 2 * groups) break;   // already two waves without this split
                const double c = estimate_ns(v, f32, tiles, groups, tp.num_kb, sp, p.accumulate != 0);
                if (c < best) { best = c; pick = i; splits = sp; }
            }
        }
    }
    if (pick < 0) return SG_ERR_INTERNAL;
    const Variant &var = kVariants[pick];
    // bf16 matmuls with whole k-blocks move two k-blocks per stage and per TMA load
    const bool b_blocked = p.N % BK == 0 && !b_km;
    const int kps = (!f32 && lay == 0 && p.spatial_rank == 0 && p.K % BK == 0 && b_blocked &&
                     !(var.bn == 256 && var.cg == 1) && ov.kps != 1) ? 2 : 1;
    // ---- filter operand ----
    {
        const int64_t s_kw = p.KW > 1 ? p.k_kw : (int64_t)p.C * p.k_c;
        const int64_t s_kh = p.KH > 1 ? p.k_kh : (int64_t)p.KW * s_kw;
        // bf16 sub-tiles are consumed by the tensor core as they land (128-byte swizzle); f32
        // sub-tiles are read by the converter warps, one 128-byte row per load: no swizzle
        const CUtensorMapSwizzle swz = f32 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B;
        const int sub_cols = BK;      // columns of one sub-tile: a 128-byte row
        tp.b_blocked = b_blocked;
        bool ok;
        if (b_km) {
            // stored [n][k], k contiguous: 2-D {k, n}, box {BK, columns of this CTA} lands K-major
            cuuint64_t dims[2] = {(cuuint64_t)p.K, (cuuint64_t)p.N};
            cuuint64_t strides[1] = {(cuuint64_t)(b_pitch * es)};
            cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)(var.bn / var.cg)};
            ok = encode_tiled_cached(&map_flt, ctx.device, in_type, 2, Flt, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B,
                                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        } else if (tp.b_blocked) {
            // whole sub-tile column blocks: 5-D {column in block, c, column block, kw, kh}; one box
            // {sub_cols, BK (two k-blocks: 2 BK), blocks of this CTA, 1, 1} is the CTA's whole filter tile of a stage
            cuuint64_t dims[5] = {(cuuint64_t)sub_cols, (cuuint64_t)p.C, (cuuint64_t)(p.N / sub_cols), (cuuint64_t)p.KW, (cuuint64_t)p.KH};
            cuuint64_t strides[4] = {(cuuint64_t)(p.k_c * es), (cuuint64_t)ROW_BYTES, (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
            cuuint32_t box[5] = {(cuuint32_t)sub_cols, (cuuint32_t)(kps * BK), (cuuint32_t)(var.bn / var.cg / sub_cols), 1, 1};
            ok = encode_tiled_cached(&map_flt, ctx.device, in_type, 5, Flt, dims, strides, box, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        } else {
            // 4-D {f, c, kw, kh}, one sub-tile per load
            cuuint64_t dims[4] = {(cuuint64_t)p.N, (cuuint64_t)p.C, (cuuint64_t)p.KW, (cuuint64_t)p.KH};
            cuuint64_t strides[3] = {(cuuint64_t)(p.k_c * es), (cuuint64_t)(s_kw * es), (cuuint64_t)(s_kh * es)};
            cuuint32_t box[4] = {(cuuint32_t)sub_cols, (cuuint32_t)BK, 1, 1};
            ok = encode_tiled_cached(&map_flt, ctx.device, in_type, 4, Flt, dims, strides, box, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        }
        if (!ok) return SG_ERR_UNSUPPORTED;
    }
    if (p.spatial_rank == 0) {
        const CUtensorMapSwizzle swz_a = (a_mn && f32) ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B;
        bool ok;
        if (a_mn) {
            // stored [k][m], m contiguous, blocked by sub-tile rows of m (a 128-byte row: BK elements):
            // {m in block, k, m block}, box {BK, BK, 128 / BK}.  bf16 lands as an M-major operand
            // (swizzled); f32 is read by the converter warps, which transpose it (no swizzle).
            cuuint64_t dims[3] = {(cuuint64_t)BK, (cuuint64_t)p.K, (cuuint64_t)(p.M / BK)};
            cuuint64_t strides[2] = {(cuuint64_t)(a_pitch * es), (cuuint64_t)ROW_BYTES};
            cuuint32_t box[3] = {(cuuint32_t)BK, (cuuint32_t)BK, (cuuint32_t)(BM / BK)};
            ok = encode_tiled_cached(&map_in, ctx.device, in_type, 3, In, dims, strides, box, swz_a, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        } else if (kps == 2) {
            // blocked by k-blocks: {k in block, m, k-block}, box {BK, 128, 2}
            cuuint64_t dims[3] = {(cuuint64_t)BK, (cuuint64_t)p.M, (cuuint64_t)(p.K / BK)};
            cuuint64_t strides[2] = {(cuuint64_t)(p.i_w * es), (cuuint64_t)ROW_BYTES};
            cuuint32_t box[3] = {(cuuint32_t)BK, BM, 2};
            ok = encode_tiled_cached(&map_in, ctx.device, in_type, 3, In, dims, strides, box, swz_a, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        } else {
            cuuint64_t dims[2] = {(cuuint64_t)p.K, (cuuint64_t)p.M};
            cuuint64_t strides[1] = {(cuuint64_t)(p.i_w * es)};
            cuuint32_t box[2] = {(cuuint32_t)BK, BM};
            ok = encode_tiled_cached(&map_in, ctx.device, in_type, 2, In, dims, strides, box, swz_a, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        }
        if (!ok) return SG_ERR_UNSUPPORTED;
    }
    // k ranges are whole stages; every range keeps at least one k-block
    int per = (tp.num_kb + splits - 1) / splits;
    per = (per + kps - 1) / kps * kps;
    splits = (tp.num_kb + per - 1) / per;
    tp.splits = splits;
    tp.kb_per_split = per;
    // Unless something below says otherwise the kernel may start while the kernel ahead of it in the stream drains
    // (programmatic dependent launch): it sets up its barriers and tensor memory, then waits for that kernel to finish
    // before its first global read or write.
    tp.wait_prior = ov.pdl == 0 ? 0 : 2;
    if (splits > 1) {
        // partial sums meet in the output by TMA reduce-add: an overwriting call clears it first
        if (!p.accumulate) {
            if (launch_zero_fill(p, O, stream) != cudaSuccess) return SG_ERR_CUDA;
            tp.wait_prior = 1;      // the clearing kernel lets its dependents start at once: only the stores wait for it
        }
        tp.accumulate = 1;
    }
    // Stream-K tail.  When whole tiles are dealt out and the last wave would be partly filled, the tiles of that wave
    // are cut along k instead: every CTA (pair) gets an equal run of their k-blocks (whole stages), so the launch ends
    // after tiles/groups waves' worth of k-blocks instead of ceil(tiles/groups).  The runs' partial sums meet in the
    // output by reduce-add (an overwriting call clears those tiles first).  Taken when the k-blocks saved clearly
    // outweigh the extra epilogues and the clearing launch (4096^3 f32 alone on the GPU: 498 -> 468 us; inside a step
    // of concurrent launches the other launches fill the last wave anyway and nothing changes).
    {
        const int groups = num_sms / var.cg;
        const int num_m_tiles = (p.M + var.cg * BM - 1) / (var.cg * BM), num_n_tiles = (p.N + var.bn - 1) / var.bn;
        const int64_t tiles = (int64_t)num_m_tiles * num_n_tiles;
        const int left = (int)(tiles % groups);
        if (ov.sk != 0 && splits == 1 && tiles > groups && left != 0 && tp.num_kb % kps == 0) {
            const int64_t units = (int64_t)left * tp.num_kb;
            int run = (int)((units + groups - 1) / groups);
            run = (run + kps - 1) / kps * kps;
            const double kb_ns = f32 ? var.mma_ns_f32 : var.mma_ns;
            const double saved = (double)(tp.num_kb - run) * kb_ns;
            const double extra = 2.0 * (1500.0 + (double)var.bn * (f32 ? 24.0 : 12.0)) + 2500.0;
            if (run >= 4 * kps && (saved > 2.0 * extra || ov.sk == 2)) {
                tp.sk_first_tile = (int)(tiles - left);
                tp.sk_units = run;
                if (!p.accumulate) {
                    zero_tiles_kernel<<<left, 256, 0, stream>>>(O, p.o_w, p.M, p.N, var.cg * BM, var.bn, num_m_tiles, num_n_tiles, tp.sk_first_tile);
                    count_launch();
                    if (cudaGetLastError() != cudaSuccess) return SG_ERR_CUDA;
                    tp.wait_prior = 1;
                }
            }
        }
    }
    t_last_choice[0] = var.bn; t_last_choice[1] = var.cg; t_last_choice[2] = splits;
    t_last_sk[0] = tp.sk_units > 0 ? tp.sk_first_tile : -1; t_last_sk[1] = tp.sk_units;
    // f32 (either operand stored either way): the split input tile goes to tensor memory.  With
    // 256-column tiles that costs the second accumulator buffer, which short reductions used to feel; since the
    // converters stopped being the bottleneck the sweep is no slower with it everywhere (5.72 to 5.79 ms per step
    // either way), so there is one rule.
    // In the plain layout the two correction products of the split run as bf16 MMAs (see split4_mix).
    int lay_k = (f32 && ov.ta != 0) ? (lay | 4) : lay;
    if (lay_k == 4 && ov.mix != 0) lay_k = 12;
    const int slot = pick + (f32 ? kNumVariants : 0) + (kps == 2 ? 2 * kNumVariants : 0) + (lay_k == 12 ? 8 : lay_k) * 3 * kNumVariants;
#define SG_LAUNCH(BN_, CG_)                                                                                \
    (f32 ? (lay_k == 12 ? launch_variant<BN_, CG_, true, 1, 12>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)   \
            : lay_k == 4 ? launch_variant<BN_, CG_, true, 1, 4>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)     \
            : lay_k == 6 ? launch_variant<BN_, CG_, true, 1, 6>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)   \
            : lay_k == 5 ? launch_variant<BN_, CG_, true, 1, 5>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)   \
            : lay_k == 7 ? launch_variant<BN_, CG_, true, 1, 7>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)   \
            : lay == 0 ? launch_variant<BN_, CG_, true, 1>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)         \
            : lay == 1 ? launch_variant<BN_, CG_, true, 1, 1>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)    \
            : lay == 2 ? launch_variant<BN_, CG_, true, 1, 2>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)    \
                       : launch_variant<BN_, CG_, true, 1, 3>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx))   \
     : lay == 1 ? launch_variant<BN_, CG_, false, 1, 1>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)    \
     : lay == 2 ? launch_variant<BN_, CG_, false, 1, 2>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)    \
     : lay == 3 ? launch_variant<BN_, CG_, false, 1, 3>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx)    \
     : kps == 2 ? launch_variant<BN_, CG_, false, 2>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx) \
                : launch_variant<BN_, CG_, false, 1>(map_in, map_flt, map_out, tp, p.M, p.N, slot, ctx))
    switch (pick) {
        case 0: return SG_LAUNCH(64, 1);
        case 1: return SG_LAUNCH(128, 1);
        case 2: return SG_LAUNCH(256, 1);
        case 3: return SG_LAUNCH(128, 2);
        default: return SG_LAUNCH(256, 2);
    }
#undef SG_LAUNCH
}

sg_status tensor_read_status(cudaStream_t stream) {
    const sg_status a = read_status_word(stream);
    const sg_status b = conv_read_status(stream);
    const sg_status c = bandwidth_read_status(stream);
    const sg_status d = depthwise_read_status(stream);
    return a != SG_OK ? a : (b != SG_OK ? b : (c != SG_OK ? c : d));
}

cudaError_t launch_wait_timeout_selftest(long long budget_cycles, cudaStream_t stream) {
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(budget_cycles);
    count_launch();
    return cudaGetLastError();
}

bool tensor_driver_ready(int *num_sms) {
    const DeviceState *d = device_state(nullptr, nullptr);
    if (!d) return false;
    if (num_sms) *num_sms = d->num_sms;
    return true;
}

bool tensor_device_info(int *device, int *num_sms, int *pdl, int *conv_single) {
    Overrides ov;
    const DeviceState *d = device_state(device, &ov);
    if (!d) return false;
    *num_sms = d->num_sms;
    *pdl = ov.pdl;
    *conv_single = ov.conv_single;
    return true;
}

bool tensor_ensure_smem_attr(int slot, const void *kernel, int bytes) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices || slot < 0 || slot >= kAttrSlots) return false;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (g_dev[dev].attr_set[slot]) return true;
    }
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(g_mu);
    g_dev[dev].attr_set[slot] = true;
    return true;
}

bool tensor_encode_tiled(CUtensorMap *map, CUtensorMapDataType type, int rank, void *base, const cuuint64_t *dims,
                         const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle,
                         CUtensorMapL2promotion promotion) {
    int dev = 0;
    if (!device_state(&dev, nullptr)) return false;
    return encode_tiled_cached(map, dev, type, rank, base, dims, strides, box, swizzle, promotion);
}

void tensor_set_tile_override(int bn, int cg, int splits) {
    std::lock_guard<std::mutex> lock(g_mu);
    read_env_locked();
    g_ov.bn = bn; g_ov.cg = cg; g_ov.split = splits;
}

void tensor_last_stream_k(int out[2]) { out[0] = t_last_sk[0]; out[1] = t_last_sk[1]; }

void tensor_last_choice(int out[3]) { out[0] = t_last_choice[0]; out[1] = t_last_choice[1]; out[2] = t_last_choice[2]; }

void tensor_map_cache_stats(long long out[2]) { out[0] = g_cache_hits.load(); out[1] = g_cache_misses.load(); }

void tensor_shutdown() {
    {
        std::lock_guard<std::mutex> lock(g_cache_mu);
        free(g_cache);
        g_cache = nullptr;
    }
    std::lock_guard<std::mutex> lock(g_mu);
    for (DeviceState &d : g_dev) d = DeviceState{};
}

}  // namespace sg

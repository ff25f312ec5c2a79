// Two-SM tensor-core contraction: a cluster of two blocks computes one 256 x 256 tile with
// tcgen05.mma.cta_group::2.  Each block loads its own 128 rows of A and HALF of the B tile (128 of the 256
// columns) and the MMA unit reads both halves, so a block fetches 32 KB per 64-deep k-step instead of 48 KB
// and six ring stages fit in shared memory.  No multicast load is used: every byte a block needs is
// fetched by that block.
//
// Work units: whole 256 x 256 tiles for as many full rounds over the pairs as there are; the tiles left for
// the last, partly filled round are cut into two 256 x 128 units when that lets the round end in half the
// time (p.tail_split = 2), so the SMs are not left idle behind a few full-size tiles.
//
// Pair protocol (rank 0 = leader):
//   full[s]      lives in the leader; both blocks' TMA loads complete on it (cta_group::2 form), the
//                leader's producer posts the expected byte count of both;
//   empty[s], tmem_full[b]   live in each block; the leader's MMA thread arrives on both copies with a
//                multicast tcgen05.commit;
//   tmem_empty[b] lives in the leader; the eight epilogue warps of the pair arrive on it (the peer's
//                remotely).
// All waits are bounded; the only unbounded synchronisations are the two cluster barriers at the start and
// the end, which every thread reaches unconditionally.
#include <algorithm>

#include "gemm.h"
#include "gemm_tc_common.cuh"

namespace relay {

using namespace gemm_tc;

relay_status_t make_tmap_2d(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                            uint32_t box_inner, uint32_t box_outer, bool swizzle128);
relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);

namespace {

constexpr int STAGES = 6;
constexpr int A_BYTES = 128 * BK * 2, BH_BYTES = 128 * BK * 2, STAGE_BYTES = A_BYTES + BH_BYTES;   // 32 KB
constexpr int NUM_THREADS = 192;
constexpr int STAGING_BYTES = 4 * 2 * 4096;
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES + STAGING_BYTES + 256;

// Work unit u of the launch: tile index, first column and width.
struct Unit {
    int tile_m, n0, width;
};
__device__ __forceinline__ Unit unit_of(const Params &p, int u)
{
    Unit w;
    int tile, sub = 0;
    w.width = BN;
    if (u < p.full_tiles) {
        tile = u;
    } else {
        const int v = u - p.full_tiles;
        tile = p.full_tiles + v / p.tail_split;
        sub = v % p.tail_split;
        w.width = BN / p.tail_split;
    }
    w.tile_m = tile % p.tiles_m;
    w.n0 = (tile / p.tiles_m) * BN + sub * w.width;
    return w;
}

template <bool A_MN, bool B_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_c, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *staging = smem + (size_t)STAGES * STAGE_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + STAGING_BYTES);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES, *tmem_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = tc::cluster_ctarank();          // 0 = leader
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int n_units = p.full_tiles + (p.tiles_m * p.tiles_n - p.full_tiles) * p.tail_split;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&tmem_full[b], 1); tc::mbar_init(&tmem_empty[b], 8); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_a);
        tc::prefetch_tmap(&tm_b);
        tc::prefetch_tmap(&tm_c);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();                                   // the peer's barriers are initialised before anyone signals them
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        // ---------------- TMA producer (both blocks) ----------------
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int u = pair; u < n_units && ok; u += n_pairs) {
                const Unit w = unit_of(p, u);
                const int m0 = w.tile_m * 256 + (int)rank * 128;                // this block's rows
                const int n0 = w.n0 + (int)rank * (w.width >> 1);               // this block's half of the B columns
                const int b_boxes = w.width >> 7;                               // boxes of 64 columns in that half
                const uint32_t tx = 2u * (A_BYTES + (uint32_t)b_boxes * MN_BOX_BYTES);   // bytes of both blocks
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY)) { ok = false; break; }
                    uint8_t *sa = smem + (size_t)s * STAGE_BYTES, *sb = sa + A_BYTES;
                    const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);       // the leader's barrier
                    if (rank == 0) tc::mbar_expect_tx_cluster(bar, tx);
                    const int k0 = kb * BK;
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < 2; ++i) tc::tma_load_2d_pair(sa + i * MN_BOX_BYTES, &tm_a, bar, m0 + i * 64, k0);
                    } else {
                        tc::tma_load_2d_pair(sa, &tm_a, bar, k0, m0);
                    }
                    // B in boxes of 64 columns: MN-major boxes are 64 x 64 k anyway; K-major boxes of 64 rows stack
                    // to the same shared-memory image as one 128-row box
                    for (int i = 0; i < b_boxes; ++i) {
                        if (B_MN) tc::tma_load_2d_pair(sb + i * MN_BOX_BYTES, &tm_b, bar, n0 + i * 64, k0);
                        else tc::tma_load_2d_pair(sb + i * MN_BOX_BYTES, &tm_b, bar, k0, n0 + i * 64);
                    }
                    if (++s == STAGES) { s = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only) ----------------
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc_full = tc::instr_desc_bf16(256, BN, A_MN, B_MN);
            constexpr uint32_t idesc_half = tc::instr_desc_bf16(256, BN / 2, A_MN, B_MN);
            constexpr uint32_t a_lbo = A_MN ? MN_BOX_BYTES : 16, b_lbo = B_MN ? MN_BOX_BYTES : 16;
            constexpr uint32_t a_step = A_MN ? 2048 : 32, b_step = B_MN ? 2048 : 32;
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(smem), a_lbo, 1024);
            const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(smem) + A_BYTES, b_lbo, 1024);
            uint32_t t_local = 0, phase = 0, stage_off = 0;
            int s = 0;
            bool ok = true;
            for (int u = pair; u < n_units && ok; u += n_pairs, ++t_local) {
                const int buf = t_local & 1;
                const uint32_t idesc = (u < p.full_tiles || p.tail_split == 1) ? idesc_full : idesc_half;
                if (!tc::mbar_wait(&tmem_empty[buf], ((t_local >> 1) & 1) ^ 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY)) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL)) { ok = false; break; }
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + stage_off, db = desc_b0 + stage_off;
                    const uint32_t acc = kb != 0;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)
                        tc::mma_bf16_pair(d_tmem, da + ((kk * a_step) >> 4), db + ((kk * b_step) >> 4), idesc, acc | (kk != 0));
                    tc::mma_commit_pair(&empty[s]);
                    stage_off += STAGE_BYTES >> 4;
                    if (++s == STAGES) { s = 0; phase ^= 1; stage_off = 0; }
                }
                if (ok) tc::mma_commit_pair(&tmem_full[buf]);
            }
        }
    } else {
        // ---------------- epilogue (both blocks: 128 rows x 256 columns each) ----------------
        const int quarter = warp & 3;
        uint8_t *my_stage = staging + (size_t)(warp - 2) * 2 * 4096;
        uint32_t t_local = 0;
        for (int u = pair; u < n_units; u += n_pairs, ++t_local) {
            const int buf = t_local & 1;
            const Unit w = unit_of(p, u);
            const int m0 = w.tile_m * 256 + (int)rank * 128, n0 = w.n0;
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[buf], (t_local >> 1) & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc::tc_fence_after_sync();
            const int row0 = m0 + quarter * 32;
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
            if (row0 < p.M) {
                if (p.out_f32) epilogue_rows<true, 2>(p, &tm_c, taddr, my_stage, lane, row0, n0, w.width);
                else epilogue_rows<false, 2>(p, &tm_c, taddr, my_stage, lane, row0, n0, w.width);
            }
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive_cluster(tc::mapa(tc::smem_u32(&tmem_empty[buf]), 0));
        }
        if (lane == 0) tc::tma_store_wait_all<0>();
    }

    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();                                   // neither block leaves while the other may still signal it
    if (warp == 1) {
        tc::tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace

bool gemm_tc2_eligible(const GemmDesc &g, int sms)
{
    if (g.M < 256 || sms < 2) return false;
    const int64_t t2 = ((g.M + 255) / 256) * ((g.N + BN - 1) / BN);
    return t2 >= sms;                                 // at least two 256 x 256 tiles per pair of SMs
}

relay_status_t launch_gemm_tc2(const GemmDesc &g, int sms, cudaStream_t st)
{
    const bool a_mn = g.a_sk != 1, b_mn = g.b_sk != 1;
    CUtensorMap tm_a, tm_b, tm_c;
    if (a_mn) RELAY_TRY(make_tmap_2d_bf16(&tm_a, g.a, g.M, g.K, g.a_sk, 64, BK));
    else RELAY_TRY(make_tmap_2d_bf16(&tm_a, g.a, g.K, g.M, g.a_sm, BK, 128));
    if (b_mn) RELAY_TRY(make_tmap_2d_bf16(&tm_b, g.b, g.N, g.K, g.b_sk, 64, BK));
    else RELAY_TRY(make_tmap_2d_bf16(&tm_b, g.b, g.K, g.N, g.b_sn, BK, 64));
    const bool f32 = g.out_dtype == RELAY_F32;
    RELAY_TRY(make_tmap_2d(&tm_c, f32, g.c, g.N, g.M, g.ldc, f32 ? 32 : 64, 32, true));
    Params p{};
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.c = g.c; p.ldc = g.ldc;
    p.bias = g.bias; p.bias_bf16 = g.bias_dtype == RELAY_BF16; p.act = g.act; p.out_f32 = f32;
    p.tiles_m = (int)((g.M + 255) / 256); p.tiles_n = (int)((g.N + BN - 1) / BN); p.k_blocks = (int)((g.K + BK - 1) / BK);
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int pairs = std::min(n_tiles, sms / 2);
    // tiles of the last, partly filled round: two half-width units each when they then still fit one round
    const int rem = n_tiles % pairs;
    p.tail_split = (rem > 0 && 2 * rem <= pairs) ? 2 : 1;
    p.full_tiles = p.tail_split == 2 ? n_tiles - rem : n_tiles;
#define LAUNCH2(AMN, BMN)                                                                                                   \
    do {                                                                                                                    \
        RELAY_CUDA(cudaFuncSetAttribute(gemm_tc2_kernel<AMN, BMN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES)); \
        RELAY_CUDA(launch_pdl(gemm_tc2_kernel<AMN, BMN>, dim3(2 * pairs), dim3(NUM_THREADS), SMEM_BYTES, st, tm_a, tm_b, tm_c, p));                         \
    } while (0)
    if (a_mn && b_mn) LAUNCH2(true, true);
    else if (a_mn) LAUNCH2(true, false);
    else if (b_mn) LAUNCH2(false, true);
    else LAUNCH2(false, false);
#undef LAUNCH2
    return check_launch("gemm_tc2");
}

}  // namespace relay

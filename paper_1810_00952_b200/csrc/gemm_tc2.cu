// Two-SM tensor-core contraction: a cluster of two blocks computes 256-row work units with
// tcgen05.mma.cta_group::2.  Each block loads its own 128 rows of A and HALF of the unit's B columns and the
// MMA unit reads both halves.  No multicast load is used: every byte a block needs is fetched by that block.
//
// What bounds these kernels is the number of bytes a block can pull from L2 per cycle (about 48 B per cycle and
// SM here), so the work units are made as wide as the accumulator memory allows: a unit is 256 rows by 128, 256,
// 384 or 512 columns ("class" 1..4 = width / 128).  The A rows of a stage are shared by all columns of the unit,
// so a block fetches 16 KB + class x 8 KB per 64-deep k-step:
//   class 4   two MMAs of N = 256 per 16-deep step, 48 KB stages (four), 48 B per MMA cycle: the tensor pipe stays busy;
//   class 3   N = 256 and N = 128, 40 KB stages (four);
//   class 2   N = 256, 32 KB stages (six);   class 1   N = 128, 24 KB stages (eight).
// Units of class 3 and 4 own both halves of the accumulator memory (their epilogue is not overlapped with the
// next unit's main loop), units of class 1 and 2 alternate between the halves (overlapped).
//
// The host cuts the output into units so that every pair of blocks gets nearly the same work in as few, as wide
// units as possible (plan_units), sorts them widest first and passes the list as a kernel parameter; pair p
// takes units p, p + pairs, ...  When the list would not fit, units follow a fixed scheme instead: whole rounds
// of class-4 units, then 256 x 256 tiles, the tiles of a last, partly filled round cut in two.
// Classes use the same ring memory with different stage sizes and their own barriers; a pair's units never grow
// in class, and at a change of class the producer waits until every stage of the old class has been released.
//
// Pair protocol (rank 0 = leader):
//   full[s]      lives in the leader; both blocks' TMA loads complete on it (cta_group::2 form), the
//                leader's producer posts the expected byte count of both;
//   empty[s], tmem_full[b]   live in each block; the leader's MMA thread arrives on both copies with a
//                multicast tcgen05.commit;
//   tmem_empty[b] lives in the leader; the thirty-two epilogue warps of the pair arrive on it (the peer's
//                remotely).
// All waits are bounded; the only unbounded synchronisations are the two cluster barriers at the start and
// the end, which every thread reaches unconditionally.
#include <algorithm>
#include <vector>

#include "gemm.h"
#include "gemm_tc_common.cuh"

namespace relay {

using namespace gemm_tc;

relay_status_t make_tmap_2d_sw64(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_outer);
relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);

namespace {

constexpr int A_BYTES = 128 * BK * 2;                      // this block's 128 rows of A: 16 KB
constexpr int CHUNK_BYTES = 64 * BK * 2;                   // this block's 64 columns of one 128-column chunk: 8 KB
constexpr int RING_BYTES = 192 * 1024;
constexpr int NUM_THREADS = 608;                           // warp 0 A producer, warp 1 MMA, warps 2-17 epilogue, warp 18 B producer
constexpr int EPI_WARPS = 16;
constexpr int kWideMinKBlocks = 32;                        // classes 3 and 4 only for contractions at least this long
constexpr int STAGING_BYTES = EPI_WARPS * 2048;        // one 32-row x 64-byte buffer per epilogue warp
constexpr int BAR_BYTES = 512;
constexpr size_t SMEM_BYTES = 1024 + (size_t)RING_BYTES + STAGING_BYTES + BAR_BYTES;
constexpr int MAX_UNITS = 640;

__host__ __device__ constexpr int cls_stages(int c) { return c == 1 ? 8 : c == 2 ? 6 : 4; }
__host__ __device__ constexpr int cls_stage_bytes(int c) { return A_BYTES + c * CHUNK_BYTES; }
__host__ __device__ constexpr int cls_bar_base(int c) { return c == 1 ? 0 : c == 2 ? 16 : c == 3 ? 28 : 36; }   // full[], then empty[]
constexpr int BAR_TMEM = 44;                                // tmem_full[2], tmem_empty[2]
static_assert(cls_stages(1) * cls_stage_bytes(1) <= RING_BYTES && cls_stages(2) * cls_stage_bytes(2) <= RING_BYTES &&
              cls_stages(3) * cls_stage_bytes(3) <= RING_BYTES && cls_stages(4) * cls_stage_bytes(4) <= RING_BYTES, "ring too small");
static_assert((BAR_TMEM + 4) * 8 + 8 <= BAR_BYTES, "barrier area too small");

// unit list: row block | first 128-column chunk << 12 | class << 24, widest class first
struct UnitTable {
    int n;
    uint32_t e[MAX_UNITS];
};

struct Unit {
    int tile_m, n0, width;
};

// Fixed scheme (no list): tiles are numbered so that 2w and 2w+1 are the two column neighbours that class-4 unit w
// covers: tile t (t < 2 * tiles_m * (tiles_n / 2)): row block (t/2) % tiles_m, column block 2 * ((t/2) / tiles_m) + t % 2;
// an odd last column block follows in row order.
__device__ __forceinline__ void tile_pos(const Params &p, int t, int &tile_m, int &tile_n)
{
    const int paired = 2 * p.tiles_m * (p.tiles_n >> 1);
    if (t < paired) {
        const int w = t >> 1;
        tile_m = w % p.tiles_m;
        tile_n = 2 * (w / p.tiles_m) + (t & 1);
    } else {
        tile_m = t - paired;
        tile_n = p.tiles_n - 1;
    }
}

__device__ __forceinline__ Unit unit_of(const Params &p, const UnitTable &tb, int u)
{
    Unit w;
    if (tb.n > 0) {
        const uint32_t e = tb.e[u];
        w.tile_m = (int)(e & 0xFFFu);
        w.n0 = (int)((e >> 12) & 0xFFFu) * 128;
        w.width = (int)(e >> 24) * 128;
        return w;
    }
    int tile_n;
    if (u < p.wide_units) {
        tile_pos(p, 2 * u, w.tile_m, tile_n);
        w.n0 = tile_n * BN;
        w.width = 2 * BN;
        return w;
    }
    const int v = u - p.wide_units;
    int tile, sub = 0;
    w.width = BN;
    if (v < p.full_tiles) {
        tile = v;
    } else {
        const int x = v - p.full_tiles;
        tile = p.full_tiles + x / p.tail_split;
        sub = x % p.tail_split;
        w.width = BN / p.tail_split;
    }
    tile_pos(p, 2 * p.wide_units + tile, w.tile_m, tile_n);
    w.n0 = tile_n * BN + sub * w.width;
    return w;
}

// One epilogue warp drains its 32 accumulator rows, the 32-column groups [g_begin, g_end) of an accumulator that
// starts at column n0: both groups' TMEM loads are issued before the first is awaited (a load takes several hundred
// cycles), then per group bias + activation + rounding, a 32-row x 64-byte staging buffer in the 64-byte swizzle
// pattern (16-byte piece c of row r at piece c ^ ((r >> 1) & 3)) and one TMA tile store (two for f32 output).
// The drain is spread over sixteen warps because one warp alone issues these instructions only every few cycles.
template <bool OUT_F32, bool TRANSC>
__device__ __forceinline__ void finish_group(const Params &p, const CUtensorMap *tm_c, uint8_t *stage, int lane, int row0, int nc,
                                             float bias_lane, uint32_t (&r)[32])
{
    float v[32];
    if (p.bias != nullptr) {                             // warp-uniform; lane j holds the bias of column nc + j
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bias_lane, j);
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
    }
    if (TRANSC) {                                        // tanh / sigmoid: their own instantiation (they need many registers)
        if (p.gate_block > 0) {                          // LSTM gates: a 32-column group lies inside one gate block (warp-uniform)
            if (nc / p.gate_block == 2) {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = 1.0f - __fdividef(2.0f, 1.0f + __expf(2.0f * v[j]));
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __fdividef(1.0f, 1.0f + __expf(-v[j]));
            }
        } else if (p.act == RELAY_ACT_TANH) {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = OUT_F32 ? tanh_<false>(v[j]) : tanh_<true>(v[j]);
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = OUT_F32 ? sigmoid_<false>(v[j]) : sigmoid_<true>(v[j]);
        }
    } else if (p.act == RELAY_ACT_RELU) {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
    }
    const int sw = (lane >> 1) & 3;
#pragma unroll
    for (int h = 0; h < (OUT_F32 ? 2 : 1); ++h) {        // 64 bytes of every row at a time
        if (tc::elect_one()) tc::tma_store_wait_read<0>();   // the previous store (same elected lane) has read the buffer
        __syncwarp();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint4 piece;
            if (OUT_F32) piece = make_uint4(__float_as_uint(v[16 * h + 4 * c]), __float_as_uint(v[16 * h + 4 * c + 1]),
                                            __float_as_uint(v[16 * h + 4 * c + 2]), __float_as_uint(v[16 * h + 4 * c + 3]));
            else piece = make_uint4(pack2(v[8 * c], v[8 * c + 1]), pack2(v[8 * c + 2], v[8 * c + 3]), pack2(v[8 * c + 4], v[8 * c + 5]),
                                    pack2(v[8 * c + 6], v[8 * c + 7]));
            *reinterpret_cast<uint4 *>(stage + lane * 64 + ((c ^ sw) << 4)) = piece;
        }
        tc::fence_proxy_async();
        __syncwarp();
        if (tc::elect_one()) {                           // the election is deterministic: always the same lane of the warp
            tc::tma_store_2d(tm_c, stage, nc + h * (OUT_F32 ? 16 : 0), row0);
            tc::tma_store_commit();
        }
    }
}

// One epilogue warp drains its 32 accumulator rows, `per` (1 or 2) 32-column groups starting at group g0 of an
// accumulator that starts at column n0: the TMEM loads of both groups are issued before the first is awaited (a load
// takes several hundred cycles), then per group bias + activation + rounding, a 32-row x 64-byte staging buffer in
// the 64-byte swizzle pattern (16-byte piece c of row r at piece c ^ ((r >> 1) & 3)) and one TMA tile store (two for
// f32 output).  The drain is spread over sixteen warps because one warp alone issues these instructions only every
// few cycles.
template <bool OUT_F32, bool TRANSC>
__device__ __forceinline__ void drain_groups(const Params &p, const CUtensorMap *tm_c, uint32_t taddr, uint8_t *stage, int lane, int row0,
                                             int n0, const float (&bias_r)[8], int g0, int per)
{
    uint32_t ra[32], rb[32];
    const int g1 = g0 + per - 1;                         // per == 1: the same group again (its copy is not used)
    tc::tmem_ld_32x32(taddr + g0 * 32, ra);
    tc::tmem_ld_32x32(taddr + g1 * 32, rb);
    tc::tmem_ld_wait();
    float bl0 = 0.0f, bl1 = 0.0f;
#pragma unroll
    for (int q = 0; q < 8; ++q) { if (q == g0) bl0 = bias_r[q]; if (q == g1) bl1 = bias_r[q]; }
    if (n0 + g0 * 32 < p.N) finish_group<OUT_F32, TRANSC>(p, tm_c, stage, lane, row0, n0 + g0 * 32, bl0, ra);
    if (per == 2 && n0 + g1 * 32 < p.N) finish_group<OUT_F32, TRANSC>(p, tm_c, stage, lane, row0, n0 + g1 * 32, bl1, rb);
}

template <bool A_MN, bool B_MN, bool TRANSC>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                const __grid_constant__ CUtensorMap tm_c, const Params p, const __grid_constant__ UnitTable tb)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *staging = smem + RING_BYTES;
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + STAGING_BYTES);
    uint64_t *tmem_full = bars + BAR_TMEM, *tmem_empty = bars + BAR_TMEM + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + BAR_TMEM + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const uint32_t rank = tc::cluster_ctarank();          // 0 = leader
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int n_units = tb.n > 0 ? tb.n
                                 : p.wide_units + p.full_tiles + (p.tiles_m * p.tiles_n - 2 * p.wide_units - p.full_tiles) * p.tail_split;

    if (threadIdx.x == 0) {
        for (int i = 0; i < BAR_TMEM; ++i) tc::mbar_init(&bars[i], 1);
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&tmem_full[b], 1); tc::mbar_init(&tmem_empty[b], 2 * EPI_WARPS); }
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

    if (warp == 0 || warp == 18) {
        // ---------------- TMA producers (both blocks): warp 0 loads A and posts the byte count, warp 18 loads B ----------------
        // (two producer warps keep the ring fed)
        const bool load_a = warp == 0;
        {   // warp-uniform loop, an elected lane issues the copies
            int cur = 0, s = 0, n_st = 0, st_bytes = 0;
            uint32_t phase = 0;
            uint64_t *full = bars, *empty = bars;
            bool ok = true;
            for (int u = pair; u < n_units && ok; u += n_pairs) {
                const Unit w = unit_of(p, tb, u);
                const int c = w.width >> 7;
                if (c != cur) {
                    // the new class's stages lie over the old one's: every old stage must have been released
                    for (int i = 0; i < n_st && ok; ++i) {
                        ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                        if (++s == n_st) { s = 0; phase ^= 1; }
                    }
                    if (!ok) break;
                    cur = c; n_st = cls_stages(c); st_bytes = cls_stage_bytes(c);
                    full = bars + cls_bar_base(c); empty = full + n_st;
                    s = 0; phase = 0;
                }
                // the first MMA of a 16-deep step covers 2*h0 columns, the second 2*h1; this block holds h0 + h1 of them
                const int h0 = c == 1 ? 64 : 128, h1 = c == 3 ? 64 : c == 4 ? 128 : 0;
                const int m0 = w.tile_m * 256 + (int)rank * 128;
                const int na = w.n0 + (int)rank * h0, nb = w.n0 + 2 * h0 + (int)rank * h1;
                const int boxes0 = h0 >> 6, boxes = (h0 + h1) >> 6;
                const uint32_t tx = 2u * (uint32_t)st_bytes;                        // bytes of both blocks
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                    if (!ok) break;
                    uint8_t *sa = smem + (size_t)s * st_bytes, *sb = sa + A_BYTES;
                    const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);       // the leader's barrier
                    const int k0 = kb * BK;
                    if (tc::elect_one()) {
                        if (load_a) {
                            if (rank == 0) tc::mbar_expect_tx_cluster(bar, tx);
                            if (A_MN) {
#pragma unroll
                                for (int i = 0; i < 2; ++i) tc::tma_load_2d_pair(sa + i * MN_BOX_BYTES, &tm_a, bar, m0 + i * 64, k0);
                            } else {
                                tc::tma_load_2d_pair(sa, &tm_a, bar, k0, m0);
                            }
                        } else {
                            // B in boxes of 64 columns: MN-major boxes are 64 x 64 k anyway; K-major boxes of 64 rows stack
                            // to the same shared-memory image as one taller box
                            for (int i = 0; i < boxes; ++i) {
                                const int n = i < boxes0 ? na + i * 64 : nb + (i - boxes0) * 64;
                                if (B_MN) tc::tma_load_2d_pair(sb + i * MN_BOX_BYTES, &tm_b, bar, n, k0);
                                else tc::tma_load_2d_pair(sb + i * MN_BOX_BYTES, &tm_b, bar, k0, n);
                            }
                        }
                    }
                    __syncwarp();
                    if (++s == n_st) { s = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader only) ----------------
        // The whole warp runs the loop with warp-uniform values and one elected lane issues: the descriptors then stay
        // in uniform registers and an MMA costs the issuing warp far fewer cycles than from a single divergent lane.
        if (rank == 0) {
            constexpr uint32_t idesc_256 = tc::instr_desc_bf16(256, 256, A_MN, B_MN);
            constexpr uint32_t idesc_128 = tc::instr_desc_bf16(256, 128, A_MN, B_MN);
            constexpr uint32_t a_lbo = A_MN ? MN_BOX_BYTES : 16, b_lbo = B_MN ? MN_BOX_BYTES : 16;
            constexpr uint32_t a_step = A_MN ? 2048 : 32, b_step = B_MN ? 2048 : 32;
            constexpr uint32_t b1_off = (2 * CHUNK_BYTES) >> 4;   // the second MMA's columns follow the first's 128 in this block
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(smem), a_lbo, 1024);
            const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(smem) + A_BYTES, b_lbo, 1024);
            uint32_t t_local = 0, phase = 0, stage_off = 0;   // t_local counts accumulator halves handed to the epilogue
            int cur = 0, s = 0, n_st = 0, st_bytes = 0;
            uint64_t *full = bars, *empty = bars;
            bool ok = true;
            for (int u = pair; u < n_units && ok; u += n_pairs) {
                const Unit w = unit_of(p, tb, u);
                const int c = w.width >> 7;
                if (c != cur) {
                    cur = c; n_st = cls_stages(c); st_bytes = cls_stage_bytes(c);
                    full = bars + cls_bar_base(c); empty = full + n_st;
                    s = 0; phase = 0; stage_off = 0;
                }
                const bool both = c >= 3;                 // the unit owns both accumulator halves (t_local is even: such units come first)
                const int buf = t_local & 1;
                const uint32_t par = ((t_local >> 1) & 1) ^ 1;
                // every lane waits; the votes reconverge the warp (the lanes leave a wait at different times)
                if (!__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[buf], par, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                if (both && !__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[1], par, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                tc::tc_fence_after_sync();
                const uint32_t d0 = tmem_base + buf * BN, d1 = tmem_base + BN;
                const uint32_t idesc0 = c == 1 ? idesc_128 : idesc_256, idesc1 = c == 3 ? idesc_128 : idesc_256;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + stage_off, db = desc_b0 + stage_off;
                    const uint32_t acc = kb != 0;
                    if (both) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            tc::mma_bf16_pair_elect(d0, da + ((kk * a_step) >> 4), db + ((kk * b_step) >> 4), idesc0, acc | (kk != 0));
                            tc::mma_bf16_pair_elect(d1, da + ((kk * a_step) >> 4), db + b1_off + ((kk * b_step) >> 4), idesc1, acc | (kk != 0));
                        }
                    } else {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk)
                            tc::mma_bf16_pair_elect(d0, da + ((kk * a_step) >> 4), db + ((kk * b_step) >> 4), idesc0, acc | (kk != 0));
                    }
                    tc::mma_commit_pair_elect(&empty[s]);
                    stage_off += (uint32_t)st_bytes >> 4;
                    if (++s == n_st) { s = 0; phase ^= 1; stage_off = 0; }
                }
                if (!ok) break;
                tc::mma_commit_pair_elect(&tmem_full[buf]);
                if (both) tc::mma_commit_pair_elect(&tmem_full[1]);
                t_local += both ? 2 : 1;
            }
        }
    } else {
        // ---------------- epilogue (both blocks: 128 rows each; four warps per 32-row TMEM lane quarter) ----------------
        const int quarter = warp & 3;                     // TMEM lanes [32*quarter, 32*quarter+32)
        const int slot = (warp - 2) >> 2;                 // which quarter of an accumulator's 32-column groups this warp drains
        uint8_t *my_stage = staging + (size_t)(warp - 2) * 2048;
        uint32_t t_local = 0;
        bool ok_all = true;
        for (int u = pair; u < n_units && ok_all; u += n_pairs) {
            const Unit w = unit_of(p, tb, u);
            const int items = w.width > BN ? 2 : 1;       // accumulator halves of this unit, in the order the issuer fills them
            for (int item = 0; item < items; ++item, ++t_local) {
                const int buf = t_local & 1;
                const int n0 = w.n0 + item * BN, width = item == 0 ? min(w.width, BN) : w.width - BN;
                const int m0 = w.tile_m * 256 + (int)rank * 128;
                float bias_r[8];
                load_bias(p, lane, n0, width, bias_r);    // before the wait: the loads' latency overlaps the main loop
                int ok = 1;
                if (lane == 0) ok = tc::mbar_wait(&tmem_full[buf], (t_local >> 1) & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { ok_all = false; break; }
                tc::tc_fence_after_sync();
                const int row0 = m0 + quarter * 32;
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
                if (row0 < p.M) {
                    const int per = width / 128;          // 32-column groups per warp: 2 for a 256-column accumulator, 1 for 128
                    if (p.out_f32) drain_groups<true, TRANSC>(p, &tm_c, taddr, my_stage, lane, row0, n0, bias_r, slot * per, per);
                    else drain_groups<false, TRANSC>(p, &tm_c, taddr, my_stage, lane, row0, n0, bias_r, slot * per, per);
                }
                tc::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive_cluster(tc::mapa(tc::smem_u32(&tmem_empty[buf]), 0));
            }
        }
        __syncwarp();
        if (tc::elect_one()) tc::tma_store_wait_all<0>();
    }

    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();                                   // neither block leaves while the other may still signal it
    if (warp == 1) {
        tc::tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// Cuts tiles_m row blocks of `cpr` 128-column chunks into units for `pairs` pairs of blocks.  A pair's share is
// ceil(chunks / pairs) chunks; rounds over the pairs take it widest class first (4, 4, ..., then the rest), since a
// 64-deep k-step of class c costs max(256 c MMA cycles, (16 + 8 c) KB / 48 B per cycle).  A unit never crosses a
// row block, so what is left at the end of a row becomes a narrower unit.  Returns false when the list would not fit.
bool plan_units(int tiles_m, int cpr, int pairs, int k_blocks, UnitTable *tb)
{
    const int max_c = k_blocks >= kWideMinKBlocks ? 4 : 2;
    const long long total = (long long)tiles_m * cpr;
    if (tiles_m > 0xFFF || cpr > 0xFFF || total > 4LL * MAX_UNITS) return false;
    long long share = (total + pairs - 1) / pairs;
    std::vector<int> rounds;
    while (share > 0) {
        const int c = (int)std::min<long long>(max_c, share);
        rounds.push_back(c);
        share -= c;
    }
    std::vector<uint32_t> units;
    size_t r = 0;
    int quota = pairs;
    for (int m = 0; m < tiles_m; ++m) {
        int at = 0;
        while (at < cpr) {
            const int want = r < rounds.size() ? rounds[r] : std::min(2, max_c);
            const int c = std::min(want, cpr - at);
            units.push_back((uint32_t)m | ((uint32_t)at << 12) | ((uint32_t)c << 24));
            at += c;
            if (--quota == 0) { quota = pairs; ++r; }
        }
    }
    if (units.size() > (size_t)MAX_UNITS) return false;
    std::stable_sort(units.begin(), units.end(), [](uint32_t a, uint32_t b) { return (a >> 24) > (b >> 24); });
    tb->n = (int)units.size();
    std::copy(units.begin(), units.end(), tb->e);
    return true;
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
    RELAY_TRY(make_tmap_2d_sw64(&tm_c, f32, g.c, g.N, g.M, g.ldc, 32));
    Params p{};
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.c = g.c; p.ldc = g.ldc;
    p.bias = g.bias; p.bias_bf16 = g.bias_dtype == RELAY_BF16; p.act = g.act; p.out_f32 = f32;
    p.gate_block = (int)g.gate_block;
    p.tiles_m = (int)((g.M + 255) / 256); p.tiles_n = (int)((g.N + BN - 1) / BN); p.k_blocks = (int)((g.K + BK - 1) / BK);
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    const int n_tiles = p.tiles_m * p.tiles_n;
    const int pairs = std::min(n_tiles, sms / 2);
    static thread_local UnitTable tb;
    tb.n = 0;
    p.tail_split = 1;
    if (!plan_units(p.tiles_m, (int)((g.N + 127) / 128), pairs, p.k_blocks, &tb)) {
        // fixed scheme: class-4 units for whole rounds over the pairs (only for a contraction long enough to pay for
        // their exposed epilogue), then 256 x 256 tiles; the tiles of a last, partly filled round become two
        // half-width units each when they then still fit one round
        tb.n = 0;
        const int wide_rounds = p.k_blocks >= kWideMinKBlocks ? std::min(n_tiles / (2 * pairs), (p.tiles_m * (p.tiles_n / 2)) / pairs) : 0;
        p.wide_units = wide_rounds * pairs;
        const int narrow = n_tiles - 2 * p.wide_units;
        const int rem = narrow % pairs;
        p.tail_split = (rem > 0 && 2 * rem <= pairs) ? 2 : 1;
        p.full_tiles = p.tail_split == 2 ? narrow - rem : narrow;
    }
    if (g.gate_block > 0 && (g.gate_block % 32 != 0 || g.N != 4 * g.gate_block))
        return fail(RELAY_ERR_UNSUPPORTED, "gate blocks of %lld columns over N = %lld", (long long)g.gate_block, (long long)g.N);
    const bool transc = g.act == RELAY_ACT_TANH || g.act == RELAY_ACT_SIGMOID || g.gate_block > 0;
#define LAUNCH3(AMN, BMN, TR)                                                                                               \
    do {                                                                                                                    \
        RELAY_CUDA(cudaFuncSetAttribute(gemm_tc2_kernel<AMN, BMN, TR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES)); \
        RELAY_CUDA(launch_pdl(gemm_tc2_kernel<AMN, BMN, TR>, dim3(2 * pairs), dim3(NUM_THREADS), SMEM_BYTES, st, tm_a, tm_b, tm_c, p, tb));                 \
    } while (0)
#define LAUNCH2(AMN, BMN)            \
    do {                             \
        if (transc) LAUNCH3(AMN, BMN, true); \
        else LAUNCH3(AMN, BMN, false);       \
    } while (0)
    if (a_mn && b_mn) LAUNCH2(true, true);
    else if (a_mn) LAUNCH2(true, false);
    else if (b_mn) LAUNCH2(false, true);
    else LAUNCH2(false, false);
#undef LAUNCH2
#undef LAUNCH3
    return check_launch("gemm_tc2");
}

}  // namespace relay

// Host-only view of the unit plan (no GPU is touched), so that its invariants can be tested for many shapes.
extern "C" int32_t relay_debug_plan_units(int64_t M, int64_t N, int64_t K, int32_t sms, uint32_t *units, int32_t max_units)
{
    using namespace relay;
    if (M < 1 || N < 1 || K < 1 || sms < 2 || !units || max_units < 0) return -2;
    const int tiles_m = (int)((M + 255) / 256), tiles_n = (int)((N + BN - 1) / BN), k_blocks = (int)((K + BK - 1) / BK);
    const int pairs = std::min(tiles_m * tiles_n, sms / 2);
    static thread_local UnitTable tb;
    tb.n = 0;
    if (!plan_units(tiles_m, (int)((N + 127) / 128), pairs, k_blocks, &tb)) return -1;   // the fixed scheme would run
    if (tb.n > max_units) return -2;
    std::copy(tb.e, tb.e + tb.n, units);
    return tb.n;
}

// Tensor-core contraction for bf16 operands with fp32 accumulation (sm_100a):
//   TMA tile loads (128-byte swizzle) -> 4-stage shared-memory ring -> tcgen05.mma issued by one
//   thread into a double-buffered TMEM accumulator -> epilogue warps read TMEM (tcgen05.ld), add the
//   bias, apply the activation, round once and store.
// One persistent block per SM walks the output tiles.  Roles: warp 0 = TMA producer, warp 1 = TMEM
// owner + MMA issuer, the remaining warps = epilogue (one TMEM lane quarter each).
// Two tile shapes (template parameter MH = number of 128-row halves):
//   MH = 1: 128 x 256 tiles, 4 stages, the two 256-column TMEM accumulators alternate between tiles so
//           that the epilogue of tile i overlaps the main loop of tile i+1;
//   MH = 2: 256 x 256 tiles (two MMAs per k-step share the B tile in shared memory, which cuts the
//           bytes fetched per FLOP by a third), 3 stages, one accumulator per half, each half drained
//           by its own four epilogue warps and released separately.
//
// Operands are described by strides (gemm.h): an operand whose contraction index is contiguous is
// "K-major", one whose M/N index is contiguous is "MN-major"; both are fed to the MMA unit as they
// lie in memory, so forward (x K-major, W MN-major), input gradient (dZ K-major, W K-major) and
// weight gradient (x MN-major, dZ MN-major) need no transpose pass.
#include <mutex>

#include "ewise_kernels.cuh"
#include "gemm.h"
#include "gemm_tc_common.cuh"
#include "tc_common.cuh"

namespace relay {

using namespace gemm_tc;

namespace {

constexpr int B_BYTES = BN * BK * 2;

template <int MH> struct Cfg {
    static constexpr int BM = 128 * MH;
    static constexpr int STAGES = MH == 1 ? 4 : 3;
    static constexpr int A_BYTES = BM * BK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int NUM_THREADS = 64 + 128 * MH;
    static constexpr int STORE_BUFS = MH == 1 ? 2 : 1;                 // 4 KB staging buffers per epilogue warp
    static constexpr int STAGING_BYTES = 4 * MH * STORE_BUFS * 4096;
    static constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + STAGING_BYTES + 256;
};

template <bool A_MN, bool B_MN, int MH>
__global__ void __launch_bounds__(Cfg<MH>::NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
               const __grid_constant__ CUtensorMap tm_c, const Params p)
{
    constexpr int BM = Cfg<MH>::BM, STAGES = Cfg<MH>::STAGES, A_BYTES = Cfg<MH>::A_BYTES, STAGE_BYTES = Cfg<MH>::STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *staging = smem + (size_t)STAGES * STAGE_BYTES;            // [epilogue warp][STORE_BUFS][4 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + Cfg<MH>::STAGING_BYTES);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES, *tmem_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const int n_tiles = p.tiles_m * p.tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&tmem_full[b], 1); tc::mbar_init(&tmem_empty[b], 4); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_a);
        tc::prefetch_tmap(&tm_b);
        tc::prefetch_tmap(&tm_c);
    }
    if (warp == 1) {
        tc::tmem_alloc(tmem_slot, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        {   // warp-uniform loop, an elected lane issues the copies (addresses stay in uniform registers)
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                    if (!ok) break;
                    uint8_t *sa = smem + (size_t)s * STAGE_BYTES, *sb = sa + A_BYTES;
                    const int k0 = kb * BK;
                    if (tc::elect_one()) {
                    tc::mbar_expect_tx(&full[s], STAGE_BYTES);
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i) tc::tma_load_2d(sa + i * MN_BOX_BYTES, &tm_a, &full[s], m0 + i * 64, k0);
                    } else {
                        tc::tma_load_2d(sa, &tm_a, &full[s], k0, m0);     // one box of BM rows
                    }
                    if (B_MN) {
#pragma unroll
                        for (int i = 0; i < BN / 64; ++i) tc::tma_load_2d(sb + i * MN_BOX_BYTES, &tm_b, &full[s], n0 + i * 64, k0);
                    } else {
                        tc::tma_load_2d(sb, &tm_b, &full[s], k0, n0);
                    }
                    }
                    __syncwarp();
                    if (++s == STAGES) { s = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        {   // warp-uniform loop, an elected lane issues (descriptors stay in uniform registers)
            constexpr uint32_t idesc = tc::instr_desc_bf16(128, BN, A_MN, B_MN);
            // K-major: 8-row atoms 1024 B apart, one MMA (16 k) = 32 bytes along the swizzled row;
            // MN-major: 64-wide M/N groups one TMA box apart, 8-k atoms 1024 B apart, one MMA = 2 atoms.
            constexpr uint32_t a_lbo = A_MN ? MN_BOX_BYTES : 16, b_lbo = B_MN ? MN_BOX_BYTES : 16;
            constexpr uint32_t a_step = A_MN ? 2048 : 32, b_step = B_MN ? 2048 : 32;
            // descriptors of a stage differ from the stage-0 ones only in the start-address field (16-byte
            // units): the issuing thread spends one add per MMA instead of rebuilding them
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(smem), a_lbo, 1024);
            const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(smem) + A_BYTES, b_lbo, 1024);
            uint32_t t_local = 0, phase = 0, stage_off = 0;
            int s = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++t_local) {
                // MH = 1: accumulator t_local & 1;  MH = 2: accumulator h for half h, both used by every tile
                const int buf = MH == 1 ? (t_local & 1) : 0;
                const uint32_t empty_parity = MH == 1 ? (((t_local >> 1) & 1) ^ 1) : ((t_local & 1) ^ 1);
                if (!__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[buf], empty_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                if (MH == 2 && !__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[1], empty_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + stage_off, db = desc_b0 + stage_off;
                    const uint32_t acc = kb != 0;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) {
#pragma unroll
                        for (int h = 0; h < MH; ++h)
                            tc::mma_bf16_elect(d_tmem + h * BN, da + ((h * (128 * BK * 2) + kk * a_step) >> 4), db + ((kk * b_step) >> 4), idesc,
                                         acc | (kk != 0));
                    }
                    tc::mma_commit_elect(&empty[s]);          // the stage is free once these MMAs have read it
                    stage_off += STAGE_BYTES >> 4;
                    if (++s == STAGES) { s = 0; phase ^= 1; stage_off = 0; }
                }
                if (ok) tc::mma_commit_elect(&tmem_full[buf]);  // the accumulator(s) are complete
            }
        }
    } else {
        // ---------------- epilogue (4 warps per 128-row half) ----------------
        const int quarter = warp & 3;                     // TMEM lanes [32*quarter, 32*quarter+32)
        const int half = (warp - 2) >> 2;                 // which 128-row half this warp drains (MH = 2)
        uint32_t t_local = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++t_local) {
            const int buf = MH == 1 ? (t_local & 1) : half;          // accumulator to read
            const int fbar = MH == 1 ? (t_local & 1) : 0;            // barrier that announces it
            const uint32_t full_parity = MH == 1 ? ((t_local >> 1) & 1) : (t_local & 1);
            const int m0 = (tile % p.tiles_m) * BM + half * 128, n0 = (tile / p.tiles_m) * BN;
            float bias_r[8];
            load_bias(p, lane, n0, BN, bias_r);                 // before the wait: the loads' latency overlaps the main loop
            // one lane polls, the warp follows its verdict (keeps the warp converged for tcgen05.ld)
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[fbar], full_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc::tc_fence_after_sync();
            const int row0 = m0 + quarter * 32;                 // this warp's 32 rows; lane = row within them
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
            uint8_t *my_stage = staging + (size_t)(warp - 2) * Cfg<MH>::STORE_BUFS * 4096;
            if (row0 < p.M) {
                if (p.out_f32) epilogue_rows<true, Cfg<MH>::STORE_BUFS>(p, &tm_c, taddr, my_stage, lane, row0, n0, bias_r, 0, BN / 32);
                else epilogue_rows<false, Cfg<MH>::STORE_BUFS>(p, &tm_c, taddr, my_stage, lane, row0, n0, bias_r, 0, BN / 64);
            }
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&tmem_empty[buf]);
        }
    }

    if (warp >= 2 && lane == 0) tc::tma_store_wait_all<0>();   // this lane's tile stores have landed
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc::tc_fence_after_sync();
        tc::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---- host ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

}  // namespace

// 2-D tensor map (bf16 or f32): `inner` contiguous elements per row, `outer` rows `row_stride` elements
// apart, box = box_inner x box_outer, 128-byte swizzle, out-of-range elements read as zero / not written
relay_status_t make_tmap_2d(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                            uint32_t box_inner, uint32_t box_outer, bool swizzle128)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {row_stride * (f32 ? 4 : 2)};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return RELAY_OK;
}

// the same with 64-byte swizzle: boxes whose rows are 64 bytes (32 bf16 or 16 f32)
relay_status_t make_tmap_2d_sw64(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_outer)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {row_stride * (f32 ? 4 : 2)};
    cuuint32_t box[2] = {f32 ? 16u : 32u, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return RELAY_OK;
}

relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer)
{
    return make_tmap_2d(m, false, base, inner, outer, row_stride, box_inner, box_outer, true);
}

bool gemm_tc_eligible(const GemmDesc &g)
{
    if (g.in_dtype != RELAY_BF16) return false;
    if (g.out_dtype != RELAY_BF16 && g.out_dtype != RELAY_F32) return false;
    if (g.M % 8 || g.N % 8 || g.K % 8 || g.ldc % 8) return false;
    if (g.M < 64 || g.N < 64 || g.K < 64) return false;                 // too small to fill a tile: SIMT kernel
    if (g.M > (1ll << 30) || g.N > (1ll << 30) || g.K > (1ll << 30)) return false;
    if (((uintptr_t)g.a | (uintptr_t)g.b | (uintptr_t)g.c) & 15) return false;
    const bool a_ok = (g.a_sk == 1 && g.a_sm % 8 == 0) || (g.a_sm == 1 && g.a_sk % 8 == 0);
    const bool b_ok = (g.b_sk == 1 && g.b_sn % 8 == 0) || (g.b_sn == 1 && g.b_sk % 8 == 0);
    return a_ok && b_ok;
}

relay_status_t launch_gemm_tc(const GemmDesc &g, cudaStream_t st)
{
    const bool a_mn = g.a_sk != 1, b_mn = g.b_sk != 1;
    // 256 x 256 tiles fetch a third fewer bytes per FLOP but their epilogue is not overlapped; take them
    // when they do not cost an extra round of tiles over the SMs
    int dev = 0, sms = 148;
    RELAY_CUDA(cudaGetDevice(&dev));
    RELAY_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    if (gemm_tc2_eligible(g, sms)) return launch_gemm_tc2(g, sms, st);
    const int64_t t1 = ((g.M + 127) / 128) * ((g.N + BN - 1) / BN), t2 = ((g.M + 255) / 256) * ((g.N + BN - 1) / BN);
    const double cost1 = (double)((t1 + sms - 1) / sms), cost2 = 1.85 * (double)((t2 + sms - 1) / sms);
    const int mh = (g.M >= 256 && cost2 < cost1) ? 2 : 1;
    const int bm = 128 * mh;
    CUtensorMap tm_a, tm_b;
    if (a_mn) RELAY_TRY(make_tmap_2d_bf16(&tm_a, g.a, g.M, g.K, g.a_sk, 64, BK));       // rows = k, inner = m
    else RELAY_TRY(make_tmap_2d_bf16(&tm_a, g.a, g.K, g.M, g.a_sm, BK, bm));             // rows = m, inner = k
    if (b_mn) RELAY_TRY(make_tmap_2d_bf16(&tm_b, g.b, g.N, g.K, g.b_sk, 64, BK));       // rows = k, inner = n
    else RELAY_TRY(make_tmap_2d_bf16(&tm_b, g.b, g.K, g.N, g.b_sn, BK, BN));             // rows = n, inner = k
    Params p{};
    p.M = (int)g.M; p.N = (int)g.N; p.K = (int)g.K;
    p.c = g.c; p.ldc = g.ldc;
    p.bias = g.bias; p.bias_bf16 = g.bias_dtype == RELAY_BF16; p.act = g.act; p.out_f32 = g.out_dtype == RELAY_F32;
    p.tiles_m = (int)((g.M + bm - 1) / bm); p.tiles_n = (int)((g.N + BN - 1) / BN); p.k_blocks = (int)((g.K + BK - 1) / BK);
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    CUtensorMap tm_c;
    const bool f32 = g.out_dtype == RELAY_F32;
    RELAY_TRY(make_tmap_2d(&tm_c, f32, g.c, g.N, g.M, g.ldc, f32 ? 32 : 64, 32, true));
    const int grid = std::min(p.tiles_m * p.tiles_n, sms);
#define LAUNCH(AMN, BMN, MHV)                                                                                             \
    do {                                                                                                                  \
        RELAY_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<AMN, BMN, MHV>, cudaFuncAttributeMaxDynamicSharedMemorySize,       \
                                        (int)Cfg<MHV>::SMEM_BYTES));                                                      \
        RELAY_CUDA(launch_pdl(gemm_tc_kernel<AMN, BMN, MHV>, dim3(grid), dim3(Cfg<MHV>::NUM_THREADS), Cfg<MHV>::SMEM_BYTES, st, tm_a, tm_b, tm_c, p));          \
    } while (0)
#define LAUNCH_MH(AMN, BMN)          \
    do {                             \
        if (mh == 2) LAUNCH(AMN, BMN, 2); \
        else LAUNCH(AMN, BMN, 1);    \
    } while (0)
    if (a_mn && b_mn) LAUNCH_MH(true, true);
    else if (a_mn) LAUNCH_MH(true, false);
    else if (b_mn) LAUNCH_MH(false, true);
    else LAUNCH_MH(false, false);
#undef LAUNCH_MH
#undef LAUNCH
    return check_launch("gemm_tc");
}

}  // namespace relay

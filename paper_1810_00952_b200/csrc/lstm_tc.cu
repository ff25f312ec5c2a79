// Recurrent half of the LSTM sequence as ONE persistent cooperative kernel (sm_100a).
//
// Block j owns 16 hidden units (64 gate columns: i, f, g, o of those units).  Its slice of W_hh
// (64 columns x H, bf16) is loaded once by TMA and stays in shared memory for all T steps; the
// running cell state of its units lives in registers.  Each step:
//   loader warps stream bf16(h_{t-1}) [B x H] from the exchange buffer in L2 through a shared memory
//   ring by TMA (as many k-blocks in flight as the ring holds)  ->  issuer warps run tcgen05.mma
//   (D[batch row, 64 gate columns] in TMEM)  ->  epilogue warps add the precomputed input projection,
//   apply the gates, update c, write h_t (fp32 to h_all, bf16 to the exchange buffer)  ->  grid barrier.
// Batch rows are independent, so the batch is split into groups of rows that run as separate sets of
// blocks (separate exchange rows, separate barrier counters) when the SM count allows: each block then
// streams fewer rows of h per step.
// The grid barrier is a counter in global memory with a bounded spin; the kernel is launched
// cooperatively so that all blocks are resident.
#include <cooperative_groups.h>

#include <algorithm>

#include "ewise_kernels.cuh"
#include "lstm.h"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);

namespace {

constexpr int UNITS = 16, NCOL = 4 * UNITS;      // hidden units and gate columns per block
constexpr int BK = 64, MAX_STAGES = 32;
constexpr int A_TILE = 128 * BK * 2;             // what one MMA reads as its A operand: 128 rows x 64 k
constexpr int RING_BYTES = 96 * 1024;
constexpr int W_KB = NCOL * BK * 2;              // one k-block of the resident W slice
// Ring stages are only as far apart as the rows a group really has (rounded up to the 1024-byte swizzle atom):
// the MMA reads 128 rows from a stage's start, so its rows beyond the group's are whatever follows in shared
// memory (later stages, then the W slice).  Row r of the product depends on row r of A alone, and the epilogue
// reads only the group's rows, so those accumulator rows are never looked at; the ring holds four times as many
// bytes in flight as it would with zero-padded 128-row stages.
constexpr int NUM_THREADS = 256;                 // warps 0-3 epilogue, warp 4 W loader + MMA issuer 0, warps 5 and 7 h loaders, warp 6 issuer 1
constexpr int MAX_ISS = 2;
// Issuing a tcgen05.mma costs the issuing warp tens of cycles even with warp-uniform operands (and about 130 from a
// single divergent lane), more than the tensor pipe needs for an N = 64 one.  With an even number of k-blocks a ring
// stage therefore holds two of them (one barrier round per stage), each of two issuer warps takes one into its own
// accumulator, and the epilogue adds the two accumulators up.

struct Params {
    int T, B, H, n_blocks, k_blocks;
    int rows_per_group, n_epi;       // batch rows per block group; epilogue warps that own rows (ceil(rows_per_group / 32))
    int tile_stride, n_stages;       // bytes between the k-block tiles of the ring (a stage is n_iss tiles); stages in the ring
    int n_iss;                       // MMA issuers = k-blocks per stage = accumulators (1 or 2)
    int n_load;                      // loader threads (1 or 2): they take the stages of a step in turn
    const float *zx;                 // [T*B][4H] input projection + bias
    const float *h0, *c0;            // [B][H]
    float *h_all, *c_final;          // [T][B][H], [B][H]
    __nv_bfloat16 *hq;               // [2][B][H] exchange buffer for bf16(h)
    unsigned int *counter;           // grid barrier
    int *err;
    long long *timing;               // null, or 8 cycle counts that block 0 leaves (see relay_debug_lstm_phase_cycles)
};

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(unsigned int *p, unsigned int v)
{
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// The gate math of a step sits on the chain of dependent steps, 80 activations per lane: one MUFU instruction each
// (tanh.approx, relative error 2^-11, far inside the bf16-operand tolerance of this path) instead of an exp2 and a
// reciprocal.
__device__ __forceinline__ float fast_tanh(float x) { return tanh_<true>(x); }
__device__ __forceinline__ float fast_sigmoid(float x) { return fmaf(0.5f, tanh_<true>(0.5f * x), 0.5f); }

__global__ void __launch_bounds__(NUM_THREADS, 1)
lstm_persistent_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h0,
                       const __grid_constant__ CUtensorMap tm_h1, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_s = smem;                                           // [n_stages][rows of the group x 128 B], RING_BYTES
    uint8_t *w_s = smem + RING_BYTES;                              // [k_blocks][64 cols x 128 B] (at least A_TILE bytes: see above)
    uint64_t *bars = reinterpret_cast<uint64_t *>(w_s + max(p.k_blocks * W_KB, A_TILE));
    uint64_t *full = bars, *empty = bars + MAX_STAGES, *w_full = bars + 2 * MAX_STAGES, *tmem_full = bars + 2 * MAX_STAGES + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const int blk = blockIdx.x % p.n_blocks, grp = blockIdx.x / p.n_blocks;
    const int j0 = blk * UNITS;
    const int b_lo = grp * p.rows_per_group;                      // first batch row of this block's group
    const int nb = min(p.rows_per_group, p.B - b_lo);             // rows the group really has
    unsigned int *counter = p.counter + grp * 32;                 // one barrier counter per group (128 B apart)

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], p.n_iss); }
        tc::mbar_init(w_full, 1);
        tc::mbar_init(tmem_full, p.n_iss);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_w);
        tc::prefetch_tmap(&tm_h0);
        tc::prefetch_tmap(&tm_h1);
    }
    // the ring starts as zeros (finite values for the accumulator rows nobody reads)
    for (int i = threadIdx.x; i < RING_BYTES / 16; i += NUM_THREADS) reinterpret_cast<uint4 *>(a_s)[i] = make_uint4(0, 0, 0, 0);
    tc::fence_proxy_async();
    if (warp == 4) { tc::tmem_alloc(tmem_slot, MAX_ISS * NCOL); tc::tmem_relinquish(); }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < 4) {
      if (warp < p.n_epi) {
        // ------------------------------ epilogue / state owners ------------------------------
        const int b = b_lo + warp * 32 + lane;        // batch row; TMEM lane = row within the group
        const bool live = warp * 32 + lane < nb;
        float c[UNITS];
#pragma unroll
        for (int i = 0; i < UNITS; ++i) c[i] = live ? p.c0[(size_t)b * p.H + j0 + i] : 0.0f;
        // publish bf16(h0) of the owned units, then arrive for "step -1"
        if (live) {
            uint32_t packed[UNITS / 2];
#pragma unroll
            for (int i = 0; i < UNITS; i += 2) packed[i / 2] = pack2(p.h0[(size_t)b * p.H + j0 + i], p.h0[(size_t)b * p.H + j0 + i + 1]);
            uint4 *dst = reinterpret_cast<uint4 *>(p.hq + (size_t)b * p.H + j0);
            dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
        }
        // every epilogue warp arrives on the grid barrier by itself (no block-level barrier that a
        // warp which has given up could leave the others waiting on); the exchange buffer is read
        // by TMA (async proxy), so the generic-proxy stores are fenced for it before the release
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
        __syncwarp();
        if (lane == 0) red_release_add(counter, 1u);

        const bool timed = p.timing != nullptr && blockIdx.x == 0 && warp == 0;
        long long t_loop = 0, t_wait = 0, t_work = 0;
        if (timed) t_loop = clock64();
        for (int t = 0; t < p.T; ++t) {
            // the input projection does not depend on h: fetch it while the recurrent product runs
            float zx[4][UNITS];
            if (live) {
                const float *zrow = p.zx + ((size_t)t * p.B + b) * 4 * p.H + j0;
#pragma unroll
                for (int g = 0; g < 4; ++g)
#pragma unroll
                    for (int i = 0; i < UNITS; i += 4) {
                        const float4 v = *reinterpret_cast<const float4 *>(zrow + (size_t)g * p.H + i);
                        zx[g][i] = v.x; zx[g][i + 1] = v.y; zx[g][i + 2] = v.z; zx[g][i + 3] = v.w;
                    }
            }
            int ok = 1;
            const long long tw0 = timed ? clock64() : 0;
            if (lane == 0) ok = tc::mbar_wait(tmem_full, t & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            const long long tw1 = timed ? clock64() : 0;
            tc::tc_fence_after_sync();
            uint32_t d0[32], d1[32];
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16);
            tc::tmem_ld_32x32(taddr, d0);
            tc::tmem_ld_32x32(taddr + 32, d1);
            if (p.n_iss == 2) {                           // warp-uniform: the second issuer's partial sums
                uint32_t e0[32], e1[32];
                tc::tmem_ld_32x32(taddr + NCOL, e0);
                tc::tmem_ld_32x32(taddr + NCOL + 32, e1);
                tc::tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    d0[i] = __float_as_uint(__uint_as_float(d0[i]) + __uint_as_float(e0[i]));
                    d1[i] = __float_as_uint(__uint_as_float(d1[i]) + __uint_as_float(e1[i]));
                }
            } else {
                tc::tmem_ld_wait();
            }
            tc::tc_fence_before_sync();
            float hn[UNITS];
            if (live) {
#pragma unroll
                for (int i = 0; i < UNITS; ++i) {
                    const float zi = __uint_as_float(d0[i]) + zx[0][i];
                    const float zf = __uint_as_float(d0[16 + i]) + zx[1][i];
                    const float zg = __uint_as_float(d1[i]) + zx[2][i];
                    const float zo = __uint_as_float(d1[16 + i]) + zx[3][i];
                    const float cn = fmaf(fast_sigmoid(zf), c[i], fast_sigmoid(zi) * fast_tanh(zg));
                    c[i] = cn;
                    hn[i] = fast_sigmoid(zo) * fast_tanh(cn);
                }
                // publish bf16(h_t) first: it is what the other blocks wait for
                uint4 *hq = reinterpret_cast<uint4 *>(p.hq + ((size_t)((t + 1) & 1) * p.B + b) * p.H + j0);
                hq[0] = make_uint4(pack2(hn[0], hn[1]), pack2(hn[2], hn[3]), pack2(hn[4], hn[5]), pack2(hn[6], hn[7]));
                hq[1] = make_uint4(pack2(hn[8], hn[9]), pack2(hn[10], hn[11]), pack2(hn[12], hn[13]), pack2(hn[14], hn[15]));
            }
            // the warp's stores are ordered before lane 0's release by the warp barrier; the release is cumulative
            asm volatile("fence.proxy.async.global;" ::: "memory");
            __syncwarp();
            if (lane == 0) red_release_add(counter, 1u);
            if (timed) { t_wait += tw1 - tw0; t_work += clock64() - tw1; }
            if (live) {   // the fp32 copy for the caller is off the critical path
                float4 *ho = reinterpret_cast<float4 *>(p.h_all + ((size_t)t * p.B + b) * p.H + j0);
#pragma unroll
                for (int i = 0; i < UNITS; i += 4) ho[i / 4] = make_float4(hn[i], hn[i + 1], hn[i + 2], hn[i + 3]);
            }
        }
        if (timed && lane == 0) { p.timing[0] = clock64() - t_loop; p.timing[1] = t_wait; p.timing[2] = t_work; p.timing[7] = p.T; }
        if (live) {
#pragma unroll
            for (int i = 0; i < UNITS; ++i) p.c_final[(size_t)b * p.H + j0 + i] = c[i];
        }
      }
    } else if (warp == 5 || warp == 7) {
        // ------------------------------ h loaders: bf16(h_{t-1}) -> ring, by TMA ------------------------------
        // Two warps take the stages of a step in turn.  Each runs its loop warp-uniform and an elected lane issues:
        // addresses and coordinates then stay in uniform registers, which costs far fewer cycles per copy than one
        // divergent lane does.
        const int ld = warp == 5 ? 0 : 1;
        if (ld < p.n_load) {
            int s = ld;
            uint32_t phase = 0;
            bool ok = true;
            const uint32_t stage_bytes = (uint32_t)(p.n_iss * p.rows_per_group * 128);
            const bool timed = p.timing != nullptr && blockIdx.x == 0 && ld == 0 && lane == 0;
            long long t_bar = 0, t_iss = 0;
            for (int t = 0; t < p.T && ok; ++t) {
                const long long tb0 = timed ? clock64() : 0;
                // grid barrier: every block has published its part of h_{t-1} (lane 0 polls, the warp follows)
                const unsigned int target = (unsigned int)(p.n_epi * p.n_blocks) * (unsigned int)(t + 1);   // n_epi arrivals per block
                if (lane == 0) {
                    const long long t0 = clock64();
                    unsigned spins = 0;
                    while (ld_acquire(counter) < target) {
                        if ((++spins & 255u) == 0 && (*abort_flag || clock64() - t0 > tc::kWaitLimitCycles)) {
                            if (!*abort_flag) { *abort_flag = 1; atomicCAS(p.err, 0, tc::ERR_WAIT_STEP); }
                            ok = false;
                            break;
                        }
                    }
                }
                __syncwarp();                                           // lane 0's acquire is ordered before the other lanes' accesses
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                asm volatile("fence.proxy.async.global;" ::: "memory");   // every lane: whichever lane is elected issues the copies
                const long long tb1 = timed ? clock64() : 0;
                const CUtensorMap *tm_h = (t & 1) ? &tm_h1 : &tm_h0;
                for (int kb = ld * p.n_iss; kb < p.k_blocks; kb += p.n_load * p.n_iss) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                    if (!ok) break;
                    uint8_t *dst = a_s + (size_t)s * p.n_iss * p.tile_stride;
                    if (tc::elect_one()) {
                        tc::mbar_expect_tx(&full[s], stage_bytes);
                        for (int i = 0; i < p.n_iss; ++i)
                            tc::tma_load_2d(dst + (size_t)i * p.tile_stride, tm_h, &full[s], (kb + i) * BK, b_lo);   // the group's rows only
                    }
                    __syncwarp();
                    s += p.n_load;
                    if (s >= p.n_stages) { s -= p.n_stages; phase ^= 1; }
                }
                if (timed) { t_bar += tb1 - tb0; t_iss += clock64() - tb1; }
            }
            if (timed) { p.timing[3] = t_bar; p.timing[4] = t_iss; }
        }
    } else {
        // ------------------------------ MMA issuers (warp 4 also loads the W slice) ------------------------------
        // The whole warp runs the loop with warp-uniform values and one elected lane issues (mma_bf16_elect).
        const int iss = warp == 4 ? 0 : 1;
        if (iss < p.n_iss) {
            if (iss == 0 && lane == 0) {
                tc::mbar_expect_tx(w_full, (uint32_t)(p.k_blocks * W_KB));
                for (int kb = 0; kb < p.k_blocks; ++kb) tc::tma_load_2d(w_s + (size_t)kb * W_KB, &tm_w, w_full, kb * BK, blk * NCOL);
            }
            __syncwarp();
            bool ok = __all_sync(0xffffffffu, tc::mbar_wait(w_full, 0, abort_flag, p.err, tc::ERR_WAIT_FULL));
            const uint32_t idesc = tc::instr_desc_bf16(128, NCOL, false, false);
            // descriptors differ from the first one only in the start-address field (16-byte units): one add per MMA
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(a_s) + (uint32_t)(iss * p.tile_stride), 16, 1024);
            const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(w_s) + (uint32_t)(iss * W_KB), 16, 1024);
            const uint32_t a_stage = (uint32_t)(p.n_iss * p.tile_stride) >> 4, b_stage = (uint32_t)(p.n_iss * W_KB) >> 4;
            const uint32_t d_tmem = tmem_base + iss * NCOL;
            int s = 0;
            uint32_t phase = 0, a_off = 0;
            const bool timed = p.timing != nullptr && blockIdx.x == 0 && iss == 0 && lane == 0;
            long long t_first = 0, t_rest = 0;          // wait for the step's first stage (barrier + first copy); first stage -> last commit
            for (int t = 0; t < p.T && ok; ++t) {
                uint32_t b_off = 0;
                const long long tm0 = timed ? clock64() : 0;
                long long tm1 = 0;
                for (int kb = 0; kb < p.k_blocks; kb += p.n_iss) {     // this issuer's k-block of the stage: kb + iss
                    // every lane waits; the vote reconverges the warp (the lanes leave the wait at different times)
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    if (timed && kb == 0) tm1 = clock64();
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + a_off, db = desc_b0 + b_off;
                    const uint32_t acc = kb != 0;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) tc::mma_bf16_elect(d_tmem, da + 2 * kk, db + 2 * kk, idesc, acc | (kk != 0));
                    tc::mma_commit_elect(&empty[s]);
                    a_off += a_stage; b_off += b_stage;
                    if (++s == p.n_stages) { s = 0; phase ^= 1; a_off = 0; }
                }
                if (ok) tc::mma_commit_elect(tmem_full);
                if (timed) { t_first += tm1 - tm0; t_rest += clock64() - tm1; }
            }
            if (timed) { p.timing[5] = t_first; p.timing[6] = t_rest; }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) { tc::tc_fence_after_sync(); tc::tmem_dealloc(tmem_base, MAX_ISS * NCOL); }
}

// wp[blk][g*16 + i][k] = w_hh[k][g*H + blk*16 + i]: block (blk, k-block of 64) moves a 64 x 64 tile with 16-byte accesses on
// both sides (a source row holds four runs of 16 columns, one per gate block; a packed row is 64 consecutive k).  Block
// (0, 0) also clears the step counters, so the call needs no memset of its own.
__global__ void __launch_bounds__(256) pack_whh_kernel(const __nv_bfloat16 *__restrict__ w_hh, __nv_bfloat16 *__restrict__ wp, int H,
                                                        unsigned int *__restrict__ counter, int n_counter)
{
    __shared__ __align__(16) __nv_bfloat16 tile[64][66];     // [column local n][k local]; 33 words per row
    const int blk = blockIdx.x, k0 = blockIdx.y * 64;
    if (blk == 0 && k0 == 0)
        for (int e = threadIdx.x; e < n_counter; e += 256) counter[e] = 0u;
    uint4 v[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int idx = threadIdx.x + r * 256, kl = idx >> 3, g = (idx >> 1) & 3, half = idx & 1;
        v[r] = *reinterpret_cast<const uint4 *>(w_hh + (size_t)(k0 + kl) * 4 * H + (size_t)g * H + blk * 16 + half * 8);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int idx = threadIdx.x + r * 256, kl = idx >> 3, g = (idx >> 1) & 3, half = idx & 1;
        const uint32_t w[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            tile[g * 16 + half * 8 + 2 * q][kl] = __ushort_as_bfloat16((unsigned short)(w[q] & 0xffffu));
            tile[g * 16 + half * 8 + 2 * q + 1][kl] = __ushort_as_bfloat16((unsigned short)(w[q] >> 16));
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int idx = threadIdx.x + r * 256, n = idx >> 3, kc = idx & 7;
        const uint32_t *row = reinterpret_cast<const uint32_t *>(&tile[n][kc * 8]);
        *reinterpret_cast<uint4 *>(wp + ((size_t)blk * 64 + n) * H + k0 + kc * 8) = make_uint4(row[0], row[1], row[2], row[3]);
    }
}

}  // namespace

bool lstm_tc_eligible(int64_t T, int64_t B, int64_t H)
{
    if (T < 1 || B < 1 || B > 128 || H % 64 || H < 64 || H > 1024) return false;
    int dev = 0, sms = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    return coop && H / UNITS <= sms;
}

size_t lstm_tc_workspace(int64_t B, int64_t H)
{
    return align_up((size_t)H * 4 * H * 2, 1024) /* packed W_hh */ + align_up((size_t)2 * B * H * 2, 1024) /* exchange */ + 1024 /* counters */;
}

relay_status_t launch_lstm_tc_prepare(int64_t B, int64_t H, const void *w_hh, void *ws, cudaStream_t st)
{
    char *base = (char *)ws;
    __nv_bfloat16 *wp = (__nv_bfloat16 *)base;
    unsigned int *counter = (unsigned int *)(base + align_up((size_t)H * 4 * H * 2, 1024) + align_up((size_t)2 * B * H * 2, 1024));
    pack_whh_kernel<<<dim3((unsigned)(H / UNITS), (unsigned)(H / 64)), 256, 0, st>>>((const __nv_bfloat16 *)w_hh, wp, (int)H, counter, 256);
    return check_launch("pack_whh");
}

relay_status_t launch_lstm_tc(int64_t T, int64_t B, int64_t H, const float *zx, const void *w_hh, const float *h0, const float *c0,
                              float *h_all, float *c_final, void *ws, cudaStream_t st, long long *timing)
{
    char *base = (char *)ws;
    __nv_bfloat16 *wp = (__nv_bfloat16 *)base;
    __nv_bfloat16 *hq = (__nv_bfloat16 *)(base + align_up((size_t)H * 4 * H * 2, 1024));
    unsigned int *counter = (unsigned int *)((char *)hq + align_up((size_t)2 * B * H * 2, 1024));
    const int n_blocks = (int)(H / UNITS);
    CUtensorMap tm_w, tm_h0, tm_h1;
    RELAY_TRY(make_tmap_2d_bf16(&tm_w, wp, (uint64_t)H, (uint64_t)n_blocks * NCOL, (uint64_t)H, BK, NCOL));
    // split the batch into groups of rows while every block still fits on its own SM (at least 8 rows a group)
    int dev = 0, sms = 148;
    RELAY_CUDA(cudaGetDevice(&dev));
    RELAY_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    int groups = std::max(1, std::min({sms / n_blocks, (int)(B / 8), 8}));
    const int rows_per_group = (int)((B + groups - 1) / groups);
    groups = (int)((B + rows_per_group - 1) / rows_per_group);
    RELAY_TRY(make_tmap_2d_bf16(&tm_h0, hq, (uint64_t)H, (uint64_t)B, (uint64_t)H, BK, (uint32_t)rows_per_group));
    RELAY_TRY(make_tmap_2d_bf16(&tm_h1, hq + (size_t)B * H, (uint64_t)H, (uint64_t)B, (uint64_t)H, BK, (uint32_t)rows_per_group));
    Params p{};
    p.T = (int)T; p.B = (int)B; p.H = (int)H; p.n_blocks = n_blocks; p.k_blocks = (int)(H / BK);
    p.rows_per_group = rows_per_group; p.n_epi = (rows_per_group + 31) / 32;
    p.zx = zx; p.h0 = h0; p.c0 = c0; p.h_all = h_all; p.c_final = c_final; p.hq = hq; p.counter = counter;
    p.err = device_error_word();
    p.timing = timing;
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    p.n_iss = p.k_blocks % 2 == 0 ? 2 : 1;
    p.tile_stride = (int)align_up((size_t)rows_per_group * 128, 1024);
    p.n_stages = std::min(MAX_STAGES, RING_BYTES / (p.n_iss * p.tile_stride));
    // two loaders when the stages of a step split evenly between them (each then walks the ring in steps of two)
    p.n_load = ((p.k_blocks / p.n_iss) % 2 == 0 && p.n_stages % 2 == 0) ? 2 : 1;
    // what follows the ring is at least one A tile long, so the rows an MMA reads past the last stage stay inside the allocation
    const size_t smem = 1024 + (size_t)RING_BYTES + std::max<size_t>((size_t)p.k_blocks * W_KB, A_TILE) + 1024;
    RELAY_CUDA(cudaFuncSetAttribute(lstm_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    void *args[] = {(void *)&tm_w, (void *)&tm_h0, (void *)&tm_h1, (void *)&p};
    RELAY_CUDA(cudaLaunchCooperativeKernel((const void *)lstm_persistent_kernel, dim3(n_blocks * groups), dim3(NUM_THREADS), args, smem, st));
    count_launch();
    return RELAY_OK;
}

}  // namespace relay

// The dependent steps of the LSTM gradient program (Section 4.2 through the recursion over time) as ONE persistent
// kernel of thread-block clusters (sm_100a).
//
// Per step the recurrent partial is  dh_rec[row, unit] = sum_col dz_{t+1}[row, col] * W_hh[unit, col]  over all 4H gate
// columns.  A cluster of four blocks owns 64 hidden units and the batch rows of one group; block k of the cluster takes
// the k-th quarter of the sum (gate block k of the columns: H of them), so that
//   * its slice of W_hh (64 units x H columns, bf16, at most 128 KB) stays in shared memory for all T steps, and
//   * per step it streams only ITS quarter of the group's dz rows from L2 (rows x H bf16): every element of dz is read
//     by H / 64 blocks, not by H / 16 as it would be if each block summed over all 4H columns for a 16-unit slice.
// Step: the loader warp waits for the group's grid barrier and streams the dz quarter through a ring by TMA (a stage =
// one k-block per issuer, brought by ONE copy through a [k-block][row][64] view of dZ) -> four issuer warps run
// tcgen05.mma, each into its own accumulator, with the W slice as the M operand and the dz rows as the N operand (D[unit, row] in TMEM, M = 64,
// N = the group's rows rounded up to 16: the tensor pipe's time grows with N, and a group has few rows) -> sixteen warps
// read the accumulator and send the 16 units that block q of the cluster does the gate math for to that block's shared
// memory (st.async: the data and the byte count that completes the receiver's barrier travel together, one way) -> the
// same warps, now as one thread per (row, unit) of the block's OWN 16 units, add the four quarters and dh_all[t], apply the
// gate derivatives, write bf16(dz_t); the block then arrives ONCE on the grid barrier.
// All waits are bounded; a block that gives up records why in the device error word.
#include <algorithm>

#include "ewise_kernels.cuh"
#include "lstm.h"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);
relay_status_t make_tmap_kblocks_bf16(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t row_stride, uint32_t box_rows,
                                      uint32_t box_kblocks);

namespace {

constexpr int KS = 4;                            // blocks per cluster = quarters of the 4H columns
constexpr int CU = 64;                           // hidden units per cluster (N of the MMAs)
constexpr int QU = CU / KS;                      // units whose gate math one block does
constexpr int BK = 64, MAX_STAGES = 32;
constexpr int A_TILE = 128 * BK * 2;             // what one MMA reads as its A operand: 128 rows x 64 k
constexpr int RING_BYTES = 64 * 1024;
constexpr int W_KB = CU * BK * 2;                // one k-block of the resident W slice
constexpr int MAX_ISS = 4;                       // issuer warps = k-blocks per ring stage = accumulators (4, 2 or 1: a divisor of H / 64)
constexpr int N_WORK = 16;                       // warps 0-15: accumulator hand-over, then the gate math
constexpr int NUM_THREADS = (N_WORK + MAX_ISS + 1) * 32;   // warps 16-19: issuers (16 also loads the W slice), warp 20: dz loader
constexpr int MAX_ROWS = 64;                     // batch rows per group
constexpr int MAX_PAIRS = MAX_ROWS * QU / (N_WORK * 32);   // (row, unit) pairs per worker thread

struct ClusterParams {
    int T, B, H, n_blocks, k_blocks;             // n_blocks: blocks per row group (H / 16); k_blocks: H / 64
    int rows_per_group;
    int n_mma, n_pad;                            // N of the MMAs (rows rounded up to 16); row length of an exchange slot (a power of two >= n_mma)
    int tmem_cols;
    int tile_stride, n_stages;
    int n_iss;                                   // issuers in use
    int box_kb;                                  // k-blocks one copy brings (n_iss: a stage in one copy; 1: tile by tile)
    const float *gates;                          // [T*B][4H] activated gates i | f | g | o
    const float *c_all, *c0;                     // [T*B][H], [B][H]
    const float *dh_all;                         // [T*B][H]
    const float *dc_final;                       // [B][H] or nullptr
    __nv_bfloat16 *dz;                           // [T*B][4H]
    float *dh0, *dc0;                            // [B][H] or nullptr
    unsigned int *counter;
    int *err;
};

__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred P;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 P, [%1], %2;\n\tselp.u32 %0, 1, 0, P;\n\t}\n"
        : "=r"(ok)
        : "r"(tc::smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded like tc::mbar_wait; acquires at cluster scope (the data behind the barrier was stored by other blocks)
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *err, int code)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned spins = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((++spins & 1023u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > tc::kWaitLimitCycles) {
                *abort_flag = 1;
                atomicCAS(err, 0, code);
                return false;
            }
        }
    }
    return true;
}
// 16 bytes into another block's shared memory; the receiver's barrier `bar` (an address in that block) counts them
__device__ __forceinline__ void st_async_v4(uint32_t addr, uint32_t bar, float a, float b, float c, float d)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d), "r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld_32x4(uint32_t taddr, uint32_t (&r)[4])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(taddr) : "memory");
}
// exchange slot of one source block: [16 units][n_pad rows] floats; the 4-row chunks of a unit's line are permuted by the
// unit so that the sixteen units of one row (what a warp of the gate math reads at once) spread over the banks
__device__ __forceinline__ int slot_index(int unit, int row, int n_pad)
{
    const int chunks = n_pad >> 2, mask = (chunks < 8 ? chunks : 8) - 1;
    return unit * n_pad + ((((row >> 2) ^ (unit & mask)) << 2) | (row & 3));
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
lstm_grad_cluster_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_dz, const ClusterParams p)
{
    extern __shared__ uint8_t smem_raw[];
    // the same offset in every block of the cluster (the dynamic segment starts at the same address in each): remote
    // addresses are formed from local ones
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *a_s = smem;                                           // [n_stages][n_iss][rows of the group x 128 B], RING_BYTES
    uint8_t *w_s = smem + RING_BYTES;                              // [k_blocks][64 units x 128 B]
    float *xbuf = reinterpret_cast<float *>(w_s + max(p.k_blocks * W_KB, A_TILE));   // [KS][QU][n_pad]: the four quarters of this block's units
    uint64_t *bars = reinterpret_cast<uint64_t *>(xbuf + (size_t)KS * QU * p.n_pad);
    uint64_t *full = bars, *empty = bars + MAX_STAGES, *w_full = bars + 2 * MAX_STAGES, *tmem_full = bars + 2 * MAX_STAGES + 1,
             *xfull = bars + 2 * MAX_STAGES + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * MAX_STAGES + 3);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const int ks = (int)tc::cluster_ctarank();                    // = blockIdx.x % KS
    const int cl = blockIdx.x / KS;                               // cluster index
    const int n_cl = p.n_blocks / KS;                             // clusters per row group
    const int ub = cl % n_cl, grp = cl / n_cl;
    const int b_lo = grp * p.rows_per_group;
    const int nb = min(p.rows_per_group, p.B - b_lo);
    unsigned int *counter = p.counter + grp * 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.n_stages; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], p.n_iss); }
        tc::mbar_init(w_full, 1);
        tc::mbar_init(tmem_full, p.n_iss);
        tc::mbar_init(xfull, 1);                                  // armed once per step with the bytes the four blocks send
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_w);
        tc::prefetch_tmap(&tm_dz);
    }
    for (int i = threadIdx.x; i < RING_BYTES / 16; i += NUM_THREADS) reinterpret_cast<uint4 *>(a_s)[i] = make_uint4(0, 0, 0, 0);
    tc::fence_proxy_async();
    if (warp == N_WORK) { tc::tmem_alloc(tmem_slot, (uint32_t)p.tmem_cols); tc::tmem_relinquish(); }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();                                           // every block's barriers exist before anyone arrives on them
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp < N_WORK) {
        // ------------------------------ hand-over of the accumulator, then the gate math ------------------------------
        // Hand-over: the accumulator row of unit n sits in TMEM lane 32 (n / 16) + n % 16 (M = 64), and warp w may read lanes
        // 32 (w % 4) .. + 31: it serves block w % 4 of the cluster, and of the rows (columns of the accumulator) it takes the 4-row
        // chunks w / 4, w / 4 + 4, ...
        const int q = warp & 3, cc = warp >> 2;
        const uint32_t x_remote = tc::mapa(tc::smem_u32(xbuf + (size_t)ks * QU * p.n_pad), (uint32_t)q);
        const uint32_t xfull_remote = tc::mapa(tc::smem_u32(xfull), (uint32_t)q);
        const uint32_t x_bytes = (uint32_t)(KS * QU * p.n_mma * sizeof(float));
        if (threadIdx.x == 0) tc::mbar_expect_tx(xfull, x_bytes);  // arms the first exchange
        // Gate math: thread i of the 512 owns pairs i, i + 512, ...; pair -> (row = pair / 16, unit = pair % 16) of this block's units
        const int u = (ub * CU + ks * QU) + (threadIdx.x & (QU - 1));
        int row[MAX_PAIRS];
        bool live[MAX_PAIRS];
        float dc[MAX_PAIRS], c_cur[MAX_PAIRS];
#pragma unroll
        for (int i = 0; i < MAX_PAIRS; ++i) {
            row[i] = (threadIdx.x >> 4) + i * (N_WORK * 32 / QU);
            live[i] = row[i] < nb;
            dc[i] = 0.0f; c_cur[i] = 0.0f;
            if (live[i]) {
                const size_t bu = (size_t)(b_lo + row[i]) * p.H + u;
                if (p.dc_final) dc[i] = p.dc_final[bu];
                c_cur[i] = p.c_all[(size_t)(p.T - 1) * p.B * p.H + bu];
            }
        }
        for (int s = 0; s <= p.T; ++s) {
            const int t = p.T - 1 - s;
            // what does not depend on the recurrent product is fetched while it runs
            float gt[MAX_PAIRS][4], c_prev[MAX_PAIRS], dh[MAX_PAIRS];
            if (s < p.T) {
#pragma unroll
                for (int i = 0; i < MAX_PAIRS; ++i) {
                    if (live[i]) {
                        const size_t r = (size_t)t * p.B + b_lo + row[i];
                        const float *grow = p.gates + r * 4 * p.H + u;
#pragma unroll
                        for (int g = 0; g < 4; ++g) gt[i][g] = grow[(size_t)g * p.H];
                        c_prev[i] = t > 0 ? p.c_all[(r - p.B) * p.H + u] : p.c0[(size_t)(b_lo + row[i]) * p.H + u];
                        dh[i] = p.dh_all[r * p.H + u];
                    }
                }
            }
            int ok = 1;                                    // a warp whose wait gave up skips the step's work but still meets the others
            if (s > 0) {
                if (lane == 0) ok = tc::mbar_wait(tmem_full, (s - 1) & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (ok) {
                    tc::tc_fence_after_sync();
                    for (int c = cc * 4; c < p.n_mma; c += 4 * (N_WORK / KS)) {
                        uint32_t d[MAX_ISS][4];                            // the issuers' partial sums
                        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + c;
#pragma unroll
                        for (int a = 0; a < MAX_ISS; ++a) tmem_ld_32x4(taddr + (a < p.n_iss ? a : 0) * p.n_mma, d[a]);   // (unused ones re-read the first)
                        tc::tmem_ld_wait();
                        float v[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            v[j] = __uint_as_float(d[0][j]);
                            if (p.n_iss >= 2) v[j] += __uint_as_float(d[1][j]);
                            if (p.n_iss == 4) v[j] = v[j] + (__uint_as_float(d[2][j]) + __uint_as_float(d[3][j]));
                        }
                        if (lane < QU) st_async_v4(x_remote + (uint32_t)slot_index(lane, c, p.n_pad) * 4, xfull_remote, v[0], v[1], v[2], v[3]);
                    }
                    tc::tc_fence_before_sync();
                    if (lane == 0) ok = mbar_wait_cluster(xfull, (s - 1) & 1, abort_flag, p.err, tc::ERR_WAIT_EXCHANGE) ? 1 : 0;
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                }
                __syncwarp();
#pragma unroll
                for (int i = 0; i < MAX_PAIRS; ++i) {
                    if (ok && live[i]) {
                        const float *xs = xbuf + slot_index(threadIdx.x & (QU - 1), row[i], p.n_pad);
                        const int qs = QU * p.n_pad;
                        const float rec = (xs[0] + xs[qs]) + (xs[2 * qs] + xs[3 * qs]);
                        if (s == p.T) { if (p.dh0) p.dh0[(size_t)(b_lo + row[i]) * p.H + u] = rec; }
                        else dh[i] += rec;
                    }
                }
                if (s == p.T) break;                        // the last pass only produces dh0: every warp leaves here
                if (ok && threadIdx.x == 0) tc::mbar_expect_tx(xfull, x_bytes);   // the phase just seen complete is over: arm the next one
            }
#pragma unroll
            for (int i = 0; i < MAX_PAIRS; ++i) {
                if (ok && live[i]) {
                    float dzv[4];
                    lstm_gate_grads(gt[i][0], gt[i][1], gt[i][2], gt[i][3], c_cur[i], c_prev[i], dh[i], dc[i], dzv);
                    c_cur[i] = c_prev[i];
                    __nv_bfloat16 *drow = p.dz + ((size_t)t * p.B + b_lo + row[i]) * 4 * p.H + u;
#pragma unroll
                    for (int g = 0; g < 4; ++g) drow[(size_t)g * p.H] = __float2bfloat16_rn(dzv[g]);
                }
            }
            // dZ[t] is read by TMA (async proxy) in the other blocks: every thread fences its generic stores for it.  Then the
            // sixteen warps meet at a barrier (which also orders their reads of the exchange slots, overwritten in the next
            // step, before the arrival) and ONE thread releases the group's counter: the release is cumulative over what the
            // barrier ordered before it.  Arrivals on one address are served one after the other (sixteen per block cost more
            // than the product itself), and a running count in shared memory whose last arrival does the release was slower
            // still.  The barrier doubles as the vote on giving up: all warps leave together if any wait ran out.
            asm volatile("fence.proxy.async.global;" ::: "memory");
            unsigned int any_bad;
            asm volatile("{\n\t.reg .pred p, q;\n\tsetp.eq.u32 p, %1, 0;\n\tbar.red.or.pred q, 1, %2, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                         : "=r"(any_bad) : "r"((unsigned int)ok), "n"(N_WORK * 32) : "memory");
            if (any_bad) break;
            if (threadIdx.x == 0) tc::red_release_add_u32(counter, 1u);
        }
#pragma unroll
        for (int i = 0; i < MAX_PAIRS; ++i)
            if (live[i] && p.dc0) p.dc0[(size_t)(b_lo + row[i]) * p.H + u] = dc[i];
    } else if (warp == N_WORK + MAX_ISS) {
        // ------------------------------ dz loader: this block's quarter of dZ[T-s], rows of the group -> ring, by TMA ------------------------------
        // warp-uniform loop, an elected lane issues
        int st = 0;
        uint32_t phase = 0;
        bool ok = true;
        const uint32_t stage_bytes = (uint32_t)(p.n_iss * p.rows_per_group * 128);
        const int kb0 = ks * p.k_blocks;
        for (int s = 1; s <= p.T && ok; ++s) {
            // grid barrier: every block of the group has written its part of dZ[T-s]
            const unsigned int target = (unsigned int)p.n_blocks * (unsigned int)s;
            if (lane == 0) {
                const long long t0 = clock64();
                unsigned spins = 0;
                while (ok && tc::ld_acquire_u32(counter) < target) {
                    if ((++spins & 255u) == 0 && (*abort_flag || clock64() - t0 > tc::kWaitLimitCycles)) {
                        if (!*abort_flag) { *abort_flag = 1; atomicCAS(p.err, 0, tc::ERR_WAIT_STEP); }
                        ok = false;
                    }
                }
            }
            __syncwarp();                                               // lane 0's acquire is ordered before the other lanes' accesses
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            asm volatile("fence.proxy.async.global;" ::: "memory");     // every lane: whichever lane is elected issues the copies
            const int row0 = (p.T - s) * p.B + b_lo;
            for (int kb = 0; kb < p.k_blocks; kb += p.n_iss) {
                ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[st], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                if (!ok) break;
                uint8_t *dst = a_s + (size_t)st * p.n_iss * p.tile_stride;
                if (tc::elect_one()) {
                    tc::mbar_expect_tx(&full[st], stage_bytes);
                    for (int i = 0; i < p.n_iss; i += p.box_kb) tc::tma_load_3d(dst + (size_t)i * p.tile_stride, &tm_dz, &full[st], 0, row0, kb0 + kb + i);
                }
                __syncwarp();
                if (++st == p.n_stages) { st = 0; phase ^= 1; }
            }
        }
    } else {
        // ------------------------------ MMA issuers (warp 16 also loads the W slice) ------------------------------
        // The whole warp runs the loop with warp-uniform values and one elected lane issues (mma_bf16_elect).
        const int iss = warp - N_WORK;
        if (iss < p.n_iss) {
        if (iss == 0 && lane == 0) {
            tc::mbar_expect_tx(w_full, (uint32_t)(p.k_blocks * W_KB));
            for (int kb = 0; kb < p.k_blocks; ++kb) tc::tma_load_2d(w_s + (size_t)kb * W_KB, &tm_w, w_full, ks * p.H + kb * BK, ub * CU);
        }
        __syncwarp();
        bool ok = __all_sync(0xffffffffu, tc::mbar_wait(w_full, 0, abort_flag, p.err, tc::ERR_WAIT_FULL));
        // D[unit, row] = W slice (M operand, 64 units) x dz rows (N operand): the rows an MMA reads beyond the group's are whatever
        // follows in shared memory, and the accumulator columns they produce are never read
        const uint32_t idesc = tc::instr_desc_bf16(CU, p.n_mma, false, false);
        // descriptors differ from the first one only in the start-address field (16-byte units): one add per MMA
        const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(a_s) + (uint32_t)(iss * p.tile_stride), 16, 1024);
        const uint64_t desc_b0 = tc::smem_desc(tc::smem_u32(w_s) + (uint32_t)(iss * W_KB), 16, 1024);
        const uint32_t a_stage = (uint32_t)(p.n_iss * p.tile_stride) >> 4, b_stage = (uint32_t)(p.n_iss * W_KB) >> 4;
        const uint32_t d_tmem = tmem_base + iss * p.n_mma;
        int st = 0;
        uint32_t phase = 0, a_off = 0;
        for (int s = 1; s <= p.T && ok; ++s) {
            uint32_t b_off = 0;
            for (int kb = 0; kb < p.k_blocks; kb += p.n_iss) {         // this issuer's k-block of the stage: kb + iss
                // every lane waits; the vote reconverges the warp (the lanes leave the wait at different times)
                ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[st], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                if (!ok) break;
                tc::tc_fence_after_sync();
                const uint64_t da = desc_a0 + a_off, db = desc_b0 + b_off;
                const uint32_t acc = kb != 0;
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) tc::mma_bf16_elect(d_tmem, db + 2 * kk, da + 2 * kk, idesc, acc | (kk != 0));
                tc::mma_commit_elect(&empty[st]);
                a_off += a_stage; b_off += b_stage;
                if (++st == p.n_stages) { st = 0; phase ^= 1; a_off = 0; }
            }
            if (ok) tc::mma_commit_elect(tmem_full);
        }
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();                                           // no block leaves while a peer may still store into its exchange slots
    if (warp == N_WORK) { tc::tc_fence_after_sync(); tc::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols); }
}

size_t smem_bytes(int k_blocks, int n_pad)
{
    return 1024 + (size_t)RING_BYTES + std::max<size_t>((size_t)k_blocks * W_KB, A_TILE) + (size_t)KS * QU * n_pad * sizeof(float) + 1024;
}

}  // namespace

relay_status_t launch_lstm_grad_cluster(int64_t T, int64_t B, int64_t H, const float *gates, const float *c_all, const float *c0,
                                        const float *dh_all, const float *dc_final, const void *w_hh, __nv_bfloat16 *dz, float *dh0,
                                        float *dc0, unsigned int *counter, cudaStream_t st, bool *launched)
{
    *launched = false;
    if (!lstm_tc_eligible(T, B, H) || H % CU) return RELAY_OK;
    const int n_blocks = (int)(H / QU);
    int dev = 0, sms = 148;
    RELAY_CUDA(cudaGetDevice(&dev));
    RELAY_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    ClusterParams p{};
    p.T = (int)T; p.B = (int)B; p.H = (int)H; p.n_blocks = n_blocks; p.k_blocks = (int)(H / BK);
    p.n_iss = p.k_blocks % 4 == 0 ? 4 : p.k_blocks % 2 == 0 ? 2 : 1;
    p.gates = gates; p.c_all = c_all; p.c0 = c0; p.dh_all = dh_all; p.dc_final = dc_final; p.dz = dz; p.dh0 = dh0; p.dc0 = dc0;
    p.counter = counter;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = KS; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeCooperative;
    attr[1].val.cooperative = 1;
    cfg.blockDim = dim3(NUM_THREADS); cfg.stream = st; cfg.attrs = attr;
    // Batch rows are independent: split them into groups that run as separate sets of clusters (fewer rows of dz per block and
    // step) as far as ALL clusters are still resident at once -- every block waits for every other block of its group.
    bool fits = false;
    for (int groups = std::max(1, std::min({sms / n_blocks, (int)(B / 8), 8})); groups >= 1 && !fits; --groups) {
        p.rows_per_group = (int)((B + groups - 1) / groups);
        const int g = (int)((B + p.rows_per_group - 1) / p.rows_per_group);
        p.n_mma = (p.rows_per_group + 15) / 16 * 16;
        for (p.n_pad = 16; p.n_pad < p.n_mma; p.n_pad *= 2) {}
        for (p.tmem_cols = 32; p.tmem_cols < p.n_iss * p.n_mma; p.tmem_cols *= 2) {}
        p.tile_stride = (int)align_up((size_t)p.rows_per_group * 128, 1024);
        p.n_stages = std::min(MAX_STAGES, RING_BYTES / (p.n_iss * p.tile_stride));
        // a stage in one copy when the tiles of its k-blocks follow one another without padding (rows a multiple of the 8-row
        // swizzle atom)
        p.box_kb = p.rows_per_group % 8 == 0 ? p.n_iss : 1;
        const size_t smem = smem_bytes(p.k_blocks, p.n_pad);
        if (p.rows_per_group > MAX_ROWS || p.n_stages < 1 || smem > 227 * 1024) continue;
        RELAY_CUDA(cudaFuncSetAttribute(lstm_grad_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        cfg.gridDim = dim3((unsigned)(n_blocks * g)); cfg.dynamicSmemBytes = smem; cfg.numAttrs = 1;
        int max_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&max_clusters, lstm_grad_cluster_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return RELAY_OK; }
        fits = max_clusters * KS >= n_blocks * g;
    }
    if (!fits) return RELAY_OK;
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    CUtensorMap tm_w, tm_dz;
    RELAY_TRY(make_tmap_2d_bf16(&tm_w, w_hh, (uint64_t)(4 * H), (uint64_t)H, (uint64_t)(4 * H), BK, CU));
    RELAY_TRY(make_tmap_kblocks_bf16(&tm_dz, dz, (uint64_t)(4 * H), (uint64_t)(T * B), (uint64_t)(4 * H), (uint32_t)p.rows_per_group, (uint32_t)p.box_kb));
    RELAY_CUDA(cudaMemsetAsync(counter, 0, 1024, st));
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, lstm_grad_cluster_kernel, tm_w, tm_dz, p) != cudaSuccess) {
        // a runtime that does not combine the cooperative attribute with clusters: residency was established above
        cudaGetLastError();
        cfg.numAttrs = 1;
        RELAY_CUDA(cudaLaunchKernelEx(&cfg, lstm_grad_cluster_kernel, tm_w, tm_dz, p));
    }
    count_launch();
    *launched = true;
    return RELAY_OK;
}

// View of a row-major bf16 matrix as [k-block][row][64 columns]: one copy brings `box_kblocks` tiles of `box_rows` rows x 128 bytes,
// stored one after the other (each 128-byte swizzled, as the MMA descriptors expect them)
relay_status_t make_tmap_kblocks_bf16(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t row_stride, uint32_t box_rows,
                                      uint32_t box_kblocks)
{
    typedef CUresult (*Fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                           const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                           CUtensorMapFloatOOBfill);
    void *fp = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
        return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {64, rows, cols / 64};
    cuuint64_t strides[2] = {row_stride * 2, 128};
    cuuint32_t box[3] = {64, box_rows, box_kblocks};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ((Fn)fp)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled (k-block view) failed with code %d", (int)r);
    return RELAY_OK;
}

}  // namespace relay

// conv2d 3x3 / stride 1 / "same" padding as implicit GEMM on the tensor cores (bf16, fp32 accumulate).
//
// Layout change first (Section 5.2 of the paper lists change of layout among the optimisations a
// whole-program IR enables): the NCHW boundary tensors are repacked once per call into NHWC, where
// a filter tap is a shift along NON-innermost tensor-map axes, so every TMA tile load starts on a
// 16-byte boundary and the zero padding is the tensor map's out-of-range fill.
//
//   forward / input gradient ("fprop" kernel):   D[o, pixel] = sum_{tap, c} Wp[o, tap, c] * Xn[pixel + tap, c]
//     A = packed weights [O][R*S*C] (K-major), B = NHWC activations (K-major, one 4-D box of
//     rows_per_tile image rows x W pixels x 64 channels per stage); the accumulator row is an output
//     channel, so the epilogue writes whole runs of an NCHW image plane with bias + activation fused.
//     The input gradient is the same kernel on dZ with the taps mirrored and the channel roles swapped.
//   weight gradient ("wgrad" kernel):             D[o, c] = sum_{pixel} dZn[pixel, o] * Xn[pixel + tap, c]
//     both operands MN-major (rows are pixels); one work unit = (tap, 128 output channels, slice of the
//     batch); slices are summed afterwards in a fixed order (split-K without atomics).
#include <algorithm>

#include "conv.h"
#include "ewise_host.h"
#include "ewise_kernels.cuh"
#include "tc_common.cuh"

namespace relay {

relay_status_t make_tmap_2d_bf16(CUtensorMap *m, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_inner, uint32_t box_outer);
relay_status_t make_tmap_nhwc_bf16(CUtensorMap *m, const void *base, uint64_t C, uint64_t W, uint64_t H, uint64_t N,
                                   uint32_t box_c, uint32_t box_w, uint32_t box_h);
relay_status_t make_tmap_2d(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                            uint32_t box_inner, uint32_t box_outer, bool swizzle128);
relay_status_t make_tmap_2d_sw64(CUtensorMap *m, bool f32, const void *base, uint64_t inner, uint64_t outer, uint64_t row_stride,
                                 uint32_t box_outer);

namespace {

constexpr int BM = 128, BK = 64;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;

// ---------------------------------------------------------------------------------------------------
// layout kernels
// ---------------------------------------------------------------------------------------------------
// out[n][hw][c] = in[n][c][hw]  (GRAD: in = dy, multiplied by act'(y) on the way: dZ in NHWC).
// 64 channels x 64 pixels per block, 16-byte global accesses on both sides (HW % 8 == 0, C % 8 == 0).
// GRAD with db_part != null also writes, per block, the sums over its 64 pixels of the stored (rounded) dZ
// of each of its 64 channels to db_part[(n * gridDim.x + blockIdx.x) * C + c]: the bias gradient's partials.
// Weight packing that rides along with a repack launch: the z-slices of the grid beyond `n_img` pack the weights
// (one output element per thread, as pack_weights_kernel below), so the 1 MB job costs no launch of its own.
struct PackJob {
    const __nv_bfloat16 *w;    // null: nothing to pack
    __nv_bfloat16 *wf, *wb;    // wf[o][tap][c], wb[c][mirror(tap)][o]; either may be null
    int O, C, taps, n_img;
};

__device__ __forceinline__ void pack_one(const PackJob &j, unsigned i)
{
    const unsigned taps = j.taps, total = (unsigned)j.O * j.C * taps;
    if (i >= total) return;
    if (j.wf) {
        const unsigned c = i % j.C, t = i / j.C, tap = t % taps, o = t / taps;
        j.wf[i] = j.w[(o * j.C + c) * taps + tap];
    }
    if (j.wb) {
        const unsigned o = i % j.O, t = i / j.O, tap2 = t % taps, c = t / taps;
        j.wb[i] = j.w[(o * j.C + c) * taps + (taps - 1 - tap2)];
    }
}

// Transposition tile of the repack kernels: 64 pixels x 64 channels as [pixel][channel pair] 32-bit words, 33 words per row.
// A thread arrives with 16 bytes = 8 pixels (chunk * 8 ..) of channel `cl`; the lane 8 further on holds the same pixels of
// channel cl ^ 1.  The two exchange half of their words, so that each ends up with four (even channel, odd channel) words
// -- the even-channel lane for the chunk's first four pixels, the odd-channel lane for the last four -- and stores 4 words
// instead of 8 half-words.  Column index XOR 2 for the upper half of the pixels: with it the 32 lanes of a store hit 32
// different banks (without it pixels 32 apart collide), and the reader undoes it by swapping the halves of its 16 bytes.
// Every lane of the warp must call tile_put together.
__device__ __forceinline__ void tile_put(uint32_t (*tile)[33], int cl, int chunk, const uint4 &val)
{
    const bool odd = cl & 1;
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, odd ? val.x : val.z, 8);
    const uint32_t r1 = __shfl_xor_sync(0xffffffffu, odd ? val.y : val.w, 8);
    const uint32_t e0 = odd ? r0 : val.x, e1 = odd ? r1 : val.y;      // even channel's two words (pixels 0,1 | 2,3 of this lane's four)
    const uint32_t o0 = odd ? val.z : r0, o1 = odd ? val.w : r1;      // odd channel's
    const int px = chunk * 8 + (odd ? 4 : 0), col = (cl >> 1) ^ ((chunk >> 2) << 1);
    tile[px + 0][col] = __byte_perm(e0, o0, 0x5410);
    tile[px + 1][col] = __byte_perm(e0, o0, 0x7632);
    tile[px + 2][col] = __byte_perm(e1, o1, 0x5410);
    tile[px + 3][col] = __byte_perm(e1, o1, 0x7632);
}
// the 8 channels cchunk * 8 .. of pixel pl
__device__ __forceinline__ uint4 tile_get(const uint32_t (*tile)[33], int pl, int cchunk)
{
    const uint32_t *row = &tile[pl][cchunk * 4];
    const uint32_t a = row[0], b = row[1], c = row[2], d = row[3];
    return (pl & 32) ? make_uint4(c, d, a, b) : make_uint4(a, b, c, d);
}

// NT: channel blocks of 64 that one thread block repacks; the loads of all of them are in flight before the first is
// transposed (16 * NT KB per block with GRAD, 8 * NT KB without).
template <bool GRAD, int NT>
__global__ void __launch_bounds__(256) nchw_to_nhwc_kernel(const __nv_bfloat16 *__restrict__ in, const __nv_bfloat16 *__restrict__ y,
                                                            __nv_bfloat16 *__restrict__ out, int C, int HW, int act,
                                                            float *__restrict__ db_part, const PackJob job)
{
    if (job.w != nullptr && (int)blockIdx.z >= job.n_img) {        // whole blocks: no barrier is skipped by part of a block
        pdl_wait();
        const unsigned blk = (((unsigned)blockIdx.z - job.n_img) * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
        pack_one(job, blk * 256u + threadIdx.x);
        return;
    }
    __shared__ uint32_t tile[NT][64][33];
    const int n = blockIdx.z, cb = blockIdx.y * (64 * NT), p0 = blockIdx.x * 64;
    const size_t img = (size_t)n * C * HW;
    pdl_wait();
    uint4 v[NT][2], yy[GRAD ? NT : 1][2];
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int idx = threadIdx.x + i * 256;
            const int cl = idx >> 3, chunk = idx & 7;
            const int c = cb + t * 64 + cl, p = p0 + chunk * 8;
            v[t][i] = make_uint4(0, 0, 0, 0);
            if (GRAD) yy[GRAD ? t : 0][i] = make_uint4(0, 0, 0, 0);
            if (c < C && p < HW) {
                const size_t off = img + (size_t)c * HW + p;
                v[t][i] = ld_stream(in + off);
                if (GRAD) yy[GRAD ? t : 0][i] = ld_stream(y + off);
            }
        }
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int idx = threadIdx.x + i * 256;
            const int cl = idx >> 3, chunk = idx & 7;
            const int c = cb + t * 64 + cl;
            uint4 val = v[t][i];
            if (GRAD) {
                float a[8], b[8];
                unpack(val, a);
                unpack(yy[GRAD ? t : 0][i], b);
#pragma unroll
                for (int j = 0; j < 8; ++j) a[j] *= act_grad_from_output(b[j], act);
                val = pack(a);
            }
            tile_put(tile[t], cl, chunk, val);
            if (GRAD && db_part != nullptr) {          // the 8 lanes that share a channel row combine in a fixed order
                float r[8];
                unpack(val, r);
                float sum = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                if (chunk == 0 && c < C) db_part[((size_t)n * gridDim.x + blockIdx.x) * C + c] = sum;
            }
        }
    __syncthreads();
    // 8 * NT lanes write the 128 * NT contiguous bytes of one pixel
#pragma unroll
    for (int i = 0; i < 2 * NT; ++i) {
        const int idx = threadIdx.x + i * 256;
        const int pl = idx / (8 * NT), cchunk = idx % (8 * NT), t = cchunk >> 3;
        const int c = cb + cchunk * 8, p = p0 + pl;
        if (c < C && p < HW) *reinterpret_cast<uint4 *>(out + ((size_t)n * HW + p) * C + c) = tile_get(tile[t], pl, cchunk & 7);
    }
}

// ---------------------------------------------------------------------------------------------------
// The same repack as a PERSISTENT kernel that runs beside the tensor-core kernel which consumes it.  Two blocks per SM
// (little shared memory, and at most a third of the registers, so that the consumer's one large block per SM still fits) walk a list of units: first the
// weight-packing units, then (image, 64-pixel block) units of up to two activation tensors, image by image.  A unit's
// loads for four channel blocks are all in flight before the first is transposed, so two blocks per SM keep enough
// bytes in flight.  Finished units are counted with release semantics: flags[0] counts packing units, flags[1 + n] the
// units of image n of the FIRST tensor; the consumer (launched behind this kernel with programmatic stream
// serialisation, and therefore started once every block here is resident and past its own wait for the stream's
// earlier work) polls them before it loads a tile.  This kernel never waits for the consumer.
struct RepackJob {
    const __nv_bfloat16 *in, *y;   // y: saved forward output (grad != 0: out = in * act'(y))
    __nv_bfloat16 *out;
    float *db_part;                // grad: per-unit sums over the 64 pixels, [n][pixel block][C], or null
    int C, grad, act, flagged;
};
struct RepackStream {
    RepackJob job[2];
    int n_jobs, Nb, HW, pbx;       // pbx: 64-pixel blocks per image
    PackJob pack;
    int pack_units;                // units of kPackPerUnit weight elements
    unsigned int *flags;
};
constexpr int kPackPerUnit = 4096;

template <bool GRAD>
__device__ __forceinline__ void repack_unit(const RepackJob &j, int HW, int pbx, int n, int pb, uint32_t (*tile)[33])
{
    // channel blocks whose loads are in flight together: 8 loads of 16 bytes per thread either way
    constexpr int NT = GRAD ? 2 : 4;
    const int p0 = pb * 64, tid = threadIdx.x;
    const size_t img = (size_t)n * j.C * HW;
    for (int cg = 0; cg < j.C; cg += 64 * NT) {
        uint4 v[NT][2], yy[GRAD ? NT : 1][2];
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int idx = tid + i * 256, cl = idx >> 3, chunk = idx & 7;
                const int c = cg + t * 64 + cl, p = p0 + chunk * 8;
                v[t][i] = make_uint4(0, 0, 0, 0);
                if (GRAD) yy[t][i] = make_uint4(0, 0, 0, 0);
                if (c < j.C && p < HW) {
                    const size_t off = img + (size_t)c * HW + p;
                    v[t][i] = ld_stream(j.in + off);
                    if (GRAD) yy[t][i] = ld_stream(j.y + off);
                }
            }
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            const int c0 = cg + t * 64;
            if (c0 >= j.C) break;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int idx = tid + i * 256, cl = idx >> 3, chunk = idx & 7;
                uint4 val = v[t][i];
                if (GRAD) {
                    float a[8], b[8];
                    unpack(val, a);
                    unpack(yy[GRAD ? t : 0][i], b);
#pragma unroll
                    for (int q = 0; q < 8; ++q) a[q] *= act_grad_from_output(b[q], j.act);
                    val = pack(a);
                }
                tile_put(tile, cl, chunk, val);
                if (GRAD && j.db_part != nullptr) {      // the 8 lanes that share a channel row combine in a fixed order
                    float r[8];
                    unpack(val, r);
                    float sum = ((r[0] + r[1]) + (r[2] + r[3])) + ((r[4] + r[5]) + (r[6] + r[7]));
                    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
                    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
                    if (chunk == 0 && c0 + cl < j.C) j.db_part[((size_t)n * pbx + pb) * j.C + c0 + cl] = sum;
                }
            }
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int idx = tid + i * 256, pl = idx >> 3, cchunk = idx & 7;
                const int c = c0 + cchunk * 8, p = p0 + pl;
                if (c < j.C && p < HW) *reinterpret_cast<uint4 *>(j.out + ((size_t)n * HW + p) * j.C + c) = tile_get(tile, pl, cchunk);
            }
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(256, 3) repack_stream_kernel(const RepackStream S)
{
    __shared__ uint32_t tile[64][33];
    // first the stream's earlier work must be complete (this kernel overwrites scratch that it may still read); only
    // then may the consumer start: whatever it reads that this kernel does not produce is then final as well
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int act_units = S.Nb * S.pbx, total = S.pack_units + S.n_jobs * act_units;
    for (int u = blockIdx.x; u < total; u += gridDim.x) {
        unsigned int *flag = nullptr;
        if (u < S.pack_units) {
#pragma unroll 1
            for (int k = 0; k < kPackPerUnit / 256; ++k) pack_one(S.pack, (unsigned)u * kPackPerUnit + k * 256 + threadIdx.x);
            flag = S.flags;
        } else {
            const int v = u - S.pack_units, ji = v / act_units, w = v - ji * act_units, n = w / S.pbx, pb = w - n * S.pbx;
            const RepackJob &j = S.job[ji];
            if (j.grad) repack_unit<true>(j, S.HW, S.pbx, n, pb, tile);
            else repack_unit<false>(j, S.HW, S.pbx, n, pb, tile);
            if (j.flagged) flag = S.flags + 1 + n;
        }
        if (flag != nullptr) {             // block-uniform
            tc::fence_proxy_async_global();   // the consumer reads these stores through TMA
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) tc::red_release_add_u32(flag, 1u);
        }
    }
}

// wf[o][tap][c] = w[o][c][tap];   wb[c][mirror(tap)][o] = w[o][c][tap]   (either may be null); one thread
// per OUTPUT element so that the stores coalesce (the 1 MB source stays in L2)
__global__ void pack_weights_kernel(const __nv_bfloat16 *__restrict__ w, __nv_bfloat16 *__restrict__ wf,
                                    __nv_bfloat16 *__restrict__ wb, int O, int C, int R, int S)
{
    const unsigned taps = R * S, total = (unsigned)O * C * taps;     // < 2^31 (checked by the plan)
    pdl_wait();
    for (unsigned i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        if (wf) {
            const unsigned c = i % C, t = i / C, tap = t % taps, o = t / taps;
            wf[i] = w[(o * C + c) * taps + tap];
        }
        if (wb) {
            const unsigned o = i % O, t = i / O, tap2 = t % taps, c = t / taps;
            wb[i] = w[(o * C + c) * taps + (taps - 1 - tap2)];
        }
    }
}

// dw[o][c][tap] = bf16( sum over slices, in slice order, of part[slice][tap][o][c] ); one thread per (o, c) adds up all
// its taps: the partial reads coalesce over (o, c) for every tap, and a warp's stores cover one contiguous run of
// 32 * taps output elements
__global__ void wgrad_reduce_kernel(const float *__restrict__ part, int n_slices, __nv_bfloat16 *__restrict__ dw, int O, int C, int taps)
{
    const unsigned oc_total = (unsigned)O * C;
    const size_t total = (size_t)oc_total * taps;
    pdl_wait();
    for (unsigned oc = blockIdx.x * blockDim.x + threadIdx.x; oc < oc_total; oc += gridDim.x * blockDim.x) {
        for (int tap = 0; tap < taps; ++tap) {
            float s = 0.0f;
            for (int j = 0; j < n_slices; ++j) s += part[(size_t)j * total + (size_t)tap * oc_total + oc];
            dw[(size_t)oc * taps + tap] = __float2bfloat16_rn(s);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// fprop kernel.  Work items are output tiles of (rows_per_tile * W) pixels by 128 * mh output channels:
//   MH = 1: every item is 128 channels wide; the two TMEM accumulators alternate between items, so the
//           epilogue of one item overlaps the main loop of the next;
//   MH = 2: "pairs" (256 channels: two MMAs per k-step share the activation tile in shared memory, a third
//           fewer bytes per FLOP) fill whole rounds over the SMs, and what is left runs as single
//           128-channel items so that the last round is half as long.  One accumulator per half, each
//           drained by its own four epilogue warps.
// The epilogue goes through a staging buffer and TMA tile stores into the NCHW output viewed as a 2-D
// tensor [Nb * Cout rows][H * W columns] (the pixels of consecutive image rows are contiguous there).
// ---------------------------------------------------------------------------------------------------
struct FpropParams {
    int Cin, Cout, H, W, Nb, taps_r, taps_s, pad;
    int rows_per_tile, nt;      // nt = rows_per_tile * W = UMMA N
    int tiles_per_img, n_tiles_total, k_blocks, stages;
    int n_pairs, pairs_per_ntile, n_items;   // items [0, n_pairs) are pairs, the rest singles (MH = 2); MH = 1: all singles
    const unsigned int *flags;  // two-SM kernel running beside the repack that feeds it (else null): flags[0] counts packed weight
    int pack_units, units_per_img;   // units, flags[1 + n] the repacked units of image n; a tile is loaded once both are complete
    int n_full;                 // two-SM kernel: items [0, n_full) are whole tiles, items beyond are HALF tiles (rows_per_tile / 2 rows)
    const void *bias;           // per output channel, or null
    int bias_bf16, act;
    int out_nhwc;               // two-SM kernel: the output tensor map is [Nb*H*W pixels][Cout], tiles are stored pixel-major
    int *err;
};

struct FpropItem { int m0, mh, img, h0; };

template <int MH>
__device__ __forceinline__ FpropItem fprop_item(const FpropParams &p, int item)
{
    FpropItem it;
    int nt_idx;
    if (MH == 2 && item < p.n_pairs) {
        it.mh = 2;
        it.m0 = (item % p.pairs_per_ntile) * 256;
        nt_idx = item / p.pairs_per_ntile;
    } else {
        const int singles_per_ntile = p.Cout / BM;
        const int j = item - (MH == 2 ? p.n_pairs : 0);
        const int base = MH == 2 ? p.n_pairs / p.pairs_per_ntile : 0;
        it.mh = 1;
        it.m0 = (j % singles_per_ntile) * BM;
        nt_idx = base + j / singles_per_ntile;
    }
    it.img = nt_idx / p.tiles_per_img;
    it.h0 = (nt_idx % p.tiles_per_img) * p.rows_per_tile;
    return it;
}

template <int MH>
__global__ void __launch_bounds__(64 + 128 * MH, 1)
conv_fprop_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                     const __grid_constant__ CUtensorMap tm_y, const FpropParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int a_bytes = MH * BM * BK * 2;
    const int b_bytes = p.nt * BK * 2;
    const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
    const int STAGES = p.stages;
    uint8_t *staging = smem + (size_t)STAGES * stage_bytes;                 // [epilogue warp][2][2 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + 4 * MH * 4096);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES, *tmem_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const int cblocks = p.Cin / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&tmem_full[b], 1); tc::mbar_init(&tmem_empty[b], 4); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_w);
        tc::prefetch_tmap(&tm_x);
        tc::prefetch_tmap(&tm_y);
    }
    if (warp == 1) { tc::tmem_alloc(tmem_slot, TMEM_COLS); tc::tmem_relinquish(); }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x) {
                const FpropItem wi = fprop_item<MH>(p, item);
                const uint32_t tx = wi.mh * (BM * BK * 2) + b_bytes;
                int kb = 0;
                for (int r = 0; r < p.taps_r && ok; ++r)
                    for (int sft = 0; sft < p.taps_s && ok; ++sft)
                        for (int cb = 0; cb < cblocks; ++cb, ++kb) {
                            if (!tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY)) { ok = false; break; }
                            uint8_t *sa = smem + (size_t)s * stage_bytes, *sb = sa + a_bytes;
                            tc::mbar_expect_tx(&full[s], tx);
                            tc::tma_load_2d(sa, &tm_w, &full[s], kb * BK, wi.m0);
                            if (MH == 2 && wi.mh == 2) tc::tma_load_2d(sa + BM * BK * 2, &tm_w, &full[s], kb * BK, wi.m0 + BM);
                            tc::tma_load_4d(sb, &tm_x, &full[s], cb * BK, sft - p.pad, wi.h0 + r - p.pad, wi.img);
                            if (++s == STAGES) { s = 0; phase ^= 1; }
                        }
            }
        }
    } else if (warp == 1) {
        {   // warp-uniform issue loop, an elected lane issues
            const uint32_t idesc = tc::instr_desc_bf16(BM, p.nt, false, false);
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(smem), 16, 1024), desc_b0 = tc::smem_desc(tc::smem_u32(smem) + a_bytes, 16, 1024);
            uint32_t t_local = 0, phase = 0, stage_off = 0;   // stage_off = s * stage_bytes in 16-byte units
            int s = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.n_items && ok; item += gridDim.x, ++t_local) {
                const FpropItem wi = fprop_item<MH>(p, item);
                const int buf = MH == 1 ? (t_local & 1) : 0;
                const uint32_t empty_parity = MH == 1 ? (((t_local >> 1) & 1) ^ 1) : ((t_local & 1) ^ 1);
                if (!__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[buf], empty_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                if (MH == 2 && !__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[1], empty_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    // descriptors differ from the stage-0 ones only in the start address field (16-byte units),
                    // so the issuing thread spends one add per MMA instead of rebuilding them
                    const uint64_t da = desc_a0 + stage_off, db = desc_b0 + stage_off;
                    const uint32_t acc = kb != 0;
                    if (MH == 2 && wi.mh == 2) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            tc::mma_bf16_elect(d_tmem, da + kk * 2, db + kk * 2, idesc, acc | (kk != 0));
                            tc::mma_bf16_elect(d_tmem + 256, da + (BM * BK * 2 >> 4) + kk * 2, db + kk * 2, idesc, acc | (kk != 0));
                        }
                    } else {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) tc::mma_bf16_elect(d_tmem, da + kk * 2, db + kk * 2, idesc, acc | (kk != 0));
                    }
                    tc::mma_commit_elect(&empty[s]);
                    stage_off += (uint32_t)stage_bytes >> 4;
                    if (++s == STAGES) { s = 0; phase ^= 1; stage_off = 0; }
                }
                if (ok) tc::mma_commit_elect(&tmem_full[buf]);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;                  // MH = 2: which accumulator this warp drains
        uint8_t *my_stage = staging + (size_t)(warp - 2) * 4096;
        uint32_t t_local = 0, blk_count = 0;
        for (int item = blockIdx.x; item < p.n_items; item += gridDim.x, ++t_local) {
            const FpropItem wi = fprop_item<MH>(p, item);
            const int buf = MH == 1 ? (t_local & 1) : half;
            const int fbar = MH == 1 ? (t_local & 1) : 0;
            const uint32_t full_parity = MH == 1 ? ((t_local >> 1) & 1) : (t_local & 1);
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[fbar], full_parity, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc::tc_fence_after_sync();
            if (half < wi.mh) {                            // a single item leaves the second accumulator unused
                const int o0 = wi.m0 + half * BM + quarter * 32;   // this warp's 32 output channels; lane = channel
                const int o = o0 + lane;
                float bias = 0.0f;
                if (p.bias != nullptr && o < p.Cout)
                    bias = p.bias_bf16 ? __bfloat162float(((const __nv_bfloat16 *)p.bias)[o]) : ((const float *)p.bias)[o];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 256;
#pragma unroll 1
                for (int c = 0; c < p.nt / 32; ++c, ++blk_count) {
                    uint32_t r[32];
                    tc::tmem_ld_32x32(taddr + c * 32, r);
                    tc::tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) + bias;
                    switch (p.act) {
                    case RELAY_ACT_RELU:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
                        break;
                    case RELAY_ACT_TANH:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = tanh_<true>(v[j]);
                        break;
                    case RELAY_ACT_SIGMOID:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = sigmoid_<true>(v[j]);
                        break;
                    default: break;
                    }
                    // 32 channels x 32 pixels (64 bytes per row) -> staging (2 buffers of 2 KB) -> TMA tile store
                    uint8_t *st = my_stage + (blk_count & 1) * 2048;
                    if (lane == 0) tc::tma_store_wait_read<1>();
                    __syncwarp();
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        *reinterpret_cast<uint4 *>(st + lane * 64 + q * 16) =
                            make_uint4(pack2(v[8 * q], v[8 * q + 1]), pack2(v[8 * q + 2], v[8 * q + 3]), pack2(v[8 * q + 4], v[8 * q + 5]),
                                       pack2(v[8 * q + 6], v[8 * q + 7]));
                    tc::fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tc::tma_store_2d(&tm_y, st, wi.h0 * p.W + c * 32, wi.img * p.Cout + o0);
                        tc::tma_store_commit();
                    }
                }
            }
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&tmem_empty[buf]);
        }
        if (lane == 0) tc::tma_store_wait_all<0>();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after_sync(); tc::tmem_dealloc(tmem_base, TMEM_COLS); }
}

// ---------------------------------------------------------------------------------------------------
// fprop kernel, two-SM form: a pair of blocks computes 256 output channels x (rows_per_tile * W) pixels
// with tcgen05.mma.cta_group::2.  Each block loads the packed weights of its 128 channels and HALF of the
// activation tile (rows_per_tile / 2 image rows), 30 KB per k-block at cfg4, so six stages fit and the two
// TMEM accumulators alternate between tiles (the epilogue overlaps the next main loop).
// ---------------------------------------------------------------------------------------------------
// Work items of the two-SM kernel.  Whole rounds over the SM pairs are made of whole tiles; the tiles that would start
// one more, mostly empty round are cut into two half tiles each (half as many image rows, N halved), so that this last
// round is about half as long and twice as many pairs share it.
struct PairItem { int m0, img, h0, rows; bool half; };
__device__ __forceinline__ PairItem pair_item(const FpropParams &p, int item)
{
    PairItem it;
    int t = item, sub = 0;
    it.half = item >= p.n_full;
    if (it.half) { const int j = item - p.n_full; t = p.n_full + (j >> 1); sub = j & 1; }
    const int nt_idx = t / p.pairs_per_ntile;
    it.m0 = (t % p.pairs_per_ntile) * 256;
    it.rows = it.half ? p.rows_per_tile >> 1 : p.rows_per_tile;
    it.img = nt_idx / p.tiles_per_img;
    it.h0 = (nt_idx % p.tiles_per_img) * p.rows_per_tile + sub * it.rows;
    return it;
}

// tm_xh: activation boxes of rows_per_tile / 2 image rows (a block's half of a whole tile); tm_xq: of rows_per_tile / 4 rows (its
// half of a half tile); tm_y: 32-pixel x 32-channel output boxes; tm_yt: 16-pixel boxes, unswizzled, for the half tiles
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
conv_fprop_tc2_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                      const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ CUtensorMap tm_xq,
                      const __grid_constant__ CUtensorMap tm_yt, const FpropParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int a_bytes = BM * BK * 2;
    const int bh_bytes = (p.nt / 2) * BK * 2;                       // this block's half of the activation tile
    const int stage_bytes = a_bytes + ((bh_bytes + 1023) & ~1023);
    const int STAGES = p.stages;
    uint8_t *staging = smem + (size_t)STAGES * stage_bytes;         // [epilogue warp][2][2 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + 4 * 4096);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES, *tmem_empty = bars + 2 * STAGES + 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 4);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const uint32_t rank = tc::cluster_ctarank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int cblocks = p.Cin / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { tc::mbar_init(&tmem_full[b], 1); tc::mbar_init(&tmem_empty[b], 8); }
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_w);
        tc::prefetch_tmap(&tm_x);
        tc::prefetch_tmap(&tm_y);
        tc::prefetch_tmap(&tm_xq);
        tc::prefetch_tmap(&tm_yt);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    // Beside a repack kernel (p.flags): that kernel has already waited for the stream's earlier work, and what it
    // produces is handed over through its counters, so this kernel starts at once and waits for the repack kernel's
    // completion only at its very end (completion of this kernel then still implies completion of all earlier ones).
    if (p.flags != nullptr) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    else pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        {   // warp-uniform loop, an elected lane issues the copies
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            // bounded poll of one of the repack kernel's counters (lane 0 polls, the warp follows)
            auto wait_count = [&](const unsigned int *counter, unsigned int target) -> bool {
                int good = 1;
                if (lane == 0) {
                    const long long t0 = clock64();
                    unsigned spins = 0;
                    while (tc::ld_acquire_u32(counter) < target) {
                        __nanosleep(100);
                        if ((++spins & 255u) == 0 && (*abort_flag || clock64() - t0 > tc::kWaitLimitCycles)) {
                            if (!*abort_flag) { *abort_flag = 1; atomicCAS(p.err, 0, tc::ERR_WAIT_STEP); }
                            good = 0;
                            break;
                        }
                    }
                }
                __syncwarp();                                  // lane 0's acquire is ordered before the other lanes' accesses
                good = __shfl_sync(0xffffffffu, good, 0);
                tc::fence_proxy_async_global();                // every lane: whichever lane is elected issues the copies
                return good != 0;
            };
            int ready_img = -1;
            if (p.flags != nullptr) ok = wait_count(p.flags, (unsigned)p.pack_units);
            for (int item = pair; item < p.n_items && ok; item += n_pairs) {
                const PairItem it = pair_item(p, item);
                if (p.flags != nullptr && it.img != ready_img) {
                    ok = wait_count(p.flags + 1 + it.img, (unsigned)p.units_per_img);
                    if (!ok) break;
                    ready_img = it.img;
                }
                const int m0 = it.m0 + (int)rank * BM;
                const int rows_cta = it.rows >> 1;                       // this block's image rows of the tile
                const int img = it.img, h0 = it.h0 + (int)rank * rows_cta;
                const uint32_t tx_bytes = 2u * (uint32_t)(a_bytes + rows_cta * p.W * 128);
                const CUtensorMap *mx = it.half ? &tm_xq : &tm_x;
                int kb = 0;
                for (int r = 0; r < p.taps_r && ok; ++r)
                    for (int sft = 0; sft < p.taps_s && ok; ++sft)
                        for (int cb = 0; cb < cblocks; ++cb, ++kb) {
                            ok = __all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY));
                            if (!ok) break;
                            uint8_t *sa = smem + (size_t)s * stage_bytes, *sb = sa + a_bytes;
                            const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);
                            if (tc::elect_one()) {
                                if (rank == 0) tc::mbar_expect_tx_cluster(bar, tx_bytes);
                                tc::tma_load_2d_pair(sa, &tm_w, bar, kb * BK, m0);
                                tc::tma_load_4d_pair(sb, mx, bar, cb * BK, sft - p.pad, h0 + r - p.pad, img);
                            }
                            __syncwarp();
                            if (++s == STAGES) { s = 0; phase ^= 1; }
                        }
            }
        }
    } else if (warp == 1) {
        // the whole warp runs the issue loop with warp-uniform values, an elected lane issues (descriptors stay in
        // uniform registers: an MMA costs the issuing warp far fewer cycles than from one divergent lane)
        if (rank == 0) {
            const uint32_t idesc_full = tc::instr_desc_bf16(256, p.nt, false, false), idesc_half = tc::instr_desc_bf16(256, p.nt >> 1, false, false);
            const uint64_t desc_a0 = tc::smem_desc(tc::smem_u32(smem), 16, 1024), desc_b0 = tc::smem_desc(tc::smem_u32(smem) + a_bytes, 16, 1024);
            uint32_t t_local = 0, phase = 0, stage_off = 0;
            int s = 0;
            bool ok = true;
            for (int item = pair; item < p.n_items && ok; item += n_pairs, ++t_local) {
                const int buf = t_local & 1;
                const uint32_t idesc = item >= p.n_full ? idesc_half : idesc_full;
                if (!__all_sync(0xffffffffu, tc::mbar_wait(&tmem_empty[buf], ((t_local >> 1) & 1) ^ 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_EMPTY))) break;
                tc::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                    if (!ok) break;
                    tc::tc_fence_after_sync();
                    const uint64_t da = desc_a0 + stage_off, db = desc_b0 + stage_off;
                    const uint32_t acc = kb != 0;
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk) tc::mma_bf16_pair_elect(d_tmem, da + kk * 2, db + kk * 2, idesc, acc | (kk != 0));
                    tc::mma_commit_pair_elect(&empty[s]);
                    stage_off += (uint32_t)stage_bytes >> 4;
                    if (++s == STAGES) { s = 0; phase ^= 1; stage_off = 0; }
                }
                if (ok) tc::mma_commit_pair_elect(&tmem_full[buf]);
            }
        }
    } else {
        const int quarter = warp & 3;
        uint8_t *my_stage = staging + (size_t)(warp - 2) * 4096;
        uint32_t t_local = 0, blk_count = 0;
        for (int item = pair; item < p.n_items; item += n_pairs, ++t_local) {
            const int buf = t_local & 1;
            const PairItem it = pair_item(p, item);
            const int m0 = it.m0 + (int)rank * BM;
            const int img = it.img, h0 = it.h0;
            int ok = 1;
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[buf], (t_local >> 1) & 1, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc::tc_fence_after_sync();
            const int o0 = m0 + quarter * 32;
            const int o = o0 + lane;
            float bias = 0.0f;
            if (p.bias != nullptr && o < p.Cout)
                bias = p.bias_bf16 ? __bfloat162float(((const __nv_bfloat16 *)p.bias)[o]) : ((const float *)p.bias)[o];
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * 256;
            if (!it.half) {
#pragma unroll 1
                for (int c = 0; c < p.nt / 32; ++c, ++blk_count) {
                    uint32_t r[32];
                    tc::tmem_ld_32x32(taddr + c * 32, r);
                    tc::tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) + bias;
                    switch (p.act) {
                    case RELAY_ACT_RELU:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
                        break;
                    case RELAY_ACT_TANH:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = tanh_<true>(v[j]);
                        break;
                    case RELAY_ACT_SIGMOID:
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = sigmoid_<true>(v[j]);
                        break;
                    default: break;
                    }
                    uint8_t *st = my_stage + (blk_count & 1) * 2048;
                    if (tc::elect_one()) tc::tma_store_wait_read<1>();   // always the same lane of the warp
                    __syncwarp();
                    // 32 rows x 64 bytes in the 64-byte swizzle pattern of the output tensor map (16-byte piece q of row r at
                    // piece q ^ ((r >> 1) & 3)): conflict-free stores
                    if (p.out_nhwc) {
                        // pixel-major block: row j = pixel j, this lane's channel is element `lane` of the row (the 32 lanes of
                        // a store fill one 64-byte row, so the 2-byte stores are conflict-free as well)
                        uint8_t *col = st + ((lane & 7) << 1);
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            *reinterpret_cast<__nv_bfloat16 *>(col + j * 64 + (((lane >> 3) ^ ((j >> 1) & 3)) << 4)) = __float2bfloat16_rn(v[j]);
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            *reinterpret_cast<uint4 *>(st + lane * 64 + ((q ^ ((lane >> 1) & 3)) << 4)) =
                                make_uint4(pack2(v[8 * q], v[8 * q + 1]), pack2(v[8 * q + 2], v[8 * q + 3]), pack2(v[8 * q + 4], v[8 * q + 5]),
                                           pack2(v[8 * q + 6], v[8 * q + 7]));
                    }
                    tc::fence_proxy_async();
                    __syncwarp();
                    if (tc::elect_one()) {
                        if (p.out_nhwc) tc::tma_store_2d(&tm_y, st, o0, (img * p.H + h0) * p.W + c * 32);
                        else tc::tma_store_2d(&tm_y, st, h0 * p.W + c * 32, img * p.Cout + o0);
                        tc::tma_store_commit();
                    }
                }
            } else {
                // half tile: nt / 2 pixels in chunks of 16 (nt / 2 is a multiple of 16, not always of 32); unswizzled staging:
                // NCHW 32 channel rows of 32 bytes, NHWC 16 pixel rows of 64 bytes
#pragma unroll 1
                for (int c = 0; c < (p.nt >> 1) / 16; ++c, ++blk_count) {
                    uint32_t r[16];
                    tc::tmem_ld_32x16(taddr + c * 16, r);
                    tc::tmem_ld_wait();
                    float v[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = act_fwd<true>(__uint_as_float(r[j]) + bias, p.act);
                    uint8_t *st = my_stage + (blk_count & 1) * 2048;
                    if (tc::elect_one()) tc::tma_store_wait_read<1>();
                    __syncwarp();
                    if (p.out_nhwc) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) *reinterpret_cast<__nv_bfloat16 *>(st + j * 64 + lane * 2) = __float2bfloat16_rn(v[j]);
                    } else {
#pragma unroll
                        for (int q = 0; q < 2; ++q)
                            *reinterpret_cast<uint4 *>(st + lane * 32 + q * 16) =
                                make_uint4(pack2(v[8 * q], v[8 * q + 1]), pack2(v[8 * q + 2], v[8 * q + 3]), pack2(v[8 * q + 4], v[8 * q + 5]),
                                           pack2(v[8 * q + 6], v[8 * q + 7]));
                    }
                    tc::fence_proxy_async();
                    __syncwarp();
                    if (tc::elect_one()) {
                        if (p.out_nhwc) tc::tma_store_2d(&tm_yt, st, o0, (img * p.H + h0) * p.W + c * 16);
                        else tc::tma_store_2d(&tm_yt, st, h0 * p.W + c * 16, img * p.Cout + o0);
                        tc::tma_store_commit();
                    }
                }
            }
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive_cluster(tc::mapa(tc::smem_u32(&tmem_empty[buf]), 0));
        }
        if (tc::elect_one()) tc::tma_store_wait_all<0>();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();
    if (warp == 1) {
        tc::tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
    if (p.flags != nullptr && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");   // see the start of the kernel
}

// ---------------------------------------------------------------------------------------------------
// wgrad kernel: one work unit = (tap, 128 output channels, NT input channels, batch slice)
// ---------------------------------------------------------------------------------------------------
struct WgradParams {
    int C, O, H, W, Nb, taps_r, taps_s, pad;
    int rows_per_kblock, kpix;           // kpix = rows_per_kblock * W pixels per k-block
    int nt;                              // input channels per unit (UMMA N)
    int m_tiles, c_tiles, n_slices, imgs_per_slice, stages;
    float *part;                         // [slice][tap][O][C]
    int *err;
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
conv_wgrad_tc_kernel(const __grid_constant__ CUtensorMap tm_dz, const __grid_constant__ CUtensorMap tm_x,
                     const __grid_constant__ CUtensorMap tm_part, const WgradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int box_bytes = p.kpix * 128;                 // 64 channels x kpix pixel rows
    const int a_bytes = (BM / 64) * box_bytes, b_bytes = (p.nt / 64) * box_bytes;
    const int stage_bytes = a_bytes + b_bytes;
    const int STAGES = p.stages;
    uint8_t *staging = smem + (size_t)STAGES * stage_bytes;           // [epilogue warp][2][4 KB]
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + 4 * 8192);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // decode the work unit of this block
    int u = blockIdx.x;
    const int slice = u % p.n_slices; u /= p.n_slices;
    const int ct = u % p.c_tiles; u /= p.c_tiles;
    const int mt = u % p.m_tiles; u /= p.m_tiles;
    const int tap = u;
    const int r = tap / p.taps_s, sft = tap % p.taps_s;
    const int img0 = slice * p.imgs_per_slice, img1 = min(p.Nb, img0 + p.imgs_per_slice);
    const int kb_per_img = p.H / p.rows_per_kblock;
    const int k_blocks = max(0, img1 - img0) * kb_per_img;
    const int o0 = mt * BM, c0 = ct * p.nt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        tc::mbar_init(&tmem_full[0], 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_dz);
        tc::prefetch_tmap(&tm_x);
    }
    if (warp == 1) { tc::tmem_alloc(tmem_slot, 256); tc::tmem_relinquish(); }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < k_blocks; ++kb) {
                const int s = kb % STAGES;
                if (!tc::mbar_wait(&empty[s], ((kb / STAGES) & 1) ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY)) break;
                uint8_t *sa = smem + (size_t)s * stage_bytes, *sb = sa + a_bytes;
                tc::mbar_expect_tx(&full[s], stage_bytes);
                const int img = img0 + kb / kb_per_img, h0 = (kb % kb_per_img) * p.rows_per_kblock;
                for (int i = 0; i < BM / 64; ++i) tc::tma_load_4d(sa + i * box_bytes, &tm_dz, &full[s], o0 + i * 64, 0, h0, img);
                for (int j = 0; j < p.nt / 64; ++j)
                    tc::tma_load_4d(sb + j * box_bytes, &tm_x, &full[s], c0 + j * 64, sft - p.pad, h0 + r - p.pad, img);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::instr_desc_bf16(BM, p.nt, true, true);
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                const int s = kb % STAGES;
                if (!tc::mbar_wait(&full[s], (kb / STAGES) & 1, abort_flag, p.err, tc::ERR_WAIT_FULL)) { ok = false; break; }
                tc::tc_fence_after_sync();
                const uint32_t sa = tc::smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
                const uint64_t da = tc::smem_desc(sa, box_bytes, 1024), db = tc::smem_desc(sb, box_bytes, 1024);
                const uint32_t acc = kb != 0;
                for (int kk = 0; kk < p.kpix / 16; ++kk) tc::mma_bf16(tmem_base, da + kk * 128, db + kk * 128, idesc, acc | (kk != 0));
                tc::mma_commit(&empty[s]);
            }
            if (ok) tc::mma_commit(&tmem_full[0]);
        }
    } else {
        const int quarter = warp & 3;
        int ok = 1;
        if (k_blocks > 0) {
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[0], 0, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
        }
        if (ok) {
            tc::tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            uint8_t *my_stage = staging + (size_t)(warp - 2) * 8192;
            const int row0 = (slice * (p.taps_r * p.taps_s) + tap) * p.O + o0 + quarter * 32;   // row of the [slice][tap][O] x [C] partial
#pragma unroll 1
            for (int c = 0; c < p.nt / 32; ++c) {
                uint32_t v[32];
                if (k_blocks > 0) {
                    tc::tmem_ld_32x32(taddr + c * 32, v);
                    tc::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                uint4 piece[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) piece[q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                tc::warp_store_block<1>(&tm_part, my_stage + (c & 1) * 4096, piece, lane, c0 + c * 32, row0);
            }
            if (lane == 0) tc::tma_store_wait_all<0>();
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) { tc::tc_fence_after_sync(); tc::tmem_dealloc(tmem_base, 256); }
}

// ---------------------------------------------------------------------------------------------------
// wgrad kernel, two-SM form: a pair of blocks owns (tap, 256 output channels, 256 input channels, batch
// slice).  Each block loads its 128 output channels of dZ and its 128 input channels of x per k-block
// (56 KB instead of 84 KB) and the pair's MMA (cta_group::2, M = 256) reads both halves.
// ---------------------------------------------------------------------------------------------------
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
conv_wgrad_tc2_kernel(const __grid_constant__ CUtensorMap tm_dz, const __grid_constant__ CUtensorMap tm_x,
                      const __grid_constant__ CUtensorMap tm_part, const WgradParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int box_bytes = p.kpix * 128;
    const int a_bytes = 2 * box_bytes, stage_bytes = 4 * box_bytes;      // 128 o + 128 c per block
    const int STAGES = p.stages;
    uint8_t *staging = smem + (size_t)STAGES * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(staging + 4 * 8192);
    uint64_t *full = bars, *empty = bars + STAGES, *tmem_full = bars + 2 * STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * STAGES + 2);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0), lane = threadIdx.x & 31;   // provably warp-uniform
    const uint32_t rank = tc::cluster_ctarank();

    int u = blockIdx.x >> 1;                           // unit of the pair
    const int slice = u % p.n_slices; u /= p.n_slices;
    const int ct = u % p.c_tiles; u /= p.c_tiles;
    const int mt = u % p.m_tiles; u /= p.m_tiles;      // m_tiles counts 256-channel tiles here
    const int tap = u;
    const int r = tap / p.taps_s, sft = tap % p.taps_s;
    const int img0 = slice * p.imgs_per_slice, img1 = min(p.Nb, img0 + p.imgs_per_slice);
    const int kb_per_img = p.H / p.rows_per_kblock;
    const int k_blocks = max(0, img1 - img0) * kb_per_img;
    const int o0 = mt * 256 + (int)rank * 128, c0 = ct * 256 + (int)rank * 128;   // this block's halves

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        tc::mbar_init(&tmem_full[0], 1);
        *abort_flag = 0;
        tc::fence_barrier_init();
        tc::prefetch_tmap(&tm_dz);
        tc::prefetch_tmap(&tm_x);
        tc::prefetch_tmap(&tm_part);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(256) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();   // set-up done; from here on the kernel touches global memory

    if (warp == 0) {
        {   // warp-uniform loop, an elected lane issues the copies
            int s = 0;
            uint32_t phase = 0;
            for (int kb = 0; kb < k_blocks; ++kb) {
                if (!__all_sync(0xffffffffu, tc::mbar_wait(&empty[s], phase ^ 1, abort_flag, p.err, tc::ERR_WAIT_EMPTY))) break;
                uint8_t *sa = smem + (size_t)s * stage_bytes, *sb = sa + a_bytes;
                const uint32_t bar = tc::mapa(tc::smem_u32(&full[s]), 0);
                const int img = img0 + kb / kb_per_img, h0 = (kb % kb_per_img) * p.rows_per_kblock;
                if (tc::elect_one()) {
                    if (rank == 0) tc::mbar_expect_tx_cluster(bar, 2 * stage_bytes);
#pragma unroll
                    for (int i = 0; i < 2; ++i) tc::tma_load_4d_pair(sa + i * box_bytes, &tm_dz, bar, o0 + i * 64, 0, h0, img);
#pragma unroll
                    for (int j = 0; j < 2; ++j) tc::tma_load_4d_pair(sb + j * box_bytes, &tm_x, bar, c0 + j * 64, sft - p.pad, h0 + r - p.pad, img);
                }
                __syncwarp();
                if (++s == STAGES) { s = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // warp-uniform issue loop, an elected lane issues
        if (rank == 0) {
            const uint32_t idesc = tc::instr_desc_bf16(256, 256, true, true);
            int s = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < k_blocks; ++kb) {
                ok = __all_sync(0xffffffffu, tc::mbar_wait(&full[s], phase, abort_flag, p.err, tc::ERR_WAIT_FULL));
                if (!ok) break;
                tc::tc_fence_after_sync();
                const uint32_t sa = tc::smem_u32(smem + (size_t)s * stage_bytes), sb = sa + a_bytes;
                const uint64_t da = tc::smem_desc(sa, box_bytes, 1024), db = tc::smem_desc(sb, box_bytes, 1024);
                const uint32_t acc = kb != 0;
                for (int kk = 0; kk < p.kpix / 16; ++kk) tc::mma_bf16_pair_elect(tmem_base, da + kk * 128, db + kk * 128, idesc, acc | (kk != 0));
                tc::mma_commit_pair_elect(&empty[s]);
                if (++s == STAGES) { s = 0; phase ^= 1; }
            }
            if (ok) tc::mma_commit_pair_elect(&tmem_full[0]);
        }
    } else {
        const int quarter = warp & 3;
        int ok = 1;
        if (k_blocks > 0) {
            if (lane == 0) ok = tc::mbar_wait(&tmem_full[0], 0, abort_flag, p.err, tc::ERR_WAIT_TMEM_FULL) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
        }
        if (ok) {
            tc::tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
            uint8_t *my_stage = staging + (size_t)(warp - 2) * 8192;
            const int row0 = (slice * (p.taps_r * p.taps_s) + tap) * p.O + o0 + quarter * 32;
            const int col0 = ct * 256;                  // the accumulator row holds all 256 input channels of the tile
#pragma unroll 1
            for (int c = 0; c < 256 / 32; ++c) {
                uint32_t v[32];
                if (k_blocks > 0) {
                    tc::tmem_ld_32x32(taddr + c * 32, v);
                    tc::tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = 0u;
                }
                uint4 piece[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) piece[q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
                tc::warp_store_block<1>(&tm_part, my_stage + (c & 1) * 4096, piece, lane, col0 + c * 32, row0);
            }
            if (lane == 0) tc::tma_store_wait_all<0>();
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::cluster_sync();
    if (warp == 1) {
        tc::tc_fence_after_sync();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------
// host plans
// ---------------------------------------------------------------------------------------------------
struct TcPlan {
    bool ok = false;
    int rows_per_tile = 0;   // fprop: image rows per tile (rows*W <= 256, multiple of 32)
    int rows_per_kblock = 0; // wgrad: image rows per k-block (rows*W multiple of 16, <= 128)
    int wg_nt = 0, wg_c_tiles = 0, wg_m_tiles = 0, wg_slices = 0, wg_imgs_per_slice = 0, wg_stages = 0;
    bool wg_pair = false;    // two-SM wgrad: units of 256 output x 256 input channels computed by pairs of blocks
    int fp_stages = 0;
    size_t x_nhwc = 0, dz_nhwc = 0, wpack = 0, part = 0, db_part = 0, flags = 0;
};

constexpr size_t kSmemLimit = 227 * 1024 - 2048;

TcPlan plan(const ConvDims &d)
{
    TcPlan pl;
    if (d.dt != RELAY_BF16 || d.stride != 1 || d.R != 3 || d.S != 3 || d.pad != 1) return pl;
    if (d.C % 128 || d.O % 128 || d.W % 8 || d.W > 256 || d.H < 1 || d.Nb < 1) return pl;
    if (d.Nb > 65535 || d.H * d.W > (1 << 24) || d.O * d.C * 9 >= (1ll << 31)) return pl;
    for (int rt = (int)std::min<int64_t>(d.H, 256 / d.W); rt >= 1; --rt)
        if (d.H % rt == 0 && (rt * d.W) % 32 == 0) { pl.rows_per_tile = rt; break; }
    for (int rk = (int)std::min<int64_t>(d.H, 128 / d.W); rk >= 1; --rk)
        if (d.H % rk == 0 && (rk * d.W) % 16 == 0) { pl.rows_per_kblock = rk; break; }
    if (!pl.rows_per_tile || !pl.rows_per_kblock) return pl;
    // fprop stages
    const size_t fp_stage = BM * BK * 2 + (((size_t)pl.rows_per_tile * d.W * BK * 2 + 1023) & ~size_t(1023));
    pl.fp_stages = (int)std::min<size_t>(6, (kSmemLimit - 1024) / fp_stage);
    if (pl.fp_stages < 2) return pl;
    // wgrad tiling
    pl.wg_nt = (int)std::min<int64_t>(256, d.C);
    const size_t box = (size_t)pl.rows_per_kblock * d.W * 128;
    auto wg_stage = [&](int nt) { return (size_t)(BM / 64 + nt / 64) * box; };
    constexpr size_t wg_fixed = 1024 + 4 * 8192;   // alignment slack + store staging
    while (pl.wg_nt > 64 && (kSmemLimit - wg_fixed) / wg_stage(pl.wg_nt) < 2) pl.wg_nt -= 64;
    if ((kSmemLimit - wg_fixed) / wg_stage(pl.wg_nt) < 2 || d.C % pl.wg_nt) return pl;
    pl.wg_stages = (int)std::min<size_t>(4, (kSmemLimit - wg_fixed) / wg_stage(pl.wg_nt));
    pl.wg_c_tiles = (int)(d.C / pl.wg_nt);
    pl.wg_m_tiles = (int)(d.O / BM);
    int workers = 148;
    const size_t pair_stage = 4 * box;
    if (d.O % 256 == 0 && d.C % 256 == 0 && (kSmemLimit - wg_fixed) / pair_stage >= 2) {
        pl.wg_pair = true;
        pl.wg_nt = 256;
        pl.wg_c_tiles = (int)(d.C / 256);
        pl.wg_m_tiles = (int)(d.O / 256);
        pl.wg_stages = (int)std::min<size_t>(4, (kSmemLimit - wg_fixed) / pair_stage);
        workers = 74;
    }
    const int base_units = 9 * pl.wg_m_tiles * pl.wg_c_tiles;
    int slices = std::max(1, workers / base_units);
    slices = (int)std::min<int64_t>(slices, d.Nb);
    pl.wg_imgs_per_slice = (int)((d.Nb + slices - 1) / slices);
    pl.wg_slices = (int)((d.Nb + pl.wg_imgs_per_slice - 1) / pl.wg_imgs_per_slice);
    pl.x_nhwc = align_up((size_t)d.Nb * d.C * d.H * d.W * 2, 1024);
    pl.dz_nhwc = align_up((size_t)d.Nb * d.O * d.H * d.W * 2, 1024);
    pl.wpack = align_up((size_t)d.O * d.C * 9 * 2, 1024);
    pl.part = align_up((size_t)pl.wg_slices * 9 * d.O * d.C * sizeof(float), 1024);
    pl.db_part = align_up((size_t)d.Nb * ((d.H * d.W + 63) / 64) * d.O * sizeof(float), 1024);   // one partial row per repack block
    pl.flags = align_up((size_t)(1 + d.Nb) * sizeof(unsigned int), 1024);                          // counters of the repack kernel that runs beside a conv
    pl.ok = true;
    return pl;
}

// the two-SM form takes every tile as a pair of blocks; it is the form that can also store pixel-major (NHWC) tiles
bool fprop_pair_form(const ConvDims &d, const TcPlan &pl, int Cout, int sms)
{
    const int nt = pl.rows_per_tile * (int)d.W;
    return Cout % 256 == 0 && pl.rows_per_tile % 2 == 0 && ((nt / 2) * 128) % 1024 == 0 && sms >= 2 &&
           (int64_t)d.Nb * (d.H / pl.rows_per_tile) * (Cout / 256) >= sms / 2;
}

int sm_count()
{
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 148;
    return sms;
}

// `out_nhwc` (only where fprop_pair_form holds): `out` is [Nb][H][W][Cout] instead of [Nb][Cout][H][W]
// `flags` (only where fprop_pair_form holds): the activations and packed weights are being produced by a repack_stream_kernel
// launched just before on the same stream; see there
relay_status_t launch_fprop(const ConvDims &d, const TcPlan &pl, const void *act_nhwc, int Cin, const void *wpacked, int Cout,
                            const void *bias, int32_t b_dt, int act, void *out_nchw, cudaStream_t st, bool out_nhwc = false,
                            const unsigned int *flags = nullptr, int pack_units = 0)
{
    CUtensorMap tm_w, tm_x, tm_y;
    RELAY_TRY(make_tmap_2d_bf16(&tm_w, wpacked, (uint64_t)9 * Cin, Cout, (uint64_t)9 * Cin, BK, BM));
    RELAY_TRY(make_tmap_nhwc_bf16(&tm_x, act_nhwc, Cin, d.W, d.H, d.Nb, BK, (uint32_t)d.W, pl.rows_per_tile));
    // output NCHW as [Nb * Cout rows][H * W columns]; 32 x 32 boxes, rows of 64 bytes, no swizzle
    RELAY_TRY(make_tmap_2d(&tm_y, false, out_nchw, (uint64_t)(d.H * d.W), (uint64_t)d.Nb * Cout, (uint64_t)(d.H * d.W), 32, 32, false));
    const int sms = sm_count();
    FpropParams p{};
    p.Cin = Cin; p.Cout = Cout; p.H = (int)d.H; p.W = (int)d.W; p.Nb = (int)d.Nb; p.taps_r = 3; p.taps_s = 3; p.pad = 1;
    p.rows_per_tile = pl.rows_per_tile; p.nt = pl.rows_per_tile * (int)d.W;
    p.tiles_per_img = (int)d.H / pl.rows_per_tile; p.n_tiles_total = (int)d.Nb * p.tiles_per_img;
    p.k_blocks = 9 * Cin / BK;
    p.bias = bias; p.bias_bf16 = b_dt == RELAY_BF16; p.act = act;
    p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    // two-SM form: every tile is computed by a pair of blocks, each loading half of the activation tile
    if ((out_nhwc || flags) && !fprop_pair_form(d, pl, Cout, sms)) return fail(RELAY_ERR_UNSUPPORTED, "conv2d: not in the one-SM kernel");
    p.flags = flags; p.pack_units = pack_units; p.units_per_img = (int)((d.H * d.W + 63) / 64);
    if (fprop_pair_form(d, pl, Cout, sms)) {
        CUtensorMap tm_xh, tm_y2, tm_xq, tm_yt;
        RELAY_TRY(make_tmap_nhwc_bf16(&tm_xh, act_nhwc, Cin, d.W, d.H, d.Nb, BK, (uint32_t)d.W, pl.rows_per_tile / 2));
        // output boxes of 32 channels x 32 pixels (NHWC: 32 pixels x 32 channels), rows of 64 bytes in the 64-byte swizzle pattern
        if (out_nhwc) RELAY_TRY(make_tmap_2d_sw64(&tm_y2, false, out_nchw, (uint64_t)Cout, (uint64_t)(d.Nb * d.H * d.W), (uint64_t)Cout, 32));
        else RELAY_TRY(make_tmap_2d_sw64(&tm_y2, false, out_nchw, (uint64_t)(d.H * d.W), (uint64_t)d.Nb * Cout, (uint64_t)(d.H * d.W), 32));
        p.out_nhwc = out_nhwc ? 1 : 0;
        const size_t stage2 = (size_t)BM * BK * 2 + (size_t)(p.nt / 2) * 128;
        p.stages = (int)std::min<size_t>(8, (kSmemLimit - 1024 - 4 * 4096) / stage2);
        p.pairs_per_ntile = Cout / 256;
        p.n_pairs = p.n_items = p.n_full = p.n_tiles_total * p.pairs_per_ntile;
        // the items that would start one more round over the pairs, if they are at most half a round, run as half tiles
        const int pairs = std::min(p.n_items, sms / 2), rest = p.n_items % pairs;
        const bool can_halve = pl.rows_per_tile % 4 == 0 && ((p.nt / 4) * 128) % 1024 == 0 && (p.nt / 2) % 16 == 0;
        tm_xq = tm_xh; tm_yt = tm_y2;
        if (can_halve && p.n_items > pairs && rest != 0 && 2 * rest <= pairs) {
            p.n_full = p.n_items - rest;
            p.n_items = p.n_full + 2 * rest;
            RELAY_TRY(make_tmap_nhwc_bf16(&tm_xq, act_nhwc, Cin, d.W, d.H, d.Nb, BK, (uint32_t)d.W, pl.rows_per_tile / 4));
            if (out_nhwc) RELAY_TRY(make_tmap_2d(&tm_yt, false, out_nchw, (uint64_t)Cout, (uint64_t)(d.Nb * d.H * d.W), (uint64_t)Cout, 32, 16, false));
            else RELAY_TRY(make_tmap_2d(&tm_yt, false, out_nchw, (uint64_t)(d.H * d.W), (uint64_t)d.Nb * Cout, (uint64_t)(d.H * d.W), 16, 32, false));
        }
        const size_t smem2 = 1024 + (size_t)p.stages * stage2 + 4 * 4096 + 256;
        RELAY_CUDA(cudaFuncSetAttribute(conv_fprop_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
        RELAY_CUDA(launch_pdl(conv_fprop_tc2_kernel, dim3(2 * pairs), dim3(NUM_THREADS), smem2, st, tm_w, tm_xh, tm_y2, tm_xq, tm_yt, p));
        return check_launch("conv_fprop_tc2");
    }
    // one-SM form: pairs fill whole rounds over the SMs; the remainder runs as singles
    const int64_t total_pairs = Cout % 256 == 0 ? (int64_t)p.n_tiles_total * (Cout / 256) : 0;
    const int mh = total_pairs >= sms ? 2 : 1;
    const size_t b_stage = ((size_t)p.nt * BK * 2 + 1023) & ~size_t(1023);
    const size_t stage = (size_t)mh * BM * BK * 2 + b_stage;
    const size_t staging = (size_t)4 * mh * 4096;
    p.stages = (int)std::min<size_t>(6, (kSmemLimit - 1024 - staging) / stage);
    if (p.stages < 2) return fail(RELAY_ERR_UNSUPPORTED, "conv2d tile does not fit in shared memory");
    const size_t smem = 1024 + (size_t)p.stages * stage + staging + 256;
    if (mh == 2) {
        p.pairs_per_ntile = Cout / 256;
        const int64_t ntiles_as_pairs = (total_pairs / sms) * sms / p.pairs_per_ntile;   // whole n-tiles only
        p.n_pairs = (int)(ntiles_as_pairs * p.pairs_per_ntile);
        p.n_items = p.n_pairs + (int)((p.n_tiles_total - ntiles_as_pairs) * (Cout / BM));
        RELAY_CUDA(cudaFuncSetAttribute(conv_fprop_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RELAY_CUDA(launch_pdl(conv_fprop_tc_kernel<2>, dim3(std::min(p.n_items, sms)), dim3(64 + 256), smem, st, tm_w, tm_x, tm_y, p));
    } else {
        p.pairs_per_ntile = 1; p.n_pairs = 0; p.n_items = p.n_tiles_total * (Cout / BM);
        RELAY_CUDA(cudaFuncSetAttribute(conv_fprop_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RELAY_CUDA(launch_pdl(conv_fprop_tc_kernel<1>, dim3(std::min(p.n_items, sms)), dim3(64 + 128), smem, st, tm_w, tm_x, tm_y, p));
    }
    return check_launch("conv_fprop_tc");
}

// `w` (optional): the same launch also packs the O x Cw x 3 x 3 weights into wf and / or wb
relay_status_t launch_transpose(bool grad, const void *in, const void *y, void *out, int64_t Nb, int64_t C, int64_t HW, int act,
                                float *db_part, cudaStream_t st, const void *w = nullptr, void *wf = nullptr, void *wb = nullptr,
                                int64_t O = 0, int64_t Cw = 0)
{
    // one channel block per thread block: two per block measured the same (97.4 us for the forward group of cfg4 either
    // way), four slower (102.6 us: fewer blocks fit an SM)
    constexpr int NT = 1;
    dim3 grid((unsigned)((HW + 63) / 64), (unsigned)((C + 64 * NT - 1) / (64 * NT)), (unsigned)Nb);
    PackJob job{};
    if (w != nullptr) {
        job.w = (const __nv_bfloat16 *)w; job.wf = (__nv_bfloat16 *)wf; job.wb = (__nv_bfloat16 *)wb;
        job.O = (int)O; job.C = (int)Cw; job.taps = 9; job.n_img = (int)Nb;
        const int64_t per_slice = (int64_t)grid.x * grid.y * 256;
        grid.z += (unsigned)((O * Cw * 9 + per_slice - 1) / per_slice);
    }
#define RELAY_REPACK(G, N_) RELAY_CUDA(launch_pdl(nchw_to_nhwc_kernel<G, N_>, grid, dim3(256), 0, st, (const __nv_bfloat16 *)in, (const __nv_bfloat16 *)(G ? y : nullptr), (__nv_bfloat16 *)out, (int)C, (int)HW, act, G ? db_part : (float *)nullptr, job))
    if (grad) RELAY_REPACK(true, NT);
    else RELAY_REPACK(false, NT);
#undef RELAY_REPACK
    return check_launch("nchw_to_nhwc");
}

// Launches the persistent repack beside which the next kernel of the stream (a two-SM conv given `flags`) runs.
// job0 is the tensor that conv consumes (counted per image); job1 (optional) only has to be complete when that conv ends.
relay_status_t launch_repack_stream(const ConvDims &d, const RepackJob &job0, const RepackJob *job1, const void *w, void *wf, void *wb,
                                    unsigned int *flags, int *pack_units, cudaStream_t st)
{
    RepackStream S{};
    S.job[0] = job0; S.n_jobs = 1;
    if (job1) { S.job[1] = *job1; S.n_jobs = 2; }
    S.Nb = (int)d.Nb; S.HW = (int)(d.H * d.W); S.pbx = (S.HW + 63) / 64;
    S.pack.w = (const __nv_bfloat16 *)w; S.pack.wf = (__nv_bfloat16 *)wf; S.pack.wb = (__nv_bfloat16 *)wb;
    S.pack.O = (int)d.O; S.pack.C = (int)d.C; S.pack.taps = 9; S.pack.n_img = 0;
    S.pack_units = (int)((d.O * d.C * 9 + kPackPerUnit - 1) / kPackPerUnit);
    S.flags = flags;
    *pack_units = S.pack_units;
    RELAY_CUDA(cudaMemsetAsync(flags, 0, (size_t)(1 + d.Nb) * sizeof(unsigned int), st));
    // the SMs must already be split for the most shared memory while this kernel runs: a consumer block that needed another
    // split could only start on an SM once it had drained
    RELAY_CUDA(cudaFuncSetAttribute(repack_stream_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
    int per_sm = 0;
    RELAY_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, repack_stream_kernel, 256, 0));
    const int64_t total = S.pack_units + (int64_t)S.n_jobs * S.Nb * S.pbx;
    const int grid = (int)std::min<int64_t>(total, (int64_t)sm_count() * std::max(1, std::min(per_sm, 2)));
    RELAY_CUDA(launch_pdl(repack_stream_kernel, dim3((unsigned)grid), dim3(256), 0, st, S));
    return check_launch("repack_stream");
}

}  // namespace

relay_status_t make_tmap_nhwc_bf16(CUtensorMap *m, const void *base, uint64_t C, uint64_t W, uint64_t H, uint64_t N,
                                   uint32_t box_c, uint32_t box_w, uint32_t box_h)
{
    typedef CUresult (*Fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                           const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                           CUtensorMapFloatOOBfill);
    void *fp = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
        return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[4] = {C, W, H, N};
    cuuint64_t strides[3] = {C * 2, W * C * 2, H * W * C * 2};
    cuuint32_t box[4] = {box_c, box_w, box_h, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = ((Fn)fp)(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(RELAY_ERR_CUDA, "cuTensorMapEncodeTiled (NHWC) failed with code %d", (int)r);
    return RELAY_OK;
}

bool conv_tc_eligible(const ConvDims &d) { return plan(d).ok; }

size_t conv_tc_fwd_workspace(const ConvDims &d)
{
    TcPlan pl = plan(d);
    return pl.ok ? pl.x_nhwc + pl.wpack : 0;
}

size_t conv_tc_grad_workspace(const ConvDims &d)
{
    TcPlan pl = plan(d);
    return pl.ok ? pl.x_nhwc + pl.dz_nhwc + pl.wpack + pl.part + pl.db_part + pl.flags : 0;
}

relay_status_t launch_conv_fwd_tc(const ConvDims &d, const void *x, bool x_is_nhwc, const void *w, const void *b, int32_t b_dt, int act,
                                  void *y, void *ws, cudaStream_t st, void *y_nhwc)
{
    TcPlan pl = plan(d);
    char *base = (char *)ws;
    void *wf = base + pl.x_nhwc;
    const void *x_nhwc = x;
    if (!x_is_nhwc) {
        // the repack launch packs the weights as well
        RELAY_TRY(launch_transpose(false, x, nullptr, base, d.Nb, d.C, d.H * d.W, 0, nullptr, st, w, wf, nullptr, d.O, d.C));
        x_nhwc = base;
    } else {
        RELAY_CUDA(launch_pdl(pack_weights_kernel, dim3((unsigned)((d.O * d.C * 9 + 255) / 256)), dim3(256), 0, st, (const __nv_bfloat16 *)w, (__nv_bfloat16 *)wf, (__nv_bfloat16 *)nullptr, (int)d.O, (int)d.C, 3, 3));
        RELAY_TRY(check_launch("pack_weights"));
    }
    if (!y_nhwc) return launch_fprop(d, pl, x_nhwc, (int)d.C, wf, (int)d.O, b, b_dt, act, y, st);
    if (fprop_pair_form(d, pl, (int)d.O, sm_count())) return launch_fprop(d, pl, x_nhwc, (int)d.C, wf, (int)d.O, b, b_dt, act, y_nhwc, st, true);
    RELAY_TRY(launch_fprop(d, pl, x_nhwc, (int)d.C, wf, (int)d.O, b, b_dt, act, y, st));
    return launch_transpose(false, y, nullptr, y_nhwc, d.Nb, d.O, d.H * d.W, 0, nullptr, st);
}

relay_status_t launch_conv_grad_tc(const ConvDims &d, const void *x, const void *w, const void *y, const void *dy, int act, void *dx,
                                   void *dw, float *db, void *ws, cudaStream_t st, bool nhwc_in, float *nhwc_partials, void *dx_nhwc)
{
    TcPlan pl = plan(d);
    char *base = (char *)ws;
    const void *x_nhwc = base;
    void *dz_nhwc = base + pl.x_nhwc;
    void *wb = base + pl.x_nhwc + pl.dz_nhwc;
    float *part = (float *)(base + pl.x_nhwc + pl.dz_nhwc + pl.wpack);
    float *db_part = (float *)(base + pl.x_nhwc + pl.dz_nhwc + pl.wpack + pl.part);
    const int64_t HW = d.H * d.W;
    const bool beside = !nhwc_in && dx && !dx_nhwc && fprop_pair_form(d, pl, (int)d.C, sm_count());
    if (beside) {
        // One persistent repack kernel writes dZ = dy (.) act'(y) in NHWC (with the bias-gradient partials), then x in NHWC, and
        // packs the mirrored weights; the input-gradient conv runs BESIDE it, taking each image of dZ as soon as it is complete.
        // That conv ends only after the repack kernel has, so the weight-gradient kernel behind it finds x complete.
        unsigned int *flags = (unsigned int *)(base + pl.x_nhwc + pl.dz_nhwc + pl.wpack + pl.part + pl.db_part);
        RepackJob jz{}, jx{};
        jz.in = (const __nv_bfloat16 *)dy; jz.y = (const __nv_bfloat16 *)y; jz.out = (__nv_bfloat16 *)dz_nhwc; jz.db_part = db ? db_part : nullptr;
        jz.C = (int)d.O; jz.grad = 1; jz.act = act; jz.flagged = 1;
        jx.in = (const __nv_bfloat16 *)x; jx.out = (__nv_bfloat16 *)base; jx.C = (int)d.C;
        int pack_units = 0;
        RELAY_TRY(launch_repack_stream(d, jz, &jx, w, nullptr, wb, flags, &pack_units, st));
        RELAY_TRY(launch_fprop(d, pl, dz_nhwc, (int)d.O, wb, (int)d.C, nullptr, RELAY_F32, RELAY_ACT_NONE, dx, st, false, flags, pack_units));
        if (db) RELAY_TRY(launch_colsum_finalize(db_part, (int)(d.Nb * ((HW + 63) / 64)), d.O, 1.0f, db, st));
    } else if (nhwc_in) {
        // x, y, dy are NHWC already: dZ = dy (.) act'(y) is one elementwise pass over [N*H*W, O] whose column sums are db;
        // x is read where it lies
        RELAY_TRY(launch_act_grad(RELAY_BF16, dy, y, dz_nhwc, db, nhwc_partials, d.Nb * HW, d.O, act, st));
        x_nhwc = x;
    } else {
        // dZ = dy (.) act'(y), written straight into NHWC; x into NHWC
        // (the same pass leaves per-block partial sums of dZ over pixels for the bias gradient)
        // (the same launch packs the mirrored weights that the input gradient needs)
        RELAY_TRY(launch_transpose(true, dy, y, dz_nhwc, d.Nb, d.O, HW, act, db ? db_part : nullptr, st, dx ? w : nullptr, nullptr, wb, d.O, d.C));
        RELAY_TRY(launch_transpose(false, x, nullptr, base, d.Nb, d.C, HW, 0, nullptr, st));
        if (db) RELAY_TRY(launch_colsum_finalize(db_part, (int)(d.Nb * ((HW + 63) / 64)), d.O, 1.0f, db, st));
    }
    if (dx && !beside) {
        if (nhwc_in) {
            RELAY_CUDA(launch_pdl(pack_weights_kernel, dim3((unsigned)((d.O * d.C * 9 + 255) / 256)), dim3(256), 0, st, (const __nv_bfloat16 *)w, (__nv_bfloat16 *)nullptr, (__nv_bfloat16 *)wb, (int)d.O, (int)d.C, 3, 3));
            RELAY_TRY(check_launch("pack_weights"));
        }
        if (dx_nhwc && fprop_pair_form(d, pl, (int)d.C, sm_count())) {
            RELAY_TRY(launch_fprop(d, pl, dz_nhwc, (int)d.O, wb, (int)d.C, nullptr, RELAY_F32, RELAY_ACT_NONE, dx_nhwc, st, true));
        } else {
            RELAY_TRY(launch_fprop(d, pl, dz_nhwc, (int)d.O, wb, (int)d.C, nullptr, RELAY_F32, RELAY_ACT_NONE, dx, st));
            if (dx_nhwc) RELAY_TRY(launch_transpose(false, dx, nullptr, dx_nhwc, d.Nb, d.C, HW, 0, nullptr, st));
        }
    }
    CUtensorMap tm_dz, tm_x;
    RELAY_TRY(make_tmap_nhwc_bf16(&tm_dz, dz_nhwc, d.O, d.W, d.H, d.Nb, 64, (uint32_t)d.W, pl.rows_per_kblock));
    RELAY_TRY(make_tmap_nhwc_bf16(&tm_x, x_nhwc, d.C, d.W, d.H, d.Nb, 64, (uint32_t)d.W, pl.rows_per_kblock));
    WgradParams p{};
    p.C = (int)d.C; p.O = (int)d.O; p.H = (int)d.H; p.W = (int)d.W; p.Nb = (int)d.Nb; p.taps_r = 3; p.taps_s = 3; p.pad = 1;
    p.rows_per_kblock = pl.rows_per_kblock; p.kpix = pl.rows_per_kblock * (int)d.W; p.nt = pl.wg_nt;
    p.m_tiles = pl.wg_m_tiles; p.c_tiles = pl.wg_c_tiles; p.n_slices = pl.wg_slices; p.imgs_per_slice = pl.wg_imgs_per_slice;
    p.stages = pl.wg_stages; p.part = part; p.err = device_error_word();
    if (!p.err) return fail(RELAY_ERR_CUDA, "no device error word");
    const size_t stage = (size_t)(BM / 64 + p.nt / 64) * p.kpix * 128;
    const size_t smem = 1024 + (size_t)p.stages * stage + 4 * 8192 + 256;
    CUtensorMap tm_part;
    RELAY_TRY(make_tmap_2d(&tm_part, true, part, (uint64_t)d.C, (uint64_t)p.n_slices * 9 * d.O, (uint64_t)d.C, 32, 32, true));
    const int grid = 9 * p.m_tiles * p.c_tiles * p.n_slices;
    if (pl.wg_pair) {
        const size_t smem2 = 1024 + (size_t)p.stages * 4 * p.kpix * 128 + 4 * 8192 + 256;
        RELAY_CUDA(cudaFuncSetAttribute(conv_wgrad_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2));
        RELAY_CUDA(launch_pdl(conv_wgrad_tc2_kernel, dim3(2 * grid), dim3(NUM_THREADS), smem2, st, tm_dz, tm_x, tm_part, p));
    } else {
        RELAY_CUDA(cudaFuncSetAttribute(conv_wgrad_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        RELAY_CUDA(launch_pdl(conv_wgrad_tc_kernel, dim3(grid), dim3(NUM_THREADS), smem, st, tm_dz, tm_x, tm_part, p));
    }
    RELAY_TRY(check_launch("conv_wgrad_tc"));
    RELAY_CUDA(launch_pdl(wgrad_reduce_kernel, dim3((unsigned)((d.O * d.C + 127) / 128)), dim3(128), 0, st, (const float *)part, p.n_slices, (__nv_bfloat16 *)dw, (int)d.O, (int)d.C, 9));
    return check_launch("wgrad_reduce");
}

}  // namespace relay

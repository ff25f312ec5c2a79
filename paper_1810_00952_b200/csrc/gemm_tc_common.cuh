// Pieces shared by the one-SM and the two-SM tensor-core contraction kernels: tile constants, kernel
// parameters and the epilogue of one warp.
#pragma once
#include "ewise_kernels.cuh"
#include "tc_common.cuh"

namespace relay {
namespace gemm_tc {

constexpr int BN = 256, BK = 64;
constexpr int MN_BOX_BYTES = 64 * BK * 2;   // one TMA box of an MN-major operand: 64 (M/N) x 64 (k)
constexpr int TMEM_COLS = 512;              // two accumulators of 256 fp32 columns

struct Params {
    int M, N, K;
    void *c;
    long long ldc;
    const void *bias;
    int bias_bf16, act, out_f32;
    int tiles_m, tiles_n, k_blocks;
    // two-SM kernel: wide_units 256 x 512 units come first; of the remaining tiles, those after the first full_tiles
    // are cut into tail_split column parts
    int wide_units, full_tiles, tail_split;
    int *err;
    // > 0 (two-SM kernel only): the columns are LSTM pre-activations in blocks of this many columns [ i | f | g | o ]; the
    // epilogue applies tanh to block 2 and the logistic function to the others (`act` is ignored)
    int gate_block;
};

// Bias values of up to 256 columns starting at n0, one 32-column group per register: lane j holds the bias of
// column n0 + 32 g + j in b[g].  Fetched before the warp waits for its accumulator, so that the latency of
// these loads is not paid per group inside the drain loop.
__device__ __forceinline__ void load_bias(const Params &p, int lane, int n0, int width, float (&b)[8])
{
#pragma unroll
    for (int g = 0; g < 8; ++g) {
        const int c = n0 + g * 32 + lane;
        b[g] = 0.0f;
        if (p.bias != nullptr && g * 32 < width && c < p.N)
            b[g] = p.bias_bf16 ? __bfloat162float(((const __nv_bfloat16 *)p.bias)[c]) : ((const float *)p.bias)[c];
    }
}

// One warp drains 32 accumulator rows, the 128-byte column blocks [blk_begin, blk_end) of an accumulator that
// starts at column n0 (block = 64 bf16 or 32 f32 columns): TMEM -> registers -> bias + activation -> rounding ->
// swizzled staging buffers -> TMA tile store of 32 rows x 128 bytes at a time.  `bias_r` comes from load_bias(n0).
template <bool OUT_F32, int BUFS>
__device__ __forceinline__ void epilogue_rows(const Params &p, const CUtensorMap *tm_c, uint32_t taddr, uint8_t *stage, int lane,
                                              int row0, int n0, const float (&bias_r)[8], int blk_begin, int blk_end)
{
    constexpr int COLS = OUT_F32 ? 32 : 64;             // columns per 128-byte block
    constexpr int SUBS = COLS / 32;
#pragma unroll 1
    for (int blk = blk_begin; blk < blk_end; ++blk) {
        const int nc = n0 + blk * COLS;
        if (nc >= p.N) break;                            // warp-uniform
        uint32_t r[SUBS][32];
#pragma unroll
        for (int sub = 0; sub < SUBS; ++sub) tc::tmem_ld_32x32(taddr + blk * COLS + sub * 32, r[sub]);
        tc::tmem_ld_wait();
        uint4 piece[8];
#pragma unroll
        for (int sub = 0; sub < SUBS; ++sub) {
            float v[32];
            if (p.bias != nullptr) {                     // warp-uniform
                // every lane reads the 32 bias values of this group by shuffle (lane j holds column j's)
                float bias_lane = 0.0f;
#pragma unroll
                for (int g = 0; g < 8; ++g) if (g == blk * SUBS + sub) bias_lane = bias_r[g];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[sub][j]) + __shfl_sync(0xffffffffu, bias_lane, j);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[sub][j]);
            }
            switch (p.act) {                             // hoisted out of the element loop
            case RELAY_ACT_RELU:
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = fmaxf(v[j], 0.0f);
                break;
            case RELAY_ACT_TANH:
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = OUT_F32 ? tanh_<false>(v[j]) : tanh_<true>(v[j]);
                break;
            case RELAY_ACT_SIGMOID:
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = OUT_F32 ? sigmoid_<false>(v[j]) : sigmoid_<true>(v[j]);
                break;
            default: break;
            }
            if (OUT_F32) {
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    piece[c] = make_uint4(__float_as_uint(v[4 * c]), __float_as_uint(v[4 * c + 1]), __float_as_uint(v[4 * c + 2]),
                                          __float_as_uint(v[4 * c + 3]));
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    piece[sub * 4 + c] = make_uint4(pack2(v[8 * c], v[8 * c + 1]), pack2(v[8 * c + 2], v[8 * c + 3]),
                                                    pack2(v[8 * c + 4], v[8 * c + 5]), pack2(v[8 * c + 6], v[8 * c + 7]));
            }
        }
        tc::warp_store_block<BUFS - 1>(tm_c, stage + ((blk - blk_begin) % BUFS) * 4096, piece, lane, nc, row0);
    }
}


}  // namespace gemm_tc
}  // namespace relay

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
    int full_tiles, tail_split;   // two-SM kernel: tiles after the first full_tiles are cut into tail_split column parts
    int *err;
};

// One warp drains its 32 accumulator rows (`width` columns, 256 unless stated): TMEM -> registers -> bias +
// activation -> rounding -> swizzled staging buffer -> TMA tile store of 32 rows x 128 bytes at a time.
template <bool OUT_F32, int BUFS>
__device__ __forceinline__ void epilogue_rows(const Params &p, const CUtensorMap *tm_c, uint32_t taddr, uint8_t *stage, int lane,
                                              int row0, int n0, int width = BN)
{
    constexpr int COLS = OUT_F32 ? 32 : 64;             // columns per 128-byte block
#pragma unroll 1
    for (int blk = 0; blk < width / COLS; ++blk) {
        const int nc = n0 + blk * COLS;
        if (nc >= p.N) break;                            // warp-uniform
        uint4 piece[8];
#pragma unroll
        for (int sub = 0; sub < COLS / 32; ++sub) {
            uint32_t r[32];
            tc::tmem_ld_32x32(taddr + blk * COLS + sub * 32, r);
            tc::tmem_ld_wait();
            const int c0 = nc + sub * 32;
            // lane j fetches the bias of column c0 + j; every lane then reads all 32 by shuffle
            float bias_lane = 0.0f;
            if (p.bias != nullptr && c0 + lane < p.N)
                bias_lane = p.bias_bf16 ? __bfloat162float(((const __nv_bfloat16 *)p.bias)[c0 + lane]) : ((const float *)p.bias)[c0 + lane];
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bias_lane, j);
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
        tc::warp_store_block<BUFS - 1>(tm_c, stage + (blk % BUFS) * 4096, piece, lane, nc, row0);
    }
}


}  // namespace gemm_tc
}  // namespace relay

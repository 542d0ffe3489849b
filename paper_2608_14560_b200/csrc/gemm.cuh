// Grouped block-scaled FP8 GEMMs of the expert MLP (stage 3 of the Fused MoE
// description): GEMM1 [rows,H] x w13[e]^T with SwiGLU and FP8 re-quantisation
// fused into its epilogue, and GEMM2 [rows,I] x w2[e]^T writing bf16 rows for
// the combine.
//
// One persistent CTA per SM walks a static list of 128 x 256 output tiles.
//   warp 0      TMA producer: A tile (128 rows x 128 K-bytes) and B tile (256
//               weight rows x 128 K-bytes) per K-block into a 4-stage ring,
//               128-byte swizzle, completion on mbarriers.
//   warp 1      MMA issuer: four tcgen05.mma (M128 N256 K32, e4m3 -> fp32) per
//               K-block into one of two 256-column TMEM accumulators; each
//               K-block starts from zero because its partial sum must be
//               multiplied by fp32 scales before it joins the running sum.
//   warps 4-11  epilogue: read the K-block partial from TMEM, multiply by
//               a_scale[row,kb] * w_scale[nblk,kb], accumulate in registers;
//               at the end of the tile apply the fused tail and store.
// Scales are arbitrary fp32 (amax/448), so the power-of-two hardware block
// scaling cannot express them; the per-K-block promotion is done on the ALUs.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "ptx.cuh"

namespace moe {

constexpr int G_STAGES = 4;
constexpr int G_BLOCK_K = 128;                                  // K bytes per stage = one scale block
constexpr int G_TILE_N = 256;                                   // accumulator columns
constexpr int G_A_BYTES = TILE_M * G_BLOCK_K;                   // 16 KB
constexpr int G_B_BYTES = G_TILE_N * G_BLOCK_K;                 // 32 KB
constexpr int G_STAGE_BYTES = G_A_BYTES + G_B_BYTES;            // 48 KB
constexpr int G_THREADS = 384;                                  // 4 control warps + 8 epilogue warps
constexpr int G_EPI_THREADS = 256;
constexpr int G_CTRL_BYTES = 4096;                              // barriers, flags, amax exchange
constexpr int G_SMEM_BYTES = G_STAGES * G_STAGE_BYTES + G_CTRL_BYTES + 1024;  // + alignment slack
constexpr uint32_t G_TMEM_COLS = 512;

struct GemmArgs {
    int num_kb;               // K / 128
    int n_tiles;              // output tiles along N per row tile
    int w_rows_per_expert;    // rows of the weight matrix per expert (2I or H)
    int row_cap;              // rows in the activation buffers (stride of transposed scales)
    int out_cols;             // I (GEMM1) or H (GEMM2)
    int gate_row0, up_row0;   // GEMM1: first weight row of the gate / up half
    const int* num_m_tiles;   // device scalars and tables built by the permute stage
    const int* tile_expert;
    const int* tile_rows;
    const float* a_scale_t;   // [num_kb, row_cap]
    const float* w_scale;     // [E_loc, w_rows/128, num_kb]
    uint8_t* out_fp8;         // GEMM1: [row_cap, I] e4m3
    float* out_scale_t;       // GEMM1: [I/128, row_cap]
    __nv_bfloat16* out_bf16;  // GEMM2: [row_cap, H]
    int* status;
};

struct GemmCtrl {
    uint64_t full[G_STAGES];
    uint64_t empty[G_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t amax_bar[2];
    uint64_t drain_bar;
    uint32_t tmem_slot;
    int abort_flag;
    float amax[2][2][TILE_M];  // [tile parity][column half][row]
};
static_assert(sizeof(GemmCtrl) <= G_CTRL_BYTES, "control block too large");

__device__ __forceinline__ void raise(GemmCtrl* c, int* status, int code) {
    *reinterpret_cast<volatile int*>(&c->abort_flag) = 1;
    atomicCAS(status, DEV_OK, code);
}

template <int MODE>
__global__ void __launch_bounds__(G_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(smem + G_STAGES * G_STAGE_BYTES);
    volatile int* abort_flag = &ctrl->abort_flag;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G_STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctrl->tmem_full[b]), 1);
            mbar_init(smem_u32(&ctrl->tmem_empty[b]), G_EPI_THREADS / 32);
            mbar_init(smem_u32(&ctrl->amax_bar[b]), G_EPI_THREADS);
        }
        mbar_init(smem_u32(&ctrl->drain_bar), 1);
        ctrl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_slot), G_TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_slot);
    const int num_tiles = __ldg(g.num_m_tiles) * g.n_tiles;
    const int num_kb = g.num_kb;

    if (warp < 4) {
        reg_dealloc<40>();
        if (warp == 0 && lane == 0) {
            // ---------------- TMA producer ----------------
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
                const int wrow = __ldg(g.tile_expert + m_tile) * g.w_rows_per_expert;
                int b_row0, b_row1;
                if (MODE == 1) {
                    b_row0 = wrow + g.gate_row0 + n * 128;
                    b_row1 = wrow + g.up_row0 + n * 128;
                } else {
                    b_row0 = wrow + n * G_TILE_N;
                    b_row1 = b_row0 + 128;
                }
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % G_STAGES, ph = (it / G_STAGES) & 1;
                    if (!mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1, abort_flag)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_PRODUCER);
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&ctrl->full[s]);
                    const uint32_t a_dst = smem_base + s * G_STAGE_BYTES, b_dst = a_dst + G_A_BYTES;
                    mbar_expect_tx(bar, G_STAGE_BYTES);
                    tma_load_2d(a_dst, &tmA, kb * G_BLOCK_K, m_tile * TILE_M, bar);
                    tma_load_2d(b_dst, &tmB, kb * G_BLOCK_K, b_row0, bar);
                    tma_load_2d(b_dst + G_B_BYTES / 2, &tmB, kb * G_BLOCK_K, b_row1, bar);
                }
            }
            if (!ok || *abort_flag) {
                // wait (bounded) until the copies still in flight have landed
                const uint32_t n_back = it < G_STAGES ? it : G_STAGES;
                int zero = 0;
                for (uint32_t j = it - n_back; j < it; ++j)
                    if (!mbar_wait(smem_u32(&ctrl->full[j % G_STAGES]), (j / G_STAGES) & 1, &zero))
                        atomicCAS(g.status, DEV_OK, DEV_TIMEOUT_DRAIN);
            }
        } else if (warp == 1 && lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = umma_idesc_f8(TILE_M, G_TILE_N);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % G_STAGES, ph = (it / G_STAGES) & 1;
                    const uint32_t b = it & 1, bph = (it >> 1) & 1;
                    if (!mbar_wait(smem_u32(&ctrl->tmem_empty[b]), bph ^ 1, abort_flag)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_MMA_TMEM);
                        ok = false;
                        break;
                    }
                    if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_MMA_SMEM);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * G_STAGE_BYTES;
                    const uint64_t a_desc = umma_desc_sw128(a_addr);
                    const uint64_t b_desc = umma_desc_sw128(a_addr + G_A_BYTES);
                    const uint32_t d_tmem = tmem_base + b * G_TILE_N;
#pragma unroll
                    for (int k = 0; k < G_BLOCK_K / 32; ++k)  // 32 K-bytes per instruction: +2 in 16-B units
                        umma_f8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k > 0);
                    umma_commit(smem_u32(&ctrl->empty[s]));
                    umma_commit(smem_u32(&ctrl->tmem_full[b]));
                }
            }
            if (!ok || *abort_flag) {  // let issued MMAs retire before TMEM is released
                umma_commit(smem_u32(&ctrl->drain_bar));
                int zero = 0;
                mbar_wait(smem_u32(&ctrl->drain_bar), 0, &zero);
            }
        }
    } else {
        // ---------------- epilogue warps ----------------
        reg_alloc<232>();
        const int half = (warp - 4) >> 2;        // which half of the tile's columns
        const int quad = warp & 3;               // TMEM lane quadrant this warp may read
        const int r_in_tile = quad * 32 + lane;  // accumulator row == TMEM lane
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quad * 32) << 16);
        const size_t row_cap = static_cast<size_t>(g.row_cap);
        uint32_t it = 0, tile_iter = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_iter) {
            const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
            const int e = __ldg(g.tile_expert + m_tile);
            const int rows_valid = __ldg(g.tile_rows + m_tile);
            const size_t row = static_cast<size_t>(m_tile) * TILE_M + r_in_tile;
            const float* a_sc = g.a_scale_t + row;
            const int sblocks = g.w_rows_per_expert / 128;
            // weight-scale rows for the two 64-column (GEMM1) or the one 128-column (GEMM2) block(s)
            const float* ws0;
            const float* ws1;
            if (MODE == 1) {
                ws0 = g.w_scale + (static_cast<size_t>(e) * sblocks + g.gate_row0 / 128 + n) * num_kb;
                ws1 = g.w_scale + (static_cast<size_t>(e) * sblocks + g.up_row0 / 128 + n) * num_kb;
            } else {
                ws0 = g.w_scale + (static_cast<size_t>(e) * sblocks + 2 * n + half) * num_kb;
                ws1 = ws0;
            }
            float acc[128];
#pragma unroll
            for (int j = 0; j < 128; ++j) acc[j] = 0.0f;
            float sa = a_sc[0], s0 = __ldg(ws0), s1 = __ldg(ws1);
            for (int kb = 0; kb < num_kb; ++kb, ++it) {
                const float f0 = sa * s0, f1 = sa * s1;
                if (kb + 1 < num_kb) {  // next block's scales travel while we wait for the MMA
                    sa = a_sc[static_cast<size_t>(kb + 1) * row_cap];
                    s0 = __ldg(ws0 + kb + 1);
                    s1 = __ldg(ws1 + kb + 1);
                }
                const uint32_t b = it & 1, bph = (it >> 1) & 1;
                if (!mbar_wait(smem_u32(&ctrl->tmem_full[b]), bph, abort_flag)) {
                    raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                    ok = false;
                    break;
                }
                tc_fence_after();
                // GEMM1: columns [64h,64h+64) are gate, [128+64h, 128+64h+64) the matching up columns.
                // GEMM2: columns [128h, 128h+128).
                const uint32_t col0 = b * G_TILE_N + (MODE == 1 ? 64 * half : 128 * half);
                const uint32_t col1 = b * G_TILE_N + (MODE == 1 ? 128 + 64 * half : 128 * half + 64);
                float v[64];
                tmem_ld64(t_lane + col0, v);
#pragma unroll
                for (int j = 0; j < 64; ++j) acc[j] = fmaf(v[j], f0, acc[j]);
                tmem_ld64(t_lane + col1, v);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[b]));
#pragma unroll
                for (int j = 0; j < 64; ++j) acc[64 + j] = fmaf(v[j], f1, acc[64 + j]);
            }
            if (!ok) break;

            if (MODE == 1) {
                // SwiGLU on this thread's 64 columns, then the row's 128-wide amax across the two halves
                float amax = 0.0f;
#pragma unroll
                for (int j = 0; j < 64; ++j) {
                    const float gt = acc[j];
                    const float c = __fdiv_rn(gt, 1.0f + expf(-gt)) * acc[64 + j];
                    acc[j] = c;
                    amax = fmaxf(amax, fabsf(c));
                }
                const uint32_t par = tile_iter & 1;
                ctrl->amax[par][half][r_in_tile] = amax;
                const uint32_t xbar = smem_u32(&ctrl->amax_bar[par]);
                mbar_arrive(xbar);
                if (!mbar_wait(xbar, (tile_iter >> 1) & 1, abort_flag)) {
                    raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                    break;
                }
                amax = fmaxf(amax, *reinterpret_cast<volatile float*>(&ctrl->amax[par][half ^ 1][r_in_tile]));
                const float sc = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 448.0f);
                if (r_in_tile < rows_valid) {
                    uint4* dst = reinterpret_cast<uint4*>(g.out_fp8 + row * g.out_cols + n * 128 + half * 64);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int j = q * 16 + i * 4;
                            const uint32_t lo = __nv_cvt_float2_to_fp8x2(
                                make_float2(__fdiv_rn(acc[j], sc), __fdiv_rn(acc[j + 1], sc)), __NV_SATFINITE, __NV_E4M3);
                            const uint32_t hi = __nv_cvt_float2_to_fp8x2(
                                make_float2(__fdiv_rn(acc[j + 2], sc), __fdiv_rn(acc[j + 3], sc)), __NV_SATFINITE,
                                __NV_E4M3);
                            w[i] = lo | (hi << 16);
                        }
                        dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (half == 0) g.out_scale_t[static_cast<size_t>(n) * row_cap + row] = sc;
                }
            } else {
                if (r_in_tile < rows_valid) {
                    uint4* dst = reinterpret_cast<uint4*>(g.out_bf16 + row * g.out_cols + n * G_TILE_N + half * 128);
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __nv_bfloat162 p = __floats2bfloat162_rn(acc[q * 8 + 2 * i], acc[q * 8 + 2 * i + 1]);
                            w[i] = *reinterpret_cast<const uint32_t*>(&p);
                        }
                        dst[q] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, G_TMEM_COLS);
    }
}

}  // namespace moe

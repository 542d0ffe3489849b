// Grouped block-scaled FP8 GEMMs of the expert MLP (stage 3 of the Fused MoE
// description): GEMM1 [rows,H] x w13[e]^T with SwiGLU and FP8 re-quantisation
// fused into its epilogue, and GEMM2 [rows,I] x w2[e]^T writing bf16 rows for
// the combine.
//
// One persistent CTA per SM walks a static list of 128 x 256 output tiles.
//   warp 0      TMA producer.  Per K-block (128 K-bytes = one scale block): the A
//               tile (128 rows), the B tile (256 weight rows) and the 128
//               activation scales of the block, into a 4-stage ring (128-byte
//               swizzle) / an 8-slot scale ring, completion on mbarriers.
//   warps 1,2   MMA issuers (even / odd K-blocks).  Four tcgen05.mma (M128 N256 K32, e4m3 -> fp32) per
//               K-block into one of two 256-column TMEM buffers, then ONE
//               tcgen05.commit: the same mbarrier tells the producer that the stage
//               is free and the epilogue that the accumulator is ready (a single
//               thread issues everything, and each MMA, commit and wait costs it
//               50-100 clocks, so the per-K-block instruction count is kept minimal).
//               Every K-block starts from zero because its partial sum must be
//               multiplied by fp32 scales before it joins the running sum.
//   warps 4-7   epilogue of columns [0,128), warps 8-11 of columns [128,256): read
//               the partial from TMEM, multiply by a_scale[row,kb] * w_scale[nblk,kb]
//               with fp32 FMAs, accumulate in registers; at the end of the
//               tile apply the fused tail and store.
// Scales are arbitrary fp32 (amax/448), so the power-of-two hardware block
// scaling cannot express them; the per-K-block promotion is done on the ALUs.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "ptx.cuh"

namespace moe {

constexpr int G_STAGES = 4;
// The two MMA issuer threads take the even and the odd K-blocks.  A thread must see EVERY phase of a barrier it
// waits on (a parity wait cannot tell the wanted phase from the one two earlier), so a stage must always fall
// to the same issuer: the stage count has to be even.
static_assert(G_STAGES % 2 == 0, "an odd stage count lets an issuer thread skip phases of full[s]");
constexpr int G_BLOCK_K = 128;                          // K bytes per stage = one scale block
constexpr int G_TILE_N = 256;                           // output columns per tile
constexpr int G_HALF_N = 128;                           // columns handled by one epilogue warpgroup
constexpr int G_ACC_BUFS = 2;                           // TMEM accumulator buffers (2 x 256 columns)
constexpr int G_A_BYTES = TILE_M * G_BLOCK_K;           // 16 KB
constexpr int G_B_BYTES = G_TILE_N * G_BLOCK_K;         // 32 KB
constexpr int G_STAGE_BYTES = G_A_BYTES + G_B_BYTES;    // 48 KB
constexpr int G_SCALE_RING = 8;                         // K-blocks of activation scales in flight
constexpr int G_SCALE_BYTES = TILE_M * 4;               // 512 B per K-block
constexpr int G_THREADS = 384;                          // 4 control warps + 8 epilogue warps
constexpr int G_EPI_WARPS = 8;
constexpr int G_STORE_WARP_BYTES = 2048;                // per-warp staging: 32 rows x 64 B (swizzled)
constexpr int G_STORE_BYTES = G_EPI_WARPS * G_STORE_WARP_BYTES;
constexpr int G_AMAX_BYTES = 2 * 2 * TILE_M * 4;               // GEMM1 row-amax exchange
constexpr int G_CTRL_BYTES = 512;
constexpr int G_SMEM_BYTES = G_STAGES * G_STAGE_BYTES + G_SCALE_RING * G_SCALE_BYTES + G_STORE_BYTES +
                             G_AMAX_BYTES + G_CTRL_BYTES + 1024;       // + alignment slack
constexpr uint32_t G_TMEM_COLS = 512;
static_assert(G_SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");

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
    __nv_bfloat16* out_bf16;  // GEMM2: tile-blocked rows, see y_block_offset()
    int* status;
    long long wait_limit;     // clocks a bounded wait may spin (WAIT_LIMIT_CLOCKS outside of tests)
    int fault_skip_it;        // test hook: the producer stops before this pipeline iteration (-1: never)
};

struct GemmCtrl {
    uint64_t full[G_STAGES];   // stage filled (TMA transaction bytes)
    uint64_t done[G_STAGES];   // the MMAs that read the stage have finished: stage free AND accumulator ready
    uint64_t tmem_empty[G_ACC_BUFS];
    uint64_t amax_bar[2];
    uint64_t drain_bar[2];
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(GemmCtrl) <= G_CTRL_BYTES, "control block too large");

__device__ __forceinline__ void raise(GemmCtrl* c, int* status, int code) {
    *reinterpret_cast<volatile int*>(&c->abort_flag) = 1;
    atomicCAS(status, DEV_OK, code);
}

// MODE 1: gate/up projection + SwiGLU + re-quantisation (B tile = 4 x 64 weight rows:
//         gate[0,64) | up[0,64) | gate[64,128) | up[64,128) of the tile's 128 columns).
//         tmOut describes the e4m3 output [row_cap, I] for 64-byte x 32-row TMA stores.
// MODE 2: down projection, bf16 rows out in the tile-blocked layout (B tile = 2 x 128 rows).
template <int MODE>
__global__ void __launch_bounds__(G_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmOut, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* scale_ring = reinterpret_cast<float*>(smem + G_STAGES * G_STAGE_BYTES);
    uint8_t* store_stage = smem + G_STAGES * G_STAGE_BYTES + G_SCALE_RING * G_SCALE_BYTES;
    GemmCtrl* ctrl = reinterpret_cast<GemmCtrl*>(store_stage + G_STORE_BYTES + G_AMAX_BYTES);
    volatile int* abort_flag = &ctrl->abort_flag;
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G_STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), 1);
            mbar_init(smem_u32(&ctrl->done[s]), 1);
        }
        for (int b = 0; b < G_ACC_BUFS; ++b) {
            mbar_init(smem_u32(&ctrl->tmem_empty[b]), G_EPI_WARPS);
        }
        mbar_init(smem_u32(&ctrl->amax_bar[0]), G_EPI_WARPS * 32);
        mbar_init(smem_u32(&ctrl->amax_bar[1]), G_EPI_WARPS * 32);
        mbar_init(smem_u32(&ctrl->drain_bar[0]), 1);
        mbar_init(smem_u32(&ctrl->drain_bar[1]), 1);
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
        if (MODE == 1) tma_prefetch_desc(&tmOut);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Everything above touched only this CTA's shared and tensor memory; the tile tables, activations and
    // scales below were written by the kernels before this one.
    pdl_launch_dependents();
    pdl_wait();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctrl->tmem_slot);
    // (the tables come from the kernels before this one, which may still be resident: coherent loads)
    const int num_tiles = __ldcg(g.num_m_tiles) * g.n_tiles;
    const int num_kb = g.num_kb;
    const long long limit = g.wait_limit;

    if (warp < 4) {
        reg_dealloc<40>();
        if (warp == 0 && lane == 0) {
            // ---------------- TMA producer ----------------
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
                const int wrow = __ldcg(g.tile_expert + m_tile) * g.w_rows_per_expert;
                const float* a_sc = g.a_scale_t + static_cast<size_t>(m_tile) * TILE_M;
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    const uint32_t s = it % G_STAGES, ph = (it / G_STAGES) & 1;
                    if (static_cast<int>(it) == g.fault_skip_it) {  // test hook: this stage is never filled
                        ok = false;
                        break;
                    }
                    if (!mbar_wait(smem_u32(&ctrl->done[s]), ph ^ 1, abort_flag, limit)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_PRODUCER);
                        ok = false;
                        break;
                    }
                    const uint32_t bar = smem_u32(&ctrl->full[s]);
                    const uint32_t a_dst = smem_base + s * G_STAGE_BYTES, b_dst = a_dst + G_A_BYTES;
                    const int k0 = kb * G_BLOCK_K;
                    // (the scale slot is free: 8 slots exceed the 4 stages + 2 accumulators the producer can be
                    // ahead of the epilogue)
                    mbar_expect_tx(bar, G_STAGE_BYTES + G_SCALE_BYTES);
                    bulk_load_1d(smem_u32(scale_ring + (it % G_SCALE_RING) * TILE_M),
                                 a_sc + static_cast<size_t>(kb) * g.row_cap, G_SCALE_BYTES, bar);
                    tma_load_2d(a_dst, &tmA, k0, m_tile * TILE_M, bar);
                    if (MODE == 1) {
                        const int gr = wrow + g.gate_row0 + n * 128, ur = wrow + g.up_row0 + n * 128;
                        tma_load_2d(b_dst, &tmB, k0, gr, bar);
                        tma_load_2d(b_dst + G_B_BYTES / 4, &tmB, k0, ur, bar);
                        tma_load_2d(b_dst + G_B_BYTES / 2, &tmB, k0, gr + 64, bar);
                        tma_load_2d(b_dst + 3 * G_B_BYTES / 4, &tmB, k0, ur + 64, bar);
                    } else {
                        const int br = wrow + n * G_TILE_N;
                        tma_load_2d(b_dst, &tmB, k0, br, bar);
                        tma_load_2d(b_dst + G_B_BYTES / 2, &tmB, k0, br + 128, bar);
                    }
                }
            }
            {
                // Before this thread may reach the end of the kernel every copy it issued has to have landed
                // (bounded wait).  On the regular path the MMA issuers have consumed all of them long ago and
                // these waits fall through; after an abort raised by any role they are what keeps the
                // copy engine from writing into shared memory of a CTA that has exited.
                int zero = 0;
                const uint32_t n_back = it < G_STAGES ? it : G_STAGES;
                for (uint32_t j = it - n_back; j < it; ++j)
                    if (!mbar_wait(smem_u32(&ctrl->full[j % G_STAGES]), (j / G_STAGES) & 1, &zero, limit))
                        atomicCAS(g.status, DEV_OK, DEV_TIMEOUT_DRAIN);
            }
        } else if ((warp == 1 || warp == 2) && lane == 0) {
            // ---------------- MMA issuers ----------------
            // Two threads share the issue work: warp 1 takes the even K-blocks (TMEM buffer 0), warp 2 the
            // odd ones (buffer 1).  A commit only tracks the MMAs of its own thread, so while one thread
            // pays for its commit and waits the other keeps the tensor pipe fed.
            const uint32_t idesc = umma_idesc_f8(TILE_M, G_TILE_N);
            const uint32_t mine = warp - 1;
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                for (int kb = 0; kb < num_kb; ++kb, ++it) {
                    if ((it & 1) != mine) continue;
                    const uint32_t s = it % G_STAGES, ph = (it / G_STAGES) & 1;
                    const uint32_t b = it & 1, bph = (it >> 1) & 1;
                    // The stage has normally landed long before the accumulator is handed back, so that
                    // wait comes first and only the hand-over itself is left on the critical path.
                    const uint32_t a_addr = smem_base + s * G_STAGE_BYTES;
                    const uint64_t a_desc = umma_desc_sw128(a_addr);
                    const uint64_t b_desc = umma_desc_sw128(a_addr + G_A_BYTES);
                    const uint32_t d_tmem = tmem_base + b * G_TILE_N;
                    if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, abort_flag, limit)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_MMA_SMEM);
                        ok = false;
                        break;
                    }
                    if (!mbar_wait(smem_u32(&ctrl->tmem_empty[b]), bph ^ 1, abort_flag, limit)) {
                        raise(ctrl, g.status, DEV_TIMEOUT_MMA_TMEM);
                        ok = false;
                        break;
                    }
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < G_BLOCK_K / 32; ++k)  // 32 K-bytes per instruction: +2 in 16-B units
                        umma_f8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k > 0);
                    umma_commit(smem_u32(&ctrl->done[s]));
                }
            }
            if (!ok || *abort_flag) {  // let issued MMAs retire before TMEM is released
                umma_commit(smem_u32(&ctrl->drain_bar[mine]));
                int zero = 0;
                mbar_wait(smem_u32(&ctrl->drain_bar[mine]), 0, &zero, limit);
            }
        }
    } else {
        // ---------------- epilogue warps ----------------
        reg_alloc<232>();
        const int widx = warp - 4;
        const int half = widx >> 2;              // which 128-column half of the tile
        const int quad = warp & 3;               // TMEM lane quadrant this warp may read
        const int r_in_tile = quad * 32 + lane;  // accumulator row == TMEM lane
        const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + half * G_HALF_N;
        const size_t row_cap = static_cast<size_t>(g.row_cap);
        float* amax_x = reinterpret_cast<float*>(store_stage + G_STORE_BYTES);  // [2][2][TILE_M], GEMM1 only
        uint8_t* stage = store_stage + widx * G_STORE_WARP_BYTES;
        uint32_t it = 0, tile_iter = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tile_iter) {
            const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
            const int e = __ldcg(g.tile_expert + m_tile);
            const int rows_valid = __ldcg(g.tile_rows + m_tile);
            const size_t row = static_cast<size_t>(m_tile) * TILE_M + r_in_tile;
            const int sblocks = g.w_rows_per_expert / 128;
            // weight-scale rows of this thread's first / second 64 columns
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

            float s0 = __ldg(ws0), s1 = __ldg(ws1);
            for (int kb = 0; kb < num_kb; ++kb, ++it) {
                const float w0 = s0, w1 = s1;
                if (kb + 1 < num_kb) {
                    s0 = __ldg(ws0 + kb + 1);
                    s1 = __ldg(ws1 + kb + 1);
                }
                const uint32_t s = it % G_STAGES, ph = (it / G_STAGES) & 1, buf = it & 1;
                // Every lane polls (a single polling lane plus a broadcast was measured 2.5 % slower); the vote
                // keeps the warp converged when a wait gives up: either all lanes go on or none does.
                if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctrl->done[s]), ph, abort_flag, limit))) {
                    if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                    ok = false;
                    break;
                }
                tc_fence_after();
                // The MMA of this K-block has finished, hence its stage -- A, B and the scales -- had landed.
                // (Fetching the scale earlier needs a barrier of its own per ring slot -- on full[s] this warp can
                // be lapped by a whole phase -- and that extra barrier test per K-block was measured to cost the
                // epilogue 110 clocks, 10 % of the kernel: barrier operations of a thread queue behind one another.)
                const float sa = ld_shared_f32(scale_ring + (it % G_SCALE_RING) * TILE_M + r_in_tile);
                const float f0 = sa * w0, f1 = sa * w1;
                // GEMM1: of this warpgroup's 128 columns, [0,64) are gate and [64,128) the matching up columns.
                const uint32_t col = t_lane + buf * G_TILE_N;
                float v[64];
                tmem_ld64(col, v);
#pragma unroll
                for (int j = 0; j < 64; ++j) acc[j] = fmaf(v[j], f0, acc[j]);
                tmem_ld64(col + 64, v);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
#pragma unroll
                for (int j = 0; j < 64; ++j) acc[64 + j] = fmaf(v[j], f1, acc[64 + j]);
            }
            if (!ok) break;

            // The staging area of this warp was handed to the TMA engine at the end of the previous tile;
            // by now (a whole tile later) that copy has long read it, so this wait does not stall.
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
            const int sw = (lane >> 1) & 3;  // 64-byte swizzle: 16-byte chunk index ^= bits 7..8 of the address

            if (MODE == 1) {
                // SwiGLU on this thread's 64 columns, then the row's 128-wide amax across the two halves
                float c[64];
                float amax = 0.0f;
#pragma unroll
                for (int j = 0; j < 64; ++j) {
                    // silu(g) * u with the hardware exp2 and reciprocal approximations (a few ulp): the
                    // tile's tail runs while the tensor pipe idles, so its instruction count matters.
                    const float gt = acc[j];
                    c[j] = __fdividef(gt, 1.0f + __expf(-gt)) * acc[64 + j];
                    amax = fmaxf(amax, fabsf(c[j]));
                }
                const uint32_t par = tile_iter & 1;
                amax_x[(par * 2 + half) * TILE_M + r_in_tile] = amax;
                const uint32_t xbar = smem_u32(&ctrl->amax_bar[par]);
                mbar_arrive(xbar);
                if (!__all_sync(0xffffffffu, mbar_wait(xbar, (tile_iter >> 1) & 1, abort_flag, limit))) {
                    if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                    break;
                }
                amax = fmaxf(amax,
                             *reinterpret_cast<volatile float*>(&amax_x[(par * 2 + (half ^ 1)) * TILE_M + r_in_tile]));
                const float sc = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 448.0f);
                const float inv_sc = __frcp_rn(sc);
                if (quad * 32 < rows_valid) {
                    // e4m3 rows out: 32 rows x 64 bytes per warp, staged with the 64-byte swizzle, one TMA store
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int j = q * 16 + i * 4;
                            const uint32_t lo = __nv_cvt_float2_to_fp8x2(
                                make_float2(c[j] * inv_sc, c[j + 1] * inv_sc), __NV_SATFINITE, __NV_E4M3);
                            const uint32_t hi = __nv_cvt_float2_to_fp8x2(
                                make_float2(c[j + 2] * inv_sc, c[j + 3] * inv_sc), __NV_SATFINITE, __NV_E4M3);
                            w[i] = lo | (hi << 16);
                        }
                        *reinterpret_cast<uint4*>(stage + lane * 64 + ((q ^ sw) << 4)) =
                            make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(&tmOut, smem_u32(stage), n * 128 + half * 64, m_tile * TILE_M + quad * 32);
                        bulk_commit_group();
                    }
                    if (half == 0 && r_in_tile < rows_valid)
                        g.out_scale_t[static_cast<size_t>(n) * row_cap + row] = sc;
                }
            } else {
                // bf16 rows out in a tile-blocked layout: block (row tile, column tile, half, quadrant) holds
                // this warp's 32 rows x 128 columns as [8 column groups][32 rows][16 bf16], so every warp
                // store instruction writes 1 KB of contiguous memory (32 bytes per lane).
                if (quad * 32 < rows_valid) {
                    uint8_t* blk = reinterpret_cast<uint8_t*>(g.out_bf16) +
                                   (((static_cast<size_t>(m_tile) * g.n_tiles + n) * 2 + half) * 4 + quad) * 8192 +
                                   lane * 32;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        uint32_t w[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const __nv_bfloat162 pr = __floats2bfloat162_rn(acc[q * 16 + 2 * i], acc[q * 16 + 2 * i + 1]);
                            w[i] = *reinterpret_cast<const uint32_t*>(&pr);
                        }
                        st_global_v8(blk + q * 1024, w);
                    }
                }
            }
        }
        if (lane == 0) bulk_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, G_TMEM_COLS);
    }
}

// Byte offset of the 32-byte group holding columns [16*c16, 16*c16+16) of padded row r in the
// tile-blocked bf16 output of GEMM2 (n_tiles = H / 256 column tiles).
__host__ __device__ __forceinline__ size_t y_block_offset(int r, int c16, int n_tiles) {
    const int m_tile = r / TILE_M, quad = (r % TILE_M) / 32, lane = r % 32;
    const int n = c16 / 16, half = (c16 % 16) / 8, q = c16 % 8;
    return (((static_cast<size_t>(m_tile) * n_tiles + n) * 2 + half) * 4 + quad) * 8192 + q * 1024 + lane * 32;
}

}  // namespace moe

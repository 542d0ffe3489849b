// The front of stage 1 of the Fused MoE description when the layer starts from
// bf16 hidden states: the router projection ("routing scores via a lightweight
// linear projection") and the input-side FP8 quantisation of the activations
// (one fp32 scale per token per 128 columns, scale = amax / 448).
//
// The expert indices selected from the logits are compared bit for bit, so the
// fp32 summation order of the projection is fixed: 32 partial sums, partial l
// takes the l-th pair of every run of 64 elements in increasing order with one
// fused multiply-add per element (bf16 x bf16 is exact in fp32), then five
// pairwise rounds p[l] += p[l xor d], d = 16, 8, 4, 2, 1.  That order is what a
// warp computes naturally: lane l owns partial l and the rounds are butterfly
// shuffles.  It runs on the fp32 pipes, not on the tensor cores, whose
// accumulation order is not specified.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <stdint.h>

#include "ptx.cuh"

namespace moe {

constexpr int RP_KC = 256;   // K elements staged per step (4 runs of 64)
constexpr int RP_MT = 8;     // tokens per warp tile
constexpr int RP_ME = 8;     // experts per warp tile

__host__ __device__ constexpr size_t router_smem_bytes(int WT, int WE) {
    return static_cast<size_t>(2) * (WT * RP_MT + WE * RP_ME) * RP_KC * 2;  // two buffers of bf16 rows
}

// logits[t, e] = sum_h x[t, h] * w[e, h] in the order stated above.  One CTA computes a
// (WT*8 tokens) x (WE*8 experts) tile; warp (wt, we) owns an 8 x 8 block of it with the K dimension
// spread over its lanes.  x [T, H] and w [E, H] bf16, H a multiple of 256, E a multiple of WE*8.
template <int WT, int WE>
__global__ void __launch_bounds__(WT * WE * 32)
router_logits_kernel(int T, int H, int E, const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                     float* __restrict__ logits) {
    extern __shared__ __align__(16) uint8_t rp_smem[];
    constexpr int ROWS_T = WT * RP_MT, ROWS_E = WE * RP_ME, ROWS = ROWS_T + ROWS_E;
    constexpr int THREADS = WT * WE * 32;
    constexpr int CHUNKS_PER_ROW = RP_KC * 2 / 16;                 // 16-byte chunks of one staged row
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wt = warp / WE, we = warp % WE;
    const int t0 = blockIdx.x * ROWS_T, e0 = blockIdx.y * ROWS_E;
    const uint32_t smem0 = smem_u32(rp_smem);

    // stage K-chunk kc of the tile's rows (tokens first, then experts) into buffer b; rows past T read as zero
    auto stage = [&](int kc, int b) {
        for (int c = tid; c < ROWS * CHUNKS_PER_ROW; c += THREADS) {
            const int r = c / CHUNKS_PER_ROW, cc = c % CHUNKS_PER_ROW;
            const __nv_bfloat16* src;
            uint32_t bytes = 16;
            if (r < ROWS_T) {
                const int t = t0 + r;
                if (t >= T) bytes = 0;
                src = x + static_cast<size_t>(t < T ? t : 0) * H + kc * RP_KC + cc * 8;
            } else {
                src = w + static_cast<size_t>(e0 + r - ROWS_T) * H + kc * RP_KC + cc * 8;
            }
            cp_async_16(smem0 + (b * ROWS + r) * (RP_KC * 2) + cc * 16, src, bytes);
        }
        cp_async_commit();
    };

    // Accumulators as pairs of tokens (2 i, 2 i + 1) for the packed fp32 FMA: one instruction, two independent
    // round-to-nearest FMAs, so every sum is bit for bit the one of the scalar form.
    uint64_t acc2[RP_MT / 2][RP_ME];
#pragma unroll
    for (int i = 0; i < RP_MT / 2; ++i)
#pragma unroll
        for (int j = 0; j < RP_ME; ++j) acc2[i][j] = 0ull;

    const int nkc = H / RP_KC;
    stage(0, 0);
    for (int kc = 0; kc < nkc; ++kc) {
        const int b = kc & 1;
        if (kc + 1 < nkc) {
            stage(kc + 1, b ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        const uint8_t* xb = rp_smem + (b * ROWS + wt * RP_MT) * (RP_KC * 2) + lane * 4;
        const uint8_t* wb = rp_smem + (b * ROWS + ROWS_T + we * RP_ME) * (RP_KC * 2) + lane * 4;
#pragma unroll
        for (int run = 0; run < RP_KC / 64; ++run) {
            uint64_t xl2[RP_MT / 2], xh2[RP_MT / 2];  // elements 2l / 2l+1 of the run for two tokens each
#pragma unroll
            for (int i = 0; i < RP_MT / 2; ++i) {
                const uint32_t u0 = *reinterpret_cast<const uint32_t*>(xb + (2 * i) * (RP_KC * 2) + run * 128);
                const uint32_t u1 = *reinterpret_cast<const uint32_t*>(xb + (2 * i + 1) * (RP_KC * 2) + run * 128);
                xl2[i] = pack_f32x2(u0 << 16, u1 << 16);
                xh2[i] = pack_f32x2(u0 & 0xffff0000u, u1 & 0xffff0000u);
            }
#pragma unroll
            for (int j = 0; j < RP_ME; ++j) {
                const uint32_t u = *reinterpret_cast<const uint32_t*>(wb + j * (RP_KC * 2) + run * 128);
                const uint64_t wl2 = pack_f32x2(u << 16, u << 16), wh2 = pack_f32x2(u & 0xffff0000u, u & 0xffff0000u);
#pragma unroll
                for (int i = 0; i < RP_MT / 2; ++i) acc2[i][j] = fma_f32x2(xl2[i], wl2, acc2[i][j]);  // element 2l of the run
#pragma unroll
                for (int i = 0; i < RP_MT / 2; ++i) acc2[i][j] = fma_f32x2(xh2[i], wh2, acc2[i][j]);  // then element 2l+1
            }
        }
        __syncthreads();  // the buffer is refilled two steps from now
    }
    float acc[RP_MT][RP_ME];
#pragma unroll
    for (int i = 0; i < RP_MT / 2; ++i)
#pragma unroll
        for (int j = 0; j < RP_ME; ++j) {
            acc[2 * i][j] = __uint_as_float(static_cast<uint32_t>(acc2[i][j]));
            acc[2 * i + 1][j] = __uint_as_float(static_cast<uint32_t>(acc2[i][j] >> 32));
        }

    // five pairwise rounds; afterwards every lane holds every logit of the warp tile
#pragma unroll
    for (int i = 0; i < RP_MT; ++i)
#pragma unroll
        for (int j = 0; j < RP_ME; ++j) {
            float v = acc[i][j];
#pragma unroll
            for (int d = 16; d >= 1; d >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, d));
            acc[i][j] = v;
        }
    // lane l stores the logits of token (l >> 2) for experts 2 (l & 3), 2 (l & 3) + 1
#pragma unroll
    for (int i = 0; i < RP_MT; ++i)
#pragma unroll
        for (int j = 0; j < RP_ME; j += 2)
            if (lane == i * 4 + j / 2) {
                const int t = t0 + wt * RP_MT + i;
                if (t < T)
                    *reinterpret_cast<float2*>(logits + static_cast<size_t>(t) * E + e0 + we * RP_ME + j) =
                        make_float2(acc[i][j], acc[i][j + 1]);
            }
}

// One warp per (token, 128-column block): amax, scale = amax / 448 (1 for an all-zero block), codes =
// e4m3(x / scale) with IEEE division, round to nearest even, saturating.  scale_layout 0: [T, H/128], 1: [H/128, T].
__global__ void __launch_bounds__(256) quantize_rows_kernel(int T, int H, int scale_layout,
                                                            const __nv_bfloat16* __restrict__ x,
                                                            uint8_t* __restrict__ q, float* __restrict__ scale) {
    const int lane = threadIdx.x & 31;
    const int nb = H / 128;
    const long long nblocks = static_cast<long long>(T) * nb;
    const long long warp0 = static_cast<long long>(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long long nwarps = static_cast<long long>(gridDim.x) * (blockDim.x >> 5);
    for (long long blk = warp0; blk < nblocks; blk += nwarps) {
        const long long t = blk / nb;
        const int b = static_cast<int>(blk - t * nb);
        const uint2 raw = *reinterpret_cast<const uint2*>(x + t * H + b * 128 + lane * 4);
        const float v0 = __uint_as_float(raw.x << 16), v1 = __uint_as_float(raw.x & 0xffff0000u);
        const float v2 = __uint_as_float(raw.y << 16), v3 = __uint_as_float(raw.y & 0xffff0000u);
        float amax = fmaxf(fmaxf(fabsf(v0), fabsf(v1)), fmaxf(fabsf(v2), fabsf(v3)));
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, d));
        const float sc = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 448.0f);
        const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(v0, sc), __fdiv_rn(v1, sc)),
                                                     __NV_SATFINITE, __NV_E4M3);
        const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(v2, sc), __fdiv_rn(v3, sc)),
                                                     __NV_SATFINITE, __NV_E4M3);
        *reinterpret_cast<uint32_t*>(q + t * H + b * 128 + lane * 4) = lo | (hi << 16);
        if (lane == 0) scale[scale_layout ? static_cast<long long>(b) * T + t : t * nb + b] = sc;
    }
}

}  // namespace moe

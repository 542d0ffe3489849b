// Stage 1 of the Fused MoE description: sigmoid scores, group-wise top-2 to
// score each of 8 groups, keep the 4 best groups, select the 8 best experts,
// weights = unbiased score / sum * scaling factor.  One warp per token.
//
// Every fp32 operation is spelled with a round-to-nearest intrinsic so the
// compiler cannot contract or reassociate: selected indices must be
// reproducible bit for bit.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "ptx.cuh"

namespace moe {

constexpr int R_EXPERTS = 256;  // global experts
constexpr int R_GROUPS = 8;     // groups of 32 consecutive experts
constexpr int R_TOPK_GROUP = 4;
constexpr int R_TOPK = 8;

// exp(x) in fp32, fixed operation by operation: clamp to [-87, 88];
// n = rint(x*log2e); r = x - n*ln2 (two-part ln2, fused); degree-7 Taylor
// polynomial by Horner with fused multiply-adds; times 2^n via the exponent field.
__device__ __forceinline__ float exp_fixed(float x) {
    x = fminf(fmaxf(x, -87.0f), 88.0f);
    const float n = rintf(__fmul_rn(x, __uint_as_float(0x3fb8aa3bu)));
    float r = __fmaf_rn(n, __uint_as_float(0xbf317200u), x);
    r = __fmaf_rn(n, __uint_as_float(0xb5bfbe8eu), r);
    float p = __uint_as_float(0x39500d01u);
    p = __fmaf_rn(p, r, __uint_as_float(0x3ab60b61u));
    p = __fmaf_rn(p, r, __uint_as_float(0x3c088889u));
    p = __fmaf_rn(p, r, __uint_as_float(0x3d2aaaabu));
    p = __fmaf_rn(p, r, __uint_as_float(0x3e2aaaabu));
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float two_n = __uint_as_float(static_cast<uint32_t>(static_cast<int>(n) + 127) << 23);
    return __fmul_rn(p, two_n);
}

__device__ __forceinline__ float sigmoid_fixed(float x) {
    return __fdiv_rn(1.0f, __fadd_rn(1.0f, exp_fixed(-x)));
}

// Monotone map fp32 -> uint32 (larger float <=> larger key); every finite key is > 0.
__device__ __forceinline__ uint32_t order_key(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Bias of the 8 experts a lane owns (lane l owns experts 8l .. 8l+7, so a group of 32 experts is 4
// neighbouring lanes), bf16 -> fp32.
__device__ __forceinline__ void load_bias8(const __nv_bfloat16* __restrict__ bias, int lane, float (&bias_f)[8]) {
    const uint4 braw = reinterpret_cast<const uint4*>(bias)[lane];
    const uint32_t w[4] = {braw.x, braw.y, braw.z, braw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        bias_f[2 * i] = __uint_as_float(w[i] << 16);
        bias_f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// Routes token t with one warp.  Lane j < 8 returns the j-th selected expert and its weight.
__device__ __forceinline__ void route_token(int t, int lane, const float* __restrict__ logits,
                                            const float (&bias_f)[8], float scaling, int& my_idx, float& my_w) {
    const float4* row = reinterpret_cast<const float4*>(logits + static_cast<size_t>(t) * R_EXPERTS);
    const float4 x0 = __ldg(row + 2 * lane), x1 = __ldg(row + 2 * lane + 1);
    const float x[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
    float sig[8], b[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        sig[i] = sigmoid_fixed(x[i]);
        b[i] = __fadd_rn(sig[i], bias_f[i]);
    }
    // two largest biased scores of my 8, then of the 4 lanes of my group
    float m1 = fmaxf(b[0], b[1]), m2 = fminf(b[0], b[1]);
#pragma unroll
    for (int i = 2; i < 8; ++i) {
        m2 = fmaxf(m2, fminf(m1, b[i]));
        m1 = fmaxf(m1, b[i]);
    }
#pragma unroll
    for (int d = 1; d <= 2; d <<= 1) {
        const float o1 = __shfl_xor_sync(0xffffffffu, m1, d);
        const float o2 = __shfl_xor_sync(0xffffffffu, m2, d);
        m2 = fmaxf(fminf(m1, o1), fmaxf(m2, o2));
        m1 = fmaxf(m1, o1);
    }
    const float gs = __fadd_rn(m1, m2);
    // rank of my group among the 8 (ties to the smaller group index)
    const int g = lane >> 2;
    int better = 0;
#pragma unroll
    for (int o = 0; o < R_GROUPS; ++o) {
        const float v = __shfl_sync(0xffffffffu, gs, o * 4);
        better += (v > gs) || (v == gs && o < g);
    }
    const bool kept = better < R_TOPK_GROUP;

    // 8 rounds of warp arg-max over the kept experts (ties to the smaller index)
    uint32_t key[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) key[i] = kept ? order_key(b[i]) : 0u;
    int sel_idx[R_TOPK];
    float sel_sig[R_TOPK];
#pragma unroll
    for (int j = 0; j < R_TOPK; ++j) {
        uint32_t bk = key[0];
        int bi = 0;
#pragma unroll
        for (int i = 1; i < 8; ++i)
            if (key[i] > bk) {
                bk = key[i];
                bi = i;
            }
        const uint32_t wk = __reduce_max_sync(0xffffffffu, bk);
        const uint32_t cand = (bk == wk) ? static_cast<uint32_t>(lane * 8 + bi) : 0xffffffffu;
        const int win = static_cast<int>(__reduce_min_sync(0xffffffffu, cand));
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (i == (win & 7)) s = sig[i];
        sel_sig[j] = __shfl_sync(0xffffffffu, s, win >> 3);
        sel_idx[j] = win;
        if (lane == (win >> 3)) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (i == (win & 7)) key[i] = 0u;
        }
    }
    float den = 0.0f;
#pragma unroll
    for (int j = 0; j < R_TOPK; ++j) den = __fadd_rn(den, sel_sig[j]);
    my_idx = 0;
    my_w = 0.0f;
#pragma unroll
    for (int j = 0; j < R_TOPK; ++j)
        if (lane == j) {
            my_idx = sel_idx[j];
            my_w = __fmul_rn(__fdiv_rn(sel_sig[j], den), scaling);
        }
}

__global__ void __launch_bounds__(256) route_topk_kernel(int T, const float* __restrict__ logits,
                                                         const __nv_bfloat16* __restrict__ bias, float scaling,
                                                         int* __restrict__ topk_idx, float* __restrict__ topk_w,
                                                         int* __restrict__ status) {
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) *status = DEV_OK;  // first kernel of a forward: clear the fault word
    const int lane = threadIdx.x & 31;
    const int warps_per_block = blockDim.x >> 5;
    const int warp0 = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
    const int nwarps = gridDim.x * warps_per_block;
    float bias_f[8];
    load_bias8(bias, lane, bias_f);
    for (int t = warp0; t < T; t += nwarps) {
        int my_idx;
        float my_w;
        route_token(t, lane, logits, bias_f, scaling, my_idx, my_w);
        if (lane < R_TOPK) {
            topk_idx[static_cast<size_t>(t) * R_TOPK + lane] = my_idx;
            topk_w[static_cast<size_t>(t) * R_TOPK + lane] = my_w;
        }
    }
}

}  // namespace moe

// Stage 4 of the Fused MoE description: bring the expert outputs back to token
// order, weighted by the routing weights.  One block per token pulls the
// token's (at most 8) bf16 rows in routing order, accumulates in fp32 and
// rounds once to bf16; tokens without a local expert are written as zeros.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "gemm.cuh"
#include "ptx.cuh"

namespace moe {

// y is the tile-blocked bf16 output of GEMM2 (see y_block_offset); each thread owns 16 columns
// (one 32-byte group) of one token.
__global__ void __launch_bounds__(256) combine_kernel(int T, int H, const int* slot_to_row, const float* topk_w,
                                                      const uint8_t* y,
                                                      __nv_bfloat16* __restrict__ out) {
    pdl_launch_dependents();
    pdl_wait();
    const int groups = H / 16, n_tiles = H / 256;
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        int rows[8];
        float w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            rows[j] = __ldcg(slot_to_row + t * 8 + j);  // written by the kernels before this one: coherent loads
            w[j] = __ldcg(topk_w + t * 8 + j);
        }
        for (int c = threadIdx.x; c < groups; c += blockDim.x) {
            float acc[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (rows[j] < 0) continue;
                uint32_t u[8];
                ld_global_v8(y + y_block_offset(rows[j], c, n_tiles), u);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    acc[2 * i] = fmaf(w[j], __uint_as_float(u[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = fmaf(w[j], __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
            uint32_t o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const __nv_bfloat162 p = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
                o[i] = *reinterpret_cast<const uint32_t*>(&p);
            }
            uint4* dst = reinterpret_cast<uint4*>(out + static_cast<size_t>(t) * H + c * 16);  // 16-byte aligned
            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
    }
}

}  // namespace moe

// Stage 4 of the Fused MoE description: bring the expert outputs back to token
// order, weighted by the routing weights.  One block per token pulls the
// token's (at most 8) bf16 rows in routing order, accumulates in fp32 and
// rounds once to bf16; tokens without a local expert are written as zeros.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace moe {

__global__ void __launch_bounds__(256) combine_kernel(int T, int H, const int* __restrict__ slot_to_row,
                                                      const float* __restrict__ topk_w,
                                                      const __nv_bfloat16* __restrict__ y,
                                                      __nv_bfloat16* __restrict__ out) {
    const int chunks = H / 8;  // 8 bf16 = 16 bytes
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        int rows[8];
        float w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            rows[j] = __ldg(slot_to_row + t * 8 + j);
            w[j] = __ldg(topk_w + t * 8 + j);
        }
        for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (rows[j] < 0) continue;
                const uint4 raw = __ldg(reinterpret_cast<const uint4*>(y + static_cast<size_t>(rows[j]) * H) + c);
                const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[2 * i] = fmaf(w[j], __uint_as_float(u[i] << 16), acc[2 * i]);
                    acc[2 * i + 1] = fmaf(w[j], __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
                }
            }
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const __nv_bfloat162 p = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
                o[i] = *reinterpret_cast<const uint32_t*>(&p);
            }
            reinterpret_cast<uint4*>(out + static_cast<size_t>(t) * H)[c] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

}  // namespace moe

// moe_fp8_expert_histogram_static: the per-expert histogram + exclusive scan of the permutation stage for
// callers that cannot allocate device memory.  Its scratch (per-block partial counts) lives in a file-scope
// device array of fixed size instead of a caller-provided workspace.
#include "../../include/moe_fp8.h"

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "limits.cuh"

namespace {

using moe::P_MAX_LOCAL;
using moe::P_TOKENS_PER_BLOCK;

constexpr int STATIC_MAX_BLOCKS =
    (MOE_FP8_STATIC_HISTOGRAM_MAX_TOKENS + P_TOKENS_PER_BLOCK - 1) / P_TOKENS_PER_BLOCK;

// Per-block partial histograms: [STATIC_MAX_BLOCKS][P_MAX_LOCAL] int32 = 64 KB, resident on every GPU that
// loads the library until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress; the device address is looked up once per device below.
static __device__ __align__(256) int g_block_hist[STATIC_MAX_BLOCKS * P_MAX_LOCAL];
static_assert(STATIC_MAX_BLOCKS * P_MAX_LOCAL * sizeof(int) == 65536, "the documented size of the fixed scratch");

constexpr int MAX_DEVICES = 64;
int* g_block_hist_addr[MAX_DEVICES] = {};
std::mutex g_setup_mutex;

// Variant of the permutation stage's counting kernel: bit t of mask[e] says that token t of this block routes
// to local expert e; the popcounts are the block's partial histogram, written to the static scratch.
__global__ void __launch_bounds__(P_TOKENS_PER_BLOCK) count_static_kernel(int T, int E_loc, int off,
                                                                          const int* __restrict__ topk_idx,
                                                                          int* __restrict__ block_hist) {
    __shared__ uint32_t mask[P_MAX_LOCAL][P_TOKENS_PER_BLOCK / 32];
    for (int i = threadIdx.x; i < E_loc * (P_TOKENS_PER_BLOCK / 32); i += blockDim.x) (&mask[0][0])[i] = 0u;
    __syncthreads();
    const int t = blockIdx.x * P_TOKENS_PER_BLOCK + threadIdx.x;
    if (t < T) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = topk_idx[t * 8 + j] - off;
            if (e >= 0 && e < E_loc) atomicOr(&mask[e][threadIdx.x >> 5], 1u << (threadIdx.x & 31));
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E_loc; e += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < P_TOKENS_PER_BLOCK / 32; ++w) c += __popc(mask[e][w]);
        block_hist[blockIdx.x * E_loc + e] = c;
    }
}

// One block; thread e sums the per-block counts of local expert e, then an exclusive scan over the experts.
__global__ void __launch_bounds__(P_MAX_LOCAL) scan_counts_kernel(int nblk, int E_loc, const int* __restrict__ block_hist,
                                                                  int* __restrict__ expert_count,
                                                                  int* __restrict__ expert_offset) {
    __shared__ int s_cnt[P_MAX_LOCAL];
    const int e = threadIdx.x;
    int total = 0;
    if (e < E_loc)
        for (int b = 0; b < nblk; ++b) total += block_hist[b * E_loc + e];
    s_cnt[e] = total;
    __syncthreads();
    if (e < E_loc) {
        int before = 0;
        for (int i = 0; i < e; ++i) before += s_cnt[i];
        expert_count[e] = total;
        expert_offset[e] = before;
        if (e == E_loc - 1) expert_offset[E_loc] = before + total;
    }
}

}  // namespace

extern "C" int moe_fp8_expert_histogram_static(int T, const int* topk_idx, int local_expert_offset,
                                               int num_local_experts, int* expert_count, int* expert_offset,
                                               void* stream_v) {
    if (T < 0 || num_local_experts <= 0 || num_local_experts > P_MAX_LOCAL || local_expert_offset < 0 ||
        local_expert_offset + num_local_experts > 256 || !expert_count || !expert_offset || (T > 0 && !topk_idx))
        return MOE_FP8_ERR_BAD_ARG;
    if (T > MOE_FP8_STATIC_HISTOGRAM_MAX_TOKENS) return MOE_FP8_ERR_STATIC_LIMIT;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return MOE_FP8_ERR_CUDA;
    int* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_block_hist_addr[dev]) {  // first call on this device: resolve the device address of the array
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_block_hist) != cudaSuccess || !p) return MOE_FP8_ERR_CUDA;
            g_block_hist_addr[dev] = static_cast<int*>(p);
        }
        scratch = g_block_hist_addr[dev];
    }

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int nblk = (T + P_TOKENS_PER_BLOCK - 1) / P_TOKENS_PER_BLOCK;
    // Every scratch entry the scan reads ([0, nblk) x [0, E_loc)) is written by count_static_kernel in this same call,
    // so nothing left behind by an earlier call can be seen and nothing needs zeroing.
    if (nblk > 0)
        count_static_kernel<<<nblk, P_TOKENS_PER_BLOCK, 0, stream>>>(T, num_local_experts, local_expert_offset,
                                                                    topk_idx, scratch);
    scan_counts_kernel<<<1, P_MAX_LOCAL, 0, stream>>>(nblk, num_local_experts, scratch, expert_count, expert_offset);
    return cudaGetLastError() == cudaSuccess ? MOE_FP8_OK : MOE_FP8_ERR_CUDA;
}

// Stage 2 of the Fused MoE description: per-expert histogram, exclusive scan,
// stable placement of the local (token, expert) slots into expert-contiguous
// rows (experts ascending, tokens ascending inside an expert), and the gather
// of FP8 activation rows and their 128-wide scales into that order.  All
// metadata stays on the device; nothing here synchronises with the host.
//
// Row numbering: "canonical" rows are dense (expert e starts at offset[e]);
// "padded" rows start every expert on a multiple of the GEMM tile height so a
// tile never straddles two experts.
#pragma once
#include <stdint.h>

#include "limits.cuh"
#include "ptx.cuh"
#include "routing.cuh"

namespace moe {

constexpr int TILE_M = 128;              // GEMM tile height (rows)

struct PermuteMeta {
    int* block_hist;     // [nblk, E_loc] per-block counts, turned into per-block bases by the scan
    int* expert_count;   // [E_loc]
    int* expert_offset;  // [E_loc+1] canonical (unpadded) exclusive scan
    int* padded_offset;  // [E_loc+1] exclusive scan of counts rounded up to TILE_M
    int* tile_expert;    // [max_m_tiles] local expert of each row tile
    int* tile_rows;      // [max_m_tiles] valid rows in each row tile (1..TILE_M)
    int* num_m_tiles;    // [1]
    int* slot_to_row;    // [T*8] padded row of each slot, -1 when the slot's expert is not local
    int* row_to_slot;    // [T*8] canonical row -> slot id (first S entries valid)
    int* row_token;      // [row_cap] padded row -> token (valid rows only)
    int* tok_nlocal;     // [T] local slots of each token (small batches only: route_permute_kernel / _in_cta)
    // small batches only, for the fused kernel: the row tiles cut into sub-tiles of at most 32 rows
    int* st_expert;      // [max sub-tiles] local expert
    int* st_row0;        // [max sub-tiles] first padded row (a multiple of 32)
    int* st_rows;        // [max sub-tiles] valid rows (1..32)
    int* num_st;         // [1]
};
constexpr int ST_ROWS = 32;

// Bit t of mask[e] says: token t of this block routes to local expert e.  The
// popcount below a token's bit is its stable rank inside the block.
// topk_idx was written by the kernel before this one, which may still be resident (programmatic dependent
// launch): it is read with coherent (.cg) loads, never through the read-only path.
__device__ __forceinline__ void build_block_masks(uint32_t (*mask)[P_TOKENS_PER_BLOCK / 32], int T, int E_loc,
                                                  int off, const int* topk_idx) {
    for (int i = threadIdx.x; i < E_loc * (P_TOKENS_PER_BLOCK / 32); i += blockDim.x)
        (&mask[0][0])[i] = 0u;
    __syncthreads();
    const int t = blockIdx.x * P_TOKENS_PER_BLOCK + threadIdx.x;
    if (t < T) {
        const int4 a = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t);
        const int4 b = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t + 1);
        const int ids[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = ids[j] - off;
            if (e >= 0 && e < E_loc) atomicOr(&mask[e][threadIdx.x >> 5], 1u << (threadIdx.x & 31));
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(P_TOKENS_PER_BLOCK) count_kernel(int T, int E_loc, int off,
                                                                   const int* topk_idx,
                                                                   int* __restrict__ block_hist) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ uint32_t mask[P_MAX_LOCAL][P_TOKENS_PER_BLOCK / 32];
    build_block_masks(mask, T, E_loc, off, topk_idx);
    for (int e = threadIdx.x; e < E_loc; e += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < P_TOKENS_PER_BLOCK / 32; ++w) c += __popc(mask[e][w]);
        block_hist[blockIdx.x * E_loc + e] = c;
    }
}

// One block.  Thread e owns local expert e.
__global__ void __launch_bounds__(P_MAX_LOCAL) scan_kernel(int nblk, int E_loc, PermuteMeta m) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int s_cnt[P_MAX_LOCAL + 1];
    __shared__ int s_pad[P_MAX_LOCAL + 1];
    const int e = threadIdx.x;
    int total = 0;
    if (e < E_loc) {
        for (int b = 0; b < nblk; ++b) {
            const int c = m.block_hist[b * E_loc + e];
            m.block_hist[b * E_loc + e] = total;  // base of block b inside expert e
            total += c;
        }
    }
    s_cnt[e] = (e < E_loc) ? total : 0;
    s_pad[e] = (e < E_loc) ? (total + TILE_M - 1) / TILE_M * TILE_M : 0;
    __syncthreads();
    if (threadIdx.x == 0) {  // 256 entries: a serial scan is a few hundred cycles
        int a = 0, p = 0;
        for (int i = 0; i < E_loc; ++i) {
            const int c = s_cnt[i], q = s_pad[i];
            s_cnt[i] = a;
            s_pad[i] = p;
            a += c;
            p += q;
        }
        s_cnt[E_loc] = a;
        s_pad[E_loc] = p;
        *m.num_m_tiles = p / TILE_M;
    }
    __syncthreads();
    if (e < E_loc) {
        m.expert_count[e] = total;
        m.expert_offset[e] = s_cnt[e];
        m.padded_offset[e] = s_pad[e];
        const int t0 = s_pad[e] / TILE_M;
        for (int i = 0; i * TILE_M < total; ++i) {
            m.tile_expert[t0 + i] = e;
            m.tile_rows[t0 + i] = min(TILE_M, total - i * TILE_M);
        }
    }
    if (e == 0) {
        m.expert_offset[E_loc] = s_cnt[E_loc];
        m.padded_offset[E_loc] = s_pad[E_loc];
    }
}

__global__ void __launch_bounds__(P_TOKENS_PER_BLOCK) place_kernel(int T, int E_loc, int off, int row_cap,
                                                                   const int* topk_idx, PermuteMeta m,
                                                                   int* __restrict__ status) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ uint32_t mask[P_MAX_LOCAL][P_TOKENS_PER_BLOCK / 32];
    build_block_masks(mask, T, E_loc, off, topk_idx);
    const int t = blockIdx.x * P_TOKENS_PER_BLOCK + threadIdx.x;
    if (t >= T) return;
    const int word = threadIdx.x >> 5, bit = threadIdx.x & 31;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int e = __ldcg(topk_idx + t * 8 + j) - off;
        int prow = -1;
        if (e >= 0 && e < E_loc) {
            int rank = __popc(mask[e][word] & ((1u << bit) - 1u));
            for (int w = 0; w < word; ++w) rank += __popc(mask[e][w]);
            const int within = m.block_hist[blockIdx.x * E_loc + e] + rank;
            prow = m.padded_offset[e] + within;
            if (prow < 0 || prow >= row_cap) {
                atomicExch(status, DEV_BAD_ROW);
                prow = -1;
            } else {
                m.row_to_slot[m.expert_offset[e] + within] = t * 8 + j;
                m.row_token[prow] = t;
            }
        }
        m.slot_to_row[t * 8 + j] = prow;
    }
}

// Batches up to P_TAIL_MAX_TOKENS: routing in parallel blocks (one warp per token), then the block that
// finishes last -- found with a ticket counter, nobody waits -- builds histogram, scan and placement for all
// tokens on its own.  One launch instead of four; same arithmetic and outputs as route_topk_kernel +
// count_kernel + scan_kernel + place_kernel.  `ticket` must be zero at launch; the last block leaves it zero
// (moe_fp8_set_workspace zeroes it once, nothing else ever writes it).
// Dynamic shared memory: E_loc * ceil(T/32) words of masks, then as many 16-bit prefix counts.
constexpr int P_TAIL_MAX_TOKENS = 512;   // measured faster than the four kernels up to here, slower at 1024
constexpr int P_TAIL_THREADS = 256;
__host__ __device__ constexpr size_t route_permute_smem_bytes(int T, int E_loc) {
    return static_cast<size_t>(E_loc) * ((T + 31) / 32) * 6;
}
__global__ void __launch_bounds__(P_TAIL_THREADS) route_permute_kernel(
    int T, int E_loc, int off, int row_cap, const float* __restrict__ logits, const __nv_bfloat16* __restrict__ bias,
    float scaling, int* __restrict__ topk_idx, float* __restrict__ topk_w, PermuteMeta m, int* __restrict__ ticket,
    int* __restrict__ status) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ uint32_t dyn_smem[];
    __shared__ int s_cnt[P_MAX_LOCAL + 1];
    __shared__ int s_pad[P_MAX_LOCAL + 1];
    __shared__ int s_st[P_MAX_LOCAL + 1];
    __shared__ int s_last;
    const int tid = threadIdx.x, lane = tid & 31;
    if (blockIdx.x == 0 && tid == 0) *status = DEV_OK;  // first kernel of a forward: clear the fault word
    {   // stage 1: one warp per token
        const int warps_per_block = blockDim.x >> 5;
        const int nwarps = gridDim.x * warps_per_block;
        float bias_f[8];
        load_bias8(bias, lane, bias_f);
        for (int t = blockIdx.x * warps_per_block + (tid >> 5); t < T; t += nwarps) {
            int my_idx;
            float my_w;
            route_token(t, lane, logits, bias_f, scaling, my_idx, my_w);
            if (lane < R_TOPK) {
                topk_idx[static_cast<size_t>(t) * R_TOPK + lane] = my_idx;
                topk_w[static_cast<size_t>(t) * R_TOPK + lane] = my_w;
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int n = atomicAdd(ticket, 1);
        s_last = (n == static_cast<int>(gridDim.x) - 1);
        if (s_last) *ticket = 0;
        // A counter that did not start at zero (somebody wrote into the workspace) would leave this forward
        // without a last block and with stale tables: say so instead of returning them silently.
        if (n < 0 || n >= static_cast<int>(gridDim.x)) {
            atomicExch(status, DEV_BAD_TICKET);
            *ticket = 0;
        }
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    // stage 2 for all tokens, in this block.  Bit t of mask[e] says: token t routes to local expert e.
    const int W = (T + 31) / 32;
    uint32_t* mask = dyn_smem;                                             // [E_loc][W]
    uint16_t* pre = reinterpret_cast<uint16_t*>(dyn_smem + E_loc * W);     // [E_loc][W] tokens of e below word w
    for (int i = tid; i < E_loc * W; i += blockDim.x) mask[i] = 0u;
    __syncthreads();
    for (int t = tid; t < T; t += blockDim.x) {
        const int4 a = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t);
        const int4 b = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t + 1);
        const int ids[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = ids[j] - off;
            if (e >= 0 && e < E_loc) atomicOr(&mask[e * W + (t >> 5)], 1u << (t & 31));
        }
    }
    __syncthreads();
    int total = 0;
    for (int e = tid; e < P_MAX_LOCAL; e += blockDim.x) {
        total = 0;
        if (e < E_loc)
            for (int w = 0; w < W; ++w) {
                pre[e * W + w] = static_cast<uint16_t>(total);
                total += __popc(mask[e * W + w]);
            }
        s_cnt[e] = total;
        s_pad[e] = (total + TILE_M - 1) / TILE_M * TILE_M;
    }
    __syncthreads();
    if (tid == 0) {  // 256 entries: a serial scan is a few hundred cycles
        int a = 0, p = 0, st = 0;
        for (int i = 0; i < E_loc; ++i) {
            const int c = s_cnt[i], q = s_pad[i];
            s_cnt[i] = a;
            s_pad[i] = p;
            s_st[i] = st;
            a += c;
            p += q;
            st += (c + ST_ROWS - 1) / ST_ROWS;
        }
        s_cnt[E_loc] = a;
        s_pad[E_loc] = p;
        *m.num_m_tiles = p / TILE_M;
        *m.num_st = st;
        m.expert_offset[E_loc] = a;
        m.padded_offset[E_loc] = p;
    }
    __syncthreads();
    for (int e = tid; e < E_loc; e += blockDim.x) {  // blockDim == P_MAX_LOCAL: `total` is still expert e's count
        m.expert_count[e] = total;
        m.expert_offset[e] = s_cnt[e];
        m.padded_offset[e] = s_pad[e];
        const int t0 = s_pad[e] / TILE_M;
        for (int i = 0; i * TILE_M < total; ++i) {
            m.tile_expert[t0 + i] = e;
            m.tile_rows[t0 + i] = min(TILE_M, total - i * TILE_M);
        }
        for (int i = 0; i * ST_ROWS < total; ++i) {
            m.st_expert[s_st[e] + i] = e;
            m.st_row0[s_st[e] + i] = s_pad[e] + i * ST_ROWS;
            m.st_rows[s_st[e] + i] = min(ST_ROWS, total - i * ST_ROWS);
        }
    }
    for (int t = tid; t < T; t += blockDim.x) {
        const int4 a = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t);
        const int4 b = __ldcg(reinterpret_cast<const int4*>(topk_idx) + 2 * t + 1);
        const int ids[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        const int word = t >> 5, bit = t & 31;
        int nlocal = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = ids[j] - off;
            int prow = -1;
            if (e >= 0 && e < E_loc) {
                ++nlocal;
                const int rank = pre[e * W + word] + __popc(mask[e * W + word] & ((1u << bit) - 1u));
                prow = s_pad[e] + rank;
                if (prow < 0 || prow >= row_cap) {
                    atomicExch(status, DEV_BAD_ROW);
                    prow = -1;
                } else {
                    m.row_to_slot[s_cnt[e] + rank] = t * 8 + j;
                    m.row_token[prow] = t;
                }
            }
            m.slot_to_row[t * 8 + j] = prow;
        }
        m.tok_nlocal[t] = nlocal;
    }
}
static_assert(P_TAIL_THREADS == P_MAX_LOCAL, "the tail keeps one expert's count per thread");
static_assert(TILE_M % ST_ROWS == 0, "sub-tiles do not straddle row tiles");

// Stages 1 and 2 for a batch of at most 32 tokens, computed by ONE thread block for itself: every CTA of the
// fused small-batch kernel runs this on the same inputs and writes the same tables (to the same addresses, with
// the same values), so no CTA ever waits for another one and no separate routing launch is needed.  Same
// arithmetic and outputs as route_permute_kernel.  `scratch` is RP_CTA_SCRATCH_INTS ints of shared memory;
// the block needs at least P_MAX_LOCAL threads and T warps are busy at a time.  Ends with a block barrier after
// which every thread of the block may read the tables.
constexpr int RP_CTA_MAX_TOKENS = 32;
constexpr int RP_CTA_SCRATCH_INTS = RP_CTA_MAX_TOKENS * 8 + P_MAX_LOCAL + 2 * (P_MAX_LOCAL + 1);
__device__ __forceinline__ void route_permute_in_cta(int* scratch, int T, int E_loc, int off, int row_cap,
                                                     const float* __restrict__ logits,
                                                     const __nv_bfloat16* __restrict__ bias, float scaling,
                                                     int* topk_idx, float* topk_w, const PermuteMeta& m, int* status) {
    int* s_idx = scratch;                                                  // [T][8] selected experts
    uint32_t* mask = reinterpret_cast<uint32_t*>(scratch + RP_CTA_MAX_TOKENS * 8);   // [P_MAX_LOCAL] bit t: token t
    int* s_cnt = scratch + RP_CTA_MAX_TOKENS * 8 + P_MAX_LOCAL;            // [P_MAX_LOCAL + 1]
    int* s_pad = s_cnt + P_MAX_LOCAL + 1;                                  // [P_MAX_LOCAL + 1]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    if (tid < P_MAX_LOCAL) mask[tid] = 0u;
    {
        float bias_f[8];
        load_bias8(bias, lane, bias_f);
        for (int t = warp; t < T; t += nwarps) {
            int my_idx;
            float my_w;
            route_token(t, lane, logits, bias_f, scaling, my_idx, my_w);
            if (lane < R_TOPK) {
                s_idx[t * R_TOPK + lane] = my_idx;
                topk_idx[t * R_TOPK + lane] = my_idx;
                topk_w[t * R_TOPK + lane] = my_w;
            }
        }
    }
    __syncthreads();
    if (tid < T) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = s_idx[tid * 8 + j] - off;
            if (e >= 0 && e < E_loc) atomicOr(&mask[e], 1u << tid);
        }
    }
    __syncthreads();
    int total = 0;
    if (tid < P_MAX_LOCAL) {
        total = tid < E_loc ? __popc(mask[tid]) : 0;
        s_cnt[tid] = total;
        s_pad[tid] = (total + TILE_M - 1) / TILE_M * TILE_M;
    }
    __syncthreads();
    if (warp == 0) {  // exclusive scans of both arrays: lane l owns entries 8l .. 8l+7
        int c[8], q[8], sc = 0, sq = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            c[i] = s_cnt[lane * 8 + i];
            q[i] = s_pad[lane * 8 + i];
            sc += c[i];
            sq += q[i];
        }
        int ec = sc, eq = sq;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int vc = __shfl_up_sync(0xffffffffu, ec, d), vq = __shfl_up_sync(0xffffffffu, eq, d);
            if (lane >= d) {
                ec += vc;
                eq += vq;
            }
        }
        int bc = ec - sc, bq = eq - sq;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            s_cnt[lane * 8 + i] = bc;
            s_pad[lane * 8 + i] = bq;
            bc += c[i];
            bq += q[i];
        }
        if (lane == 31) {
            s_cnt[P_MAX_LOCAL] = ec;
            s_pad[P_MAX_LOCAL] = eq;
        }
    }
    __syncthreads();
    if (tid < E_loc) {
        m.expert_count[tid] = total;
        m.expert_offset[tid] = s_cnt[tid];
        m.padded_offset[tid] = s_pad[tid];
        // at most RP_CTA_MAX_TOKENS = 32 rows per expert: one row tile, which is also its only sub-tile
        const int t0 = s_pad[tid] / TILE_M;
        if (total > 0) {
            m.tile_expert[t0] = tid;
            m.tile_rows[t0] = total;
            m.st_expert[t0] = tid;
            m.st_row0[t0] = s_pad[tid];
            m.st_rows[t0] = total;
        }
    }
    if (tid == 0) {  // entries past E_loc count nothing, so entry E_loc already holds the totals
        *m.num_m_tiles = s_pad[E_loc] / TILE_M;
        *m.num_st = s_pad[E_loc] / TILE_M;
        m.expert_offset[E_loc] = s_cnt[E_loc];
        m.padded_offset[E_loc] = s_pad[E_loc];
    }
    if (tid < T) {
        int nlocal = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = s_idx[tid * 8 + j] - off;
            int prow = -1;
            if (e >= 0 && e < E_loc) {
                ++nlocal;
                const int rank = __popc(mask[e] & ((1u << tid) - 1u));
                prow = s_pad[e] + rank;
                if (prow < 0 || prow >= row_cap) {
                    atomicExch(status, DEV_BAD_ROW);
                    prow = -1;
                } else {
                    m.row_to_slot[s_cnt[e] + rank] = tid * 8 + j;
                    m.row_token[prow] = tid;
                }
            }
            m.slot_to_row[tid * 8 + j] = prow;
        }
        m.tok_nlocal[tid] = nlocal;
    }
    __syncthreads();
}

// One warp per padded row: copy the token's FP8 row (K bytes) and write its
// K/128 scales transposed ([K/128, row_cap]) so the GEMM epilogue reads them
// coalesced across the rows of a tile.  Rows past an expert's count are padding
// and are left untouched (their results are never stored).
__global__ void __launch_bounds__(256) gather_rows_kernel(int H, int row_cap, int scale_layout, int T,
                                                          const uint8_t* __restrict__ hidden,
                                                          const float* __restrict__ hidden_scale, PermuteMeta m,
                                                          uint8_t* __restrict__ a1, float* __restrict__ a1_scale_t) {
    pdl_launch_dependents();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int nwarps = gridDim.x * (blockDim.x >> 5);
    const int rows = *m.num_m_tiles * TILE_M;
    const int chunks = H / 16, nkb = H / 128;
    for (int r = warp; r < rows; r += nwarps) {
        if ((r % TILE_M) >= m.tile_rows[r / TILE_M]) continue;
        const int t = m.row_token[r];
        const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<size_t>(t) * H);
        uint4* dst = reinterpret_cast<uint4*>(a1 + static_cast<size_t>(r) * H);
        for (int c = lane; c < chunks; c += 32) dst[c] = __ldg(src + c);
        for (int kb = lane; kb < nkb; kb += 32) {
            const float s = scale_layout ? hidden_scale[static_cast<size_t>(kb) * T + t]
                                         : hidden_scale[static_cast<size_t>(t) * nkb + kb];
            a1_scale_t[static_cast<size_t>(kb) * row_cap + r] = s;
        }
    }
}

}  // namespace moe

// Host side of the C ABI declared in include/moe_fp8.h: handle, workspace
// carving, TMA descriptors and the launch sequence of one forward pass.
#include "../../include/moe_fp8.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "ptx.cuh"
#include "routing.cuh"
#include "permute.cuh"
#include "gemm.cuh"
#include "combine.cuh"
#include "router.cuh"

namespace {

using namespace moe;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t WS_ALIGN = 1024;
inline size_t align_up(size_t x, size_t a = WS_ALIGN) { return (x + a - 1) / a * a; }

struct WsLayout {
    size_t topk_idx, topk_w, block_hist, expert_count, expert_offset, padded_offset, tile_expert, tile_rows,
        num_m_tiles, slot_to_row, row_to_slot, row_token, tok_nlocal, st_expert, st_row0, st_rows, num_st, counters, num_counters, max_st, raw1, raw2, status, a1, a1_scale_t, a2, a2_scale_t, y, stage_hidden,
        stage_scale, stage_logits, stage_out, stage2_hidden, stage2_scale, stage2_logits, stage2_out, total;
    int row_cap, max_m_tiles, max_blocks;
};

WsLayout make_layout(const moe_fp8_config& c) {
    WsLayout L;
    const size_t Tm = static_cast<size_t>(c.max_tokens > 0 ? c.max_tokens : 1);
    const size_t slots = Tm * 8;
    size_t pad_experts = static_cast<size_t>(c.num_local_experts) < slots ? c.num_local_experts : slots;
    L.row_cap = static_cast<int>(align_up(slots + pad_experts * (TILE_M - 1), TILE_M));
    L.max_m_tiles = L.row_cap / TILE_M;
    L.max_blocks = static_cast<int>((Tm + P_TOKENS_PER_BLOCK - 1) / P_TOKENS_PER_BLOCK);
    const size_t H = c.hidden, I = c.intermediate, EL = c.num_local_experts, rc = L.row_cap;
    size_t o = 0;
    auto take = [&](size_t bytes) {
        size_t at = o;
        o = align_up(o + bytes);
        return at;
    };
    L.topk_idx = take(slots * 4);
    L.topk_w = take(slots * 4);
    L.block_hist = take(static_cast<size_t>(L.max_blocks) * EL * 4);
    L.expert_count = take(EL * 4);
    L.expert_offset = take((EL + 1) * 4);
    L.padded_offset = take((EL + 1) * 4);
    L.tile_expert = take(static_cast<size_t>(L.max_m_tiles) * 4);
    L.tile_rows = take(static_cast<size_t>(L.max_m_tiles) * 4);
    L.num_m_tiles = take(4);
    L.slot_to_row = take(slots * 4);
    L.row_to_slot = take(slots * 4);
    L.row_token = take(rc * 4);
    L.tok_nlocal = take(Tm * 4);
    // two sets of the fused small-batch kernel's counters (per row tile, per (token, column tile)): a call uses
    // one and zeroes the other for the next call
    // sub-tiles of at most 32 rows: an expert's padded rows are whole row tiles, four sub-tiles each
    L.max_st = static_cast<size_t>(L.max_m_tiles) * (TILE_M / ST_ROWS);
    L.st_expert = take(L.max_st * 4);
    L.st_row0 = take(L.max_st * 4);
    L.st_rows = take(L.max_st * 4);
    L.num_st = take(4);
    // (a batch the fused kernel takes has at most EL + F_MAX_TOKENS * 8 / 32 sub-tiles)
    // (then the parts stored per tile by the K split of very small batches, per GEMM)
    L.num_counters = std::min<size_t>(L.max_st, EL + F_MAX_TOKENS / 4) + static_cast<size_t>(F_MAX_TOKENS) * (H / G_TILE_N) +
                     2 * SPLIT_MAX_TILES;
    L.counters = take(2 * L.num_counters * 4);
    L.raw1 = take(static_cast<size_t>(SPLIT_MAX_TILES) * (H / 128) * SPLIT_RAW_FLOATS * 4);
    L.raw2 = take(static_cast<size_t>(SPLIT_MAX_TILES) * (I / 128) * SPLIT_RAW_FLOATS * 4);
    L.status = take(8);  // device status word, then the ticket counter of route_permute_kernel
    L.a1 = take(rc * H);
    L.a1_scale_t = take(rc * (H / 128) * 4);
    L.a2 = take(rc * I);
    L.a2_scale_t = take(rc * (I / 128) * 4);
    L.y = take(rc * H * 2);
    L.stage_hidden = take(Tm * H);
    L.stage_scale = take(Tm * (H / 128) * 4);
    L.stage_logits = take(Tm * 256 * 4);
    L.stage_out = take(Tm * H * 2);
    // second staging set: moe_fp8_forward_host_async alternates between the two
    L.stage2_hidden = take(Tm * H);
    L.stage2_scale = take(Tm * (H / 128) * 4);
    L.stage2_logits = take(Tm * 256 * 4);
    L.stage2_out = take(Tm * H * 2);
    L.total = o;
    return L;
}

}  // namespace

constexpr int NUM_STAGES_MAX = 9;

struct moe_fp8_handle_s {
    moe_fp8_config cfg;
    WsLayout L;
    int sm_count;
    int last_cuda_error;
    int last_launches;
    int last_T;
    uint8_t* ws;
    size_t ws_bytes;
    EncodeTiledFn encode;
    CUtensorMap tm_a1, tm_a2, tm_a1_small, tm_a2_small, tm_a2_store, tm_w13, tm_w2;
    const void* w13_cached;
    const void* w2_cached;
    bool stage_timing;
    bool stage_times_valid;
    int fault_skip_it;         // test hook, see moe_fp8_debug_set_fault
    long long fault_wait_limit;
    cudaEvent_t ev[NUM_STAGES_MAX + 1];
    int fused_max_tokens;   // batches of at most this many tokens take the fused kernel (0: never)
    bool k_split;           // fused kernel: very small batches may cut a tile's K range over several CTAs
    int short_tile_min_tokens;   // batches of at least this many tokens run short row tiles with the weights on M (0: never)
    unsigned long long fused_calls;
    // moe_fp8_forward_host_async: copy streams and the events that order the two staging sets
    bool pipe_ready;
    unsigned pipe_calls;
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_in[2], ev_compute[2], ev_out[2];
};

namespace {

int cuda_fail(moe_fp8_handle_t h, cudaError_t e) {
    if (h) h->last_cuda_error = static_cast<int>(e);
    return MOE_FP8_ERR_CUDA;
}

// 2-D tensor [rows, cols] (cols contiguous) of 1-byte (fp8) or 2-byte (bf16) elements for tiled TMA copies
// with a box of box_cols x box_rows elements and the given shared-memory swizzle.
bool encode_2d(moe_fp8_handle_t h, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, int elem_bytes,
               uint32_t box_cols, uint32_t box_rows, CUtensorMapSwizzle swizzle) {
    cuuint64_t gdim[2] = {cols, rows};
    cuuint64_t gstride[1] = {cols * elem_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estride[2] = {1, 1};
    CUresult r = h->encode(m, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                           const_cast<void*>(base), gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <typename T>
T* at(moe_fp8_handle_t h, size_t off) {
    return reinterpret_cast<T*>(h->ws + off);
}

// Launch on `stream`; with pdl the kernel may begin (up to its pdl_wait()) while the previous kernel of the
// stream is still running, which hides launch latency and the GEMM kernels' set-up.
template <typename... KArgs, typename... Args>
cudaError_t launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                   Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

PermuteMeta meta_of(moe_fp8_handle_t h) {
    PermuteMeta m;
    m.block_hist = at<int>(h, h->L.block_hist);
    m.expert_count = at<int>(h, h->L.expert_count);
    m.expert_offset = at<int>(h, h->L.expert_offset);
    m.padded_offset = at<int>(h, h->L.padded_offset);
    m.tile_expert = at<int>(h, h->L.tile_expert);
    m.tile_rows = at<int>(h, h->L.tile_rows);
    m.num_m_tiles = at<int>(h, h->L.num_m_tiles);
    m.slot_to_row = at<int>(h, h->L.slot_to_row);
    m.row_to_slot = at<int>(h, h->L.row_to_slot);
    m.row_token = at<int>(h, h->L.row_token);
    m.tok_nlocal = at<int>(h, h->L.tok_nlocal);
    m.st_expert = at<int>(h, h->L.st_expert);
    m.st_row0 = at<int>(h, h->L.st_row0);
    m.st_rows = at<int>(h, h->L.st_rows);
    m.num_st = at<int>(h, h->L.num_st);
    return m;
}

constexpr int PDL_MAX_TOKENS = 2048;
constexpr int NUM_STAGES = 9;
const char* const STAGE_NAMES[NUM_STAGES] = {"route_topk", "count", "scan", "place", "gather_rows",
                                             "gemm1_swiglu_quant", "gemm2", "combine", "fused_small"};

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Test hook: the routing stage's sigmoid on arbitrary inputs.
__global__ void sigmoid_export_kernel(int n, const float* __restrict__ x, float* __restrict__ y) {
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) y[i] = sigmoid_fixed(x[i]);
}

// Debug: canonical row r -> padded row, then copy that row's intermediate results.
__global__ void export_rows_kernel(int E_loc, int I, int H, int row_cap, const int* __restrict__ expert_offset,
                                   const int* __restrict__ padded_offset, const uint8_t* __restrict__ a2,
                                   const float* __restrict__ a2_scale_t, const __nv_bfloat16* __restrict__ y,
                                   uint8_t* __restrict__ a2_out, float* __restrict__ a2_scale_out,
                                   __nv_bfloat16* __restrict__ y_out) {
    const int S = expert_offset[E_loc];
    for (int r = blockIdx.x; r < S; r += gridDim.x) {
        int e = 0;
        while (e + 1 < E_loc && expert_offset[e + 1] <= r) ++e;
        const size_t p = static_cast<size_t>(padded_offset[e]) + (r - expert_offset[e]);
        if (a2_out)
            for (int i = threadIdx.x; i < I; i += blockDim.x) a2_out[static_cast<size_t>(r) * I + i] = a2[p * I + i];
        if (a2_scale_out)
            for (int i = threadIdx.x; i < I / 128; i += blockDim.x)
                a2_scale_out[static_cast<size_t>(r) * (I / 128) + i] = a2_scale_t[static_cast<size_t>(i) * row_cap + p];
        if (y_out)
            for (int i = threadIdx.x; i < H; i += blockDim.x)
                y_out[static_cast<size_t>(r) * H + i] = *reinterpret_cast<const __nv_bfloat16*>(
                    reinterpret_cast<const uint8_t*>(y) + y_block_offset(static_cast<int>(p), i / 16, H / 256) + (i % 16) * 2);
    }
}

}  // namespace

extern "C" {

const char* moe_fp8_strerror(int rc) {
    switch (rc) {
        case MOE_FP8_OK: return "ok";
        case MOE_FP8_ERR_BAD_ARG: return "bad argument";
        case MOE_FP8_ERR_UNSUPPORTED_DIMS: return "unsupported layer dimensions";
        case MOE_FP8_ERR_NO_WORKSPACE: return "workspace missing or too small";
        case MOE_FP8_ERR_CUDA: return "CUDA error";
        case MOE_FP8_ERR_ARCH: return "device is not compute capability 10.x (no fallback path exists)";
        case MOE_FP8_ERR_STATIC_LIMIT: return "size exceeds the fixed capacity of the no-allocation entry point";
        default: return "unknown error";
    }
}

int moe_fp8_create(const moe_fp8_config* cfg, moe_fp8_handle_t* out) {
    if (!cfg || !out) return MOE_FP8_ERR_BAD_ARG;
    *out = nullptr;
    if (cfg->max_tokens < 0 || cfg->hidden <= 0 || cfg->intermediate <= 0 || cfg->num_local_experts <= 0)
        return MOE_FP8_ERR_BAD_ARG;
    if (cfg->num_experts != R_EXPERTS || cfg->n_group != R_GROUPS || cfg->topk_group != R_TOPK_GROUP ||
        cfg->top_k != R_TOPK || cfg->hidden % G_TILE_N != 0 || cfg->intermediate % 128 != 0 ||
        cfg->num_local_experts > P_MAX_LOCAL || cfg->max_tokens > (1 << 20) ||
        (cfg->hidden_scale_layout != 0 && cfg->hidden_scale_layout != 1))
        return MOE_FP8_ERR_UNSUPPORTED_DIMS;

    int dev = 0, major = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    if (major != 10) return MOE_FP8_ERR_ARCH;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;

    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) return MOE_FP8_ERR_CUDA;

    e = cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, GeomFull::SMEM_BYTES);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    e = cudaFuncSetAttribute(grouped_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GeomFull::SMEM_BYTES);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    e = cudaFuncSetAttribute(fused_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GeomSmall::SMEM_BYTES);
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    e = cudaFuncSetAttribute(router_logits_kernel<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(router_smem_bytes(4, 4)));
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;
    e = cudaFuncSetAttribute(route_permute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(route_permute_smem_bytes(P_TAIL_MAX_TOKENS, P_MAX_LOCAL)));
    if (e != cudaSuccess) return MOE_FP8_ERR_CUDA;

    moe_fp8_handle_s* h = new (std::nothrow) moe_fp8_handle_s();
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    memset(h, 0, sizeof(*h));
    h->cfg = *cfg;
    h->L = make_layout(*cfg);
    h->sm_count = sms;
    h->fused_max_tokens = F_DEFAULT_MAX_TOKENS;
    h->k_split = true;
    h->short_tile_min_tokens = SHORT_TILE_MIN_TOKENS;
    h->fused_calls = 0;
    h->fault_skip_it = -1;
    h->fault_wait_limit = WAIT_LIMIT_CLOCKS;
    h->encode = reinterpret_cast<EncodeTiledFn>(fn);
    *out = h;
    return MOE_FP8_OK;
}

int moe_fp8_destroy(moe_fp8_handle_t h) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    moe_fp8_set_stage_timing(h, 0);
    if (h->pipe_ready) {
        cudaStreamSynchronize(h->s_in);
        cudaStreamSynchronize(h->s_out);
        for (int k = 0; k < 2; ++k) {
            cudaEventDestroy(h->ev_in[k]);
            cudaEventDestroy(h->ev_compute[k]);
            cudaEventDestroy(h->ev_out[k]);
        }
        cudaStreamDestroy(h->s_in);
        cudaStreamDestroy(h->s_out);
    }
    delete h;
    return MOE_FP8_OK;
}

size_t moe_fp8_workspace_bytes(moe_fp8_handle_t h) { return h ? h->L.total : 0; }

int moe_fp8_set_workspace(moe_fp8_handle_t h, void* ws, size_t bytes) {
    if (!h || !ws || (reinterpret_cast<uintptr_t>(ws) % WS_ALIGN) != 0) return MOE_FP8_ERR_BAD_ARG;
    if (bytes < h->L.total) return MOE_FP8_ERR_NO_WORKSPACE;
    // The device status word and the ticket counter of route_permute_kernel start at zero.  A memset of device
    // memory is asynchronous to the host and a forward may follow on a non-blocking stream, which does not
    // order itself behind the default stream: wait for it here.
    cudaError_t e = cudaMemset(static_cast<uint8_t*>(ws) + h->L.status, 0, 2 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(static_cast<uint8_t*>(ws) + h->L.counters, 0, 2 * h->L.num_counters * sizeof(int));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    h->fused_calls = 0;
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->ws = static_cast<uint8_t*>(ws);
    h->ws_bytes = bytes;
    if (!encode_2d(h, &h->tm_a1, h->ws + h->L.a1, h->L.row_cap, h->cfg.hidden, 1, 128, TILE_M,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(h, &h->tm_a2, h->ws + h->L.a2, h->L.row_cap, h->cfg.intermediate, 1, 128, TILE_M,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(h, &h->tm_a1_small, h->ws + h->L.a1, h->L.row_cap, h->cfg.hidden, 1, 128, GeomSmall::A_ROWS,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(h, &h->tm_a2_small, h->ws + h->L.a2, h->L.row_cap, h->cfg.intermediate, 1, 128, GeomSmall::A_ROWS,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_2d(h, &h->tm_a2_store, h->ws + h->L.a2, h->L.row_cap, h->cfg.intermediate, 1, 64, 32,
                   CU_TENSOR_MAP_SWIZZLE_64B)) {
        h->ws = nullptr;
        return cuda_fail(h, cudaErrorInvalidValue);
    }
    return MOE_FP8_OK;
}

int moe_fp8_last_cuda_error(moe_fp8_handle_t h) { return h ? h->last_cuda_error : 0; }
int moe_fp8_last_launch_count(moe_fp8_handle_t h) { return h ? h->last_launches : 0; }

int moe_fp8_forward(moe_fp8_handle_t h, int T, const void* hidden_fp8, const float* hidden_scale,
                    const float* router_logits, const void* routing_bias, const void* w13, const float* w13_scale,
                    const void* w2, const float* w2_scale, int local_expert_offset, float scaling_factor, void* out,
                    void* stream_v) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    const moe_fp8_config& c = h->cfg;
    if (T < 0 || T > c.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (local_expert_offset < 0 || local_expert_offset + c.num_local_experts > c.num_experts)
        return MOE_FP8_ERR_BAD_ARG;
    if (!routing_bias || !w13 || !w13_scale || !w2 || !w2_scale || misaligned(routing_bias) || misaligned(w13) ||
        misaligned(w13_scale) || misaligned(w2) || misaligned(w2_scale))
        return MOE_FP8_ERR_BAD_ARG;
    if (T > 0 && (!hidden_fp8 || !hidden_scale || !router_logits || !out || misaligned(hidden_fp8) ||
                  misaligned(hidden_scale) || misaligned(router_logits) || misaligned(out)))
        return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    h->last_launches = 0;
    h->last_T = T;
    if (T == 0) return MOE_FP8_OK;

    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int H = c.hidden, I = c.intermediate, EL = c.num_local_experts;
    if (w13 != h->w13_cached || w2 != h->w2_cached) {
        // w13 is fetched in 64-row boxes (gate and up rows interleave in the B tile), w2 in 128-row boxes
        if (!encode_2d(h, &h->tm_w13, w13, static_cast<uint64_t>(EL) * 2 * I, H, 1, 128, 64,
                       CU_TENSOR_MAP_SWIZZLE_128B) ||
            !encode_2d(h, &h->tm_w2, w2, static_cast<uint64_t>(EL) * H, I, 1, 128, 128, CU_TENSOR_MAP_SWIZZLE_128B))
            return cuda_fail(h, cudaErrorInvalidValue);
        h->w13_cached = w13;
        h->w2_cached = w2;
    }

    PermuteMeta m = meta_of(h);
    int* topk_idx = at<int>(h, h->L.topk_idx);
    float* topk_w = at<float>(h, h->L.topk_w);
    int* status = at<int>(h, h->L.status);
    uint8_t* a1 = at<uint8_t>(h, h->L.a1);
    float* a1_scale_t = at<float>(h, h->L.a1_scale_t);
    uint8_t* a2 = at<uint8_t>(h, h->L.a2);
    float* a2_scale_t = at<float>(h, h->L.a2_scale_t);
    __nv_bfloat16* y = at<__nv_bfloat16>(h, h->L.y);
    const int row_cap = h->L.row_cap;
    const int nblk = (T + P_TOKENS_PER_BLOCK - 1) / P_TOKENS_PER_BLOCK;
    int launches = 0;
    // Programmatic dependent launch between our own kernels (not across the per-kernel timing events).  It
    // removes 10-13 us of launch gaps from a small batch; on large batches the early-resident blocks of the
    // next kernel cost the running GEMM about 6 %, so it is limited to the launch-latency-bound regime.
    const bool pdl = !h->stage_timing && T <= PDL_MAX_TOKENS;

    // No memset: the first kernel clears the status word, and the ticket counter returns to zero by itself.
    int ev_i = 0;
    auto mark = [&]() {
        if (h->stage_timing) cudaEventRecord(h->ev[ev_i++], stream);
    };
    // The first launch that fails ends the call: nothing further is enqueued behind it.
    cudaError_t lerr = cudaSuccess;
#define MOE_LAUNCH(...)                                   \
    do {                                                  \
        lerr = launch(__VA_ARGS__);                       \
        if (lerr != cudaSuccess) return cuda_fail(h, lerr); \
        ++launches;                                       \
    } while (0)
    h->stage_times_valid = false;
    mark();
    // Batches of at most fused_max_tokens tokens: gather, both GEMMs and the combine in one kernel; up to
    // F_ROUTE_MAX_TOKENS that kernel also routes and permutes (every CTA for itself: one launch per forward).
    const bool fused = T <= h->fused_max_tokens;
    const bool route_in_fused = fused && T <= F_ROUTE_MAX_TOKENS;
    int *counters = nullptr, *counters_next = nullptr;
    if (fused) {
        // this call's counter set is zero: the fused call before it zeroed it (set_workspace for the first two)
        const size_t set = h->fused_calls & 1;  // (advanced once the fused kernel is enqueued)
        counters = at<int>(h, h->L.counters) + set * h->L.num_counters;
        counters_next = at<int>(h, h->L.counters) + (set ^ 1) * h->L.num_counters;
    }

    if (route_in_fused) {
        mark();
        mark();
        mark();
        mark();
    } else if (T <= P_TAIL_MAX_TOKENS) {  // routing in parallel blocks, the last one to finish does stage 2
        const int grid = min((T + 7) / 8, h->sm_count * 8);
        MOE_LAUNCH(route_permute_kernel, grid, P_TAIL_THREADS, route_permute_smem_bytes(T, EL), stream, false, T, EL,
                   local_expert_offset, row_cap, router_logits, static_cast<const __nv_bfloat16*>(routing_bias),
                   scaling_factor, topk_idx, topk_w, m, status + 1, status);
        mark();
        mark();
        mark();
        mark();
    } else {
        {  // stage 1: routing
            const int grid = min((T + 7) / 8, h->sm_count * 8);
            MOE_LAUNCH(route_topk_kernel, grid, 256, 0, stream, false, T, router_logits,
                       static_cast<const __nv_bfloat16*>(routing_bias), scaling_factor, topk_idx, topk_w, status);
            mark();
        }
        // stage 2: histogram, scan, placement
        MOE_LAUNCH(count_kernel, nblk, P_TOKENS_PER_BLOCK, 0, stream, pdl, T, EL, local_expert_offset,
                   static_cast<const int*>(topk_idx), m.block_hist);
        mark();
        MOE_LAUNCH(scan_kernel, 1, P_MAX_LOCAL, 0, stream, pdl, nblk, EL, m);
        mark();
        MOE_LAUNCH(place_kernel, nblk, P_TOKENS_PER_BLOCK, 0, stream, pdl, T, EL, local_expert_offset, row_cap,
                   static_cast<const int*>(topk_idx), m, status);
        mark();
    }
    // the two GEMMs' arguments
    GemmArgs g1, g2;
    memset(&g1, 0, sizeof(g1));
    g1.num_kb = H / 128;
    g1.n_tiles = I / 128;
    g1.w_rows_per_expert = 2 * I;
    g1.row_cap = row_cap;
    g1.out_cols = I;
    g1.gate_row0 = c.gate_first ? 0 : I;
    g1.up_row0 = c.gate_first ? I : 0;
    g1.num_m_tiles = m.num_m_tiles;
    g1.tile_expert = m.tile_expert;
    g1.tile_rows = m.tile_rows;
    g1.a_scale_t = a1_scale_t;
    g1.w_scale = w13_scale;
    g1.out_fp8 = a2;
    g1.out_scale_t = a2_scale_t;
    g1.status = status;
    g1.wait_limit = h->fault_wait_limit;
    g1.fault_skip_it = h->fault_skip_it;
    memset(&g2, 0, sizeof(g2));
    g2.num_kb = I / 128;
    g2.n_tiles = H / G_TILE_N;
    g2.w_rows_per_expert = H;
    g2.row_cap = row_cap;
    g2.out_cols = H;
    g2.num_m_tiles = m.num_m_tiles;
    g2.tile_expert = m.tile_expert;
    g2.tile_rows = m.tile_rows;
    g2.a_scale_t = a2_scale_t;
    g2.w_scale = w2_scale;
    g2.out_bf16 = y;
    g2.status = status;
    g2.wait_limit = h->fault_wait_limit;
    g2.fault_skip_it = -1;

    if (fused) {
        // stages 2 (gather), 3 and 4 in one launch
        FusedArgs f;
        memset(&f, 0, sizeof(f));
        f.T = T;
        f.H = H;
        f.scale_layout = c.hidden_scale_layout;
        f.hidden = static_cast<const uint8_t*>(hidden_fp8);
        f.hidden_scale = hidden_scale;
        f.row_token = m.row_token;
        f.slot_to_row = m.slot_to_row;
        f.topk_w = topk_w;
        f.tok_nlocal = m.tok_nlocal;
        f.ready = counters;
        f.tok_done = counters + (h->L.num_counters - 2 * SPLIT_MAX_TILES - static_cast<size_t>(F_MAX_TOKENS) * (H / G_TILE_N));
        f.part_done[0] = counters + (h->L.num_counters - 2 * SPLIT_MAX_TILES);
        f.part_done[1] = f.part_done[0] + SPLIT_MAX_TILES;
        f.raw[0] = at<float>(h, h->L.raw1);
        f.raw[1] = at<float>(h, h->L.raw2);
        f.split = h->k_split ? 1 : 0;
        // the fused kernel works on sub-tiles of at most 32 rows
        g1.num_m_tiles = g2.num_m_tiles = m.num_st;
        g1.tile_expert = g2.tile_expert = m.st_expert;
        g1.tile_rows = g2.tile_rows = m.st_rows;
        g1.tile_row0 = g2.tile_row0 = m.st_row0;
        f.out = static_cast<__nv_bfloat16*>(out);
        f.route = route_in_fused;
        f.E_loc = EL;
        f.expert_offset = local_expert_offset;
        f.row_cap = row_cap;
        f.logits = router_logits;
        f.bias = static_cast<const __nv_bfloat16*>(routing_bias);
        f.scaling = scaling_factor;
        f.topk_idx = topk_idx;
        f.topk_w_out = topk_w;
        f.meta = m;
        f.counters_next = counters_next;
        f.num_counters = static_cast<int>(h->L.num_counters);
        mark();  // gather_rows
        mark();  // gemm1
        mark();  // gemm2
        mark();  // combine
        MOE_LAUNCH(fused_small_kernel, h->sm_count, G_THREADS, GeomSmall::SMEM_BYTES, stream, pdl, h->tm_a2_small,
                   h->tm_w13, h->tm_w2, g1, g2, f);
        ++h->fused_calls;  // only a kernel that runs zeroes the other counter set
        mark();
    } else {
        {  // stage 2, continued: gather
            const long long row_bound = static_cast<long long>(T) * 8 + static_cast<long long>(EL) * (TILE_M - 1);
            const int grid = static_cast<int>(std::min<long long>((row_bound + 7) / 8, h->sm_count * 8LL));
            MOE_LAUNCH(gather_rows_kernel, grid, 256, 0, stream, pdl, H, row_cap, c.hidden_scale_layout, T,
                       static_cast<const uint8_t*>(hidden_fp8), hidden_scale, m, a1, a1_scale_t);
            mark();
        }
        // stage 3a: GEMM1 + SwiGLU + re-quantisation
        if (h->short_tile_min_tokens > 0 && T >= h->short_tile_min_tokens) g1.wm_rows = g2.wm_rows = WM_TOKENS;
        MOE_LAUNCH(grouped_gemm_kernel<1>, h->sm_count, G_THREADS, GeomFull::SMEM_BYTES, stream, pdl, h->tm_a1,
                   h->tm_a1_small, h->tm_w13, h->tm_a2_store, g1);
        mark();
        // stage 3b: GEMM2
        MOE_LAUNCH(grouped_gemm_kernel<2>, h->sm_count, G_THREADS, GeomFull::SMEM_BYTES, stream, pdl, h->tm_a2,
                   h->tm_a2_small, h->tm_w2, h->tm_a2_store, g2);
        mark();
        {  // stage 4: weighted combine back to token order
            const int grid = min(T, h->sm_count * 16);
            MOE_LAUNCH(combine_kernel, grid, 256, 0, stream, pdl, T, H, static_cast<const int*>(m.slot_to_row),
                       static_cast<const float*>(topk_w), reinterpret_cast<const uint8_t*>(y),
                       static_cast<__nv_bfloat16*>(out));
            mark();
        }
        mark();  // fused_small (not used on this path)
    }
#undef MOE_LAUNCH
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(h, e);
    h->last_launches = launches;
    h->stage_times_valid = h->stage_timing;
    return MOE_FP8_OK;
}

int moe_fp8_debug_set_fault(moe_fp8_handle_t h, int skip_iteration, long long wait_clocks) {
    if (!h || wait_clocks < 0) return MOE_FP8_ERR_BAD_ARG;
    h->fault_skip_it = skip_iteration < 0 ? -1 : skip_iteration;
    h->fault_wait_limit = wait_clocks == 0 ? WAIT_LIMIT_CLOCKS : wait_clocks;
    return MOE_FP8_OK;
}

int moe_fp8_debug_set_k_split(moe_fp8_handle_t h, int enable) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    h->k_split = enable != 0;
    return MOE_FP8_OK;
}

int moe_fp8_debug_set_short_tiles(moe_fp8_handle_t h, int min_tokens) {
    if (!h || min_tokens < 0) return MOE_FP8_ERR_BAD_ARG;
    h->short_tile_min_tokens = min_tokens;
    return MOE_FP8_OK;
}

int moe_fp8_set_small_batch_fusion(moe_fp8_handle_t h, int enable) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if (enable < 0 || enable > F_MAX_TOKENS) return MOE_FP8_ERR_BAD_ARG;
    h->fused_max_tokens = enable == 0 ? 0 : enable == 1 ? F_DEFAULT_MAX_TOKENS : enable;
    return MOE_FP8_OK;
}

int moe_fp8_debug_sigmoid(int n, const float* x, float* y, void* stream_v) {
    if (n < 0 || (n > 0 && (!x || !y))) return MOE_FP8_ERR_BAD_ARG;
    if (n == 0) return MOE_FP8_OK;
    sigmoid_export_kernel<<<(n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256, 256, 0,
                            static_cast<cudaStream_t>(stream_v)>>>(n, x, y);
    return cudaGetLastError() == cudaSuccess ? MOE_FP8_OK : MOE_FP8_ERR_CUDA;
}

int moe_fp8_set_stage_timing(moe_fp8_handle_t h, int enable) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if ((enable != 0) == h->stage_timing) return MOE_FP8_OK;
    h->stage_times_valid = false;
    if (enable) {
        for (int i = 0; i <= NUM_STAGES; ++i) {
            cudaError_t e = cudaEventCreate(&h->ev[i]);
            if (e != cudaSuccess) {
                for (int j = 0; j < i; ++j) cudaEventDestroy(h->ev[j]);
                return cuda_fail(h, e);
            }
        }
        h->stage_timing = true;
    } else {
        for (int i = 0; i <= NUM_STAGES; ++i) cudaEventDestroy(h->ev[i]);
        h->stage_timing = false;
    }
    return MOE_FP8_OK;
}

int moe_fp8_num_stages(void) { return NUM_STAGES; }

const char* moe_fp8_stage_name(int i) { return (i >= 0 && i < NUM_STAGES) ? STAGE_NAMES[i] : ""; }

int moe_fp8_get_stage_times(moe_fp8_handle_t h, float* host_ms, int n) {
    if (!h || !host_ms || n < 0) return MOE_FP8_ERR_BAD_ARG;
    if (!h->stage_timing || !h->stage_times_valid) return MOE_FP8_ERR_BAD_ARG;
    cudaError_t e = cudaEventSynchronize(h->ev[NUM_STAGES]);
    if (e != cudaSuccess) return cuda_fail(h, e);
    const int k = n < NUM_STAGES ? n : NUM_STAGES;
    for (int i = 0; i < k; ++i) {
        e = cudaEventElapsedTime(&host_ms[i], h->ev[i], h->ev[i + 1]);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    return k;
}

int moe_fp8_forward_host(moe_fp8_handle_t h, int T, const void* host_hidden_fp8, const float* host_hidden_scale,
                         const float* host_router_logits, const void* routing_bias, const void* w13,
                         const float* w13_scale, const void* w2, const float* w2_scale, int local_expert_offset,
                         float scaling_factor, void* host_out, void* stream_v) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (T > 0 && (!host_hidden_fp8 || !host_hidden_scale || !host_router_logits || !host_out))
        return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    if (T == 0) return moe_fp8_forward(h, 0, nullptr, nullptr, nullptr, routing_bias, w13, w13_scale, w2, w2_scale,
                                       local_expert_offset, scaling_factor, nullptr, stream_v);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t H = h->cfg.hidden, Tz = T;
    uint8_t* d_hidden = at<uint8_t>(h, h->L.stage_hidden);
    float* d_scale = at<float>(h, h->L.stage_scale);
    float* d_logits = at<float>(h, h->L.stage_logits);
    void* d_out = at<uint8_t>(h, h->L.stage_out);
    cudaError_t e;
    if ((e = cudaMemcpyAsync(d_hidden, host_hidden_fp8, Tz * H, cudaMemcpyHostToDevice, stream)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_scale, host_hidden_scale, Tz * (H / 128) * 4, cudaMemcpyHostToDevice, stream)) !=
            cudaSuccess ||
        (e = cudaMemcpyAsync(d_logits, host_router_logits, Tz * 256 * 4, cudaMemcpyHostToDevice, stream)) !=
            cudaSuccess)
        return cuda_fail(h, e);
    int rc = moe_fp8_forward(h, T, d_hidden, d_scale, d_logits, routing_bias, w13, w13_scale, w2, w2_scale,
                             local_expert_offset, scaling_factor, d_out, stream_v);
    if (rc != MOE_FP8_OK) return rc;
    if ((e = cudaMemcpyAsync(host_out, d_out, Tz * H * 2, cudaMemcpyDeviceToHost, stream)) != cudaSuccess)
        return cuda_fail(h, e);
    if ((e = cudaStreamSynchronize(stream)) != cudaSuccess) return cuda_fail(h, e);
    return MOE_FP8_OK;
}

int moe_fp8_forward_from_hidden(moe_fp8_handle_t h, int T, const void* hidden_bf16, const void* router_weight,
                                const void* routing_bias, const void* w13, const float* w13_scale, const void* w2,
                                const float* w2_scale, int local_expert_offset, float scaling_factor, void* out,
                                void* stream_v) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (!router_weight || misaligned(router_weight) || (T > 0 && (!hidden_bf16 || misaligned(hidden_bf16))))
        return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int H = h->cfg.hidden, E = h->cfg.num_experts;
    uint8_t* d_hidden = at<uint8_t>(h, h->L.stage_hidden);
    float* d_scale = at<float>(h, h->L.stage_scale);
    float* d_logits = at<float>(h, h->L.stage_logits);
    if (T > 0) {
        const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(hidden_bf16);
        const __nv_bfloat16* wr = static_cast<const __nv_bfloat16*>(router_weight);
        cudaError_t e;
        if (T <= 128)  // few tokens: many small CTAs, so that the router weight streams in from many SMs
            e = launch(router_logits_kernel<1, 4>, dim3((T + 7) / 8, E / 32), 128, router_smem_bytes(1, 4), stream, false,
                       T, H, E, x, wr, d_logits);
        else
            e = launch(router_logits_kernel<4, 4>, dim3((T + 31) / 32, E / 32), 512, router_smem_bytes(4, 4), stream,
                       false, T, H, E, x, wr, d_logits);
        if (e != cudaSuccess) return cuda_fail(h, e);
        const long long blocks = (static_cast<long long>(T) * (H / 128) + 7) / 8;
        e = launch(quantize_rows_kernel, static_cast<int>(std::min<long long>(blocks, h->sm_count * 16LL)), 256, 0, stream,
                   false, T, H, h->cfg.hidden_scale_layout, x, d_hidden, d_scale);
        if (e != cudaSuccess) return cuda_fail(h, e);
    }
    const int rc = moe_fp8_forward(h, T, d_hidden, d_scale, d_logits, routing_bias, w13, w13_scale, w2, w2_scale,
                                   local_expert_offset, scaling_factor, out, stream_v);
    if (rc == MOE_FP8_OK && T > 0) h->last_launches += 2;
    return rc;
}

int moe_fp8_debug_export_inputs(moe_fp8_handle_t h, int T, float* router_logits, void* hidden_fp8,
                                float* hidden_scale, void* stream_v) {
    if (!h || T < 0 || T > h->cfg.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t Tz = T, H = h->cfg.hidden;
    cudaError_t e = cudaSuccess;
    auto copy = [&](void* dst, size_t off, size_t bytes) {
        if (dst && bytes && e == cudaSuccess)
            e = cudaMemcpyAsync(dst, h->ws + off, bytes, cudaMemcpyDeviceToDevice, stream);
    };
    copy(router_logits, h->L.stage_logits, Tz * h->cfg.num_experts * 4);
    copy(hidden_fp8, h->L.stage_hidden, Tz * H);
    copy(hidden_scale, h->L.stage_scale, Tz * (H / 128) * 4);
    if (e != cudaSuccess) return cuda_fail(h, e);
    return MOE_FP8_OK;
}

int moe_fp8_forward_host_async(moe_fp8_handle_t h, int T, const void* host_hidden_fp8, const float* host_hidden_scale,
                               const float* host_router_logits, const void* routing_bias, const void* w13,
                               const float* w13_scale, const void* w2, const float* w2_scale, int local_expert_offset,
                               float scaling_factor, void* host_out, void* stream_v) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if (T < 0 || T > h->cfg.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (T > 0 && (!host_hidden_fp8 || !host_hidden_scale || !host_router_logits || !host_out))
        return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    if (T == 0) return MOE_FP8_OK;
    cudaError_t e;
    if (!h->pipe_ready) {  // first use: two copy streams and six events (host-side objects, no device memory)
        if ((e = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail(h, e);
        if ((e = cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking)) != cudaSuccess) {
            cudaStreamDestroy(h->s_in);
            return cuda_fail(h, e);
        }
        for (int k = 0; k < 2; ++k) {
            cudaEventCreateWithFlags(&h->ev_in[k], cudaEventDisableTiming);
            cudaEventCreateWithFlags(&h->ev_compute[k], cudaEventDisableTiming);
            cudaEventCreateWithFlags(&h->ev_out[k], cudaEventDisableTiming);
        }
        if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(h, e);
        h->pipe_calls = 0;
        h->pipe_ready = true;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const int k = h->pipe_calls & 1;
    const bool used_before = h->pipe_calls >= 2;  // this staging set has a call two steps back still to respect
    const size_t H = h->cfg.hidden, Tz = T;
    uint8_t* d_hidden = at<uint8_t>(h, k ? h->L.stage2_hidden : h->L.stage_hidden);
    float* d_scale = at<float>(h, k ? h->L.stage2_scale : h->L.stage_scale);
    float* d_logits = at<float>(h, k ? h->L.stage2_logits : h->L.stage_logits);
    void* d_out = at<uint8_t>(h, k ? h->L.stage2_out : h->L.stage_out);
    // inputs: after the forward that last read this staging set
    if (used_before && (e = cudaStreamWaitEvent(h->s_in, h->ev_compute[k], 0)) != cudaSuccess) return cuda_fail(h, e);
    if ((e = cudaMemcpyAsync(d_hidden, host_hidden_fp8, Tz * H, cudaMemcpyHostToDevice, h->s_in)) != cudaSuccess ||
        (e = cudaMemcpyAsync(d_scale, host_hidden_scale, Tz * (H / 128) * 4, cudaMemcpyHostToDevice, h->s_in)) !=
            cudaSuccess ||
        (e = cudaMemcpyAsync(d_logits, host_router_logits, Tz * 256 * 4, cudaMemcpyHostToDevice, h->s_in)) !=
            cudaSuccess ||
        (e = cudaEventRecord(h->ev_in[k], h->s_in)) != cudaSuccess)
        return cuda_fail(h, e);
    // forward: after its inputs have arrived and after the copy-out that last read this set's output area
    if ((e = cudaStreamWaitEvent(stream, h->ev_in[k], 0)) != cudaSuccess) return cuda_fail(h, e);
    if (used_before && (e = cudaStreamWaitEvent(stream, h->ev_out[k], 0)) != cudaSuccess) return cuda_fail(h, e);
    const int rc = moe_fp8_forward(h, T, d_hidden, d_scale, d_logits, routing_bias, w13, w13_scale, w2, w2_scale,
                                   local_expert_offset, scaling_factor, d_out, stream_v);
    if (rc != MOE_FP8_OK) return rc;
    if ((e = cudaEventRecord(h->ev_compute[k], stream)) != cudaSuccess) return cuda_fail(h, e);
    // output: after the forward
    if ((e = cudaStreamWaitEvent(h->s_out, h->ev_compute[k], 0)) != cudaSuccess ||
        (e = cudaMemcpyAsync(host_out, d_out, Tz * H * 2, cudaMemcpyDeviceToHost, h->s_out)) != cudaSuccess ||
        (e = cudaEventRecord(h->ev_out[k], h->s_out)) != cudaSuccess)
        return cuda_fail(h, e);
    ++h->pipe_calls;
    return MOE_FP8_OK;
}

int moe_fp8_host_sync(moe_fp8_handle_t h) {
    if (!h) return MOE_FP8_ERR_BAD_ARG;
    if (!h->pipe_ready) return MOE_FP8_OK;
    cudaError_t e;
    if ((e = cudaStreamSynchronize(h->s_in)) != cudaSuccess || (e = cudaStreamSynchronize(h->s_out)) != cudaSuccess)
        return cuda_fail(h, e);
    return MOE_FP8_OK;
}

int moe_fp8_debug_export(moe_fp8_handle_t h, int T, int* topk_idx, float* topk_w, int* expert_count,
                         int* expert_offset, int* row_to_slot, void* a2_fp8, float* a2_scale, void* y_rows,
                         int* status_word, void* stream_v) {
    if (!h || T < 0 || T > h->cfg.max_tokens) return MOE_FP8_ERR_BAD_ARG;
    if (!h->ws) return MOE_FP8_ERR_NO_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const size_t slots = static_cast<size_t>(T) * 8, EL = h->cfg.num_local_experts;
    cudaError_t e = cudaSuccess;
    auto copy = [&](void* dst, size_t off, size_t bytes) {
        if (dst && bytes && e == cudaSuccess)
            e = cudaMemcpyAsync(dst, h->ws + off, bytes, cudaMemcpyDeviceToDevice, stream);
    };
    copy(status_word, h->L.status, 4);
    if (T > 0 && h->last_T == T) {
        copy(topk_idx, h->L.topk_idx, slots * 4);
        copy(topk_w, h->L.topk_w, slots * 4);
        copy(expert_count, h->L.expert_count, EL * 4);
        copy(expert_offset, h->L.expert_offset, (EL + 1) * 4);
        copy(row_to_slot, h->L.row_to_slot, slots * 4);
        if (e == cudaSuccess && (a2_fp8 || a2_scale || y_rows)) {
            export_rows_kernel<<<1024, 256, 0, stream>>>(
                static_cast<int>(EL), h->cfg.intermediate, h->cfg.hidden, h->L.row_cap,
                at<int>(h, h->L.expert_offset), at<int>(h, h->L.padded_offset), at<uint8_t>(h, h->L.a2),
                at<float>(h, h->L.a2_scale_t), at<__nv_bfloat16>(h, h->L.y), static_cast<uint8_t*>(a2_fp8), a2_scale,
                static_cast<__nv_bfloat16*>(y_rows));
            e = cudaGetLastError();
        }
    } else if (T > 0) {
        return MOE_FP8_ERR_BAD_ARG;
    }
    if (e != cudaSuccess) return cuda_fail(h, e);
    return MOE_FP8_OK;
}

}  // extern "C"

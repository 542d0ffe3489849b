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
//
// Two kernels are built from these roles:
//   grouped_gemm_kernel<MODE>   one GEMM per launch (any batch size);
//   fused_small_kernel          small batches (the host decides up to which size): the gather of stage 2, GEMM1, GEMM2
//               and the weighted combine of stage 4 in ONE launch, with the operands swapped (weights on the
//               M side of the MMA, the tile's at most 32 token rows on the N side; see "weights on M" below).
//               Every CTA first works through its GEMM1 tiles, then its GEMM2 tiles.  Warp 3 gathers the (few)
//               token rows of a GEMM1 tile straight from the token-major input with cp.async.  A GEMM2 tile
//               starts once a counter in global memory says that all GEMM1 column tiles of its row tile have
//               been stored (bounded wait; GEMM1 tiles never wait for another CTA and precede the GEMM2 tiles
//               in every CTA, and all CTAs of the one-per-SM grid are resident, so the counter always
//               arrives).  The CTA that completes the last local row of a token for a column tile -- found
//               with a per-(token, column tile) counter, nobody waits -- sums that token's rows in routing
//               order and writes the bf16 output.  Up to F_ROUTE_MAX_TOKENS tokens the kernel starts with
//               stages 1 and 2 as well: every CTA routes and permutes the whole batch for itself
//               (route_permute_in_cta) and all of them write the same tables, so the forward is one launch
//               and still no CTA waits for a table.  The counters come in two sets; CTA 0 zeroes the set of
//               the next call.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "permute.cuh"
#include "ptx.cuh"

namespace moe {



// The two MMA issuer threads take the even and the odd K-blocks.  A thread must see EVERY phase of a barrier it
// waits on (a parity wait cannot tell the wanted phase from the one two earlier), so a stage must always fall
// to the same issuer: the stage count has to be even (checked in Geometry).
constexpr int G_MAX_STAGES = 6;
constexpr int G_BLOCK_K = 128;                          // K bytes per stage = one scale block
constexpr int G_TILE_N = 256;                           // output columns per tile
constexpr int G_HALF_N = 128;                           // columns handled by one epilogue warpgroup
constexpr int G_ACC_BUFS = 2;                           // TMEM accumulator buffers (2 x 256 columns)
constexpr int G_B_BYTES = G_TILE_N * G_BLOCK_K;         // 32 KB
constexpr int G_THREADS = 384;                          // 4 control warps + 8 epilogue warps
constexpr int G_EPI_WARPS = 8;
constexpr int G_STORE_WARP_BYTES = 2048;                // per-warp staging: 32 rows x 64 B (swizzled)
constexpr int G_AMAX_BYTES = 2 * 2 * TILE_M * 4;               // GEMM1 row-amax exchange
constexpr int G_CTRL_BYTES = 512;
constexpr uint32_t G_TMEM_COLS = 512;

// Shared-memory geometry of a kernel: pipeline stages, rows of the A tile that are actually fetched (the MMA
// always reads 128 rows; with fewer fetched rows the rest of its A operand is whatever follows in shared
// memory, and those accumulator rows are never stored), slots of the activation-scale ring.
template <int STAGES_, int A_ROWS_, int SCALE_SLOTS_, int STORE_BYTES_>
struct Geometry {
    static constexpr int STAGES = STAGES_, A_ROWS = A_ROWS_, SCALE_SLOTS = SCALE_SLOTS_;
    static constexpr int A_BYTES = A_ROWS_ * G_BLOCK_K;
    static constexpr int STAGE_BYTES = A_BYTES + G_B_BYTES;
    static constexpr int SCALE_BYTES = A_ROWS_ * 4;                  // per K-block
    static constexpr int STORE_BYTES = STORE_BYTES_;                 // GEMM1 output staging
    static constexpr int SMEM_BYTES = STAGES_ * STAGE_BYTES + SCALE_SLOTS_ * SCALE_BYTES + STORE_BYTES_ + G_AMAX_BYTES +
                                      G_CTRL_BYTES + 1024;           // + alignment slack
    static_assert(STAGES_ % 2 == 0, "an odd stage count lets an issuer thread skip phases of full[s]");
    static_assert(STAGES_ <= G_MAX_STAGES, "control block holds G_MAX_STAGES barriers per kind");
    static_assert(A_BYTES % 1024 == 0, "the B tile must stay 1024-byte aligned for the 128-byte swizzle");
    static_assert(SCALE_SLOTS_ >= STAGES_ + G_ACC_BUFS + 1, "the producer may be that far ahead of the epilogue");
    static_assert(SMEM_BYTES <= 232448, "exceeds the 227 KB of shared memory a CTA may use");
};
// one GEMM per launch: full 128-row A tiles, 4 stages of 48 KB
using GeomFull = Geometry<4, TILE_M, 8, G_EPI_WARPS * G_STORE_WARP_BYTES>;
// fused small-batch kernel: a row tile holds at most 32 token rows, so their slot shrinks to 4 KB and six
// stages fit: 192 KB of weights in flight per SM instead of 128 KB, which is what a weight-streaming CTA is
// limited by; 512 bytes of output staging per epilogue warp
using GeomSmall = Geometry<6, 32, 16, G_EPI_WARPS * 512>;

// Row tiles of fused_small_kernel hold at most ST_ROWS = 32 rows (the N of its MMAs); an expert with more rows
// gets several of them (each streams the expert's weights, the later ones out of L2).  F_MAX_TOKENS is the
// capacity of the kernel's counters, not the batch size up to which it is the faster path (the host decides).
constexpr int F_MAX_TOKENS = 256;
// From this batch size up the large-tile GEMM kernels run row tiles of at most 32 rows with the weights on M.
constexpr int SHORT_TILE_MIN_TOKENS = 1;
// Up to here the fused kernel is used unless the caller says otherwise.  Measured against the separate kernels
// (cold step): 9-17 % faster from 34 to 80 tokens with uniform routing, 13-16 % faster at 40-64 tokens with
// skewed routing, 3-6 % slower at exactly 33 and at 80 skewed tokens (hot experts need a second or third
// sub-tile), 10 % slower at 100 skewed tokens, still 9-15 % faster at 128-192 uniform tokens.
constexpr int F_DEFAULT_MAX_TOKENS = 80;
static_assert(GeomSmall::A_ROWS == ST_ROWS, "the token slot of a stage holds one sub-tile");
// Largest batch whose routing and permutation run inside fused_small_kernel, by every CTA for itself (one token
// per warp and round).  Measured against a routing kernel in front: 4-6 us faster per forward up to 13 tokens,
// equal at 20, 1-6 us slower from 24 tokens up, where a CTA needs two to three rounds.
constexpr int F_ROUTE_MAX_TOKENS = 16;
static_assert(F_ROUTE_MAX_TOKENS <= RP_CTA_MAX_TOKENS, "capacity of route_permute_in_cta");
static_assert(RP_CTA_SCRATCH_INTS * 4 <= GeomSmall::STAGE_BYTES, "the routing scratch lives in the first pipeline stage");

constexpr int WM_TOKENS = 32;                       // weights-on-M tiles: N of the MMA, token rows of a tile
constexpr int WM_BUF_COLS = 2 * WM_TOKENS;          // their TMEM columns per K-block: two weight-row blocks

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
    const int* tile_row0;     // fused kernel: first padded row of each (sub-)tile; else null: tile * TILE_M
    int wm_rows;              // large-tile kernel: row tiles with at most this many rows (0 or 32) run with the
                              // weights on the M side of the MMAs, see epilogue_tile_wm
    const float* a_scale_t;   // [num_kb, row_cap]
    const float* w_scale;     // [E_loc, w_rows/128, num_kb]
    uint8_t* out_fp8;         // GEMM1: [row_cap, I] e4m3
    float* out_scale_t;       // GEMM1: [I/128, row_cap]
    __nv_bfloat16* out_bf16;  // GEMM2: tile-blocked rows, see y_block_offset()
    int* status;
    long long wait_limit;     // clocks a bounded wait may spin (WAIT_LIMIT_CLOCKS outside of tests)
    int fault_skip_it;        // test hook: the producer stops before this pipeline iteration (-1: never)
};

// What fused_small_kernel needs beyond the two GemmArgs.
struct FusedArgs {
    int T, H, scale_layout;
    const uint8_t* hidden;        // e4m3 [T, H] token-major activations
    const float* hidden_scale;    // [T, H/128] or [H/128, T]
    const int* row_token;         // padded row -> token
    const int* slot_to_row;       // [T*8]
    const float* topk_w;          // [T*8]
    const int* tok_nlocal;        // [T] local slots of each token
    int* ready;                   // [row tiles] GEMM1 column tiles stored, zero at launch
    int* tok_done;                // [T, H/256] GEMM2 rows stored per (token, column tile), zero at launch
    __nv_bfloat16* out;           // bf16 [T, H]
    // Routing and permutation inside the kernel (route != 0): every CTA computes stages 1 and 2 for itself.
    int route, E_loc, expert_offset, row_cap;
    const float* logits;          // [T, 256]
    const __nv_bfloat16* bias;    // [256]
    float scaling;
    int* topk_idx;                // [T*8] out
    float* topk_w_out;            // [T*8] out (the same buffer as topk_w)
    PermuteMeta meta;
    int* counters_next;           // the counter set of the NEXT fused call, zeroed by CTA 0 of this one
    int num_counters;
    // K split of very small batches (T <= SPLIT_MAX_TOKENS, few tiles): the parts of a tile store their per-K-block
    // partial sums here, [tile][K-block][weight-row block][128 rows][4 tokens] fp32 per GEMM, and count themselves
    float* raw[2];
    int* part_done[2];            // [tiles] per GEMM, zero at launch (part of the counter set)
    int split;                    // 1: the split may be used by this call
};
constexpr int SPLIT_MAX_TOKENS = 4;                       // rows of a tile whose K range may be split
constexpr int SPLIT_MAX_TILES = 74;                       // a split needs at least two CTAs per tile
constexpr int SPLIT_RAW_FLOATS = 2 * SPLIT_MAX_TOKENS * 128;  // per tile and K-block
constexpr int SPLIT_MAX_KB = 64;                          // K-blocks of a GEMM whose tiles may be split

struct GemmCtrl {
    uint64_t full[G_MAX_STAGES];   // stage filled (TMA transaction bytes)
    uint64_t done[G_MAX_STAGES];   // the MMAs that read the stage have finished: stage free AND accumulator ready
    uint64_t tmem_empty[G_MAX_STAGES];   // accumulator buffers: two, or one per stage (weights-on-M roles)
    uint64_t amax_bar[2];
    uint64_t drain_bar[2];
    uint64_t sync_bar[2];      // fused kernel: rendezvous of the epilogue warps at the end of a tile
    uint32_t tmem_slot;
    int abort_flag;
    int split_last;            // fused kernel, K split: this CTA stored the last part of the tile
};
static_assert(sizeof(GemmCtrl) <= G_CTRL_BYTES, "control block too large");

__device__ __forceinline__ void raise(GemmCtrl* c, int* status, int code) {
    *reinterpret_cast<volatile int*>(&c->abort_flag) = 1;
    atomicCAS(status, DEV_OK, code);
}

// Byte offset of the 32-byte group holding columns [16*c16, 16*c16+16) of padded row r in the
// tile-blocked bf16 output of GEMM2 (n_tiles = H / 256 column tiles).
__host__ __device__ __forceinline__ size_t y_block_offset(int r, int c16, int n_tiles) {
    const int m_tile = r / TILE_M, quad = (r % TILE_M) / 32, lane = r % 32;
    const int n = c16 / 16, half = (c16 % 16) / 8, q = c16 % 8;
    return (((static_cast<size_t>(m_tile) * n_tiles + n) * 2 + half) * 4 + quad) * 8192 + q * 1024 + lane * 32;
}

// The CTA's carve-up of shared memory and the values every role needs.
struct Cta {
    float* scale_ring;
    uint8_t* store_stage;
    float* amax_x;             // [2][2][TILE_M] GEMM1 row-amax exchange
    GemmCtrl* ctrl;
    volatile int* abort_flag;
    uint32_t smem_base, tmem_base;
    long long limit;
    int warp, lane;
};

// Tiles first, first + stride, ... below count.
struct TileRange {
    int first, count, stride;
};

// Very small batches of the fused kernel: a tile's K range is cut into `parts` pieces of `len` K-blocks that
// different CTAs work on (see epilogue_tile_wm).  parts = 1: a work item is a whole tile.
struct KSplit {
    int parts, len;
};
__device__ __forceinline__ KSplit ksplit_none(int num_kb) { return KSplit{1, num_kb}; }
// as many parts as keep every CTA at one item at most, eight at most
__device__ __forceinline__ KSplit ksplit_for(int num_kb, int tiles, int grid, bool allowed) {
    int want = (allowed && tiles > 0) ? grid / tiles : 1;
    want = want < 1 ? 1 : (want > 8 ? 8 : want);
    const int len = (num_kb + want - 1) / want;
    return KSplit{(num_kb + len - 1) / len, len};
}

template <class GEO>
__device__ __forceinline__ void gemm_cta_setup(Cta& c, uint8_t* smem_raw, int full_count) {
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    c.scale_ring = reinterpret_cast<float*>(smem + GEO::STAGES * GEO::STAGE_BYTES);
    c.store_stage = smem + GEO::STAGES * GEO::STAGE_BYTES + GEO::SCALE_SLOTS * GEO::SCALE_BYTES;
    c.amax_x = reinterpret_cast<float*>(c.store_stage + GEO::STORE_BYTES);
    c.ctrl = reinterpret_cast<GemmCtrl*>(c.store_stage + GEO::STORE_BYTES + G_AMAX_BYTES);
    c.abort_flag = &c.ctrl->abort_flag;
    c.smem_base = smem_u32(smem);
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    GemmCtrl* ctrl = c.ctrl;
    if (threadIdx.x == 0) {
        for (int s = 0; s < GEO::STAGES; ++s) {
            mbar_init(smem_u32(&ctrl->full[s]), full_count);
            mbar_init(smem_u32(&ctrl->done[s]), 1);
        }
        for (int b = 0; b < G_MAX_STAGES; ++b) mbar_init(smem_u32(&ctrl->tmem_empty[b]), G_EPI_WARPS);
        mbar_init(smem_u32(&ctrl->amax_bar[0]), G_EPI_WARPS * 32);
        mbar_init(smem_u32(&ctrl->amax_bar[1]), G_EPI_WARPS * 32);
        mbar_init(smem_u32(&ctrl->drain_bar[0]), 1);
        mbar_init(smem_u32(&ctrl->drain_bar[1]), 1);
        mbar_init(smem_u32(&ctrl->sync_bar[0]), G_EPI_WARPS * 32);
        mbar_init(smem_u32(&ctrl->sync_bar[1]), G_EPI_WARPS * 32);
        ctrl->abort_flag = 0;
        mbar_fence_init();
    }
    if (c.warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_slot), G_TMEM_COLS);
        tmem_relinquish();
    }
}

// ---------------- TMA producer (one thread) ----------------
// MODE 1: weight tile = 4 x 64 weight rows (gate[0,64) | up[0,64) | gate[64,128) | up[64,128) of the tile's 128
// columns; in the fused kernel gate[0,128) | up[0,128)); MODE 2: 2 x 128 rows.  FUSED and MODE 1: the token
// rows and the scales come from the gather warp instead; FUSED and MODE 2: the tile's token rows are GEMM1's
// output and must have been stored.
template <int MODE, bool FUSED, class GEO>
__device__ __forceinline__ void producer_tiles(const Cta& c, const CUtensorMap* tmA, const CUtensorMap* tmB,
                                               const GemmArgs& g, const FusedArgs* f, int ready_target, TileRange tr,
                                               uint32_t& it, bool& ok, const CUtensorMap* tmA_short = nullptr,
                                               KSplit ks = KSplit{1, 1 << 30}) {
    GemmCtrl* ctrl = c.ctrl;
    for (int item = tr.first; item < tr.count && ok; item += tr.stride) {
        const int tile = item / ks.parts, kb0 = (item - tile * ks.parts) * ks.len;
        const int kb1 = min(g.num_kb, kb0 + ks.len);
        const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
        const int wrow = __ldcg(g.tile_expert + m_tile) * g.w_rows_per_expert;
        const int row0 = FUSED ? __ldcg(g.tile_row0 + m_tile) : m_tile * TILE_M;
        const float* a_sc = g.a_scale_t + row0;
        // a short row tile of the large-tile kernel: 32 token rows fetched, weights laid out for the M side
        const bool wm = !FUSED && g.wm_rows > 0 && __ldcg(g.tile_rows + m_tile) <= g.wm_rows;
        const uint32_t TX_BYTES = (FUSED && MODE == 1) ? G_B_BYTES
                                  : wm ? WM_TOKENS * G_BLOCK_K + WM_TOKENS * 4 + G_B_BYTES
                                       : GEO::STAGE_BYTES + GEO::SCALE_BYTES;
        // claim the stage of pipeline iteration j: wait until its last reader has finished, announce the bytes
        auto claim = [&](uint32_t j) -> bool {
            const uint32_t s = j % GEO::STAGES, ph = (j / GEO::STAGES) & 1;
            if (MODE == 1 && static_cast<int>(j) == g.fault_skip_it) return false;  // test hook: never filled
            if (!mbar_wait(smem_u32(&ctrl->done[s]), ph ^ 1, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_PRODUCER);
                return false;
            }
            mbar_expect_tx(smem_u32(&ctrl->full[s]), TX_BYTES);
            return true;
        };
        auto load_b = [&](uint32_t j, int kb) {
            const uint32_t s = j % GEO::STAGES, bar = smem_u32(&ctrl->full[s]);
            const uint32_t b_dst = c.smem_base + s * GEO::STAGE_BYTES + GEO::A_BYTES;
            const int k0 = kb * G_BLOCK_K;
            if (MODE == 1) {
                const int gr = wrow + g.gate_row0 + n * 128, ur = wrow + g.up_row0 + n * 128;
                // weights on N: gate[0,64) | up[0,64) | gate[64,128) | up[64,128); on M (fused kernel):
                // gate[0,128) | up[0,128)
                tma_load_2d(b_dst, tmB, k0, gr, bar);
                tma_load_2d(b_dst + G_B_BYTES / 4, tmB, k0, (FUSED || wm) ? gr + 64 : ur, bar);
                tma_load_2d(b_dst + G_B_BYTES / 2, tmB, k0, (FUSED || wm) ? ur : gr + 64, bar);
                tma_load_2d(b_dst + 3 * G_B_BYTES / 4, tmB, k0, ur + 64, bar);
            } else {
                const int br = wrow + n * G_TILE_N;
                tma_load_2d(b_dst, tmB, k0, br, bar);
                tma_load_2d(b_dst + G_B_BYTES / 2, tmB, k0, br + 128, bar);
            }
        };
        auto load_a = [&](uint32_t j, int kb) {  // the A rows and their scales of the K-block
            const uint32_t s = j % GEO::STAGES, bar = smem_u32(&ctrl->full[s]);
            // (the scale slot is free: the ring exceeds the stages + accumulators the producer can be ahead
            // of the epilogue)
            bulk_load_1d(smem_u32(c.scale_ring + (j % GEO::SCALE_SLOTS) * GEO::A_ROWS),
                         a_sc + static_cast<size_t>(kb) * g.row_cap, wm ? WM_TOKENS * 4 : GEO::SCALE_BYTES, bar);
            tma_load_2d(c.smem_base + s * GEO::STAGE_BYTES, wm ? tmA_short : tmA, kb * G_BLOCK_K, row0, bar);
        };
        int kb = kb0;
        if (FUSED && MODE == 2) {
            // The tile's A rows are GEMM1's output and must have been stored; its weights need not wait for
            // that, so the B tiles of the first K-blocks go out before the counter is looked at.
            const int npre = kb1 - kb0 < GEO::STAGES ? kb1 - kb0 : GEO::STAGES;
            for (int k = 0; k < npre && ok; ++k) {
                ok = claim(it + k);
                if (ok) load_b(it + k, kb0 + k);
            }
            if (!ok) break;
            if (!wait_counter(f->ready + m_tile, ready_target, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_READY);
                ok = false;
                break;
            }
            fence_proxy_async();  // the rows were stored by other CTAs' copy engines; order our copies behind the acquire
            for (int k = 0; k < npre; ++k) load_a(it + k, kb0 + k);
            it += npre;
            kb = kb0 + npre;
        }
        for (; kb < kb1 && ok; ++kb, ++it) {
            ok = claim(it);
            if (!ok) break;
            if (!(FUSED && MODE == 1)) load_a(it, kb);
            load_b(it, kb);
        }
    }
}

// Before the producer thread may reach the end of the kernel every copy it issued has to have landed (bounded
// wait).  On the regular path the MMA issuers have consumed all of them long ago and these waits fall through;
// after an abort raised by any role they are what keeps the copy engine from writing into shared memory of a
// CTA that has exited.
template <class GEO>
__device__ __forceinline__ void producer_drain(const Cta& c, int* status, uint32_t it) {
    int zero = 0;
    const uint32_t n_back = it < GEO::STAGES ? it : GEO::STAGES;
    for (uint32_t j = it - n_back; j < it; ++j)
        if (!mbar_wait(smem_u32(&c.ctrl->full[j % GEO::STAGES]), (j / GEO::STAGES) & 1, &zero, c.limit))
            atomicCAS(status, DEV_OK, DEV_TIMEOUT_DRAIN);
}

// ---------------- MMA issuers (two threads) ----------------
// Two threads share the issue work: `mine` = 0 takes the even K-blocks (TMEM buffer 0), 1 the odd ones (buffer
// 1).  A commit only tracks the MMAs of its own thread, so while one thread pays for its commit and waits the
// other keeps the tensor pipe fed.
template <class GEO>
__device__ __forceinline__ void issuer_tiles(const Cta& c, const GemmArgs& g, TileRange tr, uint32_t mine,
                                             uint32_t& it, bool& ok) {
    GemmCtrl* ctrl = c.ctrl;
    const uint32_t idesc = umma_idesc_f8(TILE_M, G_TILE_N), idesc_wm = umma_idesc_f8(TILE_M, WM_TOKENS);
    for (int tile = tr.first; tile < tr.count && ok; tile += tr.stride) {
        // a short row tile: the stage's weight rows are the M side (two blocks of 128), its 32 token rows the N
        // side; the accumulator is the first 64 columns of the buffer
        const bool wm = g.wm_rows > 0 && __ldcg(g.tile_rows + tile / g.n_tiles) <= g.wm_rows;
        for (int kb = 0; kb < g.num_kb; ++kb, ++it) {
            if ((it & 1) != mine) continue;
            const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1;
            const uint32_t b = it & 1, bph = (it >> 1) & 1;
            // The stage has normally landed long before the accumulator is handed back, so that
            // wait comes first and only the hand-over itself is left on the critical path.
            const uint32_t a_addr = c.smem_base + s * GEO::STAGE_BYTES;
            const uint64_t a_desc = umma_desc_sw128(a_addr);  // 128 rows from here, fetched or not
            const uint64_t b_desc = umma_desc_sw128(a_addr + GEO::A_BYTES);
            const uint32_t d_tmem = c.tmem_base + b * G_TILE_N;
            if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_MMA_SMEM);
                ok = false;
                break;
            }
            if (!mbar_wait(smem_u32(&ctrl->tmem_empty[b]), bph ^ 1, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_MMA_TMEM);
                ok = false;
                break;
            }
            tc_fence_after();
            if (wm) {
                const uint64_t w1_desc = umma_desc_sw128(a_addr + GEO::A_BYTES + G_B_BYTES / 2);
#pragma unroll
                for (int k = 0; k < G_BLOCK_K / 32; ++k) umma_f8(d_tmem, b_desc + 2 * k, a_desc + 2 * k, idesc_wm, k > 0);
#pragma unroll
                for (int k = 0; k < G_BLOCK_K / 32; ++k)
                    umma_f8(d_tmem + WM_TOKENS, w1_desc + 2 * k, a_desc + 2 * k, idesc_wm, k > 0);
            } else {
#pragma unroll
                for (int k = 0; k < G_BLOCK_K / 32; ++k)  // 32 K-bytes per instruction: +2 in 16-B units
                    umma_f8(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k > 0);
            }
            umma_commit(smem_u32(&ctrl->done[s]));
        }
    }
}

// After an abort: let issued MMAs retire before TMEM is released.
__device__ __forceinline__ void issuer_drain(const Cta& c, uint32_t mine, bool ok) {
    if (!ok || *c.abort_flag) {
        umma_commit(smem_u32(&c.ctrl->drain_bar[mine]));
        int zero = 0;
        mbar_wait(smem_u32(&c.ctrl->drain_bar[mine]), 0, &zero, c.limit);
    }
}

// ---------------- gather warp (fused kernel) ----------------
// GEMM1 tiles: lane l copies 16-byte chunk (l & 7) of rows (l >> 3) + 4 i, i = 0..7, of every K-block from the
// token-major input, and the scale of row l.  The stage uses the 128-byte swizzle of the TMA tiles: chunk c of
// row r sits at r * 128 + ((c ^ (r & 7)) << 4), and r & 7 takes only two values per lane (i even / odd).  Rows
// past the tile's valid rows are zero-filled; the stage holds only these 32 rows (see Geometry).  Each lane's arrival on full[s] is triggered by the completion of its copies.
template <class GEO>
__device__ __forceinline__ void gather_tiles(const Cta& c, const GemmArgs& g, const FusedArgs& f, TileRange tr,
                                             uint32_t& it, bool& ok, KSplit ks) {
    GemmCtrl* ctrl = c.ctrl;
    const int lane = c.lane, sub = lane >> 3, chunk = lane & 7;
    const uint32_t dst_even = sub * 128 + ((chunk ^ sub) << 4);
    const uint32_t dst_odd = sub * 128 + ((chunk ^ (sub + 4)) << 4);
    for (int item = tr.first; item < tr.count && ok; item += tr.stride) {
        const int tile = item / ks.parts, kb0 = (item - tile * ks.parts) * ks.len;
        const int kb1 = min(g.num_kb, kb0 + ks.len);
        const int m_tile = tile / g.n_tiles;
        const int rows_valid = __ldcg(g.tile_rows + m_tile);
        // token of row `lane` (scale copy) and source rows of this lane's eight chunks
        const int my_tok = lane < rows_valid ? __ldcg(f.row_token + __ldcg(g.tile_row0 + m_tile) + lane) : -1;
        const uint8_t* src_row[GEO::A_ROWS / 4];
#pragma unroll
        for (int i = 0; i < GEO::A_ROWS / 4; ++i) {
            const int t = __shfl_sync(0xffffffffu, my_tok, sub + 4 * i);
            src_row[i] = t >= 0 ? f.hidden + static_cast<size_t>(t) * f.H + chunk * 16 : nullptr;
        }
        const float* sc_src = nullptr;
        size_t sc_step = 0;
        if (my_tok >= 0) {
            sc_src = f.scale_layout ? f.hidden_scale + my_tok : f.hidden_scale + static_cast<size_t>(my_tok) * g.num_kb;
            sc_step = f.scale_layout ? static_cast<size_t>(f.T) : 1;
        }
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctrl->done[s]), ph ^ 1, c.abort_flag, c.limit))) {
                if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_PRODUCER);
                ok = false;
                break;
            }
            const uint32_t a_dst = c.smem_base + s * GEO::STAGE_BYTES;
#pragma unroll
            for (int i = 0; i < GEO::A_ROWS / 4; ++i)
                cp_async_16(a_dst + i * 512 + ((i & 1) ? dst_odd : dst_even),
                            src_row[i] ? static_cast<const void*>(src_row[i] + kb * G_BLOCK_K)
                                       : static_cast<const void*>(f.hidden),
                            src_row[i] ? 16u : 0u);
            cp_async_4(smem_u32(c.scale_ring + (it % GEO::SCALE_SLOTS) * GEO::A_ROWS + lane),
                       sc_src ? static_cast<const void*>(sc_src + kb * sc_step) : static_cast<const void*>(f.hidden_scale),
                       sc_src ? 4u : 0u);
            cp_async_arrive_noinc(smem_u32(&ctrl->full[s]));
        }
    }
}
// GEMM2 tiles: the producer fetches everything; the lanes only keep the arrival count of full[s] uniform.
template <class GEO>
__device__ __forceinline__ void gather_idle_tiles(const Cta& c, const GemmArgs& g, TileRange tr, uint32_t& it, bool& ok,
                                                  KSplit ks) {
    GemmCtrl* ctrl = c.ctrl;
    for (int item = tr.first; item < tr.count && ok; item += tr.stride) {
        const int kb0 = (item % ks.parts) * ks.len, kb1 = min(g.num_kb, kb0 + ks.len);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
            const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctrl->done[s]), ph ^ 1, c.abort_flag, c.limit))) {
                ok = false;
                break;
            }
            mbar_arrive(smem_u32(&ctrl->full[s]));
        }
    }
}

// Rendezvous of all epilogue threads (an mbarrier, because its wait is bounded: a plain barrier would hold the
// arrived warps for ever if another warp had given up).  Orders the arrived threads' earlier writes before the
// later reads of those that leave.  `n` counts the rendezvous of this thread so far.
__device__ __forceinline__ bool epilogue_rendezvous(const Cta& c, uint32_t& n) {
    const uint32_t bar = smem_u32(&c.ctrl->sync_bar[n & 1]);
    mbar_arrive(bar);
    const bool ok = __all_sync(0xffffffffu, mbar_wait(bar, (n >> 1) & 1, c.abort_flag, c.limit));
    ++n;
    return ok;
}

template <int MODE, bool FUSED, class GEO, bool SHARED, bool SPLIT = false>
__device__ __forceinline__ bool epilogue_tile_wm(const Cta& c, const GemmArgs& g, const FusedArgs* f, int m_tile, int n,
                                                 uint32_t& it, uint32_t& tile_iter, uint32_t& sync_iter, int kb0 = 0,
                                                 int kb1 = -1, int parts = 1);

// ---------------- epilogue warps ----------------
// MODE 1: gate/up projection + SwiGLU + re-quantisation; tmOut describes the e4m3 output [row_cap, I] for
//         64-byte x 32-row TMA stores.
// MODE 2: down projection, bf16 rows out in the tile-blocked layout.
template <int MODE, class GEO>
__device__ __forceinline__ void epilogue_tiles(const Cta& c, const CUtensorMap* tmOut, const GemmArgs& g, TileRange tr,
                                               uint32_t& it, uint32_t& tile_iter, bool& ok) {
    static_assert(GEO::A_ROWS == TILE_M && GEO::STORE_BYTES == G_EPI_WARPS * G_STORE_WARP_BYTES, "full row tiles");
    GemmCtrl* ctrl = c.ctrl;
    const int warp = c.warp, lane = c.lane;
    const int widx = warp - 4;
    const int half = widx >> 2;              // which 128-column half of the tile
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    const int r_in_tile = quad * 32 + lane;  // accumulator row == TMEM lane
    const uint32_t t_lane = c.tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + half * G_HALF_N;
    const size_t row_cap = static_cast<size_t>(g.row_cap);
    float* amax_x = c.amax_x;
    uint8_t* stage = c.store_stage + widx * G_STORE_WARP_BYTES;  // staging of this warp's GEMM1 rows
    const int scale_row = r_in_tile;
    const int num_kb = g.num_kb;
    for (int tile = tr.first; tile < tr.count && ok; tile += tr.stride) {
        const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
        const int e = __ldcg(g.tile_expert + m_tile);
        const int rows_valid = __ldcg(g.tile_rows + m_tile);
        if (g.wm_rows > 0 && rows_valid <= g.wm_rows) {  // a short row tile, worked on with the weights on M
            uint32_t unused = 0;
            ok = epilogue_tile_wm<MODE, false, GEO, true>(c, g, nullptr, m_tile, n, it, tile_iter, unused);
            continue;
        }
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
            const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1, buf = it & 1;
            // Every lane polls (a single polling lane plus a broadcast was measured 2.5 % slower); the vote
            // keeps the warp converged when a wait gives up: either all lanes go on or none does.
            if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctrl->done[s]), ph, c.abort_flag, c.limit))) {
                if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                ok = false;
                break;
            }
            tc_fence_after();
            // The MMA of this K-block has finished, hence its stage -- A, B and the scales -- had landed.
            // (Fetching the scale earlier needs a barrier of its own per ring slot -- on full[s] this warp can
            // be lapped by a whole phase -- and that extra barrier test per K-block was measured to cost the
            // epilogue 110 clocks, 10 % of the kernel: barrier operations of a thread queue behind one another.)
            const float sa = ld_shared_f32(c.scale_ring + (it % GEO::SCALE_SLOTS) * GEO::A_ROWS + scale_row);
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

        if (MODE == 1) {
            // The staging area of this warp was handed to the TMA engine at the end of the previous tile;
            // by now (a whole tile later) that copy has long read it, so this wait does not stall.
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
            const int sw = (lane >> 1) & 3;  // 64-byte swizzle: 16-byte chunk index ^= bits 7..8 of the address
            // SwiGLU on this thread's 64 columns, then the row's 128-wide amax across the two halves
            float cc[64];
            float amax = 0.0f;
#pragma unroll
            for (int j = 0; j < 64; ++j) {
                // silu(g) * u with the hardware exp2 and reciprocal approximations (a few ulp): the
                // tile's tail runs while the tensor pipe idles, so its instruction count matters.
                const float gt = acc[j];
                cc[j] = __fdividef(gt, 1.0f + __expf(-gt)) * acc[64 + j];
                amax = fmaxf(amax, fabsf(cc[j]));
            }
            const uint32_t par = tile_iter & 1;
            amax_x[(par * 2 + half) * TILE_M + r_in_tile] = amax;
            const uint32_t xbar = smem_u32(&ctrl->amax_bar[par]);
            mbar_arrive(xbar);
            if (!__all_sync(0xffffffffu, mbar_wait(xbar, (tile_iter >> 1) & 1, c.abort_flag, c.limit))) {
                if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                ok = false;
                break;
            }
            ++tile_iter;
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
                            make_float2(cc[j] * inv_sc, cc[j + 1] * inv_sc), __NV_SATFINITE, __NV_E4M3);
                        const uint32_t hi = __nv_cvt_float2_to_fp8x2(
                            make_float2(cc[j + 2] * inv_sc, cc[j + 3] * inv_sc), __NV_SATFINITE, __NV_E4M3);
                        w[i] = lo | (hi << 16);
                    }
                    *reinterpret_cast<uint4*>(stage + lane * 64 + ((q ^ sw) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(tmOut, smem_u32(stage), n * 128 + half * 64, m_tile * TILE_M + quad * 32);
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
}

// ================= weights on M: the roles of the fused small-batch kernel =================
// With at most 32 token rows in a tile, a 128 x 256 accumulator holds 96 rows of padding, and the two
// epilogue warps that own the 32 real rows (TMEM lanes) do all of the per-K-block promotion.  Here the
// operands are swapped instead: the 256 weight rows of the tile are the M side (two MMAs of M = 128 per K
// step), the 32 token rows the N side.  An accumulator is then 128 lanes x 32 columns per weight-row block,
// 64 columns per K-block: every stage gets an accumulator buffer of its own (6 x 64 of the 512 columns),
// so the hand-over latencies overlap six deep, and every epilogue thread owns one weight row (an output
// column) for 16 tokens -- 32 loads and 32 FMAs per K-block instead of 128, evenly over all eight warps.
// Element for element the arithmetic is the one of the other orientation.
static_assert(G_MAX_STAGES * WM_BUF_COLS <= static_cast<int>(G_TMEM_COLS), "one accumulator buffer per stage");

template <class GEO>
__device__ __forceinline__ void issuer_tiles_wm(const Cta& c, const GemmArgs& g, TileRange tr, uint32_t mine,
                                                uint32_t& it, bool& ok, KSplit ks) {
    static_assert(GEO::A_ROWS == WM_TOKENS, "the token slot of a stage is the MMA's N operand");
    static_assert(GEO::SCALE_SLOTS >= 2 * GEO::STAGES + 1, "the gather may be two pipelines ahead of the epilogue");
    GemmCtrl* ctrl = c.ctrl;
    const uint32_t idesc = umma_idesc_f8(TILE_M, WM_TOKENS);
    for (int item = tr.first; item < tr.count && ok; item += tr.stride) {
        const int kb0 = (item % ks.parts) * ks.len, kb1 = min(g.num_kb, kb0 + ks.len);
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
            if ((it & 1) != mine) continue;
            const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1;
            const uint32_t tok_addr = c.smem_base + s * GEO::STAGE_BYTES;
            const uint64_t t_desc = umma_desc_sw128(tok_addr);
            const uint64_t w0_desc = umma_desc_sw128(tok_addr + GEO::A_BYTES);
            const uint64_t w1_desc = umma_desc_sw128(tok_addr + GEO::A_BYTES + G_B_BYTES / 2);
            const uint32_t d_tmem = c.tmem_base + s * WM_BUF_COLS;
            if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_MMA_SMEM);
                ok = false;
                break;
            }
            // the buffer of this stage was last used one pipeline round ago
            if (!mbar_wait(smem_u32(&ctrl->tmem_empty[s]), ph ^ 1, c.abort_flag, c.limit)) {
                raise(ctrl, g.status, DEV_TIMEOUT_MMA_TMEM);
                ok = false;
                break;
            }
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < G_BLOCK_K / 32; ++k) umma_f8(d_tmem, w0_desc + 2 * k, t_desc + 2 * k, idesc, k > 0);
#pragma unroll
            for (int k = 0; k < G_BLOCK_K / 32; ++k)
                umma_f8(d_tmem + WM_TOKENS, w1_desc + 2 * k, t_desc + 2 * k, idesc, k > 0);
            umma_commit(smem_u32(&ctrl->done[s]));
        }
    }
}

// MODE 1: weight-row block 0 = 128 gate rows, block 1 = the matching 128 up rows; SwiGLU, re-quantisation per
//         token over the tile's 128 output columns, e4m3 bytes and scales out, tile announced in f->ready.
// MODE 2: blocks 0 / 1 = output columns [0,128) / [128,256) of the tile; bf16 out in the tile-blocked layout,
//         then the per-(token, column tile) counters and the combine of the tokens this CTA completes.
// One tile; false: a wait gave up (the code is in the status word).  SHARED: the tile runs inside the large-tile
// kernel, between tiles of the other orientation -- its accumulators are the first 64 columns of the two
// 256-column buffers of that kernel, handed over through the same two barriers, and its staging is the first
// 512 bytes of the warp's own TMA staging area.
// SPLIT (fused kernel, batches of at most SPLIT_MAX_TOKENS tokens with few tiles, parts > 1): this call covers the
// K-blocks [kb0, kb1) only.  It stores every K-block's partial sums as they come out of the tensor memory, not
// yet multiplied by the scales; the CTA that stores the last part of a tile -- found with a counter, nobody
// waits -- then runs the whole promotion from the stored partial sums, K-block after K-block in the one order
// the unsplit tile uses, and finishes the tile.  Every fp32 operation is the one of the unsplit tile.
template <int MODE, bool FUSED, class GEO, bool SHARED, bool SPLIT>
__device__ __forceinline__ bool epilogue_tile_wm(const Cta& c, const GemmArgs& g, const FusedArgs* f, int m_tile, int n,
                                                 uint32_t& it, uint32_t& tile_iter, uint32_t& sync_iter, int kb0, int kb1,
                                                 int parts) {
    static_assert(!SPLIT || FUSED, "only the fused kernel cuts K ranges");
    GemmCtrl* ctrl = c.ctrl;
    const int warp = c.warp, lane = c.lane;
    const int th = (warp - 4) >> 2;          // which 16 of the tile's 32 token rows
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    // (lane l of quadrant q holds weight row 32 q + l of each 128-row block)
    const uint32_t t_lane = c.tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + th * 16;
    const size_t row_cap = static_cast<size_t>(g.row_cap);
    uint32_t* amax_x = reinterpret_cast<uint32_t*>(c.amax_x);   // [2 parities][256]: [2 token halves][4 quadrants][16] used
    const int num_kb = g.num_kb;
    const int e = __ldcg(g.tile_expert + m_tile);
    const int rows_valid = __ldcg(g.tile_rows + m_tile);
    const int sblocks = g.w_rows_per_expert / 128;
    const float* ws0;  // weight-scale rows of block 0 / block 1
    const float* ws1;
    if (MODE == 1) {
        ws0 = g.w_scale + (static_cast<size_t>(e) * sblocks + g.gate_row0 / 128 + n) * num_kb;
        ws1 = g.w_scale + (static_cast<size_t>(e) * sblocks + g.up_row0 / 128 + n) * num_kb;
    } else {
        ws0 = g.w_scale + (static_cast<size_t>(e) * sblocks + 2 * n) * num_kb;
        ws1 = ws0 + num_kb;
    }
    float acc[32];  // [0,16): block 0, [16,32): block 1, for tokens 16 th .. 16 th + 15
#pragma unroll
    for (int j = 0; j < 32; ++j) acc[j] = 0.0f;

    const int kb_end = kb1 < 0 ? num_kb : kb1;
    const int tile_row0 = SHARED ? m_tile * TILE_M : __ldcg(g.tile_row0 + m_tile);
    float4* raw = nullptr;  // this tile's stored partial sums (four tokens each): this thread's weight row
    if (SPLIT)
        raw = reinterpret_cast<float4*>(f->raw[MODE - 1] + static_cast<size_t>(m_tile * g.n_tiles + n) * num_kb * SPLIT_RAW_FLOATS) +
              quad * 32 + lane;
    float s0 = __ldg(ws0 + kb0), s1 = __ldg(ws1 + kb0);
    for (int kb = kb0; kb < kb_end; ++kb, ++it) {
        const float w0 = s0, w1 = s1;
        if (kb + 1 < kb_end) {
            s0 = __ldg(ws0 + kb + 1);
            s1 = __ldg(ws1 + kb + 1);
        }
        const uint32_t s = it % GEO::STAGES, ph = (it / GEO::STAGES) & 1;
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&ctrl->done[s]), ph, c.abort_flag, c.limit))) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        tc_fence_after();
        // the MMAs of this K-block have finished, hence its stage -- tokens, weights and scales -- had landed
        const float4* sp = reinterpret_cast<const float4*>(c.scale_ring + (it % GEO::SCALE_SLOTS) * GEO::A_ROWS + th * 16);
        float sa[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 x = sp[q];
            sa[4 * q] = x.x;
            sa[4 * q + 1] = x.y;
            sa[4 * q + 2] = x.z;
            sa[4 * q + 3] = x.w;
        }
        float v[32];
        const uint32_t buf = SHARED ? (it & 1) : s, t_buf = t_lane + buf * (SHARED ? G_TILE_N : WM_BUF_COLS);
        tmem_ld16x2(t_buf, t_buf + WM_TOKENS, v);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->tmem_empty[buf]));
        if (SPLIT) {
            if (th == 0) {  // (all four token columns; those past the tile's rows are never used)
                raw[(kb * 2 + 0) * 128] = make_float4(v[0], v[1], v[2], v[3]);
                raw[(kb * 2 + 1) * 128] = make_float4(v[16], v[17], v[18], v[19]);
            }
        } else {
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                acc[t] = fmaf(v[t], sa[t] * w0, acc[t]);
                acc[16 + t] = fmaf(v[16 + t], sa[t] * w1, acc[16 + t]);
            }
        }
    }

    if (SPLIT) {
        // count this part; the last one goes on, the others are done with the tile
        __threadfence();
        if (!epilogue_rendezvous(c, sync_iter)) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        if (warp == 4 && lane == 0) {
            __threadfence();
            const int before = atomicAdd(f->part_done[MODE - 1] + m_tile * g.n_tiles + n, 1);
            *reinterpret_cast<volatile int*>(&ctrl->split_last) = (before == parts - 1);
        }
        if (!epilogue_rendezvous(c, sync_iter)) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        if (!*reinterpret_cast<volatile int*>(&ctrl->split_last)) return true;
        __threadfence();
        // The finisher.  The scales of the tile's (at most four) tokens and of the two weight-row blocks go to
        // shared memory first (the row-maximum exchange area is free here: every warp has left the previous
        // tile); then the warps of token half 0 promote block 0 and those of half 1 block 1, K-block after
        // K-block, and half 1 hands its sums to half 0 through the staging area.
        float* sa_s = c.amax_x;                                   // [num_kb][4]
        float* w_s = c.amax_x + SPLIT_MAX_TOKENS * num_kb;        // [2][num_kb]
        static_assert(G_AMAX_BYTES >= (SPLIT_MAX_TOKENS + 2) * SPLIT_MAX_KB * 4, "scales of a tile's K-blocks");
        for (int i = threadIdx.x - 128; i < SPLIT_MAX_TOKENS * num_kb; i += G_EPI_WARPS * 32) {
            const int kb = i / SPLIT_MAX_TOKENS, t = i - kb * SPLIT_MAX_TOKENS;
            float v = 0.0f;
            if (t < rows_valid) {
                if (MODE == 1) {
                    const int tok = __ldcg(f->row_token + tile_row0 + t);
                    v = __ldcg(f->scale_layout ? f->hidden_scale + static_cast<size_t>(kb) * f->T + tok
                                               : f->hidden_scale + static_cast<size_t>(tok) * num_kb + kb);
                } else {
                    v = __ldcg(g.a_scale_t + static_cast<size_t>(kb) * row_cap + tile_row0 + t);
                }
            }
            sa_s[i] = v;
        }
        for (int i = threadIdx.x - 128; i < 2 * num_kb; i += G_EPI_WARPS * 32)
            w_s[i] = __ldg((i < num_kb ? ws0 : ws1 - num_kb) + i);
        if (!epilogue_rendezvous(c, sync_iter)) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f);
        {
            const float4* rp = raw + th * 128;
            const float* wp = w_s + th * num_kb;
#pragma unroll 28
            for (int kb = 0; kb < num_kb; ++kb) {
                const float4 r = __ldcg(rp + kb * 2 * 128);
                const float4 sa = *reinterpret_cast<const float4*>(sa_s + kb * SPLIT_MAX_TOKENS);
                const float w = wp[kb];
                a4.x = fmaf(r.x, sa.x * w, a4.x);
                a4.y = fmaf(r.y, sa.y * w, a4.y);
                a4.z = fmaf(r.z, sa.z * w, a4.z);
                a4.w = fmaf(r.w, sa.w * w, a4.w);
            }
        }
        float4* xchg = reinterpret_cast<float4*>(c.store_stage);  // [128 weight rows]: half 0's warps read their own staging
        if (th == 1) xchg[quad * 32 + lane] = a4;
        if (!epilogue_rendezvous(c, sync_iter)) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        if (th == 0) {
            const float4 b4 = xchg[quad * 32 + lane];
            acc[0] = a4.x, acc[1] = a4.y, acc[2] = a4.z, acc[3] = a4.w;
            acc[16] = b4.x, acc[17] = b4.y, acc[18] = b4.z, acc[19] = b4.w;
        }
        __syncwarp();
    }

    const size_t row0 = static_cast<size_t>(tile_row0) + th * 16;  // padded row of this thread's token 0
    const uint32_t wst_off = (warp - 4) * (SHARED ? G_STORE_WARP_BYTES : 512);  // this warp's staging
    if (SHARED) {  // the warp's last TMA store may still be reading the area
        if (lane == 0) bulk_wait_read_all();
        __syncwarp();
    }
    const int valid = min(16, rows_valid - th * 16);                     // tokens of this thread that exist
    if (MODE == 1) {
        float cc[16];
        uint32_t wmax[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            const float gt = acc[t];
            cc[t] = __fdividef(gt, 1.0f + __expf(-gt)) * acc[16 + t];
            // |x| as an integer orders like the float: the warp's maximum over its 32 output columns
            wmax[t] = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(cc[t])));
        }
        const uint32_t par = tile_iter & 1;
        // (inside the half of the exchange area that belongs to this parity in the other orientation as well)
        uint32_t* xq = amax_x + par * (2 * TILE_M) + th * 64;
        {
            uint32_t mine = 0;
#pragma unroll
            for (int t = 0; t < 16; ++t)
                if (lane == t) mine = wmax[t];
            if (lane < 16) xq[quad * 16 + lane] = mine;
        }
        const uint32_t xbar = smem_u32(&ctrl->amax_bar[par]);
        mbar_arrive(xbar);
        if (!__all_sync(0xffffffffu, mbar_wait(xbar, (tile_iter >> 1) & 1, c.abort_flag, c.limit))) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        ++tile_iter;
        // lane t < 16 owns the scale of token t's 128-column block; everybody fetches its reciprocal
        float my_sc = 1.0f, my_inv = 1.0f;
        if (lane < 16) {
            const volatile uint32_t* xv = xq + lane;
            const float amax = __uint_as_float(max(max(xv[0], xv[16]), max(xv[32], xv[48])));
            my_sc = (amax == 0.0f) ? 1.0f : __fdiv_rn(amax, 448.0f);
            my_inv = __frcp_rn(my_sc);
        }
        // Narrow global stores are slow (a warp's 32 single bytes cost tens of clocks): the codes are
        // transposed through this warp's 512 bytes of staging, [16 tokens][32 columns], and leave as
        // 16-byte stores -- lane l carries 16 columns of token l / 2.
        uint8_t* wst = c.store_stage + wst_off;
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            const float inv_sc = __shfl_sync(0xffffffffu, my_inv, t);
            wst[t * 32 + lane] =
                static_cast<uint8_t>(__nv_cvt_float_to_fp8(cc[t] * inv_sc, __NV_SATFINITE, __NV_E4M3));
        }
        __syncwarp();
        if ((lane >> 1) < valid)
            *reinterpret_cast<uint4*>(g.out_fp8 + (row0 + (lane >> 1)) * g.out_cols + n * 128 + quad * 32 + (lane & 1) * 16) =
                *reinterpret_cast<const uint4*>(wst + (lane >> 1) * 32 + (lane & 1) * 16);
        if (quad == 0 && lane < valid) g.out_scale_t[static_cast<size_t>(n) * row_cap + row0 + lane] = my_sc;
        __syncwarp();
        // (The rows are read by copy engines, of other CTAs or of the next kernel: plain stores here,
        // asynchronous-proxy loads there.)
        fence_proxy_async();
        if (FUSED) {
            // Announce the tile: every thread's stores are fenced before the epilogue warps meet, and the
            // announcing thread fences once more behind the barrier.
            __threadfence();
            if (!epilogue_rendezvous(c, sync_iter)) {
                if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
                return false;
            }
            if (warp == 4 && lane == 0) {
                __threadfence();
                atomicAdd(f->ready + m_tile, 1);
            }
        }
    } else {
        // bf16 out through this warp's 512 bytes of staging, eight tokens x 32 columns at a time, so that
        // the rows leave as 16-byte stores: lane l carries 8 columns of token l / 4 (half of a 32-byte
        // group of the tile-blocked layout)
        __nv_bfloat16* wst = reinterpret_cast<__nv_bfloat16*>(c.store_stage + wst_off);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int t = 0; t < 8; ++t) wst[t * 32 + lane] = __float2bfloat16_rn(acc[j * 16 + h * 8 + t]);
                __syncwarp();
                const int t = h * 8 + (lane >> 2), ch0 = quad * 32 + (lane & 3) * 8;
                if (t < valid)
                    *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(g.out_bf16) +
                                              y_block_offset(static_cast<int>(row0) + t, n * 16 + j * 8 + (ch0 >> 4), g.n_tiles) +
                                              (ch0 & 15) * 2) =
                        *reinterpret_cast<const uint4*>(wst + (lane >> 2) * 32 + (lane & 3) * 8);
                __syncwarp();
            }
        }
        // Stage 4 without a kernel of its own.  Once the tile is stored and fenced, the thread of each valid
        // row bumps the counter of (its token, this column tile); whoever brings it to the token's number of
        // local slots knows that all of the token's rows for these 256 columns are in memory and sums
        // them, in routing order, exactly as combine_kernel does.
        if (!FUSED) return true;  // (one GEMM per launch: the combine is a kernel of its own)
        __threadfence();
        if (!epilogue_rendezvous(c, sync_iter)) {
            if (lane == 0) raise(ctrl, g.status, DEV_TIMEOUT_EPILOGUE);
            return false;
        }
        {
            // epilogue warp w looks after the rows w, w + 8, w + 16, w + 24 of the tile (lanes 0..3), so up
            // to eight completed tokens are summed at the same time
            int tok = -1;
            bool last = false;
            const int r_mine = (warp - 4) + 8 * lane;
            if (lane < 4 && r_mine < rows_valid) {
                tok = __ldcg(f->row_token + tile_row0 + r_mine);
                __threadfence();
                const int before = atomicAdd(f->tok_done + static_cast<size_t>(tok) * g.n_tiles + n, 1);
                last = before == __ldcg(f->tok_nlocal + tok) - 1;
            }
            uint32_t todo = __ballot_sync(0xffffffffu, last);
            if (todo) __threadfence();
            while (todo) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int t = __shfl_sync(0xffffffffu, tok, src);
                // lane l owns columns n*256 + 8 l .. + 8: half of the 32-byte group n*16 + l/2.  All loads
                // first, then the sum in routing order.
                const int4 ra = __ldcg(reinterpret_cast<const int4*>(f->slot_to_row) + 2 * t);
                const int4 rb = __ldcg(reinterpret_cast<const int4*>(f->slot_to_row) + 2 * t + 1);
                const float4 wa = __ldcg(reinterpret_cast<const float4*>(f->topk_w) + 2 * t);
                const float4 wb = __ldcg(reinterpret_cast<const float4*>(f->topk_w) + 2 * t + 1);
                const int rr[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
                const float ww[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
                uint4 u[8];
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (rr[j] >= 0)
                        u[j] = __ldcg(reinterpret_cast<const uint4*>(
                            reinterpret_cast<const uint8_t*>(g.out_bf16) +
                            y_block_offset(rr[j], n * 16 + (lane >> 1), g.n_tiles) + (lane & 1) * 16));
                float o[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) o[i] = 0.0f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (rr[j] < 0) continue;
                    const uint32_t uu[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        o[2 * i] = fmaf(ww[j], __uint_as_float(uu[i] << 16), o[2 * i]);
                        o[2 * i + 1] = fmaf(ww[j], __uint_as_float(uu[i] & 0xffff0000u), o[2 * i + 1]);
                    }
                }
                uint32_t p[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const __nv_bfloat162 pr = __floats2bfloat162_rn(o[2 * i], o[2 * i + 1]);
                    p[i] = *reinterpret_cast<const uint32_t*>(&pr);
                }
                *reinterpret_cast<uint4*>(f->out + static_cast<size_t>(t) * f->H + n * G_TILE_N + lane * 8) =
                    make_uint4(p[0], p[1], p[2], p[3]);
            }
        }
    }
    return true;
}

template <int MODE, bool FUSED, class GEO>
__device__ __forceinline__ void epilogue_tiles_wm(const Cta& c, const GemmArgs& g, const FusedArgs* f, TileRange tr,
                                                  uint32_t& it, uint32_t& tile_iter, uint32_t& sync_iter, bool& ok,
                                                  KSplit ks) {
    for (int item = tr.first; item < tr.count && ok; item += tr.stride) {
        const int tile = item / ks.parts, kb0 = (item - tile * ks.parts) * ks.len;
        const int m_tile = tile / g.n_tiles, n = tile - m_tile * g.n_tiles;
        // (two instantiations, so that the unsplit tile's loop carries nothing of the split)
        ok = (FUSED && MODE == 1 && ks.parts > 1)
                 ? epilogue_tile_wm<MODE, FUSED, GEO, false, FUSED && MODE == 1>(c, g, f, m_tile, n, it, tile_iter, sync_iter, kb0,
                                                                                min(g.num_kb, kb0 + ks.len), ks.parts)
                 : epilogue_tile_wm<MODE, FUSED, GEO, false, false>(c, g, f, m_tile, n, it, tile_iter, sync_iter);
    }
}

// One GEMM per launch.
template <int MODE>
__global__ void __launch_bounds__(G_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAs,
                    const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmOut, const GemmArgs g) {
    extern __shared__ uint8_t smem_raw[];
    using GEO = GeomFull;
    Cta c;
    gemm_cta_setup<GEO>(c, smem_raw, 1);
    if (c.warp == 0 && c.lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmAs);
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
    c.tmem_base = *reinterpret_cast<volatile uint32_t*>(&c.ctrl->tmem_slot);
    c.limit = g.wait_limit;
    // (the tables come from the kernels before this one, which may still be resident: coherent loads)
    const TileRange tr = {static_cast<int>(blockIdx.x), __ldcg(g.num_m_tiles) * g.n_tiles, static_cast<int>(gridDim.x)};
    uint32_t it = 0;
    bool ok = true;

    if (c.warp < 4) {
        reg_dealloc<40>();
        if (c.warp == 0 && c.lane == 0) {
            producer_tiles<MODE, false, GEO>(c, &tmA, &tmB, g, nullptr, 0, tr, it, ok, &tmAs);
            producer_drain<GEO>(c, g.status, it);
        } else if ((c.warp == 1 || c.warp == 2) && c.lane == 0) {
            issuer_tiles<GEO>(c, g, tr, c.warp - 1, it, ok);
            issuer_drain(c, c.warp - 1, ok);
        }
    } else {
        reg_alloc<232>();
        uint32_t tile_iter = 0;
        epilogue_tiles<MODE, GEO>(c, &tmOut, g, tr, it, tile_iter, ok);
        if (c.lane == 0) bulk_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    if (c.warp == 1) {
        __syncwarp();
        tmem_dealloc(c.tmem_base, G_TMEM_COLS);
    }
}

// Gather + GEMM1 + GEMM2 + combine in one launch for small batches, at most F_MAX_TOKENS tokens (see the head of
// this file).  tmA2 describes GEMM1's output buffer for loads (32-row boxes), tmB1 / tmB2 the two weight
// tensors.
__global__ void __launch_bounds__(G_THREADS, 1)
fused_small_kernel(const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB1,
                   const __grid_constant__ CUtensorMap tmB2, const GemmArgs g1, const GemmArgs g2, const FusedArgs f) {
    extern __shared__ uint8_t smem_raw[];
    using GEO = GeomSmall;
    Cta c;
    gemm_cta_setup<GEO>(c, smem_raw, 33);  // the producer's arrival plus the 32 lanes of the gather warp
    if (c.warp == 0 && c.lane == 0) {
        tma_prefetch_desc(&tmA2);
        tma_prefetch_desc(&tmB1);
        tma_prefetch_desc(&tmB2);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_launch_dependents();
    pdl_wait();
    c.tmem_base = *reinterpret_cast<volatile uint32_t*>(&c.ctrl->tmem_slot);
    c.limit = g1.wait_limit;

    // The previous fused call has ended (stream order), so the counters it used can be zeroed for the call
    // after this one.
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < f.num_counters; i += blockDim.x) f.counters_next[i] = 0;
    if (f.route) {
        // Stages 1 and 2, by every CTA for itself, in the not yet used pipeline stages.
        if (blockIdx.x == 0 && threadIdx.x == 0) *g1.status = DEV_OK;  // first kernel of a forward: clear the fault word
        int* scratch = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
        route_permute_in_cta(scratch, f.T, f.E_loc, f.expert_offset, f.row_cap, f.logits, f.bias, f.scaling, f.topk_idx,
                             f.topk_w_out, f.meta, g1.status);
    }

    // tokens without a local expert: their output rows are zeros, written here by the CTAs in turn
    for (int t = blockIdx.x; t < f.T; t += gridDim.x)
        if (__ldcg(f.tok_nlocal + t) == 0)
            for (int i = threadIdx.x; i < f.H / 8; i += blockDim.x)
                reinterpret_cast<uint4*>(f.out + static_cast<size_t>(t) * f.H)[i] = make_uint4(0u, 0u, 0u, 0u);

    // The CTA's work list: its GEMM1 tiles, then its GEMM2 tiles; the grid-strided numbering runs on from one
    // phase into the next, so the CTAs that had no GEMM1 tile take the first GEMM2 tiles.
    // Very small batches with few tiles: a tile's K range is cut into parts for different CTAs (KSplit).
    const int grid = static_cast<int>(gridDim.x), m_tiles = __ldcg(g1.num_m_tiles);
    const bool may_split = f.split && f.T <= SPLIT_MAX_TOKENS && g1.num_kb <= SPLIT_MAX_KB && g2.num_kb <= SPLIT_MAX_KB;
    const KSplit ks1 = ksplit_for(g1.num_kb, m_tiles * g1.n_tiles, grid, may_split && m_tiles * g1.n_tiles <= SPLIT_MAX_TILES);
    // (GEMM2's K range is too short for it: counting the parts and the finisher's pass over the stored partial sums
    // cost 5-6 us per tile, which 16 K-blocks do not win back; measured 1-2 us slower)
    const KSplit ks2 = ksplit_none(g2.num_kb);
    const int n1 = m_tiles * g1.n_tiles * ks1.parts, n2 = m_tiles * g2.n_tiles * ks2.parts;
    const TileRange tr1 = {static_cast<int>(blockIdx.x), n1, grid};
    const TileRange tr2 = {((static_cast<int>(blockIdx.x) - n1) % grid + grid) % grid, n2, grid};
    uint32_t it = 0;
    bool ok = true;

    if (c.warp < 4) {
        reg_dealloc<40>();
        if (c.warp == 0 && c.lane == 0) {
            producer_tiles<1, true, GEO>(c, &tmA2, &tmB1, g1, &f, 0, tr1, it, ok, nullptr, ks1);
            producer_tiles<2, true, GEO>(c, &tmA2, &tmB2, g2, &f, g1.n_tiles, tr2, it, ok, nullptr, ks2);
            producer_drain<GEO>(c, g1.status, it);
        } else if ((c.warp == 1 || c.warp == 2) && c.lane == 0) {
            issuer_tiles_wm<GEO>(c, g1, tr1, c.warp - 1, it, ok, ks1);
            issuer_tiles_wm<GEO>(c, g2, tr2, c.warp - 1, it, ok, ks2);
            issuer_drain(c, c.warp - 1, ok);
        } else if (c.warp == 3) {
            gather_tiles<GEO>(c, g1, f, tr1, it, ok, ks1);
            gather_idle_tiles<GEO>(c, g2, tr2, it, ok, ks2);
            cp_async_wait_all();  // nothing may still be landing in shared memory when the CTA exits
        }
    } else {
        reg_alloc<232>();
        uint32_t tile_iter = 0, sync_iter = 0;
        epilogue_tiles_wm<1, true, GEO>(c, g1, &f, tr1, it, tile_iter, sync_iter, ok, ks1);
        epilogue_tiles_wm<2, true, GEO>(c, g2, &f, tr2, it, tile_iter, sync_iter, ok, ks2);
    }

    tc_fence_before();
    __syncthreads();
    if (c.warp == 1) {
        __syncwarp();
        tmem_dealloc(c.tmem_base, G_TMEM_COLS);
    }
}

}  // namespace moe

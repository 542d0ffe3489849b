/*
 * moe_fp8.h -- C ABI of the B200 (sm_100a) fused block-scaled FP8 MoE forward.
 *
 * The operation is the "Fused MoE" workload of the paper (Section "Kernel
 * Design and Optimization", subsection "Fused MoE"): the DeepSeek-V3 MoE block
 * in four stages -- (1) routing: sigmoid scores, group-wise top-2 over 8
 * groups, final top-K = 8; (2) gathering the active rows of each expert into a
 * contiguous FP8 layout with 128-element fp32 block scales; (3) the gated MLP:
 * FP8 block-scaled GEMM1 [T,7168]->[T,4096], SwiGLU, re-quantisation, FP8
 * block-scaled GEMM2 [T,2048]->[T,7168]; (4) scattering the expert outputs
 * back to token positions weighted by the routing scores.  As in the paper's
 * final implementation, all metadata is built on the GPU and the hot path never
 * synchronises the stream.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".
 *   - The library never allocates, frees or retains caller tensors; scratch
 *     memory is one caller-owned workspace (moe_fp8_set_workspace).
 *   - Functions return 0 on success and a negative MOE_FP8_ERR_* otherwise; on
 *     error nothing has been enqueued.  There is no CPU fallback: without a
 *     compute-capability 10.x device moe_fp8_create fails.
 *   - moe_fp8_forward only enqueues work on `stream` and returns; faults found
 *     on the device (a bounded wait that gave up, an out-of-range row) are
 *     recorded in a status word readable through moe_fp8_debug_export.
 *   - One handle serves one stream at a time.  Weights are treated as
 *     immutable while the same weight pointers are passed (their TMA
 *     descriptors are cached per pointer pair); nothing is cached on
 *     activations, logits or outputs.
 *   - Inputs must be finite.  Base addresses must be 16-byte aligned.
 */
#ifndef MOE_FP8_H_
#define MOE_FP8_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOE_FP8_OK 0
#define MOE_FP8_ERR_BAD_ARG (-1)          /* null/misaligned pointer, T out of range, offset out of range */
#define MOE_FP8_ERR_UNSUPPORTED_DIMS (-2) /* layer shape outside what the kernels are built for */
#define MOE_FP8_ERR_NO_WORKSPACE (-3)     /* workspace missing or too small */
#define MOE_FP8_ERR_CUDA (-4)             /* a CUDA call failed; see moe_fp8_last_cuda_error */
#define MOE_FP8_ERR_ARCH (-5)             /* current device is not compute capability 10.x */
#define MOE_FP8_ERR_STATIC_LIMIT (-6)     /* size beyond the fixed capacity of a no-allocation entry point */

/* Layer shape, fixed at creation.  Supported: num_experts = 256, n_group = 8,
 * topk_group = 4, top_k = 8 (the DeepSeek-V3 routing of stage 1); hidden a
 * multiple of 256, intermediate a multiple of 128; 1 <= num_local_experts <= 256. */
typedef struct moe_fp8_config {
    int hidden;              /* H, 7168 */
    int intermediate;        /* I, 2048 */
    int num_experts;         /* E, 256 global experts */
    int num_local_experts;   /* E_loc, experts whose weights live on this GPU */
    int n_group;             /* 8 */
    int topk_group;          /* 4 */
    int top_k;               /* 8 */
    int max_tokens;          /* upper bound on T; sizes the workspace */
    int hidden_scale_layout; /* 0: hidden_scale is [T, H/128]; 1: [H/128, T] */
    int gate_first;          /* 1: w13 rows [0,I) are the gate (SiLU side), [I,2I) the up projection; 0: swapped */
} moe_fp8_config;

typedef struct moe_fp8_handle_s* moe_fp8_handle_t;

/* Host only.  Validates the shape, then requires a cc 10.x current device. */
int moe_fp8_create(const moe_fp8_config* cfg, moe_fp8_handle_t* out);
int moe_fp8_destroy(moe_fp8_handle_t h);

/* Bytes of device scratch needed for cfg.max_tokens tokens. */
size_t moe_fp8_workspace_bytes(moe_fp8_handle_t h);
/* Hands the library a caller-owned device buffer (1024-byte aligned) that must
 * stay valid until it is replaced or the handle destroyed.  The call zeroes the
 * control words and counters in it and waits for the device (cudaDeviceSynchronize);
 * after that the contents belong to the library: counters live there between
 * forwards, so the caller must not write into the buffer. */
int moe_fp8_set_workspace(moe_fp8_handle_t h, void* dev_workspace, size_t bytes);

/*
 * One forward pass of the layer for T tokens (stages 1-4 above), enqueued on
 * `stream` (a cudaStream_t).  T = 0 is valid and enqueues nothing.
 *
 *   hidden_fp8     e4m3 [T, H]            activations
 *   hidden_scale   fp32 [T, H/128]        one scale per token per 128 columns
 *   router_logits  fp32 [T, 256]
 *   routing_bias   bf16 [256]             added to the sigmoid score for selection only
 *   w13            e4m3 [E_loc, 2I, H]    gate and up projections, H contiguous
 *   w13_scale      fp32 [E_loc, 2I/128, H/128]
 *   w2             e4m3 [E_loc, H, I]     down projection, I contiguous
 *   w2_scale       fp32 [E_loc, H/128, I/128]
 *   local_expert_offset  first global expert id held locally; routes to experts
 *                        outside [offset, offset+E_loc) are dropped after the
 *                        weights were normalised over all 8 selected experts
 *   scaling_factor routed scaling factor (2.5)
 *   out            bf16 [T, H], fully overwritten (zeros for tokens without a local expert)
 *
 * All pointers are device pointers, 16-byte aligned; nothing is copied or kept beyond the call's kernels.
 * Forwards on one handle share its workspace: their kernels must not overlap on the GPU (one stream, or
 * streams ordered with events); use one handle per concurrent stream otherwise.
 */
int moe_fp8_forward(moe_fp8_handle_t h, int T, const void* hidden_fp8, const float* hidden_scale,
                    const float* router_logits, const void* routing_bias, const void* w13,
                    const float* w13_scale, const void* w2, const float* w2_scale, int local_expert_offset,
                    float scaling_factor, void* out, void* stream);

/*
 * The same pass for callers whose per-step tensors live in HOST memory
 * (preferably pinned): copies hidden_fp8, hidden_scale and router_logits to
 * staging areas inside the workspace, runs moe_fp8_forward, copies `out` back
 * and waits for the stream.  Weights, their scales and the bias stay device
 * pointers.  host_* arguments are host pointers with the layouts above.
 */
int moe_fp8_forward_host(moe_fp8_handle_t h, int T, const void* host_hidden_fp8, const float* host_hidden_scale,
                         const float* host_router_logits, const void* routing_bias, const void* w13,
                         const float* w13_scale, const void* w2, const float* w2_scale, int local_expert_offset,
                         float scaling_factor, void* host_out, void* stream);

/*
 * moe_fp8_forward_host for a sequence of steps: the call returns as soon as everything is enqueued.  The
 * host-to-device copies of the step run on a copy stream of the library, the forward on `stream`, the copy of
 * `out` back to host_out on a second copy stream, chained by events; two staging sets in the workspace
 * alternate, so the copies of one step overlap the forward of its neighbours.  host_* buffers must be pinned
 * (page-locked) for the copies to be asynchronous, must not be touched until moe_fp8_host_sync (or a later
 * cudaStreamSynchronize of `stream` followed by moe_fp8_host_sync) returns, and host_out of step i may be reused
 * from step i + 2 on only after such a wait.  The first call creates the two streams and six events (host
 * objects; no device memory is allocated).  Results are those of moe_fp8_forward_host, bit for bit.
 */
int moe_fp8_forward_host_async(moe_fp8_handle_t h, int T, const void* host_hidden_fp8, const float* host_hidden_scale,
                               const float* host_router_logits, const void* routing_bias, const void* w13,
                               const float* w13_scale, const void* w2, const float* w2_scale, int local_expert_offset,
                               float scaling_factor, void* host_out, void* stream);
/* Waits until every copy enqueued by moe_fp8_forward_host_async on this handle has finished. */
int moe_fp8_host_sync(moe_fp8_handle_t h);

/*
 * The same pass started from bf16 hidden states: stage 1 of the Fused MoE description begins with "routing
 * scores via a lightweight linear projection", and the FP8 activations with their 128-wide scales are the
 * quantisation of those hidden states.  This entry computes
 *   router_logits[t, e] = sum_h hidden[t, h] * router_weight[e, h]        (bf16 inputs, fp32 result)
 *   hidden_fp8, hidden_scale = per token per 128 columns: scale = amax / 448 (1 for an all-zero block),
 *                              code = e4m3(x / scale), round to nearest even, saturating
 * into staging areas of the workspace and then runs moe_fp8_forward on them (two more kernel launches).
 * Because the selected expert indices are reproducible bit for bit, the fp32 summation order of the
 * projection is fixed: 32 partial sums, partial l takes the l-th pair of every run of 64 elements in
 * increasing order with one fused multiply-add per element, then five pairwise rounds p[l] += p[l xor d],
 * d = 16, 8, 4, 2, 1.
 *
 *   hidden_bf16    bf16 [T, H]     device
 *   router_weight  bf16 [256, H]   device
 * All other arguments as moe_fp8_forward.  The staging areas are shared with moe_fp8_forward_host.
 */
int moe_fp8_forward_from_hidden(moe_fp8_handle_t h, int T, const void* hidden_bf16, const void* router_weight,
                                const void* routing_bias, const void* w13, const float* w13_scale, const void* w2,
                                const float* w2_scale, int local_expert_offset, float scaling_factor, void* out,
                                void* stream);
/* Test hook: copies what the last moe_fp8_forward_from_hidden (or moe_fp8_forward_host) on this handle fed
 * to the forward pass -- router_logits fp32 [T,256], hidden_fp8 e4m3 [T,H], hidden_scale fp32 in the
 * configured layout -- into caller buffers (device pointers, any may be NULL), enqueued on `stream`. */
int moe_fp8_debug_export_inputs(moe_fp8_handle_t h, int T, float* router_logits, void* hidden_fp8,
                                float* hidden_scale, void* stream);

/*
 * Test hook: copies internal results of the LAST forward on this handle into
 * caller buffers (device pointers, any may be NULL), enqueued on `stream`.
 *   topk_idx       int32 [T, 8]  selected experts, descending biased score
 *   topk_w         fp32  [T, 8]
 *   expert_count   int32 [E_loc]
 *   expert_offset  int32 [E_loc+1]   exclusive scan of the counts
 *   row_to_slot    int32 [T*8]       row -> slot id t*8+j (experts ascending,
 *                                    tokens ascending inside an expert); first S valid
 *   a2_fp8         e4m3  [T*8, I]    re-quantised SwiGLU output per row (first S rows)
 *   a2_scale       fp32  [T*8, I/128]
 *   y_rows         bf16  [T*8, H]    GEMM2 output per row before the combine
 *   status_word    int32 [1]         0, or the first device-side fault code
 */
int moe_fp8_debug_export(moe_fp8_handle_t h, int T, int* topk_idx, float* topk_w, int* expert_count,
                         int* expert_offset, int* row_to_slot, void* a2_fp8, float* a2_scale, void* y_rows,
                         int* status_word, void* stream);

/*
 * Small batches run the gather of stage 2, both GEMMs of stage 3 and the combine of stage 4 as ONE kernel (the
 * paper's short regime, T = 1-16, is bounded by routing and launch overhead, and it names fusing the scatter
 * into GEMM2's epilogue as the next step; in that kernel the CTA that stores the last local row of a token
 * sums the token's rows in routing order, so results stay bit-identical to the separate kernels).  Its MMAs
 * take the weights on the M side and a tile's at most 32 token rows on the N side; an expert with more rows is
 * worked on as several such tiles.  Up to 16 tokens that kernel also does stages 1 and 2 -- every CTA routes
 * and permutes the whole batch for itself and all write the same tables -- so a forward is a single launch;
 * above that a routing kernel runs in front of it.  The kernel's cross-CTA counters live in the workspace in two
 * sets: a call uses one and zeroes the other, so a call that gave up on a bounded wait does not disturb later
 * ones.
 * enable = 1 (the default): batches of at most 80 tokens take the fused kernel (measured faster up to there
 * for uniform and for skewed routing; with well balanced routing it stays faster up to about 200 tokens);
 * enable = 0: every batch takes the separate kernels; enable = 2..256: batches of at most that many tokens
 * take the fused kernel.  Other values: MOE_FP8_ERR_BAD_ARG.
 */
int moe_fp8_set_small_batch_fusion(moe_fp8_handle_t h, int enable);

/*
 * Batches of at most 4 tokens with so few tiles that most SMs would idle: the fused kernel cuts every tile's K
 * range into up to eight parts for different CTAs.  A part stores its per-K-block partial sums unscaled; the CTA
 * that stores a tile's last part (found with a counter, nobody waits) applies the scales K-block after K-block
 * in the order of the unsplit tile and finishes the tile, so results are bit-identical.  On by default; this
 * hook turns it off (enable = 0) for the test that compares the two.
 */
int moe_fp8_debug_set_k_split(moe_fp8_handle_t h, int enable);

/*
 * Inside the two large-tile GEMM kernels a row tile that holds at most 32 rows (an expert's short last tile) is
 * worked on with the operands swapped -- weights on the M side of the MMAs, the 32 token rows on N, a 64-column
 * accumulator -- instead of as a full 128-row tile: same arithmetic, bit-identical results, less tensor and
 * epilogue time.  This hook sets the batch size from which that applies (min_tokens = 0: never).
 */
int moe_fp8_debug_set_short_tiles(moe_fp8_handle_t h, int min_tokens);

/*
 * Test hook for the failure path of the bounded device waits (every wait on an mbarrier inside the GEMM
 * kernels gives up after a limit, records a fault code in the status word and lets the kernel return with
 * its tensor memory released).  skip_iteration >= 0: in the next forwards the copy producer of every CTA
 * of the GEMM1 kernel stops before its skip_iteration-th pipeline stage, so the consumers wait for a stage
 * that nothing fills; wait_clocks > 0 shortens the limit of every wait to that many SM clocks (0 restores
 * the default of about a second).  skip_iteration < 0 switches the hook off.  Nothing traps: the forward
 * returns normally, its output is garbage and the status word holds a time-out code (1..5, 8).
 */
int moe_fp8_debug_set_fault(moe_fp8_handle_t h, int skip_iteration, long long wait_clocks);

/* Test hook: y[i] = the routing stage's sigmoid of x[i] (stage 1 of the Fused MoE description; the indices
 * it selects are compared bit for bit, so its arithmetic is fixed operation by operation).  Device
 * pointers, fp32 [n]; enqueued on `stream`. */
int moe_fp8_debug_sigmoid(int n, const float* x, float* y, void* stream);

/*
 * Measurement hook (the paper profiles each kernel of one MoE iteration, Appendix
 * "NCU Profile of the Slowest FuseMoE Workload"): when enabled, moe_fp8_forward
 * records a CUDA event on `stream` before and after each of its kernel launches.
 * Enabling creates the events (not for use inside the hot path); disabling
 * destroys them.  Off by default.
 */
int moe_fp8_set_stage_timing(moe_fp8_handle_t h, int enable);
/* Number of stages and the name of stage i ("route_topk", ..., "combine"). */
int moe_fp8_num_stages(void);
const char* moe_fp8_stage_name(int i);
/* Waits for the events of the last forward and writes the device time of each
 * stage in milliseconds to host_ms[0..n) (host pointer); returns the number of
 * stages written. */
int moe_fp8_get_stage_times(moe_fp8_handle_t h, float* host_ms, int n);

/*
 * Per-expert histogram and exclusive scan WITHOUT any caller-provided or allocated scratch (the paper has
 * no counterpart; it exists for callers that cannot allocate).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a CUDA-graph capture or a
 * latency-critical serving loop that must not take the allocator lock or trigger an implicit device
 * synchronisation, or a plug-in that is handed tensors and a stream by its host framework but owns no
 * memory pool.  Such a caller cannot size and hand over the workspace that moe_fp8_set_workspace wants, yet
 * may still need the expert load (for capacity planning, load-balance statistics or to size its own
 * buffers) from routing indices it already holds.
 *
 *   topk_idx       int32 [T, 8]  device, selected global expert ids per token (as moe_fp8_debug_export gives)
 *   expert_count   int32 [num_local_experts]    device, out
 *   expert_offset  int32 [num_local_experts+1]  device, out, exclusive scan of the counts
 *
 * The scratch (per-block partial counts) is a 64 KB array that lives in the library image on every GPU that
 * loads it, for as long as the process runs.  Capacity: T <= MOE_FP8_STATIC_HISTOGRAM_MAX_TOKENS and
 * num_local_experts <= 256; a larger T returns MOE_FP8_ERR_STATIC_LIMIT and nothing is enqueued.  The call
 * makes no cudaMalloc/cudaFree and calls no allocating library routine; it only enqueues two kernels on
 * `stream`.  The first call on each device looks up the device address of the array (a host-side query, no
 * allocation); make that first call outside of any stream capture.  All calls share the one array and it
 * keeps the previous call's contents: every entry a call reads is first written by that same call, so
 * stale contents are never seen, but two calls whose kernels overlap on the GPU (different streams, or
 * threads racing on one stream's order) would overwrite each other's partial counts -- serialise them.
 */
#define MOE_FP8_STATIC_HISTOGRAM_MAX_TOKENS 16384
int moe_fp8_expert_histogram_static(int T, const int* topk_idx, int local_expert_offset, int num_local_experts,
                                    int* expert_count, int* expert_offset, void* stream);

/* CUDA error code (cudaError_t as int) of the last MOE_FP8_ERR_CUDA on this handle. */
int moe_fp8_last_cuda_error(moe_fp8_handle_t h);
/* Kernel launches enqueued by the last moe_fp8_forward on this handle. */
int moe_fp8_last_launch_count(moe_fp8_handle_t h);
/* Static string for a return code. */
const char* moe_fp8_strerror(int rc);

#ifdef __cplusplus
}
#endif
#endif /* MOE_FP8_H_ */

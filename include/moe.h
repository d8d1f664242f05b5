/*
 * moe.h -- C ABI of the B200 (sm_100a) fused Mixture-of-Experts layer forward pass.
 *
 * The layer (K-Search paper, Sec. 4.5 "Kernel Analysis: FP8 MoE Kernel (Blackwell)"): for each
 * token the top-k experts are chosen out of E from the router scores; tokens are reordered so
 * that every expert's tokens are contiguous ("sort-scatter", Sec. 4.5 "Expert FFN computation");
 * each chosen expert applies a gate and an up projection combined through SiLU, then a down
 * projection; the k results of a token are summed with the routing weights.  This library
 * computes it in bf16 with fp32 accumulation:
 *
 *   router   p = softmax(router_logits[t,:]); topk_ids[t,0..k) = the k largest logits, ties to the
 *            lower expert index, listed from largest to smallest; topk_weights = p[ids] / sum p[ids]
 *   permute  stable counting sort of the A = T*k assignments (flat index a = t*k + j) by expert:
 *            expert_offsets[E+1] (exclusive prefix sum of per-expert counts),
 *            flat_to_sorted[a] = position of a in expert-contiguous order, sorted_to_flat = inverse
 *   gemm1    h[r,:] = SiLU(x[t(r),:] . w13[e, 0:I, :]^T) * (x[t(r),:] . w13[e, I:2I, :]^T)   (bf16)
 *   gemm2    y[r,:] = h[r,:] . w2[e,:,:]^T                                                    (bf16)
 *   combine  out[t,:] = sum_{j ascending} topk_weights[t,j] * y[flat_to_sorted[t*k+j],:]      (bf16)
 *
 * Conventions for every entry point
 *   - All tensors are row-major with the last index contiguous.  bf16 data is passed as void*.
 *   - Unless a parameter says HOST, every pointer is a DEVICE pointer owned by the caller and
 *     valid on the current device.  The library allocates and frees no device memory, launches
 *     only on the given stream (a cudaStream_t passed as void*, NULL = default stream) and does
 *     not synchronise it, except where stated.
 *   - Inputs are read-only and must not alias outputs or the workspace.
 *   - The return value is a moe_status_t: 0 on success, negative on error.  Arguments are
 *     checked on the host before anything is launched; on an error nothing has been launched.
 *   - Supported envelope: 1 <= E <= 256, 1 <= top_k <= min(E, 32), H % 128 == 0, I % 64 == 0,
 *     T >= 0, T*top_k < 2^27.  T == 0 succeeds without a launch.
 *     Pointers of the layer's tensors must be 16-byte aligned (the router-only entry points need
 *     4 bytes for their arrays), the workspace 256-byte aligned.
 *   - The current device must be compute capability 10.x (MOE_ERR_ARCH otherwise; checked after the
 *     arguments, before the first launch).
 *   - Device-side waits are bounded.  If one expires (which indicates a bug, not bad input) the
 *     kernel records MOE_ERR_DEVICE_TIMEOUT in the workspace's status word and returns; read it
 *     with moe_last_status().
 *   - Results are deterministic: no floating-point atomics, no split accumulation; two calls on
 *     the same inputs give bit-identical outputs.
 *   - The kernels of one call are launched with programmatic stream serialisation (each waits for its
 *     predecessor before reading its results), so a call can be captured into a CUDA graph and replayed.
 *
 * Variants of the layer, each with the same conventions: moe_forward_local (only the experts resident on
 * this device), moe_route_grouped / moe_forward_grouped (sigmoid scores, selection bias, group-limited
 * top-k, scaled weights), moe_forward_fp8w (FP8 weights with a scale per 128 x 128 block, dequantised on the
 * way to 16-bit MMAs), moe_forward_mxfp8 (weights and activations in MX FP8, multiplied by the block-scaled
 * MMA), the *_host forms for activations in host memory, moe_forward_staged for per-stage timing.
 */
#ifndef MOE_B200_H_
#define MOE_B200_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MOE_API __attribute__((visibility("default")))
#else
#define MOE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOE_OK = 0,
    MOE_ERR_NULL = -1,           /* a required pointer is NULL */
    MOE_ERR_SHAPE = -2,          /* a size is negative, zero where it must not be, or top_k > E */
    MOE_ERR_UNSUPPORTED = -3,    /* outside the supported envelope (see above) */
    MOE_ERR_ALIGN = -4,          /* a pointer is not aligned as required */
    MOE_ERR_WORKSPACE = -5,      /* workspace_bytes is smaller than moe_*_workspace_bytes() */
    MOE_ERR_CUDA = -6,           /* a CUDA runtime/driver call failed (launch, descriptor encoding) */
    MOE_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait expired (reported by moe_last_status) */
    MOE_ERR_ARCH = -8,           /* the current device is not compute capability 10.x */
    MOE_ERR_STATIC_LIMIT = -9    /* moe_route_static: the problem needs more than its built-in scratch */
} moe_status_t;

/* Flags for moe_forward_ex. */
#define MOE_FLAG_NONE 0u
/* Run the two grouped GEMMs on plain CUDA-core kernels instead of the tcgen05 kernels.  Meant
 * for validating the tensor-core path at sizes the CPU cannot check in full; about 100x slower. */
#define MOE_FLAG_VALIDATION_GEMM 1u
/* Keep the tcgen05 GEMMs on the one-CTA-per-tile kernel even where the CTA-pair kernel would be
 * chosen (token tiles of up to 128 / 256 rows).  For tests and A/B timing. */
#define MOE_FLAG_SINGLE_CTA_GEMM 2u
/* Let the CTA-pair kernel of the gate/up GEMM use two weight slabs per CTA (512 x N pair tiles) where
 * the shape allows it.  Off by default (slower on the measured workloads); for tests and A/B timing. */
#define MOE_FLAG_TWO_SLAB_GEMM 4u
/* Keep token tiles at 256 rows or fewer even where the wide-tile kernel (one pass over a weight slab for an
 * expert of up to 320 / 384 rows) would be chosen.  For tests and A/B timing. */
#define MOE_FLAG_NARROW_TILES 8u
/* Where the wide-tile kernel runs the gate/up GEMM, let it fetch token rows straight from x by row index (TMA
 * four-row gather) instead of reading the expert-contiguous copy; x_perm is then not written.  Opt-in: for A/B timing. */
#define MOE_FLAG_GATHER_IN_LOAD 16u

/* Byte offsets of the intermediates inside the workspace of moe_forward (so tests and tools can
 * read them after the stream has been synchronised).  Filled by moe_workspace_layout(). */
typedef struct {
    size_t total_bytes;
    size_t status;          /* int32[4]: status, site, aux0, aux1 */
    size_t topk_ids;        /* int32 [T,k] */
    size_t topk_weights;    /* f32   [T,k] */
    size_t expert_offsets;  /* int32 [E+1] */
    size_t sorted_to_flat;  /* int32 [A] */
    size_t flat_to_sorted;  /* int32 [A] */
    size_t route_scratch;   /* router/permute scratch (per-chunk histograms, tile schedule) */
    size_t x_perm;          /* bf16 [A,H]: rows of x in expert-contiguous order */
    size_t h;               /* bf16 [A,I] */
    size_t y;               /* bf16 [A,H] */
    size_t staging;         /* used only by moe_forward_host: device copies of x, logits, out */
} moe_workspace_layout_t;

/* Host-only, pure.  Size in bytes of the workspace moe_forward / moe_forward_host need for this
 * problem; 0 if the problem is outside the supported envelope.  (Sec. 4.5: the intermediates are
 * the sort-scatter's reordered tokens and the two projections' results.) */
MOE_API size_t moe_workspace_bytes(int T, int H, int I, int E, int top_k);

/* Host-only, pure.  Fills *layout for the same problem; MOE_ERR_UNSUPPORTED outside the envelope. */
MOE_API int moe_workspace_layout(int T, int H, int I, int E, int top_k, moe_workspace_layout_t *layout);

/* Host-only, pure.  Workspace bytes needed by moe_route alone; 0 if unsupported. */
MOE_API size_t moe_route_workspace_bytes(int T, int E, int top_k);

/* Router + sort-scatter (Sec. 4.5 "Routing" and step (2) of "Expert FFN computation").
 *   router_logits  [T,E] f32, in
 *   topk_ids       [T,k] int32, out: chosen experts in rank order
 *   topk_weights   [T,k] f32,   out: renormalised softmax probabilities (sum to 1 per token)
 *   expert_offsets [E+1] int32, out
 *   sorted_to_flat [T*k] int32, out
 *   flat_to_sorted [T*k] int32, out
 *   workspace      scratch of at least moe_route_workspace_bytes(T,E,top_k) bytes; contents
 *                  undefined afterwards.  Concurrent calls need distinct workspaces.
 * Non-finite logits are outside the contract but the kernels still terminate and stay in bounds. */
MOE_API int moe_route(const float *router_logits, int T, int E, int top_k, int32_t *topk_ids, float *topk_weights,
              int32_t *expert_offsets, int32_t *sorted_to_flat, int32_t *flat_to_sorted, void *workspace,
              size_t workspace_bytes, void *stream);

/* moe_route for callers that can neither allocate device memory nor hand the library a workspace.
 * (The paper has no counterpart: this is a packaging variant of moe_route, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region where the framework
 * forbids allocation (a real-time serving loop with a frozen memory plan, a plugin that is given
 * tensors but no allocator handle), or where an allocation could synchronise the device or fragment a
 * pool at a bad moment.  Such a caller passes only the inputs and outputs below; the scratch that
 * moe_route takes as `workspace` lives instead in a 512 KiB array compiled into the library's device
 * image.  Every GPU that loads the library holds those 512 KiB until the process exits.
 *
 * Same arguments and results as moe_route, without workspace / workspace_bytes.  Differences:
 *   - Limit: 256 + 4 * (ceil(T/32) * E + 3 * E + 1) bytes (rounded up to 256) must fit in 512 KiB,
 *     e.g. T <= 16256 tokens at E = 256, T <= 32640 at E = 128.  Larger problems return
 *     MOE_ERR_STATIC_LIMIT and launch nothing; use moe_route with a workspace for those.
 *   - The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - The first call on each device looks up the array's device address (a host-side query); make that
 *     first call before starting any stream capture on that device.  The address is cached per device
 *     for the life of the process: after cudaDeviceReset() the cached address is stale and this entry
 *     point must not be called again in that process.
 *   - Arguments are checked as for moe_route (NULL, 4-byte alignment of every array, architecture).
 *   - All calls on a device share the one array, and it keeps the previous call's contents: the call
 *     clears or overwrites everything it later reads, so calls that run one after another (same
 *     stream, or ordered by events) are independent, but two calls whose kernels may overlap on the
 *     GPU (different streams without ordering) race on the array and give undefined results.
 *   - moe_last_status() cannot be used (there is no workspace); these kernels contain no waits. */
MOE_API int moe_route_static(const float *router_logits, int T, int E, int top_k, int32_t *topk_ids,
                             float *topk_weights, int32_t *expert_offsets, int32_t *sorted_to_flat,
                             int32_t *flat_to_sorted, void *stream);

/* The whole layer (Sec. 4.5: routing, sort-scatter, gate+up with SiLU, down projection; then the
 * weighted combine).
 *   x              [T,H]    bf16, in
 *   router_logits  [T,E]    f32,  in
 *   w13            [E,2I,H] bf16, in: rows [0,I) of an expert are the gate projection, [I,2I) the up projection
 *   w2             [E,H,I]  bf16, in
 *   out            [T,H]    bf16, out
 *   workspace      at least moe_workspace_bytes(T,H,I,E,top_k) bytes, 256-byte aligned.  Holds the
 *                  routing arrays and intermediates at the offsets moe_workspace_layout() reports;
 *                  they stay valid until the next call that uses this workspace.
 * Launches five kernels (seven above 1024 tokens, where the router and sort-scatter take three) on
 * `stream` and returns without waiting for them. */
MOE_API int moe_forward(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I,
                int E, int top_k, void *out, void *workspace, size_t workspace_bytes, void *stream);

/* moe_forward with option flags (MOE_FLAG_*). */
MOE_API int moe_forward_ex(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I,
                   int E, int top_k, void *out, void *workspace, size_t workspace_bytes, void *stream,
                   unsigned flags);

/* The layer restricted to the experts resident on this device (the paper's kernel computes "32 local
 * experts" out of 256, Sec. 4.5): the router still chooses among all E experts from router_logits
 * [T,E], but only assignments to experts [local_expert_offset, local_expert_offset + num_local_experts)
 * are computed; the others contribute nothing to `out`, and the routing weights are NOT renormalised
 * over the local experts, so the outputs of devices that partition the experts add up to the full layer.
 *   w13_local [num_local_experts, 2I, H] bf16, w2_local [num_local_experts, H, I] bf16: the resident experts,
 *   local expert l being global expert local_expert_offset + l.
 * Workspace as for moe_forward (same size); afterwards topk_ids / topk_weights hold the full routing,
 * expert_offsets has num_local_experts + 1 entries, flat_to_sorted is -1 for dropped assignments and
 * only the first expert_offsets[num_local_experts] entries of sorted_to_flat are defined.
 * MOE_ERR_SHAPE if the local range is empty or not inside [0, E). */
MOE_API int moe_forward_local(const void *x, const float *router_logits, const void *w13_local, const void *w2_local,
                              int T, int H, int I, int E, int top_k, int local_expert_offset, int num_local_experts,
                              void *out, void *workspace, size_t workspace_bytes, void *stream, unsigned flags);

/* The layer with FP8 block-scaled expert weights (the paper's workload is an "FP8 MoE", Table 2 and
 * Sec. 4.5; its kernel converts the stored FP8 operands and multiplies 16-bit tensor-core tiles, which is
 * what this entry point does on tcgen05): weights are OCP E4M3 codes, one byte each, with one fp32 scale
 * per 128 x 128 block of every expert's matrix; a weight is decode(code) * scale[row/128][col/128].
 * Activations, routing, intermediates and the result are as in moe_forward.
 *   w13_q      [E,2I,H] uint8 E4M3 codes (rows [0,I) gate, [I,2I) up)   w13_scale [E, 2I/128, H/128] f32
 *   w2_q       [E,H,I]  uint8 E4M3 codes                                w2_scale  [E, H/128,  I/128] f32
 *   stage_events  NULL, or MOE_NUM_STAGE_EVENTS cudaEvent_t handles recorded as by moe_forward_staged.
 * Needs I % 128 == 0 in addition to the usual envelope (MOE_ERR_UNSUPPORTED otherwise).  Codes are
 * converted to bf16 and multiplied by the block scale rounded to bf16 (at most 2^-8 relative per weight);
 * scales must be below 2^7 in magnitude; NaN codes are outside the contract. */
MOE_API int moe_forward_fp8w(const void *x, const float *router_logits, const void *w13_q, const float *w13_scale,
                             const void *w2_q, const float *w2_scale, int T, int H, int I, int E, int top_k, void *out,
                             void *workspace, size_t workspace_bytes, void *stream, void *const *stage_events);

/* moe_forward_local (pass local_expert_offset = 0, num_local_experts = E for the whole layer) that also
 * records CUDA events between the stages, for per-kernel timing inside a whole step.  stage_events is a
 * HOST array of MOE_NUM_STAGE_EVENTS cudaEvent_t handles (passed as void*, created by the caller with
 * timing enabled).  Event 0 is recorded on `stream` before the first kernel, and event i+1 after
 * stage i, where the stages are
 *   0 router + sort-scatter (1 or 3 kernels), 1 token rows into expert-contiguous order, 2 gate/up GEMM + SwiGLU,
 *   3 down GEMM, 4 combine.
 * With T == 0 nothing is launched and no event is recorded. */
#define MOE_NUM_STAGE_EVENTS 6
MOE_API int moe_forward_staged(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H,
                               int I, int E, int top_k, int local_expert_offset, int num_local_experts, void *out,
                               void *workspace, size_t workspace_bytes, void *stream, unsigned flags,
                               void *const *stage_events);

/* ---- Grouped sigmoid router ("DeepSeek-V3 style, top-8 routing", paper Sec. 4.5) -------------------------
 * The paper names the style without its formula; this is the routing published with DeepSeek-V3, with every
 * constant a parameter:
 *   score_e  = sigmoid(logit_e)                          the weight an expert gets if chosen
 *   choice_e = score_e + selection_bias[e]               used for selection only
 *   the E experts form n_group contiguous groups of E / n_group; a group's score is the sum of its two largest
 *   choice values (the single value for groups of one); the topk_group best groups stay eligible; the top_k
 *   eligible experts with the largest choice values are selected, in rank order; ties go to the lower index;
 *   weight_j = score_{id_j} / (sum of the selected scores, in rank order) * route_scale.
 * All of it is evaluated in binary32 with one correctly rounded operation per step, e^x by a fixed recipe
 * (clamp to [-87, 88]; n = nearest integer of x * log2 e; r = x - n * ln 2 in two fused steps; degree-7 Taylor
 * polynomial in Horner form; times 2^n), so the selected ids are reproducible bit for bit.
 * Requirements: n_group >= 1 divides E, E / n_group is a power of two, 1 <= topk_group <= n_group,
 * topk_group * (E / n_group) >= top_k (MOE_ERR_UNSUPPORTED otherwise). */
typedef struct {
    int n_group;
    int topk_group;
    const float *selection_bias; /* DEVICE, [E] f32, or NULL for no bias */
    float route_scale;
} moe_grouped_router_t;

/* moe_route with the grouped router (same outputs, workspace and errors). */
MOE_API int moe_route_grouped(const float *router_logits, int T, int E, int top_k, const moe_grouped_router_t *router,
                              int32_t *topk_ids, float *topk_weights, int32_t *expert_offsets, int32_t *sorted_to_flat,
                              int32_t *flat_to_sorted, void *workspace, size_t workspace_bytes, void *stream);

/* moe_forward_local with the grouped router (pass local_expert_offset = 0, num_local_experts = E for all). */
MOE_API int moe_forward_grouped(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H,
                                int I, int E, int top_k, const moe_grouped_router_t *router, int local_expert_offset,
                                int num_local_experts, void *out, void *workspace, size_t workspace_bytes, void *stream,
                                unsigned flags);

/* ---- MX FP8: 8-bit weights AND activations, multiplied by the block-scaled tensor-core instruction --------
 *
 * The paper's MoE workload is an FP8 one (Table 2, "FP8 MoE"; Sec. 4.5 names FP8 packing and scaling as a
 * cost of the kernel) without fixing the scaling granularity.  This path uses the OCP Microscaling format
 * MXFP8, the one sm_100a multiplies natively: E4M3 codes, and for every 32 consecutive elements along the
 * contraction dimension one E8M0 scale byte b standing for 2^(b-127) (255 = NaN); a stored value is
 * decode(code) * 2^(b-127).  Quantising 32 values: b = clamp(floor(log2(max|v|)) - 8 + 127, 0, 254) (0 for an
 * all-zero block; 255 and NaN codes if the block holds an infinity or NaN), codes = E4M3(v / 2^(b-127)),
 * round to nearest even, saturating at +-448.  The layer quantises each token row of x along H before the
 * gate/up projections and h = SiLU(gate)*up along I (from its fp32 value) before the down projection;
 * accumulation is fp32; y and out are bf16 as in moe_forward.
 *
 * Scale bytes are consumed in 512-byte "atoms": the 4 scale bytes (128 K-elements) of 128 rows, row r's at
 * byte (r % 32) * 16 + (r / 32) * 4.  moe_mxfp8_pack_scales converts plain scale bytes to that form once. */

/* Offsets of the MX path's workspace regions; A = T*top_k. */
typedef struct {
    size_t total_bytes;
    size_t status, topk_ids, topk_weights, expert_offsets, sorted_to_flat, flat_to_sorted, route_scratch; /* as moe_workspace_layout_t */
    size_t x_q;   /* uint8 [A,H]  codes of the token rows in expert-contiguous order */
    size_t x_sf;  /* scale atoms of x_q: [H/128][sf_atoms][512].  An expert's rows are cut into token tiles of equal
                     size rows_e (the last may be partial): rows_e = tile_rows for tile_rows <= 256; for the wide
                     bounds (304, 384) an expert of count <= tile_rows rows is one tile, a larger one
                     ceil(count / 256) tiles of rows_e = ceil(count / that) rounded up to 16.  Row i of expert e
                     belongs to token tile n = expert_offsets[e] / min(tile_rows, 256) + e + i / rows_e, as its row
                     r = i % rows_e; a tile owns ceil(tile_rows / 128) atoms, and the row's scales are in atom
                     n * ceil(tile_rows / 128) + r / 128 at atom row r % 128 */
    size_t h_q;   /* uint8 [A,I]  codes of h */
    size_t h_sf;  /* scale atoms of h_q: [I/128][sf_atoms][512], same row-to-atom rule */
    size_t y;     /* bf16 [A,H] */
    size_t staging; /* used only by moe_forward_mxfp8_host: device copies of x, logits, out */
    size_t sf_atoms;  /* a count, not an offset: atoms per K-slot in x_sf / h_sf */
    size_t tile_rows; /* a count: the token-tile bound of this problem (32, 64, 128, 160, 240, 304 or 384) */
} moe_mxfp8_workspace_layout_t;

/* Host-only, pure.  Workspace bytes of moe_forward_mxfp8; 0 outside the envelope (moe_forward's, plus I % 128 == 0). */
MOE_API size_t moe_mxfp8_workspace_bytes(int T, int H, int I, int E, int top_k);
MOE_API int moe_mxfp8_workspace_layout(int T, int H, int I, int E, int top_k, moe_mxfp8_workspace_layout_t *layout);

/* Repack weight scale bytes for moe_forward_mxfp8 (done once per model; enqueues one kernel on `stream`).
 *   scales  [E, rows, K/32] uint8, DEVICE, in: plain row-major scale bytes of a weight tensor [E, rows, K]
 *   packed  E * rows * K/32 bytes, DEVICE, 16-byte aligned, out (must not alias `scales`)
 *   gate_up 1 for w13 (rows = 2I, [gate | up]): atoms follow the gate/up GEMM's tiles of 64 features, whose 128
 *           rows are, for each group of 16 features, the 16 gate rows then the 16 up rows;
 *           0 for w2 (rows = H): atoms of 128 consecutive rows.
 * Atom order: [E][rows/128 tiles][K/128][512].  Needs rows % 128 == 0 and K % 128 == 0. */
MOE_API int moe_mxfp8_pack_scales(const void *scales, int E, int rows, int K, int gate_up, void *packed, void *stream);

/* MX quantisation of bf16 rows by the rule above (the layer applies the same rule to x inside
 * moe_forward_mxfp8; this entry point exposes it).  x [R,K] bf16 DEVICE (16-byte aligned) ->
 * codes [R,K] uint8 (8-byte aligned), scales [R,K/32] uint8 plain row-major.  K % 128 == 0. */
MOE_API int moe_mxfp8_quantize_rows(const void *x, int R, int K, void *codes, void *scales, void *stream);

/* The layer in MX FP8, restricted to the resident experts as in moe_forward_local (pass 0 and E for all).
 * With the grouped router and 32 resident experts of 256 this is the configuration the paper's kernel serves
 * (Sec. 4.5: FP8, "DeepSeek-V3 style, top-8 routing", 32 local experts).
 *   x [T,H] bf16, router_logits [T,E] f32, out [T,H] bf16: as moe_forward; all DEVICE pointers
 *   router  NULL for softmax -> top-k -> renormalise, else the grouped sigmoid router (moe_grouped_router_t)
 *   w13_q [n_local,2I,H] uint8 codes, w13_sf_packed: its scale bytes packed with gate_up = 1
 *   w2_q  [n_local,H,I]  uint8 codes, w2_sf_packed : its scale bytes packed with gate_up = 0
 *   workspace  at least moe_mxfp8_workspace_bytes bytes, 256-byte aligned (layout: moe_mxfp8_workspace_layout)
 *   stage_events  NULL, or MOE_NUM_STAGE_EVENTS events recorded as by moe_forward_staged
 * Launches the same number of kernels as moe_forward (the scatter into expert-contiguous order also quantises:
 * each token row is read and quantised once and stored to its top_k destinations).  Token tiles are at most
 * 384 rows (128 when H is not a multiple of 256); moe_mxfp8_workspace_layout reports the size in use.  Errors as moe_forward; a block of x holding an infinity or NaN makes that token's output NaN. */
MOE_API int moe_forward_mxfp8(const void *x, const float *router_logits, const void *w13_q, const void *w13_sf_packed,
                              const void *w2_q, const void *w2_sf_packed, int T, int H, int I, int E, int top_k,
                              const moe_grouped_router_t *router, int local_expert_offset, int num_local_experts,
                              void *out, void *workspace, size_t workspace_bytes, void *stream,
                              void *const *stage_events);

/* moe_forward_mxfp8 for a caller whose activations live in HOST memory, as moe_forward_host: x_host [T,H] bf16,
 * router_logits_host [T,E] f32 and out_host [T,H] bf16 are HOST pointers (pinned memory makes the copies
 * asynchronous); the weight codes and packed scales stay DEVICE pointers.  Enqueues the two host-to-device
 * copies, the layer and the device-to-host copy on `stream` and returns without synchronising. */
MOE_API int moe_forward_mxfp8_host(const void *x_host, const float *router_logits_host, const void *w13_q,
                                   const void *w13_sf_packed, const void *w2_q, const void *w2_sf_packed, int T, int H,
                                   int I, int E, int top_k, const moe_grouped_router_t *router, int local_expert_offset,
                                   int num_local_experts, void *out_host, void *workspace, size_t workspace_bytes,
                                   void *stream);

/* moe_forward_local (local_expert_offset = 0, num_local_experts = E for the whole layer) for a caller
 * whose activations live in HOST memory: x_host [T,H] bf16 and router_logits_host [T,E] f32 are HOST
 * pointers (pinned memory makes the copies asynchronous), out_host [T,H] bf16 is a HOST pointer; the
 * expert weights w13 / w2 stay DEVICE pointers (they are model parameters, resident across calls).
 * The call enqueues, on `stream`, the host-to-device copies into the workspace's staging area, the
 * layer, and the device-to-host copy of the result, and returns without synchronising: out_host is
 * valid once the stream has been synchronised. */
MOE_API int moe_forward_host(const void *x_host, const float *router_logits_host, const void *w13, const void *w2, int T,
                             int H, int I, int E, int top_k, int local_expert_offset, int num_local_experts,
                             void *out_host, void *workspace, size_t workspace_bytes, void *stream);

/* Synchronises `stream`, then reads the status word the kernels of the last moe_forward /
 * moe_route call left in `workspace`.  MOE_OK, MOE_ERR_DEVICE_TIMEOUT, or MOE_ERR_CUDA if the
 * stream reports an error. */
MOE_API int moe_last_status(const void *workspace, void *stream);

/* Self-test of the device-side error path.  Every wait inside the kernels is bounded; when one expires the kernel
 * records MOE_ERR_DEVICE_TIMEOUT in the workspace's status word, stops and returns.  This call enqueues one small
 * kernel that waits, with a bound of about 0.1 s, for a flag that nothing raises; afterwards moe_last_status() on
 * the same workspace must report MOE_ERR_DEVICE_TIMEOUT and the device must be usable as before.  workspace: at
 * least 2048 bytes, 256-byte aligned (its first 2048 bytes are overwritten). */
MOE_API int moe_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream);

/* Host-only, pure.  The largest number of token rows one GEMM tile of moe_forward_ex covers for this problem and
 * these flags (32, 64, 128, 256, 320 or 384; 0 outside the envelope): experts with more rows are cut into evenly
 * sized tiles.  Reporting only: results never depend on it beyond the fp32 summation order inside a tile. */
MOE_API int moe_token_tile_rows(int T, int H, int I, int E, int top_k, unsigned flags);

/* Number of kernels moe_forward_ex launches for this problem with these flags (0 when T == 0). */
MOE_API int moe_forward_launch_count(int T, unsigned flags);

/* Static, NUL-terminated description of a status code. */
MOE_API const char *moe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MOE_B200_H_ */

// Internal declarations shared by the CUDA translation units of the MoE library.
// Nothing here is part of the public ABI (see include/moe.h).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "moe.h"

namespace moe {

constexpr int kMaxExperts = 256;        // router keeps ceil(E/32) <= 8 logits per lane
constexpr int kMaxTopK = 32;            // lane j of the token's warp owns rank j
constexpr int kRouteTokensPerBlock = 32;  // tokens per router block = one histogram chunk
constexpr int kStatusInts = 4;          // status word: {status, site, aux0, aux1}
constexpr int kDoneCounterInt = 4;      // int index, in the status word's zeroed padding, of the fused router's block counter
// A forward call's status region is larger and also holds the hand-over between its two GEMMs (all zeroed by the
// memset that opens the call): a flag the gate/up GEMM raises once it has waited for its predecessors (the tile
// schedule is then complete), and per expert a count of finished gate/up epilogue passes.  With them the down GEMM
// starts on the SMs the gate/up GEMM has already left, expert by expert, instead of waiting for its whole grid.
constexpr int kStatusBytesRoute = 256;
constexpr int kStatusBytesForward = 2048;
constexpr int kHandoverFlagInt = 8;
constexpr int kReadyTotalInt = 9;       // all experts' counts together
constexpr int kClockProbeInt = 32;      // 2 x 4 int64 (bytes 128..191): the GEMMs' clock probes (moe_tc_common.cuh)
constexpr int kReadyCounterInt = 64;    // [kMaxExperts] ints from here
// What one gate/up tile adds to its expert's counter: each of the 4 epilogue warps of each CTA counts once, and a
// token tile is covered by I / 64 CTA-tiles of 64 features whichever kernel runs it.
static inline int handover_counts_per_token_tile(int I) { return (I / 64) * 4; }

// Site ids recorded next to MOE_ERR_DEVICE_TIMEOUT (gate/up GEMM; the down GEMM adds 4).
enum : int { kSiteProducerEmpty = 1, kSiteMmaFull = 2, kSiteMmaTmemEmpty = 3, kSiteEpilogueTmemFull = 4,
              kSiteHandoverFlag = 9, kSiteHandoverCount = 10, kSiteSelfTest = 11 };

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Host-side checks shared by the entry points (defined in moe_api.cu).
//   check_device    : MOE_OK when the current device is compute capability 10.x, MOE_ERR_ARCH when it is not,
//                     MOE_ERR_CUDA when it cannot be queried.
//   check_route_args: what moe_route, moe_route_grouped and moe_route_static all require of their arguments, in the
//                     order shape, envelope, NULL, 4-byte alignment of every array.
int check_device();
int check_route_args(const float *logits, int T, int E, int k, const int32_t *ids, const float *w, const int32_t *offsets,
                     const int32_t *s2f, const int32_t *f2s);

// ---- chained launches (programmatic dependent launch) ----------------------------------------------------
// The kernels of one forward call form a chain in which each reads what its predecessors wrote.  Every kernel
// is launched with programmatic stream serialisation allowed, announces at its very start that its dependents
// may be scheduled (chain_release), and waits for the completion of everything before it in the stream
// (chain_wait) before it touches memory a predecessor writes.  A kernel's launch latency and prologue (barrier
// set-up, tensor-memory allocation) then overlap the tail of the kernel before it.  Because EVERY block of
// every kernel waits, completion is transitive: when a kernel's predecessor is complete, so is everything
// earlier in the chain.  (The down GEMM of a hand-over pair starts on flags instead of this wait, so its blocks
// make the wait at their end, before teardown: gemm_chain_finish.)
#ifdef __CUDACC__
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Scratch of the router / sort-scatter, all int32, carved out of the caller's workspace.
struct RouteScratch {
    int *chunk_counts;  // [n_chunks, E] per-chunk expert histogram, then rows of earlier chunks per expert
    int *tile_prefix;   // [E+1] exclusive prefix sum of token tiles over experts in schedule order
    int *tile_order;    // [E]   expert at each schedule position: most rows first, ties to the lower index
    int *tile_rows;     // [E]   rows per token tile of this expert (multiple of 16; 0 if empty)
    int n_chunks;
};

static inline int route_num_chunks(int T) { return (T + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock; }

static inline size_t route_scratch_bytes(int T, int E) {
    size_t ints = (size_t)route_num_chunks(T) * E + (size_t)(E + 1) + 2 * (size_t)E;
    return align_up(ints * sizeof(int), 256);
}

static inline RouteScratch carve_route_scratch(void *base, int T, int E) {
    RouteScratch s;
    s.n_chunks = route_num_chunks(T);
    s.chunk_counts = reinterpret_cast<int *>(base);
    s.tile_prefix = s.chunk_counts + (size_t)s.n_chunks * E;
    s.tile_order = s.tile_prefix + (E + 1);
    s.tile_rows = s.tile_order + E;
    return s;
}

// How a token's experts and weights are derived from its logits.
//   softmax : softmax -> top-k -> renormalise (the five workloads)
//   grouped : sigmoid scores, a per-expert bias added for selection only, experts in n_group contiguous
//             groups of which the topk_group best (by the sum of their two largest biased scores) stay
//             eligible, top-k among those, weights = unbiased scores normalised and multiplied by `scale`.
struct RouterParams {
    int grouped = 0;
    int n_group = 1, topk_group = 1;
    const float *bias = nullptr;  // [E] or nullptr
    float scale = 1.f;
};

// The experts resident on this device: ids [offset, offset + count) of the E the router chooses from.
// Assignments to other experts are dropped from the schedule (flat_to_sorted = -1).
struct LocalExperts {
    int offset, count;
};

// Router + histogram, exclusive scans + tile schedule, stable scatter.  `nt_max` is the largest
// number of rows a GEMM token tile may have (multiple of 16); tiles are sized in multiples of
// `row_quantum` rows.  Scratch and expert_offsets are sized by local.count.
cudaError_t launch_route(const float *logits, int T, int E, int k, LocalExperts local, int nt_max, int *topk_ids,
                         float *topk_w, int *expert_offsets, int *sorted_to_flat, int *flat_to_sorted,
                         RouteScratch scratch, int *status, cudaStream_t stream, int row_quantum = 16,
                         RouterParams router = RouterParams(), size_t status_bytes = kStatusBytesRoute);

// x_perm[flat_to_sorted[t*k+j], :] = x[t, :] for every assignment with flat_to_sorted >= 0
cudaError_t launch_scatter_rows(const __nv_bfloat16 *x, const int *flat_to_sorted, int T, int k, int H, __nv_bfloat16 *x_perm,
                                cudaStream_t stream);

// out[t,:] = sum_j topk_w[t,j] * y[flat_to_sorted[t*k+j],:] over the ranks with a row here (flat_to_sorted >= 0).
// resident_subset: the call serves a subset of the experts, most ranks have no row: a kernel that takes several
// tokens per block (same result).
cudaError_t launch_combine(const __nv_bfloat16 *y, const float *topk_w, const int *flat_to_sorted, int T, int k,
                           int H, __nv_bfloat16 *out, cudaStream_t stream, bool resident_subset = false);

// Grouped GEMM over expert-contiguous rows, tcgen05 / TMEM / TMA.
//   swiglu = true : act [A,K=H] x w [E,2I,H]  -> out [A,I]  = SiLU(gate) * up
//   swiglu = false: act [A,K=I] x w [E,H,I]   -> out [A,H]
// `n_out` is the number of output features per row (I resp. H).
struct GroupedGemmArgs {
    const __nv_bfloat16 *act;  // [A, K]
    const __nv_bfloat16 *w;    // [E, w_rows, K]
    __nv_bfloat16 *out;        // [A, n_out]
    int A, K, n_out, E;
    int w_rows;                // rows per expert in w (2I for gemm1, H for gemm2)
    int nt_max;                // token-tile bound the schedule was built with
    const int *expert_offsets; // [E+1]
    const int *tile_prefix;    // [E+1] in schedule order
    const int *tile_order;     // [E]
    const int *tile_rows;      // [E]
    int *status;               // status word
    bool swiglu;
    const float *w_scale = nullptr;  // FP8-weight GEMM: w points at E4M3 codes, this at [E, w_rows/128, K/128] scales
    // hand-over between the two GEMMs of a call: 0 none; 1 this GEMM raises the flag and counts finished tiles per
    // expert; 2 this GEMM waits for the flag instead of the previous grid, and per tile for its expert's count
    int handover_role = 0;
    int *handover = nullptr;            // the call's status region (flag and counters at the offsets above)
    int handover_per_token_tile = 0;    // role 2: counts that complete one token tile of an expert
    // gather-in-load (wide-tile gate/up GEMM): when gather_x is set, `act` is unused and row r of the expert-contiguous
    // order is row gather_sorted_to_flat[r] / gather_top_k of gather_x [gather_T, K]
    const __nv_bfloat16 *gather_x = nullptr;
    const int *gather_sorted_to_flat = nullptr;
    int gather_T = 0, gather_top_k = 1;
};
int launch_grouped_gemm_tc(const GroupedGemmArgs &args, cudaStream_t stream);  // returns a moe_status_t

// The same GEMM on CTA pairs (cta_group::2): 256 x N tiles (one weight slab per CTA) or 512 x N tiles
// (two slabs per CTA sharing one token tile).  grouped_gemm_tc_pair_slabs gives the largest slab count
// usable for this GEMM: 2, 1, or 0 when the pair kernel does not apply (token-tile bound below 128, or a
// feature count the pair tile does not divide).
int grouped_gemm_tc_pair_slabs(const GroupedGemmArgs &args);
int launch_grouped_gemm_tc_pair(const GroupedGemmArgs &args, int slabs, cudaStream_t stream);

// The same GEMM on CTA pairs with wide token tiles (bounds 320 and 384 rows): one pass over a weight slab per
// expert of up to that many rows, accumulators in a ring of tensor-memory columns (moe_gemm_tc_ring.cu).
bool grouped_gemm_tc_ring_applies(const GroupedGemmArgs &args);
int launch_grouped_gemm_tc_ring(const GroupedGemmArgs &args, cudaStream_t stream);

// The one-CTA kernel for FP8 (E4M3) block-scaled weights: args.w holds one code byte per weight and
// args.w_scale one fp32 scale per 128 x 128 block; converter warps rebuild bf16 operand tiles in shared
// memory and the bf16 tensor-core path does the rest.  Needs K % 128 == 0.
int launch_grouped_gemm_tc_fp8w(const GroupedGemmArgs &args, cudaStream_t stream);

// ---- MX FP8 (E4M3 codes, one E8M0 scale byte per 32 elements along K) ---------------------------------
// The block-scaled MMA reads the scale bytes of its operands from tensor memory, where they arrive from
// shared memory in 512-byte "atoms": the 4 scale bytes (4 x 32 = 128 K-elements, one ring slot) of 128
// consecutive rows, row r of the atom at byte (r % 32) * 16 + (r / 32) * 4.  Scale bytes therefore live
// in global memory in that form, one atom per (128-row group, ring slot), so a slot's scales are one
// bulk copy.
//   weights     : [E][feature tile][K/128][512]; a gate/up tile's rows are in the tile's interleaved order
//   activations : [K/128][n_atoms][512], whole atoms per token tile.  The MX schedule cuts an expert's rows into
//                 tiles of equal size (the last may be partial): exactly `tile` rows for a token-tile bound of up to
//                 256 (32, 64, 128, 160 or 240); for the wide bounds (304, 384) an expert of up to `tile` rows is one
//                 tile, and a larger one is cut into ceil(count / 256) tiles of round16(count / that) <= 256 rows,
//                 as in the bf16 schedule (two consecutive tiles of more than 248 rows would overlap in the
//                 accumulator ring).  With stride = min(tile, 256), token tile j of expert e is tile number
//                 offsets[e] / stride + e + j  (never below the number of tiles before it, so the numbers are
//                 distinct) and owns ceil(tile / 128) consecutive atoms; its row r sits in atom r / 128 of those,
//                 at atom row r % 128.  Every tile thus starts a fresh atom, and the MMA reads its token scales
//                 from the first column of the atom (an odd column offset is a misaligned address for the
//                 instruction).  n_atoms = (A / stride + E + 1) * ceil(tile / 128) bounds the atom index.
constexpr int kMxSfAtomBytes = 512;
static inline int mx_sf_stride(int tile) { return tile > 256 ? 256 : tile; }
static inline int mx_act_sf_atoms(int A, int E, int tile) { return (A / mx_sf_stride(tile) + E + 1) * ((tile + 127) / 128); }
static inline size_t mx_act_sf_bytes(int A, int E, int K, int tile) {
    return (size_t)(K / 128) * mx_act_sf_atoms(A, E, tile) * kMxSfAtomBytes;
}
__host__ __device__ inline int mx_atom_byte(int row_in_atom, int sf) {
    return (row_in_atom & 31) * 16 + (row_in_atom >> 5) * 4 + sf;
}

struct MxGemmArgs {
    const uint8_t *act_q;   // [A, K] codes, rows in expert-contiguous order
    const uint8_t *act_sf;  // activation scale atoms (layout above)
    const uint8_t *w_q;     // [E, w_rows, K] codes
    const uint8_t *w_sf;    // weight scale atoms (layout above)
    void *out;              // swiglu: [A, n_out] codes of h; else [A, n_out] bf16
    uint8_t *out_sf;        // swiglu: scale atoms of h as the next GEMM's activation (K = n_out); else unused
    int A, K, n_out, E, w_rows, nt_max, n_atoms;
    const int *expert_offsets, *tile_prefix, *tile_order, *tile_rows;
    int *status;
    bool swiglu;
    int handover_role = 0;  // as in GroupedGemmArgs
    int *handover = nullptr;
    int handover_per_token_tile = 0;
};
// One-CTA tcgen05 kernel with kind::mxf8f6f4.block_scale.  The schedule must have been built with the row
// quantum equal to nt_max (every tile nt_max rows, the last partial) and nt_max <= 128.  Needs K % 128 == 0.
int launch_grouped_gemm_tc_mx(const MxGemmArgs &args, cudaStream_t stream);
// The same GEMM on CTA pairs (cta_group::2, 256 x N tiles): nt_max 128, 160 or 240, and n_out a multiple of the
// pair tile (128 features of h, 256 output rows of the down projection).
bool grouped_gemm_tc_mx_pair_applies(const MxGemmArgs &args);
int launch_grouped_gemm_tc_mx_pair(const MxGemmArgs &args, cudaStream_t stream);
// The same on CTA pairs with wide token tiles (nt_max 304 or 384: one pass over a weight slab per expert of up to that
// many rows), accumulators handed out in 16-column chunks of tensor memory as in the bf16 wide-tile kernel.
bool grouped_gemm_tc_mx_ring_applies(const MxGemmArgs &args);
int launch_grouped_gemm_tc_mx_ring(const MxGemmArgs &args, cudaStream_t stream);

// xq[flat_to_sorted[t*k+j], :] and that row's scale atoms <- MX quantisation of x[t,:], for every assignment with
// flat_to_sorted >= 0 (token-major: each row is read and quantised once).
cudaError_t launch_mx_scatter_quantize(const __nv_bfloat16 *x, const int *flat_to_sorted, const int *topk_ids,
                                       const int *expert_offsets, const int *tile_rows, LocalExperts local, int T, int k,
                                       int H, uint8_t *xq, uint8_t *x_sf, int n_atoms, int tile, cudaStream_t stream);
// codes[r,:], scales[r, K/32] (plain row-major) <- MX quantisation of x[r,:].
cudaError_t launch_mx_quantize_rows(const __nv_bfloat16 *x, int R, int K, uint8_t *codes, uint8_t *scales,
                                    cudaStream_t stream);
// plain [E, rows, K/32] scale bytes -> weight scale atoms; gate_up: rows = 2I in [gate | up] order, tiles of
// 64 features interleaved as the gate/up GEMM reads them; else tiles of 128 consecutive rows.
cudaError_t launch_mx_pack_scales(const uint8_t *plain, int E, int rows, int K, bool gate_up, uint8_t *packed,
                                  cudaStream_t stream);

// One block waits, with a short bound, for a hand-over flag that nothing raises, and must come back with
// MOE_ERR_DEVICE_TIMEOUT in the status word: the error path of the bounded waits, exercised without a hang.
cudaError_t launch_wait_timeout_selftest(int *status, cudaStream_t stream);

// Same contract on plain CUDA cores (validation only).
cudaError_t launch_grouped_gemm_validation(const GroupedGemmArgs &args, cudaStream_t stream);

// Token-tile bound chosen from the average rows per expert: 32, 64, 128 or 256, and 320 / 384 (the wide-tile
// kernel) when experts are expected to hold more than 256 rows.  `wide_ok` = false keeps the bound at 256.
int choose_nt_max(int T, int E, int k, bool wide_ok = false);

}  // namespace moe

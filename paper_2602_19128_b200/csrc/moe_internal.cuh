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

// Site ids recorded next to MOE_ERR_DEVICE_TIMEOUT (gate/up GEMM; the down GEMM adds 4).
enum : int { kSiteProducerEmpty = 1, kSiteMmaFull = 2, kSiteMmaTmemEmpty = 3, kSiteEpilogueTmemFull = 4 };

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

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

// The experts resident on this device: ids [offset, offset + count) of the E the router chooses from.
// Assignments to other experts are dropped from the schedule (flat_to_sorted = -1).
struct LocalExperts {
    int offset, count;
};

// Router + histogram, exclusive scans + tile schedule, stable scatter.  `nt_max` is the largest
// number of rows a GEMM token tile may have (multiple of 16).  Scratch and expert_offsets are sized
// by local.count.
cudaError_t launch_route(const float *logits, int T, int E, int k, LocalExperts local, int nt_max, int *topk_ids,
                         float *topk_w, int *expert_offsets, int *sorted_to_flat, int *flat_to_sorted,
                         RouteScratch scratch, int *status, cudaStream_t stream);

// x_perm[r,:] = x[sorted_to_flat[r] / k, :] for r < *n_rows (a device-side count, at most A)
cudaError_t launch_gather_rows(const __nv_bfloat16 *x, const int *sorted_to_flat, const int *n_rows, int A, int k,
                               int H, __nv_bfloat16 *x_perm, cudaStream_t stream);

// out[t,:] = sum_j topk_w[t,j] * y[flat_to_sorted[t*k+j],:]
cudaError_t launch_combine(const __nv_bfloat16 *y, const float *topk_w, const int *flat_to_sorted, int T, int k,
                           int H, __nv_bfloat16 *out, cudaStream_t stream);

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
};
int launch_grouped_gemm_tc(const GroupedGemmArgs &args, cudaStream_t stream);  // returns a moe_status_t

// The same GEMM on CTA pairs (cta_group::2): 256 x N tiles (one weight slab per CTA) or 512 x N tiles
// (two slabs per CTA sharing one token tile).  grouped_gemm_tc_pair_slabs gives the largest slab count
// usable for this GEMM: 2, 1, or 0 when the pair kernel does not apply (token-tile bound below 128, or a
// feature count the pair tile does not divide).
int grouped_gemm_tc_pair_slabs(const GroupedGemmArgs &args);
int launch_grouped_gemm_tc_pair(const GroupedGemmArgs &args, int slabs, cudaStream_t stream);

// The one-CTA kernel for FP8 (E4M3) block-scaled weights: args.w holds one code byte per weight and
// args.w_scale one fp32 scale per 128 x 128 block; converter warps rebuild bf16 operand tiles in shared
// memory and the bf16 tensor-core path does the rest.  Needs K % 128 == 0.
int launch_grouped_gemm_tc_fp8w(const GroupedGemmArgs &args, cudaStream_t stream);

// Same contract on plain CUDA cores (validation only).
cudaError_t launch_grouped_gemm_validation(const GroupedGemmArgs &args, cudaStream_t stream);

// Token-tile bound chosen from the average rows per expert.
int choose_nt_max(int T, int E, int k);

}  // namespace moe

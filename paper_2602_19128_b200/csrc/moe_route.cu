// Router (softmax -> top-k -> renormalise) and the stable sort-scatter by expert.
//
// Paper, Sec. 4.5 "Routing": each token gets scores for E experts and the top k are picked with
// warp-level cooperation; "Expert FFN computation", step (2): tokens are reordered by expert into
// contiguous memory.  Here one warp owns one token (E <= 256 logits fit in 8 registers per lane),
// selection is k rounds of a warp arg-max (two warp reductions per round: the largest order-preserving
// key, then the lowest index holding it) under the strict order
//     e before e'  <=>  logit[e] > logit[e']  or  (logit[e] == logit[e'] and e < e'),
// and the sort-scatter is a counting sort made stable without ordered atomics:
//   1. every router block histograms the assignments of its own 32 tokens (one "chunk");
//   2. one block turns the [chunk, expert] histogram into start positions (scan over chunks per
//      expert, scan over experts) and derives the GEMM token-tile schedule;
//   3. one warp per chunk walks its assignments in flat order, 32 at a time, ranking equal
//      experts inside a group with match_any and carrying per-expert counters between groups.
// Integer results are therefore unique and reproducible.
#include "moe_internal.cuh"

#include <limits.h>
#include <math.h>

#include <mutex>

namespace moe {
namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kRouteThreads = 1024;  // one warp per token of the block's 32-token chunk
constexpr int kLogitsPerLane = kMaxExperts / 32;

// Order-preserving map from float to unsigned: a > b  <=>  ordered_key(a) > ordered_key(b) (for non-NaN values;
// -0 is first folded into +0 so that the two compare equal, as the floats do).
__device__ __forceinline__ unsigned ordered_key(float f) {
    const unsigned u = __float_as_uint(f + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// k rounds of a warp arg-max under the strict order (larger key first, ties to the lower expert index).  Expert
// e = 32 i + lane has key[i] in its lane; entries with e >= E must hold key 0 and are never selected while a real
// candidate is left.  Each round: every lane finds its best remaining entry, one warp reduction gives the largest
// key, a second one the lowest expert index among the lanes that hold it.  Lane j < k returns rank j's expert.
__device__ __forceinline__ int select_top_k(const unsigned (&key)[kLogitsPerLane], int E, int k, int lane) {
    unsigned taken = 0;
    int my_id = 0;
    for (int j = 0; j < k; ++j) {
        unsigned best = 0;
        int best_e = INT_MAX;  // no candidate
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i) {
            const int e = i * 32 + lane;
            const bool free_slot = e < E && !((taken >> i) & 1u);
            if (free_slot && (best_e == INT_MAX || key[i] > best)) { best = key[i]; best_e = e; }
        }
        const unsigned top = __reduce_max_sync(kFullMask, best_e == INT_MAX ? 0u : best);
        int winner = (int)__reduce_min_sync(kFullMask, (best_e != INT_MAX && best == top) ? (unsigned)best_e : 0xffffffffu);
        if (winner < 0 || winner >= E) winner = 0;  // unreachable for k <= E; keeps the index in range regardless
        if ((winner & 31) == lane) taken |= 1u << (winner >> 5);
        if (lane == j) my_id = winner;
    }
    return my_id;
}

// Router for one token by one warp: top-k of the E logits (8 per lane) under the strict order, then the
// renormalised softmax weights.  Softmax's normaliser cancels in the renormalisation, so only the k selected
// logits are exponentiated: w_j = exp(l_j - l_0) / sum_j' exp(l_j' - l_0), the sum in rank order.
// Lane j < k returns rank j's expert and weight.
__device__ __forceinline__ void route_one_token(const float *__restrict__ row, int E, int k, int lane, int &my_id,
                                                float &my_w) {
    float v[kLogitsPerLane];
    unsigned key[kLogitsPerLane];
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) {
        const int e = i * 32 + lane;
        v[i] = e < E ? row[e] : 0.f;
        key[i] = e < E ? ordered_key(v[i]) : 0u;
    }
    my_id = select_top_k(key, E, k, lane);
    // the selected logit lives in lane my_id % 32, register my_id / 32
    float my_l = 0.f;
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) {
        const float got = __shfl_sync(kFullMask, v[i], my_id & 31);
        if ((my_id >> 5) == i) my_l = got;
    }
    const float top_l = __shfl_sync(kFullMask, my_l, 0);  // rank 0 holds the largest logit
    const float my_p = lane < k ? expf(my_l - top_l) : 0.f;
    float denom = 0.f;  // ascending rank, the order the definition states
    for (int j = 0; j < k; ++j) denom += __shfl_sync(kFullMask, my_p, j);
    my_w = my_p / denom;
}

// ---- grouped sigmoid router ("DeepSeek-V3 style" routing, Sec. 4.5) ---------------------------------------
// Selection is an integer decision taken from floating-point values, so every operation that feeds it is one
// correctly rounded binary32 operation in a fixed order (the _rn intrinsics keep the compiler from fusing or
// reassociating them); e^x follows a fixed recipe: clamp to [-87, 88], n = nearest integer of x * log2(e),
// r = x - n * ln 2 (ln 2 in two parts, fused multiply-adds), degree-7 Taylor polynomial in Horner form, times 2^n.
__device__ __forceinline__ float exp_fixed(float x) {
    x = fminf(fmaxf(x, -87.0f), 88.0f);
    const float n = rintf(__fmul_rn(x, 1.44269502f));
    float r = __fmaf_rn(n, -0.693145752f, x);
    r = __fmaf_rn(n, -1.42860677e-06f, r);
    float p = 1.98412701e-04f;
    p = __fmaf_rn(p, r, 1.38888892e-03f);
    p = __fmaf_rn(p, r, 8.33333377e-03f);
    p = __fmaf_rn(p, r, 4.16666679e-02f);
    p = __fmaf_rn(p, r, 1.66666672e-01f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    return __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
}
__device__ __forceinline__ float sigmoid_fixed(float l) { return __fdiv_rn(1.0f, __fadd_rn(1.0f, exp_fixed(-l))); }

// Merge two (largest, second largest) pairs.
__device__ __forceinline__ void top2_merge(float &t1, float &t2, float o1, float o2) {
    const float lo = fminf(t1, o1);
    t1 = fmaxf(t1, o1);
    t2 = fmaxf(lo, fmaxf(t2, o2));
}

// One token by one warp.  Expert e = 32 i + lane lives in register i of its lane; a group is G = E / n_group
// consecutive experts, G a power of two: either a segment of G lanes within one register index (G <= 32) or all
// lanes of G / 32 consecutive register indices.
__device__ __forceinline__ void route_one_token_grouped(const float *__restrict__ row, int E, int k, int lane,
                                                        const RouterParams &rp, int &my_id, float &my_w) {
    const int G = E / rp.n_group;
    float s[kLogitsPerLane], c[kLogitsPerLane], t1[kLogitsPerLane], t2[kLogitsPerLane];
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) {
        const int e = i * 32 + lane;
        s[i] = e < E ? sigmoid_fixed(row[e]) : 0.f;
        c[i] = e < E ? (rp.bias ? __fadd_rn(s[i], rp.bias[e]) : s[i]) : -INFINITY;
        t1[i] = c[i];
        t2[i] = -INFINITY;
    }
    // the two largest biased scores of every group
    if (G > 32) {  // registers of the same group first
        const int m = G >> 5;
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i) {
            const int first = i & ~(m - 1);
            float a1 = -INFINITY, a2 = -INFINITY;
#pragma unroll
            for (int j = 0; j < kLogitsPerLane; ++j)
                if (j >= first && j < first + m) top2_merge(a1, a2, c[j], -INFINITY);
            t1[i] = a1;
            t2[i] = a2;
        }
    }
    for (int off = (G < 32 ? G : 32) >> 1; off > 0; off >>= 1) {
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i) {
            const float o1 = __shfl_xor_sync(kFullMask, t1[i], off), o2 = __shfl_xor_sync(kFullMask, t2[i], off);
            top2_merge(t1[i], t2[i], o1, o2);
        }
    }
    float gs[kLogitsPerLane];  // score of the group that holds this register's expert
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) gs[i] = G >= 2 ? __fadd_rn(t1[i], t2[i]) : t1[i];
    // a group is eligible if fewer than topk_group groups rank before it (ties to the lower group index)
    if (rp.n_group <= 32) {
        // lane g fetches group g's score from the lane and register that hold the group's first expert ...
        const int first = lane < rp.n_group ? lane * G : 0;
        float mine = 0.f;
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i) {
            const float got = __shfl_sync(kFullMask, gs[i], first & 31);
            if ((first >> 5) == i) mine = got;
        }
        // ... ranks it against the others, and the eligible groups become a bit mask
        int rank = 0;
        for (int g = 0; g < rp.n_group; ++g) {
            const float val = __shfl_sync(kFullMask, mine, g);
            rank += (val > mine || (val == mine && g < lane)) ? 1 : 0;
        }
        const unsigned eligible = __ballot_sync(kFullMask, lane < rp.n_group && rank < rp.topk_group);
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i)
            if (!((eligible >> ((i * 32 + lane) / G)) & 1u)) c[i] = -INFINITY;
    } else {  // more groups than lanes (groups of at most 4 experts): every register ranks its own group
        int rank[kLogitsPerLane];
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i) rank[i] = 0;
        for (int g = 0; g < rp.n_group; ++g) {
            const int e0 = g * G, ip = e0 >> 5;
            float pick = gs[0];
#pragma unroll
            for (int i = 1; i < kLogitsPerLane; ++i) pick = ip == i ? gs[i] : pick;
            const float val = __shfl_sync(kFullMask, pick, e0 & 31);
#pragma unroll
            for (int i = 0; i < kLogitsPerLane; ++i) {
                const int gid = (i * 32 + lane) / G;
                rank[i] += (val > gs[i] || (val == gs[i] && g < gid)) ? 1 : 0;
            }
        }
#pragma unroll
        for (int i = 0; i < kLogitsPerLane; ++i)
            if (rank[i] >= rp.topk_group) c[i] = -INFINITY;
    }

    // top-k of the eligible biased scores; the weight uses the unbiased score of the selected expert
    unsigned key[kLogitsPerLane];
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) key[i] = i * 32 + lane < E ? ordered_key(c[i]) : 0u;
    my_id = select_top_k(key, E, k, lane);
    float my_s = 0.f;
#pragma unroll
    for (int i = 0; i < kLogitsPerLane; ++i) {
        const float got = __shfl_sync(kFullMask, s[i], my_id & 31);
        if ((my_id >> 5) == i) my_s = got;
    }
    if (lane >= k) my_s = 0.f;
    float denom = 0.f;  // ascending rank
    for (int j = 0; j < k; ++j) denom = __fadd_rn(denom, __shfl_sync(kFullMask, my_s, j));
    my_w = __fmul_rn(__fdiv_rn(my_s, denom), rp.scale);
}

// Routes the block's 32 tokens (warp w takes tokens w, w + n_warps, ...), writes ids and weights, and
// leaves the block's histogram over the resident experts in hist[].
__device__ __forceinline__ void route_block_tokens(const float *__restrict__ logits, int T, int E, int k, int local_offset,
                                                   int n_local, const RouterParams &rp, int *topk_ids, float *topk_w,
                                                   int *hist) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = blockDim.x >> 5;
    for (int e = tid; e < n_local; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    const int t_base = blockIdx.x * kRouteTokensPerBlock;
    for (int tt = warp; tt < kRouteTokensPerBlock; tt += n_warps) {
        const int t = t_base + tt;
        if (t >= T) break;  // uniform over the warp
        int my_id;
        float my_w;
        if (rp.grouped)
            route_one_token_grouped(logits + (size_t)t * E, E, k, lane, rp, my_id, my_w);
        else
            route_one_token(logits + (size_t)t * E, E, k, lane, my_id, my_w);
        if (lane < k) {
            topk_ids[(size_t)t * k + lane] = my_id;
            topk_w[(size_t)t * k + lane] = my_w;
            const int local = my_id - local_offset;  // only experts resident here are scheduled
            if (local >= 0 && local < n_local) atomicAdd(&hist[local], 1);
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kRouteThreads)
route_topk_kernel(const float *__restrict__ logits, int T, int E, int k, int local_offset, int n_local,
                  const RouterParams rp, int *__restrict__ topk_ids, float *__restrict__ topk_w,
                  int *__restrict__ chunk_counts) {
    __shared__ int hist[kMaxExperts];  // indexed by local expert (expert id - local_offset)
    chain_release();
    chain_wait();
    route_block_tokens(logits, T, E, k, local_offset, n_local, rp, topk_ids, topk_w, hist);
    for (int e = threadIdx.x; e < n_local; e += kRouteThreads) chunk_counts[(size_t)blockIdx.x * n_local + e] = hist[e];
}

// Exclusive scan over threads 0..255 of the block (wider blocks may call it; their other threads pass 0
// and ignore the result); returns the exclusive prefix, total in *total.
__device__ __forceinline__ int block_exclusive_scan_256(int value, int *warp_sums, int *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = value;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int n = __shfl_up_sync(kFullMask, incl, off);
        if (lane >= off) incl += n;
    }
    if (lane == 31 && warp < 8) warp_sums[warp] = incl;
    __syncthreads();
    int base = 0, sum = 0;
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) {
        const int ws = warp_sums[wi];
        if (wi < warp) base += ws;
        sum += ws;
    }
    __syncthreads();
    *total = sum;
    return base + incl - value;
}

constexpr int kScanThreads = 1024;

// Scan phase, run by one block of a multiple of 256 threads (threads 0..255 carry one expert each for the schedule):
// per-expert running sum over chunks, exclusive scan over experts, token-tile schedule.
// (Pointers are deliberately not __restrict__ and cross-block data is read with __ldcg: in the fused
// kernel these arrays were written by other blocks, or are written here and read again by the scatter.)
__device__ __forceinline__ void scan_phase(int *chunk_counts, int n_chunks, int E, int nt_max, int row_quantum, int *expert_offsets,
                                           int *tile_prefix, int *tile_order, int *tile_rows, int *warp_sums,
                                           int *counts, int *tiles_at, int *part_sums) {
    const int e = threadIdx.x;
    const bool lane_of_scan = e < kMaxExperts;
    // Running sum over chunks per expert.  The block's threads form blockDim.x / 256 parts; part p of expert e
    // first totals its share of the chunks, then, knowing the totals of the parts before it, replaces each of its
    // chunk counts by the rows of all earlier chunks.  (16 independent loads in flight at a time: latency-bound.)
    int count = 0;
    {
        constexpr int kBatch = 16;
        const int pe = threadIdx.x % kMaxExperts, part = threadIdx.x / kMaxExperts, n_parts = blockDim.x / kMaxExperts;
        const int per = (n_chunks + n_parts - 1) / n_parts;
        const int b_begin = min(n_chunks, part * per), b_end = min(n_chunks, b_begin + per);
        const bool one_batch = b_end - b_begin <= kBatch;  // then the counts stay in registers between the passes
        int first[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) first[i] = 0;
        int sum = 0;
        if (pe < E) {
            for (int b0 = b_begin; b0 < b_end; b0 += kBatch) {
                int c[kBatch];
#pragma unroll
                for (int i = 0; i < kBatch; ++i) c[i] = b0 + i < b_end ? __ldcg(&chunk_counts[(size_t)(b0 + i) * E + pe]) : 0;
#pragma unroll
                for (int i = 0; i < kBatch; ++i) sum += c[i];
                if (b0 == b_begin) {
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) first[i] = c[i];
                }
            }
        }
        part_sums[part * kMaxExperts + pe] = sum;
        __syncthreads();
        int run = 0;
        for (int p = 0; p < n_parts; ++p) {
            const int v = part_sums[p * kMaxExperts + pe];
            if (p < part) run += v;
            count += v;
        }
        if (pe < E) {
            for (int b0 = b_begin; b0 < b_end; b0 += kBatch) {
                int c[kBatch];
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    c[i] = one_batch ? first[i] : (b0 + i < b_end ? __ldcg(&chunk_counts[(size_t)(b0 + i) * E + pe]) : 0);
#pragma unroll
                for (int i = 0; i < kBatch; ++i) {
                    if (b0 + i < b_end) chunk_counts[(size_t)(b0 + i) * E + pe] = run;
                    run += c[i];
                }
            }
        }
        if (!lane_of_scan || e >= E) count = 0;  // the schedule below is built by threads 0..E-1
    }
    if (lane_of_scan) {
        counts[e] = e < E ? count : -1;
        tiles_at[e] = 0;
    }
    // token tiles of this expert: one tile if it fits under nt_max; otherwise as few as fit under min(nt_max, 256) --
    // a wide bound (320 / 384) exists to keep an expert in ONE pass over its weights, and consecutive tiles wider than
    // half of tensor memory cannot overlap their epilogues, so experts that need several tiles get 256-row ones --
    // evenly sized, rounded up to the row quantum
    // (16 rows, the MMA's N granularity; the MX path with a bound of up to 256 passes its tile size, so that every tile
    // is exactly that many rows)
    int n_tiles = 0, rows = 0;
    if (count > 0) {
        const int multi = nt_max > 256 ? 256 : nt_max;
        n_tiles = count <= nt_max ? 1 : (count + multi - 1) / multi;
        rows = (((count + n_tiles - 1) / n_tiles) + row_quantum - 1) / row_quantum * row_quantum;
    }
    int total_rows, total_tiles;
    const int row_start = block_exclusive_scan_256(count, warp_sums, &total_rows);  // (syncs: counts[] is visible)
    // Schedule order: experts with more rows first (ties to the lower index), so that tiles of similar
    // cost are adjacent and the GEMMs' static tile assignment stays balanced; the small tiles come last.
    // (all-pairs ranking, E^2 comparisons: every part of the block takes a share of the opponents)
    {
        const int pe = threadIdx.x % kMaxExperts, part = threadIdx.x / kMaxExperts, n_parts = blockDim.x / kMaxExperts;
        part_sums[threadIdx.x] = 0;
        if (pe < E) {
            const int mine = counts[pe];
            const int per = (E + n_parts - 1) / n_parts, o_end = min(E, (part + 1) * per);
            int before = 0;
#pragma unroll 4
            for (int o = part * per; o < o_end; ++o) before += (counts[o] > mine || (counts[o] == mine && o < pe)) ? 1 : 0;
            part_sums[threadIdx.x] = before;
        }
        __syncthreads();
        if (e < E) {
            int pos = 0;
            for (int p = 0; p < n_parts; ++p) pos += part_sums[p * kMaxExperts + e];
            tiles_at[pos] = n_tiles;
            tile_order[pos] = e;
        }
    }
    __syncthreads();
    const int tile_start = block_exclusive_scan_256(lane_of_scan ? tiles_at[e] : 0, warp_sums, &total_tiles);
    if (e < E) {
        expert_offsets[e] = row_start;
        tile_prefix[e] = tile_start;  // indexed by schedule position
        tile_rows[e] = rows;
    }
    if (e == 0) {
        expert_offsets[E] = total_rows;
        tile_prefix[E] = total_tiles;
    }
}

__global__ void __launch_bounds__(kScanThreads)
route_scan_kernel(int *chunk_counts, int n_chunks, int E, int nt_max, int row_quantum, int *expert_offsets,
                  int *tile_prefix, int *tile_order, int *tile_rows) {
    __shared__ int warp_sums[8];
    __shared__ int counts[kMaxExperts], tiles_at[kMaxExperts], part_sums[kScanThreads];
    chain_release();
    chain_wait();
    scan_phase(chunk_counts, n_chunks, E, nt_max, row_quantum, expert_offsets, tile_prefix, tile_order, tile_rows, warp_sums,
               counts, tiles_at, part_sums);
}

// Stable scatter of one chunk (32 tokens) by one warp; next[] is that warp's per-expert cursor.
__device__ __forceinline__ void scatter_chunk(int chunk, const int *topk_ids, const int *chunk_starts,
                                              const int *expert_offsets, int A, int n_local, int local_offset, int k,
                                              int *sorted_to_flat, int *flat_to_sorted, int *next, int lane) {
    // first position of this chunk's assignments to expert e = segment start + rows of earlier chunks
    // (all loads issued before the first use: the loop is a chain of L2 round trips otherwise)
    {
        int start[kMaxExperts / 32];
#pragma unroll
        for (int i = 0; i < kMaxExperts / 32; ++i) {
            const int e = i * 32 + lane;
            start[i] = e < n_local ? __ldcg(&expert_offsets[e]) + __ldcg(&chunk_starts[(size_t)chunk * n_local + e]) : 0;
        }
#pragma unroll
        for (int i = 0; i < kMaxExperts / 32; ++i)
            if (i * 32 + lane < n_local) next[i * 32 + lane] = start[i];
    }
    __syncwarp();
    const int a0 = chunk * kRouteTokensPerBlock * k;
    const int a1 = min(A, a0 + kRouteTokensPerBlock * k);
    constexpr int kAhead = 4;  // groups of 32 assignments whose ids are fetched together
    for (int base0 = a0; base0 < a1; base0 += 32 * kAhead) {
        int ids[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int a = base0 + u * 32 + lane;
            ids[u] = a < a1 ? __ldcg(&topk_ids[a]) - local_offset : -1;
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int a = base0 + u * 32 + lane;
            if (base0 + u * 32 >= a1) break;  // uniform over the warp
            const bool valid = a < a1;
            const int e = ids[u];
            const bool kept = valid && e >= 0 && e < n_local;  // assignments to experts that are not resident are dropped
            const int key = kept ? e : -1 - lane;             // ... and never match anything
            const unsigned same = __match_any_sync(kFullMask, key);
            const int rank = __popc(same & ((1u << lane) - 1u));
            const int pos = kept ? next[e] + rank : -1;
            __syncwarp();
            if (kept && rank == 0) next[e] += __popc(same);
            __syncwarp();
            if (valid) flat_to_sorted[a] = pos;
            if (kept) sorted_to_flat[pos] = a;
        }
    }
}

__global__ void __launch_bounds__(32)
route_scatter_kernel(const int *topk_ids, const int *chunk_starts, const int *expert_offsets, int A, int n_local,
                     int local_offset, int k, int *sorted_to_flat, int *flat_to_sorted) {
    __shared__ int next[kMaxExperts];
    chain_release();
    chain_wait();
    scatter_chunk(blockIdx.x, topk_ids, chunk_starts, expert_offsets, A, n_local, local_offset, k, sorted_to_flat,
                  flat_to_sorted, next, threadIdx.x);
}

// Small batches (at most kFusedMaxChunks chunks = 1024 tokens): the three phases in ONE launch.  Every
// block routes its 32 tokens with one warp per token; the block that finishes last (a counter in the
// status word's padding, zeroed by the caller's memset) then runs the scan phase and scatters every
// chunk, one warp per chunk.  Which block is last does not affect any result.
constexpr int kFusedThreads = 1024;
constexpr int kFusedMaxChunks = kFusedThreads / 32;

__global__ void __launch_bounds__(kFusedThreads)
route_fused_kernel(const float *__restrict__ logits, int T, int E, int k, int local_offset, int n_local, int nt_max,
                   int row_quantum, const RouterParams rp, int *topk_ids, float *topk_w, int *chunk_counts, int *expert_offsets, int *tile_prefix,
                   int *tile_order, int *tile_rows, int *sorted_to_flat, int *flat_to_sorted, int *done_counter) {
    __shared__ int hist[kMaxExperts], counts[kMaxExperts], tiles_at[kMaxExperts], warp_sums[8], part_sums[kFusedThreads];
    __shared__ int next[kFusedMaxChunks][kMaxExperts];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    chain_release();
    chain_wait();
    route_block_tokens(logits, T, E, k, local_offset, n_local, rp, topk_ids, topk_w, hist);
    for (int e = tid; e < n_local; e += kFusedThreads) chunk_counts[(size_t)blockIdx.x * n_local + e] = hist[e];
    __threadfence();  // this block's ids, weights and histogram are visible before it is counted as done
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(done_counter, 1) == (int)gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int n_chunks = gridDim.x;
    scan_phase(chunk_counts, n_chunks, n_local, nt_max, row_quantum, expert_offsets, tile_prefix, tile_order, tile_rows,
               warp_sums, counts, tiles_at, part_sums);
    __syncthreads();  // expert_offsets and the chunk starts written above are read below (same block)
    const int warp = tid >> 5;
    if (warp < n_chunks)
        scatter_chunk(warp, topk_ids, chunk_counts, expert_offsets, T * k, n_local, local_offset, k, sorted_to_flat,
                      flat_to_sorted, next[warp], tid & 31);
}

// Token rows into expert-contiguous order, token-major: a warp reads (a share of) token t's row once and stores
// it to the up to top_k rows flat_to_sorted[t*k + j] >= 0.  Reading each row once instead of once per assignment
// halves the traffic of a top-8 layer; the copies are streamed past L2 (the GEMM reads them from memory anyway).
__global__ void __launch_bounds__(256)
scatter_rows_kernel(const uint4 *__restrict__ x, const int *__restrict__ flat_to_sorted, int T, int k, int vec_per_row,
                    int warps_per_token, uint4 *__restrict__ x_perm) {
    chain_release();
    chain_wait();
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int t = (int)(w / warps_per_token), part = (int)(w % warps_per_token);
    if (t >= T) return;
    const int my_row = lane < k ? flat_to_sorted[(size_t)t * k + lane] : -1;  // lane j holds rank j's destination
    if (!__any_sync(kFullMask, my_row >= 0)) return;  // none of the token's experts is resident here: nothing to copy
    const uint4 *src = x + (size_t)t * vec_per_row;
    constexpr int kInFlight = 4;  // independent 16-byte loads per lane before the first is used
    const int stride = 32 * warps_per_token;
    for (int i0 = part * 32 + lane; i0 < vec_per_row + lane; i0 += kInFlight * stride) {  // (i0 - lane) uniform
        uint4 v[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u)
            if (i0 + u * stride < vec_per_row) v[u] = src[i0 + u * stride];
        for (int j = 0; j < k; ++j) {
            const int row = __shfl_sync(kFullMask, my_row, j);
            if (row < 0) continue;  // assignment to an expert that is not resident here
            uint4 *dst = x_perm + (size_t)row * vec_per_row;
#pragma unroll
            for (int u = 0; u < kInFlight; ++u)
                if (i0 + u * stride < vec_per_row) __stcs(dst + i0 + u * stride, v[u]);
        }
    }
}

// One thread per 16-byte column of one token: the up to eight rows of a batch are fetched together (eight independent
// 16-byte loads in flight per thread), then added one rank after the other, so the summation order is fixed.
constexpr int kCombineThreads = 128, kCombineBatch = 8;
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const uint4 *__restrict__ y, const float *__restrict__ topk_w, const int *__restrict__ flat_to_sorted,
               int k, int vec_per_row, int blocks_per_token, uint4 *__restrict__ out) {
    __shared__ int rows[kMaxTopK];
    __shared__ float weights[kMaxTopK];
    chain_release();
    chain_wait();
    const int t = blockIdx.x / blocks_per_token;
    const int i = (blockIdx.x - t * blocks_per_token) * kCombineThreads + threadIdx.x;
    if (threadIdx.x < k) {
        rows[threadIdx.x] = flat_to_sorted[(size_t)t * k + threadIdx.x];
        weights[threadIdx.x] = topk_w[(size_t)t * k + threadIdx.x];
    }
    __syncthreads();
    if (i >= vec_per_row) return;
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.f;
    for (int j0 = 0; j0 < k; j0 += kCombineBatch) {
        uint4 v[kCombineBatch];
#pragma unroll
        for (int u = 0; u < kCombineBatch; ++u) {
            const bool live = j0 + u < k && rows[j0 + u] >= 0;  // rank exists and its expert is resident here
            v[u] = live ? __ldcs(&y[(size_t)rows[j0 + u] * vec_per_row + i]) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kCombineBatch; ++u) {  // ascending rank
            if (j0 + u >= k || rows[j0 + u] < 0) continue;  // contributes nothing (not even a signed zero)
            const float wj = weights[j0 + u];
            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&v[u]);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 f = __bfloat1622float2(h2[c]);
                acc[2 * c] = fmaf(wj, f.x, acc[2 * c]);
                acc[2 * c + 1] = fmaf(wj, f.y, acc[2 * c + 1]);
            }
        }
    }
    uint4 o;
    __nv_bfloat162 *o2 = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
    for (int c = 0; c < 4; ++c) o2[c] = __floats2bfloat162_rn(acc[2 * c], acc[2 * c + 1]);
    out[(size_t)t * vec_per_row + i] = o;
}

// The same sum for a layer with a resident subset of the experts, where most ranks of most tokens have no row here
// (the paper's 32 of 256: one live rank per token on average).  There the kernel above has one 16-byte load in flight
// per thread and is bound by the latency of that load (3.1 TB/s alone on the machine, 0.09 ms for 8192 tokens).
// Here a block takes kSparseTokens consecutive tokens, lists their live (token, rank) pairs in order, and every
// thread fetches up to kSparseBatch rows at once before it sums them, token after token, rank after rank: the
// same order of summation, the same result, sixteen loads in flight.
constexpr int kSparseTokens = 16, kSparseBatch = 16;
__global__ void __launch_bounds__(kCombineThreads)
combine_sparse_kernel(const uint4 *__restrict__ y, const float *__restrict__ topk_w, const int *__restrict__ flat_to_sorted,
                      int T, int k, int vec_per_row, int blocks_per_group, uint4 *__restrict__ out) {
    __shared__ int live_row[kSparseTokens * kMaxTopK], live_tok[kSparseTokens * kMaxTopK];
    __shared__ float live_w[kSparseTokens * kMaxTopK];
    __shared__ int n_live;
    chain_release();
    chain_wait();
    const int group = blockIdx.x / blocks_per_group;
    const int t0 = group * kSparseTokens, i = (blockIdx.x - group * blocks_per_group) * kCombineThreads + threadIdx.x;
    const int n_tok = min(kSparseTokens, T - t0);
    if (threadIdx.x < 32) {  // warp 0 compacts the live pairs, in (token, rank) order
        int count = 0;
        for (int e0 = 0; e0 < n_tok * k; e0 += 32) {
            const int e = e0 + threadIdx.x;
            const int row = e < n_tok * k ? flat_to_sorted[(size_t)t0 * k + e] : -1;
            const unsigned mask = __ballot_sync(kFullMask, row >= 0);
            if (row >= 0) {
                const int at = count + __popc(mask & ((1u << threadIdx.x) - 1u));
                live_row[at] = row;
                live_tok[at] = e / k;
                live_w[at] = topk_w[(size_t)t0 * k + e];
            }
            count += __popc(mask);
        }
        if (threadIdx.x == 0) n_live = count;
    }
    __syncthreads();
    if (i >= vec_per_row) return;
    const int L = n_live;
    float acc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = 0.f;
    int cur = 0;  // the token whose sum is in acc
    auto flush = [&]() {
        uint4 o;
        __nv_bfloat162 *o2 = reinterpret_cast<__nv_bfloat162 *>(&o);
#pragma unroll
        for (int c = 0; c < 4; ++c) o2[c] = __floats2bfloat162_rn(acc[2 * c], acc[2 * c + 1]);
        out[(size_t)(t0 + cur) * vec_per_row + i] = o;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[c] = 0.f;
        ++cur;
    };
    for (int base = 0; base < L; base += kSparseBatch) {
        uint4 v[kSparseBatch];
#pragma unroll
        for (int u = 0; u < kSparseBatch; ++u)
            v[u] = base + u < L ? __ldcs(&y[(size_t)live_row[base + u] * vec_per_row + i]) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < kSparseBatch; ++u) {
            if (base + u >= L) break;  // (uniform over the block)
            const int tok = live_tok[base + u];
            while (cur < tok) flush();
            const float wj = live_w[base + u];
            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&v[u]);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float2 f = __bfloat1622float2(h2[c]);
                acc[2 * c] = fmaf(wj, f.x, acc[2 * c]);
                acc[2 * c + 1] = fmaf(wj, f.y, acc[2 * c + 1]);
            }
        }
    }
    while (cur < n_tok) flush();
}

}  // namespace

int choose_nt_max(int T, int E, int k, bool wide_ok) {
    const double avg = (double)T * k / E;
    const int options[3] = {32, 64, 128};
    for (int nt : options)
        if (1.5 * avg <= nt) return nt;
    // Between about 160 and 350 rows per expert on average, experts with 257..384 rows are common: a wide bound
    // keeps each of them in one tile (320 while the mean plus 2.5 standard deviations of a uniform routing fits, else
    // 384).  With more rows than that nearly every expert needs several tiles anyway, and those are 256-row tiles.
    if (!wide_ok || avg <= 160.0 || avg > 352.0) return 256;
    return avg + 2.5 * sqrt(avg) <= 320.0 ? 320 : 384;
}

cudaError_t launch_route(const float *logits, int T, int E, int k, LocalExperts local, int nt_max, int *topk_ids,
                         float *topk_w, int *expert_offsets, int *sorted_to_flat, int *flat_to_sorted,
                         RouteScratch scratch, int *status, cudaStream_t stream, int row_quantum, RouterParams router,
                         size_t status_bytes) {
    cudaError_t err = cudaMemsetAsync(status, 0, status_bytes, stream);  // the status word and what shares its region
    if (err != cudaSuccess) return err;
    const int A = T * k;
    if (scratch.n_chunks <= kFusedMaxChunks) {
        return launch_chained(route_fused_kernel, scratch.n_chunks, kFusedThreads, 0, stream, logits, T, E, k, local.offset,
                              local.count, nt_max, row_quantum, router, topk_ids, topk_w, scratch.chunk_counts, expert_offsets,
                              scratch.tile_prefix, scratch.tile_order, scratch.tile_rows, sorted_to_flat, flat_to_sorted,
                              status + kDoneCounterInt);
    }
    err = launch_chained(route_topk_kernel, scratch.n_chunks, kRouteThreads, 0, stream, logits, T, E, k, local.offset,
                         local.count, router, topk_ids, topk_w, scratch.chunk_counts);
    if (err != cudaSuccess) return err;
    err = launch_chained(route_scan_kernel, 1, kScanThreads, 0, stream, scratch.chunk_counts, scratch.n_chunks, local.count,
                         nt_max, row_quantum, expert_offsets, scratch.tile_prefix, scratch.tile_order, scratch.tile_rows);
    if (err != cudaSuccess) return err;
    return launch_chained(route_scatter_kernel, scratch.n_chunks, 32, 0, stream, topk_ids, scratch.chunk_counts,
                          expert_offsets, A, local.count, local.offset, k, sorted_to_flat, flat_to_sorted);
}

// Warps per token: enough warps to fill the device when there are few tokens, at most one per 32 vectors.
static int scatter_warps_per_token(long long tokens, int vec_per_row) {
    const long long target = 32768;
    long long per = tokens > 0 ? (target + tokens - 1) / tokens : 1;
    const int most = (vec_per_row + 31) / 32;
    if (per > most) per = most;
    return per < 1 ? 1 : (int)per;
}

cudaError_t launch_scatter_rows(const __nv_bfloat16 *x, const int *flat_to_sorted, int T, int k, int H, __nv_bfloat16 *x_perm,
                                cudaStream_t stream) {
    const int wpt = scatter_warps_per_token(T, H / 8);
    const long long warps = (long long)T * wpt;
    return launch_chained(scatter_rows_kernel, (unsigned)((warps + 7) / 8), 256, 0, stream,
                          reinterpret_cast<const uint4 *>(x), flat_to_sorted, T, k, H / 8, wpt, reinterpret_cast<uint4 *>(x_perm));
}

cudaError_t launch_combine(const __nv_bfloat16 *y, const float *topk_w, const int *flat_to_sorted, int T, int k,
                           int H, __nv_bfloat16 *out, cudaStream_t stream, bool resident_subset) {
    const int vec_per_row = H / 8, blocks_per_token = (vec_per_row + kCombineThreads - 1) / kCombineThreads;
    if (resident_subset) {
        const long long groups = ((long long)T + kSparseTokens - 1) / kSparseTokens;
        return launch_chained(combine_sparse_kernel, (unsigned)(groups * blocks_per_token), kCombineThreads, 0, stream,
                              reinterpret_cast<const uint4 *>(y), topk_w, flat_to_sorted, T, k, vec_per_row, blocks_per_token,
                              reinterpret_cast<uint4 *>(out));
    }
    return launch_chained(combine_kernel, (unsigned)((long long)T * blocks_per_token), kCombineThreads, 0, stream,
                          reinterpret_cast<const uint4 *>(y), topk_w, flat_to_sorted, k, vec_per_row, blocks_per_token,
                          reinterpret_cast<uint4 *>(out));
}

}  // namespace moe

// ---- moe_route_static: the router + sort-scatter for callers that cannot allocate --------------------
//
// The scratch (status word, per-chunk histograms, tile schedule) lives in a file-scope device array,
// so the caller passes only inputs and outputs.  In host code the array's name is only a handle for
// the runtime, not a device address: its address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that pointer is what the kernels receive.
namespace moe {
namespace {

constexpr size_t kStaticScratchBytes = 512 * 1024;
static __device__ __align__(256) unsigned char g_route_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch on the current device (looked up on the first call per device).
cudaError_t static_scratch_address(void **out) {
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_scratch_ptr[dev]) {
        void *ptr = nullptr;
        err = cudaGetSymbolAddress(&ptr, g_route_static_scratch);
        if (err != cudaSuccess) return err;
        g_static_scratch_ptr[dev] = ptr;
    }
    *out = g_static_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace moe

extern "C" int moe_route_static(const float *router_logits, int T, int E, int top_k, int32_t *topk_ids,
                                float *topk_weights, int32_t *expert_offsets, int32_t *sorted_to_flat,
                                int32_t *flat_to_sorted, void *stream) {
    using namespace moe;
    const int args = check_route_args(router_logits, T, E, top_k, topk_ids, topk_weights, expert_offsets, sorted_to_flat,
                                      flat_to_sorted);
    if (args == MOE_ERR_SHAPE || args == MOE_ERR_UNSUPPORTED) return args;
    if (256 + route_scratch_bytes(T, E) > kStaticScratchBytes) return MOE_ERR_STATIC_LIMIT;
    if (args != MOE_OK) return args;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (T == 0)
        return cudaMemsetAsync(expert_offsets, 0, (size_t)(E + 1) * sizeof(int), s) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
    void *scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess || !scratch) return MOE_ERR_CUDA;
    char *base = static_cast<char *>(scratch);
    // The array keeps the previous call's contents.  The status word is cleared by launch_route; the
    // histogram and schedule regions are fully overwritten for this T and E before they are read.
    RouteScratch rs = carve_route_scratch(base + 256, T, E);
    const cudaError_t err = launch_route(router_logits, T, E, top_k, LocalExperts{0, E}, 256, topk_ids, topk_weights,
                                         expert_offsets, sorted_to_flat, flat_to_sorted, rs,
                                         reinterpret_cast<int *>(base), s);
    return err == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}


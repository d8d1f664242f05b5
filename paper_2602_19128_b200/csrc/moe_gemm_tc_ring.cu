// Grouped expert GEMMs on CTA pairs with WIDE token tiles: one pass over a weight slab serves up to
// NT_MAX (320 or 384) token rows, and the accumulators live in a ring of tensor-memory columns.
//
// What is computed is as in moe_gemm_tc.cu / moe_gemm_tc_pair.cu (paper Sec. 4.5 "Expert FFN computation":
// per expert, gate and up projections combined through SiLU, then the down projection).  What differs:
//
//  * Prefill-sized batches give every expert roughly T*k/E rows; with a 256-row bound an expert with 257..512
//    rows was cut into two tiles of ~half the size, so its weight slab crossed from L2 to the SMs twice and each
//    ring slot carried little MMA time (a slot of N = 144 is 288 tensor-pipe cycles: a 7-slot ring then covers
//    barely 2000 cycles of load latency).  Here such an expert is ONE tile: bytes pulled from L2 per useful flop
//    drop from (1/144 + 1/256) to (1/288 + 1/256), and a slot lasts twice as long.
//  * A tile of N columns no longer fits a fixed half of tensor memory (2 x 320 > 512), so the 512 columns are
//    handed out in 32 chunks of 16 columns, alternately from the two ends: even tiles of a CTA pair occupy columns
//    [0, N), odd tiles [512 - N, 512).  Two consecutive tiles that together exceed 512 columns overlap in the
//    middle, in the LAST columns of the even tile and the FIRST columns of the odd one; the epilogue drains an even
//    tile from its highest column down and an odd tile from its lowest column up, handing chunks back one at a time,
//    and the MMA warp waits (one chunk per lane) only until the previous occupant of each of ITS chunks has been
//    read.  The tensor pipe therefore waits for the first few columns of one epilogue, not for a whole one.
//    (Measured: with 64-column chunks the down GEMM, whose tiles are short, lost 15 % to those waits; handing a
//    chunk back with release semantics made every hand-back wait for the epilogue's global stores.)
//  * An MMA writes at most 256 contiguous columns, so a tile wider than that is issued as two MMAs per K step
//    ("parts" of about N / 2 columns each -- a narrow remainder part would cost as much pipe time as a wide one),
//    both reading the same weight slab.  Each CTA still stages ONE contiguous half of the token tile with ONE copy;
//    part p reads rows [o_p, o_p + n_p / 2) of both halves, so its accumulator columns [0, n_p / 2) are tile rows
//    o_p.., and columns [n_p / 2, n_p) are tile rows N / 2 + o_p...  The epilogue applies that map.
//  * The MMA warp decodes nothing: the leader's weight producer, which runs ahead by the depth of the ring, writes
//    each tile's column count into a small queue in shared memory before it arms the tile's first slot, and the
//    MMA warp reads it after that slot's barrier (release / acquire through the barrier).  Between two tiles the
//    tensor pipe therefore waits for no global load.
//
// Roles, barriers and the bounded waits are those of moe_gemm_tc_pair.cu.
#include "moe_tc_pair.cuh"

namespace moe {
namespace {

using namespace tc;

constexpr int kRingThreads = 224;   // warp 0 weight TMA, warp 1 MMA, warps 2..5 epilogue, warp 6 token TMA
constexpr int kChunkCols = 16;      // granularity of the accumulator ring: the MMA's N granularity
constexpr int kNumChunks = 32;      // 512 columns of tensor memory
constexpr int kAccFullBars = 32;    // tiles between the MMA warp and the epilogue: each holds at least one chunk
constexpr int kTileQueue = 16;      // more entries than ring slots: the producer is at most STAGES tiles ahead
constexpr int kRingActMaps = 24;    // act[i]: box of 8 * (i + 1) rows, up to 192 rows per CTA (N = 384)
constexpr int kOutStageBytes = 16 * kTileM * 2;  // one 16-column group of a CTA's 128 output rows, token-major

struct RingMaps {
    CUtensorMap w;
    CUtensorMap act[kRingActMaps];
    CUtensorMap x;  // gather-in-load only: the layer's input [T, H] with a box of ONE row of 64 columns
};

// Four rows of a 2-D tensor, given by their row indices, into four consecutive 128-byte rows of shared memory
// (TMA tile::gather4); completes on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_gather4_pair(uint32_t dst, const CUtensorMap *map, int col, int r0, int r1, int r2, int r3,
                                                 uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

template <int NT_MAX, int STAGES>
struct RingSmem {
    static constexpr int kSlotBBytes = (NT_MAX / 2) * kRowBytes;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kSlotABytes;
    static constexpr int kOutStage = kB + STAGES * kSlotBBytes;  // down projection: two [16 tokens][128 rows] bf16 tiles
    static constexpr int kBars = kOutStage + 2 * kOutStageBytes;  // full[S], empty[S], acc_full[32], acc_empty[32]
    static constexpr int kQueue = kBars + (2 * STAGES + kAccFullBars + kNumChunks) * 8;
    static constexpr int kTmemSlot = kQueue + kTileQueue * 4;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kPairDynamicSmemBytes;  // (kBytes + 1024 of it are used)
};

// The MMAs of one tile: part i writes `cols[i]` accumulator columns starting at absolute column `col[i]` and reads
// rows [row[i], row[i] + cols[i] / 2) of each CTA's staged half of the token tile.  Even tiles are anchored at
// column 0, odd tiles at the top of tensor memory.
struct Parts {
    int n, first_col;
    int col[2], cols[2], row[2];
};
__device__ __forceinline__ Parts split_tile(int seq, int n_cols) {
    Parts s;
    s.first_col = (seq & 1) ? kNumChunks * kChunkCols - n_cols : 0;
    s.n = n_cols > 256 ? 2 : 1;
    s.cols[0] = n_cols > 256 ? (((n_cols >> 1) + 15) & ~15) : n_cols;
    s.cols[1] = n_cols - s.cols[0];
    s.col[0] = s.first_col;
    s.col[1] = s.first_col + s.cols[0];
    s.row[0] = 0;
    s.row[1] = s.cols[0] >> 1;
    return s;
}

template <int NT_MAX, int STAGES, bool SWIGLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kRingThreads, 1)
grouped_gemm_tc_ring_kernel(const __grid_constant__ RingMaps maps, const KernelParams p) {
    using L = RingSmem<NT_MAX, STAGES>;
    static_assert(NT_MAX % 16 == 0 && NT_MAX <= 16 * kRingActMaps && NT_MAX <= 384, "token-tile bound");
    static_assert(STAGES < kTileQueue, "the tile queue must outlast the ring");
    constexpr int kTmemCols = kNumChunks * kChunkCols;   // all of tensor memory (a power of two)
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;          // the down GEMM reports sites 5..8
    constexpr int kFeatPerCta = SWIGLU ? kTileM / 2 : kTileM;
    constexpr int kFeatPerTile = 2 * kFeatPerCta;
    chain_release();  // the next kernel of the forward call may be scheduled; it waits for this grid to finish
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBars, bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + STAGES * 8, bar_acc_empty = bar_acc_full + kAccFullBars * 8;
    volatile int *queue = reinterpret_cast<volatile int *>(base_ptr + L::kQueue);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const uint32_t peer_abort = map_to_cta(base + L::kAbort, rank ^ 1u);
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + s * 8, 1);
            mbar_init(bar_empty + s * 8, 1);
        }
        for (int a = 0; a < kAccFullBars; ++a) mbar_init(bar_acc_full + a * 8, 1);
        for (int c = 0; c < kNumChunks; ++c) mbar_init(bar_acc_empty + c * 8, 2 * kEpilogueWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {  // collective over the same warp of both CTAs
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + L::kTmemSlot),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything can signal them
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above overlapped the previous kernel; its results are read from here on
    const bool started = gemm_chain_start(p.handover_role, p.handover, abort_flag, p.status);
    const int total_tiles = started ? p.tile_prefix[p.E] * p.n_feature_tiles : 0;
    const int n_pairs = gridDim.x >> 1, pair = blockIdx.x >> 1;
    clock_probe_begin(p.status, SWIGLU ? 0 : 1);

    // ---------------- TMA producers (both CTAs): weight slab and token rows from two different warps ----------------
    auto producer_loop = [&](const bool load_w, const bool load_act) {  // run by a whole warp
        int stage = 0, seq = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round, ++seq) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15, half = n_mma >> 1;  // each CTA stages half: a multiple of 8 rows
            const int feat0 = t.f * kFeatPerTile + (int)rank * kFeatPerCta;
            if (load_act) {  // the token rows of a down GEMM are the gate/up GEMM's output for this expert
                ok = handover_wait_expert(p.handover_role, p.handover, t.e, t.n_tok_tiles, p.handover_per_token_tile,
                                          p.tile_prefix[p.E], gate_up_done, abort_flag, p.status, lane);
                if (!ok) { store_cluster_u32(peer_abort, 1u); break; }
            }
            // Gather-in-load: this CTA's half of the token tile is fetched straight from the layer's input, four rows
            // per copy; lane l owns rows 4l..4l+3 and 128+4l..131+4l of the half.  Rows past the expert's end read token 0.
            int tok[2][4];
            if (load_act && p.gather_tokens) {
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int row = (int)rank * half + r * 128 + 4 * lane + u;  // within the tile
                        tok[r][u] = (r * 128 + 4 * lane + u < half && row < t.n_valid) ? p.sorted_to_flat[t.row0 + row] / p.top_k : 0;
                    }
            }
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = __all_sync(0xffffffffu, pair_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, peer_abort, p.status,
                                                       kSiteProducerEmpty + kSiteOffset));
                if (!ok) break;
                if (load_act && p.gather_tokens) {  // every lane issues its own copies
                    const uint32_t full = map_to_cta(bar_full + stage * 8, 0);
                    const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                    const int k0 = kb * kBlockK;
                    if (4 * lane < half)
                        tma_gather4_pair(sb + lane * 4 * kRowBytes, &maps.x, k0, tok[0][0], tok[0][1], tok[0][2], tok[0][3], full);
                    if (128 + 4 * lane < half)
                        tma_gather4_pair(sb + (32 + lane) * 4 * kRowBytes, &maps.x, k0, tok[1][0], tok[1][1], tok[1][2], tok[1][3],
                                         full);
                } else if (elect_one()) {
                    const uint32_t full = map_to_cta(bar_full + stage * 8, 0);
                    const int k0 = kb * kBlockK;
                    if (load_w) {
                        if (rank == 0) {
                            // the MMA warp learns the tile's width from here, after this slot's barrier
                            if (kb == 0) queue[seq & (kTileQueue - 1)] = n_mma;
                            mbar_expect_tx(bar_full + stage * 8, 2 * kSlotABytes + n_mma * kRowBytes);
                        }
                        const uint32_t sa = base + L::kA + stage * kSlotABytes;
                        if (SWIGLU)  // 64 features = 4 groups of 16, gate and up rows interleaved per group
                            tma_load_5d_pair(sa, &maps.w, k0, 0, 0, feat0 >> 4, t.e, full);
                        else
                            tma_load_2d_pair(sa, &maps.w, k0, t.e * p.w_rows + feat0, full);
                    }
                    if (load_act) {
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                        tma_load_2d_pair(sb, &maps.act[half / 8 - 1], k0, t.row0 + (int)rank * half, full);
                    }
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        // wait until every slot has been handed back: no commit may arrive here after exit
        for (int s = 0; ok && s < STAGES; ++s) {
            ok = __all_sync(0xffffffffu, pair_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, peer_abort, p.status,
                                                   kSiteProducerEmpty + kSiteOffset));
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    };
    if (warp == 0) {
        producer_loop(true, false);
    } else if (warp == kRingThreads / 32 - 1) {
        producer_loop(false, true);
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only): the warp walks the ring, one elected lane issues ----------------
        if (rank == 0) {
            int stage = 0, seq = 0;
            uint32_t phase = 0, chunk_phase = 0;  // bit c: parity of chunk c's next hand-back
            bool ok = true;
            for (int round = 0; ok; ++round, ++seq) {
                const int tile = tile_of_round(round, pair, n_pairs);
                if (tile >= total_tiles) break;
                Parts parts;
                parts.n = 0;
                for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, pair_wait(bar_full + stage * 8, phase, abort_flag, peer_abort, p.status,
                                                           kSiteMmaFull + kSiteOffset));
                    if (!ok) break;
                    if (kb == 0) {
                        // the tile's width, then its chunks of the accumulator ring, each free of its last occupant
                        const int n_mma = queue[seq & (kTileQueue - 1)];
                        const int n_chunks = n_mma / kChunkCols;
                        parts = split_tile(seq, n_mma);
                        {   // lane c waits for the tile's c-th chunk
                            const int first = parts.first_col / kChunkCols, chunk = (first + lane) & (kNumChunks - 1);
                            bool mine = true;
                            if (lane < n_chunks)
                                mine = pair_wait(bar_acc_empty + chunk * 8, ((chunk_phase >> chunk) & 1u) ^ 1u, abort_flag, peer_abort,
                                                 p.status, kSiteMmaTmemEmpty + kSiteOffset);
                            ok = __all_sync(0xffffffffu, mine);
                            chunk_phase ^= (n_chunks >= 32 ? 0xffffffffu : ((1u << n_chunks) - 1u)) << first;
                        }
                        if (!ok) break;
                    }
                    tcgen05_fence_after();
                    if (elect_one()) {
                        const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kA + stage * kSlotABytes);
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            if (i < parts.n) {
                                const uint64_t b_desc = smem_desc_k_major_sw128(sb + parts.row[i] * kRowBytes);
                                const uint32_t idesc = instr_desc_bf16(2 * kTileM, parts.cols[i]);
#pragma unroll
                                for (int kk = 0; kk < kBlockK / 16; ++kk)  // 16 K-elements = 32 bytes = 2 descriptor units
                                    umma_bf16_pair(tmem_base + parts.col[i], a_desc + 2 * kk, b_desc + 2 * kk, idesc,
                                                   (kb | kk) != 0);
                            }
                        }
                        umma_commit_pair(bar_empty + stage * 8);
                        if (kb == p.n_k_blocks - 1) umma_commit_pair(bar_acc_full + (seq & (kAccFullBars - 1)) * 8);
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // wait until every chunk has been handed back by both CTAs' epilogues (lane c: chunk c)
            if (ok)
                ok = __all_sync(0xffffffffu, pair_wait(bar_acc_empty + lane * 8, ((chunk_phase >> lane) & 1u) ^ 1u, abort_flag,
                                                       peer_abort, p.status, kSiteMmaTmemEmpty + kSiteOffset));
        }
    } else {
        // ---------------- epilogue (both CTAs): own 128 weight rows x all N tokens ----------------
        const int q = warp & 3;  // a warp may only read TMEM lanes 32*(warp%4) .. +31
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        int seq = 0, out_flip = 0;
        bool ok = true;
        for (int round = 0; ok; ++round, ++seq) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15, half_tile = n_mma >> 1;
            const Parts parts = split_tile(seq, n_mma);
            ok = pair_wait(bar_acc_full + (seq & (kAccFullBars - 1)) * 8, (uint32_t)(seq / kAccFullBars) & 1u, abort_flag, peer_abort,
                           p.status, kSiteEpilogueTmemFull + kSiteOffset);
            if (epilogue_any(!ok)) break;  // the four warps synchronise inside a down-projection tile: they leave together
            tcgen05_fence_after();
            const int lane_feat = SWIGLU ? q * 16 + (lane & 15) : q * 32 + lane;
            __nv_bfloat16 *dst_rows = p.out + (size_t)t.row0 * p.n_out + t.f * kFeatPerTile + (int)rank * kFeatPerCta;
            __nv_bfloat16 *dst = dst_rows + lane_feat;
            const size_t row_stride = (size_t)p.n_out;
            // An even tile is drained from its highest 16 columns down, an odd tile from its lowest up: the columns the
            // next tile of this pair is waiting for go back first.
            const int n_groups = n_mma >> 4;
#pragma unroll 1
            for (int g = 0; g < n_groups; ++g) {
                const int tile_col = ((seq & 1) ? g : n_groups - 1 - g) << 4;        // first column of the group, within the tile
                const int part = tile_col >= parts.cols[0] ? 1 : 0;
                const int c0 = tile_col - (part ? parts.cols[0] : 0);               // ... within its part
                const int half = (part ? parts.cols[1] : parts.cols[0]) >> 1;
                // Accumulator column j of a part is tile row  j < half ? row + j : N/2 + row + (j - half).  `half` is a
                // multiple of 8, so the group's columns 0..7 are eight consecutive rows and so are its columns 8..15.
                const int row_lo = part ? parts.row[1] : 0, row_hi = half_tile + row_lo - half;
                const int row_a = c0 < half ? row_lo + c0 : row_hi + c0;
                const int row_b = c0 + 8 < half ? row_lo + c0 + 8 : row_hi + c0 + 8;
                float v[16];
                tmem_load_16(lane_base + parts.first_col + tile_col, v);
                // the chunk goes back as soon as its columns have been read
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0)
                    mbar_arrive_cluster_relaxed(map_to_cta(bar_acc_empty + ((parts.first_col + tile_col) / kChunkCols) * 8, 0));
                const bool all_valid = row_a + 8 <= t.n_valid && row_b + 8 <= t.n_valid;  // (uniform over the warp)
                if (SWIGLU) {  // lanes 0..15 hold gate, lanes 16..31 up of the same 16 features
                    const int hi = lane >> 4;
                    const int row0 = hi ? row_b : row_a;  // this lane stores columns hi*8 .. hi*8+7 of the group
                    __nv_bfloat16 *out_row = dst + (size_t)row0 * row_stride;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const float other = __shfl_xor_sync(0xffffffffu, hi ? v[u] : v[8 + u], 16);
                        const float gt = hi ? other : v[u];
                        const float up = hi ? v[8 + u] : other;
                        if (all_valid || row0 + u < t.n_valid) *out_row = __float2bfloat16_rn(swiglu(gt, up));
                        out_row += row_stride;
                    }
                } else {
                    // A lane holds one output feature of 16 tokens; stored from here a warp instruction would write
                    // 32 x 2 bytes of one token.  The four warps transpose the group through shared memory instead and
                    // each stores four whole 256-byte token rows, 16 bytes per lane.
                    out_flip ^= 1;  // (across tiles too: two consecutive groups never share a buffer)
                    uint8_t *stage_buf = base_ptr + L::kOutStage + out_flip * kOutStageBytes;
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        reinterpret_cast<__nv_bfloat16 *>(stage_buf)[i * kTileM + q * 32 + lane] = __float2bfloat16_rn(v[i]);
                    asm volatile("bar.sync 2, 128;" ::: "memory");  // (two buffers: the next group's writes cannot pass this)
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int r = q * 4 + it * 2 + (lane >> 4);          // column of the group
                        const int row = r < 8 ? row_a + r : row_b + r - 8;   // ... and its tile row
                        const uint4 val = *reinterpret_cast<const uint4 *>(stage_buf + r * (kTileM * 2) + (lane & 15) * 16);
                        if (row < t.n_valid)
                            *reinterpret_cast<uint4 *>(dst_rows + (size_t)row * row_stride + (lane & 15) * 8) = val;
                    }
                }
            }
            handover_count_tile(p.handover_role, p.handover, t.e, lane);  // (after the accumulator has been handed back)
        }
    }

    // ---------------- teardown ----------------
    gemm_chain_finish(p.handover_role);
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    clock_probe_end(p.status, SWIGLU ? 0 : 1);
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    tmem_release_pair(tmem_base, kTmemCols, warp);
}

template <int NT_MAX, int STAGES, bool SWIGLU>
int launch_ring_instance(const RingMaps &maps, const KernelParams &p, int grid, cudaStream_t stream) {
    using L = RingSmem<NT_MAX, STAGES>;
    static_assert(L::kBytes + 1024 <= L::kDynamicBytes, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_ring_kernel<NT_MAX, STAGES, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kRingThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace

// The wide-tile kernel serves token-tile bounds 320 and 384 on shapes its 256-row (128-feature for gate/up) pair
// tile divides.
bool grouped_gemm_tc_ring_applies(const GroupedGemmArgs &a) {
    if (!(a.nt_max == 320 || a.nt_max == 384) || a.K % kBlockK != 0 || a.A <= 0) return false;
    return a.n_out % (a.swiglu ? kTileM : 2 * kTileM) == 0;
}

int launch_grouped_gemm_tc_ring(const GroupedGemmArgs &a, cudaStream_t stream) {
    if (!grouped_gemm_tc_ring_applies(a)) return MOE_ERR_UNSUPPORTED;
    RingMaps maps;
    const bool ok_w = a.swiglu ? encode_weight_map_gate_up(&maps.w, a.w, a.E, a.n_out, a.K)
                               : encode_weight_map_2d(&maps.w, a.w, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w) return MOE_ERR_CUDA;
    if (a.gather_x) {  // token rows come straight from x [T, K]: one map whose box is a single row of 64 columns
        if (!a.swiglu || !encode_row_map(&maps.x, a.gather_x, (uint64_t)a.gather_T, a.K)) return MOE_ERR_CUDA;
    } else if (!encode_act_maps(maps.act, a.act, a.A, a.K, 8, a.nt_max / 16)) {
        return MOE_ERR_CUDA;
    }

    KernelParams p;
    p.out = a.out;
    p.expert_offsets = a.expert_offsets;
    p.tile_prefix = a.tile_prefix;
    p.tile_order = a.tile_order;
    p.tile_rows = a.tile_rows;
    p.status = a.status;
    p.E = a.E;
    p.n_k_blocks = a.K / kBlockK;
    p.n_out = a.n_out;
    p.w_rows = a.w_rows;
    p.w_scale = nullptr;
    p.handover_role = a.handover_role;
    p.handover = a.handover;
    p.handover_per_token_tile = a.handover_per_token_tile;
    p.n_feature_tiles = a.n_out / (a.swiglu ? kTileM : 2 * kTileM);
    p.gather_tokens = a.gather_x != nullptr;
    p.sorted_to_flat = a.gather_sorted_to_flat;
    p.top_k = a.gather_top_k;

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / 256;  // (experts above the bound: 256-row tiles)
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int pairs_on_device = sm_count() / 2;
    const int n_pairs = (int)(max_tiles < pairs_on_device ? max_tiles : pairs_on_device);
    const int grid = 2 * (n_pairs > 0 ? n_pairs : 1);
    if (a.nt_max == 320)
        return a.swiglu ? launch_ring_instance<320, 6, true>(maps, p, grid, stream)
                        : launch_ring_instance<320, 6, false>(maps, p, grid, stream);
    return a.swiglu ? launch_ring_instance<384, 5, true>(maps, p, grid, stream)
                    : launch_ring_instance<384, 5, false>(maps, p, grid, stream);
}

}  // namespace moe

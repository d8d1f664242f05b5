// Grouped expert GEMMs in MX FP8 on CTA pairs with WIDE token tiles (up to 304 / 384 rows): the block-scaled MMA of
// moe_gemm_tc_mx_pair.cu on the accumulator ring of moe_gemm_tc_ring.cu.
//
// What is computed: paper Sec. 4.5 "Expert FFN computation" (gate/up with SiLU, then down) on the FP8 workload of
// Table 2, with the MX operands described in moe_gemm_tc_mx.cu.  Why: with the 240-row bound of the pair kernel
// (two accumulators of 240 columns and the scale columns fill tensor memory) a prefill-sized expert of 241..480 rows
// is two tiles, its weight slab crosses from L2 to the SMs twice, and the second, narrow tile costs almost as much
// as the first, because a ring slot is bound by the rows the copy engine brings (128 weight rows either way), not by
// the MMAs.  Here such an expert is ONE tile.
//
// Tensor memory: columns [0, 496) are the accumulator ring, 31 chunks of 16 columns handed out from the two ends
// (even tiles of a pair at column 0, odd tiles ending at column 496; the epilogue drains an even tile from its
// highest chunk down and an odd one from its lowest up and hands chunks back one by one); columns [496, 500) hold the
// weight scales of the current K slot and [500, 512) the token scales (three atoms of 128 rows).
//
// An MMA writes at most 256 columns, so a wider tile is two MMAs per K step: rows [0, 128) and rows [128, N) of the
// tile.  Unlike the bf16 ring kernel each part is staged on its own -- each CTA copies its half of the first 128 rows
// and its half of the rest, two copies per slot -- so that accumulator column j is tile row j and the token scales,
// whose atoms are 128 rows, are read in place: part 0 uses atom 0, part 1 atoms 1 and 2.
//
// Roles, barriers, the tile-width queue and the bounded waits are those of the two kernels this one combines.
#include "moe_mx_tc.cuh"
#include "moe_tc_pair.cuh"

namespace moe {
namespace {

using namespace tc;
using namespace mxtc;

constexpr int kMxRingThreads = 224;  // warp 0 weight TMA, warp 1 MMA, warps 2..5 epilogue, warp 6 token TMA
constexpr int kChunkCols = 16;       // granularity of the accumulator ring: the MMA's N granularity
constexpr int kAccCols = 496;        // accumulator columns; the scales take the last 16 of tensor memory
constexpr int kNumChunks = kAccCols / kChunkCols;  // 31
constexpr int kAccFullBars = 32;     // tiles between the MMA warp and the epilogue: each holds at least one chunk
constexpr int kTileQueue = 16;       // more entries than ring slots: the producer is at most STAGES tiles ahead
constexpr uint32_t kSfACol = kAccCols, kSfBCol = kAccCols + 4;
constexpr int kOutStageBytes = 16 * kTileM * 2;  // one 16-column group of a CTA's 128 output rows, token-major

struct MxRingMaps {
    TensorMaps ops;            // weight codes, token codes (boxes of 8, 16, ..., 128 rows)
    CUtensorMap w_sf, act_sf;  // scale atoms
};

// In both CTAs of the pair: one scale atom from that CTA's shared memory to its tensor memory.
__device__ __forceinline__ void tmem_copy_sf_atom_pair(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
__device__ __forceinline__ void umma_mx_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate, uint32_t sfa_tmem, uint32_t sfb_tmem) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

template <int NT_MAX, int STAGES, bool SWIGLU>
struct MxRingSmem {
    static constexpr int kAtomsB = (NT_MAX + 127) / 128;
    static constexpr int kSlotBBytes = (NT_MAX / 2) * kMxSlotK;
    static constexpr int kSfBBytes = kAtomsB * kMxSfAtomBytes;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kMxSlotABytes;
    static constexpr int kSfA = kB + STAGES * kSlotBBytes;
    static constexpr int kSfB = kSfA + STAGES * kMxSfAtomBytes;
    static constexpr int kAmax = kSfB + STAGES * kSfBBytes;
    static constexpr int kOutStage = kAmax + 2 * 4 * 16 * 4;  // down projection only: two [16 tokens][128 rows] bf16 tiles
    static constexpr int kBars = kOutStage + (SWIGLU ? 0 : 2 * kOutStageBytes);  // full[S], empty[S], acc_full[32], acc_empty[32 (31 used)]
    static constexpr int kQueue = kBars + (2 * STAGES + kAccFullBars + 32) * 8;
    static constexpr int kTmemSlot = kQueue + kTileQueue * 4;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kPairDynamicSmemBytes;  // (kBytes + 1024 of it are used)
};

// The MMAs of one tile: part i writes `cols[i]` accumulator columns starting at absolute column `col[i]`; they are
// tile rows [row[i], row[i] + cols[i]).  Even tiles are anchored at column 0, odd tiles end at the ring's last column.
struct MxParts {
    int n, first_col;
    int col[2], cols[2], row[2];
};
__device__ __forceinline__ MxParts split_mx_tile(int seq, int n_cols) {
    MxParts s;
    s.first_col = (seq & 1) ? kAccCols - n_cols : 0;
    s.n = n_cols > 256 ? 2 : 1;
    s.cols[0] = n_cols > 256 ? 128 : n_cols;  // (one scale atom: part 1 starts on an atom boundary)
    s.cols[1] = n_cols - s.cols[0];
    s.col[0] = s.first_col;
    s.col[1] = s.first_col + s.cols[0];
    s.row[0] = 0;
    s.row[1] = s.cols[0];
    return s;
}

template <int NT_MAX, int STAGES, bool SWIGLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kMxRingThreads, 1)
grouped_gemm_tc_mx_ring_kernel(const __grid_constant__ MxRingMaps maps, const MxParams p) {
    using L = MxRingSmem<NT_MAX, STAGES, SWIGLU>;
    static_assert(NT_MAX % 16 == 0 && NT_MAX <= 384 && NT_MAX > 256, "token-tile bound of the wide-tile kernel");
    static_assert(L::kAtomsB == 3, "three token scale atoms next to the weight scales");
    static_assert(STAGES < kTileQueue, "the tile queue must outlast the ring");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;
    constexpr int kFeatPerCta = SWIGLU ? kTileM / 2 : kTileM;  // h features resp. output rows per CTA of a pair tile
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
                     "r"(kTmemColsMx)
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
    const int w_tiles_per_expert = p.n_out / kFeatPerCta;  // weight scale atoms are stored per 128-row CTA tile

    // ---------------- TMA producers (both CTAs): weight side in warp 0, token side in warp 6 ----------------
    auto producer_loop = [&](const bool load_w, const bool load_act) {
        int stage = 0, seq = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round, ++seq) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const MxParts parts = split_mx_tile(seq, n_mma);
            const int cta_tile = 2 * t.f + (int)rank;  // this CTA's 128 weight rows
            const int w_sf_row = (t.e * w_tiles_per_expert + cta_tile) * p.n_k_blocks;
            if (load_act) {  // the token rows of a down GEMM are the gate/up GEMM's output for this expert
                ok = handover_wait_expert(p.handover_role, p.handover, t.e, t.n_tok_tiles, p.handover_per_token_tile,
                                          p.tile_prefix[p.E], gate_up_done, abort_flag, p.status, lane);
                if (!ok) { store_cluster_u32(peer_abort, 1u); break; }
            }
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = __all_sync(0xffffffffu, pair_wait(bar_empty + stage * 8, phase ^ 1u, abort_flag, peer_abort, p.status,
                                                       kSiteProducerEmpty + kSiteOffset));
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = map_to_cta(bar_full + stage * 8, 0);
                    const int k0 = kb * kMxSlotK;
                    if (load_w) {
                        if (rank == 0) {
                            // the MMA warp learns the tile's width from here, after this slot's barrier
                            if (kb == 0) queue[seq & (kTileQueue - 1)] = n_mma;
                            mbar_expect_tx(bar_full + stage * 8,
                                           2 * (kMxSlotABytes + kMxSfAtomBytes + L::kSfBBytes) + n_mma * kMxSlotK);
                        }
                        const uint32_t sa = base + L::kA + stage * kMxSlotABytes;
                        if (SWIGLU)  // 64 features = 4 groups of 16, gate and up rows interleaved per group
                            tma_load_5d_pair(sa, &maps.ops.w, k0, 0, 0, cta_tile * 4, t.e, full);
                        else
                            tma_load_2d_pair(sa, &maps.ops.w, k0, t.e * p.w_rows + cta_tile * kTileM, full);
                        tma_load_2d_pair(base + L::kSfA + stage * kMxSfAtomBytes, &maps.w_sf, 0, w_sf_row + kb, full);
                    }
                    if (load_act) {
                        // this CTA's half of each part, one copy per part: part 1 lands behind part 0's 64 rows
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            if (i < parts.n) {
                                const int half = parts.cols[i] >> 1;
                                tma_load_2d_pair(sb + (i ? (parts.cols[0] >> 1) * kMxSlotK : 0), act_map<8>(maps.ops, half), k0,
                                                 t.row0 + parts.row[i] + (int)rank * half, full);
                            }
                        }
                        tma_load_2d_pair(base + L::kSfB + stage * L::kSfBBytes, &maps.act_sf, 0, kb * p.n_atoms + t.atom, full);
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
    } else if (warp == kMxRingThreads / 32 - 1) {
        producer_loop(false, true);
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only): the warp walks the ring, one elected lane issues ----------------
        if (rank == 0) {
            int stage = 0, seq = 0;
            uint32_t phase = 0, chunk_phase = 0;  // bit c: parity of chunk c's next hand-back
            bool ok = true;
            const uint32_t sfa_tmem = tmem_base + kSfACol, sfb_tmem = tmem_base + kSfBCol;
            for (int round = 0; ok; ++round, ++seq) {
                const int tile = tile_of_round(round, pair, n_pairs);
                if (tile >= total_tiles) break;
                MxParts parts;
                parts.n = 0;
                for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, pair_wait(bar_full + stage * 8, phase, abort_flag, peer_abort, p.status,
                                                           kSiteMmaFull + kSiteOffset));
                    if (!ok) break;
                    if (kb == 0) {
                        // the tile's width, then its chunks of the accumulator ring, each free of its last occupant
                        const int n_mma = queue[seq & (kTileQueue - 1)];
                        const int n_chunks = n_mma / kChunkCols;
                        parts = split_mx_tile(seq, n_mma);
                        {   // lane c waits for the tile's c-th chunk (a tile has at most 24)
                            const int first = parts.first_col / kChunkCols, chunk = first + lane;
                            bool mine = true;
                            if (lane < n_chunks)
                                mine = pair_wait(bar_acc_empty + chunk * 8, ((chunk_phase >> chunk) & 1u) ^ 1u, abort_flag, peer_abort,
                                                 p.status, kSiteMmaTmemEmpty + kSiteOffset);
                            ok = __all_sync(0xffffffffu, mine);
                            chunk_phase ^= ((1u << n_chunks) - 1u) << first;
                        }
                        if (!ok) break;
                    }
                    tcgen05_fence_after();
                    if (elect_one()) {
                        tmem_copy_sf_atom_pair(sfa_tmem, smem_desc_sf_atom(base + L::kSfA + stage * kMxSfAtomBytes));
#pragma unroll
                        for (int a = 0; a < L::kAtomsB; ++a)
                            tmem_copy_sf_atom_pair(sfb_tmem + 4 * a,
                                                   smem_desc_sf_atom(base + L::kSfB + stage * L::kSfBBytes + a * kMxSfAtomBytes));
                        const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kA + stage * kMxSlotABytes);
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            if (i < parts.n) {
                                const uint64_t b_desc = smem_desc_k_major_sw128(sb + (i ? (parts.cols[0] >> 1) * kMxSlotK : 0));
                                const uint32_t sfb_part = sfb_tmem + (i ? 4u : 0u);  // part 1 starts at tile row 128: atom 1
#pragma unroll
                                for (int kk = 0; kk < kMxSlotK / 32; ++kk)
                                    umma_mx_pair(tmem_base + parts.col[i], a_desc + 2 * kk, b_desc + 2 * kk,
                                                 instr_desc_mx(2 * kTileM, parts.cols[i], kk), (kb | kk) != 0, sfa_tmem, sfb_part);
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
            if (ok) {
                bool mine = true;
                if (lane < kNumChunks)
                    mine = pair_wait(bar_acc_empty + lane * 8, ((chunk_phase >> lane) & 1u) ^ 1u, abort_flag, peer_abort, p.status,
                                     kSiteMmaTmemEmpty + kSiteOffset);
                ok = __all_sync(0xffffffffu, mine);
            }
        }
    } else {
        // ---------------- epilogue (both CTAs): own 128 weight rows x all N tokens ----------------
        const int q = warp & 3;  // a warp may only read TMEM lanes 32*(warp%4) .. +31
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t *amax_s = reinterpret_cast<uint32_t *>(base_ptr + L::kAmax);
        int buf = 0, seq = 0, out_flip = 0;
        for (int round = 0;; ++round, ++seq) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const MxParts parts = split_mx_tile(seq, n_mma);
            const bool ok = pair_wait(bar_acc_full + (seq & (kAccFullBars - 1)) * 8, (uint32_t)(seq / kAccFullBars) & 1u, abort_flag,
                                      peer_abort, p.status, kSiteEpilogueTmemFull + kSiteOffset);
            if (epilogue_any(!ok)) break;  // the four warps synchronise inside the tile, so they leave together
            tcgen05_fence_after();
            const int feat0 = (2 * t.f + (int)rank) * kFeatPerCta;  // first feature / output row of this CTA
            // An even tile is drained from its highest 16 columns down, an odd tile from its lowest up: the columns the
            // next tile of this pair is waiting for go back first.  Accumulator column j is tile row j.
            const int n_groups = n_mma >> 4;
            const int hi = lane >> 4, j16 = lane & 15;
            uint8_t *dst_q = nullptr, *sf_dst = nullptr;
            __nv_bfloat16 *dst_rows = nullptr;
            if (SWIGLU) {
                dst_q = static_cast<uint8_t *>(p.out) + (size_t)t.row0 * p.n_out + feat0 + q * 16 + j16;
                const int block = (feat0 + q * 16) >> 5;  // 32-feature block = scale byte `block % 4` of K-slot `block / 4`
                sf_dst = p.out_sf + ((size_t)(block >> 2) * p.n_atoms + t.atom) * kMxSfAtomBytes + (block & 3);
            } else {
                dst_rows = static_cast<__nv_bfloat16 *>(p.out) + (size_t)t.row0 * p.n_out + feat0;
            }
#pragma unroll 1
            for (int g = 0; g < n_groups; ++g) {
                const int c0 = ((seq & 1) ? g : n_groups - 1 - g) << 4;  // first column of the group = its first tile row
                float v[16];
                tmem_load_16(lane_base + parts.first_col + c0, v);
                // the chunk goes back as soon as its columns have been read
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0)
                    mbar_arrive_cluster_relaxed(map_to_cta(bar_acc_empty + ((parts.first_col + c0) / kChunkCols) * 8, 0));
                if (SWIGLU) {
                    // lanes 0..15 hold gate, lanes 16..31 up of the same 16 features; h is quantised in blocks of 32
                    // features: this warp's 16 and its partner's (warps q and q ^ 1), maxima exchanged through amax_s
                    float hv[8];
                    uint32_t mag[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float other = __shfl_xor_sync(0xffffffffu, hi ? v[i] : v[8 + i], 16);
                        const float gt = hi ? other : v[i];
                        const float up = hi ? v[8 + i] : other;
                        hv[i] = swiglu(gt, up);
                        mag[i] = __float_as_uint(hv[i]) & 0x7FFFFFFFu;  // magnitudes compare as integers; NaN and inf on top
                    }
                    const uint32_t col_max = half_warp_max8(mag, j16);  // of column c0 + hi * 8 + j16 / 2, this warp's 16 features
                    buf ^= 1;
                    if ((j16 & 1) == 0) amax_s[(buf * 4 + q) * 16 + hi * 8 + (j16 >> 1)] = col_max;
                    pair_sync(q >> 1);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const uint32_t block_mag = max(amax_s[(buf * 4 + q) * 16 + hi * 8 + i],
                                                       amax_s[(buf * 4 + (q ^ 1)) * 16 + hi * 8 + i]);
                        const uint32_t sb = mx_scale_byte(block_mag);
                        const int col = c0 + hi * 8 + i;
                        if (col < t.n_valid) {
                            uint8_t code = 0x7F;
                            if (sb != 255u)
                                code = (uint8_t)__nv_cvt_float_to_fp8(hv[i] * __uint_as_float((254u - sb) << 23), __NV_SATFINITE,
                                                                      __NV_E4M3);
                            dst_q[(size_t)col * p.n_out] = code;
                            if ((q & 1) == 0 && j16 == 0)  // row `col` of the tile: atom col / 128, atom row col % 128
                                sf_dst[(size_t)(col >> 7) * kMxSfAtomBytes + mx_atom_byte(col & 127, 0)] = (uint8_t)sb;
                        }
                    }
                } else {
                    // Output rows are the token's: a lane holds one output feature of 16 tokens, and stored from here
                    // a warp instruction would write 32 x 2 bytes of one token -- measured, those stores took as long
                    // as the MMAs of a tile.  The four warps transpose the group through shared memory instead and
                    // each stores four whole 256-byte token rows, 16 bytes per lane.
                    out_flip ^= 1;  // (across tiles too: two consecutive groups never share a buffer)
                    uint8_t *stage_buf = base_ptr + L::kOutStage + out_flip * kOutStageBytes;
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        reinterpret_cast<__nv_bfloat16 *>(stage_buf)[i * kTileM + q * 32 + lane] = __float2bfloat16_rn(v[i]);
                    asm volatile("bar.sync 2, 128;" ::: "memory");  // (two buffers: the next group's writes cannot pass this)
#pragma unroll
                    for (int it = 0; it < 2; ++it) {
                        const int r = q * 4 + it * 2 + (lane >> 4);  // token of the group
                        const uint4 val = *reinterpret_cast<const uint4 *>(stage_buf + r * (kTileM * 2) + (lane & 15) * 16);
                        if (c0 + r < t.n_valid)
                            *reinterpret_cast<uint4 *>(dst_rows + (size_t)(c0 + r) * p.n_out + (lane & 15) * 8) = val;
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
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    tmem_release_pair(tmem_base, kTmemColsMx, warp);
}

template <int NT_MAX, int STAGES, bool SWIGLU>
int launch_mx_ring_instance(const MxRingMaps &maps, const MxParams &p, int grid, cudaStream_t stream) {
    using L = MxRingSmem<NT_MAX, STAGES, SWIGLU>;
    static_assert(L::kBytes + 1024 <= L::kDynamicBytes, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_mx_ring_kernel<NT_MAX, STAGES, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kMxRingThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace

bool grouped_gemm_tc_mx_ring_applies(const MxGemmArgs &a) {
    if (!(a.nt_max == 304 || a.nt_max == 384) || a.K % kMxSlotK != 0 || a.A <= 0) return false;
    return a.n_out % (a.swiglu ? kTileM : 2 * kTileM) == 0;
}

int launch_grouped_gemm_tc_mx_ring(const MxGemmArgs &a, cudaStream_t stream) {
    if (!grouped_gemm_tc_mx_ring_applies(a)) return MOE_ERR_UNSUPPORTED;
    const int atoms_per_tile = (a.nt_max + 127) / 128;
    const int cta_feat = a.swiglu ? kTileM / 2 : kTileM;
    MxRingMaps maps;
    const bool ok_w = a.swiglu ? encode_mx_weight_map_gate_up(&maps.ops.w, a.w_q, a.E, a.n_out, a.K)
                               : encode_mx_weight_map_2d(&maps.ops.w, a.w_q, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w || !encode_mx_act_maps(maps.ops.act, a.act_q, a.A, a.K, 8)) return MOE_ERR_CUDA;
    const uint64_t w_atoms = (uint64_t)a.E * (a.n_out / cta_feat) * (a.K / kMxSlotK);
    const uint64_t act_atoms = (uint64_t)(a.K / kMxSlotK) * a.n_atoms;
    if (!encode_mx_scale_map(&maps.w_sf, a.w_sf, w_atoms, 1) ||
        !encode_mx_scale_map(&maps.act_sf, a.act_sf, act_atoms, (uint32_t)atoms_per_tile))
        return MOE_ERR_CUDA;

    MxParams p;
    p.out = a.out;
    p.out_sf = a.out_sf;
    p.w_sf = a.w_sf;
    p.act_sf = a.act_sf;
    p.expert_offsets = a.expert_offsets;
    p.tile_prefix = a.tile_prefix;
    p.tile_order = a.tile_order;
    p.tile_rows = a.tile_rows;
    p.status = a.status;
    p.E = a.E;
    p.n_k_blocks = a.K / kMxSlotK;
    p.n_out = a.n_out;
    p.w_rows = a.w_rows;
    p.n_feature_tiles = a.n_out / (2 * cta_feat);
    p.n_atoms = a.n_atoms;
    p.tile_stride = mx_sf_stride(a.nt_max);
    p.atoms_per_tile = atoms_per_tile;
    p.handover_role = a.handover_role;
    p.handover = a.handover;
    p.handover_per_token_tile = a.handover_per_token_tile;

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / 256;  // (experts above the bound: tiles of up to 256 rows)
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int pairs_on_device = sm_count() / 2;
    const int n_pairs = (int)(max_tiles < pairs_on_device ? max_tiles : pairs_on_device);
    const int grid = 2 * (n_pairs > 0 ? n_pairs : 1);
    if (a.nt_max == 304)  // (the gate/up kernel has no output staging buffer: room for a sixth ring slot)
        return a.swiglu ? launch_mx_ring_instance<304, 6, true>(maps, p, grid, stream)
                        : launch_mx_ring_instance<304, 5, false>(maps, p, grid, stream);
    return a.swiglu ? launch_mx_ring_instance<384, 5, true>(maps, p, grid, stream)
                    : launch_mx_ring_instance<384, 5, false>(maps, p, grid, stream);
}

}  // namespace moe

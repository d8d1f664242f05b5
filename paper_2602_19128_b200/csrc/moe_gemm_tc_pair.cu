// Grouped expert GEMMs on CTA pairs: tcgen05.mma.cta_group::2, a 256 x N or 512 x N tile per pair.
//
// Same role split, ring and tile schedule as the one-CTA kernel (moe_gemm_tc.cu; paper Sec. 4.5
// "Expert FFN computation" for what is computed), but two CTAs of a cluster work on one tile:
// each CTA stages its own 128 weight rows and only HALF of the token tile (N/2 rows), and the
// pair's MMA reads both halves.  Per useful flop the SMs pull (1/N + 1/256) bytes from L2 instead
// of (1/N + 1/128), which is what bounds the prefill-sized workloads; no load is multicast, every
// CTA fetches what it stages.
//
// Protocol (rank 0 = leader):
//   full[s]      lives in the leader.  The leader's producer arms it with the bytes of BOTH CTAs;
//                both producers' TMA copies (cta_group::2 form) complete on it.
//   empty[s]     one per CTA.  The leader's MMA thread commits ring slots back with a commit that
//                arrives on the barrier of both CTAs.
//   acc_full[a]  one per CTA, same commit form; each CTA's epilogue warps drain their own TMEM
//                (128 weight rows x N tokens) and arrive on the LEADER's acc_empty[a] (8 arrivals).
// Before leaving, each producer waits until every ring slot has been handed back and the leader
// waits for both accumulators to be released, so no arrival can reach a CTA that has exited; a
// cluster barrier then precedes the TMEM release.  Every wait is bounded as in the one-CTA kernel.
//
// SLABS = 2 gives each CTA two 128-row weight slabs per ring slot that share one token tile (two MMAs
// per K step, two accumulators): (1/N + 1/512) bytes per flop through the copy engine, which keeps
// the tensor pipe busy for token tiles well below 256 rows.  The two accumulators fill TMEM
// (2 x 256 columns), so the epilogue is not overlapped with the next tile's MMAs; measured slower than
// one slab on every benchmark workload, it is opt-in (MOE_FLAG_TWO_SLAB_GEMM) and kept for shapes
// with much longer K.
#include "moe_tc_pair.cuh"

namespace moe {
namespace {

using namespace tc;

constexpr int kPairThreads = 224;  // warp 0 weight TMA, warp 1 MMA, warps 2..5 epilogue, warp 6 token TMA

// D[tmem of both CTAs] (+)= A * B^T over the pair: M = 256 (128 rows per CTA), B halves from both CTAs.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
template <int NT_MAX, int STAGES, int SLABS>
struct PairSmem {
    static constexpr int kSlotABytesAll = SLABS * kSlotABytes;
    static constexpr int kSlotBBytes = (NT_MAX / 2) * kRowBytes;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kSlotABytesAll;
    static constexpr int kBars = kB + STAGES * kSlotBBytes;  // full[S], empty[S], acc_full[2], acc_empty[2]
    static constexpr int kTmemSlot = kBars + (2 * STAGES + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kPairDynamicSmemBytes;  // (kBytes + 1024 of it are used)
};

// Drain one accumulator (this warp's 32 TMEM lanes x n_mma columns) to global memory.
//   SWIGLU: lanes 0..15 hold gate, lanes 16..31 up of the same 16 features; dst points at this lane's
//           feature in row 0 of the tile.  Plain: one output feature per lane.
template <bool SWIGLU>
__device__ __forceinline__ void drain_accumulator(uint32_t taddr, int n_mma, int n_valid, __nv_bfloat16 *dst,
                                                  size_t row_stride, int lane) {
    if (SWIGLU) {
        const int hi = lane >> 4;
        for (int c0 = 0; c0 < n_mma; c0 += 16) {
            float v[16];
            tmem_load_16(taddr + c0, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float other = __shfl_xor_sync(0xffffffffu, hi ? v[i] : v[8 + i], 16);
                const float g = hi ? other : v[i];
                const float u = hi ? v[8 + i] : other;
                const int col = c0 + hi * 8 + i;
                if (col < n_valid) dst[(size_t)col * row_stride] = __float2bfloat16_rn(swiglu(g, u));
            }
        }
    } else {
        for (int c0 = 0; c0 < n_mma; c0 += 16) {
            float v[16];
            tmem_load_16(taddr + c0, v);
#pragma unroll
            for (int i = 0; i < 16; ++i)
                if (c0 + i < n_valid) dst[(size_t)(c0 + i) * row_stride] = __float2bfloat16_rn(v[i]);
        }
    }
}

template <int NT_MAX, int STAGES, int SLABS, bool SWIGLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
grouped_gemm_tc_pair_kernel(const __grid_constant__ TensorMaps maps, const KernelParams p) {
    using L = PairSmem<NT_MAX, STAGES, SLABS>;
    constexpr int kAccBufs = SLABS == 1 ? 2 : 1;          // accumulator sets in TMEM
    // accumulator columns (2 * NT_MAX either way), rounded up to the power of two an allocation must be
    constexpr int kAccCols = SLABS * kAccBufs * NT_MAX;
    constexpr int kTmemCols = kAccCols <= 32 ? 32 : kAccCols <= 64 ? 64 : kAccCols <= 128 ? 128 : kAccCols <= 256 ? 256 : 512;
    static_assert(kAccCols <= 512, "accumulators exceed tensor memory");
    static_assert((kTmemCols & (kTmemCols - 1)) == 0, "a tensor-memory allocation must be a power of two");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;           // the down GEMM reports sites 5..8
    // weight rows (plain) resp. h features (SwiGLU) covered by one pair tile, one slab of it, one CTA of a slab
    constexpr int kFeatPerCta = SWIGLU ? kTileM / 2 : kTileM;
    constexpr int kFeatPerSlab = 2 * kFeatPerCta;
    constexpr int kFeatPerTile = SLABS * kFeatPerSlab;
    chain_release();  // the next kernel of the forward call may be scheduled; it waits for this grid to finish
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBars, bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + STAGES * 8, bar_acc_empty = bar_acc_full + 16;
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
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_acc_full + a * 8, 1);
            mbar_init(bar_acc_empty + a * 8, 2 * kEpilogueWarps);
        }
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

    // ---------------- TMA producers (both CTAs) ----------------
    // The weight slabs and the token rows of a slot are issued by two different warps: a copy
    // instruction occupies its issuing thread for a while, and two issuers keep the ring ahead.
    auto producer_loop = [&](const bool load_w, const bool load_act) {  // run by a whole warp
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15, half = n_mma >> 1;  // each CTA stages half: a multiple of 8 rows
            const int feat0 = t.f * kFeatPerTile + (int)rank * kFeatPerCta;  // this CTA's part of slab 0
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
                    const int k0 = kb * kBlockK;
                    if (load_w) {
                        if (rank == 0) mbar_expect_tx(bar_full + stage * 8, 2 * L::kSlotABytesAll + n_mma * kRowBytes);
#pragma unroll
                        for (int s = 0; s < SLABS; ++s) {
                            const uint32_t sa = base + L::kA + stage * L::kSlotABytesAll + s * kSlotABytes;
                            const int feat = feat0 + s * kFeatPerSlab;
                            if (SWIGLU)  // 64 features = 4 groups of 16, gate and up rows interleaved per group
                                tma_load_5d_pair(sa, &maps.w, k0, 0, 0, feat >> 4, t.e, full);
                            else
                                tma_load_2d_pair(sa, &maps.w, k0, t.e * p.w_rows + feat, full);
                        }
                    }
                    if (load_act) {
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                        tma_load_2d_pair(sb, act_map<8>(maps, half), k0, t.row0 + (int)rank * half, full);
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
    } else if (warp == kPairThreads / 32 - 1) {
        producer_loop(false, true);
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only): the warp walks the ring, one elected lane issues ----------------
        if (rank == 0) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int round = 0; ok; ++round) {
                const int tile = tile_of_round(round, pair, n_pairs);
                if (tile >= total_tiles) break;
                const Tile t = decode_tile(tile, p);
                const uint32_t idesc = instr_desc_bf16(2 * kTileM, (t.n_valid + 15) & ~15);
                ok = __all_sync(0xffffffffu, pair_wait(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, peer_abort,
                                                       p.status, kSiteMmaTmemEmpty + kSiteOffset));
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + acc * SLABS * NT_MAX;
                for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, pair_wait(bar_full + stage * 8, phase, abort_flag, peer_abort, p.status,
                                                           kSiteMmaFull + kSiteOffset));
                    if (!ok) break;
                    tcgen05_fence_after();
                    if (elect_one()) {
                        const uint64_t b_desc = smem_desc_k_major_sw128(base + L::kB + stage * L::kSlotBBytes);
#pragma unroll
                        for (int s = 0; s < SLABS; ++s) {
                            const uint64_t a_desc =
                                smem_desc_k_major_sw128(base + L::kA + stage * L::kSlotABytesAll + s * kSlotABytes);
#pragma unroll
                            for (int kk = 0; kk < kBlockK / 16; ++kk)  // 16 K-elements = 32 bytes = 2 descriptor units
                                umma_bf16_pair(d_tmem + s * NT_MAX, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
                        }
                        umma_commit_pair(bar_empty + stage * 8);
                        if (kb == p.n_k_blocks - 1) umma_commit_pair(bar_acc_full + acc * 8);
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
            }
            // wait until every accumulator set has been released by both CTAs' epilogues
            for (int a = 0; ok && a < kAccBufs; ++a) {
                ok = __all_sync(0xffffffffu, pair_wait(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, peer_abort,
                                                       p.status, kSiteMmaTmemEmpty + kSiteOffset));
                if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue (both CTAs): own 128 weight rows per slab x all N tokens ----------------
        const int q = warp & 3;  // a warp may only read TMEM lanes 32*(warp%4) .. +31
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            ok = pair_wait(bar_acc_full + acc * 8, acc_phase, abort_flag, peer_abort, p.status, kSiteEpilogueTmemFull + kSiteOffset);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tcgen05_fence_after();
            const int lane_feat = SWIGLU ? q * 16 + (lane & 15) : q * 32 + lane;
#pragma unroll
            for (int s = 0; s < SLABS; ++s) {
                const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (acc * SLABS + s) * NT_MAX;
                __nv_bfloat16 *dst = p.out + (size_t)t.row0 * p.n_out + t.f * kFeatPerTile + s * kFeatPerSlab +
                                     (int)rank * kFeatPerCta + lane_feat;
                drain_accumulator<SWIGLU>(taddr, n_mma, t.n_valid, dst, (size_t)p.n_out, lane);
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(bar_acc_empty + acc * 8, 0));
            handover_count_tile(p.handover_role, p.handover, t.e, lane);  // (after the accumulator is handed back)
            if (++acc == kAccBufs) { acc = 0; acc_phase ^= 1u; }
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

template <int NT_MAX, int STAGES, int SLABS, bool SWIGLU>
int launch_pair_instance(const TensorMaps &maps, const KernelParams &p, int grid, cudaStream_t stream) {
    using L = PairSmem<NT_MAX, STAGES, SLABS>;
    static_assert(L::kBytes + 1024 <= L::kDynamicBytes, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_pair_kernel<NT_MAX, STAGES, SLABS, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kPairThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int features_per_pair_tile(const GroupedGemmArgs &a, int slabs) { return slabs * (a.swiglu ? kTileM : 2 * kTileM); }

}  // namespace

// Largest number of weight slabs per CTA (2, 1) the pair kernel supports for this GEMM, 0 if none.
int grouped_gemm_tc_pair_slabs(const GroupedGemmArgs &a) {
    if (!(a.nt_max == 128 || a.nt_max == 256) || a.K % kBlockK != 0 || a.A <= 0) return 0;
    if (a.nt_max == 256 && a.n_out % features_per_pair_tile(a, 2) == 0) return 2;
    return a.n_out % features_per_pair_tile(a, 1) == 0 ? 1 : 0;
}

int launch_grouped_gemm_tc_pair(const GroupedGemmArgs &a, int slabs, cudaStream_t stream) {
    const int max_slabs = grouped_gemm_tc_pair_slabs(a);
    if (slabs < 1 || slabs > max_slabs) return MOE_ERR_UNSUPPORTED;
    TensorMaps maps;
    const bool ok_w = a.swiglu ? encode_weight_map_gate_up(&maps.w, a.w, a.E, a.n_out, a.K)
                               : encode_weight_map_2d(&maps.w, a.w, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w || !encode_act_maps(maps.act, a.act, a.A, a.K, 8)) return MOE_ERR_CUDA;

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
    p.handover_role = slabs == 1 ? a.handover_role : 0;  // (the two-slab tile counts differently; the caller does not combine them)
    p.handover = a.handover;
    p.handover_per_token_tile = a.handover_per_token_tile;
    p.n_feature_tiles = a.n_out / features_per_pair_tile(a, slabs);

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / a.nt_max;
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int pairs_on_device = sm_count() / 2;
    const int n_pairs = (int)(max_tiles < pairs_on_device ? max_tiles : pairs_on_device);
    const int grid = 2 * (n_pairs > 0 ? n_pairs : 1);
    if (slabs == 2)
        return a.swiglu ? launch_pair_instance<256, 4, 2, true>(maps, p, grid, stream)
                        : launch_pair_instance<256, 4, 2, false>(maps, p, grid, stream);
    if (a.nt_max == 256)
        return a.swiglu ? launch_pair_instance<256, 7, 1, true>(maps, p, grid, stream)
                        : launch_pair_instance<256, 7, 1, false>(maps, p, grid, stream);
    return a.swiglu ? launch_pair_instance<128, 9, 1, true>(maps, p, grid, stream)
                    : launch_pair_instance<128, 9, 1, false>(maps, p, grid, stream);
}

}  // namespace moe

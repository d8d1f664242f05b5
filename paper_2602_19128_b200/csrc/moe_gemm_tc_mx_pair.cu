// Grouped expert GEMMs in MX FP8 on CTA pairs: tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale, a
// 256 x N tile per pair with N up to 240 token rows.
//
// What is computed: paper Sec. 4.5 "Expert FFN computation" (gate/up with SiLU, then down), on the FP8
// workload of Table 2, with the MX operands described in moe_gemm_tc_mx.cu.  Why pairs: at 8 bits the
// tensor core needs half the time per K-slot, so the one-CTA kernel is bound by the bytes an SM pulls
// from L2 per slot.  Here each CTA stages its own 128 weight rows and only HALF of the token tile, and
// one token tile may be 240 rows, so a weight byte is fetched once per 240 tokens and a token byte once
// per 256 weight rows.
//
// Protocol: as the bf16 pair kernel (leader = cluster rank 0 owns full[s] and issues every MMA; commits
// arrive on both CTAs' barriers; epilogues of both CTAs release the accumulator on the leader).  Added:
//   * Scale atoms travel by TMA tensor copies (cta_group::2 form, completing on the leader's barrier):
//     each CTA loads the atom of its own 128 weight rows and ALL atoms of the token tile -- the MMA reads
//     the token scales of every column from the tensor memory of the CTA whose rows it computes.
//   * Before a slot's MMAs the leader issues tcgen05.cp.cta_group::2, which copies, in both CTAs, the
//     atoms from that CTA's shared memory to its tensor memory.
//   * Tensor memory per CTA: two accumulators of NT_MAX columns, 4 columns of weight scales, 4 columns
//     per token atom.  2 * 240 + 32 = 512 is why the largest tile is 240 rows and not 256.
// Every wait is bounded; on expiry both CTAs are told, every role stops and tensor memory is released.
#include "moe_mx_tc.cuh"
#include "moe_tc_pair.cuh"

namespace moe {
namespace {

using namespace tc;
using namespace mxtc;

constexpr int kPairThreads = 224;  // warp 0 weight TMA, warp 1 MMA, warps 2..5 epilogue, warp 6 token TMA

struct MxPairMaps {
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
template <int NT_MAX, int STAGES>
struct MxPairSmem {
    static constexpr int kAtomsB = (NT_MAX + 127) / 128;
    static constexpr int kSlotBBytes = (NT_MAX / 2) * kMxSlotK;
    static constexpr int kSfBBytes = kAtomsB * kMxSfAtomBytes;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kMxSlotABytes;
    static constexpr int kSfA = kB + STAGES * kSlotBBytes;
    static constexpr int kSfB = kSfA + STAGES * kMxSfAtomBytes;
    static constexpr int kAmax = kSfB + STAGES * kSfBBytes;
    static constexpr int kBars = kAmax + 2 * 4 * 16 * 4;  // full[S], empty[S], acc_full[2], acc_empty[2]
    static constexpr int kTmemSlot = kBars + (2 * STAGES + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kPairDynamicSmemBytes;  // (kBytes + 1024 of it are used)
};

template <int NT_MAX, int STAGES, bool SWIGLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
grouped_gemm_tc_mx_pair_kernel(const __grid_constant__ MxPairMaps maps, const MxParams p) {
    using L = MxPairSmem<NT_MAX, STAGES>;
    static_assert(2 * NT_MAX + 16 + 4 * L::kAtomsB <= kTmemColsMx, "accumulators and scale columns exceed tensor memory");
    static_assert(NT_MAX % 16 == 0 && (NT_MAX / 2) % 8 == 0, "token tile halves must be whole 8-row swizzle groups");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;
    constexpr uint32_t kSfACol = 2 * NT_MAX, kSfBCol = 2 * NT_MAX + 16;
    constexpr int kFeatPerCta = SWIGLU ? kTileM / 2 : kTileM;  // h features resp. output rows per CTA of a pair tile
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
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15, half = n_mma >> 1;
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
                        if (rank == 0)
                            mbar_expect_tx(bar_full + stage * 8,
                                           2 * (kMxSlotABytes + kMxSfAtomBytes + L::kSfBBytes) + n_mma * kMxSlotK);
                        const uint32_t sa = base + L::kA + stage * kMxSlotABytes;
                        if (SWIGLU)  // 64 features = 4 groups of 16, gate and up rows interleaved per group
                            tma_load_5d_pair(sa, &maps.ops.w, k0, 0, 0, cta_tile * 4, t.e, full);
                        else
                            tma_load_2d_pair(sa, &maps.ops.w, k0, t.e * p.w_rows + cta_tile * kTileM, full);
                        tma_load_2d_pair(base + L::kSfA + stage * kMxSfAtomBytes, &maps.w_sf, 0, w_sf_row + kb, full);
                    }
                    if (load_act) {
                        const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                        tma_load_2d_pair(sb, act_map<8>(maps.ops, half), k0, t.row0 + (int)rank * half, full);
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
    } else if (warp == kPairThreads / 32 - 1) {
        producer_loop(false, true);
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (rank == 0) {
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            const uint32_t sfa_tmem = tmem_base + kSfACol, sfb_tmem = tmem_base + kSfBCol;
            for (int round = 0; ok; ++round) {
                const int tile = tile_of_round(round, pair, n_pairs);
                if (tile >= total_tiles) break;
                const MxTile t = decode_mx_tile(tile, p);
                const int n_mma = (t.n_valid + 15) & ~15;
                ok = __all_sync(0xffffffffu, pair_wait(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, peer_abort,
                                                       p.status, kSiteMmaTmemEmpty + kSiteOffset));
                if (!ok) break;
                tcgen05_fence_after();
                const uint32_t d_tmem = tmem_base + acc * NT_MAX;
                for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                    ok = __all_sync(0xffffffffu, pair_wait(bar_full + stage * 8, phase, abort_flag, peer_abort, p.status,
                                                           kSiteMmaFull + kSiteOffset));
                    if (!ok) break;
                    tcgen05_fence_after();
                    if (elect_one()) {
                        tmem_copy_sf_atom_pair(sfa_tmem, smem_desc_sf_atom(base + L::kSfA + stage * kMxSfAtomBytes));
#pragma unroll
                        for (int a = 0; a < L::kAtomsB; ++a)
                            tmem_copy_sf_atom_pair(sfb_tmem + 4 * a,
                                                   smem_desc_sf_atom(base + L::kSfB + stage * L::kSfBBytes + a * kMxSfAtomBytes));
                        const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kA + stage * kMxSlotABytes);
                        const uint64_t b_desc = smem_desc_k_major_sw128(base + L::kB + stage * L::kSlotBBytes);
#pragma unroll
                        for (int kk = 0; kk < kMxSlotK / 32; ++kk)
                            umma_mx_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, instr_desc_mx(2 * kTileM, n_mma, kk),
                                         (kb | kk) != 0, sfa_tmem, sfb_tmem);
                        umma_commit_pair(bar_empty + stage * 8);
                        if (kb == p.n_k_blocks - 1) umma_commit_pair(bar_acc_full + acc * 8);
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            // wait until both accumulators have been released by both CTAs' epilogues
            for (int a = 0; ok && a < 2; ++a) {
                ok = __all_sync(0xffffffffu, pair_wait(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, peer_abort,
                                                       p.status, kSiteMmaTmemEmpty + kSiteOffset));
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue (both CTAs): own 128 weight rows x all N tokens ----------------
        const int q = warp & 3;
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t *amax_s = reinterpret_cast<uint32_t *>(base_ptr + L::kAmax);
        int buf = 0;
        for (int round = 0;; ++round) {
            const int tile = tile_of_round(round, pair, n_pairs);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const bool ok = pair_wait(bar_acc_full + acc * 8, acc_phase, abort_flag, peer_abort, p.status,
                                      kSiteEpilogueTmemFull + kSiteOffset);
            if (epilogue_any(!ok)) break;  // the four warps synchronise inside the tile, so they leave together
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * NT_MAX;
            const int feat0 = (2 * t.f + (int)rank) * kFeatPerCta;  // first feature / output row of this CTA
            if (SWIGLU) {
                uint8_t *dst = static_cast<uint8_t *>(p.out) + (size_t)t.row0 * p.n_out + feat0 + q * 16 + (lane & 15);
                const int block = (feat0 + q * 16) >> 5;  // 32-feature block = scale byte `block % 4` of K-slot `block / 4`
                uint8_t *sf_dst = p.out_sf + ((size_t)(block >> 2) * p.n_atoms + t.atom) * kMxSfAtomBytes + (block & 3);
                drain_swiglu_mx(taddr, n_mma, t.n_valid, dst, (size_t)p.n_out, sf_dst, amax_s, buf, q, lane);
            } else {
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) + (size_t)t.row0 * p.n_out + feat0 + q * 32 + lane;
                for (int c0 = 0; c0 < n_mma; c0 += 16) {
                    float v[16];
                    tmem_load_16(taddr + c0, v);
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (c0 + i < t.n_valid) dst[(size_t)(c0 + i) * p.n_out] = __float2bfloat16_rn(v[i]);
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(bar_acc_empty + acc * 8, 0));
            handover_count_tile(p.handover_role, p.handover, t.e, lane);  // (after the accumulator is handed back)
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
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
int launch_pair_instance(const MxPairMaps &maps, const MxParams &p, int grid, cudaStream_t stream) {
    using L = MxPairSmem<NT_MAX, STAGES>;
    static_assert(L::kBytes + 1024 <= L::kDynamicBytes, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_mx_pair_kernel<NT_MAX, STAGES, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kPairThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // namespace

bool grouped_gemm_tc_mx_pair_applies(const MxGemmArgs &a) {
    if (!(a.nt_max == 128 || a.nt_max == 160 || a.nt_max == 240) || a.K % kMxSlotK != 0 || a.A <= 0) return false;
    return a.n_out % (a.swiglu ? kTileM : 2 * kTileM) == 0;
}

int launch_grouped_gemm_tc_mx_pair(const MxGemmArgs &a, cudaStream_t stream) {
    if (!grouped_gemm_tc_mx_pair_applies(a)) return MOE_ERR_UNSUPPORTED;
    const int atoms_per_tile = (a.nt_max + 127) / 128;
    const int cta_feat = a.swiglu ? kTileM / 2 : kTileM;
    MxPairMaps maps;
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

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / a.nt_max;
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int pairs_on_device = sm_count() / 2;
    const int n_pairs = (int)(max_tiles < pairs_on_device ? max_tiles : pairs_on_device);
    const int grid = 2 * (n_pairs > 0 ? n_pairs : 1);
    if (a.nt_max == 240)
        return a.swiglu ? launch_pair_instance<240, 6, true>(maps, p, grid, stream)
                        : launch_pair_instance<240, 6, false>(maps, p, grid, stream);
    if (a.nt_max == 160)  // a smaller token slot buys two more ring slots: more weight bytes in flight per SM
        return a.swiglu ? launch_pair_instance<160, 8, true>(maps, p, grid, stream)
                        : launch_pair_instance<160, 8, false>(maps, p, grid, stream);
    return a.swiglu ? launch_pair_instance<128, 8, true>(maps, p, grid, stream)
                    : launch_pair_instance<128, 8, false>(maps, p, grid, stream);
}

}  // namespace moe

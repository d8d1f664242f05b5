// Grouped expert GEMMs in MX FP8 on the Blackwell tensor cores: tcgen05.mma kind::mxf8f6f4.block_scale.
// Both operands are E4M3 codes with one E8M0 scale byte per 32 K-elements; the tensor core applies the
// scales itself, reading them from tensor memory, so nothing is dequantised in software and the weights
// cross HBM at one byte each.
//
// Paper, Sec. 4.5 ("Expert FFN computation"; the workload is the FP8 MoE of Table 2): gate and up
// projections combined through SiLU, then the down projection, over expert-contiguous token rows.  The
// paper's kernel converted FP8 tiles for 16-bit WMMA; on sm_100a the 8-bit block-scaled MMA does that
// work.  Structure as in the bf16 kernel (weights on the M side, tokens on the N side, persistent CTAs on
// a device-built schedule, warp 0 TMA, warp 1 MMA, warps 2..5 epilogue, double-buffered accumulators),
// plus:
//
//  * A ring slot is 128 K-elements: 16 KiB of weight codes, the token codes, the 512-byte atom of weight
//    scale bytes (4 per row) and the token tile's own atom of scale bytes (every tile of the MX schedule
//    starts a fresh atom).  Four copies per slot, all completing on the slot's mbarrier.
//  * Before a slot's four K=32 MMAs the issuing lane copies the slot's scale atoms from shared to tensor
//    memory (tcgen05.cp 32x128b.warpx4: 32 rows x 16 bytes, replicated to the four lane quadrants).  Row
//    r of an atom then sits in lane r % 32, column r / 32, byte = the K-block within the slot, which the
//    instruction descriptor selects (a_sf_id / b_sf_id).  Copies and MMAs execute in issue order, so the
//    next slot's copies may overwrite the columns without a wait.
//  * The gate/up epilogue quantises h itself: after SiLU(gate)*up a warp holds 16 features x 16 tokens;
//    the largest magnitude over a block of 32 features comes from a 16-lane shuffle reduction and one
//    exchange with the neighbouring warp through shared memory, then each lane scales and encodes its
//    values and the scale byte goes straight into the atom layout the down GEMM loads.
#include "moe_mx_tc.cuh"

namespace moe {
namespace {

using namespace tc;
using namespace mxtc;

constexpr int kMxSfBBytes = kMxSfAtomBytes;            // one atom per token tile (at most 128 rows)

__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tmem_copy_sf_atom(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
__device__ __forceinline__ void umma_mx(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate, uint32_t sfa_tmem, uint32_t sfb_tmem) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int NT_MAX, int STAGES>
struct MxSmem {
    static constexpr int kSlotBBytes = NT_MAX * kMxSlotK;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kMxSlotABytes;
    static constexpr int kSfA = kB + STAGES * kSlotBBytes;
    static constexpr int kSfB = kSfA + STAGES * kMxSfAtomBytes;
    static constexpr int kAmax = kSfB + STAGES * kMxSfBBytes;     // [2 buffers][4 warps][16 tokens] magnitudes
    static constexpr int kBars = kAmax + 2 * 4 * 16 * 4;          // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
    static constexpr int kTmemSlot = kBars + (2 * STAGES + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kBytes + 1024;
};

template <int NT_MAX, int STAGES, bool SWIGLU>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_tc_mx_kernel(const __grid_constant__ TensorMaps maps, const MxParams p) {
    using L = MxSmem<NT_MAX, STAGES>;
    static_assert(2 * NT_MAX + 32 <= kTmemColsMx, "accumulators and scale columns exceed tensor memory");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;
    constexpr uint32_t kSfACol = 2 * NT_MAX, kSfBCol = 2 * NT_MAX + 16;
    chain_release();  // the next kernel of the forward call may be scheduled; it waits for this grid to finish
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full = base + L::kBars, bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + STAGES * 8, bar_acc_empty = bar_acc_full + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_full + s * 8, 1);
            mbar_init(bar_empty + s * 8, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_acc_full + a * 8, 1);
            mbar_init(bar_acc_empty + a * 8, kEpilogueWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + L::kTmemSlot),
                     "r"(kTmemColsMx)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above overlapped the previous kernel; its results are read from here on
    const bool started = gemm_chain_start(p.handover_role, p.handover, abort_flag, p.status);
    const int total_tiles = started ? p.tile_prefix[p.E] * p.n_feature_tiles : 0;

    if (warp == 0) {
        // ---------------- producer: codes by TMA, scale atoms by bulk copies ----------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const int w_row = t.e * p.w_rows + t.f * kTileM;
            const uint32_t tx_bytes = kMxSlotABytes + n_mma * kMxSlotK + kMxSfAtomBytes + kMxSfBBytes;
            const uint8_t *w_sf = p.w_sf + ((size_t)t.e * p.n_feature_tiles + t.f) * p.n_k_blocks * kMxSfAtomBytes;
            const uint8_t *a_sf = p.act_sf + (size_t)t.atom * kMxSfAtomBytes;
            ok = handover_wait_expert(p.handover_role, p.handover, t.e, t.n_tok_tiles, p.handover_per_token_tile,
                                      p.tile_prefix[p.E], gate_up_done, abort_flag, p.status, lane);
            if (!ok) break;
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = mbar_wait_warp(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status, kSiteProducerEmpty + kSiteOffset);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = bar_full + stage * 8;
                    mbar_expect_tx(full, tx_bytes);
                    const uint32_t sa = base + L::kA + stage * kMxSlotABytes;
                    const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                    const int k0 = kb * kMxSlotK;
                    if (SWIGLU)
                        tma_load_5d(sa, &maps.w, k0, 0, 0, t.f * 4, t.e, full);
                    else
                        tma_load_2d(sa, &maps.w, k0, w_row, full);
                    tma_load_2d(sb, act_map<16>(maps, n_mma), k0, t.row0, full);
                    bulk_load(base + L::kSfA + stage * kMxSfAtomBytes, w_sf + (size_t)kb * kMxSfAtomBytes, kMxSfAtomBytes, full);
                    bulk_load(base + L::kSfB + stage * kMxSfBBytes, a_sf + (size_t)kb * p.n_atoms * kMxSfAtomBytes,
                              kMxSfBBytes, full);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        const uint32_t sfa_tmem = tmem_base + kSfACol, sfb_tmem = tmem_base + kSfBCol;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            ok = mbar_wait_warp(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, p.status, kSiteMmaTmemEmpty + kSiteOffset);
            if (!ok) break;
            tcgen05_fence_after();
            const uint32_t d_tmem = tmem_base + acc * NT_MAX;
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = mbar_wait_warp(bar_full + stage * 8, phase, abort_flag, p.status, kSiteMmaFull + kSiteOffset);
                if (!ok) break;
                tcgen05_fence_after();
                if (elect_one()) {
                    const uint32_t sfa_smem = base + L::kSfA + stage * kMxSfAtomBytes;
                    const uint32_t sfb_smem = base + L::kSfB + stage * kMxSfBBytes;
                    tmem_copy_sf_atom(sfa_tmem, smem_desc_sf_atom(sfa_smem));
                    tmem_copy_sf_atom(sfb_tmem, smem_desc_sf_atom(sfb_smem));
                    const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kA + stage * kMxSlotABytes);
                    const uint64_t b_desc = smem_desc_k_major_sw128(base + L::kB + stage * L::kSlotBBytes);
#pragma unroll
                    for (int kk = 0; kk < kMxSlotK / 32; ++kk)  // 32 K-elements = 32 bytes = 2 descriptor units
                        umma_mx(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, instr_desc_mx(kTileM, n_mma, kk), (kb | kk) != 0,
                                sfa_tmem, sfb_tmem);
                    umma_commit(bar_empty + stage * 8);
                    if (kb == p.n_k_blocks - 1) umma_commit(bar_acc_full + acc * 8);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;  // a warp may only read TMEM lanes 32*(warp%4) .. +31
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t *amax_s = reinterpret_cast<uint32_t *>(base_ptr + L::kAmax);
        int buf = 0;  // exchange buffer, flipped every 16-token chunk (across tiles too): a warp may run one chunk ahead of its partner
        for (int round = 0;; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const MxTile t = decode_mx_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const bool ok = mbar_wait(bar_acc_full + acc * 8, acc_phase, abort_flag, p.status, kSiteEpilogueTmemFull + kSiteOffset);
            // the four warps synchronise inside the tile (SwiGLU), so they must agree on leaving
            if (epilogue_any(!ok)) break;
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * NT_MAX;
            if (SWIGLU) {
                uint8_t *dst = static_cast<uint8_t *>(p.out) + (size_t)t.row0 * p.n_out + t.f * (kTileM / 2) + q * 16 + (lane & 15);
                // scale bytes of h: features 64f + 16q.. lie in block 2f + q/2 = K-slot block/4 of the down GEMM
                const int block = 2 * t.f + (q >> 1);
                uint8_t *sf_dst = p.out_sf + ((size_t)(block >> 2) * p.n_atoms + t.atom) * kMxSfAtomBytes + (block & 3);
                drain_swiglu_mx(taddr, n_mma, t.n_valid, dst, (size_t)p.n_out, sf_dst, amax_s, buf, q, lane);
            } else {
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.out) + (size_t)t.row0 * p.n_out + t.f * kTileM + q * 32 + lane;
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
            if (lane == 0) mbar_arrive(bar_acc_empty + acc * 8);
            handover_count_tile(p.handover_role, p.handover, t.e, lane);  // (after the accumulator is handed back)
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // ---------------- teardown ----------------
    gemm_chain_finish(p.handover_role);
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemColsMx) : "memory");
    }
}

template <int NT_MAX, int STAGES, bool SWIGLU>
int launch_instance(const TensorMaps &maps, const MxParams &p, int grid, cudaStream_t stream) {
    using L = MxSmem<NT_MAX, STAGES>;
    static_assert(L::kDynamicBytes <= 232448, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_mx_kernel<NT_MAX, STAGES, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

template <bool SWIGLU>
int dispatch(int nt_max, const TensorMaps &maps, const MxParams &p, int grid, cudaStream_t s) {
    switch (nt_max) {
        case 32: return launch_instance<32, 10, SWIGLU>(maps, p, grid, s);
        case 64: return launch_instance<64, 8, SWIGLU>(maps, p, grid, s);
        case 128: return launch_instance<128, 6, SWIGLU>(maps, p, grid, s);
        default: return MOE_ERR_UNSUPPORTED;
    }
}

}  // namespace

int launch_grouped_gemm_tc_mx(const MxGemmArgs &a, cudaStream_t stream) {
    if (a.K % kMxSlotK != 0 || a.A <= 0 || a.nt_max > 128) return MOE_ERR_UNSUPPORTED;
    const int features_per_tile = a.swiglu ? kTileM / 2 : kTileM;
    if (a.n_out % features_per_tile != 0) return MOE_ERR_UNSUPPORTED;
    if (a.swiglu && a.n_out % 128 != 0) return MOE_ERR_UNSUPPORTED;  // h is the next GEMM's K

    TensorMaps maps;
    const bool ok_w = a.swiglu ? encode_mx_weight_map_gate_up(&maps.w, a.w_q, a.E, a.n_out, a.K)
                               : encode_mx_weight_map_2d(&maps.w, a.w_q, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w || !encode_mx_act_maps(maps.act, a.act_q, a.A, a.K, 16)) return MOE_ERR_CUDA;

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
    p.n_feature_tiles = a.n_out / features_per_tile;
    p.n_atoms = a.n_atoms;
    p.tile_stride = mx_sf_stride(a.nt_max);
    p.atoms_per_tile = 1;
    p.handover_role = a.handover_role;
    p.handover = a.handover;
    p.handover_per_token_tile = a.handover_per_token_tile;

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / a.nt_max;
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int sms = sm_count();
    const int grid = (int)(max_tiles < sms ? max_tiles : sms);
    return a.swiglu ? dispatch<true>(a.nt_max, maps, p, grid, stream) : dispatch<false>(a.nt_max, maps, p, grid, stream);
}

}  // namespace moe

// Grouped expert GEMMs on the Blackwell tensor cores: tcgen05.mma with TMEM accumulators, operands
// staged in shared memory by TMA, warp-specialised and persistent.
//
// Paper, Sec. 4.5 "Expert FFN computation": after the sort-scatter every expert's tokens are
// contiguous; the gate and up projections are computed together and combined through SiLU, the
// down projection follows; experts without tokens are skipped.  The paper's kernel used 16x16
// WMMA tiles with double buffering.  Here:
//
//  * The weights sit on the MMA's M side (128 weight rows per tile, the hardware's full-rate
//    shape) and the tokens on its N side, so a token tile can have any multiple of 16 rows up
//    to NT_MAX.  An expert with 4 tokens costs one N=16 instruction per 128x16 weight slab
//    instead of a mostly empty 128-row token tile, and every weight byte is fetched once per
//    token tile.  D[128, N] = W_tile[128, K] * X_tile[N, K]^T, both operands K-major.
//  * gemm1 interleaves gate and up rows inside one 128-row A tile in groups of 16
//    (rows 32q..32q+15 = gate features, 32q+16..32q+31 = the matching up features), so each
//    epilogue warp finds gate and up of the same 16 features in its own 32 TMEM lanes and
//    pairs them with one shuffle; SiLU(gate)*up is applied before anything is stored.
//  * One CTA per SM walks tiles  tile = blockIdx.x + i*gridDim.x  of a device-built schedule
//    (no host round trip, no atomics).  Tiles of the same expert and weight slab are adjacent in
//    that order, so they run at the same time on neighbouring SMs and share the slab in L2.
//  * Warp 0 issues TMA loads into a STAGES-deep ring; warp 1 issues the MMAs and commits ring
//    slots back; warps 2..5 drain the accumulator (double-buffered in TMEM, so the epilogue of
//    one tile overlaps the MMAs of the next).
//  * Every wait is bounded: if one expires the CTA records MOE_ERR_DEVICE_TIMEOUT and the site in
//    the status word, every role stops, TMEM is released and the kernel returns.
#include "moe_tc_common.cuh"

namespace moe {
namespace {

using namespace tc;

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int NT_MAX, int STAGES>
struct SmemLayout {
    static constexpr int kSlotBBytes = NT_MAX * kRowBytes;
    static constexpr int kA = 0;
    static constexpr int kB = STAGES * kSlotABytes;
    static constexpr int kBars = kB + STAGES * kSlotBBytes;  // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
    static constexpr int kTmemSlot = kBars + (2 * STAGES + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kBytes + 1024;  // slack to align the base to 1024 bytes
};

template <int NT_MAX, int STAGES, bool SWIGLU>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_tc_kernel(const __grid_constant__ TensorMaps maps, const KernelParams p) {
    using L = SmemLayout<NT_MAX, STAGES>;
    constexpr int kTmemCols = 2 * NT_MAX;
    static_assert(kTmemCols >= 32 && kTmemCols <= 512 && (kTmemCols & (kTmemCols - 1)) == 0,
                  "a tensor-memory allocation must be a power of two between 32 and 512 columns");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;  // the down GEMM reports sites 5..8
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
                     "r"(kTmemCols)
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
        // ---------------- TMA producer: the warp walks the ring, one elected lane issues ----------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true, gate_up_done = false;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const int w_row = t.e * p.w_rows + t.f * kTileM;  // down projection: 128 rows of w2[e]
            const uint32_t tx_bytes = kSlotABytes + n_mma * kRowBytes;
            ok = handover_wait_expert(p.handover_role, p.handover, t.e, t.n_tok_tiles, p.handover_per_token_tile,
                                      p.tile_prefix[p.E], gate_up_done, abort_flag, p.status, lane);
            if (!ok) break;
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = mbar_wait_warp(bar_empty + stage * 8, phase ^ 1u, abort_flag, p.status, kSiteProducerEmpty + kSiteOffset);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = bar_full + stage * 8;
                    mbar_expect_tx(full, tx_bytes);
                    const uint32_t sa = base + L::kA + stage * kSlotABytes;
                    const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                    const int k0 = kb * kBlockK;
                    if (SWIGLU)  // 64 features = groups 4f..4f+3 of 16, gate and up rows interleaved per group
                        tma_load_5d(sa, &maps.w, k0, 0, 0, t.f * 4, t.e, full);
                    else
                        tma_load_2d(sa, &maps.w, k0, w_row, full);
                    tma_load_2d(sb, act_map<16>(maps, n_mma), k0, t.row0, full);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: same structure; MMAs and their commits come from one lane ----------------
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const uint32_t idesc = instr_desc_bf16(kTileM, (t.n_valid + 15) & ~15);
            ok = mbar_wait_warp(bar_acc_empty + acc * 8, acc_phase ^ 1u, abort_flag, p.status, kSiteMmaTmemEmpty + kSiteOffset);
            if (!ok) break;
            tcgen05_fence_after();
            const uint32_t d_tmem = tmem_base + acc * NT_MAX;
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = mbar_wait_warp(bar_full + stage * 8, phase, abort_flag, p.status, kSiteMmaFull + kSiteOffset);
                if (!ok) break;
                tcgen05_fence_after();
                if (elect_one()) {
                    const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kA + stage * kSlotABytes);
                    const uint64_t b_desc = smem_desc_k_major_sw128(base + L::kB + stage * L::kSlotBBytes);
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk)  // 16 K-elements = 32 bytes = 2 descriptor units
                        umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
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
        // ---------------- epilogue: TMEM -> registers -> global ----------------
        const int q = warp & 3;  // a warp may only read TMEM lanes 32*(warp%4) .. +31
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            ok = mbar_wait(bar_acc_full + acc * 8, acc_phase, abort_flag, p.status, kSiteEpilogueTmemFull + kSiteOffset);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tcgen05_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + acc * NT_MAX;
            if (SWIGLU) {
                const int hi = lane >> 4;
                __nv_bfloat16 *dst = p.out + (size_t)t.row0 * p.n_out + t.f * (kTileM / 2) + q * 16 + (lane & 15);
                for (int c0 = 0; c0 < n_mma; c0 += 16) {
                    float v[16];
                    tmem_load_16(taddr + c0, v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float other = __shfl_xor_sync(0xffffffffu, hi ? v[i] : v[8 + i], 16);
                        const float g = hi ? other : v[i];
                        const float u = hi ? v[8 + i] : other;
                        const int col = c0 + hi * 8 + i;
                        if (col < t.n_valid)
                            dst[(size_t)col * p.n_out] = __float2bfloat16_rn(swiglu(g, u));
                    }
                }
            } else {
                __nv_bfloat16 *dst = p.out + (size_t)t.row0 * p.n_out + t.f * kTileM + q * 32 + lane;
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
        // give copies that may still be in flight time to land before the CTA's memory is released
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <int NT_MAX, int STAGES, bool SWIGLU>
int launch_instance(const TensorMaps &maps, const KernelParams &p, int grid, cudaStream_t stream) {
    using L = SmemLayout<NT_MAX, STAGES>;
    static_assert(L::kDynamicBytes <= 232448, "ring does not fit in shared memory");
    auto kernel = grouped_gemm_tc_kernel<NT_MAX, STAGES, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kThreads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

template <bool SWIGLU>
int dispatch(int nt_max, const TensorMaps &maps, const KernelParams &p, int grid, cudaStream_t s) {
    switch (nt_max) {
        case 32: return launch_instance<32, 10, SWIGLU>(maps, p, grid, s);
        case 64: return launch_instance<64, 8, SWIGLU>(maps, p, grid, s);
        case 128: return launch_instance<128, 6, SWIGLU>(maps, p, grid, s);
        case 256: return launch_instance<256, 4, SWIGLU>(maps, p, grid, s);
        default: return MOE_ERR_UNSUPPORTED;
    }
}

__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(int *status) {
    __shared__ int abort_flag;
    if (threadIdx.x == 0) abort_flag = 0;
    __syncwarp();
    // the flag was zeroed by the caller's memset and nobody sets it: the poll must give up after its limit
    if (threadIdx.x == 0) poll_at_least(status + kHandoverFlagInt, 1, &abort_flag, status, kSiteSelfTest, 200000000LL);
}

}  // namespace

cudaError_t launch_wait_timeout_selftest(int *status, cudaStream_t stream) {
    cudaError_t err = cudaMemsetAsync(status, 0, kStatusBytesForward, stream);
    if (err != cudaSuccess) return err;
    wait_timeout_selftest_kernel<<<1, 32, 0, stream>>>(status);
    return cudaGetLastError();
}

int launch_grouped_gemm_tc(const GroupedGemmArgs &a, cudaStream_t stream) {
    if (a.K % kBlockK != 0 || a.A <= 0) return MOE_ERR_UNSUPPORTED;
    const int features_per_tile = a.swiglu ? kTileM / 2 : kTileM;
    if (a.n_out % features_per_tile != 0) return MOE_ERR_UNSUPPORTED;

    TensorMaps maps;
    const bool ok_w = a.swiglu ? encode_weight_map_gate_up(&maps.w, a.w, a.E, a.n_out, a.K)
                               : encode_weight_map_2d(&maps.w, a.w, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w || !encode_act_maps(maps.act, a.act, a.A, a.K, 16)) return MOE_ERR_CUDA;

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
    p.n_feature_tiles = a.n_out / features_per_tile;

    // The tile count is only known on the device; this is its upper bound.
    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / a.nt_max;
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int sms = sm_count();
    const int grid = (int)(max_tiles < sms ? max_tiles : sms);
    return a.swiglu ? dispatch<true>(a.nt_max, maps, p, grid, stream) : dispatch<false>(a.nt_max, maps, p, grid, stream);
}

}  // namespace moe

// Grouped expert GEMMs with FP8 (E4M3) block-scaled weights, one CTA per 128 x N tile.
//
// Paper: the workload is an "FP8 MoE" (Table 2; Sec. 4.5) and the paper's kernel feeds 16-bit
// tensor-core tiles, so stored FP8 weights are converted and rescaled on their way to the MMA.  Here
// the weights stay FP8 in HBM (half the bytes of the bf16 layer, which is what bounds the decode- and
// Mixtral-sized workloads) and the conversion happens in shared memory:
//
//   warp 0      TMA: per ring slot (128 K-elements = one scale block) the 128 x 128 tile of FP8 codes
//               (16 KiB, unswizzled) and the bf16 token tile as two 128-byte-swizzled 64-wide chunks,
//               each with ONE copy (a copy has a fixed cost, so slots are as large as the bf16 kernel's)
//   warps 6..9  converters: wait for the slot, turn the codes into bf16 * block scale and write them in
//               the 128-byte-swizzled K-major layout the MMA reads (two 32 KiB buffers),
//               fence towards the tensor core's proxy, signal
//   warp 1      MMA: A operand from the converted buffer, B operand straight from the slot
//   warps 2..5  epilogue (unchanged: SwiGLU or plain, double-buffered TMEM)
//
// A weight is decode(code) * scale[row/128][k/128].  A CTA's 128 weight rows lie in one scale block
// (down projection) or in one gate block and one up block (gate/up), and a slot is one 128-wide K
// block, so a slot needs one or two scalar scales.  Conversion: the code's exponent and
// mantissa bits are moved into a bf16 bit pattern worth value * 2^-120 (two byte permutes and three
// logic operations per four codes), then one bf16x2 multiply by scale * 2^120 per pair.  The scale is
// rounded to bf16 once per slot and the product once per weight: at most 2^-8 relative on a weight, an
// order of magnitude inside the layer's tolerance.  Scales must stay below 2^7 for scale * 2^120 to be finite.
#include "moe_tc_common.cuh"

namespace moe {
namespace {

using namespace tc;

constexpr int kConvWarps = 16;  // four per scheduler: the conversion is ALU work (2.5 instructions per weight) and
                                // needs the issue slots; measured 4 / 8 / 16 warps: 2.79 / 2.20 / 2.05 ms on the
                                // decode-sized gate/up GEMM
constexpr int kFp8Threads = (6 + kConvWarps) * 32;
constexpr int kSlotK = 128;                         // K elements per ring slot: one scale block, two MMA K-chunks of 64
constexpr int kSlotQBytes = kTileM * kSlotK;       // 16 KiB of codes
constexpr int kConvBytes = 2 * kSlotABytes;        // 32 KiB: two 128-byte-swizzled bf16 tiles (K 0..63 | 64..127)

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Four E4M3 codes (one 32-bit word, lowest byte first) -> four bf16 values times the block scale.
// A code byte placed in the high byte of a 16-bit lane and shifted so that its 4 exponent and 3 mantissa
// bits sit at the top of bf16's exponent-low/mantissa-high positions is a bf16 number equal to the
// code's value times 2^-120, for normal AND subnormal codes alike (E4M3's bias is 7, bf16's 127, and a
// zero exponent field means "no hidden one" in both); one bf16x2 multiply by scale * 2^120 finishes it.
__device__ __forceinline__ void convert_four(uint32_t codes, __nv_bfloat162 scale2, uint32_t &lo, uint32_t &hi) {
    const uint32_t t0 = __byte_perm(codes, 0u, 0x1404);  // bytes 0,1 -> high bytes of the two 16-bit lanes
    const uint32_t t1 = __byte_perm(codes, 0u, 0x3424);  // bytes 2,3
    const uint32_t r0 = ((t0 & 0x7F007F00u) >> 4) | (t0 & 0x80008000u);
    const uint32_t r1 = ((t1 & 0x7F007F00u) >> 4) | (t1 & 0x80008000u);
    __nv_bfloat162 v0, v1;
    *reinterpret_cast<uint32_t *>(&v0) = r0;
    *reinterpret_cast<uint32_t *>(&v1) = r1;
    v0 = __hmul2(v0, scale2);
    v1 = __hmul2(v1, scale2);
    lo = *reinterpret_cast<uint32_t *>(&v0);
    hi = *reinterpret_cast<uint32_t *>(&v1);
}

template <int NT_MAX, int STAGES, int CONV>
struct Fp8Smem {
    static constexpr int kSlotBBytes = 2 * NT_MAX * kRowBytes;       // two swizzled token tiles (K 0..63 | 64..127)
    static constexpr int kConv = 0;                                  // CONV x 32 KiB bf16 operand buffers (1024-aligned)
    static constexpr int kB = CONV * kConvBytes;                     // STAGES token-tile pairs
    static constexpr int kQ = kB + STAGES * kSlotBBytes;             // STAGES code tiles
    static constexpr int kBars = kQ + STAGES * kSlotQBytes;          // raw_full[S], raw_empty[S], conv_full[C], conv_empty[C], acc_full[2], acc_empty[2]
    static constexpr int kTmemSlot = kBars + (2 * STAGES + 2 * CONV + 4) * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kBytes = kAbort + 4;
    static constexpr int kDynamicBytes = kBytes + 1024;
};

template <int NT_MAX, int STAGES, int CONV, bool SWIGLU>
__global__ void __launch_bounds__(kFp8Threads, 1)
grouped_gemm_tc_fp8w_kernel(const __grid_constant__ TensorMaps maps, const KernelParams p) {
    using L = Fp8Smem<NT_MAX, STAGES, CONV>;
    constexpr int kTmemCols = 2 * NT_MAX;
    static_assert(kTmemCols >= 32 && kTmemCols <= 512 && (kTmemCols & (kTmemCols - 1)) == 0,
                  "a tensor-memory allocation must be a power of two between 32 and 512 columns");
    constexpr int kSiteOffset = SWIGLU ? 0 : 4;
    chain_release();  // the next kernel of the forward call may be scheduled; it waits for this grid to finish
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_raw_full = base + L::kBars, bar_raw_empty = bar_raw_full + STAGES * 8;
    const uint32_t bar_conv_full = bar_raw_empty + STAGES * 8, bar_conv_empty = bar_conv_full + CONV * 8;
    const uint32_t bar_acc_full = bar_conv_empty + CONV * 8, bar_acc_empty = bar_acc_full + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar_raw_full + s * 8, 1);
            mbar_init(bar_raw_empty + s * 8, 1);
        }
        for (int c = 0; c < CONV; ++c) {
            mbar_init(bar_conv_full + c * 8, kConvWarps);
            mbar_init(bar_conv_empty + c * 8, 1);
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
    chain_wait();  // everything above overlapped the previous kernel; its results are read from here on
    const int total_tiles = p.tile_prefix[p.E] * p.n_feature_tiles;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            const int w_row = t.e * p.w_rows + t.f * kTileM;
            const uint32_t tx_bytes = kSlotQBytes + 2 * n_mma * kRowBytes;
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                ok = mbar_wait_warp(bar_raw_empty + stage * 8, phase ^ 1u, abort_flag, p.status, kSiteProducerEmpty + kSiteOffset);
                if (!ok) break;
                if (elect_one()) {
                    const uint32_t full = bar_raw_full + stage * 8;
                    mbar_expect_tx(full, tx_bytes);
                    const uint32_t sq = base + L::kQ + stage * kSlotQBytes;
                    const uint32_t sb = base + L::kB + stage * L::kSlotBBytes;
                    const int k0 = kb * kSlotK;
                    if (SWIGLU)
                        tma_load_5d(sq, &maps.w, k0, 0, 0, t.f * 4, t.e, full);
                    else
                        tma_load_2d(sq, &maps.w, k0, w_row, full);
                    // one copy: rows x (two 64-wide K chunks), each chunk landing as its own swizzled tile of n_mma rows
                    tma_load_3d(sb, act_map<16>(maps, n_mma), 0, t.row0, 2 * kb, full);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        int stage = 0, conv = 0, acc = 0;
        uint32_t phase = 0, conv_phase = 0, acc_phase = 0;
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
                // the converted weights imply the slot has landed; the token tile is read from the slot itself
                ok = mbar_wait_warp(bar_conv_full + conv * 8, conv_phase, abort_flag, p.status, kSiteMmaFull + kSiteOffset);
                if (ok) ok = mbar_wait_warp(bar_raw_full + stage * 8, phase, abort_flag, p.status, kSiteMmaFull + kSiteOffset);
                if (!ok) break;
                tcgen05_fence_after();
                if (elect_one()) {
                    const int n_mma = (t.n_valid + 15) & ~15;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {  // the slot's two 64-wide K chunks
                        const uint64_t a_desc = smem_desc_k_major_sw128(base + L::kConv + conv * kConvBytes + j * kSlotABytes);
                        const uint64_t b_desc =
                            smem_desc_k_major_sw128(base + L::kB + stage * L::kSlotBBytes + j * n_mma * kRowBytes);
#pragma unroll
                        for (int kk = 0; kk < kBlockK / 16; ++kk)
                            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | j | kk) != 0);
                    }
                    umma_commit(bar_conv_empty + conv * 8);
                    umma_commit(bar_raw_empty + stage * 8);
                    if (kb == p.n_k_blocks - 1) umma_commit(bar_acc_full + acc * 8);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                if (++conv == CONV) { conv = 0; conv_phase ^= 1u; }
            }
            if (!ok) break;
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    } else if (warp >= 6) {
        // ---------------- converters: FP8 codes -> scaled bf16 in the MMA's swizzled layout ----------------
        // A slot holds 128 rows x 128 codes.  Warp cw owns rows (128/kConvWarps)*cw ..; per iteration lanes
        // 8m..8m+7 take the eight 16-byte pieces of row base + 4i + m (512 contiguous bytes per
        // instruction), and each lane writes its 16 weights as two 16-byte chunks of the bf16 row in
        // K-chunk tile (piece / 4): chunk c of row r at r*128 + ((c ^ (r & 7)) * 16).
        const int cw = warp - 6, piece = lane & 7, sub_row = lane >> 3;
        constexpr int kRowsPerWarp = kTileM / kConvWarps;
        int stage = 0, conv = 0;
        uint32_t phase = 0, conv_phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            // scale rows: the tile's gate block and up block (gate/up), or its single block (down)
            const int row_blocks = p.w_rows >> 7;
            const float *scale_a = p.w_scale + ((size_t)t.e * row_blocks + (SWIGLU ? (t.f * 64) >> 7 : t.f)) * p.n_k_blocks;
            const float *scale_b = SWIGLU ? p.w_scale + ((size_t)t.e * row_blocks + ((p.n_out + t.f * 64) >> 7)) * p.n_k_blocks
                                          : scale_a;
            float next_a = __ldg(scale_a), next_b = __ldg(scale_b);
            for (int kb = 0; kb < p.n_k_blocks; ++kb) {
                const float two120 = 1329227995784915872903807060280344576.0f;  // 2^120
                const __nv_bfloat162 sa = __float2bfloat162_rn(next_a * two120);
                const __nv_bfloat162 sb = SWIGLU ? __float2bfloat162_rn(next_b * two120) : sa;
                if (kb + 1 < p.n_k_blocks) {  // next slot's scales, off the critical path
                    next_a = __ldg(scale_a + kb + 1);
                    next_b = __ldg(scale_b + kb + 1);
                }
                ok = mbar_wait_warp(bar_raw_full + stage * 8, phase, abort_flag, p.status, kSiteMmaFull + kSiteOffset);
                if (ok) ok = mbar_wait_warp(bar_conv_empty + conv * 8, conv_phase ^ 1u, abort_flag, p.status, kSiteProducerEmpty + kSiteOffset);
                if (!ok) break;
                const uint8_t *src = base_ptr + L::kQ + stage * kSlotQBytes;
                uint8_t *dst = base_ptr + L::kConv + conv * kConvBytes + (piece >> 2) * kSlotABytes;
                const int chunk = 2 * (piece & 3);
#pragma unroll
                for (int i = 0; i < kRowsPerWarp / 4; ++i) {
                    const int row = cw * kRowsPerWarp + i * 4 + sub_row;
                    // gate/up slots interleave 16 gate rows and 16 up rows
                    const __nv_bfloat162 s2 = (SWIGLU && (row & 16)) ? sb : sa;
                    const uint4 q = *reinterpret_cast<const uint4 *>(src + row * kSlotK + piece * 16);
                    uint4 lo, hi;
                    convert_four(q.x, s2, lo.x, lo.y);
                    convert_four(q.y, s2, lo.z, lo.w);
                    convert_four(q.z, s2, hi.x, hi.y);
                    convert_four(q.w, s2, hi.z, hi.w);
                    uint8_t *drow = dst + row * kRowBytes;
                    *reinterpret_cast<uint4 *>(drow + ((chunk ^ (row & 7)) << 4)) = lo;
                    *reinterpret_cast<uint4 *>(drow + (((chunk + 1) ^ (row & 7)) << 4)) = hi;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy stores -> visible to the MMA
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_conv_full + conv * 8);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                if (++conv == CONV) { conv = 0; conv_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> global ----------------
        const int q = warp & 3;
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int round = 0; ok; ++round) {
            const int tile = tile_of_round(round, blockIdx.x, gridDim.x);
            if (tile >= total_tiles) break;
            const Tile t = decode_tile(tile, p);
            const int n_mma = (t.n_valid + 15) & ~15;
            ok = mbar_wait_warp(bar_acc_full + acc * 8, acc_phase, abort_flag, p.status, kSiteEpilogueTmemFull + kSiteOffset);
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
                        if (col < t.n_valid) dst[(size_t)col * p.n_out] = __float2bfloat16_rn(swiglu(g, u));
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
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
    }

    // ---------------- teardown ----------------
    tcgen05_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <int NT_MAX, int STAGES, int CONV, bool SWIGLU>
int launch_fp8_instance(const TensorMaps &maps, const KernelParams &p, int grid, cudaStream_t stream) {
    using L = Fp8Smem<NT_MAX, STAGES, CONV>;
    static_assert(L::kDynamicBytes <= 232448, "rings do not fit in shared memory");
    auto kernel = grouped_gemm_tc_fp8w_kernel<NT_MAX, STAGES, CONV, SWIGLU>;
    if (!set_max_dynamic_smem_once(reinterpret_cast<const void *>(kernel), L::kDynamicBytes))
        return MOE_ERR_CUDA;
    return launch_chained(kernel, grid, kFp8Threads, L::kDynamicBytes, stream, maps, p) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

template <bool SWIGLU>
int dispatch_fp8(int nt_max, const TensorMaps &maps, const KernelParams &p, int grid, cudaStream_t s) {
    switch (nt_max) {
        case 32: return launch_fp8_instance<32, 5, 2, SWIGLU>(maps, p, grid, s);
        case 64: return launch_fp8_instance<64, 4, 2, SWIGLU>(maps, p, grid, s);
        case 128: return launch_fp8_instance<128, 3, 2, SWIGLU>(maps, p, grid, s);
        case 256: return launch_fp8_instance<256, 2, 2, SWIGLU>(maps, p, grid, s);
        default: return MOE_ERR_UNSUPPORTED;
    }
}

}  // namespace

int launch_grouped_gemm_tc_fp8w(const GroupedGemmArgs &a, cudaStream_t stream) {
    if (a.K % 128 != 0 || a.A <= 0 || !a.w_scale || a.w_rows % 128 != 0) return MOE_ERR_UNSUPPORTED;
    const int features_per_tile = a.swiglu ? kTileM / 2 : kTileM;
    if (a.n_out % 128 != 0) return MOE_ERR_UNSUPPORTED;  // gate and up halves must both start on a scale block

    TensorMaps maps;
    const bool ok_w = a.swiglu ? encode_weight_map_gate_up_fp8(&maps.w, a.w, a.E, a.n_out, a.K)
                               : encode_weight_map_2d_fp8(&maps.w, a.w, (uint64_t)a.E * a.w_rows, a.K);
    if (!ok_w || !encode_act_maps_k128(maps.act, a.act, a.A, a.K, 16)) return MOE_ERR_CUDA;

    KernelParams p;
    p.out = a.out;
    p.expert_offsets = a.expert_offsets;
    p.tile_prefix = a.tile_prefix;
    p.tile_order = a.tile_order;
    p.tile_rows = a.tile_rows;
    p.status = a.status;
    p.E = a.E;
    p.n_k_blocks = a.K / kSlotK;  // slots of 128 K-elements
    p.n_out = a.n_out;
    p.w_rows = a.w_rows;
    p.n_feature_tiles = a.n_out / features_per_tile;
    p.w_scale = a.w_scale;
    p.handover_role = 0;
    p.handover = nullptr;
    p.handover_per_token_tile = 0;

    const long long max_token_tiles = (long long)(a.A < a.E ? a.A : a.E) + a.A / a.nt_max;
    const long long max_tiles = max_token_tiles * p.n_feature_tiles;
    const int sms = sm_count();
    const int grid = (int)(max_tiles < sms ? max_tiles : sms);
    return a.swiglu ? dispatch_fp8<true>(a.nt_max, maps, p, grid, stream) : dispatch_fp8<false>(a.nt_max, maps, p, grid, stream);
}

}  // namespace moe

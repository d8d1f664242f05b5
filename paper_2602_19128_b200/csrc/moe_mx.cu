// MX FP8 support kernels: quantisation of bf16 rows to E4M3 codes with one E8M0 scale byte per 32
// elements (fused with the scatter into expert-contiguous order), and the repacking of weight scale bytes
// into the 512-byte atoms the block-scaled MMA consumes.
//
// Paper, Sec. 4.5: the MoE workload is an FP8 one and names FP8 packing and scaling as a cost of the
// kernel; the granularity is not given.  This path uses the OCP Microscaling rule: for 32 values,
// scale = 2^(floor(log2(amax)) - 8), codes = E4M3(value / scale) rounded to nearest even, saturating.
#include <cuda_fp8.h>

#include "moe_internal.cuh"

namespace moe {
namespace {

// Scale byte from the largest |value| bit pattern of a block: exponent field - 8, floored at 0 (zero and
// tiny blocks); 255 (NaN) when the block holds an infinity or a NaN.
__device__ __forceinline__ uint32_t mx_scale_byte(uint32_t amax_bits) {
    const uint32_t e = amax_bits >> 23;
    if (e == 255u) return 255u;
    return e > 8u ? e - 8u : 0u;
}
// 2^(127 - b): the factor that divides by the scale, exactly.
__device__ __forceinline__ float mx_inverse_scale(uint32_t scale_byte) { return __uint_as_float((254u - scale_byte) << 23); }

__device__ __forceinline__ uint32_t e4m3x2(float lo, float hi) {
    return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);
}

// Quantise the 8 bf16 values a lane holds; 4 neighbouring lanes form one block of 32.  Returns the codes
// packed low-to-high and the block's scale byte (the same in the 4 lanes).  All 32 lanes must call.
__device__ __forceinline__ uint2 quantize_8_of_32(const uint4 v, uint32_t &scale_byte) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t amax = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {  // bf16 magnitude bits widened to fp32 bit patterns compare like the values
        amax = max(amax, (w[i] << 16) & 0x7FFFFFFFu);
        amax = max(amax, w[i] & 0x7FFF0000u);
    }
    amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    scale_byte = mx_scale_byte(amax);
    if (scale_byte == 255u) return make_uint2(0x7F7F7F7Fu, 0x7F7F7F7Fu);
    const float inv = mx_inverse_scale(scale_byte);
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
        c[i] = e4m3x2(__uint_as_float(w[i] << 16) * inv, __uint_as_float(w[i] & 0xFFFF0000u) * inv);
    return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

// MX quantisation of bf16 rows, 256 elements (32 lanes x 8) at a time.  A row is shared by `warps_per_row` warps,
// warp s taking segments s, s + warps_per_row, ...: small batches spread one row over many warps so the device is
// not left idle, large ones keep one warp per row.
//   kScatter = false: codes[r,:] and row-major scale bytes of row r (the plain quantiser).
//   kScatter = true : token-major scatter into expert-contiguous order.  Token t's row is read and quantised ONCE
//                     and its codes and scale bytes are stored to the up to top_k rows flat_to_sorted[t*k + j] >= 0,
//                     the scale bytes straight into the atom layout of each destination row.
template <bool kScatter>
__global__ void __launch_bounds__(256)
mx_quantize_rows_kernel(const uint4 *__restrict__ x, const int *__restrict__ flat_to_sorted,
                        const int *__restrict__ topk_ids, const int *__restrict__ expert_offsets,
                        const int *__restrict__ tile_rows, int local_offset, int n_local, int n_rows, int k, int vec_per_row,
                        int warps_per_row, uint2 *__restrict__ codes, uint8_t *__restrict__ scales, int n_atoms, int tile) {
    chain_release();
    chain_wait();
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int r = (int)(w / warps_per_row), first_seg = (int)(w % warps_per_row);
    if (r >= n_rows) return;
    // kScatter: lane j holds rank j's destination row and where its scale bytes go inside one K-slot's atoms
    int my_row = -1;
    long long my_sf_base = 0;
    if (kScatter && lane < k) {
        my_row = flat_to_sorted[(size_t)r * k + lane];
        if (my_row >= 0) {
            const int e = topk_ids[(size_t)r * k + lane] - local_offset;  // resident, or the row would be -1
            const int begin = expert_offsets[e], i = my_row - begin;
            // row tr of token tile i / rows of this expert, whose tiles all have `rows` rows (the schedule's choice)
            const int rows = tile_rows[e], stride = tile > 256 ? 256 : tile;
            const int atoms_per_tile = (tile + 127) / 128, tr = i % rows;
            my_sf_base = (long long)((begin / stride + e + i / rows) * atoms_per_tile + tr / 128) * kMxSfAtomBytes +
                         mx_atom_byte(tr % 128, 0);
        }
    }
    (void)n_local;
    if (kScatter && !__any_sync(0xffffffffu, my_row >= 0)) return;  // none of the token's experts is resident here
    const uint4 *src = x + (size_t)r * vec_per_row;
    constexpr int kInFlight = 4;  // independent 16-byte loads per lane before the first is used
    const int n_segs = (vec_per_row + 31) / 32;
    for (int s0 = first_seg; s0 < n_segs; s0 += kInFlight * warps_per_row) {  // uniform over the warp
        uint4 in[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int v = (s0 + u * warps_per_row) * 32 + lane;
            in[u] = (s0 + u * warps_per_row < n_segs && v < vec_per_row) ? src[v] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            if (s0 + u * warps_per_row >= n_segs) break;  // uniform
            const int v = (s0 + u * warps_per_row) * 32 + lane;
            uint32_t sb;
            const uint2 q = quantize_8_of_32(in[u], sb);  // every lane takes part in the shuffles
            const int block = v >> 2;  // 32-element block along the row; 4 blocks per 128-element slot
            if (kScatter) {
                for (int j = 0; j < k; ++j) {
                    const int row = __shfl_sync(0xffffffffu, my_row, j);
                    const long long sf_base = __shfl_sync(0xffffffffu, my_sf_base, j);
                    if (row < 0 || v >= vec_per_row) continue;
                    __stcs(codes + (size_t)row * vec_per_row + v, q);  // streaming: the GEMM reads it from memory anyway
                    if ((lane & 3) == 0)
                        scales[(size_t)(block >> 2) * n_atoms * kMxSfAtomBytes + sf_base + (block & 3)] = (uint8_t)sb;
                }
            } else if (v < vec_per_row) {
                codes[(size_t)r * vec_per_row + v] = q;
                if ((lane & 3) == 0) scales[(size_t)r * (vec_per_row >> 2) + block] = (uint8_t)sb;
            }
        }
    }
}

// Warps per row: enough warps to fill the device (about 16 per SM slot) when there are few rows.
int mx_quantize_warps_per_row(long long rows, int n_segs) {
    const long long target = 32768;
    long long per_row = rows > 0 ? (target + rows - 1) / rows : 1;
    if (per_row > n_segs) per_row = n_segs;
    return per_row < 1 ? 1 : (int)per_row;
}

// One thread per (expert, tile, slot, row): moves the row's 4 scale bytes of that slot into its atom.
__global__ void __launch_bounds__(256)
mx_pack_scales_kernel(const uint32_t *__restrict__ plain, int E, int rows, int slots, int tiles, int gate_up,
                      uint32_t *__restrict__ packed) {
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long total = (long long)E * tiles * slots * 128;
    if (idx >= total) return;
    const int m = (int)(idx % 128);
    const int slot = (int)((idx / 128) % slots);
    const int tile = (int)((idx / 128 / slots) % tiles);
    const int e = (int)(idx / 128 / slots / tiles);
    int row;
    if (gate_up) {  // tile row m = 32q + 16 * half + j  <->  feature 64 * tile + 16q + j of the gate (half 0) or up (half 1) rows
        const int q = m >> 5, half = (m >> 4) & 1, j = m & 15;
        row = half * (rows / 2) + 64 * tile + 16 * q + j;
    } else {
        row = 128 * tile + m;
    }
    const uint32_t four = plain[((size_t)e * rows + row) * slots + slot];
    packed[(((size_t)e * tiles + tile) * slots + slot) * (kMxSfAtomBytes / 4) + mx_atom_byte(m, 0) / 4] = four;
}

}  // namespace

cudaError_t launch_mx_scatter_quantize(const __nv_bfloat16 *x, const int *flat_to_sorted, const int *topk_ids,
                                       const int *expert_offsets, const int *tile_rows, LocalExperts local, int T, int k,
                                       int H, uint8_t *xq, uint8_t *x_sf, int n_atoms, int tile, cudaStream_t stream) {
    const int wpr = mx_quantize_warps_per_row(T, (H / 8 + 31) / 32);
    const long long warps = (long long)T * wpr;
    return launch_chained(mx_quantize_rows_kernel<true>, (unsigned)((warps + 7) / 8), 256, 0, stream,
                          reinterpret_cast<const uint4 *>(x), flat_to_sorted, topk_ids, expert_offsets, tile_rows, local.offset,
                          local.count, T, k, H / 8, wpr, reinterpret_cast<uint2 *>(xq), x_sf, n_atoms, tile);
}

cudaError_t launch_mx_quantize_rows(const __nv_bfloat16 *x, int R, int K, uint8_t *codes, uint8_t *scales,
                                    cudaStream_t stream) {
    const int wpr = mx_quantize_warps_per_row(R, (K / 8 + 31) / 32);
    const long long warps = (long long)R * wpr;
    return launch_chained(mx_quantize_rows_kernel<false>, (unsigned)((warps + 7) / 8), 256, 0, stream,
                          reinterpret_cast<const uint4 *>(x), nullptr, nullptr, nullptr, nullptr, 0, 0, R, 1, K / 8, wpr,
                          reinterpret_cast<uint2 *>(codes), scales, 0, 1);
}

cudaError_t launch_mx_pack_scales(const uint8_t *plain, int E, int rows, int K, bool gate_up, uint8_t *packed,
                                  cudaStream_t stream) {
    const int slots = K / 128;
    const int tiles = gate_up ? rows / 2 / 64 : rows / 128;
    const long long total = (long long)E * tiles * slots * 128;
    mx_pack_scales_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const uint32_t *>(plain), E, rows, slots, tiles, gate_up ? 1 : 0,
        reinterpret_cast<uint32_t *>(packed));
    return cudaGetLastError();
}

}  // namespace moe

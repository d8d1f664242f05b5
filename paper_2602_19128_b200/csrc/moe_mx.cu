// MX FP8 support kernels: quantisation of bf16 rows to E4M3 codes with one E8M0 scale byte per 32
// elements (fused with the gather into expert-contiguous order), and the repacking of weight scale bytes
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

// Byte offset, inside one K-slot's atoms, of the scale bytes of sorted row r: finds the expert whose segment holds
// the row (last e with offsets[e] <= r: a 32-way search in two steps; offsets are non-decreasing, so the lanes that
// satisfy the test form a prefix), then its token tile and the row's place in the tile's atoms.  Whole warp.
__device__ __forceinline__ size_t locate_sorted_row(int r, const int *__restrict__ expert_offsets, int E, int tile, int lane) {
    const int stride = (E + 31) / 32;
    const int coarse = __popc(__ballot_sync(0xffffffffu, lane * stride < E && expert_offsets[lane * stride] <= r)) - 1;
    const int cand = coarse * stride + lane;
    const int e = coarse * stride + __popc(__ballot_sync(0xffffffffu, lane < stride && cand < E && expert_offsets[cand] <= r)) - 1;
    const int begin = expert_offsets[e], i = r - begin;
    const int atoms_per_tile = (tile + 127) / 128, tr = i % tile;  // row tr of token tile i / tile of this expert
    return (size_t)((begin / tile + e + i / tile) * atoms_per_tile + tr / 128) * kMxSfAtomBytes + mx_atom_byte(tr % 128, 0);
}

// A row is cut into 256-element segments (32 lanes x 8 elements = 8 blocks of 32) and shared by
// `warps_per_row` warps, warp s taking segments s, s + warps_per_row, ...: small batches spread one row
// over many warps so the device is not left idle, large ones keep one warp per row.  kGather: row r of
// the output is token sorted_to_flat[r] / k and the scale bytes go to the activation atoms; otherwise
// row r is row r and the scale bytes are stored row-major.
template <bool kGather>
__global__ void __launch_bounds__(256)
mx_quantize_rows_kernel(const uint4 *__restrict__ x, const int *__restrict__ sorted_to_flat,
                        const int *__restrict__ expert_offsets, int E, int n_rows_plain, int k, int vec_per_row,
                        int warps_per_row, uint2 *__restrict__ codes, uint8_t *__restrict__ scales, int n_atoms, int tile) {
    chain_release();
    chain_wait();
    const int lane = threadIdx.x & 31;
    const long long w = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int r = (int)(w / warps_per_row), first_seg = (int)(w % warps_per_row);
    int src_row = r;
    size_t sf_base = 0;
    if (kGather) {
        if (r >= expert_offsets[E]) return;  // rows actually scheduled
        sf_base = locate_sorted_row(r, expert_offsets, E, tile, lane);
        src_row = sorted_to_flat[r] / k;
    } else {
        if (r >= n_rows_plain) return;
    }
    const uint4 *src = x + (size_t)src_row * vec_per_row;
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
            if (v < vec_per_row) {
                if (kGather)
                    __stcs(codes + (size_t)r * vec_per_row + v, q);  // streaming: the GEMM reads it from memory anyway; keep x in L2
                else
                    codes[(size_t)r * vec_per_row + v] = q;
                if ((lane & 3) == 0) {
                    const int block = v >> 2;  // 32-element block along the row; 4 blocks per 128-element slot
                    if (kGather)
                        scales[(size_t)(block >> 2) * n_atoms * kMxSfAtomBytes + sf_base + (block & 3)] = (uint8_t)sb;
                    else
                        scales[(size_t)r * (vec_per_row >> 2) + block] = (uint8_t)sb;
                }
            }
        }
    }
}

// Second step of the two-step form for large batches: x was quantised once per TOKEN (codes [T,H], scale bytes
// [T,H/32] row-major, 60 MB for 8192 tokens: resident in L2), and every sorted row copies its token's codes and
// scatters its scale bytes into the atoms.  Against quantising each of the top_k copies of a token this reads the
// 16-bit rows once instead of top_k times and moves half the bytes per copy.  One warp per sorted row.
__global__ void __launch_bounds__(256)
mx_gather_codes_kernel(const uint4 *__restrict__ tok_codes, const uint8_t *__restrict__ tok_scales,
                       const int *__restrict__ sorted_to_flat, const int *__restrict__ expert_offsets, int E, int k,
                       int vec_per_row, int blocks_per_row, uint4 *__restrict__ codes, uint8_t *__restrict__ scales,
                       int n_atoms, int tile) {
    chain_release();
    chain_wait();
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (r >= expert_offsets[E]) return;
    const size_t sf_base = locate_sorted_row(r, expert_offsets, E, tile, lane);
    const int t = sorted_to_flat[r] / k;
    const uint4 *src = tok_codes + (size_t)t * vec_per_row;
    uint4 *dst = codes + (size_t)r * vec_per_row;
    int i = lane;
    for (; i + 96 < vec_per_row; i += 128) {  // four independent 16-byte loads in flight per lane
        const uint4 a = src[i], b = src[i + 32], c = src[i + 64], d = src[i + 96];
        __stcs(dst + i, a); __stcs(dst + i + 32, b); __stcs(dst + i + 64, c); __stcs(dst + i + 96, d);
    }
    for (; i < vec_per_row; i += 32) __stcs(dst + i, src[i]);
    for (int b = lane; b < blocks_per_row; b += 32)
        scales[(size_t)(b >> 2) * n_atoms * kMxSfAtomBytes + sf_base + (b & 3)] = tok_scales[(size_t)t * blocks_per_row + b];
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

cudaError_t launch_mx_gather_quantize(const __nv_bfloat16 *x, const int *sorted_to_flat, const int *expert_offsets, int E,
                                      int A, int k, int H, uint8_t *xq, uint8_t *x_sf, int n_atoms, int tile,
                                      cudaStream_t stream) {
    const int segs = mx_quantize_warps_per_row(A, (H / 8 + 31) / 32);
    const long long warps = (long long)A * segs;
    return launch_chained(mx_quantize_rows_kernel<true>, (unsigned)((warps + 7) / 8), 256, 0, stream,
                          reinterpret_cast<const uint4 *>(x), sorted_to_flat, expert_offsets, E, 0, k, H / 8, segs,
                          reinterpret_cast<uint2 *>(xq), x_sf, n_atoms, tile);
}

cudaError_t launch_mx_gather_codes(const uint8_t *tok_codes, const uint8_t *tok_scales, const int *sorted_to_flat,
                                   const int *expert_offsets, int E, int A, int k, int H, uint8_t *xq, uint8_t *x_sf,
                                   int n_atoms, int tile, cudaStream_t stream) {
    return launch_chained(mx_gather_codes_kernel, (A + 7) / 8, 256, 0, stream, reinterpret_cast<const uint4 *>(tok_codes),
                          tok_scales, sorted_to_flat, expert_offsets, E, k, H / 16, H / 32, reinterpret_cast<uint4 *>(xq), x_sf,
                          n_atoms, tile);
}

cudaError_t launch_mx_quantize_rows(const __nv_bfloat16 *x, int R, int K, uint8_t *codes, uint8_t *scales,
                                    cudaStream_t stream) {
    const int segs = mx_quantize_warps_per_row(R, (K / 8 + 31) / 32);
    const long long warps = (long long)R * segs;
    return launch_chained(mx_quantize_rows_kernel<false>, (unsigned)((warps + 7) / 8), 256, 0, stream,
                          reinterpret_cast<const uint4 *>(x), nullptr, nullptr, 0, R, 1, K / 8, segs,
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

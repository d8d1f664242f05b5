// Device helpers shared by the two MX FP8 grouped-GEMM kernels (one CTA per tile, and CTA pairs):
// the tile decoder with the scale-atom index, descriptors of the block-scaled MMA and of the scale
// copies, and the gate/up epilogue that quantises h.
#pragma once

#include <cuda_fp8.h>

#include "moe_tc_common.cuh"

namespace moe {
namespace mxtc {

using namespace tc;

constexpr int kMxSlotK = 128;                     // K elements = bytes per operand row per ring slot
constexpr int kMxSlotABytes = kTileM * kMxSlotK;  // 16 KiB
constexpr int kTmemColsMx = 512;

struct MxParams {
    void *out;
    uint8_t *out_sf;
    const uint8_t *w_sf, *act_sf;
    const int *expert_offsets, *tile_prefix, *tile_order, *tile_rows;
    int *status;
    int E, n_k_blocks, n_out, w_rows, n_feature_tiles, n_atoms;
    int tile_stride;     // stride of the tile numbering: min(token-tile bound, 256) (moe_internal.cuh)
    int atoms_per_tile;  // ceil(token-tile bound / 128)
    int handover_role;   // hand-over between the two GEMMs of a call (moe_internal.cuh)
    int *handover;
    int handover_per_token_tile;
};

struct MxTile {
    int e, f, row0, n_valid;
    int atom;         // first activation scale atom of the tile
    int n_tok_tiles;  // token tiles of this tile's expert
};

__device__ __forceinline__ MxTile decode_mx_tile(int tile, const MxParams &p) {
    int lo = 0, hi = p.E;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.tile_prefix[mid] * p.n_feature_tiles <= tile) lo = mid; else hi = mid;
    }
    MxTile t;
    t.e = p.tile_order[lo];
    const int first = p.tile_prefix[lo], n_tok_tiles = p.tile_prefix[lo + 1] - first;
    const int local = tile - first * p.n_feature_tiles;
    t.f = local / n_tok_tiles;
    const int j = local - t.f * n_tok_tiles;
    const int rows = p.tile_rows[t.e];  // rows of every tile of this expert (the bound itself for bounds up to 256)
    const int begin = p.expert_offsets[t.e], count = p.expert_offsets[t.e + 1] - begin;
    t.row0 = begin + j * rows;
    t.n_valid = min(rows, count - j * rows);
    t.atom = (begin / p.tile_stride + t.e + j) * p.atoms_per_tile;
    t.n_tok_tiles = n_tok_tiles;
    return t;
}

// Shared-memory descriptor of one scale atom: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sf_atom(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(128 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
// Block-scaled instruction descriptor: E4M3 A and B (format 0), both K-major, E8M0 scales, M = m (128, or
// 256 for a CTA pair), N = n, scale byte `sf` of each row (the K-block within the slot) for both operands.
__device__ __forceinline__ uint32_t instr_desc_mx(int m, int n, int sf) {
    return ((uint32_t)sf << 4) | ((uint32_t)(n >> 3) << 17) | (1u << 23) | ((uint32_t)(m >> 4) << 24) |
           ((uint32_t)sf << 29);
}

// Barrier of the two epilogue warps (64 threads) that share a block of 32 features.
__device__ __forceinline__ void pair_sync(int pair) {
    asm volatile("bar.sync %0, 64;" ::"r"(2 + pair) : "memory");
}

__device__ __forceinline__ uint32_t mx_scale_byte(uint32_t amax_bits) {
    const uint32_t e = amax_bits >> 23;
    if (e == 255u) return 255u;
    return e > 8u ? e - 8u : 0u;
}

// Maxima of eight values over the 16 lanes of a half-warp by recursive halving: 8 shuffles instead of the 32 of a
// butterfly per value.  Afterwards lanes j and j ^ 1 (j = lane % 16) both hold the maximum of value j / 2.
__device__ __forceinline__ uint32_t half_warp_max8(const uint32_t (&mag)[8], int j) {
    uint32_t m4[4], m2[2];
    const bool b8 = (j & 8) != 0, b4 = (j & 4) != 0, b2 = (j & 2) != 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, b8 ? mag[i] : mag[4 + i], 8);
        m4[i] = max(b8 ? mag[4 + i] : mag[i], recv);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const uint32_t recv = __shfl_xor_sync(0xffffffffu, b4 ? m4[i] : m4[2 + i], 4);
        m2[i] = max(b4 ? m4[2 + i] : m4[i], recv);
    }
    uint32_t m1 = max(b2 ? m2[1] : m2[0], __shfl_xor_sync(0xffffffffu, b2 ? m2[0] : m2[1], 2));
    return max(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
}

// Gate/up epilogue of one warp: its 32 TMEM lanes hold, for 16 features, the gate rows (lanes 0..15) and
// the up rows (lanes 16..31) of n_mma token columns.  Computes h = SiLU(gate) * up, quantises it in
// blocks of 32 features (this warp's 16 and its partner warp's 16, warps q and q^1), and stores the
// codes and the scale bytes.
//   dst      -> code of this lane's feature in the tile's first row; row stride n_out bytes
//   sf_dst   -> byte of the block's scale in row 0 of the tile's first atom (K-slot and block already applied)
//   amax_s   [2][4][16] exchange buffer in shared memory; buf is flipped every chunk (across tiles too): a
//            warp may run one chunk ahead of its partner
__device__ __forceinline__ void drain_swiglu_mx(uint32_t taddr, int n_mma, int n_valid, uint8_t *dst, size_t n_out,
                                                uint8_t *sf_dst, uint32_t *amax_s, int &buf, int q, int lane) {
    const int hi = lane >> 4, j = lane & 15;
    for (int c0 = 0; c0 < n_mma; c0 += 16) {
        float v[16];
        tmem_load_16(taddr + c0, v);
        float hv[8];
        uint32_t mag[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float other = __shfl_xor_sync(0xffffffffu, hi ? v[i] : v[8 + i], 16);
            const float g = hi ? other : v[i];
            const float u = hi ? v[8 + i] : other;
            hv[i] = swiglu(g, u);
            mag[i] = __float_as_uint(hv[i]) & 0x7FFFFFFFu;  // magnitudes compare as integers; NaN and inf on top
        }
        const uint32_t col_max = half_warp_max8(mag, j);  // of column c0 + hi * 8 + j / 2 over this warp's 16 features
        buf ^= 1;
        if ((j & 1) == 0) amax_s[(buf * 4 + q) * 16 + hi * 8 + (j >> 1)] = col_max;
        pair_sync(q >> 1);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t block_mag = max(amax_s[(buf * 4 + q) * 16 + hi * 8 + i], amax_s[(buf * 4 + (q ^ 1)) * 16 + hi * 8 + i]);
            const uint32_t sb = mx_scale_byte(block_mag);
            const int col = c0 + hi * 8 + i;
            if (col < n_valid) {
                uint8_t code = 0x7F;
                if (sb != 255u)
                    code = (uint8_t)__nv_cvt_float_to_fp8(hv[i] * __uint_as_float((254u - sb) << 23), __NV_SATFINITE, __NV_E4M3);
                dst[(size_t)col * n_out] = code;
                if ((q & 1) == 0 && j == 0)  // row `col` of the tile: atom col / 128, atom row col % 128
                    sf_dst[(size_t)(col >> 7) * kMxSfAtomBytes + mx_atom_byte(col & 127, 0)] = (uint8_t)sb;
            }
        }
    }
}

// Scale tensor maps (host side): the atom arrays seen as [rows of 512 bytes] of 32-bit words.
bool encode_mx_scale_map(CUtensorMap *map, const void *atoms, uint64_t n_atoms, uint32_t atoms_per_box);

}  // namespace mxtc
}  // namespace moe

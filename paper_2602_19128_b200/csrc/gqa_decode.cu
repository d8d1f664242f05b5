// One decode step of grouped-query attention over a paged key-value cache (paper, Sec. 4.6 "Kernel Analysis: GQA
// Paged Decode"): every batch item has one query token, which attends over the keys and values stored in its pages.
//
// The work is HBM-bound (every cached key and value is read once; 8 flops per byte at a group of 8 query heads), so
// the design is about the stream, not the tensor pipe:
//   * one block per (sequence split, key-value head, batch item); its 4 warps keep the 16 x 128 query tile of the
//     group (Hq / Hkv heads, padded to the MMA's 16 rows) in registers, so a key or value byte is fetched from
//     memory once for all heads of the group (Sec. 4.6 / Table 2: "fusing multiple query heads per KV head");
//   * tokens arrive in chunks of 64 through a three-stage cp.async pipeline of 16-byte copies that follow the page
//     table ("vectorized/async paged-KV gather with pipelined global to shared memory prefetch"); two blocks per SM
//     keep about 128 KiB in flight per SM; rows past the end of the sequence are zero-filled;
//   * each warp owns 16 tokens of a chunk: S = Q K^T (mma.sync m16n8k16, bf16 in, fp32 out: the tile is 16 rows, far
//     too small for a tcgen05 tile, and the kernel is bound by the copy stream), an online softmax in the base-2
//     domain, O += P V with the probabilities re-used from the accumulator registers;
//   * the four warps' (max, sum, O) are merged in shared memory; a split writes its unnormalised result to the
//     workspace, bumps the (item, head) counter, and the block that finds itself last merges the splits and writes
//     out / lse (Sec. 4.6 "Parallelism over the sequence").  A sequence with one active split skips the round trip.
// The merge is a fixed-order sum over splits, so results do not depend on which block arrives last.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "gqa_decode.h"

namespace gqa {
namespace {

constexpr int kD = 128;            // head dimension
constexpr int kRows = 16;          // query heads per block: the MMA's M; groups of up to 16 heads
constexpr int kChunk = 64;         // tokens per pipeline stage
constexpr int kWarps = 4;          // each owns 16 tokens of a chunk
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 3;
constexpr int kRowBytes = kD * 2;  // 256 bytes per token and head
constexpr int kStageBytes = 2 * kChunk * kRowBytes;  // keys, then values: 32 KiB
constexpr int kSmemBytes = kStages * kStageBytes;    // 96 KiB: two blocks per SM
constexpr int kMaxSplits = 64;
constexpr float kLog2e = 1.4426950408889634f;

struct Params {
    const __nv_bfloat16 *q, *k_cache, *v_cache;
    const int *kv_indptr, *kv_indices, *kv_last_page_len;
    __nv_bfloat16 *out;
    float *lse;
    int *counters;     // [B * Hkv], zeroed before the launch
    float *part_ml;    // [B * Hkv, n_splits, group, 2]  (max in the base-2 domain, sum)
    float *part_o;     // [B * Hkv, n_splits, group, D]  unnormalised
    int B, Hq, Hkv, group, page_size, split_tokens, n_splits;
    float scale_log2;  // sm_scale * log2(e)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16 bytes global -> shared, or 16 zero bytes when `valid` is false (src-size 0; the source address is not read).
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid) {
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, f32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Byte offset, inside a 64-token tile of 256-byte rows, of 16-byte piece `piece` of token row `row`: the piece index
// is XOR-ed with the row's low bits so that the eight rows an ldmatrix reads fall into different banks.
__device__ __forceinline__ uint32_t tile_offset(int row, int piece) { return row * kRowBytes + ((piece ^ (row & 7)) << 4); }

__global__ void __launch_bounds__(kThreads, 2) gqa_paged_decode_kernel(const Params p) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ int is_last;
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pages = p.kv_indptr[b + 1] - p.kv_indptr[b];
    const int L = pages > 0 ? (pages - 1) * p.page_size + p.kv_last_page_len[b] : 0;
    const int head0 = kvh * p.group;

    if (L <= 0) {  // nothing cached: out = 0, lse = -inf (written by the first split's block)
        if (split == 0) {
            for (int i = tid; i < p.group * kD; i += kThreads)
                p.out[((size_t)b * p.Hq + head0 + i / kD) * kD + (i % kD)] = __float2bfloat16_rn(0.f);
            if (p.lse && tid < p.group) p.lse[(size_t)b * p.Hq + head0 + tid] = -INFINITY;
        }
        return;
    }
    const int n_active = min(p.n_splits, (L + p.split_tokens - 1) / p.split_tokens);
    if (split >= n_active) return;
    const int begin = split * p.split_tokens;
    const int end = split == n_active - 1 ? L : begin + p.split_tokens;  // the last active split runs to the end
    const int n_chunks = (end - begin + kChunk - 1) / kChunk;

    // ---- the group's queries as MMA A fragments: 8 K-steps of 16 dims, rows = heads (zero beyond the group) ----
    uint32_t qa[kD / 16][4];
    {
        const int r0 = lane >> 2, c0 = (lane & 3) * 2;
        const __nv_bfloat16 *q0 = p.q + ((size_t)b * p.Hq + head0 + r0) * kD;
        const __nv_bfloat16 *q1 = q0 + 8 * kD;
#pragma unroll
        for (int ks = 0; ks < kD / 16; ++ks) {
            const int c = ks * 16 + c0;
            qa[ks][0] = r0 < p.group ? *reinterpret_cast<const uint32_t *>(q0 + c) : 0u;
            qa[ks][1] = r0 + 8 < p.group ? *reinterpret_cast<const uint32_t *>(q1 + c) : 0u;
            qa[ks][2] = r0 < p.group ? *reinterpret_cast<const uint32_t *>(q0 + c + 8) : 0u;
            qa[ks][3] = r0 + 8 < p.group ? *reinterpret_cast<const uint32_t *>(q1 + c + 8) : 0u;
        }
    }

    // ---- the copy pipeline: thread i moves pieces i, i + 128, ... (8 of the keys and 8 of the values per chunk) ----
    const int *page_list = p.kv_indices + p.kv_indptr[b];
    const size_t token_stride = (size_t)p.Hkv * kD;  // elements between consecutive slots of a page
    const uint32_t smem_base = smem_u32(smem);
    auto issue_chunk = [&](int chunk) {
        if (chunk < n_chunks) {
            const uint32_t stage = smem_base + (chunk % kStages) * kStageBytes;
            const int tok0 = begin + chunk * kChunk;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int piece_id = tid + j * kThreads, row = piece_id >> 4, piece = piece_id & 15;
                const int tok = tok0 + row;
                const bool valid = tok < end;
                size_t off = 0;
                if (valid) {
                    const int page = page_list[tok / p.page_size];
                    off = ((size_t)page * p.page_size + (tok % p.page_size)) * token_stride + (size_t)kvh * kD + piece * 8;
                }
                const uint32_t dst = stage + tile_offset(row, piece);
                cp_async_16(dst, p.k_cache + off, valid);
                cp_async_16(dst + kChunk * kRowBytes, p.v_cache + off, valid);
            }
        }
        cp_async_commit();  // (an empty group keeps the wait counts uniform)
    };

    float o_acc[kD / 8][4];  // this warp's 16 x 128 output tile: 16 n-tiles of 8 dims
#pragma unroll
    for (int n = 0; n < kD / 8; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) o_acc[n][i] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows lane/4 and lane/4 + 8

    for (int c = 0; c < kStages - 1; ++c) issue_chunk(c);
    for (int chunk = 0; chunk < n_chunks; ++chunk) {
        cp_async_wait<kStages - 2>();
        __syncthreads();                      // chunk `chunk` has landed for every thread; stage (chunk-1) is free
        issue_chunk(chunk + kStages - 1);
        const uint32_t k_tile = smem_base + (chunk % kStages) * kStageBytes, v_tile = k_tile + kChunk * kRowBytes;
        const int row_base = warp * 16;       // this warp's tokens of the chunk
        const int tok_base = begin + chunk * kChunk + row_base;
        if (tok_base < end) {                 // (uniform over the warp)
            // S = Q K^T for 16 tokens: two n-tiles of 8 tokens, 8 K-steps
            float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            const int m4 = lane >> 3, rr = lane & 7;
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
                uint32_t kb[4];
                ldmatrix_x4(kb, k_tile + tile_offset(row_base + ((m4 >> 1) << 3) + rr, 2 * ks + (m4 & 1)));
                mma_bf16(s[0], qa[ks], kb[0], kb[1]);
                mma_bf16(s[1], qa[ks], kb[2], kb[3]);
            }
            // online softmax in the base-2 domain; columns past the end of the sequence are masked
            float row_max[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int tok = tok_base + n * 8 + (lane & 3) * 2 + (i & 1);
                    s[n][i] = tok < end ? s[n][i] * p.scale_log2 : -INFINITY;
                    row_max[i >> 1] = fmaxf(row_max[i >> 1], s[n][i]);
                }
            float alpha[2];
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                row_max[r] = fmaxf(row_max[r], __shfl_xor_sync(0xffffffffu, row_max[r], 1));
                row_max[r] = fmaxf(row_max[r], __shfl_xor_sync(0xffffffffu, row_max[r], 2));
                const float m_new = fmaxf(m_run[r], row_max[r]);  // finite: the warp's first token is valid
                alpha[r] = exp2f(m_run[r] - m_new);               // 0 on the first chunk (m_run = -inf)
                m_run[r] = m_new;
            }
            float row_sum[2] = {0.f, 0.f};
            uint32_t pa[4];
            {
                float pv[2][4];
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        pv[n][i] = exp2f(s[n][i] - m_run[i >> 1]);
                        row_sum[i >> 1] += pv[n][i];
                    }
                // the probabilities as the A operand of P V: (row, k) and (row, k+8) are n-tiles 0 and 1
                pa[0] = pack_bf16(pv[0][0], pv[0][1]);
                pa[1] = pack_bf16(pv[0][2], pv[0][3]);
                pa[2] = pack_bf16(pv[1][0], pv[1][1]);
                pa[3] = pack_bf16(pv[1][2], pv[1][3]);
            }
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                row_sum[r] += __shfl_xor_sync(0xffffffffu, row_sum[r], 1);
                row_sum[r] += __shfl_xor_sync(0xffffffffu, row_sum[r], 2);
                l_run[r] = l_run[r] * alpha[r] + row_sum[r];
            }
            // O = O * alpha + P V: 16 n-tiles of 8 dims, two per transposed ldmatrix
#pragma unroll
            for (int n = 0; n < kD / 8; n += 2) {
                uint32_t vb[4];
                ldmatrix_x4_trans(vb, v_tile + tile_offset(row_base + ((m4 & 1) << 3) + rr, n + (m4 >> 1)));
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    o_acc[n][i] *= alpha[i >> 1];
                    o_acc[n + 1][i] *= alpha[i >> 1];
                }
                mma_bf16(o_acc[n], pa, vb[0], vb[1]);
                mma_bf16(o_acc[n + 1], pa, vb[2], vb[3]);
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();  // every warp is done with the pipeline's shared memory: it becomes the merge buffer

    // ---- merge the four warps: (max, sum, O) per head, in warp order ----
    float *merge_o = reinterpret_cast<float *>(smem);                    // [4 warps][16 rows][128]
    float *merge_ml = merge_o + kWarps * kRows * kD;                      // [4 warps][16 rows][2]
    {
        const int r0 = lane >> 2, c0 = (lane & 3) * 2;
#pragma unroll
        for (int n = 0; n < kD / 8; ++n) {
            float *dst = merge_o + (warp * kRows + r0) * kD + n * 8 + c0;
            *reinterpret_cast<float2 *>(dst) = make_float2(o_acc[n][0], o_acc[n][1]);
            *reinterpret_cast<float2 *>(dst + 8 * kD) = make_float2(o_acc[n][2], o_acc[n][3]);
        }
        if ((lane & 3) == 0) {
            merge_ml[(warp * kRows + r0) * 2] = m_run[0];
            merge_ml[(warp * kRows + r0) * 2 + 1] = l_run[0];
            merge_ml[(warp * kRows + r0 + 8) * 2] = m_run[1];
            merge_ml[(warp * kRows + r0 + 8) * 2 + 1] = l_run[1];
        }
    }
    __syncthreads();
    const size_t bh = (size_t)b * p.Hkv + kvh;
    float *part_o = p.part_o + (bh * p.n_splits + split) * p.group * kD;
    float *part_ml = p.part_ml + (bh * p.n_splits + split) * p.group * 2;
    for (int i = tid; i < p.group * kD; i += kThreads) {
        const int g = i / kD, d = i - g * kD;
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) m = fmaxf(m, merge_ml[(w * kRows + g) * 2]);
        float l = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float mw = merge_ml[(w * kRows + g) * 2];
            const float f = mw == -INFINITY ? 0.f : exp2f(mw - m);  // a warp without valid tokens contributes nothing
            l += merge_ml[(w * kRows + g) * 2 + 1] * f;
            o += merge_o[(w * kRows + g) * kD + d] * f;
        }
        if (n_active == 1) {  // no other split: finish here
            p.out[((size_t)b * p.Hq + head0 + g) * kD + d] = __float2bfloat16_rn(o / l);
            if (p.lse && d == 0) p.lse[(size_t)b * p.Hq + head0 + g] = (m + log2f(l)) * 0.6931471805599453f;
        } else {
            part_o[i] = o;
            if (d == 0) { part_ml[g * 2] = m; part_ml[g * 2 + 1] = l; }
        }
    }
    if (n_active == 1) return;

    // ---- the block that arrives last merges the splits (Sec. 4.6: "detects that it is last via a lightweight counter") ----
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(&p.counters[bh], 1) == n_active - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const float *all_o = p.part_o + bh * p.n_splits * p.group * kD;
    const float *all_ml = p.part_ml + bh * p.n_splits * p.group * 2;
    for (int i = tid; i < p.group * kD; i += kThreads) {
        const int g = i / kD, d = i - g * kD;
        float m = -INFINITY;
        for (int s = 0; s < n_active; ++s) m = fmaxf(m, __ldcg(&all_ml[(s * p.group + g) * 2]));
        float l = 0.f, o = 0.f;
        for (int s = 0; s < n_active; ++s) {  // ascending split order: the sum is the same whichever block is last
            const float f = exp2f(__ldcg(&all_ml[(s * p.group + g) * 2]) - m);
            l += __ldcg(&all_ml[(s * p.group + g) * 2 + 1]) * f;
            o += __ldcg(&all_o[(size_t)(s * p.group + g) * kD + d]) * f;
        }
        p.out[((size_t)b * p.Hq + head0 + g) * kD + d] = __float2bfloat16_rn(o / l);
        if (p.lse && d == 0) p.lse[(size_t)b * p.Hq + head0 + g] = (m + log2f(l)) * 0.6931471805599453f;
    }
}

bool envelope_ok(long long B, int Hq, int Hkv, int D, long long max_kv_len) {
    if (B < 0 || Hq < 1 || Hkv < 1 || D != kD || max_kv_len < 0) return false;
    if (Hq % Hkv != 0 || Hq / Hkv > kRows) return false;
    return B <= 65535 && Hkv <= 65535;  // grid dimensions y and z
}

// Sequence splits: enough blocks to fill the device a few times over, no split shorter than four chunks.
void choose_split(int B, int Hkv, int max_kv_len, int *split_tokens, int *n_splits) {
    const long long base = (long long)B * Hkv;
    long long want = base > 0 ? (4 * 148 * 2 + base - 1) / base : 1;  // about four waves of two blocks per SM
    const long long most = (max_kv_len + 4 * kChunk - 1) / (4 * kChunk);
    if (want > most) want = most;
    if (want > kMaxSplits) want = kMaxSplits;
    if (want < 1) want = 1;
    long long st = (max_kv_len + want - 1) / want;
    st = (st + kChunk - 1) / kChunk * kChunk;
    if (st < kChunk) st = kChunk;
    long long n = (max_kv_len + st - 1) / st;
    if (n < 1) n = 1;
    *split_tokens = (int)st;
    *n_splits = (int)n;
}

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace
}  // namespace gqa

extern "C" {

size_t gqa_decode_workspace_bytes(int B, int Hq, int Hkv, int D, int max_kv_len) {
    using namespace gqa;
    if (!envelope_ok(B, Hq, Hkv, D, max_kv_len)) return 0;
    int st, ns;
    choose_split(B, Hkv, max_kv_len, &st, &ns);
    const size_t bh = (size_t)B * Hkv, group = Hq / Hkv;
    return align_up(bh * sizeof(int), 256) + align_up(bh * ns * group * 2 * sizeof(float), 256) +
           align_up(bh * ns * group * kD * sizeof(float), 256) + 256;
}

int gqa_decode_split_tokens(int B, int Hq, int Hkv, int D, int max_kv_len) {
    using namespace gqa;
    if (!envelope_ok(B, Hq, Hkv, D, max_kv_len)) return 0;
    int st, ns;
    choose_split(B, Hkv, max_kv_len, &st, &ns);
    return st;
}

int gqa_paged_decode(const void *q, const void *k_cache, const void *v_cache, const int32_t *kv_indptr,
                     const int32_t *kv_indices, const int32_t *kv_last_page_len, int B, int Hq, int Hkv, int D,
                     int page_size, int num_pages, int max_kv_len, float sm_scale, void *out, float *lse, void *workspace,
                     size_t workspace_bytes, void *stream) {
    using namespace gqa;
    if (B < 0 || Hq < 1 || Hkv < 1 || D < 1 || page_size < 1 || num_pages < 0 || max_kv_len < 0) return MOE_ERR_SHAPE;
    if (!envelope_ok(B, Hq, Hkv, D, max_kv_len)) return MOE_ERR_UNSUPPORTED;
    if (B == 0) return MOE_OK;
    if (!q || !k_cache || !v_cache || !kv_indptr || !kv_indices || !kv_last_page_len || !out || !workspace) return MOE_ERR_NULL;
    auto misaligned = [](const void *ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) != 0; };
    if (misaligned(q, 16) || misaligned(k_cache, 16) || misaligned(v_cache, 16) || misaligned(out, 16) ||
        misaligned(kv_indptr, 4) || misaligned(kv_indices, 4) || misaligned(kv_last_page_len, 4) || misaligned(lse, 4) ||
        misaligned(workspace, 256))
        return MOE_ERR_ALIGN;
    if (workspace_bytes < gqa_decode_workspace_bytes(B, Hq, Hkv, D, max_kv_len)) return MOE_ERR_WORKSPACE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (major != 10) return MOE_ERR_ARCH;

    Params p;
    p.q = static_cast<const __nv_bfloat16 *>(q);
    p.k_cache = static_cast<const __nv_bfloat16 *>(k_cache);
    p.v_cache = static_cast<const __nv_bfloat16 *>(v_cache);
    p.kv_indptr = kv_indptr;
    p.kv_indices = kv_indices;
    p.kv_last_page_len = kv_last_page_len;
    p.out = static_cast<__nv_bfloat16 *>(out);
    p.lse = lse;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.group = Hq / Hkv; p.page_size = page_size;
    choose_split(B, Hkv, max_kv_len, &p.split_tokens, &p.n_splits);
    p.scale_log2 = sm_scale * kLog2e;
    const size_t bh = (size_t)B * Hkv;
    char *ws = static_cast<char *>(workspace);
    p.counters = reinterpret_cast<int *>(ws);
    ws += align_up(bh * sizeof(int), 256);
    p.part_ml = reinterpret_cast<float *>(ws);
    ws += align_up(bh * p.n_splits * p.group * 2 * sizeof(float), 256);
    p.part_o = reinterpret_cast<float *>(ws);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(p.counters, 0, bh * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
    static bool attr_set[64];
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(gqa_paged_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess)
            return MOE_ERR_CUDA;
        attr_set[dev] = true;
    }
    gqa_paged_decode_kernel<<<dim3(p.n_splits, Hkv, B), kThreads, kSmemBytes, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // extern "C"

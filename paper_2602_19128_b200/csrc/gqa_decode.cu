// One decode step of grouped-query attention over a paged key-value cache (paper, Sec. 4.6 "Kernel Analysis: GQA
// Paged Decode"): every batch item has one query token, which attends over the keys and values stored in its pages.
//
// The work is HBM-bound (every cached key and value is read once; 8 flops per byte at a group of 8 query heads), so
// the design is about the stream, not the tensor pipe:
//   * one block per (sequence split, key-value head, batch item); its 4 warps keep the 16 x 128 query tile of the
//     group (Hq / Hkv heads, padded to the MMA's 16 rows) in registers, so a key or value byte is fetched from
//     memory once for all heads of the group (Sec. 4.6 / Table 2: "fusing multiple query heads per KV head");
//   * tokens arrive in chunks of 64 through a pipeline of TMA copies that follow the page table and complete on the
//     stage's mbarrier ("vectorized/async paged-KV gather with pipelined global to shared memory prefetch").  Page
//     sizes that are powers of two of at least 8 take the TILED gather: the cache is a 5-D tensor (64 dims, slot,
//     half of the dims, head, page) and one `cp.async.bulk.tensor` box brings a page's slots (up to 64) of one head
//     as two 128-byte-swizzled blocks, so a chunk of 16-token pages is eight boxes.  A fifth warp issues them and
//     does nothing else, three stages deep, two blocks per SM; full / empty mbarriers hand the stages back and
//     forth, and the compute warps' loop has no block-wide barrier.  Other page sizes take the ROW gather, one
//     256-byte `cp.async.bulk` per token row and compute thread into rows padded to 272 bytes, two stages in three
//     blocks per SM.  What was measured on the way, B = 64 x 16k tokens: sixteen 16-byte cp.async per thread and
//     chunk, 4.0 TB/s (800 instructions per warp and chunk, instruction-latency bound at 8 warps per SM); the row
//     gather 4.0 TB/s with and 5.2 TB/s without the arithmetic, one 256-byte request per 14 cycles and SM being all
//     the copy engine took; the tiled gather with one compute warp issuing 6.1 TB/s, with the boxes dealt out to
//     the four compute warps 6.3 TB/s (a thread is held 5 to 9 cycles per 128-byte row of a box it issues), with
//     the copy warp 6.6-6.9 TB/s, the measured copy bandwidth;
//   * each warp owns 16 tokens of a chunk: S = Q K^T (mma.sync m16n8k16, bf16 in, fp32 out: the tile is 16 rows, far
//     too small for a tcgen05 tile, and the kernel is bound by the copy stream), an online softmax in the base-2
//     domain, O += P V with the probabilities re-used from the accumulator registers;
//   * the four warps' (max, sum, O) are merged in shared memory; a split writes its unnormalised result to the
//     workspace, bumps the (item, head) counter, and the block that finds itself last merges the splits and writes
//     out / lse (Sec. 4.6 "Parallelism over the sequence").  A sequence with one active split skips the round trip.
// The merge is a fixed-order sum over splits, so results do not depend on which block arrives last.
// Every wait on a stage's barrier is bounded: a block that gives up records MOE_ERR_DEVICE_TIMEOUT in the
// workspace's status word (read it with moe_last_status) and leaves without writing a result.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include "gqa_decode.h"

namespace moe {
namespace tc {
// (moe_tc_host.cu) 5-D bf16 tensor map of a paged cache [num_pages, page_size, Hkv, 128], dimensions ordered (64
// dims, slot, half of the dims, head, page): box = 64 dims x box_rows slots x both halves of one head of one page,
// 128-byte swizzle; encoded through the driver entry point and cached.
bool encode_kv_cache_map(CUtensorMap *map, const void *cache, uint64_t num_pages, uint32_t page_size, uint32_t Hkv,
                         uint32_t box_rows);
// (moe_tc_host.cu) cudaFuncAttributeMaxDynamicSharedMemorySize, set once per kernel and device, under a mutex.
bool set_max_dynamic_smem_once(const void *kernel, int bytes);
}  // namespace tc
// (moe_api.cu) MOE_OK when the current device has compute capability 10.x (cached per device), else an error code.
int check_device();
}  // namespace moe

namespace gqa {
namespace {

constexpr int kD = 128;            // head dimension
constexpr int kRows = 16;          // query heads per block: the MMA's M; groups of up to 16 heads
constexpr int kChunk = 64;         // tokens per pipeline stage
constexpr int kWarps = 4;          // each owns 16 tokens of a chunk
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 2;         // one chunk in flight while the previous one is used ...
constexpr int kBlocksPerSm = 3;    // ... in each of three blocks per SM (168 registers per thread, 69 KiB each)
constexpr int kRowBytes = kD * 2;  // 256 bytes per token and head in the cache
// Two layouts of a 64-token tile in shared memory, one per gather mode, inside the same 17 KiB:
//   tiled: one block per TMA box, [64 / box_rows boxes][2 halves of the dims][box_rows rows][128 bytes], each half
//          block in TMA's 128-byte swizzle (16 KiB);
//   rows:  [64 rows][272 bytes], the 16 bytes of padding keeping ldmatrix free of bank conflicts.
constexpr int kRowPitch = kRowBytes + 16;
constexpr int kTileBytes = kChunk * kRowPitch;        // 17 KiB, a multiple of 1024 (the swizzle's alignment)
constexpr int kStageBytes = 2 * kTileBytes;           // keys, then values: 34 KiB
constexpr int kModelBlocksPerSm = 2;  // blocks per SM the split model counts with (the copy-warp variant's)
constexpr int kStagesProducer = 3;  // the variant with a copy warp: three stages in each of two blocks per SM
constexpr int kSmemBytes = kStages * kStageBytes + 1024;  // (the base is rounded up to 1024 bytes)
constexpr int kSmemBytesProducer = kStagesProducer * kStageBytes + 1024;
static_assert(kTileBytes % 1024 == 0, "tiles must keep the swizzle's alignment");
constexpr int kWaitLimit = 1 << 22;                   // polls of a stage's barrier before the block gives up
constexpr int kMaxSplits = 128;
constexpr float kLog2e = 1.4426950408889634f;

struct Params {
    const __nv_bfloat16 *q, *k_cache, *v_cache;
    const int *kv_indptr, *kv_indices, *kv_last_page_len;
    __nv_bfloat16 *out;
    float *lse;
    int *status;       // the workspace's status word, zeroed before the launch
    int *counters;     // [B * Hkv], zeroed before the launch
    float *part_ml;    // [B * Hkv, n_splits, group, 2]  (max in the base-2 domain, sum)
    float *part_o;     // [B * Hkv, n_splits, group, D]  unnormalised
    int B, Hq, Hkv, group, page_size, split_tokens, n_splits;
    int box_rows;      // tiled gather: token rows one TMA box brings (min(page_size, 64))
    float scale_log2;  // sm_scale * log2(e)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}
// One bulk copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) that completes on an mbarrier.
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// One box of the cache's 5-D tensor map -- coordinates (dim 0, slot, half 0, head, page): the innermost is always 0 --
// that completes on an mbarrier.
__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap *map, int slot, int head, int page, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(0), "r"(slot), "r"(0), "r"(head), "r"(page), "r"(bar) : "memory");
}

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

// Bounded wait on an mbarrier: false once `limit` polls have passed (the status word then says so: the call's first
// expired wait records MOE_ERR_DEVICE_TIMEOUT, site 12 and the block) or once another thread of the block has given up.
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, int limit, volatile int *gave_up, int *status) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*gave_up) return false;
    }
    *gave_up = 1;
    if (atomicCAS(status, 0, (int)MOE_ERR_DEVICE_TIMEOUT) == 0) { status[1] = 12; status[2] = blockIdx.x; }
    return false;
}

// Self-test of that error path: one warp waits, with a small bound, on a barrier at which nothing arrives.
__global__ void gqa_wait_timeout_selftest_kernel(int *status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int gave_up;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    bounded_wait(smem_u32(&bar), 0, 1 << 14, &gave_up, status);
}

// Byte offset, inside a 64-token tile, of 16-byte piece `piece` (0..15) of token row `row`.
// `sh` = log2(box_rows) (tiled only).
template <bool kTiled>
__device__ __forceinline__ uint32_t tile_offset(int row, int piece, int sh) {
    if (kTiled)
        return ((row >> sh) << (sh + 8)) + ((piece >> 3) << (sh + 7)) + ((row & ((1 << sh) - 1)) << 7) +
               (((piece & 7) ^ (row & 7)) << 4);
    return row * kRowPitch + (piece << 4);
}

// kTiled: the page size is a power of two of at least 8, and the gather is one TMA box per (page, keys or values),
// issued by a fifth warp that does nothing else, three stages deep, in two blocks per SM: the four compute warps never
// touch the copy engine, and stages are handed back and forth on full / empty mbarriers, so the loop has no block-wide
// barrier.  (A thread is held for as long as the engine takes to turn its box into requests, 5 to 9 cycles per
// 128-byte row: 600 cycles per chunk and warp when the four compute warps shared the issuing, against 1000 for the
// arithmetic.)  Otherwise: one 256-byte bulk copy per token row, issued by the 128 compute threads themselves, two
// stages in three blocks per SM, a block barrier per chunk.
template <bool kTiled>
__global__ void __launch_bounds__(kTiled ? kThreads + 32 : kThreads, kTiled ? 2 : kBlocksPerSm)
gqa_paged_decode_kernel(const Params p, const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map) {
    constexpr bool kProducer = kTiled;  // a copy warp
    constexpr int kNumStages = kProducer ? kStagesProducer : kStages;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    uint8_t *smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    __shared__ int is_last, gave_up;
    __shared__ __align__(8) unsigned long long full_bar[kStagesProducer], empty_bar[kStagesProducer];
    // the compute warps' barrier: the whole block without a copy warp, a named barrier of 128 threads with one
    auto sync_compute = [&]() {
        if (kProducer) asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory");
        else __syncthreads();
    };
    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pages = p.kv_indptr[b + 1] - p.kv_indptr[b];
    const int L = pages > 0 ? (pages - 1) * p.page_size + p.kv_last_page_len[b] : 0;
    const int head0 = kvh * p.group;

    if (L <= 0) {  // nothing cached: out = 0, lse = -inf (written by the first split's block)
        if (split == 0 && tid < kThreads) {
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

    // ---- the copy pipeline ----
    // tiled: a chunk is 128 / box_rows boxes -- (page of the chunk, keys or values), both halves of the dims in one box
    //        -- one per lane of the copy warp, which alone arrives on the stage's barrier;
    // rows:  thread i brings ONE token row per chunk -- row i % 64 of the keys (i < 64) or of the values.
    //        Every thread arrives on the stage's barrier once per chunk, with its bytes when its row exists.
    const int *page_list = p.kv_indices + p.kv_indptr[b];
    const size_t token_stride = (size_t)p.Hkv * kD;  // elements between consecutive slots of a page
    const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(full_bar);
    const int sh = 31 - __clz(p.box_rows);                              // (tiled) log2 of the rows of a box
    const int n_boxes = 2 * kChunk >> sh;                               // 2 (64-row boxes) .. 16 (8-row boxes)
    const int my_box = lane;                                            // tiled: page my_box / 2 of the chunk, values?
    const int my_row = kTiled ? (my_box >> 1) << sh : (tid & (kChunk - 1));  // first row of the box / the row
    const bool my_values = kTiled ? (my_box & 1) : (tid >= kChunk);
    const __nv_bfloat16 *my_cache = (my_values ? p.v_cache : p.k_cache) + (size_t)kvh * kD;
    const uint32_t my_dst = (my_values ? (uint32_t)kTileBytes : 0u) +
                            (kTiled ? (uint32_t)(my_row * kRowBytes) : (uint32_t)(my_row * kRowPitch));
    const bool has_box = kTiled ? (warp == kWarps && my_box < n_boxes) : true;
    const uint32_t empty_base = smem_u32(empty_bar);
    if (tid == 0) {
        for (int s = 0; s < kNumStages; ++s) {
            mbar_init(bar_base + s * 8, kProducer ? 32 : kThreads);  // arrivals per chunk: the copy warp's lanes / every thread
            mbar_init(empty_base + s * 8, kWarps);                    // (copy-warp variant) one arrival per compute warp
        }
        gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Where this thread's row (rows: its slot in the cache; tiled: its page) of a chunk lives, -1 past the end of the
    // split.  The page table is read ONE CHUNK AHEAD of the copy that needs it, so its latency never sits between copies.
    auto locate = [&](int chunk) -> int {
        const int tok = begin + chunk * kChunk + my_row;
        if (!has_box || chunk >= n_chunks || tok >= end) return -1;
        const int page = __ldg(&page_list[tok / p.page_size]);
        return kTiled ? page : page * p.page_size + tok % p.page_size;
    };
    int next_loc = locate(0);
    auto issue_chunk = [&](int chunk) {  // called for chunk 0, 1, 2, ... in order
        if (chunk < n_chunks) {
            const int stage = chunk % kNumStages;
            const uint32_t dst = smem_base + stage * kStageBytes + my_dst, bar = bar_base + stage * 8;
            if (kTiled) {
                if (next_loc >= 0) {
                    mbar_arrive_expect_tx(bar, p.box_rows * kRowBytes);
                    tma_load_box(dst, my_values ? &v_map : &k_map, (begin + chunk * kChunk + my_row) & (p.page_size - 1), kvh,
                                 next_loc, bar);
                } else {
                    mbar_arrive(bar);
                }
            } else if (next_loc >= 0) {
                mbar_arrive_expect_tx(bar, kRowBytes);
                bulk_copy(dst, my_cache + (size_t)next_loc * token_stride, kRowBytes, bar);
            } else {  // a row past the end: zeros, so that a masked probability of 0 meets a finite value
#pragma unroll
                for (int i = 0; i < kRowBytes / 16; ++i)
                    asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst + i * 16), "r"(0) : "memory");
                mbar_arrive(bar);
            }
        }
        next_loc = locate(chunk + 1);
    };
    auto wait_bar = [&](uint32_t bar, uint32_t parity) -> bool {
        return bounded_wait(bar, parity, kWaitLimit, &gave_up, p.status);
    };
    auto wait_chunk = [&](int chunk) -> bool {
        return wait_bar(bar_base + (chunk % kNumStages) * 8, (uint32_t)(chunk / kNumStages) & 1u);
    };

    if (kProducer && warp == kWarps) {
        // ---- the copy warp: chunk after chunk into the ring, each stage as soon as the four compute warps are done
        // with its previous use ----
        for (int chunk = 0; chunk < n_chunks; ++chunk) {
            const int use = chunk / kNumStages;
            bool free_ = use == 0 || wait_bar(empty_base + (chunk % kNumStages) * 8, (uint32_t)(use - 1) & 1u);
            if (!__all_sync(0xffffffffu, free_)) break;
            issue_chunk(chunk);
        }
        return;
    }

    float o_acc[kD / 8][4];  // this warp's 16 x 128 output tile: 16 n-tiles of 8 dims
#pragma unroll
    for (int n = 0; n < kD / 8; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i) o_acc[n][i] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};  // rows lane/4 and lane/4 + 8

    if (!kProducer)
        for (int c = 0; c < kNumStages - 1; ++c) issue_chunk(c);
    bool ok = true;
    for (int chunk = 0; chunk < n_chunks; ++chunk) {
        ok = wait_chunk(chunk);
        if (kProducer) {
            ok = __all_sync(0xffffffffu, ok);     // chunk `chunk` has landed
            if (!ok) break;
        } else {
            ok = __syncthreads_and(ok);           // ... and every thread is done with chunk - 1's stage
            if (!ok) break;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // (that stage is about to be overwritten by copies)
            issue_chunk(chunk + kNumStages - 1);
        }
        const uint32_t k_tile = smem_base + (chunk % kNumStages) * kStageBytes, v_tile = k_tile + kTileBytes;
        const int row_base = warp * 16;       // this warp's tokens of the chunk
        const int tok_base = begin + chunk * kChunk + row_base;
        if (tok_base < end) {                 // (uniform over the warp)
            if (kTiled && tok_base + 16 > end) {
                // A box brings whole pages: value rows past the end of the sequence hold whatever the cache holds there
                // (and rows of pages that were not fetched, whatever the stage held).  Zero them, so that a masked
                // probability of 0 meets a finite value.  The rows are this warp's own.
                const int valid = end - tok_base;  // 1..15
                for (int i = lane; i < 16 * 16; i += 32) {
                    const int r = i >> 4;
                    if (r >= valid)
                        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};"
                                     ::"r"(v_tile + tile_offset<true>(row_base + r, i & 15, sh)), "r"(0) : "memory");
                }
                __syncwarp();
            }
            // S = Q K^T for 16 tokens: two n-tiles of 8 tokens, 8 K-steps.  A warp is one of one to three on its
            // scheduler, so the latency of its own chain is what counts: fragments are fetched two steps ahead of the
            // MMAs that use them, and even and odd K-steps accumulate separately (chains of four instead of eight).
            float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            float s_odd[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            const int m4 = lane >> 3, rr = lane & 7;
            const int k_row = row_base + ((m4 >> 1) << 3) + rr, v_row = row_base + ((m4 & 1) << 3) + rr;
            constexpr int kAhead = 2;
            uint32_t kb[kAhead + 1][4];
#pragma unroll
            for (int ks = 0; ks < kAhead; ++ks) ldmatrix_x4(kb[ks], k_tile + tile_offset<kTiled>(k_row, 2 * ks + (m4 & 1), sh));
#pragma unroll
            for (int ks = 0; ks < kD / 16; ++ks) {
                if (ks + kAhead < kD / 16)
                    ldmatrix_x4(kb[(ks + kAhead) % (kAhead + 1)], k_tile + tile_offset<kTiled>(k_row, 2 * (ks + kAhead) + (m4 & 1), sh));
                const uint32_t(&f)[4] = kb[ks % (kAhead + 1)];
                if (ks & 1) {
                    mma_bf16(s_odd[0], qa[ks], f[0], f[1]);
                    mma_bf16(s_odd[1], qa[ks], f[2], f[3]);
                } else {
                    mma_bf16(s[0], qa[ks], f[0], f[1]);
                    mma_bf16(s[1], qa[ks], f[2], f[3]);
                }
            }
            // the first value fragments are on their way while the softmax runs
            uint32_t vb[kAhead + 1][4];
#pragma unroll
            for (int j = 0; j < kAhead; ++j) ldmatrix_x4_trans(vb[j], v_tile + tile_offset<kTiled>(v_row, 2 * j + (m4 >> 1), sh));
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) s[n][i] += s_odd[n][i];
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
            // O = O * alpha + P V: 16 n-tiles of 8 dims, two per transposed ldmatrix.  Once the running maxima have
            // settled alpha is exactly 1 for every row, and the 64 multiplications are skipped (same result).
            if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
                for (int n = 0; n < kD / 8; ++n)
#pragma unroll
                    for (int i = 0; i < 4; ++i) o_acc[n][i] *= alpha[i >> 1];
            }
#pragma unroll
            for (int j = 0; j < kD / 16; ++j) {  // n-tiles 2j and 2j + 1
                if (j + kAhead < kD / 16)
                    ldmatrix_x4_trans(vb[(j + kAhead) % (kAhead + 1)], v_tile + tile_offset<kTiled>(v_row, 2 * (j + kAhead) + (m4 >> 1), sh));
                const uint32_t(&f)[4] = vb[j % (kAhead + 1)];
                mma_bf16(o_acc[2 * j], pa, f[0], f[1]);
                mma_bf16(o_acc[2 * j + 1], pa, f[2], f[3]);
            }
        }
        if (kProducer) {  // this warp is done with the stage (also when none of its tokens exist)
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_base + (chunk % kNumStages) * 8);
        }
    }
    // every warp is done with the pipeline's shared memory (all copies were waited for): it becomes the merge buffer
    if (kProducer) {
        sync_compute();
        ok = *(volatile int *)&gave_up == 0;
    }
    // A block that gave up waits (bounded) for its copies in flight, then leaves without a result: the status word says so.
    if (!ok) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        return;
    }
    if (!kProducer) __syncthreads();

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
    sync_compute();
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
    sync_compute();
    if (tid == 0) is_last = atomicAdd(&p.counters[bh], 1) == n_active - 1;
    sync_compute();
    if (!is_last) return;
    __threadfence();
    const float *all_o = p.part_o + bh * p.n_splits * p.group * kD;
    const float *all_ml = p.part_ml + bh * p.n_splits * p.group * 2;
    // The merge is a chain of round trips to L2 for one block, so every step is laid out for loads in flight: the
    // (max, sum) pairs of all splits come to shared memory in one sweep, the scale factors are computed from there,
    // and the sum over the splits runs over all of a thread's outputs at once, eight splits deep.
    float2 *ml = reinterpret_cast<float2 *>(smem);                       // [n_active][group] (max, sum)
    float *scale = reinterpret_cast<float *>(ml + kMaxSplits * kRows);   // [n_active][group]
    float *head_m = scale + kMaxSplits * kRows;                          // [16]
    float *head_l = head_m + kRows;                                      // [16]
    sync_compute();                                                     // (the warps' merge buffer is free again)
    for (int i = tid; i < n_active * p.group; i += kThreads) ml[i] = __ldcg(reinterpret_cast<const float2 *>(all_ml) + i);
    sync_compute();
    if (tid < p.group) {
        float m = -INFINITY;
        for (int s = 0; s < n_active; ++s) m = fmaxf(m, ml[s * p.group + tid].x);
        head_m[tid] = m;
    }
    sync_compute();
    for (int i = tid; i < n_active * p.group; i += kThreads) scale[i] = exp2f(ml[i].x - head_m[i % p.group]);
    sync_compute();
    if (tid < p.group) {
        float l = 0.f;
        for (int s = 0; s < n_active; ++s) l += ml[s * p.group + tid].y * scale[s * p.group + tid];  // ascending splits
        head_l[tid] = l;
        if (p.lse) p.lse[(size_t)b * p.Hq + head0 + tid] = (head_m[tid] + log2f(l)) * 0.6931471805599453f;
    }
    sync_compute();
    // thread t owns (head, four dims) items t, t + 128, ...: at most four (16 heads x 32 groups of four dims)
    constexpr int kItems = kRows * (kD / 4) / kThreads;
    const int n_items = p.group * (kD / 4);
    float4 o[kItems];
#pragma unroll
    for (int j = 0; j < kItems; ++j) o[j] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
    for (int s = 0; s < n_active; ++s) {  // ascending split order: the sum is the same whichever block is last
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            const int i = tid + j * kThreads;
            if (i < n_items) {
                const int g = i / (kD / 4), d = (i - g * (kD / 4)) * 4;
                const float4 v = __ldcg(reinterpret_cast<const float4 *>(&all_o[(size_t)(s * p.group + g) * kD + d]));
                const float f = scale[s * p.group + g];
                o[j].x += v.x * f; o[j].y += v.y * f; o[j].z += v.z * f; o[j].w += v.w * f;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < kItems; ++j) {
        const int i = tid + j * kThreads;
        if (i >= n_items) break;
        const int g = i / (kD / 4), d = (i - g * (kD / 4)) * 4;
        const float l = head_l[g];
        __nv_bfloat162 lo = __floats2bfloat162_rn(o[j].x / l, o[j].y / l), hi = __floats2bfloat162_rn(o[j].z / l, o[j].w / l);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t *>(&lo);
        packed.y = *reinterpret_cast<uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(&p.out[((size_t)b * p.Hq + head0 + g) * kD + d]) = packed;
    }
}

bool envelope_ok(long long B, int Hq, int Hkv, int D, long long max_kv_len) {
    if (B < 0 || Hq < 1 || Hkv < 1 || D != kD || max_kv_len < 0) return false;
    if (Hq % Hkv != 0 || Hq / Hkv > kRows) return false;
    return B <= 65535 && Hkv <= 65535;  // grid dimensions y and z
}

// Sequence splits, from a model of the kernel's time in units of one chunk streamed by a block on a full machine
// (1.4 us).  148 SMs x 2 blocks are resident at a time (the copy-warp variant), so blocks run in waves; a block costs
// its chunks plus 3 (pipeline fill, the warps' merge); a wave that fills a fraction f of the machine runs in
// max(0.47, f) of a full wave's time (a block alone streams a chunk in 0.47 of the time, and 0.86 of a wave already
// saturates the memory); a split sequence pays the partial results' round trip and the last block's merge once,
// 5 + n / 10; and while the machine is not full, 0.3 x (the idle share) of a block's length is added for the tail that
// sequences shorter than max_kv_len leave (their lengths are known to the device only; on a full machine the blocks
// that remain speed up as others finish, on a part-empty one they already run at their own limit).  The constants
// were fitted to measured split sweeps (batches of 1 to 256, 2k to 64k tokens, equal and ragged lengths); the chosen
// count was within 10 % of the best measured one in each.  Ties go to fewer splits; no split is shorter than four
// chunks.
void choose_split(int B, int Hkv, int max_kv_len, int *split_tokens, int *n_splits) {
    const long long base = (long long)B * Hkv, slots = 148 * kModelBlocksPerSm;
    const long long chunks = max_kv_len > 0 ? ((long long)max_kv_len + kChunk - 1) / kChunk : 1;
    long long most = (chunks + 3) / 4;
    if (most > kMaxSplits) most = kMaxSplits;
    if (most < 1) most = 1;
    long long best_n = 1;
    double best_cost = -1.0;
    for (long long n = 1; n <= most; ++n) {
        const long long per_block = (chunks + n - 1) / n, n_eff = (chunks + per_block - 1) / per_block;
        if (n_eff != n) continue;  // (the same split as a smaller n)
        const long long blocks = (base > 0 ? base : 1) * n, full_waves = blocks / slots;
        const double f = (double)(blocks - full_waves * slots) / (double)slots;
        const double last_wave = f > 0.0 ? (f > 0.47 ? f : 0.47) : 0.0;
        const double idle = blocks < slots ? 1.0 - (double)blocks / (double)slots : 0.0;
        const double cost = ((double)per_block + 3.0) * ((double)full_waves + last_wave) +
                            0.3 * idle * (double)per_block + (n > 1 ? 5.0 + 0.1 * (double)n : 0.0);
        if (best_cost < 0 || cost < best_cost * (1.0 - 1e-9)) { best_cost = cost; best_n = n; }
    }
    const long long per_block = (chunks + best_n - 1) / best_n;
    *split_tokens = (int)(per_block * kChunk);
    *n_splits = (int)((chunks + per_block - 1) / per_block);
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
    return 256 + align_up(bh * sizeof(int), 256) + align_up(bh * ns * group * 2 * sizeof(float), 256) +
           align_up(bh * ns * group * kD * sizeof(float), 256) + 256;
}

int gqa_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream) {
    using namespace gqa;
    if (!workspace) return MOE_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return MOE_ERR_ALIGN;
    if (workspace_bytes < 256) return MOE_ERR_WORKSPACE;
    const int arch = moe::check_device();
    if (arch != MOE_OK) return arch;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) return MOE_ERR_CUDA;
    gqa_wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(static_cast<int *>(workspace));
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
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
    if ((long long)num_pages * page_size >= (1ll << 31)) return MOE_ERR_UNSUPPORTED;  // slot numbers are 32-bit
    if (B == 0) return MOE_OK;
    if (!q || !k_cache || !v_cache || !kv_indptr || !kv_indices || !kv_last_page_len || !out || !workspace) return MOE_ERR_NULL;
    auto misaligned = [](const void *ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) != 0; };
    if (misaligned(q, 16) || misaligned(k_cache, 16) || misaligned(v_cache, 16) || misaligned(out, 16) ||
        misaligned(kv_indptr, 4) || misaligned(kv_indices, 4) || misaligned(kv_last_page_len, 4) || misaligned(lse, 4) ||
        misaligned(workspace, 256))
        return MOE_ERR_ALIGN;
    if (workspace_bytes < gqa_decode_workspace_bytes(B, Hq, Hkv, D, max_kv_len)) return MOE_ERR_WORKSPACE;
    const int arch = moe::check_device();
    if (arch != MOE_OK) return arch;

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
    p.status = reinterpret_cast<int *>(ws);  // status word first, as in the layer's workspace: moe_last_status reads it
    p.counters = reinterpret_cast<int *>(ws + 256);
    ws += 256 + align_up(bh * sizeof(int), 256);
    p.part_ml = reinterpret_cast<float *>(ws);
    ws += align_up(bh * p.n_splits * p.group * 2 * sizeof(float), 256);
    p.part_o = reinterpret_cast<float *>(ws);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(p.status, 0, 256 + bh * sizeof(int), st) != cudaSuccess) return MOE_ERR_CUDA;
    if (!moe::tc::set_max_dynamic_smem_once(reinterpret_cast<const void *>(gqa_paged_decode_kernel<true>), kSmemBytesProducer) ||
        !moe::tc::set_max_dynamic_smem_once(reinterpret_cast<const void *>(gqa_paged_decode_kernel<false>), kSmemBytes))
        return MOE_ERR_CUDA;
    // Page sizes that are powers of two of at least 8 take the tiled gather: one 5-D tensor map per cache,
    // (64 dims, slot, half, head, page), a box of min(page_size, 64) slots x both halves in the 128-byte swizzle.
    const bool tiled = page_size >= 8 && (page_size & (page_size - 1)) == 0 && num_pages > 0;
    CUtensorMap k_map, v_map;
    memset(&k_map, 0, sizeof(k_map));
    memset(&v_map, 0, sizeof(v_map));
    p.box_rows = page_size < kChunk ? page_size : kChunk;
    if (tiled && (!moe::tc::encode_kv_cache_map(&k_map, k_cache, (uint64_t)num_pages, (uint32_t)page_size, (uint32_t)Hkv, (uint32_t)p.box_rows) ||
                  !moe::tc::encode_kv_cache_map(&v_map, v_cache, (uint64_t)num_pages, (uint32_t)page_size, (uint32_t)Hkv, (uint32_t)p.box_rows)))
        return MOE_ERR_CUDA;
    const dim3 grid(p.n_splits, Hkv, B);
    if (tiled) gqa_paged_decode_kernel<true><<<grid, kThreads + 32, kSmemBytesProducer, st>>>(p, k_map, v_map);
    else gqa_paged_decode_kernel<false><<<grid, kThreads, kSmemBytes, st>>>(p, k_map, v_map);
    return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

}  // extern "C"

// Device-side PTX wrappers, descriptors and the tile schedule decoder shared by the tcgen05 grouped-GEMM
// kernels (bf16, FP8-dequantising and MX FP8; one CTA per tile and CTA pairs), plus the host-side tensor-map
// encoders.
#pragma once

#include "moe_internal.cuh"

namespace moe {
namespace tc {

constexpr int kBlockK = 64;                        // K elements per ring slot = one 128-byte swizzle row
constexpr int kTileM = 128;                        // weight rows per CTA (MMA M per CTA)
constexpr int kSlotABytes = kTileM * kBlockK * 2;  // 16 KiB
constexpr int kRowBytes = kBlockK * 2;             // 128
constexpr int kThreads = 192;                      // warp 0 TMA, warp 1 MMA, warps 2..5 epilogue
constexpr int kEpilogueWarps = 4;
constexpr long long kWaitLimitCycles = 4000000000LL;  // about two seconds at full clock
constexpr uint32_t kWaitSuspendNs = 20000;            // upper bound of one hardware-suspended wait
constexpr int kNumActMaps = 16;                    // activation boxes of q, 2q, ..., 16q rows (q = 16, or 8 for pairs)

// Tensor maps of one grouped GEMM.  `w` is either a 2-D map over [E*w_rows, K] with a 128-row box
// (down projection) or a 5-D map over w13 viewed as [E][I/16][gate|up][16][H] whose
// {64,16,2,4,1} box delivers 64 features as 4 x (16 gate rows, 16 up rows) in one copy.
struct TensorMaps {
    CUtensorMap w;
    CUtensorMap act[kNumActMaps];  // act[i]: box of q * (i + 1) rows, so any token tile is ONE copy
};

struct KernelParams {
    __nv_bfloat16 *out;
    const int *expert_offsets, *tile_prefix, *tile_order, *tile_rows;
    int *status;
    int E, n_k_blocks, n_out, w_rows, n_feature_tiles;
    const float *w_scale;  // FP8-weight kernels only: [E, w_rows/128, K/128] block scales
    int handover_role;     // hand-over between the two GEMMs of a call (moe_internal.cuh)
    int *handover;
    int handover_per_token_tile;
    // gather-in-load (wide-tile gate/up GEMM only): token rows are fetched from the layer's input by row index
    int gather_tokens = 0;
    const int *sorted_to_flat = nullptr;
    int top_k = 1;
};

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done != 0;
}
// The same test, but the thread may be suspended by the hardware for up to `hint_ns` (it is woken
// when the phase completes), so a long wait costs neither issue slots nor power.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return done != 0;
}
// Bounded wait.  Returns false if the CTA is aborting (this wait expired, or another role's did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          int site) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long start = clock64();
    while (true) {
        if (mbar_try_wait_suspend(bar, parity, kWaitSuspendNs)) {
            return true;
        }
        if (*abort_flag) return false;
        if (clock64() - start > kWaitLimitCycles) {
            *abort_flag = 1;
            if (atomicCAS(status, 0, (int)MOE_ERR_DEVICE_TIMEOUT) == 0) {
                status[1] = site;
                status[2] = blockIdx.x;
            }
            return false;
        }
    }
}

// True in exactly one lane of a converged warp, always the same lane.  The role loops are run by
// whole warps and only the issuing instructions sit under this predicate: loop state then stays
// warp-uniform and the descriptors of TMA / tcgen05 instructions (which take uniform-register
// operands) need no per-instruction transfer.  Measured: with a single lane running the whole loop
// under `lane == 0`, every TMA or MMA instruction cost about 150 cycles to issue.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// Bounded wait by a whole warp; the result is made uniform.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                               int site) {
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, status, site));
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            int c4, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_load_16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Shared-memory matrix descriptor for a K-major bf16 tile whose rows are 128 bytes with the 128-byte
// swizzle TMA applies: start address, leading offset 1 (unused for swizzled K-major), stride between
// 8-row groups 1024 bytes, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = m (128, or 256 for a CTA
// pair), N = n.
__device__ __forceinline__ uint32_t instr_desc_bf16(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// The map whose box holds exactly n_rows activation rows (n_rows a multiple of the quantum the maps
// were encoded with: 16 rows up to 256 for the one-CTA kernel, 8 rows up to 128 for each CTA of a pair).
// One copy per ring slot and operand: every TMA copy has a fixed cost in the copy engine that is
// comparable to moving several KiB, so a token tile is never assembled from smaller boxes.
// OR of `flag` over the 128 epilogue threads (named barrier 1), so that they leave their loop together.
__device__ __forceinline__ bool epilogue_any(bool flag) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, 128, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)flag)
        : "memory");
    return r != 0;
}
template <int kQuantum>
__device__ __forceinline__ const CUtensorMap *act_map(const TensorMaps &maps, int n_rows) {
    return &maps.act[n_rows / kQuantum - 1];
}

struct Tile {
    int e, f, row0, n_valid;
    int n_tok_tiles;  // token tiles of this tile's expert
};
// Tile order: experts in schedule order (most rows first), then weight slab, then the expert's token
// tiles (fastest), so tiles that share a weight slab run at the same time on neighbouring CTAs.
__device__ __forceinline__ Tile decode_tile(int tile, const KernelParams &p) {
    int lo = 0, hi = p.E;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (p.tile_prefix[mid] * p.n_feature_tiles <= tile) lo = mid; else hi = mid;
    }
    Tile t;
    t.e = p.tile_order[lo];
    const int first = p.tile_prefix[lo], n_tok_tiles = p.tile_prefix[lo + 1] - first;
    const int local = tile - first * p.n_feature_tiles;
    t.f = local / n_tok_tiles;
    const int j = local - t.f * n_tok_tiles;
    const int rows = p.tile_rows[t.e];
    const int begin = p.expert_offsets[t.e], count = p.expert_offsets[t.e + 1] - begin;
    t.row0 = begin + j * rows;
    t.n_valid = min(rows, count - j * rows);
    t.n_tok_tiles = n_tok_tiles;
    return t;
}

// ---- hand-over between the gate/up and the down GEMM of one call -------------------------------------------
// Bounded poll of an int in global memory until it reaches `target` (acquire); on expiry the CTA aborts as for an
// expired barrier wait.
__device__ __forceinline__ bool poll_at_least(const int *addr, int target, volatile int *abort_flag, int *status, int site,
                                              long long limit_cycles = kWaitLimitCycles) {
    const long long start = clock64();
    while (true) {
        int v;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(addr) : "memory");
        if (v >= target) return true;
        if (*abort_flag) return false;
        if (clock64() - start > limit_cycles) {
            *abort_flag = 1;
            if (atomicCAS(status, 0, (int)MOE_ERR_DEVICE_TIMEOUT) == 0) {
                status[1] = site;
                status[2] = blockIdx.x;
            }
            return false;
        }
        __nanosleep(200);
    }
}
// Start of a GEMM kernel's work, after its prologue.  Role 2 (down GEMM with hand-over) does not wait for the
// whole gate/up grid: it waits until that grid has raised the flag, i.e. has itself waited for the router and the
// gather, so the tile schedule is complete.  Every other kernel waits for its predecessors; role 1 then raises the flag.
__device__ __forceinline__ bool gemm_chain_start(int role, int *handover, volatile int *abort_flag, int *status) {
    if (role == 2) {
        bool ok = true;
        if (threadIdx.x == 0) ok = poll_at_least(handover + kHandoverFlagInt, 1, abort_flag, status, kSiteHandoverFlag);
        __syncthreads();
        return !*abort_flag && ok;
    }
    chain_wait();
    if (role == 1 && threadIdx.x == 0) {
        asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(handover + kHandoverFlagInt), "r"(1) : "memory");
    }
    return true;
}
// End of a GEMM kernel's work, before its teardown.  A role-2 grid never waited for the grid before it, only for that
// grid's flag and counts; it waits here (the gate/up grid is finished or finishing by now, so this costs nothing), so
// that "this grid is complete" again implies "everything before it in the stream is complete" for whatever follows.
__device__ __forceinline__ void gemm_chain_finish(int role) {
    if (role == 2) chain_wait();
}
// Role 1, called by every epilogue warp after it has stored its part of a tile: the stores of all its lanes are
// made visible, then the expert's count goes up by one.
__device__ __forceinline__ void handover_count_tile(int role, int *handover, int expert, int lane) {
    if (role != 1) return;
    __threadfence();
    __syncwarp();
    if (lane == 0) {
        atomicAdd(handover + kReadyCounterInt + expert, 1);
        atomicAdd(handover + kReadyTotalInt, 1);
    }
}
// Role 2, called by the token-side producer warp before the first load of a tile: all gate/up tiles of the expert
// must have been counted; then generic-proxy writes become visible to the TMA loads that follow.
// Once the total over all experts has been seen complete (`all_done`, kept by the caller across tiles) nothing is
// read any more: a load from global memory in front of every tile would starve the ring of a memory-bound GEMM.
// (whole warp: lane 0 reads, every lane fences, the result is uniform)
__device__ __forceinline__ bool handover_wait_expert(int role, int *handover, int expert, int n_tok_tiles, int per_token_tile,
                                                     int total_token_tiles, bool &all_done, volatile int *abort_flag,
                                                     int *status, int lane) {
    if (role != 2 || all_done) return true;
    bool ok = true, done = false;
    if (lane == 0) {
        int total;
        asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(total) : "l"(handover + kReadyTotalInt) : "memory");
        done = total >= total_token_tiles * per_token_tile;
        if (!done)
            ok = poll_at_least(handover + kReadyCounterInt + expert, n_tok_tiles * per_token_tile, abort_flag, status,
                               kSiteHandoverCount);
    }
    ok = __all_sync(0xffffffffu, ok);
    all_done = __any_sync(0xffffffffu, done);
    asm volatile("fence.proxy.async;" ::: "memory");
    return ok;
}

// Clock probe: block 0 of a GEMM grid leaves its SM cycle counter and the global nanosecond timer, at the start of its
// work and at its end, in the call's status region (kClockProbeInt, 4 x int64 per GEMM: cycles begin / end, ns begin /
// end).  Their quotient is the clock the SM really ran at during THAT kernel, which a benchmark needs to tell a slow
// kernel from a power-capped GPU; two stores per block-0 thread-0, nothing else.
__device__ __forceinline__ void clock_probe_begin(int *status, int which) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        long long *slot = reinterpret_cast<long long *>(status + kClockProbeInt) + 4 * which;
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        slot[0] = clock64();
        slot[2] = (long long)ns;
    }
}
__device__ __forceinline__ void clock_probe_end(int *status, int which) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        long long *slot = reinterpret_cast<long long *>(status + kClockProbeInt) + 4 * which;
        unsigned long long ns;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns));
        slot[1] = clock64();
        slot[3] = (long long)ns;
    }
}

// Static tile assignment: worker w of n_workers takes, in round i, tile i*n_workers + w on even rounds
// and i*n_workers + (n_workers-1-w) on odd rounds.  With tiles ordered by decreasing cost this
// back-and-forth deal keeps every worker's total within about 1 % of the mean, without atomics.
__device__ __forceinline__ int tile_of_round(int round, int worker, int n_workers) {
    return round * n_workers + ((round & 1) ? n_workers - 1 - worker : worker);
}

// SiLU(g) * u with the fast exponential; exp overflow gives g / inf = -0 for very negative g.
__device__ __forceinline__ float swiglu(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

// ---- host side ----------------------------------------------------------------------------------
bool encode_weight_map_2d(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K);
bool encode_weight_map_gate_up(CUtensorMap *map, const void *w13, int E, int I, int H);
bool encode_weight_map_2d_fp8(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K);
bool encode_act_maps_k128(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum);
bool encode_weight_map_gate_up_fp8(CUtensorMap *map, const void *w13, int E, int I, int H);
bool encode_act_maps(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum, int count = kNumActMaps);
bool encode_row_map(CUtensorMap *map, const void *act, uint64_t rows, uint64_t K);
bool encode_mx_weight_map_2d(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K);
bool encode_mx_weight_map_gate_up(CUtensorMap *map, const void *w13, int E, int I, int H);
bool encode_mx_act_maps(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum);
int sm_count();
bool set_max_dynamic_smem_once(const void *kernel, int bytes);

}  // namespace tc
}  // namespace moe

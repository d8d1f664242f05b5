// Grouped GEMMs of the MoE layer on plain CUDA cores (fp32 FMA, shared-memory tiles).
// Selected only by MOE_FLAG_VALIDATION_GEMM: it exists so the tcgen05 path can be checked in full
// at sizes a CPU cannot evaluate, by a kernel that shares nothing with it (no TMA, no tensor
// cores, no tile schedule: one block per (feature tile, expert) walks that expert's rows).
#include "moe_internal.cuh"

namespace moe {
namespace {

constexpr int kTile = 64;   // rows and features per block tile
constexpr int kStep = 16;   // K elements staged per iteration

template <bool kSwiglu>
__global__ void __launch_bounds__(256)
grouped_gemm_validation_kernel(const __nv_bfloat16 *__restrict__ act, const __nv_bfloat16 *__restrict__ w,
                               __nv_bfloat16 *__restrict__ out, int K, int n_out, int w_rows,
                               const int *__restrict__ expert_offsets) {
    const int e = blockIdx.y, f0 = blockIdx.x * kTile;
    const int r_begin = expert_offsets[e], r_end = expert_offsets[e + 1];
    if (r_begin == r_end) return;  // experts without tokens are skipped
    __shared__ float xs[kStep][kTile + 1], wa[kStep][kTile + 1], wb[kStep][kTile + 1];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int lrow = tid >> 2, lk = (tid & 3) * 4;
    const __nv_bfloat16 *wg = w + ((size_t)e * w_rows + f0) * K;          // gate rows (or the only rows)
    const __nv_bfloat16 *wu = wg + (size_t)n_out * K;                      // up rows: I rows further down
    for (int r0 = r_begin; r0 < r_end; r0 += kTile) {
        float acc_a[4][4] = {}, acc_b[4][4] = {};
        for (int k0 = 0; k0 < K; k0 += kStep) {
            const int r = r0 + lrow;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                xs[lk + c][lrow] = r < r_end ? __bfloat162float(act[(size_t)r * K + k0 + lk + c]) : 0.f;
                wa[lk + c][lrow] = __bfloat162float(wg[(size_t)lrow * K + k0 + lk + c]);
                if (kSwiglu) wb[lk + c][lrow] = __bfloat162float(wu[(size_t)lrow * K + k0 + lk + c]);
            }
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < kStep; ++kk) {
                float a[4], b[4], c[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    a[i] = xs[kk][ty * 4 + i];
                    b[i] = wa[kk][tx * 4 + i];
                    c[i] = kSwiglu ? wb[kk][tx * 4 + i] : 0.f;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc_a[i][j] = fmaf(a[i], b[j], acc_a[i][j]);
                        if (kSwiglu) acc_b[i][j] = fmaf(a[i], c[j], acc_b[i][j]);
                    }
            }
            __syncthreads();
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + ty * 4 + i;
            if (r >= r_end) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float g = acc_a[i][j];
                const float v = kSwiglu ? g / (1.f + expf(-g)) * acc_b[i][j] : g;
                out[(size_t)r * n_out + f0 + tx * 4 + j] = __float2bfloat16_rn(v);
            }
        }
    }
}

}  // namespace

cudaError_t launch_grouped_gemm_validation(const GroupedGemmArgs &a, cudaStream_t stream) {
    dim3 grid(a.n_out / kTile, a.E);
    if (a.swiglu)
        grouped_gemm_validation_kernel<true><<<grid, 256, 0, stream>>>(a.act, a.w, a.out, a.K, a.n_out, a.w_rows,
                                                                      a.expert_offsets);
    else
        grouped_gemm_validation_kernel<false><<<grid, 256, 0, stream>>>(a.act, a.w, a.out, a.K, a.n_out, a.w_rows,
                                                                       a.expert_offsets);
    return cudaGetLastError();
}

}  // namespace moe

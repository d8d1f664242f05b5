// C ABI of the MoE library: argument checking, workspace layout, and the launch sequence
//   router+histogram -> scan+schedule -> stable scatter -> gather rows -> gemm1 (SwiGLU) -> gemm2 -> combine
// (paper, Sec. 4.5: routing, sort-scatter, gate+up with SiLU, down projection; then the weighted sum).
#include "moe_internal.cuh"

#include <math.h>

namespace moe {

int check_device() {
    static int verdict[64];  // per device: 0 not asked yet, 1 compute capability 10.x, 2 anything else
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_CUDA;
    if (dev >= 0 && dev < 64 && verdict[dev]) return verdict[dev] == 1 ? MOE_OK : MOE_ERR_ARCH;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return MOE_ERR_CUDA;
    if (dev >= 0 && dev < 64) verdict[dev] = major == 10 ? 1 : 2;
    return major == 10 ? MOE_OK : MOE_ERR_ARCH;
}

int check_route_args(const float *logits, int T, int E, int k, const int32_t *ids, const float *w, const int32_t *offsets,
                     const int32_t *s2f, const int32_t *f2s) {
    if (T < 0 || E <= 0 || k <= 0 || k > E) return MOE_ERR_SHAPE;
    if (E > kMaxExperts || k > kMaxTopK || (long long)T * k >= (1LL << 27)) return MOE_ERR_UNSUPPORTED;
    if (!offsets) return MOE_ERR_NULL;
    if (T > 0 && (!logits || !ids || !w || !s2f || !f2s)) return MOE_ERR_NULL;
    auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) % 4) != 0; };
    if (misaligned(logits) || misaligned(ids) || misaligned(w) || misaligned(offsets) || misaligned(s2f) || misaligned(f2s))
        return MOE_ERR_ALIGN;
    return MOE_OK;
}

}  // namespace moe

namespace {

using namespace moe;

bool envelope_ok(long long T, int H, int I, int E, int k) {
    if (E < 1 || E > kMaxExperts || k < 1 || k > E || k > kMaxTopK) return false;
    if (H < 128 || I < 64 || H % 128 != 0 || I % 64 != 0) return false;
    if (T < 0 || T * k >= (1LL << 27)) return false;
    return true;
}

bool route_envelope_ok(long long T, int E, int k) {
    return !(E < 1 || E > kMaxExperts || k < 1 || k > E || k > kMaxTopK || T < 0 || T * k >= (1LL << 27));
}

// Checks a grouped-router description against the kernel's envelope and converts it.
int make_router(const moe_grouped_router_t *r, int E, int k, RouterParams *out) {
    if (!r) return MOE_ERR_NULL;
    if (r->n_group < 1 || r->topk_group < 1) return MOE_ERR_SHAPE;
    if (E % r->n_group != 0 || r->topk_group > r->n_group) return MOE_ERR_UNSUPPORTED;
    const int G = E / r->n_group;
    if ((G & (G - 1)) != 0 || (long long)r->topk_group * G < k) return MOE_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(r->selection_bias) % 4 != 0) return MOE_ERR_ALIGN;
    out->grouped = 1;
    out->n_group = r->n_group;
    out->topk_group = r->topk_group;
    out->bias = r->selection_bias;
    out->scale = r->route_scale;
    return MOE_OK;
}

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

void fill_layout(int T, int H, int I, int E, int k, moe_workspace_layout_t *L) {
    const size_t A = (size_t)T * k;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += align_up(bytes, 256); return at; };
    L->status = take(kStatusBytesForward);
    L->topk_ids = take(A * sizeof(int));
    L->topk_weights = take(A * sizeof(float));
    L->expert_offsets = take((size_t)(E + 1) * sizeof(int));
    L->sorted_to_flat = take(A * sizeof(int));
    L->flat_to_sorted = take(A * sizeof(int));
    L->route_scratch = take(route_scratch_bytes(T, E));
    L->x_perm = take(A * H * 2);
    L->h = take(A * I * 2);
    L->y = take(A * H * 2);
    L->staging = take((size_t)T * H * 2) /* x */;
    take((size_t)T * E * sizeof(float)) /* logits */;
    take((size_t)T * H * 2) /* out */;
    L->total_bytes = off;
}

// Token-tile bound of the bf16 layer for this problem and these flags: the wide bounds (320 / 384) need the
// wide-tile kernel for BOTH GEMMs (I a multiple of 128, H of 256) and none of the flags that pin another kernel.
int layer_token_tile_bound(int T, int H, int I, int E, int k, unsigned flags, bool fp8w) {
    const bool pinned = fp8w || (flags & (MOE_FLAG_SINGLE_CTA_GEMM | MOE_FLAG_TWO_SLAB_GEMM | MOE_FLAG_NARROW_TILES)) != 0;
    const bool wide_ok = !pinned && I % 128 == 0 && H % 256 == 0;
    return choose_nt_max(T, E, k, wide_ok);
}

int forward_impl(const void *x, const float *logits, const void *w13, const void *w2, int T, int H, int I, int E, int k,
                 void *out, void *workspace, size_t workspace_bytes, cudaStream_t stream, unsigned flags,
                 void *const *stage_events = nullptr, int local_offset = 0, int n_local = -1,
                 const float *w13_scale = nullptr, const float *w2_scale = nullptr, RouterParams router = RouterParams()) {
    if (n_local < 0) n_local = E;  // every expert is resident
    const bool fp8w = w13_scale != nullptr;  // w13 / w2 then hold E4M3 codes, one byte per weight
    if (T < 0 || H <= 0 || I <= 0 || E <= 0 || k <= 0 || k > E) return MOE_ERR_SHAPE;
    if (!envelope_ok(T, H, I, E, k)) return MOE_ERR_UNSUPPORTED;
    if (local_offset < 0 || n_local < 1 || (long long)local_offset + n_local > E) return MOE_ERR_SHAPE;
    if (flags & ~(MOE_FLAG_VALIDATION_GEMM | MOE_FLAG_SINGLE_CTA_GEMM | MOE_FLAG_TWO_SLAB_GEMM | MOE_FLAG_NARROW_TILES |
                  MOE_FLAG_GATHER_IN_LOAD))
        return MOE_ERR_UNSUPPORTED;
    if (fp8w && (I % 128 != 0 || flags != MOE_FLAG_NONE)) return MOE_ERR_UNSUPPORTED;
    if (T == 0) return MOE_OK;
    if (!x || !logits || !w13 || !w2 || !out || !workspace || (fp8w && !w2_scale)) return MOE_ERR_NULL;
    if (!aligned(x, 16) || !aligned(logits, 16) || !aligned(w13, 16) || !aligned(w2, 16) || !aligned(out, 16) ||
        !aligned(workspace, 256))
        return MOE_ERR_ALIGN;
    moe_workspace_layout_t L;
    fill_layout(T, H, I, E, k, &L);
    if (workspace_bytes < L.total_bytes) return MOE_ERR_WORKSPACE;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;

    char *ws = static_cast<char *>(workspace);
    int *status = reinterpret_cast<int *>(ws + L.status);
    int *ids = reinterpret_cast<int *>(ws + L.topk_ids);
    float *wts = reinterpret_cast<float *>(ws + L.topk_weights);
    int *offsets = reinterpret_cast<int *>(ws + L.expert_offsets);
    int *s2f = reinterpret_cast<int *>(ws + L.sorted_to_flat);
    int *f2s = reinterpret_cast<int *>(ws + L.flat_to_sorted);
    RouteScratch rs = carve_route_scratch(ws + L.route_scratch, T, n_local);
    __nv_bfloat16 *x_perm = reinterpret_cast<__nv_bfloat16 *>(ws + L.x_perm);
    __nv_bfloat16 *h = reinterpret_cast<__nv_bfloat16 *>(ws + L.h);
    __nv_bfloat16 *y = reinterpret_cast<__nv_bfloat16 *>(ws + L.y);
    const int A = T * k;
    const int nt_max = layer_token_tile_bound(T, H, I, E, k, flags, fp8w);

    auto mark = [&](int i) {
        return !stage_events || cudaEventRecord(static_cast<cudaEvent_t>(stage_events[i]), stream) == cudaSuccess;
    };
    if (!mark(0)) return MOE_ERR_CUDA;
    if (launch_route(logits, T, E, k, LocalExperts{local_offset, n_local}, nt_max, ids, wts, offsets, s2f, f2s, rs, status,
                     stream, 16, router, kStatusBytesForward) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(1)) return MOE_ERR_CUDA;
    // Gather-in-load (opt-in): the wide-tile gate/up GEMM fetches token rows from x itself and x_perm is not written.
    const bool gather_in_load = (flags & MOE_FLAG_GATHER_IN_LOAD) != 0 && (nt_max == 320 || nt_max == 384) &&
                                !(flags & MOE_FLAG_VALIDATION_GEMM);
    if (!gather_in_load &&
        launch_scatter_rows(static_cast<const __nv_bfloat16 *>(x), f2s, T, k, H, x_perm, stream) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(2)) return MOE_ERR_CUDA;

    GroupedGemmArgs g1;
    g1.act = x_perm; g1.w = static_cast<const __nv_bfloat16 *>(w13); g1.out = h;
    g1.A = A; g1.K = H; g1.n_out = I; g1.E = n_local; g1.w_rows = 2 * I; g1.nt_max = nt_max;
    g1.expert_offsets = offsets; g1.tile_prefix = rs.tile_prefix; g1.tile_order = rs.tile_order; g1.tile_rows = rs.tile_rows;
    g1.status = status; g1.swiglu = true;
    GroupedGemmArgs g2 = g1;
    g2.act = h; g2.w = static_cast<const __nv_bfloat16 *>(w2); g2.out = y;
    g2.K = I; g2.n_out = H; g2.w_rows = H; g2.swiglu = false;
    if (gather_in_load) {
        g1.gather_x = static_cast<const __nv_bfloat16 *>(x);
        g1.gather_sorted_to_flat = s2f;
        g1.gather_T = T;
        g1.gather_top_k = k;
    }

    if (fp8w) {
        g1.w_scale = w13_scale;
        g2.w_scale = w2_scale;
        int st = launch_grouped_gemm_tc_fp8w(g1, stream);
        if (st != MOE_OK) return st;
        if (!mark(3)) return MOE_ERR_CUDA;
        st = launch_grouped_gemm_tc_fp8w(g2, stream);
        if (st != MOE_OK) return st;
    } else if (flags & MOE_FLAG_VALIDATION_GEMM) {
        if (launch_grouped_gemm_validation(g1, stream) != cudaSuccess) return MOE_ERR_CUDA;
        if (!mark(3)) return MOE_ERR_CUDA;
        if (launch_grouped_gemm_validation(g2, stream) != cudaSuccess) return MOE_ERR_CUDA;
    } else {
        // CTA pairs where the token tiles are large enough for the halved token-tile traffic to matter.
        // Two weight slabs per CTA (512 x N pair tiles) are opt-in: measured on the prefill-sized and
        // skewed workloads they are 5 % resp. 25 % slower than one slab, because the accumulators then
        // fill TMEM and the epilogue no longer overlaps the next tile's MMAs.
        const bool single = (flags & MOE_FLAG_SINGLE_CTA_GEMM) != 0;
        const bool dense_tiles = (flags & MOE_FLAG_TWO_SLAB_GEMM) != 0;
        // Hand-over: the down GEMM starts expert by expert as the gate/up GEMM finishes them (not with the opt-in
        // two-slab tiles, whose epilogue counts differently).
        if (!dense_tiles) {
            g1.handover_role = 1;
            g2.handover_role = 2;
            g1.handover = g2.handover = status;
            g2.handover_per_token_tile = handover_counts_per_token_tile(I);
        }
        auto run = [&](const GroupedGemmArgs &g, bool allow_two_slabs) {
            if (!single && grouped_gemm_tc_ring_applies(g)) return launch_grouped_gemm_tc_ring(g, stream);
            int slabs = single ? 0 : grouped_gemm_tc_pair_slabs(g);
            if (slabs == 2 && !(dense_tiles && allow_two_slabs)) slabs = grouped_gemm_tc_pair_slabs(g) >= 1 ? 1 : 0;
            if (slabs == 2 || slabs == 1) {
                // a one-slab launch needs its own divisibility (256 resp. 128 features)
                const int st = launch_grouped_gemm_tc_pair(g, slabs, stream);
                if (st != MOE_ERR_UNSUPPORTED) return st;
            }
            return launch_grouped_gemm_tc(g, stream);
        };
        int st = run(g1, true);
        if (st != MOE_OK) return st;
        if (!mark(3)) return MOE_ERR_CUDA;
        st = run(g2, false);
        if (st != MOE_OK) return st;
    }
    if (!mark(4)) return MOE_ERR_CUDA;
    if (launch_combine(y, wts, f2s, T, k, H, static_cast<__nv_bfloat16 *>(out), stream, n_local < E) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(5)) return MOE_ERR_CUDA;
    return MOE_OK;
}

// ---- MX FP8 ---------------------------------------------------------------------------------------------
bool mx_envelope_ok(long long T, int H, int I, int E, int k) { return envelope_ok(T, H, I, E, k) && I % 128 == 0; }

// Token-tile rows of the MX path.  Scale columns sit next to the accumulators in tensor memory, so the largest tile
// of the kernel with two fixed accumulators is 240 rows (2 * 240 + 32 columns); only the CTA-pair kernels have the
// instances above 128 rows, and their down projection needs H to be a multiple of the 256-row pair tile.  Where the
// bf16 layer takes its wide tiles (160 to 352 rows per expert on average) so does this one, on the accumulator ring,
// one pass over an expert's weights: 304 rows while the mean plus 2.5 standard deviations of a uniform routing fits
// (a 304-row token slot leaves the gate/up kernel room for a sixth ring slot, which the weight-stream-bound calls
// need), else 384.  160-row tiles (a deeper ring still) are taken when the mean plus 2.5 standard deviations fits.
int mx_tile_rows(int T, int H, int E, int k) {
    const int nt = choose_nt_max(T, E, k, true);
    if (nt <= 128) return nt;
    if (H % 256 != 0) return 128;
    const double mean = (double)T * k / E;
    if (nt > 256) return mean + 2.5 * sqrt(mean) <= 304.0 ? 304 : 384;
    return mean + 2.5 * sqrt(mean) <= 160.0 ? 160 : 240;
}

void fill_mx_layout(int T, int H, int I, int E, int k, moe_mxfp8_workspace_layout_t *L) {
    const size_t A = (size_t)T * k;
    const int tile = mx_tile_rows(T, H, E, k);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += align_up(bytes, 256); return at; };
    L->status = take(kStatusBytesForward);
    L->topk_ids = take(A * sizeof(int));
    L->topk_weights = take(A * sizeof(float));
    L->expert_offsets = take((size_t)(E + 1) * sizeof(int));
    L->sorted_to_flat = take(A * sizeof(int));
    L->flat_to_sorted = take(A * sizeof(int));
    L->route_scratch = take(route_scratch_bytes(T, E));
    L->x_q = take(A * H);
    L->x_sf = take(mx_act_sf_bytes((int)A, E, H, tile));
    L->h_q = take(A * I);
    L->h_sf = take(mx_act_sf_bytes((int)A, E, I, tile));
    L->y = take(A * H * 2);
    L->staging = take((size_t)T * H * 2) /* x */;
    take((size_t)T * E * sizeof(float)) /* logits */;
    take((size_t)T * H * 2) /* out */;
    L->sf_atoms = (size_t)mx_act_sf_atoms((int)A, E, tile);
    L->tile_rows = (size_t)tile;
    L->total_bytes = off;
}

int forward_mx_impl(const void *x, const float *logits, const void *w13_q, const void *w13_sf, const void *w2_q,
                    const void *w2_sf, int T, int H, int I, int E, int k, int local_offset, int n_local, void *out,
                    void *workspace, size_t workspace_bytes, cudaStream_t stream, void *const *stage_events,
                    const moe_grouped_router_t *grouped) {
    if (T < 0 || H <= 0 || I <= 0 || E <= 0 || k <= 0 || k > E) return MOE_ERR_SHAPE;
    if (!mx_envelope_ok(T, H, I, E, k)) return MOE_ERR_UNSUPPORTED;
    if (local_offset < 0 || n_local < 1 || (long long)local_offset + n_local > E) return MOE_ERR_SHAPE;
    RouterParams router;
    if (grouped) {
        const int rs_status = make_router(grouped, E, k, &router);
        if (rs_status != MOE_OK) return rs_status;
    }
    if (stage_events)
        for (int i = 0; i < MOE_NUM_STAGE_EVENTS; ++i)
            if (!stage_events[i]) return MOE_ERR_NULL;
    if (T == 0) return MOE_OK;
    if (!x || !logits || !w13_q || !w13_sf || !w2_q || !w2_sf || !out || !workspace) return MOE_ERR_NULL;
    if (!aligned(x, 16) || !aligned(logits, 16) || !aligned(w13_q, 16) || !aligned(w2_q, 16) || !aligned(w13_sf, 16) ||
        !aligned(w2_sf, 16) || !aligned(out, 16) || !aligned(workspace, 256))
        return MOE_ERR_ALIGN;
    moe_mxfp8_workspace_layout_t L;
    fill_mx_layout(T, H, I, E, k, &L);
    if (workspace_bytes < L.total_bytes) return MOE_ERR_WORKSPACE;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;

    char *ws = static_cast<char *>(workspace);
    int *status = reinterpret_cast<int *>(ws + L.status);
    int *ids = reinterpret_cast<int *>(ws + L.topk_ids);
    float *wts = reinterpret_cast<float *>(ws + L.topk_weights);
    int *offsets = reinterpret_cast<int *>(ws + L.expert_offsets);
    int *s2f = reinterpret_cast<int *>(ws + L.sorted_to_flat);
    int *f2s = reinterpret_cast<int *>(ws + L.flat_to_sorted);
    RouteScratch rs = carve_route_scratch(ws + L.route_scratch, T, n_local);
    uint8_t *x_q = reinterpret_cast<uint8_t *>(ws + L.x_q), *x_sf = reinterpret_cast<uint8_t *>(ws + L.x_sf);
    uint8_t *h_q = reinterpret_cast<uint8_t *>(ws + L.h_q), *h_sf = reinterpret_cast<uint8_t *>(ws + L.h_sf);
    __nv_bfloat16 *y = reinterpret_cast<__nv_bfloat16 *>(ws + L.y);
    const int A = T * k;
    const int n_atoms = (int)L.sf_atoms;
    const int nt_max = (int)L.tile_rows;

    auto mark = [&](int i) {
        return !stage_events || cudaEventRecord(static_cast<cudaEvent_t>(stage_events[i]), stream) == cudaSuccess;
    };
    if (!mark(0)) return MOE_ERR_CUDA;
    // Bounds up to 256: every token tile exactly nt_max rows (the last of an expert partial).  Wide bounds: the bf16
    // schedule's rule (row quantum 16; experts above the bound get evenly sized tiles of at most 256 rows).  Either
    // way each tile owns its own scale atoms (moe_internal.cuh).
    if (launch_route(logits, T, E, k, LocalExperts{local_offset, n_local}, nt_max, ids, wts, offsets, s2f, f2s, rs, status,
                     stream, nt_max > 256 ? 16 : nt_max, router, kStatusBytesForward) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(1)) return MOE_ERR_CUDA;
    if (launch_mx_scatter_quantize(static_cast<const __nv_bfloat16 *>(x), f2s, ids, offsets, rs.tile_rows,
                                   LocalExperts{local_offset, n_local}, T, k, H, x_q, x_sf, n_atoms, nt_max, stream) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(2)) return MOE_ERR_CUDA;

    MxGemmArgs g1;
    g1.act_q = x_q; g1.act_sf = x_sf; g1.w_q = static_cast<const uint8_t *>(w13_q);
    g1.w_sf = static_cast<const uint8_t *>(w13_sf); g1.out = h_q; g1.out_sf = h_sf;
    g1.A = A; g1.K = H; g1.n_out = I; g1.E = n_local; g1.w_rows = 2 * I; g1.nt_max = nt_max; g1.n_atoms = n_atoms;
    g1.expert_offsets = offsets; g1.tile_prefix = rs.tile_prefix; g1.tile_order = rs.tile_order; g1.tile_rows = rs.tile_rows;
    g1.status = status; g1.swiglu = true;
    MxGemmArgs g2 = g1;
    g2.act_q = h_q; g2.act_sf = h_sf; g2.w_q = static_cast<const uint8_t *>(w2_q);
    g2.w_sf = static_cast<const uint8_t *>(w2_sf); g2.out = y; g2.out_sf = nullptr;
    g2.K = I; g2.n_out = H; g2.w_rows = H; g2.swiglu = false;
    g1.handover_role = 1;
    g2.handover_role = 2;
    g1.handover = g2.handover = status;
    g2.handover_per_token_tile = handover_counts_per_token_tile(I);
    auto run = [&](const MxGemmArgs &g) {
        if (grouped_gemm_tc_mx_ring_applies(g)) return launch_grouped_gemm_tc_mx_ring(g, stream);
        return grouped_gemm_tc_mx_pair_applies(g) ? launch_grouped_gemm_tc_mx_pair(g, stream) : launch_grouped_gemm_tc_mx(g, stream);
    };
    int st = run(g1);
    if (st != MOE_OK) return st;
    if (!mark(3)) return MOE_ERR_CUDA;
    st = run(g2);
    if (st != MOE_OK) return st;
    if (!mark(4)) return MOE_ERR_CUDA;
    if (launch_combine(y, wts, f2s, T, k, H, static_cast<__nv_bfloat16 *>(out), stream, n_local < E) != cudaSuccess)
        return MOE_ERR_CUDA;
    if (!mark(5)) return MOE_ERR_CUDA;
    return MOE_OK;
}

}  // namespace

extern "C" {

size_t moe_mxfp8_workspace_bytes(int T, int H, int I, int E, int top_k) {
    if (!mx_envelope_ok(T, H, I, E, top_k)) return 0;
    moe_mxfp8_workspace_layout_t L;
    fill_mx_layout(T, H, I, E, top_k, &L);
    return L.total_bytes;
}

int moe_mxfp8_workspace_layout(int T, int H, int I, int E, int top_k, moe_mxfp8_workspace_layout_t *layout) {
    if (!layout) return MOE_ERR_NULL;
    if (!mx_envelope_ok(T, H, I, E, top_k)) return MOE_ERR_UNSUPPORTED;
    fill_mx_layout(T, H, I, E, top_k, layout);
    return MOE_OK;
}

int moe_mxfp8_pack_scales(const void *scales, int E, int rows, int K, int gate_up, void *packed, void *stream) {
    if (E < 1 || rows < 1 || K < 1) return MOE_ERR_SHAPE;
    if (K % 128 != 0 || rows % 128 != 0) return MOE_ERR_UNSUPPORTED;
    if (!scales || !packed) return MOE_ERR_NULL;
    if (!aligned(scales, 4) || !aligned(packed, 16)) return MOE_ERR_ALIGN;
    return launch_mx_pack_scales(static_cast<const uint8_t *>(scales), E, rows, K, gate_up != 0,
                                 static_cast<uint8_t *>(packed), static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MOE_OK
               : MOE_ERR_CUDA;
}

int moe_mxfp8_quantize_rows(const void *x, int R, int K, void *codes, void *scales, void *stream) {
    if (R < 0 || K < 1) return MOE_ERR_SHAPE;
    if (K % 128 != 0) return MOE_ERR_UNSUPPORTED;
    if (R == 0) return MOE_OK;
    if (!x || !codes || !scales) return MOE_ERR_NULL;
    if (!aligned(x, 16) || !aligned(codes, 8)) return MOE_ERR_ALIGN;
    return launch_mx_quantize_rows(static_cast<const __nv_bfloat16 *>(x), R, K, static_cast<uint8_t *>(codes),
                                   static_cast<uint8_t *>(scales), static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MOE_OK
               : MOE_ERR_CUDA;
}

int moe_forward_mxfp8_host(const void *x_host, const float *router_logits_host, const void *w13_q,
                           const void *w13_sf_packed, const void *w2_q, const void *w2_sf_packed, int T, int H, int I, int E,
                           int top_k, const moe_grouped_router_t *router, int local_expert_offset, int num_local_experts,
                           void *out_host, void *workspace, size_t workspace_bytes, void *stream) {
    if (T < 0 || H <= 0 || I <= 0 || E <= 0 || top_k <= 0 || top_k > E || num_local_experts < 1) return MOE_ERR_SHAPE;
    if (!mx_envelope_ok(T, H, I, E, top_k)) return MOE_ERR_UNSUPPORTED;
    if (T == 0) return MOE_OK;
    if (!x_host || !router_logits_host || !out_host || !workspace) return MOE_ERR_NULL;
    if (!aligned(workspace, 256)) return MOE_ERR_ALIGN;
    moe_mxfp8_workspace_layout_t L;
    fill_mx_layout(T, H, I, E, top_k, &L);
    if (workspace_bytes < L.total_bytes) return MOE_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(workspace);
    const size_t x_bytes = (size_t)T * H * 2, l_bytes = (size_t)T * E * sizeof(float);
    char *x_dev = ws + L.staging;
    char *l_dev = x_dev + align_up(x_bytes, 256);
    char *out_dev = l_dev + align_up(l_bytes, 256);
    if (cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemcpyAsync(l_dev, router_logits_host, l_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return MOE_ERR_CUDA;
    const int st = forward_mx_impl(x_dev, reinterpret_cast<const float *>(l_dev), w13_q, w13_sf_packed, w2_q, w2_sf_packed, T,
                                   H, I, E, top_k, local_expert_offset, num_local_experts, out_dev, workspace,
                                   workspace_bytes, s, nullptr, router);
    if (st != MOE_OK) return st;
    if (cudaMemcpyAsync(out_host, out_dev, x_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
}

int moe_forward_mxfp8(const void *x, const float *router_logits, const void *w13_q, const void *w13_sf_packed,
                      const void *w2_q, const void *w2_sf_packed, int T, int H, int I, int E, int top_k,
                      const moe_grouped_router_t *router, int local_expert_offset, int num_local_experts, void *out,
                      void *workspace, size_t workspace_bytes, void *stream, void *const *stage_events) {
    return forward_mx_impl(x, router_logits, w13_q, w13_sf_packed, w2_q, w2_sf_packed, T, H, I, E, top_k,
                           local_expert_offset, num_local_experts, out, workspace, workspace_bytes,
                           static_cast<cudaStream_t>(stream), stage_events, router);
}

size_t moe_workspace_bytes(int T, int H, int I, int E, int top_k) {
    if (!envelope_ok(T, H, I, E, top_k)) return 0;
    moe_workspace_layout_t L;
    fill_layout(T, H, I, E, top_k, &L);
    return L.total_bytes;
}

int moe_workspace_layout(int T, int H, int I, int E, int top_k, moe_workspace_layout_t *layout) {
    if (!layout) return MOE_ERR_NULL;
    if (!envelope_ok(T, H, I, E, top_k)) return MOE_ERR_UNSUPPORTED;
    fill_layout(T, H, I, E, top_k, layout);
    return MOE_OK;
}

size_t moe_route_workspace_bytes(int T, int E, int top_k) {
    if (!route_envelope_ok(T, E, top_k)) return 0;
    return 256 + route_scratch_bytes(T, E);
}

int moe_route(const float *router_logits, int T, int E, int top_k, int32_t *topk_ids, float *topk_weights,
              int32_t *expert_offsets, int32_t *sorted_to_flat, int32_t *flat_to_sorted, void *workspace,
              size_t workspace_bytes, void *stream) {
    const int args = check_route_args(router_logits, T, E, top_k, topk_ids, topk_weights, expert_offsets, sorted_to_flat,
                                      flat_to_sorted);
    if (args != MOE_OK) return args;
    if (!workspace) return MOE_ERR_NULL;
    if (!aligned(workspace, 256)) return MOE_ERR_ALIGN;
    if (workspace_bytes < moe_route_workspace_bytes(T, E, top_k)) return MOE_ERR_WORKSPACE;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (T == 0) {  // no assignments: every segment is empty
        return cudaMemsetAsync(expert_offsets, 0, (size_t)(E + 1) * sizeof(int), s) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
    }
    char *ws = static_cast<char *>(workspace);
    RouteScratch rs = carve_route_scratch(ws + 256, T, E);
    const cudaError_t err = launch_route(router_logits, T, E, top_k, LocalExperts{0, E}, 256, topk_ids, topk_weights,
                                         expert_offsets, sorted_to_flat, flat_to_sorted, rs, reinterpret_cast<int *>(ws), s);
    return err == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_route_grouped(const float *router_logits, int T, int E, int top_k, const moe_grouped_router_t *router,
                      int32_t *topk_ids, float *topk_weights, int32_t *expert_offsets, int32_t *sorted_to_flat,
                      int32_t *flat_to_sorted, void *workspace, size_t workspace_bytes, void *stream) {
    if (T < 0 || E <= 0 || top_k <= 0 || top_k > E) return MOE_ERR_SHAPE;
    if (!route_envelope_ok(T, E, top_k)) return MOE_ERR_UNSUPPORTED;
    RouterParams rp;
    const int rs_status = make_router(router, E, top_k, &rp);
    if (rs_status != MOE_OK) return rs_status;
    const int args = check_route_args(router_logits, T, E, top_k, topk_ids, topk_weights, expert_offsets, sorted_to_flat,
                                      flat_to_sorted);
    if (args != MOE_OK) return args;
    if (!workspace) return MOE_ERR_NULL;
    if (!aligned(workspace, 256)) return MOE_ERR_ALIGN;
    if (workspace_bytes < moe_route_workspace_bytes(T, E, top_k)) return MOE_ERR_WORKSPACE;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (T == 0)
        return cudaMemsetAsync(expert_offsets, 0, (size_t)(E + 1) * sizeof(int), s) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
    char *ws = static_cast<char *>(workspace);
    RouteScratch rs = carve_route_scratch(ws + 256, T, E);
    const cudaError_t err = launch_route(router_logits, T, E, top_k, LocalExperts{0, E}, 256, topk_ids, topk_weights,
                                         expert_offsets, sorted_to_flat, flat_to_sorted, rs, reinterpret_cast<int *>(ws), s,
                                         16, rp);
    return err == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_forward_grouped(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I,
                        int E, int top_k, const moe_grouped_router_t *router, int local_expert_offset,
                        int num_local_experts, void *out, void *workspace, size_t workspace_bytes, void *stream,
                        unsigned flags) {
    if (num_local_experts < 1 || E <= 0 || top_k <= 0 || top_k > E) return MOE_ERR_SHAPE;
    RouterParams rp;
    const int rs_status = make_router(router, E, top_k, &rp);
    if (rs_status != MOE_OK) return rs_status;
    return forward_impl(x, router_logits, w13, w2, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), flags, nullptr, local_expert_offset, num_local_experts, nullptr,
                        nullptr, rp);
}

int moe_forward(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I, int E,
                int top_k, void *out, void *workspace, size_t workspace_bytes, void *stream) {
    return forward_impl(x, router_logits, w13, w2, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), MOE_FLAG_NONE);
}

int moe_forward_ex(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I,
                   int E, int top_k, void *out, void *workspace, size_t workspace_bytes, void *stream, unsigned flags) {
    return forward_impl(x, router_logits, w13, w2, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), flags);
}

int moe_forward_local(const void *x, const float *router_logits, const void *w13_local, const void *w2_local, int T, int H,
                      int I, int E, int top_k, int local_expert_offset, int num_local_experts, void *out, void *workspace,
                      size_t workspace_bytes, void *stream, unsigned flags) {
    if (num_local_experts < 1) return MOE_ERR_SHAPE;
    return forward_impl(x, router_logits, w13_local, w2_local, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), flags, nullptr, local_expert_offset, num_local_experts);
}

int moe_forward_fp8w(const void *x, const float *router_logits, const void *w13_q, const float *w13_scale,
                     const void *w2_q, const float *w2_scale, int T, int H, int I, int E, int top_k, void *out,
                     void *workspace, size_t workspace_bytes, void *stream, void *const *stage_events) {
    if (!w13_scale || !w2_scale) return MOE_ERR_NULL;
    if (!aligned(w13_scale, 4) || !aligned(w2_scale, 4)) return MOE_ERR_ALIGN;
    if (stage_events)
        for (int i = 0; i < MOE_NUM_STAGE_EVENTS; ++i)
            if (!stage_events[i]) return MOE_ERR_NULL;
    return forward_impl(x, router_logits, w13_q, w2_q, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), MOE_FLAG_NONE, stage_events, 0, -1, w13_scale, w2_scale);
}

int moe_forward_staged(const void *x, const float *router_logits, const void *w13, const void *w2, int T, int H, int I,
                       int E, int top_k, int local_expert_offset, int num_local_experts, void *out, void *workspace,
                       size_t workspace_bytes, void *stream, unsigned flags, void *const *stage_events) {
    if (!stage_events) return MOE_ERR_NULL;
    for (int i = 0; i < MOE_NUM_STAGE_EVENTS; ++i)
        if (!stage_events[i]) return MOE_ERR_NULL;
    if (num_local_experts < 1) return MOE_ERR_SHAPE;
    return forward_impl(x, router_logits, w13, w2, T, H, I, E, top_k, out, workspace, workspace_bytes,
                        static_cast<cudaStream_t>(stream), flags, stage_events, local_expert_offset, num_local_experts);
}

int moe_forward_host(const void *x_host, const float *router_logits_host, const void *w13, const void *w2, int T, int H,
                     int I, int E, int top_k, int local_expert_offset, int num_local_experts, void *out_host,
                     void *workspace, size_t workspace_bytes, void *stream) {
    if (T < 0 || H <= 0 || I <= 0 || E <= 0 || top_k <= 0 || top_k > E || num_local_experts < 1) return MOE_ERR_SHAPE;
    if (!envelope_ok(T, H, I, E, top_k)) return MOE_ERR_UNSUPPORTED;
    if (T == 0) return MOE_OK;
    if (!x_host || !router_logits_host || !out_host || !workspace) return MOE_ERR_NULL;
    if (!aligned(workspace, 256)) return MOE_ERR_ALIGN;
    moe_workspace_layout_t L;
    fill_layout(T, H, I, E, top_k, &L);
    if (workspace_bytes < L.total_bytes) return MOE_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(workspace);
    const size_t x_bytes = (size_t)T * H * 2, l_bytes = (size_t)T * E * sizeof(float);
    char *x_dev = ws + L.staging;
    char *l_dev = x_dev + align_up(x_bytes, 256);
    char *out_dev = l_dev + align_up(l_bytes, 256);
    if (cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return MOE_ERR_CUDA;
    if (cudaMemcpyAsync(l_dev, router_logits_host, l_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return MOE_ERR_CUDA;
    const int st = forward_impl(x_dev, reinterpret_cast<const float *>(l_dev), w13, w2, T, H, I, E, top_k, out_dev,
                                workspace, workspace_bytes, s, MOE_FLAG_NONE, nullptr, local_expert_offset,
                                num_local_experts);
    if (st != MOE_OK) return st;
    if (cudaMemcpyAsync(out_host, out_dev, x_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MOE_ERR_CUDA;
    return MOE_OK;
}

int moe_last_status(const void *workspace, void *stream) {
    if (!workspace) return MOE_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(s) != cudaSuccess) return MOE_ERR_CUDA;
    int status[moe::kStatusInts] = {0, 0, 0, 0};
    if (cudaMemcpy(status, workspace, sizeof(status), cudaMemcpyDeviceToHost) != cudaSuccess) return MOE_ERR_CUDA;
    return status[0];
}

int moe_token_tile_rows(int T, int H, int I, int E, int top_k, unsigned flags) {
    if (!envelope_ok(T, H, I, E, top_k)) return 0;
    return layer_token_tile_bound(T, H, I, E, top_k, flags, false);
}

int moe_forward_launch_count(int T, unsigned flags) {
    (void)flags;
    if (T <= 0) return 0;
    // router + sort-scatter: one fused kernel up to 1024 tokens, three kernels beyond; then gather, two GEMMs, combine
    return (route_num_chunks(T) <= 32 ? 1 : 3) + 4;
}

int moe_selftest_wait_timeout(void *workspace, size_t workspace_bytes, void *stream) {
    if (!workspace) return MOE_ERR_NULL;
    if (!aligned(workspace, 256)) return MOE_ERR_ALIGN;
    if (workspace_bytes < (size_t)kStatusBytesForward) return MOE_ERR_WORKSPACE;
    const int arch = check_device();
    if (arch != MOE_OK) return arch;
    return launch_wait_timeout_selftest(static_cast<int *>(workspace), static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? MOE_OK
               : MOE_ERR_CUDA;
}

const char *moe_status_string(int status) {
    switch (status) {
        case MOE_OK: return "ok";
        case MOE_ERR_NULL: return "a required pointer is NULL";
        case MOE_ERR_SHAPE: return "invalid shape (negative size, zero dimension, or top_k > E)";
        case MOE_ERR_UNSUPPORTED: return "outside the supported envelope (E<=256, top_k<=32, H%128==0, I%64==0, T*top_k<2^27)";
        case MOE_ERR_ALIGN: return "pointer not sufficiently aligned";
        case MOE_ERR_WORKSPACE: return "workspace too small";
        case MOE_ERR_CUDA: return "a CUDA call failed";
        case MOE_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case MOE_ERR_ARCH: return "device is not compute capability 10.x";
        case MOE_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of moe_route_static (512 KiB)";
        default: return "unknown status";
    }
}

}  // extern "C"

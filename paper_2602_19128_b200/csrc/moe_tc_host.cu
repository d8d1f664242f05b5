// Host-side helpers of the tcgen05 grouped GEMMs: TMA tensor-map encoding (through the driver entry
// point, so the library links against no driver stub and loads on a machine without a GPU) and the
// SM count.
#include "moe_mx_tc.cuh"

#include <string.h>

#include <mutex>

namespace moe {
namespace tc {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// ---- tensor-map cache ------------------------------------------------------------------------------------
// A forward call needs 34 tensor maps (one weight map and sixteen activation maps per GEMM); encoding them through
// the driver costs more host time than everything else in a call.  An encoded map is a pure function of the
// arguments of the encode call (address, element type, rank, extents, strides, box, swizzle): it does not depend on
// the memory's contents, so an entry can never go stale -- a buffer freed and allocated again at the same address
// with the same shape has the same map.  The cache is a fixed table of kCacheSlots entries keyed by ALL those
// arguments, direct-mapped with a short probe, overwritten in place when full, and guarded by one mutex (look-ups
// copy the 128-byte map out under the lock), so concurrent callers on different streams are safe.
struct EncodeKey {
    const void *base;
    uint32_t rank, dtype, swizzle, pad;
    uint64_t dims[5], strides[4];
    uint32_t box[5], pad2;
};
struct CacheSlot {
    EncodeKey key;
    CUtensorMap map;
    bool used;
};
constexpr int kCacheSlots = 1024, kCacheProbe = 8;
std::mutex g_cache_mutex;
CacheSlot *g_cache = nullptr;  // allocated on first use (host memory), never freed

static_assert(sizeof(EncodeKey) % 8 == 0, "the key is hashed and compared as 64-bit words");
uint64_t key_hash(const EncodeKey &k) {  // word-wise multiply-xorshift: a few nanoseconds for the 14 words of a key
    uint64_t words[sizeof(EncodeKey) / 8];
    memcpy(words, &k, sizeof(EncodeKey));
    uint64_t h = 0x9e3779b97f4a7c15ull;
    for (size_t i = 0; i < sizeof(EncodeKey) / 8; ++i) {
        h = (h ^ words[i]) * 0xff51afd7ed558ccdull;
        h ^= h >> 29;
    }
    return h;
}

bool encode_cached(CUtensorMap *map, CUtensorMapDataType dtype, int rank, const void *base, const cuuint64_t *dims,
                   const cuuint64_t *strides, const cuuint32_t *box, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    EncodeKey key;
    memset(&key, 0, sizeof(key));  // (padding bytes take part in the comparison)
    key.base = base;
    key.rank = (uint32_t)rank;
    key.dtype = (uint32_t)dtype;
    key.swizzle = (uint32_t)swizzle;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides[i];
    const uint64_t h = key_hash(key);
    {
        std::lock_guard<std::mutex> lock(g_cache_mutex);
        if (!g_cache) g_cache = new CacheSlot[kCacheSlots]();
        for (int i = 0; i < kCacheProbe; ++i) {
            const CacheSlot &s = g_cache[(h + i) % kCacheSlots];
            if (s.used && memcmp(&s.key, &key, sizeof(key)) == 0) { *map = s.map; return true; }
        }
    }
    const cuuint32_t elem_strides[5] = {1, 1, 1, 1, 1};
    if (fn(map, dtype, rank, const_cast<void *>(base), dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
           swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    int at = (int)(h % kCacheSlots);  // a free slot within the probe window, else the home slot is replaced
    for (int i = 0; i < kCacheProbe; ++i)
        if (!g_cache[(h + i) % kCacheSlots].used) { at = (int)((h + i) % kCacheSlots); break; }
    g_cache[at].key = key;
    g_cache[at].map = *map;
    g_cache[at].used = true;
    return true;
}

// bf16 operands and MX codes land in the 128-byte-swizzled layout the MMA reads; the FP8 codes of the
// dequantising kernel are staged unswizzled for its converter warps.
enum class Operand { kBf16, kCodesForConverter, kCodesForMma };

bool encode(CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides,
            const cuuint32_t *box, Operand kind = Operand::kBf16) {
    return encode_cached(map, kind == Operand::kBf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8,
                         rank, base, dims, strides, box,
                         kind == Operand::kCodesForConverter ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B);
}

}  // namespace

// 5-D bf16 tensor map of a paged key-value cache [num_pages, page_size, Hkv, 128] (decode attention), with the
// dimensions ordered (64 dims, slot, half of the dims, head, page) -- strides need not ascend -- so that one box,
// 64 dims x box_rows slots x 2 halves of one head of one page, lands as two 128-byte-swizzled blocks of box_rows rows.
bool encode_kv_cache_map(CUtensorMap *map, const void *cache, uint64_t num_pages, uint32_t page_size, uint32_t Hkv,
                         uint32_t box_rows) {
    const cuuint64_t dims[5] = {64, page_size, 2, Hkv, num_pages};
    const cuuint64_t strides[4] = {256ull * Hkv, 128, 256, 256ull * Hkv * page_size};
    const cuuint32_t box[5] = {64, box_rows, 2, 1, 1};
    return encode(map, cache, 5, dims, strides, box);
}

namespace {

// 2-D bf16 tensor [rows, cols] row-major; box = box_rows x 64 columns, 128-byte swizzle, zero fill.
bool encode_2d(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    return encode(map, base, 2, dims, strides, box);
}

}  // namespace

bool encode_weight_map_2d(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K) {
    return encode_2d(map, w, rows, K, kTileM);
}

// w13 [E, 2I, H] viewed as [E][I/16 groups][2 halves][16 rows][H]: coordinates (k, row, half, group,
// expert).  The {64,16,2,4,1} box lands in shared memory as, for each of 4 consecutive groups, 16
// gate rows followed by the 16 up rows of the same features: one copy per 128-row A slot.
bool encode_weight_map_gate_up(CUtensorMap *map, const void *w13, int E, int I, int H) {
    const cuuint64_t row_bytes = (cuuint64_t)H * 2;
    const cuuint64_t dims[5] = {(cuuint64_t)H, 16, 2, (cuuint64_t)(I / 16), (cuuint64_t)E};
    const cuuint64_t strides[4] = {row_bytes, (cuuint64_t)I * row_bytes, 16 * row_bytes, 2 * (cuuint64_t)I * row_bytes};
    const cuuint32_t box[5] = {(cuuint32_t)kBlockK, 16, 2, 4, 1};
    return encode(map, w13, 5, dims, strides, box);
}

// The same two weight maps over FP8 codes (one byte per element): [rows, K] with a 128-row x 64-byte box,
// and the gate/up view [E][I/16][2][16][H] with the {64,16,2,4,1} box.
// (FP8 slots are 128 K-elements wide: 128-byte rows of codes.)
bool encode_weight_map_2d_fp8(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K) {
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K};
    const cuuint32_t box[2] = {128, (cuuint32_t)kTileM};
    return encode(map, w, 2, dims, strides, box, Operand::kCodesForConverter);
}

bool encode_weight_map_gate_up_fp8(CUtensorMap *map, const void *w13, int E, int I, int H) {
    const cuuint64_t row_bytes = (cuuint64_t)H;
    const cuuint64_t dims[5] = {(cuuint64_t)H, 16, 2, (cuuint64_t)(I / 16), (cuuint64_t)E};
    const cuuint64_t strides[4] = {row_bytes, (cuuint64_t)I * row_bytes, 16 * row_bytes, 2 * (cuuint64_t)I * row_bytes};
    const cuuint32_t box[5] = {128, 16, 2, 4, 1};
    return encode(map, w13, 5, dims, strides, box, Operand::kCodesForConverter);
}

// MX operands: one byte per element, 128 K-elements (one 128-byte swizzle row) per ring slot.
bool encode_mx_weight_map_2d(CUtensorMap *map, const void *w, uint64_t rows, uint64_t K) {
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K};
    const cuuint32_t box[2] = {128, (cuuint32_t)kTileM};
    return encode(map, w, 2, dims, strides, box, Operand::kCodesForMma);
}

bool encode_mx_weight_map_gate_up(CUtensorMap *map, const void *w13, int E, int I, int H) {
    const cuuint64_t row_bytes = (cuuint64_t)H;
    const cuuint64_t dims[5] = {(cuuint64_t)H, 16, 2, (cuuint64_t)(I / 16), (cuuint64_t)E};
    const cuuint64_t strides[4] = {row_bytes, (cuuint64_t)I * row_bytes, 16 * row_bytes, 2 * (cuuint64_t)I * row_bytes};
    const cuuint32_t box[5] = {128, 16, 2, 4, 1};
    return encode(map, w13, 5, dims, strides, box, Operand::kCodesForMma);
}

bool encode_mx_act_maps(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum) {
    for (int i = 0; i < kNumActMaps; ++i) {
        const cuuint64_t dims[2] = {K, rows};
        const cuuint64_t strides[1] = {K};
        const cuuint32_t box[2] = {128, (cuuint32_t)row_quantum * (cuuint32_t)(i + 1)};
        if (!encode(&maps[i], act, 2, dims, strides, box, Operand::kCodesForMma)) return false;
    }
    return true;
}

// Activation maps whose box spans 128 K-elements: the tensor [rows, K] viewed as [K/64][rows][64], box
// {64, q*(i+1), 2}, so one copy delivers two consecutive 128-byte-swizzled tiles (K 0..63, then 64..127).
bool encode_act_maps_k128(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum) {
    for (int i = 0; i < kNumActMaps; ++i) {
        const cuuint64_t dims[3] = {(cuuint64_t)kBlockK, rows, K / kBlockK};
        const cuuint64_t strides[2] = {K * 2, (cuuint64_t)kBlockK * 2};
        const cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)row_quantum * (cuuint32_t)(i + 1), 2};
        if (!encode(&maps[i], act, 3, dims, strides, box)) return false;
    }
    return true;
}

bool encode_act_maps(CUtensorMap *maps, const void *act, uint64_t rows, uint64_t K, int row_quantum, int count) {
    for (int i = 0; i < count; ++i)
        if (!encode_2d(&maps[i], act, rows, K, (uint32_t)row_quantum * (uint32_t)(i + 1))) return false;
    return true;
}

// [rows, K] bf16 with a box of ONE row of 64 columns: the form TMA's four-row gather (tile::gather4) takes.
bool encode_row_map(CUtensorMap *map, const void *act, uint64_t rows, uint64_t K) { return encode_2d(map, act, rows, K, 1); }

// Scale atoms as a 2-D tensor of 32-bit words: [n_atoms][128 words], box = atoms_per_box whole atoms, unswizzled.
bool encode_scale_atoms(CUtensorMap *map, const void *atoms, uint64_t n_atoms, uint32_t atoms_per_box) {
    const cuuint64_t dims[2] = {kMxSfAtomBytes / 4, n_atoms};
    const cuuint64_t strides[1] = {kMxSfAtomBytes};
    const cuuint32_t box[2] = {kMxSfAtomBytes / 4, atoms_per_box};
    return encode_cached(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, atoms, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per kernel and device instead of once per launch (it is a
// driver call on the host path of every forward call otherwise).  A small table under the cache's mutex.
bool set_max_dynamic_smem_once(const void *kernel, int bytes) {
    struct Entry { const void *kernel; unsigned long long devices; };
    static Entry table[64];
    static int used = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(g_cache_mutex);
    Entry *e = nullptr;
    for (int i = 0; i < used; ++i)
        if (table[i].kernel == kernel) { e = &table[i]; break; }
    if (e && ((e->devices >> dev) & 1ull)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (!e && used < 64) { e = &table[used++]; e->kernel = kernel; e->devices = 0; }
    if (e) e->devices |= 1ull << dev;
    return true;
}

int sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (cached[dev] == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        cached[dev] = n > 0 ? n : 1;
    }
    return cached[dev];
}

}  // namespace tc

namespace mxtc {
bool encode_mx_scale_map(CUtensorMap *map, const void *atoms, uint64_t n_atoms, uint32_t atoms_per_box) {
    return tc::encode_scale_atoms(map, atoms, n_atoms, atoms_per_box);
}
}  // namespace mxtc
}  // namespace moe

// Host-side construction of the TMA tensor map over the int8 activations qa[M,K]:
// tiles of 128 k (one quantisation group, 128 bytes) x `box_rows` tokens, 128-byte swizzle,
// rows past M read as zeros.  The driver entry point is resolved through the runtime so the
// library carries no link-time dependency on libcuda.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstring>
#include <mutex>
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Encoding a map costs the host about a microsecond and depends only on the pointer and the shape, not on
// the memory's contents: the maps of the small-M kernel (three per call) are kept in a small table.
struct MapKey {
    const void* ptr;
    int kind, a, b, c, d;
    bool operator==(const MapKey& o) const {
        return ptr == o.ptr && kind == o.kind && a == o.a && b == o.b && c == o.c && d == o.d;
    }
};
constexpr int MAP_CACHE_SIZE = 64;
struct MapCache {
    std::mutex mu;
    MapKey keys[MAP_CACHE_SIZE];
    CUtensorMap maps[MAP_CACHE_SIZE];
    bool used[MAP_CACHE_SIZE] = {false};
    int next = 0;
    bool find(const MapKey& k, CUtensorMap* out) {
        std::lock_guard<std::mutex> g(mu);
        for (int i = 0; i < MAP_CACHE_SIZE; ++i)
            if (used[i] && keys[i] == k) { std::memcpy(out, &maps[i], sizeof(CUtensorMap)); return true; }
        return false;
    }
    void put(const MapKey& k, const CUtensorMap* m) {
        std::lock_guard<std::mutex> g(mu);
        keys[next] = k;
        std::memcpy(&maps[next], m, sizeof(CUtensorMap));
        used[next] = true;
        next = (next + 1) % MAP_CACHE_SIZE;
    }
};
MapCache& map_cache() {
    static MapCache c;
    return c;
}
}  // namespace

// Views of the packed weights for the strip kernel: a strip is R < 128 consecutive rows of a 128-channel tile
// (whole tiles are fetched with plain bulk copies and need no map).
//   nib    4-D: 16 words of a row, 128 rows (stride 64 B), G groups (stride one blob), tiles; box = one row
//          x R rows x GS groups: the strip's nibbles of GS consecutive groups, laid out [group][row][64 B]
//   scale  3-D over a blob's 128 fp16 scales: box = the strip's R scales x GS groups
//   zero   3-D over a blob's 64 bytes of zero points: box = the strip's R / 2 bytes (16 at least) x GS groups
// A box that reaches past the last group reads zeros there (zero scales: such a group adds nothing).
cudaError_t make_strip_weight_maps(CUtensorMap* nib, CUtensorMap* scale, CUtensorMap* zero, const void* packed,
                                   int N, int K, int R, int GS) {
    if (R >= TILE_N) {
        std::memset(nib, 0, sizeof(CUtensorMap));
        std::memset(scale, 0, sizeof(CUtensorMap));
        std::memset(zero, 0, sizeof(CUtensorMap));
        return cudaSuccess;
    }
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    int dev = 0;
    cudaGetDevice(&dev);
    const MapKey kn = {packed, 1, N, K, R * 256 + GS, dev}, ks = {packed, 2, N, K, R * 256 + GS, dev},
                 kz = {packed, 4, N, K, R * 256 + GS, dev};
    const cuuint64_t G = (cuuint64_t)(K / GROUP), tiles = (cuuint64_t)(N / TILE_N);
    uint8_t* base = static_cast<uint8_t*>(const_cast<void*>(packed));
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    if (!map_cache().find(kn, nib)) {
        const cuuint64_t dims[4] = {16, (cuuint64_t)TILE_N, G, tiles};
        const cuuint64_t strides[3] = {64, (cuuint64_t)BLOB_BYTES, G * BLOB_BYTES};
        const cuuint32_t box[4] = {16, (cuuint32_t)R, (cuuint32_t)GS, 1};
        if (encode(nib, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        map_cache().put(kn, nib);
    }
    const cuuint64_t strides[2] = {(cuuint64_t)BLOB_BYTES, G * BLOB_BYTES};
    if (!map_cache().find(ks, scale)) {
        const cuuint64_t dims[3] = {(cuuint64_t)TILE_N, G, tiles};
        const cuuint32_t box[3] = {(cuuint32_t)R, (cuuint32_t)GS, 1};
        if (encode(scale, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, base + BLOB_SCALE_OFF, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        map_cache().put(ks, scale);
    }
    if (!map_cache().find(kz, zero)) {
        const cuuint64_t dims[3] = {(cuuint64_t)TILE_N / 2, G, tiles};
        const cuuint32_t box[3] = {(cuuint32_t)(R / 2 < 16 ? 16 : R / 2), (cuuint32_t)GS, 1};
        if (encode(zero, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, base + BLOB_ZERO_OFF, dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
        map_cache().put(kz, zero);
    }
    return cudaSuccess;
}

// 3-D view of qa[M,K] as (128 bytes of a group, M tokens, G groups): a box of box_rows tokens x box_groups
// groups lands as [group][token][128 B], i.e. as box_groups of the 2-D map's tiles one after the other
// (128-byte swizzle, tokens past M and groups past G read as zeros).
cudaError_t make_qa_group_map(CUtensorMap* out, const int8_t* qa, int M, int K, int box_rows, int box_groups) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    int dev = 0;
    cudaGetDevice(&dev);
    const MapKey k = {qa, 3, M, K, box_rows * 256 + box_groups, dev};
    if (map_cache().find(k, out)) return cudaSuccess;
    const cuuint64_t dims[3] = {(cuuint64_t)GROUP, (cuuint64_t)M, (cuuint64_t)(K / GROUP)};
    const cuuint64_t strides[2] = {(cuuint64_t)K, (cuuint64_t)GROUP};
    const cuuint32_t box[3] = {(cuuint32_t)GROUP, (cuuint32_t)box_rows, (cuuint32_t)box_groups};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<int8_t*>(qa), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    map_cache().put(k, out);
    return cudaSuccess;
}

// 3-D view of bf16 activations x[M,K] as (64 elements = 128 bytes, M tokens, K / 64 half-groups): a box of box_rows
// tokens x box_halves half-groups lands as [half-group][token][128 B] (128-byte swizzle, zeros past M and K).
cudaError_t make_x_half_group_map(CUtensorMap* out, const void* x, int M, int K, int box_rows, int box_halves) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    int dev = 0;
    cudaGetDevice(&dev);
    const MapKey k = {x, 5, M, K, box_rows * 256 + box_halves, dev};
    if (map_cache().find(k, out)) return cudaSuccess;
    const cuuint64_t dims[3] = {64, (cuuint64_t)M, (cuuint64_t)(K / 64)};
    const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_halves};
    const cuuint32_t estr[3] = {1, 1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    map_cache().put(k, out);
    return cudaSuccess;
}

cudaError_t make_qa_tensor_map(CUtensorMap* out, const int8_t* qa, int M, int K, int box_rows) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K};
    const cuuint32_t box[2] = {(cuuint32_t)GROUP, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<int8_t*>(qa), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    return cudaSuccess;
}

// Map over the bf16 output y[M,N] for the tensor-core kernel's tile stores: boxes of 32 tokens x 32 channels
// (64 bytes per row), no swizzle; rows past M are not written.
cudaError_t make_y_tensor_map(CUtensorMap* out, void* y, int M, int N) {
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return cudaErrorNotSupported;
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)N * 2};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    return cudaSuccess;
}

}  // namespace w4a8

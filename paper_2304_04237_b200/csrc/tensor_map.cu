// Host-side encoder of the TMA tensor maps shared by the tiled kernels: a [B][H][W][C] bf16 tensor
// seen as 4-D (C, W, H, B) with a box of one head's 32 channels x bw columns x bh rows.  Elements
// outside the map read as zero, which is the zero padding of the depthwise convolution (Fig. 2).
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace slide_attn {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

bool tensor_map_available() { return encode_fn() != nullptr; }

namespace {

bool encode_tile_map(EncodeTiledFn fn, CUtensorMap* map, const void* base, int elem_bytes, int B, int H, int W, int C,
                     int box_c, int box_w, int box_h);

// A tensor map is a pure function of the arguments below (it holds the address and the geometry, no
// device state), so recently encoded maps are kept: a forward on buffers it has seen before makes
// no driver call.
struct MapKey {
    const void* base;
    int elem_bytes, B, H, W, C, box_c, box_w, box_h;
    bool operator==(const MapKey& o) const {
        return base == o.base && elem_bytes == o.elem_bytes && B == o.B && H == o.H && W == o.W && C == o.C &&
               box_c == o.box_c && box_w == o.box_w && box_h == o.box_h;
    }
};
constexpr int kCacheSlots = 64;
struct MapCache {
    std::mutex mu;
    MapKey key[kCacheSlots];
    CUtensorMap map[kCacheSlots];
    bool used[kCacheSlots] = {};
    int next = 0;
} g_cache;

}  // namespace

bool make_tile_map(CUtensorMap* map, const void* base, int elem_bytes, int B, int H, int W, int C,
                   int box_c, int box_w, int box_h) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || (elem_bytes != 2 && elem_bytes != 4)) return false;
    const MapKey key = {base, elem_bytes, B, H, W, C, box_c, box_w, box_h};
    {
        std::lock_guard<std::mutex> lock(g_cache.mu);
        for (int i = 0; i < kCacheSlots; ++i)
            if (g_cache.used[i] && g_cache.key[i] == key) { *map = g_cache.map[i]; return true; }
    }
    if (!encode_tile_map(fn, map, base, elem_bytes, B, H, W, C, box_c, box_w, box_h)) return false;
    std::lock_guard<std::mutex> lock(g_cache.mu);
    const int slot = g_cache.next;
    g_cache.next = (slot + 1) % kCacheSlots;
    g_cache.key[slot] = key; g_cache.map[slot] = *map; g_cache.used[slot] = true;
    return true;
}

namespace {

bool encode_tile_map(EncodeTiledFn fn, CUtensorMap* map, const void* base, int elem_bytes, int B, int H, int W, int C,
                     int box_c, int box_w, int box_h) {
    const cuuint64_t eb = (cuuint64_t)elem_bytes;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    const cuuint64_t strides[3] = {(cuuint64_t)C * eb, (cuuint64_t)W * C * eb, (cuuint64_t)H * W * C * eb};
    const cuuint32_t box[4] = {(cuuint32_t)box_c, (cuuint32_t)box_w, (cuuint32_t)box_h, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(map, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

}  // namespace slide_attn

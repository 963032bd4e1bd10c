// Tensor-map (TMA descriptor) construction, cached per context.
#include <cstring>

#include "tc_common.cuh"

namespace ghd {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is looked up through the runtime so that the library does not link libcuda.
EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

bool cached(ghd_ctx* c, const TmapKey& key, CUtensorMap* out) {
    auto it = c->tmaps->find(key);
    if (it == c->tmaps->end()) return false;
    memcpy(out, it->second.data(), sizeof(CUtensorMap));
    return true;
}

void remember(ghd_ctx* c, const TmapKey& key, const CUtensorMap& tm) {
    std::vector<uint64_t> blob(sizeof(CUtensorMap) / 8);
    memcpy(blob.data(), &tm, sizeof(CUtensorMap));
    if (c->tmaps->size() > 8192) c->tmaps->clear();
    (*c->tmaps)[key] = blob;
}

}  // namespace

bool tmap_rows_x_k(ghd_ctx* c, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows, CUtensorMap* out) {
    const TmapKey key{ptr, rows, cols, 1, 0, box_rows, 64};
    if (cached(c, key, out)) return true;
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMap tm;
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    remember(c, key, tm);
    *out = tm;
    return true;
}

bool tmap_slabs(ghd_ctx* c, const void* ptr, uint64_t rows, uint64_t cols, uint32_t halves, uint32_t box_rows, uint32_t ks,
                CUtensorMap* out) {
    const TmapKey key{ptr, rows, cols, halves, 0x51ab0000ull + ks, box_rows, 64};
    if (cached(c, key, out)) return true;
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64 || rows % halves) return false;
    const uint64_t half_rows = rows / halves;
    cuuint64_t dims[4] = {64, half_rows, halves, cols / 64};
    cuuint64_t strides[3] = {cols * 2, half_rows * cols * 2, 128};
    cuuint32_t box[4] = {64, box_rows, halves, ks};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap tm;
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    remember(c, key, tm);
    *out = tm;
    return true;
}

bool tmap_planes_slabs(ghd_ctx* c, const void* ptr, uint64_t planes, uint64_t rows_alloc, uint64_t rows, uint64_t cols,
                       uint32_t box_rows, CUtensorMap* out) {
    const TmapKey key{ptr, rows, cols, planes, rows_alloc + (0x51abull << 48), box_rows, 64};
    if (cached(c, key, out)) return true;
    EncodeTiledFn fn = encode_fn();
    if (!fn || cols % 64) return false;
    cuuint64_t dims[4] = {64, rows, cols / 64, planes};
    cuuint64_t strides[3] = {cols * 2, 128, rows_alloc * cols * 2};
    cuuint32_t box[4] = {64, box_rows, (cuuint32_t)(cols / 64), 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap tm;
    if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    remember(c, key, tm);
    *out = tm;
    return true;
}

}  // namespace ghd

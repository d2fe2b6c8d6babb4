// Host-side construction of TMA tensor maps (driver entry point fetched through the runtime, so
// the library does not link against libcuda).
#pragma once
#include <cstdint>
#include <string>

#include <cuda.h>
#include <cuda_runtime.h>

namespace tessera {

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn(std::string *err) {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        if (err) *err = "cuTensorMapEncodeTiled entry point not available";
        return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

// Tensor of rank 3 or 4 (dims fastest first), 128-byte swizzle, zero fill outside the tensor.
inline bool make_tmap(CUtensorMap *out, CUtensorMapDataType type, const void *base, int rank, const uint64_t *dims,
                      const uint64_t *strides_bytes /* rank-1 entries */, const uint32_t *box, std::string *err) {
    EncodeTiledFn fn = encode_tiled_fn(err);
    if (!fn) return false;
    cuuint32_t elem[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(out, type, (cuuint32_t)rank, const_cast<void *>(base),
                    reinterpret_cast<const cuuint64_t *>(dims), reinterpret_cast<const cuuint64_t *>(strides_bytes),
                    reinterpret_cast<const cuuint32_t *>(box), elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (err) *err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
        return false;
    }
    return true;
}

inline bool make_tmap_bf16(CUtensorMap *out, const void *base, int rank, const uint64_t *dims,
                           const uint64_t *strides_bytes, const uint32_t *box, std::string *err) {
    return make_tmap(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, rank, dims, strides_bytes, box, err);
}

// 8-bit pool [num_pages][page_size][H_kv][D] (one byte per element): box = one page of one head, 128 bytes of D.
inline bool make_pool_tmap8(CUtensorMap *out, const void *pool, int num_pages, int page_size, int H_kv, int D,
                            std::string *err) {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)H_kv, (uint64_t)page_size, (uint64_t)num_pages};
    const uint64_t strides[3] = {(uint64_t)D, (uint64_t)H_kv * D, (uint64_t)page_size * H_kv * D};
    const uint32_t box[4] = {128, 1, (uint32_t)page_size, 1};
    return make_tmap(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, pool, 4, dims, strides, box, err);
}

// 8-bit Q [n_q][H_q][D]: box = (tile_tokens tokens) x (g heads of one KV group) x 128 bytes of D.
inline bool make_q_tmap8(CUtensorMap *out, const void *q, int64_t n_q, int H_q, int D, int g, int tile_tokens,
                         std::string *err) {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)H_q, (uint64_t)n_q};
    const uint64_t strides[2] = {(uint64_t)D, (uint64_t)H_q * D};
    const uint32_t box[3] = {128, (uint32_t)g, (uint32_t)tile_tokens};
    return make_tmap(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, q, 3, dims, strides, box, err);
}

// KV pool [num_pages][page_size][H_kv][D]: box = one page of one head, 64 elements of D.
inline bool make_pool_tmap(CUtensorMap *out, const void *pool, int num_pages, int page_size, int H_kv, int D,
                           std::string *err) {
    const uint64_t dims[4] = {(uint64_t)D, (uint64_t)H_kv, (uint64_t)page_size, (uint64_t)num_pages};
    const uint64_t strides[3] = {(uint64_t)D * 2, (uint64_t)H_kv * D * 2, (uint64_t)page_size * H_kv * D * 2};
    const uint32_t box[4] = {64, 1, (uint32_t)page_size, 1};
    return make_tmap_bf16(out, pool, 4, dims, strides, box, err);
}

// Q [n_q][H_q][D]: box = (tile_tokens tokens) x (g heads of one KV group) x 64 elements of D; the
// box lands in shared memory as rows ordered token-major, head-minor.
inline bool make_q_tmap(CUtensorMap *out, const void *q, int64_t n_q, int H_q, int D, int g, int tile_tokens,
                        std::string *err) {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)H_q, (uint64_t)n_q};
    const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)H_q * D * 2};
    const uint32_t box[3] = {64, (uint32_t)g, (uint32_t)tile_tokens};
    return make_tmap_bf16(out, q, 3, dims, strides, box, err);
}

}  // namespace tessera

// Cached units stored as 8-bit floats (e4m3: 4 exponent bits, 3 mantissa bits, no infinities, largest
// value 448; a stored code c stands for c * scale, one scale per pool).  The paper's system keeps
// conventional 16-bit K/V (Sec. 8); this tier halves the bytes a cache hit moves (Sec. 2.4) and is
// this library's extension.  Two directions, both driven by the plan's copy list and shift table:
//   expand : 8-bit source pool -> the request's 16-bit pages (keys rotated on the way, Sec. 5.3)
//   retain : 16-bit pages -> 8-bit storage pages (keys rotated by the plan's shifts - normally back
//            to the position-free form - then scaled and rounded to nearest-even, saturating)
// A task is the same pair-chunk as in the 16-bit gather: 8 elements of a head and their partners
// D/2 elements later - 8-byte accesses on the 8-bit side, 16-byte accesses on the 16-bit side.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <type_traits>

#include "launch.h"
#include "plan.h"

namespace tessera {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void unpack_bf16x8(const uint4 &v, float (&f)[8]) {
    const uint32_t *w = reinterpret_cast<const uint32_t *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float (&f)[8]) {
    uint4 v;
    uint32_t *w = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t *>(&p);
    }
    return v;
}
// 8 codes -> 8 floats (exact) times mul (one fp32 rounding).
__device__ __forceinline__ void unpack_e4m3x8(const uint2 &v, float mul, float (&f)[8]) {
    const uint32_t w[2] = {v.x, v.y};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_fp8x2_storage_t two = (__nv_fp8x2_storage_t)((w[i >> 1] >> (16 * (i & 1))) & 0xffffu);
        const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(two, __NV_E4M3);
        const float2 x = __half22float2(*reinterpret_cast<const __half2 *>(&h));
        f[2 * i] = __fmul_rn(x.x, mul);
        f[2 * i + 1] = __fmul_rn(x.y, mul);
    }
}
// 8 floats times mul (one fp32 rounding) -> 8 codes, nearest-even, saturating at +-448.
__device__ __forceinline__ uint2 pack_e4m3x8(const float (&f)[8], float mul) {
    uint32_t w[2] = {0u, 0u};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 x = make_float2(__fmul_rn(f[2 * i], mul), __fmul_rn(f[2 * i + 1], mul));
        const uint32_t two = (uint32_t)__nv_cvt_float2_to_fp8x2(x, __NV_SATFINITE, __NV_E4M3);
        w[i >> 1] |= two << (16 * (i & 1));
    }
    return make_uint2(w[0], w[1]);
}

// x' = x cos - y sin, y' = y cos + x sin in fp32, the arithmetic of the 16-bit gather; a table entry
// that is exactly (1, 0) leaves the pair untouched (signed zeros and infinities survive a zero shift).
__device__ __forceinline__ void rotate_pair(float &x, float &y, const float2 c) {
    const bool identity = c.x == 1.f && c.y == 0.f;
    const float a = fmaf(-y, c.y, x * c.x), b = fmaf(x, c.y, y * c.x);
    x = identity ? x : a;
    y = identity ? y : b;
}
template <bool INTERLEAVED>
__device__ __forceinline__ void rotate_f(float (&lo)[8], float (&hi)[8], const float2 *cs) {
    if (INTERLEAVED) {
        // lo holds pairs (0,1) (2,3) .. with cs[0..3]; hi the chunk D/2 elements later with cs[4..7]
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            rotate_pair(lo[2 * i], lo[2 * i + 1], cs[i]);
            rotate_pair(hi[2 * i], hi[2 * i + 1], cs[4 + i]);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) rotate_pair(lo[i], hi[i], cs[i]);
    }
}
template <int D, bool INTERLEAVED>
__device__ __forceinline__ int cs_index(int c, int i) {
    return INTERLEAVED ? (i < 4 ? 4 * c + i : 4 * c + D / 4 + (i - 4)) : c * 8 + i;
}

// One thread block per GatherItem.  TO_8BIT false: sources are e4m3 (mul = scale), destinations bf16;
// TO_8BIT true: sources are bf16, destinations e4m3 (mul = 1 / scale, applied after the rotation); with V16
// only the keys go 8-bit and the value rows are bit copies into a 16-bit pool (key pages for the 8-bit
// attention path, values as everywhere else).
template <int D, bool TO_8BIT, bool ROTATE, bool INTERLEAVED, bool V16 = false>
__global__ void __launch_bounds__(kThreads)
kv_fp8_kernel(const void *__restrict__ k_src, const void *__restrict__ v_src, void *__restrict__ k_dst,
              void *__restrict__ v_dst, const int32_t *__restrict__ g_src, const int32_t *__restrict__ g_dst,
              const GatherItem *__restrict__ items, int n_items, const float2 *__restrict__ rope, int H_kv, float k_mul,
              float v_mul) {
    constexpr int CPH = D / 16;          // pair-chunks per head
    constexpr int HALF = D / 16;         // distance (in 8-element chunks) between pair partners
    __shared__ float2 s_rope[kGatherItemTokens * (D / 2)];
    __shared__ int32_t s_src[kGatherItemTokens], s_dst[kGatherItemTokens];

    const int tid = threadIdx.x;
    // one item per thread block, or - when launched with fewer blocks than items - a walk through the list
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const GatherItem it = items[item];
    const int n_rows = ROTATE ? (it.row_step ? it.count : 1) : 0;
    const int first_row = it.row_step < 0 ? it.row0 - (it.count - 1) : it.row0;
    for (int i = tid; i < n_rows * (D / 2); i += kThreads) s_rope[i] = rope[(size_t)first_row * (D / 2) + i];
    if (tid < it.count) {
        s_dst[tid] = g_dst[it.begin + tid];
        s_src[tid] = g_src[it.begin + tid];
    }
    __syncthreads();

    const int tasks_per_row = H_kv * CPH;
    const int row_chunks = H_kv * (D / 8);
    const int n_tasks = it.count * tasks_per_row;
    const int c = tid % CPH;
    using Raw = typename std::conditional<TO_8BIT, uint4, uint2>::type;   // one 8-element chunk of the source
    const Raw *ks = static_cast<const Raw *>(k_src), *vs = static_cast<const Raw *>(v_src);
    constexpr int U = 2;                 // tasks in flight per thread: all loads of both are issued first
    for (int t0 = tid; t0 < n_tasks; t0 += U * kThreads) {
        Raw rk[U][2], rv[U][2];
        size_t dso[U];
        int tok[U];
        bool ok[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int t = t0 + u * kThreads;
            ok[u] = t < n_tasks;
            if (!ok[u]) continue;
            tok[u] = t / tasks_per_row;
            const int w = t - tok[u] * tasks_per_row;
            const int chunk = (w / CPH) * (D / 8) + c;
            const size_t so = (size_t)s_src[tok[u]] * row_chunks + chunk;
            dso[u] = (size_t)s_dst[tok[u]] * row_chunks + chunk;
            rk[u][0] = __ldg(ks + so);
            rk[u][1] = __ldg(ks + so + HALF);
            rv[u][0] = __ldg(vs + so);
            rv[u][1] = __ldg(vs + so + HALF);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            float klo[8], khi[8], vlo[8], vhi[8];
            if constexpr (TO_8BIT) {
                unpack_bf16x8(rk[u][0], klo);
                unpack_bf16x8(rk[u][1], khi);
                unpack_bf16x8(rv[u][0], vlo);
                unpack_bf16x8(rv[u][1], vhi);
            } else {
                unpack_e4m3x8(rk[u][0], k_mul, klo);
                unpack_e4m3x8(rk[u][1], k_mul, khi);
                unpack_e4m3x8(rv[u][0], v_mul, vlo);
                unpack_e4m3x8(rv[u][1], v_mul, vhi);
            }
            if (ROTATE) {
                const int sr = it.row_step == 0 ? 0 : (it.row_step < 0 ? it.count - 1 - tok[u] : tok[u]);
                const float2 *row = s_rope + (size_t)sr * (D / 2);
                float2 cr[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) cr[i] = row[cs_index<D, INTERLEAVED>(c, i)];
                rotate_f<INTERLEAVED>(klo, khi, cr);
            }
            if constexpr (TO_8BIT) {
                uint2 *kd = static_cast<uint2 *>(k_dst);
                kd[dso[u]] = pack_e4m3x8(klo, k_mul);
                kd[dso[u] + HALF] = pack_e4m3x8(khi, k_mul);
                if constexpr (V16) {
                    uint4 *vd = static_cast<uint4 *>(v_dst);
                    vd[dso[u]] = rv[u][0];
                    vd[dso[u] + HALF] = rv[u][1];
                } else {
                    uint2 *vd = static_cast<uint2 *>(v_dst);
                    vd[dso[u]] = pack_e4m3x8(vlo, v_mul);
                    vd[dso[u] + HALF] = pack_e4m3x8(vhi, v_mul);
                }
            } else {
                uint4 *kd = static_cast<uint4 *>(k_dst), *vd = static_cast<uint4 *>(v_dst);
                kd[dso[u]] = pack_bf16x8(klo);
                kd[dso[u] + HALF] = pack_bf16x8(khi);
                vd[dso[u]] = pack_bf16x8(vlo);
                vd[dso[u] + HALF] = pack_bf16x8(vhi);
            }
        }
    }
    __syncthreads();          // the staged rows are rewritten by the next item
    }
}

// bf16 -> e4m3 codes of (value * mul): 8 elements per thread, grid-stride.
__global__ void __launch_bounds__(256)
quantize_e4m3_kernel(const uint4 *__restrict__ src, uint2 *__restrict__ dst, int64_t n_chunks, float mul) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_chunks; e += (int64_t)gridDim.x * blockDim.x) {
        float f[8];
        unpack_bf16x8(__ldg(src + e), f);
        dst[e] = pack_e4m3x8(f, mul);
    }
}

// Fresh rows of the recompute tokens into an 8-bit key pool and a 16-bit value pool (Sec. 5.3: recomputed
// states override cached ones): K as the e4m3 code of (k * k_mul), V as a bit copy.
__global__ void __launch_bounds__(256)
scatter_fresh_k8_kernel(uint2 *__restrict__ k_pool8, uint4 *__restrict__ v_pool, const uint4 *__restrict__ k_new,
                        const uint4 *__restrict__ v_new, const int32_t *__restrict__ fresh_dst, int64_t n_chunks,
                        int row_chunks, float k_mul) {
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_chunks; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = e / row_chunks;
        const int c = (int)(e - j * row_chunks);
        const size_t o = (size_t)fresh_dst[j] * row_chunks + c;
        if (k_new) {
            float f[8];
            unpack_bf16x8(__ldg(k_new + e), f);
            k_pool8[o] = pack_e4m3x8(f, k_mul);
        }
        if (v_new) v_pool[o] = __ldg(v_new + e);
    }
}

template <int D, bool TO_8BIT, bool IL>
cudaError_t launch_d(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst, bool rotate,
                     float k_mul, float v_mul, const int32_t *g_src, int first_item, int n, int max_blocks, cudaStream_t st) {
    if (n == 0) return cudaSuccess;
    const int grid = max_blocks > 0 ? (n < max_blocks ? n : max_blocks) : n;
    const DeviceTables &d = pl->dev;
    const GatherItem *items = d.items + first_item;
    const int H = pl->cfg.num_kv_heads;
    if (rotate)
        kv_fp8_kernel<D, TO_8BIT, true, IL><<<grid, kThreads, 0, st>>>(k_src, v_src, k_dst, v_dst, g_src, d.g_dst, items, n, d.rope, H, k_mul, v_mul);
    else
        kv_fp8_kernel<D, TO_8BIT, false, IL><<<grid, kThreads, 0, st>>>(k_src, v_src, k_dst, v_dst, g_src, d.g_dst, items, n, d.rope, H, k_mul, v_mul);
    count_launch();
    return cudaGetLastError();
}

template <bool TO_8BIT>
cudaError_t launch_dir(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst, bool rotate,
                       float k_mul, float v_mul, const int32_t *g_src, int first_item, int n, int max_blocks, cudaStream_t st) {
    const bool il = pl->cfg.rope_pairing == 1;
    if (pl->cfg.head_dim == 128)
        return il ? launch_d<128, TO_8BIT, true>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n, max_blocks, st)
                  : launch_d<128, TO_8BIT, false>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n, max_blocks, st);
    return il ? launch_d<64, TO_8BIT, true>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n, max_blocks, st)
              : launch_d<64, TO_8BIT, false>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n, max_blocks, st);
}

}  // namespace

// Keys rotated and quantised into an 8-bit pool, values copied into a 16-bit pool (sources 16-bit).
cudaError_t launch_compose_k8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst8, void *v_dst,
                              bool rotate, float k_mul, cudaStream_t st) {
    const int n = (int)pl->items.size();
    if (n == 0) return cudaSuccess;
    const DeviceTables &d = pl->dev;
    const int H = pl->cfg.num_kv_heads;
    const bool il = pl->cfg.rope_pairing == 1;
#define TESSERA_K8_LAUNCH(DD, ROT, IL) \
    kv_fp8_kernel<DD, true, ROT, IL, true><<<n, kThreads, 0, st>>>(k_src, v_src, k_dst8, v_dst, d.g_src, d.g_dst, d.items, n, d.rope, H, k_mul, 1.f)
    if (pl->cfg.head_dim == 128) {
        if (rotate) { if (il) TESSERA_K8_LAUNCH(128, true, true); else TESSERA_K8_LAUNCH(128, true, false); }
        else { if (il) TESSERA_K8_LAUNCH(128, false, true); else TESSERA_K8_LAUNCH(128, false, false); }
    } else {
        if (rotate) { if (il) TESSERA_K8_LAUNCH(64, true, true); else TESSERA_K8_LAUNCH(64, true, false); }
        else { if (il) TESSERA_K8_LAUNCH(64, false, true); else TESSERA_K8_LAUNCH(64, false, false); }
    }
#undef TESSERA_K8_LAUNCH
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_quantize_e4m3(const void *src_bf16, void *dst8, int64_t n_elems, float mul, cudaStream_t st) {
    const int64_t n_chunks = n_elems / 8;
    if (n_chunks == 0) return cudaSuccess;
    const int blocks = (int)std::min<int64_t>((n_chunks + 255) / 256, 148 * 16);
    quantize_e4m3_kernel<<<blocks, 256, 0, st>>>(static_cast<const uint4 *>(src_bf16), static_cast<uint2 *>(dst8), n_chunks, mul);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_scatter_fresh_k8(const tessera_plan *pl, void *k_pool8, void *v_pool, const void *k_new,
                                    const void *v_new, float k_mul, cudaStream_t st) {
    if (pl->n_q == 0 || (!k_new && !v_new)) return cudaSuccess;
    const int row_chunks = pl->cfg.num_kv_heads * pl->cfg.head_dim / 8;
    const int64_t n_chunks = pl->n_q * row_chunks;
    const int blocks = (int)std::min<int64_t>((n_chunks + 255) / 256, (int64_t)pl->num_sms * 16);
    scatter_fresh_k8_kernel<<<blocks, 256, 0, st>>>(static_cast<uint2 *>(k_pool8), static_cast<uint4 *>(v_pool),
                                                   static_cast<const uint4 *>(k_new), static_cast<const uint4 *>(v_new),
                                                   pl->dev.fresh_dst, n_chunks, row_chunks, k_mul);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_kv_fp8_range(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst,
                                bool to_8bit, bool rotate, float k_mul, float v_mul, const int32_t *g_src, int first_item,
                                int n_items, int max_blocks, cudaStream_t st) {
    return to_8bit ? launch_dir<true>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n_items, max_blocks, st)
                   : launch_dir<false>(pl, k_src, v_src, k_dst, v_dst, rotate, k_mul, v_mul, g_src, first_item, n_items, max_blocks, st);
}

cudaError_t launch_kv_fp8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst,
                          bool to_8bit, bool rotate, float k_mul, float v_mul, cudaStream_t st) {
    return launch_kv_fp8_range(pl, k_src, v_src, k_dst, v_dst, to_8bit, rotate, k_mul, v_mul, pl->dev.g_src, 0,
                               (int)pl->items.size(), 0, st);
}

}  // namespace tessera

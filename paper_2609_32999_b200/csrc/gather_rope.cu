// Gather + RoPE shift (HBM-bound) and the fresh-row scatter.
//
// gather_rope_kernel moves cached token rows from their source slots to the request's destination
// slots (Sec. 5.3 "Preparing cache hits").  V rows are bit copies; K rows are either bit copies or
// rotated by the unit's shift on the way (Sec. 2.2: keys carry the rotation, values do not).
// Every global access is a 16-byte chunk; the two halves of a rotary pair (m, m + D/2) of one head
// are loaded by the same thread, so no data crosses lanes.  The cos/sin rows an item needs are
// staged in shared memory once per thread block.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "launch.h"
#include "plan.h"

namespace tessera {

namespace {

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 ldg_plain(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void stg(uint4 *p, const uint4 &v) {
    asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// One rotary pair in fp32: (x, y) -> (x cos - y sin, y cos + x sin).  A table entry that is exactly
// (1, 0) - a shift of zero, or a frequency of zero - returns the inputs themselves, so such elements
// stay bit copies (the fused multiply-add would turn -0.0 into +0.0 and 0 x Inf into NaN).
__device__ __forceinline__ void rotate_pair(float &x, float &y, const float2 c) {
    const bool identity = c.x == 1.f && c.y == 0.f;
    const float a = fmaf(-y, c.y, x * c.x), b = fmaf(x, c.y, y * c.x);
    x = identity ? x : a;
    y = identity ? y : b;
}

// Rotates 8 pairs: lo holds x_m, hi holds x_{m + D/2}, cs[i] = (cos, sin) of pair i; one
// round-to-nearest-even to bf16 (exact for elements that were left alone).
__device__ __forceinline__ void rotate8(uint4 &lo, uint4 &hi, const float2 *cs) {
    uint32_t *l = reinterpret_cast<uint32_t *>(&lo);
    uint32_t *h = reinterpret_cast<uint32_t *>(&hi);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float x0 = __uint_as_float(l[i] << 16), x1 = __uint_as_float(l[i] & 0xffff0000u);
        float y0 = __uint_as_float(h[i] << 16), y1 = __uint_as_float(h[i] & 0xffff0000u);
        rotate_pair(x0, y0, cs[2 * i]);
        rotate_pair(x1, y1, cs[2 * i + 1]);
        __nv_bfloat162 pa = __floats2bfloat162_rn(x0, x1), pb = __floats2bfloat162_rn(y0, y1);
        l[i] = *reinterpret_cast<uint32_t *>(&pa);
        h[i] = *reinterpret_cast<uint32_t *>(&pb);
    }
}

// Interleaved pairing: pair m = (element 2m, element 2m + 1).  One 16-byte chunk holds 4 whole pairs;
// cs[0..3] are the (cos, sin) of the chunk's pairs.
__device__ __forceinline__ void rotate4_interleaved(uint4 &v, const float2 *cs) {
    uint32_t *w = reinterpret_cast<uint32_t *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float x = __uint_as_float(w[i] << 16), y = __uint_as_float(w[i] & 0xffff0000u);
        rotate_pair(x, y, cs[i]);
        __nv_bfloat162 p = __floats2bfloat162_rn(x, y);
        w[i] = *reinterpret_cast<uint32_t *>(&p);
    }
}
// Rotates the two chunks a task holds.  Half-split pairing: lo / hi are the two halves of 8 pairs and
// cs = the 8 (cos, sin) of pairs 8c .. 8c+7.  Interleaved: lo holds pairs 4c .. 4c+3 (cs[0..3]) and hi,
// D/2 elements later, pairs 4c + D/4 .. (cs[4..7]).
template <bool INTERLEAVED>
__device__ __forceinline__ void rotate_task(uint4 &lo, uint4 &hi, const float2 *cs) {
    if (INTERLEAVED) {
        rotate4_interleaved(lo, cs);
        rotate4_interleaved(hi, cs + 4);
    } else {
        rotate8(lo, hi, cs);
    }
}
// Index (within a D/2-entry cos/sin row) of entry i of the 8 a task with chunk index c needs.
template <int D, bool INTERLEAVED>
__device__ __forceinline__ int cs_index(int c, int i) {
    return INTERLEAVED ? (i < 4 ? 4 * c + i : 4 * c + D / 4 + (i - 4)) : c * 8 + i;
}

constexpr int kThreads = 256;

// One thread block per GatherItem.  A "task" is one rotary pair-chunk of one token row: the 16-byte
// chunk holding elements [8c, 8c+8) of a head and its partner chunk D/2 elements later (K), plus the
// same two chunks of the V row.  IN_PLACE: source = destination, K only (the standalone shift).
template <int D, bool DO_V, bool ROTATE, bool IN_PLACE, bool INTERLEAVED>
__global__ void __launch_bounds__(kThreads)
gather_rope_kernel(const uint4 *k_src, const uint4 *v_src, uint4 *k_pool, uint4 *v_pool,
                   const int32_t *__restrict__ g_src, const int32_t *__restrict__ g_dst,
                   const GatherItem *__restrict__ items, int n_items, const float2 *__restrict__ rope, int H_kv) {
    constexpr int CPH = D / 16;          // pair-chunks per head
    constexpr int HALF = D / 16;         // distance (in 16-byte chunks) between pair partners
    __shared__ float2 s_rope[kGatherItemTokens * (D / 2)];
    __shared__ int32_t s_src[kGatherItemTokens], s_dst[kGatherItemTokens];

    const int tid = threadIdx.x;
    // one item per thread block in the ordinary launch; a launch with fewer blocks than items (the
    // host-tier reader, which must leave most SMs to the attention kernel) walks the list
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const GatherItem it = items[item];
    // rows row0, row0 + step, ... of the table; with step = -1 they are staged in ascending order
    const int n_rows = ROTATE ? (it.row_step ? it.count : 1) : 0;
    const int first_row = it.row_step < 0 ? it.row0 - (it.count - 1) : it.row0;
    for (int i = tid; i < n_rows * (D / 2); i += kThreads) s_rope[i] = rope[(size_t)first_row * (D / 2) + i];
    if (tid < it.count) {
        s_dst[tid] = g_dst[it.begin + tid];
        s_src[tid] = IN_PLACE ? s_dst[tid] : g_src[it.begin + tid];
    }
    __syncthreads();

    const int tasks_per_row = H_kv * CPH;
    const int row_chunks = H_kv * (D / 8);
    const int n_tasks = it.count * tasks_per_row;
    const int c = tid % CPH;             // kThreads and tasks_per_row are multiples of CPH
    float2 cs[8];
    if (ROTATE && it.row_step == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) cs[i] = s_rope[cs_index<D, INTERLEAVED>(c, i)];
    }

    constexpr int U = 2;                 // tasks in flight per thread
    for (int t0 = tid; t0 < n_tasks; t0 += U * kThreads) {
        uint4 klo[U], khi[U], vlo[U], vhi[U];
        size_t dsto[U];
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
            dsto[u] = (size_t)s_dst[tok[u]] * row_chunks + chunk;
            if (IN_PLACE) {
                klo[u] = ldg_plain(k_pool + so);
                khi[u] = ldg_plain(k_pool + so + HALF);
            } else {
                klo[u] = ldg_stream(k_src + so);
                khi[u] = ldg_stream(k_src + so + HALF);
            }
            if (DO_V) {
                vlo[u] = ldg_stream(v_src + so);
                vhi[u] = ldg_stream(v_src + so + HALF);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!ok[u]) continue;
            if (DO_V) {
                stg(v_pool + dsto[u], vlo[u]);
                stg(v_pool + dsto[u] + HALF, vhi[u]);
            }
            if (ROTATE) {
                if (it.row_step != 0) {
                    const int sr = it.row_step < 0 ? it.count - 1 - tok[u] : tok[u];
                    const float2 *row = s_rope + (size_t)sr * (D / 2);
                    float2 cr[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) cr[i] = row[cs_index<D, INTERLEAVED>(c, i)];
                    rotate_task<INTERLEAVED>(klo[u], khi[u], cr);
                } else {
                    rotate_task<INTERLEAVED>(klo[u], khi[u], cs);
                }
            }
            stg(k_pool + dsto[u], klo[u]);
            stg(k_pool + dsto[u] + HALF, khi[u]);
        }
    }
    __syncthreads();          // the staged rows are rewritten by the next item
    }
}

// Writes the recomputed K / V rows into their destination slots (Sec. 5.3 "Completing prefill":
// recomputed states are private to the request and override the cached ones).
__global__ void __launch_bounds__(256)
scatter_fresh_kernel(uint4 *__restrict__ k_pool, uint4 *__restrict__ v_pool,
                     const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                     const int32_t *__restrict__ fresh_dst, int64_t first_chunk, int64_t n_chunks, int row_chunks) {
    for (int64_t e = first_chunk + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < first_chunk + n_chunks;
         e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = e / row_chunks;
        const int c = (int)(e - j * row_chunks);
        const size_t o = (size_t)fresh_dst[j] * row_chunks + c;
        if (k_new) stg(k_pool + o, ldg_stream(k_new + e));
        if (v_new) stg(v_pool + o, ldg_stream(v_new + e));
    }
}

// Rotates the fresh q and k_new rows of recompute row j for position q_pos[j] (Sec. 2.2 / 5.3).  One
// thread block per row: the first D/2 threads evaluate cos / sin of (position x frequency) in fp64,
// then every thread rotates pair-chunks exactly as the gather kernel does.
template <int D, bool INTERLEAVED>
__global__ void __launch_bounds__(128)
rope_fresh_kernel(uint4 *__restrict__ q, uint4 *__restrict__ k_new, const int32_t *__restrict__ q_pos,
                  const double *__restrict__ inv_freq, int H_q, int H_kv) {
    constexpr int CPH = D / 16, HALF = D / 16;
    __shared__ float2 s_cs[D / 2];
    const int j = blockIdx.x, tid = threadIdx.x;
    if (tid < D / 2) {
        double sn, cs;
        sincos((double)q_pos[j] * inv_freq[tid], &sn, &cs);
        s_cs[tid] = make_float2((float)cs, (float)sn);
    }
    __syncthreads();
    const int c = tid % CPH;
    float2 cr[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) cr[i] = s_cs[cs_index<D, INTERLEAVED>(c, i)];
    for (int pass = 0; pass < 2; ++pass) {
        uint4 *base = pass ? k_new : q;
        const int heads = pass ? H_kv : H_q;
        if (!base) continue;
        uint4 *row = base + (size_t)j * heads * (D / 8);
        for (int t = tid; t < heads * CPH; t += 128) {
            uint4 *plo = row + (t / CPH) * (D / 8) + c, *phi = plo + HALF;
            uint4 lo = *plo, hi = *phi;
            rotate_task<INTERLEAVED>(lo, hi, cr);
            *plo = lo;
            *phi = hi;
        }
    }
}


// Write side of the extend pass in one pass over the fresh rows (Sec. 5.3 "Completing prefill"; Sec. 6.1:
// the forward path captures pre-RoPE keys and values).  A thread block owns kExtendRows consecutive
// recompute rows: D/2 threads per row evaluate cos / sin of (position x frequency) in fp64, then the
// block walks the rows' pair-chunk tasks.  A key task reads the un-rotated chunk pair once, stores the
// raw bits to the captured unit's cache slot (if any), rotates and stores to the request's slot; a
// value task copies to both; a query task rotates in place.
constexpr int kExtendRows = 4;
template <int D, bool INTERLEAVED>
__global__ void __launch_bounds__(256)
extend_write_kernel(uint4 *__restrict__ q, const uint4 *__restrict__ k_raw, const uint4 *__restrict__ v_new,
                    uint4 *k_pool, uint4 *v_pool, uint4 *k_cache, uint4 *v_cache, const int32_t *__restrict__ q_pos, const int32_t *__restrict__ fresh_dst,
                    const int32_t *__restrict__ retain_dst, const double *__restrict__ inv_freq, int n_q, int H_q, int H_kv) {
    constexpr int CPH = D / 16, HALF = D / 16;
    __shared__ float2 s_cs[kExtendRows][D / 2];
    __shared__ int32_t s_dst[kExtendRows], s_keep[kExtendRows];
    const int tid = threadIdx.x;
    const int j0 = blockIdx.x * kExtendRows;
    const int rows = min(kExtendRows, n_q - j0);
    for (int i = tid; i < rows * (D / 2); i += 256) {
        const int r = i / (D / 2), m = i % (D / 2);
        double sn, cs;
        sincos((double)q_pos[j0 + r] * inv_freq[m], &sn, &cs);
        s_cs[r][m] = make_float2((float)cs, (float)sn);
    }
    if (tid < rows) {
        s_dst[tid] = fresh_dst[j0 + tid];
        s_keep[tid] = retain_dst ? retain_dst[j0 + tid] : -1;
    }
    __syncthreads();
    const int c = tid % CPH;                        // 256 and every task count below are multiples of CPH
    const int kv_tasks = H_kv * CPH, q_tasks = q ? H_q * CPH : 0;
    const int row_chunks = H_kv * (D / 8);
    // keys and values: task t of row r = head t / CPH, pair-chunk c
    for (int t = tid; t < rows * kv_tasks; t += 256) {
        const int r = t / kv_tasks, w = t - r * kv_tasks;
        const int chunk = (w / CPH) * (D / 8) + c;
        const size_t so = (size_t)(j0 + r) * row_chunks + chunk;
        uint4 klo = ldg_stream(k_raw + so), khi = ldg_stream(k_raw + so + HALF);
        const uint4 vlo = ldg_stream(v_new + so), vhi = ldg_stream(v_new + so + HALF);
        const size_t dso = (size_t)s_dst[r] * row_chunks + chunk;
        stg(v_pool + dso, vlo);
        stg(v_pool + dso + HALF, vhi);
        if (s_keep[r] >= 0) {
            const size_t co = (size_t)s_keep[r] * row_chunks + chunk;
            stg(k_cache + co, klo);
            stg(k_cache + co + HALF, khi);
            stg(v_cache + co, vlo);
            stg(v_cache + co + HALF, vhi);
        }
        float2 cr[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) cr[i] = s_cs[r][cs_index<D, INTERLEAVED>(c, i)];
        rotate_task<INTERLEAVED>(klo, khi, cr);
        stg(k_pool + dso, klo);
        stg(k_pool + dso + HALF, khi);
    }
    // queries, in place
    const int q_chunks = H_q * (D / 8);
    for (int t = tid; t < rows * q_tasks; t += 256) {
        const int r = t / q_tasks, w = t - r * q_tasks;
        uint4 *plo = q + (size_t)(j0 + r) * q_chunks + (w / CPH) * (D / 8) + c, *phi = plo + HALF;
        uint4 lo = ldg_plain(plo), hi = ldg_plain(phi);
        float2 cr[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) cr[i] = s_cs[r][cs_index<D, INTERLEAVED>(c, i)];
        rotate_task<INTERLEAVED>(lo, hi, cr);
        stg(plo, lo);
        stg(phi, hi);
    }
}

template <int D, bool IL>
cudaError_t launch_gather_d(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                            GatherMode mode, const int32_t *g_src, int first_item, int n, int max_blocks, cudaStream_t st) {
    if (n == 0) return cudaSuccess;
    const int grid = max_blocks > 0 ? std::min(n, max_blocks) : n;
    auto *kp = static_cast<uint4 *>(k_pool);
    auto *vp = static_cast<uint4 *>(v_pool);
    auto *ks = static_cast<const uint4 *>(k_src);
    auto *vs = static_cast<const uint4 *>(v_src);
    const DeviceTables &d = pl->dev;
    const GatherItem *items = d.items + first_item;
    const int H = pl->cfg.num_kv_heads;
    switch (mode) {
        case GatherMode::kCopy:
            gather_rope_kernel<D, true, false, false, IL><<<grid, kThreads, 0, st>>>(ks, vs, kp, vp, g_src, d.g_dst, items, n, d.rope, H);
            break;
        case GatherMode::kCopyRotate:
            gather_rope_kernel<D, true, true, false, IL><<<grid, kThreads, 0, st>>>(ks, vs, kp, vp, g_src, d.g_dst, items, n, d.rope, H);
            break;
        case GatherMode::kShiftInPlace:
            gather_rope_kernel<D, false, true, true, IL><<<grid, kThreads, 0, st>>>(ks, vs, kp, vp, g_src, d.g_dst, items, n, d.rope, H);
            break;
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_gather_range(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                                GatherMode mode, const int32_t *g_src, int first_item, int n_items, int max_blocks,
                                cudaStream_t st) {
    const bool il = pl->cfg.rope_pairing == 1;
    if (pl->cfg.head_dim == 128)
        return il ? launch_gather_d<128, true>(pl, k_src, v_src, k_pool, v_pool, mode, g_src, first_item, n_items, max_blocks, st)
                  : launch_gather_d<128, false>(pl, k_src, v_src, k_pool, v_pool, mode, g_src, first_item, n_items, max_blocks, st);
    return il ? launch_gather_d<64, true>(pl, k_src, v_src, k_pool, v_pool, mode, g_src, first_item, n_items, max_blocks, st)
              : launch_gather_d<64, false>(pl, k_src, v_src, k_pool, v_pool, mode, g_src, first_item, n_items, max_blocks, st);
}

cudaError_t launch_gather(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                          GatherMode mode, cudaStream_t st) {
    return launch_gather_range(pl, k_src, v_src, k_pool, v_pool, mode, pl->dev.g_src, 0, (int)pl->items.size(), 0, st);
}

cudaError_t launch_rope_fresh(const tessera_plan *pl, void *q, void *k_new, cudaStream_t st) {
    if (pl->n_q == 0 || (!q && !k_new)) return cudaSuccess;
    const DeviceTables &d = pl->dev;
    auto *qp = static_cast<uint4 *>(q);
    auto *kp = static_cast<uint4 *>(k_new);
    const int Hq = pl->cfg.num_q_heads, Hkv = pl->cfg.num_kv_heads;
    const unsigned n = (unsigned)pl->n_q;
    const bool il = pl->cfg.rope_pairing == 1;
    if (pl->cfg.head_dim == 128) {
        if (il) rope_fresh_kernel<128, true><<<n, 128, 0, st>>>(qp, kp, d.q_pos, d.inv_freq, Hq, Hkv);
        else rope_fresh_kernel<128, false><<<n, 128, 0, st>>>(qp, kp, d.q_pos, d.inv_freq, Hq, Hkv);
    } else {
        if (il) rope_fresh_kernel<64, true><<<n, 128, 0, st>>>(qp, kp, d.q_pos, d.inv_freq, Hq, Hkv);
        else rope_fresh_kernel<64, false><<<n, 128, 0, st>>>(qp, kp, d.q_pos, d.inv_freq, Hq, Hkv);
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_extend_write(const tessera_plan *pl, void *k_pool, void *v_pool, void *q, const void *k_new_raw,
                                const void *v_new, void *k_cache, void *v_cache, cudaStream_t st) {
    if (pl->n_q == 0) return cudaSuccess;
    const DeviceTables &d = pl->dev;
    const int Hq = pl->cfg.num_q_heads, Hkv = pl->cfg.num_kv_heads, n_q = (int)pl->n_q;
    const unsigned blocks = (unsigned)((n_q + kExtendRows - 1) / kExtendRows);
    auto *qp = static_cast<uint4 *>(q);
    auto *kr = static_cast<const uint4 *>(k_new_raw), *vn = static_cast<const uint4 *>(v_new);
    auto *kp = static_cast<uint4 *>(k_pool), *vp = static_cast<uint4 *>(v_pool);
    auto *kc = static_cast<uint4 *>(k_cache), *vc = static_cast<uint4 *>(v_cache);
    const int32_t *keep = pl->retained_tokens > 0 ? d.retain_dst : nullptr;
    const bool il = pl->cfg.rope_pairing == 1;
    if (pl->cfg.head_dim == 128) {
        if (il) extend_write_kernel<128, true><<<blocks, 256, 0, st>>>(qp, kr, vn, kp, vp, kc, vc, d.q_pos, d.fresh_dst, keep, d.inv_freq, n_q, Hq, Hkv);
        else extend_write_kernel<128, false><<<blocks, 256, 0, st>>>(qp, kr, vn, kp, vp, kc, vc, d.q_pos, d.fresh_dst, keep, d.inv_freq, n_q, Hq, Hkv);
    } else {
        if (il) extend_write_kernel<64, true><<<blocks, 256, 0, st>>>(qp, kr, vn, kp, vp, kc, vc, d.q_pos, d.fresh_dst, keep, d.inv_freq, n_q, Hq, Hkv);
        else extend_write_kernel<64, false><<<blocks, 256, 0, st>>>(qp, kr, vn, kp, vp, kc, vc, d.q_pos, d.fresh_dst, keep, d.inv_freq, n_q, Hq, Hkv);
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_scatter_fresh(const tessera_plan *pl, void *k_pool, void *v_pool, const void *k_new,
                                 const void *v_new, int chunk, cudaStream_t st) {
    if (pl->n_q == 0 || (!k_new && !v_new)) return cudaSuccess;
    const int row_chunks = pl->cfg.num_kv_heads * pl->cfg.head_dim / 8;
    const int64_t row0 = chunk < 0 ? 0 : pl->chunk_row_off[chunk];
    const int64_t rows = chunk < 0 ? pl->n_q : pl->chunk_row_off[chunk + 1] - row0;
    if (rows == 0) return cudaSuccess;
    const int64_t n_chunks = rows * row_chunks;
    const int blocks = (int)std::min<int64_t>((n_chunks + 255) / 256, (int64_t)pl->num_sms * 16);
    scatter_fresh_kernel<<<blocks, 256, 0, st>>>(static_cast<uint4 *>(k_pool), static_cast<uint4 *>(v_pool),
                                                static_cast<const uint4 *>(k_new), static_cast<const uint4 *>(v_new),
                                                pl->dev.fresh_dst, row0 * row_chunks, n_chunks, row_chunks);
    count_launch();
    return cudaGetLastError();
}

}  // namespace tessera

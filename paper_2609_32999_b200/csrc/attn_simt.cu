// Generic partial-prefill attention on CUDA cores, for shapes outside the tensor-core kernel's range
// (small head_dim / page_size).  One thread block per (recompute row, KV head); warp w serves query
// head kvh * g + w.  Keys are spread over lanes for the scores, head_dim over lanes for P.V.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "launch.h"
#include "plan.h"

namespace tessera {
namespace {

template <int D>
__global__ void attn_simt_kernel(const __nv_bfloat16 *__restrict__ k_pool, const __nv_bfloat16 *__restrict__ v_pool,
                                 const __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ out,
                                 float *__restrict__ lse, const int32_t *__restrict__ q_pos,
                                 const int32_t *__restrict__ q_req, const int32_t *__restrict__ page_off,
                                 const int32_t *__restrict__ pages, int H_q, int H_kv, int page_size,
                                 float scale_log2, int row0) {
    constexpr int EPL = D / 32;                      // output elements per lane
    extern __shared__ float s_q[];                   // [g][D]
    const int j = row0 + blockIdx.x, kvh = blockIdx.y;
    const int g = H_q / H_kv;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int h = kvh * g + warp;
    const int p = q_pos[j];
    const int32_t *bt = pages + page_off[q_req[j]];
    const int page_shift = __ffs(page_size) - 1;

    float *qs = s_q + warp * D;
    for (int d = lane; d < D; d += 32) qs[d] = __bfloat162float(q[((size_t)j * H_q + h) * D + d]) * scale_log2;
    __syncwarp();

    float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;

    for (int t0 = 0; t0 <= p; t0 += 32) {
        const int t = t0 + lane;
        const bool valid = t <= p;
        int slot = 0;
        float s = -INFINITY;
        if (valid) {
            slot = bt[t >> page_shift] * page_size + (t & (page_size - 1));
            const uint4 *kr = reinterpret_cast<const uint4 *>(k_pool + ((size_t)slot * H_kv + kvh) * D);
            float dot = 0.f;
#pragma unroll
            for (int c = 0; c < D / 8; ++c) {
                const uint4 kv = kr[c];
                const uint32_t *w = reinterpret_cast<const uint32_t *>(&kv);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    dot = fmaf(qs[c * 8 + 2 * i], __uint_as_float(w[i] << 16), dot);
                    dot = fmaf(qs[c * 8 + 2 * i + 1], __uint_as_float(w[i] & 0xffff0000u), dot);
                }
            }
            s = dot;
        }
        float mx = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float m_new = fmaxf(m, mx);              // finite: lane 0 of every chunk is valid
        const float pr = valid ? exp2f(s - m_new) : 0.f;
        const float corr = exp2f(m - m_new);
        float ps = pr;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
        l = l * corr + ps;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= corr;
        m = m_new;
        const int n_valid = min(32, p - t0 + 1);
        for (int kk = 0; kk < n_valid; ++kk) {
            const float pk = __shfl_sync(0xffffffffu, pr, kk);
            const int sk = __shfl_sync(0xffffffffu, slot, kk);
            const __nv_bfloat16 *vr = v_pool + ((size_t)sk * H_kv + kvh) * D + lane * EPL;
            if (EPL == 4) {
                const uint2 vv = *reinterpret_cast<const uint2 *>(vr);
                acc[0] = fmaf(pk, __uint_as_float(vv.x << 16), acc[0]);
                acc[1] = fmaf(pk, __uint_as_float(vv.x & 0xffff0000u), acc[1]);
                acc[2] = fmaf(pk, __uint_as_float(vv.y << 16), acc[2]);
                acc[3] = fmaf(pk, __uint_as_float(vv.y & 0xffff0000u), acc[3]);
            } else {
                const uint32_t vv = *reinterpret_cast<const uint32_t *>(vr);
                acc[0] = fmaf(pk, __uint_as_float(vv << 16), acc[0]);
                acc[1] = fmaf(pk, __uint_as_float(vv & 0xffff0000u), acc[1]);
            }
        }
    }
    const float inv = 1.f / l;
    __nv_bfloat16 *o = out + ((size_t)j * H_q + h) * D + lane * EPL;
#pragma unroll
    for (int e = 0; e < EPL; e += 2)
        *reinterpret_cast<__nv_bfloat162 *>(o + e) = __floats2bfloat162_rn(acc[e] * inv, acc[e + 1] * inv);
    if (lse && lane == 0) lse[(size_t)j * H_q + h] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

cudaError_t launch_attn_simt(const tessera_plan *pl, const void *k_pool, const void *v_pool, const void *q,
                             void *out, float *lse, int chunk, cudaStream_t st) {
    if (pl->n_q == 0) return cudaSuccess;
    const int row0 = chunk < 0 ? 0 : pl->chunk_row_off[chunk];
    const int64_t rows = chunk < 0 ? pl->n_q : pl->chunk_row_off[chunk + 1] - row0;
    if (rows == 0) return cudaSuccess;
    const int Hq = pl->cfg.num_q_heads, Hkv = pl->cfg.num_kv_heads, D = pl->cfg.head_dim, g = Hq / Hkv;
    const float scale_log2 = pl->sm_scale * 1.4426950408889634f;
    dim3 grid((unsigned)rows, (unsigned)Hkv);
    const DeviceTables &d = pl->dev;
    auto *kp = static_cast<const __nv_bfloat16 *>(k_pool);
    auto *vp = static_cast<const __nv_bfloat16 *>(v_pool);
    auto *qp = static_cast<const __nv_bfloat16 *>(q);
    auto *op = static_cast<__nv_bfloat16 *>(out);
    const size_t smem = (size_t)g * D * sizeof(float);
    if (D == 128)
        attn_simt_kernel<128><<<grid, g * 32, smem, st>>>(kp, vp, qp, op, lse, d.q_pos, d.q_req, d.page_off, d.pages, Hq, Hkv, pl->cfg.page_size, scale_log2, row0);
    else
        attn_simt_kernel<64><<<grid, g * 32, smem, st>>>(kp, vp, qp, op, lse, d.q_pos, d.q_req, d.page_off, d.pages, Hq, Hkv, pl->cfg.page_size, scale_log2, row0);
    count_launch();
    return cudaGetLastError();
}

}  // namespace tessera

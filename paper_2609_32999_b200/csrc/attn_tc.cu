// Partial-prefill GQA attention on the 5th-generation tensor cores (Sec. 5.3 "Completing prefill":
// only the recompute rows are queries; they attend causally over the request's assembled pages).
//
// One thread block works on one KV head and up to TWO query tiles of the same request (128 rows
// each: 128/g recompute tokens x the g query heads of the group), which share every K/V page they
// read.  Warp roles:
//   warps 0-3 / 4-7 : softmax of tile 0 / tile 1 - thread i owns accumulator row i (TMEM lane i)
//   warp 8          : TMA producer - Q tiles once, then one K page and one V page per step through
//                     a ring of shared-memory stages; page ids come from the request's block table
//   warp 9          : issues tcgen05.mma (one lane): S = Q K^T into double-buffered TMEM columns,
//                     O += P V with P read from shared memory; owns the TMEM allocation
// Pages past a tile's last query position are never loaded; only pages that cross some row's causal
// limit are masked.  The running maximum is only refreshed when it grows by more than 2^8, so the
// accumulator in TMEM is rescaled rarely.  Every wait is bounded (see ptx::mbar_wait).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "launch.h"
#include "plan.h"
#include "sm100_ptx.cuh"
#include "tma_desc.h"

namespace tessera {
namespace {

using namespace ptx;

constexpr int kD = 128;            // head_dim
constexpr int kPage = 64;          // keys per step (= page size)
constexpr int kRows = 128;         // rows per query tile
constexpr int kStages = 3;
constexpr int kThreads = 320;

constexpr uint32_t kQTileBytes = kRows * kD * 2;         // 32 KB, two 16 KB halves of 64 elements
constexpr uint32_t kKVStageBytes = kPage * kD * 2;       // 16 KB, two 8 KB halves
constexpr uint32_t kPBytes = kRows * kPage * 2;          // 16 KB
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemK = kSmemQ + 2 * kQTileBytes;
constexpr uint32_t kSmemV = kSmemK + kStages * kKVStageBytes;
constexpr uint32_t kSmemP = kSmemV + kStages * kKVStageBytes;
constexpr uint32_t kSmemTotal = kSmemP + 2 * kPBytes;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;       // slack for the 1024-byte alignment

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0;      // S[tile][buf] at tile * 128 + buf * 64
constexpr uint32_t kTmemO = 256;    // O[tile] at 256 + tile * 128

constexpr float kRescaleThreshold = 8.f;   // log2 units

struct Barriers {
    uint64_t q_full[2];
    uint64_t k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
    uint64_t s_full[2][2];
    uint64_t p_full[2];
    uint64_t pv_done[2];
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const AttnTile *__restrict__ tiles,
               const AttnWork *__restrict__ work, const int32_t *__restrict__ q_pos,
               const int32_t *__restrict__ page_off, const int32_t *__restrict__ pages,
               const int32_t *__restrict__ seq_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ lse,
               int H_q, int g, float scale_log2, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) Barriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const AttnWork wk = work[blockIdx.x];
    const int n_tiles = wk.tile_b >= 0 ? 2 : 1;
    const AttnTile t0 = tiles[wk.tile_a];
    const AttnTile t1 = tiles[n_tiles == 2 ? wk.tile_b : wk.tile_a];
    const int kvh = wk.kvh;
    const int n_pages0 = (t0.kv_len + kPage - 1) / kPage;
    const int n_pages1 = n_tiles == 2 ? (t1.kv_len + kPage - 1) / kPage : 0;
    const int n_steps = max(n_pages0, n_pages1);
    const int32_t *bt = pages + page_off[t0.req];

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.q_full[i]), 1);
            mbar_init(smem_u32(&bars.p_full[i]), kRows);
            mbar_init(smem_u32(&bars.pv_done[i]), 1);
            mbar_init(smem_u32(&bars.s_full[i][0]), 1);
            mbar_init(smem_u32(&bars.s_full[i][1]), 1);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(smem_u32(&bars.k_full[i]), 1);
            mbar_init(smem_u32(&bars.k_empty[i]), 1);
            mbar_init(smem_u32(&bars.v_full[i]), 1);
            mbar_init(smem_u32(&bars.v_empty[i]), 1);
        }
        fence_barrier_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        prefetch_tmap(&tmap_q);
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int q = 0; q < n_tiles; ++q) {
                const AttnTile &t = q ? t1 : t0;
                const uint32_t bar = smem_u32(&bars.q_full[q]);
                mbar_expect_tx(bar, kQTileBytes);
                tma_load_3d(smem_u32(sm + kSmemQ + q * kQTileBytes), &tmap_q, bar, 0, kvh * g, t.q_begin);
                tma_load_3d(smem_u32(sm + kSmemQ + q * kQTileBytes + kQTileBytes / 2), &tmap_q, bar, 64, kvh * g, t.q_begin);
            }
        }
        for (int j0 = 0; j0 < n_steps; j0 += 32) {
            const int my_page = (j0 + lane < n_steps) ? bt[j0 + lane] : 0;
            const int jn = min(32, n_steps - j0);
            for (int jj = 0; jj < jn; ++jj) {
                const int page = __shfl_sync(0xffffffffu, my_page, jj);
                if (lane == 0) {
                    const int j = j0 + jj, st = j % kStages;
                    const uint32_t par = ((j / kStages) & 1) ^ 1;
                    mbar_wait(smem_u32(&bars.k_empty[st]), par, abort_flag, status, 1);
                    const uint32_t kb = smem_u32(&bars.k_full[st]);
                    mbar_expect_tx(kb, kKVStageBytes);
                    const uint32_t kdst = smem_u32(sm + kSmemK + st * kKVStageBytes);
                    tma_load_4d(kdst, &tmap_k, kb, 0, kvh, 0, page);
                    tma_load_4d(kdst + kKVStageBytes / 2, &tmap_k, kb, 64, kvh, 0, page);
                    mbar_wait(smem_u32(&bars.v_empty[st]), par, abort_flag, status, 2);
                    const uint32_t vb = smem_u32(&bars.v_full[st]);
                    mbar_expect_tx(vb, kKVStageBytes);
                    const uint32_t vdst = smem_u32(sm + kSmemV + st * kKVStageBytes);
                    tma_load_4d(vdst, &tmap_v, vb, 0, kvh, 0, page);
                    tma_load_4d(vdst + kKVStageBytes / 2, &tmap_v, vb, 64, kvh, 0, page);
                }
                __syncwarp();
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc_s = idesc_bf16(kRows, kPage, false);
        constexpr uint32_t idesc_o = idesc_bf16(kRows, kD, true);
        const int T = seq_len[t0.req];
        const int tail_page = (T % kPage) ? T / kPage : -1;       // page holding slots past the sequence end

        auto issue_s = [&](int j) {                               // S_j = Q K_j^T for every tile active at step j
            const int st = j % kStages;
            mbar_wait(smem_u32(&bars.k_full[st]), (j / kStages) & 1, abort_flag, status, 3);
            tc_fence_after();
            if (lane == 0) {
                const uint32_t kbase = smem_u32(sm + kSmemK + st * kKVStageBytes);
                for (int q = 0; q < n_tiles; ++q) {
                    if (j >= (q ? n_pages1 : n_pages0)) continue;
                    const uint32_t qbase = smem_u32(sm + kSmemQ + q * kQTileBytes);
                    const uint32_t d = tmem + kTmemS + q * 128 + (j & 1) * 64;
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) {
                        const uint64_t a = smem_desc_sw128(qbase + (k / 4) * (kQTileBytes / 2) + (k % 4) * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(kbase + (k / 4) * (kKVStageBytes / 2) + (k % 4) * 32, 16, 1024);
                        umma_ss(d, a, b, idesc_s, k > 0);
                    }
                    umma_commit(smem_u32(&bars.s_full[q][j & 1]));
                }
                umma_commit(smem_u32(&bars.k_empty[st]));
            }
            __syncwarp();
        };

        for (int q = 0; q < n_tiles; ++q) mbar_wait(smem_u32(&bars.q_full[q]), 0, abort_flag, status, 4);
        issue_s(0);
        for (int j = 0; j < n_steps; ++j) {
            if (j + 1 < n_steps) issue_s(j + 1);
            const int st = j % kStages;
            mbar_wait(smem_u32(&bars.v_full[st]), (j / kStages) & 1, abort_flag, status, 5);
            if (j == tail_page) {
                // V rows past the end of the sequence hold whatever the page held before; their
                // probabilities are zero, but 0 x NaN would still poison the accumulator.
                uint8_t *v = sm + kSmemV + st * kKVStageBytes;
                for (int r = T % kPage; r < kPage; ++r)
                    for (int c = lane; c < 16; c += 32) {
                        *reinterpret_cast<uint4 *>(v + (c >> 3) * (kKVStageBytes / 2) + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
                    }
                fence_proxy_async_smem();
                __syncwarp();
            }
            const uint32_t vbase = smem_u32(sm + kSmemV + st * kKVStageBytes);
            for (int q = 0; q < n_tiles; ++q) {
                if (j >= (q ? n_pages1 : n_pages0)) continue;
                mbar_wait(smem_u32(&bars.p_full[q]), j & 1, abort_flag, status, 6);
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t pbase = smem_u32(sm + kSmemP + q * kPBytes);
                    const uint32_t d = tmem + kTmemO + q * 128;
#pragma unroll
                    for (int k = 0; k < kPage / 16; ++k) {
                        const uint64_t a = smem_desc_sw128(pbase + k * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(vbase + k * 2048, kKVStageBytes / 2, 1024);
                        umma_ss(d, a, b, idesc_o, (j > 0) || (k > 0));
                    }
                    umma_commit(smem_u32(&bars.pv_done[q]));
                }
                __syncwarp();
            }
            if (lane == 0) umma_commit(smem_u32(&bars.v_empty[st]));
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        const int q = warp >> 2;                       // tile handled by this warp group
        if (q < n_tiles) {
            const AttnTile &t = q ? t1 : t0;
            const int my_pages = q ? n_pages1 : n_pages0;
            const int row = tid & 127;
            const int tok = min(row / g, t.n_tok - 1);
            const bool row_valid = row / g < t.n_tok;
            const int p_row = q_pos[t.q_begin + tok];
            const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tS = tmem + kTmemS + q * 128 + lane_base;
            const uint32_t tO = tmem + kTmemO + q * 128 + lane_base;
            uint8_t *p_row_smem = sm + kSmemP + q * kPBytes + row * 128;
            float m_row = -INFINITY, l_row = 0.f;

            for (int j = 0; j < my_pages; ++j) {
                mbar_wait(smem_u32(&bars.s_full[q][j & 1]), (j >> 1) & 1, abort_flag, status, 7);
                tc_fence_after();
                uint32_t s[64];
                {
                    uint32_t(&lo)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[0]);
                    uint32_t(&hi)[32] = *reinterpret_cast<uint32_t(*)[32]>(&s[32]);
                    tmem_ld32(tS + (j & 1) * 64, lo);
                    tmem_ld32(tS + (j & 1) * 64 + 32, hi);
                    tmem_wait_ld();
                }
                const int key0 = j * kPage;
                if (key0 + kPage > t.kv_full) {        // some row's causal limit falls inside this page
#pragma unroll
                    for (int i = 0; i < 64; ++i)
                        if (key0 + i > p_row) s[i] = 0xff800000u;   // -inf
                }
                float mx = -INFINITY;
#pragma unroll
                for (int i = 0; i < 64; ++i) mx = fmaxf(mx, __uint_as_float(s[i]));
                const float mc = fmaxf(m_row, mx * scale_log2);
                float factor = 1.f;
                bool rescale = false;
                if (mc > m_row + kRescaleThreshold) {  // also true on the first step (m_row = -inf)
                    factor = ex2(m_row - mc);          // 0 on the first step
                    m_row = mc;
                    rescale = j > 0;
                }
                uint32_t pk[32];
                float sum = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float a = ex2(fmaf(__uint_as_float(s[2 * i]), scale_log2, -m_row));
                    const float b = ex2(fmaf(__uint_as_float(s[2 * i + 1]), scale_log2, -m_row));
                    sum += a + b;
                    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                    pk[i] = *reinterpret_cast<uint32_t *>(&h);
                }
                l_row = l_row * factor + sum;
                if (j > 0) {
                    // P buffer free and O_{j-1} complete
                    mbar_wait(smem_u32(&bars.pv_done[q]), (j - 1) & 1, abort_flag, status, 8);
                    tc_fence_after();
                    if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t o[32];
                            tmem_ld32(tO + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                            tmem_st32(tO + c * 32, o);
                        }
                        tmem_wait_st();
                    }
                }
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4 *>(p_row_smem + ((c ^ (row & 7)) << 4)) =
                        make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_full[q]));
            }

            // epilogue: O / l -> bf16, LSE
            mbar_wait(smem_u32(&bars.pv_done[q]), (my_pages - 1) & 1, abort_flag, status, 9);
            tc_fence_after();
            const float inv = 1.f / l_row;
            const int head = kvh * g + row % g;
            __nv_bfloat16 *orow = out + ((size_t)(t.q_begin + tok) * H_q + head) * kD;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t o[32];
                tmem_ld32(tO + c * 32, o);
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(o[v * 8 + 2 * i]) * inv,
                                                                     __uint_as_float(o[v * 8 + 2 * i + 1]) * inv);
                            w[i] = *reinterpret_cast<uint32_t *>(&h);
                        }
                        *reinterpret_cast<uint4 *>(orow + c * 32 + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            if (lse && row_valid)
                lse[(size_t)(t.q_begin + tok) * H_q + head] = (m_row + log2f(l_row)) * 0.6931471805599453f;
        }
    }

    if (*abort_flag) {            // a wait gave up: let copies still in flight land before the block exits
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

}  // namespace

cudaError_t launch_attn_tc(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, void *out,
                           float *lse, cudaStream_t st, std::string *err) {
    if (pl->n_q == 0 || pl->work.empty()) return cudaSuccess;
    const int Hq = pl->cfg.num_q_heads, Hkv = pl->cfg.num_kv_heads, g = Hq / Hkv;
    if (pl->cfg.head_dim != kD || pl->cfg.page_size != kPage || kRows % g != 0) {
        *err = "shape outside the tcgen05 kernel's range";
        return cudaErrorNotSupported;
    }
    CUtensorMap tq, tk, tv;
    if (!make_q_tmap(&tq, q, pl->n_q, Hq, kD, g, kRows / g, err)) return cudaErrorInvalidValue;
    if (!make_pool_tmap(&tk, k_pool, pl->num_pool_pages, kPage, Hkv, kD, err)) return cudaErrorInvalidValue;
    if (!make_pool_tmap(&tv, v_pool, pl->num_pool_pages, kPage, Hkv, kD, err)) return cudaErrorInvalidValue;
    {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemAlloc);
        if (e != cudaSuccess) { *err = "cudaFuncSetAttribute(shared memory)"; return e; }
    }
    const DeviceTables &d = pl->dev;
    const float scale_log2 = pl->sm_scale * 1.4426950408889634f;
    attn_tc_kernel<<<(unsigned)pl->work.size(), kThreads, kSmemAlloc, st>>>(
        tq, tk, tv, d.tiles, d.work, d.q_pos, d.page_off, d.pages, d.seq_len,
        static_cast<__nv_bfloat16 *>(out), lse, Hq, g, scale_log2, d.status);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) *err = "kernel launch";
    return e;
}

}  // namespace tessera

// Partial-prefill GQA attention on the 5th-generation tensor cores (Sec. 5.3 "Completing prefill":
// only the recompute rows are queries; they attend causally over the request's assembled pages).
//
// One thread block works on one KV head and up to TWO query tiles of the same request (128 rows
// each: 128/g recompute tokens x the g query heads of the group), which share every K/V page they
// read.  A step covers 128 keys (two pages).  Warp roles:
//   warps 0-3 / 4-7 : softmax of tile 0 / tile 1 - thread i owns accumulator row i (TMEM lane i)
//   warp 8          : TMA producer - Q tiles once, then K and V of every step through one ring of
//                     32 KB shared-memory slots; page ids come from the request's block table
//   warp 9          : issues tcgen05.mma (one lane) and owns the TMEM allocation
// Per tile and step:  S = Q K^T (both operands in shared memory) -> 128 fp32 TMEM columns;
// softmax reads S, writes P as bf16 over the first 64 of those columns; O += P V takes P straight
// from TMEM, so probabilities never touch shared memory.  The MMA warp issues P.V of step j and
// then S of step j+1 of the same tile; while one tile is in softmax the tensor pipe works for the
// other.  Pages past a tile's last query position are never loaded; only steps that cross some
// row's causal limit are masked.  The running maximum is refreshed only when it grows by more than
// 2^8, so the accumulator in TMEM is rescaled rarely.  Every wait is bounded (ptx::mbar_wait).
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
constexpr int kPage = 64;          // page size
constexpr int kStep = 128;         // keys per step (two pages)
constexpr int kRows = 128;         // rows per query tile
constexpr int kRing = 5;           // K/V ring slots
constexpr int kThreads = 320;

constexpr uint32_t kQTileBytes = kRows * kD * 2;         // 32 KB: [d half][128 rows][128 B]
constexpr uint32_t kSlotBytes = kStep * kD * 2;          // 32 KB: [d half][128 keys][128 B]
constexpr uint32_t kHalfBytes = kSlotBytes / 2;          // 16 KB
constexpr uint32_t kPageHalfBytes = kPage * 128;         // 8 KB: one page inside a d half
constexpr uint32_t kSmemQ = 0;
constexpr uint32_t kSmemRing = kSmemQ + 2 * kQTileBytes;
constexpr uint32_t kSmemTotal = kSmemRing + kRing * kSlotBytes;
constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;       // slack for the 1024-byte alignment

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0;      // S[tile] at tile * 128 (P[tile] = its first 64 columns)
constexpr uint32_t kTmemO = 256;    // O[tile] at 256 + tile * 128

constexpr float kRescaleThreshold = 8.f;   // log2 units

struct Barriers {
    uint64_t q_full[2];
    uint64_t full[kRing], empty[kRing];
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t pv_done[2];
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// (d0, d1) = (a0, a1) * b + c with one packed instruction.
__device__ __forceinline__ void fma2(float &d0, float &d1, float a0, float a1, float b, float c) {
    asm("{\n .reg .b64 ra, rb, rc, rd;\n mov.b64 ra, {%2, %3};\n mov.b64 rb, {%4, %4};\n mov.b64 rc, {%5, %5};\n"
        " fma.rn.f32x2 rd, ra, rb, rc;\n mov.b64 {%0, %1}, rd;\n}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const AttnTile *__restrict__ tiles,
               const AttnWork *__restrict__ work, const int32_t *__restrict__ q_pos,
               const int32_t *__restrict__ page_off, const int32_t *__restrict__ pages,
               const int32_t *__restrict__ seq_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ lse,
               int H_q, int g, int num_pool_pages, float scale_log2, int *status) {
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
    const int n_steps0 = (t0.kv_len + kStep - 1) / kStep;
    const int n_steps1 = n_tiles == 2 ? (t1.kv_len + kStep - 1) / kStep : 0;
    const int n_steps = max(n_steps0, n_steps1);
    const int T = seq_len[t0.req];
    const int req_pages = (T + kPage - 1) / kPage;
    const int32_t *bt = pages + page_off[t0.req];

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.q_full[i]), 1);
            mbar_init(smem_u32(&bars.s_full[i]), 1);
            mbar_init(smem_u32(&bars.p_full[i]), kRows);
            mbar_init(smem_u32(&bars.pv_done[i]), 1);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&bars.full[i]), 1);
            mbar_init(smem_u32(&bars.empty[i]), 1);
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
        // ring item 2j = K of step j, item 2j+1 = V of step j
        for (int j0 = 0; j0 < n_steps; j0 += 16) {
            // lane l holds the id of page (2 * j0 + l); a page past the request's last one is fetched
            // from outside the pool, which TMA fills with zeros
            const int pi = 2 * j0 + lane;
            const int my_page = pi < req_pages ? bt[pi] : num_pool_pages;
            const int jn = min(16, n_steps - j0);
            for (int jj = 0; jj < jn; ++jj) {
                const int pg0 = __shfl_sync(0xffffffffu, my_page, 2 * jj);
                const int pg1 = __shfl_sync(0xffffffffu, my_page, 2 * jj + 1);
                if (lane == 0) {
                    const int j = j0 + jj;
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        const int item = 2 * j + kv, slot = item % kRing;
                        mbar_wait(smem_u32(&bars.empty[slot]), ((item / kRing) & 1) ^ 1, abort_flag, status, 1 + kv);
                        const uint32_t fb = smem_u32(&bars.full[slot]);
                        mbar_expect_tx(fb, kSlotBytes);
                        const uint32_t dst = smem_u32(sm + kSmemRing + slot * kSlotBytes);
                        const CUtensorMap *tm = kv ? &tmap_v : &tmap_k;
                        tma_load_4d(dst, tm, fb, 0, kvh, 0, pg0);
                        tma_load_4d(dst + kPageHalfBytes, tm, fb, 0, kvh, 0, pg1);
                        tma_load_4d(dst + kHalfBytes, tm, fb, 64, kvh, 0, pg0);
                        tma_load_4d(dst + kHalfBytes + kPageHalfBytes, tm, fb, 64, kvh, 0, pg1);
                    }
                }
                __syncwarp();
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        constexpr uint32_t idesc_s = idesc_bf16(kRows, kStep, false);
        constexpr uint32_t idesc_o = idesc_bf16(kRows, kD, true);
        const int tail_step = (T % kStep) ? T / kStep : -1;        // step holding slots past the sequence end

        auto ring_wait = [&](int item, int code) {
            mbar_wait(smem_u32(&bars.full[item % kRing]), (item / kRing) & 1, abort_flag, status, code);
            tc_fence_after();
        };
        auto issue_s = [&](int q, int j) {                         // S[q] = Q_q K_j^T (lane 0)
            const uint32_t kbase = smem_u32(sm + kSmemRing + ((2 * j) % kRing) * kSlotBytes);
            const uint32_t qbase = smem_u32(sm + kSmemQ + q * kQTileBytes);
            const uint32_t d = tmem + kTmemS + q * 128;
#pragma unroll
            for (int k = 0; k < kD / 16; ++k) {
                const uint64_t a = smem_desc_sw128(qbase + (k / 4) * (kQTileBytes / 2) + (k % 4) * 32, 16, 1024);
                const uint64_t b = smem_desc_sw128(kbase + (k / 4) * kHalfBytes + (k % 4) * 32, 16, 1024);
                umma_ss(d, a, b, idesc_s, k > 0);
            }
            umma_commit(smem_u32(&bars.s_full[q]));
        };

        for (int q = 0; q < n_tiles; ++q) mbar_wait(smem_u32(&bars.q_full[q]), 0, abort_flag, status, 4);
        ring_wait(0, 3);
        if (lane == 0) {
            for (int q = 0; q < n_tiles; ++q) issue_s(q, 0);
            umma_commit(smem_u32(&bars.empty[0]));
        }
        __syncwarp();
        for (int j = 0; j < n_steps; ++j) {
            ring_wait(2 * j + 1, 5);                               // V_j
            const int vslot = (2 * j + 1) % kRing;
            if (j == tail_step) {
                // V rows past the end of the sequence hold whatever the page held before; their
                // probabilities are zero, but 0 x NaN would still poison the accumulator.
                uint8_t *v = sm + kSmemRing + vslot * kSlotBytes;
                for (int r = T - j * kStep; r < kStep; ++r)
                    if (lane < 16) *reinterpret_cast<uint4 *>(v + (lane >> 3) * kHalfBytes + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                fence_proxy_async_smem();
                __syncwarp();
            }
            const bool more = j + 1 < n_steps;
            if (more) ring_wait(2 * j + 2, 3);                     // K_{j+1}
            const uint32_t vbase = smem_u32(sm + kSmemRing + vslot * kSlotBytes);
            for (int q = 0; q < n_tiles; ++q) {
                const int my_steps = q ? n_steps1 : n_steps0;
                if (j >= my_steps) continue;
                mbar_wait(smem_u32(&bars.p_full[q]), j & 1, abort_flag, status, 6);
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t d = tmem + kTmemO + q * 128;
                    const uint32_t p = tmem + kTmemS + q * 128;
#pragma unroll
                    for (int k = 0; k < kStep / 16; ++k) {
                        const uint64_t b = smem_desc_sw128(vbase + k * 2048, kHalfBytes, 1024);
                        umma_ts(d, p + k * 8, b, idesc_o, (j > 0) || (k > 0));
                    }
                    umma_commit(smem_u32(&bars.pv_done[q]));
                    if (j + 1 < my_steps) issue_s(q, j + 1);
                }
                __syncwarp();
            }
            if (lane == 0) {
                umma_commit(smem_u32(&bars.empty[vslot]));
                if (more) umma_commit(smem_u32(&bars.empty[(2 * j + 2) % kRing]));
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        const int q = warp >> 2;                       // tile handled by this warp group
        if (q < n_tiles) {
            const AttnTile &t = q ? t1 : t0;
            const int my_steps = q ? n_steps1 : n_steps0;
            const int row = tid & 127;
            const int tok = min(row / g, t.n_tok - 1);
            const bool row_valid = row / g < t.n_tok;
            const int p_row = q_pos[t.q_begin + tok];
            const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t tS = tmem + kTmemS + q * 128 + lane_base;
            const uint32_t tO = tmem + kTmemO + q * 128 + lane_base;
            float m_row = -INFINITY, l_row = 0.f;

            for (int j = 0; j < my_steps; ++j) {
                // S_j complete; this also means P.V of step j-1 has completed (it was issued earlier)
                mbar_wait(smem_u32(&bars.s_full[q]), j & 1, abort_flag, status, 7);
                tc_fence_after();
                const int key0 = j * kStep;
                const bool masked = key0 + kStep > t.kv_full;   // some row's causal limit falls in this step

                // pass 1: row maximum
                float mxa[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t s[32];
                    tmem_ld32(tS + c * 32, s);
                    tmem_wait_ld();
                    if (masked) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (key0 + c * 32 + i > p_row) s[i] = 0xff800000u;   // -inf
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i) mxa[i & 3] = fmaxf(mxa[i & 3], __uint_as_float(s[i]));
                }
                const float mx = fmaxf(fmaxf(mxa[0], mxa[1]), fmaxf(mxa[2], mxa[3]));
                const float mc = fmaxf(m_row, mx * scale_log2);
                float factor = 1.f;
                bool rescale = false;
                if (mc > m_row + kRescaleThreshold) {  // also true on the first step (m_row = -inf)
                    factor = ex2(m_row - mc);          // 0 on the first step
                    m_row = mc;
                    rescale = j > 0;
                }
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
                }

                // pass 2: probabilities, written as bf16 over the first 64 columns of S
                float suma[4] = {0.f, 0.f, 0.f, 0.f};
                const float neg_m = -m_row;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t s[32];
                    tmem_ld32(tS + c * 32, s);
                    tmem_wait_ld();
                    if (masked) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (key0 + c * 32 + i > p_row) s[i] = 0xff800000u;
                    }
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float x0, x1;
                        fma2(x0, x1, __uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1]), scale_log2, neg_m);
                        const float a = ex2(x0), b = ex2(x1);
                        suma[i & 3] += a + b;
                        pk[i] = pack_bf16(a, b);
                    }
                    tmem_st16(tS + c * 16, pk);
                }
                l_row = l_row * factor + ((suma[0] + suma[1]) + (suma[2] + suma[3]));
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_full[q]));
            }

            // epilogue: O / l -> bf16, LSE
            mbar_wait(smem_u32(&bars.pv_done[q]), (my_steps - 1) & 1, abort_flag, status, 9);
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
                        for (int i = 0; i < 4; ++i)
                            w[i] = pack_bf16(__uint_as_float(o[v * 8 + 2 * i]) * inv, __uint_as_float(o[v * 8 + 2 * i + 1]) * inv);
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
        static_cast<__nv_bfloat16 *>(out), lse, Hq, g, pl->num_pool_pages, scale_log2, d.status);
    count_launch();
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) *err = "kernel launch";
    return e;
}

}  // namespace tessera

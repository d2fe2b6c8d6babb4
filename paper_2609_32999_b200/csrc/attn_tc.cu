// Partial-prefill GQA attention on the 5th-generation tensor cores (Sec. 5.3 "Completing prefill":
// only the recompute rows are queries; they attend causally over the request's assembled pages).
//
// One thread block works on one KV head and up to TWO query tiles of the same request (128 rows
// each: 128/g recompute tokens x the g query heads of the group), which share every K/V page they
// read.  A step covers 128 keys (1, 2, 4, 8 or 16 pages of 128, 64, 32, 16 or 8 tokens).  Warp roles (384 threads):
//   warps 0-7  : softmax.  All eight work on one tile at a time and alternate between the tiles; a
//                warp owns 16 rows (TMEM lanes) and reads them as an MMA accumulator fragment, the
//                four threads of a row in one warp - no two warps ever exchange anything
//   warp 8     : TMA producer - Q tiles once per item, then K and V of every step through one ring of
//                four 32 KB shared-memory slots; page ids come from the request's block table
//   warp 9, 10 : issue tcgen05.mma for tile 0 / tile 1 (one lane each); warp 9 owns the TMEM allocation
//   warp 11    : idle (completes the warp group that hands its registers to the softmax warps)
// Per tile and step:  S = Q K^T (both operands in shared memory) -> 128 fp32 TMEM columns;
// softmax reads S and writes P as bf16 back over part of those columns; O += P V takes P straight
// from TMEM, so probabilities never touch shared memory.  Each issuing warp sends P.V of step j and
// then S of step j+1 of its tile; while the softmax warps are on one tile the tensor pipe works
// for the other.  Pages past a tile's last query position are never loaded; only steps that cross
// some row's causal limit are masked.  Probabilities are taken against a reference maximum that is
// refreshed only when a row's partial sum would exceed 2^8, so the accumulator in TMEM is rescaled
// rarely.  Every wait is bounded (ptx::mbar_wait).  A finished tile leaves through a shared-memory
// output tile and a tiled bulk store.
// The kernel is persistent: one thread block per SM walks through its share of the work list, so the
// barriers, the TMEM allocation and the tensor maps are set up once, and the next item's Q, K and V
// loads and first S run while the softmax warps still write the previous item's result.
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

constexpr int kStep = 128;         // keys per step (two pages)
constexpr int kRows = 128;         // rows per query tile
constexpr int kRing = 4;           // K/V ring slots (two steps of look-ahead; a fifth slot measured no faster)
constexpr int kThreads = 384;        // 8 softmax warps, producer, MMA, 2 idle warps (register donors)
// setmaxnreg moves registers inside the pool the block got at launch (threads x registers per thread
// under __launch_bounds__): the raised and lowered counts together must fit in it, or the raise
// waits forever.
constexpr int kRegsLaunch = (65536 / kThreads) / 8 * 8;
constexpr int kRegsSoftmax = 208, kRegsOther = 80;
static_assert(256 * kRegsSoftmax + 128 * kRegsOther <= kThreads * kRegsLaunch, "register pool of the block exceeded");

// Shared-memory geometry for head_dim D (64 or 128): a tile of 128 rows is stored as D/64 "halves" of
// [128 rows][128 B] (64 elements per row, 128-byte swizzle).
constexpr uint32_t kHalfBytes = 128 * 128;                                     // 16 KB
template <int D> struct Geo {
    static constexpr int kHalves = D / 64;
    static constexpr uint32_t kQTileBytes = kHalves * kHalfBytes;              // Q tile: 16 / 32 KB
    static constexpr uint32_t kSlotBytes = kHalves * kHalfBytes;               // K or V of one step
    static constexpr uint32_t kSmemQ = 0;
    static constexpr uint32_t kSmemRing = kSmemQ + 2 * kQTileBytes;
    static constexpr uint32_t kSmemStage = kSmemRing + kRing * kSlotBytes;     // one output tile (bf16), laid out like a Q tile
    static constexpr uint32_t kSmemTotal = kSmemStage + kQTileBytes;
    static constexpr uint32_t kSmemAlloc = kSmemTotal + 1024;                  // slack for the 1024-byte alignment
};

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0;      // S[tile] at tile * 128 (P[tile] = its first 64 columns)
constexpr uint32_t kTmemO = 256;    // O[tile] at 256 + tile * 128


struct Barriers {
    uint64_t q_full[2], q_empty[2];
    uint64_t full[kRing], empty[kRing];
    uint64_t s_full[2];
    uint64_t p_half[2][2];     // probabilities of keys [0, 64) / [64, 128) of the tile's current step are in TMEM
    uint64_t pv_half[2];       // P.V of the first 64 keys has completed (read only when a reference maximum is refreshed mid-step)
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
template <int N> __device__ __forceinline__ void reg_alloc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void reg_dealloc() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }
__device__ __forceinline__ void named_sync(int id, int count) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
// (a0, a1) += (b0, b1) with one packed instruction.
__device__ __forceinline__ void add2(float &a0, float &a1, float b0, float b1) {
    asm("{\n .reg .b64 ra, rb;\n mov.b64 ra, {%0, %1};\n mov.b64 rb, {%2, %3};\n add.rn.f32x2 ra, ra, rb;\n mov.b64 {%0, %1}, ra;\n}"
        : "+f"(a0), "+f"(a1) : "f"(b0), "f"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// What one work item means for every role of the block.
struct Item {
    AttnWork wk;
    AttnTile t0, t1;
    int n_tiles, step0, n_steps0, n_steps1, n_steps, T, req_pages;
    const int32_t *bt;
};

// kMaxPages: most pages a 128-key step can consist of in this instantiation - 8 (pages of 16 tokens or
// more) or 16 (pages of 8 tokens); the wider producer loop is kept out of the common instantiation.
// K8: queries and keys are 8-bit floats (e4m3 codes; the scales are folded into scale_log2 by the host):
// S = Q K^T runs as kind::f8f6f4 with 32 elements of head_dim per instruction, a Q tile and a K step are
// 128 rows of 128 bytes (one swizzle atom wide, head_dim 128 only); V, P and the accumulator stay as they are.
template <int D, int kMaxPages, bool K8>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
               const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
               const AttnTile *__restrict__ tiles,
               const AttnWork *__restrict__ work, int n_work, const int32_t *__restrict__ q_pos,
               const int32_t *__restrict__ page_off, const int32_t *__restrict__ pages,
               const int32_t *__restrict__ seq_len, __nv_bfloat16 *__restrict__ out, float *__restrict__ lse,
               int H_q, int g, int H_kv, int page_size, int num_pool_pages, float scale_log2, int max_parts,
               float *__restrict__ ws_o, float2 *__restrict__ ws_ml, int *status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sm = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    using G = Geo<D>;
    constexpr int kD = D;
    constexpr uint32_t kQTileBytes = G::kQTileBytes, kSlotBytes = G::kSlotBytes;
    constexpr int kQKHalves = K8 ? 1 : G::kHalves;      // 128-byte-wide halves of a Q tile / a K step
    constexpr uint32_t kSmemQ = G::kSmemQ, kSmemRing = G::kSmemRing;
    __shared__ __align__(8) Barriers bars;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    // A block of a launch in which another block already gave up on a wait does not start, so a
    // stalled launch ends after one round of timeouts rather than one per block.
    if (*reinterpret_cast<volatile int *>(status) != 0) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int pps = kStep / page_size;                 // pages per step: 1, 2, 4, 8 or 16

    // The block's share of the work list: round k of the grid takes items [k G, (k + 1) G), this block
    // the b-th of them in even rounds and the b-th from the end in odd rounds.  For a list sorted by
    // cost the serpentine evens out the sums, and blocks that run at the same time work on neighbours
    // in the list, i.e. on the same request and KV head, and share their K/V pages in L2.  When a batch
    // has few items per block the host lays the list out so that this very walk hands each block a
    // greedily balanced share (holes are marked tile_a = -1).  Taking items off a global counter at
    // run time measured 1-1.5 % slower on the long-context configurations.  Every role walks the
    // same sequence; -1 = nothing in this round.
    const int n_rounds = (n_work + (int)gridDim.x - 1) / (int)gridDim.x;
    auto item_index = [&](int round) {
        const int b = (round & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
        const int w = round * (int)gridDim.x + b;
        return w < n_work ? w : -1;
    };
    auto load_item = [&](int w) {
        Item it;
        it.wk = work[w];
        if (it.wk.tile_a < 0) {            // a hole of the assignment: nothing to do in this round
            it.n_tiles = 0;
            return it;
        }
        it.n_tiles = it.wk.tile_b >= 0 ? 2 : 1;
        it.t0 = tiles[it.wk.tile_a];
        it.t1 = tiles[it.n_tiles == 2 ? it.wk.tile_b : it.wk.tile_a];
        // the item covers the 128-key steps [step0, step_end) of its tiles (all of them unless it was
        // split); step indices below are relative to step0
        it.step0 = it.wk.step_begin;
        it.n_steps0 = min(it.wk.step_end, (it.t0.kv_len + kStep - 1) / kStep) - it.step0;
        it.n_steps1 = it.n_tiles == 2 ? min(it.wk.step_end, (it.t1.kv_len + kStep - 1) / kStep) - it.step0 : 0;
        it.n_steps = max(it.n_steps0, it.n_steps1);
        it.T = seq_len[it.t0.req];
        it.req_pages = (it.T + page_size - 1) / page_size;
        it.bt = pages + page_off[it.t0.req];
        return it;
    };

    if (tid == 0) {
        s_abort = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(smem_u32(&bars.q_full[i]), 1);
            mbar_init(smem_u32(&bars.q_empty[i]), 1);
            mbar_init(smem_u32(&bars.s_full[i]), 1);
            mbar_init(smem_u32(&bars.p_half[i][0]), 2 * kRows);
            mbar_init(smem_u32(&bars.p_half[i][1]), 2 * kRows);
            mbar_init(smem_u32(&bars.pv_half[i]), 1);
            mbar_init(smem_u32(&bars.pv_done[i]), 1);
        }
        for (int i = 0; i < kRing; ++i) {
            mbar_init(smem_u32(&bars.full[i]), 1);
            mbar_init(smem_u32(&bars.empty[i]), 2);       // both MMA-issuing warps release every slot
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
        prefetch_tmap(&tmap_o);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    // Registers move from the producer / MMA warp group to the softmax warps, which hold a whole
    // 128-column row of S plus the packed probabilities.
    if (warp >= 8) {
    reg_dealloc<kRegsOther>();
    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        // A tile holds (128 / g) tokens x g heads = q_rows rows; when g does not divide 128 the last
        // rows of the 128-row MMA tile are padding and are zeroed once (TMA never writes them; their
        // results are never stored).
        const int q_rows = (kRows / g) * g;
        if (q_rows < kRows) {
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int hf = 0; hf < kQKHalves; ++hf) {
                    uint8_t *base = sm + kSmemQ + q * kQTileBytes + hf * kHalfBytes;
                    for (int o = q_rows * 128 + lane * 16; o < kRows * 128; o += 32 * 16)
                        *reinterpret_cast<uint4 *>(base + o) = make_uint4(0, 0, 0, 0);
                }
            fence_proxy_async_smem();
            __syncwarp();
        }
        const int steps_per_fetch = 32 / pps;
        const uint32_t page_bytes = (uint32_t)page_size * 128;     // one page inside a d half
        int ring_base = 0;                  // ring items issued for earlier work items
        int q_uses[2] = {0, 0};             // how often each Q tile buffer has been filled
        for (int round = 0; round < n_rounds; ++round) {
            const int w = item_index(round);
            if (w < 0) continue;
            const Item it = load_item(w);
            if (it.n_tiles == 0) continue;
            const int kvh = it.wk.kvh;
            if (lane == 0) {
                for (int q = 0; q < it.n_tiles; ++q) {
                    const AttnTile &t = q ? it.t1 : it.t0;
                    // the previous item's last S MMA has read this buffer
                    if (q_uses[q] > 0) mbar_wait(smem_u32(&bars.q_empty[q]), (q_uses[q] - 1) & 1, abort_flag, status, 10);
                    const uint32_t bar = smem_u32(&bars.q_full[q]);
                    mbar_expect_tx(bar, (uint32_t)(kQKHalves * q_rows * 128));
#pragma unroll
                    for (int hf = 0; hf < kQKHalves; ++hf)
                        tma_load_3d(smem_u32(sm + kSmemQ + q * kQTileBytes + hf * kHalfBytes), &tmap_q, bar, hf * 64, kvh * g, t.q_begin);
                }
            }
            for (int q = 0; q < it.n_tiles; ++q) ++q_uses[q];
            // ring item ring_base + 2j = K of step j, + 2j + 1 = V of step j
            for (int j0 = 0; j0 < it.n_steps; j0 += steps_per_fetch) {
                // lane l holds the id of page (pps * (step0 + j0) + l); a page past the request's last one
                // is fetched from outside the pool, which TMA fills with zeros
                const int pi = pps * (it.step0 + j0) + lane;
                const int my_page = pi < it.req_pages ? it.bt[pi] : num_pool_pages;
                const int jn = min(steps_per_fetch, it.n_steps - j0);
                for (int jj = 0; jj < jn; ++jj) {
                    int pg[kMaxPages];
#pragma unroll
                    for (int k = 0; k < kMaxPages; ++k) pg[k] = __shfl_sync(0xffffffffu, my_page, (pps * jj + k) & 31);
                    if (lane == 0) {
                        const int j = j0 + jj;
#pragma unroll
                        for (int kv = 0; kv < 2; ++kv) {
                            const int item = ring_base + 2 * j + kv, slot = item % kRing;
                            mbar_wait(smem_u32(&bars.empty[slot]), ((item / kRing) & 1) ^ 1, abort_flag, status, 1 + kv);
                            const uint32_t fb = smem_u32(&bars.full[slot]);
                            const int halves = kv ? G::kHalves : kQKHalves;
                            mbar_expect_tx(fb, (uint32_t)halves * kHalfBytes);
                            const uint32_t dst = smem_u32(sm + kSmemRing + slot * kSlotBytes);
                            const CUtensorMap *tm = kv ? &tmap_v : &tmap_k;
#pragma unroll
                            for (int k = 0; k < kMaxPages; ++k)
                                if (k < pps) {
#pragma unroll
                                    for (int hf = 0; hf < G::kHalves; ++hf)
                                        if (hf < halves) tma_load_4d(dst + hf * kHalfBytes + k * page_bytes, tm, fb, hf * 64, kvh, 0, pg[k]);
                                }
                        }
                    }
                    __syncwarp();
                }
            }
            ring_base += 2 * it.n_steps;
        }
    } else if (warp == 9 || warp == 10) {
        // ------------------------------------------------------------------ MMA issuers: warp 9 for
        // tile 0, warp 10 for tile 1.  Each runs its own tile's chain, so the waits of one overlap
        // the MMAs of the other; a ring slot is free again once both have released it (the warp of a
        // tile that is absent or already finished only releases).
        constexpr uint32_t idesc_s = K8 ? idesc_e4m3(kRows, kStep) : idesc_bf16(kRows, kStep, false);
        constexpr uint32_t idesc_o = idesc_bf16(kRows, kD, true);
        const int q = warp - 9;
        const uint32_t qbase = smem_u32(sm + kSmemQ + q * kQTileBytes);
        const uint32_t tS = tmem + kTmemS + q * 128, tO = tmem + kTmemO + q * 128;
        int ring_base = 0, step_base = 0, q_uses = 0;

        for (int round = 0; round < n_rounds; ++round) {
            const int w = item_index(round);
            if (w < 0) continue;
            const Item it = load_item(w);
            if (it.n_tiles == 0) continue;
            const int n_steps = it.n_steps;
            const int my_steps = q ? it.n_steps1 : it.n_steps0;
            const int T = it.T, step0 = it.step0;
            const int tail_step = (T % kStep) ? T / kStep - step0 : -1;   // step holding slots past the sequence end

            auto ring_wait = [&](int item, int code) {
                item += ring_base;
                mbar_wait(smem_u32(&bars.full[item % kRing]), (item / kRing) & 1, abort_flag, status, code);
                tc_fence_after();
            };
            auto slot_of = [&](int item) { return (ring_base + item) % kRing; };
            auto issue_s = [&](int j) {                                // S[q] = Q_q K_j^T (lane 0)
                const uint32_t kbase = smem_u32(sm + kSmemRing + slot_of(2 * j) * kSlotBytes);
                if constexpr (K8) {
#pragma unroll
                    for (int k = 0; k < kD / 32; ++k) {                // 32 bytes = 32 elements of head_dim per instruction
                        const uint64_t a = smem_desc_sw128(qbase + k * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(kbase + k * 32, 16, 1024);
                        umma_ss_f8(tS, a, b, idesc_s, k > 0);
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < kD / 16; ++k) {
                        const uint64_t a = smem_desc_sw128(qbase + (k / 4) * kHalfBytes + (k % 4) * 32, 16, 1024);
                        const uint64_t b = smem_desc_sw128(kbase + (k / 4) * kHalfBytes + (k % 4) * 32, 16, 1024);
                        umma_ss(tS, a, b, idesc_s, k > 0);
                    }
                }
                umma_commit(smem_u32(&bars.s_full[q]));
                umma_commit(smem_u32(&bars.empty[slot_of(2 * j)]));    // K_j no longer needed by this tile
                if (j == my_steps - 1) umma_commit(smem_u32(&bars.q_empty[q]));   // the item's last read of Q
            };

            ring_wait(0, 3);
            if (my_steps > 0) {
                mbar_wait(smem_u32(&bars.q_full[q]), q_uses & 1, abort_flag, status, 4);
                ++q_uses;
                tc_fence_after();
                if (lane == 0) issue_s(0);
            } else if (lane == 0) {
                mbar_arrive(smem_u32(&bars.empty[slot_of(0)]));
            }
            __syncwarp();
            for (int j = 0; j < n_steps; ++j) {
                ring_wait(2 * j + 1, 5);                               // V_j
                const int vslot = slot_of(2 * j + 1);
                const bool more = j + 1 < n_steps;
                if (j >= my_steps) {
                    // this tile is finished or absent: only release the slots
                    if (more) ring_wait(2 * j + 2, 3);
                    if (lane == 0) {
                        mbar_arrive(smem_u32(&bars.empty[vslot]));
                        if (more) mbar_arrive(smem_u32(&bars.empty[slot_of(2 * j + 2)]));
                    }
                    __syncwarp();
                    continue;
                }
                if (j == tail_step) {
                    // V rows past the end of the sequence hold whatever the page held before; their
                    // probabilities are zero, but 0 x NaN would still poison the accumulator.  (Both
                    // issuing warps may write these zeros; the values agree.)
                    uint8_t *v = sm + kSmemRing + vslot * kSlotBytes;
                    for (int r = T - (step0 + j) * kStep; r < kStep; ++r)
                        if (lane < 8 * G::kHalves) *reinterpret_cast<uint4 *>(v + (lane >> 3) * kHalfBytes + r * 128 + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                const bool next_s = j + 1 < my_steps;
                if (more) ring_wait(2 * j + 2, 3);                     // K_{j+1}
                const uint32_t vbase = smem_u32(sm + kSmemRing + vslot * kSlotBytes);
                // P arrives in two halves: P.V of the first 64 keys runs while the softmax warps are still
                // on the exponentials of the other 64
                mbar_wait(smem_u32(&bars.p_half[q][0]), (step_base + j) & 1, abort_flag, status, 6);
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int k = 0; k < kStep / 32; ++k) {
                        const uint64_t b = smem_desc_sw128(vbase + k * 2048, kHalfBytes, 1024);
                        umma_ts(tO, tS + k * 8, b, idesc_o, (j > 0) || (k > 0));   // P of keys [16k, 16k + 16): columns 8k .. 8k + 7
                    }
                    umma_commit(smem_u32(&bars.pv_half[q]));
                }
                __syncwarp();
                mbar_wait(smem_u32(&bars.p_half[q][1]), (step_base + j) & 1, abort_flag, status, 11);
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int k = kStep / 32; k < kStep / 16; ++k) {
                        const uint64_t b = smem_desc_sw128(vbase + k * 2048, kHalfBytes, 1024);
                        umma_ts(tO, tS + k * 8, b, idesc_o, true);
                    }
                    umma_commit(smem_u32(&bars.pv_done[q]));
                    umma_commit(smem_u32(&bars.empty[vslot]));
                    if (next_s) issue_s(j + 1);
                    else if (more) mbar_arrive(smem_u32(&bars.empty[slot_of(2 * j + 2)]));
                }
                __syncwarp();
            }
            ring_base += 2 * n_steps;
            step_base += my_steps;
        }
    }
    } else {
        reg_alloc<kRegsSoftmax>();
        // ------------------------------------------------------------------ softmax + epilogue
        // All eight warps work on ONE tile at a time and alternate between the tiles.  A warp owns 16
        // rows (TMEM lanes) with all their 128 columns - warp w the first 16 lanes of lane quarter
        // w % 4, warp w + 4 the other 16 - and reads S in the layout of an MMA accumulator fragment:
        // a thread holds two rows (t/4 and t/4 + 8 of the warp's 16) and, of every group of 8 columns,
        // columns 2 (t%4) and 2 (t%4) + 1.  The four threads that share a row sit in one warp, so row
        // maxima and sums are two shuffles away and no two warps ever have to agree on anything.
        const int lane16 = (warp & 3) * 32 + (warp >> 2) * 16;         // first TMEM lane of this warp
        const uint32_t lane_base = (uint32_t)lane16 << 16;
        const int rows[2] = {lane16 + (lane >> 2), lane16 + (lane >> 2) + 8};
        const int cq = (lane & 3) * 2;                                 // first of the thread's two columns in every group of 8
        int step_base[2] = {0, 0};                     // steps of each tile in earlier work items (barrier phases go on)
        // where this thread's two bf16 of (row, column group kk) go in the swizzled output tile: rows r and
        // r + 8 share r % 8, so one table of eight offsets serves both
        uint32_t stage_off[8];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) stage_off[kk] = (uint32_t)(rows[0] * 128 + ((kk ^ (rows[0] & 7)) << 4) + cq * 2);
        auto quad_max = [](float v) {
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
            return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
        };
        auto quad_sum = [](float v) {
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            return v + __shfl_xor_sync(0xffffffffu, v, 2);
        };

        for (int round = 0; round < n_rounds; ++round) {
        const int w = item_index(round);
        if (w < 0) continue;
        const Item it = load_item(w);
        if (it.n_tiles == 0) continue;
        const int n_tiles = it.n_tiles, n_steps = it.n_steps, n_steps0 = it.n_steps0, n_steps1 = it.n_steps1;
        const int step0 = it.step0, kvh = it.wk.kvh;
        const AttnTile &t0 = it.t0, &t1 = it.t1;
        int tok[2][2], p_row[2][2];
        bool row_valid[2][2];
        // reference maximum (identical in the four threads of a row) and this thread's share of the row sum
        float m_row[2][2] = {{-INFINITY, -INFINITY}, {-INFINITY, -INFINITY}}, l_row[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const AttnTile &t = q ? t1 : t0;
#pragma unroll
            for (int rr = 0; rr < 2; ++rr) {
                tok[q][rr] = min(rows[rr] / g, t.n_tok - 1);
                row_valid[q][rr] = rows[rr] / g < t.n_tok;
                p_row[q][rr] = q_pos[t.q_begin + tok[q][rr]];
            }
        }

        for (int j = 0; j < n_steps; ++j) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                if (q >= n_tiles || j >= (q ? n_steps1 : n_steps0)) continue;
                const uint32_t tS = tmem + kTmemS + q * 128 + lane_base;
                const int par = (step_base[q] + j) & 1;
                // S_j complete; this also means P.V of step j-1 has completed (it was issued earlier)
                mbar_wait(smem_u32(&bars.s_full[q]), par, abort_flag, status, 7);
                tc_fence_after();
                const int key0 = (step0 + j) * kStep;
                const bool masked = key0 + kStep > (q ? t1.kv_full : t0.kv_full);   // a causal limit falls in this step

                // The thread's 2 x 64 scores (rows t/4 and t/4 + 8 of the warp's 16; of every group of 8
                // columns, columns 2 (t%4) and 2 (t%4) + 1) stay in registers for the whole step.
                uint32_t s[64];
                tmem_ld_16x256b_x16(tS, s);
                tmem_wait_ld();
                if (masked) {
#pragma unroll
                    for (int k = 0; k < 16; ++k)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (key0 + 8 * k + cq + (e & 1) > p_row[q][e >> 1]) s[4 * k + e] = 0xff800000u;   // -inf
                }
                uint32_t pk[16];
                // Probabilities of column groups [8 h, 8 h + 8) (keys [64 h, 64 h + 64)) against the current
                // reference maxima: packed into pk, this thread's share of the two row sums into sum.
                auto exp_half = [&](int h, float (&sum)[2]) {
                    float sa[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, sb[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
                    // a row that has seen no visible key yet (possible in a later split-KV part) keeps
                    // the reference at 0: its scores are all -inf and its probabilities 0
                    const float neg_m[2] = {m_row[q][0] == -INFINITY ? 0.f : -m_row[q][0],
                                            m_row[q][1] == -INFINITY ? 0.f : -m_row[q][1]};
#pragma unroll
                    for (int k = 0; k < 8; ++k)
#pragma unroll
                        for (int rr = 0; rr < 2; ++rr) {
                            const int i = 4 * (8 * h + k) + 2 * rr;
                            float x0, x1;
                            fma2(x0, x1, __uint_as_float(s[i]), __uint_as_float(s[i + 1]), scale_log2, neg_m[rr]);
                            const float e0 = ex2(x0), e1 = ex2(x1);
                            add2(sa[rr][k & 1], sb[rr][k & 1], e0, e1);
                            pk[2 * k + rr] = pack_bf16(e0, e1);          // P column 4 (8 h + k) + t%4 of row rr
                        }
                    sum[0] = (sa[0][0] + sb[0][0]) + (sa[0][1] + sb[0][1]);
                    sum[1] = (sa[1][0] + sb[1][0]) + (sa[1][1] + sb[1][1]);
                };
                // P as bf16 over the first 64 columns of S (column c holds keys 2c and 2c + 1), one half at
                // a time; the MMA warp starts P.V of a half as soon as all 256 threads have stored it.
                auto release_half = [&](int h) {
                    tmem_st_16x128b_x8(tS + 32 * h, pk);
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&bars.p_half[q][h]));
                };
                // The step's true row maxima become the reference (per warp: all its rows together); the
                // accumulator and the running sum are brought to the new reference.
                auto refresh = [&](bool rescale_o, float (&factor)[2]) {
#pragma unroll
                    for (int rr = 0; rr < 2; ++rr) {
                        float ma = -INFINITY, mb = -INFINITY;
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            ma = fmaxf(ma, __uint_as_float(s[4 * k + 2 * rr]));
                            mb = fmaxf(mb, __uint_as_float(s[4 * k + 2 * rr + 1]));
                        }
                        const float mx = quad_max(fmaxf(ma, mb));
                        const float mc = fmaxf(m_row[q][rr], mx * scale_log2);
                        factor[rr] = 1.f;
                        if (mc != -INFINITY) {
                            factor[rr] = ex2(m_row[q][rr] - mc);   // 0 when the row had no visible key before
                            m_row[q][rr] = mc;
                        }
                    }
                    if (rescale_o) {
                        const uint32_t tO = tmem + kTmemO + q * 128 + lane_base;
                        uint32_t o[kD / 2];
                        if constexpr (kD == 128) tmem_ld_16x256b_x16(tO, o); else tmem_ld_16x256b_x8(tO, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < kD / 2; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor[(i >> 1) & 1]);
                        if constexpr (kD == 128) tmem_st_16x256b_x16(tO, o); else tmem_st_16x256b_x8(tO, o);
                    }
                };

                // Fast path: probabilities against the current reference maxima.  While every thread's
                // share of a row sum stays below 2^6 the row sum stays below 2^8, every probability
                // does too and the reference is good enough; otherwise (and on the first step) the
                // warp's rows take the step's true maxima.  The decision is per warp, and it is taken
                // after each half: once the first half has been released, a refresh concerns only the
                // second half (the first half's P.V is brought to the new reference with the accumulator).
                float sum_a[2], sum_b[2], factor[2];
                bool fresh = j == 0;
                if (!fresh) {
                    exp_half(0, sum_a);
                    fresh = __any_sync(0xffffffffu, !(sum_a[0] <= 64.f && sum_a[1] <= 64.f));
                }
                if (fresh) {
                    refresh(j > 0, factor);       // S_j complete means P.V of step j - 1 has completed: O is at rest
                    exp_half(0, sum_a);
                    l_row[q][0] *= factor[0];
                    l_row[q][1] *= factor[1];
                }
                release_half(0);
                exp_half(1, sum_b);
                if (!fresh && __any_sync(0xffffffffu, !(sum_a[0] + sum_b[0] <= 64.f && sum_a[1] + sum_b[1] <= 64.f))) {
                    // the first half is already with the MMA warp, in units of the old reference: wait until
                    // its P.V has landed in the accumulator, then move accumulator and sums to the new one
                    mbar_wait(smem_u32(&bars.pv_half[q]), par, abort_flag, status, 12);
                    tc_fence_after();
                    refresh(true, factor);
                    l_row[q][0] = (l_row[q][0] + sum_a[0]) * factor[0];
                    l_row[q][1] = (l_row[q][1] + sum_a[1]) * factor[1];
                    sum_a[0] = sum_a[1] = 0.f;
                    exp_half(1, sum_b);
                }
                l_row[q][0] += sum_a[0] + sum_b[0];
                l_row[q][1] += sum_a[1] + sum_b[1];
                release_half(1);
            }
        }

        // epilogue of the item: O / l -> bf16, LSE.  The producer and the MMA warps are already on
        // the next item; its first P.V needs the P these warps write after this epilogue, so the
        // accumulators are not touched before they have been read here.
        for (int q = 0; q < n_tiles; ++q) {
            const AttnTile &t = q ? t1 : t0;
            const int my_steps = q ? n_steps1 : n_steps0;
            mbar_wait(smem_u32(&bars.pv_done[q]), (step_base[q] + my_steps - 1) & 1, abort_flag, status, 9);
            tc_fence_after();
            const float l_tot[2] = {quad_sum(l_row[q][0]), quad_sum(l_row[q][1])};
            const uint32_t tO = tmem + kTmemO + q * 128 + lane_base;
            uint32_t o[kD / 2];
            if (it.wk.n_parts > 1) {
                // split-KV part: unnormalised accumulator, reference maximum and sum go to the workspace
                const size_t slot = ((size_t)(q ? it.wk.tile_b : it.wk.tile_a) * H_kv + kvh) * max_parts + it.wk.part;
                if constexpr (kD == 128) tmem_ld_16x256b_x16(tO, o); else tmem_ld_16x256b_x8(tO, o);
                tmem_wait_ld();
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    float *po = ws_o + (slot * kRows + rows[rr]) * kD + cq;
#pragma unroll
                    for (int k = 0; k < kD / 8; ++k)
                        *reinterpret_cast<uint2 *>(po + 8 * k) = make_uint2(o[4 * k + 2 * rr], o[4 * k + 2 * rr + 1]);
                    if ((lane & 3) == 0) ws_ml[slot * kRows + rows[rr]] = make_float2(m_row[q][rr], l_tot[rr]);
                }
                continue;
            }
            const float inv[2] = {__frcp_rn(l_tot[0]), __frcp_rn(l_tot[1])};
#pragma unroll
            for (int rr = 0; rr < 2; ++rr)
                if (lse && row_valid[q][rr] && (lane & 3) == 0)
                    lse[(size_t)(t.q_begin + tok[q][rr]) * H_q + kvh * g + rows[rr] % g] =
                        (m_row[q][rr] + log2f(l_tot[rr])) * 0.6931471805599453f;
            const bool full_tile = t.n_tok == kRows / g;
            uint8_t *stage = sm + G::kSmemStage;
            if (full_tile) {
                // A full tile leaves through shared memory and one tiled bulk store per 64 columns: the
                // tile is laid out like a Q tile (row = token * g + head, 128-byte swizzle), so the
                // store writes whole 128-byte lines.
                if (tid == 0) bulk_wait_read();            // the previous tile's store has read the buffer
                named_sync(5, 256);
            }
            if constexpr (kD == 128) tmem_ld_16x256b_x16(tO, o); else tmem_ld_16x256b_x8(tO, o);
            tmem_wait_ld();
            if (full_tile) {
#pragma unroll
                for (int rr = 0; rr < 2; ++rr)
#pragma unroll
                    for (int k = 0; k < kD / 8; ++k) {
                        // columns 8k + cq, + 1 of row rows[rr]: 16-byte chunk k % 8 of 64-column half k / 8
                        float y0, y1;
                        fma2(y0, y1, __uint_as_float(o[4 * k + 2 * rr]), __uint_as_float(o[4 * k + 2 * rr + 1]), inv[rr], 0.f);
                        *reinterpret_cast<uint32_t *>(stage + (k >> 3) * kHalfBytes + rr * (8 * 128) + stage_off[k & 7]) = pack_bf16(y0, y1);
                    }
            } else {
                // a request's last, partly filled tile: 4-byte stores straight to `out`
#pragma unroll
                for (int rr = 0; rr < 2; ++rr) {
                    if (!row_valid[q][rr]) continue;
                    __nv_bfloat16 *orow = out + ((size_t)(t.q_begin + tok[q][rr]) * H_q + kvh * g + rows[rr] % g) * kD + cq;
#pragma unroll
                    for (int k = 0; k < kD / 8; ++k)
                        *reinterpret_cast<uint32_t *>(orow + 8 * k) =
                            pack_bf16(__uint_as_float(o[4 * k + 2 * rr]) * inv[rr], __uint_as_float(o[4 * k + 2 * rr + 1]) * inv[rr]);
                }
            }
            if (full_tile) {
                fence_proxy_async_smem();
                named_sync(5, 256);
                if (tid == 0) {
#pragma unroll
                    for (int hf = 0; hf < G::kHalves; ++hf)
                        tma_store_3d(&tmap_o, smem_u32(stage + hf * kHalfBytes), hf * 64, kvh * g, t.q_begin);
                    bulk_commit();
                }
            }
        }
        step_base[0] += n_steps0;
        step_base[1] += n_steps1;
        }
    }

    if (tid == 0) bulk_wait_all();    // the block's output stores are complete
    if (*abort_flag) {            // a wait gave up: let copies still in flight land before the block exits
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) {}
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

// Merges the parts of a split-KV launch: for every row, O = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m)
// with m = max_p m_p.  One warp per row (lanes walk head_dim), 8 rows per block, kRows / 8 blocks per
// (tile, KV head) item; all parts of a row are loaded before any is used.
template <int kD>
__global__ void __launch_bounds__(256)
attn_combine_kernel(const CombineItem *__restrict__ items, const AttnTile *__restrict__ tiles,
                    const float *__restrict__ ws_o, const float2 *__restrict__ ws_ml, __nv_bfloat16 *__restrict__ out,
                    float *__restrict__ lse, int H_q, int H_kv, int g, int max_parts) {
    constexpr int kBlocksPerItem = kRows / 8;
    const CombineItem it = items[blockIdx.x / kBlocksPerItem];
    const AttnTile t = tiles[it.tile];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = (blockIdx.x % kBlocksPerItem) * 8 + warp;
    if (row >= t.n_tok * g) return;
    const size_t slot0 = ((size_t)it.tile * H_kv + it.kvh) * max_parts;
    float2 ml[kSplitMaxParts];
    float4 o[kSplitMaxParts];
#pragma unroll
    for (int p = 0; p < kSplitMaxParts; ++p)
        if (p < it.n_parts) {
            ml[p] = ws_ml[(slot0 + p) * kRows + row];
            o[p] = lane * 4 < kD ? *reinterpret_cast<const float4 *>(ws_o + ((slot0 + p) * kRows + row) * kD + lane * 4)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    float m = -INFINITY;
#pragma unroll
    for (int p = 0; p < kSplitMaxParts; ++p)
        if (p < it.n_parts) m = fmaxf(m, ml[p].x);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
#pragma unroll
    for (int p = 0; p < kSplitMaxParts; ++p)
        if (p < it.n_parts) {
            const float w = exp2f(ml[p].x - m);
            l += ml[p].y * w;
            acc.x = fmaf(o[p].x, w, acc.x); acc.y = fmaf(o[p].y, w, acc.y);
            acc.z = fmaf(o[p].z, w, acc.z); acc.w = fmaf(o[p].w, w, acc.w);
        }
    const float inv = 1.f / l;
    const int tok = t.q_begin + row / g, head = it.kvh * g + row % g;
    uint2 pk;
    pk.x = pack_bf16(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16(acc.z * inv, acc.w * inv);
    if (lane * 4 < kD) *reinterpret_cast<uint2 *>(out + ((size_t)tok * H_q + head) * kD + lane * 4) = pk;
    if (lse && lane == 0) lse[(size_t)tok * H_q + head] = (m + log2f(l)) * 0.6931471805599453f;
}

template <int D, int kMaxPages, bool K8>
cudaError_t launch_attn_tc_d(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, void *out,
                             float *lse, int chunk, int max_blocks, float qk_scale, cudaStream_t st, std::string *err) {
    const AttnWork *work = chunk < 0 ? pl->dev.work : pl->dev.work_chunked + pl->chunk_work_off[chunk];
    const size_t n_work = chunk < 0 ? pl->work.size() : (size_t)(pl->chunk_work_off[chunk + 1] - pl->chunk_work_off[chunk]);
    if (n_work == 0) return cudaSuccess;
    const int Hq = pl->cfg.num_q_heads, Hkv = pl->cfg.num_kv_heads, g = Hq / Hkv, ps = pl->cfg.page_size;
    CUtensorMap tq, tk, tv, to;
    if (K8) {      // q and k_pool hold one byte per element
        if (!make_q_tmap8(&tq, q, pl->n_q, Hq, D, g, kRows / g, err)) return cudaErrorInvalidValue;
        if (!make_pool_tmap8(&tk, k_pool, pl->num_pool_pages, ps, Hkv, D, err)) return cudaErrorInvalidValue;
    } else {
        if (!make_q_tmap(&tq, q, pl->n_q, Hq, D, g, kRows / g, err)) return cudaErrorInvalidValue;
        if (!make_pool_tmap(&tk, k_pool, pl->num_pool_pages, ps, Hkv, D, err)) return cudaErrorInvalidValue;
    }
    if (!make_q_tmap(&to, out, pl->n_q, Hq, D, g, kRows / g, err)) return cudaErrorInvalidValue;   // `out` has the layout of a 16-bit q
    if (!make_pool_tmap(&tv, v_pool, pl->num_pool_pages, ps, Hkv, D, err)) return cudaErrorInvalidValue;
    {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<D, kMaxPages, K8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Geo<D>::kSmemAlloc);
        if (e != cudaSuccess) { *err = "cudaFuncSetAttribute(shared memory)"; return e; }
    }
    const DeviceTables &d = pl->dev;
    const float scale_log2 = pl->sm_scale * 1.4426950408889634f * qk_scale;
    // persistent: one thread block per SM (fewer when the list is shorter)
    const int sms = max_blocks > 0 ? std::min(max_blocks, pl->num_sms) : pl->num_sms;
    const unsigned grid = (unsigned)std::min<size_t>(n_work, (size_t)sms);
    attn_tc_kernel<D, kMaxPages, K8><<<grid, kThreads, Geo<D>::kSmemAlloc, st>>>(
        tq, tk, tv, to, d.tiles, work, (int)n_work, d.q_pos, d.page_off, d.pages, d.seq_len,
        static_cast<__nv_bfloat16 *>(out), lse, Hq, g, Hkv, ps, pl->num_pool_pages, scale_log2, pl->max_parts, d.ws_o, d.ws_ml, d.status);
    count_launch();
    if (pl->max_parts > 1) {
        const int c0 = chunk < 0 ? 0 : pl->chunk_combine_off[chunk];
        const int c1 = chunk < 0 ? (int)pl->combine.size() : pl->chunk_combine_off[chunk + 1];
        if (c1 > c0) {
            attn_combine_kernel<D><<<(c1 - c0) * (kRows / 8), 256, 0, st>>>(d.combine + c0, d.tiles, d.ws_o, d.ws_ml, static_cast<__nv_bfloat16 *>(out),
                                                                          lse, Hq, Hkv, g, pl->max_parts);
            count_launch();
        }
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) *err = "kernel launch";
    return e;
}

}  // namespace

cudaError_t launch_attn_tc(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, void *out,
                           float *lse, int chunk, int max_blocks, cudaStream_t st, std::string *err) {
    if (pl->n_q == 0 || pl->work.empty()) return cudaSuccess;
    const int D = pl->cfg.head_dim, ps = pl->cfg.page_size, g = pl->cfg.num_q_heads / pl->cfg.num_kv_heads;
    if ((D != 64 && D != 128) || (ps != 8 && ps != 16 && ps != 32 && ps != 64 && ps != 128) || g > 16) {
        *err = "shape outside the tcgen05 kernel's range";
        return cudaErrorNotSupported;
    }
    if (ps == 8)
        return D == 128 ? launch_attn_tc_d<128, 16, false>(pl, k_pool, v_pool, q, out, lse, chunk, max_blocks, 1.f, st, err)
                        : launch_attn_tc_d<64, 16, false>(pl, k_pool, v_pool, q, out, lse, chunk, max_blocks, 1.f, st, err);
    return D == 128 ? launch_attn_tc_d<128, 8, false>(pl, k_pool, v_pool, q, out, lse, chunk, max_blocks, 1.f, st, err)
                    : launch_attn_tc_d<64, 8, false>(pl, k_pool, v_pool, q, out, lse, chunk, max_blocks, 1.f, st, err);
}

cudaError_t launch_attn_tc_k8(const tessera_plan *pl, void *k_pool8, void *v_pool, const void *q8, void *out,
                              float *lse, float qk_scale, cudaStream_t st, std::string *err) {
    if (pl->n_q == 0 || pl->work.empty()) return cudaSuccess;
    const int D = pl->cfg.head_dim, ps = pl->cfg.page_size, g = pl->cfg.num_q_heads / pl->cfg.num_kv_heads;
    if (D != 128 || (ps != 8 && ps != 16 && ps != 32 && ps != 64 && ps != 128) || g > 16) {
        *err = "8-bit keys: head_dim 128 only";
        return cudaErrorNotSupported;
    }
    return ps == 8 ? launch_attn_tc_d<128, 16, true>(pl, k_pool8, v_pool, q8, out, lse, -1, 0, qk_scale, st, err)
                   : launch_attn_tc_d<128, 8, true>(pl, k_pool8, v_pool, q8, out, lse, -1, 0, qk_scale, st, err);
}

}  // namespace tessera

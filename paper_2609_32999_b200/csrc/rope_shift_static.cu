// tessera_rope_shift_static: the in-place RoPE shift for callers that may not allocate device
// memory.  The regular path keeps its cos/sin table in memory that tessera_plan_create obtains with
// cudaMalloc; code running inside a memory-pool-owning serving engine, in a phase where the
// allocator must stay untouched, or under a strict no-allocation policy after start-up cannot do
// that.  Here the table lives in a fixed array that is
// part of the library image, so a call allocates nothing - neither through cudaMalloc nor through
// any allocating library routine.
#include <cmath>
#include <cstring>
#include <string>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "launch.h"
#include "plan.h"

namespace tessera {
int32_t api_set_error(int32_t code, const std::string &msg);   // defined in api.cu
}

namespace {

constexpr int kMaxShifts = TESSERA_STATIC_MAX_SHIFTS;   // distinct shift amounts per call
constexpr int kMaxHalf = 64;                            // head_dim / 2 at most

// Scratch: (cos, sin) of every (shift, pair).  256 KB held by every device that loads the library,
// shared by all calls and keeping the last call's contents.
static __device__ __align__(256) float2 g_rope_scratch[kMaxShifts * kMaxHalf];

constexpr int kMaxDevices = 64;
float2 *g_scratch_addr[kMaxDevices] = {};               // device address of the array, per device

// The call's shift amounts and rotary frequencies travel by value as a kernel parameter (2.5 KB), so
// no host buffer has to outlive the call and nothing is copied from pageable memory.
struct ShiftParams {
    int32_t shifts[kMaxShifts];
    double inv_freq[kMaxHalf];
};

// Fills rows [0, n_shifts) of the scratch table: one thread block per shift amount, thread m
// evaluates the angle shift x frequency_m, its cosine and sine in fp64 and stores them as fp32.
__global__ void __launch_bounds__(kMaxHalf)
rope_static_fill_kernel(const __grid_constant__ ShiftParams prm, float2 *__restrict__ table, int half) {
    const int m = threadIdx.x;
    if (m >= half) return;
    double sn, cs;
    sincos((double)prm.shifts[blockIdx.x] * prm.inv_freq[m], &sn, &cs);
    table[(size_t)blockIdx.x * half + m] = make_float2((float)cs, (float)sn);
}

// (x, y) -> (x cos - y sin, y cos + x sin) in fp32; an entry that is exactly (1, 0) leaves the pair's
// bits alone, so a zero shift is a bit copy (signed zeros included).
__device__ __forceinline__ void rotate_pair(float &x, float &y, const float2 c) {
    const bool identity = c.x == 1.f && c.y == 0.f;
    const float a = fmaf(-y, c.y, x * c.x), b = fmaf(x, c.y, y * c.x);
    x = identity ? x : a;
    y = identity ? y : b;
}

// One warp per slot: lane handles pair-chunks (a 16-byte chunk of a head's first half and its
// partner D/2 elements later), the arithmetic of the plan-based shift kernel.  A listed slot outside
// [0, num_pool_slots) or a shift index outside the table is skipped, never dereferenced.
template <int D>
__global__ void __launch_bounds__(256)
rope_shift_static_kernel(uint4 *__restrict__ k_pool, const int32_t *__restrict__ slots,
                         const int32_t *__restrict__ slot_shift, int n, int n_shifts, int64_t num_pool_slots,
                         const float2 *__restrict__ table, int H_kv) {
    constexpr int CPH = D / 16, HALF = D / 16;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= n) return;
    const int row = slot_shift[warp];
    const int64_t slot = slots[warp];
    if (row < 0 || row >= n_shifts || slot < 0 || slot >= num_pool_slots) return;
    const size_t base = (size_t)slot * (H_kv * (D / 8));
    const float2 *cs = table + (size_t)row * (D / 2);
    for (int t = lane; t < H_kv * CPH; t += 32) {
        const int c = t % CPH;
        uint4 *plo = k_pool + base + (t / CPH) * (D / 8) + c, *phi = plo + HALF;
        uint4 lo = *plo, hi = *phi;
        uint32_t *l = reinterpret_cast<uint32_t *>(&lo), *h = reinterpret_cast<uint32_t *>(&hi);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float x0 = __uint_as_float(l[i] << 16), x1 = __uint_as_float(l[i] & 0xffff0000u);
            float y0 = __uint_as_float(h[i] << 16), y1 = __uint_as_float(h[i] & 0xffff0000u);
            rotate_pair(x0, y0, cs[c * 8 + 2 * i]);
            rotate_pair(x1, y1, cs[c * 8 + 2 * i + 1]);
            __nv_bfloat162 pa = __floats2bfloat162_rn(x0, x1), pb = __floats2bfloat162_rn(y0, y1);
            l[i] = *reinterpret_cast<uint32_t *>(&pa);
            h[i] = *reinterpret_cast<uint32_t *>(&pb);
        }
        *plo = lo;
        *phi = hi;
    }
}

}  // namespace

extern "C" int32_t tessera_rope_shift_static(const tessera_model_cfg *cfg, void *k_pool, int64_t num_pool_slots,
                                             const int32_t *slots, const int32_t *slot_shift, int32_t n_slots,
                                             const int32_t *shifts, int32_t n_shifts, void *stream) {
    using tessera::api_set_error;
    if (!cfg || !k_pool || n_slots < 0 || n_shifts < 0 || num_pool_slots < 0 ||
        (n_slots > 0 && (!slots || !slot_shift || !shifts)))
        return api_set_error(TESSERA_INVALID_ARG, "rope_shift_static: null pointer or negative count");
    if ((reinterpret_cast<uintptr_t>(k_pool) & 15) != 0)
        return api_set_error(TESSERA_INVALID_ARG, "rope_shift_static: k_pool must be 16-byte aligned");
    const int D = cfg->head_dim, H = cfg->num_kv_heads;
    if ((D != 64 && D != 128) || H <= 0 || cfg->rope_pairing != 0)
        return api_set_error(TESSERA_UNSUPPORTED_SHAPE, "rope_shift_static: head_dim 64 or 128, half-split pairs only");
    if (n_shifts > kMaxShifts)
        return api_set_error(TESSERA_UNSUPPORTED_SHAPE,
                             "rope_shift_static: " + std::to_string(n_shifts) + " distinct shifts exceed the fixed table of " +
                                 std::to_string(kMaxShifts));
    if (!cfg->inv_freq && !(cfg->rope_theta > 0.0))
        return api_set_error(TESSERA_INVALID_ARG, "rope_shift_static: rope_theta must be positive");
    if (n_slots == 0 || n_shifts == 0) return TESSERA_OK;

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: cudaGetDevice: ") + cudaGetErrorString(e));
    if (!g_scratch_addr[dev]) {
        // The array's name is only a host-side handle; the kernels need its address on THIS device.
        float2 *p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_rope_scratch);
        if (e != cudaSuccess || !p)
            return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    float2 *table = g_scratch_addr[dev];

    // Frequencies are fixed on the host (the numbers the plan-based path uses); the angles, cosines
    // and sines are evaluated by the fill kernel in fp64 and rounded once to fp32.
    static thread_local ShiftParams prm;
    std::memcpy(prm.shifts, shifts, sizeof(int32_t) * (size_t)n_shifts);
    for (int m = 0; m < D / 2; ++m)
        prm.inv_freq[m] = cfg->inv_freq ? cfg->inv_freq[m] : std::pow(cfg->rope_theta, -2.0 * m / D);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rope_static_fill_kernel<<<n_shifts, kMaxHalf, 0, st>>>(prm, table, D / 2);
    tessera::count_launch();
    const int blocks = (n_slots + 7) / 8;
    auto *kp = static_cast<uint4 *>(k_pool);
    if (D == 128)
        rope_shift_static_kernel<128><<<blocks, 256, 0, st>>>(kp, slots, slot_shift, n_slots, n_shifts, num_pool_slots, table, H);
    else
        rope_shift_static_kernel<64><<<blocks, 256, 0, st>>>(kp, slots, slot_shift, n_slots, n_shifts, num_pool_slots, table, H);
    tessera::count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess)
        return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: launch: ") + cudaGetErrorString(e));
    return TESSERA_OK;
}

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
#include <vector>

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

// One warp per slot: lane handles pair-chunks (a 16-byte chunk of a head's first half and its
// partner D/2 elements later), exactly the arithmetic of the plan-based shift kernel.
template <int D>
__global__ void __launch_bounds__(256)
rope_shift_static_kernel(uint4 *__restrict__ k_pool, const int32_t *__restrict__ slots,
                         const int32_t *__restrict__ slot_shift, int n, int n_shifts,
                         const float2 *__restrict__ table, int H_kv) {
    constexpr int CPH = D / 16, HALF = D / 16;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= n) return;
    const int row = slot_shift[warp];
    if (row < 0 || row >= n_shifts) return;             // never index outside the table
    const size_t base = (size_t)slots[warp] * (H_kv * (D / 8));
    const float2 *cs = table + (size_t)row * (D / 2);
    for (int t = lane; t < H_kv * CPH; t += 32) {
        const int c = t % CPH;
        uint4 *plo = k_pool + base + (t / CPH) * (D / 8) + c, *phi = plo + HALF;
        uint4 lo = *plo, hi = *phi;
        uint32_t *l = reinterpret_cast<uint32_t *>(&lo), *h = reinterpret_cast<uint32_t *>(&hi);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float x0 = __uint_as_float(l[i] << 16), x1 = __uint_as_float(l[i] & 0xffff0000u);
            const float y0 = __uint_as_float(h[i] << 16), y1 = __uint_as_float(h[i] & 0xffff0000u);
            const float2 c0 = cs[c * 8 + 2 * i], c1 = cs[c * 8 + 2 * i + 1];
            __nv_bfloat162 pa = __floats2bfloat162_rn(fmaf(-y0, c0.y, x0 * c0.x), fmaf(-y1, c1.y, x1 * c1.x));
            __nv_bfloat162 pb = __floats2bfloat162_rn(fmaf(x0, c0.y, y0 * c0.x), fmaf(x1, c1.y, y1 * c1.x));
            l[i] = *reinterpret_cast<uint32_t *>(&pa);
            h[i] = *reinterpret_cast<uint32_t *>(&pb);
        }
        *plo = lo;
        *phi = hi;
    }
}

}  // namespace

extern "C" int32_t tessera_rope_shift_static(const tessera_model_cfg *cfg, void *k_pool, const int32_t *slots,
                                             const int32_t *slot_shift, int32_t n_slots, const int32_t *shifts,
                                             int32_t n_shifts, void *stream) {
    using tessera::api_set_error;
    if (!cfg || !k_pool || n_slots < 0 || n_shifts < 0 || (n_slots > 0 && (!slots || !slot_shift || !shifts)))
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
        // The array's name is only a host-side handle; the kernel needs its address on THIS device.
        float2 *p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_rope_scratch);
        if (e != cudaSuccess || !p)
            return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
        g_scratch_addr[dev] = p;
    }
    float2 *table = g_scratch_addr[dev];

    // cos/sin in fp64, one rounding to fp32 - the same numbers the plan-based path tabulates.
    std::vector<float> host_table((size_t)n_shifts * (D / 2) * 2);   // host memory only; staged by the copy below
    for (int r = 0; r < n_shifts; ++r)
        for (int m = 0; m < D / 2; ++m) {
            const double w = cfg->inv_freq ? cfg->inv_freq[m] : std::pow(cfg->rope_theta, -2.0 * m / D);
            const double ang = (double)shifts[r] * w;
            host_table[(r * (D / 2) + m) * 2 + 0] = (float)std::cos(ang);
            host_table[(r * (D / 2) + m) * 2 + 1] = (float)std::sin(ang);
        }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    e = cudaMemcpyAsync(table, host_table.data(), (size_t)n_shifts * (D / 2) * sizeof(float2), cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess)
        return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: table upload: ") + cudaGetErrorString(e));
    const int blocks = (n_slots + 7) / 8;
    auto *kp = static_cast<uint4 *>(k_pool);
    if (D == 128)
        rope_shift_static_kernel<128><<<blocks, 256, 0, st>>>(kp, slots, slot_shift, n_slots, n_shifts, table, H);
    else
        rope_shift_static_kernel<64><<<blocks, 256, 0, st>>>(kp, slots, slot_shift, n_slots, n_shifts, table, H);
    tessera::count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess)
        return api_set_error(TESSERA_CUDA_ERROR, std::string("rope_shift_static: launch: ") + cudaGetErrorString(e));
    return TESSERA_OK;
}

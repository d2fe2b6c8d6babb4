// Launch entry points of the individual kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>

#include "plan.h"

namespace tessera {

enum class GatherMode { kCopy, kCopyRotate, kShiftInPlace };

void count_launch();   // bumps the process-wide kernel-launch counter

// Sources are read from (k_src, v_src) - the destination pools themselves unless the plan names a
// separate source pool - and written to the plan's destination slots in (k_pool, v_pool).
cudaError_t launch_gather(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                          GatherMode mode, cudaStream_t st);
// The same kernels over items [first_item, first_item + n_items) of the plan, with the source slots taken
// from `g_src` (device, indexed like the plan's copy list).  max_blocks > 0 caps the grid: the blocks
// then walk the items, so the launch occupies only a few SMs (host-tier reader beside the attention kernel).
cudaError_t launch_gather_range(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                                GatherMode mode, const int32_t *g_src, int first_item, int n_items, int max_blocks,
                                cudaStream_t st);
cudaError_t launch_kv_fp8_range(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst,
                                bool to_8bit, bool rotate, float k_mul, float v_mul, const int32_t *g_src, int first_item,
                                int n_items, int max_blocks, cudaStream_t st);
// 8-bit (e4m3) tier.  to_8bit false: (k_src, v_src) hold codes, (k_dst, v_dst) 16-bit pages, mul = scale;
// to_8bit true: the reverse, mul = 1 / scale.  Copy list and shift table are the plan's.
cudaError_t launch_kv_fp8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst, void *v_dst,
                          bool to_8bit, bool rotate, float k_mul, float v_mul, cudaStream_t st);
// In-place rotation of the fresh q / k_new rows for their target positions (either may be null).
cudaError_t launch_rope_fresh(const tessera_plan *pl, void *q, void *k_new, cudaStream_t st);
// Fused write side of the extend pass: rotate q in place, write rotated K / V rows to their slots and raw
// K / V rows of captured units to their cache slots (k_cache / v_cache may be null when nothing is captured).
cudaError_t launch_extend_write(const tessera_plan *pl, void *k_pool, void *v_pool, void *q, const void *k_new_raw,
                                const void *v_new, void *k_cache, void *v_cache, cudaStream_t st);
// chunk < 0: the whole batch; otherwise only request chunk `chunk` (see tessera_plan::chunk_row_off).
// k_new / v_new / q / out / lse always point at row 0 of the whole batch.
cudaError_t launch_scatter_fresh(const tessera_plan *pl, void *k_pool, void *v_pool, const void *k_new,
                                 const void *v_new, int chunk, cudaStream_t st);
// tcgen05 attention; returns cudaErrorNotSupported when the plan's shape is outside its range (the plan
// builder accepts no such shape).
// max_blocks > 0 caps the persistent grid below one block per SM (SMs left to a concurrent reader kernel).
cudaError_t launch_attn_tc(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, void *out,
                           float *lse, int chunk, int max_blocks, cudaStream_t st, std::string *err);

// The same kernel with 8-bit (e4m3) queries and keys: q8 [n_q][H_q][D] and k_pool8 hold codes, qk_scale is the
// product of their two scales; head_dim 128 only; the whole batch on the full grid.
cudaError_t launch_attn_tc_k8(const tessera_plan *pl, void *k_pool8, void *v_pool, const void *q8, void *out,
                              float *lse, float qk_scale, cudaStream_t st, std::string *err);
// Compose for the 8-bit-key attention path: 16-bit sources -> keys (rotated, times k_mul) as e4m3 codes in
// k_dst8, values as bit copies in the 16-bit v_dst.
cudaError_t launch_compose_k8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst8, void *v_dst,
                              bool rotate, float k_mul, cudaStream_t st);
// bf16 rows -> e4m3 codes of (value * mul), nearest-even, saturating: n_elems elements (a multiple of 8).
cudaError_t launch_quantize_e4m3(const void *src_bf16, void *dst8, int64_t n_elems, float mul, cudaStream_t st);
// Fresh rows into an 8-bit key pool (codes of k_new * k_mul) and a 16-bit value pool (bit copies).
cudaError_t launch_scatter_fresh_k8(const tessera_plan *pl, void *k_pool8, void *v_pool, const void *k_new,
                                    const void *v_new, float k_mul, cudaStream_t st);

}  // namespace tessera

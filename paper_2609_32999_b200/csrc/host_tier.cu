// Local-hit tier, overlapped (Sec. 5.3 "Preparing cache hits": a local hit is copied from the node's
// pinned host-memory cache into the request's KV slots while the engine keeps serving what is already
// prepared; Sec. 4: the host cache belongs to the generation node).
//
// The cached units live in a pinned host pool.  Per chunk of whole requests, a READER launch of the
// gather kernel - a handful of thread blocks that walk the chunk's copy list - pulls the rows over the
// interconnect straight into their destination slots (keys rotated on the way: no staging buffer at
// all), on a side stream; as soon as a chunk has arrived, its fresh-row scatter and attention run on
// the caller's stream with a persistent grid that leaves the reader's SMs alone.  The link (about
// 50 GB/s) is the bound; what overlaps is the attention of chunk c with the transfer of chunk c + 1.
//
// Why a reader kernel and not the copy engine: units are stored as non-adjacent fixed-size blocks
// (Sec. 5.1), so a DMA path needs one copy per block and tensor.  Measured on a B200 with 128 KB
// blocks, 3 500 cudaMemcpyAsync calls per layer into a device staging area cost 25 ms for 537 MB
// (21 GB/s) against 10.5 ms for the reader kernel.  And why a capped grid: the attention kernel takes a
// whole SM per thread block (all registers, all shared memory), so nothing runs beside it on an SM; a
// full-size gather launch would hold every SM until its slow host reads return.
#include <algorithm>
#include <string>

#include <cuda_runtime.h>

#include "launch.h"
#include "plan.h"

namespace tessera {
int32_t api_set_error(int32_t code, const std::string &msg);   // defined in api.cu
int32_t api_attention(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, const void *k_new,
                      const void *v_new, void *out, float *lse, int chunk, int max_blocks, cudaStream_t st);
int32_t api_ensure_pipeline(tessera_plan *pl);
}  // namespace tessera

namespace {

using namespace tessera;

int32_t cuda_fail(cudaError_t e, const char *what) {
    return api_set_error(TESSERA_CUDA_ERROR, std::string("host tier: ") + what + ": " + cudaGetErrorString(e));
}
#define HT_CUDA(call)                                       \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

constexpr int kDefaultReaderBlocks = 16;   // 16 x 256 threads x 128 B in flight = 512 KB: several times what the link needs

bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

}  // namespace

extern "C" int32_t tessera_composed_prefill_host_tier(tessera_plan *pl, const void *k_src_host, const void *v_src_host,
                                                      int32_t src_format, float k_scale, float v_scale, void *k_pool,
                                                      void *v_pool, const void *q, const void *k_new, const void *v_new,
                                                      void *out, float *lse, int32_t reader_blocks, void *stream) {
    if (!pl) return api_set_error(TESSERA_INVALID_ARG, "null plan");
    if (pl->host_only) return api_set_error(TESSERA_INVALID_ARG, "plan was created with TESSERA_PLAN_HOST_ONLY");
    if (pl->num_source_pages <= 0)
        return api_set_error(TESSERA_INVALID_ARG, "the plan was created without a separate source pool (desc.num_source_pages)");
    if (src_format != 0 && src_format != 1) return api_set_error(TESSERA_INVALID_ARG, "src_format: 0 (bf16 units) or 1 (e4m3 units)");
    if (src_format == 1 && (!(k_scale > 0.f) || !(v_scale > 0.f) || k_scale > 3.0e38f || v_scale > 3.0e38f))
        return api_set_error(TESSERA_INVALID_ARG, "k_scale / v_scale must be positive and finite");
    if (!k_src_host || !v_src_host || !k_pool || !v_pool || misaligned(k_src_host) || misaligned(v_src_host) ||
        misaligned(k_pool) || misaligned(v_pool))
        return api_set_error(TESSERA_INVALID_ARG, "k_src_host / v_src_host / k_pool / v_pool must be non-null and 16-byte aligned");
    if (pl->n_q > 0 && (!q || !out)) return api_set_error(TESSERA_INVALID_ARG, "q and out must be non-null");
    if (misaligned(q) || misaligned(out) || misaligned(k_new) || misaligned(v_new))
        return api_set_error(TESSERA_INVALID_ARG, "q / out / k_new / v_new must be 16-byte aligned");
    if (reader_blocks < 0 || reader_blocks > pl->num_sms / 2)
        return api_set_error(TESSERA_INVALID_ARG, "reader_blocks: 0 (default) up to half the SM count");
    const int readers = reader_blocks > 0 ? reader_blocks : std::min(kDefaultReaderBlocks, pl->num_sms / 2);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (int32_t rc = api_ensure_pipeline(pl)) return rc;

    const int n_chunks = (int)pl->chunk_item_off.size() - 1;
    // the reader starts after everything already queued on the caller's stream (an earlier layer may
    // still be reading these destination pages)
    HT_CUDA(cudaEventRecord(pl->ev_start, st));
    HT_CUDA(cudaStreamWaitEvent(pl->s_in, pl->ev_start, 0));
    for (int c = 0; c < n_chunks; ++c) {
        const int first = pl->chunk_item_off[c], n = pl->chunk_item_off[c + 1] - first;
        // the last chunk has nothing to overlap with: it takes the whole GPU
        const int cap = c + 1 < n_chunks ? readers : 0;
        if (src_format == 0)
            HT_CUDA(launch_gather_range(pl, k_src_host, v_src_host, k_pool, v_pool, GatherMode::kCopyRotate, pl->dev.g_src,
                                        first, n, cap, pl->s_in));
        else
            HT_CUDA(launch_kv_fp8_range(pl, k_src_host, v_src_host, k_pool, v_pool, false, true, k_scale, v_scale,
                                        pl->dev.g_src, first, n, cap, pl->s_in));
        HT_CUDA(cudaEventRecord(pl->ev_in[c], pl->s_in));
    }
    for (int c = 0; c < n_chunks; ++c) {
        HT_CUDA(cudaStreamWaitEvent(st, pl->ev_in[c], 0));
        // while a later chunk is still on the link, attention leaves the reader's SMs alone
        const int max_blocks = c + 1 < n_chunks ? pl->num_sms - readers : 0;
        if (int32_t rc = api_attention(pl, k_pool, v_pool, q, k_new, v_new, out, lse, c, max_blocks, st)) return rc;
    }
    return TESSERA_OK;
}

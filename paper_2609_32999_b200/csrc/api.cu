// extern "C" boundary: argument checks, plan upload, kernel launches on the caller's stream.
#include <atomic>
#include <cstring>
#include <new>
#include <string>

#include <cmath>
#include <cuda_runtime.h>

#include "launch.h"
#include "plan.h"

namespace tessera {

namespace {
thread_local std::string g_last_error;
std::atomic<int64_t> g_launches{0};

int32_t set_error(int32_t code, const std::string &msg) {
    g_last_error = msg;
    return code;
}

int32_t cuda_fail(cudaError_t e, const char *what) {
    return set_error(TESSERA_CUDA_ERROR, std::string(what) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")");
}

#define TS_CUDA(call)                                       \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call); \
    } while (0)

size_t align_up(size_t x) { return (x + 255) & ~size_t(255); }

// Multiprocessor count of the current device, asked once per device.
int32_t device_sm_count(int *out) {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cache[kMaxDevices];
    int dev = 0;
    TS_CUDA(cudaGetDevice(&dev));
    int n = (dev >= 0 && dev < kMaxDevices) ? cache[dev].load(std::memory_order_relaxed) : 0;
    if (n <= 0) {
        TS_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        if (n <= 0) return set_error(TESSERA_CUDA_ERROR, "device reports no multiprocessors");
        if (dev >= 0 && dev < kMaxDevices) cache[dev].store(n, std::memory_order_relaxed);
    }
    *out = n;
    return TESSERA_OK;
}

template <class T>
size_t place(size_t &off, size_t n) {
    size_t o = off;
    off = align_up(off + n * sizeof(T));
    return o;
}

int32_t upload(tessera_plan *pl, cudaStream_t st) {
    using namespace tessera;
    DeviceTables &d = pl->dev;
    TS_CUDA(cudaGetDevice(&pl->device));
    size_t off = 0;
    const size_t o_src = place<int32_t>(off, pl->g_src.size());
    const size_t o_dst = place<int32_t>(off, pl->g_dst.size());
    const size_t o_items = place<GatherItem>(off, pl->items.size());
    const size_t o_rope = place<float>(off, pl->rope_table.size());
    const size_t o_fresh = place<int32_t>(off, pl->fresh_dst.size());
    const size_t o_retain = place<int32_t>(off, pl->retain_dst.size());
    const size_t o_qpos = place<int32_t>(off, pl->recompute_pos.size());
    const size_t o_qreq = place<int32_t>(off, pl->q_req.size());
    const size_t o_poff = place<int32_t>(off, pl->page_off.size());
    const size_t o_pages = place<int32_t>(off, pl->pages.size());
    const size_t o_tiles = place<AttnTile>(off, pl->tiles.size());
    const size_t o_work = place<AttnWork>(off, pl->work.size());
    const size_t o_workc = place<AttnWork>(off, pl->work_chunked.size());
    const size_t o_comb = place<CombineItem>(off, pl->combine.size());
    const size_t o_seq = place<int32_t>(off, pl->seq_len.size());
    const size_t o_status = place<int32_t>(off, 4);
    const size_t o_invf = place<double>(off, pl->inv_freq.size());
    // split-KV workspace: one slot per (tile, KV head, part)
    const size_t n_slots = pl->max_parts > 1 ? pl->tiles.size() * pl->cfg.num_kv_heads * pl->max_parts : 0;
    const size_t o_wsml = place<float2>(off, n_slots * kAttnTileRows);
    const size_t o_wso = place<float>(off, n_slots * kAttnTileRows * pl->cfg.head_dim);
    const size_t table_bytes = o_wsml;    // the workspace behind it needs no upload
    pl->host_blob.assign(table_bytes, 0);
    char *hb = pl->host_blob.data();
    auto put = [&](size_t o, const void *src, size_t bytes) { if (bytes) std::memcpy(hb + o, src, bytes); };
    put(o_src, pl->g_src.data(), pl->g_src.size() * 4);
    put(o_dst, pl->g_dst.data(), pl->g_dst.size() * 4);
    put(o_items, pl->items.data(), pl->items.size() * sizeof(GatherItem));
    put(o_rope, pl->rope_table.data(), pl->rope_table.size() * 4);
    put(o_fresh, pl->fresh_dst.data(), pl->fresh_dst.size() * 4);
    put(o_retain, pl->retain_dst.data(), pl->retain_dst.size() * 4);
    put(o_qpos, pl->recompute_pos.data(), pl->recompute_pos.size() * 4);
    put(o_qreq, pl->q_req.data(), pl->q_req.size() * 4);
    put(o_poff, pl->page_off.data(), pl->page_off.size() * 4);
    put(o_pages, pl->pages.data(), pl->pages.size() * 4);
    put(o_tiles, pl->tiles.data(), pl->tiles.size() * sizeof(AttnTile));
    put(o_work, pl->work.data(), pl->work.size() * sizeof(AttnWork));
    put(o_workc, pl->work_chunked.data(), pl->work_chunked.size() * sizeof(AttnWork));
    put(o_comb, pl->combine.data(), pl->combine.size() * sizeof(CombineItem));
    put(o_invf, pl->inv_freq.data(), pl->inv_freq.size() * sizeof(double));
    put(o_seq, pl->seq_len.data(), pl->seq_len.size() * 4);
    TS_CUDA(cudaMalloc(&d.blob, off));
    TS_CUDA(cudaMemcpyAsync(d.blob, hb, table_bytes, cudaMemcpyHostToDevice, st));
    char *db = static_cast<char *>(d.blob);
    d.g_src = reinterpret_cast<int32_t *>(db + o_src);
    d.g_dst = reinterpret_cast<int32_t *>(db + o_dst);
    d.items = reinterpret_cast<GatherItem *>(db + o_items);
    d.rope = reinterpret_cast<float2 *>(db + o_rope);
    d.fresh_dst = reinterpret_cast<int32_t *>(db + o_fresh);
    d.retain_dst = pl->retain_dst.empty() ? nullptr : reinterpret_cast<int32_t *>(db + o_retain);
    d.q_pos = reinterpret_cast<int32_t *>(db + o_qpos);
    d.q_req = reinterpret_cast<int32_t *>(db + o_qreq);
    d.page_off = reinterpret_cast<int32_t *>(db + o_poff);
    d.pages = reinterpret_cast<int32_t *>(db + o_pages);
    d.tiles = reinterpret_cast<AttnTile *>(db + o_tiles);
    d.work = reinterpret_cast<AttnWork *>(db + o_work);
    d.work_chunked = reinterpret_cast<AttnWork *>(db + o_workc);
    d.combine = reinterpret_cast<CombineItem *>(db + o_comb);
    d.ws_ml = reinterpret_cast<float2 *>(db + o_wsml);
    d.ws_o = reinterpret_cast<float *>(db + o_wso);
    d.seq_len = reinterpret_cast<int32_t *>(db + o_seq);
    d.status = reinterpret_cast<int32_t *>(db + o_status);
    d.inv_freq = reinterpret_cast<double *>(db + o_invf);
    return TESSERA_OK;
}

int32_t check_device_plan(const tessera_plan *pl) {
    if (!pl) return set_error(TESSERA_INVALID_ARG, "null plan");
    if (pl->host_only) return set_error(TESSERA_INVALID_ARG, "plan was created with TESSERA_PLAN_HOST_ONLY");
    return TESSERA_OK;
}

bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) != 0; }

// Fresh-row scatter + attention of the whole batch (chunk < 0) or of one request chunk.
int32_t attention(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, const void *k_new,
                  const void *v_new, void *out, float *lse, int chunk, cudaStream_t st, int max_blocks = 0) {
    TS_CUDA(launch_scatter_fresh(pl, k_pool, v_pool, k_new, v_new, chunk, st));
    std::string err;
    cudaError_t e = launch_attn_tc(pl, k_pool, v_pool, q, out, lse, chunk, max_blocks, st, &err);
    if (e != cudaSuccess) return set_error(TESSERA_CUDA_ERROR, "tcgen05 attention launch: " + err + " / " + cudaGetErrorString(e));
    return TESSERA_OK;
}

// Streams and events of the host-buffer entry point, created once per plan.
int32_t ensure_pipeline(tessera_plan *pl) {
    if (pl->s_in) return TESSERA_OK;
    const size_t n = pl->chunk_row_off.size() - 1;
    TS_CUDA(cudaStreamCreateWithFlags(&pl->s_in, cudaStreamNonBlocking));
    TS_CUDA(cudaStreamCreateWithFlags(&pl->s_out, cudaStreamNonBlocking));
    TS_CUDA(cudaEventCreateWithFlags(&pl->ev_start, cudaEventDisableTiming));
    TS_CUDA(cudaEventCreateWithFlags(&pl->ev_out, cudaEventDisableTiming));
    pl->ev_in.assign(n, nullptr);
    pl->ev_comp.assign(n, nullptr);
    for (size_t c = 0; c < n; ++c) {
        TS_CUDA(cudaEventCreateWithFlags(&pl->ev_in[c], cudaEventDisableTiming));
        TS_CUDA(cudaEventCreateWithFlags(&pl->ev_comp[c], cudaEventDisableTiming));
    }
    return TESSERA_OK;
}

}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// Lets entry points defined in other files record the calling thread's error text, run scatter +
// attention of one request chunk (optionally on a capped grid), and create the plan's side streams.
int32_t api_set_error(int32_t code, const std::string &msg) { return set_error(code, msg); }
int32_t api_attention(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q, const void *k_new,
                      const void *v_new, void *out, float *lse, int chunk, int max_blocks, cudaStream_t st) {
    return attention(pl, k_pool, v_pool, q, k_new, v_new, out, lse, chunk, st, max_blocks);
}
int32_t api_ensure_pipeline(tessera_plan *pl) { return ensure_pipeline(pl); }

}  // namespace tessera

using namespace tessera;

extern "C" {

int32_t tessera_plan_create(const tessera_model_cfg *cfg, const tessera_compose_desc *desc, int32_t num_pool_pages,
                            uint32_t flags, tessera_plan **out, void *stream) {
    if (!out) return set_error(TESSERA_INVALID_ARG, "null out pointer");
    *out = nullptr;
    if (flags & ~uint32_t(TESSERA_PLAN_HOST_ONLY)) return set_error(TESSERA_INVALID_ARG, "unknown plan flag");
    tessera_plan *pl = new (std::nothrow) tessera_plan();
    if (!pl) return set_error(TESSERA_INVALID_ARG, "out of host memory");
    std::string err;
    int32_t st = TESSERA_INVALID_ARG;
    int num_sms = kDefaultSMs;               // a host-only plan touches no device and is sized for a B200
    if (!(flags & TESSERA_PLAN_HOST_ONLY)) {
        if (int32_t rc = device_sm_count(&num_sms)) {
            delete pl;
            return rc;
        }
    }
    try {
        st = build_plan_host(cfg, desc, num_pool_pages, num_sms, pl, &err);
    } catch (const std::bad_alloc &) {
        err = "out of host memory while building the plan";
    }
    if (st != TESSERA_OK) {
        delete pl;
        return set_error(st, err);
    }
    pl->host_only = (flags & TESSERA_PLAN_HOST_ONLY) != 0;
    if (!pl->host_only) {
        st = upload(pl, static_cast<cudaStream_t>(stream));
        if (st != TESSERA_OK) {
            if (pl->dev.blob) cudaFree(pl->dev.blob);
            delete pl;
            return st;
        }
    }
    *out = pl;
    return TESSERA_OK;
}

int32_t tessera_plan_destroy(tessera_plan *pl) {
    if (!pl) return TESSERA_OK;
    int32_t rc = TESSERA_OK;
    if (!pl->host_only) {
        for (cudaEvent_t e : pl->ev_in) if (e) cudaEventDestroy(e);
        for (cudaEvent_t e : pl->ev_comp) if (e) cudaEventDestroy(e);
        if (pl->ev_start) cudaEventDestroy(pl->ev_start);
        if (pl->ev_out) cudaEventDestroy(pl->ev_out);
        if (pl->s_in) cudaStreamDestroy(pl->s_in);
        if (pl->s_out) cudaStreamDestroy(pl->s_out);
        void *bufs[] = {pl->dev.blob, pl->dev.st_q, pl->dev.st_k, pl->dev.st_v, pl->dev.st_o, pl->dev.st_lse, pl->dev.q8};
        for (void *b : bufs)
            if (b) {
                cudaError_t e = cudaFree(b);
                if (e != cudaSuccess) rc = cuda_fail(e, "cudaFree");
            }
    }
    delete pl;
    return rc;
}

int32_t tessera_plan_block_table(const tessera_plan *pl, const int32_t **page_off, const int32_t **pages,
                                 const int32_t **src_slot) {
    if (!pl) return set_error(TESSERA_INVALID_ARG, "null plan");
    if (page_off) *page_off = pl->page_off.data();
    if (pages) *pages = pl->pages.data();
    if (src_slot) *src_slot = pl->src_slot.data();
    return TESSERA_OK;
}

int32_t tessera_plan_get_info(const tessera_plan *pl, tessera_plan_info *info) {
    if (!pl || !info) return set_error(TESSERA_INVALID_ARG, "null plan or info");
    info->total_tokens = pl->total_tokens;
    info->n_q = pl->n_q;
    info->cached_tokens = pl->cached_tokens;
    info->qk_pairs = pl->qk_pairs;
    info->gather_bytes = pl->cached_tokens * pl->cfg.num_kv_heads * pl->cfg.head_dim * 2 * 2 * 2;
    info->attn_flops = 4LL * pl->cfg.head_dim * pl->cfg.num_q_heads * pl->qk_pairs;
    info->n_rope_rows = (int32_t)pl->rope_delta.size();
    info->n_gather_items = (int32_t)pl->items.size();
    info->n_attn_items = pl->n_work_items;
    info->attn_kernel = pl->attn_kernel;
    info->retained_tokens = pl->retained_tokens;
    info->attn_mma_pairs = pl->mma_pairs;
    return TESSERA_OK;
}

int32_t tessera_plan_status(tessera_plan *pl, int32_t *detail, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t word[4] = {0, 0, 0, 0};
    TS_CUDA(cudaMemcpyAsync(word, pl->dev.status, sizeof word, cudaMemcpyDeviceToHost, st));
    TS_CUDA(cudaStreamSynchronize(st));
    if (word[0] != 0) TS_CUDA(cudaMemsetAsync(pl->dev.status, 0, sizeof word, st));
    if (detail) *detail = word[0];
    if (word[0] != 0)
        return set_error(TESSERA_DEVICE_TIMEOUT, "a bounded wait inside a kernel gave up, code " + std::to_string(word[0]));
    return TESSERA_OK;
}

int32_t tessera_kv_compose(const tessera_plan *pl, void *k_pool, void *v_pool, uint32_t flags, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (flags & ~uint32_t(TESSERA_FUSE_ROPE)) return set_error(TESSERA_INVALID_ARG, "unknown compose flag");
    if (!k_pool || !v_pool || misaligned(k_pool) || misaligned(v_pool))
        return set_error(TESSERA_INVALID_ARG, "k_pool / v_pool must be non-null and 16-byte aligned");
    if (pl->num_source_pages > 0)
        return set_error(TESSERA_INVALID_ARG, "this plan reads a separate source pool: use tessera_kv_compose_from");
    TS_CUDA(launch_gather(pl, k_pool, v_pool, k_pool, v_pool, (flags & TESSERA_FUSE_ROPE) ? GatherMode::kCopyRotate : GatherMode::kCopy,
                          static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_kv_compose_from(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool, void *v_pool,
                                uint32_t flags, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (flags & ~uint32_t(TESSERA_FUSE_ROPE)) return set_error(TESSERA_INVALID_ARG, "unknown compose flag");
    if (pl->num_source_pages <= 0)
        return set_error(TESSERA_INVALID_ARG, "the plan was created without a separate source pool (desc.num_source_pages)");
    if (!k_pool || !v_pool || !k_src || !v_src || misaligned(k_pool) || misaligned(v_pool) || misaligned(k_src) || misaligned(v_src))
        return set_error(TESSERA_INVALID_ARG, "k_src / v_src / k_pool / v_pool must be non-null and 16-byte aligned");
    TS_CUDA(launch_gather(pl, k_src, v_src, k_pool, v_pool, (flags & TESSERA_FUSE_ROPE) ? GatherMode::kCopyRotate : GatherMode::kCopy,
                          static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

namespace {
int32_t check_fp8_call(const tessera_plan *pl, const void *a, const void *b, const void *c, const void *d, uint32_t flags,
                       float k_scale, float v_scale) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (flags & ~uint32_t(TESSERA_FUSE_ROPE)) return set_error(TESSERA_INVALID_ARG, "unknown compose flag");
    if (pl->num_source_pages <= 0)
        return set_error(TESSERA_INVALID_ARG, "the plan was created without a separate source pool (desc.num_source_pages)");
    if (!a || !b || !c || !d || misaligned(a) || misaligned(b) || misaligned(c) || misaligned(d))
        return set_error(TESSERA_INVALID_ARG, "source and destination pools must be non-null and 16-byte aligned");
    if (!(k_scale > 0.f) || !(v_scale > 0.f) || std::isinf(k_scale) || std::isinf(v_scale))
        return set_error(TESSERA_INVALID_ARG, "k_scale / v_scale must be positive and finite");
    return TESSERA_OK;
}
}  // namespace

int32_t tessera_kv_compose_from_fp8(const tessera_plan *pl, const void *k_src8, const void *v_src8, float k_scale,
                                    float v_scale, void *k_pool, void *v_pool, uint32_t flags, void *stream) {
    if (int32_t rc = check_fp8_call(pl, k_src8, v_src8, k_pool, v_pool, flags, k_scale, v_scale)) return rc;
    TS_CUDA(launch_kv_fp8(pl, k_src8, v_src8, k_pool, v_pool, false, (flags & TESSERA_FUSE_ROPE) != 0, k_scale, v_scale,
                          static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_kv_retain_fp8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_dst8, void *v_dst8,
                              float k_scale, float v_scale, uint32_t flags, void *stream) {
    if (int32_t rc = check_fp8_call(pl, k_src, v_src, k_dst8, v_dst8, flags, k_scale, v_scale)) return rc;
    // the reciprocal is taken once, in fp32: every element is multiplied by it (one rounding) and then rounded to e4m3
    TS_CUDA(launch_kv_fp8(pl, k_src, v_src, k_dst8, v_dst8, true, (flags & TESSERA_FUSE_ROPE) != 0, 1.0f / k_scale,
                          1.0f / v_scale, static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_kv_compose_k8(const tessera_plan *pl, const void *k_src, const void *v_src, void *k_pool8, void *v_pool,
                              float k_scale, uint32_t flags, void *stream) {
    if (int32_t rc = check_fp8_call(pl, k_src, v_src, k_pool8, v_pool, flags, k_scale, 1.0f)) return rc;
    TS_CUDA(launch_compose_k8(pl, k_src, v_src, k_pool8, v_pool, (flags & TESSERA_FUSE_ROPE) != 0, 1.0f / k_scale,
                              static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_rope_shift(const tessera_plan *pl, void *k_pool, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (!k_pool || misaligned(k_pool)) return set_error(TESSERA_INVALID_ARG, "k_pool must be non-null and 16-byte aligned");
    TS_CUDA(launch_gather(pl, k_pool, k_pool, k_pool, k_pool, GatherMode::kShiftInPlace, static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_rope_fresh(const tessera_plan *pl, void *q, void *k_new, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (misaligned(q) || misaligned(k_new)) return set_error(TESSERA_INVALID_ARG, "q / k_new must be 16-byte aligned");
    TS_CUDA(launch_rope_fresh(pl, q, k_new, static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_extend_write(const tessera_plan *pl, void *k_pool, void *v_pool, void *q, const void *k_new_raw,
                             const void *v_new, void *k_cache, void *v_cache, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (!k_pool || !v_pool || misaligned(k_pool) || misaligned(v_pool))
        return set_error(TESSERA_INVALID_ARG, "k_pool / v_pool must be non-null and 16-byte aligned");
    if (pl->n_q > 0 && (!k_new_raw || !v_new)) return set_error(TESSERA_INVALID_ARG, "k_new_raw and v_new must be non-null");
    if (misaligned(q) || misaligned(k_new_raw) || misaligned(v_new) || misaligned(k_cache) || misaligned(v_cache))
        return set_error(TESSERA_INVALID_ARG, "q / k_new_raw / v_new / k_cache / v_cache must be 16-byte aligned");
    if (pl->retained_tokens > 0 && (!k_cache || !v_cache))
        return set_error(TESSERA_INVALID_ARG, "the plan captures units: k_cache and v_cache must be non-null");
    if (pl->retained_tokens > 0 && pl->retain_pool_pages == 0 && (k_cache != k_pool || v_cache != v_pool))
        return set_error(TESSERA_INVALID_ARG, "the plan's cache pages are pages of the destination pool: pass k_pool / v_pool as k_cache / v_cache");
    TS_CUDA(launch_extend_write(pl, k_pool, v_pool, q, k_new_raw, v_new, k_cache, v_cache, static_cast<cudaStream_t>(stream)));
    return TESSERA_OK;
}

int32_t tessera_partial_prefill_attn(const tessera_plan *pl, void *k_pool, void *v_pool, const void *q,
                                     const void *k_new, const void *v_new, void *out, float *lse, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (!k_pool || !v_pool || misaligned(k_pool) || misaligned(v_pool))
        return set_error(TESSERA_INVALID_ARG, "k_pool / v_pool must be non-null and 16-byte aligned");
    if (pl->n_q > 0 && (!q || !out)) return set_error(TESSERA_INVALID_ARG, "q and out must be non-null");
    if (misaligned(q) || misaligned(out) || misaligned(k_new) || misaligned(v_new))
        return set_error(TESSERA_INVALID_ARG, "q / out / k_new / v_new must be 16-byte aligned");
    return attention(pl, k_pool, v_pool, q, k_new, v_new, out, lse, -1, static_cast<cudaStream_t>(stream));
}

int32_t tessera_partial_prefill_attn_k8(tessera_plan *pl, void *k_pool8, float k_scale, void *v_pool, const void *q,
                                        float q_scale, const void *k_new, const void *v_new, void *out, float *lse,
                                        void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (pl->cfg.head_dim != 128) return set_error(TESSERA_UNSUPPORTED_SHAPE, "8-bit keys: head_dim 128 only");
    if (!k_pool8 || !v_pool || misaligned(k_pool8) || misaligned(v_pool))
        return set_error(TESSERA_INVALID_ARG, "k_pool8 / v_pool must be non-null and 16-byte aligned");
    if (!(k_scale > 0.f) || !(q_scale > 0.f) || std::isinf(k_scale) || std::isinf(q_scale))
        return set_error(TESSERA_INVALID_ARG, "k_scale / q_scale must be positive and finite");
    if (pl->n_q > 0 && (!q || !out)) return set_error(TESSERA_INVALID_ARG, "q and out must be non-null");
    if (misaligned(q) || misaligned(out) || misaligned(k_new) || misaligned(v_new))
        return set_error(TESSERA_INVALID_ARG, "q / out / k_new / v_new must be 16-byte aligned");
    if (pl->n_q == 0) return TESSERA_OK;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t q_elems = pl->n_q * pl->cfg.num_q_heads * pl->cfg.head_dim;
    if (!pl->dev.q8) TS_CUDA(cudaMalloc(&pl->dev.q8, (size_t)q_elems));
    // the reciprocals are taken once, in fp32: every element is multiplied by it and rounded to e4m3
    TS_CUDA(launch_quantize_e4m3(q, pl->dev.q8, q_elems, 1.0f / q_scale, st));
    TS_CUDA(launch_scatter_fresh_k8(pl, k_pool8, v_pool, k_new, v_new, 1.0f / k_scale, st));
    std::string err;
    cudaError_t e = launch_attn_tc_k8(pl, k_pool8, v_pool, pl->dev.q8, out, lse, q_scale * k_scale, st, &err);
    if (e != cudaSuccess) return set_error(TESSERA_CUDA_ERROR, "tcgen05 attention launch (8-bit keys): " + err + " / " + cudaGetErrorString(e));
    return TESSERA_OK;
}

int32_t tessera_composed_prefill_host(tessera_plan *pl, void *k_pool, void *v_pool, const void *q_host,
                                      const void *k_new_host, const void *v_new_host, void *out_host,
                                      float *lse_host, void *stream) {
    if (int32_t rc = check_device_plan(pl)) return rc;
    if (!k_pool || !v_pool || misaligned(k_pool) || misaligned(v_pool))
        return set_error(TESSERA_INVALID_ARG, "k_pool / v_pool must be non-null and 16-byte aligned");
    if (pl->num_source_pages > 0)
        return set_error(TESSERA_INVALID_ARG, "this plan reads a separate source pool: compose with tessera_kv_compose_from");
    if (pl->n_q > 0 && (!q_host || !k_new_host || !v_new_host || !out_host))
        return set_error(TESSERA_INVALID_ARG, "q / k_new / v_new / out host buffers must be non-null");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceTables &d = pl->dev;
    const size_t q_bytes = (size_t)pl->n_q * pl->cfg.num_q_heads * pl->cfg.head_dim * 2;
    const size_t kv_bytes = (size_t)pl->n_q * pl->cfg.num_kv_heads * pl->cfg.head_dim * 2;
    const size_t lse_bytes = (size_t)pl->n_q * pl->cfg.num_q_heads * sizeof(float);
    if (!d.st_q && pl->n_q > 0) {
        TS_CUDA(cudaMalloc(&d.st_q, q_bytes));
        TS_CUDA(cudaMalloc(&d.st_k, kv_bytes));
        TS_CUDA(cudaMalloc(&d.st_v, kv_bytes));
        TS_CUDA(cudaMalloc(&d.st_o, q_bytes));
        TS_CUDA(cudaMalloc(reinterpret_cast<void **>(&d.st_lse), lse_bytes));
        TS_CUDA(cudaMemsetAsync(d.st_q, 0, q_bytes, st));   // rows of later chunks are read (and discarded) as tile padding
    }
    if (pl->n_q == 0) {
        TS_CUDA(launch_gather(pl, k_pool, v_pool, k_pool, v_pool, GatherMode::kCopyRotate, st));
        TS_CUDA(cudaStreamSynchronize(st));
        return TESSERA_OK;
    }
    // Chunks of whole requests flow through three streams: host->device copies of chunk c+1, compute
    // of chunk c and device->host copies of chunk c-1 overlap.  The gather needs no activations and
    // runs while the first chunk is on its way.
    if (int32_t rc = ensure_pipeline(pl)) return rc;
    const size_t q_row = (size_t)pl->cfg.num_q_heads * pl->cfg.head_dim * 2;
    const size_t kv_row = (size_t)pl->cfg.num_kv_heads * pl->cfg.head_dim * 2;
    const size_t lse_row = (size_t)pl->cfg.num_q_heads * sizeof(float);
    const int n_chunks = (int)pl->chunk_row_off.size() - 1;
    auto at = [](const void *p, size_t off) { return static_cast<const char *>(p) + off; };
    auto at_w = [](void *p, size_t off) { return static_cast<char *>(p) + off; };
    TS_CUDA(cudaEventRecord(pl->ev_start, st));
    TS_CUDA(cudaStreamWaitEvent(pl->s_in, pl->ev_start, 0));
    TS_CUDA(cudaStreamWaitEvent(pl->s_out, pl->ev_start, 0));
    for (int c = 0; c < n_chunks; ++c) {
        const size_t r0 = pl->chunk_row_off[c], rows = pl->chunk_row_off[c + 1] - r0;
        if (rows) {
            TS_CUDA(cudaMemcpyAsync(at_w(d.st_q, r0 * q_row), at(q_host, r0 * q_row), rows * q_row, cudaMemcpyHostToDevice, pl->s_in));
            TS_CUDA(cudaMemcpyAsync(at_w(d.st_k, r0 * kv_row), at(k_new_host, r0 * kv_row), rows * kv_row, cudaMemcpyHostToDevice, pl->s_in));
            TS_CUDA(cudaMemcpyAsync(at_w(d.st_v, r0 * kv_row), at(v_new_host, r0 * kv_row), rows * kv_row, cudaMemcpyHostToDevice, pl->s_in));
        }
        TS_CUDA(cudaEventRecord(pl->ev_in[c], pl->s_in));
    }
    TS_CUDA(launch_gather(pl, k_pool, v_pool, k_pool, v_pool, GatherMode::kCopyRotate, st));
    for (int c = 0; c < n_chunks; ++c) {
        const size_t r0 = pl->chunk_row_off[c], rows = pl->chunk_row_off[c + 1] - r0;
        TS_CUDA(cudaStreamWaitEvent(st, pl->ev_in[c], 0));
        if (int32_t rc = attention(pl, k_pool, v_pool, d.st_q, d.st_k, d.st_v, d.st_o, d.st_lse, c, st)) return rc;
        TS_CUDA(cudaEventRecord(pl->ev_comp[c], st));
        TS_CUDA(cudaStreamWaitEvent(pl->s_out, pl->ev_comp[c], 0));
        if (rows) {
            TS_CUDA(cudaMemcpyAsync(at_w(out_host, r0 * q_row), at(d.st_o, r0 * q_row), rows * q_row, cudaMemcpyDeviceToHost, pl->s_out));
            if (lse_host)
                TS_CUDA(cudaMemcpyAsync(at_w(lse_host, r0 * lse_row), at(d.st_lse, r0 * lse_row), rows * lse_row, cudaMemcpyDeviceToHost, pl->s_out));
        }
    }
    TS_CUDA(cudaEventRecord(pl->ev_out, pl->s_out));
    TS_CUDA(cudaStreamWaitEvent(st, pl->ev_out, 0));
    TS_CUDA(cudaStreamSynchronize(st));
    return TESSERA_OK;
}

int32_t tessera_last_error(char *buf, int32_t len) {
    const std::string &e = g_last_error;
    if (buf && len > 0) {
        const size_t n = std::min<size_t>(e.size(), (size_t)len - 1);
        std::memcpy(buf, e.data(), n);
        buf[n] = 0;
    }
    return (int32_t)e.size();
}

int64_t tessera_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// Internal plan representation shared by the host builder and the launch code.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include <cuda_runtime.h>
#include <vector_types.h>

#include "tessera.h"

namespace tessera {

constexpr int kGatherItemTokens = 32;   // token rows per thread block of the gather kernel
constexpr int kAttnTileRows = 128;      // query rows (tokens x grouped heads) per tcgen05 tile
constexpr int kDefaultSMs = 148;         // SM count assumed by a host-only plan (a B200); device plans ask the device
constexpr int kSplitMinSteps = 4;        // never split below this many 128-key steps per part
constexpr int kSplitMaxParts = 8;
constexpr int kHostChunks = 4;          // request chunks of the host-buffer entry point's copy / compute pipeline
constexpr int kLptMaxItemsPerBlock = 16;  // above this many attention items per thread block the plain serpentine walk is kept
constexpr int kAttnCostBands = 16;      // cost bands of the attention work list (longest band first)

// One thread block of the gather / shift kernel: `count` consecutive entries of the copy list that
// belong to one cached unit.  Entry i uses row (row0 + i * row_step) of the cos/sin table.
struct GatherItem {
    int32_t begin, count, row0, row_step;
};

// One query tile of the attention kernel: `n_tok` consecutive recompute rows [q_begin, q_begin+n_tok)
// of request `req`; the tile reads keys [0, kv_len).  Keys below `kv_full` are visible to every row.
struct AttnTile {
    int32_t req, q_begin, n_tok, kv_len, kv_full, pad0, pad1, pad2;
};

// One thread block of the tcgen05 attention kernel: KV head `kvh` of query tiles tile_a and tile_b
// (consecutive tiles of one request; tile_b = -1 when the request has an odd tile left over).
// With split-KV the item covers only the 128-key steps [step_begin, step_end) and is part `part` of
// `n_parts`; a part in which tile_a would have nothing to do names the longer tile alone.
struct AttnWork {
    int32_t tile_a, tile_b, kvh, step_begin, step_end, part, n_parts;
    int32_t cost;      // (tile, step) count of the item: the host's sort key, not read by the kernel
};

// One (query tile, KV head) whose partial results have to be merged after a split-KV launch.
struct CombineItem {
    int32_t tile, kvh, n_parts, pad;
};

struct DeviceTables {
    void *blob = nullptr;          // one allocation holding everything below
    int32_t *g_src = nullptr, *g_dst = nullptr;
    GatherItem *items = nullptr;
    float2 *rope = nullptr;        // [n_rope_rows][D/2] (cos, sin)
    int32_t *fresh_dst = nullptr;  // [n_q] destination slot of each recompute row
    int32_t *retain_dst = nullptr; // [n_q] cache slot of a captured row, -1 otherwise (null: nothing is captured)
    int32_t *q_pos = nullptr;      // [n_q]
    int32_t *q_req = nullptr;      // [n_q]
    int32_t *page_off = nullptr;   // [batch+1]
    int32_t *pages = nullptr;      // block tables
    AttnTile *tiles = nullptr;
    AttnWork *work = nullptr;      // tcgen05 work items, longest first
    AttnWork *work_chunked = nullptr;  // the same items grouped by request chunk (host-buffer entry)
    CombineItem *combine = nullptr;    // (tile, head) pairs to merge, grouped by request chunk
    float *ws_o = nullptr;             // split-KV partials: [slot][128 rows][128] unnormalised O ...
    float2 *ws_ml = nullptr;           // ... and [slot][128] (reference maximum in log2 units, sum)
    int32_t *seq_len = nullptr;    // [batch]
    int32_t *status = nullptr;     // device status word(s)
    double *inv_freq = nullptr;    // [D/2] rotary frequencies
    // staging for the host-buffer entry point (allocated on first use)
    void *q8 = nullptr;            // 8-bit copy of q for the 8-bit-key attention entry (allocated on first use)
    void *st_q = nullptr, *st_k = nullptr, *st_v = nullptr, *st_o = nullptr;
    float *st_lse = nullptr;
};

}  // namespace tessera

struct tessera_plan {
    tessera_model_cfg cfg{};
    std::vector<double> inv_freq;          // [D/2], always filled
    float sm_scale = 0.f;
    int32_t num_pool_pages = 0;
    int32_t num_source_pages = 0;          // > 0: cached units are read from a separate source pool
    int32_t batch = 0;
    bool host_only = false;
    int device = -1;
    int num_sms = tessera::kDefaultSMs;    // multiprocessors of the plan's device: grid of the persistent attention
                                           // kernel, target block count of split-KV and of the small-batch gather

    std::vector<int32_t> seq_len, tok_off, page_off, pages, src_slot;
    std::vector<int32_t> recompute_off, recompute_pos, q_req, fresh_dst;
    std::vector<int32_t> retain_dst;       // [n_q] or empty: cache slot of every captured recompute row
    int32_t retain_pool_pages = 0;         // > 0: captured units go to a separate cache pool of this many pages
    int64_t retained_tokens = 0;
    std::vector<int32_t> g_src, g_dst;
    std::vector<tessera::GatherItem> items;
    std::vector<int32_t> rope_delta;       // sorted distinct shift amounts
    std::vector<float> rope_table;         // [rows][D/2][2]
    std::vector<tessera::AttnTile> tiles;
    std::vector<tessera::AttnWork> work;
    // The host-buffer entry point pipelines copies against compute over chunks of whole requests.
    std::vector<tessera::AttnWork> work_chunked;   // items of chunk c: [chunk_work_off[c], chunk_work_off[c+1])
    std::vector<int32_t> chunk_work_off, chunk_row_off;   // [n_chunks + 1]; rows = recompute rows
    std::vector<int32_t> chunk_item_off;                  // [n_chunks + 1]; gather items of the chunk's requests
    std::vector<tessera::CombineItem> combine;     // grouped by chunk: [chunk_combine_off[c], chunk_combine_off[c+1])
    std::vector<int32_t> chunk_combine_off;
    int32_t n_work_items = 0;                      // real items of `work` (the list may hold holes)
    int32_t max_parts = 1;                         // split-KV parts per item (1 = no split)
    int32_t attn_kernel = 0;
    int32_t tile_tokens = 0;

    int64_t total_tokens = 0, n_q = 0, cached_tokens = 0, qk_pairs = 0, mma_pairs = 0;

    std::vector<char> host_blob;           // staging image of the device tables
    tessera::DeviceTables dev;
    // streams / events of the host-buffer entry point (created on first use)
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr;
    std::vector<cudaEvent_t> ev_in, ev_comp;
};

namespace tessera {
// Builds and validates all host tables.  Returns a status; on failure `err` holds the reason.
// `num_sms`: multiprocessor count the work lists are sized for.
int32_t build_plan_host(const tessera_model_cfg *cfg, const tessera_compose_desc *desc,
                        int32_t num_pool_pages, int num_sms, tessera_plan *plan, std::string *err);
}  // namespace tessera

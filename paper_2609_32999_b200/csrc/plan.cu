// Host-side placement: validation of a batch descriptor and construction of every table the
// kernels read (Sec. 5.3 "Placement before preparation"; storage blocks of Sec. 5.1).
// Pure host code: it makes no CUDA call, so it also runs where no GPU exists.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <numeric>
#include <tuple>

#include <vector_types.h>

#include "plan.h"

namespace tessera {

namespace {

std::string fmt(const char *f, long a = 0, long b = 0, long c = 0) {
    char buf[256];
    snprintf(buf, sizeof buf, f, a, b, c);
    return buf;
}

bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

}  // namespace

int32_t build_plan_host(const tessera_model_cfg *cfg, const tessera_compose_desc *d,
                        int32_t num_pool_pages, int num_sms, tessera_plan *pl, std::string *err) {
    auto fail = [&](int32_t code, const std::string &msg) { *err = msg; return code; };
    if (!cfg || !d || !pl) return fail(TESSERA_INVALID_ARG, "null cfg / desc / plan");
    if (num_sms <= 0) return fail(TESSERA_INVALID_ARG, "multiprocessor count must be positive");
    pl->num_sms = num_sms;
    if (d->batch < 0 || num_pool_pages < 0 || d->n_free < 0)
        return fail(TESSERA_INVALID_ARG, "negative batch, pool size or free-list length");
    if (d->batch > 0 && (!d->seq_len || !d->unit_off || !d->recompute_off))
        return fail(TESSERA_INVALID_ARG, "null seq_len / unit_off / recompute_off");

    // ---- shapes the kernels cover
    const int Hq = cfg->num_q_heads, Hkv = cfg->num_kv_heads, D = cfg->head_dim, B = cfg->page_size;
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0)
        return fail(TESSERA_UNSUPPORTED_SHAPE, fmt("num_q_heads %ld must be a positive multiple of num_kv_heads %ld", Hq, Hkv));
    if (Hq / Hkv > 16) return fail(TESSERA_UNSUPPORTED_SHAPE, "group size H_q/H_kv above 16");
    if (D != 64 && D != 128) return fail(TESSERA_UNSUPPORTED_SHAPE, fmt("head_dim %ld: only 64 and 128", D));
    if (B <= 0 || B % 8 != 0 || B > 128 || !is_pow2(B))
        return fail(TESSERA_UNSUPPORTED_SHAPE, fmt("page_size %ld: a power of two in 8..128", B));
    if (cfg->rope_pairing != 0 && cfg->rope_pairing != 1)
        return fail(TESSERA_UNSUPPORTED_SHAPE, "rope_pairing: 0 (half-split pairs) or 1 (interleaved pairs)");
    if (!cfg->inv_freq && !(cfg->rope_theta > 0.0)) return fail(TESSERA_INVALID_ARG, "rope_theta must be positive");
    if ((int64_t)num_pool_pages * B > (int64_t)INT32_MAX)
        return fail(TESSERA_UNSUPPORTED_SHAPE, "pool has more than 2^31 slots");

    pl->cfg = *cfg;
    pl->inv_freq.resize(D / 2);
    for (int m = 0; m < D / 2; ++m)
        pl->inv_freq[m] = cfg->inv_freq ? cfg->inv_freq[m] : std::pow(cfg->rope_theta, -2.0 * m / D);
    pl->cfg.inv_freq = nullptr;
    pl->sm_scale = cfg->sm_scale != 0.f ? cfg->sm_scale : (float)(1.0 / std::sqrt((double)D));
    pl->num_pool_pages = num_pool_pages;
    if (d->num_source_pages < 0) return fail(TESSERA_INVALID_ARG, "negative num_source_pages");
    if ((int64_t)d->num_source_pages * B > (int64_t)INT32_MAX) return fail(TESSERA_UNSUPPORTED_SHAPE, "source pool has more than 2^31 slots");
    pl->num_source_pages = d->num_source_pages;
    pl->batch = d->batch;

    const int batch = d->batch;
    // ---- CSR sanity
    if (batch > 0) {
        if (d->unit_off[0] != 0 || d->recompute_off[0] != 0) return fail(TESSERA_INVALID_ARG, "CSR offsets must start at 0");
        for (int r = 0; r < batch; ++r) {
            if (d->seq_len[r] < 0) return fail(TESSERA_INVALID_ARG, fmt("request %ld: negative seq_len", r));
            if (d->unit_off[r + 1] < d->unit_off[r] || d->recompute_off[r + 1] < d->recompute_off[r])
                return fail(TESSERA_INVALID_ARG, fmt("request %ld: CSR offsets decrease", r));
        }
    }
    const int n_units = batch ? d->unit_off[batch] : 0;
    const int n_q = batch ? d->recompute_off[batch] : 0;
    if (n_units > 0 && (!d->unit_len || !d->unit_cached_pos || !d->unit_cached_stride || !d->unit_target_pos || !d->unit_page_off))
        return fail(TESSERA_INVALID_ARG, "null unit array");
    if (n_q > 0 && !d->recompute_pos) return fail(TESSERA_INVALID_ARG, "null recompute_pos");
    if (n_units > 0) {
        if (d->unit_page_off[0] != 0) return fail(TESSERA_INVALID_ARG, "unit_page_off must start at 0");
        for (int u = 0; u < n_units; ++u) {
            if (d->unit_len[u] < 0) return fail(TESSERA_INVALID_ARG, fmt("unit %ld: negative length", u));
            int np = d->unit_page_off[u + 1] - d->unit_page_off[u];
            if (np < 0) return fail(TESSERA_INVALID_ARG, fmt("unit %ld: unit_page_off decreases", u));
            const int off = d->unit_src_offset ? d->unit_src_offset[u] : 0;
            if (off < 0 || off >= B) return fail(TESSERA_INVALID_ARG, fmt("unit %ld: source offset %ld outside [0, page_size)", u, off));
            if (np != 0 && np != (off + d->unit_len[u] + B - 1) / B)
                return fail(TESSERA_INVALID_ARG, fmt("unit %ld: %ld source pages for %ld tokens", u, np, d->unit_len[u]));
            if (d->unit_target_stride && d->unit_target_stride[u] != 0 && d->unit_target_stride[u] != 1)
                return fail(TESSERA_INVALID_ARG, fmt("unit %ld: target stride must be 0 or 1", u));
            if (np != 0 && d->unit_cached_stride[u] != 0 && d->unit_cached_stride[u] != 1)
                return fail(TESSERA_INVALID_ARG, fmt("unit %ld: cached stride must be 0 or 1", u));
        }
        if (d->unit_page_off[n_units] > 0 && !d->unit_pages) return fail(TESSERA_INVALID_ARG, "null unit_pages");
        if (d->unit_retain_page_off) {
            if (d->unit_retain_page_off[0] != 0) return fail(TESSERA_INVALID_ARG, "unit_retain_page_off must start at 0");
            for (int u = 0; u < n_units; ++u) {
                const int np = d->unit_retain_page_off[u + 1] - d->unit_retain_page_off[u];
                if (np < 0) return fail(TESSERA_INVALID_ARG, fmt("unit %ld: unit_retain_page_off decreases", u));
                if (np != 0 && np != (d->unit_len[u] + B - 1) / B)
                    return fail(TESSERA_INVALID_ARG, fmt("unit %ld: %ld cache pages for %ld tokens", u, np, d->unit_len[u]));
            }
            if (d->unit_retain_page_off[n_units] > 0 && !d->unit_retain_pages) return fail(TESSERA_INVALID_ARG, "null unit_retain_pages");
        }
    }
    if (d->retain_pool_pages < 0) return fail(TESSERA_INVALID_ARG, "negative retain_pool_pages");
    if ((int64_t)d->retain_pool_pages * B > (int64_t)INT32_MAX) return fail(TESSERA_UNSUPPORTED_SHAPE, "cache pool has more than 2^31 slots");
    pl->retain_pool_pages = d->retain_pool_pages;

    // ---- block tables: request r takes the next ceil(T_r / B) free pages
    pl->seq_len.assign(d->seq_len, d->seq_len + batch);
    pl->tok_off.assign(batch + 1, 0);
    pl->page_off.assign(batch + 1, 0);
    int64_t total = 0, need_pages = 0;
    for (int r = 0; r < batch; ++r) {
        total += d->seq_len[r];
        need_pages += (d->seq_len[r] + B - 1) / B;
        if (total > INT32_MAX) return fail(TESSERA_UNSUPPORTED_SHAPE, "batch has more than 2^31 tokens");
        pl->tok_off[r + 1] = (int32_t)total;
        pl->page_off[r + 1] = (int32_t)need_pages;
    }
    if (need_pages > d->n_free)
        return fail(TESSERA_OUT_OF_PAGES, fmt("batch needs %ld destination pages, free list has %ld", need_pages, d->n_free));
    if (need_pages > 0 && !d->free_pages) return fail(TESSERA_INVALID_ARG, "null free_pages");
    pl->pages.assign(d->free_pages, d->free_pages + need_pages);

    // page ids: range, destinations distinct, destinations disjoint from sources
    std::vector<uint8_t> page_use(num_pool_pages, 0);   // 1 = source, 2 = destination
    const int n_src_pages = n_units ? d->unit_page_off[n_units] : 0;
    for (int k = 0; k < n_src_pages; ++k) {
        int pg = d->unit_pages[k];
        const int src_limit = d->num_source_pages > 0 ? d->num_source_pages : num_pool_pages;
        if (pg < 0 || pg >= src_limit) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("source page %ld outside pool of %ld pages", pg, src_limit));
        if (d->num_source_pages == 0) page_use[pg] = 1;    // a separate source pool cannot alias destinations
    }
    for (int64_t k = 0; k < need_pages; ++k) {
        int pg = pl->pages[k];
        if (pg < 0 || pg >= num_pool_pages) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("free page %ld outside pool of %ld pages", pg, num_pool_pages));
        if (page_use[pg] == 1) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("free page %ld is also a source page of this batch", pg));
        if (page_use[pg] == 2) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("free page %ld listed twice", pg));
        page_use[pg] = 2;
    }

    // cache pages of captured units: in range, distinct, and - when they live in the destination pool -
    // neither sources nor destinations of this batch
    const int n_retain_pages = (n_units && d->unit_retain_page_off) ? d->unit_retain_page_off[n_units] : 0;
    if (n_retain_pages > 0) {
        const int limit = d->retain_pool_pages > 0 ? d->retain_pool_pages : num_pool_pages;
        std::vector<uint8_t> seen(limit, 0);
        for (int k = 0; k < n_retain_pages; ++k) {
            const int pg = d->unit_retain_pages[k];
            if (pg < 0 || pg >= limit) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("cache page %ld outside pool of %ld pages", pg, limit));
            if (seen[pg]) return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("cache page %ld listed twice", pg));
            seen[pg] = 1;
            if (d->retain_pool_pages == 0 && page_use[pg] != 0)
                return fail(TESSERA_PAGE_OUT_OF_RANGE, fmt("cache page %ld is also a source or destination page of this batch", pg));
        }
    }

    // ---- per-position sources, recompute rows, coverage
    pl->src_slot.assign((size_t)total, -1);
    pl->recompute_off.assign(d->recompute_off, d->recompute_off + batch + 1);
    pl->recompute_pos.assign(d->recompute_pos, d->recompute_pos + n_q);
    pl->q_req.resize(n_q);
    pl->fresh_dst.resize(n_q);
    pl->g_src.clear(); pl->g_dst.clear(); pl->items.clear();
    std::vector<int32_t> unit_of((size_t)total, -1);
    std::vector<uint8_t> fresh((size_t)total, 0);
    std::vector<int32_t> fresh_row((size_t)total, -1);     // recompute row index of a position
    pl->retain_dst.assign(n_retain_pages > 0 ? n_q : 0, -1);
    pl->retained_tokens = 0;
    std::vector<int64_t> deltas;     // shift amounts needed, with repeats
    pl->qk_pairs = 0;
    for (int r = 0; r < batch; ++r) {
        const int T = d->seq_len[r];
        const int64_t base = pl->tok_off[r];
        for (int u = d->unit_off[r]; u < d->unit_off[r + 1]; ++u) {
            const int len = d->unit_len[u], tp = d->unit_target_pos[u];
            if (tp < 0 || (int64_t)tp + len > T)
                return fail(TESSERA_UNIT_OVERLAP, fmt("unit %ld leaves its request's positions [0, %ld)", u, T));
            const bool cached = d->unit_page_off[u + 1] > d->unit_page_off[u];
            for (int i = 0; i < len; ++i) {
                if (unit_of[base + tp + i] != -1)
                    return fail(TESSERA_UNIT_OVERLAP, fmt("units %ld and %ld both claim position %ld", unit_of[base + tp + i], u, tp + i));
                unit_of[base + tp + i] = u;
                if (cached) {
                    const int si = i + (d->unit_src_offset ? d->unit_src_offset[u] : 0);
                    pl->src_slot[base + tp + i] = d->unit_pages[d->unit_page_off[u] + si / B] * B + si % B;
                }
            }
        }
        for (int j = d->recompute_off[r]; j < d->recompute_off[r + 1]; ++j) {
            const int p = d->recompute_pos[j];
            if (p < 0 || p >= T) return fail(TESSERA_INVALID_ARG, fmt("request %ld: recompute position %ld outside [0, %ld)", r, p, T));
            if (j > d->recompute_off[r] && d->recompute_pos[j - 1] >= p)
                return fail(TESSERA_UNSORTED_POSITIONS, fmt("request %ld: recompute positions not strictly ascending at index %ld", r, j));
            fresh[base + p] = 1;
            fresh_row[base + p] = j;
            pl->q_req[j] = r;
            pl->fresh_dst[j] = pl->pages[pl->page_off[r] + p / B] * B + p % B;
            pl->qk_pairs += (int64_t)p + 1;
        }
        for (int p = 0; p < T; ++p)
            if (pl->src_slot[base + p] < 0 && !fresh[base + p])
                return fail(TESSERA_UNCOVERED_POSITION, fmt("request %ld: position %ld has no cached unit and is not recomputed", r, p));
        // captured units: every token is a recompute row; row j also goes to the unit's cache slot
        if (n_retain_pages > 0)
            for (int u = d->unit_off[r]; u < d->unit_off[r + 1]; ++u) {
                const int first = d->unit_retain_page_off[u], np = d->unit_retain_page_off[u + 1] - first;
                if (np == 0) continue;
                for (int i = 0; i < d->unit_len[u]; ++i) {
                    const int j = fresh_row[base + d->unit_target_pos[u] + i];
                    if (j < 0)
                        return fail(TESSERA_INVALID_ARG, fmt("unit %ld is to be captured but its token %ld is not recomputed", u, i));
                    pl->retain_dst[j] = d->unit_retain_pages[first + i / B] * B + i % B;
                }
                pl->retained_tokens += d->unit_len[u];
            }
    }

    // ---- copy list + shift table.  One item = up to kGatherItemTokens rows of one unit.
    for (int r = 0; r < batch; ++r)
        for (int u = d->unit_off[r]; u < d->unit_off[r + 1]; ++u) {
            if (d->unit_page_off[u + 1] <= d->unit_page_off[u]) continue;
            // token i is shifted by (target_pos + ts * i) - (cached_pos + cs * i)
            const int64_t d0 = (int64_t)d->unit_target_pos[u] - d->unit_cached_pos[u];
            const int step = (d->unit_target_stride ? d->unit_target_stride[u] : 1) - d->unit_cached_stride[u];
            if (step == 0) deltas.push_back(d0);
            else for (int i = 0; i < d->unit_len[u]; ++i) deltas.push_back(d0 + (int64_t)step * i);
        }
    std::sort(deltas.begin(), deltas.end());
    deltas.erase(std::unique(deltas.begin(), deltas.end()), deltas.end());
    for (int64_t x : deltas)
        if (x > INT32_MAX || x < INT32_MIN) return fail(TESSERA_INVALID_ARG, "shift amount overflows int32");
    pl->rope_delta.assign(deltas.begin(), deltas.end());
    pl->rope_table.resize(deltas.size() * (size_t)D);     // [row][D/2][cos, sin]
    for (size_t row = 0; row < deltas.size(); ++row)
        for (int m = 0; m < D / 2; ++m) {
            // angle, cosine and sine in fp64; a single rounding to fp32 each
            const double ang = (double)deltas[row] * pl->inv_freq[m];
            pl->rope_table[(row * (D / 2) + m) * 2 + 0] = (float)std::cos(ang);
            pl->rope_table[(row * (D / 2) + m) * 2 + 1] = (float)std::sin(ang);
        }
    auto row_of = [&](int64_t delta) {
        return (int32_t)(std::lower_bound(deltas.begin(), deltas.end(), delta) - deltas.begin());
    };
    // Rows per gather block: 32, fewer when the batch is so small that the grid would not fill the GPU.
    int item_tokens = kGatherItemTokens;
    {
        int64_t cached = 0;
        for (int u = 0; u < n_units; ++u)
            if (d->unit_page_off[u + 1] > d->unit_page_off[u]) cached += d->unit_len[u];
        while (item_tokens > 8 && cached / item_tokens < 4 * num_sms) item_tokens /= 2;
    }
    pl->cached_tokens = 0;
    std::vector<int32_t> req_item_off(batch + 1, 0);       // gather items are emitted request by request
    for (int r = 0; r < batch; ++r) {
        req_item_off[r] = (int32_t)pl->items.size();
        for (int u = d->unit_off[r]; u < d->unit_off[r + 1]; ++u) {
            if (d->unit_page_off[u + 1] <= d->unit_page_off[u]) continue;
            const int len = d->unit_len[u], tp = d->unit_target_pos[u];
            const int64_t d0 = (int64_t)tp - d->unit_cached_pos[u];
            const int step = (d->unit_target_stride ? d->unit_target_stride[u] : 1) - d->unit_cached_stride[u];
            const int32_t row0 = row_of(d0);       // step +-1: consecutive integers are consecutive rows
            for (int i0 = 0; i0 < len; i0 += item_tokens) {
                const int cnt = std::min(item_tokens, len - i0);
                pl->items.push_back({(int32_t)pl->g_src.size(), cnt, row0 + i0 * step, step});
                for (int i = i0; i < i0 + cnt; ++i) {
                    const int p = tp + i;
                    pl->g_src.push_back(pl->src_slot[pl->tok_off[r] + p]);
                    pl->g_dst.push_back(pl->pages[pl->page_off[r] + p / B] * B + p % B);
                }
            }
            pl->cached_tokens += len;
        }
    }
    req_item_off[batch] = (int32_t)pl->items.size();

    // ---- attention work list: tiles of consecutive recompute rows of one request
    const int g = Hq / Hkv;
    pl->tile_tokens = kAttnTileRows / g;
    pl->attn_kernel = 1;       // the tcgen05 kernel covers every accepted shape (page size 8..128, head_dim 64 / 128, g <= 16)
    pl->tiles.clear();
    for (int r = 0; r < batch; ++r)
        for (int j0 = d->recompute_off[r]; j0 < d->recompute_off[r + 1]; j0 += pl->tile_tokens) {
            const int n = std::min(pl->tile_tokens, d->recompute_off[r + 1] - j0);
            AttnTile t{};
            t.req = r; t.q_begin = j0; t.n_tok = n;
            t.kv_len = d->recompute_pos[j0 + n - 1] + 1;
            t.kv_full = d->recompute_pos[j0] + 1;
            pl->tiles.push_back(t);
        }
    // tcgen05 work items: consecutive tiles of a request share one thread block (and every K/V page
    // they read); longest first, so that the tail of the grid is made of short items.
    pl->work.clear();
    {
        const int page = 128;        // keys per step of the tensor-core kernel
        std::vector<std::pair<int32_t, int32_t>> pairs;
        size_t first = 0;
        while (first < pl->tiles.size()) {
            size_t last = first;
            while (last < pl->tiles.size() && pl->tiles[last].req == pl->tiles[first].req) ++last;
            for (size_t k = first; k < last; k += 2) {
                const int32_t a = (int32_t)k, b2 = (k + 1 < last) ? (int32_t)(k + 1) : -1;
                pairs.push_back({a, b2});
            }
            first = last;
        }
        auto steps_of = [&](int32_t tile) { return (pl->tiles[tile].kv_len + page - 1) / page; };
        // Split-KV: a batch with fewer items than SMs (a single request, typically) splits each item's
        // key range into parts that run as separate thread blocks and are merged afterwards.
        pl->max_parts = 1;
        if (!pairs.empty() && (int)pairs.size() * Hkv < num_sms) {
            int longest = 1;
            for (auto &pr : pairs) longest = std::max(longest, steps_of(pr.second >= 0 ? pr.second : pr.first));
            const int want = num_sms / ((int)pairs.size() * Hkv);     // stay within one wave of blocks
            pl->max_parts = std::max(1, std::min({want, kSplitMaxParts, longest / kSplitMinSteps}));
        }
        pl->combine.clear();
        for (auto &pr : pairs) {
            const int32_t a = pr.first, b2 = pr.second;
            const int sa = steps_of(a), sl = steps_of(b2 >= 0 ? b2 : a);       // sa <= sl: positions ascend
            const int parts = std::max(1, std::min(pl->max_parts, sl / kSplitMinSteps));
            const int chunk = (sl + parts - 1) / parts;
            for (int h = 0; h < Hkv; ++h) {
                int parts_a = 0, parts_b = 0;
                for (int p2 = 0; p2 < parts; ++p2) {
                    const int sb = p2 * chunk, se = std::min(sl, sb + chunk);
                    if (sb >= se) break;
                    if (b2 < 0 || sb < sa) {
                        pl->work.push_back({a, b2, h, sb, se, p2, parts, 0});
                        ++parts_a;
                        if (b2 >= 0) ++parts_b;
                    } else {
                        pl->work.push_back({b2, -1, h, sb, se, p2, parts, 0});   // tile a is already finished
                        ++parts_b;
                    }
                }
                if (parts > 1) {
                    pl->combine.push_back({a, h, parts_a, 0});
                    if (b2 >= 0) pl->combine.push_back({b2, h, parts_b, 0});
                }
            }
        }
        // cost of an item = its (tile, 128-key step) count, kept in the item for the sorts
        for (AttnWork &w : pl->work) {
            int c = std::min(w.step_end, steps_of(w.tile_a)) - w.step_begin;
            if (w.tile_b >= 0) c += std::min(w.step_end, steps_of(w.tile_b)) - w.step_begin;
            w.cost = c;
        }
        pl->mma_pairs = 0;
        for (const AttnWork &w : pl->work) pl->mma_pairs += (int64_t)w.cost * kAttnTileRows * page;
        auto cost = [](const AttnWork &w) { return w.cost; };
        auto sort_items = [&](std::vector<AttnWork>::iterator first_it, std::vector<AttnWork>::iterator last_it) {
            int max_cost = 1;
            for (auto it = first_it; it != last_it; ++it) max_cost = std::max(max_cost, cost(*it));
            const int band = std::max(1, max_cost / kAttnCostBands);
            const AttnTile *tl = pl->tiles.data();
            std::stable_sort(first_it, last_it, [=](const AttnWork &x, const AttnWork &y) {
                const int bx = x.cost / band, by = y.cost / band;
                if (bx != by) return bx > by;
                const int rx = tl[x.tile_a].req, ry = tl[y.tile_a].req;
                if (rx != ry) return rx < ry;
                if (x.kvh != y.kvh) return x.kvh < y.kvh;
                return x.cost > y.cost;
            });
        };
        // chunks of whole requests with about equal attention cost, for the host-buffer pipeline
        std::vector<int64_t> req_cost(batch, 0);
        for (const AttnWork &w : pl->work) req_cost[pl->tiles[w.tile_a].req] += cost(w);
        int64_t total_cost = 0;
        for (int64_t c : req_cost) total_cost += c;
        const int n_chunks = std::max(1, std::min(batch, kHostChunks));
        std::vector<int> chunk_of(batch, 0);
        pl->chunk_row_off.assign(1, 0);
        {
            int64_t acc = 0;
            int c = 0;
            for (int r = 0; r < batch; ++r) {
                chunk_of[r] = c;
                acc += req_cost[r];
                const bool last_req = r + 1 == batch;
                // close the chunk when its share of the cost is reached, keeping one request per remaining chunk
                if (!last_req && c + 1 < n_chunks && (acc * n_chunks >= total_cost * (c + 1) || batch - (r + 1) <= n_chunks - (c + 1))) {
                    pl->chunk_row_off.push_back(d->recompute_off[r + 1]);
                    ++c;
                }
            }
            pl->chunk_row_off.push_back(n_q);
        }
        const int used_chunks = (int)pl->chunk_row_off.size() - 1;
        pl->chunk_item_off.assign(used_chunks + 1, (int32_t)pl->items.size());
        pl->chunk_item_off[0] = 0;
        for (int r = 1; r < batch; ++r)
            if (chunk_of[r] != chunk_of[r - 1]) pl->chunk_item_off[chunk_of[r]] = req_item_off[r];
        pl->work_chunked = pl->work;
        std::stable_sort(pl->work_chunked.begin(), pl->work_chunked.end(), [&](const AttnWork &x, const AttnWork &y) {
            return chunk_of[pl->tiles[x.tile_a].req] < chunk_of[pl->tiles[y.tile_a].req];
        });
        pl->chunk_work_off.assign(used_chunks + 1, 0);
        for (const AttnWork &w : pl->work_chunked) ++pl->chunk_work_off[chunk_of[pl->tiles[w.tile_a].req] + 1];
        for (int c = 0; c < used_chunks; ++c) pl->chunk_work_off[c + 1] += pl->chunk_work_off[c];
        for (int c = 0; c < used_chunks; ++c)
            sort_items(pl->work_chunked.begin() + pl->chunk_work_off[c], pl->work_chunked.begin() + pl->chunk_work_off[c + 1]);
        std::stable_sort(pl->combine.begin(), pl->combine.end(), [&](const CombineItem &x, const CombineItem &y) {
            return chunk_of[pl->tiles[x.tile].req] < chunk_of[pl->tiles[y.tile].req];
        });
        pl->chunk_combine_off.assign(used_chunks + 1, 0);
        for (const CombineItem &ci : pl->combine) ++pl->chunk_combine_off[chunk_of[pl->tiles[ci.tile].req] + 1];
        for (int c = 0; c < used_chunks; ++c) pl->chunk_combine_off[c + 1] += pl->chunk_combine_off[c];
        // Longest first in coarse cost bands; inside a band, items of one (request, KV head) stay
        // together, so thread blocks that run at the same time stream the same K/V pages and find
        // them in L2.
        sort_items(pl->work.begin(), pl->work.end());
        // With few items per thread block the spread of the blocks' finishing times is what costs (config 3:
        // 7 items per block, slowest block 8-10 % above the mean with the plain walk): the items are then
        // assigned greedily to the least-loaded block by modelled cycles (item fetch 700, epilogue + first
        // step 3 150 per tile, 3 180 per step of both tiles, 1 650 per step of one - measured with clock64)
        // and laid out so that the kernel's serpentine walk (round k, block b -> index k G + (k odd ? G - 1
        // - b : b)) hands every block its own list; holes are marked tile_a = -1.  Measured: config 3 +6 %,
        // config 4 +-0.  With many items per block (config 5: 131) the plain walk is already even and keeps
        // neighbours in the list - the same request and head - on the GPU at the same time, which the
        // greedy assignment does not: it measured 3 % slower there, so it is not used.
        auto lpt_layout = [&](std::vector<AttnWork> &list) {
            const int G = num_sms;
            if ((int)list.size() <= G || (int)list.size() > kLptMaxItemsPerBlock * G) return;
            auto cycles = [&](const AttnWork &w) -> int64_t {
                const int sa = std::min(w.step_end, steps_of(w.tile_a)) - w.step_begin;
                const int sb = w.tile_b >= 0 ? std::min(w.step_end, steps_of(w.tile_b)) - w.step_begin : 0;
                const int both = std::min(sa, sb), single = std::max(sa, sb) - both, nt = w.tile_b >= 0 ? 2 : 1;
                return 700 + (int64_t)nt * 3150 + (int64_t)both * 3180 + (int64_t)single * 1650;
            };
            std::vector<int> order(list.size());
            std::iota(order.begin(), order.end(), 0);
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cycles(list[a]) > cycles(list[b]); });
            std::vector<int64_t> load(G, 0);
            std::vector<std::vector<int>> mine(G);
            for (int i : order) {
                const int b = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                load[b] += cycles(list[i]);
                mine[b].push_back(i);
            }
            size_t rounds = 0;
            for (auto &m : mine) rounds = std::max(rounds, m.size());
            AttnWork hole{};
            hole.tile_a = -1; hole.tile_b = -1;
            std::vector<AttnWork> out(rounds * G, hole);
            for (int b = 0; b < G; ++b)
                for (size_t k = 0; k < mine[b].size(); ++k)
                    out[k * G + ((k & 1) ? G - 1 - b : b)] = list[mine[b][k]];
            list.swap(out);
        };
        pl->n_work_items = (int32_t)pl->work.size();
        lpt_layout(pl->work);
    }

    pl->total_tokens = total;
    pl->n_q = n_q;
    return TESSERA_OK;
}

}  // namespace tessera

/*
 * tessera.h - C ABI of the composed-prefill hot path on one B200 (sm_100a).
 *
 * The path is the per-layer GPU work of a prompt whose context units already
 * have cached KV (Sec. 5.3 of the paper, "Coordinated Request Execution"):
 *
 *   placement  -> tessera_plan_create          (host, once per batch)
 *   gather     -> tessera_kv_compose           (device, per layer)
 *   RoPE shift -> tessera_rope_shift           (device, per layer; normally fused into compose)
 *   attention  -> tessera_partial_prefill_attn (device, per layer)
 *
 * Conventions
 *   - Every function returns a tessera_status (0 = OK, negative = error).  A failed call
 *     launches nothing and leaves the pool untouched; tessera_last_error() gives the text
 *     of the calling thread's last failure.  Nothing throws, aborts or traps.
 *   - "host" / "device" beside a pointer says where the memory lives.  The caller owns every
 *     buffer it passes; host arrays may be freed as soon as the call returns.  The library owns
 *     only the opaque plan (its host tables, device tables and staging buffers).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Device
 *     work is enqueued on it and the call returns without waiting, unless stated otherwise.
 *   - One plan serves every layer of its batch, one call after the other.  Calls on the SAME plan
 *     must not overlap on the GPU (two streams without ordering): a plan owns one status word, one
 *     split-KV workspace and one set of staging buffers.  Different plans are independent.
 *   - All K/V/Q/O tensors are bf16 (2 bytes, raw bits), indices are int32.
 *   - KV pool layout (one K pool and one V pool per layer, same page ids in every layer):
 *         [num_pool_pages][page_size][num_kv_heads][head_dim]   bf16, contiguous,
 *     i.e. a page is a storage block of page_size tokens (Sec. 5.1) and one token's row over all
 *     KV heads is contiguous.  Slot id = page * page_size + offset.  Base pointers must be
 *     16-byte aligned.
 */
#ifndef TESSERA_H_
#define TESSERA_H_

#include <stdint.h>

#if defined(__GNUC__)
#define TESSERA_API __attribute__((visibility("default")))
#else
#define TESSERA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum tessera_status {
    TESSERA_OK = 0,
    TESSERA_INVALID_ARG = -1,          /* null pointer, negative size, malformed CSR arrays        */
    TESSERA_UNSORTED_POSITIONS = -2,   /* recompute_pos not strictly ascending inside a request     */
    TESSERA_UNIT_OVERLAP = -3,         /* two cached units claim one position, or a unit leaves [0,T) */
    TESSERA_UNCOVERED_POSITION = -4,   /* a position has neither a cached unit nor a recompute entry */
    TESSERA_PAGE_OUT_OF_RANGE = -5,    /* page id outside [0, num_pool_pages), or dest == source    */
    TESSERA_OUT_OF_PAGES = -6,         /* free_pages too short for the batch                        */
    TESSERA_UNSUPPORTED_SHAPE = -7,    /* head_dim / page_size / head counts outside the kernels' range */
    TESSERA_CUDA_ERROR = -8,           /* a CUDA runtime or driver call failed; see tessera_last_error */
    TESSERA_DEVICE_TIMEOUT = -9        /* a bounded wait inside a kernel gave up (tessera_plan_status) */
} tessera_status;

/* Model-side constants of one attention layer. */
typedef struct tessera_model_cfg {
    int32_t num_q_heads;        /* H_q                                                        */
    int32_t num_kv_heads;       /* H_kv, divides H_q; query head h reads KV head h / (H_q/H_kv) */
    int32_t head_dim;           /* D: 64 or 128                                               */
    int32_t page_size;          /* tokens per storage block, a multiple of 8, at most 128      */
    double  rope_theta;         /* pair m turns by theta^(-2m/D) per position                  */
    const double *inv_freq;     /* host, optional [D/2]: overrides rope_theta when non-null     */
    int32_t rope_pairing;       /* 0 = pair (m, m + D/2) (Llama / Qwen); 1 = pair (2m, 2m + 1) (interleaved) */
    float   sm_scale;           /* softmax scale; 0 means 1/sqrt(D)                             */
} tessera_model_cfg;

/*
 * One batch of composed prompts: the outcome of the paper's per-unit plan (Sec. 5.1) as the
 * generation node sees it - an ORDERED list of context units per request, where each one was
 * cached, where it lands, and which positions are recomputed (Sec. 5.3).  All arrays on the host.
 */
typedef struct tessera_compose_desc {
    int32_t batch;
    const int32_t *seq_len;             /* [batch] composed length T_r                              */
    const int32_t *unit_off;            /* [batch+1] CSR into the unit arrays                        */
    const int32_t *unit_len;            /* [n_units] tokens                                          */
    const int32_t *unit_cached_pos;     /* [n_units] position of the unit's token 0 when cached       */
    const int32_t *unit_cached_stride;  /* [n_units] 1: key i was cached rotated at cached_pos + i;
                                                     0: keys were cached before rotation             */
    const int32_t *unit_target_pos;     /* [n_units] position of token 0 in this prompt               */
    const int32_t *unit_page_off;       /* [n_units+1] CSR into unit_pages; an empty range marks an
                                           uncached unit, all of whose tokens must be recomputed      */
    const int32_t *unit_pages;          /* source page ids, ceil(len/page_size) per cached unit       */
    const int32_t *recompute_off;       /* [batch+1] CSR into recompute_pos                           */
    const int32_t *recompute_pos;       /* query rows: positions, strictly ascending per request      */
    const int32_t *free_pages;          /* destination page ids, consumed in order, request by request */
    int32_t n_free;
    /* Optional (NULL = default), used to RETAIN freshly computed units in reusable form (Sec. 5.3: the
       miss prefill keeps an unrotated copy for the cache; Sec. 6.1: pre-RoPE keys are captured): */
    const int32_t *unit_src_offset;     /* [n_units] offset (0 .. page_size-1) of the unit's token 0 inside
                                           its first source page; default 0.  Lets a unit be read out of the
                                           middle of another request's pages; it then spans
                                           ceil((offset + len) / page_size) source pages                 */
    int32_t num_source_pages;           /* 0 (default): unit_pages index the destination pool.  > 0: the
                                           cached units live in a SEPARATE source pool of this many pages
                                           (same page layout) - the node's pinned host-memory unit cache of
                                           Sec. 4 / 5.3 "local hit", or any other device-visible buffer;
                                           such a plan is executed with tessera_kv_compose_from           */
    const int32_t *unit_target_stride;  /* [n_units] 1 (default): token i is rotated for position
                                           target_pos + i; 0: every token is rotated for position
                                           target_pos (with target_pos = 0: written without rotation)     */
    /* Optional (NULL = nothing is kept): units that tessera_extend_write CAPTURES for the cache while it
       writes the request's fresh rows (Sec. 6.1: the forward path captures pre-RoPE keys and values;
       Sec. 5.3: the miss prefill keeps the same unrotated copy for the cache). */
    const int32_t *unit_retain_page_off;/* [n_units+1] CSR into unit_retain_pages.  A non-empty range marks a
                                           unit to keep: every one of its tokens must be a recompute row (an
                                           uncached unit, or a cached one recomputed in full), and the range
                                           must hold ceil(len / page_size) pages.  Token i of the unit lands in
                                           slot pages[i / page_size] * page_size + i % page_size               */
    const int32_t *unit_retain_pages;   /* cache page ids, all distinct                                          */
    int32_t retain_pool_pages;          /* 0 (default): the cache pages are pages of the destination pool itself
                                           (k_cache = k_pool) and must be neither source nor destination pages of
                                           this batch.  > 0: they index a separate cache pool of this many pages */
} tessera_compose_desc;

typedef struct tessera_plan tessera_plan;

enum { TESSERA_PLAN_HOST_ONLY = 1u };   /* plan_create flag: build and validate host tables only,
                                           touch no device (the plan then serves only the two
                                           inspection calls below and plan_destroy)               */
enum { TESSERA_FUSE_ROPE = 1u };        /* kv_compose flag: rotate keys while copying them        */

typedef struct tessera_plan_info {
    int64_t total_tokens;       /* sum of T_r                                                   */
    int64_t n_q;                /* recompute rows                                               */
    int64_t cached_tokens;      /* rows moved by kv_compose                                     */
    int64_t qk_pairs;           /* sum over query rows of (position + 1)                        */
    int64_t gather_bytes;       /* cached_tokens * H_kv * D * 2 bytes * 2 (K,V) * 2 (read,write) */
    int64_t attn_flops;         /* 4 * D * H_q * qk_pairs                                       */
    int32_t n_rope_rows;        /* distinct shift amounts in the cos/sin table                  */
    int32_t n_gather_items;     /* thread blocks of the gather kernel                           */
    int32_t n_attn_items;       /* (q tile, kv head) work items of the attention kernel         */
    int32_t attn_kernel;        /* always 1: the tcgen05 kernel covers every shape the plan accepts      */
    int64_t retained_tokens;    /* recompute rows that tessera_extend_write also writes to cache pages      */
    int64_t attn_mma_pairs;     /* (query row, key) products the attention kernel issues to the tensor cores:
                                   128 rows x 128 keys per (tile, step), summed over the work list.  The
                                   algorithmic count is qk_pairs * H_q; the difference is padding rows, keys
                                   above a row's causal limit inside a tile, and the ragged last step       */
} tessera_plan_info;

/*
 * Placement before preparation (Sec. 5.3): fixes every request's layout and its final KV slots.
 * Validates the batch, hands request r the next ceil(T_r/page_size) ids of free_pages, derives the
 * per-position source slot, the copy list, the table of shift amounts (cos/sin evaluated in fp64,
 * stored fp32) and the attention work list, and uploads them on `stream`.  The plan depends on the
 * layout only, so one plan serves every layer of the batch.
 *   num_pool_pages: pages in each pool tensor.   flags: 0 or TESSERA_PLAN_HOST_ONLY.
 * Returns the plan in *out; errors: every code above except DEVICE_TIMEOUT.
 */
TESSERA_API int32_t tessera_plan_create(const tessera_model_cfg *cfg, const tessera_compose_desc *desc,
                            int32_t num_pool_pages, uint32_t flags, tessera_plan **out, void *stream);

/* Frees host and device tables.  The caller must have synchronised every stream that used the plan. */
TESSERA_API int32_t tessera_plan_destroy(tessera_plan *plan);

/*
 * Host views of the placement result, valid until plan_destroy: page_off [batch+1], pages (the
 * request's block table, in position order), src_slot [sum T_r] (pool slot whose cached row lands at
 * each position, -1 where no cached unit covers it).  Any out pointer may be NULL.
 */
TESSERA_API int32_t tessera_plan_block_table(const tessera_plan *plan, const int32_t **page_off,
                                 const int32_t **pages, const int32_t **src_slot);

TESSERA_API int32_t tessera_plan_get_info(const tessera_plan *plan, tessera_plan_info *info);

/*
 * Reads the plan's device status word (synchronises `stream` first).  0 when no kernel of this plan
 * hit a bounded-wait limit since the last call; otherwise TESSERA_DEVICE_TIMEOUT and *detail (host,
 * nullable) receives a code naming the wait.  The word is cleared by the call.  While the word is
 * non-zero the attention kernel's blocks return at once (a stalled launch ends after one round of
 * timeouts), so after a timeout this call must be made before the plan is used again.
 */
TESSERA_API int32_t tessera_plan_status(tessera_plan *plan, int32_t *detail, void *stream);

/*
 * Preparing cache hits, on-GPU part (Sec. 5.3): copies every cached unit's K and V token rows from
 * its source pages into the request's destination pages at the unit's target offset.  V rows are bit
 * copies (values carry no rotation, Sec. 2.2).  With TESSERA_FUSE_ROPE the K rows are rotated from
 * their cached position to their new position on the way (fp32 math, one round-to-nearest-even to
 * bf16; a shift of 0 is a bit copy); without it K rows are bit copies and tessera_rope_shift must
 * follow.  k_pool, v_pool: device, layout above; source and destination pages live in the same pool.
 * The same call retains units: a plan whose "requests" are cache entries, whose sources are the pages
 * of a finished request (unit_src_offset) and whose unit_target_stride is 0 writes the un-rotated form.
 */
TESSERA_API int32_t tessera_kv_compose(const tessera_plan *plan, void *k_pool, void *v_pool, uint32_t flags, void *stream);

/*
 * Local-hit path of Sec. 5.3: the cached units are copied out of a separate source pool - the
 * node's PINNED HOST-MEMORY unit cache, read by the kernel straight over the interconnect (the memory
 * must be device-addressable: cudaHostAlloc / cudaHostRegister), or another device buffer - into the
 * request's destination pages in k_pool / v_pool, with the same flags and arithmetic as
 * tessera_kv_compose.  The plan must have been created with desc.num_source_pages > 0, and such a plan
 * is refused by tessera_kv_compose.  k_src, v_src: [num_source_pages][page_size][H_kv][D] bf16,
 * 16-byte aligned, never written.  Throughput is bounded by the link to the source memory, not by HBM.
 */
TESSERA_API int32_t tessera_kv_compose_from(const tessera_plan *plan, const void *k_src, const void *v_src,
                                            void *k_pool, void *v_pool, uint32_t flags, void *stream);

/*
 * 8-bit storage tier for cached units.  The paper's system stores conventional 16-bit K/V (Sec. 8,
 * "Algorithm and Model Compatibility") and has no counterpart of these two calls; they halve the
 * bytes a cache hit moves (Sec. 2.4: transfer volume is what a hit costs).  A stored byte is an
 * e4m3 code c (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities, largest finite
 * value 448, 0x7f / 0xff = NaN) and stands for c * scale, one positive finite scale per pool and
 * tensor (k_scale, v_scale).  Both calls need a plan created with desc.num_source_pages > 0 and use
 * its copy list and shift table exactly as tessera_kv_compose_from does.
 *
 * tessera_kv_compose_from_fp8 - expand: k_src8 / v_src8 [num_source_pages][page_size][H_kv][D] bytes
 *   (device-addressable, 16-byte aligned, never written) -> the request's destination pages in the
 *   16-bit pools k_pool / v_pool.  V and un-shifted K rows: bf16_rne(fp32(c) * scale) (the fp32
 *   product is rounded once, then once more to bf16; exact when scale is a power of two).  With
 *   TESSERA_FUSE_ROPE shifted K rows are rotated in fp32 from those fp32 products and rounded once
 *   to bf16; without it every K row is treated as un-shifted and tessera_rope_shift must follow.
 *
 * tessera_kv_retain_fp8 - retain: the reverse direction.  k_src / v_src are 16-bit pools
 *   [num_source_pages] (e.g. a finished request's pages), k_dst8 / v_dst8 8-bit pools of
 *   num_pool_pages pages whose free pages the plan consumed.  Every element is (rotated by the
 *   plan's shift when TESSERA_FUSE_ROPE is given - a retention plan shifts keys back to their
 *   position-free form -) multiplied in fp32 by the fp32 reciprocal 1.0f / scale and rounded to the
 *   nearest e4m3 value, ties to even, magnitudes above 448 saturating to +-448, NaN to 0x7f.
 *
 * Errors: as tessera_kv_compose_from; TESSERA_INVALID_ARG also for a scale that is not positive and
 * finite.  Nothing is allocated; one kernel is launched on `stream`.
 */
TESSERA_API int32_t tessera_kv_compose_from_fp8(const tessera_plan *plan, const void *k_src8, const void *v_src8,
                                                float k_scale, float v_scale, void *k_pool, void *v_pool,
                                                uint32_t flags, void *stream);
TESSERA_API int32_t tessera_kv_retain_fp8(const tessera_plan *plan, const void *k_src, const void *v_src, void *k_dst8,
                                          void *v_dst8, float k_scale, float v_scale, uint32_t flags, void *stream);

/*
 * "Applying RoPE to the keys at their new positions" (Sec. 5.3; the fused placement kernel of
 * Sec. 6.1) as a call of its own: rotates, in place, the destination-page K rows of every cached
 * unit by (new position - cached position).  NOT idempotent: call exactly once after a compose
 * without TESSERA_FUSE_ROPE, never after a fused compose.
 */
TESSERA_API int32_t tessera_rope_shift(const tessera_plan *plan, void *k_pool, void *stream);

/*
 * Neighbour of the extend pass (Sec. 5.3 "Completing prefill"; Sec. 2.2: queries and keys are rotated,
 * values are not): rotates, in place, the fresh queries q [n_q][H_q][D] and fresh keys k_new
 * [n_q][H_kv][D] (device, bf16) of the recompute rows for their target positions recompute_pos[j].
 * Either pointer may be NULL.  Angles, cosines and sines are evaluated in fp64 on the device and used
 * as fp32; fp32 math, one round-to-nearest-even to bf16.  Call it when the caller hands over
 * un-rotated projections; tessera_partial_prefill_attn itself expects rotated q and k_new.
 */
TESSERA_API int32_t tessera_rope_fresh(const tessera_plan *plan, void *q, void *k_new, void *stream);

/*
 * The write side of the extend pass in ONE pass over the fresh rows (Sec. 5.3 "Completing prefill";
 * Sec. 6.1: "the forward path captures pre-RoPE keys and values").  The caller hands over the layer's
 * projections BEFORE rotation.  For every recompute row j at position p_j = recompute_pos[j]:
 *   - k_new_raw[j] is read once; rotated for p_j it is written to the row's destination slot in
 *     k_pool (overriding a cached value: recomputed states belong to this request), and - when the
 *     row belongs to a unit marked by desc.unit_retain_page_off - its UNROTATED bits are also written
 *     to the unit's cache page in k_cache;
 *   - v_new[j] is copied to the destination slot in v_pool and, for a retained unit, to v_cache
 *     (bit copies: values carry no rotation, Sec. 2.2);
 *   - q[j] (nullable) is rotated for p_j in place.
 * Angle, cosine and sine are evaluated in fp64 on the device and used as fp32; fp32 math, one
 * round-to-nearest-even to bf16; a row at position 0 comes through bit for bit.  The captured unit is
 * position-free: a later plan reuses it as a cached unit with unit_cached_stride = 0.
 *   q [n_q][H_q][D], k_new_raw / v_new [n_q][H_kv][D]: device bf16, 16-byte aligned; k_new_raw and v_new
 *   are never written.  k_cache / v_cache: device pools in the pool layout with retain_pool_pages pages
 *   (or k_pool / v_pool themselves when retain_pool_pages is 0); nullable when the plan retains nothing.
 * After this call tessera_partial_prefill_attn is called with k_new = v_new = NULL (its own scatter is
 * then skipped) and the rotated q.  One kernel launch; nothing is allocated.
 */
TESSERA_API int32_t tessera_extend_write(const tessera_plan *plan, void *k_pool, void *v_pool, void *q,
                                         const void *k_new_raw, const void *v_new, void *k_cache, void *v_cache,
                                         void *stream);

/*
 * Completing prefill (Sec. 5.3): the extend pass restricted to the recompute rows.
 *   1. writes k_new / v_new (device, [n_q][H_kv][D], keys already rotated at their target
 *      positions) into the rows' destination slots, overriding cached values - recomputed states
 *      belong to this request only.  Skipped when k_new and v_new are both NULL.
 *   2. out[j][h] = softmax(sm_scale * q[j][h] . K[0..p_j][h/g]) . V[0..p_j][h/g] over the request's
 *      assembled pages, p_j = recompute_pos[j]; bf16 inputs, fp32 accumulation and softmax.
 *   q, out: device [n_q][H_q][D] bf16, 16-byte aligned (both are addressed through tiled bulk copies).
 *   lse: device [n_q][H_q] fp32 natural-log sum of exponentials, nullable.
 *   One persistent kernel (one thread block per SM) runs the whole batch; a batch too small to fill the
 *   GPU is split along the keys and merged by a second kernel.
 */
TESSERA_API int32_t tessera_partial_prefill_attn(const tessera_plan *plan, void *k_pool, void *v_pool,
                                     const void *q, const void *k_new, const void *v_new,
                                     void *out, float *lse, void *stream);

/*
 * Partial-prefill attention over 8-BIT KEY PAGES.  The paper stores and attends over 16-bit K/V
 * (Sec. 8, "Algorithm and Model Compatibility") and has no counterpart of this call; it is the extend
 * pass of Sec. 5.3 as a different numerical method: queries and keys are e4m3 codes (1-4-3 float, largest
 * value 448), S = Q K^T runs on the 8-bit tensor-core path, probabilities, values and the accumulator stay
 * as in tessera_partial_prefill_attn.
 *   k_pool8   device [num_pool_pages][page_size][H_kv][D] bytes: code c stands for c * k_scale.  The
 *             request's destination pages must hold its assembled keys as codes (written by
 *             tessera_kv_compose_k8, which rotates and quantises on the way).
 *   v_pool    device, 16-bit pool as everywhere else
 *   q         device [n_q][H_q][D] bf16, already rotated; quantised by the call itself into a buffer the
 *             plan owns (allocated on the first call): code = e4m3_rne(q * fp32(1 / q_scale)), saturating
 *   k_new, v_new  fresh rows (nullable together): k_new is written to the rows' slots of k_pool8 as
 *             e4m3_rne(k_new * fp32(1 / k_scale)), v_new to v_pool as bit copies
 *   out, lse  as in tessera_partial_prefill_attn: out[j][h] = softmax(sm_scale * (q8 q_scale) . (k8 k_scale)) . V
 * head_dim 128 only (TESSERA_UNSUPPORTED_SHAPE otherwise).  The result is compared with fp64 attention
 * over the DECODED operands (the codes times their scales) at the usual tolerance: the quantisation is
 * part of the method, not an error of the kernel.
 */
/*
 * Companion of the call below: "preparing cache hits" (Sec. 5.3) for the 8-bit-key attention path.  Like
 * tessera_kv_compose_from (16-bit units in a separate source pool, desc.num_source_pages > 0), but the
 * key rows land in the 8-bit pool k_pool8 - rotated (with TESSERA_FUSE_ROPE) in fp32, multiplied by
 * fp32(1 / k_scale) and rounded to the nearest e4m3 code, ties to even, saturating - while the value rows
 * are bit copies into the 16-bit v_pool.  No counterpart in the paper.  One kernel; nothing is allocated.
 */
TESSERA_API int32_t tessera_kv_compose_k8(const tessera_plan *plan, const void *k_src, const void *v_src, void *k_pool8,
                                          void *v_pool, float k_scale, uint32_t flags, void *stream);

TESSERA_API int32_t tessera_partial_prefill_attn_k8(tessera_plan *plan, void *k_pool8, float k_scale, void *v_pool,
                                                    const void *q, float q_scale, const void *k_new, const void *v_new,
                                                    void *out, float *lse, void *stream);

/*
 * The whole per-layer path for callers whose activations live in HOST memory: copies q, k_new,
 * v_new (host, pinned for full speed) to staging buffers owned by the plan, runs fused compose and
 * attention, copies out (and lse when non-null) back to the host and waits for `stream`.
 * The pools stay on the device: they are the resident KV cache.
 */
TESSERA_API int32_t tessera_composed_prefill_host(tessera_plan *plan, void *k_pool, void *v_pool,
                                      const void *q_host, const void *k_new_host, const void *v_new_host,
                                      void *out_host, float *lse_host, void *stream);

/*
 * The per-layer path when the cached units sit in the node's PINNED HOST-MEMORY cache (Sec. 5.3
 * "Preparing cache hits": a local hit is copied from the pinned host cache into the request's KV slots
 * while the engine keeps working on what is already prepared).  The plan must have been created with
 * desc.num_source_pages > 0.  The batch is cut into chunks of whole requests.  For each chunk a reader
 * launch of the gather kernel - `reader_blocks` thread blocks walking the chunk's copy list on a side
 * stream of the plan - pulls the rows over the interconnect straight into their destination slots, keys
 * rotated on the way (no staging buffer is needed: the bound on extra device memory is zero); when a
 * chunk has arrived, its fresh-row scatter + attention run on `stream` with a grid that leaves the
 * reader's SMs free, so attention of chunk c overlaps the transfer of chunk c + 1.  Results are
 * bit-identical to tessera_kv_compose_from + tessera_partial_prefill_attn.
 *   k_src_host, v_src_host  host, pinned and device-addressable (cudaHostAlloc / cudaHostRegister),
 *                           [num_source_pages][page_size][H_kv][D], 16-byte aligned, never written; bf16
 *                           when src_format is 0, e4m3 codes standing for code * k_scale / v_scale when
 *                           src_format is 1 (the scales are ignored for format 0)
 *   q, k_new, v_new, out, lse   device, as in tessera_partial_prefill_attn
 *   reader_blocks           thread blocks (of 256 threads) of the reader; 0 = 16; at most half the SM count
 * All work is enqueued on `stream` and on the side stream; the call returns without waiting.  The host
 * pools must stay valid and unchanged until `stream` has drained.
 */
TESSERA_API int32_t tessera_composed_prefill_host_tier(tessera_plan *plan, const void *k_src_host, const void *v_src_host,
                                                       int32_t src_format, float k_scale, float v_scale,
                                                       void *k_pool, void *v_pool, const void *q, const void *k_new,
                                                       const void *v_new, void *out, float *lse, int32_t reader_blocks,
                                                       void *stream);

/*
 * In-place RoPE shift for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a service entry of this library.)  Some callers run where cudaMalloc is off
 * limits: inside a serving engine that owns the whole device through its own memory pool, in a
 * phase where the allocator must stay untouched, or under a no-allocation-after-start-up rule.
 * tessera_plan_create allocates its tables, so such callers cannot use the plan-based shift.  This
 * call needs no plan and allocates nothing: its cos/sin table sits in a fixed 256 KB array inside
 * the library image, which every device that loads the library holds until the process exits.
 *
 * Rotates, in place, row slots[i] of k_pool (device, pool layout above) by shifts[slot_shift[i]]
 * positions, with the arithmetic of tessera_rope_shift (angle, cosine and sine in fp64 stored as
 * fp32, fp32 math, one round-to-nearest-even to bf16; a shift of 0 leaves the bits unchanged).
 *   cfg            host: head_dim (64 or 128), num_kv_heads and rope_theta / inv_freq are read.
 *                  rope_pairing must be 0: only half-split pairs (m, m + D/2) are supported here;
 *                  rope_pairing = 1 is refused with TESSERA_UNSUPPORTED_SHAPE
 *   num_pool_slots rows in k_pool (num_pool_pages * page_size): the bound every listed slot is checked
 *                  against on the device
 *   slots          device [n_slots] pool slot ids (page * page_size + offset); each listed once.
 *                  An id outside [0, num_pool_slots) is skipped: that row is neither read nor written
 *   slot_shift     device [n_slots] index into shifts; entries outside [0, n_shifts) are skipped too
 *   shifts         host   [n_shifts] shift amounts; n_shifts <= TESSERA_STATIC_MAX_SHIFTS, otherwise
 *                  TESSERA_UNSUPPORTED_SHAPE and nothing is launched.  The values are copied into the
 *                  launch itself, so the array may be freed as soon as the call returns
 * The first call on a device looks up the array's device address (once per device, with that device
 * current); make that first call before any stream capture begins.  All calls on a device share
 * the array and each call overwrites the rows it uses (nothing in it has to start at zero), so two
 * calls whose GPU work can overlap - different streams without ordering - race on it; calls on one
 * stream are safe.  Two kernels (table fill, rotation) are enqueued on `stream`; the call does not
 * wait for them and copies nothing from host memory.
 */
#define TESSERA_STATIC_MAX_SHIFTS 512
TESSERA_API int32_t tessera_rope_shift_static(const tessera_model_cfg *cfg, void *k_pool, int64_t num_pool_slots,
                                              const int32_t *slots, const int32_t *slot_shift, int32_t n_slots,
                                              const int32_t *shifts, int32_t n_shifts, void *stream);

/*
 * Diagnostic (the paper has no counterpart): exercises the bounded wait that every kernel of this
 * library uses around its mbarriers.  Launches one small thread block that waits on a barrier nobody
 * arrives on; the wait must give up after max_cycles SM cycles (1 .. 2e9), record code 42 and let the
 * kernel end normally.  Synchronises `stream`.  Returns TESSERA_DEVICE_TIMEOUT when the wait ran out
 * as intended (code_out = 42), TESSERA_OK if it did not (a defect).  cycles_out (host, nullable, 3
 * entries): cycles spent in the first wait, cycles spent in a second wait issued after the abort flag
 * was up (must be small), and a bit mask of waits that reported success (must be 0).
 */
TESSERA_API int32_t tessera_selftest_bounded_wait(int64_t max_cycles, int32_t *code_out, int64_t *cycles_out, void *stream);

/* Copies the calling thread's last error text into buf (host); returns its length. */
TESSERA_API int32_t tessera_last_error(char *buf, int32_t len);

/* Kernels this library has launched in this process so far (all plans, all streams). */
TESSERA_API int64_t tessera_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TESSERA_H_ */

/*
 * libcompact_attn -- attention for parallel context compaction on one B200 (sm_100a).
 *
 * Problem statement (paper, Section 4 "Parallel Compaction"): when a history
 * exceeds the threshold it is snapshotted and cut into N contiguous blocks
 * ("Snapshot & partition", N = ceil(|X| / B), last block possibly short); every
 * block is handed to its own summarisation sequence and all N run concurrently
 * ("Dispatch"); the N summaries are concatenated in block order ("Merge").  This
 * library runs the attention of those N concurrent sequences in the
 * "independent chunks" layout of Section 4: a sequence sees its own block only,
 * so attention is block-diagonal and causal inside each block.  Sequential
 * compaction (Section 2.2, Eq. 1) is the N = 1 case of the same calls.  The same
 * kernels serve the paper's own prefix-aware layout (cpa_plan_create_prefix: a
 * worker reads the cached history up to its block, then runs its own tokens),
 * prefill in chunks beside the decode of other blocks (cpa_plan_create_chunked,
 * cpa_step_mixed), summaries of unknown length without reserved pages
 * (cpa_plan_create_dynamic) and whole events from host memory (cpa_event_host).
 *
 * The paper does not spell out attention; it is the textbook operation
 *     O[i,h,:] = sum_{j<=i} softmax_j(scale * q[i,h,:].k[j,g,:]) v[j,g,:],  g = h div G,
 * with G = num_q_heads / num_kv_heads (contiguous head groups), keys restricted
 * to the query's own block.
 *
 * Conventions for every call
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global
 *     memory of the current device.  The library allocates NO device memory: all
 *     device buffers belong to the caller, with sizes taken from cpa_plan_param.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Device work is enqueued asynchronously on it.
 *   - Tensors are bf16.  Packed token-major layout [tokens, heads, head_dim] for
 *     Q/K/V/O, blocks back to back in block order (offsets = cu_seqlens).
 *     KV pools are [num_pages, num_kv_heads, page_size, head_dim], one pool for K
 *     and one for V; a (page, head) chunk is contiguous.  Inside a row the 16-byte
 *     pieces are permuted: piece j of the row in slot r is stored at position
 *     (j & ~7) | ((j & 7) ^ (r & 7)), so that a chunk copied verbatim into shared
 *     memory is read without bank conflicts.  Only this library reads the pools.
 *   - Every call returns 0 (CPA_OK) or a negative cpa_status.  Nothing throws,
 *     exits, or traps the device.  Device-side waits are bounded; if one gives up
 *     the kernel stops issuing work, lets the copies and MMAs it has in flight
 *     finish (again with a bound), frees its tensor memory and returns, and the
 *     plan's device status word (the first int32 of the index buffer) keeps the
 *     first code recorded: 1 = a wait gave up, 2 = an append found no room.
 *     cpa_plan_status reads it back.  After a non-zero status the results of that
 *     launch are void and the plan must be uploaded again before further use.
 *   - Thread safety: a plan is used by one host thread at a time.  Different
 *     plans may be used from different threads; the library's only process-wide
 *     state are per-device flags and addresses that every thread sets to the same
 *     value (kept in relaxed atomics).
 *   - Limits: group size G <= 8, num_sms <= 4095, block lengths and page counts
 *     below 2^30, and at most 65535 workers in a plan with cached prefixes.
 *   - There is no CPU fallback: without a CUDA device the compute calls return
 *     CPA_ECUDA.
 */
#ifndef COMPACT_ATTN_H_
#define COMPACT_ATTN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define CPA_API __attribute__((visibility("default")))
#else
#define CPA_API
#endif

typedef enum cpa_status {
    CPA_OK = 0,
    CPA_EINVAL = -1,       /* bad argument: null/misaligned pointer, length < 1, heads not divisible ... */
    CPA_ENOSPC = -2,       /* free list too short, caller buffer too small, or append beyond the reservation */
    CPA_EUNSUPPORTED = -3, /* head_dim not in {64,128}, page_size != 16, group size > 8 ... */
    CPA_ECUDA = -4,        /* a CUDA runtime/driver call failed (no device, launch error) */
    CPA_ETIMEOUT = -5,     /* a bounded device-side wait gave up (read from the status word) */
    CPA_ESTATE = -6        /* call order violated (e.g. compute before cpa_plan_upload) */
} cpa_status;

typedef struct cpa_config {
    int32_t num_q_heads;
    int32_t num_kv_heads;    /* must divide num_q_heads; group size G <= 8 */
    int32_t head_dim;        /* 64 or 128 */
    int32_t page_size;       /* 16 */
    float   scale;           /* softmax scale, normally 1/sqrt(head_dim) */
    int32_t q_tile_rows;     /* query rows per prefill work item: 128, 256, or 512 (items of 512 rows run on pairs of
                                CTAs, cta_group::2: head_dim 128, plans without cached prefixes or chunks only;
                                measured no faster than 256, kept as an option); 0 = default (256) */
    int32_t pages_per_split; /* KV pages per decode work item (<= 1024); 0 = chosen per block from the batch */
    int32_t num_sms;         /* SMs this plan's kernels may fill: the persistent prefill launches min(num_sms, units)
                                CTAs (one per SM) and the decode wave is sized for 3 * num_sms CTAs; 0 = the SM
                                count of the device that is current when the plan is created (148 if there is
                                none); at most 4095.  A value below the device's SM count leaves SMs to other
                                streams (a CTA of the prefill keeps its SM for the whole launch, stream priority
                                does not preempt it) */
} cpa_config;

typedef struct cpa_plan cpa_plan; /* opaque; host memory owned by the library */

/* Index arrays a plan holds (all int32), for cpa_plan_export. */
enum {
    CPA_ARR_CU_SEQLENS = 0,    /* [B+1] prefix sums of block lengths */
    CPA_ARR_PAGE_INDPTR = 1,   /* [B+1] prefix sums of pages per block */
    CPA_ARR_PAGE_INDICES = 2,  /* [page_indptr[B]] pool page ids, block-major */
    CPA_ARR_SEQ_LENS = 3,      /* [B] tokens cached per block (host mirror) */
    CPA_ARR_SLOT_MAPPING = 4,  /* [tokens] pool slot (page*P + offset) of every prefill token */
    CPA_ARR_PREFILL_ITEMS = 5, /* [n,2] (block, q_tile) in launch order */
    CPA_ARR_DECODE_ITEMS = 6,  /* [n,3] (block, kv_head, split) in launch order */
    CPA_ARR_SPLIT_INDPTR = 7,  /* [B+1] prefix sums of decode splits per block */
    CPA_ARR_SPLIT_PAGES = 8,   /* [B] pages per decode split of each block (the last split may be shorter) */
    CPA_ARR_PREFILL_SCHED = 9, /* [rounds * CPA_PARAM_PREFILL_CTAS] prefill unit (item * num_q_heads + head) of CTA c
                                  in round k at k * ctas + c, -1 = none; every unit appears exactly once */
    CPA_ARR_DEC_START = 10,    /* [B] chunked plans: the step at which each block starts to decode */
    CPA_ARR_CHUNK_ROWS = 11,   /* [CPA_PARAM_CHUNK_STEPS * (B+1)] chunked plans: per chunk index, prefix sums of the
                                  rows each block prefills in it */
    CPA_ARR_PAGES_ASSIGNED = 12, /* [B] plans with pages on demand: pages each block holds (as of creation or the last cpa_plan_sync) */
    CPA_ARR_FREE_RING = 13,    /* plans with pages on demand: the pages of the common reserve, in the order they will be handed out */
    CPA_ARR_SPLIT_RANGES = 14  /* [own splits, 2] (first own page, pages) of every decode split of a block's own pages,
                                  block-major (the splits of block b are entries split_indptr[b] + slots of the shared
                                  scan .. split_indptr[b+1]) */
};

/* Scalars of a plan, for cpa_plan_param. */
enum {
    CPA_PARAM_NUM_BLOCKS = 0,
    CPA_PARAM_TOTAL_TOKENS = 1,
    CPA_PARAM_Q_TILE_ROWS = 2,
    CPA_PARAM_PAGES_PER_SPLIT = 3,       /* largest split size over the blocks */
    CPA_PARAM_PAGES_USED = 4,            /* page_indptr[B] */
    CPA_PARAM_INDEX_BYTES = 5,           /* size of the device index buffer for cpa_plan_upload */
    CPA_PARAM_DECODE_WORKSPACE_BYTES = 6,/* size of cpa_decode's device workspace */
    CPA_PARAM_TOTAL_SPLITS = 7,          /* split_indptr[B] */
    CPA_PARAM_MAX_NEW_TOKENS = 8,
    CPA_PARAM_PREFILL_CTAS = 9,          /* columns of CPA_ARR_PREFILL_SCHED: the CTAs of the prefill launch,
                                            min(num_sms, prefill units), or for 512-row items its PAIRS of CTAs,
                                            min(num_sms / 2 (at most what the device holds at a time), units) */
    CPA_PARAM_SHARED_CHUNK_PAGES = 10,   /* pages per chunk of the shared-prefix decode scan; 0 without cached prefixes */
    CPA_PARAM_CHUNK_TOKENS = 11,         /* tokens per prefill chunk; 0 = not a chunked plan */
    CPA_PARAM_NUM_STEPS = 12,            /* steps of a chunked plan's schedule */
    CPA_PARAM_CHUNK_STEPS = 13,          /* chunk indices of the schedule (the most chunks of any block) */
    CPA_PARAM_DECODE_SMS = 14,           /* SMs a chunked plan leaves to the decode wave while a chunk is prefilled */
    CPA_PARAM_NUM_SMS = 15,              /* the plan's SM budget (cfg.num_sms, or the device's SM count for 0) */
    CPA_PARAM_DECODE_STEPS_PER_CHUNK = 16, /* decode steps a chunked plan's schedule gives a chunk */
    CPA_PARAM_DECODE_EVEN_CUT = 17,      /* 1: the decode splits come from the even cut (see cpa_plan_create), 0: uniform per block */
    CPA_PARAM_DECODE_CTAS = 18,          /* CTAs of a decode launch */
    CPA_PARAM_HOST_STAGE_BYTES = 19      /* size of cpa_event_host's device staging buffer */
};

/*
 * cpa_plan -- "Snapshot & partition" + "Dispatch" bookkeeping (Section 4).
 * Builds, on the host, everything the kernels index with:
 *   cu_seqlens; per block ceil((L_b + max_new_tokens) / page_size) pages taken in
 *   order from `free_pages` (block 0 first); seq_lens (0: nothing cached yet);
 *   the slot of every prefill token; the prefill work list of (block, q_tile)
 *   ordered by descending cost (keys seen by the tile's last row), ties by
 *   ascending block then tile; the deal of the prefill units (item, query head) to
 *   the CTAs of the persistent prefill kernel (kv head by kv head, in rounds of one unit
 *   per CTA, the most expensive unit of a round to the least loaded CTA, see
 *   CPA_ARR_PREFILL_SCHED); the decode work list of (block, kv_head, split),
 *   split s = pages [s*C_b, (s+1)*C_b) of the block, ordered by descending page
 *   count, ties by ascending block, kv head, split.  C_b is cfg->pages_per_split, or
 *   with 0 it is chosen per block so that all items fill one wave of CTAs (three per
 *   SM): splits start at one per block and the block with the largest splits is
 *   split further while kv_heads more items still fit (never below 4 pages).  With 0 the
 *   planner also tries the EVEN CUT: all blocks' pages laid end to end are cut into equal
 *   ranges, one per group of kv_heads CTAs of the wave, so that every CTA streams the same
 *   number of pages; block b then has a first split that ends at the next cut, full splits
 *   of C pages and a remainder (CPA_ARR_SPLIT_RANGES lists them), and a CTA whose range
 *   crosses a block boundary has two items.  It is taken when it loads the busiest SM at
 *   least 5 % less than the uniform cut, a second item in a CTA counted as 16 pages (CPA_PARAM_DECODE_EVEN_CUT); CPA_ARR_DECODE_ITEMS
 *   is then in launch order (CTA-major rounds) instead of descending size.
 * block_lens, free_pages: host int32 arrays (copied; caller keeps ownership).
 * Page ids must be >= 0, at most (2^31 - 1) / max(64, 32 * num_kv_heads) (the pools' rows are addressed with
 * 32-bit coordinates; far beyond what fits a device), and distinct (distinctness is the caller's contract).
 * Errors: CPA_EINVAL (null pointer, num_blocks < 1, a length < 1,
 * max_new_tokens < 0, page id out of range, heads not divisible), CPA_EUNSUPPORTED,
 * CPA_ENOSPC (num_free too small).  On error *out is NULL.
 */
CPA_API int cpa_plan_create(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                    int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                    cpa_plan** out);

/*
 * cpa_partition -- "Snapshot & partition" (Section 4): a history of |X| tokens is cut into N = ceil(|X| / B)
 * contiguous blocks of B tokens, the last one possibly shorter (Section 5, "Threshold and block size
 * interaction": 96k tokens at 16k per block are 6 workers, at 4k per block 24).  Writes the N block lengths
 * to the host array `block_lens` (capacity `capacity` entries) and N to `num_blocks`; the lengths are what
 * cpa_plan_create takes, and i * B what cpa_plan_create_prefix takes as worker i's prefix.  Host arithmetic
 * only.  Errors: CPA_EINVAL (a length below 1, a null pointer), CPA_ENOSPC (more than `capacity` blocks;
 * `num_blocks` still says how many), CPA_EUNSUPPORTED (more than 2^31 - 1 blocks).
 */
CPA_API int cpa_partition(int64_t history_tokens, int32_t block_tokens, int32_t* block_lens, int32_t capacity,
                          int32_t* num_blocks);

/*
 * cpa_plan_create_prefix -- the plan for the paper's own layout (Section 4, "Dispatch" and
 * "Prefix-aware target-at-end layout"): the prompt of worker w is blocks 1..w-1 of the history
 * followed by block w wrapped in its markers, every worker's prefix extends the previous worker's,
 * and that prefix is not recomputed but read from the KV cache the history already has.
 *   own_lens[w]    : tokens worker w runs itself (its target block plus markers), >= 1
 *   prefix_lens[w] : history tokens worker w reads from the cache; a multiple of 128 (the
 *                    prefill kernel reads a cached prefix in whole KV tiles of 128 keys; a
 *                    block boundary that is not a multiple of 128 is handled by the caller
 *                    giving the remainder to own_lens, as a serving engine's block-granular
 *                    prefix cache does with a partial block)
 *   shared_pages   : host int32 [num_shared] pool pages that hold the history, page i = history
 *                    tokens [16 i, 16 i + 16); they must be filled (cpa_kv_append through a plan
 *                    that owns them) before cpa_prefill_prefix or a decode call reads them, and
 *                    no call through this plan ever writes them
 * Worker w's page list is shared_pages[0 .. prefix_lens[w]/16) followed by
 * ceil((own_lens[w] + max_new_tokens) / 16) pages of its own from `free_pages`; its cached
 * length (seq_lens) starts at prefix_lens[w]; positions and slots count from the start of the
 * prompt; the cost of a prefill item includes the prefix.  Decode runs in two levels: the shared
 * pages are scanned once for all workers in chunks of CPA_PARAM_SHARED_CHUNK_PAGES pages (a kernel
 * of its own inside cpa_decode / cpa_decode_append), worker w has
 * ceil(prefix pages / chunk) partial slots for that scan in front of the slots of its splits, and
 * its splits (CPA_ARR_DECODE_ITEMS, CPA_ARR_SPLIT_PAGES) cover its own pages only.  Everything else is
 * as for cpa_plan_create, which is the case prefix_lens == 0.  Errors as for cpa_plan_create,
 * plus CPA_EINVAL for a prefix that is negative, not a multiple of 128, or longer than
 * 16 * num_shared.
 */
CPA_API int cpa_plan_create_prefix(const cpa_config* cfg, int32_t num_workers, const int32_t* own_lens,
                                   const int32_t* prefix_lens, const int32_t* shared_pages, int32_t num_shared,
                                   int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                                   cpa_plan** out);

/*
 * cpa_plan_create_chunked -- the plan for an event whose prefill runs in chunks.  The paper's serving
 * engine runs with chunked prefill enabled (Section 4.2, "Hardware and Serving Infrastructure"), and its
 * finding that 16k blocks are prefill-bound (Section 6, "Prefill cost limits parallelism") is the case
 * this is for: a long block's prompt is cut into chunks, and the blocks that are past their prompt
 * decode meanwhile instead of waiting behind it.  The paper gives no rule; this library's is
 * (C = chunk_tokens, r = decode_steps_per_chunk):
 *   a block of L_b tokens has n_b = ceil(L_b / C) chunks; chunk c, rows [c * C, min((c + 1) * C, L_b)),
 *   starts at step c * r; the block decodes summary token t at step n_b * r + t, t < max_new_tokens;
 *   the schedule has max_b(n_b) * r + max_new_tokens steps (CPA_PARAM_NUM_STEPS), run one by one with
 *   cpa_step_mixed.
 * chunk_tokens: a multiple of 128 (a later chunk reads the earlier ones from the block's pages in whole
 * KV tiles of 128 keys).  decode_steps_per_chunk >= 1: how many decode steps a chunk is given; a chunk
 * costs far more than a decode step, so with r = 1 the decoding blocks produce tokens at the chunks' pace,
 * and with r near (chunk time / decode step time) both sides stay busy.  decode_sms: SMs left to the
 * decode wave while a chunk is under way (the chunk's persistent grid takes the other num_sms -
 * decode_sms); 0 = a quarter of the plan's SMs.
 * Everything else (pages, slots, whole-block prefill list, decode items) is as for cpa_plan_create, and
 * the plan also works with the whole-block calls (cpa_prefill, cpa_kv_append, cpa_decode_append) as long
 * as the two ways are not mixed within one event.  Errors as for cpa_plan_create, plus CPA_EINVAL for a
 * chunk size below 128 or not a multiple of 128, decode_steps_per_chunk < 1 and decode_sms >= the plan's SMs.
 */
CPA_API int cpa_plan_create_chunked(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                                    int32_t max_new_tokens, int32_t chunk_tokens, int32_t decode_steps_per_chunk,
                                    int32_t decode_sms, const int32_t* free_pages, int32_t num_free, cpa_plan** out);

/*
 * cpa_plan_create_prefix_chunked -- the prefix-aware layout and chunked prefill together, which is how the
 * paper's serving engine runs (Section 4.2: automatic prefix caching and chunked prefill both enabled;
 * Section 4, "Dispatch": every worker's prompt extends the previous worker's).  Worker w reads prefix_lens[w]
 * cached history tokens from `shared_pages` (as for cpa_plan_create_prefix) and runs its own_lens[w] tokens
 * in chunks of chunk_tokens (as for cpa_plan_create_chunked): chunk c of worker w attends the cached history,
 * then the worker's earlier chunks (already in its own pages), then causally itself; its keys and values land
 * at sequence positions prefix_lens[w] + c * chunk_tokens + i; the worker's first decode step starts from the
 * length prefix_lens[w] + own_lens[w].  The schedule (chunk c at step c * r, summary token t at step
 * n_w * r + t), the arguments and cpa_step_mixed are those of cpa_plan_create_chunked; decode runs in the
 * two levels of cpa_plan_create_prefix.  Errors: the union of the two creators'.
 */
CPA_API int cpa_plan_create_prefix_chunked(const cpa_config* cfg, int32_t num_workers, const int32_t* own_lens,
                                           const int32_t* prefix_lens, const int32_t* shared_pages,
                                           int32_t num_shared, int32_t max_new_tokens, int32_t chunk_tokens,
                                           int32_t decode_steps_per_chunk, int32_t decode_sms,
                                           const int32_t* free_pages, int32_t num_free, cpa_plan** out);

/*
 * cpa_plan_create_dynamic -- a plan that reserves no pages for the summaries.  The paper's outlook (Section 8,
 * "Dynamic block size and prompt selection") wants block sizes and summary lengths that are not fixed in
 * advance, and its second benchmark (Section 3.1: documents of about 0.7k tokens, six questions each) is many
 * short sequences whose summaries stop at different lengths; reserving max_new_tokens for each wastes most of
 * the pool.  The paper has no rule; this library's is:
 *   a block starts with the pages for its tokens plus the next one, L_b / page_size + 1 of them (never more than
 *   its row of the page table holds, ceil((L_b + max_new_tokens) / page_size): max_new_tokens only bounds growth),
 *   dealt in order from `free_pages`; the rest of `free_pages` becomes a common reserve, a ring in the index
 *   buffer; the decode launch that fills a block's page takes the next page for it from the ring; a block that
 *   has stopped gives its pages back with cpa_release_blocks.
 * CPA_ARR_PAGE_INDICES is then a table of B rows (row b = page_indptr[b] .. page_indptr[b+1]), valid up to
 * CPA_ARR_PAGES_ASSIGNED[b] entries; the host copies are those of plan creation until cpa_plan_sync refreshes
 * them.  Decode with cpa_decode_append or cpa_decode_append_dynamic (cpa_kv_append with new_lens == NULL
 * returns CPA_EUNSUPPORTED: it takes no pages).  Errors as for cpa_plan_create (CPA_ENOSPC: the free list does
 * not cover the first pages).
 */
CPA_API int cpa_plan_create_dynamic(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                                    int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                                    cpa_plan** out);

/* Synchronise `stream` and read the device's lengths (CPA_ARR_SEQ_LENS) and, for a plan with pages on demand, its
 * page table, pages per block and reserve back into the host copies that cpa_plan_export shows.  (The paper has
 * no counterpart.)  Errors: CPA_EINVAL, CPA_ESTATE (not uploaded), CPA_ECUDA. */
CPA_API int cpa_plan_sync(cpa_plan* plan, void* stream);

/* Borrow a host view of one index array (valid until the plan is destroyed or,
 * for CPA_ARR_SEQ_LENS, until the next cpa_kv_append).  Errors: CPA_EINVAL. */
CPA_API int cpa_plan_export(const cpa_plan* plan, int which, const int32_t** ptr, int64_t* count);

/* One scalar of the plan, or a negative cpa_status for an unknown `which`. */
CPA_API int64_t cpa_plan_param(const cpa_plan* plan, int which);

/*
 * Copy the index arrays into the caller's device buffer (>= CPA_PARAM_INDEX_BYTES
 * bytes, 16-byte aligned) on `stream` and bind the plan to that buffer; device
 * seq_lens and the status word start at 0.  The buffer must stay alive and
 * untouched by the caller until the plan is destroyed.  Errors: CPA_EINVAL,
 * CPA_ENOSPC (bytes too small), CPA_ECUDA.
 */
CPA_API int cpa_plan_upload(cpa_plan* plan, void* d_index_buf, int64_t bytes, void* stream);

/* Synchronise `stream`, read the device status word: CPA_OK, CPA_ETIMEOUT (a bounded
 * device-side wait gave up), CPA_ENOSPC (an append found no page or slot left), or
 * CPA_ECUDA if the stream reports an error.  CPA_ESTATE before upload. */
CPA_API int cpa_plan_status(cpa_plan* plan, void* stream);

CPA_API void cpa_plan_destroy(cpa_plan* plan);

/*
 * cpa_prefill -- causal attention of every block over itself (the prefill each
 * concurrent summarisation sequence runs over its block, Section 4 "Dispatch";
 * block-diagonal because of the independent-chunks layout).
 *   q, o : device bf16 [total_tokens, num_q_heads, head_dim]
 *   k, v : device bf16 [total_tokens, num_kv_heads, head_dim]
 * All four 16-byte aligned; o must not alias the inputs.  One launch of
 * CPA_PARAM_PREFILL_CTAS persistent CTAs covers all (block, q_tile, head) units.
 * d_workspace is unused (may be NULL).
 * Errors: CPA_EINVAL, CPA_ESTATE (plan not uploaded), CPA_ECUDA.
 */
CPA_API int cpa_prefill(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o,
                void* d_workspace, void* stream);

/*
 * cpa_prefill_prefix -- the prefill of the prefix-aware layout (Section 4, "Dispatch"; Section 6
 * observes that every worker still has to prefill its own block, which the prefix cache does not
 * hold): row i of worker w attends over the prefix_lens[w] cached history
 * tokens and over its own tokens 0..i,
 *     O[i,h,:] = sum_{j < prefix or j-prefix <= i} softmax_j(scale * q[i,h,:].k[j,g,:]) v[j,g,:].
 *   q, o   : device bf16 [sum(own_lens), num_q_heads, head_dim], the workers' own tokens
 *   k, v   : device bf16 [sum(own_lens), num_kv_heads, head_dim], the same tokens' keys/values
 *   k_pool, v_pool : the pools; only the shared pages of each worker's prefix are read
 * The plan must come from cpa_plan_create_prefix (or cpa_plan_create: then nothing is read from
 * the pools and the result is cpa_prefill's).  Prefix tiles are staged straight from the pool
 * pages into the kernel's shared-memory tiles.  Follow with cpa_kv_append(own_lens) to cache the
 * own tokens behind the prefix.  Errors: as cpa_prefill.
 */
CPA_API int cpa_prefill_prefix(const cpa_plan* plan, const void* q, const void* k, const void* v, const void* k_pool,
                               const void* v_pool, void* o, void* stream);

/*
 * cpa_prefill_variant -- cpa_prefill with the kernel chosen by the caller; for
 * cross-checking one kernel against the other on the device and for profiling.
 * (The paper has no counterpart.)  Same arguments, layouts and errors as
 * cpa_prefill; CPA_EINVAL for an unknown variant.
 *   CPA_PREFILL_TENSOR_CORE  TMA-staged tiles, tcgen05 MMAs, accumulators in TMEM
 *   CPA_PREFILL_WARP_MMA     warp-level mma.sync kernel (the earlier, slower design)
 */
enum { CPA_PREFILL_TENSOR_CORE = 0, CPA_PREFILL_WARP_MMA = 1 };
CPA_API int cpa_prefill_variant(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o,
                                void* stream, int variant);

/*
 * cpa_kv_append -- write new K/V rows into the blocks' pages and advance
 * seq_lens (the KV cache each sequence keeps while it decodes its summary).
 * The paper has no counterpart: Section 4.2 names the serving engine whose paged
 * cache does this underneath and says nothing about it; the slot rule below is
 * this library's own.
 *   k_new, v_new : device bf16 [sum(new_lens), num_kv_heads, head_dim], block-major
 *   new_lens     : host int32 [B] tokens to add per block, or NULL = one token
 *                  per block (a decode step; then k_new is [B, kv_heads, head_dim]).
 * Token i of block b goes to position seq_lens[b] + i, i.e. pool slot
 * page_indices[page_indptr[b] + pos / P] * P + pos % P.  With new_lens == NULL,
 * or new_lens == block_lens on an empty cache, nothing is copied from the host,
 * so the call enqueues device work only; otherwise B+1 offsets are copied
 * to the device first.  Errors: CPA_EINVAL, CPA_ESTATE, CPA_ENOSPC (a block would
 * outgrow L_b + max_new_tokens; nothing is launched), CPA_ECUDA.
 */
CPA_API int cpa_kv_append(cpa_plan* plan, const void* k_new, const void* v_new, const int32_t* new_lens,
                  void* k_pool, void* v_pool, void* stream);

/*
 * cpa_decode -- one batched decode step (Section 4, "Dispatch": the N summarisation
 * sequences run concurrently, so every step produces one token of every block's
 * summary; Section 2.1 notes that the per-token cost of this step grows with the
 * context length): the newest token of every block
 * attends over that block's whole cache, the token itself included (call
 * cpa_kv_append for the step first).  Split-K over the block's pages, then a
 * log-sum-exp merge of the split partials
 *     m = max_s m_s,  l = sum_s l_s e^(m_s - m),  O = sum_s acc_s e^(m_s - m) / l.
 *   q, o        : device bf16 [B, num_q_heads, head_dim]
 *   k_pool/v_pool: device bf16 pools (read only)
 *   d_workspace : device scratch, >= CPA_PARAM_DECODE_WORKSPACE_BYTES, 16-byte aligned;
 *                 contents are overwritten; calls sharing one workspace must not overlap.
 * Lengths are read from the device seq_lens, so T steps can be enqueued back to
 * back without host synchronisation.  Errors: CPA_EINVAL, CPA_ESTATE (also: a worker
 * of a prefix-aware plan has none of its own tokens cached yet), CPA_ECUDA.
 */
CPA_API int cpa_decode(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool,
               void* o, void* d_workspace, void* stream);

/*
 * cpa_decode_append -- one decode step with its append fused in: exactly
 * cpa_kv_append(plan, k_new, v_new, NULL, ...) followed by cpa_decode(...), in one launch
 * (the per-step work of a summarisation sequence, Section 4 "Dispatch": store the new
 * token's key/value, then attend over the block's cache including it).
 *   q, o          : device bf16 [B, num_q_heads, head_dim]
 *   k_new, v_new  : device bf16 [B, num_kv_heads, head_dim], the new token of every block
 *   k_pool/v_pool : device bf16 pools; the new rows are written into them
 *   d_workspace   : as for cpa_decode
 * The CTA that scans the page holding the new position stores the row and uses it from its
 * staged copy; the device lengths are double buffered, so the call needs no separate kernel
 * to advance them.  Results are those of the two separate calls.  Errors: CPA_EINVAL,
 * CPA_ESTATE, CPA_ENOSPC (a block would outgrow L_b + max_new_tokens; nothing is launched),
 * CPA_ECUDA.
 */
CPA_API int cpa_decode_append(cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                              void* v_pool, void* o, void* d_workspace, void* stream);

/*
 * cpa_decode_append_steps -- `num_steps` consecutive cpa_decode_append calls enqueued by one call, for
 * callers whose inputs of several steps are on the device already (a benchmark, a replay; in a model the next
 * step's query depends on this step's output, so there it is one step per call).
 *   q, o          : device bf16 [num_steps, B, num_q_heads, head_dim]; step t uses slice t
 *   k_new, v_new  : device bf16 [num_steps, B, num_kv_heads, head_dim]
 * Everything else, and the errors, as for cpa_decode_append; the capacity of every block is checked for all
 * steps before the first launch (CPA_ENOSPC: nothing is launched).  num_steps < 0: CPA_EINVAL; 0: nothing to do.
 */
CPA_API int cpa_decode_append_steps(cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                                    void* v_pool, void* o, void* d_workspace, int32_t num_steps, void* stream);

/*
 * cpa_decode_append_dynamic -- cpa_decode_append for a plan with pages on demand (cpa_plan_create_dynamic;
 * Section 8, "Dynamic block size and prompt selection"), with per-block stop flags that live on the device, so
 * that summaries of different, unknown lengths need neither a new plan nor a host round trip per step.
 *   d_active : device int32 [B], or NULL = every block takes part.  Block b decodes in this step iff
 *              d_active[b] != 0; a block that sits out keeps its length, and its rows of o are not written.
 * A block whose new token fills a page takes the page for the next one from the reserve inside the launch.  If
 * the reserve is empty the block stops growing: in its next step it sits out and the status word reads back as
 * CPA_ENOSPC (cpa_plan_status); nothing is written outside the block's pages.  The host's CPA_ARR_SEQ_LENS counts
 * a token per call for every block (an upper bound; cpa_plan_sync reads the true lengths), and the call returns
 * CPA_ENOSPC without launching once that bound would pass L_b + max_new_tokens.  Other arguments, layouts and
 * errors as for cpa_decode_append; CPA_ESTATE for a plan of another kind.
 */
CPA_API int cpa_decode_append_dynamic(cpa_plan* plan, const void* q, const void* k_new, const void* v_new,
                                      const int32_t* d_active, void* k_pool, void* v_pool, void* o,
                                      void* d_workspace, void* stream);

/*
 * cpa_release_blocks -- pages on demand: every block with d_active[b] == 0 that still holds pages gives them back
 * to the reserve (device int32 [B] flags, as for cpa_decode_append_dynamic; Section 8 as cited there).  A
 * released block takes part in no later step.  Enqueued on `stream`, ordered against the decode launches of the
 * same stream.  Errors: CPA_EINVAL, CPA_ESTATE (not uploaded, or a plan of another kind), CPA_ECUDA.
 */
CPA_API int cpa_release_blocks(cpa_plan* plan, const int32_t* d_active, void* stream);

/*
 * cpa_step_mixed -- step `step` of a chunked plan's schedule (cpa_plan_create_chunked; Section 4.2 and
 * Section 6 of the paper as cited there).  If a chunk starts at this step (step = c * r), the blocks that
 * have a chunk c prefill it and cache it; the blocks whose turn it is decode one token (append fused in).
 * The two touch different blocks and run side by side: chunks one after the other on a second stream the
 * plan owns (created at the first chunk; no device memory is allocated), decode launches on `stream`.
 * `stream` waits for the chunks started so far when a block decodes its first token, and at the last
 * step of the schedule: the prefill rows of a chunk are complete on `stream` from the step in which one
 * of its blocks starts to decode, and all of them after the last step.  The first chunk is ordered behind
 * what `stream` held when step 0 was called, every later chunk behind the chunk before it and nothing else
 * (so the chunks run back to back whatever the decode steps between them take): the inputs of all chunks
 * must be complete on `stream` when step 0 is called, and must be the same buffers in every step.
 *   q, k, v, o : the packed tensors of the whole event ([total_tokens, heads, head_dim]); a chunk reads
 *                and writes only its rows, rows cu_seqlens[b] + [c * C, ...) of every block that has a
 *                chunk c.  Row i of a chunk attends over the block's
 *                cached tokens [0, c * C) and the chunk's tokens up to itself: exactly the rows
 *                cpa_prefill gives.  May be NULL in steps that start no chunk.
 *   q_dec, o_dec       : device bf16 [B, num_q_heads, head_dim]; only the rows of the decoding blocks are
 *                        read / written.  k_new, v_new: [B, num_kv_heads, head_dim] likewise.  May be
 *                        NULL in steps in which no block decodes.
 *   k_pool, v_pool, d_workspace : as for cpa_decode_append
 * Steps run in order: `step` must be the number of steps run since cpa_plan_upload (CPA_ESTATE
 * otherwise, and for a plan that is not chunked).  Errors: CPA_EINVAL, CPA_ESTATE, CPA_ECUDA.
 */
CPA_API int cpa_step_mixed(cpa_plan* plan, int32_t step, const void* q, const void* k, const void* v, void* o,
                           const void* q_dec, const void* k_new, const void* v_new, void* o_dec, void* k_pool,
                           void* v_pool, void* d_workspace, void* stream);

/*
 * cpa_step_mixed_range -- steps first_step .. first_step + num_steps - 1 of the schedule enqueued by one call
 * (cpa_step_mixed in a loop inside the library), for callers whose decode inputs of several steps are on the
 * device already.  q_dec, o_dec: device bf16 [num_steps, B, num_q_heads, head_dim], slice i for step
 * first_step + i (rows of the blocks that decode in that step, as for cpa_step_mixed); k_new, v_new likewise
 * with num_kv_heads.  Everything else and the errors as for cpa_step_mixed; a step that fails ends the range
 * (the steps before it have been enqueued).
 */
CPA_API int cpa_step_mixed_range(cpa_plan* plan, int32_t first_step, int32_t num_steps, const void* q, const void* k,
                                 const void* v, void* o, const void* q_dec, const void* k_new, const void* v_new,
                                 void* o_dec, void* k_pool, void* v_pool, void* d_workspace, void* stream);

/*
 * cpa_event_host -- a whole compaction event with inputs and outputs in HOST memory: the prefill of every
 * block (Section 4, "Dispatch": each worker runs its prompt), the append of the prompts' K/V, and
 * max_new_tokens decode steps over all blocks, each with its append (the workers' summaries, Section 4).  The
 * paper has no counterpart for the copy order; it is this library's way of hiding the PCIe transfers.
 *   h_q, h_o            : host bf16 [total_tokens, num_q_heads, head_dim]  (h_o is written)
 *   h_k, h_v            : host bf16 [total_tokens, num_kv_heads, head_dim]
 *   h_q_dec, h_o_dec    : host bf16 [max_new_tokens, B, num_q_heads, head_dim]  (step t's row of every block;
 *                         h_o_dec is written); h_k_dec, h_v_dec likewise with num_kv_heads.  May be NULL when
 *                         max_new_tokens == 0.
 *   d_stage             : device scratch, >= CPA_PARAM_HOST_STAGE_BYTES, 256-byte aligned; holds the device
 *                         copies of all eight arrays (the caller may read them there after the call)
 *   k_pool, v_pool, d_workspace : as for cpa_decode_append
 * Host buffers should be page-locked (cudaHostAlloc / cudaHostRegister): with pageable memory the copies
 * are still correct but do not overlap the kernels.  On a chunked plan (cpa_plan_create_chunked or
 * cpa_plan_create_prefix_chunked; decode_sms = 1 leaves the chunks all SMs but one) the prompts go up chunk by
 * chunk on a copy stream of the plan, chunk c of all blocks is prefilled in one launch as soon as its rows
 * have landed, and the output rows go home on another stream once the last input is up (behind the remaining
 * chunks and the decode steps); the decode steps then run for all blocks together (not the schedule of cpa_step_mixed, which this call uses up).
 * On any other plan the same steps run without overlap.  Everything is enqueued; the results are in place
 * when `stream` has been synchronised, and cpa_plan_status tells whether a kernel gave up.
 * Errors: CPA_EINVAL (null or misaligned pointer), CPA_ESTATE (plan not uploaded, or something was
 * already appended or stepped since the upload), CPA_EUNSUPPORTED (a plan with pages on demand), CPA_ECUDA.
 * After CPA_ECUDA part of the event may have been enqueued: synchronise `stream` and upload the plan again
 * before using it further.
 */
CPA_API int cpa_event_host(cpa_plan* plan, const void* h_q, const void* h_k, const void* h_v, void* h_o,
                           const void* h_q_dec, const void* h_k_dec, const void* h_v_dec, void* h_o_dec,
                           void* d_stage, void* k_pool, void* v_pool, void* d_workspace, void* stream);

/*
 * cpa_decode_static -- cpa_decode for callers that cannot hand over scratch memory.
 * (The paper has no counterpart; this is a packaging variant of cpa_decode.)
 *
 * Some hosts of this library may not allocate device memory where they decode:
 * a plugin that only gets fixed buffers from the framework around it, a service
 * whose device memory is budgeted in full at start-up, or a latency-critical
 * loop that cannot afford the device-wide synchronisation cudaMalloc and
 * cudaFree imply.  For them the split partials go to a fixed 16 MiB array
 * (CPA_STATIC_SCRATCH_BYTES) that is part of the library image on the device;
 * every GPU that loads the library keeps those 16 MiB until the process exits.
 * The call allocates and frees nothing.
 *
 * Arguments, layouts, results and errors are those of cpa_decode without
 * d_workspace, plus: CPA_ENOSPC when the plan needs more scratch than the array
 * holds (CPA_PARAM_DECODE_WORKSPACE_BYTES > CPA_STATIC_SCRATCH_BYTES); nothing is
 * launched then.  Use a smaller batch or larger pages_per_split, or cpa_decode.
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All calls
 * on a device share the one array and it keeps the previous call's contents;
 * the kernels overwrite every element they later read, so nothing needs
 * clearing, but two calls whose device work overlaps (different streams,
 * different plans) race on it: serialise them.
 */
#define CPA_STATIC_SCRATCH_BYTES (16ll << 20)
CPA_API int cpa_decode_static(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool,
                              void* o, void* stream);

/* Static text for a cpa_status value. */
CPA_API const char* cpa_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* COMPACT_ATTN_H_ */

// Internal definitions shared by the host planner and the kernel launchers.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "compact_attn.h"

// Device-side view of the uploaded index buffer.
struct cpa_dev_index {
    int32_t* status;               // [4]  word 0: first timeout/error code recorded by a kernel
    const int32_t* cu_seqlens;     // [B+1]
    const int32_t* page_indptr;    // [B+1]
    const int32_t* split_indptr;   // [B+1]
    int32_t* seq_lens;             // [B]   tokens cached per block (advanced by the append kernels)
    int32_t* seq_lens_next;        // [B]   the other length buffer: a fused decode+append writes the new lengths here
    int32_t* append_indptr;        // [B+1] source-row offsets of a general append
    const int32_t* page_indices;   // [pages_used]
    const int32_t* prefill_items;  // [n_prefill, 4]: (first token of the block, block length, q item | prefix KV tiles << 16,
                                   //   first entry of the sequence in page_indices), 16-byte aligned
    const int32_t* prefill_sched;  // [prefill_rounds, prefill_ctas]: unit (item * Hq + head) of CTA c in round k, -1 = none
    const int32_t* decode_items;   // [n_decode, item_stride]: (block, kv_head, split, pages, split size, first page of the
                                   //   split in the sequence's page list, partial slot, slots filled by the shared scan) + page ids
    const int32_t* prefix_lens;    // [B] cached prefix tokens of each sequence
    const int32_t* shared_items;   // [n_shared, 4]: (first worker | workers << 16, kv head, chunk, pages) of the shared-prefix scan
    const int32_t* shared_page_ids;// [longest prefix in pages] pool pages of the shared history
    int32_t shared_chunk;          // pages per chunk of the shared-prefix scan (0: no shared prefix)
    int32_t* merge_tickets;        // [B * Hkv] arrival counters of the fused split merge (zero between launches)
    int32_t item_stride;           // int32 words per decode item: 8 + largest split size rounded up to 4
    const int32_t* dec_start;      // [B] chunked plans: the step at which a block starts to decode
    // plans with pages on demand: page_indices is a table of B rows (row b holds page_indptr[b+1] - page_indptr[b]
    // entries, the first pages_assigned[b] of them valid) that the decode kernel extends from the reserve
    int32_t* page_table;           // page_indices again, writable
    int32_t* pages_assigned;       // [B]
    int32_t* ring_ctrl;            // [4]: pops so far (head), pushes so far (tail), ring size
    int32_t* ring;                 // [ring size] page ids of the reserve; entry i of the sequence of pushes sits at i % size
};

// Which blocks take part in a decode launch.
struct cpa_decode_mode {
    int32_t step;             // >= 0: a step of a chunked plan's schedule, block b decodes iff 0 <= step - dec_start[b] < T;
                              // -1: every block decodes
    int32_t T;                // decode steps per block (chunked plans)
    int32_t dynamic;          // pages on demand: page ids come from the table, a block that fills a page takes the next
    const int32_t* d_active;  // dynamic plans: device flags [B], block b takes part iff d_active[b] != 0; nullptr: all do
};

// One chunk of a chunked plan's prefill (chunk c of every block that has one): its items, their deal to CTAs, and
// the rows it appends.
struct cpa_chunk_step {
    int64_t off_items = 0;    // [n_items, 4] item records of the step (same format as prefill_items)
    int64_t off_sched = 0;    // [rounds, ctas]
    int64_t off_rows = 0;     // [B+1] prefix sums of the rows each block prefills in this step
    int32_t n_items = 0, ctas = 0, rounds = 0, rows = 0;
};

struct cpa_plan {
    cpa_config cfg;
    int32_t B = 0;
    int32_t T = 0;          // max_new_tokens
    int32_t num_sms = 0;    // SM budget of the plan's kernels: cfg.num_sms, or the device's SM count for 0
    int32_t q_tile = 0;     // query rows per prefill item
    int32_t C = 0;          // largest pages-per-split over the blocks
    int64_t total_tokens = 0;
    int32_t pool_pages = 0; // largest page id in the page table + 1 (extent of the pools the prefill reads a prefix from)
    std::vector<int32_t> prefix_lens;   // [B] tokens of each sequence that are cached before the plan starts (0: none)
    std::vector<int32_t> block_lens, cu_seqlens, page_indptr, page_indices, seq_lens, slot_mapping,
        prefill_items, prefill_sched, decode_items, split_indptr, split_pages;
    std::vector<int32_t> split_ranges;   // [own splits, 2] (first own page, pages) of every own split, block-major
    bool even_cut = false;               // the decode items come from the even cut of all own pages (see plan.cpp)
    int32_t decode_grid = 0;             // CTAs of a decode launch (one wave at most; the even cut fixes it exactly)
    int32_t n_prefill = 0, n_decode = 0; // n_decode: device items, fillers of the even cut included
    int32_t prefill_ctas = 0, prefill_rounds = 0;   // shape of prefill_sched
    // two-level decode of the prefix-aware layout: partial slots of each sequence that the shared-prefix
    // scan fills, its chunk size in pages, its work items and the shared pages' ids
    std::vector<int32_t> n_fixed, shared_items, shared_page_ids;
    int32_t shared_chunk = 0, n_shared = 0;
    // chunked prefill: tokens per chunk (0: none), SMs left to the decode wave while a chunk is prefilled,
    // the step at which each block starts to decode, the per-step prefill work, and the schedule's position
    int32_t chunk = 0, decode_sms = 0, n_steps = 0, next_step = 0;
    int32_t steps_per_chunk = 1;      // decode steps the schedule gives a chunk (chunk c starts at step c * steps_per_chunk)
    bool chunk_pending = false;       // a chunk has been started on the second stream and not been joined yet
    std::vector<int32_t> dec_start, chunk_rows;   // chunk_rows: [chunk steps][B+1] prefix sums of the rows a step prefills
    std::vector<cpa_chunk_step> chunk_steps;
    int64_t off_decstart = 0;
    // pages on demand: no pages are reserved for the summaries; the reserve lives in a ring in the index buffer
    bool dynamic = false;
    std::vector<int32_t> pages_assigned, free_ring;   // host mirrors (as of plan creation or the last cpa_plan_sync)
    int32_t ring_size = 0;
    int64_t off_assigned = 0, off_ringctrl = 0, off_ring = 0;
    // a mixed step runs its prefill chunk beside its decode launch: a second stream and two events, created
    // at the first mixed step on the device that is current then, destroyed with the plan
    cudaStream_t side_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // an event from host memory copies in and out on two streams of its own, ordered by events; made at the
    // first such event on the device that is current then, destroyed with the plan
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    std::vector<cudaEvent_t> host_events;

    // packed image of the device index buffer (int32 words) and offsets into it
    std::vector<int32_t> image;
    int64_t off_status = 0, off_cu = 0, off_pindptr = 0, off_sindptr = 0, off_seqlens = 0,
            off_append = 0, off_pidx = 0, off_pitems = 0, off_psched = 0, off_prefix = 0, off_shitems = 0, off_shpages = 0, off_ditems = 0, off_tickets = 0, off_seqlens2 = 0,
            words = 0;
    int cur_lens = 0;            // which of the two device length buffers is current
    int32_t item_stride = 0;
    int32_t* d_base = nullptr;   // caller's device buffer after cpa_plan_upload
    mutable uint32_t decode_calls = 0;  // decode launches so far; its parity picks the scan direction
    std::vector<int32_t> append_stage;  // host staging for general appends

    int64_t index_bytes() const { return words * 4; }
    int64_t decode_workspace_bytes() const {
        // [rows, 2] (max, sum) padded to 16 bytes, then [rows, head_dim] accumulators, fp32
        int64_t rows = (int64_t)split_indptr[B] * cfg.num_q_heads;
        int64_t bytes = ((rows * 2 + 3) / 4 * 4 + rows * cfg.head_dim) * 4;
        return (bytes + 255) / 256 * 256;
    }
    cpa_dev_index dev() const {
        cpa_dev_index d;
        d.status = d_base + off_status;
        d.cu_seqlens = d_base + off_cu;
        d.page_indptr = d_base + off_pindptr;
        d.split_indptr = d_base + off_sindptr;
        d.seq_lens = d_base + (cur_lens ? off_seqlens2 : off_seqlens);
        d.seq_lens_next = d_base + (cur_lens ? off_seqlens : off_seqlens2);
        d.append_indptr = d_base + off_append;
        d.page_indices = d_base + off_pidx;
        d.prefill_items = d_base + off_pitems;
        d.prefill_sched = d_base + off_psched;
        d.decode_items = d_base + off_ditems;
        d.prefix_lens = d_base + off_prefix;
        d.shared_items = d_base + off_shitems;
        d.shared_page_ids = d_base + off_shpages;
        d.shared_chunk = shared_chunk;
        d.merge_tickets = d_base + off_tickets;
        d.item_stride = item_stride;
        d.dec_start = d_base + off_decstart;
        d.page_table = d_base + off_pidx;
        d.pages_assigned = d_base + off_assigned;
        d.ring_ctrl = d_base + off_ringctrl;
        d.ring = d_base + off_ring;
        return d;
    }
};

// largest SM budget a plan takes (the schedule's sort keys hold a CTA id in 12 bits)
constexpr int32_t kMaxPlanSms = 4095;
// largest pages-per-split the planner produces: the decode kernel parks a split's page ids in shared memory
constexpr int32_t kMaxSplitPages = 1024;
// Which kernel scans the shared pages in the decode of the prefix-aware layout: the tensor-core one takes
// the rows of a worker group as one 128-row tile (it needs a head group size that divides 8); the
// warp-MMA one takes 64 rows.
#ifndef CPA_SCAN_ON_TENSOR_CORES
#define CPA_SCAN_ON_TENSOR_CORES 1
#endif
constexpr bool kScanOnTensorCores = CPA_SCAN_ON_TENSOR_CORES != 0;
static inline int32_t cpa_scan_rows(int32_t group) { return (kScanOnTensorCores && 8 % group == 0) ? 128 : 64; }

// largest chunk of the shared-prefix scan (its page ids are parked in shared memory too)
constexpr int32_t kMaxSharedChunkPages = 1024;

// Pool rows are stored with their 16-byte pieces permuted: piece j of the row in slot r sits at
// position cpa_pool_piece(j, r) (an involution inside every group of 8 pieces = 128 bytes).  A
// (page, head) chunk copied to shared memory as it is can then be read by the decode kernel's
// fragment pattern without bank conflicts on the V side.
__host__ __device__ static inline int cpa_pool_piece(int j, int slot) { return (j & ~7) | ((j & 7) ^ (slot & 7)); }

static inline bool cpa_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Shared-prefix scan of the prefix-aware decode on the tensor-core path (prefill_tc.cu): partials of every
// (worker, head) row for every chunk of shared pages go to part_ml / part_o.
int cpa_scan_tc(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool, float* part_ml,
                float* part_o, int wave_sms, void* stream);

// The prefill on pairs of CTAs (prefill_tc2.cu): plans whose q items have 512 rows (head_dim 128, no cached prefix).
int cpa_prefill_pairs(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, void* stream);
// Pairs of that kernel's CTAs the current device holds at a time; 0 without a device.
int cpa_prefill_pair_capacity();

// The tensor-core prefill over an explicit work list (a chunk step's items and deal); `items`, `sched` are device
// pointers into the index buffer.  cpa_prefill_tc runs the plan's whole-block list.
int cpa_prefill_tc_list(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, const void* k_pool,
                        const void* v_pool, const int32_t* items, const int32_t* sched, int ctas, int rounds, void* stream);
// Chunk c's append: rows [c * chunk, ...) of every block that has them go to the block's pages.
// device staging an event from host memory needs: q, k, v, o, then the decode steps' q, k, v, o (256-byte aligned each)
int64_t cpa_host_stage_bytes(const cpa_plan* plan);
int cpa_append_chunk(cpa_plan* plan, int chunk, const void* k, const void* v, void* k_pool, void* v_pool, void* stream);
// One decode launch (append fused in when k_new is given) over the blocks `mode` selects.
int cpa_decode_launch(const cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                      void* v_pool, void* o, void* ws, cpa_decode_mode mode, int wave_sms, void* stream);

// Host planner: partition bookkeeping for one compaction event (Section 4,
// "Snapshot & partition" and "Dispatch"): block offsets, page table, token slots
// and the CTA work lists for the prefill and decode kernels.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "cpa_internal.h"

namespace {

int64_t align4(int64_t words) { return (words + 3) / 4 * 4; }  // 16-byte alignment of every array

// SM count of the current device; 148 (a B200) when no device can be asked, so that plans can be
// built and compared on a host without one.
int32_t device_sm_count() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        (void)cudaGetLastError();
        return 148;
    }
    return sms;
}

// Deal of prefill units to the CTAs of the persistent kernel (one CTA per SM).  A unit is (item, query
// head).  Units are listed kv head by kv head, inside a kv head in item order, the G query heads of
// the group side by side: CTAs that run at the same time then stream the same few K/V ranges, which
// stay in L2.  The list is dealt in rounds of one unit per CTA: in every round the CTAs are ranked by
// the work they have so far (least first, ties to the lower CTA), the round's units by cost (largest
// first, ties in list order), and the i-th unit goes to the i-th CTA.  `item_cost[i]` is the cost of
// every unit of item i.  Returns the table [rounds][ctas] (-1 = none) and sets ctas / rounds.
std::vector<int32_t> deal_prefill_units(const std::vector<int32_t>& item_cost, int32_t Hq, int32_t G, int32_t max_ctas,
                                        int32_t* ctas_out, int32_t* rounds_out) {
    const int32_t n_items = (int32_t)item_cost.size();
    const int64_t n_units = (int64_t)n_items * Hq;
    const int32_t ctas = (int32_t)std::max<int64_t>(1, std::min<int64_t>(max_ctas, n_units));
    const int32_t rounds = (int32_t)((n_units + ctas - 1) / ctas);
    *ctas_out = ctas;
    *rounds_out = rounds;
    std::vector<int32_t> sched((size_t)rounds * (size_t)ctas, -1);
    std::vector<int64_t> load((size_t)ctas, 0);
    std::vector<uint64_t> rank((size_t)ctas), batch((size_t)ctas);   // packed sort keys
    const int64_t per_head = (int64_t)n_items * G;                    // units of one kv head
    for (int32_t r = 0; r < rounds; ++r) {
        const int64_t u0 = (int64_t)r * ctas, n = std::min<int64_t>(ctas, n_units - u0);
        for (int64_t j = 0; j < n; ++j) {
            // unit u0 + j of the list -> (kv head, item, head inside the group)
            const int64_t u = u0 + j, g = u / per_head, rem = u - g * per_head;
            const int32_t i = (int32_t)(rem / G), h = (int32_t)(rem - (int64_t)i * G);
            // descending cost, then list order: the position j breaks ties
            batch[(size_t)j] = ((uint64_t)(0xFFFFFu - (uint32_t)item_cost[(size_t)i]) << 44) | ((uint64_t)j << 32) |
                               (uint32_t)(i * Hq + (int32_t)g * G + h);
        }
        std::sort(batch.begin(), batch.begin() + n);
        for (int32_t c = 0; c < ctas; ++c) rank[(size_t)c] = ((uint64_t)load[(size_t)c] << 16) | (uint32_t)c;
        std::sort(rank.begin(), rank.end());
        for (int64_t j = 0; j < n; ++j) {
            const int32_t c = (int32_t)(rank[(size_t)j] & 0xFFFFu);
            sched[(size_t)r * (size_t)ctas + (size_t)c] = (int32_t)(batch[(size_t)j] & 0xFFFFFFFFu);
            load[(size_t)c] += 0xFFFFF - (int64_t)(batch[(size_t)j] >> 44);
        }
    }
    return sched;
}

}  // namespace

namespace {
// Both layouts: `prefix_lens` == nullptr is the independent-chunks layout (no cached prefix).
int plan_create(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens, const int32_t* prefix_lens,
                const int32_t* shared_pages, int32_t num_shared, int32_t max_new_tokens, const int32_t* free_pages,
                int32_t num_free, int32_t chunk_tokens, int32_t decode_sms, int32_t steps_per_chunk, bool dynamic,
                cpa_plan** out) {
    if (out) *out = nullptr;
    if (!cfg || !block_lens || !out || num_blocks < 1 || max_new_tokens < 0 || num_free < 0 ||
        (num_free > 0 && !free_pages) || num_shared < 0 || (num_shared > 0 && !shared_pages))
        return CPA_EINVAL;
    if (cfg->num_q_heads < 1 || cfg->num_kv_heads < 1 || cfg->num_q_heads % cfg->num_kv_heads != 0 ||
        cfg->q_tile_rows < 0 || cfg->pages_per_split < 0 || cfg->num_sms < 0 || !(cfg->scale > 0.f))
        return CPA_EINVAL;
    if ((cfg->head_dim != 64 && cfg->head_dim != 128) || cfg->page_size != 16 ||
        cfg->num_q_heads / cfg->num_kv_heads > 8)
        return CPA_EUNSUPPORTED;
    if (cfg->q_tile_rows != 0 && cfg->q_tile_rows != 128 && cfg->q_tile_rows != 256 && cfg->q_tile_rows != 512)
        return CPA_EUNSUPPORTED;
    // 512-row items run on pairs of CTAs: head_dim 128, whole blocks without cached prefix or chunks
    const bool pairs_possible = cfg->head_dim == 128 && !prefix_lens && chunk_tokens == 0 &&
                                (cfg->num_sms == 0 || cfg->num_sms >= 2);
    if (cfg->q_tile_rows == 512 && !pairs_possible) return CPA_EUNSUPPORTED;
    if (cfg->pages_per_split > kMaxSplitPages) return CPA_EUNSUPPORTED;
    // the schedule's sort keys hold a CTA id in 12 bits; the shared-scan items pack worker ranges in 16
    if (cfg->num_sms > kMaxPlanSms) return CPA_EUNSUPPORTED;
    if (prefix_lens && num_blocks > 0xFFFF) return CPA_EUNSUPPORTED;
    // a chunk is read back as a cached prefix of whole 128-key tiles
    if (chunk_tokens < 0 || chunk_tokens % 128 != 0 || decode_sms < 0 || steps_per_chunk < 1) return CPA_EINVAL;
    if (dynamic && (chunk_tokens > 0 || prefix_lens)) return CPA_EUNSUPPORTED;

    cpa_plan* p = new (std::nothrow) cpa_plan();
    if (!p) return CPA_ENOSPC;
    p->cfg = *cfg;
    p->num_sms = cfg->num_sms ? cfg->num_sms : std::min(device_sm_count(), kMaxPlanSms);
    p->B = num_blocks;
    p->T = max_new_tokens;
    p->q_tile = cfg->q_tile_rows ? cfg->q_tile_rows : 256;
    const int32_t P = cfg->page_size;
    const int32_t B = num_blocks;
    // a pool's rows (page * Hkv + head) * P + slot are 32-bit tensor-map coordinates, and a slot is page * P + offset
    const int32_t max_page_id = INT32_MAX / std::max(64, 2 * P * cfg->num_kv_heads);

    p->block_lens.assign(block_lens, block_lens + B);
    p->prefix_lens.assign(B, 0);
    if (prefix_lens) p->prefix_lens.assign(prefix_lens, prefix_lens + B);
    p->cu_seqlens.assign(B + 1, 0);
    p->page_indptr.assign(B + 1, 0);
    std::vector<int32_t> pages_per_block(B), own_pages(B);
    int64_t own_total = 0;
    for (int32_t b = 0; b < B; ++b) {
        if (block_lens[b] < 1) { delete p; return CPA_EINVAL; }
        const int32_t pre = p->prefix_lens[b];
        // a cached prefix is read in whole KV tiles of 128 keys (so also in whole pages)
        if (pre < 0 || pre % 128 != 0 || pre > (int64_t)num_shared * P) { delete p; return CPA_EINVAL; }
        // the device item record packs the q item and the prefix tile count into 16 bits each (which also
        // keeps a unit's cost far below the 20 bits the schedule's sort key gives it)
        if (pre / 128 > 0x7FFF || (block_lens[b] + 127) / 128 > 0xFFFF) { delete p; return CPA_EUNSUPPORTED; }
        int64_t cu = (int64_t)p->cu_seqlens[b] + block_lens[b];
        int64_t own = ((int64_t)block_lens[b] + max_new_tokens + P - 1) / P;
        int64_t ip = (int64_t)p->page_indptr[b] + pre / P + own;
        if (cu > INT32_MAX / 2 || ip > INT32_MAX / 64 || (int64_t)pre + block_lens[b] + max_new_tokens > INT32_MAX / 2) {
            delete p;
            return CPA_EUNSUPPORTED;
        }
        p->cu_seqlens[b + 1] = (int32_t)cu;
        p->page_indptr[b + 1] = (int32_t)ip;
        own_pages[b] = (int32_t)own;
        pages_per_block[b] = (int32_t)(pre / P + own);
        own_total += own;
    }
    p->total_tokens = p->cu_seqlens[B];
    const int32_t pages_used = p->page_indptr[B];
    // Pages on demand: a block starts with the pages for its tokens plus the next one (never more than its row of
    // the table holds); the rest of the free list is the common reserve.
    p->dynamic = dynamic;
    std::vector<int32_t> first_pages(own_pages);
    if (dynamic) {
        own_total = 0;
        for (int32_t b = 0; b < B; ++b) {
            first_pages[b] = std::min(block_lens[b] / P + 1, own_pages[b]);
            own_total += first_pages[b];
        }
        p->pages_assigned = first_pages;
    }
    if (own_total > num_free) { delete p; return CPA_ENOSPC; }
    // a sequence's pages: the shared pages of its cached prefix first, then pages of its own, dealt
    // in order from the free list
    p->page_indices.reserve((size_t)pages_used);
    int64_t taken = 0;
    for (int32_t b = 0; b < B; ++b) {
        p->page_indices.insert(p->page_indices.end(), shared_pages, shared_pages + p->prefix_lens[b] / P);
        p->page_indices.insert(p->page_indices.end(), free_pages + taken, free_pages + taken + first_pages[b]);
        p->page_indices.insert(p->page_indices.end(), (size_t)(own_pages[b] - first_pages[b]), 0);   // not assigned yet
        taken += first_pages[b];
    }
    if (dynamic) {
        p->free_ring.assign(free_pages + taken, free_pages + num_free);
        p->ring_size = std::max(1, num_free);
        for (int32_t id : p->free_ring)
            if (id < 0 || id > max_page_id) { delete p; return CPA_EINVAL; }
    }
    int32_t max_page = 0;
    for (int32_t id : p->page_indices) {
        if (id < 0 || id > max_page_id) { delete p; return CPA_EINVAL; }
        max_page = std::max(max_page, id);
    }
    p->pool_pages = max_page + 1;
    p->seq_lens = p->prefix_lens;   // the prefix is cached already

    // slot of every prefill token (positions count from the start of the sequence, prefix included)
    p->slot_mapping.resize((size_t)p->total_tokens);
    for (int32_t b = 0; b < B; ++b) {
        const int32_t* pages = p->page_indices.data() + p->page_indptr[b];
        int32_t* slots = p->slot_mapping.data() + p->cu_seqlens[b];
        for (int32_t i = 0; i < block_lens[b]; ++i) {
            const int32_t pos = p->prefix_lens[b] + i;
            slots[i] = pages[pos / P] * P + pos % P;
        }
    }

    // prefill work list: longest tiles first (later q tiles of a causal block see more keys)
    struct PItem { int32_t cost, block, tile; };
    std::vector<PItem> pit;
    for (int32_t b = 0; b < B; ++b) {
        int32_t n_tiles = (block_lens[b] + p->q_tile - 1) / p->q_tile;
        for (int32_t t = 0; t < n_tiles; ++t)
            pit.push_back({p->prefix_lens[b] + std::min((t + 1) * p->q_tile, block_lens[b]), b, t});
    }
    std::stable_sort(pit.begin(), pit.end(), [](const PItem& a, const PItem& c) {
        if (a.cost != c.cost) return a.cost > c.cost;
        if (a.block != c.block) return a.block < c.block;
        return a.tile < c.tile;
    });
    p->n_prefill = (int32_t)pit.size();
    p->prefill_items.reserve(pit.size() * 2);
    for (const PItem& it : pit) { p->prefill_items.push_back(it.block); p->prefill_items.push_back(it.tile); }

    // Prefill schedule for the persistent kernel: see deal_prefill_units.  A unit's cost is its KV tile
    // count plus a fixed part.
    {
        const int32_t Hq = cfg->num_q_heads, G = Hq / cfg->num_kv_heads;
        const int64_t n_units = (int64_t)p->n_prefill * Hq;
        if (n_units > INT32_MAX / 4) { delete p; return CPA_EUNSUPPORTED; }
        const int32_t sub_per_item = p->q_tile / 128;
        std::vector<int32_t> item_cost((size_t)p->n_prefill);
        for (int32_t i = 0; i < p->n_prefill; ++i) {
            const int32_t b = p->prefill_items[2 * i], q0 = p->prefill_items[2 * i + 1] * p->q_tile;
            if (p->q_tile == 512) {
                // a pair of CTAs runs the item: slot s covers sub-tiles 2s and 2s+1 and streams tiles 0 .. t0+2s+1
                const int32_t n_sub = std::min(4, (block_lens[b] - q0 + 127) / 128);
                int32_t steps = q0 / 128 + (n_sub > 1 ? 2 : 1);
                if (n_sub > 2) steps += q0 / 128 + (n_sub > 3 ? 4 : 3);
                item_cost[(size_t)i] = 10 * steps + 18;
                continue;
            }
            const int32_t n_sub = (sub_per_item > 1 && block_lens[b] - q0 > 128) ? 2 : 1;
            item_cost[(size_t)i] = 10 * (p->prefix_lens[b] / 128 + q0 / 128 + n_sub) + 18;
        }
        // one schedule column per CTA, or per pair of CTAs for 512-row items (as many pairs as the device holds at
        // a time, when there is a device to ask)
        int32_t workers = p->num_sms;
        if (p->q_tile == 512) {
            workers = p->num_sms / 2;
            const int32_t cap = cpa_prefill_pair_capacity();
            if (cap > 0 && cfg->num_sms == 0) workers = std::min(workers, cap);
        }
        p->prefill_sched = deal_prefill_units(item_cost, Hq, G, workers, &p->prefill_ctas, &p->prefill_rounds);
    }

    // Decode splits.  Every CTA pays a fixed start-up and merge cost, so the planner aims at
    // ONE wave of resident CTAs (three per SM): starting from one split per block, it keeps
    // splitting the block whose splits are largest while the item count (kv heads x splits)
    // still fits.  split_pages[b] is the page count of block b's splits (the last may be
    // shorter).  A fixed pages_per_split from the configuration overrides the search.
    //
    // Prefix-aware layout: the cached prefixes are shared pages, and reading them once per worker
    // would multiply the traffic by about half the worker count.  They are scanned by a kernel of
    // their own instead: the shared pages are cut into chunks of `shared_chunk` pages, workers are
    // grouped (as many consecutive workers as give 128 (worker, head) rows per kv head), and one
    // item = (group, kv head, chunk) computes a partial for every worker of the group whose prefix
    // reaches into the chunk.  Worker b gets ceil(prefix pages / shared_chunk) partial slots for
    // them in front of the slots of its own splits, which cover its own pages only.
    bool two_level = false;
    int32_t max_pre_pages = 0;
    for (int32_t b = 0; b < B; ++b) max_pre_pages = std::max(max_pre_pages, p->prefix_lens[b] / P);
    two_level = max_pre_pages > 0;
    std::vector<int32_t> dec_pages(pages_per_block);   // pages the per-block splits cover
    p->n_fixed.assign(B, 0);
    p->shared_chunk = 0;
    if (two_level) {
        const int32_t G = cfg->num_q_heads / cfg->num_kv_heads;
        const int32_t per_group = cpa_scan_rows(G) / G;                     // workers per group
        const int32_t n_groups = (B + per_group - 1) / per_group;
        const int64_t sms = p->num_sms;
        const int64_t want = std::max<int64_t>(1, 3 * sms / ((int64_t)cfg->num_kv_heads * n_groups));   // chunks per (group, head)
        int64_t ch = (max_pre_pages + want - 1) / want;
        ch = std::min<int64_t>(kMaxSharedChunkPages, std::max<int64_t>(8, (ch + 7) / 8 * 8));   // whole 128-key tiles
        p->shared_chunk = (int32_t)ch;
        for (int32_t b = 0; b < B; ++b) {
            dec_pages[b] = pages_per_block[b] - p->prefix_lens[b] / P;
            p->n_fixed[b] = (p->prefix_lens[b] / P + p->shared_chunk - 1) / p->shared_chunk;
        }
        for (int32_t r = 0; r < n_groups; ++r) {
            const int32_t w0 = r * per_group, nw = std::min(per_group, B - w0);
            int32_t reach = 0;
            for (int32_t b = w0; b < w0 + nw; ++b) reach = std::max(reach, p->prefix_lens[b] / P);
            for (int32_t c = 0; c * p->shared_chunk < reach; ++c)
                for (int32_t g = 0; g < cfg->num_kv_heads; ++g) {
                    p->shared_items.push_back(w0 | (nw << 16));
                    p->shared_items.push_back(g);
                    p->shared_items.push_back(c);
                    p->shared_items.push_back(std::min(p->shared_chunk, reach - c * p->shared_chunk));
                }
        }
        p->shared_page_ids.assign(shared_pages, shared_pages + max_pre_pages);
    }
    p->n_shared = (int32_t)(p->shared_items.size() / 4);
    p->split_pages.assign(B, 0);
    std::vector<int32_t> n_splits(B, 1);
    if (cfg->pages_per_split > 0) {
        for (int32_t b = 0; b < B; ++b) p->split_pages[b] = cfg->pages_per_split;
    } else {
        const int64_t slots = 3LL * p->num_sms;
        int64_t items = (int64_t)B * cfg->num_kv_heads;
        while (items + cfg->num_kv_heads <= slots) {
            int32_t best = -1;
            int32_t best_size = 4;  // never split below 4 pages
            for (int32_t b = 0; b < B; ++b) {
                const int32_t size = (dec_pages[b] + n_splits[b] - 1) / n_splits[b];
                if (size > best_size) { best_size = size; best = b; }
            }
            if (best < 0) break;
            ++n_splits[best];
            items += cfg->num_kv_heads;
        }
        for (int32_t b = 0; b < B; ++b) {
            int32_t size = (dec_pages[b] + n_splits[b] - 1) / n_splits[b];
            p->split_pages[b] = std::min(size, kMaxSplitPages);
        }
    }
    // The uniform cut: block b in splits of split_pages[b] pages, one item per (block, kv head, split), largest first.
    struct DItem { int32_t pages, block, head, split, first; };   // first: first own page of the split; block < 0: filler
    auto uniform_items = [&]() {
        std::vector<DItem> v;
        for (int32_t b = 0; b < B; ++b) {
            const int32_t Cb = p->split_pages[b];
            const int32_t ns = (dec_pages[b] + Cb - 1) / Cb;
            for (int32_t g = 0; g < cfg->num_kv_heads; ++g)
                for (int32_t s2 = 0; s2 < ns; ++s2)
                    v.push_back({std::min(Cb, dec_pages[b] - s2 * Cb), b, g, s2, s2 * Cb});
        }
        std::stable_sort(v.begin(), v.end(), [](const DItem& x, const DItem& y) {
            if (x.pages != y.pages) return x.pages > y.pages;
            if (x.block != y.block) return x.block < y.block;
            if (x.head != y.head) return x.head < y.head;
            return x.split < y.split;
        });
        return v;
    };
    // What a launch costs with a given item list: CTA c takes items c, c + grid, ...; CTA c runs on SM c mod num_sms
    // (three to an SM), which shares its bandwidth between them; every item also pays a fixed cost, the CTA's ring of
    // stages running empty and filling again plus the merge, worth about sixteen pages of streaming (measured: a
    // second item in a CTA costs about 9 us where a CTA streams 1.8 pages per us).  The figure is the load of the
    // busiest SM.
    auto busiest_sm = [&](const std::vector<DItem>& v, int64_t grid) {
        std::vector<int64_t> load((size_t)p->num_sms, 0);
        for (size_t i = 0; i < v.size(); ++i)
            if (v[i].block >= 0) load[(size_t)(((int64_t)i % grid) % p->num_sms)] += v[i].pages + 16;
        return *std::max_element(load.begin(), load.end());
    };
    std::vector<DItem> dit = uniform_items();
    // The even cut (only when the split size is the planner's choice): all own pages of all blocks, laid end to end,
    // are cut into equal ranges of `cut` pages, one range per group of kv_heads CTAs, so that every CTA of the wave
    // streams the same number of pages whatever the blocks' lengths; a range that crosses a block boundary becomes
    // two items of its CTAs.  Block b then has a first split that ends at the next cut, full splits behind it and a
    // remainder.  Taken when the busiest SM gets at least 5 % less than with the uniform cut, which happens when
    // there are more (block, kv head) pairs than CTAs in a wave, so that some CTAs would run two whole items.
    p->even_cut = false;
    if (cfg->pages_per_split == 0) {
        int64_t total = 0;
        for (int32_t b = 0; b < B; ++b) total += dec_pages[b];
        const int64_t groups = std::max<int64_t>(1, 3LL * p->num_sms / cfg->num_kv_heads);
        const int64_t cut = std::min<int64_t>(kMaxSplitPages, std::max<int64_t>(4, (total + groups - 1) / groups));
        const int64_t n_ranges = (total + cut - 1) / cut;
        const int64_t workers = std::min(groups, n_ranges);          // groups of kv_heads CTAs
        std::vector<std::vector<DItem>> per_worker((size_t)workers);
        // a block's first split is not left shorter than `least` pages: it takes the following range's pages along
        // (that range's CTAs then stream up to `least` pages more than the others)
        const int32_t least = cut + cut / 16 + 2 <= kMaxSplitPages ? (int32_t)std::max<int64_t>(2, cut / 16) : 0;
        int64_t off = 0;
        for (int32_t b = 0; b < B; ++b) {
            int32_t pos = 0, s2 = 0;
            while (pos < dec_pages[b]) {
                int64_t range = (off + pos) / cut;
                int32_t len = (int32_t)std::min<int64_t>(dec_pages[b] - pos, (range + 1) * cut - (off + pos));
                if (s2 == 0 && len < least && dec_pages[b] > len) {
                    ++range;
                    len = (int32_t)std::min<int64_t>(dec_pages[b], (range + 1) * cut - off);
                }
                per_worker[(size_t)(range % workers)].push_back({len, b, 0, s2, pos});
                pos += len;
                ++s2;
            }
            off += dec_pages[b];
        }
        size_t rounds = 0;
        for (const auto& w : per_worker) rounds = std::max(rounds, w.size());
        std::vector<DItem> even;
        even.reserve(rounds * (size_t)workers * (size_t)cfg->num_kv_heads);
        for (size_t k = 0; k < rounds; ++k)
            for (int64_t w = 0; w < workers; ++w)
                for (int32_t g = 0; g < cfg->num_kv_heads; ++g) {
                    if (k < per_worker[(size_t)w].size()) {
                        DItem it = per_worker[(size_t)w][k];
                        it.head = g;
                        even.push_back(it);
                    } else {
                        even.push_back({0, -1, g, -1, 0});     // this CTA has nothing in this round
                    }
                }
        p->decode_grid = (int32_t)std::min<int64_t>((int64_t)dit.size(), 3LL * p->num_sms);
        if (busiest_sm(even, workers * cfg->num_kv_heads) * 100 < busiest_sm(dit, p->decode_grid) * 95) {
            p->even_cut = true;
            p->decode_grid = (int32_t)(workers * cfg->num_kv_heads);
            dit.swap(even);
            for (int32_t b = 0; b < B; ++b) p->split_pages[b] = (int32_t)cut;
        }
    }
    if (!p->even_cut) p->decode_grid = (int32_t)std::min<int64_t>((int64_t)dit.size(), 3LL * p->num_sms);
    p->C = *std::max_element(p->split_pages.begin(), p->split_pages.end());
    p->split_indptr.assign(B + 1, 0);
    {
        std::vector<int32_t> n_own_splits(B, 0);
        for (const DItem& it : dit)
            if (it.block >= 0 && it.head == 0) n_own_splits[it.block] = std::max(n_own_splits[it.block], it.split + 1);
        for (int32_t b = 0; b < B; ++b) p->split_indptr[b + 1] = p->split_indptr[b] + p->n_fixed[b] + n_own_splits[b];
        // (first own page, pages) of every own split, block-major
        p->split_ranges.assign((size_t)2 * (size_t)(p->split_indptr[B]), 0);
        for (const DItem& it : dit)
            if (it.block >= 0 && it.head == 0) {
                const size_t at = (size_t)2 * (size_t)(p->split_indptr[it.block] + p->n_fixed[it.block] + it.split);
                p->split_ranges[at] = it.first;
                p->split_ranges[at + 1] = it.pages;
            }
    }
    p->n_decode = (int32_t)dit.size();
    p->decode_items.reserve(dit.size() * 3);
    for (const DItem& it : dit) {
        if (it.block < 0) continue;      // the host's list names the real items, in launch order
        p->decode_items.push_back(it.block);
        p->decode_items.push_back(it.head);
        p->decode_items.push_back(it.split);
    }

    // Chunked prefill: chunk c of a block, rows [c*C, min((c+1)*C, L_b)), starts at step c*r (r = steps_per_chunk: a
    // chunk is given the time of r decode steps) and reads the block's earlier chunks from its pages exactly like a
    // cached prefix; a block decodes in the T steps from step n_b*r on.  Every chunk index gets its own item list
    // and deal.  While some block decodes during a chunk's r steps, the chunk's persistent grid leaves
    // `decode_sms` SMs to the decode wave that runs beside it.
    std::vector<int32_t> chunk_items, chunk_sched, chunk_rows;
    if (chunk_tokens > 0) {
        const int32_t Cc = chunk_tokens, Hq = cfg->num_q_heads, G = Hq / cfg->num_kv_heads, r = steps_per_chunk;
        p->chunk = Cc;
        p->steps_per_chunk = r;
        p->decode_sms = decode_sms ? decode_sms : std::max(1, p->num_sms / 4);
        if (p->decode_sms >= p->num_sms) { delete p; return CPA_EINVAL; }
        p->dec_start.assign(B, 0);
        int32_t n_chunk_steps = 0;
        std::vector<int32_t> n_chunks(B);
        for (int32_t b = 0; b < B; ++b) {
            n_chunks[b] = (block_lens[b] + Cc - 1) / Cc;
            if ((int64_t)n_chunks[b] * r + max_new_tokens > INT32_MAX / 2) { delete p; return CPA_EUNSUPPORTED; }
            p->dec_start[b] = n_chunks[b] * r;
            n_chunk_steps = std::max(n_chunk_steps, n_chunks[b]);
        }
        p->n_steps = n_chunk_steps * r + max_new_tokens;
        p->chunk_steps.resize((size_t)n_chunk_steps);
        for (int32_t st = 0; st < n_chunk_steps; ++st) {
            cpa_chunk_step& cs = p->chunk_steps[(size_t)st];
            bool any_decode = false;   // does some block decode during the r steps of this chunk?
            for (int32_t b = 0; b < B; ++b)
                any_decode |= p->dec_start[b] < (st + 1) * r && st * r < p->dec_start[b] + max_new_tokens;
            std::vector<PItem> cit;
            cs.off_rows = (int64_t)chunk_rows.size();
            int32_t rows = 0;
            for (int32_t b = 0; b < B; ++b) {
                chunk_rows.push_back(rows);
                if (st >= n_chunks[b]) continue;
                const int32_t len = std::min(Cc, block_lens[b] - st * Cc);
                rows += len;
                for (int32_t t = 0; t * p->q_tile < len; ++t)
                    cit.push_back({p->prefix_lens[b] + st * Cc + std::min((t + 1) * p->q_tile, len), b, t});
            }
            chunk_rows.push_back(rows);
            cs.rows = rows;
            std::stable_sort(cit.begin(), cit.end(), [](const PItem& a, const PItem& c) {
                if (a.cost != c.cost) return a.cost > c.cost;
                if (a.block != c.block) return a.block < c.block;
                return a.tile < c.tile;
            });
            cs.n_items = (int32_t)cit.size();
            cs.off_items = (int64_t)chunk_items.size();
            std::vector<int32_t> item_cost(cit.size());
            for (size_t i = 0; i < cit.size(); ++i) {
                const int32_t b = cit[i].block, q0 = cit[i].tile * p->q_tile;
                const int32_t len = std::min(Cc, block_lens[b] - st * Cc);
                const int32_t n_sub = (p->q_tile > 128 && len - q0 > 128) ? 2 : 1;
                // the chunk is a "block" of its own whose cached prefix is the sequence's cached history (prefix-aware
                // layout) followed by the block's earlier chunks
                const int32_t pre_tiles = (p->prefix_lens[b] + st * Cc) / 128;
                if (pre_tiles > 0x7FFF) { delete p; return CPA_EUNSUPPORTED; }
                item_cost[i] = 10 * (pre_tiles + q0 / 128 + n_sub) + 18;
                chunk_items.push_back(p->cu_seqlens[b] + st * Cc);
                chunk_items.push_back(len);
                chunk_items.push_back(cit[i].tile | (pre_tiles << 16));
                chunk_items.push_back(p->page_indptr[b]);
            }
            const int32_t budget = any_decode ? p->num_sms - p->decode_sms : p->num_sms;
            std::vector<int32_t> sched = deal_prefill_units(item_cost, Hq, G, budget, &cs.ctas, &cs.rounds);
            cs.off_sched = (int64_t)chunk_sched.size();
            chunk_sched.insert(chunk_sched.end(), sched.begin(), sched.end());
        }
    }

    // device image
    int64_t w = 0;
    p->off_status = w;  w = align4(w + 4);
    p->off_cu = w;      w = align4(w + B + 1);
    p->off_pindptr = w; w = align4(w + B + 1);
    p->off_sindptr = w; w = align4(w + B + 1);
    p->off_seqlens = w; w = align4(w + B);
    p->off_append = w;  w = align4(w + B + 1);
    p->off_pidx = w;    w = align4(w + pages_used);
    p->off_pitems = w;  w = align4(w + 4LL * p->n_prefill);
    p->off_psched = w;  w = align4(w + (int64_t)p->prefill_sched.size());
    int32_t most_pages = p->C;      // (a first split of the even cut may be a little longer than the cut)
    for (const DItem& it : dit) most_pages = std::max(most_pages, it.pages);
    p->item_stride = 8 + (most_pages + 3) / 4 * 4;
    p->off_ditems = w;  w = align4(w + (int64_t)p->item_stride * p->n_decode);
    p->off_tickets = w; w = align4(w + (int64_t)B * cfg->num_kv_heads);
    p->off_seqlens2 = w; w = align4(w + B);
    p->off_prefix = w;  w = align4(w + B);
    p->off_shitems = w; w = align4(w + (int64_t)p->shared_items.size());
    p->off_shpages = w; w = align4(w + (int64_t)p->shared_page_ids.size());
    p->off_decstart = w; w = align4(w + (int64_t)p->dec_start.size());
    p->off_assigned = w; w = align4(w + (int64_t)p->pages_assigned.size());
    p->off_ringctrl = w; w = align4(w + (dynamic ? 4 : 0));
    p->off_ring = w;     w = align4(w + (dynamic ? p->ring_size : 0));
    const int64_t off_citems = w; w = align4(w + (int64_t)chunk_items.size());
    const int64_t off_csched = w; w = align4(w + (int64_t)chunk_sched.size());
    const int64_t off_crows = w;  w = align4(w + (int64_t)chunk_rows.size());
    for (cpa_chunk_step& cs : p->chunk_steps) { cs.off_items += off_citems; cs.off_sched += off_csched; cs.off_rows += off_crows; }
    p->chunk_rows = chunk_rows;
    p->words = w;
    p->image.assign((size_t)w, 0);
    int32_t* im = p->image.data();
    std::memcpy(im + p->off_cu, p->cu_seqlens.data(), sizeof(int32_t) * (B + 1));
    std::memcpy(im + p->off_pindptr, p->page_indptr.data(), sizeof(int32_t) * (B + 1));
    std::memcpy(im + p->off_sindptr, p->split_indptr.data(), sizeof(int32_t) * (B + 1));
    std::memcpy(im + p->off_pidx, p->page_indices.data(), sizeof(int32_t) * pages_used);
    for (int32_t i = 0; i < p->n_prefill; ++i) {
        // a prefill item carries its block's token range and cached prefix (one 16-byte record), so a
        // kernel needs no dependent loads per item
        const int32_t b = p->prefill_items[2 * i];
        int32_t* it = im + p->off_pitems + 4LL * i;
        it[0] = p->cu_seqlens[b];                                             // first token of the block
        it[1] = p->block_lens[b];
        it[2] = p->prefill_items[2 * i + 1] | ((p->prefix_lens[b] / 128) << 16);   // q item, KV tiles of the cached prefix
        it[3] = p->page_indptr[b];                                            // where the sequence's page ids start
    }
    for (int32_t b = 0; b < B; ++b) im[p->off_seqlens + b] = im[p->off_seqlens2 + b] = p->prefix_lens[b];
    std::memcpy(im + p->off_psched, p->prefill_sched.data(), sizeof(int32_t) * p->prefill_sched.size());
    std::memcpy(im + p->off_prefix, p->prefix_lens.data(), sizeof(int32_t) * B);
    if (dynamic) {
        std::memcpy(im + p->off_assigned, p->pages_assigned.data(), sizeof(int32_t) * B);
        im[p->off_ringctrl + 0] = 0;                                 // pops so far
        im[p->off_ringctrl + 1] = (int32_t)p->free_ring.size();      // pushes so far
        im[p->off_ringctrl + 2] = p->ring_size;
        if (!p->free_ring.empty())
            std::memcpy(im + p->off_ring, p->free_ring.data(), sizeof(int32_t) * p->free_ring.size());
    }
    if (!p->dec_start.empty()) {
        std::memcpy(im + p->off_decstart, p->dec_start.data(), sizeof(int32_t) * p->dec_start.size());
        std::memcpy(im + off_citems, chunk_items.data(), sizeof(int32_t) * chunk_items.size());
        std::memcpy(im + off_csched, chunk_sched.data(), sizeof(int32_t) * chunk_sched.size());
        std::memcpy(im + off_crows, chunk_rows.data(), sizeof(int32_t) * chunk_rows.size());
    }
    if (!p->shared_items.empty()) {
        std::memcpy(im + p->off_shitems, p->shared_items.data(), sizeof(int32_t) * p->shared_items.size());
        std::memcpy(im + p->off_shpages, p->shared_page_ids.data(), sizeof(int32_t) * p->shared_page_ids.size());
    }
    for (int32_t i = 0; i < p->n_decode; ++i) {
        // a decode item carries its own page ids, so the kernel's first KV load depends on
        // one prior load only
        int32_t* it = im + p->off_ditems + (int64_t)p->item_stride * i;
        if (dit[i].block < 0) {          // filler: no pages, belongs to nobody (split -1 never takes a block's chores)
            it[0] = 0; it[1] = dit[i].head; it[2] = -1; it[3] = 0; it[4] = 1; it[5] = 0; it[6] = 0; it[7] = 0;
            continue;
        }
        it[0] = dit[i].block;
        it[1] = dit[i].head;
        it[2] = dit[i].split;
        it[3] = dit[i].pages;
        it[4] = p->split_pages[dit[i].block];
        // where the split starts inside the sequence's page list (behind the pages the shared scan
        // covers), its partial slot among the sequence's slots, and how many slots come before
        const int32_t skip = two_level ? p->prefix_lens[dit[i].block] / P : 0;
        it[5] = skip + dit[i].first;
        it[6] = p->n_fixed[dit[i].block] + dit[i].split;
        it[7] = p->n_fixed[dit[i].block];
        const int32_t* src = p->page_indices.data() + p->page_indptr[dit[i].block] + it[5];
        for (int32_t j = 0; j < dit[i].pages; ++j) it[8 + j] = src[j];
    }
    p->append_stage.assign(B + 1, 0);
    *out = p;
    return CPA_OK;
}
}  // namespace

extern "C" int cpa_partition(int64_t history_tokens, int32_t block_tokens, int32_t* block_lens, int32_t capacity,
                             int32_t* num_blocks) {
    if (history_tokens < 1 || block_tokens < 1 || !num_blocks || capacity < 0 || (capacity > 0 && !block_lens))
        return CPA_EINVAL;
    const int64_t n = (history_tokens + block_tokens - 1) / block_tokens;
    if (n > INT32_MAX) return CPA_EUNSUPPORTED;
    *num_blocks = (int32_t)n;
    if (n > capacity) return CPA_ENOSPC;
    for (int64_t i = 0; i + 1 < n; ++i) block_lens[i] = block_tokens;
    block_lens[n - 1] = (int32_t)(history_tokens - (n - 1) * block_tokens);   // the last block may be short
    return CPA_OK;
}

extern "C" int cpa_plan_create(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                               int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                               cpa_plan** out) {
    return plan_create(cfg, num_blocks, block_lens, nullptr, nullptr, 0, max_new_tokens, free_pages, num_free, 0, 0, 1, false, out);
}

extern "C" int cpa_plan_create_dynamic(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                                       int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                                       cpa_plan** out) {
    return plan_create(cfg, num_blocks, block_lens, nullptr, nullptr, 0, max_new_tokens, free_pages, num_free, 0, 0, 1, true,
                       out);
}

extern "C" int cpa_plan_sync(cpa_plan* plan, void* stream) {
    if (!plan) return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    cudaStream_t st = (cudaStream_t)stream;
    const int B = plan->B;
    std::vector<int32_t> ctrl(4, 0), ring((size_t)plan->ring_size, 0);
    bool ok = cudaMemcpyAsync(plan->seq_lens.data(), plan->d_base + (plan->cur_lens ? plan->off_seqlens2 : plan->off_seqlens),
                              sizeof(int32_t) * B, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (ok && plan->dynamic) {
        ok = cudaMemcpyAsync(plan->page_indices.data(), plan->d_base + plan->off_pidx,
                             sizeof(int32_t) * plan->page_indices.size(), cudaMemcpyDeviceToHost, st) == cudaSuccess &&
             cudaMemcpyAsync(plan->pages_assigned.data(), plan->d_base + plan->off_assigned, sizeof(int32_t) * B,
                             cudaMemcpyDeviceToHost, st) == cudaSuccess &&
             cudaMemcpyAsync(ctrl.data(), plan->d_base + plan->off_ringctrl, sizeof(int32_t) * 4, cudaMemcpyDeviceToHost,
                             st) == cudaSuccess &&
             cudaMemcpyAsync(ring.data(), plan->d_base + plan->off_ring, sizeof(int32_t) * ring.size(),
                             cudaMemcpyDeviceToHost, st) == cudaSuccess;
    }
    if (ok) ok = cudaStreamSynchronize(st) == cudaSuccess;
    if (!ok) { (void)cudaGetLastError(); return CPA_ECUDA; }
    if (plan->dynamic) {
        plan->free_ring.clear();
        for (int32_t i = ctrl[0]; i < ctrl[1]; ++i) plan->free_ring.push_back(ring[(size_t)(i % plan->ring_size)]);
    }
    return CPA_OK;
}

extern "C" int cpa_plan_create_chunked(const cpa_config* cfg, int32_t num_blocks, const int32_t* block_lens,
                                       int32_t max_new_tokens, int32_t chunk_tokens, int32_t decode_steps_per_chunk,
                                       int32_t decode_sms, const int32_t* free_pages, int32_t num_free,
                                       cpa_plan** out) {
    if (out) *out = nullptr;
    if (chunk_tokens < 128) return CPA_EINVAL;
    return plan_create(cfg, num_blocks, block_lens, nullptr, nullptr, 0, max_new_tokens, free_pages, num_free,
                       chunk_tokens, decode_sms, decode_steps_per_chunk, false, out);
}

extern "C" int cpa_plan_create_prefix(const cpa_config* cfg, int32_t num_workers, const int32_t* own_lens,
                                      const int32_t* prefix_lens, const int32_t* shared_pages, int32_t num_shared,
                                      int32_t max_new_tokens, const int32_t* free_pages, int32_t num_free,
                                      cpa_plan** out) {
    if (out) *out = nullptr;
    if (!prefix_lens) return CPA_EINVAL;
    return plan_create(cfg, num_workers, own_lens, prefix_lens, shared_pages, num_shared, max_new_tokens, free_pages,
                       num_free, 0, 0, 1, false, out);
}

extern "C" int cpa_plan_create_prefix_chunked(const cpa_config* cfg, int32_t num_workers, const int32_t* own_lens,
                                              const int32_t* prefix_lens, const int32_t* shared_pages, int32_t num_shared,
                                              int32_t max_new_tokens, int32_t chunk_tokens, int32_t decode_steps_per_chunk,
                                              int32_t decode_sms, const int32_t* free_pages, int32_t num_free,
                                              cpa_plan** out) {
    if (out) *out = nullptr;
    if (!prefix_lens || chunk_tokens < 128) return CPA_EINVAL;
    return plan_create(cfg, num_workers, own_lens, prefix_lens, shared_pages, num_shared, max_new_tokens, free_pages,
                       num_free, chunk_tokens, decode_sms, decode_steps_per_chunk, false, out);
}

extern "C" int cpa_plan_export(const cpa_plan* plan, int which, const int32_t** ptr, int64_t* count) {
    if (!plan || !ptr || !count) return CPA_EINVAL;
    const std::vector<int32_t>* v = nullptr;
    int64_t div = 1;
    switch (which) {
        case CPA_ARR_CU_SEQLENS: v = &plan->cu_seqlens; break;
        case CPA_ARR_PAGE_INDPTR: v = &plan->page_indptr; break;
        case CPA_ARR_PAGE_INDICES: v = &plan->page_indices; break;
        case CPA_ARR_SEQ_LENS: v = &plan->seq_lens; break;
        case CPA_ARR_SLOT_MAPPING: v = &plan->slot_mapping; break;
        case CPA_ARR_PREFILL_ITEMS: v = &plan->prefill_items; div = 2; break;
        case CPA_ARR_DECODE_ITEMS: v = &plan->decode_items; div = 3; break;
        case CPA_ARR_SPLIT_INDPTR: v = &plan->split_indptr; break;
        case CPA_ARR_SPLIT_PAGES: v = &plan->split_pages; break;
        case CPA_ARR_PREFILL_SCHED: v = &plan->prefill_sched; break;
        case CPA_ARR_DEC_START: v = &plan->dec_start; break;
        case CPA_ARR_CHUNK_ROWS: v = &plan->chunk_rows; break;
        case CPA_ARR_PAGES_ASSIGNED: v = &plan->pages_assigned; break;
        case CPA_ARR_FREE_RING: v = &plan->free_ring; break;
        case CPA_ARR_SPLIT_RANGES: v = &plan->split_ranges; div = 2; break;
        default: return CPA_EINVAL;
    }
    *ptr = v->data();
    *count = (int64_t)v->size() / div;
    return CPA_OK;
}

extern "C" int64_t cpa_plan_param(const cpa_plan* plan, int which) {
    if (!plan) return CPA_EINVAL;
    switch (which) {
        case CPA_PARAM_NUM_BLOCKS: return plan->B;
        case CPA_PARAM_TOTAL_TOKENS: return plan->total_tokens;
        case CPA_PARAM_Q_TILE_ROWS: return plan->q_tile;
        case CPA_PARAM_PAGES_PER_SPLIT: return plan->C;
        case CPA_PARAM_PAGES_USED: {
            if (!plan->dynamic) return plan->page_indptr[plan->B];
            int64_t n = 0;
            for (int32_t a : plan->pages_assigned) n += a;
            return n;
        }
        case CPA_PARAM_INDEX_BYTES: return plan->index_bytes();
        case CPA_PARAM_DECODE_WORKSPACE_BYTES: return plan->decode_workspace_bytes();
        case CPA_PARAM_TOTAL_SPLITS: return plan->split_indptr[plan->B];
        case CPA_PARAM_MAX_NEW_TOKENS: return plan->T;
        case CPA_PARAM_PREFILL_CTAS: return plan->prefill_ctas;
        case CPA_PARAM_SHARED_CHUNK_PAGES: return plan->shared_chunk;
        case CPA_PARAM_CHUNK_TOKENS: return plan->chunk;
        case CPA_PARAM_NUM_STEPS: return plan->n_steps;
        case CPA_PARAM_CHUNK_STEPS: return (int64_t)plan->chunk_steps.size();
        case CPA_PARAM_DECODE_SMS: return plan->decode_sms;
        case CPA_PARAM_NUM_SMS: return plan->num_sms;
        case CPA_PARAM_DECODE_STEPS_PER_CHUNK: return plan->steps_per_chunk;
        case CPA_PARAM_DECODE_EVEN_CUT: return plan->even_cut ? 1 : 0;
        case CPA_PARAM_DECODE_CTAS: return plan->decode_grid;
        case CPA_PARAM_HOST_STAGE_BYTES: return cpa_host_stage_bytes(plan);
        default: return CPA_EINVAL;
    }
}

extern "C" int cpa_plan_upload(cpa_plan* plan, void* d_index_buf, int64_t bytes, void* stream) {
    if (!plan || !d_index_buf || !cpa_aligned16(d_index_buf)) return CPA_EINVAL;
    if (bytes < plan->index_bytes()) return CPA_ENOSPC;
    // the device copy starts with nothing but the cached prefixes, so the host mirror does too
    plan->seq_lens = plan->prefix_lens;
    plan->cur_lens = 0;
    plan->next_step = 0;
    plan->chunk_pending = false;
    if (plan->dynamic) {   // the device starts from the plan's first assignment again, and so do the host mirrors
        const int32_t* im = plan->image.data();
        plan->page_indices.assign(im + plan->off_pidx, im + plan->off_pidx + plan->page_indices.size());
        plan->pages_assigned.assign(im + plan->off_assigned, im + plan->off_assigned + plan->B);
        plan->free_ring.assign(im + plan->off_ring, im + plan->off_ring + im[plan->off_ringctrl + 1]);
    }
    cudaError_t e = cudaMemcpyAsync(d_index_buf, plan->image.data(), (size_t)plan->index_bytes(),
                                    cudaMemcpyHostToDevice, (cudaStream_t)stream);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
    plan->d_base = static_cast<int32_t*>(d_index_buf);
    return CPA_OK;
}

extern "C" int cpa_plan_status(cpa_plan* plan, void* stream) {
    if (!plan) return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    int32_t word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, plan->d_base + plan->off_status, sizeof(word),
                                    cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
    // the first code a kernel recorded: 1 = a bounded wait gave up, 2 = an append found no room
    return word == 0 ? CPA_OK : word == 2 ? CPA_ENOSPC : CPA_ETIMEOUT;
}

extern "C" void cpa_plan_destroy(cpa_plan* plan) {
    if (!plan) return;
    if (plan->ev_fork) cudaEventDestroy(plan->ev_fork);
    if (plan->ev_join) cudaEventDestroy(plan->ev_join);
    if (plan->side_stream) cudaStreamDestroy(plan->side_stream);
    for (cudaEvent_t e : plan->host_events) cudaEventDestroy(e);
    if (plan->in_stream) cudaStreamDestroy(plan->in_stream);
    if (plan->out_stream) cudaStreamDestroy(plan->out_stream);
    (void)cudaGetLastError();
    delete plan;
}

extern "C" const char* cpa_strerror(int status) {
    switch (status) {
        case CPA_OK: return "ok";
        case CPA_EINVAL: return "invalid argument";
        case CPA_ENOSPC: return "not enough pages or buffer space";
        case CPA_EUNSUPPORTED: return "unsupported configuration";
        case CPA_ECUDA: return "CUDA call failed";
        case CPA_ETIMEOUT: return "a bounded device-side wait gave up";
        case CPA_ESTATE: return "call order violated";
        default: return "unknown status";
    }
}

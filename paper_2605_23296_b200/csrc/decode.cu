// Batched paged-KV decode attention: one query token per block over that block's
// pages, split over the KV length, then a log-sum-exp merge of the split partials.
//
// The step is a streaming scan of the KV pool and is bound by HBM bandwidth: every K
// and V element is read once per kv head.  A (page, kv head) chunk of the pool is
// contiguous (16 keys x head_dim bf16), so it moves with ONE bulk asynchronous copy
// (cp.async.bulk, global -> shared, completion counted on an mbarrier).  Each warp
// owns a ring of stages in shared memory and keeps several pages in flight without
// spending registers or L1 miss slots on them; that depth, not arithmetic, decides
// the bandwidth reached.
//
// The per-key arithmetic runs on the warp-level MMA (m16n8k16, bf16 in, fp32
// accumulate), which costs nothing next to the memory stream and keeps the fp32 ALU
// free at G = 8; the G query heads of a kv-head group share every byte read:
//   S  [heads(16, G used) x keys(8)]   = Q [heads x dims] . K^T      (A = Q, B = K rows)
//   O^T[dims(16) x heads(8, G used)]  += V^T[dims x keys(16)] . P^T  (A = V^T, B = P)
// Both contractions are invariant under a permutation of the contracted index, so a
// thread reads whole 16-byte chunks from the staged page and pairs registers up as
// the MMA fragments need them; no transposes, no ldmatrix.
#include <algorithm>
#include <atomic>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "cpa_device.cuh"
#include "cpa_internal.h"

namespace {

constexpr int kDecodeWarps = 4;
constexpr int kDecodeThreads = kDecodeWarps * 32;
constexpr int kDecodeSmemBytes = 64 * 1024;          // stage rings of the four warps (three CTAs per SM)
constexpr uint32_t kSpinLimit = 1u << 18;            // bounded mbarrier wait (each try suspends briefly)
constexpr uint32_t kDrainLimit = 1u << 12;           // last look at a copy in flight after a wait gave up

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

__device__ __forceinline__ uint32_t sel(const uint4& v, int i) {
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

// Contiguous global -> shared copy; both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// Optional fused append (cpa_decode_append): k_new == nullptr means plain decode.
struct cpa_fused_append {
    const __nv_bfloat16* k_new;   // [B, Hkv, D] the step's new key rows
    const __nv_bfloat16* v_new;
    __nv_bfloat16* k_pool;        // the pools again, writable
    __nv_bfloat16* v_pool;
};

// One work item = (block, kv head, split of up to C pages); the item record carries the
// split's page ids.  Four warps take the split's pages round-robin; each streams its pages
// through its own ring of STAGES shared-memory stages (K chunk + V chunk per stage; two
// stages at head_dim 128 so that three CTAs = twelve warps fit an SM: once the pool is partly
// served from L2 the per-page arithmetic latency, not the copy depth, is what needs hiding) and
// keeps its own running (max, sum, acc).  The CTA then merges the four warps in shared
// memory.  A block with a single active split is normalised and stored directly; otherwise
// the CTA writes one partial per query head and takes a ticket: the last CTA of a
// (block, kv head) to arrive merges all partials
//     m = max_s m_s,  l = sum_s l_s 2^(m_s - m),  O = sum_s acc_s 2^(m_s - m) / l
// and resets the ticket counter for the next launch.
//   part_ml : [total_splits, Hq, 2]  (max in log2 units, sum), fp32
//   part_o  : [total_splits, Hq, D]  unnormalised accumulators, fp32
template <int D>
__global__ void __launch_bounds__(kDecodeThreads, 3)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_pool,
                    const __nv_bfloat16* __restrict__ v_pool, float* __restrict__ part_ml,
                    float* __restrict__ part_o, __nv_bfloat16* __restrict__ out, cpa_dev_index ix, int Hq,
                    int Hkv, int G, float scale_log2, int reverse, cpa_fused_append fa, int n_items, int late_wait,
                    cpa_decode_mode mode) {
    constexpr int P = 16;
    constexpr int KC = D / 32;  // 16-byte K chunks per thread per 8-key group
    constexpr int VC = D / 64;  // 16-byte V chunks per thread per key row
    constexpr uint32_t kChunkBytes = P * D * 2;                  // one (page, head) chunk of K or of V
    constexpr uint32_t kStageBytes = 2 * kChunkBytes;
    constexpr int STAGES = kDecodeSmemBytes / kDecodeWarps / kStageBytes;   // 2 at d=128, 4 at d=64
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(8) uint64_t sm_bar[kDecodeWarps][STAGES];
    __shared__ float sm_m[kDecodeWarps][8];
    __shared__ float sm_l[kDecodeWarps][8];
    __shared__ int sm_last;
    __shared__ int sm_pages[kDecodeWarps][kMaxSplitPages / kDecodeWarps];  // page ids of each warp's pages

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(dsm) + warp * (STAGES * kStageBytes);
    const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(&sm_bar[warp][0]);
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < STAGES; ++st) mbar_init(bar0 + 8 * st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    __syncwarp();

    bool gave_up = false;  // a bounded wait ran out: stop waiting, results are void, status says so
    int ring_pos = 0;      // pages this warp has pushed through its ring so far (stage and phase carry over)
    // A CTA takes items blockIdx.x, blockIdx.x + gridDim.x, ...: the grid is at most one wave, so when
    // there are more items than resident CTAs nobody waits for a second, half-empty wave.
    for (int item_idx = blockIdx.x; item_idx < n_items; item_idx += gridDim.x) {
    if (item_idx != (int)blockIdx.x) __syncthreads();  // the previous item's merge buffer aliases the rings
    const int32_t* item = ix.decode_items + (int64_t)item_idx * ix.item_stride;
    const int4 hdr = *reinterpret_cast<const int4*>(item);
    const int b = hdr.x, g = hdr.y, s = hdr.z, n_reserved = hdr.w;
    if (n_reserved == 0) continue;   // a filler of the even cut: this CTA has nothing in this round
    // A step of a chunked plan: only the blocks whose turn it is decode; the others sit the step out and their
    // output rows are not touched.  A block that is through with its tokens has its length carried into the
    // other length buffer by its first CTA (below); one that is still being prefilled has no length yet.
    int sched_pos = 0;   // chunked plans: the block's token number in this step
    if (mode.step >= 0) {
        sched_pos = mode.step - __ldg(ix.dec_start + b);
        if (sched_pos < 0) continue;
        if (sched_pos >= mode.T) {
            if (fa.k_new != nullptr && g == 0 && s == 0 && threadIdx.x == 0) {
                asm volatile("griddepcontrol.wait;\n" ::: "memory");   // the previous launch wrote the length read here
                ix.seq_lens_next[b] = ix.seq_lens[b];
            }
            continue;
        }
    }
    const int C = item[4];  // pages per split of this block
    const int first = item[5];           // first page of the split inside the block's page list
    const int slot = item[6];            // its partial slot among the block's slots
    const int n_fixed = item[7];         // slots in front that the shared-prefix scan has filled
    // this warp's pages are warp, warp+4, ... of the split: park their ids in shared memory (the item record
    // carries them; a plan with pages on demand reads them from the page table further down)
    if (!mode.dynamic)
        for (int j = lane; warp + kDecodeWarps * j < n_reserved; j += 32)
            sm_pages[warp][j] = item[8 + warp + kDecodeWarps * j];
    // Everything above reads plan constants only.  The launch may have started while the
    // previous kernel in the stream (normally the step's append) was still running; from here
    // on its writes (cached length, the new K/V row) are needed, so wait for it to finish.
    // (When the launch follows the shared-prefix scan of the same step, that earlier kernel is the only
    // one still running; its partials are needed for the merge only, so the wait moves down there.)
    if (!late_wait) asm volatile("griddepcontrol.wait;\n" ::: "memory");
    // Fused append: the block's newest token (position len_old) is not in the pool yet.  The
    // CTA whose split holds that position stores the row (for later steps) and patches its own
    // staged copy of the page; every CTA counts the token.  Lengths are double buffered: this
    // launch reads one array and the owner CTA of kv head 0 writes the other, so no CTA can see
    // a length that already moved.
    const bool fused = fa.k_new != nullptr;
    // (a block of a chunked plan enters its first decode step with its whole prompt cached, whatever the
    // length buffers hold: the chunks that cached it ran beside earlier decode launches)
    const int len_old = (mode.step >= 0 && sched_pos == 0)
                            ? ix.prefix_lens[b] + ix.cu_seqlens[b + 1] - ix.cu_seqlens[b] : ix.seq_lens[b];
    if (mode.dynamic) {
        // Pages on demand.  A block takes part unless the caller's flag says it has stopped.  The page its new
        // token goes to was taken from the reserve when the page before it filled up; if the reserve was empty
        // then, the block cannot grow: it sits the step out and the status word says why.  The first CTA of a
        // block that sits out carries its length over.
        const bool idle = mode.d_active != nullptr && mode.d_active[b] == 0;
        const bool no_room = !idle && fused && len_old / P >= ix.pages_assigned[b];
        if (idle || no_room) {
            if (fused && g == 0 && s == 0 && threadIdx.x == 0) {
                ix.seq_lens_next[b] = len_old;
                if (no_room) atomicCAS(ix.status, 0, kStatusNoSpace);
            }
            continue;
        }
    }
    const int len = len_old + (fused ? 1 : 0);
    __syncwarp();
    const int pages_active = (len + P - 1) / P;
    if (mode.dynamic) {   // the ids of the pages that hold keys, from the block's row of the page table
        const int32_t* row = ix.page_indices + ix.page_indptr[b] + first;
        for (int j = lane; warp + kDecodeWarps * j < n_reserved && first + warp + kDecodeWarps * j < pages_active; j += 32)
            sm_pages[warp][j] = row[warp + kDecodeWarps * j];
        __syncwarp();
    }
    const int pg_new = fused ? len_old / P : -1;   // page (inside the block) of the new token
    const bool owner = fused && pg_new >= first && pg_new < first + n_reserved;
    uint4 new_chunk = make_uint4(0, 0, 0, 0);      // lanes 0-15: a 16-byte piece of the K row, 16-31: of the V row
    if (owner && warp == (pg_new - first) % kDecodeWarps) {
        const int piece = lane & 15;
        if (piece < D / 8) {
            const __nv_bfloat16* src = (lane < 16 ? fa.k_new : fa.v_new) + ((int64_t)b * Hkv + g) * D + piece * 8;
            new_chunk = *reinterpret_cast<const uint4*>(src);
            const int64_t page = sm_pages[warp][(pg_new - first) / kDecodeWarps];
            __nv_bfloat16* dst = (lane < 16 ? fa.k_pool : fa.v_pool) +
                                 (((page * Hkv + g) * P) + (len_old % P)) * D + cpa_pool_piece(piece, len_old % P) * 8;
            *reinterpret_cast<uint4*>(dst) = new_chunk;
        }
        if (g == 0 && lane == 0) {
            ix.seq_lens_next[b] = len;
            if (mode.dynamic && len % P == 0) {
                // this token filled its page: take the page of the next one from the reserve now, so that every
                // CTA of the next launch finds it in the table (pushes happen in other launches only, so the
                // count of pushes is a constant here)
                const int next_pg = len / P, cap = ix.page_indptr[b + 1] - ix.page_indptr[b];
                if (next_pg < cap) {
                    const int h = atomicAdd(ix.ring_ctrl, 1);
                    if (h < ix.ring_ctrl[1]) {
                        ix.page_table[ix.page_indptr[b] + next_pg] = ix.ring[h % ix.ring_ctrl[2]];
                        ix.pages_assigned[b] = next_pg + 1;
                    } else {
                        atomicSub(ix.ring_ctrl, 1);   // the reserve is empty: the block's next step will say so
                    }
                }
            }
        }
    }
    const int n_active = min(n_reserved, pages_active - first);  // pages of this split that hold keys
    if (n_active <= 0) continue;  // split lies beyond the cached length (uniform per CTA)
    const int n_mine = (n_active - warp + kDecodeWarps - 1) / kDecodeWarps;  // pages of this warp (may be <= 0)

    auto issue = [&](int st, int page) {  // lane 0 only
        const uint32_t bar = bar0 + 8 * st;
        const uint32_t dst = ring + st * kStageBytes;
        const int64_t chunk = ((int64_t)page * Hkv + g) * (P * D);
        mbar_expect_tx(bar, kStageBytes);
        bulk_load(dst, k_pool + chunk, kChunkBytes, bar);
        bulk_load(dst + kChunkBytes, v_pool + chunk, kChunkBytes, bar);
    };
    // Consecutive decode steps walk the pages in opposite directions: what the previous step
    // read last is what this step reads first, so a pool of about the L2's size is served
    // largely from L2 instead of being evicted just before its reuse.  The online softmax does
    // not care about the order of the keys.
    auto local_index = [&](int i) { return reverse ? n_mine - 1 - i : i; };
#pragma unroll
    for (int st = 0; st < STAGES; ++st)
        if (st < n_mine && lane == 0) issue((ring_pos + st) % STAGES, sm_pages[warp][local_index(st)]);

    // Q fragments: row gid of the A tile is query head g*G + gid (zero rows beyond G)
    uint4 qf[KC];
#pragma unroll
    for (int c = 0; c < KC; ++c) qf[c] = make_uint4(0, 0, 0, 0);
    if (gid < G) {
        const __nv_bfloat16* qrow = q + ((int64_t)b * Hq + g * G + gid) * D;
#pragma unroll
        for (int c = 0; c < KC; ++c) qf[c] = *reinterpret_cast<const uint4*>(qrow + (c * 4 + tig) * 8);
    }

    float acc[VC][4][4];
#pragma unroll
    for (int c = 0; c < VC; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[c][i][e] = 0.f;
    float m_run = -INFINITY;  // running max of raw scores, row gid
    float l_run = 0.f;        // this thread's share of the running sum, row gid

    for (int i = 0; i < n_mine; ++i) {
        const int st = (ring_pos + i) % STAGES;
        const uint32_t parity = (uint32_t)((ring_pos + i) / STAGES) & 1u;
        const int pg = first + warp + kDecodeWarps * local_index(i);  // page index inside the block
        mbar_wait(bar0 + 8 * st, parity, gave_up, ix.status, kSpinLimit);
        if (__any_sync(0xffffffffu, gave_up)) {
            // The page never arrived: nothing more is issued, and the copies still on their way into
            // this warp's stages (pages i .. i + STAGES - 1) get one last bounded look, so that the CTA
            // does not end under a copy in flight.  The CTA returns below; the status word says why.
            gave_up = true;
            if (lane == 0)
                for (int k2 = i; k2 < n_mine && k2 < i + STAGES; ++k2)
                    mbar_drain(bar0 + 8 * ((ring_pos + k2) % STAGES), (uint32_t)((ring_pos + k2) / STAGES) & 1u, kDrainLimit);
            break;
        }
        const uint32_t ks = ring + st * kStageBytes;
        const uint32_t vs = ks + kChunkBytes;
        if (pg == pg_new) {   // (only the owning warp ever sees this page) put the new row into the staged copy
            const int piece = lane & 15;
            if (piece < D / 8) {
                const uint32_t addr = (lane < 16 ? ks : vs) + (len_old % P) * (D * 2) + cpa_pool_piece(piece, len_old % P) * 16;
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n"
                             :: "r"(addr), "r"(new_chunk.x), "r"(new_chunk.y), "r"(new_chunk.z), "r"(new_chunk.w) : "memory");
            }
            __syncwarp();
        }
        // ---- S = Q K^T for the 16 keys of this page
        float sc[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            // two accumulators per 8-key group halve the length of the dependent MMA chain
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < KC; ++c) {
                const uint4 kr = lds128(ks + (gid + 8 * t) * (D * 2) + cpa_pool_piece(c * 4 + tig, gid) * 16);
                mma_bf16_16816(sa, qf[c].x, 0u, qf[c].y, 0u, kr.x, kr.y);
                mma_bf16_16816(sb, qf[c].z, 0u, qf[c].w, 0u, kr.z, kr.w);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[t][e] = sa[e] + sb[e];
        }
        // ---- mask the tail of the last page by index, then online softmax (row gid)
        const int key0 = pg * P + tig * 2;
        const bool partial = (pg + 1) * P > len;
        if (partial) {
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    if (key0 + 8 * t + e >= len) sc[t][e] = -INFINITY;
        }
        float mx = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);  // finite: every visited page holds a valid key
        const float alpha = (m_run == -INFINITY) ? 0.f : exp2f((m_run - m_new) * scale_log2);
        const float mb = m_new * scale_log2;
        float p[2][2];
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int e = 0; e < 2; ++e) p[t][e] = exp2f(fmaf(sc[t][e], scale_log2, -mb));
        // the row sum is taken over the bf16-rounded weights the MMA will multiply with
        const uint32_t pb0 = pack_bf16x2(p[0][0], p[0][1]);
        const uint32_t pb1 = pack_bf16x2(p[1][0], p[1][1]);
        l_run = l_run * alpha + (__uint_as_float(pb0 << 16) + __uint_as_float(pb0 & 0xffff0000u)) +
                (__uint_as_float(pb1 << 16) + __uint_as_float(pb1 & 0xffff0000u));
        m_run = m_new;

        // accumulator columns are heads 2*tig, 2*tig+1; their factors live in lanes of row = head
        const float a0 = __shfl_sync(0xffffffffu, alpha, (2 * tig) * 4);
        const float a1 = __shfl_sync(0xffffffffu, alpha, (2 * tig + 1) * 4);

        // ---- O^T += V^T P^T
#pragma unroll
        for (int c = 0; c < VC; ++c) {
            uint4 vr[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int row = 2 * tig + (r & 1) + 8 * (r >> 1);
                vr[r] = lds128(vs + row * (D * 2) + cpa_pool_piece(c * 8 + gid, row) * 16);
                // unused slots may hold anything (even NaN): select them away
                if (partial && pg * P + row >= len) vr[r] = make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int i2 = 0; i2 < 4; ++i2) {
                acc[c][i2][0] *= a0; acc[c][i2][1] *= a1; acc[c][i2][2] *= a0; acc[c][i2][3] *= a1;
                const uint32_t r0 = sel(vr[0], i2), r1 = sel(vr[1], i2);
                const uint32_t r2 = sel(vr[2], i2), r3 = sel(vr[3], i2);
                mma_bf16_16816(acc[c][i2], __byte_perm(r0, r1, 0x5410), __byte_perm(r0, r1, 0x7632),
                               __byte_perm(r2, r3, 0x5410), __byte_perm(r2, r3, 0x7632), pb0, pb1);
            }
        }
        // every lane has taken what it needs from this stage: refill it
        __syncwarp();
        const int nxt = i + STAGES;
        if (nxt < n_mine && lane == 0) issue(st, sm_pages[warp][local_index(nxt)]);
    }
    if (n_mine > 0) ring_pos += n_mine;
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);

    // ---- merge the four warps; the stage rings are idle now (every issued copy was consumed)
    if (__syncthreads_or((int)gave_up)) return;   // a wait gave up: no copy is in flight any more, results are void
    float (*sm_o)[8][D + 4] = reinterpret_cast<float (*)[8][D + 4]>(dsm);
    if (tig == 0) { sm_m[warp][gid] = m_run * scale_log2; sm_l[warp][gid] = l_run; }
#pragma unroll
    for (int c = 0; c < VC; ++c)
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                sm_o[warp][2 * tig + (e & 1)][8 * (8 * c + gid) + 2 * i + (e >> 1)] = acc[c][i][e];
    __syncthreads();

    // Active splits of this block's own pages.  The own pages (behind `skip` pages the shared scan covers) are cut
    // into a first split of `head` pages and splits of C pages behind it (uniform cut: head = C; even cut: the first
    // split ends where the cut through all blocks' pages falls).
    const int skip = late_wait ? __ldg(ix.prefix_lens + b) / P : 0;
    const int head = s == 0 ? n_reserved : (first - skip) - (s - 1) * C;
    const int own_active = pages_active - skip;
    const int n_own = own_active <= head ? 1 : 1 + (own_active - head + C - 1) / C;
    const int n_splits = n_fixed + n_own;                            // partials to merge
    const int64_t out_row = (int64_t)b * Hq + g * G;
    const int64_t prow = (int64_t)(ix.split_indptr[b] + slot) * Hq + g * G;
    constexpr int HP = D / 2;  // dim pairs per head
    for (int idx = threadIdx.x; idx < G * HP; idx += kDecodeThreads) {
        const int h = idx / HP, dim = 2 * (idx - h * HP);
        float m = sm_m[0][h];
#pragma unroll
        for (int w = 1; w < kDecodeWarps; ++w) m = fmaxf(m, sm_m[w][h]);
        float o0 = 0.f, o1 = 0.f, l = 0.f;
#pragma unroll
        for (int w = 0; w < kDecodeWarps; ++w) {
            const float mw = sm_m[w][h];
            const float f = (mw == -INFINITY) ? 0.f : exp2f(mw - m);
            const float2 t = *reinterpret_cast<const float2*>(&sm_o[w][h][dim]);
            o0 = fmaf(f, t.x, o0);
            o1 = fmaf(f, t.y, o1);
            l = fmaf(f, sm_l[w][h], l);
        }
        if (n_splits == 1) {
            const float inv = 1.f / l;
            *reinterpret_cast<__nv_bfloat162*>(out + (out_row + h) * D + dim) = __floats2bfloat162_rn(o0 * inv, o1 * inv);
        } else {
            *reinterpret_cast<float2*>(part_o + (prow + h) * D + dim) = make_float2(o0, o1);
            if (dim == 0) *reinterpret_cast<float2*>(part_ml + (prow + h) * 2) = make_float2(m, l);
        }
    }
    if (n_splits == 1) continue;

    // ---- the last CTA of this (block, kv head) merges the splits
    if (late_wait) asm volatile("griddepcontrol.wait;\n" ::: "memory");   // the shared scan's partials are complete
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        int* ticket = ix.merge_tickets + b * Hkv + g;
        const int t = atomicAdd(ticket, 1);
        sm_last = (t == n_own - 1);
        if (sm_last) *ticket = 0;  // every other split has arrived; ready for the next launch
    }
    __syncthreads();
    if (!sm_last) continue;
    __threadfence();
    const int64_t base = (int64_t)ix.split_indptr[b] * Hq + g * G;
    constexpr int kMergeTable = kDecodeSmemBytes / 64;   // splits whose (factor, sum) pairs fit the idle rings
    if (n_splits <= kMergeTable) {
        // The (max, sum) pairs are fetched once, in parallel, into the idle stage rings and turned into
        // scale factors there; the accumulator loop then issues nothing but independent loads.
        float* sm_f = reinterpret_cast<float*>(dsm);              // [n_splits][8] max, then factor
        float* sm_s = sm_f + kMergeTable * 8;                     // [n_splits][8] sum
        __shared__ float sm_tot[8];
        for (int idx = threadIdx.x; idx < n_splits * G; idx += kDecodeThreads) {
            const int sp = idx / G, h = idx - sp * G;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + (base + (int64_t)sp * Hq + h) * 2));
            sm_f[sp * 8 + h] = ml.x;
            sm_s[sp * 8 + h] = ml.y;
        }
        __syncthreads();
        for (int h = warp; h < G; h += kDecodeWarps) {            // one warp per head: max, factors, total
            float m = -INFINITY;
            for (int sp = lane; sp < n_splits; sp += 32) m = fmaxf(m, sm_f[sp * 8 + h]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float l = 0.f;
            for (int sp = lane; sp < n_splits; sp += 32) {
                const float f = exp2f(sm_f[sp * 8 + h] - m);
                sm_f[sp * 8 + h] = f;
                l = fmaf(f, sm_s[sp * 8 + h], l);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
            if (lane == 0) sm_tot[h] = l;
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < G * HP; idx += kDecodeThreads) {
            const int h = idx / HP, dim = 2 * (idx - h * HP);
            float o0 = 0.f, o1 = 0.f;
#pragma unroll 8
            for (int sp = 0; sp < n_splits; ++sp) {
                const float2 t = __ldcg(reinterpret_cast<const float2*>(part_o + (base + (int64_t)sp * Hq + h) * D + dim));
                const float f = sm_f[sp * 8 + h];
                o0 = fmaf(f, t.x, o0);
                o1 = fmaf(f, t.y, o1);
            }
            const float inv = 1.f / sm_tot[h];
            *reinterpret_cast<__nv_bfloat162*>(out + (out_row + h) * D + dim) = __floats2bfloat162_rn(o0 * inv, o1 * inv);
        }
        continue;   // (the next item's first __syncthreads separates these reads from its ring writes)
    }
    for (int idx = threadIdx.x; idx < G * HP; idx += kDecodeThreads) {
        const int h = idx / HP, dim = 2 * (idx - h * HP);
        float m = -INFINITY;
        for (int sp = 0; sp < n_splits; ++sp) m = fmaxf(m, __ldcg(part_ml + (base + (int64_t)sp * Hq + h) * 2));
        float o0 = 0.f, o1 = 0.f, l = 0.f;
        for (int sp = 0; sp < n_splits; ++sp) {
            const int64_t r = base + (int64_t)sp * Hq + h;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(part_ml + r * 2));
            const float2 t = __ldcg(reinterpret_cast<const float2*>(part_o + r * D + dim));
            const float f = exp2f(ml.x - m);
            o0 = fmaf(f, t.x, o0);
            o1 = fmaf(f, t.y, o1);
            l = fmaf(f, ml.y, l);
        }
        const float inv = 1.f / l;
        *reinterpret_cast<__nv_bfloat162*>(out + (out_row + h) * D + dim) = __floats2bfloat162_rn(o0 * inv, o1 * inv);
    }
    }  // items
}

// Shared-prefix scan of the prefix-aware layout: one work item = (group of consecutive workers,
// kv head, chunk of shared history pages).  Every page of the chunk is read ONCE into a ring of
// stages that all four warps consume; warp w owns rows 16w .. 16w+15 of the group's (worker, query
// head) rows (row = worker * G + head; up to 64 rows), sixteen rows on the M side of S = Q K^T and
// two groups of eight on the N side of O^T += V^T P^T.  A row sees the keys below its worker's
// prefix length only (masked by index), so the workers whose prefix ends inside or before the
// chunk are handled by the same pass, and a warp skips the pages none of its rows sees.  Each row
// that sees at least one key of the chunk leaves a partial (max, sum, acc) in slot `chunk` of its
// worker; the per-worker kernel that follows in the stream merges them with the partials of the
// worker's own pages.  Lane 0 of warp 0 also feeds the ring, two pages behind its own position, so
// that it rarely has to wait for the other warps to release a stage.
constexpr int kSharedThreads = 4 * 32;
constexpr int kSharedSmemBytes = 64 * 1024;          // the ring (three CTAs per SM)
constexpr int kSharedLag = 2;

template <int D>
__global__ void __launch_bounds__(kSharedThreads, 3)
decode_shared_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_pool,
                     const __nv_bfloat16* __restrict__ v_pool, float* __restrict__ part_ml,
                     float* __restrict__ part_o, cpa_dev_index ix, int Hq, int Hkv, int G, float scale_log2) {
    constexpr int P = 16;
    constexpr int KC = D / 32;  // 16-byte K chunks per thread per 8-key group
    constexpr int VC = D / 64;  // 16-byte V chunks per thread per key row
    constexpr uint32_t kChunkBytes = P * D * 2;
    constexpr uint32_t kStageBytes = 2 * kChunkBytes;
    constexpr int STAGES = kSharedSmemBytes / kStageBytes;   // 8 at d=128, 16 at d=64
    extern __shared__ __align__(128) unsigned char dsm[];
    __shared__ __align__(8) uint64_t sm_full[STAGES], sm_empty[STAGES];
    __shared__ int sm_ids[kMaxSharedChunkPages];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const uint32_t ring = (uint32_t)__cvta_generic_to_shared(dsm);
    const uint32_t full0 = (uint32_t)__cvta_generic_to_shared(&sm_full[0]);
    const uint32_t empty0 = (uint32_t)__cvta_generic_to_shared(&sm_empty[0]);
    if (threadIdx.x == 0) {
        for (int st = 0; st < STAGES; ++st) { mbar_init(full0 + 8 * st, 1); mbar_init(empty0 + 8 * st, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    // The per-worker kernel of this step is next in the stream and does not need anything from this one
    // before its merge: let it start as soon as there is room for its CTAs.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int4 hdr = *reinterpret_cast<const int4*>(ix.shared_items + 4 * (int64_t)blockIdx.x);
    const int w0 = hdr.x & 0xFFFF, nw = hdr.x >> 16, g = hdr.y, chunk = hdr.z, n_pages = hdr.w;
    const int first = chunk * ix.shared_chunk;      // first history page of the chunk
    for (int i = threadIdx.x; i < n_pages; i += kSharedThreads) sm_ids[i] = __ldg(ix.shared_page_ids + first + i);
    __syncthreads();
    bool gave_up = false;

    auto issue = [&](int i) {   // lane 0 of warp 0: page i of the chunk into its stage
        const int st = i % STAGES;
        const uint32_t dst = ring + st * kStageBytes;
        const int64_t src = ((int64_t)sm_ids[i] * Hkv + g) * (P * D);
        mbar_expect_tx(full0 + 8 * st, kStageBytes);
        bulk_load(dst, k_pool + src, kChunkBytes, full0 + 8 * st);
        bulk_load(dst + kChunkBytes, v_pool + src, kChunkBytes, full0 + 8 * st);
    };
    int n_issued = 0;   // pages handed to the copy engine so far (thread 0)
    if (threadIdx.x == 0)
        for (int i = 0; i < STAGES && i < n_pages; ++i) { issue(i); n_issued = i + 1; }

    // -------------------------------------------------------------------- compute warps
    // rows of this thread: A = 16*warp + gid, B = A + 8 (row = worker * G + head inside the group)
    const int n_rows = nw * G;
    int vis[2], wk[2], hd[2];          // visible prefix length (tokens), worker, head of rows A and B
    uint4 qa[KC], qb[KC];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = 16 * warp + gid + 8 * r;
        const bool real = row < n_rows;
        wk[r] = w0 + (real ? row / G : 0);
        hd[r] = real ? row % G : 0;
        vis[r] = real ? __ldg(ix.prefix_lens + wk[r]) : 0;
        const __nv_bfloat16* qrow = q + ((int64_t)wk[r] * Hq + g * G + hd[r]) * D;
#pragma unroll
        for (int c = 0; c < KC; ++c) {
            const uint4 v = real ? *reinterpret_cast<const uint4*>(qrow + (c * 4 + tig) * 8) : make_uint4(0, 0, 0, 0);
            if (r == 0) qa[c] = v; else qb[c] = v;
        }
    }
    float acc[2][VC][4][4];
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int c = 0; c < VC; ++c)
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[n][c][i][e] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY};   // running max of raw scores, rows A and B
    float l_run[2] = {0.f, 0.f};               // this thread's share of the running sums
    int vis_warp = max(vis[0], vis[1]);        // no row of this warp sees keys from here on
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) vis_warp = max(vis_warp, __shfl_xor_sync(0xffffffffu, vis_warp, o));

    for (int i = 0; i < n_pages; ++i) {
        const int st = i % STAGES;
        const uint32_t parity = (uint32_t)(i / STAGES) & 1u;
        if (threadIdx.x == 0) {
            // refill: page j takes the stage of page j - STAGES, which every warp must have released
            const int j = i + STAGES - kSharedLag;
            if (j >= STAGES && j < n_pages) {
                mbar_wait(empty0 + 8 * (j % STAGES), ((uint32_t)(j / STAGES) & 1u) ^ 1u, gave_up, ix.status, kSpinLimit);
                if (!gave_up) { issue(j); n_issued = j + 1; }
            }
        }
        gave_up = __shfl_sync(0xffffffffu, gave_up, 0) || gave_up;
        mbar_wait(full0 + 8 * st, parity, gave_up, ix.status, kSpinLimit);
        if (__any_sync(0xffffffffu, gave_up)) { gave_up = true; break; }   // stop consuming; the CTA drains and returns below
        if ((first + i) * P >= vis_warp) {
            // Nothing on this page for this warp's rows.  It still waits for the page before it releases
            // the stage: a warp that ran ahead would add its releases of later pages to the current
            // phase of the stage's barrier.
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" :: "r"(empty0 + 8 * st) : "memory");
            continue;
        }
        const uint32_t ks = ring + st * kStageBytes;
        const uint32_t vs = ks + kChunkBytes;
        // ---- S = Q K^T: 16 rows x 16 keys
        float sc[2][4];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            float sa[4] = {0.f, 0.f, 0.f, 0.f}, sb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int c = 0; c < KC; ++c) {
                const uint4 kr = lds128(ks + (gid + 8 * t) * (D * 2) + cpa_pool_piece(c * 4 + tig, gid) * 16);
                mma_bf16_16816(sa, qa[c].x, qb[c].x, qa[c].y, qb[c].y, kr.x, kr.y);
                mma_bf16_16816(sb, qa[c].z, qb[c].z, qa[c].w, qb[c].w, kr.z, kr.w);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) sc[t][e] = sa[e] + sb[e];
        }
        // ---- a row sees the keys below its worker's prefix length; then the online softmax per row
        const int key0 = (first + i) * P + tig * 2;
        uint32_t pk[2][2];     // bf16 weights of rows A / B for key groups t = 0 / 1
        float alpha[2];
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float s00 = sc[0][2 * r], s01 = sc[0][2 * r + 1], s10 = sc[1][2 * r], s11 = sc[1][2 * r + 1];
            if (key0 + 9 >= vis[r]) {   // the page reaches beyond this row's prefix
                if (key0 >= vis[r]) s00 = -INFINITY;
                if (key0 + 1 >= vis[r]) s01 = -INFINITY;
                if (key0 + 8 >= vis[r]) s10 = -INFINITY;
                if (key0 + 9 >= vis[r]) s11 = -INFINITY;
            }
            float mx = fmaxf(fmaxf(s00, s01), fmaxf(s10, s11));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[r], mx);                     // -inf while the row has seen no key
            alpha[r] = (m_run[r] == -INFINITY) ? 0.f : exp2f((m_run[r] - m_new) * scale_log2);
            const float mb = (m_new == -INFINITY) ? 0.f : m_new * scale_log2;
            const float p00 = exp2f(fmaf(s00, scale_log2, -mb)), p01 = exp2f(fmaf(s01, scale_log2, -mb));
            const float p10 = exp2f(fmaf(s10, scale_log2, -mb)), p11 = exp2f(fmaf(s11, scale_log2, -mb));
            // the row sum is taken over the bf16-rounded weights the MMA will multiply with
            pk[r][0] = pack_bf16x2(p00, p01);
            pk[r][1] = pack_bf16x2(p10, p11);
            l_run[r] = l_run[r] * alpha[r] + (__uint_as_float(pk[r][0] << 16) + __uint_as_float(pk[r][0] & 0xffff0000u)) +
                       (__uint_as_float(pk[r][1] << 16) + __uint_as_float(pk[r][1] & 0xffff0000u));
            m_run[r] = m_new;
        }
        // Rescale the accumulators only when some row's max moved (after the first pages it rarely
        // does).  Accumulator columns are rows 2*tig, 2*tig+1 of each group of eight; their factors
        // live in the lanes whose gid is that row.
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                const float a0 = __shfl_sync(0xffffffffu, alpha[n], (2 * tig) * 4);
                const float a1 = __shfl_sync(0xffffffffu, alpha[n], (2 * tig + 1) * 4);
#pragma unroll
                for (int c = 0; c < VC; ++c)
#pragma unroll
                    for (int i2 = 0; i2 < 4; ++i2) {
                        acc[n][c][i2][0] *= a0; acc[n][c][i2][1] *= a1; acc[n][c][i2][2] *= a0; acc[n][c][i2][3] *= a1;
                    }
            }
        }
        // ---- O^T += V^T P^T, the V fragments shared by both groups of eight rows
#pragma unroll
        for (int c = 0; c < VC; ++c) {
            uint4 vr[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const int row = 2 * tig + (r & 1) + 8 * (r >> 1);
                vr[r] = lds128(vs + row * (D * 2) + cpa_pool_piece(c * 8 + gid, row) * 16);
            }
#pragma unroll
            for (int i2 = 0; i2 < 4; ++i2) {
                const uint32_t r0 = sel(vr[0], i2), r1 = sel(vr[1], i2);
                const uint32_t r2 = sel(vr[2], i2), r3 = sel(vr[3], i2);
                const uint32_t f0 = __byte_perm(r0, r1, 0x5410), f1 = __byte_perm(r0, r1, 0x7632);
                const uint32_t f2 = __byte_perm(r2, r3, 0x5410), f3 = __byte_perm(r2, r3, 0x7632);
#pragma unroll
                for (int n = 0; n < 2; ++n) mma_bf16_16816(acc[n][c][i2], f0, f1, f2, f3, pk[n][0], pk[n][1]);
            }
        }
        // this warp is done with the stage
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" :: "r"(empty0 + 8 * st) : "memory");
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
        l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
    }
    // ---- partials: slot `chunk` of every worker whose prefix reaches into the chunk
    if (__syncthreads_or((int)gave_up)) {
        // a wait gave up: the copies of the last pages issued may still be on their way into the ring;
        // thread 0 gives each one last bounded look, so that no copy is in flight when the CTA ends
        if (threadIdx.x == 0)
            for (int j = max(0, n_issued - STAGES); j < n_issued; ++j)
                mbar_drain(full0 + 8 * (j % STAGES), (uint32_t)(j / STAGES) & 1u, kDrainLimit);
        return;
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        const int row = 16 * warp + gid + 8 * r;
        if (tig == 0 && row < n_rows && vis[r] > first * P) {
            const int64_t prow = (int64_t)(ix.split_indptr[wk[r]] + chunk) * Hq + g * G + hd[r];
            *reinterpret_cast<float2*>(part_ml + prow * 2) = make_float2(m_run[r] * scale_log2, l_run[r]);
        }
    }
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e01 = 0; e01 < 2; ++e01) {
            // accumulator column 2*tig + e01 of group n = row 16*warp + 8n + 2*tig + e01
            const int row = 16 * warp + 8 * n + 2 * tig + e01;
            if (row >= n_rows) continue;
            const int wrk = w0 + row / G, h = row % G;
            if (__ldg(ix.prefix_lens + wrk) <= first * P) continue;
            float* dst = part_o + ((int64_t)(ix.split_indptr[wrk] + chunk) * Hq + g * G + h) * D;
#pragma unroll
            for (int c = 0; c < VC; ++c)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    *reinterpret_cast<float2*>(dst + 8 * (8 * c + gid) + 2 * i) =
                        make_float2(acc[n][c][i][e01], acc[n][c][i][e01 + 2]);
        }
}

// A block whose cache is still empty has no active split and gets a zero output row.
__global__ void decode_empty_rows_kernel(__nv_bfloat16* __restrict__ out, cpa_dev_index ix, int B, int row_elems) {
    const int b = blockIdx.x;
    if (b >= B || ix.seq_lens[b] > 0) return;
    for (int i = threadIdx.x; i < row_elems; i += blockDim.x) out[(int64_t)b * row_elems + i] = __float2bfloat16(0.f);
}

template <int D>
int launch_decode(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool, void* o,
                  void* ws, cudaStream_t st, cpa_fused_append fa = cpa_fused_append{nullptr, nullptr, nullptr, nullptr},
                  cpa_decode_mode mode = cpa_decode_mode{-1, 0, 0, nullptr}, int wave_sms = 0) {
    if (plan->dynamic) mode.dynamic = 1;
    const cpa_config& c = plan->cfg;
    const int G = c.num_q_heads / c.num_kv_heads;
    const cpa_dev_index ix = plan->dev();
    float* part_ml = static_cast<float*>(ws);
    float* part_o = part_ml + ((int64_t)plan->split_indptr[plan->B] * c.num_q_heads * 2 + 3) / 4 * 4;
    const float scale_log2 = c.scale * 1.4426950408889634f;
    bool any_empty = false;  // host mirror of the cached lengths
    for (int b = 0; b < plan->B && mode.step < 0; ++b) {   // (in a chunked plan's step the schedule says who decodes)
        any_empty |= plan->seq_lens[b] == 0;
        // A worker of the prefix-aware layout that has cached none of its own tokens yet has no own split to
        // run the merge of the shared scan's partials: the own tokens are appended before the first decode.
        if (plan->prefix_lens[b] > 0 && plan->seq_lens[b] == plan->prefix_lens[b]) return CPA_ESTATE;
    }
    // the attribute is per device: remember which devices have it (setting it twice is harmless, so a
    // relaxed flag is enough when several host threads arrive together)
    static std::atomic<bool> configured_dev[64];
    int dev_id = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess || dev_id < 0 || dev_id >= 64) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    std::atomic<bool>& configured = configured_dev[dev_id];
    if (!configured.load(std::memory_order_relaxed)) {
        if (cudaFuncSetAttribute(decode_split_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kDecodeSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(decode_shared_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kSharedSmemBytes) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        configured.store(true, std::memory_order_relaxed);
    }
    if (any_empty)
        decode_empty_rows_kernel<<<plan->B, 128, 0, st>>>((__nv_bfloat16*)o, ix, plan->B, c.num_q_heads * D);
    // Prefix-aware layout: the shared history pages are scanned once for all workers; the partials go
    // to the first slots of every worker and are merged by the launch below, which follows in the stream.
    if (plan->n_shared > 0) {
        if (cpa_scan_rows(G) == 128) {   // the tensor-core scan (its query tile is loaded in boxes of 8/G sequences)
            const int rc = cpa_scan_tc(plan, q, k_pool, v_pool, part_ml, part_o, wave_sms, st);
            if (rc != CPA_OK) return rc;
        } else {
            decode_shared_kernel<D><<<plan->n_shared, kSharedThreads, kSharedSmemBytes, st>>>(
                (const __nv_bfloat16*)q, (const __nv_bfloat16*)k_pool, (const __nv_bfloat16*)v_pool, part_ml, part_o, ix,
                (int)c.num_q_heads, (int)c.num_kv_heads, G, scale_log2);
        }
    }
    // Programmatic dependent launch: the grid may be scheduled while the previous kernel of the
    // stream drains; the kernel itself waits (griddepcontrol.wait) before it reads anything
    // that kernel wrote.
    cudaLaunchConfig_t cfg = {};
    // one wave at most: the plan's grid (three CTAs per SM of its budget; with the even cut exactly the CTAs the cut
    // was made for), or what fits beside a prefill chunk; CTAs loop over the items when there are more
    cfg.gridDim = dim3(wave_sms > 0 ? std::min(plan->decode_grid, 3 * wave_sms) : plan->decode_grid);
    cfg.blockDim = dim3(kDecodeThreads);
    cfg.dynamicSmemBytes = kDecodeSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, decode_split_kernel<D>, (const __nv_bfloat16*)q,
                                       (const __nv_bfloat16*)k_pool, (const __nv_bfloat16*)v_pool, part_ml, part_o,
                                       (__nv_bfloat16*)o, ix, (int)c.num_q_heads, (int)c.num_kv_heads, G, scale_log2,
                                       (int)(plan->decode_calls++ & 1), fa, (int)plan->n_decode,
                                       (int)(plan->n_shared > 0), mode);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

// Scratch for cpa_decode_static: lives in the library image, so every GPU that loads the
// library holds these bytes until the process exits.
constexpr int64_t kStaticScratchBytes = 16ll << 20;
static_assert(kStaticScratchBytes == CPA_STATIC_SCRATCH_BYTES, "the header promises this size");
static __device__ __align__(256) unsigned char g_static_decode_scratch[kStaticScratchBytes];

}  // namespace

int cpa_decode_launch(const cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                      void* v_pool, void* o, void* ws, cpa_decode_mode mode, int wave_sms, void* stream) {
    cpa_fused_append fa{(const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, (__nv_bfloat16*)k_pool,
                        (__nv_bfloat16*)v_pool};
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_decode<128>(plan, q, k_pool, v_pool, o, ws, st, fa, mode, wave_sms)
                                     : launch_decode<64>(plan, q, k_pool, v_pool, o, ws, st, fa, mode, wave_sms);
}

extern "C" int cpa_decode(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool, void* o,
                          void* d_workspace, void* stream) {
    if (!plan || !q || !k_pool || !v_pool || !o || !d_workspace) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k_pool) || !cpa_aligned16(v_pool) || !cpa_aligned16(o) ||
        !cpa_aligned16(d_workspace))
        return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_decode<128>(plan, q, k_pool, v_pool, o, d_workspace, st)
                                     : launch_decode<64>(plan, q, k_pool, v_pool, o, d_workspace, st);
}

extern "C" int cpa_decode_static(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool,
                                 void* o, void* stream) {
    if (!plan || !q || !k_pool || !v_pool || !o) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k_pool) || !cpa_aligned16(v_pool) || !cpa_aligned16(o))
        return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    if (plan->decode_workspace_bytes() > kStaticScratchBytes) return CPA_ENOSPC;
    // In host code the array's name is only a handle; its device address has to be asked for,
    // once per device, with that device current.
    constexpr int kMaxDevices = 64;
    // the address is the same for every thread that looks it up, so a relaxed atomic slot per device is enough
    static std::atomic<void*> scratch_addr[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    void* scratch = scratch_addr[dev].load(std::memory_order_relaxed);
    if (!scratch) {
        if (cudaGetSymbolAddress(&scratch, g_static_decode_scratch) != cudaSuccess || !scratch) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        scratch_addr[dev].store(scratch, std::memory_order_relaxed);
    }
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_decode<128>(plan, q, k_pool, v_pool, o, scratch, st)
                                     : launch_decode<64>(plan, q, k_pool, v_pool, o, scratch, st);
}

extern "C" int cpa_decode_append(cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                                 void* v_pool, void* o, void* d_workspace, void* stream) {
    if (!plan || !q || !k_new || !v_new || !k_pool || !v_pool || !o || !d_workspace) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k_new) || !cpa_aligned16(v_new) || !cpa_aligned16(k_pool) ||
        !cpa_aligned16(v_pool) || !cpa_aligned16(o) || !cpa_aligned16(d_workspace))
        return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    for (int b = 0; b < plan->B; ++b)
        if ((int64_t)plan->seq_lens[b] + 1 > (int64_t)plan->prefix_lens[b] + plan->block_lens[b] + plan->T) return CPA_ENOSPC;
    // the kernel counts the new token itself; the host mirror moves first so that the launcher
    // sees non-empty caches, and moves back if the launch fails
    for (int b = 0; b < plan->B; ++b) plan->seq_lens[b] += 1;
    cpa_fused_append fa{(const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, (__nv_bfloat16*)k_pool,
                        (__nv_bfloat16*)v_pool};
    cudaStream_t st = (cudaStream_t)stream;
    // the device still holds the old lengths in the current buffer; they are read there
    const int rc = plan->cfg.head_dim == 128 ? launch_decode<128>(plan, q, k_pool, v_pool, o, d_workspace, st, fa)
                                             : launch_decode<64>(plan, q, k_pool, v_pool, o, d_workspace, st, fa);
    if (rc != CPA_OK) {
        for (int b = 0; b < plan->B; ++b) plan->seq_lens[b] -= 1;
        return rc;
    }
    plan->cur_lens ^= 1;   // the other buffer now holds the lengths
    return CPA_OK;
}

extern "C" int cpa_decode_append_steps(cpa_plan* plan, const void* q, const void* k_new, const void* v_new, void* k_pool,
                                       void* v_pool, void* o, void* d_workspace, int32_t num_steps, void* stream) {
    if (!plan || num_steps < 0) return CPA_EINVAL;
    if (num_steps == 0) return CPA_OK;
    if (!plan->d_base) return CPA_ESTATE;
    for (int b = 0; b < plan->B; ++b)
        if ((int64_t)plan->seq_lens[b] + num_steps > (int64_t)plan->prefix_lens[b] + plan->block_lens[b] + plan->T)
            return CPA_ENOSPC;
    const int64_t q_step = (int64_t)plan->B * plan->cfg.num_q_heads * plan->cfg.head_dim * 2;     // bytes per step
    const int64_t kv_step = (int64_t)plan->B * plan->cfg.num_kv_heads * plan->cfg.head_dim * 2;
    for (int32_t t = 0; t < num_steps; ++t) {
        const int rc = cpa_decode_append(plan, static_cast<const char*>(q) + t * q_step,
                                         static_cast<const char*>(k_new) + t * kv_step,
                                         static_cast<const char*>(v_new) + t * kv_step, k_pool, v_pool,
                                         static_cast<char*>(o) + t * q_step, d_workspace, stream);
        if (rc != CPA_OK) return rc;
    }
    return CPA_OK;
}

extern "C" int cpa_decode_append_dynamic(cpa_plan* plan, const void* q, const void* k_new, const void* v_new,
                                         const int32_t* d_active, void* k_pool, void* v_pool, void* o,
                                         void* d_workspace, void* stream) {
    if (!plan || !q || !k_new || !v_new || !k_pool || !v_pool || !o || !d_workspace) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k_new) || !cpa_aligned16(v_new) || !cpa_aligned16(k_pool) ||
        !cpa_aligned16(v_pool) || !cpa_aligned16(o) || !cpa_aligned16(d_workspace) || (reinterpret_cast<uintptr_t>(d_active) & 3u))
        return CPA_EINVAL;
    if (!plan->d_base || !plan->dynamic) return CPA_ESTATE;
    // The host mirror counts a token for every block, stopped or not (the flags live on the device): it is an upper
    // bound of the true lengths, which is what the capacity check needs.  cpa_plan_sync reads the true ones back.
    for (int b = 0; b < plan->B; ++b)
        if ((int64_t)plan->seq_lens[b] + 1 > (int64_t)plan->block_lens[b] + plan->T) return CPA_ENOSPC;
    for (int b = 0; b < plan->B; ++b) plan->seq_lens[b] += 1;
    const int rc = cpa_decode_launch(plan, q, k_new, v_new, k_pool, v_pool, o, d_workspace,
                                     cpa_decode_mode{-1, 0, 1, d_active}, 0, stream);
    if (rc != CPA_OK) {
        for (int b = 0; b < plan->B; ++b) plan->seq_lens[b] -= 1;
        return rc;
    }
    plan->cur_lens ^= 1;
    return CPA_OK;
}

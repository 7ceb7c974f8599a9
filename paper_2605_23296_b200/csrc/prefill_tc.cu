// Varlen causal prefill attention with grouped-query heads on the 5th-generation tensor
// cores: TMA-staged tiles, tcgen05.mma with accumulators in tensor memory (TMEM), online
// softmax in fp32 registers.
//
// One unit of work = one (block, q item, query head); a q item is 256 query rows handled as two
// 128-row sub-tiles that share every K/V tile.  The grid is persistent (one CTA per SM, each
// walking its share of the units).  Twelve warps with fixed roles:
//   warps 0-3  softmax + epilogue of sub-tile 0: thread r owns query row r (TMEM lane r), so
//   warps 4-7  ... of sub-tile 1                 row max and row sum need no shuffles
//   warp 8     TMA producer (one elected lane; eight lanes for tiles of a cached prefix, which are
//              gathered from pool pages): both Q sub-tiles of a unit, then K and V tiles of 128
//              keys through rings of two (head_dim 128) or four (head_dim 64) stages
//   warp 9     MMA issuer (one elected lane) and owner of the TMEM allocation
//   warps 10-11 idle; they complete the third warpgroup so that its registers can be handed
//              to the softmax warpgroups (setmaxnreg works on whole warpgroups)
// Per KV tile j and sub-tile u (a "step"; steps are numbered n = n_sub*j + u):
//                  S    = Q_u K_j^T            (both operands K-major in shared memory)
//                  P    = exp2(scale*S - m)    (registers -> bf16 -> TMEM, over the first 64 columns of S)
//                  O_u += P V_j                (A = P from TMEM, B = V MN-major in shared memory)
// TMEM holds NBUF score buffers of 128 fp32 columns and the two O_u accumulators behind them;
// step n uses score buffer n mod NBUF.  head_dim 128 has room for two buffers (one per
// sub-tile), head_dim 64 for three.  The issuer queues PV(n), then QK(n + NBUF) into the buffer
// PV(n) has just read: MMAs of one thread execute in issue order, so that is safe, and while
// one warpgroup does its softmax the tensor core runs the other sub-tile's MMAs.  With three
// buffers the scores of a sub-tile's next KV tile are computed while its warpgroup is still
// busy with the current one, so neither side waits for the other's round trip.  O stays in
// TMEM across tiles; it is rescaled only when a row's running max grows by more than 2^8
// (the stale max is used meanwhile, which is exact after the final division by the row sum).
//
// Shared-memory tiles use the 128-byte swizzle that both TMA and the MMA descriptors
// understand: a tile is a set of column blocks of 64 bf16 (128 B) x rows, rows 128 B apart,
// 16-byte chunk c of row r stored at chunk c ^ (r & 7); every tile base is 1024-byte aligned.
//
// Every mbarrier wait is bounded: when one gives up the CTA records it in the status word,
// stops waiting, still frees its TMEM and returns.
#include <atomic>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "cpa_internal.h"
#include "cpa_tcgen05.cuh"

namespace {

constexpr int kMaxStages = 4;
struct __align__(8) TcBarriers {
    uint64_t q_full[2], q_empty[2], k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    // [sub-tile][that sub-tile's step count mod 4]: at most three steps are ever ahead of a waiter, so a
    // waiter can never meet the phase after the one it is waiting for
    uint64_t s_full[2][4], p_full[2][4], pv_done[2];
    uint64_t p_half[2][4];   // the first 64 keys' weights of a step are in TMEM (the PV MMAs over them start while the rest is computed)
    uint64_t drain;   // only used after a wait gave up: tracks the MMAs still queued, so that TMEM is not freed under them
    uint32_t tmem_base;
};

template <int D>
struct TcShape {
    static constexpr int NB = D / 64;                          // 64-wide column blocks of a Q/K/V tile
    static constexpr uint32_t kTileBytes = NB * kBlockBytes;   // one Q sub-tile, K tile or V tile
    static constexpr int kBufs = (D == 64) ? 3 : 2;            // score buffers in TMEM
    static constexpr int kStages = (D == 64) ? 4 : 2;          // K ring and V ring depth
    static constexpr bool kSplitP = (D == 128);                // the weights of a step are handed to the issuer in two halves
    static constexpr uint32_t kColO = kBufs * 128;             // O_u at kColO + u*D
    static constexpr uint32_t kTmemCols = 512;
    static constexpr int kSmem = (2 + 2 * kStages) * (int)kTileBytes + 1024;   // Q sub-tiles + rings + alignment slack
    static_assert(kColO + 2 * D <= kTmemCols, "TMEM layout");
    static_assert(kBufs <= 3 && kStages <= kMaxStages, "barrier arrays");
};

// One unit of work = one (block, q item of `q_rows` = 128 or 256 rows, query head).  A 256-row item is
// two 128-row sub-tiles u = 0, 1 that share every K/V tile; sub-tile u has its own softmax
// warpgroup and its own O_u columns in TMEM, and sees KV tiles 0 .. t0+u; the last of them touches
// the diagonal.  In the prefix-aware layout the sequence's cached prefix (whole tiles, every row sees
// all of it) comes first and is staged from the paged pool; t0 = prefix tiles + index of sub-tile 0
// among the sequence's own 128-row tiles.
struct TcWork {
    int h, g, tok0, L, q0, t0, n_sub, n_total;   // n_total: KV tiles streamed; sub-tile u uses the first t0+1+u
    int n_pre, page_base;                        // the first n_pre KV tiles are the sequence's cached prefix, read from
                                                 // pool pages page_indices[page_base ...]; t0 counts them too
    bool valid;                                  // false: this CTA has no unit in that round
};

// The grid is persistent: CTA c walks column c of the planner's schedule (units dealt greedily by
// cost, listed kv head by kv head so that the CTAs running at one time stream the same few K/V
// ranges out of L2).  Every role walks the same list with its own running counters, so the
// pipeline never drains between units: the producer is already loading the next unit's Q and
// K/V, and the issuer its first scores, while a softmax warpgroup still writes the previous
// unit's output.
template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_kpool,
                  const __grid_constant__ CUtensorMap tm_vpool, __nv_bfloat16* __restrict__ o, cpa_dev_index ix, int Hq,
                  int Hkv, int q_rows, float scale_log2, int n_rounds) {
    using Sh = TcShape<D>;
    constexpr int NB = Sh::NB;
    constexpr uint32_t kTileBytes = Sh::kTileBytes;
    constexpr int NBUF = Sh::kBufs, KS = Sh::kStages;
    constexpr bool kSplitP = Sh::kSplitP;
    constexpr uint32_t kColO = Sh::kColO;
    extern __shared__ unsigned char dsm_raw[];
    __shared__ TcBarriers bars;

    const uint32_t base = (smem_u32(dsm_raw) + 1023u) & ~1023u;
    const uint32_t s_q = base;                       // two sub-tiles
    const uint32_t s_k = s_q + 2 * kTileBytes;       // KS stages
    const uint32_t s_v = s_k + KS * kTileBytes;      // KS stages

    // (the broadcast tells the compiler that the warp index, and every role, address and counter that follows from
    // it, is the same in all lanes, so that it can keep them out of the per-thread registers)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int G = gridDim.x;
    const int group = Hq / Hkv;
    // Unit of round k for this CTA, from the planner's schedule.  Every role keeps the schedule entry of
    // round k+2 and the item record of round k+1 in flight while it works on round k, so neither of the
    // two dependent global loads sits between two units.
    auto fetch_code = [&](int k) { return k < n_rounds ? __ldg(ix.prefill_sched + (int64_t)k * G + blockIdx.x) : -1; };
    struct Rec { int4 a; int h; };   // raw item record: (first token, length, q item | prefix tiles << 16, page base)
    auto fetch = [&](int code, Rec& r) {
        r.a = make_int4(0, 0, 0, 0);                  // block length 0: no unit in that round
        r.h = 0;
        if (code >= 0) {
            const int it = code / Hq;
            r.h = code - it * Hq;
            r.a = __ldg(reinterpret_cast<const int4*>(ix.prefill_items) + it);
        }
    };
    // a value that is the same in all lanes of a warp by construction; said so to the compiler (see `warp`)
    auto uniform = [&](int x) { return __shfl_sync(0xffffffffu, x, 0); };
    auto decode = [&](const Rec& r, TcWork& w) {
        w.valid = r.a.y > 0;
        w.h = r.h;
        w.g = r.h / group;
        w.tok0 = r.a.x;
        w.L = r.a.y;
        w.q0 = (r.a.z & 0xFFFF) * q_rows;
        w.n_pre = r.a.z >> 16;
        w.page_base = r.a.w;
        w.t0 = w.n_pre + w.q0 / kTileM;
        w.n_sub = (q_rows > kTileM && w.L - w.q0 > kTileM) ? 2 : 1;
        w.n_total = w.t0 + w.n_sub;
    };

    auto bar = [&](uint64_t* p) { return smem_u32(p); };

    if (threadIdx.x == 0) {
        for (int u = 0; u < 2; ++u) {
            mbar_init(bar(&bars.q_full[u]), 1);
            mbar_init(bar(&bars.q_empty[u]), 1);
            mbar_init(bar(&bars.pv_done[u]), 1);
            for (int i = 0; i < 4; ++i) {
                mbar_init(bar(&bars.s_full[u][i]), 1);
                mbar_init(bar(&bars.p_full[u][i]), 128);
                mbar_init(bar(&bars.p_half[u][i]), 128);
            }
        }
        mbar_init(bar(&bars.drain), 1);
        for (int s = 0; s < KS; ++s) {
            mbar_init(bar(&bars.k_full[s]), 1);
            mbar_init(bar(&bars.k_empty[s]), 1);
            mbar_init(bar(&bars.v_full[s]), 1);
            mbar_init(bar(&bars.v_empty[s]), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 9) {  // TMEM allocation is warp-wide
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&bars.tmem_base)), "r"(Sh::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;
    bool dead = false;

    if (warp >= 8) {
    // the control warpgroup hands most of its registers to the softmax warpgroups
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" :: "n"(kRegsControl));
    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        // Lane 0 waits and issues the loads from the packed tensors.  A KV tile of a cached prefix is
        // eight pool pages: lanes 0-7 take one page each.  A (page, head) chunk of the pool is 16 rows
        // whose 128-byte groups are stored in the swizzled order already (see cpa_pool_piece), so a
        // plain copy of 16 rows x 128 bytes lands as rows 16p .. 16p+15 of a swizzled column block.
        {
            int kt = 0;                   // K/V tiles loaded so far: stage kt % KS, use count kt / KS
            int k_issued = 0, v_issued = 0; // K / V tiles handed to the copy engine (they differ only after a wait gave up)
            uint32_t q_loads[2] = {0, 0};   // loads of Q_u so far
            TcWork w;
            Rec rec;
            fetch(fetch_code(0), rec);
            int code = fetch_code(1);
            for (int k = 0; k < n_rounds; ++k) {
                // once a wait has given up nothing more is issued (lane 0 does the waiting: its verdict counts)
                dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                if (dead) break;
                decode(rec, w);
                fetch(code, rec);
                code = fetch_code(k + 2);
                if (!w.valid) continue;
                if (lane == 0) {
                    for (int u = 0; u < w.n_sub; ++u) {
                        // the buffer is free once the last score MMA of its previous unit has run
                        tc_wait(bar(&bars.q_empty[u]), (q_loads[u] & 1u) ^ 1u, dead, ix.status);
                        if (dead) break;
                        ++q_loads[u];
                        mbar_expect_tx(bar(&bars.q_full[u]), kTileBytes);
#pragma unroll
                        for (int c = 0; c < NB; ++c)
                            tma_load_2d(s_q + u * kTileBytes + c * kBlockBytes, &tm_q, w.h * D + 64 * c,
                                        w.tok0 + w.q0 + u * kTileM, bar(&bars.q_full[u]));
                    }
                }
                if (w.n_pre == 0) {
                    // no cached prefix: one lane streams the K/V tiles of the packed tensors
                    if (lane == 0) {
                        for (int j = 0; j < w.n_total; ++j, ++kt) {
                            const int s = kt % KS;
                            const uint32_t par = (uint32_t)(kt / KS) & 1u;
                            const int row = w.tok0 + j * kTileN;
                            tc_wait(bar(&bars.k_empty[s]), par ^ 1u, dead, ix.status);
                            if (dead) break;
                            mbar_expect_tx(bar(&bars.k_full[s]), kTileBytes);
#pragma unroll
                            for (int c = 0; c < NB; ++c)
                                tma_load_2d(s_k + s * kTileBytes + c * kBlockBytes, &tm_k, w.g * D + 64 * c, row, bar(&bars.k_full[s]));
                            ++k_issued;
                            tc_wait(bar(&bars.v_empty[s]), par ^ 1u, dead, ix.status);
                            if (dead) break;
                            mbar_expect_tx(bar(&bars.v_full[s]), kTileBytes);
#pragma unroll
                            for (int c = 0; c < NB; ++c)
                                tma_load_2d(s_v + s * kTileBytes + c * kBlockBytes, &tm_v, w.g * D + 64 * c, row, bar(&bars.v_full[s]));
                            ++v_issued;
                        }
                    } else {
                        kt += w.n_total;
                    }
                    __syncwarp();
                    continue;
                }
                // page of this lane in the next prefix tile, fetched one tile ahead
                int page = lane < 8 ? __ldg(ix.page_indices + w.page_base + lane) : 0;
                for (int j = 0; j < w.n_total; ++j, ++kt) {
                    const int s = kt % KS;
                    const uint32_t par = (uint32_t)(kt / KS) & 1u;
                    const bool cached = j < w.n_pre;
                    const int my_page = page;
                    if (lane < 8 && j + 1 < w.n_pre) page = __ldg(ix.page_indices + w.page_base + 8 * (j + 1) + lane);
                    const int row = cached ? (my_page * Hkv + w.g) * 16 : w.tok0 + (j - w.n_pre) * kTileN;
                    if (lane == 0) {
                        tc_wait(bar(&bars.k_empty[s]), par ^ 1u, dead, ix.status);
                        if (!dead) mbar_expect_tx(bar(&bars.k_full[s]), kTileBytes);
                    }
                    dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                    if (dead) break;
                    if (cached) {
                        if (lane < 8) {
#pragma unroll
                            for (int c = 0; c < NB; ++c)
                                tma_load_2d(s_k + s * kTileBytes + c * kBlockBytes + lane * 2048, &tm_kpool, 64 * c, row,
                                            bar(&bars.k_full[s]));
                        }
                    } else if (lane == 0) {
#pragma unroll
                        for (int c = 0; c < NB; ++c)
                            tma_load_2d(s_k + s * kTileBytes + c * kBlockBytes, &tm_k, w.g * D + 64 * c, row, bar(&bars.k_full[s]));
                    }
                    ++k_issued;
                    if (lane == 0) {
                        tc_wait(bar(&bars.v_empty[s]), par ^ 1u, dead, ix.status);
                        if (!dead) mbar_expect_tx(bar(&bars.v_full[s]), kTileBytes);
                    }
                    dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                    if (dead) break;
                    if (cached) {
                        if (lane < 8) {
#pragma unroll
                            for (int c = 0; c < NB; ++c)
                                tma_load_2d(s_v + s * kTileBytes + c * kBlockBytes + lane * 2048, &tm_vpool, 64 * c, row,
                                            bar(&bars.v_full[s]));
                        }
                    } else if (lane == 0) {
#pragma unroll
                        for (int c = 0; c < NB; ++c)
                            tma_load_2d(s_v + s * kTileBytes + c * kBlockBytes, &tm_v, w.g * D + 64 * c, row, bar(&bars.v_full[s]));
                    }
                    ++v_issued;
                }
            }
            // After a wait gave up: the copies issued last may still be on their way into this CTA's
            // shared memory.  Lane 0 gives the latest phase of every barrier that had a copy one more
            // bounded look before the CTA goes on to its end.
            if (__shfl_sync(0xffffffffu, (int)dead, 0) != 0 && lane == 0) {
                for (int u = 0; u < 2; ++u)
                    if (q_loads[u] > 0) mbar_drain(bar(&bars.q_full[u]), (q_loads[u] - 1u) & 1u, kDrainLimit);
                for (int t = max(0, k_issued - KS); t < k_issued; ++t)
                    mbar_drain(bar(&bars.k_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
                for (int t = max(0, v_issued - KS); t < v_issued; ++t)
                    mbar_drain(bar(&bars.v_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        // Everything the issuing thread executes between two MMAs delays the tensor core, so the
        // loops below are written out per case with as little index arithmetic as possible.
        uint32_t leader = (lane == 0);   // cleared once a wait has given up: nothing more is issued then
        constexpr uint32_t idesc_qk = instr_desc(kTileM, kTileN, false);
        constexpr uint32_t idesc_pv = instr_desc(kTileM, D, true);
        constexpr uint32_t kTile16 = kTileBytes >> 4;        // descriptor address units are 16 bytes
        // Descriptors are kept as 32-bit halves; an operand advances by adding a constant to the low half.
        const uint64_t dqk = smem_desc(0, 16, 1024), dvv = smem_desc(0, kBlockBytes, 1024);
        const uint32_t qk_hi = (uint32_t)(dqk >> 32), pv_hi = (uint32_t)(dvv >> 32);
        const uint32_t q_lo = (uint32_t)dqk | (s_q >> 4), k_lo = (uint32_t)dqk | (s_k >> 4), v_lo = (uint32_t)dvv | (s_v >> 4);
        uint32_t n_qk[2] = {0, 0}, n_pv[2] = {0, 0};   // score / PV steps issued so far per sub-tile (they pick the barrier)
        uint32_t q_uses[2] = {0, 0};                    // units that used Q_u so far
        int kt0 = 0;                                    // K/V tiles of earlier units
        auto qk = [&](int u, int buf, int kt) {   // S[buf] = Q_u K[tile kt]^T
            const uint32_t a = q_lo + u * kTile16, bq = k_lo + (kt % KS) * kTile16, d_tmem = tmem + buf * 128;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                // 16 head dims per instruction: 32 B inside the 128-B swizzled row, next block after 4 steps
                const uint32_t off = (k >> 2) * (kBlockBytes >> 4) + (k & 3) * 2;
                tc_mma_ss_lo(d_tmem, a + off, bq + off, qk_hi, idesc_qk, k > 0, leader);
            }
            tc_commit(bar(&bars.s_full[u][n_qk[u] & 3u]), leader);
            ++n_qk[u];
        };
        auto pv = [&](int u, int buf, int kt, uint32_t acc0) {   // O_u += P[buf] V[tile kt]
            const uint32_t bv = v_lo + (kt % KS) * kTile16, d_tmem = tmem + kColO + u * D, a_tmem = tmem + buf * 128;
            // With kSplitP the weights arrive in two halves of 64 keys, and the MMAs over the first half run while the
            // softmax warpgroup is still computing the second (head_dim 128, where a sub-tile's steps form one chain
            // softmax -> PV -> QK; at head_dim 64 the third score buffer has cut that chain already and the extra
            // barrier round only costs).
            if (kSplitP) {
                tc_wait(bar(&bars.p_half[u][n_pv[u] & 3u]), (n_pv[u] >> 2) & 1u, dead, ix.status);
                if (dead) leader = 0u;
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < kTileN / 32; ++k)
                    // 16 keys per instruction: 8 TMEM columns of A; 16 rows of 128 B of V, column blocks kBlockBytes apart
                    tc_mma_ts_lo(d_tmem, a_tmem + k * 8, bv + k * (2048 >> 4), pv_hi, idesc_pv, k > 0 ? 1u : acc0, leader);
            }
            tc_wait(bar(&bars.p_full[u][n_pv[u] & 3u]), (n_pv[u] >> 2) & 1u, dead, ix.status);
            if (dead) leader = 0u;
            ++n_pv[u];
            tc_fence_after();
#pragma unroll
            for (int k = kSplitP ? kTileN / 32 : 0; k < kTileN / 16; ++k)
                tc_mma_ts_lo(d_tmem, a_tmem + k * 8, bv + k * (2048 >> 4), pv_hi, idesc_pv, k > 0 ? 1u : acc0, leader);
        };
        auto wait_k = [&](int kt) {
            tc_wait(bar(&bars.k_full[kt % KS]), (uint32_t)(kt / KS) & 1u, dead, ix.status);
            if (dead) leader = 0u;
            tc_fence_after();
        };
        auto wait_v = [&](int kt) {
            tc_wait(bar(&bars.v_full[kt % KS]), (uint32_t)(kt / KS) & 1u, dead, ix.status);
            if (dead) leader = 0u;
        };
        auto wait_q = [&](int u) {
            tc_wait(bar(&bars.q_full[u]), q_uses[u] & 1u, dead, ix.status);
            if (dead) leader = 0u;
            ++q_uses[u];
        };
        // Within a unit, steps are numbered n = n_sub*j + u (KV tile j, sub-tile u); step n uses score
        // buffer n mod NBUF, and QK(n + NBUF) is queued right behind PV(n), which reads the buffer it
        // overwrites.  All buffers are free again once the last PV of a unit has been queued.
        TcWork w;
        Rec rec;
        fetch(fetch_code(0), rec);
        int code = fetch_code(1);
        for (int r = 0; r < n_rounds; ++r) {
            decode(rec, w);
            fetch(code, rec);
            code = fetch_code(r + 2);
            if (!w.valid) continue;
            const int t0 = w.t0;
            if (w.n_sub == 2) {
                int b0 = 0, b1 = 1;       // step 2j uses buffer b0, step 2j+1 buffer b1
                wait_q(0);
                wait_q(1);
                wait_k(kt0);
                qk(0, 0, kt0);
                qk(1, 1, kt0);
                tc_commit(bar(&bars.k_empty[kt0 % KS]), leader);
                if (NBUF == 3 && t0 >= 1) { wait_k(kt0 + 1); qk(0, 2, kt0 + 1); }
                // Q_u may be overwritten once the last score MMA that reads it has run
                const int last_q0 = (NBUF == 2) ? (t0 > 0 ? t0 - 1 : 0) : t0 - 2;   // iteration that queues QK_0(t0); < 0: done above
                if (NBUF == 3 && last_q0 < 0) tc_commit(bar(&bars.q_empty[0]), leader);
                for (int j = 0; j <= t0; ++j) {      // tiles both sub-tiles have; sub-tile 1 also has tile t0+1
                    const int kt = kt0 + j;
                    wait_v(kt);
                    pv(0, b0, kt, j > 0);
                    if (j == t0) tc_commit(bar(&bars.pv_done[0]), leader);
                    if (NBUF == 2) {                 // buffer b0 next holds step 2j+2 = (sub-tile 0, tile j+1)
                        if (j < t0) { wait_k(kt + 1); qk(0, b0, kt + 1); }
                        if (j == last_q0) tc_commit(bar(&bars.q_empty[0]), leader);
                    } else {                         // buffer b0 next holds step 2j+3 = (sub-tile 1, tile j+1)
                        if (j == t0) wait_k(kt + 1);  // otherwise (sub-tile 0, tile j+1) has been issued already
                        qk(1, b0, kt + 1);
                        tc_commit(bar(&bars.k_empty[(kt + 1) % KS]), leader);    // sub-tile 1 is the last reader of a K tile
                        if (j == t0) tc_commit(bar(&bars.q_empty[1]), leader);
                    }
                    pv(1, b1, kt, j > 0);
                    tc_commit(bar(&bars.v_empty[kt % KS]), leader);
                    if (NBUF == 2) {                 // buffer b1 next holds step 2j+3 = (sub-tile 1, tile j+1)
                        if (j == t0) wait_k(kt + 1);
                        qk(1, b1, kt + 1);
                        tc_commit(bar(&bars.k_empty[(kt + 1) % KS]), leader);
                        if (j == t0) tc_commit(bar(&bars.q_empty[1]), leader);
                    } else if (j + 2 <= t0) {        // buffer b1 next holds step 2j+4 = (sub-tile 0, tile j+2)
                        wait_k(kt + 2);
                        qk(0, b1, kt + 2);
                        if (j == last_q0) tc_commit(bar(&bars.q_empty[0]), leader);
                    }
                    b0 += 2; if (b0 >= NBUF) b0 -= NBUF;
                    b1 += 2; if (b1 >= NBUF) b1 -= NBUF;
                }
                wait_v(kt0 + t0 + 1);
                pv(1, b1, kt0 + t0 + 1, 1u);
                tc_commit(bar(&bars.v_empty[(kt0 + t0 + 1) % KS]), leader);
                tc_commit(bar(&bars.pv_done[1]), leader);
            } else {
                // one sub-tile: step n = tile n; with two or three buffers the scores run ahead of the softmax
                wait_q(0);
                for (int i = 0; i < NBUF && i <= t0; ++i) {
                    wait_k(kt0 + i);
                    qk(0, i, kt0 + i);
                    tc_commit(bar(&bars.k_empty[(kt0 + i) % KS]), leader);
                }
                if (t0 < NBUF) tc_commit(bar(&bars.q_empty[0]), leader);
                int buf = 0;
                for (int j = 0; j <= t0; ++j) {
                    const int kt = kt0 + j;
                    wait_v(kt);
                    pv(0, buf, kt, j > 0);
                    tc_commit(bar(&bars.v_empty[kt % KS]), leader);
                    if (j + NBUF <= t0) {
                        wait_k(kt + NBUF);
                        qk(0, buf, kt + NBUF);
                        tc_commit(bar(&bars.k_empty[(kt + NBUF) % KS]), leader);
                        if (j + NBUF == t0) tc_commit(bar(&bars.q_empty[0]), leader);
                    }
                    if (++buf == NBUF) buf = 0;
                }
                tc_commit(bar(&bars.pv_done[0]), leader);
            }
            kt0 += w.n_total;
        }
        // After a wait gave up: MMAs queued before that may still be running.  A last commit tracks them
        // and gets a bounded look, so that the tensor memory is not freed under them.
        if (__shfl_sync(0xffffffffu, (int)dead, 0) != 0) {
            tc_commit(bar(&bars.drain), (uint32_t)(lane == 0));
            if (lane == 0) mbar_drain(bar(&bars.drain), 0u, kDrainLimit);
            __syncwarp();
        }
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" :: "n"(kRegsSoftmax));
    {
        // ------------------------------------------------------------ softmax + epilogue (one warpgroup per sub-tile)
        const int u = warp >> 2;
        const int r = threadIdx.x & 127;                                  // query row inside the sub-tile = TMEM lane
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32) << 16);   // this warp's 32 TMEM lanes
        const uint32_t t_o = tmem + lane_addr + kColO + u * D;
        uint32_t n_steps = 0;       // steps of this sub-tile so far (they pick the barrier)
        uint32_t n_units = 0;       // units this sub-tile took part in
        int kt0 = 0;                // K/V tiles of earlier units
        TcWork w;
        Rec rec;
        fetch(fetch_code(0), rec);
        int code = fetch_code(1);
        for (int rd = 0; rd < n_rounds; ++rd) {
        rec.a.x = uniform(rec.a.x); rec.a.y = uniform(rec.a.y); rec.a.z = uniform(rec.a.z); rec.h = uniform(rec.h);
        decode(rec, w);
        fetch(code, rec);
        code = uniform(fetch_code(rd + 2));
        if (!w.valid) continue;
        if (u < w.n_sub) {
        const int n_kv = w.t0 + 1 + u;
        int buf = u;                // score buffer of this sub-tile's step n = n_sub*j + u, i.e. n mod NBUF
        float m_used = -INFINITY;   // row max the weights are currently scaled with (log2 units)
        float l_run = 0.f;
        for (int j = 0; j < n_kv; ++j, ++n_steps) {
            const uint32_t t_s = tmem + lane_addr + buf * 128;
            tc_wait(bar(&bars.s_full[u][n_steps & 3u]), (n_steps >> 2) & 1u, dead, ix.status);
            tc_fence_after();
            const bool diag = (j == n_kv - 1);
            uint32_t sv[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc_ld32_nowait(t_s + c * 32, sv[c]);
            tc_wait_ld();
            if (diag) {   // only the last tile touches the diagonal: keys in the row's future become -inf
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c * 32 + i > r) sv[c][i] = 0xff800000u;
            }
            // row max as a tree of 3-input max over eight independent accumulators
            float mxa[8];
#pragma unroll
            for (int a = 0; a < 8; ++a) mxa[a] = max3(__uint_as_float(sv[0][a]), __uint_as_float(sv[0][a + 8]), __uint_as_float(sv[0][a + 16]));
#pragma unroll
            for (int a = 0; a < 8; ++a) mxa[a] = fmaxf(mxa[a], __uint_as_float(sv[0][a + 24]));
#pragma unroll
            for (int c = 1; c < 4; ++c)
#pragma unroll
                for (int a = 0; a < 8; ++a) {
                    mxa[a] = max3(mxa[a], __uint_as_float(sv[c][a]), __uint_as_float(sv[c][a + 8]));
                    mxa[a] = max3(mxa[a], __uint_as_float(sv[c][a + 16]), __uint_as_float(sv[c][a + 24]));
                }
            float mx = max3(max3(mxa[0], mxa[1], mxa[2]), max3(mxa[3], mxa[4], mxa[5]), fmaxf(mxa[6], mxa[7]));
            mx *= scale_log2;       // scale > 0, so the max commutes with the scaling
            // lazy rescale: keep the old reference max unless the new one is more than 2^8 above it
            float alpha = 1.f;
            if (mx > m_used + 8.f) {
                alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - mx);
                m_used = mx;
            }
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                // O_u must hold every earlier tile before it is rescaled, and the scores of this tile may
                // have been ready before PV of the previous one has run.  The release of V tile j-1 is
                // committed behind the last PV that reads it, which is issued after PV_u(j-1).
                const int kt = kt0 + j - 1;
                tc_wait(bar(&bars.v_empty[kt % KS]), (uint32_t)(kt / KS) & 1u, dead, ix.status);
                tc_fence_after();
                // (rare, and the tile's scores are live in registers meanwhile: eight columns at a time, so that this
                // path does not make the compiler spill in the loop around it)
#pragma unroll 1
                for (int c = 0; c < D / 8; ++c) {
                    float v[8];
                    tc_ld8(t_o + c * 8, v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] *= alpha;
                    tc_st8(t_o + c * 8, v);
                }
            }
            l_run *= alpha;
            // weights, rounded to bf16, two keys per 32-bit TMEM column (P over the first 64 columns of S)
            float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            const float neg_m = -m_used;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float x0 = __uint_as_float(sv[c][i]), x1 = __uint_as_float(sv[c][i + 1]);
                    fma_x2(x0, x1, scale_log2, neg_m);
                    const uint32_t w2 = pack_bf16(exp2f(x0), exp2f(x1));
                    pk[i >> 1] = w2;
                    // row sum over the rounded weights (numerator and denominator stay consistent);
                    // the bf16 halves are added to the fp32 sum directly
                    add_bf16x2(sum[(i >> 1) & 7], w2);
                }
                tc_st16(t_s + c * 16, pk);
                if (kSplitP && c == 1) {   // the first 64 keys' weights are in place: let their MMAs start
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(bar(&bars.p_half[u][n_steps & 3u]));
                }
            }
            l_run += ((sum[0] + sum[1]) + (sum[2] + sum[3])) + ((sum[4] + sum[5]) + (sum[6] + sum[7]));
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(&bars.p_full[u][n_steps & 3u]));
            buf += w.n_sub;
            if (buf >= NBUF) buf -= NBUF;
        }
        // ---- epilogue: O / l -> bf16 -> global; thread r owns row r and writes it in 64-byte runs.
        // O_u is overwritten by the next unit's first PV, which waits for this warpgroup's next weights.
        tc_wait(bar(&bars.pv_done[u]), n_units & 1u, dead, ix.status);
        ++n_units;
        tc_fence_after();
        const float inv = 1.f / l_run;
        // rows past the end of the block belong to the next block (or to nobody): never store them
        const bool row_ok = !dead && r < w.L - (w.q0 + u * kTileM);
        __nv_bfloat16* dst = o + ((int64_t)(w.tok0 + w.q0 + u * kTileM + r) * Hq + w.h) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            float v[32];
            tc_ld32(t_o + c * 32, v);
            if (row_ok) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 q4;
                    q4.x = pack_bf16(v[i] * inv, v[i + 1] * inv);
                    q4.y = pack_bf16(v[i + 2] * inv, v[i + 3] * inv);
                    q4.z = pack_bf16(v[i + 4] * inv, v[i + 5] * inv);
                    q4.w = pack_bf16(v[i + 6] * inv, v[i + 7] * inv);
                    *reinterpret_cast<uint4*>(dst + c * 32 + i) = q4;
                }
            }
        }
        tc_fence_before();
        }
        kt0 += w.n_total;
        }
    }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(Sh::kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- shared-prefix scan (decode, prefix-aware layout)
// The decode step of the prefix-aware layout reads the cached history once for all workers: one
// unit = (group of consecutive workers, kv head, chunk of shared pages).  The group's (worker, query
// head) rows (row = worker * G + head, at most 128) are the rows of ONE 128-row tile, the chunk's
// pages are its KV tiles (eight pages each, gathered from the pool like a cached prefix in the
// prefill kernel), and the loop is the prefill kernel's single-sub-tile loop without a diagonal:
// a row sees a KV tile iff the tile lies below its worker's prefix (prefixes are whole tiles).
// Instead of a normalised output every row that saw a tile leaves a partial
// (reference max in log2 units, sum, unnormalised accumulator) in slot `chunk` of its worker;
// the per-worker decode kernel that follows in the stream merges those with its own partials.
// Eight warps: 0-3 softmax (thread r owns row r), 4 producer, 5 MMA issuer, 6-7 idle.
constexpr int kScanThreads = 256;

template <int D>
struct ScanShape {
    static constexpr int NB = D / 64;
    static constexpr uint32_t kTileBytes = NB * kBlockBytes;
    static constexpr int kBufs = 2;                            // score buffers in TMEM
    static constexpr int kStages = (D == 64) ? 6 : 3;          // K ring and V ring depth
    static constexpr uint32_t kColO = kBufs * 128;
    static constexpr uint32_t kTmemCols = 512;
    static constexpr int kSmem = (1 + 2 * kStages) * (int)kTileBytes + 1024;
};

struct __align__(8) ScanBarriers {
    uint64_t q_full, q_empty, k_full[6], k_empty[6], v_full[6], v_empty[6], s_full[4], p_full[4], pv_done;
    uint64_t drain;   // only used after a wait gave up (see TcBarriers)
    uint32_t tmem_base;
};

template <int D>
__global__ void __launch_bounds__(kScanThreads, 1)
scan_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kpool,
               const __grid_constant__ CUtensorMap tm_vpool, float* __restrict__ part_ml, float* __restrict__ part_o,
               cpa_dev_index ix, int Hq, int Hkv, int G, float scale_log2, int n_units) {
    using Sh = ScanShape<D>;
    constexpr int NB = Sh::NB;
    constexpr uint32_t kTileBytes = Sh::kTileBytes;
    constexpr int NBUF = Sh::kBufs, KS = Sh::kStages;
    constexpr uint32_t kColO = Sh::kColO;
    extern __shared__ unsigned char dsm_raw[];
    __shared__ ScanBarriers bars;

    const uint32_t base = (smem_u32(dsm_raw) + 1023u) & ~1023u;
    const uint32_t s_q = base;
    const uint32_t s_k = s_q + kTileBytes;
    const uint32_t s_v = s_k + KS * kTileBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    auto bar = [&](uint64_t* p) { return smem_u32(p); };

    if (threadIdx.x == 0) {
        mbar_init(bar(&bars.q_full), 1);
        mbar_init(bar(&bars.q_empty), 1);
        mbar_init(bar(&bars.pv_done), 1);
        mbar_init(bar(&bars.drain), 1);
        for (int s = 0; s < KS; ++s) {
            mbar_init(bar(&bars.k_full[s]), 1);
            mbar_init(bar(&bars.k_empty[s]), 1);
            mbar_init(bar(&bars.v_full[s]), 1);
            mbar_init(bar(&bars.v_empty[s]), 1);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar(&bars.s_full[i]), 1);
            mbar_init(bar(&bars.p_full[i]), 128);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&bars.tmem_base)), "r"(Sh::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // the per-worker kernel of this step is next in the stream and needs this one only for its merge
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const uint32_t tmem = bars.tmem_base;
    bool dead = false;
    // unit u of this CTA: (first worker | workers << 16, kv head, chunk, pages)
    auto unit = [&](int u) { return __ldg(reinterpret_cast<const int4*>(ix.shared_items) + u); };

    if (warp == 4) {
        // ------------------------------------------------------------ producer (whole warp)
        int kt = 0, k_issued = 0, v_issued = 0;
        uint32_t q_loads = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int4 it = unit(u);
            const int w0 = it.x & 0xFFFF, nw = it.x >> 16, g = it.y, first = it.z * ix.shared_chunk, n_tiles = it.w / 8;
            // The query rows come in boxes of eight tile rows = 8/G workers x G heads of this kv group (a whole
            // swizzle atom each); a box that reaches past the last worker is filled with zeros.
            const int per_box = 8 / G, n_boxes = (nw + per_box - 1) / per_box;
            if (lane == 0) {
                tc_wait(bar(&bars.q_empty), (q_loads & 1u) ^ 1u, dead, ix.status);
                if (!dead) mbar_expect_tx(bar(&bars.q_full), (uint32_t)(n_boxes * NB * 1024));
            }
            // once a wait has given up nothing more is issued (lane 0 does the waiting: its verdict counts)
            dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
            if (dead) break;
            ++q_loads;
            for (int bx = lane; bx < n_boxes; bx += 32) {
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    tma_load_3d(s_q + c * kBlockBytes + bx * 1024, &tm_q, 64 * c, g * G, w0 + bx * per_box, bar(&bars.q_full));
            }
            int page = lane < 8 ? __ldg(ix.shared_page_ids + first + lane) : 0;
            for (int j = 0; j < n_tiles; ++j, ++kt) {
                const int s = kt % KS;
                const uint32_t par = (uint32_t)(kt / KS) & 1u;
                const int row = (page * Hkv + g) * 16;
                if (lane < 8 && j + 1 < n_tiles) page = __ldg(ix.shared_page_ids + first + 8 * (j + 1) + lane);
                if (lane == 0) {
                    tc_wait(bar(&bars.k_empty[s]), par ^ 1u, dead, ix.status);
                    if (!dead) mbar_expect_tx(bar(&bars.k_full[s]), kTileBytes);
                }
                dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                if (dead) break;
                if (lane < 8) {
#pragma unroll
                    for (int c = 0; c < NB; ++c)
                        tma_load_2d(s_k + s * kTileBytes + c * kBlockBytes + lane * 2048, &tm_kpool, 64 * c, row, bar(&bars.k_full[s]));
                }
                ++k_issued;
                if (lane == 0) {
                    tc_wait(bar(&bars.v_empty[s]), par ^ 1u, dead, ix.status);
                    if (!dead) mbar_expect_tx(bar(&bars.v_full[s]), kTileBytes);
                }
                dead = __shfl_sync(0xffffffffu, (int)dead, 0) != 0;
                if (dead) break;
                if (lane < 8) {
#pragma unroll
                    for (int c = 0; c < NB; ++c)
                        tma_load_2d(s_v + s * kTileBytes + c * kBlockBytes + lane * 2048, &tm_vpool, 64 * c, row, bar(&bars.v_full[s]));
                }
                ++v_issued;
            }
            if (dead) break;
        }
        // after a wait gave up: one last bounded look at the copies that may still be in flight (see the prefill kernel)
        if (dead && lane == 0) {
            if (q_loads > 0) mbar_drain(bar(&bars.q_full), (q_loads - 1u) & 1u, kDrainLimit);
            for (int t = max(0, k_issued - KS); t < k_issued; ++t)
                mbar_drain(bar(&bars.k_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
            for (int t = max(0, v_issued - KS); t < v_issued; ++t)
                mbar_drain(bar(&bars.v_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer (whole warp, one lane issues)
        uint32_t leader = (lane == 0);   // cleared once a wait has given up
        constexpr uint32_t idesc_qk = instr_desc(kTileM, kTileN, false);
        constexpr uint32_t idesc_pv = instr_desc(kTileM, D, true);
        constexpr uint32_t kTile16 = kTileBytes >> 4;
        const uint64_t dqk = smem_desc(0, 16, 1024), dvv = smem_desc(0, kBlockBytes, 1024);
        const uint32_t qk_hi = (uint32_t)(dqk >> 32), pv_hi = (uint32_t)(dvv >> 32);
        const uint32_t q_lo = (uint32_t)dqk | (s_q >> 4), k_lo = (uint32_t)dqk | (s_k >> 4), v_lo = (uint32_t)dvv | (s_v >> 4);
        uint32_t n_qk = 0, n_pv = 0, q_uses = 0;
        int kt0 = 0;
        auto qk = [&](int buf, int kt) {
            const uint32_t bq = k_lo + (kt % KS) * kTile16, d_tmem = tmem + buf * 128;
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = (k >> 2) * (kBlockBytes >> 4) + (k & 3) * 2;
                tc_mma_ss_lo(d_tmem, q_lo + off, bq + off, qk_hi, idesc_qk, k > 0, leader);
            }
            tc_commit(bar(&bars.s_full[n_qk & 3u]), leader);
            ++n_qk;
            tc_commit(bar(&bars.k_empty[kt % KS]), leader);
        };
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int t_last = unit(u).w / 8 - 1;      // tiles 0 .. t_last
            tc_wait(bar(&bars.q_full), q_uses & 1u, dead, ix.status);
            if (dead) leader = 0u;
            ++q_uses;
            for (int i = 0; i < NBUF && i <= t_last; ++i) {
                tc_wait(bar(&bars.k_full[(kt0 + i) % KS]), (uint32_t)((kt0 + i) / KS) & 1u, dead, ix.status);
                if (dead) leader = 0u;
                tc_fence_after();
                qk(i, kt0 + i);
            }
            if (t_last < NBUF) tc_commit(bar(&bars.q_empty), leader);
            int buf = 0;
            for (int j = 0; j <= t_last; ++j) {
                const int kt = kt0 + j;
                tc_wait(bar(&bars.v_full[kt % KS]), (uint32_t)(kt / KS) & 1u, dead, ix.status);
                tc_wait(bar(&bars.p_full[n_pv & 3u]), (n_pv >> 2) & 1u, dead, ix.status);
                if (dead) leader = 0u;
                ++n_pv;
                tc_fence_after();
                const uint32_t bv = v_lo + (kt % KS) * kTile16, d_tmem = tmem + kColO, a_tmem = tmem + buf * 128;
#pragma unroll
                for (int k = 0; k < kTileN / 16; ++k)
                    tc_mma_ts_lo(d_tmem, a_tmem + k * 8, bv + k * (2048 >> 4), pv_hi, idesc_pv, k > 0 ? 1u : (uint32_t)(j > 0), leader);
                tc_commit(bar(&bars.v_empty[kt % KS]), leader);
                if (j + NBUF <= t_last) {
                    tc_wait(bar(&bars.k_full[(kt + NBUF) % KS]), (uint32_t)((kt + NBUF) / KS) & 1u, dead, ix.status);
                    if (dead) leader = 0u;
                    tc_fence_after();
                    qk(buf, kt + NBUF);
                    if (j + NBUF == t_last) tc_commit(bar(&bars.q_empty), leader);
                }
                if (++buf == NBUF) buf = 0;
            }
            tc_commit(bar(&bars.pv_done), leader);
            kt0 += t_last + 1;
        }
        // after a wait gave up: track the MMAs still queued, so that the tensor memory is not freed under them
        if (__shfl_sync(0xffffffffu, (int)dead, 0) != 0) {
            tc_commit(bar(&bars.drain), (uint32_t)(lane == 0));
            if (lane == 0) mbar_drain(bar(&bars.drain), 0u, kDrainLimit);
            __syncwarp();
        }
    } else if (warp < 4) {
        // ------------------------------------------------------------ softmax + partial write-out (thread r owns row r)
        const int r = threadIdx.x;
        const uint32_t lane_addr = ((uint32_t)(warp * 32) << 16);
        const uint32_t t_o = tmem + lane_addr + kColO;
        uint32_t n_steps = 0, n_units_done = 0;
        int kt0 = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const int4 it = unit(u);
            const int w0 = it.x & 0xFFFF, nw = it.x >> 16, g = it.y, chunk = it.z, n_tiles = it.w / 8;
            const int tile0 = chunk * ix.shared_chunk / 8;            // first KV tile of the chunk in the history
            const bool real = r < nw * G;
            const int wk = w0 + (real ? r / G : 0), hd = real ? r % G : 0;
            const int vis_tiles = real ? __ldg(ix.prefix_lens + wk) / kTileN : 0;   // the row sees history tiles below this
            float m_used = -INFINITY, l_run = 0.f;
            int buf = 0;
            for (int j = 0; j < n_tiles; ++j, ++n_steps) {
                const uint32_t t_s = tmem + lane_addr + buf * 128;
                tc_wait(bar(&bars.s_full[n_steps & 3u]), (n_steps >> 2) & 1u, dead, ix.status);
                tc_fence_after();
                const bool visible = tile0 + j < vis_tiles;
                uint32_t sv[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tc_ld32_nowait(t_s + c * 32, sv[c]);
                tc_wait_ld();
                float mxa[8];
#pragma unroll
                for (int a = 0; a < 8; ++a) mxa[a] = max3(__uint_as_float(sv[0][a]), __uint_as_float(sv[0][a + 8]), __uint_as_float(sv[0][a + 16]));
#pragma unroll
                for (int a = 0; a < 8; ++a) mxa[a] = fmaxf(mxa[a], __uint_as_float(sv[0][a + 24]));
#pragma unroll
                for (int c = 1; c < 4; ++c)
#pragma unroll
                    for (int a = 0; a < 8; ++a) {
                        mxa[a] = max3(mxa[a], __uint_as_float(sv[c][a]), __uint_as_float(sv[c][a + 8]));
                        mxa[a] = max3(mxa[a], __uint_as_float(sv[c][a + 16]), __uint_as_float(sv[c][a + 24]));
                    }
                float mx = max3(max3(mxa[0], mxa[1], mxa[2]), max3(mxa[3], mxa[4], mxa[5]), fmaxf(mxa[6], mxa[7])) * scale_log2;
                // a row that does not see the tile (or is no row at all) contributes zeros and keeps its state;
                // its scores may be anything, NaN included, so they are not looked at
                float alpha = 1.f;
                if (visible && mx > m_used + 8.f) {       // lazy reference max, as in the prefill kernel
                    alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - mx);
                    m_used = mx;
                }
                if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    const int kt = kt0 + j - 1;   // O must hold every earlier tile: V tile j-1 is released behind PV(j-1)
                    tc_wait(bar(&bars.v_empty[kt % KS]), (uint32_t)(kt / KS) & 1u, dead, ix.status);
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        float v[32];
                        tc_ld32(t_o + c * 32, v);
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] *= alpha;
                        tc_st32(t_o + c * 32, v);
                    }
                }
                l_run *= alpha;
                float sum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                const float neg_m = -m_used;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0 = __uint_as_float(sv[c][i]), x1 = __uint_as_float(sv[c][i + 1]);
                        fma_x2(x0, x1, scale_log2, neg_m);
                        const uint32_t w2 = visible ? pack_bf16(exp2f(x0), exp2f(x1)) : 0u;
                        pk[i >> 1] = w2;
                        add_bf16x2(sum[(i >> 1) & 7], w2);
                    }
                    tc_st16(t_s + c * 16, pk);
                }
                l_run += ((sum[0] + sum[1]) + (sum[2] + sum[3])) + ((sum[4] + sum[5]) + (sum[6] + sum[7]));
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(&bars.p_full[n_steps & 3u]));
                if (++buf == NBUF) buf = 0;
            }
            // ---- the row's partial: (reference max, sum) and the unnormalised accumulator
            tc_wait(bar(&bars.pv_done), n_units_done & 1u, dead, ix.status);
            ++n_units_done;
            tc_fence_after();
            const bool write = real && !dead && m_used != -INFINITY;
            const int64_t prow = write ? (int64_t)(__ldg(ix.split_indptr + wk) + chunk) * Hq + g * G + hd : 0;
            if (write) *reinterpret_cast<float2*>(part_ml + prow * 2) = make_float2(m_used, l_run);
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                float v[32];
                tc_ld32(t_o + c * 32, v);
                if (write) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4*>(part_o + prow * D + c * 32 + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                }
            }
            tc_fence_before();
            kt0 += n_tiles;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(Sh::kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
// 2-D view [rows = tokens][cols = heads*D] of a packed token-major tensor; box = 64 cols x 128 rows.
bool make_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D view [rows = pages * kv_heads * 16 slots][cols = D] of a paged pool; box = 64 cols x 16 rows (one
// 128-byte group of every slot of a (page, head) chunk), copied as stored.
bool make_pool_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, 16};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int launch_prefill_tc(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, const void* k_pool,
                      const void* v_pool, const int32_t* items, const int32_t* sched, int ctas, int rounds,
                      cudaStream_t st) {
    const cpa_config& c = plan->cfg;
    constexpr int smem = TcShape<D>::kSmem;
    // the attribute is per device: remember which devices have it (relaxed flags: setting it twice is harmless)
    static std::atomic<bool> configured_dev[64];
    int dev_id = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess || dev_id < 0 || dev_id >= 64) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    std::atomic<bool>& configured = configured_dev[dev_id];
    if (!configured.load(std::memory_order_relaxed)) {
        cudaFuncAttributes attr;
        if (cudaFuncGetAttributes(&attr, prefill_tc_kernel<D>) != cudaSuccess ||
            cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        // The in-kernel register split may only hand out what the launch allocates; a kernel
        // that asked for more would wait for registers forever, so refuse to launch it.
        if (attr.numRegs * kThreads < 2 * 128 * kRegsSoftmax + 128 * kRegsControl) return CPA_EUNSUPPORTED;
        configured.store(true, std::memory_order_relaxed);
    }
    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, q, plan->total_tokens, (int64_t)c.num_q_heads * D) ||
        !make_map(&tm_k, k, plan->total_tokens, (int64_t)c.num_kv_heads * D) ||
        !make_map(&tm_v, v, plan->total_tokens, (int64_t)c.num_kv_heads * D))
        return CPA_ECUDA;
    // pools are only read for sequences with a cached prefix; without pools the maps are never used
    CUtensorMap tm_kpool = tm_k, tm_vpool = tm_v;
    if (k_pool && v_pool) {
        const int64_t pool_rows = (int64_t)plan->pool_pages * c.num_kv_heads * c.page_size;
        if (!make_pool_map(&tm_kpool, k_pool, pool_rows, D) || !make_pool_map(&tm_vpool, v_pool, pool_rows, D))
            return CPA_ECUDA;
    }
    // persistent grid: one CTA per SM, each walks its column of the planner's schedule (the plan's whole-block
    // list, or the list of one chunk step)
    cpa_dev_index ix = plan->dev();
    if (items) {
        ix.prefill_items = items;
        ix.prefill_sched = sched;
    } else {
        ctas = plan->prefill_ctas;
        rounds = plan->prefill_rounds;
    }
    if (ctas < 1) return CPA_OK;   // nothing to prefill
    prefill_tc_kernel<D><<<ctas, kThreads, smem, st>>>(tm_q, tm_k, tm_v, tm_kpool, tm_vpool, (__nv_bfloat16*)o, ix,
                                                     c.num_q_heads, c.num_kv_heads, plan->q_tile,
                                                     c.scale * 1.4426950408889634f, rounds);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

// 3-D view [sequences][heads][D] of the decode queries; box = 64 cols x G heads (one kv group) x 8/G
// sequences = eight rows of the scan's query tile.
bool make_q_rows_map(CUtensorMap* map, const void* ptr, int64_t seqs, int64_t heads, int64_t cols, int group) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)heads, (cuuint64_t)seqs};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)heads * cols * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)group, (cuuint32_t)(8 / group)};
    const cuuint32_t elem[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
int launch_scan_tc(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool, float* part_ml,
                   float* part_o, int wave_sms, cudaStream_t st) {
    const cpa_config& c = plan->cfg;
    constexpr int smem = ScanShape<D>::kSmem;
    static std::atomic<bool> configured_dev[64];
    int dev_id = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess || dev_id < 0 || dev_id >= 64) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    if (!configured_dev[dev_id].load(std::memory_order_relaxed)) {
        if (cudaFuncSetAttribute(scan_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        configured_dev[dev_id].store(true, std::memory_order_relaxed);
    }
    const int G = c.num_q_heads / c.num_kv_heads;
    if (8 % G != 0) return CPA_EUNSUPPORTED;   // the query tile is loaded in boxes of 8/G sequences
    CUtensorMap tm_q, tm_kpool, tm_vpool;
    const int64_t pool_rows = (int64_t)plan->pool_pages * c.num_kv_heads * c.page_size;
    if (!make_q_rows_map(&tm_q, q, plan->B, c.num_q_heads, D, G) ||
        !make_pool_map(&tm_kpool, k_pool, pool_rows, D) || !make_pool_map(&tm_vpool, v_pool, pool_rows, D))
        return CPA_ECUDA;
    const int sms = wave_sms > 0 ? wave_sms : plan->num_sms;   // (beside a prefill chunk: the SMs left to the decode)
    const int grid = plan->n_shared < sms ? plan->n_shared : sms;
    scan_tc_kernel<D><<<grid, kScanThreads, smem, st>>>(tm_q, tm_kpool, tm_vpool, part_ml, part_o, plan->dev(),
                                                       c.num_q_heads, c.num_kv_heads, G, c.scale * 1.4426950408889634f,
                                                       plan->n_shared);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

}  // namespace

int cpa_scan_tc(const cpa_plan* plan, const void* q, const void* k_pool, const void* v_pool, float* part_ml,
                float* part_o, int wave_sms, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_scan_tc<128>(plan, q, k_pool, v_pool, part_ml, part_o, wave_sms, st)
                                     : launch_scan_tc<64>(plan, q, k_pool, v_pool, part_ml, part_o, wave_sms, st);
}

int cpa_prefill_tc_list(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, const void* k_pool,
                        const void* v_pool, const int32_t* items, const int32_t* sched, int ctas, int rounds, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128
               ? launch_prefill_tc<128>(plan, q, k, v, o, k_pool, v_pool, items, sched, ctas, rounds, st)
               : launch_prefill_tc<64>(plan, q, k, v, o, k_pool, v_pool, items, sched, ctas, rounds, st);
}

int cpa_prefill_tc(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, const void* k_pool,
                   const void* v_pool, void* stream) {
    if (plan->q_tile == 512) return cpa_prefill_pairs(plan, q, k, v, o, stream);   // 512-row items run on pairs of CTAs
    return cpa_prefill_tc_list(plan, q, k, v, o, k_pool, v_pool, nullptr, nullptr, 0, 0, stream);
}

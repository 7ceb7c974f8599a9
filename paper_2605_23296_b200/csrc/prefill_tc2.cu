// Varlen causal prefill attention on PAIRS of CTAs (thread-block clusters of two, tcgen05 cta_group::2), for
// head_dim 128 and plans without cached prefixes.
//
// Why pairs.  In the one-CTA kernel (prefill_tc.cu) the thread that issues the MMAs is the bottleneck: an
// instruction costs it 85-100 cycles while the tensor core needs 64 (head_dim 128) for it.  With cta_group::2
// one instruction of the pair's leader drives the tensor cores of both SMs: D rows 0-127 live in the leader's
// tensor memory, rows 128-255 in its peer's, A comes from each CTA's own shared memory (or tensor memory), and
// each CTA supplies HALF of B from its shared memory.  The issue cost is paid once for twice the work, and a
// CTA stages only half of every K and V tile.
//
// One unit of work = one (block, q item of 512 rows, query head).  The rows are four sub-tiles of 128; CTA r of
// the pair owns sub-tiles r and 2 + r ("slot" 0 and 1, each with its own softmax warpgroup, score buffer and O
// accumulator, exactly as in the one-CTA kernel), so that one MMA covers sub-tiles (2p, 2p+1) = slot p of both
// CTAs.  Sub-tile i sees KV tiles 0 .. t0+i; slot p therefore runs tiles 0 .. t0+2p+1, the last of which is past
// the diagonal for the leader's sub-tile (its weights are zero and its state stays).
//
// Per CTA: warps 0-3 / 4-7 softmax + epilogue of slot 0 / 1 (thread r owns row r), warp 8 TMA producer (its own Q
// sub-tiles, keys 64r..64r+63 of every K tile, head dims 64r..64r+63 of every V tile), warp 9 MMA issuer (leader
// only) and owner of the CTA's tensor-memory allocation, warps 10-11 idle (register donors).
//
// Synchronisation across the pair:
//   - "full" barriers (Q, K, V landed) live in the leader; both CTAs' TMA loads count their bytes there
//     (cp.async.bulk.tensor with .cta_group::2 may complete on the peer's barrier); the leader arms them.
//   - "empty" / "scores ready" / "output ready" barriers exist in both CTAs and are arrived at by the leader's
//     tcgen05.commit with .multicast::cluster.
//   - "weights ready" barriers live in the leader and count 8 arrivals, one per softmax warp of the slot: 4 local,
//     4 remote (mbarrier.arrive.release.cluster on the mapped address).
// Every wait is bounded; a wait that gives up records it in the status word and the kernel runs to its end.
#include <atomic>

#include "cpa_internal.h"
#include "cpa_tcgen05.cuh"

namespace {

constexpr int kPairStages = 4;          // K ring and V ring depth (half tiles of 16 KB)
constexpr int kPairRows = 512;          // query rows of a unit

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;\n" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// Arrival at a barrier of the peer CTA.  Relaxed: what the arrival publishes is tensor memory, whose stores have
// completed (tcgen05.wait::st) and are ordered by tcgen05.fence::before_thread_sync; a release at cluster scope
// would add a fence over all of the thread's memory traffic to every step of the softmax.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];\n" :: "r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait on a barrier that threads of the peer CTA arrive at (acquire at cluster scope).
__device__ __forceinline__ void pair_wait(uint32_t bar, uint32_t parity, bool& dead, int32_t* status) {
    if (dead) return;
    uint32_t spins = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
        if (++spins > kSpinLimit) {
            dead = true;
            atomicCAS(status, 0, kStatusWaitGaveUp);
            return;
        }
    }
}
// TMA tile load into this CTA's shared memory whose bytes are counted on `bar`, a shared::cluster address that may
// belong to the peer CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
        :: "r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// tcgen05.commit of the pair's MMAs, arriving at the barrier at this shared-memory offset in both CTAs.
__device__ __forceinline__ void pair_commit(uint32_t bar, uint32_t leader) {
    asm volatile("{\n .reg .pred q;\n .reg .b16 m;\n setp.ne.b32 q, %1, 0;\n mov.b16 m, 3;\n"
                 " @q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n}\n"
                 :: "r"(bar), "r"(leader) : "memory");
}
__device__ __forceinline__ void pair_commit_local(uint32_t bar, uint32_t leader) {
    asm volatile("{\n .reg .pred q;\n setp.ne.b32 q, %1, 0;\n"
                 " @q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n"
                 :: "r"(bar), "r"(leader) : "memory");
}
__device__ __forceinline__ void pair_mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                            uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n .reg .pred p, q;\n .reg .b64 da, db;\n setp.ne.b32 p, %5, 0;\n setp.ne.b32 q, %6, 0;\n"
        " mov.b64 da, {%1, %3};\n mov.b64 db, {%2, %3};\n"
        " @q tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %4, p;\n}\n"
        :: "r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}
__device__ __forceinline__ void pair_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                            uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n .reg .pred p, q;\n .reg .b64 db;\n setp.ne.b32 p, %5, 0;\n setp.ne.b32 q, %6, 0;\n"
        " mov.b64 db, {%2, %3};\n"
        " @q tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %4, p;\n}\n"
        :: "r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}

struct __align__(8) PairBarriers {
    uint64_t q_full[2];                                    // leader: both CTAs' Q sub-tiles of a slot have landed
    uint64_t q_empty[2];                                   // both: the slot's Q may be overwritten
    uint64_t k_full[kPairStages], v_full[kPairStages];     // leader
    uint64_t k_empty[kPairStages], v_empty[kPairStages];   // both
    uint64_t s_full[2][4];                                 // both: scores of a step are in tensor memory
    uint64_t p_half[2][4], p_full[2][4];                   // leader: weights of a step (first 64 keys / all) of both CTAs
    uint64_t pv_done[2];                                   // both: a slot's output is complete
    uint64_t drain;                                        // leader, only after a wait gave up
    uint32_t tmem_base;
};

// Work of one round for the pair, from the item record (first token of the block, block length, q item, unused).
struct PairWork {
    int h, g, tok0, L, q0, t0, n_pt, n_total;
    int T0, T1;      // KV tiles slot 0 / 1 runs: tiles 0 .. T-1
    bool valid;
    __device__ __forceinline__ int T(int p) const { return p ? T1 : T0; }
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_khalf,
                    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, cpa_dev_index ix, int Hq,
                    int Hkv, float scale_log2, int n_rounds, int n_pairs) {
    static_assert(D == 128, "the pair kernel is written for head_dim 128");
    constexpr int NB = D / 64;
    constexpr uint32_t kTileBytes = NB * kBlockBytes;          // one Q sub-tile: 128 rows x D
    constexpr uint32_t kKHalfBlock = 64 * 128;                 // 64 keys x 128 B: one column block of a K half
    constexpr uint32_t kHalfBytes = 16 * 1024;                 // a K half (64 keys x D) or a V half (128 keys x 64 dims)
    constexpr int KS = kPairStages;
    constexpr uint32_t kColO = 2 * 128;                        // O of slot p at kColO + p * D
    extern __shared__ unsigned char dsm_raw[];
    __shared__ PairBarriers bars;

    const uint32_t base = (smem_u32(dsm_raw) + 1023u) & ~1023u;
    const uint32_t s_q = base;                       // two slots
    const uint32_t s_k = s_q + 2 * kTileBytes;       // KS stages of K halves
    const uint32_t s_v = s_k + KS * kHalfBytes;      // KS stages of V halves

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();         // 0 = leader of the pair
    const int pair = blockIdx.x >> 1;
    const int group = Hq / Hkv;

    auto fetch_code = [&](int k) { return k < n_rounds ? __ldg(ix.prefill_sched + (int64_t)k * n_pairs + pair) : -1; };
    struct Rec { int4 a; int h; };
    auto fetch = [&](int code, Rec& r) {
        r.a = make_int4(0, 0, 0, 0);
        r.h = 0;
        if (code >= 0) {
            const int it = code / Hq;
            r.h = code - it * Hq;
            r.a = __ldg(reinterpret_cast<const int4*>(ix.prefill_items) + it);
        }
    };
    auto decode = [&](const Rec& r, PairWork& w) {
        w.valid = r.a.y > 0;
        w.h = r.h;
        w.g = r.h / group;
        w.tok0 = r.a.x;
        w.L = r.a.y;
        w.q0 = (r.a.z & 0xFFFF) * kPairRows;
        w.t0 = w.q0 / kTileM;
        const int n_sub = min(4, (w.L - w.q0 + kTileM - 1) / kTileM);   // sub-tiles that hold rows of the block
        w.n_pt = (n_sub + 1) / 2;
        // slot p = sub-tiles 2p (leader) and 2p+1 (peer); without rows in the peer's sub-tile the tile past the
        // leader's diagonal is not needed
        w.T0 = w.t0 + (n_sub > 1 ? 2 : 1);
        w.T1 = w.n_pt == 2 ? w.t0 + (n_sub > 3 ? 4 : 3) : 0;
        w.n_total = w.n_pt == 2 ? w.T1 : w.T0;
    };
    auto bar = [&](uint64_t* p) { return smem_u32(p); };

    if (threadIdx.x == 0) {
        for (int p = 0; p < 2; ++p) {
            mbar_init(bar(&bars.q_full[p]), 1);
            mbar_init(bar(&bars.q_empty[p]), 1);
            mbar_init(bar(&bars.pv_done[p]), 1);
            for (int i = 0; i < 4; ++i) {
                mbar_init(bar(&bars.s_full[p][i]), 1);
                mbar_init(bar(&bars.p_half[p][i]), 8);    // one arrival per softmax warp of the slot, both CTAs
                mbar_init(bar(&bars.p_full[p][i]), 8);
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
    if (warp == 9) {  // each CTA of the pair allocates its tensor memory with the pair-wide form
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&bars.tmem_base)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();      // both CTAs' barriers are initialised before anything arrives at them from the other side
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;
    bool dead = false;

    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" :: "n"(kRegsControl));
    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            // the leader's copies of the "full" barriers, as seen from this CTA
            const uint32_t q_full0 = map_to_cta(bar(&bars.q_full[0]), 0), k_full0 = map_to_cta(bar(&bars.k_full[0]), 0),
                           v_full0 = map_to_cta(bar(&bars.v_full[0]), 0);
            int kt = 0, k_issued = 0, v_issued = 0;
            uint32_t q_loads[2] = {0, 0};
            PairWork w;
            Rec rec;
            fetch(fetch_code(0), rec);
            int code = fetch_code(1);
            for (int k = 0; k < n_rounds && !dead; ++k) {
                decode(rec, w);
                fetch(code, rec);
                code = fetch_code(k + 2);
                if (!w.valid) continue;
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    if (p >= w.n_pt) break;
                    tc_wait(bar(&bars.q_empty[p]), (q_loads[p] & 1u) ^ 1u, dead, ix.status);
                    if (dead) break;
                    ++q_loads[p];
                    if (rank == 0) mbar_expect_tx(bar(&bars.q_full[p]), 2 * kTileBytes);
#pragma unroll
                    for (int c = 0; c < NB; ++c)
                        tma_load_2d_pair(s_q + p * kTileBytes + c * kBlockBytes, &tm_q, w.h * D + 64 * c,
                                         w.tok0 + w.q0 + (2 * p + (int)rank) * kTileM, q_full0 + 8 * p);
                }
                for (int j = 0; j < w.n_total && !dead; ++j, ++kt) {
                    const int s = kt % KS;
                    const uint32_t par = (uint32_t)(kt / KS) & 1u;
                    const int row = w.tok0 + j * kTileN;
                    tc_wait(bar(&bars.k_empty[s]), par ^ 1u, dead, ix.status);
                    if (dead) break;
                    if (rank == 0) mbar_expect_tx(bar(&bars.k_full[s]), 2 * kHalfBytes);
#pragma unroll
                    for (int c = 0; c < NB; ++c)   // keys 64r .. 64r+63 of the tile, all head dims
                        tma_load_2d_pair(s_k + s * kHalfBytes + c * kKHalfBlock, &tm_khalf, w.g * D + 64 * c,
                                         row + 64 * (int)rank, k_full0 + 8 * s);
                    ++k_issued;
                    tc_wait(bar(&bars.v_empty[s]), par ^ 1u, dead, ix.status);
                    if (dead) break;
                    if (rank == 0) mbar_expect_tx(bar(&bars.v_full[s]), 2 * kHalfBytes);
                    // all 128 keys of the tile, head dims 64r .. 64r+63
                    tma_load_2d_pair(s_v + s * kHalfBytes, &tm_v, w.g * D + 64 * (int)rank, row, v_full0 + 8 * s);
                    ++v_issued;
                }
            }
            // After a wait gave up: the leader, whose barriers count both CTAs' bytes, gives the copies issued last
            // one more bounded look; its peer cannot leave before the leader reaches the cluster barrier at the end.
            if (dead && rank == 0) {
#pragma unroll
                for (int p = 0; p < 2; ++p)
                    if (q_loads[p] > 0) mbar_drain(bar(&bars.q_full[p]), (q_loads[p] - 1u) & 1u, kDrainLimit);
                for (int t = max(0, k_issued - KS); t < k_issued; ++t)
                    mbar_drain(bar(&bars.k_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
                for (int t = max(0, v_issued - KS); t < v_issued; ++t)
                    mbar_drain(bar(&bars.v_full[t % KS]), (uint32_t)(t / KS) & 1u, kDrainLimit);
            }
        }
        __syncwarp();
    } else if (warp == 9 && rank == 0) {
        // ------------------------------------------------------------ MMA issuer of the pair (leader CTA only)
        uint32_t leader = (lane == 0);
        constexpr uint32_t idesc_qk = instr_desc(256, kTileN, false);
        constexpr uint32_t idesc_pv = instr_desc(256, D, true);
        const uint64_t dqk = smem_desc(0, 16, 1024), dvv = smem_desc(0, kBlockBytes, 1024);
        const uint32_t qk_hi = (uint32_t)(dqk >> 32), pv_hi = (uint32_t)(dvv >> 32);
        const uint32_t q_lo = (uint32_t)dqk | (s_q >> 4), k_lo = (uint32_t)dqk | (s_k >> 4), v_lo = (uint32_t)dvv | (s_v >> 4);
        uint32_t n_qk[2] = {0, 0}, n_pv[2] = {0, 0}, q_uses[2] = {0, 0};
        int kt0 = 0;
        auto qk = [&](int p, int kt) {   // S[slot p] = Q_p K[tile kt]^T for both CTAs' sub-tiles
            const uint32_t a = q_lo + p * (kTileBytes >> 4), bq = k_lo + (kt % KS) * (kHalfBytes >> 4), d_tmem = tmem + p * 128;
#pragma unroll
            for (int k = 0; k < D / 16; ++k)
                pair_mma_ss(d_tmem, a + (k >> 2) * (kBlockBytes >> 4) + (k & 3) * 2, bq + (k >> 2) * (kKHalfBlock >> 4) + (k & 3) * 2,
                            qk_hi, idesc_qk, k > 0, leader);
            pair_commit(bar(&bars.s_full[p][n_qk[p] & 3u]), leader);
            ++n_qk[p];
        };
        auto pv = [&](int p, int kt, uint32_t acc0) {   // O[slot p] += P[slot p] V[tile kt]
            const uint32_t bv = v_lo + (kt % KS) * (kHalfBytes >> 4), d_tmem = tmem + kColO + p * D, a_tmem = tmem + p * 128;
            pair_wait(bar(&bars.p_half[p][n_pv[p] & 3u]), (n_pv[p] >> 2) & 1u, dead, ix.status);
            if (dead) leader = 0u;
            tc_fence_after();
#pragma unroll
            for (int k = 0; k < kTileN / 32; ++k)
                pair_mma_ts(d_tmem, a_tmem + k * 8, bv + k * (2048 >> 4), pv_hi, idesc_pv, k > 0 ? 1u : acc0, leader);
            pair_wait(bar(&bars.p_full[p][n_pv[p] & 3u]), (n_pv[p] >> 2) & 1u, dead, ix.status);
            if (dead) leader = 0u;
            ++n_pv[p];
            tc_fence_after();
#pragma unroll
            for (int k = kTileN / 32; k < kTileN / 16; ++k)
                pair_mma_ts(d_tmem, a_tmem + k * 8, bv + k * (2048 >> 4), pv_hi, idesc_pv, 1u, leader);
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
        PairWork w;
        Rec rec;
        fetch(fetch_code(0), rec);
        int code = fetch_code(1);
        for (int r = 0; r < n_rounds; ++r) {
            decode(rec, w);
            fetch(code, rec);
            code = fetch_code(r + 2);
            if (!w.valid) continue;
            const int last = w.n_pt - 1;     // the slot that reads every tile last
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                if (p >= w.n_pt) break;
                tc_wait(bar(&bars.q_full[p]), q_uses[p] & 1u, dead, ix.status);
                if (dead) leader = 0u;
                ++q_uses[p];
            }
            wait_k(kt0);
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                if (p >= w.n_pt) break;
                qk(p, kt0);
                if (w.T(p) == 1) pair_commit(bar(&bars.q_empty[p]), leader);
            }
            pair_commit(bar(&bars.k_empty[kt0 % KS]), leader);
            for (int j = 0; j < w.n_total; ++j) {
                const int kt = kt0 + j;
                wait_v(kt);
#pragma unroll
                for (int p = 0; p < 2; ++p) {
                    if (p >= w.n_pt || j >= w.T(p)) continue;
                    pv(p, kt, j > 0);
                    if (p == last) pair_commit(bar(&bars.v_empty[kt % KS]), leader);
                    if (j == w.T(p) - 1) pair_commit(bar(&bars.pv_done[p]), leader);
                    if (j + 1 < w.T(p)) {     // the slot's next scores go into the buffer its PV has just read
                        wait_k(kt + 1);
                        qk(p, kt + 1);
                        if (p == last) pair_commit(bar(&bars.k_empty[(kt + 1) % KS]), leader);
                        if (j + 1 == w.T(p) - 1) pair_commit(bar(&bars.q_empty[p]), leader);
                    }
                }
            }
            kt0 += w.n_total;
        }
        if (__shfl_sync(0xffffffffu, (int)dead, 0) != 0) {
            pair_commit_local(bar(&bars.drain), (uint32_t)(lane == 0));
            if (lane == 0) mbar_drain(bar(&bars.drain), 0u, kDrainLimit);
            __syncwarp();
        }
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" :: "n"(kRegsSoftmax));
    {
        // ------------------------------------------------------------ softmax + epilogue (one warpgroup per slot)
        const int p = warp >> 2;
        const int r = threadIdx.x & 127;
        const uint32_t lane_addr = ((uint32_t)((warp & 3) * 32) << 16);
        const uint32_t t_o = tmem + lane_addr + kColO + p * D;
        const uint32_t t_s = tmem + lane_addr + p * 128;
        // the leader's "weights ready" barriers: local for the leader, mapped for its peer
        const uint32_t p_half0 = rank == 0 ? bar(&bars.p_half[p][0]) : map_to_cta(bar(&bars.p_half[p][0]), 0);
        const uint32_t p_full0 = rank == 0 ? bar(&bars.p_full[p][0]) : map_to_cta(bar(&bars.p_full[p][0]), 0);
        uint32_t n_steps = 0, n_units = 0;
        int kt0 = 0;
        PairWork w;
        Rec rec;
        fetch(fetch_code(0), rec);
        int code = fetch_code(1);
        for (int rd = 0; rd < n_rounds; ++rd) {
        decode(rec, w);
        fetch(code, rec);
        code = fetch_code(rd + 2);
        if (!w.valid) continue;
        if (p < w.n_pt) {
        const int sub = 2 * p + (int)rank;          // this CTA's sub-tile of the slot
        const int diag_j = w.t0 + sub;              // the tile that holds its diagonal; later tiles are all in its future
        const int n_kv = w.T(p);
        float m_used = -INFINITY, l_run = 0.f;
        for (int j = 0; j < n_kv; ++j, ++n_steps) {
            tc_wait(bar(&bars.s_full[p][n_steps & 3u]), (n_steps >> 2) & 1u, dead, ix.status);
            tc_fence_after();
            const bool visible = j <= diag_j;
            uint32_t sv[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc_ld32_nowait(t_s + c * 32, sv[c]);
            tc_wait_ld();
            if (j == diag_j) {
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c * 32 + i > r) sv[c][i] = 0xff800000u;
            }
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
            mx *= scale_log2;
            float alpha = 1.f;
            if (visible && mx > m_used + 8.f) {       // lazy reference max, as in the one-CTA kernel
                alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - mx);
                m_used = mx;
            }
            if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                const int kt = kt0 + j - 1;   // O must hold every earlier tile: V tile j-1 is released behind the last PV that reads it
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
                    // a tile past the diagonal (the leader's sub-tile in its slot's last step) contributes nothing
                    const uint32_t w2 = visible ? pack_bf16(exp2f(x0), exp2f(x1)) : 0u;
                    pk[i >> 1] = w2;
                    add_bf16x2(sum[(i >> 1) & 7], w2);
                }
                tc_st16(t_s + c * 16, pk);
                if (c == 1) {
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();     // one arrival per warp: the peer's cross the pair as 4 messages instead of 128
                    if (lane == 0) {
                        if (rank == 0) mbar_arrive(p_half0 + 8 * (n_steps & 3u)); else mbar_arrive_cluster(p_half0 + 8 * (n_steps & 3u));
                    }
                }
            }
            l_run += ((sum[0] + sum[1]) + (sum[2] + sum[3])) + ((sum[4] + sum[5]) + (sum[6] + sum[7]));
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(p_full0 + 8 * (n_steps & 3u)); else mbar_arrive_cluster(p_full0 + 8 * (n_steps & 3u));
            }
        }
        // ---- epilogue: O / l -> bf16 -> global
        tc_wait(bar(&bars.pv_done[p]), n_units & 1u, dead, ix.status);
        ++n_units;
        tc_fence_after();
        const float inv = 1.f / l_run;
        const bool row_ok = !dead && r < w.L - (w.q0 + sub * kTileM);
        __nv_bfloat16* dst = o + ((int64_t)(w.tok0 + w.q0 + sub * kTileM + r) * Hq + w.h) * D;
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

    // Neither CTA may leave, or free its tensor memory, while the other may still read its shared memory, write its
    // barriers or run MMAs over its tensor memory.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(512) : "memory");
    }
}

// 2-D view [rows = tokens][cols = heads*D] with a box of 64 cols x `box_rows` rows, 128-byte swizzle.
bool make_map_rows(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kPairSmem = 2 * 2 * (int)kBlockBytes + 2 * kPairStages * 16 * 1024 + 1024;

}  // namespace

// Pairs of CTAs of the prefill kernel that the current device can hold at the same time (0: none, or no device).
int cpa_prefill_pair_capacity() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 0; }
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n != 0) return n > 0 ? n : 0;
    int sms = 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kPairSmem;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_pair_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem) != cudaSuccess) {
        (void)cudaGetLastError();
        cached[dev].store(-1, std::memory_order_relaxed);
        return 0;
    }
    cfg.gridDim = dim3(2 * (sms / 2));
    if (cudaOccupancyMaxActiveClusters(&clusters, prefill_pair_kernel<128>, &cfg) != cudaSuccess || clusters < 1) {
        (void)cudaGetLastError();
        cached[dev].store(-1, std::memory_order_relaxed);
        return 0;
    }
    cached[dev].store(clusters, std::memory_order_relaxed);
    return clusters;
}

int cpa_prefill_pairs(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, void* stream) {
    const cpa_config& c = plan->cfg;
    constexpr int D = 128;
    if (c.head_dim != D || plan->q_tile != kPairRows) return CPA_EUNSUPPORTED;
    cudaFuncAttributes fattr;
    if (cudaFuncGetAttributes(&fattr, prefill_pair_kernel<D>) != cudaSuccess ||
        cudaFuncSetAttribute(prefill_pair_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmem) != cudaSuccess) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    // the in-kernel register split may only hand out what the launch allocates
    if (fattr.numRegs * kThreads < 2 * 128 * kRegsSoftmax + 128 * kRegsControl) return CPA_EUNSUPPORTED;
    CUtensorMap tm_q, tm_khalf, tm_v;
    if (!make_map_rows(&tm_q, q, plan->total_tokens, (int64_t)c.num_q_heads * D, 128) ||
        !make_map_rows(&tm_khalf, k, plan->total_tokens, (int64_t)c.num_kv_heads * D, 64) ||
        !make_map_rows(&tm_v, v, plan->total_tokens, (int64_t)c.num_kv_heads * D, 128))
        return CPA_ECUDA;
    const int pairs = plan->prefill_ctas;      // schedule columns: one per pair
    if (pairs < 1) return CPA_OK;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kPairSmem;
    cfg.stream = (cudaStream_t)stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_pair_kernel<D>, tm_q, tm_khalf, tm_v, (__nv_bfloat16*)o, plan->dev(),
                                       (int)c.num_q_heads, (int)c.num_kv_heads, c.scale * 1.4426950408889634f,
                                       (int)plan->prefill_rounds, pairs);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

// Varlen causal prefill attention with grouped-query heads on the 5th-generation tensor
// cores: TMA-staged tiles, tcgen05.mma with accumulators in tensor memory (TMEM), online
// softmax in fp32 registers.
//
// One CTA = one (block, q_tile of 128 rows, query head) item; 6 warps with fixed roles:
//   warps 0-3  softmax + epilogue: thread r owns query row r (TMEM lane r), so row max and
//              row sum need no shuffles
//   warp 4     TMA producer (one elected lane): Q once, then K and V tiles of 128 keys
//              through two-stage rings
//   warp 5     MMA issuer (one elected lane) and owner of the TMEM allocation
// TMEM columns: S0 [0,128), S1 [128,256) (fp32 scores, double buffered), O [256,256+D).
// Per KV tile j:   S[j&1] = Q K_j^T          (SS MMA, both operands K-major in smem)
//                  P_j    = exp2(scale*S - m) (registers -> bf16 -> swizzled smem)
//                  O     += P_j V_j           (A = P K-major, B = V MN-major)
// The issuer runs QK(j+1) ahead of PV(j), so the tensor core works on the next scores while
// the softmax warps work on the current ones.  O stays in TMEM across tiles; it is rescaled
// only when a row's running max grows by more than 2^8 (the stale max is used meanwhile,
// which is exact after the final division by the row sum).
//
// Shared-memory tiles use the 128-byte swizzle that both TMA and the MMA descriptors
// understand: a tile is a set of column blocks of 64 bf16 (128 B) x rows, rows 128 B apart,
// 16-byte chunk c of row r stored at chunk c ^ (r & 7); every tile base is 1024-byte aligned.
//
// Every mbarrier wait is bounded: when one gives up the CTA records it in the status word,
// stops waiting, still frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "cpa_internal.h"

namespace {

constexpr int kTileM = 128;        // query rows per CTA
constexpr int kTileN = 128;        // keys per KV tile
constexpr int kThreads = 192;
constexpr uint32_t kSpinLimit = 1u << 20;
constexpr uint32_t kBlockBytes = 128 * 128;   // one column block: 128 rows x 128 B

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" :: "r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait.  Returns false (and records it) when the limit is hit; `dead` makes all later waits no-ops.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, bool& dead, int32_t* status) {
    if (dead) return;
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if (++spins > kSpinLimit) {
            dead = true;
            atomicCAS(status, 0, 1);
            return;
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
        :: "r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" :: "r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]; `accumulate` = 0 overwrites D.
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const float (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
        "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
        :: "r"(taddr),
           "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
           "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
           "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
           "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
           "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
           "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
           "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
           "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

// Shared-memory matrix descriptor, 128-byte swizzle, descriptor version 1 (sm_100).
//   K-major operand  : rows 128 B apart, 8-row groups `sbo` bytes apart (1024); lbo unused (1 unit)
//   MN-major operand : 64-element column blocks `lbo` bytes apart, 8-row (k) groups `sbo` bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}
// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, M x N, optional MN-major B.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

struct __align__(8) TcBarriers {
    uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], s_empty[2], p_full, pv_done;
    uint32_t tmem_base;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                  const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, cpa_dev_index ix, int Hq,
                  int Hkv, float scale_log2) {
    constexpr int NB = D / 64;                         // 64-wide column blocks of a Q/K/V tile
    constexpr uint32_t kTileBytes = NB * kBlockBytes;  // one Q, K or V tile
    constexpr uint32_t kTmemCols = 512;
    constexpr uint32_t kColS0 = 0, kColO = 256;
    extern __shared__ unsigned char dsm_raw[];
    __shared__ TcBarriers bars;

    const uint32_t base = (smem_u32(dsm_raw) + 1023u) & ~1023u;
    const uint32_t s_q = base;
    const uint32_t s_k = s_q + kTileBytes;           // two stages
    const uint32_t s_v = s_k + 2 * kTileBytes;       // two stages
    const uint32_t s_p = s_v + 2 * kTileBytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = ix.prefill_items[2 * blockIdx.x], tile = ix.prefill_items[2 * blockIdx.x + 1];
    const int h = blockIdx.y, g = h / (Hq / Hkv);
    const int tok0 = ix.cu_seqlens[b];
    const int L = ix.cu_seqlens[b + 1] - tok0;
    const int q0 = tile * kTileM;
    const int n_tiles = tile + 1;  // KV tiles 0..tile; only the last one touches the diagonal

    const uint32_t b_q_full = smem_u32(&bars.q_full), b_p_full = smem_u32(&bars.p_full), b_pv_done = smem_u32(&bars.pv_done);
    const uint32_t b_k_full = smem_u32(&bars.k_full[0]), b_k_empty = smem_u32(&bars.k_empty[0]);
    const uint32_t b_v_full = smem_u32(&bars.v_full[0]), b_v_empty = smem_u32(&bars.v_empty[0]);
    const uint32_t b_s_full = smem_u32(&bars.s_full[0]), b_s_empty = smem_u32(&bars.s_empty[0]);

    if (threadIdx.x == 0) {
        mbar_init(b_q_full, 1);
        mbar_init(b_p_full, 128);
        mbar_init(b_pv_done, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(b_k_full + 8 * s, 1);
            mbar_init(b_k_empty + 8 * s, 1);
            mbar_init(b_v_full + 8 * s, 1);
            mbar_init(b_v_empty + 8 * s, 1);
            mbar_init(b_s_full + 8 * s, 1);
            mbar_init(b_s_empty + 8 * s, 128);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 5) {  // TMEM allocation is warp-wide
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&bars.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars.tmem_base;
    bool dead = false;

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            mbar_expect_tx(b_q_full, kTileBytes);
#pragma unroll
            for (int c = 0; c < NB; ++c) tma_load_2d(s_q + c * kBlockBytes, &tm_q, h * D + 64 * c, tok0 + q0, b_q_full);
            for (int j = 0; j < n_tiles; ++j) {
                const int s = j & 1;
                const uint32_t par = (uint32_t)(j >> 1) & 1u;
                const int row = tok0 + j * kTileN;
                mbar_wait(b_k_empty + 8 * s, par ^ 1u, dead, ix.status);
                mbar_expect_tx(b_k_full + 8 * s, kTileBytes);
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    tma_load_2d(s_k + s * kTileBytes + c * kBlockBytes, &tm_k, g * D + 64 * c, row, b_k_full + 8 * s);
                mbar_wait(b_v_empty + 8 * s, par ^ 1u, dead, ix.status);
                mbar_expect_tx(b_v_full + 8 * s, kTileBytes);
#pragma unroll
                for (int c = 0; c < NB; ++c)
                    tma_load_2d(s_v + s * kTileBytes + c * kBlockBytes, &tm_v, g * D + 64 * c, row, b_v_full + 8 * s);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kTileM, kTileN, false);
            constexpr uint32_t idesc_pv = instr_desc(kTileM, D, true);
            auto issue_qk = [&](int j) {
                const int s = j & 1;
                const uint32_t par = (uint32_t)(j >> 1) & 1u;
                mbar_wait(b_k_full + 8 * s, par, dead, ix.status);
                mbar_wait(b_s_empty + 8 * s, par ^ 1u, dead, ix.status);
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    // 16 head dims per instruction: 32 B inside the 128-B swizzled row, next block after 4 steps
                    const uint32_t off = (k >> 2) * kBlockBytes + (k & 3) * 32;
                    tc_mma_ss(tmem + kColS0 + s * 128, smem_desc(s_q + off, 16, 1024),
                              smem_desc(s_k + s * kTileBytes + off, 16, 1024), idesc_qk, k > 0);
                }
                tc_commit(b_k_empty + 8 * s);
                tc_commit(b_s_full + 8 * s);
            };
            auto issue_pv = [&](int j) {
                const int s = j & 1;
                mbar_wait(b_v_full + 8 * s, (uint32_t)(j >> 1) & 1u, dead, ix.status);
                mbar_wait(b_p_full, (uint32_t)j & 1u, dead, ix.status);
                tc_fence_after();
#pragma unroll
                for (int k = 0; k < kTileN / 16; ++k) {
                    // A = P: 16 keys per step (32 B inside the row, next column block after 4 steps)
                    // B = V: 16 keys per step = 16 rows of 128 B; column blocks kBlockBytes apart
                    const uint32_t a_off = (k >> 2) * kBlockBytes + (k & 3) * 32;
                    tc_mma_ss(tmem + kColO, smem_desc(s_p + a_off, 16, 1024),
                              smem_desc(s_v + s * kTileBytes + k * 2048, kBlockBytes, 1024), idesc_pv, (j > 0 || k > 0));
                }
                tc_commit(b_v_empty + 8 * s);
                tc_commit(b_pv_done);
            };
            mbar_wait(b_q_full, 0, dead, ix.status);
            for (int j = 0; j < n_tiles; ++j) {
                issue_qk(j);
                if (j > 0) issue_pv(j - 1);
            }
            issue_pv(n_tiles - 1);
        }
    } else {
        // ------------------------------------------------------------ softmax + epilogue (128 threads)
        const int r = threadIdx.x;                                   // query row inside the tile = TMEM lane
        const uint32_t lane_addr = ((uint32_t)(warp * 32) << 16);    // this warp's 32 TMEM lanes
        const uint32_t p_row = s_p + r * 128;
        float m_used = -INFINITY;   // row max the weights are currently scaled with (log2 units)
        float l_run = 0.f;
        for (int j = 0; j < n_tiles; ++j) {
            const int s = j & 1;
            mbar_wait(b_s_full + 8 * s, (uint32_t)(j >> 1) & 1u, dead, ix.status);
            tc_fence_after();
            const uint32_t t_s = tmem + lane_addr + kColS0 + s * 128;
            const bool diag = (j == n_tiles - 1);
            // pass 1: row max of this tile
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float v[32];
                tc_ld32(t_s + c * 32, v);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const bool masked = diag && (c * 32 + i > r);
                    mx = fmaxf(mx, masked ? -INFINITY : v[i]);
                }
            }
            mx *= scale_log2;       // scale > 0, so the max commutes with the scaling
            // lazy rescale: keep the old reference max unless the new one is more than 2^8 above it
            float alpha = 1.f;
            if (mx > m_used + 8.f) {
                alpha = (m_used == -INFINITY) ? 0.f : exp2f(m_used - mx);
                m_used = mx;
            }
            // P of the previous tile must have been consumed (and O settled) before P is overwritten
            if (j > 0) {
                mbar_wait(b_pv_done, (uint32_t)(j - 1) & 1u, dead, ix.status);
                tc_fence_after();
            }
            const bool rescale = __any_sync(0xffffffffu, alpha != 1.f) && j > 0;
            if (rescale) {
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    float v[32];
                    tc_ld32(tmem + lane_addr + kColO + c * 32, v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] *= alpha;
                    tc_st32(tmem + lane_addr + kColO + c * 32, v);
                }
                tc_wait_st();
            }
            l_run *= alpha;
            // pass 2: weights, rounded to bf16, written K-major into the swizzled P tile
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                float v[32];
                tc_ld32(t_s + c * 32, v);
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const bool m0 = diag && (c * 32 + i > r), m1 = diag && (c * 32 + i + 1 > r);
                    const float p0 = m0 ? 0.f : exp2f(fmaf(v[i], scale_log2, -m_used));
                    const float p1 = m1 ? 0.f : exp2f(fmaf(v[i + 1], scale_log2, -m_used));
                    const uint32_t w = pack_bf16(p0, p1);
                    pk[i >> 1] = w;
                    // row sum over the rounded weights: numerator and denominator stay consistent
                    sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int chunk = c * 4 + q4;            // 16-byte chunk (8 keys) of this row: 0..15
                    const uint32_t addr = p_row + (chunk >> 3) * kBlockBytes + (((chunk & 7) ^ (r & 7)) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n"
                                 :: "r"(addr), "r"(pk[4 * q4]), "r"(pk[4 * q4 + 1]), "r"(pk[4 * q4 + 2]), "r"(pk[4 * q4 + 3]) : "memory");
                }
            }
            l_run += sum;
            // S[s] may be overwritten by QK(j+2); P is ready for PV(j)
            tc_fence_before();
            mbar_arrive(b_s_empty + 8 * s);
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            mbar_arrive(b_p_full);
        }
        // ---- epilogue: O / l, rows past the end of the block are never stored
        mbar_wait(b_pv_done, (uint32_t)(n_tiles - 1) & 1u, dead, ix.status);
        tc_fence_after();
        const float inv = 1.f / l_run;
        const bool valid = (q0 + r < L) && !dead;
        __nv_bfloat16* dst = o + ((int64_t)(tok0 + q0 + r) * Hq + h) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
            float v[32];
            tc_ld32(tmem + lane_addr + kColO + c * 32, v);
            if (valid) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 w;
                    w.x = pack_bf16(v[i] * inv, v[i + 1] * inv);
                    w.y = pack_bf16(v[i + 2] * inv, v[i + 3] * inv);
                    w.z = pack_bf16(v[i + 4] * inv, v[i + 5] * inv);
                    w.w = pack_bf16(v[i + 6] * inv, v[i + 7] * inv);
                    *reinterpret_cast<uint4*>(dst + c * 32 + i) = w;
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

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

template <int D>
int launch_prefill_tc(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, cudaStream_t st) {
    const cpa_config& c = plan->cfg;
    constexpr int NB = D / 64;
    constexpr int smem = (5 * NB + 2) * (int)kBlockBytes + 1024;   // Q + 2K + 2V tiles, P tile, alignment slack
    static bool configured = false;  // per instantiation; one device per process assumed for this cache
    if (!configured) {
        if (cudaFuncSetAttribute(prefill_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        configured = true;
    }
    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, q, plan->total_tokens, (int64_t)c.num_q_heads * D) ||
        !make_map(&tm_k, k, plan->total_tokens, (int64_t)c.num_kv_heads * D) ||
        !make_map(&tm_v, v, plan->total_tokens, (int64_t)c.num_kv_heads * D))
        return CPA_ECUDA;
    dim3 grid(plan->n_prefill, c.num_q_heads);
    prefill_tc_kernel<D><<<grid, kThreads, smem, st>>>(tm_q, tm_k, tm_v, (__nv_bfloat16*)o, plan->dev(), c.num_q_heads,
                                                      c.num_kv_heads, c.scale * 1.4426950408889634f);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

}  // namespace

int cpa_prefill_tc(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_prefill_tc<128>(plan, q, k, v, o, st)
                                     : launch_prefill_tc<64>(plan, q, k, v, o, st);
}

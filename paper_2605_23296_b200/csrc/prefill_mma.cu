// Varlen causal prefill attention with grouped-query heads, warp-level MMA version.
//
// One CTA = one (block, q_tile of 128 rows, query head) item; 8 warps, 16 query rows
// each.  K/V tiles of 64 keys are staged in shared memory with cp.async (two
// stages), fragments come from ldmatrix, scores and the running softmax stay in
// registers (fp32).  Only tiles at or below the diagonal are visited; keys are
// restricted to the query's own block by construction (tile ranges come from
// cu_seqlens), rows past the block's end are never stored.
#include <atomic>

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "cpa_internal.h"

namespace {

constexpr int kQTile = 128;
constexpr int kKVTile = 64;
constexpr int kPrefillThreads = 256;

__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}

// 16-byte async copy; src_bytes = 0 zero-fills the destination.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" :: "r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" :: "n"(N)); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

// Shared-memory tile [rows][D] bf16; 16-byte chunk c of row r is stored at chunk c ^ (r & 7).
template <int D>
__device__ __forceinline__ uint32_t tile_addr(uint32_t base, int row, int chunk) {
    return base + (uint32_t)(row * D * 2 + ((chunk ^ (row & 7)) << 4));
}

// Copy `rows` rows (row stride `stride_elems`) into a swizzled tile; rows >= valid_rows are zero-filled.
template <int D>
__device__ __forceinline__ void load_tile(uint32_t smem, const __nv_bfloat16* src, int64_t stride_elems,
                                          int rows, int valid_rows) {
    constexpr int CH = D / 8;
    for (int i = threadIdx.x; i < rows * CH; i += kPrefillThreads) {
        const int r = i / CH, c = i - r * CH;
        const bool ok = r < valid_rows;
        cp_async16(tile_addr<D>(smem, r, c), src + (ok ? (int64_t)r * stride_elems + c * 8 : 0), ok ? 16 : 0);
    }
}

template <int D>
__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                   const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, cpa_dev_index ix,
                   int Hq, int Hkv, int subs, float scale_log2) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    constexpr int KSTEPS = D / 16;   // k-steps of the QK^T contraction
    constexpr int NT_S = kKVTile / 8;  // 8-key n-tiles of S
    constexpr int NT_O = D / 8;        // 8-dim n-tiles of O
    const uint32_t s_q = (uint32_t)__cvta_generic_to_shared(smem_raw);
    const uint32_t s_k = s_q + kQTile * D * 2;
    const uint32_t s_v = s_k + 2 * kKVTile * D * 2;

    // a work item of subs*128 query rows is covered by `subs` CTAs of 128 rows each
    const int item = blockIdx.x / subs;
    const int tile = (ix.prefill_items[4 * item + 2] & 0xFFFF) * subs + (blockIdx.x - item * subs);
    const int h = blockIdx.y, g = h / (Hq / Hkv);
    const int tok0 = ix.prefill_items[4 * item];
    const int L = ix.prefill_items[4 * item + 1];
    const int q0 = tile * kQTile;
    if (q0 >= L) return;
    const int q_rows = min(kQTile, L - q0);
    const int kv_end = q0 + q_rows;  // keys visible to the tile's last row
    const int n_tiles = (kv_end + kKVTile - 1) / kKVTile;

    const __nv_bfloat16* qg = q + ((int64_t)(tok0 + q0) * Hq + h) * D;
    const __nv_bfloat16* kg = k + ((int64_t)tok0 * Hkv + g) * D;
    const __nv_bfloat16* vg = v + ((int64_t)tok0 * Hkv + g) * D;

    load_tile<D>(s_q, qg, (int64_t)Hq * D, kQTile, q_rows);
    load_tile<D>(s_k, kg, (int64_t)Hkv * D, kKVTile, min(kKVTile, L));
    load_tile<D>(s_v, vg, (int64_t)Hkv * D, kKVTile, min(kKVTile, L));
    cp_async_commit();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gid = lane >> 2, tig = lane & 3;
    const int row_lo = q0 + warp * 16 + gid;  // block-local query index of accumulator rows c0,c1
    const int row_hi = row_lo + 8;            // ... and of c2,c3

    uint32_t qf[KSTEPS][4];
    float oacc[NT_O][4];
#pragma unroll
    for (int n = 0; n < NT_O; ++n) oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f;
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    for (int j = 0; j < n_tiles; ++j) {
        const int stage = j & 1;
        if (j + 1 < n_tiles) {  // prefetch the next K/V tile into the other stage
            const int kv1 = (j + 1) * kKVTile;
            load_tile<D>(s_k + (stage ^ 1) * kKVTile * D * 2, kg + (int64_t)kv1 * Hkv * D, (int64_t)Hkv * D,
                         kKVTile, min(kKVTile, L - kv1));
            load_tile<D>(s_v + (stage ^ 1) * kKVTile * D * 2, vg + (int64_t)kv1 * Hkv * D, (int64_t)Hkv * D,
                         kKVTile, min(kKVTile, L - kv1));
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (j == 0) {
#pragma unroll
            for (int kk = 0; kk < KSTEPS; ++kk)
                ldsm_x4(qf[kk], tile_addr<D>(s_q, warp * 16 + (lane & 15), 2 * kk + (lane >> 4)));
        }
        const int kv0 = j * kKVTile;
        if (kv0 <= q0 + warp * 16 + 15) {  // some key of this tile is visible to this warp's rows
            const uint32_t sk = s_k + stage * kKVTile * D * 2;
            const uint32_t sv = s_v + stage * kKVTile * D * 2;
            float sc[NT_S][4];
#pragma unroll
            for (int n = 0; n < NT_S; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
                for (int np = 0; np < NT_S / 2; ++np) {
                    uint32_t kb[4];
                    ldsm_x4(kb, tile_addr<D>(sk, np * 16 + ((lane >> 4) << 3) + (lane & 7), 2 * kk + ((lane >> 3) & 1)));
                    mma_16816(sc[2 * np], qf[kk], kb[0], kb[1]);
                    mma_16816(sc[2 * np + 1], qf[kk], kb[2], kb[3]);
                }
            }
            // causal mask on tiles that touch the diagonal
            if (kv0 + kKVTile - 1 > q0 + warp * 16) {
#pragma unroll
                for (int n = 0; n < NT_S; ++n) {
                    const int key = kv0 + n * 8 + tig * 2;
                    if (key > row_lo) sc[n][0] = -INFINITY;
                    if (key + 1 > row_lo) sc[n][1] = -INFINITY;
                    if (key > row_hi) sc[n][2] = -INFINITY;
                    if (key + 1 > row_hi) sc[n][3] = -INFINITY;
                }
            }
            float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
            for (int n = 0; n < NT_S; ++n) {
                mx_lo = fmaxf(mx_lo, fmaxf(sc[n][0], sc[n][1]));
                mx_hi = fmaxf(mx_hi, fmaxf(sc[n][2], sc[n][3]));
            }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
            const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
            // a row that has seen no key yet keeps max = -inf; use 0 as a stand-in so nothing turns NaN
            const float mb_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo * scale_log2;
            const float mb_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi * scale_log2;
            const float al_lo = (m_lo == -INFINITY) ? 0.f : exp2f(m_lo * scale_log2 - mb_lo);
            const float al_hi = (m_hi == -INFINITY) ? 0.f : exp2f(m_hi * scale_log2 - mb_hi);
            m_lo = mn_lo; m_hi = mn_hi;
#pragma unroll
            for (int n = 0; n < NT_S; ++n) {
                sc[n][0] = exp2f(fmaf(sc[n][0], scale_log2, -mb_lo));
                sc[n][1] = exp2f(fmaf(sc[n][1], scale_log2, -mb_lo));
                sc[n][2] = exp2f(fmaf(sc[n][2], scale_log2, -mb_hi));
                sc[n][3] = exp2f(fmaf(sc[n][3], scale_log2, -mb_hi));
            }
            // Weights go to the tensor core as bf16; the row sum is taken over the SAME rounded
            // values so that numerator and denominator of the softmax stay consistent.
            uint32_t pk[NT_S][2];
            float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
            for (int n = 0; n < NT_S; ++n) {
                pk[n][0] = pack2(sc[n][0], sc[n][1]);
                pk[n][1] = pack2(sc[n][2], sc[n][3]);
                sum_lo += __uint_as_float(pk[n][0] << 16) + __uint_as_float(pk[n][0] & 0xffff0000u);
                sum_hi += __uint_as_float(pk[n][1] << 16) + __uint_as_float(pk[n][1] & 0xffff0000u);
            }
            l_lo = l_lo * al_lo + sum_lo;
            l_hi = l_hi * al_hi + sum_hi;
#pragma unroll
            for (int n = 0; n < NT_O; ++n) {
                oacc[n][0] *= al_lo; oacc[n][1] *= al_lo; oacc[n][2] *= al_hi; oacc[n][3] *= al_hi;
            }
            // O += P V
#pragma unroll
            for (int ks = 0; ks < kKVTile / 16; ++ks) {
                uint32_t pa[4];
                pa[0] = pk[2 * ks][0];
                pa[1] = pk[2 * ks][1];
                pa[2] = pk[2 * ks + 1][0];
                pa[3] = pk[2 * ks + 1][1];
#pragma unroll
                for (int np = 0; np < NT_O / 2; ++np) {
                    uint32_t vb[4];
                    ldsm_x4_trans(vb, tile_addr<D>(sv, ks * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), 2 * np + (lane >> 4)));
                    mma_16816(oacc[2 * np], pa, vb[0], vb[1]);
                    mma_16816(oacc[2 * np + 1], pa, vb[2], vb[3]);
                }
            }
        }
        __syncthreads();  // everyone is done with this stage before it is refilled
    }

    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
    // rows past the end of the block belong to the next block (or to nobody): never store them
    if (row_lo < L) {
        __nv_bfloat16* dst = o + ((int64_t)(tok0 + row_lo) * Hq + h) * D + tig * 2;
#pragma unroll
        for (int n = 0; n < NT_O; ++n)
            *reinterpret_cast<__nv_bfloat162*>(dst + n * 8) = __floats2bfloat162_rn(oacc[n][0] * inv_lo, oacc[n][1] * inv_lo);
    }
    if (row_hi < L) {
        __nv_bfloat16* dst = o + ((int64_t)(tok0 + row_hi) * Hq + h) * D + tig * 2;
#pragma unroll
        for (int n = 0; n < NT_O; ++n)
            *reinterpret_cast<__nv_bfloat162*>(dst + n * 8) = __floats2bfloat162_rn(oacc[n][2] * inv_hi, oacc[n][3] * inv_hi);
    }
}

template <int D>
int launch_prefill_mma(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, cudaStream_t st) {
    const cpa_config& c = plan->cfg;
    constexpr int smem = (kQTile + 4 * kKVTile) * D * 2;
    static std::atomic<bool> configured_dev[64];  // the attribute is per device: remember which devices have it
    int dev_id = 0;
    if (cudaGetDevice(&dev_id) != cudaSuccess || dev_id < 0 || dev_id >= 64) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    std::atomic<bool>& configured = configured_dev[dev_id];
    if (!configured.load(std::memory_order_relaxed)) {
        if (cudaFuncSetAttribute(prefill_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        configured.store(true, std::memory_order_relaxed);
    }
    const int subs = plan->q_tile / kQTile;
    dim3 grid(plan->n_prefill * subs, c.num_q_heads);
    prefill_mma_kernel<D><<<grid, kPrefillThreads, smem, st>>>(
        (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)o, plan->dev(),
        c.num_q_heads, c.num_kv_heads, subs, c.scale * 1.4426950408889634f);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

}  // namespace

int cpa_prefill_mma(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    return plan->cfg.head_dim == 128 ? launch_prefill_mma<128>(plan, q, k, v, o, st)
                                     : launch_prefill_mma<64>(plan, q, k, v, o, st);
}

int cpa_prefill_tc(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o, const void* k_pool,
                   const void* v_pool, void* stream);

namespace {
bool has_prefix(const cpa_plan* plan) {
    for (int32_t n : plan->prefix_lens)
        if (n > 0) return true;
    return false;
}
}  // namespace

extern "C" int cpa_prefill_variant(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o,
                                   void* stream, int variant) {
    if (!plan || !q || !k || !v || !o) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k) || !cpa_aligned16(v) || !cpa_aligned16(o)) return CPA_EINVAL;
    if (o == q || o == k || o == v) return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    if (has_prefix(plan)) return CPA_EINVAL;   // a cached prefix is read from the pools: cpa_prefill_prefix
    if (variant == CPA_PREFILL_TENSOR_CORE) return cpa_prefill_tc(plan, q, k, v, o, nullptr, nullptr, stream);
    if (variant == CPA_PREFILL_WARP_MMA) return cpa_prefill_mma(plan, q, k, v, o, stream);
    return CPA_EINVAL;
}

extern "C" int cpa_prefill(const cpa_plan* plan, const void* q, const void* k, const void* v, void* o,
                           void* d_workspace, void* stream) {
    (void)d_workspace;
    return cpa_prefill_variant(plan, q, k, v, o, stream, CPA_PREFILL_TENSOR_CORE);
}

extern "C" int cpa_prefill_prefix(const cpa_plan* plan, const void* q, const void* k, const void* v, const void* k_pool,
                                  const void* v_pool, void* o, void* stream) {
    if (!plan || !q || !k || !v || !o || !k_pool || !v_pool) return CPA_EINVAL;
    if (!cpa_aligned16(q) || !cpa_aligned16(k) || !cpa_aligned16(v) || !cpa_aligned16(o) || !cpa_aligned16(k_pool) ||
        !cpa_aligned16(v_pool))
        return CPA_EINVAL;
    if (o == q || o == k || o == v) return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    return cpa_prefill_tc(plan, q, k, v, o, k_pool, v_pool, stream);
}

// Paged KV append: scatter new K/V rows into the pages each block owns and advance
// the per-block cached length.  Pure data movement (bit-exact), bound by HBM.
#include <cuda_runtime.h>

#include "cpa_device.cuh"
#include "cpa_internal.h"

namespace {

// One 16-byte chunk of one (token, kv head) row.
__device__ __forceinline__ void copy_row_chunks(const uint4* __restrict__ k_src, const uint4* __restrict__ v_src,
                                                uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                                                int64_t page, int off, int Hkv, int chunks_per_head, int P) {
    const int chunks = Hkv * chunks_per_head;
    for (int c = threadIdx.x; c < chunks; c += blockDim.x) {
        const int g = c / chunks_per_head;
        const int j = c - g * chunks_per_head;
        const int64_t dst = ((page * Hkv + g) * P + off) * chunks_per_head + cpa_pool_piece(j, off);
        k_pool[dst] = k_src[c];
        v_pool[dst] = v_src[c];
    }
}

// Decode step: one new token per block.  CTA b is the only reader and writer of
// seq_lens[b], so the length can be advanced in the same launch.
__global__ void kv_append_step_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                      uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                                      cpa_dev_index ix, int Hkv, int chunks_per_head, int P) {
    // let a dependent launch (the step's decode) start its own set-up now; it waits for this
    // grid to finish before it reads what is written here
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int b = blockIdx.x;
    const int pos = ix.seq_lens[b];
    const int capacity = (ix.page_indptr[b + 1] - ix.page_indptr[b]) * P;
    __syncthreads();  // every thread has read the length before thread 0 advances it
    if (pos >= capacity) {  // host checks make this unreachable; never write outside the block's pages
        if (threadIdx.x == 0) atomicCAS(ix.status, 0, kStatusNoSpace);
        return;
    }
    const int64_t page = ix.page_indices[ix.page_indptr[b] + pos / P];
    const int64_t row = (int64_t)b * Hkv * chunks_per_head;
    copy_row_chunks(k_new + row, v_new + row, k_pool, v_pool, page, pos % P, Hkv, chunks_per_head, P);
    if (threadIdx.x == 0) ix.seq_lens[b] = pos + 1;
}

// Bulk append: `rows` new tokens, block-major; src_indptr[b] is the first row of block b.
__global__ void kv_append_bulk_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                      uint4* __restrict__ k_pool, uint4* __restrict__ v_pool,
                                      cpa_dev_index ix, const int32_t* __restrict__ src_indptr, int B,
                                      int64_t rows, int Hkv, int chunks_per_head, int P) {
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        // block that owns row r: last b with src_indptr[b] <= r
        int lo = 0, hi = B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((int64_t)src_indptr[mid] <= r) lo = mid; else hi = mid - 1;
        }
        const int b = lo;
        const int pos = ix.seq_lens[b] + (int)(r - src_indptr[b]);
        const int64_t page = ix.page_indices[ix.page_indptr[b] + pos / P];
        const int64_t row = r * Hkv * chunks_per_head;
        copy_row_chunks(k_new + row, v_new + row, k_pool, v_pool, page, pos % P, Hkv, chunks_per_head, P);
    }
}

// Chunk step of a chunked prefill: `rows` tokens, block-major; rows_indptr[b] is the first row of block b's
// chunk, whose tokens are positions first_pos .. of the block (its earlier chunks are cached already), read
// from rows cu_seqlens[b] + first_pos .. of the packed tensors.
__global__ void kv_append_chunk_kernel(const uint4* __restrict__ k, const uint4* __restrict__ v,
                                       uint4* __restrict__ k_pool, uint4* __restrict__ v_pool, cpa_dev_index ix,
                                       const int32_t* __restrict__ rows_indptr, int B, int rows, int first_pos,
                                       int Hkv, int chunks_per_head, int P) {
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        int lo = 0, hi = B - 1;   // block that owns row r: last b with rows_indptr[b] <= r
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (rows_indptr[mid] <= r) lo = mid; else hi = mid - 1;
        }
        const int b = lo;
        const int own = first_pos + (r - rows_indptr[b]);       // position among the block's own tokens
        const int pos = ix.prefix_lens[b] + own;                 // position in the sequence (behind a cached prefix)
        const int64_t page = ix.page_indices[ix.page_indptr[b] + pos / P];
        const int64_t row = ((int64_t)ix.cu_seqlens[b] + own) * Hkv * chunks_per_head;
        copy_row_chunks(k + row, v + row, k_pool, v_pool, page, pos % P, Hkv, chunks_per_head, P);
    }
}

// Pages on demand: a block whose flag says it has stopped gives its pages back to the reserve.  One CTA per
// block; pops happen in decode launches only, which are ordered against this one by the stream.
__global__ void release_pages_kernel(cpa_dev_index ix, const int32_t* __restrict__ d_active, int B) {
    __shared__ int base;
    const int b = blockIdx.x;
    if (b >= B || d_active[b] != 0) return;
    const int n = ix.pages_assigned[b];
    if (n == 0) return;
    if (threadIdx.x == 0) base = atomicAdd(ix.ring_ctrl + 1, n);
    __syncthreads();
    const int size = ix.ring_ctrl[2];
    const int32_t* row = ix.page_indices + ix.page_indptr[b];
    for (int i = threadIdx.x; i < n; i += blockDim.x) ix.ring[(base + i) % size] = row[i];
    __syncthreads();
    if (threadIdx.x == 0) ix.pages_assigned[b] = 0;
}

__global__ void seq_lens_advance_kernel(cpa_dev_index ix, const int32_t* __restrict__ src_indptr, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) ix.seq_lens[b] += src_indptr[b + 1] - src_indptr[b];
}

}  // namespace

extern "C" int cpa_kv_append(cpa_plan* plan, const void* k_new, const void* v_new, const int32_t* new_lens,
                             void* k_pool, void* v_pool, void* stream) {
    if (!plan || !k_new || !v_new || !k_pool || !v_pool) return CPA_EINVAL;
    if (!cpa_aligned16(k_new) || !cpa_aligned16(v_new) || !cpa_aligned16(k_pool) || !cpa_aligned16(v_pool))
        return CPA_EINVAL;
    if (!plan->d_base) return CPA_ESTATE;
    const int B = plan->B, P = plan->cfg.page_size, Hkv = plan->cfg.num_kv_heads;
    const int chunks_per_head = plan->cfg.head_dim / 8;
    cudaStream_t st = (cudaStream_t)stream;
    const cpa_dev_index ix = plan->dev();

    // capacity check on the host mirror before anything is enqueued
    bool is_prefill_bulk = new_lens != nullptr;
    int64_t rows = 0;
    for (int b = 0; b < B; ++b) {
        const int n = new_lens ? new_lens[b] : 1;
        if (n < 0) return CPA_EINVAL;
        if ((int64_t)plan->seq_lens[b] + n > (int64_t)plan->prefix_lens[b] + plan->block_lens[b] + plan->T) return CPA_ENOSPC;
        if (new_lens && (plan->seq_lens[b] != plan->prefix_lens[b] || n != plan->block_lens[b])) is_prefill_bulk = false;
        rows += n;
    }
    if (rows == 0) return CPA_OK;
    // a single-token append does not take pages from the reserve: plans with pages on demand append inside the
    // decode launch (cpa_decode_append, cpa_decode_append_dynamic)
    if (plan->dynamic && !new_lens) return CPA_EUNSUPPORTED;

    const int threads = std::min(256, std::max(32, (Hkv * chunks_per_head + 31) / 32 * 32));
    if (!new_lens) {
        kv_append_step_kernel<<<B, threads, 0, st>>>((const uint4*)k_new, (const uint4*)v_new, (uint4*)k_pool,
                                                     (uint4*)v_pool, ix, Hkv, chunks_per_head, P);
    } else {
        const int32_t* src_indptr = ix.cu_seqlens;
        if (!is_prefill_bulk) {
            plan->append_stage[0] = 0;
            for (int b = 0; b < B; ++b) plan->append_stage[b + 1] = plan->append_stage[b] + new_lens[b];
            if (cudaMemcpyAsync(ix.append_indptr, plan->append_stage.data(), sizeof(int32_t) * (B + 1),
                                cudaMemcpyHostToDevice, st) != cudaSuccess) {
                (void)cudaGetLastError();
                return CPA_ECUDA;
            }
            src_indptr = ix.append_indptr;
        }
        const int grid = (int)std::min<int64_t>(rows, (int64_t)plan->num_sms * 32);
        kv_append_bulk_kernel<<<grid, threads, 0, st>>>((const uint4*)k_new, (const uint4*)v_new, (uint4*)k_pool,
                                                        (uint4*)v_pool, ix, src_indptr, B, rows, Hkv,
                                                        chunks_per_head, P);
        seq_lens_advance_kernel<<<(B + 127) / 128, 128, 0, st>>>(ix, src_indptr, B);
    }
    if (cudaGetLastError() != cudaSuccess) return CPA_ECUDA;
    for (int b = 0; b < B; ++b) plan->seq_lens[b] += new_lens ? new_lens[b] : 1;
    return CPA_OK;
}

int cpa_append_chunk(cpa_plan* plan, int chunk, const void* k, const void* v, void* k_pool, void* v_pool, void* stream) {
    const int B = plan->B, P = plan->cfg.page_size, Hkv = plan->cfg.num_kv_heads;
    const int chunks_per_head = plan->cfg.head_dim / 8;
    cudaStream_t st = (cudaStream_t)stream;
    const cpa_chunk_step& cs = plan->chunk_steps[(size_t)chunk];
    const int threads = std::min(256, std::max(32, (Hkv * chunks_per_head + 31) / 32 * 32));
    const int grid = (int)std::min<int64_t>(cs.rows, (int64_t)plan->num_sms * 32);
    kv_append_chunk_kernel<<<grid, threads, 0, st>>>((const uint4*)k, (const uint4*)v, (uint4*)k_pool, (uint4*)v_pool,
                                                     plan->dev(), plan->d_base + cs.off_rows, B, cs.rows,
                                                     chunk * plan->chunk, Hkv, chunks_per_head, P);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

extern "C" int cpa_release_blocks(cpa_plan* plan, const int32_t* d_active, void* stream) {
    if (!plan || !d_active || (reinterpret_cast<uintptr_t>(d_active) & 3u)) return CPA_EINVAL;
    if (!plan->d_base || !plan->dynamic) return CPA_ESTATE;
    release_pages_kernel<<<plan->B, 128, 0, (cudaStream_t)stream>>>(plan->dev(), d_active, plan->B);
    return cudaGetLastError() == cudaSuccess ? CPA_OK : CPA_ECUDA;
}

// A whole compaction event from host memory (Section 4, "Dispatch": every block's prompt is prefilled and
// its summary decoded; the paper's engine receives its inputs from the host side of the serving stack).
// The inputs cross PCIe once and the outputs once; what this file adds to the device-side calls is the
// order of the copies: on a chunked plan the prompt goes up chunk by chunk on a copy stream, chunk c is
// prefilled (all blocks' rows [c*C, (c+1)*C) in one launch, attending over the blocks' pages for the earlier
// chunks) as soon as its rows have landed, and the output rows go home on a third stream behind the last
// input (the two directions slow each other down; the inputs are on the critical path, the outputs have the
// decode steps to hide behind).  The decode steps are the ordinary fused launches over all blocks.
#include <cuda_runtime.h>

#include <algorithm>
#include <vector>

#include "cpa_internal.h"

namespace {

__global__ void lens_after_prefill_kernel(cpa_dev_index ix, int B) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) ix.seq_lens[b] = ix.prefix_lens[b] + ix.cu_seqlens[b + 1] - ix.cu_seqlens[b];
}

inline int64_t align256(int64_t x) { return (x + 255) / 256 * 256; }

// The two copy streams and the events of an event from host memory, made on first use.
int ensure_host_streams(cpa_plan* plan, size_t n_events) {
    if (!plan->in_stream && cudaStreamCreateWithFlags(&plan->in_stream, cudaStreamNonBlocking) != cudaSuccess) goto fail;
    if (!plan->out_stream && cudaStreamCreateWithFlags(&plan->out_stream, cudaStreamNonBlocking) != cudaSuccess) goto fail;
    while (plan->host_events.size() < n_events) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) goto fail;
        plan->host_events.push_back(e);
    }
    return CPA_OK;
fail:
    (void)cudaGetLastError();
    return CPA_ECUDA;
}

}  // namespace

int64_t cpa_host_stage_bytes(const cpa_plan* plan) {
    const int64_t d = plan->cfg.head_dim, Hq = plan->cfg.num_q_heads, Hkv = plan->cfg.num_kv_heads;
    const int64_t q = align256(plan->total_tokens * Hq * d * 2), kv = align256(plan->total_tokens * Hkv * d * 2);
    const int64_t qd = align256((int64_t)plan->T * plan->B * Hq * d * 2), kvd = align256((int64_t)plan->T * plan->B * Hkv * d * 2);
    return 2 * q + 2 * kv + 2 * qd + 2 * kvd;
}

extern "C" int cpa_event_host(cpa_plan* plan, const void* h_q, const void* h_k, const void* h_v, void* h_o,
                              const void* h_q_dec, const void* h_k_dec, const void* h_v_dec, void* h_o_dec,
                              void* d_stage, void* k_pool, void* v_pool, void* d_workspace, void* stream) {
    if (!plan || !h_q || !h_k || !h_v || !h_o || !d_stage || !k_pool || !v_pool) return CPA_EINVAL;
    const int B = plan->B, T = plan->T;
    if (T > 0 && (!h_q_dec || !h_k_dec || !h_v_dec || !h_o_dec || !d_workspace)) return CPA_EINVAL;
    if ((reinterpret_cast<uintptr_t>(d_stage) & 255u) || !cpa_aligned16(k_pool) || !cpa_aligned16(v_pool) ||
        (d_workspace && !cpa_aligned16(d_workspace)))
        return CPA_EINVAL;
    if (!plan->d_base || plan->next_step != 0) return CPA_ESTATE;
    if (plan->dynamic) return CPA_EUNSUPPORTED;
    for (int b = 0; b < B; ++b)
        if (plan->seq_lens[b] != plan->prefix_lens[b]) return CPA_ESTATE;   // the event starts from empty caches

    const int64_t d = plan->cfg.head_dim, Hq = plan->cfg.num_q_heads, Hkv = plan->cfg.num_kv_heads;
    const int64_t q_row = Hq * d * 2, kv_row = Hkv * d * 2;     // bytes of one token's row
    const int64_t q_bytes = align256(plan->total_tokens * q_row), kv_bytes = align256(plan->total_tokens * kv_row);
    const int64_t qd_bytes = align256((int64_t)T * B * q_row), kvd_bytes = align256((int64_t)T * B * kv_row);
    char* base = static_cast<char*>(d_stage);
    char* d_q = base;
    char* d_k = d_q + q_bytes;
    char* d_v = d_k + kv_bytes;
    char* d_o = d_v + kv_bytes;
    char* d_qd = d_o + q_bytes;
    char* d_kd = d_qd + qd_bytes;
    char* d_vd = d_kd + kvd_bytes;
    char* d_od = d_vd + kvd_bytes;

    const int n_chunks = plan->chunk > 0 ? (int)plan->chunk_steps.size() : 1;
    // events: [0] fork, [1 + c] chunk c has landed, [1 + n + c] chunk c is computed, then decode inputs, outputs home
    const size_t n_events = 3 + 2 * (size_t)n_chunks;
    if (int rc = ensure_host_streams(plan, n_events)) return rc;
    cudaEvent_t* ev = plan->host_events.data();
    cudaEvent_t ev_fork = ev[0], ev_dec_in = ev[1 + 2 * n_chunks], ev_home = ev[2 + 2 * n_chunks];
    cudaStream_t main_st = (cudaStream_t)stream, in_st = plan->in_stream, out_st = plan->out_stream;

#define CPA_CK(call)                                   \
    do {                                               \
        if ((call) != cudaSuccess) {                   \
            (void)cudaGetLastError();                  \
            return CPA_ECUDA;                          \
        }                                              \
    } while (0)

    // the copies follow whatever the caller has enqueued on `stream` (an earlier event may still read the stage)
    CPA_CK(cudaEventRecord(ev_fork, main_st));
    CPA_CK(cudaStreamWaitEvent(in_st, ev_fork, 0));
    CPA_CK(cudaStreamWaitEvent(out_st, ev_fork, 0));

    // rows [first, first + n) of block b, for chunk c (the whole block on a plan without chunks)
    auto chunk_rows = [&](int c, int b, int64_t* first, int64_t* n) {
        if (plan->chunk == 0) { *first = plan->cu_seqlens[b]; *n = plan->block_lens[b]; return; }
        const int64_t lo = std::min<int64_t>((int64_t)c * plan->chunk, plan->block_lens[b]);
        const int64_t hi = std::min<int64_t>((int64_t)(c + 1) * plan->chunk, plan->block_lens[b]);
        *first = plan->cu_seqlens[b] + lo;
        *n = hi - lo;
    };

    // ---- inputs up, chunk by chunk, then the decode steps' inputs
    for (int c = 0; c < n_chunks; ++c) {
        for (int b = 0; b < B; ++b) {
            int64_t first, n;
            chunk_rows(c, b, &first, &n);
            if (n == 0) continue;
            CPA_CK(cudaMemcpyAsync(d_k + first * kv_row, (const char*)h_k + first * kv_row, (size_t)(n * kv_row), cudaMemcpyHostToDevice, in_st));
            CPA_CK(cudaMemcpyAsync(d_v + first * kv_row, (const char*)h_v + first * kv_row, (size_t)(n * kv_row), cudaMemcpyHostToDevice, in_st));
            CPA_CK(cudaMemcpyAsync(d_q + first * q_row, (const char*)h_q + first * q_row, (size_t)(n * q_row), cudaMemcpyHostToDevice, in_st));
        }
        CPA_CK(cudaEventRecord(ev[1 + c], in_st));
    }
    if (T > 0) {
        CPA_CK(cudaMemcpyAsync(d_qd, h_q_dec, (size_t)((int64_t)T * B * q_row), cudaMemcpyHostToDevice, in_st));
        CPA_CK(cudaMemcpyAsync(d_kd, h_k_dec, (size_t)((int64_t)T * B * kv_row), cudaMemcpyHostToDevice, in_st));
        CPA_CK(cudaMemcpyAsync(d_vd, h_v_dec, (size_t)((int64_t)T * B * kv_row), cudaMemcpyHostToDevice, in_st));
    }
    CPA_CK(cudaEventRecord(ev_dec_in, in_st));
    // outputs start home when the last input has landed: copies in both directions at once slow each other down,
    // and the inputs are on the critical path while the outputs have the decode steps to hide behind
    CPA_CK(cudaStreamWaitEvent(out_st, ev_dec_in, 0));

    // ---- prefill and append per chunk; the chunk's output rows are queued for the way home (behind the inputs)
    bool any_prefix = false;
    for (int b = 0; b < B; ++b) any_prefix |= plan->prefix_lens[b] > 0;
    for (int c = 0; c < n_chunks; ++c) {
        CPA_CK(cudaStreamWaitEvent(main_st, ev[1 + c], 0));
        int rc;
        if (plan->chunk > 0) {
            const cpa_chunk_step& cs = plan->chunk_steps[(size_t)c];
            rc = cpa_prefill_tc_list(plan, d_q, d_k, d_v, d_o, k_pool, v_pool, plan->d_base + cs.off_items,
                                     plan->d_base + cs.off_sched, cs.ctas, cs.rounds, main_st);
            if (rc == CPA_OK) rc = cpa_append_chunk(plan, c, d_k, d_v, k_pool, v_pool, main_st);
        } else {
            rc = any_prefix ? cpa_prefill_prefix(plan, d_q, d_k, d_v, k_pool, v_pool, d_o, main_st)
                            : cpa_prefill(plan, d_q, d_k, d_v, d_o, d_workspace, main_st);
            if (rc == CPA_OK) rc = cpa_kv_append(plan, d_k, d_v, plan->block_lens.data(), k_pool, v_pool, main_st);
        }
        if (rc != CPA_OK) return rc;
        CPA_CK(cudaEventRecord(ev[1 + n_chunks + c], main_st));
        CPA_CK(cudaStreamWaitEvent(out_st, ev[1 + n_chunks + c], 0));
        for (int b = 0; b < B; ++b) {
            int64_t first, n;
            chunk_rows(c, b, &first, &n);
            if (n == 0) continue;
            CPA_CK(cudaMemcpyAsync((char*)h_o + first * q_row, d_o + first * q_row, (size_t)(n * q_row), cudaMemcpyDeviceToHost, out_st));
        }
    }
    if (plan->chunk > 0) {
        // the chunk appends wrote by position; the decode steps read the lengths
        lens_after_prefill_kernel<<<(B + 127) / 128, 128, 0, main_st>>>(plan->dev(), B);
        CPA_CK(cudaGetLastError());
        for (int b = 0; b < B; ++b) plan->seq_lens[b] = plan->prefix_lens[b] + plan->block_lens[b];
        plan->next_step = plan->n_steps;    // the schedule of mixed steps is not available for this upload any more
    }

    // ---- decode steps over all blocks, each with its append; their outputs go home together
    CPA_CK(cudaStreamWaitEvent(main_st, ev_dec_in, 0));
    for (int t = 0; t < T; ++t) {
        const int64_t qo = (int64_t)t * B * q_row, ko = (int64_t)t * B * kv_row;
        if (int rc = cpa_decode_append(plan, d_qd + qo, d_kd + ko, d_vd + ko, k_pool, v_pool, d_od + qo, d_workspace, main_st))
            return rc;
    }
    if (T > 0)
        CPA_CK(cudaMemcpyAsync(h_o_dec, d_od, (size_t)((int64_t)T * B * q_row), cudaMemcpyDeviceToHost, main_st));
    CPA_CK(cudaEventRecord(ev_home, out_st));
    CPA_CK(cudaStreamWaitEvent(main_st, ev_home, 0));
#undef CPA_CK
    return CPA_OK;
}

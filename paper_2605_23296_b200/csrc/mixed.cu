// Steps of an event with chunked prefill (the serving engine of the paper's Section 4.2 runs with chunked
// prefill enabled; Section 6 finds that 16k blocks are prefill-bound): in one step the blocks that still have
// prompt left prefill their next chunk, and the blocks that are past their prompt decode one token.  The two
// halves touch different blocks, so they run side by side: the chunk's persistent prefill grid on most SMs
// (second stream), the decode wave on the SMs the plan keeps free for it (caller's stream), joined by an
// event before the call's work counts as done on the caller's stream.
#include <cuda_runtime.h>

#include "cpa_internal.h"

namespace {

// The second stream and the two events of a plan, made on first use.
int ensure_side_stream(cpa_plan* plan) {
    if (plan->side_stream) return CPA_OK;
    if (cudaStreamCreateWithFlags(&plan->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&plan->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&plan->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        (void)cudaGetLastError();
        return CPA_ECUDA;
    }
    return CPA_OK;
}

}  // namespace

extern "C" int cpa_step_mixed(cpa_plan* plan, int32_t step, const void* q, const void* k, const void* v, void* o,
                              const void* q_dec, const void* k_new, const void* v_new, void* o_dec, void* k_pool,
                              void* v_pool, void* d_workspace, void* stream) {
    if (!plan || !k_pool || !v_pool) return CPA_EINVAL;
    if (plan->chunk == 0) return CPA_ESTATE;                 // not a chunked plan
    if (!plan->d_base || step != plan->next_step) return CPA_ESTATE;
    if (step < 0 || step >= plan->n_steps) return CPA_EINVAL;
    const int B = plan->B, T = plan->T;
    const bool has_prefill = step < (int)plan->chunk_steps.size();
    bool has_decode = false;
    for (int b = 0; b < B; ++b) has_decode |= plan->dec_start[b] <= step && step < plan->dec_start[b] + T;
    if (has_prefill && (!q || !k || !v || !o || o == q || o == k || o == v)) return CPA_EINVAL;
    if (has_decode && (!q_dec || !k_new || !v_new || !o_dec || !d_workspace)) return CPA_EINVAL;
    const void* ptrs[] = {q, k, v, o, q_dec, k_new, v_new, o_dec, k_pool, v_pool, d_workspace};
    for (const void* ptr : ptrs)
        if (ptr && !cpa_aligned16(ptr)) return CPA_EINVAL;

    cudaStream_t main_st = (cudaStream_t)stream;
    cudaStream_t pre_st = main_st;
    const bool side_by_side = has_prefill && has_decode;
    if (side_by_side) {
        if (int rc = ensure_side_stream(plan)) return rc;
        pre_st = plan->side_stream;
        if (cudaEventRecord(plan->ev_fork, main_st) != cudaSuccess ||
            cudaStreamWaitEvent(pre_st, plan->ev_fork, 0) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
    }
    int rc = CPA_OK;
    if (has_prefill) {
        // the chunk's rows attend over the block's earlier chunks (cached pages) and over the chunk itself
        const cpa_chunk_step& cs = plan->chunk_steps[(size_t)step];
        rc = cpa_prefill_tc_list(plan, q, k, v, o, k_pool, v_pool, plan->d_base + cs.off_items, plan->d_base + cs.off_sched,
                                 cs.ctas, cs.rounds, pre_st);
    }
    // the chunk's K/V go to the pages, and every block that does not decode gets its next length
    if (rc == CPA_OK) rc = cpa_append_chunk(plan, step, k, v, k_pool, v_pool, pre_st);
    if (rc == CPA_OK && has_decode)
        rc = cpa_decode_launch(plan, q_dec, k_new, v_new, k_pool, v_pool, o_dec, d_workspace, cpa_decode_mode{step, T, 0, nullptr},
                               has_prefill ? plan->decode_sms : 0, main_st);
    if (side_by_side) {
        // joined even after a failed launch, so that the caller's stream never runs ahead of the second one
        if (cudaEventRecord(plan->ev_join, pre_st) != cudaSuccess ||
            cudaStreamWaitEvent(main_st, plan->ev_join, 0) != cudaSuccess) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
    }
    if (rc != CPA_OK) return rc;
    // host mirror of the lengths, and the other length buffer is now the current one
    for (int b = 0; b < B; ++b) {
        if (plan->dec_start[b] <= step && step < plan->dec_start[b] + T) plan->seq_lens[b] += 1;
        else if (step < plan->dec_start[b]) plan->seq_lens[b] = std::min(plan->block_lens[b], (step + 1) * plan->chunk);
    }
    plan->cur_lens ^= 1;
    plan->next_step = step + 1;
    return CPA_OK;
}

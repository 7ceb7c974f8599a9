// Steps of an event with chunked prefill (the serving engine of the paper's Section 4.2 runs with chunked
// prefill enabled; Section 6 finds that 16k blocks are prefill-bound): the blocks that still have prompt left
// prefill it chunk by chunk, and the blocks that are past their prompt decode meanwhile.  The two touch
// different blocks, so they run side by side: the chunks one after the other on a second stream the plan owns,
// each on most SMs; the decode launches on the caller's stream, on the SMs the plan keeps free for them.  A
// chunk is given the time of `steps_per_chunk` decode steps by the schedule (which fixes when a block may start
// to decode), but the chunks themselves run back to back; the caller's stream waits for them only when a block
// goes from its last chunk to its first decode step, and at the end of the schedule.
#include <cuda_runtime.h>

#include <algorithm>

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
    const int B = plan->B, T = plan->T, r = plan->steps_per_chunk;
    const int n_chunks = (int)plan->chunk_steps.size();
    const int chunk = step / r;
    const bool starts_chunk = step % r == 0 && chunk < n_chunks;
    const bool beside_chunk = chunk < n_chunks;              // by the schedule a chunk is under way during this step
    bool has_decode = false, first_decode = false;
    for (int b = 0; b < B; ++b) {
        const int pos = step - plan->dec_start[b];
        has_decode |= pos >= 0 && pos < T;
        first_decode |= pos == 0 && T > 0;
    }
    const bool last = step == plan->n_steps - 1;
    if (starts_chunk && (!q || !k || !v || !o || o == q || o == k || o == v)) return CPA_EINVAL;
    if (has_decode && (!q_dec || !k_new || !v_new || !o_dec || !d_workspace)) return CPA_EINVAL;
    const void* ptrs[] = {q, k, v, o, q_dec, k_new, v_new, o_dec, k_pool, v_pool, d_workspace};
    for (const void* ptr : ptrs)
        if (ptr && !cpa_aligned16(ptr)) return CPA_EINVAL;

    cudaStream_t main_st = (cudaStream_t)stream;
    auto join = [&]() -> int {   // the caller's stream waits for every chunk started so far
        if (!plan->chunk_pending) return CPA_OK;
        if (cudaStreamWaitEvent(main_st, plan->ev_join, 0) != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
        plan->chunk_pending = false;
        return CPA_OK;
    };
    // a block that decodes its first token now needs its last chunk, which is the one started most recently
    if (first_decode)
        if (int rc = join()) return rc;
    int rc = CPA_OK;
    if (starts_chunk) {
        if ((rc = ensure_side_stream(plan)) != CPA_OK) return rc;
        // The first chunk follows whatever the caller has enqueued on `stream` so far (the inputs of all chunks);
        // later chunks follow only the chunk before them, so that they run back to back instead of at the pace
        // of the decode steps in between.
        if (chunk == 0 && (cudaEventRecord(plan->ev_fork, main_st) != cudaSuccess ||
                           cudaStreamWaitEvent(plan->side_stream, plan->ev_fork, 0) != cudaSuccess)) {
            (void)cudaGetLastError();
            return CPA_ECUDA;
        }
        // the chunk's rows attend over the block's earlier chunks (cached pages) and over the chunk itself; then
        // its K/V go to the block's pages, where the next chunk and the decode steps find them
        const cpa_chunk_step& cs = plan->chunk_steps[(size_t)chunk];
        rc = cpa_prefill_tc_list(plan, q, k, v, o, k_pool, v_pool, plan->d_base + cs.off_items, plan->d_base + cs.off_sched,
                                 cs.ctas, cs.rounds, plan->side_stream);
        if (rc == CPA_OK) rc = cpa_append_chunk(plan, chunk, k, v, k_pool, v_pool, plan->side_stream);
        if (cudaEventRecord(plan->ev_join, plan->side_stream) != cudaSuccess) { (void)cudaGetLastError(); return CPA_ECUDA; }
        plan->chunk_pending = true;
        if (rc != CPA_OK) return rc;
    }
    if (has_decode) {
        rc = cpa_decode_launch(plan, q_dec, k_new, v_new, k_pool, v_pool, o_dec, d_workspace,
                               cpa_decode_mode{step, T, 0, nullptr}, beside_chunk ? plan->decode_sms : 0, main_st);
        if (rc != CPA_OK) return rc;
        // host mirror of the lengths; the other length buffer is now the current one
        for (int b = 0; b < B; ++b) {
            const int pos = step - plan->dec_start[b];
            if (pos >= 0 && pos < T) plan->seq_lens[b] = plan->prefix_lens[b] + plan->block_lens[b] + pos + 1;
        }
        plan->cur_lens ^= 1;
    }
    for (int b = 0; b < B; ++b)   // (mirror: a block's prompt counts as cached once its last chunk has been started)
        if (starts_chunk && step < plan->dec_start[b])
            plan->seq_lens[b] = plan->prefix_lens[b] + std::min(plan->block_lens[b], (chunk + 1) * plan->chunk);
    if (last)
        if ((rc = join()) != CPA_OK) return rc;
    plan->next_step = step + 1;
    return CPA_OK;
}

extern "C" int cpa_step_mixed_range(cpa_plan* plan, int32_t first_step, int32_t num_steps, const void* q, const void* k,
                                    const void* v, void* o, const void* q_dec, const void* k_new, const void* v_new,
                                    void* o_dec, void* k_pool, void* v_pool, void* d_workspace, void* stream) {
    if (!plan || num_steps < 0) return CPA_EINVAL;
    const int64_t q_step = (int64_t)plan->B * plan->cfg.num_q_heads * plan->cfg.head_dim * 2;     // bytes per step
    const int64_t kv_step = (int64_t)plan->B * plan->cfg.num_kv_heads * plan->cfg.head_dim * 2;
    auto at = [](const void* base, int64_t off) -> const void* {
        return base ? static_cast<const char*>(base) + off : nullptr;
    };
    for (int32_t i = 0; i < num_steps; ++i) {
        const int rc = cpa_step_mixed(plan, first_step + i, q, k, v, o, at(q_dec, i * q_step), at(k_new, i * kv_step),
                                      at(v_new, i * kv_step), const_cast<void*>(at(o_dec, i * q_step)), k_pool, v_pool,
                                      d_workspace, stream);
        if (rc != CPA_OK) return rc;
    }
    return CPA_OK;
}

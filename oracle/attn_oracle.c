/*
 * CPU fp64 oracle for block-diagonal causal attention.  TEST INFRASTRUCTURE ONLY:
 * it exists so that the CUDA path can be checked against the plain definition;
 * the product never calls it and it shares no code with the CUDA path.
 *
 * What it follows.  The paper (Section 4, "Snapshot & partition" / "Dispatch" /
 * "Merge") cuts a history into N contiguous blocks and gives every block to its
 * own summarisation sequence; in the "independent chunks" layout each sequence
 * sees only its own block.  The paper does not spell out attention, so the
 * arithmetic below is the textbook definition of causal softmax attention with
 * grouped-query heads, applied per block:
 *
 *     s_j  = scale * sum_c q[i,h,c] * k[j,g,c]        0 <= j <= i, g = h div G
 *     m    = max_j s_j
 *     p_j  = exp(s_j - m)
 *     O[i,h,:] = sum_j p_j v[j,g,:] / sum_j p_j
 *
 * Three nested loops, no tiling, no running (online) softmax.  Inputs are bf16
 * bit patterns widened exactly to double; everything else is double.
 *
 * Threads only partition the outermost (row, head) loop; each output element is
 * produced by exactly one thread with the same operation order as a serial run.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static inline double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * One query row against the first n_visible keys of one sequence.
 *   q_row : [d]           bf16 bits (one head)
 *   k, v  : [*, Hkv, d]   bf16 bits, row stride Hkv*d; head g selected
 *   out   : [d] doubles;  p_out (optional) : [n_visible] softmax weights
 */
static void attend_row(const uint16_t* q_row, const uint16_t* k, const uint16_t* v,
                       int64_t n_visible, int Hkv, int g, int d, double scale,
                       double* out, double* p_out, double* scratch /* [n_visible] */) {
    const int64_t stride = (int64_t)Hkv * d;
    double m = -INFINITY;
    for (int64_t j = 0; j < n_visible; ++j) {
        const uint16_t* kj = k + j * stride + (int64_t)g * d;
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += bf16_to_double(q_row[c]) * bf16_to_double(kj[c]);
        s *= scale;
        scratch[j] = s;
        if (s > m) m = s;
    }
    double denom = 0.0;
    for (int64_t j = 0; j < n_visible; ++j) {
        scratch[j] = exp(scratch[j] - m);
        denom += scratch[j];
    }
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    for (int64_t j = 0; j < n_visible; ++j) {
        const uint16_t* vj = v + j * stride + (int64_t)g * d;
        const double p = scratch[j];
        for (int c = 0; c < d; ++c) out[c] += p * bf16_to_double(vj[c]);
    }
    for (int c = 0; c < d; ++c) out[c] /= denom;
    if (p_out)
        for (int64_t j = 0; j < n_visible; ++j) p_out[j] = scratch[j] / denom;
}

/* ------------------------------------------------------------------------- */

typedef struct {
    const uint16_t *q, *k, *v;
    const int32_t* cu_seqlens;
    int B, Hq, Hkv, d;
    double scale;
    const int64_t* rows; /* global token ids, or NULL for all rows */
    int64_t n_rows;
    double* out;
    int64_t max_len;
    int tid, n_threads;
} prefill_job;

static void* prefill_worker(void* arg) {
    prefill_job* J = (prefill_job*)arg;
    const int G = J->Hq / J->Hkv;
    double* scratch = (double*)malloc(sizeof(double) * (size_t)(J->max_len > 0 ? J->max_len : 1));
    const int64_t n_items = J->n_rows * J->Hq;
    for (int64_t it = J->tid; it < n_items; it += J->n_threads) {
        const int64_t r = it / J->Hq;
        const int h = (int)(it % J->Hq);
        const int64_t tok = J->rows ? J->rows[r] : r;
        /* block that holds this token */
        int b = 0;
        while (b + 1 < J->B && tok >= J->cu_seqlens[b + 1]) ++b;
        const int64_t start = J->cu_seqlens[b];
        const int64_t i = tok - start; /* position inside its block */
        const uint16_t* q_row = J->q + (tok * J->Hq + h) * (int64_t)J->d;
        const uint16_t* kb = J->k + start * (int64_t)J->Hkv * J->d;
        const uint16_t* vb = J->v + start * (int64_t)J->Hkv * J->d;
        attend_row(q_row, kb, vb, i + 1, J->Hkv, h / G, J->d, J->scale,
                   J->out + (r * J->Hq + h) * (int64_t)J->d, NULL, scratch);
    }
    free(scratch);
    return NULL;
}

/*
 * Causal prefill over a packed ragged batch of blocks.
 *   q [tokens,Hq,d], k,v [tokens,Hkv,d]: bf16 bits; cu_seqlens [B+1]
 *   rows: n_rows global token ids to evaluate (NULL = every token, n_rows = tokens)
 *   out : [n_rows, Hq, d] doubles
 * Returns 0, or -1 on bad arguments.
 */
int oracle_prefill(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                   const int32_t* cu_seqlens, int B, int Hq, int Hkv, int d, double scale,
                   const int64_t* rows, int64_t n_rows, double* out, int n_threads) {
    if (B < 1 || Hq < 1 || Hkv < 1 || d < 1 || Hq % Hkv != 0 || n_threads < 1) return -1;
    int64_t max_len = 0;
    for (int b = 0; b < B; ++b) {
        int64_t L = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        if (L < 0) return -1;
        if (L > max_len) max_len = L;
    }
    if (n_threads > 256) n_threads = 256;
    pthread_t th[256];
    prefill_job jobs[256];
    for (int t = 0; t < n_threads; ++t) {
        prefill_job j = {q, k, v, cu_seqlens, B, Hq, Hkv, d, scale, rows, n_rows, out, max_len, t, n_threads};
        jobs[t] = j;
    }
    for (int t = 1; t < n_threads; ++t) pthread_create(&th[t], NULL, prefill_worker, &jobs[t]);
    prefill_worker(&jobs[0]);
    for (int t = 1; t < n_threads; ++t) pthread_join(th[t], NULL);
    return 0;
}

/*
 * One query token (all Hq heads) over a contiguous sequence of n keys.
 *   q [Hq,d], k,v [n,Hkv,d] bf16 bits; out [Hq,d] doubles;
 *   p_out optional [Hq,n] softmax weights.
 */
int oracle_attend_token(const uint16_t* q, const uint16_t* k, const uint16_t* v, int64_t n,
                        int Hq, int Hkv, int d, double scale, double* out, double* p_out) {
    if (n < 1 || Hq < 1 || Hkv < 1 || d < 1 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    double* scratch = (double*)malloc(sizeof(double) * (size_t)n);
    for (int h = 0; h < Hq; ++h)
        attend_row(q + (int64_t)h * d, k, v, n, Hkv, h / G, d, scale, out + (int64_t)h * d,
                   p_out ? p_out + (int64_t)h * n : NULL, scratch);
    free(scratch);
    return 0;
}

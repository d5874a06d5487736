/*
 * CPU oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * Plain fp64 masked grouped-query softmax attention over explicitly concatenated K/V, one
 * (request, query row, query head) at a time: no tiling, no online softmax, no splitting.  It is
 * the definition the GPU path must reproduce; it shares no code, header, table or helper with the
 * CUDA library and must only be used by the tests, the smoke check and the benchmark's CPU
 * baseline leg.
 *
 * What it follows:
 *  - attention over a request's whole cached K/V seen as one contiguous array (xTensor section,
 *    "Operator Adaptation": operators receive a start address and offsets, no block table);
 *  - speculative verification: m+1 query rows of one sequence against the same K (Optimized
 *    Speculative Decoding, "MLA Optimization"), read here as a linear draft chain, i.e. a causal
 *    mask among the q_len newest tokens and full visibility of the older context;
 *  - merging partial results of a split sequence (Hierarchical DP Load Balance, Layer 3, and the
 *    "aggregation operator" of Layer 2), written as the exact log-sum-exp identity;
 *  - the xTensor address identity (Eq. 2): page index and in-page offset of a virtual address.
 *
 * Conventions: head h of H_q uses KV head h / (H_q / H_kv); kv_len counts the q_len newest tokens;
 * query row i sits at position kv_len - q_len + i and sees keys 0..that position inclusive; LSE is
 * a natural logarithm; inputs are bf16 bit patterns widened exactly to double.
 *
 * Parity pins (tests/test_oracle_pins.py): single key returns V; identical keys return mean(V);
 * weights sum to one; split + merge equals unsplit; GQA equals MHA with repeated heads; verify row
 * equals decode on the truncated context; two-key logistic closed form; shift / permutation
 * invariance; huge-score stability; 50-digit decimal brute force; torch fp64 SDPA special case;
 * Eq. 2 against integer divmod identities.  No function here is "parity unpinned".
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* scores s_j = scale * <q, k_j> for j < n, d ascending */
static void scores_row(const uint16_t *q_row, const uint16_t *k, int n, int n_kv_heads, int g, int D,
                       double scale, double *s) {
    for (int j = 0; j < n; ++j) {
        const uint16_t *k_row = k + ((size_t)j * n_kv_heads + g) * D;
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += bf16_to_double(q_row[d]) * bf16_to_double(k_row[d]);
        s[j] = scale * acc;
    }
}

/*
 * One request.  q [q_len][H_q][D], k/v [kv_len][H_kv][D] (bf16 bits), out [q_len][H_q][D] fp64,
 * lse [q_len][H_q] fp64 (may be NULL).  Returns 0, or -1 on invalid sizes.
 */
int oracle_gqa_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v, int q_len, int kv_len,
                         int n_q_heads, int n_kv_heads, int head_dim, double scale, double *out,
                         double *lse) {
    if (q_len < 1 || kv_len < q_len || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0 || head_dim < 1)
        return -1;
    const int G = n_q_heads / n_kv_heads, D = head_dim;
    double *s = (double *)malloc(sizeof(double) * (size_t)kv_len);
    if (!s) return -2;
    for (int i = 0; i < q_len; ++i) {
        for (int h = 0; h < n_q_heads; ++h) {
            const int g = h / G;
            const int n = kv_len - q_len + i + 1; /* visible keys */
            const uint16_t *q_row = q + ((size_t)i * n_q_heads + h) * D;
            scores_row(q_row, k, n, n_kv_heads, g, D, scale, s);
            double m = s[0];
            for (int j = 1; j < n; ++j)
                if (s[j] > m) m = s[j];
            double l = 0.0;
            for (int j = 0; j < n; ++j) {
                s[j] = exp(s[j] - m);
                l += s[j];
            }
            double *o = out + ((size_t)i * n_q_heads + h) * D;
            for (int d = 0; d < D; ++d) {
                double acc = 0.0;
                for (int j = 0; j < n; ++j)
                    acc += s[j] * bf16_to_double(v[((size_t)j * n_kv_heads + g) * D + d]);
                o[d] = acc / l;
            }
            if (lse) lse[(size_t)i * n_q_heads + h] = m + log(l);
        }
    }
    free(s);
    return 0;
}

/* Softmax weights p_j (j < kv_len - q_len + i + 1) of query row i, head h: debugging / pin P3. */
int oracle_softmax_weights(const uint16_t *q, const uint16_t *k, int q_len, int kv_len, int n_q_heads,
                           int n_kv_heads, int head_dim, double scale, int i, int h, double *p) {
    if (q_len < 1 || kv_len < q_len || n_q_heads % n_kv_heads != 0 || i < 0 || i >= q_len || h < 0 ||
        h >= n_q_heads)
        return -1;
    const int G = n_q_heads / n_kv_heads, D = head_dim, g = h / G;
    const int n = kv_len - q_len + i + 1;
    scores_row(q + ((size_t)i * n_q_heads + h) * D, k, n, n_kv_heads, g, D, scale, p);
    double m = p[0];
    for (int j = 1; j < n; ++j)
        if (p[j] > m) m = p[j];
    double l = 0.0;
    for (int j = 0; j < n; ++j) {
        p[j] = exp(p[j] - m);
        l += p[j];
    }
    for (int j = 0; j < n; ++j) p[j] /= l;
    return n;
}

/*
 * Merge n_parts partial results of ONE query row: o_parts [n_parts][D] (each already normalised
 * by its own sum), lse_parts [n_parts].  M = max lse; w_s = exp(lse_s - M); O = sum w_s O_s / sum w_s;
 * LSE = M + log(sum w_s).  A part with lse = -inf (no visible key) has weight zero.
 */
int oracle_merge_lse(int n_parts, int D, const double *o_parts, const double *lse_parts, double *o,
                     double *lse) {
    if (n_parts < 1 || D < 1) return -1;
    double M = -INFINITY;
    for (int s = 0; s < n_parts; ++s)
        if (lse_parts[s] > M) M = lse_parts[s];
    if (M == -INFINITY) return -1; /* no visible key anywhere: undefined */
    double W = 0.0;
    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int s = 0; s < n_parts; ++s) {
        if (lse_parts[s] == -INFINITY) continue;
        const double w = exp(lse_parts[s] - M);
        W += w;
        for (int d = 0; d < D; ++d) o[d] += w * o_parts[(size_t)s * D + d];
    }
    for (int d = 0; d < D; ++d) o[d] /= W;
    if (lse) *lse = M + log(W);
    return 0;
}

/* xTensor Eq. 2: physical page index and in-page offset of a virtual address inside a request's range. */
int oracle_xtensor_locate(uint64_t virt_addr, uint64_t virt_start, uint64_t page_size, uint64_t *phypage_idx,
                          uint64_t *offset) {
    if (page_size == 0 || virt_addr < virt_start) return -1;
    *phypage_idx = (virt_addr - virt_start) / page_size;
    *offset = (virt_addr - virt_start) % page_size;
    return 0;
}

/* ---- batch driver: the same per-request routine spread over host threads, nothing else ---- */
typedef struct {
    int n_req, next;
    pthread_mutex_t mu;
    const uint16_t *const *q, *const *k, *const *v;
    const int32_t *q_len, *kv_len;
    int n_q_heads, n_kv_heads, head_dim;
    double scale;
    double *const *out, *const *lse;
    int status;
} batch_job;

static void *batch_worker(void *arg) {
    batch_job *job = (batch_job *)arg;
    for (;;) {
        pthread_mutex_lock(&job->mu);
        int r = job->next++;
        pthread_mutex_unlock(&job->mu);
        if (r >= job->n_req) break;
        int st = oracle_gqa_attention(job->q[r], job->k[r], job->v[r], job->q_len[r], job->kv_len[r],
                                      job->n_q_heads, job->n_kv_heads, job->head_dim, job->scale, job->out[r],
                                      job->lse ? job->lse[r] : NULL);
        if (st != 0) {
            pthread_mutex_lock(&job->mu);
            job->status = st;
            pthread_mutex_unlock(&job->mu);
        }
    }
    return NULL;
}

/* Requests are handed out one at a time to n_threads workers (order given by the caller). */
int oracle_gqa_attention_batch(int n_req, const uint16_t *const *q, const uint16_t *const *k,
                               const uint16_t *const *v, const int32_t *q_len, const int32_t *kv_len,
                               int n_q_heads, int n_kv_heads, int head_dim, double scale, double *const *out,
                               double *const *lse, int n_threads) {
    if (n_req < 1) return -1;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > n_req) n_threads = n_req;
    batch_job job = {n_req, 0,  PTHREAD_MUTEX_INITIALIZER, q, k, v, q_len, kv_len, n_q_heads, n_kv_heads,
                     head_dim, scale, out, lse, 0};
    pthread_t *th = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)n_threads);
    if (!th) return -2;
    for (int t = 0; t < n_threads; ++t) pthread_create(&th[t], NULL, batch_worker, &job);
    for (int t = 0; t < n_threads; ++t) pthread_join(th[t], NULL);
    free(th);
    return job.status;
}

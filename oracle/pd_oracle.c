/*
 * CPU oracle for paged grouped-query decode attention and the 1-token KV append.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the
 * path computes. It shares no code with the CUDA library, is never linked into
 * it and must never be called from a product path.
 *
 * What it states. The paper's decode cost model has a per-sequence term b whose
 * source is the extra KV-cache HBM reads of every concurrently decoding
 * sequence (Eq. 1, text below it), and every generated token joins the context
 * of its trajectory (Sec. 2.1, p_{i+1} = p_i + r_i + o_i). The paper prints no
 * attention formula; the computation behind the b term is scaled dot-product
 * attention of one new query token over the cached tokens, with each KV head
 * shared by a contiguous group of query heads:
 *
 *   kvh = h / g,            g = num_q_heads / num_kv_heads
 *   K_t = k_pages[page_table[b][t / P]][kvh][t % P][:]     t = 0 .. L_b - 1
 *   s_t = sm_scale * <q[b][h], K_t>
 *   out[b][h] = sum_t softmax(s)_t * V_t,    lse[b][h] = log sum_t exp(s_t)
 *
 * Everything is evaluated in fp64 in index order, two passes (max, then sums),
 * no blocking, no online rescaling. bf16 inputs convert to fp64 exactly.
 *
 * Pins (tests/test_oracle_pins.py): one-token context, identical keys, two
 * closed forms (tanh(1/2); a three-token softmax), brute force on tiny inputs,
 * an independently written NumPy formulation, page-permutation invariance,
 * shift invariance, poison in masked slots, overflow safety, split + LSE merge
 * over every partition of a short context.
 *
 * Pool layout (a choice of this repository, the paper describes none):
 *   k_pages, v_pages : [num_pages][num_kv_heads][page_size][head_dim] bf16
 *   page_table       : [batch][max_pages_per_seq] int32, entry i = physical
 *                      page of tokens [i*P, (i+1)*P); entries past
 *                      ceil(L/P) are never read
 *   ctx_lens         : [batch] int32
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

typedef struct {
    const uint16_t *q, *k_pages, *v_pages;
    const int32_t *page_table, *ctx_lens;
    const int32_t *t_begin, *t_end; /* optional per-sequence token range */
    int B, Hq, Hkv, d, P, MP;
    double scale;
    double *out, *lse;
    int next_row; /* work counter, guarded by mu */
    pthread_mutex_t mu;
} attn_job;

/* One (sequence, query head) row: the definition, written out. */
static void attn_row(const attn_job *J, int b, int h, double *s_buf)
{
    const int d = J->d, P = J->P;
    const int g = J->Hq / J->Hkv;
    const int kvh = h / g;
    int t0 = 0, t1 = J->ctx_lens[b];
    if (J->t_begin) t0 = J->t_begin[b];
    if (J->t_end) t1 = J->t_end[b];
    double *o = J->out + ((size_t)b * J->Hq + h) * d;
    for (int j = 0; j < d; ++j) o[j] = 0.0;
    if (t1 <= t0) { /* empty context: zero output, lse = -inf */
        J->lse[(size_t)b * J->Hq + h] = -INFINITY;
        return;
    }
    const uint16_t *qrow = J->q + ((size_t)b * J->Hq + h) * d;
    const size_t page_stride = (size_t)J->Hkv * P * d;
    /* pass 1: logits and their maximum */
    double m = -INFINITY;
    for (int t = t0; t < t1; ++t) {
        int32_t page = J->page_table[(size_t)b * J->MP + t / P];
        const uint16_t *krow = J->k_pages + (size_t)page * page_stride + ((size_t)kvh * P + t % P) * d;
        double dot = 0.0;
        for (int j = 0; j < d; ++j) dot += bf16_to_f64(qrow[j]) * bf16_to_f64(krow[j]);
        double s = J->scale * dot;
        s_buf[t - t0] = s;
        if (s > m) m = s;
    }
    /* pass 2: normaliser and weighted sum of V */
    double Z = 0.0;
    for (int t = t0; t < t1; ++t) {
        double p = exp(s_buf[t - t0] - m);
        Z += p;
        int32_t page = J->page_table[(size_t)b * J->MP + t / P];
        const uint16_t *vrow = J->v_pages + (size_t)page * page_stride + ((size_t)kvh * P + t % P) * d;
        for (int j = 0; j < d; ++j) o[j] += p * bf16_to_f64(vrow[j]);
    }
    for (int j = 0; j < d; ++j) o[j] /= Z;
    J->lse[(size_t)b * J->Hq + h] = m + log(Z);
}

static void *attn_worker(void *arg)
{
    attn_job *J = (attn_job *)arg;
    int maxlen = 1;
    for (int b = 0; b < J->B; ++b) {
        int t0 = J->t_begin ? J->t_begin[b] : 0;
        int t1 = J->t_end ? J->t_end[b] : J->ctx_lens[b];
        if (t1 - t0 > maxlen) maxlen = t1 - t0;
    }
    double *s_buf = (double *)malloc(sizeof(double) * (size_t)maxlen);
    if (!s_buf) return (void *)1;
    const int rows = J->B * J->Hq;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int r = J->next_row++;
        pthread_mutex_unlock(&J->mu);
        if (r >= rows) break;
        attn_row(J, r / J->Hq, r % J->Hq, s_buf);
    }
    free(s_buf);
    return NULL;
}

/*
 * Attention over tokens [t_begin[b], t_end[b]) of every sequence (NULL range
 * pointers mean [0, ctx_lens[b])). out: [B][Hq][d] fp64, lse: [B][Hq] fp64.
 * Returns 0, or -1 on bad arguments / allocation failure.
 */
int pd_oracle_decode_attn(const uint16_t *q, const uint16_t *k_pages, const uint16_t *v_pages,
                          const int32_t *page_table, const int32_t *ctx_lens,
                          const int32_t *t_begin, const int32_t *t_end,
                          int B, int Hq, int Hkv, int d, int P, int MP, float sm_scale,
                          double *out, double *lse, int nthreads)
{
    if (B < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || P <= 0 || MP <= 0) return -1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    attn_job J;
    J.q = q; J.k_pages = k_pages; J.v_pages = v_pages;
    J.page_table = page_table; J.ctx_lens = ctx_lens;
    J.t_begin = t_begin; J.t_end = t_end;
    J.B = B; J.Hq = Hq; J.Hkv = Hkv; J.d = d; J.P = P; J.MP = MP;
    J.scale = (double)sm_scale; /* the fp32 value the caller passes, widened */
    J.out = out; J.lse = lse; J.next_row = 0;
    pthread_mutex_init(&J.mu, NULL);
    int rc = 0;
    if (nthreads == 1) {
        if (attn_worker(&J) != NULL) rc = -1;
    } else {
        pthread_t th[256];
        int started = 0;
        for (int i = 0; i < nthreads; ++i) {
            if (pthread_create(&th[i], NULL, attn_worker, &J) != 0) break;
            ++started;
        }
        if (started == 0) rc = -1;
        for (int i = 0; i < started; ++i) {
            void *ret = NULL;
            pthread_join(th[i], &ret);
            if (ret != NULL) rc = -1;
        }
    }
    pthread_mutex_destroy(&J.mu);
    return rc;
}

/*
 * Merge of n partial results of ONE row, each the attention over a disjoint
 * part of the context: o_parts [n][d] (each already normalised over its part),
 * lse_parts [n]. With w_i = exp(lse_i - max lse):
 *   out = sum_i w_i o_i / sum_i w_i,   lse = max lse + log sum_i w_i
 * Parts with lse = -inf (empty) carry no weight.
 */
int pd_oracle_lse_merge(const double *o_parts, const double *lse_parts, int n, int d,
                        double *out, double *lse)
{
    if (n < 0 || d <= 0) return -1;
    double M = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (lse_parts[i] > M) M = lse_parts[i];
    for (int j = 0; j < d; ++j) out[j] = 0.0;
    if (M == -INFINITY) {
        *lse = -INFINITY;
        return 0;
    }
    double W = 0.0;
    for (int i = 0; i < n; ++i) {
        if (lse_parts[i] == -INFINITY) continue;
        double w = exp(lse_parts[i] - M);
        W += w;
        for (int j = 0; j < d; ++j) out[j] += w * o_parts[(size_t)i * d + j];
    }
    for (int j = 0; j < d; ++j) out[j] /= W;
    *lse = M + log(W);
    return 0;
}

/*
 * One-token append (Sec. 2.1: each generated token extends its trajectory's
 * context): for every sequence b, pos = ctx_lens[b], the d bf16 values of each
 * KV head of k_new[b] / v_new[b] ([B][Hkv][d]) are copied into slot pos % P of
 * page page_table[b][pos / P]; then ctx_lens[b] += 1 when advance != 0.
 * Pure byte copy. Returns 0, or -(b+1) for the first sequence whose position
 * or page id is out of range (nothing is written for that sequence).
 */
int pd_oracle_kv_append(const uint16_t *k_new, const uint16_t *v_new,
                        uint16_t *k_pages, uint16_t *v_pages,
                        const int32_t *page_table, int32_t *ctx_lens,
                        int B, int Hkv, int d, int P, int MP, int64_t num_pages, int advance)
{
    int rc = 0;
    const size_t page_stride = (size_t)Hkv * P * d;
    for (int b = 0; b < B; ++b) {
        int pos = ctx_lens[b];
        if (pos < 0 || pos / P >= MP) { if (!rc) rc = -(b + 1); continue; }
        int32_t page = page_table[(size_t)b * MP + pos / P];
        if (page < 0 || (int64_t)page >= num_pages) { if (!rc) rc = -(b + 1); continue; }
        for (int kvh = 0; kvh < Hkv; ++kvh) {
            size_t dst = (size_t)page * page_stride + ((size_t)kvh * P + pos % P) * d;
            size_t src = ((size_t)b * Hkv + kvh) * d;
            memcpy(k_pages + dst, k_new + src, sizeof(uint16_t) * (size_t)d);
            memcpy(v_pages + dst, v_new + src, sizeof(uint16_t) * (size_t)d);
        }
        if (advance) ctx_lens[b] = pos + 1;
    }
    return rc;
}

/*
 * KV page gather / scatter: the data movement behind the cross-pool KV transfer
 * term of the disaggregated prefill model (Eq. 3, B * dL * K / BW): the pages
 * that hold a sequence's new tokens are packed into one contiguous buffer on the
 * prefill side and unpacked into freshly assigned pages on the decode side.
 *
 * For sequence b the logical pages [page_begin[b], page_end[b]) are moved. The
 * packed buffer holds whole pages: packed page (dst_page_offset[b] + i) is
 *   [2][num_kv_heads][page_size][head_dim] bf16   (K block, then V block)
 * of logical page page_begin[b] + i. Pure byte copies in index order.
 * Return 0, or -(b+1) for the first sequence with an out-of-range page id
 * (that sequence is skipped).
 */
int pd_oracle_kv_gather(const uint16_t *k_pages, const uint16_t *v_pages, const int32_t *page_table,
                        const int32_t *page_begin, const int32_t *page_end, const int64_t *dst_page_offset,
                        uint16_t *packed, int B, int Hkv, int d, int P, int MP, int64_t num_pages)
{
    int rc = 0;
    const size_t tile = (size_t)Hkv * P * d; /* elements of one pool page */
    for (int b = 0; b < B; ++b) {
        for (int lp = page_begin[b]; lp < page_end[b]; ++lp) {
            int32_t page = (lp >= 0 && lp < MP) ? page_table[(size_t)b * MP + lp] : -1;
            if (page < 0 || (int64_t)page >= num_pages) { if (!rc) rc = -(b + 1); continue; }
            uint16_t *dst = packed + ((size_t)dst_page_offset[b] + (size_t)(lp - page_begin[b])) * 2 * tile;
            memcpy(dst, k_pages + (size_t)page * tile, sizeof(uint16_t) * tile);
            memcpy(dst + tile, v_pages + (size_t)page * tile, sizeof(uint16_t) * tile);
        }
    }
    return rc;
}

int pd_oracle_kv_scatter(const uint16_t *packed, const int64_t *src_page_offset, uint16_t *k_pages, uint16_t *v_pages,
                         const int32_t *page_table, const int32_t *page_begin, const int32_t *page_end,
                         int B, int Hkv, int d, int P, int MP, int64_t num_pages)
{
    int rc = 0;
    const size_t tile = (size_t)Hkv * P * d;
    for (int b = 0; b < B; ++b) {
        for (int lp = page_begin[b]; lp < page_end[b]; ++lp) {
            int32_t page = (lp >= 0 && lp < MP) ? page_table[(size_t)b * MP + lp] : -1;
            if (page < 0 || (int64_t)page >= num_pages) { if (!rc) rc = -(b + 1); continue; }
            const uint16_t *src = packed + ((size_t)src_page_offset[b] + (size_t)(lp - page_begin[b])) * 2 * tile;
            memcpy(k_pages + (size_t)page * tile, src, sizeof(uint16_t) * tile);
            memcpy(v_pages + (size_t)page * tile, src + tile, sizeof(uint16_t) * tile);
        }
    }
    return rc;
}

/*
 * Append-prefill attention: the step that opens every turn of a multi-turn
 * rollout. The new turn's tokens (observation plus template, dL per trajectory
 * in the prefill terms of Eq. 1 and Eq. 3) are appended to the cached context
 * (Sec. 2.1) and each of them attends causally over the cached prefix and the
 * new tokens up to and including itself; with prefix caching only these dL
 * tokens are computed, but they read the whole context.
 *
 * Queries are packed: q [total_q][num_q_heads][head_dim], sequence b owns rows
 * [q_indptr[b], q_indptr[b+1]). Its K/V (new tokens included) are already in the
 * cache, ctx_lens[b] = L_b counts them. Query i of sequence b sits at absolute
 * position pos = L_b - q_len_b + i and sees tokens 0 .. pos:
 *   out[row][h] = softmax(sm_scale * q[row][h] . K_{0..pos}^T) V_{0..pos}
 * Two passes in fp64 per (row, head), exactly as the decode definition.
 */
typedef struct {
    attn_job base;          /* q points at the packed queries; B is unused here */
    const int32_t *q_indptr;
    int n_seq;
    int next_item;
} prefill_job;

static void *prefill_worker(void *arg)
{
    prefill_job *J = (prefill_job *)arg;
    attn_job *A = &J->base;
    int maxlen = 1;
    for (int b = 0; b < J->n_seq; ++b)
        if (A->ctx_lens[b] > maxlen) maxlen = A->ctx_lens[b];
    double *s_buf = (double *)malloc(sizeof(double) * (size_t)maxlen);
    if (!s_buf) return (void *)1;
    const int total_q = J->q_indptr[J->n_seq];
    const int items = total_q * A->Hq;
    const int d = A->d, P = A->P, g = A->Hq / A->Hkv;
    const size_t page_stride = (size_t)A->Hkv * P * d;
    for (;;) {
        pthread_mutex_lock(&A->mu);
        int it = J->next_item++;
        pthread_mutex_unlock(&A->mu);
        if (it >= items) break;
        const int row = it / A->Hq, h = it % A->Hq, kvh = h / g;
        int b = 0;
        while (J->q_indptr[b + 1] <= row) ++b; /* sequence that owns this query row */
        const int q_len = J->q_indptr[b + 1] - J->q_indptr[b];
        const int pos = A->ctx_lens[b] - q_len + (row - J->q_indptr[b]);
        double *o = A->out + ((size_t)row * A->Hq + h) * d;
        for (int j = 0; j < d; ++j) o[j] = 0.0;
        if (pos < 0) { A->lse[(size_t)row * A->Hq + h] = -INFINITY; continue; }
        const uint16_t *qrow = A->q + ((size_t)row * A->Hq + h) * d;
        double m = -INFINITY;
        for (int t = 0; t <= pos; ++t) {
            int32_t page = A->page_table[(size_t)b * A->MP + t / P];
            const uint16_t *krow = A->k_pages + (size_t)page * page_stride + ((size_t)kvh * P + t % P) * d;
            double dot = 0.0;
            for (int j = 0; j < d; ++j) dot += bf16_to_f64(qrow[j]) * bf16_to_f64(krow[j]);
            s_buf[t] = A->scale * dot;
            if (s_buf[t] > m) m = s_buf[t];
        }
        double Z = 0.0;
        for (int t = 0; t <= pos; ++t) {
            double p = exp(s_buf[t] - m);
            Z += p;
            int32_t page = A->page_table[(size_t)b * A->MP + t / P];
            const uint16_t *vrow = A->v_pages + (size_t)page * page_stride + ((size_t)kvh * P + t % P) * d;
            for (int j = 0; j < d; ++j) o[j] += p * bf16_to_f64(vrow[j]);
        }
        for (int j = 0; j < d; ++j) o[j] /= Z;
        A->lse[(size_t)row * A->Hq + h] = m + log(Z);
    }
    free(s_buf);
    return NULL;
}

int pd_oracle_prefill_attn(const uint16_t *q, const int32_t *q_indptr, const uint16_t *k_pages, const uint16_t *v_pages,
                           const int32_t *page_table, const int32_t *ctx_lens, int n_seq, int Hq, int Hkv, int d,
                           int P, int MP, float sm_scale, double *out, double *lse, int nthreads)
{
    if (n_seq < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || P <= 0 || MP <= 0) return -1;
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    prefill_job J;
    memset(&J, 0, sizeof J);
    J.base.q = q; J.base.k_pages = k_pages; J.base.v_pages = v_pages;
    J.base.page_table = page_table; J.base.ctx_lens = ctx_lens;
    J.base.Hq = Hq; J.base.Hkv = Hkv; J.base.d = d; J.base.P = P; J.base.MP = MP;
    J.base.scale = (double)sm_scale;
    J.base.out = out; J.base.lse = lse;
    J.q_indptr = q_indptr; J.n_seq = n_seq; J.next_item = 0;
    pthread_mutex_init(&J.base.mu, NULL);
    int rc = 0;
    pthread_t th[256];
    int started = 0;
    for (int i = 0; i < nthreads; ++i) {
        if (pthread_create(&th[i], NULL, prefill_worker, &J) != 0) break;
        ++started;
    }
    if (started == 0) rc = (prefill_worker(&J) != NULL) ? -1 : 0;
    for (int i = 0; i < started; ++i) {
        void *ret = NULL;
        pthread_join(th[i], &ret);
        if (ret != NULL) rc = -1;
    }
    pthread_mutex_destroy(&J.base.mu);
    return rc;
}

/*
 * Multi-token append: sequence b receives the rows [q_indptr[b], q_indptr[b+1])
 * of k_new / v_new ([total][Hkv][d]) at positions ctx_lens[b], ctx_lens[b]+1, ...
 * and its length grows by that count. Byte copies; a sequence with any position
 * or page id out of range is skipped whole and reported as -(b+1).
 */
int pd_oracle_kv_append_tokens(const uint16_t *k_new, const uint16_t *v_new, const int32_t *q_indptr,
                               uint16_t *k_pages, uint16_t *v_pages, const int32_t *page_table, int32_t *ctx_lens,
                               int n_seq, int Hkv, int d, int P, int MP, int64_t num_pages)
{
    int rc = 0;
    const size_t page_stride = (size_t)Hkv * P * d;
    for (int b = 0; b < n_seq; ++b) {
        const int n = q_indptr[b + 1] - q_indptr[b];
        const int L = ctx_lens[b];
        int ok = L >= 0 && n >= 0 && (L + n + P - 1) / P <= MP;
        for (int i = 0; ok && i < n; ++i) {
            int32_t page = page_table[(size_t)b * MP + (L + i) / P];
            if (page < 0 || (int64_t)page >= num_pages) ok = 0;
        }
        if (!ok) { if (!rc) rc = -(b + 1); continue; }
        for (int i = 0; i < n; ++i) {
            const int pos = L + i;
            const int32_t page = page_table[(size_t)b * MP + pos / P];
            for (int kvh = 0; kvh < Hkv; ++kvh) {
                size_t dst = (size_t)page * page_stride + ((size_t)kvh * P + pos % P) * d;
                size_t src = ((size_t)(q_indptr[b] + i) * Hkv + kvh) * d;
                memcpy(k_pages + dst, k_new + src, sizeof(uint16_t) * (size_t)d);
                memcpy(v_pages + dst, v_new + src, sizeof(uint16_t) * (size_t)d);
            }
        }
        ctx_lens[b] = L + n;
    }
    return rc;
}

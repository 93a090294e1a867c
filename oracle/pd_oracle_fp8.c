/*
 * CPU oracle for the FP8 variant of the paged KV cache: e4m3 pages with one scale per (page, KV head).
 *
 * TEST INFRASTRUCTURE ONLY, like pd_oracle.c: plain, slow, independent of the CUDA library.
 *
 * The paper has no counterpart (its decode cost b is "extra KV-cache HBM reads", Eq. 1; halving the
 * bytes per cached token halves that term). Everything below is a definition of this repository:
 *
 *   k8, v8    : [num_pages][num_kv_heads][page_size][head_dim] bytes, OCP FP8 E4M3 (bias 7, no
 *               infinities, 0x7f / 0xff = NaN, largest finite value 448)
 *   scales    : [num_pages][num_kv_heads][4] fp32: {k_scale, v_scale, 0, 0}
 *   K_t[j]    = k_scale(page of t, kvh) * e4m3(k8[...][t % P][j]), likewise V
 *   attention : the definition of pd_oracle.c over those K_t, V_t, in fp64, two passes
 *
 * Quantisation of a whole page (all tokens known): amax = max |x| over the page's slots that hold
 * tokens, scale = amax / 448 in fp32 (1 if amax = 0), code = e4m3(x / scale) with the division in fp32,
 * rounding to nearest even and saturation at +-448.
 * One-token append: a token that opens a page (slot 0) sets both scales of that page from its own rows,
 * scale = (amax * 2) / 448 (headroom of a factor two for the 15 tokens that follow; 1 if amax = 0);
 * any other token is quantised with the page's stored scales, saturating.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

double pd_oracle_e4m3_to_f64(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);          /* subnormal */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* fp32 -> e4m3, round to nearest even, saturating to +-448; NaN -> 0x7f. */
uint8_t pd_oracle_f32_to_e4m3(float x)
{
    if (x != x) return 0x7f;
    const uint8_t sign = signbit(x) ? 0x80 : 0x00;
    const double a = fabs((double)x);
    if (a > 448.0) return sign | 0x7e; /* everything above the largest finite value saturates */
    if (a < ldexp(1.0, -6)) {          /* subnormal range: multiples of 2^-9 */
        const int q = (int)nearbyint(ldexp(a, 9)); /* 0 .. 8; 8 is the smallest normal, code 0x08 */
        return sign | (uint8_t)q;
    }
    int e;
    const double f = frexp(a, &e); /* a = f * 2^e, f in [0.5, 1) */
    int exp_unb = e - 1;
    int m = (int)nearbyint((2.0 * f - 1.0) * 8.0); /* 0 .. 8 */
    if (m == 8) {
        m = 0;
        exp_unb += 1;
    }
    int code = ((exp_unb + 7) << 3) | m;
    if (code > 0x7e) code = 0x7e;
    return sign | (uint8_t)code;
}

static float bf16_to_f32(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* amax over n bf16 values (NaN ignored). */
static float amax_bf16(const uint16_t *x, size_t n)
{
    float a = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        const float v = fabsf(bf16_to_f32(x[i]));
        if (v > a) a = v;
    }
    return a;
}

static void quantize_rows(const uint16_t *src, uint8_t *dst, size_t n, float scale)
{
    for (size_t i = 0; i < n; ++i) dst[i] = pd_oracle_f32_to_e4m3(bf16_to_f32(src[i]) / scale);
}

/*
 * Whole-page quantisation. tokens_in_page[p] = number of leading slots of page p that hold tokens
 * (0 .. P); slots past it do not contribute to amax and are written as code 0.
 */
int pd_oracle_fp8_quantize_pages(const uint16_t *k_pages, const uint16_t *v_pages, const int32_t *tokens_in_page,
                                 int64_t num_pages, int Hkv, int P, int d, uint8_t *k8, uint8_t *v8, float *scales)
{
    for (int64_t p = 0; p < num_pages; ++p) {
        const int n = tokens_in_page[p];
        if (n < 0 || n > P) return -1;
        for (int h = 0; h < Hkv; ++h) {
            const size_t tile = ((size_t)p * Hkv + h) * P * d;
            float *sc = scales + ((size_t)p * Hkv + h) * 4;
            for (int which = 0; which < 2; ++which) {
                const uint16_t *src = (which ? v_pages : k_pages) + tile;
                uint8_t *dst = (which ? v8 : k8) + tile;
                const float amax = amax_bf16(src, (size_t)n * d);
                const float scale = amax > 0.0f ? amax / 448.0f : 1.0f;
                sc[which] = scale;
                quantize_rows(src, dst, (size_t)n * d, scale);
                memset(dst + (size_t)n * d, 0, (size_t)(P - n) * d);
            }
            sc[2] = 0.0f;
            sc[3] = 0.0f;
        }
    }
    return 0;
}

/* One-token append into FP8 pages; returns the number of sequences appended (others are skipped). */
int pd_oracle_fp8_kv_append(const uint16_t *k_new, const uint16_t *v_new, uint8_t *k8, uint8_t *v8, float *scales,
                            const int32_t *page_table, int32_t *ctx_lens, int B, int Hkv, int d, int P, int MP,
                            int64_t num_pages, int advance)
{
    int done = 0;
    for (int b = 0; b < B; ++b) {
        const int pos = ctx_lens[b];
        if (pos < 0 || pos / P >= MP) continue;
        const int page = page_table[(size_t)b * MP + pos / P];
        if (page < 0 || page >= num_pages) continue;
        const int slot = pos % P;
        for (int h = 0; h < Hkv; ++h) {
            float *sc = scales + ((size_t)page * Hkv + h) * 4;
            for (int which = 0; which < 2; ++which) {
                const uint16_t *src = (which ? v_new : k_new) + ((size_t)b * Hkv + h) * d;
                uint8_t *dst = (which ? v8 : k8) + (((size_t)page * Hkv + h) * P + slot) * d;
                if (slot == 0) {
                    const float amax = amax_bf16(src, (size_t)d);
                    sc[which] = amax > 0.0f ? (amax * 2.0f) / 448.0f : 1.0f;
                }
                quantize_rows(src, dst, (size_t)d, sc[which]);
            }
        }
        if (advance) ctx_lens[b] = pos + 1;
        ++done;
    }
    return done;
}

/* ---- attention over FP8 pages: the definition, one (sequence, query head) row at a time */
typedef struct {
    const uint16_t *q;
    const uint8_t *k8, *v8;
    const float *scales;
    const int32_t *page_table, *ctx_lens;
    int B, Hq, Hkv, d, P, MP;
    double scale;
    double *out, *lse;
    int next_row;
    pthread_mutex_t mu;
} attn8_job;

static void attn8_row(const attn8_job *J, int b, int h, double *s_buf)
{
    const int d = J->d, P = J->P, g = J->Hq / J->Hkv, kvh = h / g, L = J->ctx_lens[b];
    double *o = J->out + ((size_t)b * J->Hq + h) * d;
    for (int j = 0; j < d; ++j) o[j] = 0.0;
    if (L <= 0) {
        J->lse[(size_t)b * J->Hq + h] = -INFINITY;
        return;
    }
    const uint16_t *qrow = J->q + ((size_t)b * J->Hq + h) * d;
    double m = -INFINITY;
    for (int t = 0; t < L; ++t) {
        const int page = J->page_table[(size_t)b * J->MP + t / P];
        const uint8_t *krow = J->k8 + (((size_t)page * J->Hkv + kvh) * P + t % P) * d;
        const double ks = (double)J->scales[((size_t)page * J->Hkv + kvh) * 4 + 0];
        double acc = 0.0;
        for (int j = 0; j < d; ++j) acc += (double)bf16_to_f32(qrow[j]) * (ks * pd_oracle_e4m3_to_f64(krow[j]));
        s_buf[t] = J->scale * acc;
        if (s_buf[t] > m) m = s_buf[t];
    }
    double Z = 0.0;
    for (int t = 0; t < L; ++t) {
        const int page = J->page_table[(size_t)b * J->MP + t / P];
        const uint8_t *vrow = J->v8 + (((size_t)page * J->Hkv + kvh) * P + t % P) * d;
        const double vs = (double)J->scales[((size_t)page * J->Hkv + kvh) * 4 + 1];
        const double p = exp(s_buf[t] - m);
        Z += p;
        for (int j = 0; j < d; ++j) o[j] += p * (vs * pd_oracle_e4m3_to_f64(vrow[j]));
    }
    for (int j = 0; j < d; ++j) o[j] /= Z;
    J->lse[(size_t)b * J->Hq + h] = m + log(Z);
}

static void *attn8_worker(void *arg)
{
    attn8_job *J = (attn8_job *)arg;
    int maxL = 1;
    for (int b = 0; b < J->B; ++b)
        if (J->ctx_lens[b] > maxL) maxL = J->ctx_lens[b];
    double *s_buf = (double *)malloc((size_t)maxL * sizeof(double));
    if (!s_buf) return NULL;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        const int row = J->next_row++;
        pthread_mutex_unlock(&J->mu);
        if (row >= J->B * J->Hq) break;
        attn8_row(J, row / J->Hq, row % J->Hq, s_buf);
    }
    free(s_buf);
    return NULL;
}

int pd_oracle_fp8_decode_attn(const uint16_t *q, const uint8_t *k8, const uint8_t *v8, const float *scales,
                              const int32_t *page_table, const int32_t *ctx_lens, int B, int Hq, int Hkv, int d, int P,
                              int MP, float sm_scale, int n_threads, double *out, double *lse)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    attn8_job J;
    memset(&J, 0, sizeof J);
    J.q = q; J.k8 = k8; J.v8 = v8; J.scales = scales;
    J.page_table = page_table; J.ctx_lens = ctx_lens;
    J.B = B; J.Hq = Hq; J.Hkv = Hkv; J.d = d; J.P = P; J.MP = MP;
    J.scale = (double)sm_scale;
    J.out = out; J.lse = lse;
    pthread_mutex_init(&J.mu, NULL);
    if (n_threads < 1) n_threads = 1;
    if (n_threads > 256) n_threads = 256;
    pthread_t th[256];
    int started = 0;
    for (int i = 1; i < n_threads; ++i)
        if (pthread_create(&th[started], NULL, attn8_worker, &J) == 0) ++started;
    attn8_worker(&J);
    for (int i = 0; i < started; ++i) pthread_join(th[i], NULL);
    pthread_mutex_destroy(&J.mu);
    return 0;
}

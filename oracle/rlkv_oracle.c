/*
 * CPU oracle for decode attention over a head-mixed KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the CUDA
 * library must compute.  It shares no code, header, table or helper with the CUDA
 * path; only tests, the smoke check and the benchmark's cpu-baseline leg may call it.
 *
 * What it states (paper, Section 3.3 last paragraph; Section 4.3 "Inference
 * Efficiency"; Appendix B "Local Attention Implementation"):
 *   - every KV head is either FULL (keeps all tokens) or COMPRESSED (keeps only the
 *     first `sink` tokens and the most recent `window` tokens, in a fixed-size
 *     circular buffer);
 *   - attention itself is ordinary scaled-dot-product attention (Section 3.1, Eq. 1
 *     context: softmax(q.K^T / sqrt(D)).V) restricted to the tokens a head retains;
 *     the G = q_heads / kv_heads query heads j with j / G == h read KV head h.
 *
 * Precision: inputs are bf16 bit patterns (uint16).  Scores, softmax and the output
 * are accumulated in RLKV_ORACLE_ACC (float by default; compile with
 * -DRLKV_ORACLE_ACC=double for the reference-of-the-reference build).  Sums run
 * left-to-right in d and in ascending token order.  No blocking, no fusion.
 *
 * Readings of points the paper leaves open (each also listed in the design notes):
 *   - the token appended in this step is inside the window (append, then attend);
 *   - while n <= sink + window nothing is evicted; the ring starts at token `sink`;
 *   - physical slot of token t in a compressed head: t if t < sink,
 *     else sink + ((t - sink) mod window)   (normative, so state can be bit-compared);
 *   - one length counter per layer, shared by the whole batch (lock-step decode).
 *
 * Parity pins (tests/test_oracle_pins.py): all-full == library causal attention's
 * last row; sink+window >= n == full; brute-force masked softmax; ring invariants;
 * closed forms; planted needle; Table 3's "theoretical" column for the retained-token
 * count; the mixed form of Eq. 1 has its own pins, listed at rlkv_oracle_decode_mixed.
 * The paper prints no numeric attention values, so beyond those pins the
 * numeric output is "parity unpinned" by any printed example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef RLKV_ORACLE_ACC
#define RLKV_ORACLE_ACC float
#endif
typedef RLKV_ORACLE_ACC acc_t;

typedef struct {
    int layers, kv_heads, q_heads, head_dim, batch, max_len, sink, window;
    uint8_t *is_full;        /* [layers*kv_heads] */
    int *len;                /* [layers] */
    uint16_t **k, **v;       /* [layers*batch*kv_heads] -> rows*head_dim bf16 bits */
    int32_t **token_of_slot; /* compressed heads: [cap], -1 = empty; NULL for full heads */
    int threads;
    /* 8-bit storage (rlkv_oracle_set_fp8): the k, v entries of every head hold E4M3 codes */
    int fp8;
    float *k_scale, *v_scale; /* [layers*kv_heads] */
} oracle_t;

static float bf16_to_float(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* ---- 8-bit K/V (the paper's Limitations and Future Work: head-level
 * compression "can be combined with" KV-cache quantisation; no format is given there).
 * Reading taken: the OCP 8-bit floating-point format E4M3 -- 1 sign bit, 4 exponent bits with bias
 * 7, 3 mantissa bits; exponent field 0 holds the subnormals m/8 * 2^-6; there are no infinities and
 * only exponent 15 with mantissa 7 is NaN, so the largest finite value is 1.75 * 2^8 = 448 -- with
 * one scale per (layer, KV head) for K and one for V, given by the caller:
 *     code  = E4M3( fl32( fl32(x) * fl32(1 / scale) ) )    round to nearest, ties to even,
 *                                                           magnitudes above 448 saturate to 448
 *     x_hat = value(code) * scale
 * and attention runs on x_hat as before.  Every head is stored this way, full heads and the sink +
 * window rings of compressed heads alike (one storage format per cache).
 * Pins: every code's value against torch.float8_e4m3fn; the encoder against torch's cast on a
 * sweep that holds every midpoint between neighbouring codes; closed forms. */
float rlkv_oracle_e4m3_value(uint8_t code)
{
    int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    float mag;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) mag = ldexpf((float)m / 8.0f, -6);
    else mag = ldexpf(1.0f + (float)m / 8.0f, e - 7);
    return sign ? -mag : mag;
}

/* Nearest code by search over the 127 finite magnitudes (they grow with the code). */
uint8_t rlkv_oracle_e4m3_encode(float x)
{
    if (x != x) return 0x7f;
    uint8_t sign = signbit(x) ? 0x80 : 0;
    double a = fabs((double)x);
    if (a >= 448.0) return sign | 0x7e;
    int lo = 0;
    for (int c = 0; c <= 0x7e; ++c)
        if ((double)rlkv_oracle_e4m3_value((uint8_t)c) <= a) lo = c;
    double below = a - (double)rlkv_oracle_e4m3_value((uint8_t)lo);
    double above = (double)rlkv_oracle_e4m3_value((uint8_t)(lo + 1)) - a;
    int c = below < above ? lo : (above < below ? lo + 1 : ((lo & 1) ? lo + 1 : lo));
    return sign | (uint8_t)c;
}

static size_t unit_index(const oracle_t *o, int layer, int b, int h)
{
    return ((size_t)layer * o->batch + b) * o->kv_heads + h;
}

static int head_rows(const oracle_t *o, int layer, int h)
{
    return o->is_full[layer * o->kv_heads + h] ? o->max_len : o->sink + o->window;
}

int rlkv_oracle_acc_bytes(void) { return (int)sizeof(acc_t); }

void rlkv_oracle_destroy(oracle_t *o)
{
    if (!o) return;
    if (o->k && o->v && o->token_of_slot) {
        size_t units = (size_t)o->layers * o->batch * o->kv_heads;
        for (size_t u = 0; u < units; ++u) {
            free(o->k[u]);
            free(o->v[u]);
            free(o->token_of_slot[u]);
        }
    }
    free(o->k);
    free(o->v);
    free(o->token_of_slot);
    free(o->is_full);
    free(o->len);
    free(o->k_scale);
    free(o->v_scale);
    free(o);
}

oracle_t *rlkv_oracle_create(int layers, int kv_heads, int q_heads, int head_dim, int batch,
                             int max_len, const uint8_t *head_is_full, int sink, int window)
{
    if (layers < 1 || kv_heads < 1 || q_heads < 1 || q_heads % kv_heads || head_dim < 1 ||
        batch < 1 || max_len < 1 || !head_is_full || sink < 0 || window < 1)
        return NULL;
    oracle_t *o = calloc(1, sizeof *o);
    if (!o) return NULL;
    o->layers = layers; o->kv_heads = kv_heads; o->q_heads = q_heads; o->head_dim = head_dim;
    o->batch = batch; o->max_len = max_len; o->sink = sink; o->window = window;
    o->threads = 1;
    size_t heads = (size_t)layers * kv_heads, units = heads * batch;
    o->is_full = malloc(heads);
    o->len = calloc(layers, sizeof(int));
    o->k = calloc(units, sizeof *o->k);
    o->v = calloc(units, sizeof *o->v);
    o->token_of_slot = calloc(units, sizeof *o->token_of_slot);
    if (!o->is_full || !o->len || !o->k || !o->v || !o->token_of_slot) {
        rlkv_oracle_destroy(o);
        return NULL;
    }
    for (size_t i = 0; i < heads; ++i) o->is_full[i] = head_is_full[i] ? 1 : 0;
    for (int l = 0; l < layers; ++l)
        for (int b = 0; b < batch; ++b)
            for (int h = 0; h < kv_heads; ++h) {
                size_t u = unit_index(o, l, b, h);
                size_t rows = (size_t)head_rows(o, l, h);
                o->k[u] = calloc(rows * head_dim, sizeof(uint16_t));
                o->v[u] = calloc(rows * head_dim, sizeof(uint16_t));
                if (!o->k[u] || !o->v[u]) { rlkv_oracle_destroy(o); return NULL; }
                if (!o->is_full[l * kv_heads + h]) {
                    o->token_of_slot[u] = malloc(rows * sizeof(int32_t));
                    if (!o->token_of_slot[u]) { rlkv_oracle_destroy(o); return NULL; }
                    for (size_t s = 0; s < rows; ++s) o->token_of_slot[u][s] = -1;
                }
            }
    return o;
}

/* Switches the cache to 8-bit storage.  k_scale, v_scale: [layers*kv_heads], positive and finite.
 * Only while the cache is empty.  Returns 0, -7 otherwise. */
int rlkv_oracle_set_fp8(oracle_t *o, const float *k_scale, const float *v_scale)
{
    size_t heads = (size_t)o->layers * o->kv_heads;
    for (int l = 0; l < o->layers; ++l)
        if (o->len[l] != 0) return -7;
    for (size_t i = 0; i < heads; ++i)
        if (!(k_scale[i] > 0) || !(v_scale[i] > 0) || isinf(k_scale[i]) || isinf(v_scale[i])) return -7;
    free(o->k_scale);
    free(o->v_scale);
    o->k_scale = malloc(heads * sizeof(float));
    o->v_scale = malloc(heads * sizeof(float));
    if (!o->k_scale || !o->v_scale) return -4;
    memcpy(o->k_scale, k_scale, heads * sizeof(float));
    memcpy(o->v_scale, v_scale, heads * sizeof(float));
    o->fp8 = 1;
    return 0;
}

/* The 16 stored bits of one element as a number: a bf16 value, or in 8-bit storage the E4M3 code's
 * value times the head's scale. */
static acc_t stored(const oracle_t *o, int layer, int h, uint16_t bits, int is_v)
{
    if (o->fp8) {
        float scale = (is_v ? o->v_scale : o->k_scale)[layer * o->kv_heads + h];
        return (acc_t)rlkv_oracle_e4m3_value((uint8_t)bits) * (acc_t)scale;
    }
    return (acc_t)bf16_to_float(bits);
}

void rlkv_oracle_set_threads(oracle_t *o, int threads) { o->threads = threads < 1 ? 1 : threads; }

int rlkv_oracle_length(const oracle_t *o, int layer)
{
    return (layer < 0 || layer >= o->layers) ? -1 : o->len[layer];
}

/* Slot rule of the compressed ring (Section 4.3: "fixed-size circular buffer (sink + local)"). */
static int slot_of_token(const oracle_t *o, int t)
{
    return t < o->sink ? t : o->sink + ((t - o->sink) % o->window);
}

/* Append one token for every (batch row, KV head) of a layer.
 * k, v: bf16 bits [batch][kv_heads][head_dim].  Returns 0, or -1 when the layer is at max_len
 * (state unchanged). */
int rlkv_oracle_append(oracle_t *o, int layer, const uint16_t *k, const uint16_t *v)
{
    if (layer < 0 || layer >= o->layers) return -2;
    int t = o->len[layer];
    if (t >= o->max_len) return -1;
    int D = o->head_dim;
    for (int b = 0; b < o->batch; ++b)
        for (int h = 0; h < o->kv_heads; ++h) {
            size_t u = unit_index(o, layer, b, h);
            const uint16_t *ks = k + ((size_t)b * o->kv_heads + h) * D;
            const uint16_t *vs = v + ((size_t)b * o->kv_heads + h) * D;
            int row;
            if (o->is_full[layer * o->kv_heads + h]) {
                row = t;
            } else {
                row = slot_of_token(o, t);
                o->token_of_slot[u][row] = t;
            }
            if (o->fp8) {
                float ik = 1.0f / o->k_scale[layer * o->kv_heads + h], iv = 1.0f / o->v_scale[layer * o->kv_heads + h];
                for (int d = 0; d < D; ++d) {
                    o->k[u][(size_t)row * D + d] = rlkv_oracle_e4m3_encode(bf16_to_float(ks[d]) * ik);
                    o->v[u][(size_t)row * D + d] = rlkv_oracle_e4m3_encode(bf16_to_float(vs[d]) * iv);
                }
                continue;
            }
            memcpy(o->k[u] + (size_t)row * D, ks, D * sizeof(uint16_t));
            memcpy(o->v[u] + (size_t)row * D, vs, D * sizeof(uint16_t));
        }
    o->len[layer] = t + 1;
    return 0;
}

/* Row that holds token t of a compressed head, found through token_of_slot (never by
 * assuming a physical order); -1 if the token is not retained. */
static int find_row(const oracle_t *o, size_t u, int t)
{
    int cap = o->sink + o->window;
    for (int s = 0; s < cap; ++s)
        if (o->token_of_slot[u][s] == t) return s;
    return -1;
}

/* Number of tokens a head retains at length n (used by the cost-model pin). */
int rlkv_oracle_retained(const oracle_t *o, int layer, int h)
{
    int n = o->len[layer], count = 0;
    if (o->is_full[layer * o->kv_heads + h]) return n;
    for (int t = 0; t < n; ++t)
        if (t < o->sink || t >= n - o->window) ++count;
    return count;
}

static void attend_one(const oracle_t *o, int layer, int b, int j, const uint16_t *q, float *out,
                       acc_t *s, int *rows)
{
    int D = o->head_dim, G = o->q_heads / o->kv_heads, h = j / G, n = o->len[layer];
    size_t u = unit_index(o, layer, b, h);
    int full = o->is_full[layer * o->kv_heads + h];
    const uint16_t *qj = q + ((size_t)b * o->q_heads + j) * D;
    acc_t scale = (acc_t)1 / (acc_t)sqrt((double)D);

    /* 1. retained set, ascending token order */
    int cnt = 0;
    for (int t = 0; t < n; ++t) {
        if (full) {
            rows[cnt++] = t;
        } else if (t < o->sink || t >= n - o->window) {
            rows[cnt++] = find_row(o, u, t);
        }
    }
    /* 2. scores */
    acc_t m = -INFINITY;
    for (int i = 0; i < cnt; ++i) {
        const uint16_t *kr = o->k[u] + (size_t)rows[i] * D;
        acc_t dot = 0;
        for (int d = 0; d < D; ++d) dot += (acc_t)bf16_to_float(qj[d]) * stored(o, layer, h, kr[d], 0);
        s[i] = dot * scale;
        if (s[i] > m) m = s[i];
    }
    /* 3. softmax and weighted sum of V */
    acc_t l = 0;
    for (int i = 0; i < cnt; ++i) {
        s[i] = sizeof(acc_t) == sizeof(float) ? (acc_t)expf((float)(s[i] - m)) : (acc_t)exp((double)(s[i] - m));
        l += s[i];
    }
    float *oj = out + ((size_t)b * o->q_heads + j) * D;
    for (int d = 0; d < D; ++d) {
        acc_t a = 0;
        for (int i = 0; i < cnt; ++i) a += s[i] * stored(o, layer, h, o->v[u][(size_t)rows[i] * D + d], 1);
        oj[d] = (float)(a / l);
    }
}

/* q: bf16 bits [batch][q_heads][head_dim]; out: float [batch][q_heads][head_dim].
 * Returns 0, -3 if the layer is empty. */
int rlkv_oracle_decode(const oracle_t *o, int layer, const uint16_t *q, float *out)
{
    if (layer < 0 || layer >= o->layers) return -2;
    int n = o->len[layer];
    if (n < 1) return -3;
    int fail = 0;
#pragma omp parallel num_threads(o->threads)
    {
        acc_t *s = malloc((size_t)n * sizeof(acc_t));
        int *rows = malloc((size_t)n * sizeof(int));
        if (!s || !rows) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int b = 0; b < o->batch; ++b)
            for (int j = 0; j < o->q_heads; ++j)
                if (s && rows) attend_one(o, layer, b, j, q, out, s, rows);
        free(s);
        free(rows);
    }
    return fail ? -4 : 0;
}

/* ---- mixed attention with gating adapters (Section 3.1, Eq. 1) ----------------------------
 * The form attention takes while the gates are trained and while samples are generated for that
 * training: every head keeps its full cache, and head h of layer l carries a gate alpha in [0, 1].
 *   out_full_attn  = softmax over all n tokens                     (mask M_causal, last row)
 *   out_local_attn = softmax over {t < sink} U {t >= n - window}   (mask M_local, last row)
 *   out_mix_attn   = alpha * out_full_attn + (1 - alpha) * out_local_attn
 * The gate belongs to the KV head; its G query heads share it.  Scores, both softmaxes and the
 * mix run in acc_t; the query's own token (the last one appended) is inside the window.
 * Pins (tests/test_oracle_pins.py): alpha = 1 against rlkv_oracle_decode on the same cache;
 * alpha = 0 against rlkv_oracle_decode on a cache that holds the same history in compressed
 * heads; a masked softmax written out with boolean mask matrices in numpy; n <= sink + window
 * (both branches equal, so alpha drops out). */
static void attend_masked(const oracle_t *o, int layer, int b, int j, const uint16_t *q, int local,
                          acc_t *res, acc_t *p)
{
    int D = o->head_dim, G = o->q_heads / o->kv_heads, h = j / G, n = o->len[layer];
    size_t u = unit_index(o, layer, b, h);
    const uint16_t *qj = q + ((size_t)b * o->q_heads + j) * D;
    acc_t scale = (acc_t)1 / (acc_t)sqrt((double)D);
    acc_t m = -INFINITY;
    for (int t = 0; t < n; ++t) {
        int keep = !local || t < o->sink || t >= n - o->window;
        p[t] = -INFINITY;
        if (!keep) continue;
        const uint16_t *kr = o->k[u] + (size_t)t * D;
        acc_t dot = 0;
        for (int d = 0; d < D; ++d) dot += (acc_t)bf16_to_float(qj[d]) * (acc_t)bf16_to_float(kr[d]);
        p[t] = dot * scale;
        if (p[t] > m) m = p[t];
    }
    acc_t l = 0;
    for (int t = 0; t < n; ++t) {
        if (p[t] == -INFINITY) { p[t] = 0; continue; }
        p[t] = sizeof(acc_t) == sizeof(float) ? (acc_t)expf((float)(p[t] - m)) : (acc_t)exp((double)(p[t] - m));
        l += p[t];
    }
    for (int d = 0; d < D; ++d) {
        acc_t a = 0;
        for (int t = 0; t < n; ++t)
            if (p[t] != 0) a += p[t] * (acc_t)bf16_to_float(o->v[u][(size_t)t * D + d]);
        res[d] = a / l;
    }
}

/* q: bf16 bits [batch][q_heads][head_dim]; alpha: float [kv_heads], the gates of this layer;
 * out: float [batch][q_heads][head_dim].
 * Returns 0, -3 if the layer is empty, -5 if a head of the layer is compressed (its cache no
 * longer holds what out_full_attn needs), -6 if a gate lies outside [0, 1]. */
int rlkv_oracle_decode_mixed(const oracle_t *o, int layer, const uint16_t *q, const float *alpha, float *out)
{
    if (layer < 0 || layer >= o->layers) return -2;
    int n = o->len[layer], D = o->head_dim, G = o->q_heads / o->kv_heads;
    if (n < 1) return -3;
    if (o->fp8) return -7; /* the training-time form keeps 16-bit rows */
    for (int h = 0; h < o->kv_heads; ++h) {
        if (!o->is_full[layer * o->kv_heads + h]) return -5;
        if (!(alpha[h] >= 0.0f && alpha[h] <= 1.0f)) return -6;
    }
    int fail = 0;
#pragma omp parallel num_threads(o->threads)
    {
        acc_t *p = malloc((size_t)n * sizeof(acc_t));
        acc_t *full = malloc((size_t)D * sizeof(acc_t)), *loc = malloc((size_t)D * sizeof(acc_t));
        if (!p || !full || !loc) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp for collapse(2) schedule(dynamic, 1)
        for (int b = 0; b < o->batch; ++b)
            for (int j = 0; j < o->q_heads; ++j) {
                if (!p || !full || !loc) continue;
                acc_t a = (acc_t)alpha[j / G];
                attend_masked(o, layer, b, j, q, 0, full, p);
                attend_masked(o, layer, b, j, q, 1, loc, p);
                float *oj = out + ((size_t)b * o->q_heads + j) * D;
                for (int d = 0; d < D; ++d) oj[d] = (float)(a * full[d] + ((acc_t)1 - a) * loc[d]);
            }
        free(p);
        free(full);
        free(loc);
    }
    return fail ? -4 : 0;
}

/* Copy one head's physical rows out. k_out, v_out: [rows][head_dim] bf16 bits; token_of_slot_out:
 * [rows] (for a full head: t for t < len, -1 above).  Returns the number of rows. */
int rlkv_oracle_export_head(const oracle_t *o, int layer, int b, int h, uint16_t *k_out,
                            uint16_t *v_out, int32_t *token_of_slot_out)
{
    size_t u = unit_index(o, layer, b, h);
    int rows = head_rows(o, layer, h), D = o->head_dim;
    memcpy(k_out, o->k[u], (size_t)rows * D * sizeof(uint16_t));
    memcpy(v_out, o->v[u], (size_t)rows * D * sizeof(uint16_t));
    for (int s = 0; s < rows; ++s)
        token_of_slot_out[s] = o->token_of_slot[u] ? o->token_of_slot[u][s]
                                                   : (s < o->len[layer] ? s : -1);
    return rows;
}

int rlkv_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Lethe hot-path ORACLE — test infrastructure, not product code.
 *
 * A plain, slow, scalar CPU statement of what the decode loop of Lethe computes
 * on its KV cache, written from the paper's equations.  It exists so that tests
 * can compare the CUDA library against it; it shares no source with that
 * library and nothing on the product path may call it.
 *
 * What is here, and the passage each function follows:
 *   oracle_decode_attend      Sec. 4.1 (cache grows one token per step), the
 *                             softmax attention implied by Sec. 4.2 ("raw
 *                             attention tensor"), Eq. 3 (grouped heads share a
 *                             key without expanding it) and Eq. 5 (the decayed
 *                             relevance recurrence of RASR, Sec. 4.3).
 *   oracle_estimate_sparsity  Eq. 1 (Hoyer sparsity, Sec. 3.1) applied to the
 *                             accumulated relevance vector of each KV head and
 *                             averaged over the KV heads of a layer (Sec. 4.2).
 *   oracle_alloc_budgets      Sec. 4.2, first paragraph: budgets follow measured
 *                             sparsity (sparse layers need fewer tokens, dense
 *                             layers more).  The paper prints no formula; this is
 *                             the proportional-to-density, largest-remainder rule
 *                             the build adopts.  PARITY UNPINNED against the
 *                             paper for the formula itself; pinned by invariants
 *                             and by exact-rational recomputation.
 *   oracle_rasr_prune         Sec. 4.3 last paragraph + Algorithm 1 (top-k by
 *                             score, sinks and the recent window always kept),
 *                             multi-round carry-over of Sec. 4.4.
 *   oracle_prefill_seed       Eq. 2 with Q > 1 (token importance from the prefill
 *                             attention) folded through the recurrence of Eq. 5:
 *                             the relevance the prompt tokens would have had if the
 *                             prompt had been fed one token at a time.
 *   oracle_segment_prune      Algorithm 1 as a whole (segmented breakpoint search
 *                             of Sec. 4.2 / Eq. 4, retention set, eviction-threshold
 *                             update) with the size trigger of Sec. 4.1, applied per
 *                             (sequence, KV head).  Eq. 4 is read as
 *                             v_head >= tau * v_cut (as printed, v_head / v_cut <= tau
 *                             with tau > 1 could only fire at the first cut or never).
 *   oracle_collapsed_prune    Eq. 2 as printed: ONE score per token per layer, the relevance
 *                             summed over all heads (and, in the wider scope, over the
 *                             batch), and one retention set shared by everything summed
 *                             over; same protected top-k and compaction as oracle_rasr_prune.
 *
 * K and V may also be stored quantised (e4m3 bytes with one scale per layer): the paper's
 * related-work section notes that quantised caches compose with eviction; it defines no
 * format, so the format is this build's choice (stated at oracle_decode_attend).
 *
 * Arithmetic: every floating-point step is done in double; stored results are
 * rounded once to their storage type (fp32, or bf16 round-to-nearest-even).
 * Integer steps (budgets, selection, compaction) have exactly one right answer.
 *
 * Layouts (all row-major, caller-owned):
 *   contiguous: K, V  [L][B][Hkv][cap][D]
 *   paged:      K, V  pools [n_pages][page_tokens][D]; page_table [L][B][Hkv][cap_pages]
 *   rel fp32, pos int32: [L][B][Hkv][cap_tokens] by logical slot
 *   len int32: [L][B][Hkv]
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_OK = 0, ORACLE_ERR_INVALID_ARG = 1, ORACLE_ERR_CAPACITY = 2, ORACLE_ERR_BUDGET = 3 };
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_FP8 = 2, ORACLE_FP8_E5M2 = 3 };
#define ORACLE_IS_FP8(dt) ((dt) == ORACLE_FP8 || (dt) == ORACLE_FP8_E5M2)

typedef struct {
    int32_t n_layers, batch, n_q_heads, n_kv_heads, head_dim;
    int32_t dtype;       /* storage type of K and V: ORACLE_F32, ORACLE_BF16 (held as uint16), ORACLE_FP8 (e4m3fn
                            bytes) or ORACLE_FP8_E5M2 (e5m2 bytes); with bytes, q, k_new, v_new, out are bf16 */
    int32_t paged;       /* 0 contiguous, 1 paged */
    int32_t capacity;    /* contiguous: token slots per item; paged: pages per item */
    int32_t page_tokens; /* tokens per page when paged, else ignored */
    void *k, *v;
    float *rel;
    int32_t *pos;
    int32_t *len;
    int32_t *page_table;
    int64_t n_pages;
    const float *k_scale; /* ORACLE_FP8 only, [n_layers] or NULL (= 1): a stored key byte x means k_scale[l] * x */
    const float *v_scale; /* the same for values */
} oracle_cache;

static int g_threads = 1;

void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }

int oracle_get_threads(void) {
#ifdef _OPENMP
    return g_threads;
#else
    return 1;
#endif
}

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_num_procs();
#else
    return 1;
#endif
}

/* ---- storage-type helpers ------------------------------------------------ */

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* double -> float (one IEEE rounding) -> bf16, round to nearest, ties to even. */
static uint16_t double_to_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* e4m3fn (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; S.1111.111 is NaN; largest
 * finite value 448; subnormals are multiples of 2^-9). */
static double e4m3_to_double(uint8_t b) {
    const int e = (b >> 3) & 15, m = b & 7;
    double x;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) x = ldexp((double)m, -9);
    else x = ldexp(1.0 + (double)m / 8.0, e - 7);
    return (b & 0x80) ? -x : x;
}

/* float -> e4m3fn: round to nearest, ties to even; magnitudes beyond the largest finite value saturate to it
 * (the conversion a quantised cache uses: no value becomes NaN by overflow). */
static uint8_t float_to_e4m3(float f) {
    if (f != f) return 0x7f;
    const uint8_t sign = signbit(f) ? 0x80 : 0x00;
    const float a = fabsf(f);
    if (a > 448.0f) return sign | 0x7e;
    if (a < 0.015625f) return sign | (uint8_t)rintf(a * 512.0f); /* subnormal step 2^-9; 8 is the smallest normal */
    int ex;
    const float fr = frexpf(a, &ex);                  /* a = fr * 2^ex, fr in [0.5, 1) */
    int q = (int)rintf((2.0f * fr - 1.0f) * 8.0f);    /* mantissa in eighths, 0..8 (rintf: ties to even) */
    int e = ex - 1 + 7;
    if (q == 8) {
        q = 0;
        e += 1;
    }
    const int code = (e << 3) | q;
    return sign | (uint8_t)(code > 0x7e ? 0x7e : code);
}

/* e5m2 (1 sign, 5 exponent bits with bias 15, 2 mantissa bits: the upper byte of an IEEE half).  Largest finite
 * value 57344; subnormals are multiples of 2^-16.  Exponent 31 (infinity, NaN) never occurs in a cache: the
 * encoder saturates. */
static double e5m2_to_double(uint8_t b) {
    const int e = (b >> 2) & 31, m = b & 3;
    double x;
    if (e == 31) return m ? NAN : INFINITY * ((b & 0x80) ? -1.0 : 1.0);
    if (e == 0) x = ldexp((double)m, -16);
    else x = ldexp(1.0 + (double)m / 4.0, e - 15);
    return (b & 0x80) ? -x : x;
}

/* float -> e5m2: round to nearest, ties to even; magnitudes beyond the largest finite value saturate to it. */
static uint8_t float_to_e5m2(float f) {
    if (f != f) return 0x7f;
    const uint8_t sign = signbit(f) ? 0x80 : 0x00;
    const float a = fabsf(f);
    if (a > 57344.0f) return sign | 0x7b;
    if (a < 6.103515625e-05f) return sign | (uint8_t)rintf(a * 65536.0f); /* below 2^-14: step 2^-16; 4 is the smallest normal */
    int ex;
    const float fr = frexpf(a, &ex);
    int q = (int)rintf((2.0f * fr - 1.0f) * 4.0f); /* mantissa in quarters, 0..4 */
    int e = ex - 1 + 15;
    if (q == 4) {
        q = 0;
        e += 1;
    }
    const int code = (e << 2) | q;
    return sign | (uint8_t)(code > 0x7b ? 0x7b : code);
}

static double load_elt(const void *base, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) return bf16_to_double(((const uint16_t *)base)[idx]);
    if (dtype == ORACLE_FP8) return e4m3_to_double(((const uint8_t *)base)[idx]);
    if (dtype == ORACLE_FP8_E5M2) return e5m2_to_double(((const uint8_t *)base)[idx]);
    return (double)((const float *)base)[idx];
}

static void store_elt(void *base, int dtype, int64_t idx, double x) {
    if (dtype == ORACLE_BF16) ((uint16_t *)base)[idx] = double_to_bf16(x);
    else ((float *)base)[idx] = (float)x;
}

static size_t elt_size(int dtype) { return dtype == ORACLE_BF16 ? 2 : (ORACLE_IS_FP8(dtype) ? 1 : 4); }

/* type of q, k_new, v_new and out: the cache's own, except that a quantised cache takes bf16 activations */
static int act_dtype(int dtype) { return ORACLE_IS_FP8(dtype) ? ORACLE_BF16 : dtype; }

/* test hooks for the two conversions */
double oracle_e4m3_decode(uint8_t b) { return e4m3_to_double(b); }
uint8_t oracle_e4m3_encode(float f) { return float_to_e4m3(f); }
double oracle_e5m2_decode(uint8_t b) { return e5m2_to_double(b); }
uint8_t oracle_e5m2_encode(float f) { return float_to_e5m2(f); }

static int64_t cap_tokens(const oracle_cache *c) {
    return c->paged ? (int64_t)c->capacity * c->page_tokens : (int64_t)c->capacity;
}

/* item = (layer, sequence, kv head) flattened */
static int64_t item_index(const oracle_cache *c, int l, int b, int h) {
    return ((int64_t)l * c->batch + b) * c->n_kv_heads + h;
}

/* element offset of row `slot` of an item inside K (or V) */
static int64_t row_offset(const oracle_cache *c, int64_t item, int64_t slot) {
    if (!c->paged) return (item * c->capacity + slot) * c->head_dim;
    int64_t page = c->page_table[item * c->capacity + slot / c->page_tokens];
    return (page * c->page_tokens + slot % c->page_tokens) * c->head_dim;
}

static int check_cache(const oracle_cache *c) {
    if (!c || !c->k || !c->v || !c->rel || !c->pos || !c->len) return ORACLE_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->batch < 1 || c->n_kv_heads < 1 || c->head_dim < 1) return ORACLE_ERR_INVALID_ARG;
    if (c->n_q_heads < c->n_kv_heads || c->n_q_heads % c->n_kv_heads) return ORACLE_ERR_INVALID_ARG;
    if (c->dtype != ORACLE_F32 && c->dtype != ORACLE_BF16 && !ORACLE_IS_FP8(c->dtype)) return ORACLE_ERR_INVALID_ARG;
    if (c->capacity < 1) return ORACLE_ERR_INVALID_ARG;
    if (c->paged && (!c->page_table || c->page_tokens < 1)) return ORACLE_ERR_INVALID_ARG;
    return ORACLE_OK;
}

/* ---- decode step: append, attend, relevance (Sec. 4.1, Eq. 3, Eq. 5) ------ */
/*
 * For layers [layer_begin, layer_end), with li = layer - layer_begin:
 *   q, out        [layers][B][Hq][D]   (cache dtype; bf16 when the cache is ORACLE_FP8)
 *   k_new, v_new  [layers][B][Hkv][D]  (same type as q) or both NULL = attend only
 * A quantised (ORACLE_FP8, ORACLE_FP8_E5M2) cache holds K / k_scale[l] and V / v_scale[l] as e4m3fn or e5m2 bytes: an appended row is
 * divided by the layer's scale in fp32 (one IEEE division) and rounded to nearest-even with saturation; when
 * read, a byte x counts as scale * x exactly.  Quantisation composes with pruning (Sec. 2, related work on
 * quantised caches): rows are moved as bytes, scores never see the storage type.
 *   token_pos     [B] original position written to pos[] for the appended token
 *   scale         [n_layers] softmax scale of each layer (indexed by absolute layer)
 *   lse           optional [layers][B][Hq]   log-sum-exp of the scaled logits
 *   probs         optional [layers][B][Hq][cap_tokens] doubles: the softmax row
 *                 (test hook: lets a test check that rows sum to one)
 * Returns ORACLE_ERR_CAPACITY if any item is full when a token must be appended
 * (nothing is changed in that case).
 */
int oracle_decode_attend(oracle_cache *c, int layer_begin, int layer_end, const void *q, const void *k_new,
                         const void *v_new, const int32_t *token_pos, const float *scale, float gamma, void *out,
                         float *lse, double *probs) {
    int st = check_cache(c);
    if (st) return st;
    if (!q || !out || !scale) return ORACLE_ERR_INVALID_ARG;
    if (layer_begin < 0 || layer_end > c->n_layers || layer_begin >= layer_end) return ORACLE_ERR_INVALID_ARG;
    if ((k_new == NULL) != (v_new == NULL)) return ORACLE_ERR_INVALID_ARG;
    if (k_new && !token_pos) return ORACLE_ERR_INVALID_ARG;
    if (!(gamma > 0.0f && gamma <= 1.0f)) return ORACLE_ERR_INVALID_ARG;

    const int B = c->batch, Hq = c->n_q_heads, Hkv = c->n_kv_heads, D = c->head_dim;
    const int G = Hq / Hkv;
    const int64_t capT = cap_tokens(c);
    const int n_items = (layer_end - layer_begin) * B * Hkv;

    if (k_new) {
        for (int l = layer_begin; l < layer_end; ++l)
            for (int b = 0; b < B; ++b)
                for (int h = 0; h < Hkv; ++h)
                    if (c->len[item_index(c, l, b, h)] >= capT) return ORACLE_ERR_CAPACITY;
    }

#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 1)
#endif
    for (int w = 0; w < n_items; ++w) {
        const int li = w / (B * Hkv);
        const int l = layer_begin + li;
        const int b = (w / Hkv) % B;
        const int hkv = w % Hkv;
        const int64_t item = item_index(c, l, b, hkv);
        int64_t n = c->len[item];
        const int act = act_dtype(c->dtype);
        const float ks = (ORACLE_IS_FP8(c->dtype) && c->k_scale) ? c->k_scale[l] : 1.0f;
        const float vs = (ORACLE_IS_FP8(c->dtype) && c->v_scale) ? c->v_scale[l] : 1.0f;

        /* Sec. 4.1: the cache grows by the token just generated.  It enters with
         * zero relevance and takes part in this step's attention. */
        if (k_new) {
            const int64_t src = (((int64_t)li * B + b) * Hkv + hkv) * D;
            const int64_t dst = row_offset(c, item, n);
            if (ORACLE_IS_FP8(c->dtype)) {
                for (int d = 0; d < D; ++d) {
                    const float kx = (float)load_elt(k_new, ORACLE_BF16, src + d), vx = (float)load_elt(v_new, ORACLE_BF16, src + d);
                    ((uint8_t *)c->k)[dst + d] = c->dtype == ORACLE_FP8 ? float_to_e4m3(kx / ks) : float_to_e5m2(kx / ks);
                    ((uint8_t *)c->v)[dst + d] = c->dtype == ORACLE_FP8 ? float_to_e4m3(vx / vs) : float_to_e5m2(vx / vs);
                }
            } else {
                memcpy((char *)c->k + dst * elt_size(c->dtype), (const char *)k_new + src * elt_size(c->dtype),
                       D * elt_size(c->dtype));
                memcpy((char *)c->v + dst * elt_size(c->dtype), (const char *)v_new + src * elt_size(c->dtype),
                       D * elt_size(c->dtype));
            }
            c->rel[item * capT + n] = 0.0f;
            c->pos[item * capT + n] = token_pos[b];
            n += 1;
            c->len[item] = (int32_t)n;
        }

        double *mass = (double *)calloc((size_t)(n > 0 ? n : 1), sizeof(double)); /* sum over the group's heads of p */
        double *p = (double *)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
        double *o = (double *)malloc((size_t)D * sizeof(double));

        /* Eq. 3: the G query heads hkv*G .. hkv*G+G-1 read the same K/V rows. */
        for (int g = 0; g < G; ++g) {
            const int h = hkv * G + g;
            const int64_t qoff = (((int64_t)li * B + b) * Hq + h) * D;
            if (n == 0) {
                for (int d = 0; d < D; ++d) store_elt(out, act, qoff + d, 0.0);
                if (lse) lse[((int64_t)li * B + b) * Hq + h] = -INFINITY;
                continue;
            }
            double m = -INFINITY;
            for (int64_t j = 0; j < n; ++j) {
                const int64_t koff = row_offset(c, item, j);
                double s = 0.0;
                for (int d = 0; d < D; ++d) s += load_elt(q, act, qoff + d) * ((double)ks * load_elt(c->k, c->dtype, koff + d));
                s *= (double)scale[l];
                p[j] = s;
                if (s > m) m = s;
            }
            double Z = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                p[j] = exp(p[j] - m);
                Z += p[j];
            }
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            for (int64_t j = 0; j < n; ++j) {
                p[j] /= Z;
                mass[j] += p[j];
                const int64_t voff = row_offset(c, item, j);
                for (int d = 0; d < D; ++d) o[d] += p[j] * ((double)vs * load_elt(c->v, c->dtype, voff + d));
                if (probs) probs[(((int64_t)li * B + b) * Hq + h) * capT + j] = p[j];
            }
            for (int d = 0; d < D; ++d) store_elt(out, act, qoff + d, o[d]);
            if (lse) lse[((int64_t)li * B + b) * Hq + h] = (float)(m + log(Z));
        }

        /* Eq. 5 at decode (one query): s_t[j] = gamma * s_{t-1}[j] + sum over the
         * group's heads of the attention weight that token j received. */
        for (int64_t j = 0; j < n; ++j) {
            float *r = &c->rel[item * capT + j];
            *r = (float)((double)gamma * (double)(*r) + mass[j]);
        }
        free(mass);
        free(p);
        free(o);
    }
    return ORACLE_OK;
}

/* ---- Eq. 1: Hoyer sparsity of the relevance vector, mean over KV heads ---- */
/* sparsity [L][B] fp32.  A vector of length <= 1 or of zero norm has sparsity 0. */
int oracle_estimate_sparsity(const oracle_cache *c, float *sparsity) {
    int st = check_cache(c);
    if (st) return st;
    if (!sparsity) return ORACLE_ERR_INVALID_ARG;
    const int64_t capT = cap_tokens(c);
    for (int l = 0; l < c->n_layers; ++l)
        for (int b = 0; b < c->batch; ++b) {
            double acc = 0.0;
            for (int h = 0; h < c->n_kv_heads; ++h) {
                const int64_t item = item_index(c, l, b, h);
                const int64_t n = c->len[item];
                double l1 = 0.0, l2sq = 0.0;
                for (int64_t j = 0; j < n; ++j) {
                    const double a = (double)c->rel[item * capT + j];
                    l1 += fabs(a);
                    l2sq += a * a;
                }
                double s = 0.0;
                if (n > 1 && l2sq > 0.0) {
                    const double rn = sqrt((double)n);
                    s = (rn - l1 / sqrt(l2sq)) / (rn - 1.0);
                    if (s < 0.0) s = 0.0;
                    if (s > 1.0) s = 1.0;
                }
                acc += s;
            }
            sparsity[(int64_t)l * c->batch + b] = (float)(acc / (double)c->n_kv_heads);
        }
    return ORACLE_OK;
}

/* ---- layerwise budget allocation (Sec. 4.2; the build's integer rule) ----- */
/*
 * Per sequence b: density weight w_l = max(1, round((1 - S_l) * 2^20)) from one
 * fp32 subtraction and an exact power-of-two scaling; the budget above the floor
 * k_min is split in proportion to w_l with largest-remainder rounding (ties to
 * the lower layer), so that sum_l k_l == total_budget[b] exactly.
 * budgets [L][B] int32.  Returns ORACLE_ERR_BUDGET when total < L * k_min.
 */
int oracle_alloc_budgets(int n_layers, int batch, const float *sparsity, const int64_t *total_budget, int32_t k_min,
                         int32_t *budgets) {
    if (n_layers < 1 || batch < 1 || !sparsity || !total_budget || !budgets || k_min < 0) return ORACLE_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b)
        if (total_budget[b] < (int64_t)n_layers * k_min) return ORACLE_ERR_BUDGET;
    int64_t *w = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_layers);
    int64_t *rem = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_layers);
    int64_t *base = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_layers);
    char *bonus = (char *)malloc((size_t)n_layers);
    for (int b = 0; b < batch; ++b) {
        int64_t W = 0;
        for (int l = 0; l < n_layers; ++l) {
            float s = sparsity[(int64_t)l * batch + b];
            if (!(s >= 0.0f)) s = 0.0f; /* NaN and negatives read as dense */
            if (s > 1.0f) s = 1.0f;
            const float d = 1.0f - s;
            int64_t wl = (int64_t)rintf(d * 1048576.0f);
            if (wl < 1) wl = 1;
            w[l] = wl;
            W += wl;
        }
        const int64_t F = total_budget[b] - (int64_t)n_layers * k_min;
        int64_t given = 0;
        for (int l = 0; l < n_layers; ++l) {
            base[l] = (w[l] * F) / W;
            rem[l] = (w[l] * F) % W;
            given += base[l];
            bonus[l] = 0;
        }
        int64_t R = F - given; /* 0 <= R < L */
        while (R > 0) {
            int best = -1;
            for (int l = 0; l < n_layers; ++l)
                if (!bonus[l] && (best < 0 || rem[l] > rem[best])) best = l; /* strict > keeps the lower layer on ties */
            bonus[best] = 1;
            --R;
        }
        for (int l = 0; l < n_layers; ++l)
            budgets[(int64_t)l * batch + b] = (int32_t)((int64_t)k_min + base[l] + bonus[l]);
    }
    free(w);
    free(rem);
    free(base);
    free(bonus);
    return ORACLE_OK;
}

/* ---- RASR retention: protected top-k and stable compaction ---------------- */

typedef struct {
    float score;
    int32_t idx;
} cand_t;

static int cand_cmp(const void *a, const void *b) {
    const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx); /* equal scores: older (lower) slot first */
}

static int int_cmp(const void *a, const void *b) {
    const int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 * For every (layer, sequence, KV head) with n = len tokens and k = budgets[l][b]:
 *   k >= n : nothing changes.
 *   else   : keep the first `sink` slots, the last `recent` slots (Algorithm 1's
 *            sink and recent index sets) and, among the others, the highest
 *            relevance scores (ties to the lower slot) until k are kept; if the
 *            protected slots alone exceed k, exactly they are kept and the call
 *            reports ORACLE_ERR_BUDGET.  Kept rows of K, V, rel and pos move to
 *            slots 0..k'-1 in their old order (Sec. 4.4: later rounds see earlier
 *            survivors plus newer tokens); len becomes k'.
 * keep_idx (optional) [L][B][Hkv][max_k]: old slot of each survivor, ascending,
 * padded with -1; an unpruned item lists 0..n-1 (as many as fit).
 */
int oracle_rasr_prune(oracle_cache *c, const int32_t *budgets, int32_t recent, int32_t sink, int32_t *keep_idx,
                      int32_t max_k) {
    int st = check_cache(c);
    if (st) return st;
    if (!budgets || recent < 0 || sink < 0) return ORACLE_ERR_INVALID_ARG;
    if (keep_idx && max_k < 1) return ORACLE_ERR_INVALID_ARG;
    const int64_t capT = cap_tokens(c);
    const int D = c->head_dim;
    const size_t row_bytes = (size_t)D * elt_size(c->dtype);
    int result = ORACLE_OK;
    const int n_items = c->n_layers * c->batch * c->n_kv_heads;

#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 1)
#endif
    for (int w = 0; w < n_items; ++w) {
        const int l = w / (c->batch * c->n_kv_heads);
        const int b = (w / c->n_kv_heads) % c->batch;
        const int64_t item = w;
        const int64_t n = c->len[item];
        int64_t k = budgets[(int64_t)l * c->batch + b];
        if (k < 0) k = 0;
        int32_t *kout = keep_idx ? keep_idx + item * max_k : NULL;
        if (kout)
            for (int i = 0; i < max_k; ++i) kout[i] = -1;

        if (k >= n) { /* identity */
            if (kout)
                for (int64_t i = 0; i < n && i < max_k; ++i) kout[i] = (int32_t)i;
            continue;
        }
        const int64_t n_sink = sink < n ? sink : n;
        const int64_t n_recent = recent < n ? recent : n;
        int64_t cand_lo = n_sink, cand_hi = n - n_recent; /* candidates: [cand_lo, cand_hi) */
        if (cand_hi < cand_lo) cand_hi = cand_lo;
        const int64_t n_prot = n - (cand_hi - cand_lo);
        if (n_prot > k) {
            k = n_prot;
#ifdef _OPENMP
#pragma omp critical
#endif
            result = ORACLE_ERR_BUDGET;
        }
        const int64_t take = k - n_prot;

        int32_t *keep = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
        int64_t nk = 0;
        for (int64_t j = 0; j < cand_lo; ++j) keep[nk++] = (int32_t)j;
        for (int64_t j = cand_hi; j < n; ++j) keep[nk++] = (int32_t)j;
        if (take > 0) {
            const int64_t nc = cand_hi - cand_lo;
            cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)nc);
            for (int64_t j = 0; j < nc; ++j) {
                cand[j].score = c->rel[item * capT + cand_lo + j];
                cand[j].idx = (int32_t)(cand_lo + j);
            }
            qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
            for (int64_t i = 0; i < take; ++i) keep[nk++] = cand[i].idx;
            free(cand);
        }
        qsort(keep, (size_t)nk, sizeof(int32_t), int_cmp);

        /* stable in-place gather: destination i <= source keep[i], ascending */
        for (int64_t i = 0; i < nk; ++i) {
            const int64_t s = keep[i];
            if (kout && i < max_k) kout[i] = (int32_t)s;
            if (s == i) continue;
            const int64_t so = row_offset(c, item, s), d_o = row_offset(c, item, i);
            memmove((char *)c->k + d_o * elt_size(c->dtype), (char *)c->k + so * elt_size(c->dtype), row_bytes);
            memmove((char *)c->v + d_o * elt_size(c->dtype), (char *)c->v + so * elt_size(c->dtype), row_bytes);
            c->rel[item * capT + i] = c->rel[item * capT + s];
            c->pos[item * capT + i] = c->pos[item * capT + s];
        }
        c->len[item] = (int32_t)nk;
        free(keep);
    }
    return result;
}

/* ---- Algorithm 1: segmented breakpoint, retention set, eviction threshold ---- */
/*
 * For every (layer, sequence, KV head) with n = len tokens and threshold Le = l_evict[item]:
 *   n <= Le : not triggered (Sec. 4.1): nothing changes.
 *   else    : sort the scores (descending, equal scores: lower slot first); cut points
 *             c_d = floor(n d / D), d = 1..D-1; the breakpoint is the first c_d with
 *             top[0] >= tau * top[c_d] (one fp32 multiply, fp32 compare);
 *             found    : keep the first `sink` slots, the last `recent` slots and the
 *                        breakpoint highest-scoring slots; compact as oracle_rasr_prune
 *                        does; Le <- max(Le, breakpoint + recent);
 *             not found: keep everything ("conservatively delay pruning");
 *                        Le <- min(2 Le, 2^30).
 * l_evict [L][B][Hkv] int32 is read and updated in place.  keep_idx as in oracle_rasr_prune.
 */
int oracle_segment_prune(oracle_cache *c, int32_t n_segments, float tau, int32_t recent, int32_t sink,
                         int32_t *l_evict, int32_t *keep_idx, int32_t max_k) {
    int st = check_cache(c);
    if (st) return st;
    if (!l_evict || n_segments < 2 || !(tau >= 1.0f) || recent < 0 || sink < 0) return ORACLE_ERR_INVALID_ARG;
    if (keep_idx && max_k < 1) return ORACLE_ERR_INVALID_ARG;
    const int64_t capT = cap_tokens(c);
    const size_t row_bytes = (size_t)c->head_dim * elt_size(c->dtype);
    const int n_items = c->n_layers * c->batch * c->n_kv_heads;
    for (int w = 0; w < n_items; ++w) {
        const int64_t item = w;
        const int64_t n = c->len[item];
        const int64_t Le = l_evict[item];
        int32_t *kout = keep_idx ? keep_idx + item * max_k : NULL;
        if (kout)
            for (int i = 0; i < max_k; ++i) kout[i] = (i < n) ? i : -1;
        if (n <= Le) continue; /* not triggered */

        cand_t *top = (cand_t *)malloc(sizeof(cand_t) * (size_t)n);
        for (int64_t j = 0; j < n; ++j) {
            top[j].score = c->rel[item * capT + j];
            top[j].idx = (int32_t)j;
        }
        qsort(top, (size_t)n, sizeof(cand_t), cand_cmp);
        int64_t breakpoint = -1;
        for (int d = 1; d < n_segments; ++d) {
            const int64_t cut = (n * d) / n_segments;
            if (cut >= n) break;
            const float v_head = top[0].score, v_cut = top[cut].score;
            const float rhs = tau * v_cut; /* one IEEE fp32 multiply (no contraction: built with -ffp-contract=off) */
            if (v_head >= rhs) {
                breakpoint = cut;
                break;
            }
        }
        if (breakpoint < 0) { /* no sharp drop: delay pruning */
            int64_t twice = 2 * Le;
            if (twice > (1 << 30)) twice = (1 << 30);
            l_evict[item] = (int32_t)twice;
            free(top);
            continue;
        }
        char *keep = (char *)calloc((size_t)n, 1);
        for (int64_t j = 0; j < sink && j < n; ++j) keep[j] = 1;
        for (int64_t j = (n - recent > 0 ? n - recent : 0); j < n; ++j) keep[j] = 1;
        for (int64_t i = 0; i < breakpoint; ++i) keep[top[i].idx] = 1;
        int64_t m = 0;
        for (int64_t s = 0; s < n; ++s) {
            if (!keep[s]) continue;
            if (kout && m < max_k) kout[m] = (int32_t)s;
            if (s != m) {
                const int64_t so = row_offset(c, item, s), d_o = row_offset(c, item, m);
                memmove((char *)c->k + d_o * elt_size(c->dtype), (char *)c->k + so * elt_size(c->dtype), row_bytes);
                memmove((char *)c->v + d_o * elt_size(c->dtype), (char *)c->v + so * elt_size(c->dtype), row_bytes);
                c->rel[item * capT + m] = c->rel[item * capT + s];
                c->pos[item * capT + m] = c->pos[item * capT + s];
            }
            ++m;
        }
        if (kout)
            for (int64_t i = m; i < max_k; ++i) kout[i] = -1;
        c->len[item] = (int32_t)m;
        const int64_t grown = breakpoint + recent;
        l_evict[item] = (int32_t)(grown > Le ? grown : Le);
        free(keep);
        free(top);
    }
    return ORACLE_OK;
}

/* ---- Eq. 2 as printed: one collapsed score, one retention set per group ---- */
/*
 * scope 0: a group is the Hkv items of one (layer, sequence); budgets [L][B].
 * scope 1: a group is the B * Hkv items of one layer (Eq. 2 also sums over b); budgets [L].
 * Slot j must mean the same token in every item of a group, so all of them must have the same
 * len (true when they were only ever appended to and pruned together); a group that breaks this
 * is left untouched and the call reports ORACLE_ERR_INVALID_ARG.
 *   score[j] = sum over the group's items, in ascending (b, h) order, of rel[item][j]
 * The sum decides an integer result (who is kept), so it is taken in fp32 — the precision rel is
 * stored in — one rounded add per item.  With k = the group's budget: k >= n keeps everything;
 * otherwise sinks, the recent window and the highest scores among the rest (ties to the lower
 * slot) are kept exactly as in oracle_rasr_prune, and the same slot list compacts every item of
 * the group (each keeps its own K, V, rel and pos rows).
 * keep_idx (optional) [groups][max_k]: the survivors' old slots, ascending, padded with -1.
 */
int oracle_collapsed_prune(oracle_cache *c, const int32_t *budgets, int32_t recent, int32_t sink, int32_t scope,
                           int32_t *keep_idx, int32_t max_k) {
    int st = check_cache(c);
    if (st) return st;
    if (!budgets || recent < 0 || sink < 0 || (scope != 0 && scope != 1)) return ORACLE_ERR_INVALID_ARG;
    if (keep_idx && max_k < 1) return ORACLE_ERR_INVALID_ARG;
    const int64_t capT = cap_tokens(c);
    const size_t row_bytes = (size_t)c->head_dim * elt_size(c->dtype);
    const int per_group = scope == 0 ? c->n_kv_heads : c->batch * c->n_kv_heads;
    const int n_groups = scope == 0 ? c->n_layers * c->batch : c->n_layers;
    int result = ORACLE_OK;
    for (int g = 0; g < n_groups; ++g) {
        const int64_t first = (int64_t)g * per_group; /* items of a group are consecutive in [L][B][Hkv] order */
        const int64_t n = c->len[first];
        int32_t *kout = keep_idx ? keep_idx + (int64_t)g * max_k : NULL;
        if (kout)
            for (int i = 0; i < max_k; ++i) kout[i] = -1;
        int aligned = 1;
        for (int t = 1; t < per_group; ++t)
            if (c->len[first + t] != n) aligned = 0;
        if (!aligned) {
            if (result == ORACLE_OK) result = ORACLE_ERR_INVALID_ARG;
            continue;
        }
        int64_t k = budgets[g];
        if (k < 0) k = 0;
        if (k >= n) {
            if (kout)
                for (int64_t i = 0; i < n && i < max_k; ++i) kout[i] = (int32_t)i;
            continue;
        }
        const int64_t n_sink = sink < n ? sink : n;
        const int64_t n_recent = recent < n ? recent : n;
        int64_t cand_lo = n_sink, cand_hi = n - n_recent;
        if (cand_hi < cand_lo) cand_hi = cand_lo;
        const int64_t n_prot = n - (cand_hi - cand_lo);
        if (n_prot > k) {
            k = n_prot;
            if (result == ORACLE_OK) result = ORACLE_ERR_BUDGET;
        }
        const int64_t take = k - n_prot;

        char *keep = (char *)calloc((size_t)(n > 0 ? n : 1), 1);
        for (int64_t j = 0; j < cand_lo; ++j) keep[j] = 1;
        for (int64_t j = cand_hi; j < n; ++j) keep[j] = 1;
        if (take > 0) {
            const int64_t nc = cand_hi - cand_lo;
            cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)nc);
            for (int64_t j = 0; j < nc; ++j) {
                float score = 0.0f;
                for (int t = 0; t < per_group; ++t) score = score + c->rel[(first + t) * capT + cand_lo + j];
                cand[j].score = score;
                cand[j].idx = (int32_t)(cand_lo + j);
            }
            qsort(cand, (size_t)nc, sizeof(cand_t), cand_cmp);
            for (int64_t i = 0; i < take; ++i) keep[cand[i].idx] = 1;
            free(cand);
        }
        for (int t = 0; t < per_group; ++t) {
            const int64_t item = first + t;
            int64_t m = 0;
            for (int64_t s = 0; s < n; ++s) {
                if (!keep[s]) continue;
                if (t == 0 && kout && m < max_k) kout[m] = (int32_t)s;
                if (s != m) {
                    const int64_t so = row_offset(c, item, s), d_o = row_offset(c, item, m);
                    memmove((char *)c->k + d_o * elt_size(c->dtype), (char *)c->k + so * elt_size(c->dtype), row_bytes);
                    memmove((char *)c->v + d_o * elt_size(c->dtype), (char *)c->v + so * elt_size(c->dtype), row_bytes);
                    c->rel[item * capT + m] = c->rel[item * capT + s];
                    c->pos[item * capT + m] = c->pos[item * capT + s];
                }
                ++m;
            }
            c->len[item] = (int32_t)m;
        }
        free(keep);
    }
    return result;
}

/* ---- relevance of the prompt from the prefill attention (Eq. 2, Q > 1; Eq. 5) ---- */
/*
 * q_prompt [L][B][P][Hq][D] (cache dtype): the queries of the P prompt tokens; their keys are slots 0..P-1 of
 * every item (len >= P required).  With causal attention rows
 *   A_h(i, j) = softmax over j <= i of scale_l * q_{i,h} . K_j        (i, j < P)
 * Eq. 5 run over the prompt positions as steps gives, for every slot j < P,
 *   rel[j] = sum_{i = j}^{P-1} gamma^(P-1-i) * sum_{h in group} A_h(i, j).
 * rel[0..P) is overwritten; nothing else changes.
 */
int oracle_prefill_seed(oracle_cache *c, const void *q_prompt, int32_t prompt_len, const float *scale, float gamma) {
    int st = check_cache(c);
    if (st) return st;
    if (!q_prompt || !scale || prompt_len < 1 || !(gamma > 0.0f && gamma <= 1.0f)) return ORACLE_ERR_INVALID_ARG;
    if (ORACLE_IS_FP8(c->dtype)) return ORACLE_ERR_INVALID_ARG; /* prompt keys are seeded before quantisation */
    const int B = c->batch, Hq = c->n_q_heads, Hkv = c->n_kv_heads, D = c->head_dim, P = prompt_len;
    const int G = Hq / Hkv;
    const int64_t capT = cap_tokens(c);
    const int n_items = c->n_layers * B * Hkv;
    for (int w = 0; w < n_items; ++w)
        if (c->len[w] < P) return ORACLE_ERR_CAPACITY;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(dynamic, 1)
#endif
    for (int w = 0; w < n_items; ++w) {
        const int l = w / (B * Hkv), b = (w / Hkv) % B, hkv = w % Hkv;
        const int64_t item = w;
        double *acc = (double *)calloc((size_t)P, sizeof(double));
        double *p = (double *)malloc((size_t)P * sizeof(double));
        for (int i = 0; i < P; ++i) {
            const double wgt = pow((double)gamma, (double)(P - 1 - i));
            for (int g = 0; g < G; ++g) {
                const int h = hkv * G + g;
                const int64_t qoff = ((((int64_t)l * B + b) * P + i) * Hq + h) * D;
                double m = -INFINITY;
                for (int j = 0; j <= i; ++j) {
                    const int64_t koff = row_offset(c, item, j);
                    double s = 0.0;
                    for (int d = 0; d < D; ++d) s += load_elt(q_prompt, c->dtype, qoff + d) * load_elt(c->k, c->dtype, koff + d);
                    s *= (double)scale[l];
                    p[j] = s;
                    if (s > m) m = s;
                }
                double Z = 0.0;
                for (int j = 0; j <= i; ++j) {
                    p[j] = exp(p[j] - m);
                    Z += p[j];
                }
                for (int j = 0; j <= i; ++j) acc[j] += wgt * p[j] / Z;
            }
        }
        for (int j = 0; j < P; ++j) c->rel[item * capT + j] = (float)acc[j];
        free(acc);
        free(p);
    }
    return ORACLE_OK;
}

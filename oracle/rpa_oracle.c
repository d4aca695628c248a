/*
 * Ragged paged attention -- fp64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA path is compared
 * against.  It is plain, slow and written straight from the definition; it is
 * not a fallback and the product never calls it.  It shares no code, header,
 * table or helper with the CUDA sources.
 *
 * What it computes (the paper's problem statement, Sections 2.4 and 3, and
 * Algorithm 1's result):
 *
 *   step 1 (cache update, Algorithm 1 "Update U_kv"; Section 3.4): for every
 *     sequence r and every new token i in [0, q_r), the projected K and V rows
 *     of that token are copied bit for bit into the paged cache slot of
 *     absolute position  pos = L_r - q_r + i  (L_r counts cached plus new
 *     tokens, Section 4.1.1).  The cache is the merged, head-interleaved KV
 *     tensor of Section 3.1.3: one token slot holds K and V of every KV head;
 *     combined head 2h is K of head h, 2h+1 is V of head h.
 *
 *   step 2 (attention, Algorithm 1 inner loop and its final diag(l)^-1
 *     normalisation): for every query token and query head a, with KV head
 *     h = a / h_g (grouped heads are contiguous, Section 3.1.2),
 *         s_t = scale * <q, K_t>           for t = 0 .. hi
 *         out = sum_t softmax(s)_t * V_t
 *     where hi = pos under the causal mask and L_r - 1 without it.  Algorithm 1
 *     reaches this value through the online (m, l) recurrences; the result has
 *     the plain closed form above, so the oracle is that closed form as a
 *     two-pass softmax in double precision.  K_t and V_t are read back from the
 *     updated cache through the page table, so step 2 also checks step 1.
 *
 * Quantised cache (Section 3.8, per-tensor quantisation: one scalar scale per tensor).  With
 * kv_fp8 set, a cache element is one FP8 E4M3 byte and stands for byte_value * k_scale (K) or
 * byte_value * v_scale (V).  Step 1 then stores  e4m3(float(new) * (1.0f / scale))  -- one fp32
 * multiply by the fp32 reciprocal, round to nearest even, saturating at +-448 -- and step 2 reads
 * every key and value, the batch's own new tokens included, back from the cache, i.e. in
 * quantised precision (Algorithm 1 composes its KV block in the cache's type and writes that same
 * block back).  The paper does not spell out the conversion; this is the reading taken.
 * Section 3.8 gives Q a scalar scale of its own as well: with q_scale > 0 (FP8 cache only) every
 * query element is taken in E4M3 precision too, as  e4m3(float(q) * (1.0f / q_scale)) * q_scale  --
 * the same conversion as for K -- before the scores are formed; q_scale = 0 leaves Q in bf16.
 *
 * Layouts (row-major): q [T, h_q, d], new_k/new_v [T, h_kv, d],
 * kv_cache [num_pages, page_size, 2*h_kv, d], all bf16 bit patterns in
 * uint16_t; page_table [num_seqs, max_pages_per_seq] int32; cu_q_lens
 * [num_seqs+1]; kv_lens [num_seqs]; out [T, h_q, d] double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;
    int32_t page_size;
    int32_t num_pages;
    int32_t max_pages_per_seq;
    int32_t causal;
    double scale;
    int32_t kv_fp8; /* 0: bf16 cache, 1: FP8 E4M3 cache with per-tensor scales */
    float k_scale;
    float v_scale;
    float q_scale; /* > 0: Q is quantised to E4M3 with this per-tensor scale (FP8 cache only); 0: Q stays bf16 */
} oracle_shape_t;

static double bf16_to_double(uint16_t bits) {
    uint32_t w = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* value of an FP8 E4M3 ("fn": no infinities, 0x7F/0xFF are NaN) byte */
double rpa_oracle_e4m3_to_double(uint8_t code) {
    int sign = code >> 7, ex = (code >> 3) & 15, man = code & 7;
    double v;
    if (ex == 15 && man == 7) return NAN;
    if (ex == 0)
        v = ldexp((double)man, -9); /* subnormal: man * 2^-6 / 8 */
    else
        v = ldexp(1.0 + man / 8.0, ex - 7);
    return sign ? -v : v;
}

/* fp32 -> FP8 E4M3, round to nearest even, saturating to the largest finite value (448) */
uint8_t rpa_oracle_float_to_e4m3(float x) {
    if (isnan(x)) return 0x7F;
    uint8_t sign = signbit(x) ? 0x80 : 0;
    double a = fabs((double)x);
    if (a > 448.0) return sign | 0x7E; /* everything above the largest finite value saturates */
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e); /* a = m * 2^e, m in [0.5, 1) -> floor(log2 a) = e - 1 */
    int ex = e - 1;
    if (ex < -6) ex = -6;                   /* subnormals share the quantum of the smallest normal binade */
    double quantum = ldexp(1.0, ex - 3);    /* 3 mantissa bits */
    double q = nearbyint(a / quantum);      /* ties to even (default rounding mode) */
    double v = q * quantum;
    if (v > 448.0) return sign | 0x7E;
    if (v < ldexp(1.0, -6)) return sign | (uint8_t)q; /* subnormal (or zero): exponent field 0 */
    (void)frexp(v, &e);
    ex = e - 1; /* rounding may have carried into the next binade */
    int man = (int)(v / ldexp(1.0, ex - 3)) - 8;
    return sign | (uint8_t)(((ex + 7) << 3) | man);
}

/* address (in elements) of combined head ch of the slot holding position pos of sequence r */
static int64_t slot_offset(const oracle_shape_t *sh, const int32_t *page_table, int r, int64_t pos, int ch) {
    int64_t page = page_table[(int64_t)r * sh->max_pages_per_seq + pos / sh->page_size];
    int64_t slot = pos % sh->page_size;
    return ((page * sh->page_size + slot) * (2 * sh->num_kv_heads) + ch) * (int64_t)sh->head_dim;
}

int rpa_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* returns 0, or a negative code naming the first malformed length / page id found */
int rpa_oracle_check(const oracle_shape_t *sh, const int32_t *page_table, const int32_t *cu_q_lens,
                     const int32_t *kv_lens, int num_seqs) {
    if (sh->num_kv_heads <= 0 || sh->num_q_heads % sh->num_kv_heads != 0) return -1;
    if (sh->kv_fp8 && !(sh->k_scale > 0.f && sh->v_scale > 0.f)) return -8;
    if (!(sh->q_scale >= 0.f) || (sh->q_scale > 0.f && !sh->kv_fp8)) return -9;
    if (cu_q_lens[0] != 0) return -2;
    for (int r = 0; r < num_seqs; ++r) {
        int q_r = cu_q_lens[r + 1] - cu_q_lens[r];
        int L_r = kv_lens[r];
        if (q_r < 0 || L_r < q_r) return -3;
        int pages = (L_r + sh->page_size - 1) / sh->page_size;
        if (pages > sh->max_pages_per_seq) return -4;
        for (int p = 0; p < pages; ++p) {
            int32_t id = page_table[(int64_t)r * sh->max_pages_per_seq + p];
            if (id < 0 || id >= sh->num_pages) return -5;
        }
    }
    return 0;
}

/* step 1: bit copy of the new K/V rows into their cache slots */
int rpa_oracle_update_cache(const oracle_shape_t *sh, const uint16_t *new_k, const uint16_t *new_v,
                            uint16_t *kv_cache, const int32_t *page_table, const int32_t *cu_q_lens,
                            const int32_t *kv_lens, int num_seqs) {
    int rc = rpa_oracle_check(sh, page_table, cu_q_lens, kv_lens, num_seqs);
    if (rc) return rc;
    const int d = sh->head_dim, h_kv = sh->num_kv_heads;
    for (int r = 0; r < num_seqs; ++r) {
        int q_r = cu_q_lens[r + 1] - cu_q_lens[r];
        int L_r = kv_lens[r];
        for (int i = 0; i < q_r; ++i) {
            int64_t pos = (int64_t)L_r - q_r + i;
            int64_t tok = (int64_t)cu_q_lens[r] + i;
            for (int h = 0; h < h_kv; ++h) {
                const uint16_t *src_k = new_k + (tok * h_kv + h) * d;
                const uint16_t *src_v = new_v + (tok * h_kv + h) * d;
                if (sh->kv_fp8) {
                    uint8_t *c8 = (uint8_t *)kv_cache;
                    const float inv_k = 1.0f / sh->k_scale, inv_v = 1.0f / sh->v_scale;
                    int64_t ok_ = slot_offset(sh, page_table, r, pos, 2 * h);
                    int64_t ov_ = slot_offset(sh, page_table, r, pos, 2 * h + 1);
                    for (int e = 0; e < d; ++e) {
                        c8[ok_ + e] = rpa_oracle_float_to_e4m3((float)bf16_to_double(src_k[e]) * inv_k);
                        c8[ov_ + e] = rpa_oracle_float_to_e4m3((float)bf16_to_double(src_v[e]) * inv_v);
                    }
                } else {
                    memcpy(kv_cache + slot_offset(sh, page_table, r, pos, 2 * h), src_k, (size_t)d * 2);
                    memcpy(kv_cache + slot_offset(sh, page_table, r, pos, 2 * h + 1), src_v, (size_t)d * 2);
                }
            }
        }
    }
    return 0;
}

/* step 2 for one (sequence r, new token i, query head a); out_row has d doubles */
static void attend_one(const oracle_shape_t *sh, const uint16_t *q, const uint16_t *kv_cache,
                       const int32_t *page_table, const int32_t *cu_q_lens, const int32_t *kv_lens, int r,
                       int i, int a, double *score, double *out_row) {
    const int d = sh->head_dim;
    const int h_g = sh->num_q_heads / sh->num_kv_heads;
    const int h = a / h_g;
    const int q_r = cu_q_lens[r + 1] - cu_q_lens[r];
    const int L_r = kv_lens[r];
    const int64_t pos = (int64_t)L_r - q_r + i;
    const int64_t hi = sh->causal ? pos : (int64_t)L_r - 1; /* last visible key position */
    const uint16_t *q_row = q + (((int64_t)cu_q_lens[r] + i) * sh->num_q_heads + a) * d;

    const uint8_t *cache8 = (const uint8_t *)kv_cache;
    /* the query row as the scores see it: bf16, or its E4M3 image under the per-tensor scale of Q */
    double *q_val = (double *)malloc(sizeof(double) * (size_t)d);
    for (int e = 0; e < d; ++e) {
        q_val[e] = bf16_to_double(q_row[e]);
        if (sh->q_scale > 0.f) {
            const float inv_q = 1.0f / sh->q_scale;
            q_val[e] = rpa_oracle_e4m3_to_double(rpa_oracle_float_to_e4m3((float)q_val[e] * inv_q)) * (double)sh->q_scale;
        }
    }
    double M = -INFINITY;
    for (int64_t t = 0; t <= hi; ++t) {
        const int64_t k_off = slot_offset(sh, page_table, r, t, 2 * h);
        double dot = 0.0;
        for (int e = 0; e < d; ++e) {
            double k_val = sh->kv_fp8 ? rpa_oracle_e4m3_to_double(cache8[k_off + e]) * (double)sh->k_scale
                                      : bf16_to_double(kv_cache[k_off + e]);
            dot += q_val[e] * k_val;
        }
        score[t] = sh->scale * dot;
        if (score[t] > M) M = score[t];
    }
    double Z = 0.0;
    for (int e = 0; e < d; ++e) out_row[e] = 0.0;
    for (int64_t t = 0; t <= hi; ++t) {
        double w = exp(score[t] - M);
        Z += w;
        const int64_t v_off = slot_offset(sh, page_table, r, t, 2 * h + 1);
        for (int e = 0; e < d; ++e) {
            double v_val = sh->kv_fp8 ? rpa_oracle_e4m3_to_double(cache8[v_off + e]) * (double)sh->v_scale
                                      : bf16_to_double(kv_cache[v_off + e]);
            out_row[e] += w * v_val;
        }
    }
    for (int e = 0; e < d; ++e) out_row[e] /= Z;
    free(q_val);
}

/*
 * step 2 on a list of (sequence, token-in-sequence, query head) triples, reading an ALREADY
 * UPDATED cache.  out has n_rows * d doubles, row k for triple k.
 */
int rpa_oracle_attend_rows(const oracle_shape_t *sh, const uint16_t *q, const uint16_t *kv_cache,
                           const int32_t *page_table, const int32_t *cu_q_lens, const int32_t *kv_lens,
                           int num_seqs, const int32_t *rows, int64_t n_rows, double *out) {
    int rc = rpa_oracle_check(sh, page_table, cu_q_lens, kv_lens, num_seqs);
    if (rc) return rc;
    int max_L = 1;
    for (int r = 0; r < num_seqs; ++r)
        if (kv_lens[r] > max_L) max_L = kv_lens[r];
    for (int64_t k = 0; k < n_rows; ++k) {
        int r = rows[3 * k], i = rows[3 * k + 1], a = rows[3 * k + 2];
        if (r < 0 || r >= num_seqs || a < 0 || a >= sh->num_q_heads) return -6;
        if (i < 0 || i >= cu_q_lens[r + 1] - cu_q_lens[r]) return -6;
    }
    int failed = 0;
#pragma omp parallel
    {
        double *score = (double *)malloc(sizeof(double) * (size_t)max_L);
        if (!score) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t k = 0; k < n_rows; ++k) {
            if (score)
                attend_one(sh, q, kv_cache, page_table, cu_q_lens, kv_lens, rows[3 * k], rows[3 * k + 1],
                           rows[3 * k + 2], score, out + k * sh->head_dim);
        }
        free(score);
    }
    return failed ? -7 : 0;
}

/* the whole call: step 1, then step 2 for every (token, query head); out is [T, h_q, d] doubles */
int rpa_oracle_forward(const oracle_shape_t *sh, const uint16_t *q, const uint16_t *new_k,
                       const uint16_t *new_v, uint16_t *kv_cache, const int32_t *page_table,
                       const int32_t *cu_q_lens, const int32_t *kv_lens, int num_seqs, double *out) {
    int rc = rpa_oracle_update_cache(sh, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens, num_seqs);
    if (rc) return rc;
    int64_t T = cu_q_lens[num_seqs];
    int64_t n_rows = T * sh->num_q_heads;
    int32_t *rows = (int32_t *)malloc(sizeof(int32_t) * 3 * (size_t)(n_rows > 0 ? n_rows : 1));
    if (!rows) return -7;
    int64_t k = 0;
    for (int r = 0; r < num_seqs; ++r)
        for (int i = 0; i < cu_q_lens[r + 1] - cu_q_lens[r]; ++i)
            for (int a = 0; a < sh->num_q_heads; ++a) {
                rows[3 * k] = r;
                rows[3 * k + 1] = i;
                rows[3 * k + 2] = a;
                ++k;
            }
    /* rows are emitted in (token, head) order, so row k lands at out[k*d] = out[tok][a][:] */
    rc = rpa_oracle_attend_rows(sh, q, kv_cache, page_table, cu_q_lens, kv_lens, num_seqs, rows, n_rows, out);
    free(rows);
    return rc;
}

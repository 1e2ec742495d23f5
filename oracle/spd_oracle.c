/*
 * CPU oracle for partitioned decode attention -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain, slow, float64.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call this; the CUDA library shares no code with it.
 *
 * What it computes, per user u and query head h (kv head = h / (Hq/Hkv)):
 *   full        : Y = softmax(scale * q K^T) V over the private tokens followed by the public
 *                 tokens -- the left-hand side of Theorem 1 (Eq. 1), softmax as in Sec. 2.1.
 *   partial     : m = max_i s_i, l = sum_i exp(s_i - m), O = sum_i exp(s_i - m) v_i over ONE
 *                 partition -- the max-stabilised denominators of Sec. 4.2 and the
 *                 unnormalised numerator that goes with them.
 *   merge       : combine two partials into Y (Theorem 1 with both sides brought to the
 *                 common maximum), plus the alpha-form coefficients of Sec. 4.2 as a second
 *                 derivation, plus an n-way merge (Theorem 1 applied repeatedly).
 * Keys and values are fetched through the page tables:
 *   token t of user u -> pool[page_indices[page_indptr[u] + t / P]][kvh][t % P][:].
 * Inputs are the exact fp32 or bf16 bit patterns the GPU sees, widened to double.
 *
 * Every function here is pinned by tests/test_oracle_pins.py (brute force on tiny inputs,
 * the split-point identity of Theorem 1, closed forms, a textbook dense softmax).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };

typedef struct {
    const void    *k_pool;       /* [num_pages][Hkv][P][D] */
    const void    *v_pool;
    int64_t        num_pages;
    const int32_t *page_indptr;  /* [B+1] */
    const int32_t *page_indices;
    const int32_t *seq_lens;     /* [B] */
} oracle_kv;

typedef struct {
    int32_t batch, num_q_heads, num_kv_heads, head_dim, page_size, dtype;
    double  sm_scale;
} oracle_shape;

static double widen(const void *base, int64_t idx, int dtype)
{
    if (dtype == ORACLE_F32) {
        return (double)((const float *)base)[idx];
    } else {
        /* bfloat16 = the upper 16 bits of an IEEE binary32 */
        uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
}

/* element offset of row (token t of user u, kv head kvh) in a pool */
static int64_t row_offset(const oracle_shape *s, const oracle_kv *kv, int u, int kvh, int64_t t)
{
    int64_t P = s->page_size, D = s->head_dim;
    int64_t page = kv->page_indices[(int64_t)kv->page_indptr[u] + t / P];
    return ((page * s->num_kv_heads + kvh) * P + t % P) * D;
}

/* scores of one partition for (u, h): s_i = scale * <q, k_i>; returns count */
static int64_t scores(const oracle_shape *s, const void *q, const oracle_kv *kv, int u, int h, double *out)
{
    int D = s->head_dim;
    int kvh = h / (s->num_q_heads / s->num_kv_heads);
    int64_t n = kv ? kv->seq_lens[u] : 0;
    int64_t qoff = ((int64_t)u * s->num_q_heads + h) * D;
    for (int64_t t = 0; t < n; ++t) {
        int64_t ro = row_offset(s, kv, u, kvh, t);
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += widen(q, qoff + d, s->dtype) * widen(kv->k_pool, ro + d, s->dtype);
        out[t] = s->sm_scale * acc;
    }
    return n;
}

int spd_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Unpartitioned attention (left side of Eq. 1): softmax over ALL cached tokens,
 * exp(s - max) / sum as in Sec. 2.1.  y: [B][Hq][D] double.
 * user_lo/user_hi restrict the users computed (others untouched).
 */
void spd_oracle_full(const oracle_shape *s, const void *q, const oracle_kv *priv, const oracle_kv *pub,
                     int user_lo, int user_hi, double *y)
{
    int Hq = s->num_q_heads, D = s->head_dim;
    int g = Hq / s->num_kv_heads;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int u = user_lo; u < user_hi; ++u) {
        for (int h = 0; h < Hq; ++h) {
            int64_t n_in = priv ? priv->seq_lens[u] : 0;
            int64_t n_out = pub ? pub->seq_lens[u] : 0;
            int64_t n = n_in + n_out;
            double *yo = y + ((int64_t)u * Hq + h) * D;
            for (int d = 0; d < D; ++d) yo[d] = 0.0;
            if (n == 0) continue;
            double *sc = (double *)malloc(sizeof(double) * (size_t)n);
            scores(s, q, priv, u, h, sc);
            scores(s, q, pub, u, h, sc + n_in);
            double mx = -INFINITY;
            for (int64_t i = 0; i < n; ++i) if (sc[i] > mx) mx = sc[i];
            double den = 0.0;
            for (int64_t i = 0; i < n; ++i) { sc[i] = exp(sc[i] - mx); den += sc[i]; }
            int kvh = h / g;
            for (int64_t i = 0; i < n; ++i) {
                const oracle_kv *kv = i < n_in ? priv : pub;
                int64_t t = i < n_in ? i : i - n_in;
                int64_t ro = row_offset(s, kv, u, kvh, t);
                double w = sc[i] / den;
                for (int d = 0; d < D; ++d) yo[d] += w * widen(kv->v_pool, ro + d, s->dtype);
            }
            free(sc);
        }
    }
}

/*
 * Partial attention over tokens [tok_lo, min(tok_hi, len_u)) of ONE partition (Sec. 4.2):
 *   m = max s_i ; l = sum exp(s_i - m) ; O = sum exp(s_i - m) v_i   (unnormalised)
 * An empty range gives m = -inf, l = 0, O = 0.
 * o: [B][Hq][D], m,l: [B][Hq], all double.
 */
void spd_oracle_partial(const oracle_shape *s, const void *q, const oracle_kv *kv,
                        int64_t tok_lo, int64_t tok_hi, double *o, double *m, double *l)
{
    int Hq = s->num_q_heads, D = s->head_dim;
    int g = Hq / s->num_kv_heads;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int u = 0; u < s->batch; ++u) {
        for (int h = 0; h < Hq; ++h) {
            int64_t idx = (int64_t)u * Hq + h;
            double *oo = o + idx * D;
            for (int d = 0; d < D; ++d) oo[d] = 0.0;
            m[idx] = -INFINITY;
            l[idx] = 0.0;
            int64_t len = kv->seq_lens[u];
            int64_t hi = tok_hi < len ? tok_hi : len;
            if (hi <= tok_lo) continue;
            double *sc = (double *)malloc(sizeof(double) * (size_t)len);
            scores(s, q, kv, u, h, sc);
            double mx = -INFINITY;
            for (int64_t t = tok_lo; t < hi; ++t) if (sc[t] > mx) mx = sc[t];
            double den = 0.0;
            int kvh = h / g;
            for (int64_t t = tok_lo; t < hi; ++t) {
                double p = exp(sc[t] - mx);
                den += p;
                int64_t ro = row_offset(s, kv, u, kvh, t);
                for (int d = 0; d < D; ++d) oo[d] += p * widen(kv->v_pool, ro + d, s->dtype);
            }
            m[idx] = mx;
            l[idx] = den;
            free(sc);
        }
    }
}

/*
 * n-way merge of partials (Theorem 1 applied repeatedly, everything brought to the common
 * maximum M): w_c = exp(m_c - M) with exp(-inf) = 0; L = sum w_c l_c; O = sum w_c O_c.
 * parts_o: [n][rows][D]; parts_m, parts_l: [n][rows].  Writes the merged partial
 * (o_out, m_out, l_out) and, if y != NULL, the normalised output y = O / L (0 where L = 0).
 */
void spd_oracle_merge_n(int n, int64_t rows, int D, const double *parts_o, const double *parts_m,
                        const double *parts_l, double *o_out, double *m_out, double *l_out, double *y)
{
    for (int64_t r = 0; r < rows; ++r) {
        double M = -INFINITY;
        for (int c = 0; c < n; ++c) if (parts_m[c * rows + r] > M) M = parts_m[c * rows + r];
        double L = 0.0;
        for (int d = 0; d < D; ++d) o_out[r * D + d] = 0.0;
        for (int c = 0; c < n; ++c) {
            double mc = parts_m[c * rows + r];
            double w = (mc == -INFINITY) ? 0.0 : exp(mc - M);
            L += w * parts_l[c * rows + r];
            for (int d = 0; d < D; ++d) o_out[r * D + d] += w * parts_o[((int64_t)c * rows + r) * D + d];
        }
        m_out[r] = M;
        l_out[r] = L;
        if (y) for (int d = 0; d < D; ++d) y[r * D + d] = L > 0.0 ? o_out[r * D + d] / L : 0.0;
    }
}

/*
 * Two-way merge written with the coefficients the paper prints (Sec. 4.2, after Eq. 1):
 *   A_x = O_x / gamma_x ; alpha = exp(m_out - m_in)
 *   Y = gamma_in / (gamma_in + alpha gamma_out) A_in + gamma_out / (gamma_in / alpha + gamma_out) A_out
 * Both partitions must be non-empty and |m_out - m_in| small enough for exp() in double.
 */
void spd_oracle_merge_alpha(int64_t rows, int D, const double *o_in, const double *m_in, const double *l_in,
                            const double *o_out, const double *m_out, const double *l_out, double *y)
{
    for (int64_t r = 0; r < rows; ++r) {
        double alpha = exp(m_out[r] - m_in[r]);
        double c_in = l_in[r] / (l_in[r] + alpha * l_out[r]);
        double c_out = l_out[r] / (l_in[r] / alpha + l_out[r]);
        for (int d = 0; d < D; ++d)
            y[r * D + d] = c_in * (o_in[r * D + d] / l_in[r]) + c_out * (o_out[r * D + d] / l_out[r]);
    }
}

/*
 * Prefill: causal self-attention over each user's prompt (protocol step 2; Fig. 3 step 0; the causal
 * property of Sec. 2.1: token i attends to tokens 0..i of its own prompt).  q: [T][Hq][D], k, v:
 * [T][Hkv][D], dense, users laid end to end; tok_indptr[B+1] are token offsets.  Computes the rows
 * listed in `rows` (global token indices, n_rows of them): y[r][h][:] for r-th listed row.
 */
void spd_oracle_prefill(const oracle_shape *s, const void *q, const void *k, const void *v,
                        const int32_t *tok_indptr, const int64_t *rows, int64_t n_rows, double *y)
{
    int Hq = s->num_q_heads, Hkv = s->num_kv_heads, D = s->head_dim;
    int g = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t r = 0; r < n_rows; ++r) {
        for (int h = 0; h < Hq; ++h) {
            int64_t i = rows[r];
            int u = 0;
            while (u + 1 < s->batch && tok_indptr[u + 1] <= i) ++u;
            int64_t first = tok_indptr[u], n = i - first + 1;       /* keys first..i */
            int kvh = h / g;
            double *yo = y + (r * Hq + h) * D;
            for (int d = 0; d < D; ++d) yo[d] = 0.0;
            double *sc = (double *)malloc(sizeof(double) * (size_t)n);
            double mx = -INFINITY;
            for (int64_t j = 0; j < n; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d)
                    acc += widen(q, (i * Hq + h) * D + d, s->dtype) * widen(k, ((first + j) * Hkv + kvh) * D + d, s->dtype);
                sc[j] = s->sm_scale * acc;
                if (sc[j] > mx) mx = sc[j];
            }
            double den = 0.0;
            for (int64_t j = 0; j < n; ++j) { sc[j] = exp(sc[j] - mx); den += sc[j]; }
            for (int64_t j = 0; j < n; ++j)
                for (int d = 0; d < D; ++d)
                    yo[d] += sc[j] / den * widen(v, ((first + j) * Hkv + kvh) * D + d, s->dtype);
            free(sc);
        }
    }
}

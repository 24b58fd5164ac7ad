/*
 * fp64 CPU oracle for the Cross-Loop-Parallel (CLP) decode-step attention of
 * the Parallel Loop Transformer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  Nothing in the product package may import,
 * link or call it; it shares no code, header or table with the CUDA sources.
 *
 * What it computes, for every sequence b, loop l (1-indexed) and query head h
 * (Algorithm 3, Eq. 2, and the CLP description of Sec. 2.2.1):
 *
 *   cut      = max(0, N_b - delta_l)                      delta_l = l-1 by default
 *   y_global = softmax(sm_scale * q . K_share[0:cut]) V_share[0:cut]   (Alg. 3, global)
 *   l == 1 :  O = y_global                               (first loop = vanilla attention)
 *   l >= 2 :  wl = win_lens ? win_lens[b,l-2] : min(w, cut)
 *             y_local = softmax(sm_scale * q . K_win[0:wl]) V_win[0:wl] (Alg. 3, local)
 *             g = 1 / (1 + exp(-gate_logit))              (Alg. 3, gate)  
 *             O = g * y_local + (1 - g) * y_global        (Alg. 3 / Eq. 2)
 *   cut == 0:  O = 0 (the loop has no token to serve yet)
 *   wl  == 0 with cut > 0:  y_local = 0
 *
 * The two softmaxes are normalised separately (Eq. 2 mixes finished outputs).
 * GQA: query head h reads KV head h / (Hq / Hkv) (contiguous groups; a
 * convention the paper does not state: parity unpinned by the paper, pinned
 * here only against that convention).
 *
 * Softmax is written out as its definition: subtract the maximum score,
 * exponentiate, divide by the sum.  No tiling, no online rescaling, no
 * reordering; every accumulation is a plain left-to-right fp64 loop.
 *
 * Storage types: inputs are float32 or bfloat16 (passed as uint16 bit
 * patterns, widened exactly); all arithmetic and the output are fp64.
 * The caches and windows may instead hold 8-bit E4M3 codes (OCP 8-bit floating
 * point: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities,
 * S.1111.111 is NaN) with one fp32 scale per KV head for K and one for V; the
 * attention is then the same definition applied to the dequantised values
 * code_value * scale, formed in fp64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define PLT_ORACLE_F32 0
#define PLT_ORACLE_BF16 1
#define PLT_ORACLE_E4M3 3

typedef struct {
    int32_t dtype;            /* PLT_ORACLE_F32 or PLT_ORACLE_BF16: type of q, caches, windows */
    int32_t B, L, Hq, Hkv, d; /* batch, loops, query heads, KV heads, head dim */
    int32_t w;                /* window capacity (slots per non-first loop) */
    int32_t page_size;        /* 0: contiguous cache; >0: tokens per page */
    int32_t max_pages;        /* row length of page_table (paged only) */
    int32_t kv_dtype;         /* 0: caches and windows stored like q; PLT_ORACLE_E4M3: 8-bit codes */
    int64_t kv_stride_b;      /* contiguous cache strides in elements */
    int64_t kv_stride_n;      /* contiguous: token stride; paged: token-in-page stride */
    int64_t kv_stride_h;      /* KV-head stride */
    int64_t kv_stride_page;   /* paged: stride between pages */
    double sm_scale;          /* score scale (1/sqrt(d) when the caller follows the default) */
    const void* q;            /* [B, L, Hq, d] */
    const void* k_cache;      /* shared first-loop keys */
    const void* v_cache;      /* shared first-loop values */
    const int32_t* seq_lens;  /* [B]   N_b, current token included */
    const int32_t* page_table;/* [B, max_pages] or NULL */
    const void* k_win;        /* [B, L-1, w, Hkv, d] */
    const void* v_win;        /* [B, L-1, w, Hkv, d] */
    const int32_t* win_lens;  /* [B, L-1] or NULL */
    const float* gate_logits; /* [B, L-1, Hq] pre-sigmoid */
    const int32_t* loop_offset; /* [L] delta_l, or NULL for delta_l = l-1 */
    const float* k_scale;     /* [Hkv] dequantisation scale of K codes, or NULL (= 1) */
    const float* v_scale;     /* [Hkv] dequantisation scale of V codes, or NULL (= 1) */
} plt_oracle_problem;

static double load_elem(const void* base, int64_t idx, int dtype) {
    if (dtype == PLT_ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float*)base)[idx];
}

/* Value of an E4M3 code, from the format's definition. */
double plt_oracle_e4m3_value(uint8_t code) {
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);            /* subnormal: 0.m * 2^(1-bias) */
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* Element of a cache or window: stored like q, or an E4M3 code times the KV head's scale. */
static double load_kv(const plt_oracle_problem* p, const void* base, int64_t idx, const float* scale, int kvh) {
    if (p->kv_dtype == PLT_ORACLE_E4M3)
        return plt_oracle_e4m3_value(((const uint8_t*)base)[idx]) * (scale ? (double)scale[kvh] : 1.0);
    return load_elem(base, idx, p->dtype);
}

/* Element offset of the shared cache row (b, token j, KV head kvh). */
static int64_t shared_row(const plt_oracle_problem* p, int b, int j, int kvh) {
    if (p->page_size > 0) {
        int page = p->page_table[(int64_t)b * p->max_pages + j / p->page_size];
        return (int64_t)page * p->kv_stride_page + (int64_t)(j % p->page_size) * p->kv_stride_n +
               (int64_t)kvh * p->kv_stride_h;
    }
    return (int64_t)b * p->kv_stride_b + (int64_t)j * p->kv_stride_n + (int64_t)kvh * p->kv_stride_h;
}

/* Element offset of the window row (b, loop l>=2, slot j, KV head kvh). */
static int64_t window_row(const plt_oracle_problem* p, int b, int l, int j, int kvh) {
    return ((((int64_t)b * (p->L - 1) + (l - 2)) * p->w + j) * p->Hkv + kvh) * p->d;
}

/*
 * y[0:d] = softmax(scale * q.K[rows]) V[rows] over `n` rows whose element
 * offsets are produced by rowfn.  n == 0 gives y = 0.  `scores` is scratch of n doubles.
 */
typedef int64_t (*rowfn_t)(const plt_oracle_problem*, int, int, int, int);

static void attend(const plt_oracle_problem* p, const double* qv, const void* kbase, const void* vbase,
                   rowfn_t rowfn, int b, int l, int kvh, int n, double* scores, double* y) {
    const int d = p->d;
    for (int c = 0; c < d; ++c) y[c] = 0.0;
    if (n <= 0) return;
    double smax = -INFINITY;
    for (int j = 0; j < n; ++j) {
        int64_t off = rowfn(p, b, l, j, kvh);
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += qv[c] * load_kv(p, kbase, off + c, p->k_scale, kvh);
        s *= p->sm_scale;
        scores[j] = s;
        if (s > smax) smax = s;
    }
    double denom = 0.0;
    for (int j = 0; j < n; ++j) {
        scores[j] = exp(scores[j] - smax);
        denom += scores[j];
    }
    for (int j = 0; j < n; ++j) {
        int64_t off = rowfn(p, b, l, j, kvh);
        double pj = scores[j] / denom;
        for (int c = 0; c < d; ++c) y[c] += pj * load_kv(p, vbase, off + c, p->v_scale, kvh);
    }
}

static int64_t shared_rowfn(const plt_oracle_problem* p, int b, int l, int j, int kvh) {
    (void)l;
    return shared_row(p, b, j, kvh);
}

static int cutoff(const plt_oracle_problem* p, int b, int l) {
    int delta = p->loop_offset ? p->loop_offset[l - 1] : (l - 1);
    int cut = p->seq_lens[b] - delta;
    return cut > 0 ? cut : 0;
}

/* One output row O[b, l, h, 0:d] (l is 1-indexed).  Returns 0, or -1 on allocation failure. */
static int one_row(const plt_oracle_problem* p, int b, int l, int h, double* out) {
    const int d = p->d;
    const int kvh = h / (p->Hq / p->Hkv);
    const int cut = cutoff(p, b, l);
    for (int c = 0; c < d; ++c) out[c] = 0.0;
    if (cut == 0) return 0;

    int wl = 0;
    if (l >= 2) {
        wl = p->win_lens ? p->win_lens[(int64_t)b * (p->L - 1) + (l - 2)] : (p->w < cut ? p->w : cut);
        if (wl < 0) wl = 0;
        if (wl > p->w) wl = p->w;
    }
    int nmax = cut > wl ? cut : wl;
    double* scores = (double*)malloc(sizeof(double) * (size_t)nmax);
    double* qv = (double*)malloc(sizeof(double) * (size_t)d * 3);
    if (!scores || !qv) {
        free(scores);
        free(qv);
        return -1;
    }
    double* yg = qv + d;
    double* yl = qv + 2 * d;
    int64_t qoff = (((int64_t)b * p->L + (l - 1)) * p->Hq + h) * d;
    for (int c = 0; c < d; ++c) qv[c] = load_elem(p->q, qoff + c, p->dtype);

    attend(p, qv, p->k_cache, p->v_cache, shared_rowfn, b, l, kvh, cut, scores, yg);
    if (l == 1) {
        for (int c = 0; c < d; ++c) out[c] = yg[c];
    } else {
        attend(p, qv, p->k_win, p->v_win, window_row, b, l, kvh, wl, scores, yl);
        double x = (double)p->gate_logits[((int64_t)b * (p->L - 1) + (l - 2)) * p->Hq + h];
        double g = 1.0 / (1.0 + exp(-x));
        for (int c = 0; c < d; ++c) out[c] = g * yl[c] + (1.0 - g) * yg[c];
    }
    free(scores);
    free(qv);
    return 0;
}

/*
 * Full output: out[B, L, Hq, d] in fp64.  Rows are independent; the loop over
 * them is the only thing OpenMP touches (when compiled with -fopenmp).
 * Returns 0 on success, 1 on bad arguments, 2 on allocation failure.
 */
int plt_oracle_decode_attn(const plt_oracle_problem* p, double* out) {
    if (!p || !out || p->B < 0 || p->L < 1 || p->Hkv < 1 || p->Hq % p->Hkv != 0 || p->d < 1) return 1;
    const int64_t rows = (int64_t)p->B * p->L * p->Hq;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < rows; ++r) {
        int h = (int)(r % p->Hq);
        int l = (int)((r / p->Hq) % p->L) + 1;
        int b = (int)(r / ((int64_t)p->Hq * p->L));
        if (one_row(p, b, l, h, out + r * p->d) != 0) failed = 1;
    }
    return failed ? 2 : 0;
}

/*
 * Sampled output: rows[i] = (b, l0, h) with l0 = l-1 zero-indexed;
 * out[n_rows, d].  Used where the full problem is too large to finish in seconds.
 */
int plt_oracle_decode_attn_rows(const plt_oracle_problem* p, const int32_t* rows, int64_t n_rows, double* out) {
    if (!p || !out || (!rows && n_rows > 0)) return 1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_rows; ++i) {
        int b = rows[3 * i], l = rows[3 * i + 1] + 1, h = rows[3 * i + 2];
        if (b < 0 || b >= p->B || l < 1 || l > p->L || h < 0 || h >= p->Hq) {
            failed = 1;
            continue;
        }
        if (one_row(p, b, l, h, out + i * p->d) != 0) failed = 1;
    }
    return failed ? 2 : 0;
}

/* Number of threads the row loop will use (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int plt_oracle_threads(void) { return omp_get_max_threads(); }
void plt_oracle_set_threads(int n) { if (n > 0) omp_set_num_threads(n); }
#else
int plt_oracle_threads(void) { return 1; }
void plt_oracle_set_threads(int n) { (void)n; }
#endif

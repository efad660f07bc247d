/*
 * CPU oracle for the APMSqueeze hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the method computes.  It is
 * used by the test-suite, by the smoke check and by the benchmark's CPU
 * baseline leg, and by nothing else; the CUDA library never links, includes
 * or calls it, and the two share no code.
 *
 * What it follows
 *   - Warmup phase: "Original Adam" with bias correction (Section 3.2), run on
 *     the average of the n workers' gradients (distributed Adam, Algorithm 1
 *     line 2).
 *   - Phase switch: the variance v stops being updated after warmup
 *     (Section 3.3, first paragraph); all compression errors start at zero
 *     (Algorithm 1, initialisation); Adam's raw momentum m carries over.
 *   - Compression phase: Section 3.3 steps 1-6 / Algorithm 1 lines 4-11,
 *     equivalently the parameter-server form of Supplement Section A run on
 *     every chunk independently (Supplement A, first sentence).
 *   - Compressor: 1-bit compression of Section 5.1: the sign of every element
 *     plus one scaling factor  |compensated vector| / |sign vector|, so that the
 *     decompressed vector has the magnitude of the compensated one.
 *
 * Readings taken where the paper is silent
 *   - "magnitude" is the l2 norm (the paper's ||.||), so the scale of a chunk of
 *     length L is ||z||_2 / sqrt(L).  A mean-|z| scale is available as a switch.
 *   - sign(0) = +1 (bit 1), so the sign vector always has norm sqrt(L);
 *     -0.0f counts as >= 0; NaN gives bit 0.
 *   - A chunk is `chunk` consecutive elements of the flat vector; the last one
 *     may be shorter and is scaled with its true length.  The paper's layout
 *     (n chunks, chunk k served by worker k) is chunk = d/n.
 *   - The error update is delta <- (m + delta) - C[m + delta] (Section 3.1 and
 *     Supplement A); Algorithm 1 line 7 prints C[m], a slip.
 *   - The compressed-phase denominator is sqrt(v_Tw) + eps with the raw
 *     (not bias-corrected) frozen v; eps plays the role of Adam's constant.
 *   - The average is over all n workers, summed in worker order, divided by n.
 *   - Top-k compression (Section 5.1, second item) keeps "the top k% elements ... sorted by absolute
 *     magnitude": per chunk K = ceil(k L) elements (at least one), equal magnitudes resolved in favour
 *     of the lower index, the others are sent as nothing and decompress to 0.
 *   - The gradient variant (Section 5.3, item 4) is described in one sentence; read as: workers
 *     send C[g_i + delta_i], servers average and recompress as in the method, and every worker
 *     forms m <- b1 m + (1-b1) g^ from the received g^ and updates the model with that m.
 *   - Arithmetic: IEEE binary32, every named operation rounded once, no
 *     contraction other than the fmaf written; sums of squares are accumulated
 *     in binary64 in element order and rounded to binary32 after the sqrt.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py
 * (closed forms, invariants, hand-worked fixtures, library Adam, exact-rational
 * brute force).  The convergence claims of the paper (Theorem 1, the training
 * curves) need its datasets and are not covered: parity unpinned for those.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_COMPRESSOR_ONEBIT = 0, ORACLE_COMPRESSOR_IDENTITY = 1, ORACLE_COMPRESSOR_TOPK = 2 };
enum { ORACLE_SCALE_L2 = 0, ORACLE_SCALE_L1_MEAN = 1 };
/* What the workers compress and send.  MOMENTUM is the method (Section 3.3).  GRADIENT is the
 * "APGSqueeze" variant of Section 5.3 (Implementations and setups, item 4): the error-compensated
 * compression is applied to the gradient g_t instead of the momentum; what comes back from the
 * servers is then a compressed averaged gradient, from which every worker updates the (uncompressed,
 * identical) momentum m <- b1 m + (1-b1) g^ before the model update with the frozen variance. */
enum { ORACLE_VARIANT_MOMENTUM = 0, ORACLE_VARIANT_GRADIENT = 1 };

typedef struct apms_oracle {
    int64_t d;          /* parameters */
    int     n;          /* workers */
    int64_t chunk;      /* compressor block length */
    int64_t C;          /* ceil(d / chunk) */
    int64_t W;          /* ceil(d / 32) sign words */
    float beta1, beta2, eps, lr;
    int   t;            /* Adam steps taken */
    int   frozen;       /* 0 = warmup phase, 1 = compression phase */
    int   compressor;   /* ORACLE_COMPRESSOR_* */
    int   scale_kind;   /* ORACLE_SCALE_* */
    int   variant;      /* ORACLE_VARIANT_* */
    double topk_frac;   /* top-k compressor: fraction of a chunk's elements that is kept */
    uint8_t *sel;       /* top-k: 1 where worker i kept element j last step, n x d */
    uint8_t *selbar;    /* top-k: the same for the server, d */
    int   threads;      /* OpenMP threads over chunks (chunks are independent) */
    float *x, *m, *v;   /* d each */
    float *ebar;        /* server error, d */
    float *e;           /* worker errors, n x d */
    float *s;           /* worker scales, n x C */
    float *Sbar;        /* server scales, C */
    uint32_t *B;        /* worker sign words, n x W */
    uint32_t *Bbar;     /* server sign words, W */
} apms_oracle;

/* ------------------------------------------------------------------ compressor */

/* 1-bit compressor C[z] of Section 5.1 on one chunk z[0..L): sign bits + scale.
 * Bit j of the chunk goes to bit (j mod 32) of word (j div 32), LSB first;
 * 1 means z >= 0.  Unused high bits of the last word are 0. */
void apms_oracle_compress_1bit(const float *z, int64_t L, int scale_kind,
                               uint32_t *bits, float *scale)
{
    double acc = 0.0;
    for (int64_t j = 0; j < L; ++j) {
        if (scale_kind == ORACLE_SCALE_L1_MEAN) acc += fabs((double)z[j]);
        else                                    acc += (double)z[j] * (double)z[j];
    }
    if (scale_kind == ORACLE_SCALE_L1_MEAN) *scale = (float)(acc / (double)L);
    else                                    *scale = (float)sqrt(acc / (double)L);
    for (int64_t w = 0; w < (L + 31) / 32; ++w) bits[w] = 0u;
    for (int64_t j = 0; j < L; ++j)
        if (z[j] >= 0.0f) bits[j / 32] |= (uint32_t)1 << (j % 32);
}

/* Top-k compressor of Section 5.1 on one chunk: keep the K elements of largest absolute value,
 * send nothing for the others (they decompress to 0).  Equal magnitudes: the lower index wins,
 * so that the choice is unique.  Magnitudes are compared through the bit pattern of |z| (for
 * finite values the same order; a NaN ranks above everything).  q receives C[z]; sel (may be
 * NULL) the 0/1 mask of the kept elements. */
typedef struct { uint32_t key; int64_t idx; } topk_item;
static int topk_cmp(const void *a, const void *b)
{
    const topk_item *x = (const topk_item *)a, *y = (const topk_item *)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;      /* larger magnitude first */
    return x->idx < y->idx ? -1 : (x->idx > y->idx ? 1 : 0);    /* then lower index       */
}
void apms_oracle_compress_topk(const float *z, int64_t L, int64_t K, float *q, uint8_t *sel)
{
    topk_item *items = (topk_item *)malloc((size_t)L * sizeof *items);
    for (int64_t j = 0; j < L; ++j) {
        uint32_t bits;
        memcpy(&bits, &z[j], sizeof bits);
        items[j].key = bits & 0x7fffffffu;
        items[j].idx = j;
    }
    qsort(items, (size_t)L, sizeof *items, topk_cmp);
    for (int64_t j = 0; j < L; ++j) { q[j] = 0.0f; if (sel) sel[j] = 0; }
    for (int64_t r = 0; r < K && r < L; ++r) { q[items[r].idx] = z[items[r].idx]; if (sel) sel[items[r].idx] = 1; }
    free(items);
}

/* "top k% elements" of a chunk of L elements: K = ceil(frac * L), at least 1, at most L. */
int64_t apms_oracle_topk_count(double frac, int64_t L)
{
    int64_t K = (int64_t)ceil(frac * (double)L);
    if (K < 1) K = 1;
    if (K > L) K = L;
    return K;
}

/* Decompression: scale * sign vector. */
void apms_oracle_decompress_1bit(const uint32_t *bits, float scale, int64_t L, float *q)
{
    for (int64_t j = 0; j < L; ++j)
        q[j] = ((bits[j / 32] >> (j % 32)) & 1u) ? scale : -scale;
}

/* ------------------------------------------------------------------ lifetime */

apms_oracle *apms_oracle_create(int64_t d, int n, float beta1, float beta2, float eps,
                                float lr, int64_t chunk)
{
    if (d < 1 || n < 1 || chunk < 32 || chunk % 32 != 0) return NULL;
    apms_oracle *o = (apms_oracle *)calloc(1, sizeof *o);
    if (!o) return NULL;
    o->d = d; o->n = n; o->chunk = chunk;
    o->C = (d + chunk - 1) / chunk;
    o->W = (d + 31) / 32;
    o->beta1 = beta1; o->beta2 = beta2; o->eps = eps; o->lr = lr;
    o->threads = 1;
    o->x = (float *)calloc((size_t)d, sizeof(float));
    o->m = (float *)calloc((size_t)d, sizeof(float));
    o->v = (float *)calloc((size_t)d, sizeof(float));
    o->ebar = (float *)calloc((size_t)d, sizeof(float));
    o->e = (float *)calloc((size_t)d * (size_t)n, sizeof(float));
    o->s = (float *)calloc((size_t)o->C * (size_t)n, sizeof(float));
    o->Sbar = (float *)calloc((size_t)o->C, sizeof(float));
    o->B = (uint32_t *)calloc((size_t)o->W * (size_t)n, sizeof(uint32_t));
    o->Bbar = (uint32_t *)calloc((size_t)o->W, sizeof(uint32_t));
    o->sel = (uint8_t *)calloc((size_t)d * (size_t)n, 1);
    o->selbar = (uint8_t *)calloc((size_t)d, 1);
    o->topk_frac = 0.01;
    return o;
}

void apms_oracle_destroy(apms_oracle *o)
{
    if (!o) return;
    free(o->x); free(o->m); free(o->v); free(o->ebar); free(o->e);
    free(o->s); free(o->Sbar); free(o->B); free(o->Bbar); free(o->sel); free(o->selbar); free(o);
}

void apms_oracle_set_params(apms_oracle *o, const float *x0)
{
    memcpy(o->x, x0, (size_t)o->d * sizeof(float));
    memset(o->m, 0, (size_t)o->d * sizeof(float));
    memset(o->v, 0, (size_t)o->d * sizeof(float));
    o->t = 0; o->frozen = 0;
}

void apms_oracle_set_lr(apms_oracle *o, float lr) { o->lr = lr; }
void apms_oracle_set_compressor(apms_oracle *o, int c) { o->compressor = c; }
void apms_oracle_set_scale_kind(apms_oracle *o, int k) { o->scale_kind = k; }
void apms_oracle_set_variant(apms_oracle *o, int v) { o->variant = v; }
void apms_oracle_set_topk_fraction(apms_oracle *o, double f) { o->topk_frac = f; }
uint8_t *apms_oracle_worker_selected(apms_oracle *o, int i) { return o->sel + (size_t)i * (size_t)o->d; }
uint8_t *apms_oracle_server_selected(apms_oracle *o) { return o->selbar; }
void apms_oracle_set_threads(apms_oracle *o, int t) { o->threads = t < 1 ? 1 : t; }
int  apms_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

float *apms_oracle_x(apms_oracle *o) { return o->x; }
float *apms_oracle_m(apms_oracle *o) { return o->m; }
float *apms_oracle_v(apms_oracle *o) { return o->v; }
float *apms_oracle_server_err(apms_oracle *o) { return o->ebar; }
float *apms_oracle_worker_err(apms_oracle *o, int i) { return o->e + (size_t)i * (size_t)o->d; }
float *apms_oracle_worker_scales(apms_oracle *o, int i) { return o->s + (size_t)i * (size_t)o->C; }
float *apms_oracle_server_scales(apms_oracle *o) { return o->Sbar; }
uint32_t *apms_oracle_worker_bits(apms_oracle *o, int i) { return o->B + (size_t)i * (size_t)o->W; }
uint32_t *apms_oracle_server_bits(apms_oracle *o) { return o->Bbar; }
int apms_oracle_t(const apms_oracle *o) { return o->t; }
int apms_oracle_frozen(const apms_oracle *o) { return o->frozen; }

/* ------------------------------------------------------------------ warmup: Adam, Section 3.2 */

int apms_oracle_warmup_step(apms_oracle *o, const float *const *g)
{
    if (o->frozen) return 2;
    o->t += 1;
    const float omb1 = 1.0f - o->beta1, omb2 = 1.0f - o->beta2;
    const float bc1 = (float)(1.0 - pow((double)o->beta1, (double)o->t));   /* 1 - beta1^t */
    const float bc2 = (float)(1.0 - pow((double)o->beta2, (double)o->t));   /* 1 - beta2^t */
    for (int64_t j = 0; j < o->d; ++j) {
        float gs = 0.0f;
        for (int i = 0; i < o->n; ++i) gs += g[i][j];
        const float gbar = gs / (float)o->n;                 /* averaged stochastic gradient */
        o->m[j] = fmaf(o->beta1, o->m[j], omb1 * gbar);      /* m <- b1 m + (1-b1) g   */
        o->v[j] = fmaf(o->beta2, o->v[j], omb2 * (gbar * gbar)); /* v <- b2 v + (1-b2) g^2 */
        const float mhat = o->m[j] / bc1;
        const float vhat = o->v[j] / bc2;
        o->x[j] = o->x[j] - (o->lr * mhat) / (sqrtf(vhat) + o->eps);
    }
    return 0;
}

/* End of warmup: v is frozen from here on; every compression error starts at 0. */
int apms_oracle_freeze_v(apms_oracle *o)
{
    if (o->frozen) return 2;
    o->frozen = 1;
    memset(o->ebar, 0, (size_t)o->d * sizeof(float));
    memset(o->e, 0, (size_t)o->d * (size_t)o->n * sizeof(float));
    memset(o->s, 0, (size_t)o->C * (size_t)o->n * sizeof(float));
    memset(o->Sbar, 0, (size_t)o->C * sizeof(float));
    memset(o->B, 0, (size_t)o->W * (size_t)o->n * sizeof(uint32_t));
    memset(o->Bbar, 0, (size_t)o->W * sizeof(uint32_t));
    return 0;
}

/* ------------------------------------------------------------------ compression phase, one chunk */

static void compressed_step_chunk(apms_oracle *o, const float *const *g, int64_t c)
{
    const int64_t lo = c * o->chunk;
    const int64_t hi = (lo + o->chunk < o->d) ? lo + o->chunk : o->d;
    const int64_t L = hi - lo;
    const int n = o->n;
    const float omb1 = 1.0f - o->beta1;
    float *z  = (float *)malloc((size_t)L * sizeof(float));             /* compensated vector      */
    float *q  = (float *)malloc((size_t)L * (size_t)n * sizeof(float)); /* what the server receives */
    float *qb = (float *)malloc((size_t)L * sizeof(float));             /* what the workers receive */

    /* Steps 1-3 on every worker i: local momentum, error-compensated compression, send. */
    for (int i = 0; i < n; ++i) {
        float *e = o->e + (size_t)i * (size_t)o->d + lo;
        float *qi = q + (size_t)i * (size_t)L;
        for (int64_t j = 0; j < L; ++j) {
            const float mi = (o->variant == ORACLE_VARIANT_GRADIENT)
                                 ? g[i][lo + j]                                      /* the gradient itself is sent */
                                 : fmaf(o->beta1, o->m[lo + j], omb1 * g[i][lo + j]);
            z[j] = mi + e[j];
        }
        if (o->compressor == ORACLE_COMPRESSOR_IDENTITY) {
            memcpy(qi, z, (size_t)L * sizeof(float));
        } else if (o->compressor == ORACLE_COMPRESSOR_TOPK) {
            apms_oracle_compress_topk(z, L, apms_oracle_topk_count(o->topk_frac, L), qi,
                                      o->sel + (size_t)i * (size_t)o->d + lo);
        } else {
            uint32_t *bits = o->B + (size_t)i * (size_t)o->W + lo / 32;
            float *scale = o->s + (size_t)i * (size_t)o->C + c;
            apms_oracle_compress_1bit(z, L, o->scale_kind, bits, scale);
            apms_oracle_decompress_1bit(bits, *scale, L, qi);
        }
        for (int64_t j = 0; j < L; ++j) e[j] = z[j] - qi[j];
    }

    /* Step 4 on the chunk's server: average what arrived, add the server error, recompress. */
    for (int64_t j = 0; j < L; ++j) {
        float acc = 0.0f;
        for (int i = 0; i < n; ++i) acc += q[(size_t)i * (size_t)L + j];
        z[j] = acc / (float)n + o->ebar[lo + j];
    }
    if (o->compressor == ORACLE_COMPRESSOR_IDENTITY) {
        memcpy(qb, z, (size_t)L * sizeof(float));
    } else if (o->compressor == ORACLE_COMPRESSOR_TOPK) {
        apms_oracle_compress_topk(z, L, apms_oracle_topk_count(o->topk_frac, L), qb, o->selbar + lo);
    } else {
        apms_oracle_compress_1bit(z, L, o->scale_kind, o->Bbar + lo / 32, o->Sbar + c);
        apms_oracle_decompress_1bit(o->Bbar + lo / 32, o->Sbar[c], L, qb);
    }
    for (int64_t j = 0; j < L; ++j) o->ebar[lo + j] = z[j] - qb[j];

    /* Steps 5-6 on every worker (all identical): the received chunk replaces the
     * momentum (gradient variant: it is the gradient the momentum is updated with);
     * model update preconditioned by the frozen variance. */
    for (int64_t j = 0; j < L; ++j) {
        if (o->variant == ORACLE_VARIANT_GRADIENT) o->m[lo + j] = fmaf(o->beta1, o->m[lo + j], omb1 * qb[j]);
        else                                       o->m[lo + j] = qb[j];
        o->x[lo + j] = o->x[lo + j] - (o->lr * o->m[lo + j]) / (sqrtf(o->v[lo + j]) + o->eps);
    }
    free(z); free(q); free(qb);
}

int apms_oracle_compressed_step(apms_oracle *o, const float *const *g)
{
    if (!o->frozen) return 2;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(o->threads)
#endif
    for (int64_t c = 0; c < o->C; ++c) compressed_step_chunk(o, g, c);
    return 0;
}

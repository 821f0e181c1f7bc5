/*
 * Float64 CPU oracle for the SparQ decode attention step, in plain C.
 *
 * TEST INFRASTRUCTURE ONLY: the same algorithm as oracle/sparq_oracle.py, step by step in
 * the paper's order (arXiv 2312.04985, Section 4, Steps 1-3; Eqs. (7)-(10)), for the sizes
 * where the numpy version is too slow and for the timed CPU baseline.  It shares no code
 * with the CUDA library.  Only tests, the smoke check and the benchmark's CPU-baseline leg
 * may load it.  Parallelism is over independent (batch, head) units only; inside a unit the
 * loops are sequential and in the paper's order.
 *
 * Inputs are fp16 bit patterns (uint16_t) widened exactly to double here.
 * Layouts: q [B,Hq,d]; K,V [B,Hkv,S_max,d]; seq_lens [B]; query head h reads KV head h/g.
 * Readings where the paper is silent: ties to the smaller index; selection on the
 * approximate logits; k clipped to n; all-zero q gives tau = 1.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o liboracle.so sparq_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double half_to_double(uint16_t h) {
    int sign = (h >> 15) & 1, e = (h >> 10) & 31, m = h & 1023;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return sign ? -v : v;
}

typedef struct { double v; int32_t i; } item_t;

/* descending by value, equal values by ascending index */
static int cmp_desc(const void* a, const void* b) {
    const item_t* x = (const item_t*)a; const item_t* y = (const item_t*)b;
    if (x->v > y->v) return -1;
    if (x->v < y->v) return 1;
    return (x->i > y->i) - (x->i < y->i);
}
static int cmp_int(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}
static double rel_gap(double a, double b) {
    double m = fmax(fmax(fabs(a), fabs(b)), 1e-300);
    return fabs(a - b) / m;
}

/* One (b, h) unit.  Kh, Vh point at the KV head's [S_max, d] fp16 slab.
 * vbar_in may be NULL: then v_bar is the double mean of the n valid rows of V. */
static void sparq_unit(const uint16_t* qh, const uint16_t* Kh, const uint16_t* Vh, const double* vbar_in,
                       int n, int d, int r, int k, double* out, int32_t* i1, int32_t* i2,
                       double* alpha_out, double* gap_r, double* gap_k) {
    double* q = (double*)malloc(sizeof(double) * d);
    item_t* qa = (item_t*)malloc(sizeof(item_t) * d);
    item_t* lh = (item_t*)malloc(sizeof(item_t) * (n > 0 ? n : 1));
    double* vbar = (double*)malloc(sizeof(double) * d);
    int k_eff = k < n ? k : n;
    if (k_eff < 0) k_eff = 0;

    /* Step 1: the r largest |q_j| */
    double l1_all = 0.0, l1_sel = 0.0;
    for (int j = 0; j < d; ++j) { q[j] = half_to_double(qh[j]); qa[j].v = fabs(q[j]); qa[j].i = j; l1_all += qa[j].v; }
    qsort(qa, d, sizeof(item_t), cmp_desc);
    *gap_r = (r == d) ? INFINITY : rel_gap(qa[r - 1].v, qa[r].v);
    for (int j = 0; j < r; ++j) i1[j] = qa[j].i;
    qsort(i1, r, sizeof(int32_t), cmp_int);
    for (int j = 0; j < r; ++j) l1_sel += fabs(q[i1[j]]);
    /* Eq. (9) */
    double tau = (l1_all == 0.0) ? 1.0 : sqrt((double)d * l1_sel / l1_all);

    /* Eq. (7): approximate logits over the r gathered components */
    double lmax = -INFINITY;
    for (int t = 0; t < n; ++t) {
        double acc = 0.0;
        for (int j = 0; j < r; ++j) acc += q[i1[j]] * half_to_double(Kh[(size_t)t * d + i1[j]]);
        lh[t].v = acc / tau; lh[t].i = t;
        if (lh[t].v > lmax) lmax = lh[t].v;
    }
    double Z = 0.0;
    for (int t = 0; t < n; ++t) Z += exp(lh[t].v - lmax);

    /* mean value vector */
    if (vbar_in) memcpy(vbar, vbar_in, sizeof(double) * d);
    else {
        for (int c = 0; c < d; ++c) vbar[c] = 0.0;
        for (int t = 0; t < n; ++t) for (int c = 0; c < d; ++c) vbar[c] += half_to_double(Vh[(size_t)t * d + c]);
        for (int c = 0; c < d; ++c) vbar[c] /= (double)n;
    }

    for (int j = 0; j < k; ++j) i2[j] = -1;
    if (k_eff == 0) {
        *alpha_out = 0.0; *gap_k = INFINITY;
        for (int c = 0; c < d; ++c) out[c] = vbar[c];
    } else {
        /* Step 2: top-k positions of the approximate scores; Step 3: their mass alpha */
        qsort(lh, n, sizeof(item_t), cmp_desc);
        *gap_k = (k_eff == n) ? INFINITY : rel_gap(lh[k_eff - 1].v, lh[k_eff].v);
        double a = 0.0;
        for (int j = 0; j < k_eff; ++j) { a += exp(lh[j].v - lmax) / Z; i2[j] = lh[j].i; }
        qsort(i2, k_eff, sizeof(int32_t), cmp_int);
        *alpha_out = a;
        /* Eq. (8): exact attention over the selected positions */
        double* z = (double*)malloc(sizeof(double) * k_eff);
        double zmax = -INFINITY, zs = 0.0;
        for (int j = 0; j < k_eff; ++j) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += q[c] * half_to_double(Kh[(size_t)i2[j] * d + c]);
            z[j] = acc / sqrt((double)d);
            if (z[j] > zmax) zmax = z[j];
        }
        for (int j = 0; j < k_eff; ++j) { z[j] = exp(z[j] - zmax); zs += z[j]; }
        for (int c = 0; c < d; ++c) {
            double y = 0.0;
            for (int j = 0; j < k_eff; ++j) y += (z[j] / zs) * half_to_double(Vh[(size_t)i2[j] * d + c]);
            /* Eq. (10) */
            out[c] = a * y + (1.0 - a) * vbar[c];
        }
        free(z);
    }
    free(q); free(qa); free(lh); free(vbar);
}

/* SparQ decode for the listed (b, h) units (heads == NULL: all B*Hq units in order).
 * heads: [n_units, 2] int32 pairs.  Outputs are indexed by unit: out [n_units, d],
 * i1 [n_units, r], i2 [n_units, k] (-1 padded), alpha, gap_r, gap_k [n_units].
 * vbar: NULL or [B, Hkv, d] doubles.  Returns 0, or 1 on a bad argument. */
int sparq_oracle_decode(const uint16_t* q, const uint16_t* K, const uint16_t* V, const double* vbar,
                        const int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                        const int32_t* heads, int n_units, double* out, int32_t* i1, int32_t* i2,
                        double* alpha, double* gap_r, double* gap_k, int n_threads) {
    if (B < 1 || Hkv < 1 || Hq % Hkv || r < 1 || r > d || k < 0) return 1;
    int g = Hq / Hkv;
    if (!heads) n_units = B * Hq;
    for (int b = 0; b < B; ++b) if (seq_lens[b] < 1 || seq_lens[b] > S_max) return 1;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < n_units; ++u) {
        int b = heads ? heads[2 * u] : u / Hq, h = heads ? heads[2 * u + 1] : u % Hq;
        size_t kv = ((size_t)b * Hkv + h / g) * (size_t)S_max * d;
        sparq_unit(q + ((size_t)b * Hq + h) * d, K + kv, V + kv,
                   vbar ? vbar + ((size_t)b * Hkv + h / g) * d : NULL, seq_lens[b], d, r, k,
                   out + (size_t)u * d, i1 + (size_t)u * r, i2 + (size_t)u * (k > 0 ? k : 0),
                   alpha + u, gap_r + u, gap_k + u);
    }
    return 0;
}

/* Eq. (2): dense attention for the listed units. */
int sparq_oracle_dense(const uint16_t* q, const uint16_t* K, const uint16_t* V, const int32_t* seq_lens,
                       int B, int Hq, int Hkv, int d, int S_max, const int32_t* heads, int n_units,
                       double* out, int n_threads) {
    if (B < 1 || Hkv < 1 || Hq % Hkv) return 1;
    int g = Hq / Hkv;
    if (!heads) n_units = B * Hq;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel for schedule(dynamic, 1)
    for (int u = 0; u < n_units; ++u) {
        int b = heads ? heads[2 * u] : u / Hq, h = heads ? heads[2 * u + 1] : u % Hq;
        int n = seq_lens[b];
        size_t kv = ((size_t)b * Hkv + h / g) * (size_t)S_max * d;
        const uint16_t* qh = q + ((size_t)b * Hq + h) * d;
        double* z = (double*)malloc(sizeof(double) * (n > 0 ? n : 1));
        double zmax = -INFINITY, zs = 0.0;
        for (int t = 0; t < n; ++t) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += half_to_double(qh[c]) * half_to_double(K[kv + (size_t)t * d + c]);
            z[t] = acc / sqrt((double)d);
            if (z[t] > zmax) zmax = z[t];
        }
        for (int t = 0; t < n; ++t) { z[t] = exp(z[t] - zmax); zs += z[t]; }
        for (int c = 0; c < d; ++c) {
            double y = 0.0;
            for (int t = 0; t < n; ++t) y += (z[t] / zs) * half_to_double(V[kv + (size_t)t * d + c]);
            out[(size_t)u * d + c] = y;
        }
        free(z);
    }
    return 0;
}

int sparq_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

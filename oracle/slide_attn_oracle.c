/*
 * CPU oracle for the Slide Attention forward.  TEST INFRASTRUCTURE ONLY: it is
 * called by the tests, by the smoke check and by the benchmark's CPU-baseline
 * leg, never by the library.  It shares no code with the CUDA path.
 *
 * It is the plain definition, in double precision, evaluated step by step in
 * the paper's order and notation:
 *
 *   1. keys/values of slot (u,v) = depthwise k x k convolution of the zero-padded
 *      K / V map with that slot's kernel (Sec. 4.2, Eq. 12; the k*k kernels
 *      form one group convolution, last paragraph of Sec. 4.2).  The kernel
 *      passed in is the merged one: fixed shift (Eq. 11) + learned deformed
 *      shift (Sec. 4.3, re-parameterised into a single convolution).
 *   2. logits = q . key_slot / sqrt(d) per head (Eq. 2), + optional per-slot bias
 *   3. softmax over the k*k slots (sigma in Eq. 2)
 *   4. out = sum over slots of attention * value_slot (Eq. 2)
 *
 * Indexing (the paper's Eq. 4-5 index ranges are inconsistent; this is the
 * reading used): i is the row in [0,H), j the column in [0,W); window offsets
 * u,v in [-r, r], r = floor(k/2); slot index s = (u+r)*k + (v+r); kernel tap
 * index t = p*k + q_ for kernel position (p,q_) in [0,k)^2, which reads the map
 * at (i+p-r, j+q_-r) exactly as Eq. 12 does for k = 3 (cross-correlation, no
 * kernel flip).  Positions outside the map read as zero ("[1,1] padding",
 * caption of Fig. 2); padded slots stay in the softmax.
 *
 * Layouts: q,k,v [B][H][W][heads][d] (channel c = h*d + e), float holding the
 * exact stored values (fp32, or bf16 widened); w [C][k*k slot][k*k tap] float;
 * bias [heads][k*k] float or NULL.  Everything is accumulated in double.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    const float *q, *k, *v, *wk, *wv, *bias;
    int B, H, W, heads, d, ksize;
} problem_t;

/* zero-padded read of a [B][H][W][C] map (Fig. 2 caption: padding) */
static double padded(const float *f, const problem_t *P, int b, int i, int j, int c)
{
    if (i < 0 || i >= P->H || j < 0 || j >= P->W) return 0.0;
    size_t C = (size_t)P->heads * P->d;
    return (double)f[(((size_t)b * P->H + i) * P->W + j) * C + c];
}

/* Eq. 12 with the merged kernel of one slot:
 * f_dwc[i,j,c] = sum_{p,q_} Kern[p,q_,c] * f[i+p-r, j+q_-r, c] */
static double dwconv_slot(const float *f, const float *w, const problem_t *P,
                          int b, int i, int j, int c, int s)
{
    int k = P->ksize, r = k / 2, k2 = k * k;
    const float *kern = w + ((size_t)c * k2 + s) * k2;
    double acc = 0.0;
    for (int p = 0; p < k; ++p)
        for (int q_ = 0; q_ < k; ++q_)
            acc += (double)kern[p * k + q_] * padded(f, P, b, i + p - r, j + q_ - r, c);
    return acc;
}

/* Eq. 2 for one query pixel (b,i,j): all heads.  out_px: C doubles.
 * attn_px: heads*k*k doubles or NULL.  scratch: 2*k*k*d doubles. */
static void one_pixel(const problem_t *P, int b, int i, int j,
                      double *out_px, double *attn_px, double *scratch)
{
    int d = P->d, k2 = P->ksize * P->ksize;
    size_t C = (size_t)P->heads * d;
    const float *qp = P->q + (((size_t)b * P->H + i) * P->W + j) * C;
    double *Ks = scratch, *Vs = scratch + (size_t)k2 * d;
    double *l = (double *)malloc(sizeof(double) * k2);
    for (int h = 0; h < P->heads; ++h) {
        for (int s = 0; s < k2; ++s)
            for (int e = 0; e < d; ++e) {
                int c = h * d + e;
                Ks[s * d + e] = dwconv_slot(P->k, P->wk, P, b, i, j, c, s);
                Vs[s * d + e] = dwconv_slot(P->v, P->wv, P, b, i, j, c, s);
            }
        for (int s = 0; s < k2; ++s) {
            double dot = 0.0;
            for (int e = 0; e < d; ++e) dot += (double)qp[h * d + e] * Ks[s * d + e];
            l[s] = dot / sqrt((double)d);
            if (P->bias) l[s] += (double)P->bias[h * k2 + s];
        }
        double m = l[0];
        for (int s = 1; s < k2; ++s) if (l[s] > m) m = l[s];
        double z = 0.0;
        for (int s = 0; s < k2; ++s) { l[s] = exp(l[s] - m); z += l[s]; }
        for (int s = 0; s < k2; ++s) l[s] /= z;
        if (attn_px) for (int s = 0; s < k2; ++s) attn_px[h * k2 + s] = l[s];
        for (int e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int s = 0; s < k2; ++s) acc += l[s] * Vs[s * d + e];
            out_px[h * d + e] = acc;
        }
    }
    free(l);
}

static int check(const problem_t *P)
{
    if (!P->q || !P->k || !P->v || !P->wk || !P->wv) return 1;
    if (P->B < 0 || P->H < 1 || P->W < 1 || P->heads < 1 || P->d < 1) return 1;
    if (P->ksize < 1 || (P->ksize & 1) == 0) return 1;   /* odd windows only */
    return 0;
}

/* Full forward.  out [B][H][W][C] double; attn [B][H][W][heads][k*k] double or NULL.
 * Returns 0 on success, 1 on invalid arguments. */
int slide_attn_oracle(const float *q, const float *k, const float *v,
                      const float *wk, const float *wv, const float *bias,
                      int B, int H, int W, int heads, int d, int ksize,
                      double *out, double *attn)
{
    problem_t P = {q, k, v, wk, wv, bias, B, H, W, heads, d, ksize};
    if (check(&P) || !out) return 1;
    long long npx = (long long)B * H * W;
    size_t C = (size_t)heads * d;
    int k2 = ksize * ksize;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * 2 * (size_t)k2 * d);
#pragma omp for schedule(static)
        for (long long n = 0; n < npx; ++n) {
            int j = (int)(n % W), i = (int)((n / W) % H), b = (int)(n / ((long long)W * H));
            one_pixel(&P, b, i, j, out + (size_t)n * C,
                      attn ? attn + (size_t)n * heads * k2 : NULL, scratch);
        }
        free(scratch);
    }
    return 0;
}

/* The same definition on a list of query pixels (flat index n = (b*H + i)*W + j)
 * of the full-size problem.  out [npix][C] double. */
int slide_attn_oracle_pixels(const float *q, const float *k, const float *v,
                             const float *wk, const float *wv, const float *bias,
                             int B, int H, int W, int heads, int d, int ksize,
                             const long long *pix, long long npix, double *out)
{
    problem_t P = {q, k, v, wk, wv, bias, B, H, W, heads, d, ksize};
    if (check(&P) || !out || (npix > 0 && !pix)) return 1;
    long long npx = (long long)B * H * W;
    for (long long a = 0; a < npix; ++a) if (pix[a] < 0 || pix[a] >= npx) return 1;
    size_t C = (size_t)heads * d;
    int k2 = ksize * ksize;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * 2 * (size_t)k2 * d);
#pragma omp for schedule(static)
        for (long long a = 0; a < npix; ++a) {
            long long n = pix[a];
            int j = (int)(n % W), i = (int)((n / W) % H), b = (int)(n / ((long long)W * H));
            one_pixel(&P, b, i, j, out + (size_t)a * C, NULL, scratch);
        }
        free(scratch);
    }
    return 0;
}

/* Step 1 alone: the k*k-expanded map of Sec. 4.2, out [B][H][W][k*k][C] double. */
int slide_attn_oracle_dwconv(const float *f, const float *w,
                             int B, int H, int W, int C, int ksize, double *out)
{
    problem_t P = {f, f, f, w, w, NULL, B, H, W, 1, C, ksize};
    if (check(&P) || !out) return 1;
    int k2 = ksize * ksize;
    long long npx = (long long)B * H * W;
#pragma omp parallel for schedule(static)
    for (long long n = 0; n < npx; ++n) {
        int j = (int)(n % W), i = (int)((n / W) % H), b = (int)(n / ((long long)W * H));
        for (int s = 0; s < k2; ++s)
            for (int c = 0; c < C; ++c)
                out[((size_t)n * k2 + s) * C + c] = dwconv_slot(f, w, &P, b, i, j, c, s);
    }
    return 0;
}

int slide_attn_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

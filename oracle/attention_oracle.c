/* fp64 CPU oracle: attention rows restricted to a list of key blocks, plain loops.
 *
 * TEST INFRASTRUCTURE -- checks the CUDA kernels; shares no code with them and is never on
 * the product path.
 *
 * For query token t of segment j with critical block list I_j (Algorithm 2, lines 6-11),
 * with token-level causality inside the selected blocks:
 *     U_t  = { u : floor(u / blk) in I_j  and  u <= t }
 *     O[t] = sum_{u in U_t} softmax_u( sm_scale * q_t . k_u ) * v_u        (Eq. 2 on U_t)
 *     lse[t] = ln sum_{u in U_t} exp( sm_scale * q_t . k_u )
 * The dense baseline (Eq. 2, causal) is the same with U_t = { u <= t }.
 * Inputs are float (every bf16 value is a float) and are widened to double before any
 * arithmetic.  One row is computed at a time, in the order score -> max -> exp/sum ->
 * weighted sum; rows are independent and OpenMP only distributes them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

static void one_row(const float *q, const float *Kh, const float *Vh, int d, double sm_scale,
                    const int64_t *keys, int64_t n_keys, double *o, double *lse, double *w)
{
    double mx = -INFINITY;
    for (int64_t i = 0; i < n_keys; ++i) {
        const float *k = Kh + keys[i] * (int64_t)d;
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += (double)q[c] * (double)k[c];
        w[i] = s * sm_scale;
        if (w[i] > mx) mx = w[i];
    }
    double z = 0.0;
    for (int64_t i = 0; i < n_keys; ++i) { w[i] = exp(w[i] - mx); z += w[i]; }
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int64_t i = 0; i < n_keys; ++i) {
        const float *v = Vh + keys[i] * (int64_t)d;
        double p = w[i] / z;
        for (int c = 0; c < d; ++c) o[c] += p * (double)v[c];
    }
    *lse = mx + log(z);
}

/* rows: n_rows triples (b, h, t).  idx [B,Hq,n1,k] / cnt [B,Hq,n1]; idx == NULL means dense.
 * Q [B,Hq,n,d], K,V [B,Hkv,n,d] contiguous float.  O [n_rows,d], lse [n_rows] double. */
int oracle_attention_rows(const float *Q, const float *K, const float *V,
                          const int32_t *idx, const int32_t *cnt,
                          int B, int Hq, int Hkv, int64_t n, int d,
                          int seg, int blk, int k, double sm_scale,
                          const int64_t *rows, int64_t n_rows, double *O, double *lse)
{
    (void)B;
    int g = Hq / Hkv;
    int64_t n1 = (n + seg - 1) / seg;   /* the last segment may be shorter */
    int err = 0;
#pragma omp parallel
    {
        int64_t *keys = (int64_t *)malloc(sizeof(int64_t) * (size_t)n);
        double *w = (double *)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < n_rows; ++r) {
            int64_t b = rows[3 * r], h = rows[3 * r + 1], t = rows[3 * r + 2];
            int64_t j = t / seg;
            int64_t nk = 0;
            if (idx == NULL) {
                for (int64_t u = 0; u <= t; ++u) keys[nk++] = u;
            } else {
                const int32_t *list = idx + ((b * Hq + h) * n1 + j) * (int64_t)k;
                int c = cnt[(b * Hq + h) * n1 + j];
                for (int i = 0; i < c; ++i) {
                    int64_t blkid = list[i];
                    if (blkid < 0 || blkid * blk >= n) { err = 1; continue; }
                    for (int64_t u = blkid * blk; u < (blkid + 1) * blk; ++u)
                        if (u <= t) keys[nk++] = u;
                }
            }
            const float *q = Q + ((b * Hq + h) * n + t) * (int64_t)d;
            const float *Kh = K + ((b * Hkv + h / g) * n) * (int64_t)d;
            const float *Vh = V + ((b * Hkv + h / g) * n) * (int64_t)d;
            one_row(q, Kh, Vh, d, sm_scale, keys, nk, O + r * (int64_t)d, lse + r, w);
        }
        free(keys);
        free(w);
    }
    return err;
}

/*
 * CPU oracle for the dense linear layers (forward and backward) of the GPT-2
 * 124M training step. TEST INFRASTRUCTURE ONLY: plain, slow, and independent of
 * the CUDA library. Only the tests, the smoke check and the benchmark's CPU
 * baseline may load it.
 *
 * Two instances of the same source: suffix _f32 computes and accumulates in
 * float (the arithmetic the training step's precision statement names), suffix
 * _f64 in double (used to bound the float instance's own rounding and as the
 * parity reference). See nb_oracle_impl.inc for the definitions followed.
 *
 * Every exported function is pinned by tests that do not use this file:
 * library GELU/SiLU, library autograd, integer-exact products, finite
 * differences and adjoint identities.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define NBO_ACT_NONE 0
#define NBO_ACT_GELU 1
#define NBO_ACT_SWIGLU 2

#define REAL float
#define SUFFIX _f32
#define TANH tanhf
#define EXP expf
#include "nb_oracle_impl.inc"
#undef REAL
#undef SUFFIX
#undef TANH
#undef EXP

#define REAL double
#define SUFFIX _f64
#define TANH tanh
#define EXP exp
#include "nb_oracle_impl.inc"
#undef REAL
#undef SUFFIX
#undef TANH
#undef EXP

/* Column sum used by the stand-alone dbias reduction: dbias[o] (+)= sum_m dout[m,o]. */
int nbo_reduce_dbias_f64(double *dbias, const float *dout, int64_t BT, int64_t OC, int accumulate)
{
    if (!dbias || !dout || BT < 0 || OC < 0) return -1;
    for (int64_t o = 0; o < OC; ++o) {
        double s = 0.0;
        for (int64_t m = 0; m < BT; ++m) s += (double)dout[m * OC + o];
        if (accumulate)
            dbias[o] += s;
        else
            dbias[o] = s;
    }
    return 0;
}

/*
 * fp32 -> bf16, round to nearest, ties to even (the master-weight cast done once per optimizer
 * step; paper: Results/Speed, the table of levers, the row on reusing the cast across micro-steps).
 * Written on the bit patterns: keep the top 16 bits, add one when the discarded half is above
 * one half of the last kept bit, or exactly one half and the kept value is odd. Infinities stay,
 * a carry out of the largest finite value gives infinity, NaN stays NaN (quiet, sign kept).
 */
void nbo_cast_f32_bf16(uint16_t *dst, const float *src, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) {
        uint32_t u;
        memcpy(&u, &src[i], 4);
        const uint32_t exp = (u >> 23) & 0xFFu, man = u & 0x7FFFFFu;
        if (exp == 0xFFu && man != 0) { /* NaN */
            dst[i] = (uint16_t)((u >> 16) | 0x0040u);
            continue;
        }
        const uint32_t kept = u >> 16, rest = u & 0xFFFFu;
        uint32_t r = kept;
        if (rest > 0x8000u || (rest == 0x8000u && (kept & 1u))) r = kept + 1u;
        dst[i] = (uint16_t)r;
    }
}

/*
 * Cross-entropy of the head's logits over the first V of Vp columns (paper: Figure 1, the loss box:
 * only the 50,257 real tokens take part, the padding columns get neither probability nor gradient; loss in f32).
 *   lse[i]       = log sum_{j<V} exp(logits[i,j])
 *   loss[i]      = lse[i] - logits[i, target[i]]
 *   dlogits[i,j] = gscale * (exp(logits[i,j] - lse[i]) - [j == target[i]])   for j <  V
 *                = 0                                                          for j >= V
 * logits are floats holding the stored bf16 values; everything else is double. dlogits may be
 * NULL. Returns -1 on a malformed request (a target outside [0, V) included).
 */
int nbo_cross_entropy_f64(double *loss, double *lse, double *dlogits, const float *logits,
                          const int32_t *targets, int64_t BT, int64_t Vp, int64_t V, double gscale)
{
    if (!loss || !lse || !logits || !targets || BT < 0 || V <= 0 || Vp < V) return -1;
    for (int64_t i = 0; i < BT; ++i)
        if (targets[i] < 0 || targets[i] >= V) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < BT; ++i) {
        const float *row = logits + i * Vp;
        double mx = (double)row[0];
        for (int64_t j = 1; j < V; ++j)
            if ((double)row[j] > mx) mx = (double)row[j];
        double sum = 0.0;
        for (int64_t j = 0; j < V; ++j) sum += exp((double)row[j] - mx);
        lse[i] = mx + log(sum);
        loss[i] = lse[i] - (double)row[targets[i]];
        if (dlogits) {
            double *d = dlogits + i * Vp;
            for (int64_t j = 0; j < V; ++j)
                d[j] = gscale * (exp((double)row[j] - lse[i]) - (j == targets[i] ? 1.0 : 0.0));
            for (int64_t j = V; j < Vp; ++j) d[j] = 0.0;
        }
    }
    return 0;
}

/*
 * Low-rank adapter beside a frozen linear layer (paper: Method/The clinical stage: rank-16
 * adapters, rank-stabilised scaling, on the projections of Qwen3-0.6B; base weights frozen).
 *   t        = inp . A^T                                  [BT, r]      A: [r, C]
 *   out      = inp . W^T (+ b) + scale * t . B^T          [BT, OC]     B: [OC, r]
 *   u        = dout . B                                   [BT, r]
 *   dinp     = dout . W + scale * u . A                   [BT, C]
 *   dA (+)=    scale * u^T . inp                          [r, C]
 *   dB (+)=    scale * dout^T . t                         [OC, r]
 * Intermediates t and u are kept unrounded. Any output pointer may be NULL.
 */
int nbo_lora_forward_f64(double *out, const float *inp, const float *W, const float *bias,
                         const float *A, const float *B, double scale, int64_t BT, int64_t C,
                         int64_t OC, int64_t r)
{
    if (!out || !inp || !W || !A || !B || BT < 0 || C <= 0 || OC <= 0 || r <= 0 || r > 256) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < BT; ++m) {
        double t[256];
        for (int64_t j = 0; j < r; ++j) {
            double acc = 0.0;
            for (int64_t k = 0; k < C; ++k) acc += (double)inp[m * C + k] * (double)A[j * C + k];
            t[j] = acc;
        }
        for (int64_t o = 0; o < OC; ++o) {
            double acc = 0.0;
            for (int64_t k = 0; k < C; ++k) acc += (double)inp[m * C + k] * (double)W[o * C + k];
            if (bias) acc += (double)bias[o];
            double lo = 0.0;
            for (int64_t j = 0; j < r; ++j) lo += t[j] * (double)B[o * r + j];
            out[m * OC + o] = acc + scale * lo;
        }
    }
    return 0;
}

int nbo_lora_backward_f64(double *dinp, double *dA, double *dB, const float *dout, const float *inp,
                          const float *W, const float *A, const float *B, double scale, int64_t BT,
                          int64_t C, int64_t OC, int64_t r, int accumulate)
{
    if (!dout || !inp || !W || !A || !B || BT < 0 || C <= 0 || OC <= 0 || r <= 0 || r > 256) return -1;
    double *t = (double *)malloc(sizeof(double) * (size_t)(BT * r > 0 ? BT * r : 1));
    double *u = (double *)malloc(sizeof(double) * (size_t)(BT * r > 0 ? BT * r : 1));
    if (!t || !u) return -2;
    for (int64_t m = 0; m < BT; ++m)
        for (int64_t j = 0; j < r; ++j) {
            double a = 0.0, b = 0.0;
            for (int64_t k = 0; k < C; ++k) a += (double)inp[m * C + k] * (double)A[j * C + k];
            for (int64_t o = 0; o < OC; ++o) b += (double)dout[m * OC + o] * (double)B[o * r + j];
            t[m * r + j] = a;
            u[m * r + j] = b;
        }
    if (dinp) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < BT; ++m)
            for (int64_t c = 0; c < C; ++c) {
                double acc = 0.0;
                for (int64_t o = 0; o < OC; ++o) acc += (double)dout[m * OC + o] * (double)W[o * C + c];
                double lo = 0.0;
                for (int64_t j = 0; j < r; ++j) lo += u[m * r + j] * (double)A[j * C + c];
                dinp[m * C + c] = acc + scale * lo;
            }
    }
    if (dA) {
        for (int64_t j = 0; j < r; ++j)
            for (int64_t c = 0; c < C; ++c) {
                double acc = 0.0;
                for (int64_t m = 0; m < BT; ++m) acc += u[m * r + j] * (double)inp[m * C + c];
                if (accumulate) dA[j * C + c] += scale * acc;
                else dA[j * C + c] = scale * acc;
            }
    }
    if (dB) {
        for (int64_t o = 0; o < OC; ++o)
            for (int64_t j = 0; j < r; ++j) {
                double acc = 0.0;
                for (int64_t m = 0; m < BT; ++m) acc += (double)dout[m * OC + o] * t[m * r + j];
                if (accumulate) dB[o * r + j] += scale * acc;
                else dB[o * r + j] = scale * acc;
            }
    }
    free(t);
    free(u);
    return 0;
}

int nbo_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

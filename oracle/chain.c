/*
 * TEST INFRASTRUCTURE -- part of the CPU oracle, never of the product path.
 *
 * The two pieces of the noisy-gating logits (Eq. 4) whose rounding decides an
 * integer (which experts a token is routed to, Eq. 5) and therefore have a
 * fixed single-precision evaluation order:
 *
 *   (x . W)_j   = one chain of fused multiply-adds over q = 0, 1, ..., d-1,
 *                 starting from +0, one rounding per step;
 *   H_j         = fma(noise_j, sigma_j, clean_j), one rounding.
 *
 * Build: gcc -O2 -mfma -ffp-contract=off -shared -fPIC (see oracle/__init__.py).
 * -ffp-contract=off keeps the compiler from fusing or splitting anything that is
 * not written as fmaf() here.
 */
#include <math.h>
#include <stdint.h>

/* out[t, j] = (((0 + x[t,0] W[0,j]) + x[t,1] W[1,j]) + ...) with fmaf at every step.
 * x is [T, d] with row stride ldx, W is [d, n] row-major, out is [T, n]. */
void oracle_proj_chain_f32(int64_t T, int64_t d, int64_t n, const float *x, int64_t ldx,
                           const float *W, float *out)
{
    for (int64_t t = 0; t < T; ++t) {
        float *o = out + t * n;
        for (int64_t j = 0; j < n; ++j) o[j] = 0.0f;
        for (int64_t q = 0; q < d; ++q) {
            const float xq = x[t * ldx + q];
            const float *w = W + q * n;
            for (int64_t j = 0; j < n; ++j) o[j] = fmaf(xq, w[j], o[j]);
        }
    }
}

/* out[i] = fma(a[i], b[i], c[i]) in single precision. */
void oracle_fma_f32(int64_t N, const float *a, const float *b, const float *c, float *out)
{
    for (int64_t i = 0; i < N; ++i) out[i] = fmaf(a[i], b[i], c[i]);
}

/*
 * dpclip_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded fp64 CPU statement of what the per-example
 * clipping path computes, written from the paper.  It shares no code with the
 * CUDA library and must never be called from the product path: only the test
 * suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every per-example gradient is materialised explicitly (this is exactly the
 * memory cost the method avoids on the GPU):
 *
 *   dense layer          dL/dW = dL/dz (outer) x              Eq. "grad_linear_layer", Algorithm 2
 *   bias                 dL/db = dL/dz                        Sec. "Fully-connected Layers"
 *   convolution          G = deltaZ . im2col(X)               Algorithm 3
 *   recurrent / LSTM     dL/dW = sum_t dL/dz(t) (outer) h(t-1), dL/db = sum_t dL/dz(t)   Algorithm 4
 *   attention projection dL/dW^Q = (dL/dQ)^T Q_prev           Sec. "Multi-head attention"
 *   LayerNorm gain/shift dL/dgamma = dL/dh (.) hbar, dL/dbeta = dL/dh   Sec. "LayerNorm Layers" and its Algorithm
 *
 * All of these are one formula once the layer input is given as A (T rows of
 * d_in) and the back-propagated signal as Zbar (T rows of d_out):
 *       G_i = sum_t zbar_{i,t} (outer) a_{i,t}     (d_out x d_in, row-major)
 *       gb_i = sum_t zbar_{i,t}
 * The total per-example norm is the square root of the sum over layers of the
 * squared weight- and bias-gradient norms (Sec. "algorithm", text after
 * Eq. "weighted_loss"); the clip factor is nu_i = min(1, c/||g_i||)
 * (Eq. "per_example_weight"), with nu_i = 1 when the norm is zero, which is
 * what clip_c(z) = z / max(1, ||z||/c) gives; the released quantity is the
 * SUM over the batch of nu_i * G_i plus Gaussian noise of standard deviation
 * sigma*C per coordinate (Algorithm 1, last line, without its 1/tau factor).
 *
 * The noise generator is not specified by the paper.  Reading used by both
 * sides: Philox4x32-10 (Salmon et al., SC'11) keyed by the 64-bit seed,
 * counter = (block index lo, hi, stream id lo, hi); 32-bit words mapped to
 * u in (0,1] by ONE float fma  u = x*2^-32 + 2^-33;  Box-Muller on word pairs
 * (0,1) -> elements 4q,4q+1 (cos, sin) and (2,3) -> 4q+2,4q+3.  The oracle
 * evaluates log/sqrt/cos/sin in double from that float u.
 *
 * Parity pins (tests marked "not gpu"): brute-force autodiff and finite
 * differences on tiny networks, the T=1 closed form, clip invariants, the
 * C->infinity limit against a library matmul, and for Philox the C++26
 * check value and two independent host engines.  Nothing here is unpinned.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---------------------------------------------------------------- gradients */

/* One example, one layer.  A: T x d_in, Z: T x d_out (row-major, dense).
 * G (d_out x d_in) and gb (d_out) are OVERWRITTEN. */
void oracle_example_grad(const double* A, const double* Z, int T, int d_in, int d_out,
                         double* G, double* gb)
{
    memset(G, 0, sizeof(double) * (size_t)d_out * d_in);
    memset(gb, 0, sizeof(double) * (size_t)d_out);
    for (int t = 0; t < T; ++t) {
        const double* a = A + (size_t)t * d_in;
        const double* z = Z + (size_t)t * d_out;
        for (int o = 0; o < d_out; ++o) {
            double zo = z[o];
            double* g = G + (size_t)o * d_in;
            for (int k = 0; k < d_in; ++k) g[k] += zo * a[k];
            gb[o] += zo;
        }
    }
}

static double sum_squares(const double* x, size_t n)
{
    double s = 0.0;
    for (size_t j = 0; j < n; ++j) s += x[j] * x[j];
    return s;
}

/* Squared per-example gradient norm of one layer, for every example.
 * A: B x T x d_in, Z: B x T x d_out.  sq[B] overwritten.  Returns 0, or -1 if
 * scratch memory could not be obtained. */
int oracle_layer_sqnorms(const double* A, const double* Z, int B, int T, int d_in, int d_out,
                         int has_bias, double* sq)
{
    double* G = (double*)malloc(sizeof(double) * (size_t)d_out * d_in);
    double* gb = (double*)malloc(sizeof(double) * (size_t)d_out);
    if (!G || !gb) { free(G); free(gb); return -1; }
    for (int i = 0; i < B; ++i) {
        oracle_example_grad(A + (size_t)i * T * d_in, Z + (size_t)i * T * d_out, T, d_in, d_out, G, gb);
        double s = sum_squares(G, (size_t)d_out * d_in);
        if (has_bias) s += sum_squares(gb, (size_t)d_out);
        sq[i] = s;
    }
    free(G); free(gb);
    return 0;
}

/* sq_layers: L x B (row l = layer l).  norms[B], clip[B] overwritten. */
void oracle_factors(const double* sq_layers, int L, int B, double C, double* norms, double* clip)
{
    for (int i = 0; i < B; ++i) {
        double s = 0.0;
        for (int l = 0; l < L; ++l) s += sq_layers[(size_t)l * B + i];
        double n = sqrt(s);
        norms[i] = n;
        double m = n / C;                 /* clip_c(z) = z / max(1, ||z||/c) */
        clip[i] = 1.0 / (m > 1.0 ? m : 1.0);
    }
}

/* Clipped sum of one layer: gW = sum_i clip[i] * G_i (d_out x d_in),
 * gb = sum_i clip[i] * gb_i.  clip == NULL means all ones. */
int oracle_clipped_grad(const double* A, const double* Z, int B, int T, int d_in, int d_out,
                        const double* clip, double* gW, double* gb_out)
{
    size_t nW = (size_t)d_out * d_in;
    double* G = (double*)malloc(sizeof(double) * nW);
    double* gb = (double*)malloc(sizeof(double) * (size_t)d_out);
    if (!G || !gb) { free(G); free(gb); return -1; }
    memset(gW, 0, sizeof(double) * nW);
    memset(gb_out, 0, sizeof(double) * (size_t)d_out);
    for (int i = 0; i < B; ++i) {
        oracle_example_grad(A + (size_t)i * T * d_in, Z + (size_t)i * T * d_out, T, d_in, d_out, G, gb);
        double c = clip ? clip[i] : 1.0;
        for (size_t j = 0; j < nW; ++j) gW[j] += c * G[j];
        for (int o = 0; o < d_out; ++o) gb_out[o] += c * gb[o];
    }
    free(G); free(gb);
    return 0;
}

/* ------------------------------------------- element-wise parameter layers */

/* LayerNorm-style layer h = gamma (.) hbar + beta (Sec. "LayerNorm Layers"): for one position the
 * per-example gradients are dL/dgamma = dL/dh (.) hbar and dL/dbeta = dL/dh (the section's Algorithm is
 * the product Z (.) H).  gamma and beta are shared by the T positions of an example, so, as for every
 * shared parameter, the per-position terms are summed BEFORE the norm is taken:
 *     ggamma_i = sum_t zbar_{i,t} (.) hbar_{i,t},   gbeta_i = sum_t zbar_{i,t}.
 * H: T x d normalised inputs, Z: T x d back-propagated signals; gg[d], gs[d] OVERWRITTEN. */
void oracle_elementwise_example_grad(const double* H, const double* Z, int T, int d, double* gg, double* gs)
{
    for (int j = 0; j < d; ++j) { gg[j] = 0.0; gs[j] = 0.0; }
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < d; ++j) {
            gg[j] += Z[(size_t)t * d + j] * H[(size_t)t * d + j];
            gs[j] += Z[(size_t)t * d + j];
        }
}

/* Squared per-example norms of such a layer: ||ggamma_i||^2 (+ ||gbeta_i||^2 with a shift).  sq[B]. */
int oracle_elementwise_sqnorms(const double* H, const double* Z, int B, int T, int d, int has_shift, double* sq)
{
    double* gg = (double*)malloc(sizeof(double) * (size_t)d);
    double* gs = (double*)malloc(sizeof(double) * (size_t)d);
    if (!gg || !gs) { free(gg); free(gs); return -1; }
    for (int i = 0; i < B; ++i) {
        oracle_elementwise_example_grad(H + (size_t)i * T * d, Z + (size_t)i * T * d, T, d, gg, gs);
        double s = sum_squares(gg, (size_t)d);
        if (has_shift) s += sum_squares(gs, (size_t)d);
        sq[i] = s;
    }
    free(gg); free(gs);
    return 0;
}

/* Clipped sums: g_scale = sum_i clip[i] ggamma_i, g_shift = sum_i clip[i] gbeta_i (clip NULL = ones). */
int oracle_elementwise_clipped_grad(const double* H, const double* Z, int B, int T, int d, const double* clip,
                                    double* g_scale, double* g_shift)
{
    double* gg = (double*)malloc(sizeof(double) * (size_t)d);
    double* gs = (double*)malloc(sizeof(double) * (size_t)d);
    if (!gg || !gs) { free(gg); free(gs); return -1; }
    for (int j = 0; j < d; ++j) { g_scale[j] = 0.0; g_shift[j] = 0.0; }
    for (int i = 0; i < B; ++i) {
        oracle_elementwise_example_grad(H + (size_t)i * T * d, Z + (size_t)i * T * d, T, d, gg, gs);
        double c = clip ? clip[i] : 1.0;
        for (int j = 0; j < d; ++j) { g_scale[j] += c * gg[j]; g_shift[j] += c * gs[j]; }
    }
    free(gg); free(gs);
    return 0;
}

/* -------------------------------------------------------------------- noise */

/* Philox4x32 with 10 rounds: one 128-bit counter block under a 64-bit key. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;     /* multipliers */
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;     /* key increments (Weyl) */
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 32 random bits -> float in (0, 1], by a single correctly rounded fma. */
static float u01(uint32_t x)
{
    return fmaf((float)x, 2.3283064365386963e-10f /* 2^-32 */, 1.1641532182693481e-10f /* 2^-33 */);
}

/* Standard normals xi[j], j in [0, n): element j uses block q = j/4 of stream
 * (seed, stream_id).  Box-Muller on (word0, word1) and (word2, word3). */
void oracle_normals(size_t n, uint64_t seed, uint64_t stream_id, double* xi)
{
    const double two_pi = 6.283185307179586476925286766559;
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (size_t q = 0; 4 * q < n; ++q) {
        uint32_t ctr[4] = { (uint32_t)q, (uint32_t)((uint64_t)q >> 32),
                            (uint32_t)stream_id, (uint32_t)(stream_id >> 32) };
        uint32_t x[4];
        oracle_philox4x32_10(ctr, key, x);
        double v[4];
        for (int h = 0; h < 2; ++h) {
            double u1 = (double)u01(x[2 * h]);
            double u2 = (double)u01(x[2 * h + 1]);
            double r = sqrt(-2.0 * log(u1));
            v[2 * h] = r * cos(two_pi * u2);
            v[2 * h + 1] = r * sin(two_pi * u2);
        }
        for (int e = 0; e < 4 && 4 * q + e < n; ++e) xi[4 * q + e] = v[e];
    }
}

/* g[j] += sigma * C * xi_j  (Gaussian mechanism with per-coordinate standard
 * deviation sigma*C). */
int oracle_add_noise(double* g, size_t n, double sigma, double C, uint64_t seed, uint64_t stream_id)
{
    double* xi = (double*)malloc(sizeof(double) * (n ? n : 1));
    if (!xi) return -1;
    oracle_normals(n, seed, stream_id, xi);
    for (size_t j = 0; j < n; ++j) g[j] += sigma * C * xi[j];
    free(xi);
    return 0;
}

/* -------------------------------------------------------- parameter updates */

/* The update of Algorithm 1's last line, theta <- theta - eta * (noise + (1/tau) * clipped sum), with the
 * noise read as in the rest of this file: N(0, sigma^2 C^2) on the SUM, so the noisy mean gradient is
 *     g[j] = (gsum[j] + sigma * C * xi_j) / tau.
 * inv_tau = 1/tau.  theta[n] is updated in place. */
int oracle_dp_sgd_step(double* theta, const double* gsum, size_t n, double inv_tau, double C, double sigma,
                       uint64_t seed, uint64_t stream_id, double lr)
{
    double* xi = (double*)malloc(sizeof(double) * (n ? n : 1));
    if (!xi) return -1;
    oracle_normals(n, seed, stream_id, xi);
    for (size_t j = 0; j < n; ++j) theta[j] -= lr * (gsum[j] + sigma * C * xi[j]) * inv_tau;
    free(xi);
    return 0;
}

/* The private Adam of the experiments (Sec. "Experiments": the non-private Adam of Kingma & Ba fed with the
 * noisy clipped gradient; step size 0.001, beta1 = 0.9, beta2 = 0.999 there).  With g as above and t the
 * 1-based step count:
 *     m <- beta1 m + (1 - beta1) g,   v <- beta2 v + (1 - beta2) g^2,
 *     theta <- theta - lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps). */
int oracle_dp_adam_step(double* theta, double* m, double* v, const double* gsum, size_t n, double inv_tau, double C,
                        double sigma, uint64_t seed, uint64_t stream_id, double lr, double beta1, double beta2,
                        double eps, int t)
{
    double* xi = (double*)malloc(sizeof(double) * (n ? n : 1));
    if (!xi) return -1;
    oracle_normals(n, seed, stream_id, xi);
    const double c1 = 1.0 - pow(beta1, (double)t), c2 = 1.0 - pow(beta2, (double)t);
    for (size_t j = 0; j < n; ++j) {
        const double g = (gsum[j] + sigma * C * xi[j]) * inv_tau;
        m[j] = beta1 * m[j] + (1.0 - beta1) * g;
        v[j] = beta2 * v[j] + (1.0 - beta2) * g * g;
        theta[j] -= lr * (m[j] / c1) / (sqrt(v[j] / c2) + eps);
    }
    free(xi);
    return 0;
}

/*
 * dp_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, float64 CPU statement of the DPSGD gradient-privatisation step
 * (paper section 2 "Algorithm", the equation for g_t; section 3.5 for the
 * per-group clipping rule).  It exists so that the CUDA library can be checked
 * against something that can be verified by eye.  Only the tests, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.  It shares no
 * code, header, table or constant with the CUDA path.
 *
 * Conventions
 *   - inputs (X, dY, flattened gradients) arrive as float32 arrays; every value
 *     the GPU sees (fp32, or bf16 widened) is exactly representable in them.
 *     All arithmetic is done in double, all results are double.
 *   - tensors are channels-last and contiguous:
 *       X  [B,H,W,Cin]   dY [B,OH,OW,Kout]   dW [B,Kout,R,S,Cin]   db [B,Kout]
 *   - convolution is cross-correlation with zero padding, dilation 1, groups 1.
 *   - OpenMP parallelism is over examples (and output channels) only.
 *
 * Pins (see tests/test_oracle_*.py): finite differences of <dY, conv(X,W)>,
 * PyTorch float64 autograd one example at a time, the 1x1 matmul special case,
 * the rank-1 closed form of the dense norm, the published Philox4x32-10
 * known-answer vectors, closed-form Box-Muller values and distribution tests.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Per-example weight gradients (section 2: "per-example gradients are       */
/* computed"; the layer formulas are the standard ones).                      */
/* ------------------------------------------------------------------------- */

/* dW_n[k,r,s,c] = sum_{oh,ow} dY_n[oh,ow,k] * Xpad_n[oh*st+r-p, ow*st+s-p, c]
 * db_n[k]       = sum_{oh,ow} dY_n[oh,ow,k]                (db may be NULL)  */
void oracle_conv_wgrad(const float *X, const float *dY, int B, int H, int W,
                       int Cin, int Kout, int R, int S, int stride, int pad,
                       double *dW, double *db)
{
    const int OH = (H + 2 * pad - R) / stride + 1;
    const int OW = (W + 2 * pad - S) / stride + 1;
    const size_t wsz = (size_t)Kout * R * S * Cin;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int n = 0; n < B; ++n) {
        for (int k = 0; k < Kout; ++k) {
            double *dWk = dW + (size_t)n * wsz + (size_t)k * R * S * Cin;
            memset(dWk, 0, sizeof(double) * (size_t)R * S * Cin);
            double bsum = 0.0;
            for (int oh = 0; oh < OH; ++oh) {
                for (int ow = 0; ow < OW; ++ow) {
                    const double g = (double)dY[(((size_t)n * OH + oh) * OW + ow) * Kout + k];
                    bsum += g;
                    for (int r = 0; r < R; ++r) {
                        const int ih = oh * stride + r - pad;
                        if (ih < 0 || ih >= H) continue;          /* zero padding */
                        for (int s = 0; s < S; ++s) {
                            const int iw = ow * stride + s - pad;
                            if (iw < 0 || iw >= W) continue;      /* zero padding */
                            const float *x = X + (((size_t)n * H + ih) * W + iw) * Cin;
                            double *d = dWk + ((size_t)r * S + s) * Cin;
                            for (int c = 0; c < Cin; ++c) d[c] += g * (double)x[c];
                        }
                    }
                }
            }
            if (db) db[(size_t)n * Kout + k] = bsum;
        }
    }
}

/* dense layer: dW_n[o,i] = dY[n,o] * X[n,i];  db_n[o] = dY[n,o] */
void oracle_dense_wgrad(const float *X, const float *dY, int B, int Cin, int Kout,
                        double *dW, double *db)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        for (int o = 0; o < Kout; ++o) {
            const double g = (double)dY[(size_t)n * Kout + o];
            for (int i = 0; i < Cin; ++i)
                dW[((size_t)n * Kout + o) * Cin + i] = g * (double)X[(size_t)n * Cin + i];
            if (db) db[(size_t)n * Kout + o] = g;
        }
    }
}

/* normalisation affine (scale gamma, shift beta applied per channel to the
 * normalised activation xhat):
 *   dgamma_n[c] = sum_{h,w} dY_n[h,w,c] * xhat_n[h,w,c];  dbeta_n[c] = sum dY_n[h,w,c] */
void oracle_norm_affine_wgrad(const float *xhat, const float *dY, int B, int HW, int C,
                              double *dgamma, double *dbeta)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        for (int c = 0; c < C; ++c) {
            double sg = 0.0, sb = 0.0;
            for (int p = 0; p < HW; ++p) {
                const size_t idx = ((size_t)n * HW + p) * C + c;
                sg += (double)dY[idx] * (double)xhat[idx];
                sb += (double)dY[idx];
            }
            dgamma[(size_t)n * C + c] = sg;
            dbeta[(size_t)n * C + c] = sb;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Norm, clip, accumulate (section 2, equation for g_t; section 3.5).         */
/* ------------------------------------------------------------------------- */

/* s[n] += sum_i G[n,i]^2  (double input; adds so several tensors can be chained) */
void oracle_sqnorm_add_f64(const double *G, int B, size_t P, double *s)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        double a = 0.0;
        for (size_t i = 0; i < P; ++i) a += G[(size_t)n * P + i] * G[(size_t)n * P + i];
        s[n] += a;
    }
}

/* same for float32 input (flattened per-example gradients handed in directly) */
void oracle_sqnorm_add_f32(const float *G, int B, size_t P, double *s)
{
#pragma omp parallel for
    for (int n = 0; n < B; ++n) {
        double a = 0.0;
        for (size_t i = 0; i < P; ++i) {
            const double v = (double)G[(size_t)n * P + i];
            a += v * v;
        }
        s[n] += a;
    }
}

/* clip(g, C) = g * min(1, C/||g||_2): the factor, from the squared norm.
 * Written as a branch so that ||g|| = 0 and C = +inf both give exactly 1. */
void oracle_clip_factor(const double *sq, size_t count, double C, double *factor)
{
    for (size_t j = 0; j < count; ++j)
        factor[j] = (sq[j] <= C * C) ? 1.0 : C / sqrt(sq[j]);
}

/* acc[i] += sum_n factor[n] * G[n,i]  (the clipped sum; acc persists over chunks) */
void oracle_clip_accumulate_f64(const double *G, int B, size_t P, const double *factor, double *acc)
{
#pragma omp parallel for
    for (size_t i = 0; i < P; ++i) {
        double a = 0.0;
        for (int n = 0; n < B; ++n) a += factor[n] * G[(size_t)n * P + i];
        acc[i] += a;
    }
}

void oracle_clip_accumulate_f32(const float *G, int B, size_t P, const double *factor, double *acc)
{
#pragma omp parallel for
    for (size_t i = 0; i < P; ++i) {
        double a = 0.0;
        for (int n = 0; n < B; ++n) a += factor[n] * (double)G[(size_t)n * P + i];
        acc[i] += a;
    }
}

/* ------------------------------------------------------------------------- */
/* Noise: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) + Box-Muller.     */
/* The paper only asks for N(0, sigma^2 C^2); the generator and the bit       */
/* layout below are this library's contract.                                  */
/* ------------------------------------------------------------------------- */

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint64_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint64_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = 0xD2511F53ull * c0;     /* 32x32 -> 64 bit products */
        const uint64_t p1 = 0xCD9E8D57ull * c2;
        const uint64_t n0 = ((p1 >> 32) ^ c1 ^ k0) & 0xffffffffull;
        const uint64_t n1 = p1 & 0xffffffffull;
        const uint64_t n2 = ((p0 >> 32) ^ c3 ^ k1) & 0xffffffffull;
        const uint64_t n3 = p0 & 0xffffffffull;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 = (k0 + 0x9E3779B9ull) & 0xffffffffull;  /* Weyl key schedule */
        k1 = (k1 + 0xBB67AE85ull) & 0xffffffffull;
    }
    out[0] = (uint32_t)c0; out[1] = (uint32_t)c1; out[2] = (uint32_t)c2; out[3] = (uint32_t)c3;
}

/* raw words of block j: counter = (j lo, j hi, step lo, step hi), key = (seed lo, seed hi) */
void oracle_philox_block(uint64_t seed, uint64_t step, uint64_t block, uint32_t out[4])
{
    const uint32_t ctr[4] = {(uint32_t)block, (uint32_t)(block >> 32), (uint32_t)step, (uint32_t)(step >> 32)};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    oracle_philox4x32_10(ctr, key, out);
}

/* the two uniforms of a Box-Muller pair: u1 in (0,1), u2 in [0,1), both exact in fp32 */
static void uniforms(uint32_t ra, uint32_t rb, double *u1, double *u2)
{
    *u1 = ((double)(ra >> 9) + 0.5) * (1.0 / 8388608.0);   /* 2^-23 */
    *u2 = (double)(rb >> 8) * (1.0 / 16777216.0);          /* 2^-24 */
}

/* z_i for global parameter index i.
 * index i -> block i/4, lane i%4; words (0,1) give lanes 0 (cos) and 1 (sin),
 * words (2,3) give lanes 2 (cos) and 3 (sin). */
static double noise_z_one(uint64_t seed, uint64_t step, uint64_t i)
{
    const double two_pi = 6.283185307179586476925286766559;
    uint32_t w[4];
    oracle_philox_block(seed, step, i >> 2, w);
    const int lane = (int)(i & 3);
    double u1, u2;
    uniforms(w[lane & 2], w[(lane & 2) + 1], &u1, &u2);
    const double radius = sqrt(-2.0 * log(u1));
    return (lane & 1) ? radius * sin(two_pi * u2) : radius * cos(two_pi * u2);
}

/* z[t] for global parameter indices first_index .. first_index+count-1 */
void oracle_noise_z(uint64_t seed, uint64_t step, uint64_t first_index, size_t count, double *z)
{
#pragma omp parallel for
    for (size_t t = 0; t < count; ++t) z[t] = noise_z_one(seed, step, first_index + t);
}

/* out[i] = (acc[i] + sigma*C*z_{offset+i}) / total_batch   (equation for g_t).
 * sigma = 0 means "no noise term" whatever C is (C = +inf with sigma = 0 is the
 * non-private average; 0 * inf must not poison it). */
void oracle_noise_average(const double *acc, size_t P, uint64_t param_offset, double sigma, double C,
                          double total_batch, uint64_t seed, uint64_t step, double *out)
{
#pragma omp parallel for
    for (size_t i = 0; i < P; ++i) {
        const double noise = (sigma == 0.0) ? 0.0 : sigma * C * noise_z_one(seed, step, param_offset + i);
        out[i] = (acc[i] + noise) / total_batch;
    }
}

/* Parameter update that consumes g_t (section 2: "gradients are then used to update the parameters via SGD"; the
 * CIFAR experiments add momentum 0.9).  Heavy-ball form, no dampening, no Nesterov:
 *     m <- mu * m + g        theta <- theta - lr * m        (mu = 0: plain SGD, m is then just g) */
void oracle_sgd_update(const double *g, size_t P, double lr, double mu, double *theta, double *m)
{
    for (size_t i = 0; i < P; ++i) {
        const double v = (m ? mu * m[i] : 0.0) + g[i];
        if (m) m[i] = v;
        theta[i] -= lr * v;
    }
}

/* The paper's own variant (section 2, the align block after the equation for g_t): every clipped example gets
 * its own noise of variance sigma^2 C^2 / |B| before accumulation, which is equal in distribution to one draw of
 * variance sigma^2 C^2 on the sum.  Example e of the step draws from its own stream: the Philox counter carries
 * (lo32(g/4), 0x80000000 | e, step lo, step hi) for global parameter index g, same key, same Box-Muller lanes. */
static double example_noise_z_one(uint64_t seed, uint64_t step, uint32_t example, uint64_t g)
{
    const double two_pi = 6.283185307179586476925286766559;
    const uint32_t ctr[4] = {(uint32_t)(g >> 2), 0x80000000u | example, (uint32_t)step, (uint32_t)(step >> 32)};
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    const int lane = (int)(g & 3);
    double u1, u2;
    uniforms(w[lane & 2], w[(lane & 2) + 1], &u1, &u2);
    const double radius = sqrt(-2.0 * log(u1));
    return (lane & 1) ? radius * sin(two_pi * u2) : radius * cos(two_pi * u2);
}

void oracle_example_noise_z(uint64_t seed, uint64_t step, uint32_t example, uint64_t first_index, size_t count, double *z)
{
    for (size_t t = 0; t < count; ++t) z[t] = example_noise_z_one(seed, step, example, first_index + t);
}

/* acc[i] += sum_n ( factor[n] * G[n,i] + sd * z_{example0+n}(param_offset + i) ),  sd = sigma*C/sqrt(|B|) */
void oracle_clip_accumulate_noised_f32(const float *G, int B, size_t P, const double *factor, double sd, uint64_t seed,
                                       uint64_t step, uint32_t example0, uint64_t param_offset, double *acc)
{
#pragma omp parallel for
    for (size_t i = 0; i < P; ++i) {
        double a = 0.0;
        for (int n = 0; n < B; ++n)
            a += factor[n] * (double)G[(size_t)n * P + i] +
                 (sd == 0.0 ? 0.0 : sd * example_noise_z_one(seed, step, example0 + (uint32_t)n, param_offset + i));
        acc[i] += a;
    }
}

// Internal launch interface of the CUDA-core per-example weight-gradient kernels.
#pragma once
#include "common.cuh"

namespace dp {

struct ConvGeom {
    int B, H, W, Cin, Kout, R, S, stride, pad, OH, OW;
    int M;   // Kout                     (rows of the per-example gradient matrix)
    int N;   // R*S*Cin                  (columns)
    int K;   // OH*OW                    (reduction length per example)
};

constexpr int kFmaTile = 64;          // output tile edge of the CUDA-core kernel
constexpr int kBiasCols = 64;         // output channels per bias-reduction block

inline int fma_tiles_m(const ConvGeom &g) { return (g.M + kFmaTile - 1) / kFmaTile; }
inline int fma_tiles_n(const ConvGeom &g) { return (g.N + kFmaTile - 1) / kFmaTile; }
inline int bias_blocks(const ConvGeom &g) { return (g.Kout + kBiasCols - 1) / kBiasCols; }

// mode: 0 store + norm partials, 1 norm partials only, 2 clip-accumulate (factor[n*2] scales example n).
// Mode 2 cuts the batch into fma_clip_splits(g) example ranges; with more than one range the partial sums go
// through sum_ws ([splits][M*N] floats) and are folded into acc_w in range order.
int fma_clip_splits(const ConvGeom &g);
dp_status launch_conv_fma(int dtype, int mode, const void *X, const void *dY, const ConvGeom &g, float *G_w,
                          float *partial, int slots, const float *factor, float *acc_w, float *sum_ws,
                          cudaStream_t stream);
// Thin convolutions (at most 32 gradient columns, 32 or 64 output channels, input of one example fits shared memory):
// gradient (G_w may be null), bias gradient and both squared norms in one launch; partial slot 0 = weights, 1 = bias.
bool thin_conv_eligible(const ConvGeom &g);
dp_status launch_conv_thin(int dtype, const void *X, const void *dY, const ConvGeom &g, float *G_w, float *db,
                           float *partial, int slots, int has_bias, cudaStream_t stream);
// 3x3 convolutions on three input channels with a multiple of 32 output channels: gradient (G_w may be null), bias
// gradient and the published squared norms (sqnorm[n*sq_stride + {0,1}] when `separate`, else their sum) in one launch.
bool rgb3_conv_eligible(const ConvGeom &g);
dp_status launch_conv_rgb3(int dtype, const void *X, const void *dY, const ConvGeom &g, float *G_w, float *db,
                           int has_bias, int separate, float *sqnorm, long long sq_stride,
                           cudaStream_t stream);
// db[n,k] = sum over pixels of dY; also sum_k db^2 per block into partial[n*slots + slot0 + block]
dp_status launch_bias(int dtype, const void *dY, const ConvGeom &g, float *db, float *partial, int slots, int slot0,
                      cudaStream_t stream);
// folds the partial slots of every example into sqnorm (and clip factors when clip != 0)
dp_status launch_finalize(const float *partial, int B, int slots, int w_slots, int separate, float *sqnorm,
                          long long sq_stride, int clip, float C_l, float *factor, float *clip_out,
                          cudaStream_t stream);
// acc_b[k] += sum_n factor[n*2+which] * db[n,k]
dp_status launch_bias_accum(const float *db, int B, int Kout, const float *factor, float *acc_b, cudaStream_t stream,
                            int which = 1);
// dense layer: acc_w[o, i] += sum_n factor[n*f_stride] * dY[n, o] * X[n, i]; with acc_b also (same launch)
// acc_b[o] += sum_n factor_b[n*fb_stride] * dY[n, o]
dp_status launch_dense_scaled_sum(int dtype, const void *X, const void *dY, const float *factor, long long f_stride, int B,
                                  int Cin, int Kout, float *acc_w, cudaStream_t stream, const float *factor_b = nullptr,
                                  long long fb_stride = 0, float *acc_b = nullptr);
// factor2[n] = (factor_w[n*stride], factor_b[n*stride])
dp_status launch_expand_factor(const float *factor_w, const float *factor_b, long long stride, int B, float *factor2,
                               cudaStream_t stream);

dp_status launch_dense_store(int dtype, const void *X, const void *dY, int B, int Cin, int Kout, float *G_w,
                             float *G_b, cudaStream_t stream);
// closed-form squared norms (|dY_n|^2 |X_n|^2 and |dY_n|^2), db = dY as fp32 (optional), norms and clip factors published
dp_status launch_dense_norm(int dtype, const void *X, const void *dY, int B, int Cin, int Kout, int has_bias, float *db,
                            int separate, float *sqnorm, long long sq_stride, int clip, float C_l, float *factor,
                            float *clip_out, cudaStream_t stream);

// stage 1: per pixel-chunk partial sums; stage 2: fold, store, squared norms into partial2[n*2 + {0,1}]
dp_status launch_norm_affine(int dtype, const void *X, const void *dY, int B, int HW, int C, float *chunk_partial,
                             float *dgamma, float *dbeta, float *partial2, cudaStream_t stream);

// One-launch form of the normalisation layer (see the kernel): needs B + 1 cleared ticket counters.
bool affine_fused_eligible(int B);
dp_status launch_norm_affine_fused(int dtype, const void *X, const void *dY, int B, int HW, int C, float *chunk_partial,
                                   float *dgamma, float *dbeta, float *factor, int *counters, int clip, float C_l,
                                   int separate, float *sqnorm, long long sq_stride, float *clip_out, float *acc_w,
                                   float *acc_b, cudaStream_t stream);

// fused: factors from partial2 (two squared norms per example), publish norms / factors, accumulate both tensors
dp_status launch_affine_clip_accum(const float *partial2, int B, float C_l, int separate, float *sqnorm, long long sq_stride,
                                   float *clip_out, const float *dgamma, const float *dbeta, int C, float *acc_w,
                                   float *acc_b, cudaStream_t stream);

// Shape of the norm-affine reduction: channel vectors per block (tcv) and pixels per block (pix).  Starts from whole
// channel rows and 256 pixels and narrows both until the grid has a couple of blocks per SM, so that layers with
// many channels on few pixels (2048 x 7 x 7) do not run on a handful of blocks.
inline void norm_shape(int dtype, int B, int HW, int C, int &vec, int &tcv, int &pix) {
    vec = (dtype == DP_F32) ? ((C & 3) ? 1 : 4) : ((C & 7) ? 1 : 8);
    const int cv = (C + vec - 1) / vec;
    tcv = cv < 256 ? cv : 256;
    pix = 256;
    auto blocks = [&]() { return (long long)((cv + tcv - 1) / tcv) * ((HW + pix - 1) / pix) * B; };
    if (blocks() < 296 && tcv > 32) tcv = 32;
    while (blocks() < 296 && pix > 32) pix /= 2;
}
inline int norm_chunks(int dtype, int B, int HW, int C) {
    int vec, tcv, pix;
    norm_shape(dtype, B, HW, C, vec, tcv, pix);
    return (HW + pix - 1) / pix;
}

}  // namespace dp

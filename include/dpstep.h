/*
 * dpstep.h -- C ABI of the DPSGD gradient-privatisation step for one NVIDIA B200 (sm_100a).
 *
 * The step (paper section 2, "Algorithm", equation for g_t):
 *
 *     g_t = ( N(0, sigma^2 C^2 I) + sum_{x_j in B} clip(grad L(theta, x_j), C) ) / |B|
 *
 * with clip(g, C) = g * min(1, C / ||g||_2), the batch B reached by accumulating chunks
 * of examples (section 2, "gradient accumulation"), and optionally each of M parameter
 * groups clipped on its own to C / sqrt(M) (section 3.5).
 *
 * General rules for every entry point
 *   - Every data pointer is a DEVICE pointer unless its comment says "host".  All device
 *     buffers are allocated, owned and freed by the caller; the library allocates no
 *     device memory and keeps no state between calls (scratch comes in as `workspace`).
 *     One exception, stated at its declaration: dp_clip_accumulate_static works in a fixed
 *     device array that is part of the library image.
 *   - Device pointers must be 16-byte aligned; tensors are dense, row-major, channels-last:
 *       conv   X [B,H,W,C_in]   dY [B,OH,OW,K_out]   G_w [B,K_out,R,S,C_in]   G_b [B,K_out]
 *       dense  X [B,C_in]       dY [B,K_out]         G_w [B,K_out,C_in]       G_b [B,K_out]
 *       norm   X = normalised activation [B,H,W,C_in], dY [B,H,W,C_in], G_w = dgamma [B,C_in],
 *              G_b = dbeta [B,C_in]
 *     with OH = (H + 2*pad - R)/stride + 1 (integer division), likewise OW.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising.  Arguments are validated on the host
 *     before anything is launched; on error nothing has been launched.
 *   - Functions return a dp_status; they never abort, throw or print.
 */
#ifndef DPSTEP_H
#define DPSTEP_H

#include <stddef.h>

#if defined(__GNUC__)
#define DP_API __attribute__((visibility("default")))
#else
#define DP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DP_OK = 0,
    DP_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, non-positive size, bad enum, bad C or sigma */
    DP_ERR_UNSUPPORTED = 2,   /* a valid request this build has no kernel for */
    DP_ERR_WORKSPACE = 3,     /* workspace missing, misaligned or smaller than dp_workspace_bytes() */
    DP_ERR_CUDA = 4,          /* a CUDA runtime / driver call or a launch failed */
    DP_ERR_TIMEOUT = 5        /* a bounded device-side wait gave up (reported through dp_wgrad_check) */
} dp_status;

typedef enum {
    DP_F32 = 0,               /* X and dY are fp32; tensor-core layers run them as three tf32 products of a hi/lo split
                                 (error about 4e-6 relative), everything else in plain fp32 */
    DP_BF16 = 1,              /* X and dY are bf16, products exact in fp32 */
    DP_TF32 = 2               /* X and dY are fp32; tensor-core layers round them to tf32 (nearest even) and run ONE
                                 product: per-example norms stay within 1e-4, gradients within 2e-3 relative L2, at
                                 two thirds of the shared-memory traffic and a third of the tensor work of DP_F32.
                                 Layers that do not run on tensor cores behave exactly as under DP_F32. */
} dp_dtype;                   /* every output is fp32 */
typedef enum { DP_LAYER_DENSE = 0, DP_LAYER_CONV2D = 1, DP_LAYER_NORM_AFFINE = 2 } dp_layer_kind;
typedef enum { DP_CLIP_GLOBAL = 0, DP_CLIP_PER_LAYER = 1 } dp_clip_mode;
typedef enum {
    DP_EPI_STORE_NORM = 0,    /* write per-example gradients G_w (and G_b) and sqnorm[B]          */
    DP_EPI_NORM_ONLY = 1,     /* write sqnorm[B] only; no per-example gradient reaches memory     */
    DP_EPI_CLIP_ACCUM = 2     /* clip each example of this layer to C_l and add the sum to acc    */
} dp_epilogue;
typedef enum {
    DP_IMPL_AUTO = 0,         /* tensor-core kernel when the shape allows it, else the CUDA-core one */
    DP_IMPL_CUDA_CORE = 1,    /* force the fp32 FMA kernel (any shape)                              */
    DP_IMPL_TENSOR_CORE = 2   /* force the tcgen05 kernel; DP_ERR_UNSUPPORTED if the shape is not eligible */
} dp_impl;

typedef struct {
    int kind;                 /* dp_layer_kind */
    int dtype;                /* dp_dtype of X and dY */
    int B;                    /* examples in this chunk, >= 1 */
    int C_in, H, W;           /* input channels and spatial size (dense: H = W = 1) */
    int K_out, R, S;          /* output channels and filter size (dense: R = S = 1; norm: K_out = C_in, R = S = 1) */
    int stride, pad;          /* conv only (dense / norm: 1, 0); dilation 1 and groups 1 are the only ones built */
    int has_bias;             /* conv / dense: 1 if a bias gradient is wanted; norm: ignored, dbeta always exists */
    int bias_separate;        /* 0: weight and bias form ONE parameter group (one norm, one clip factor per example);
                                 1: they are TWO groups (section 3.5 counts parameter tensors), so sqnorm and
                                    clip_out carry two values per example: (weight, bias) */
    int impl;                 /* dp_impl */
} dp_layer_desc;

/* Number of parameter groups the layer reports per example: 2 when bias_separate != 0 and the
 * layer has a bias-like tensor, else 1 (0 for an invalid descriptor). */
DP_API int dp_layer_groups(const dp_layer_desc *desc);

/* Bytes of device scratch dp_per_example_wgrad needs for this layer and epilogue
 * (0 for an invalid descriptor).  The scratch holds per-tile partial squared norms and,
 * for some paths, per-example bias gradients or clip factors. */
DP_API size_t dp_workspace_bytes(const dp_layer_desc *desc, int epilogue);

/* How many SMs one tensor-core launch of dp_per_example_wgrad(_scaled) should spread over (0 = all, the default).
 * A chunk of few examples gives one layer only a few microseconds of work for a whole GPU, most of which a launch then
 * spends starting and draining; a caller that runs several layer calls side by side on different streams gets more
 * out of the GPU when each call takes a share of the SMs and keeps them busy for longer.  The value is process-wide,
 * applies to launches made afterwards, and changes nothing but speed: results do not depend on it bit for bit only
 * within one setting (the fused clipped sum splits the batch over thread blocks by it), so keep it fixed for a run that
 * must be reproducible.  Workspace sizes depend on it: query dp_workspace_bytes after setting it.
 * Errors: DP_ERR_INVALID_ARG for a negative value. */
DP_API dp_status dp_set_sm_target(int sms);

/* Prepares a freshly allocated (or otherwise overwritten) workspace of dp_per_example_wgrad /
 * dp_per_example_wgrad_scaled: clears its header, i.e. the status word dp_wgrad_check reports and the ticket
 * counters with which the last thread block to finish an example finds out that it is the last.  Call it once
 * per workspace before the first layer call (it enqueues one small memset on `cuda_stream`); the layer calls
 * leave the counters cleared again, so one workspace serves any number of calls, of any layers, one after the
 * other.  Between calls the caller must not write to the workspace.
 * Errors: DP_ERR_WORKSPACE (null, not 256-byte aligned, or smaller than any dp_workspace_bytes() result). */
DP_API dp_status dp_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Per-example weight gradients of one layer for a chunk of B examples
 * (section 2: "per-example gradients are computed"; the layer formulas are the standard
 * weight gradients given X and dY):
 *     conv   G_w[n,k,r,s,c] = sum_{oh,ow} dY[n,oh,ow,k] * Xpad[n, oh*stride+r-pad, ow*stride+s-pad, c]
 *            G_b[n,k]       = sum_{oh,ow} dY[n,oh,ow,k]
 *     dense  G_w[n,o,i] = dY[n,o] * X[n,i];   G_b[n,o] = dY[n,o]
 *     norm   G_w[n,c] = sum_{h,w} dY[n,h,w,c] * X[n,h,w,c];   G_b[n,c] = sum_{h,w} dY[n,h,w,c]
 * and the squared L2 norm of each example's gradient of this layer, taken from the accumulators
 * before they leave the chip (for the rank-1 dense gradient: the closed form |dY_n|^2 |X_n|^2).
 *
 *   X, dY      inputs, type desc->dtype.
 *   G_w, G_b   [B, P_w], [B, P_b] fp32 outputs; required for DP_EPI_STORE_NORM (G_b only when
 *              the layer has a bias), ignored otherwise.
 *   sqnorm     fp32 output, always written: sqnorm[n*sqnorm_stride + g] for example n and group g
 *              (g < dp_layer_groups()); sqnorm_stride >= groups lets a layer write its column(s) of the
 *              [B, L] table dp_clip_accumulate reads.
 *   C_l        clip threshold of this layer, used by DP_EPI_CLIP_ACCUM only (> 0, +inf allowed).
 *   acc_w/b    [P_w], [P_b] fp32, read-modify-write; DP_EPI_CLIP_ACCUM only:
 *              acc += sum_n min(1, C_l/||g_n||) * g_n  (section 3.5, one group = this layer).
 *   clip_out   optional [B, groups] fp32: the factors that were applied (DP_EPI_CLIP_ACCUM).
 *   workspace  at least dp_workspace_bytes(desc, epilogue) bytes, 256-byte aligned, prepared once by
 *              dp_workspace_init.  Calls that may overlap on the GPU need a workspace each.  Usually a few hundred KB; layers
 *              with very few input channels (C_in <= 8) that run on tensor cores keep an unfolded copy of X there
 *              (B*OH*OW*pad(R*S*C_in) elements), and the fused clip keeps partial sums when it splits the batch.
 *
 * The first tensor-core call of a process raises a kernel attribute (shared-memory size); make one call of each
 * kind before capturing calls into a CUDA graph.
 * Results are bit-reproducible from run to run (fixed reduction orders, no float atomics).
 * Errors: DP_ERR_INVALID_ARG, DP_ERR_UNSUPPORTED, DP_ERR_WORKSPACE, DP_ERR_CUDA. */
DP_API dp_status dp_per_example_wgrad(const dp_layer_desc *desc, const void *X, const void *dY,
                               float *G_w, float *G_b, float *sqnorm, long long sqnorm_stride,
                               int epilogue, float C_l, float *acc_w, float *acc_b, float *clip_out,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* The clipped sum of one layer with the factors already known: acc_w += sum_n factor_w[n*factor_stride] * g_w,n and
 * acc_b += sum_n factor_b[n*factor_stride] * g_b,n, the per-example gradients formed on the fly and never written
 * (section 2: the sum over the batch of clip(g_j, C), whose factor min(1, C/||g_j||) needs every layer's norm first).
 * Together with DP_EPI_NORM_ONLY and dp_clip_factors this gives whole-model clipping without materialising a layer's
 * per-example gradients: the layer's inputs are read twice instead of its B gradients being written and read back,
 * which is cheaper whenever a gradient is larger than the inputs it comes from (late convolutions, dense layers).
 *
 *   factor_w, factor_b   device fp32, one value per example at stride factor_stride (>= 1).  factor_b = NULL uses
 *                        factor_w for the bias-like tensor too (whole-model clipping: one factor per example).
 *   acc_w, acc_b         [P_w], [P_b] fp32, read-modify-write (acc_b only when the layer has a bias-like tensor).
 *   workspace            at least dp_workspace_bytes(desc, DP_EPI_CLIP_ACCUM) bytes, 256-byte aligned.
 * Errors as for dp_per_example_wgrad. */
DP_API dp_status dp_per_example_wgrad_scaled(const dp_layer_desc *desc, const void *X, const void *dY,
                                             const float *factor_w, const float *factor_b, long long factor_stride,
                                             float *acc_w, float *acc_b, void *workspace, size_t workspace_bytes,
                                             void *cuda_stream);

/* Bytes of device scratch dp_clip_accumulate needs (per-block partial norms and factors). */
DP_API size_t dp_clip_workspace_bytes(int B, int L, const long long *P_l /* host, [L] */);

/* Norm, clip and accumulate over materialised per-example gradients
 * (section 2, the sum over x_j in B of clip(.,C); section 3.5 for the per-layer mode):
 *     GLOBAL     s_n = sum_l ||G_l[n]||^2,  f_n = min(1, C/sqrt(s_n)),            acc_l += sum_n f_n * G_l[n]
 *     PER_LAYER  s_{n,l} = ||G_l[n]||^2,    f_{n,l} = min(1, (C/sqrt(L))/sqrt(s_{n,l})), acc_l += sum_n f_{n,l} * G_l[n]
 * The factor is exactly 1 when s <= threshold^2 (so a zero gradient and C = +inf are safe).
 * Calling it once per chunk accumulates over chunks (section 2, gradient accumulation).
 *
 *   G        host array of L device pointers, G[l] = [B, P_l] fp32.  L = 1 is a flat [B, P] matrix.
 *   P_l      host array of L sizes (> 0).
 *   sqnorm   device [B, L] fp32 (row n holds the L per-tensor squared norms of example n, as
 *            written by dp_per_example_wgrad) or NULL, in which case the norms are computed
 *            here with one extra pass over G.
 *   C        clip norm of the whole gradient, > 0, +inf allowed.
 *   acc      host array of L device pointers, acc[l] = [P_l] fp32, read-modify-write.
 *   norms_out  optional device fp32: GLOBAL [B] whole-gradient L2 norms; PER_LAYER [B, L].
 *   clip_out   optional device fp32, same shape: the factors applied.
 *   workspace  at least dp_clip_workspace_bytes(B, L, P_l) bytes, 256-byte aligned. */
DP_API dp_status dp_clip_accumulate(int mode, int B, int L, const float *const *G, const long long *P_l,
                             const float *sqnorm, float C, float *const *acc,
                             float *norms_out, float *clip_out,
                             void *workspace, size_t workspace_bytes, void *cuda_stream);

/* dp_clip_accumulate with the noise added per example, before the sum (section 2, the block after the equation for
 * g_t: each clipped example receives its own draw of variance sigma^2 C^2 / |B|, which is equal in distribution to one
 * draw of variance sigma^2 C^2 on the sum; this is the form the paper's own implementation uses):
 *     acc_l[i] += sum_n ( f_n * G_l[n,i] + sd * z_{example0+n}(param_offset_l[l] + i) ),   sd = sigma*C/sqrt(total_batch)
 * with f_n as in dp_clip_accumulate (both modes).  After the last chunk the step ends with dp_noise_average(sigma = 0),
 * the plain division by |B|.
 * z_e(g) is example e's own stream: Philox4x32-10 with counter (lo32(g/4), 0x80000000 | e, lo32(step), hi32(step)),
 * key (lo32(seed), hi32(seed)), and the Box-Muller lanes of dp_noise_average; it depends only on
 * (seed, step, e, g), never on chunking or launch shape, and never meets the per-parameter stream of dp_noise_average.
 *
 *   param_offset_l  host array of L global indices: where each tensor starts in the model's parameter vector (>= 0,
 *                   offset + P_l <= 2^34).  Multiples of four take the fast path.
 *   sigma, C        sigma >= 0 (0 adds nothing); with sigma > 0, C must be finite.  C is always the whole-gradient
 *                   bound, also in PER_LAYER mode.
 *   total_batch     |B| of the whole step (all chunks, all ranks), > 0.
 *   example0        index within the step of this chunk's first example (>= 0, example0 + B <= 2^31); chunks of one
 *                   step must use disjoint ranges, or two examples would share a draw.
 * Everything else, and the errors, as for dp_clip_accumulate.  The work is B*P normals per chunk: arithmetic-bound,
 * where the once-per-step form costs P normals per step. */
DP_API dp_status dp_clip_accumulate_noised(int mode, int B, int L, const float *const *G, const long long *P_l,
                                           const long long *param_offset_l, const float *sqnorm, float C, float sigma,
                                           long long total_batch, unsigned long long seed, unsigned long long step,
                                           long long example0, float *const *acc, float *norms_out, float *clip_out,
                                           void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Test hook: the standard normals of example `example`'s stream for global indices first_index .. +count-1. */
DP_API dp_status dp_debug_example_noise_z(float *z, long long count, long long first_index, long long example,
                                          unsigned long long seed, unsigned long long step, void *cuda_stream);

/* The two halves of dp_clip_accumulate on their own, for steps that keep only some tensors' per-example gradients in
 * memory and form the others' clipped sums with dp_per_example_wgrad_scaled.
 *
 * dp_clip_factors: the factors from a table of squared norms (section 2 / 3.5, as in dp_clip_accumulate):
 *   sqnorm       device [B, L] fp32: per-tensor squared norms of every example (all L tensors of the model).
 *   factors_out  device fp32: GLOBAL [B], PER_LAYER [B, L].   norms_out  optional, same shape: the L2 norms.
 * dp_scale_accumulate: acc_l += sum_n f * G_l[n] with f = factor[n] (per_tensor = 0) or factor[n*L + l] (per_tensor = 1);
 *   G, P_l, acc as for dp_clip_accumulate.  Neither call needs a workspace. */
DP_API dp_status dp_clip_factors(int mode, int B, int L, const float *sqnorm, float C, float *norms_out,
                                 float *factors_out, void *cuda_stream);
DP_API dp_status dp_scale_accumulate(int B, int L, const float *const *G, const long long *P_l, const float *factor,
                                     int per_tensor, float *const *acc, void *cuda_stream);

/* dp_clip_accumulate with the parameter tensors gathered into M groups, each clipped on its own to C/sqrt(M)
 * (section 3.5: the groups are the paper's pipeline stages; no stage needs another stage's norm, and the bound on the
 * whole gradient stays C because the squares of the M bounds add up to C^2):
 *     s_{n,m} = sum over tensors l of group m of ||G_l[n]||^2,   f_{n,m} = min(1, (C/sqrt(M)) / sqrt(s_{n,m})),
 *     acc_l += sum_n f_{n,group_of[l]} * G_l[n].
 * One tensor per group is DP_CLIP_PER_LAYER, a single group is DP_CLIP_GLOBAL.
 *   group_of   host array of L group indices in [0, M); every group must own at least one tensor.  L <= 1024.
 *   sqnorm     device [B, L] per-tensor squared norms or NULL (computed here), as for dp_clip_accumulate.
 *   norms_out, clip_out   optional device [B, M]: the groups' L2 norms and factors.
 * Everything else, and the errors, as for dp_clip_accumulate. */
DP_API dp_status dp_clip_accumulate_grouped(int B, int L, int M, const int *group_of, const float *const *G,
                                            const long long *P_l, const float *sqnorm, float C, float *const *acc,
                                            float *norms_out, float *clip_out, void *workspace, size_t workspace_bytes,
                                            void *cuda_stream);

/* Micro-batch clipping (the option of the paper's first table, which the paper advises against: it trades accuracy for
 * speed): the B examples of the chunk form B/micro runs of `micro` consecutive examples; each run is averaged, the
 * average is clipped to C over the whole model and the clipped averages are added:
 *     gbar_j = (1/micro) sum_{n in run j} g_n,   f_j = min(1, C/||gbar_j||),   acc += sum_j f_j * gbar_j.
 * The unit that is clipped is the run, so the step ends with dp_noise_average(total_batch = number of runs).
 *   micro      >= 1, must divide B (1 is plain whole-model clipping).
 *   norms_out, clip_out   optional device [B/micro].
 * The norms are always computed here (a run's norm does not follow from its examples' norms): two passes over G.
 * Everything else, and the errors, as for dp_clip_accumulate in DP_CLIP_GLOBAL mode. */
DP_API dp_status dp_clip_accumulate_micro(int B, int L, int micro, const float *const *G, const long long *P_l, float C,
                                          float *const *acc, float *norms_out, float *clip_out, void *workspace,
                                          size_t workspace_bytes, void *cuda_stream);

/* dp_clip_accumulate for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this exists for deployment reasons only.)
 *
 * Some callers have no way to hand over a workspace: code running inside a framework whose caching
 * allocator already owns the whole device, plug-ins and callbacks that are forbidden to call cudaMalloc
 * because it synchronises the device, and services that pre-reserve every byte at start-up.  For them
 * the scratch of the norm / factor stages lives inside the library, in one fixed device array of
 * dp_clip_static_scratch_bytes() bytes (2 MiB) that every GPU loading the library holds until exit.
 * Arguments and results are those of dp_clip_accumulate without the workspace pair.
 *
 *   - Limit: problems whose dp_clip_workspace_bytes(B, L, P_l) exceeds the array are refused with
 *     DP_ERR_WORKSPACE (dp_last_cuda_error() says why); nothing is launched.
 *   - Every call looks up the array's device address (cudaGetSymbolAddress, with the caller's device current);
 *     the first look-up on a device loads the library image there, so make that first call outside any stream
 *     capture.  No call allocates or frees memory, and no address is kept across calls.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing in it has to start at
 *     zero (each call writes what it later reads), but two calls whose kernels overlap on the GPU -- different
 *     streams, or different host threads on the same device -- race on it: keep such calls ordered. */
DP_API dp_status dp_clip_accumulate_static(int mode, int B, int L, const float *const *G, const long long *P_l,
                                           const float *sqnorm, float C, float *const *acc,
                                           float *norms_out, float *clip_out, void *cuda_stream);

/* Size in bytes of the built-in scratch array dp_clip_accumulate_static works in. */
DP_API size_t dp_clip_static_scratch_bytes(void);

/* Noise and average (section 2): out[i] = (acc[i] + sigma * C * z_{param_offset+i}) / total_batch,
 * one pass, `out` may alias `acc`.  z is a standard normal that depends only on
 * (seed, step, global parameter index g = param_offset + i):
 *   Philox4x32-10 (Salmon et al., SC'11) with counter (lo32(g/4), hi32(g/4), lo32(step), hi32(step))
 *   and key (lo32(seed), hi32(seed)) gives words r0..r3;  for the pair (a,b) = (0,1) resp. (2,3):
 *   u1 = ((r_a >> 9) + 0.5) * 2^-23, u2 = (r_b >> 8) * 2^-24, radius = sqrt(-2 ln u1),
 *   lane g%4 = 0,2 takes radius*cos(2 pi u2), lane 1,3 takes radius*sin(2 pi u2).
 * sigma = 0 adds nothing, whatever C is; with sigma > 0, C must be finite.
 * seed and step are call arguments: a call captured into a CUDA graph keeps the values it was captured with, so
 * replaying it repeats the same draw.  Keep this call outside graphs that are replayed across training steps (or
 * update the kernel node's parameters), or every step gets the same noise and the privacy guarantee is void.
 * In per-layer mode C is still the whole-gradient bound (the per-group thresholds are chosen so
 * that the whole gradient keeps sensitivity C).
 * Errors: DP_ERR_INVALID_ARG for P <= 0, param_offset < 0, total_batch <= 0, sigma < 0, C <= 0. */
DP_API dp_status dp_noise_average(const float *acc, long long P, long long param_offset,
                           float sigma, float C, long long total_batch,
                           unsigned long long seed, unsigned long long step,
                           float *out, void *cuda_stream);

/* dp_noise_average fused with the parameter update that consumes its result (section 2: the noised, averaged
 * gradient is "used to update the parameters via SGD"; the CIFAR experiments use momentum 0.9):
 *     g_i = (acc[i] + sigma*C*z_{param_offset+i}) / total_batch
 *     m_i <- momentum * m_i + g_i      (only when momentum_buf is given; heavy ball, no dampening, no Nesterov)
 *     theta_i <- theta_i - lr * m_i    (or - lr * g_i without a momentum buffer)
 * One pass over the parameters instead of two.  theta [P] and momentum_buf [P] (optional) are fp32, read-modify-write;
 * g_out [P] is optional and receives g.  Noise stream, argument rules and errors as for dp_noise_average; lr and
 * momentum must be finite, momentum >= 0. */
DP_API dp_status dp_noise_average_sgd(const float *acc, long long P, long long param_offset,
                               float sigma, float C, long long total_batch,
                               unsigned long long seed, unsigned long long step,
                               float lr, float momentum, float *theta, float *momentum_buf, float *g_out,
                               void *cuda_stream);

/* Test hook: the raw Philox words of blocks first_block .. first_block+n_blocks-1 of the
 * (seed, step) stream described above, out4 = [n_blocks, 4] uint32 on the device. */
DP_API dp_status dp_debug_philox_raw(unsigned int *out4, long long n_blocks, long long first_block,
                              unsigned long long seed, unsigned long long step, void *cuda_stream);

/* Test hook: the standard normals z_g for g = first_index .. first_index+count-1, fp32 on the device. */
DP_API dp_status dp_debug_noise_z(float *z, long long count, long long first_index,
                           unsigned long long seed, unsigned long long step, void *cuda_stream);

/* Reads (with a synchronising copy) the status word at the start of `workspace`: DP_OK, or DP_ERR_TIMEOUT when
 * a bounded wait inside a tensor-core kernel expired in ANY call that used this workspace since the word was last
 * cleared (that kernel returned early; its outputs, and everything computed from them, are invalid).  The word is
 * sticky: kernels only ever set it, later calls do not hide it.  Reporting a time-out clears it and re-initialises
 * the workspace header, as dp_workspace_init does. */
DP_API dp_status dp_wgrad_check(void *workspace, void *cuda_stream);

/* Test hook: 0 makes DP_EPI_CLIP_ACCUM always run its two-pass form (norm pass, then clipped sum), 1 (the default)
 * lets layers whose per-example gradient fits one thread-block cluster run the single-pass form.  Process-wide. */
DP_API void dp_debug_set_single_pass(int on);

/* Test hook: the number of polls (each about a microsecond) after which the bounded waits of the tensor-core kernel
 * give up; 0 makes every wait give up before anything is copied or multiplied, a negative value restores the
 * default (about two seconds).  Process-wide; applies to launches enqueued afterwards. */
DP_API void dp_debug_set_wait_polls(long long polls);

/* 1 if dp_per_example_wgrad would run this layer on the tcgen05 tensor-core kernel under
 * DP_IMPL_AUTO, else 0 (also 0 for an invalid descriptor). */
DP_API int dp_wgrad_uses_tensor_cores(const dp_layer_desc *desc, int epilogue);

DP_API const char *dp_status_string(int status);

/* Text of the last CUDA error this thread's calls ran into ("" if none). Host memory owned by the library. */
DP_API const char *dp_last_cuda_error(void);

/* Test / report hook: the tiling the tensor-core kernel would use for a conv layer and epilogue, as up to 12 ints
 * {rows-are-input-columns, row extent, column extent, row tiles, column tiles, columns per tile,
 *  pixel-tile width, pixel-tile height, pixels per stage, pixel tiles, pipeline stages, bytes per stage}.
 * `epilogue` is a dp_epilogue value, or 3 (the fused clip as one contraction per cluster), 4 (the clipped sum as one
 * product over all examples) or 5 (norms from the pixel Gram matrices: row and column extent = pixels of the box,
 * pixel tiles = loads per row tile).
 * Returns the number of values available (0 when the layer is not eligible). `out` is host memory. */
DP_API int dp_debug_wgrad_plan(const dp_layer_desc *desc, int epilogue, int *out, int n);

/* Number of kernels this process has launched through the library so far (a host-side counter;
 * benchmarks report the difference over their timed region). */
DP_API unsigned long long dp_debug_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DPSTEP_H */

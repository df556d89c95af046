// Internal launch interface of the tcgen05 (5th-generation tensor core) per-example conv weight-gradient kernel.
#pragma once
#include "wgrad_simple.cuh"

namespace dp {

// true when the layer can run on the tensor-core kernel (channel counts, sizes and TMA alignment rules)
bool tc_eligible(int dtype, const ConvGeom &g, int epilogue);
// number of per-example partial squared-norm slots the kernel writes
int tc_norm_slots(int dtype, const ConvGeom &g, int epilogue);
size_t tc_workspace_bytes(int dtype, const ConvGeom &g, int epilogue);
// tiling chosen for the layer: {a_is_x, a_ext, b_ext, m_tiles, n_tiles, NT, OWt, OHt, Kt, k_tiles, stages, stage_bytes}
// acc[i] += sum_s part[s][i] in index order of s (P a multiple of 4)
dp_status launch_fold_partial_sums(const float *part, int splits, long long P, float *acc, cudaStream_t stream);
int tc_describe_plan(int dtype, const ConvGeom &g, int epilogue, int *out, int n);
// When given to a CLIP_ACCUM launch, the kernel derives each example's factor from the norm pass's partial sums
// itself (threshold C_l) and writes sqnorm[n*sq_stride] and clip_out[n] (optional), so no finalising launch is needed.
struct TcInlineClip { float C_l; float *sqnorm; long long sq_stride; float *clip_out; };

// When given to a STORE_NORM / NORM_ONLY launch, the last CTA to finish folds every example's partial squared norms
// (slots [0, w_slots) = weights, the rest = bias, written earlier in the stream) and writes sqnorm[n*sq_stride]
// (+1 for the bias when `separate`), so no finalising launch is needed.  counters: one cleared ticket word.
// factor_out (optional): also the clip factors against C_l, [B][2] = (weight, bias), and clip_out as dp_per_example_wgrad defines it.
struct TcPublish { int *counters; int w_slots; int separate; float *sqnorm; long long sq_stride; float *factor_out; float C_l; float *clip_out; };

// epilogue as dp_epilogue; factor[n*2] scales example n (CLIP_ACCUM); status: device word set to nonzero on a timed-out wait
dp_status launch_conv_tc(int dtype, int epilogue, const void *X, const void *dY, const ConvGeom &g, float *G_w,
                         float *partial, int slots, const float *factor, float *acc_w, void *tc_workspace,
                         int *status, cudaStream_t stream, bool second_pass = false,
                         const TcInlineClip *inline_clip = nullptr, const TcPublish *publish = nullptr);

// The fused clipped sum of a bf16 layer whose per-example gradient fits the tensor memory of one thread-block cluster
// runs as ONE contraction (norm, factor and scaled sum from the same accumulators); tc_clip_single_pass says whether
// this layer qualifies.  Writes sqnorm / clip_out like a CLIP_ACCUM launch with TcInlineClip; layers without bias only.
bool tc_clip_single_pass(int dtype, const ConvGeom &g);
dp_status launch_conv_clip1(int dtype, const void *X, const void *dY, const ConvGeom &g, float *partial, int slots,
                            const TcInlineClip &clipinfo, float *acc_w, void *tc_workspace, int *status, cudaStream_t stream);

// bf16 layers too large for one cluster: after the norm pass has published the factors (factor[2n]), the clipped sum is
// ONE matrix product over all examples with f_n dY split into hi + lo bf16 copies (kept in tc_workspace).  No bias, not unfolded.
bool tc_clip_scaled_sum(int dtype, const ConvGeom &g);
dp_status launch_conv_ssum(int dtype, const void *X, const void *dY, const ConvGeom &g, const float *factor, float *acc_w,
                           void *tc_workspace, int *status, cudaStream_t stream);

// The same clipped sum with known factors, per example through tensor memory (one tile per CTA, an example range per
// CTA, each finished tile read once and scaled into registers): the better form when an example has 128 pixels or more.
bool tc_clip_scaled_tiles(int dtype, const ConvGeom &g);
dp_status launch_conv_scaled_tiles(int dtype, const void *X, const void *dY, const ConvGeom &g, const float *factor, float *acc_w,
                                   void *tc_workspace, int *status, cudaStream_t stream);

// bf16 layers whose whole output plane is at most 256 pixels: per-example squared norms (and factors against
// clipinfo.C_l into factor_out[2n], factor_out[2n+1], when given) from the Gram matrices of dY and of the unfolded
// input over the pixels, without forming the gradient.  Weight group only; not for unfolded layers.
bool tc_gram_norm(int dtype, const ConvGeom &g);
dp_status launch_conv_gram_norm(int dtype, const void *X, const void *dY, const ConvGeom &g, const TcInlineClip &clipinfo,
                                float *factor_out, int *status, cudaStream_t stream);

// Test hook: the number of polls after which a bounded wait of the kernel gives up (0 makes every wait give up at once).
void set_wait_polls(uint32_t polls);
uint32_t default_wait_polls();

}  // namespace dp

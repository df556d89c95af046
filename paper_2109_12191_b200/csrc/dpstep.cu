// Host side of dp_per_example_wgrad: argument checks, workspace layout, and the choice between
// the tcgen05 tensor-core kernel and the CUDA-core kernels.
#include "wgrad_simple.cuh"
#include "wgrad_tc.cuh"
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <atomic>

namespace dp {

static thread_local char g_last_error[256] = "";
static std::atomic<unsigned long long> g_launches{0};

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

dp_status cuda_fail(cudaError_t e, const char *where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    return DP_ERR_CUDA;
}

void note_error(const char *message) { snprintf(g_last_error, sizeof(g_last_error), "%s", message); }

static std::atomic<int> g_sm_target{0};
static std::atomic<int> g_single_pass{1};
bool single_pass_enabled() { return g_single_pass.load(std::memory_order_relaxed) != 0; }

bool sm_target_set() { return g_sm_target.load(std::memory_order_relaxed) > 0; }

int sm_target() {
    const int all = sm_count(), t = g_sm_target.load(std::memory_order_relaxed);
    return (t > 0 && t < all) ? t : all;
}

int sm_count() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v > 0) return v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    cached[dev].store(v, std::memory_order_relaxed);
    return v;
}

static bool valid_desc(const dp_layer_desc *d) {
    if (!d) return false;
    if (d->kind != DP_LAYER_DENSE && d->kind != DP_LAYER_CONV2D && d->kind != DP_LAYER_NORM_AFFINE) return false;
    if (d->dtype != DP_F32 && d->dtype != DP_BF16 && d->dtype != DP_TF32) return false;
    if (d->impl != DP_IMPL_AUTO && d->impl != DP_IMPL_CUDA_CORE && d->impl != DP_IMPL_TENSOR_CORE) return false;
    if (d->B <= 0 || d->C_in <= 0 || d->K_out <= 0 || d->H <= 0 || d->W <= 0) return false;
    if (d->kind == DP_LAYER_CONV2D) {
        if (d->R <= 0 || d->S <= 0 || d->stride <= 0 || d->pad < 0) return false;
        if (d->H + 2 * d->pad < d->R || d->W + 2 * d->pad < d->S) return false;
    } else {
        if (d->R != 1 || d->S != 1 || d->stride != 1 || d->pad != 0) return false;
        if (d->kind == DP_LAYER_DENSE && (d->H != 1 || d->W != 1)) return false;
        if (d->kind == DP_LAYER_NORM_AFFINE && d->K_out != d->C_in) return false;
    }
    return true;
}

static ConvGeom geom_of(const dp_layer_desc *d) {
    ConvGeom g;
    g.B = d->B; g.H = d->H; g.W = d->W; g.Cin = d->C_in; g.Kout = d->K_out; g.R = d->R; g.S = d->S;
    g.stride = d->stride; g.pad = d->pad;
    g.OH = (d->H + 2 * d->pad - d->R) / d->stride + 1;
    g.OW = (d->W + 2 * d->pad - d->S) / d->stride + 1;
    g.M = d->K_out; g.N = d->R * d->S * d->C_in; g.K = g.OH * g.OW;
    return g;
}

// Element type of X and dY in memory: DP_TF32 only changes the arithmetic of the tensor-core kernel.
static int storage_type(const dp_layer_desc *d) { return d->dtype == DP_TF32 ? DP_F32 : d->dtype; }

static bool has_bias_tensor(const dp_layer_desc *d) { return d->kind == DP_LAYER_NORM_AFFINE || d->has_bias != 0; }
static int groups_of(const dp_layer_desc *d) { return (d->bias_separate && has_bias_tensor(d)) ? 2 : 1; }

struct WgradPlan {
    bool use_tc, use_thin;
    int slots, w_slots;
    size_t status_off, partial_off, factor_off, db_off, chunk_off, dg_off, tc_off, total;
};

static bool make_plan(const dp_layer_desc *d, int epi, WgradPlan &pl) {
    const ConvGeom g = geom_of(d);
    const size_t B = (size_t)d->B;
    pl.use_tc = false;
    pl.use_thin = d->kind == DP_LAYER_CONV2D && d->impl == DP_IMPL_AUTO && epi != DP_EPI_CLIP_ACCUM && thin_conv_eligible(g);
    if (d->kind == DP_LAYER_CONV2D && d->impl != DP_IMPL_CUDA_CORE && !pl.use_thin) pl.use_tc = tc_eligible(d->dtype, g, epi);
    size_t off = 0;
    pl.status_off = off; off += kWsHeaderBytes;      // status word, then the ticket counters
    if (d->kind == DP_LAYER_CONV2D) {
        const int tiles = pl.use_thin ? 1 : (pl.use_tc ? tc_norm_slots(d->dtype, g, epi) : fma_tiles_m(g) * fma_tiles_n(g));
        pl.w_slots = tiles;
        pl.slots = tiles + (d->has_bias ? (pl.use_thin ? 1 : bias_blocks(g)) : 0);
    } else {
        pl.w_slots = 1; pl.slots = 2;
    }
    pl.partial_off = off; off = round_up(off + sizeof(float) * B * pl.slots, 256);
    pl.factor_off = off;  off = round_up(off + sizeof(float) * B * 2, 256);
    pl.db_off = off;
    if (d->kind != DP_LAYER_NORM_AFFINE && d->has_bias) off = round_up(off + sizeof(float) * B * d->K_out, 256);
    pl.chunk_off = off; pl.dg_off = off;
    if (d->kind == DP_LAYER_NORM_AFFINE) {
        off = round_up(off + sizeof(float) * B * norm_chunks(storage_type(d), d->B, d->H * d->W, d->C_in) * 2 * d->C_in, 256);
        pl.dg_off = off;
        off = round_up(off + sizeof(float) * B * 2 * d->C_in, 256);
    }
    off = round_up(off, 1024);
    pl.tc_off = off;       // tensor-core scratch (unfolded input, partial sums) or the CUDA-core path's partial sums
    if (d->kind != DP_LAYER_NORM_AFFINE) {
        size_t bytes = 0;
        if (pl.use_tc) bytes = tc_workspace_bytes(d->dtype, g, epi);
        else if (epi == DP_EPI_CLIP_ACCUM) { const int sp = fma_clip_splits(g); bytes = sp > 1 ? sizeof(float) * (size_t)sp * g.M * g.N : 0; }
        off = round_up(off + bytes, 256);
    }
    pl.total = off;
    return true;
}

}  // namespace dp

using namespace dp;

extern "C" int dp_layer_groups(const dp_layer_desc *desc) { return valid_desc(desc) ? groups_of(desc) : 0; }

extern "C" size_t dp_workspace_bytes(const dp_layer_desc *desc, int epilogue) {
    if (!valid_desc(desc) || epilogue < 0 || epilogue > 2) return 0;
    WgradPlan pl;
    make_plan(desc, epilogue, pl);
    return pl.total;
}

extern "C" int dp_wgrad_uses_tensor_cores(const dp_layer_desc *desc, int epilogue) {
    if (!valid_desc(desc) || epilogue < 0 || epilogue > 2) return 0;
    WgradPlan pl;
    make_plan(desc, epilogue, pl);
    return pl.use_tc ? 1 : 0;
}

extern "C" dp_status dp_per_example_wgrad(const dp_layer_desc *d, const void *X, const void *dY, float *G_w, float *G_b,
                                          float *sqnorm, long long sqnorm_stride, int epi, float C_l, float *acc_w,
                                          float *acc_b, float *clip_out, void *workspace, size_t workspace_bytes,
                                          void *cuda_stream) {
    if (!valid_desc(d) || epi < 0 || epi > 2) return DP_ERR_INVALID_ARG;
    if (!X || !dY || !sqnorm || !aligned(X, 16) || !aligned(dY, 16) || !aligned(sqnorm, 4)) return DP_ERR_INVALID_ARG;
    const int groups = groups_of(d);
    const bool bias = has_bias_tensor(d);
    if (sqnorm_stride < groups) return DP_ERR_INVALID_ARG;
    if (epi == DP_EPI_STORE_NORM) {
        if (!G_w || !aligned(G_w, 16) || (bias && (!G_b || !aligned(G_b, 16)))) return DP_ERR_INVALID_ARG;
    }
    if (epi == DP_EPI_CLIP_ACCUM) {
        if (!(C_l > 0.0f)) return DP_ERR_INVALID_ARG;
        if (!acc_w || !aligned(acc_w, 16) || (bias && (!acc_b || !aligned(acc_b, 16)))) return DP_ERR_INVALID_ARG;
        if (clip_out && !aligned(clip_out, 4)) return DP_ERR_INVALID_ARG;
    }
    WgradPlan pl;
    make_plan(d, epi, pl);
    if (d->impl == DP_IMPL_TENSOR_CORE && !pl.use_tc) return DP_ERR_UNSUPPORTED;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < pl.total) return DP_ERR_WORKSPACE;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    float *partial = reinterpret_cast<float *>(ws + pl.partial_off);
    float *factor = reinterpret_cast<float *>(ws + pl.factor_off);
    float *db_ws = reinterpret_cast<float *>(ws + pl.db_off);
    const ConvGeom g = geom_of(d);
    const int clip = (epi == DP_EPI_CLIP_ACCUM);
    dp_status rc;
    // The status word is sticky: dp_workspace_init clears it, a tensor-core launch whose bounded wait expired sets it,
    // and only dp_wgrad_check clears it again after reporting it.

    if (d->kind == DP_LAYER_CONV2D) {
        float *db = (epi == DP_EPI_STORE_NORM) ? G_b : db_ws;
        if (pl.use_thin && rgb3_conv_eligible(g))
            return launch_conv_rgb3(storage_type(d), X, dY, g, epi == DP_EPI_STORE_NORM ? G_w : nullptr, db, d->has_bias, groups == 2,
                                    sqnorm, sqnorm_stride, st);
        if (pl.use_thin) {
            rc = launch_conv_thin(storage_type(d), X, dY, g, epi == DP_EPI_STORE_NORM ? G_w : nullptr, db, partial, pl.slots, d->has_bias, st);
            if (rc != DP_OK) return rc;
            return launch_finalize(partial, d->B, pl.slots, pl.w_slots, groups == 2, sqnorm, sqnorm_stride, 0, 0.f, factor, nullptr, st);
        }
        if (d->has_bias) {
            rc = launch_bias(storage_type(d), dY, g, db, partial, pl.slots, pl.w_slots, st);
            if (rc != DP_OK) return rc;
        }
        if (epi != DP_EPI_CLIP_ACCUM) {
            if (pl.use_tc && epi == DP_EPI_NORM_ONLY && !d->has_bias && single_pass_enabled() && sm_target_set() &&
                tc_gram_norm(d->dtype, g) && !tc_clip_single_pass(d->dtype, g)) {
                // norms only, a large gradient over a small plane, calls running side by side: from the pixel Gram matrices,
                // without forming the gradient (far less SM time; a call that has the GPU to itself is quicker on all SMs)
                const TcInlineClip ic = {0.f, sqnorm, sqnorm_stride, nullptr};
                return launch_conv_gram_norm(d->dtype, X, dY, g, ic, nullptr, reinterpret_cast<int *>(ws + pl.status_off), st);
            }
            if (pl.use_tc) {
                // one launch: the kernel's last CTA folds the partial norms (a ticket in the workspace header)
                const TcPublish pub = {reinterpret_cast<int *>(ws + kWsCounterOffset), pl.w_slots, groups == 2, sqnorm, sqnorm_stride, nullptr, 0.f, nullptr};
                return launch_conv_tc(d->dtype, epi, X, dY, g, G_w, partial, pl.slots, nullptr, nullptr, ws + pl.tc_off,
                                      reinterpret_cast<int *>(ws + pl.status_off), st, false, nullptr, &pub);
            }
            if (pl.use_tc) rc = launch_conv_tc(d->dtype, epi, X, dY, g, G_w, partial, pl.slots, nullptr, nullptr, ws + pl.tc_off, reinterpret_cast<int *>(ws + pl.status_off), st);
            else rc = launch_conv_fma(storage_type(d), epi, X, dY, g, G_w, partial, pl.slots, nullptr, nullptr, nullptr, st);
            if (rc != DP_OK) return rc;
            return launch_finalize(partial, d->B, pl.slots, pl.w_slots, groups == 2, sqnorm, sqnorm_stride, 0, 0.f, factor, nullptr, st);
        }
        if (pl.use_tc && !d->has_bias && single_pass_enabled() && tc_clip_single_pass(d->dtype, g)) {
            // per-layer clipping from ONE contraction: norm, factor and scaled sum come from the same accumulators
            const TcInlineClip ic = {C_l, sqnorm, sqnorm_stride, clip_out};
            return launch_conv_clip1(d->dtype, X, dY, g, partial, pl.slots, ic, acc_w, ws + pl.tc_off,
                                     reinterpret_cast<int *>(ws + pl.status_off), st);
        }
        // per-layer clipping: norms of every example first, then the clipped sum with the factors known
        if (pl.use_tc) {
            if (!d->has_bias && single_pass_enabled() && tc_clip_scaled_sum(d->dtype, g) && tc_gram_norm(d->dtype, g)) {
                // small planes: norms and factors from the pixel Gram matrices, then the clipped sum as one product
                const TcInlineClip ic = {C_l, sqnorm, sqnorm_stride, clip_out};
                rc = launch_conv_gram_norm(d->dtype, X, dY, g, ic, factor, reinterpret_cast<int *>(ws + pl.status_off), st);
                if (rc != DP_OK) return rc;
                if (tc_clip_scaled_tiles(d->dtype, g))     // enough pixels an example: scaled per example out of tensor memory
                    return launch_conv_scaled_tiles(d->dtype, X, dY, g, factor, acc_w, ws + pl.tc_off, reinterpret_cast<int *>(ws + pl.status_off), st);
                return launch_conv_ssum(d->dtype, X, dY, g, factor, acc_w, ws + pl.tc_off, reinterpret_cast<int *>(ws + pl.status_off), st);
            }
            // the norm pass's last CTA folds the partial norms (bias slots included) into norms and factors
            const TcPublish pub = {reinterpret_cast<int *>(ws + kWsCounterOffset), pl.w_slots, groups == 2, sqnorm, sqnorm_stride, factor, C_l, clip_out};
            rc = launch_conv_tc(d->dtype, DP_EPI_NORM_ONLY, X, dY, g, nullptr, partial, pl.slots, nullptr, nullptr, ws + pl.tc_off,
                                reinterpret_cast<int *>(ws + pl.status_off), st, false, nullptr, &pub);
            if (rc != DP_OK) return rc;
            if (!d->has_bias && single_pass_enabled() && tc_clip_scaled_sum(d->dtype, g))
                return launch_conv_ssum(d->dtype, X, dY, g, factor, acc_w, ws + pl.tc_off, reinterpret_cast<int *>(ws + pl.status_off), st);
            rc = launch_conv_tc(d->dtype, DP_EPI_CLIP_ACCUM, X, dY, g, nullptr, partial, pl.slots, factor, acc_w, ws + pl.tc_off,
                                reinterpret_cast<int *>(ws + pl.status_off), st, true);
            if (rc != DP_OK) return rc;
            if (d->has_bias) return launch_bias_accum(db, d->B, d->K_out, factor, acc_b, st);
            return DP_OK;
        }
        rc = launch_conv_fma(storage_type(d), DP_EPI_NORM_ONLY, X, dY, g, nullptr, partial, pl.slots, nullptr, nullptr, nullptr, st);
        if (rc != DP_OK) return rc;
        rc = launch_finalize(partial, d->B, pl.slots, pl.w_slots, groups == 2, sqnorm, sqnorm_stride, 1, C_l, factor, clip_out, st);
        if (rc != DP_OK) return rc;
        if (pl.use_tc) rc = launch_conv_tc(d->dtype, DP_EPI_CLIP_ACCUM, X, dY, g, nullptr, partial, pl.slots, factor, acc_w, ws + pl.tc_off, reinterpret_cast<int *>(ws + pl.status_off), st, true);
        else rc = launch_conv_fma(storage_type(d), DP_EPI_CLIP_ACCUM, X, dY, g, nullptr, partial, pl.slots, factor, acc_w, reinterpret_cast<float *>(ws + pl.tc_off), st);
        if (rc != DP_OK) return rc;
        if (d->has_bias) return launch_bias_accum(db, d->B, d->K_out, factor, acc_b, st);
        return DP_OK;
    }

    if (d->kind == DP_LAYER_DENSE) {
        if (epi == DP_EPI_STORE_NORM) {
            rc = launch_dense_store(storage_type(d), X, dY, d->B, d->C_in, d->K_out, G_w, d->has_bias ? G_b : nullptr, st);
            if (rc != DP_OK) return rc;
        }
        float *db_dst = !d->has_bias ? nullptr : (epi == DP_EPI_STORE_NORM ? G_b : (clip ? db_ws : nullptr));
        rc = launch_dense_norm(storage_type(d), X, dY, d->B, d->C_in, d->K_out, d->has_bias, db_dst, groups == 2, sqnorm,
                               sqnorm_stride, clip, C_l, factor, clip_out, st);
        if (rc != DP_OK || !clip) return rc;
        // sum_n f_n dY_n^T X_n is one matrix product with the batch as the reduction axis
        // (the bias gradient of a dense layer is dY: its clipped sum rides in the same launch, with the bias factor)
        return launch_dense_scaled_sum(storage_type(d), X, dY, factor, 2, d->B, d->C_in, d->K_out, acc_w, st,
                                       d->has_bias ? factor + 1 : nullptr, 2, d->has_bias ? acc_b : nullptr);
    }

    // normalisation affine
    {
        float *chunk_partial = reinterpret_cast<float *>(ws + pl.chunk_off);
        float *dg = (epi == DP_EPI_STORE_NORM) ? G_w : reinterpret_cast<float *>(ws + pl.dg_off);
        float *dbt = (epi == DP_EPI_STORE_NORM) ? G_b : reinterpret_cast<float *>(ws + pl.dg_off) + (size_t)d->B * d->C_in;
        if (affine_fused_eligible(d->B))
            return launch_norm_affine_fused(storage_type(d), X, dY, d->B, d->H * d->W, d->C_in, chunk_partial, dg, dbt, factor,
                                            reinterpret_cast<int *>(ws + kWsCounterOffset), clip, C_l, groups == 2, sqnorm,
                                            sqnorm_stride, clip_out, acc_w, acc_b, st);
        rc = launch_norm_affine(storage_type(d), X, dY, d->B, d->H * d->W, d->C_in, chunk_partial, dg, dbt, partial, st);
        if (rc != DP_OK) return rc;
        if (clip)
            return launch_affine_clip_accum(partial, d->B, C_l, groups == 2, sqnorm, sqnorm_stride, clip_out, dg, dbt, d->C_in,
                                            acc_w, acc_b, st);
        return launch_finalize(partial, d->B, 2, 1, groups == 2, sqnorm, sqnorm_stride, 0, 0.f, factor, nullptr, st);
    }
}

extern "C" dp_status dp_per_example_wgrad_scaled(const dp_layer_desc *d, const void *X, const void *dY,
                                                 const float *factor_w, const float *factor_b, long long factor_stride,
                                                 float *acc_w, float *acc_b, void *workspace, size_t workspace_bytes,
                                                 void *cuda_stream) {
    if (!valid_desc(d)) return DP_ERR_INVALID_ARG;
    if (!X || !dY || !aligned(X, 16) || !aligned(dY, 16)) return DP_ERR_INVALID_ARG;
    if (!factor_w || !aligned(factor_w, 4) || (factor_b && !aligned(factor_b, 4)) || factor_stride < 1) return DP_ERR_INVALID_ARG;
    const bool bias = has_bias_tensor(d);
    if (!acc_w || !aligned(acc_w, 16) || (bias && (!acc_b || !aligned(acc_b, 16)))) return DP_ERR_INVALID_ARG;
    if (!factor_b) factor_b = factor_w;
    WgradPlan pl;
    make_plan(d, DP_EPI_CLIP_ACCUM, pl);
    if (d->impl == DP_IMPL_TENSOR_CORE && !pl.use_tc) return DP_ERR_UNSUPPORTED;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < pl.total) return DP_ERR_WORKSPACE;

    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    float *partial = reinterpret_cast<float *>(ws + pl.partial_off);
    float *factor = reinterpret_cast<float *>(ws + pl.factor_off);
    float *db_ws = reinterpret_cast<float *>(ws + pl.db_off);
    const ConvGeom g = geom_of(d);
    int *status_word = reinterpret_cast<int *>(ws + pl.status_off);
    dp_status rc;
    if (d->kind == DP_LAYER_DENSE) {
        // sum_n f_n dY_n^T X_n is one matrix product with the batch as the reduction axis; the bias gradient is dY itself.
        // One launch does both and reads the caller's factors in place.
        return launch_dense_scaled_sum(storage_type(d), X, dY, factor_w, factor_stride, d->B, d->C_in, d->K_out, acc_w, st,
                                       d->has_bias ? factor_b : nullptr, factor_stride, d->has_bias ? acc_b : nullptr);
    }
    // the clipped-sum kernels read one (weight, bias) pair of factors per example
    rc = launch_expand_factor(factor_w, factor_b, factor_stride, d->B, factor, st);
    if (rc != DP_OK) return rc;

    if (d->kind == DP_LAYER_CONV2D) {
        if (d->has_bias) {
            rc = launch_bias(storage_type(d), dY, g, db_ws, partial, pl.slots, pl.w_slots, st);
            if (rc != DP_OK) return rc;
        }
        if (pl.use_tc) rc = launch_conv_tc(d->dtype, DP_EPI_CLIP_ACCUM, X, dY, g, nullptr, partial, pl.slots, factor, acc_w, ws + pl.tc_off, status_word, st);
        else rc = launch_conv_fma(storage_type(d), DP_EPI_CLIP_ACCUM, X, dY, g, nullptr, partial, pl.slots, factor, acc_w, reinterpret_cast<float *>(ws + pl.tc_off), st);
        if (rc != DP_OK) return rc;
        if (d->has_bias) return launch_bias_accum(db_ws, d->B, d->K_out, factor, acc_b, st);
        return DP_OK;
    }
    {
        float *chunk_partial = reinterpret_cast<float *>(ws + pl.chunk_off);
        float *dg = reinterpret_cast<float *>(ws + pl.dg_off);
        float *dbt = dg + (size_t)d->B * d->C_in;
        rc = launch_norm_affine(storage_type(d), X, dY, d->B, d->H * d->W, d->C_in, chunk_partial, dg, dbt, partial, st);
        if (rc != DP_OK) return rc;
        rc = launch_bias_accum(dg, d->B, d->C_in, factor, acc_w, st, 0);
        if (rc != DP_OK) return rc;
        return launch_bias_accum(dbt, d->B, d->C_in, factor, acc_b, st, 1);
    }
}

extern "C" int dp_debug_wgrad_plan(const dp_layer_desc *desc, int epilogue, int *out, int n) {
    if (!valid_desc(desc) || desc->kind != DP_LAYER_CONV2D || epilogue < 0 || epilogue > 5 || !out || n <= 0) return 0;   // 3: the single-pass form of the fused clip, 4: the clipped sum as one product, 5: norms from Gram matrices
    return tc_describe_plan(desc->dtype, geom_of(desc), epilogue, out, n);
}

extern "C" dp_status dp_workspace_init(void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < kWsHeaderBytes) return DP_ERR_WORKSPACE;
    DP_CUDA_TRY(cudaMemsetAsync(workspace, 0, kWsHeaderBytes, static_cast<cudaStream_t>(cuda_stream)));
    return DP_OK;
}

extern "C" dp_status dp_wgrad_check(void *workspace, void *cuda_stream) {
    if (!workspace) return DP_ERR_INVALID_ARG;
    int status = 0;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    DP_CUDA_TRY(cudaMemcpyAsync(&status, workspace, sizeof(int), cudaMemcpyDeviceToHost, st));
    DP_CUDA_TRY(cudaStreamSynchronize(st));
    if (status == 0) return DP_OK;
    // reported once: a launch that gave up may also have left ticket counters behind, so the whole header starts over
    DP_CUDA_TRY(cudaMemsetAsync(workspace, 0, kWsHeaderBytes, st));
    DP_CUDA_TRY(cudaStreamSynchronize(st));
    return DP_ERR_TIMEOUT;
}

extern "C" dp_status dp_set_sm_target(int sms) {
    if (sms < 0) return DP_ERR_INVALID_ARG;
    dp::g_sm_target.store(sms, std::memory_order_relaxed);
    return DP_OK;
}

extern "C" void dp_debug_set_single_pass(int on) { dp::g_single_pass.store(on ? 1 : 0, std::memory_order_relaxed); }

extern "C" void dp_debug_set_wait_polls(long long polls) {
    set_wait_polls(polls < 0 ? default_wait_polls() : (uint32_t)(polls > 0xffffffffll ? 0xffffffffll : polls));
}

extern "C" const char *dp_status_string(int status) {
    switch (status) {
        case DP_OK: return "ok";
        case DP_ERR_INVALID_ARG: return "invalid argument";
        case DP_ERR_UNSUPPORTED: return "unsupported";
        case DP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DP_ERR_CUDA: return "CUDA error";
        case DP_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" const char *dp_last_cuda_error(void) { return dp::g_last_error; }

extern "C" unsigned long long dp_debug_launch_count(void) { return dp::g_launches.load(std::memory_order_relaxed); }

// Gaussian noise and averaging: out = (acc + sigma*C*z) / |B|  (paper section 2, equation for g_t).
// z comes from Philox4x32-10 (Salmon et al., SC'11) and the Box-Muller transform, addressed by
// (seed, step, global parameter index), so the result does not depend on the launch shape.
#include "common.cuh"
#include "philox.cuh"

namespace dp {

// Thread t owns Philox block first_block + t, i.e. global indices 4*(first_block+t) .. +3;
// local index = global - param_offset.  VEC: param_offset % 4 == 0, so a block is one float4.
template <bool VEC>
__global__ void __launch_bounds__(256)
noise_average_kernel(const float *acc, float *out, long long P,   // out may alias acc
                     unsigned long long param_offset, unsigned long long n_blocks,
                     float noise_std, float inv_batch, unsigned long long seed, unsigned long long step) {
    const unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_blocks) return;
    const unsigned long long block = (param_offset >> 2) + t;
    float z[4] = {0.f, 0.f, 0.f, 0.f};
    if (noise_std != 0.0f) normals4(seed, step, block, z);
    const long long i0 = (long long)(4ull * block - param_offset);   // may be negative for the first block
    if (VEC && i0 + 3 < P) {
        const float4 a = __ldcs(reinterpret_cast<const float4 *>(acc + i0));
        float4 r;
        r.x = (a.x + noise_std * z[0]) * inv_batch;
        r.y = (a.y + noise_std * z[1]) * inv_batch;
        r.z = (a.z + noise_std * z[2]) * inv_batch;
        r.w = (a.w + noise_std * z[3]) * inv_batch;
        __stcs(reinterpret_cast<float4 *>(out + i0), r);
    } else {
#pragma unroll
        for (int lane = 0; lane < 4; ++lane) {
            const long long i = i0 + lane;
            if (i >= 0 && i < P) out[i] = (acc[i] + noise_std * z[lane]) * inv_batch;
        }
    }
}

// Noise, average and the parameter update in one pass: g = (acc + std*z) / |B|;  m <- mu*m + g (when a momentum
// buffer is given);  theta <- theta - lr*m (or - lr*g).  Same thread-to-Philox-block mapping as above.
__global__ void __launch_bounds__(256)
noise_average_sgd_kernel(const float *acc, long long P, unsigned long long param_offset, unsigned long long n_blocks,
                         float noise_std, float inv_batch, unsigned long long seed, unsigned long long step, float lr,
                         float mu, float *theta, float *mom, float *g_out) {
    const unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_blocks) return;
    const unsigned long long block = (param_offset >> 2) + t;
    float z[4] = {0.f, 0.f, 0.f, 0.f};
    if (noise_std != 0.0f) normals4(seed, step, block, z);
    const long long i0 = (long long)(4ull * block - param_offset);
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
        const long long i = i0 + lane;
        if (i < 0 || i >= P) continue;
        const float g = (acc[i] + noise_std * z[lane]) * inv_batch;
        float v = g;
        if (mom) { v = fmaf(mu, mom[i], g); mom[i] = v; }
        theta[i] = fmaf(-lr, v, theta[i]);
        if (g_out) g_out[i] = g;
    }
}

__global__ void philox_raw_kernel(uint32_t *out4, long long n_blocks, unsigned long long first_block,
                                  unsigned long long seed, unsigned long long step) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_blocks) return;
    const Words4 w = philox_block(seed, step, first_block + (unsigned long long)t);
    reinterpret_cast<uint4 *>(out4)[t] = make_uint4(w.w0, w.w1, w.w2, w.w3);
}

__global__ void noise_z_kernel(float *z, long long count, unsigned long long first_index,
                               unsigned long long n_blocks, unsigned long long seed, unsigned long long step) {
    const unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_blocks) return;
    const unsigned long long block = (first_index >> 2) + t;
    float v[4];
    normals4(seed, step, block, v);
    const long long i0 = (long long)(4ull * block - first_index);
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
        const long long i = i0 + lane;
        if (i >= 0 && i < count) z[i] = v[lane];
    }
}

// z[t] = normal of example `example`'s stream at global index first_index + t (one thread per Philox block)
__global__ void example_noise_z_kernel(float *z, long long count, unsigned long long first_index,
                                       unsigned long long n_blocks, uint32_t example, unsigned long long seed,
                                       unsigned long long step) {
    const unsigned long long t = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_blocks) return;
    const unsigned long long block = (first_index >> 2) + t;
    float v[4];
    example_normals4(seed, step, example, (uint32_t)block, v);
    const long long i0 = (long long)(4ull * block - first_index);
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
        const long long i = i0 + lane;
        if (i >= 0 && i < count) z[i] = v[lane];
    }
}

}  // namespace dp

extern "C" dp_status dp_noise_average(const float *acc, long long P, long long param_offset, float sigma, float C,
                                      long long total_batch, unsigned long long seed, unsigned long long step,
                                      float *out, void *cuda_stream) {
    if (!acc || !out || P <= 0 || param_offset < 0 || total_batch <= 0) return DP_ERR_INVALID_ARG;
    if (!(sigma >= 0.0f) || !(C > 0.0f)) return DP_ERR_INVALID_ARG;                 // also rejects NaN
    if (sigma > 0.0f && isinf(C)) return DP_ERR_INVALID_ARG;
    if (isinf(sigma)) return DP_ERR_INVALID_ARG;
    if (!dp::aligned(acc, 16) || !dp::aligned(out, 16)) return DP_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned long long off = (unsigned long long)param_offset;
    const unsigned long long n_blocks = ((off & 3ull) + (unsigned long long)P + 3ull) >> 2;
    const float noise_std = (sigma == 0.0f) ? 0.0f : sigma * C;
    const float inv_batch = 1.0f / (float)total_batch;
    const unsigned long long grid = (n_blocks + 255) / 256;
    if (grid > 0x7fffffffull) return DP_ERR_UNSUPPORTED;
    if ((off & 3ull) == 0)
        dp::noise_average_kernel<true><<<(unsigned)grid, 256, 0, stream>>>(acc, out, P, off, n_blocks, noise_std,
                                                                          inv_batch, seed, step);
    else
        dp::noise_average_kernel<false><<<(unsigned)grid, 256, 0, stream>>>(acc, out, P, off, n_blocks, noise_std,
                                                                           inv_batch, seed, step);
    DP_LAUNCH_CHECK("noise_average_kernel");
    return DP_OK;
}

extern "C" dp_status dp_noise_average_sgd(const float *acc, long long P, long long param_offset, float sigma, float C,
                                          long long total_batch, unsigned long long seed, unsigned long long step,
                                          float lr, float momentum, float *theta, float *momentum_buf, float *g_out,
                                          void *cuda_stream) {
    if (!acc || !theta || P <= 0 || param_offset < 0 || total_batch <= 0) return DP_ERR_INVALID_ARG;
    if (!(sigma >= 0.0f) || !(C > 0.0f) || isinf(sigma) || (sigma > 0.0f && isinf(C))) return DP_ERR_INVALID_ARG;
    if (!(lr == lr) || isinf(lr) || !(momentum >= 0.0f) || isinf(momentum)) return DP_ERR_INVALID_ARG;
    if (!dp::aligned(acc, 4) || !dp::aligned(theta, 4) || (momentum_buf && !dp::aligned(momentum_buf, 4)) ||
        (g_out && !dp::aligned(g_out, 4)))
        return DP_ERR_INVALID_ARG;
    const unsigned long long off = (unsigned long long)param_offset;
    const unsigned long long n_blocks = ((off & 3ull) + (unsigned long long)P + 3ull) >> 2;
    const unsigned long long grid = (n_blocks + 255) / 256;
    if (grid > 0x7fffffffull) return DP_ERR_UNSUPPORTED;
    dp::noise_average_sgd_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        acc, P, off, n_blocks, (sigma == 0.0f) ? 0.0f : sigma * C, 1.0f / (float)total_batch, seed, step, lr, momentum,
        theta, momentum_buf, g_out);
    DP_LAUNCH_CHECK("noise_average_sgd_kernel");
    return DP_OK;
}

extern "C" dp_status dp_debug_philox_raw(unsigned int *out4, long long n_blocks, long long first_block,
                                         unsigned long long seed, unsigned long long step, void *cuda_stream) {
    if (!out4 || n_blocks <= 0 || first_block < 0 || !dp::aligned(out4, 16)) return DP_ERR_INVALID_ARG;
    const long long grid = (n_blocks + 255) / 256;
    if (grid > 0x7fffffffll) return DP_ERR_UNSUPPORTED;
    dp::philox_raw_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        out4, n_blocks, (unsigned long long)first_block, seed, step);
    DP_LAUNCH_CHECK("philox_raw_kernel");
    return DP_OK;
}

extern "C" dp_status dp_debug_noise_z(float *z, long long count, long long first_index, unsigned long long seed,
                                      unsigned long long step, void *cuda_stream) {
    if (!z || count <= 0 || first_index < 0) return DP_ERR_INVALID_ARG;
    const unsigned long long off = (unsigned long long)first_index;
    const unsigned long long n_blocks = ((off & 3ull) + (unsigned long long)count + 3ull) >> 2;
    const unsigned long long grid = (n_blocks + 255) / 256;
    if (grid > 0x7fffffffull) return DP_ERR_UNSUPPORTED;
    dp::noise_z_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(z, count, off, n_blocks,
                                                                                         seed, step);
    DP_LAUNCH_CHECK("noise_z_kernel");
    return DP_OK;
}

extern "C" dp_status dp_debug_example_noise_z(float *z, long long count, long long first_index, long long example,
                                              unsigned long long seed, unsigned long long step, void *cuda_stream) {
    if (!z || count <= 0 || first_index < 0 || example < 0 || example >= 0x80000000ll) return DP_ERR_INVALID_ARG;
    const unsigned long long off = (unsigned long long)first_index;
    if (off + (unsigned long long)count > (1ull << 34)) return DP_ERR_UNSUPPORTED;
    const unsigned long long n_blocks = ((off & 3ull) + (unsigned long long)count + 3ull) >> 2;
    const unsigned long long grid = (n_blocks + 255) / 256;
    if (grid > 0x7fffffffull) return DP_ERR_UNSUPPORTED;
    dp::example_noise_z_kernel<<<(unsigned)grid, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        z, count, off, n_blocks, (uint32_t)example, seed, step);
    DP_LAUNCH_CHECK("example_noise_z_kernel");
    return DP_OK;
}

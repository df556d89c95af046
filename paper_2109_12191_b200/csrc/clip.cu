// Norm, clip and accumulate over materialised per-example gradients
// (paper section 2: sum over the batch of clip(g_j, C); section 3.5: per-group threshold C/sqrt(M)).
//
// Three memory-bound stages, all with fixed reduction orders:
//   1. (only when the caller has no norms) per-block partial sums of squares of every example row,
//      then one block per (tensor, example) folds the partials;
//   2. one small kernel turns squared norms into clip factors;
//   3. every thread owns four neighbouring parameters, streams the B example rows through
//      registers with 128-bit loads, and touches the accumulator once.
#include "common.cuh"
#include "philox.cuh"
#include <math.h>
#include <mutex>

namespace dp {

constexpr int kMaxSeg = 40;          // tensors per launch (table travels as a kernel parameter)
constexpr int kNormChunk = 8192;     // floats of one example row reduced by one block (stage 1)
constexpr int kAccCols = 1024;       // parameters per block in stage 3 (256 threads x float4)

struct SegTable {
    const float *G[kMaxSeg];         // [B, P] per tensor
    float *acc[kMaxSeg];             // [P] per tensor
    long long P[kMaxSeg];
    int blk_start[kMaxSeg + 1];      // first block of each tensor within this launch
    int col[kMaxSeg];                // index l of the tensor in the [B, L] norm / factor tables
    long long part_start[kMaxSeg];   // first partial slot of each tensor within one example's row of partials
    long long goff[kMaxSeg];         // global index of the tensor's first parameter (per-example noise only)
    int nseg;
};

// Per-example noise (the paper's own implementation, section 2, the block after the equation for g_t):
// example e of the step adds sd * z_e(g), sd = sigma*C/sqrt(|B|), to its clipped gradient before the sum.
struct ExampleNoise {
    float sd;
    unsigned long long seed, step;
    uint32_t example0;               // index within the step of this chunk's first example
};

__device__ __forceinline__ int find_seg(const SegTable &t, int blk) {
    int s = 0;
    while (s + 1 < t.nseg && blk >= t.blk_start[s + 1]) ++s;
    return s;
}

// stage 1a: partial[n][part_start[seg] + j] = sum of squares of G_seg[n, j*chunk .. (j+1)*chunk)
__global__ void __launch_bounds__(256)
sqnorm_partial_kernel(const __grid_constant__ SegTable tab, float *__restrict__ partial, long long parts_per_example) {
    __shared__ float scratch[32];
    const int seg = find_seg(tab, blockIdx.x);
    const int j = blockIdx.x - tab.blk_start[seg];
    const int n = blockIdx.y;
    const long long P = tab.P[seg];
    const long long c0 = (long long)j * kNormChunk;
    const int len = (int)min((long long)kNormChunk, P - c0);
    const float *row = tab.G[seg] + (long long)n * P + c0;
    float a = 0.f;
    if ((reinterpret_cast<uintptr_t>(row) & 15) == 0) {
        const float4 *row4 = reinterpret_cast<const float4 *>(row);
        const int n4 = len >> 2;
        float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 4
        for (int i = threadIdx.x; i < n4; i += 256) {
            const float4 v = __ldg(row4 + i);
            a0 = fmaf(v.x, v.x, a0); a1 = fmaf(v.y, v.y, a1); a2 = fmaf(v.z, v.z, a2); a3 = fmaf(v.w, v.w, a3);
        }
        a = (a0 + a1) + (a2 + a3);
        for (int i = (n4 << 2) + threadIdx.x; i < len; i += 256) a = fmaf(row[i], row[i], a);
    } else {
        for (int i = threadIdx.x; i < len; i += 256) a = fmaf(row[i], row[i], a);
    }
    a = block_sum(a, scratch);
    if (threadIdx.x == 0) partial[(long long)n * parts_per_example + tab.part_start[seg] + j] = a;
}

// stage 1b: sq[n][col[seg]] = sum over the tensor's partials, in index order, in double
__global__ void __launch_bounds__(128)
sqnorm_fold_kernel(const __grid_constant__ SegTable tab, const float *__restrict__ partial,
                   long long parts_per_example, float *__restrict__ sq, int L) {
    __shared__ double scratch[32];
    const int seg = blockIdx.x, n = blockIdx.y;
    const long long nparts = (tab.P[seg] + kNormChunk - 1) / kNormChunk;
    const float *p = partial + (long long)n * parts_per_example + tab.part_start[seg];
    double a = 0.0;
    for (long long i = threadIdx.x; i < nparts; i += 128) a += (double)p[i];
    a = block_sum(a, scratch);
    if (threadIdx.x == 0) sq[(long long)n * L + tab.col[seg]] = (float)a;
}

// stage 2: factors.  GLOBAL: one factor per example from the sum over its L tensors (thread per example).
// PER_LAYER: one factor per (example, tensor) against C/sqrt(L).
__global__ void clip_factor_kernel(const float *__restrict__ sq, int B, int L, int per_layer, float C,
                                   float *__restrict__ factor, float *norms_out, float *clip_out) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (per_layer) {
        if (idx >= B * L) return;
        const float thr = (float)((double)C / sqrt((double)L));
        const double s = (double)sq[idx];
        const float f = clip_factor(s, thr);
        factor[idx] = f;
        if (norms_out) norms_out[idx] = (float)sqrt(s);
        if (clip_out) clip_out[idx] = f;
    } else {
        if (idx >= B) return;
        double s = 0.0;
        for (int l = 0; l < L; ++l) s += (double)sq[(long long)idx * L + l];
        const float f = clip_factor(s, C);
        factor[idx] = f;
        if (norms_out) norms_out[idx] = (float)sqrt(s);
        if (clip_out) clip_out[idx] = f;
    }
}

// stage 1a for micro-batch clipping: row j of the partials belongs to the MEAN of examples j*micro .. j*micro+micro-1
// (the unit that is clipped), so the rows are added before they are squared.
__global__ void __launch_bounds__(256)
sqnorm_partial_micro_kernel(const __grid_constant__ SegTable tab, float *__restrict__ partial,
                            long long parts_per_example, int micro) {
    __shared__ float scratch[32];
    const int seg = find_seg(tab, blockIdx.x);
    const int j = blockIdx.x - tab.blk_start[seg];
    const long long P = tab.P[seg];
    const long long c0 = (long long)j * kNormChunk;
    const int len = (int)min((long long)kNormChunk, P - c0);
    const float *row = tab.G[seg] + (long long)blockIdx.y * micro * P + c0;
    const float inv = 1.0f / (float)micro;
    float a = 0.f;
    if (((reinterpret_cast<uintptr_t>(row) | (uintptr_t)(P * 4)) & 15) == 0) {
        const int n4 = len >> 2;
        for (int i = threadIdx.x; i < n4; i += 256) {
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int r = 0; r < micro; ++r) {
                const float4 x = __ldg(reinterpret_cast<const float4 *>(row + (long long)r * P) + i);
                v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
            }
            v.x *= inv; v.y *= inv; v.z *= inv; v.w *= inv;
            a = fmaf(v.x, v.x, a); a = fmaf(v.y, v.y, a); a = fmaf(v.z, v.z, a); a = fmaf(v.w, v.w, a);
        }
        for (int i = (n4 << 2) + threadIdx.x; i < len; i += 256) {
            float v = 0.f;
            for (int r = 0; r < micro; ++r) v += row[(long long)r * P + i];
            v *= inv;
            a = fmaf(v, v, a);
        }
    } else {
        for (int i = threadIdx.x; i < len; i += 256) {
            float v = 0.f;
            for (int r = 0; r < micro; ++r) v += row[(long long)r * P + i];
            v *= inv;
            a = fmaf(v, v, a);
        }
    }
    a = block_sum(a, scratch);
    if (threadIdx.x == 0) partial[(long long)blockIdx.y * parts_per_example + tab.part_start[seg] + j] = a;
}

// stage 2 for micro-batch clipping: one factor per micro-batch from the norm of its mean; every example of the
// micro-batch then carries factor / micro, so that stage 3 adds factor * mean.
__global__ void clip_factor_micro_kernel(const float *__restrict__ sq, int n_micro, int L, int micro, float C,
                                         float *__restrict__ factor, float *norms_out, float *clip_out) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n_micro) return;
    double s = 0.0;
    for (int l = 0; l < L; ++l) s += (double)sq[(long long)j * L + l];
    const float f = clip_factor(s, C);
    const float each = f / (float)micro;
    for (int i = 0; i < micro; ++i) factor[(long long)j * micro + i] = each;
    if (norms_out) norms_out[j] = (float)sqrt(s);
    if (clip_out) clip_out[j] = f;
}

// stage 2 for groups of tensors (section 3.5: M pipeline stages, each clipped to C/sqrt(M)): one block per example
// sums the squared norms of each group's tensors in tensor order, then every tensor gets its group's factor.
constexpr int kMaxGroupedTensors = 1024;
struct GroupTable {
    int M;
    unsigned short of[kMaxGroupedTensors];   // group of tensor l
};
__global__ void __launch_bounds__(128)
clip_factor_grouped_kernel(const float *__restrict__ sq, int L, const __grid_constant__ GroupTable gt, float C,
                           float *__restrict__ factor, float *norms_out, float *clip_out) {
    __shared__ float f_sh[kMaxGroupedTensors];
    const int n = blockIdx.x;
    const float thr = (float)((double)C / sqrt((double)gt.M));
    for (int m = threadIdx.x; m < gt.M; m += 128) {
        double s = 0.0;
        for (int l = 0; l < L; ++l)
            if (gt.of[l] == m) s += (double)sq[(long long)n * L + l];
        const float f = clip_factor(s, thr);
        f_sh[m] = f;
        if (norms_out) norms_out[(long long)n * gt.M + m] = (float)sqrt(s);
        if (clip_out) clip_out[(long long)n * gt.M + m] = f;
    }
    __syncthreads();
    for (int l = threadIdx.x; l < L; l += 128) factor[(long long)n * L + l] = f_sh[gt.of[l]];
}

// stage 3: acc[i] += sum_n factor * G[n, i].  factor index: GLOBAL n, PER_LAYER n*L + col.
template <int UNROLL>
__global__ void __launch_bounds__(256)
scale_accumulate_kernel(const __grid_constant__ SegTable tab, const float *__restrict__ factor, int B, int L,
                        int per_layer) {
    __shared__ float f_sh[256];
    const int seg = find_seg(tab, blockIdx.x);
    const long long P = tab.P[seg];
    const long long c0 = (long long)(blockIdx.x - tab.blk_start[seg]) * kAccCols;
    const float *G = tab.G[seg];
    float *acc = tab.acc[seg];
    const int f_stride = per_layer ? L : 1;
    const int f_off = per_layer ? tab.col[seg] : 0;
    // vector path needs every row start 16-byte aligned: base aligned and P a multiple of 4
    const bool vec = ((P & 3) == 0) && ((reinterpret_cast<uintptr_t>(G) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(acc) & 15) == 0);
    if (vec) {
        const long long i = c0 + 4 * threadIdx.x;
        const bool live = i < P;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int n0 = 0; n0 < B; n0 += 256) {
            const int nb = min(256, B - n0);
            __syncthreads();
            if (threadIdx.x < nb) f_sh[threadIdx.x] = factor[(long long)(n0 + threadIdx.x) * f_stride + f_off];
            __syncthreads();
            if (live) {
                const float *g = G + (long long)n0 * P + i;
                int n = 0;
                for (; n + UNROLL <= nb; n += UNROLL) {
                    float4 v[UNROLL];
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u)
                        v[u] = __ldcs(reinterpret_cast<const float4 *>(g + (long long)(n + u) * P));
#pragma unroll
                    for (int u = 0; u < UNROLL; ++u) {
                        const float f = f_sh[n + u];
                        s.x = fmaf(f, v[u].x, s.x); s.y = fmaf(f, v[u].y, s.y);
                        s.z = fmaf(f, v[u].z, s.z); s.w = fmaf(f, v[u].w, s.w);
                    }
                }
                for (; n < nb; ++n) {
                    const float4 v = __ldcs(reinterpret_cast<const float4 *>(g + (long long)n * P));
                    const float f = f_sh[n];
                    s.x = fmaf(f, v.x, s.x); s.y = fmaf(f, v.y, s.y); s.z = fmaf(f, v.z, s.z); s.w = fmaf(f, v.w, s.w);
                }
            }
        }
        if (live) {
            float4 a = *reinterpret_cast<const float4 *>(acc + i);
            a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
            *reinterpret_cast<float4 *>(acc + i) = a;
        }
    } else {
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        for (int n0 = 0; n0 < B; n0 += 256) {
            const int nb = min(256, B - n0);
            __syncthreads();
            if (threadIdx.x < nb) f_sh[threadIdx.x] = factor[(long long)(n0 + threadIdx.x) * f_stride + f_off];
            __syncthreads();
            for (int n = 0; n < nb; ++n) {
                const float f = f_sh[n];
                const float *g = G + (long long)(n0 + n) * P + c0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const long long i = threadIdx.x + 256 * q;
                    if (c0 + i < P) s[q] = fmaf(f, g[i], s[q]);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long i = c0 + threadIdx.x + 256 * q;
            if (i < P) acc[i] += s[q];
        }
    }
}

// stage 3 for small models with many examples: too few 1024-parameter blocks exist to fill the GPU, so a block takes
// only 128 parameters and splits the example rows over its eight warps (warp w owns rows w, w+8, ...), sixteen rows in
// flight per thread; the eight partial sums are folded in warp order through shared memory.
constexpr int kSplitCols = 128;
__global__ void __launch_bounds__(256)
scale_accumulate_rowsplit_kernel(const __grid_constant__ SegTable tab, const float *__restrict__ factor, int B, int L,
                                 int per_layer) {
    __shared__ float f_sh[256];
    __shared__ float4 part[8][32];
    const int seg = find_seg(tab, blockIdx.x);
    const long long P = tab.P[seg];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const long long i = (long long)(blockIdx.x - tab.blk_start[seg]) * kSplitCols + 4 * lane;
    const float *G = tab.G[seg];
    float *acc = tab.acc[seg];
    const int f_stride = per_layer ? L : 1;
    const int f_off = per_layer ? tab.col[seg] : 0;
    const bool vec = ((P & 3) == 0) && ((reinterpret_cast<uintptr_t>(G) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(acc) & 15) == 0);
    const int live = i >= P ? 0 : (int)min(4ll, P - i);           // parameters this thread owns (vec: 0 or 4)
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int n0 = 0; n0 < B; n0 += 256) {
        const int nb = min(256, B - n0);
        __syncthreads();
        if (threadIdx.x < nb) f_sh[threadIdx.x] = factor[(long long)(n0 + threadIdx.x) * f_stride + f_off];
        __syncthreads();
        if (live == 0) continue;
        const float *g = G + (long long)n0 * P + i;
        if (vec) {
            int n = w;
            for (; n + 8 * 15 < nb; n += 8 * 16) {
                float4 v[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) v[u] = __ldcs(reinterpret_cast<const float4 *>(g + (long long)(n + 8 * u) * P));
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const float f = f_sh[n + 8 * u];
                    s.x = fmaf(f, v[u].x, s.x); s.y = fmaf(f, v[u].y, s.y);
                    s.z = fmaf(f, v[u].z, s.z); s.w = fmaf(f, v[u].w, s.w);
                }
            }
            for (; n < nb; n += 8) {
                const float4 v = __ldcs(reinterpret_cast<const float4 *>(g + (long long)n * P));
                const float f = f_sh[n];
                s.x = fmaf(f, v.x, s.x); s.y = fmaf(f, v.y, s.y); s.z = fmaf(f, v.z, s.z); s.w = fmaf(f, v.w, s.w);
            }
        } else {
            for (int n = w; n < nb; n += 8) {
                const float *row = g + (long long)n * P;
                const float f = f_sh[n];
                s.x = fmaf(f, row[0], s.x);
                if (live > 1) s.y = fmaf(f, row[1], s.y);
                if (live > 2) s.z = fmaf(f, row[2], s.z);
                if (live > 3) s.w = fmaf(f, row[3], s.w);
            }
        }
    }
    part[w][lane] = s;
    __syncthreads();
    if (w == 0 && live > 0) {
        float4 t = part[0][lane];
#pragma unroll
        for (int q = 1; q < 8; ++q) {
            const float4 v = part[q][lane];
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        if (vec) {
            float4 a = *reinterpret_cast<const float4 *>(acc + i);
            a.x += t.x; a.y += t.y; a.z += t.z; a.w += t.w;
            *reinterpret_cast<float4 *>(acc + i) = a;
        } else {
            acc[i] += t.x;
            if (live > 1) acc[i + 1] += t.y;
            if (live > 2) acc[i + 2] += t.z;
            if (live > 3) acc[i + 3] += t.w;
        }
    }
}

// stage 3 with per-example noise: acc[i] += sum_n ( factor * G[n, i] + sd * z_{example0+n}(goff + i) ).
// Every thread owns the four parameters of one Philox block when the tensor starts on a multiple of four global
// indices; otherwise each parameter draws its own block and keeps one lane.  Bound by the integer and
// transcendental work of B*P normals, not by memory.
__global__ void __launch_bounds__(256)
scale_accumulate_noised_kernel(const __grid_constant__ SegTable tab, const float *__restrict__ factor, int B, int L,
                               int per_layer, const ExampleNoise nz) {
    __shared__ float f_sh[256];
    const int seg = find_seg(tab, blockIdx.x);
    const long long P = tab.P[seg];
    const long long c0 = (long long)(blockIdx.x - tab.blk_start[seg]) * kAccCols;
    const float *G = tab.G[seg];
    float *acc = tab.acc[seg];
    const long long goff = tab.goff[seg];
    const int f_stride = per_layer ? L : 1;
    const int f_off = per_layer ? tab.col[seg] : 0;
    const bool vec = ((P & 3) == 0) && ((goff & 3) == 0) && ((reinterpret_cast<uintptr_t>(G) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(acc) & 15) == 0);
    if (vec) {
        const long long i = c0 + 4 * threadIdx.x;
        const bool live = i < P;
        const uint32_t block = (uint32_t)((unsigned long long)(goff + i) >> 2);
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int n0 = 0; n0 < B; n0 += 256) {
            const int nb = min(256, B - n0);
            __syncthreads();
            if (threadIdx.x < nb) f_sh[threadIdx.x] = factor[(long long)(n0 + threadIdx.x) * f_stride + f_off];
            __syncthreads();
            if (live) {
                const float *g = G + (long long)n0 * P + i;
                int n = 0;
                for (; n + 4 <= nb; n += 4) {
                    float4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u] = __ldcs(reinterpret_cast<const float4 *>(g + (long long)(n + u) * P));
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float z[4];
                        example_normals4(nz.seed, nz.step, nz.example0 + (uint32_t)(n0 + n + u), block, z);
                        const float f = f_sh[n + u];
                        s.x += fmaf(f, v[u].x, nz.sd * z[0]); s.y += fmaf(f, v[u].y, nz.sd * z[1]);
                        s.z += fmaf(f, v[u].z, nz.sd * z[2]); s.w += fmaf(f, v[u].w, nz.sd * z[3]);
                    }
                }
                for (; n < nb; ++n) {
                    const float4 v = __ldcs(reinterpret_cast<const float4 *>(g + (long long)n * P));
                    float z[4];
                    example_normals4(nz.seed, nz.step, nz.example0 + (uint32_t)(n0 + n), block, z);
                    const float f = f_sh[n];
                    s.x += fmaf(f, v.x, nz.sd * z[0]); s.y += fmaf(f, v.y, nz.sd * z[1]);
                    s.z += fmaf(f, v.z, nz.sd * z[2]); s.w += fmaf(f, v.w, nz.sd * z[3]);
                }
            }
        }
        if (live) {
            float4 a = *reinterpret_cast<const float4 *>(acc + i);
            a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
            *reinterpret_cast<float4 *>(acc + i) = a;
        }
    } else {
        float s[4] = {0.f, 0.f, 0.f, 0.f};
        for (int n0 = 0; n0 < B; n0 += 256) {
            const int nb = min(256, B - n0);
            __syncthreads();
            if (threadIdx.x < nb) f_sh[threadIdx.x] = factor[(long long)(n0 + threadIdx.x) * f_stride + f_off];
            __syncthreads();
            for (int n = 0; n < nb; ++n) {
                const float f = f_sh[n];
                const float *g = G + (long long)(n0 + n) * P + c0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const long long i = threadIdx.x + 256 * q;
                    if (c0 + i < P) {
                        const unsigned long long gi = (unsigned long long)(goff + c0 + i);
                        float z[4];
                        example_normals4(nz.seed, nz.step, nz.example0 + (uint32_t)(n0 + n), (uint32_t)(gi >> 2), z);
                        s[q] += fmaf(f, g[i], nz.sd * z[gi & 3]);
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long i = c0 + threadIdx.x + 256 * q;
            if (i < P) acc[i] += s[q];
        }
    }
}

struct ClipPlan {
    size_t partial_off, sq_off, factor_off, total;
    long long parts_per_example;
};

static bool plan(int B, int L, const long long *P_l, ClipPlan &pl) {
    long long parts = 0;
    for (int l = 0; l < L; ++l) {
        if (P_l[l] <= 0) return false;
        parts += (P_l[l] + kNormChunk - 1) / kNormChunk;
    }
    pl.parts_per_example = parts;
    size_t off = 0;
    pl.partial_off = off; off = round_up(off + sizeof(float) * (size_t)parts * B, 256);
    pl.sq_off = off;      off = round_up(off + sizeof(float) * (size_t)B * L, 256);
    pl.factor_off = off;  off = round_up(off + sizeof(float) * (size_t)B * L, 256);
    pl.total = off;
    return true;
}

}  // namespace dp

extern "C" size_t dp_clip_workspace_bytes(int B, int L, const long long *P_l) {
    dp::ClipPlan pl;
    if (B <= 0 || L <= 0 || !P_l || !dp::plan(B, L, P_l, pl)) return 0;
    return pl.total;
}

namespace dp {
// What differs from plain dp_clip_accumulate in the other entry points.
struct ClipVariant {
    const ExampleNoise *noise = nullptr;   // stage 3 also adds each example's own noise draw ...
    const long long *goff_l = nullptr;     // ... addressed by the tensors' global offsets
    const GroupTable *groups = nullptr;    // factors per (example, group of tensors) instead of per tensor
    int micro = 1;                         // examples averaged before clipping
    const float *given_factor = nullptr;   // stage 3 only, with the caller's factors ([B] or [B, L]); no workspace
};

// Host side of dp_clip_accumulate and its variants.
static dp_status clip_accumulate_impl(int mode, int B, int L, const float *const *G, const long long *P_l,
                                      const float *sqnorm, float C, float *const *acc, float *norms_out,
                                      float *clip_out, void *workspace, size_t workspace_bytes, void *cuda_stream,
                                      const ClipVariant &var = ClipVariant()) {
    const ExampleNoise *noise = var.noise;
    const long long *goff_l = var.goff_l;
    const int micro = var.micro;
    if (mode != DP_CLIP_GLOBAL && mode != DP_CLIP_PER_LAYER) return DP_ERR_INVALID_ARG;
    if (B <= 0 || L <= 0 || !G || !P_l || !acc || !(C > 0.0f)) return DP_ERR_INVALID_ARG;
    if (B > 65535) return DP_ERR_UNSUPPORTED;
    const bool stage3_only = var.given_factor != nullptr;
    ClipPlan pl;
    if (!plan(B, L, P_l, pl)) return DP_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (!G[l] || !acc[l] || !aligned(G[l], 4) || !aligned(acc[l], 4)) return DP_ERR_INVALID_ARG;
        if ((P_l[l] + kSplitCols - 1) / kSplitCols > 0x3fffffffll) return DP_ERR_UNSUPPORTED;
    }
    if (sqnorm && !aligned(sqnorm, 4)) return DP_ERR_INVALID_ARG;
    if (!stage3_only && (!workspace || !aligned(workspace, 256) || workspace_bytes < pl.total)) return DP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    char *ws = static_cast<char *>(workspace);
    float *partial = stage3_only ? nullptr : reinterpret_cast<float *>(ws + pl.partial_off);
    float *sq_ws = stage3_only ? nullptr : reinterpret_cast<float *>(ws + pl.sq_off);
    const float *factor = stage3_only ? var.given_factor : reinterpret_cast<float *>(ws + pl.factor_off);
    float *factor_ws = stage3_only ? nullptr : reinterpret_cast<float *>(ws + pl.factor_off);
    const int per_layer = (mode == DP_CLIP_PER_LAYER);

    // tensors go to the kernels in tables of at most kMaxSeg entries
    long long wide_blocks = 0;
    for (int l = 0; l < L; ++l) wide_blocks += (P_l[l] + kAccCols - 1) / kAccCols;
    // A small model gives few blocks, and each thread would walk all B rows alone: with many rows the block narrows
    // to 128 parameters and its warps share the rows.
    const bool split = B >= 64 && wide_blocks < 8 * sm_count();
    const int acc_cols = (split && !noise) ? kSplitCols : kAccCols;

    auto fill = [&](int l0, SegTable &t, bool norm_blocks, long long &part_cursor) {
        t.nseg = 0;
        int blk = 0;
        for (int l = l0; l < L && t.nseg < kMaxSeg; ++l) {
            const int s = t.nseg++;
            t.G[s] = G[l]; t.acc[s] = acc[l]; t.P[s] = P_l[l]; t.col[s] = l;
            t.goff[s] = goff_l ? goff_l[l] : 0;
            t.blk_start[s] = blk;
            t.part_start[s] = part_cursor;
            const long long nparts = (P_l[l] + kNormChunk - 1) / kNormChunk;
            part_cursor += nparts;
            const long long nb = norm_blocks ? nparts : (P_l[l] + acc_cols - 1) / acc_cols;
            if ((long long)blk + nb > 0x7fffffffll) { --t.nseg; part_cursor -= nparts; break; }
            blk += (int)nb;
        }
        t.blk_start[t.nseg] = blk;
        return blk;
    };

    const float *sq = sqnorm;
    if (!sq && !stage3_only) {
        long long cursor = 0;
        for (int l0 = 0; l0 < L;) {
            SegTable t;
            const int blocks = fill(l0, t, true, cursor);
            if (t.nseg == 0) return DP_ERR_UNSUPPORTED;
            if (micro > 1)
                sqnorm_partial_micro_kernel<<<dim3((unsigned)blocks, (unsigned)(B / micro)), 256, 0, stream>>>(t, partial, pl.parts_per_example, micro);
            else
                sqnorm_partial_kernel<<<dim3((unsigned)blocks, (unsigned)B), 256, 0, stream>>>(t, partial, pl.parts_per_example);
            DP_LAUNCH_CHECK("sqnorm_partial_kernel");
            sqnorm_fold_kernel<<<dim3((unsigned)t.nseg, (unsigned)(B / micro)), 128, 0, stream>>>(t, partial, pl.parts_per_example, sq_ws, L);
            DP_LAUNCH_CHECK("sqnorm_fold_kernel");
            l0 += t.nseg;
        }
        sq = sq_ws;
    }
    if (!stage3_only) {
        const long long count = per_layer ? (long long)B * L : B;
        if (var.groups)
            clip_factor_grouped_kernel<<<(unsigned)B, 128, 0, stream>>>(sq, L, *var.groups, C, factor_ws, norms_out, clip_out);
        else if (micro > 1)
            clip_factor_micro_kernel<<<(unsigned)((B / micro + 127) / 128), 128, 0, stream>>>(sq, B / micro, L, micro, C, factor_ws, norms_out, clip_out);
        else
            clip_factor_kernel<<<(unsigned)((count + 127) / 128), 128, 0, stream>>>(sq, B, L, per_layer, C, factor_ws, norms_out, clip_out);
        DP_LAUNCH_CHECK("clip_factor_kernel");
    }
    {
        long long cursor = 0;
        for (int l0 = 0; l0 < L;) {
            SegTable t;
            const int blocks = fill(l0, t, false, cursor);
            if (t.nseg == 0) return DP_ERR_UNSUPPORTED;
            if (noise) scale_accumulate_noised_kernel<<<(unsigned)blocks, 256, 0, stream>>>(t, factor, B, L, per_layer, *noise);
            else if (split) scale_accumulate_rowsplit_kernel<<<(unsigned)blocks, 256, 0, stream>>>(t, factor, B, L, per_layer);
            else scale_accumulate_kernel<8><<<(unsigned)blocks, 256, 0, stream>>>(t, factor, B, L, per_layer);
            DP_LAUNCH_CHECK("scale_accumulate_kernel");
            l0 += t.nseg;
        }
    }
    return DP_OK;
}
}  // namespace dp

extern "C" dp_status dp_clip_accumulate(int mode, int B, int L, const float *const *G, const long long *P_l,
                                        const float *sqnorm, float C, float *const *acc, float *norms_out,
                                        float *clip_out, void *workspace, size_t workspace_bytes, void *cuda_stream) {
    return dp::clip_accumulate_impl(mode, B, L, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace, workspace_bytes,
                                    cuda_stream);
}

extern "C" dp_status dp_clip_factors(int mode, int B, int L, const float *sqnorm, float C, float *norms_out,
                                     float *factors_out, void *cuda_stream) {
    if (mode != DP_CLIP_GLOBAL && mode != DP_CLIP_PER_LAYER) return DP_ERR_INVALID_ARG;
    if (B <= 0 || L <= 0 || !sqnorm || !factors_out || !(C > 0.0f)) return DP_ERR_INVALID_ARG;
    if (!dp::aligned(sqnorm, 4) || !dp::aligned(factors_out, 4) || (norms_out && !dp::aligned(norms_out, 4))) return DP_ERR_INVALID_ARG;
    const int per_layer = (mode == DP_CLIP_PER_LAYER);
    const long long count = per_layer ? (long long)B * L : B;
    dp::clip_factor_kernel<<<(unsigned)((count + 127) / 128), 128, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        sqnorm, B, L, per_layer, C, factors_out, norms_out, nullptr);
    DP_LAUNCH_CHECK("clip_factor_kernel");
    return DP_OK;
}

extern "C" dp_status dp_scale_accumulate(int B, int L, const float *const *G, const long long *P_l, const float *factor,
                                         int per_tensor, float *const *acc, void *cuda_stream) {
    if (!factor || !dp::aligned(factor, 4) || (per_tensor != 0 && per_tensor != 1)) return DP_ERR_INVALID_ARG;
    dp::ClipVariant var;
    var.given_factor = factor;
    return dp::clip_accumulate_impl(per_tensor ? DP_CLIP_PER_LAYER : DP_CLIP_GLOBAL, B, L, G, P_l, nullptr, 1.0f, acc,
                                    nullptr, nullptr, nullptr, 0, cuda_stream, var);
}

extern "C" dp_status dp_clip_accumulate_grouped(int B, int L, int M, const int *group_of, const float *const *G,
                                                const long long *P_l, const float *sqnorm, float C, float *const *acc,
                                                float *norms_out, float *clip_out, void *workspace,
                                                size_t workspace_bytes, void *cuda_stream) {
    if (L <= 0 || M <= 0 || M > L || !group_of) return DP_ERR_INVALID_ARG;
    if (L > dp::kMaxGroupedTensors) return DP_ERR_UNSUPPORTED;
    dp::GroupTable gt;
    gt.M = M;
    unsigned char used[dp::kMaxGroupedTensors] = {0};
    for (int l = 0; l < L; ++l) {
        if (group_of[l] < 0 || group_of[l] >= M) return DP_ERR_INVALID_ARG;
        gt.of[l] = (unsigned short)group_of[l];
        used[group_of[l]] = 1;
    }
    for (int m = 0; m < M; ++m)
        if (!used[m]) return DP_ERR_INVALID_ARG;                 // an empty group would still count in C/sqrt(M)
    dp::ClipVariant var;
    var.groups = &gt;
    return dp::clip_accumulate_impl(DP_CLIP_PER_LAYER, B, L, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace,
                                    workspace_bytes, cuda_stream, var);
}

extern "C" dp_status dp_clip_accumulate_micro(int B, int L, int micro, const float *const *G, const long long *P_l,
                                              float C, float *const *acc, float *norms_out, float *clip_out,
                                              void *workspace, size_t workspace_bytes, void *cuda_stream) {
    if (micro <= 0 || B <= 0 || B % micro != 0) return DP_ERR_INVALID_ARG;
    dp::ClipVariant var;
    var.micro = micro;
    return dp::clip_accumulate_impl(DP_CLIP_GLOBAL, B, L, G, P_l, nullptr, C, acc, norms_out, clip_out, workspace,
                                    workspace_bytes, cuda_stream, var);
}

extern "C" dp_status dp_clip_accumulate_noised(int mode, int B, int L, const float *const *G, const long long *P_l,
                                               const long long *param_offset_l, const float *sqnorm, float C,
                                               float sigma, long long total_batch, unsigned long long seed,
                                               unsigned long long step, long long example0, float *const *acc,
                                               float *norms_out, float *clip_out, void *workspace,
                                               size_t workspace_bytes, void *cuda_stream) {
    if (!param_offset_l || L <= 0 || B <= 0 || !P_l) return DP_ERR_INVALID_ARG;
    if (!(sigma >= 0.0f) || isinf(sigma) || total_batch <= 0 || example0 < 0) return DP_ERR_INVALID_ARG;
    if (sigma > 0.0f && (isinf(C) || !(C > 0.0f))) return DP_ERR_INVALID_ARG;
    if (example0 + (long long)B > 0x80000000ll) return DP_ERR_INVALID_ARG;
    for (int l = 0; l < L; ++l) {
        if (param_offset_l[l] < 0 || P_l[l] <= 0) return DP_ERR_INVALID_ARG;
        if (((unsigned long long)param_offset_l[l] + (unsigned long long)P_l[l]) > (1ull << 34)) return DP_ERR_UNSUPPORTED;
    }
    if (sigma == 0.0f)
        return dp::clip_accumulate_impl(mode, B, L, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace,
                                        workspace_bytes, cuda_stream);
    dp::ExampleNoise nz;
    nz.sd = (float)((double)sigma * (double)C / sqrt((double)total_batch));
    nz.seed = seed; nz.step = step; nz.example0 = (uint32_t)example0;
    dp::ClipVariant var;
    var.noise = &nz;
    var.goff_l = param_offset_l;
    return dp::clip_accumulate_impl(mode, B, L, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace, workspace_bytes,
                                    cuda_stream, var);
}

// ----------------------------------------------------------------------------------------------------
// Variant of dp_clip_accumulate for callers that cannot supply scratch memory of their own.
// The scratch lives in this file-scope device array, so every GPU that loads the library carries
// kStaticScratchBytes of it until the process exits.
namespace dp {
constexpr size_t kStaticScratchBytes = 2u << 20;   // 2 MiB
static __device__ __align__(256) unsigned char g_clip_scratch[kStaticScratchBytes];

// Device address of g_clip_scratch on the current device.  In host code the array's name is only a
// stand-in for the symbol, never a usable address, so the address is asked for with the caller's
// device current.  It is asked for on every call (after the first one on a device this is a table
// look-up inside the runtime and allocates nothing), so no address outlives a cudaDeviceReset.
static dp_status static_scratch(void **out) {
    void *ptr = nullptr;
    DP_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_clip_scratch));
    if (!ptr) return cuda_fail(cudaErrorInvalidSymbol, "cudaGetSymbolAddress(g_clip_scratch)");
    *out = ptr;
    return DP_OK;
}
}  // namespace dp

extern "C" size_t dp_clip_static_scratch_bytes(void) { return dp::kStaticScratchBytes; }

extern "C" dp_status dp_clip_accumulate_static(int mode, int B, int L, const float *const *G, const long long *P_l,
                                               const float *sqnorm, float C, float *const *acc, float *norms_out,
                                               float *clip_out, void *cuda_stream) {
    if (B <= 0 || L <= 0 || !P_l) return DP_ERR_INVALID_ARG;
    const size_t need = dp_clip_workspace_bytes(B, L, P_l);
    if (need == 0) return DP_ERR_INVALID_ARG;
    if (need > dp::kStaticScratchBytes) {
        dp::note_error("dp_clip_accumulate_static: this problem needs more scratch than the built-in 2 MiB array; "
                       "use dp_clip_accumulate with a caller-owned workspace");
        return DP_ERR_WORKSPACE;
    }
    void *scratch = nullptr;
    const dp_status rc = dp::static_scratch(&scratch);
    if (rc != DP_OK) return rc;
    // every scratch word the kernels read is written earlier in the same call, so nothing needs clearing
    return dp_clip_accumulate(mode, B, L, G, P_l, sqnorm, C, acc, norms_out, clip_out, scratch, dp::kStaticScratchBytes,
                              cuda_stream);
}

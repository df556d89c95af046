// CUDA-core (fp32 FMA) per-example weight gradients: the any-shape path for convolutions, the
// dense outer product, the normalisation-affine reduction, bias sums, and the small kernels that
// fold per-tile squared norms into per-example norms and clip factors.
// Formulas: paper section 2 (per-example gradient, its L2 norm, clip) and section 3.5 (per-layer threshold).
#include "wgrad_simple.cuh"
#include <math.h>

namespace dp {

constexpr int TM = kFmaTile, TN = kFmaTile, TK = 16;

// Per-example gradient matrix D_n[m, j] = sum_q A[q, m] * Bm[q, j] with
//   A[q, m]  = dY[n, pix, m]                       q = n*K + pix
//   Bm[q, j] = Xpad[n, oh*st + r - pad, ow*st + s - pad, c],  j = (r*S + s)*Cin + c
// MODE 0/1: the block owns one example (blockIdx.z) and reduces q over that example's pixels.
// MODE 2:   the block owns the tile for a RANGE of examples (blockIdx.z picks the range): q runs over
//           those examples' pixels and A is scaled by the example's clip factor, so the accumulator ends
//           as sum_n f_n D_n[m, j].  With one range the sum is added to acc_w; with several, range z
//           writes its partial sum to sum_ws[z] and a fold kernel adds them in order.
template <typename T, int MODE>
__global__ void __launch_bounds__(256)
conv_wgrad_fma_kernel(const T *__restrict__ X, const T *__restrict__ dY, const ConvGeom g, float *__restrict__ G_w,
                      float *__restrict__ partial, int slots, const float *__restrict__ factor,
                      float *__restrict__ acc_w, int per_split, float *__restrict__ sum_ws) {
    __shared__ __align__(16) float sA[TK][TM];
    __shared__ __align__(16) float sB[TK][TN];
    __shared__ float scratch[32];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
    const int n_fixed = (MODE == 2) ? 0 : blockIdx.z;
    const long long q_begin = (MODE == 2) ? (long long)blockIdx.z * per_split * g.K : (long long)n_fixed * g.K;
    const long long q_end = (MODE == 2) ? (long long)min(g.B, ((int)blockIdx.z + 1) * per_split) * g.K : q_begin + g.K;
    const bool add_to_acc = (MODE == 2) && gridDim.z == 1;

    // loader role: this thread fills column lm of sA and column lj of sB for rows lp, lp+4, lp+8, lp+12
    const int lcol = tid & 63, lp = tid >> 6;
    const bool a_ok = (m0 + lcol) < g.M;
    const int jj = j0 + lcol;
    const bool b_ok = jj < g.N;
    const int c = b_ok ? jj % g.Cin : 0;
    const int rs = b_ok ? jj / g.Cin : 0;
    const int r = rs / g.S, s = rs % g.S;

    float ra[4], rb[4];
    auto fetch = [&](long long qc) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long q = qc + lp + 4 * i;
            ra[i] = 0.f; rb[i] = 0.f;
            if (q < q_end) {
                const int n = (int)(q / g.K);
                const int pix = (int)(q - (long long)n * g.K);
                if (a_ok) {
                    float v = to_float(dY[q * g.Kout + m0 + lcol]);
                    if (MODE == 2) v *= factor[2 * n];
                    ra[i] = v;
                }
                if (b_ok) {
                    const int oh = pix / g.OW, ow = pix - oh * g.OW;
                    const int ih = oh * g.stride + r - g.pad, iw = ow * g.stride + s - g.pad;
                    if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W)
                        rb[i] = to_float(X[(((long long)n * g.H + ih) * g.W + iw) * g.Cin + c]);
                }
            }
        }
    };

    const int ty = tid >> 4, tx = tid & 15;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[i][k] = 0.f;

    fetch(q_begin);
    for (long long qc = q_begin; qc < q_end; qc += TK) {
#pragma unroll
        for (int i = 0; i < 4; ++i) { sA[lp + 4 * i][lcol] = ra[i]; sB[lp + 4 * i][lcol] = rb[i]; }
        __syncthreads();
        if (qc + TK < q_end) fetch(qc + TK);
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            const float4 a = *reinterpret_cast<const float4 *>(&sA[kk][ty * 4]);
            const float4 b = *reinterpret_cast<const float4 *>(&sB[kk][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int k = 0; k < 4; ++k) acc[i][k] = fmaf(av[i], bv[k], acc[i][k]);
        }
        __syncthreads();
    }

    const int jb = j0 + tx * 4;
    if (MODE == 0 || MODE == 1) {
        float sq = 0.f;   // rows / columns outside the matrix hold exact zeros, no masking needed
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) sq = fmaf(acc[i][k], acc[i][k], sq);
        sq = block_sum(sq, scratch);
        if (tid == 0) partial[(long long)n_fixed * slots + blockIdx.y * gridDim.x + blockIdx.x] = sq;
    }
    if (MODE == 0 || MODE == 2) {
        float *base = (MODE == 0) ? G_w + (long long)n_fixed * g.M * g.N
                                  : (add_to_acc ? acc_w : sum_ws + (long long)blockIdx.z * g.M * g.N);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int m = m0 + ty * 4 + i;
            if (m >= g.M) continue;
            float *row = base + (long long)m * g.N;
            if ((g.N & 3) == 0) {
                if (jb < g.N) {
                    float4 v = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
                    if (add_to_acc) {
                        const float4 o = *reinterpret_cast<const float4 *>(row + jb);
                        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
                    }
                    *reinterpret_cast<float4 *>(row + jb) = v;
                }
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (jb + k < g.N) row[jb + k] = add_to_acc ? row[jb + k] + acc[i][k] : acc[i][k];
            }
        }
    }
}

// Thin convolutions (R*S*Cin <= 32 columns, e.g. a 3x3 conv on RGB): one block per example.  The zero-padded
// input of the example sits in shared memory; thread = (pixel group, output channel lane) keeps one gradient row
// (all columns) per owned output channel in registers and walks its share of the pixels, reading dY coalesced and
// the input patch by shared-memory broadcast.  The eight pixel groups are folded in order; the bias gradient and
// both squared norms come out of the same pass.
// RT x SCT > 0 fixes the filter rows and the run length S*Cin at compile time (3 x 9 for a 3x3 conv on RGB), which
// turns every patch read into a shared-memory load with an immediate offset; RT = 0 is the any-shape version.
template <typename T, int KPT, int RT, int SCT>
__global__ void __launch_bounds__(256)
conv_wgrad_thin_kernel(const T *__restrict__ X, const T *__restrict__ dY, const ConvGeom g, float *__restrict__ G_w,
                       float *__restrict__ db, float *__restrict__ partial, int slots, int has_bias) {
    extern __shared__ float thin_smem[];
    __shared__ float scratch[32];
    const int Hp = g.H + 2 * g.pad, Wp = g.W + 2 * g.pad;
    const int xs_count = Hp * Wp * g.Cin;
    float *xs = thin_smem;                                   // [Hp][Wp][Cin], zero border
    float *red = thin_smem + ((xs_count + 3) & ~3);          // [8][Kout*N] then [8][Kout]
    const int n = blockIdx.x, lane = threadIdx.x & 31, pg = threadIdx.x >> 5;
    {
        const int row_in = g.W * g.Cin, row_p = Wp * g.Cin;
        for (int i = threadIdx.x; i < xs_count; i += 256) xs[i] = 0.f;
        __syncthreads();
        const T *Xn = X + (long long)n * g.H * row_in;
        for (int i = threadIdx.x; i < g.H * row_in; i += 256) {
            const int h = i / row_in, rest = i - h * row_in;
            xs[(h + g.pad) * row_p + g.pad * g.Cin + rest] = to_float(Xn[i]);
        }
    }
    int off[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const int jj = j < g.N ? j : 0;
        const int c = jj % g.Cin, rs = jj / g.Cin;
        off[j] = ((rs / g.S) * Wp + rs % g.S) * g.Cin + c;
    }
    float acc[KPT][32], bsum[KPT];
#pragma unroll
    for (int kk = 0; kk < KPT; ++kk) {
        bsum[kk] = 0.f;
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[kk][j] = 0.f;
    }
    __syncthreads();
    int oh = pg / g.OW, ow = pg - oh * g.OW;
    const T *dYn = dY + (long long)n * g.K * g.Kout;
    // U pixels per trip, and the next trip's dY loads are issued before this trip's arithmetic: a warp always has
    // U (then 2U) 128-byte rows in flight, which is what hides the memory latency at one or two blocks per SM.
    constexpr int U = 8;
    float gy[U][KPT], gyn[U][KPT];
    int base[U], basen[U];
    auto load_trip = [&](int pix, float (&y)[U][KPT], int (&b)[U]) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int pu = pix + 8 * u;
            b[u] = pu < g.K ? (oh * g.stride * Wp + ow * g.stride) * g.Cin : 0;
#pragma unroll
            for (int kk = 0; kk < KPT; ++kk)
                y[u][kk] = pu < g.K ? to_float(dYn[(long long)pu * g.Kout + lane + 32 * kk]) : 0.f;
            ow += 8;
            while (ow >= g.OW) { ow -= g.OW; ++oh; }
        }
    };
    load_trip(pg, gy, base);
    for (int pix = pg; pix < g.K; pix += 8 * U) {
        if (pix + 8 * U < g.K) load_trip(pix + 8 * U, gyn, basen);
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int kk = 0; kk < KPT; ++kk) bsum[kk] += gy[u][kk];
            if constexpr (RT > 0) {
                const float *patch = xs + base[u];
                const int row_p = Wp * g.Cin;
                // the whole warp reads the same patch (broadcast); 64-bit loads halve the shared-memory instructions,
                // with the pairing chosen by the parity of the patch start (the same for every lane and every row)
                const bool pairs = ((row_p | SCT) & 1) != 0 ? ((row_p & 1) == 0) : true;
                const int lead = (base[u] & 1);          // 1: element 0 is unaligned, pairs start at element 1
#pragma unroll
                for (int r = 0; r < RT; ++r) {
                    float x[SCT];
                    const float *row = patch + r * row_p;
                    if (pairs && (row_p & 1) == 0) {
                        if (lead == 0) {
#pragma unroll
                            for (int t = 0; t + 1 < SCT; t += 2) { const float2 v = *reinterpret_cast<const float2 *>(row + t); x[t] = v.x; x[t + 1] = v.y; }
                            if (SCT & 1) x[SCT - 1] = row[SCT - 1];
                        } else {
                            x[0] = row[0];
#pragma unroll
                            for (int t = 1; t + 1 < SCT; t += 2) { const float2 v = *reinterpret_cast<const float2 *>(row + t); x[t] = v.x; x[t + 1] = v.y; }
                            if (!(SCT & 1)) x[SCT - 1] = row[SCT - 1];
                        }
                    } else {
#pragma unroll
                        for (int t = 0; t < SCT; ++t) x[t] = row[t];
                    }
#pragma unroll
                    for (int t = 0; t < SCT; ++t) {
#pragma unroll
                        for (int kk = 0; kk < KPT; ++kk) acc[kk][r * SCT + t] = fmaf(gy[u][kk], x[t], acc[kk][r * SCT + t]);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    if (j < g.N) {
                        const float x = xs[base[u] + off[j]];
#pragma unroll
                        for (int kk = 0; kk < KPT; ++kk) acc[kk][j] = fmaf(gy[u][kk], x, acc[kk][j]);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            base[u] = basen[u];
#pragma unroll
            for (int kk = 0; kk < KPT; ++kk) gy[u][kk] = gyn[u][kk];
        }
    }
    const int MN = g.Kout * g.N;
    float *bred = red + 8 * MN;
#pragma unroll
    for (int kk = 0; kk < KPT; ++kk) {
        const int k = lane + 32 * kk;
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (j < g.N) red[pg * MN + k * g.N + j] = acc[kk][j];
        bred[pg * g.Kout + k] = bsum[kk];
    }
    __syncthreads();
    float sq = 0.f, sqb = 0.f;
    for (int t = threadIdx.x; t < MN; t += 256) {
        float v = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) v += red[q * MN + t];
        if (G_w) G_w[(long long)n * MN + t] = v;
        sq = fmaf(v, v, sq);
    }
    if (has_bias) {
        for (int k = threadIdx.x; k < g.Kout; k += 256) {
            float v = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) v += bred[q * g.Kout + k];
            db[(long long)n * g.Kout + k] = v;
            sqb = fmaf(v, v, sqb);
        }
    }
    sq = block_sum(sq, scratch);
    sqb = block_sum(sqb, scratch);
    if (threadIdx.x == 0) {
        partial[(long long)n * slots] = sq;
        if (has_bias) partial[(long long)n * slots + 1] = sqb;
    }
}

static size_t thin_smem_bytes(const ConvGeom &g) {
    const size_t xs = ((size_t)(g.H + 2 * g.pad) * (g.W + 2 * g.pad) * g.Cin + 3) & ~(size_t)3;
    return sizeof(float) * (xs + 8 * (size_t)g.Kout * g.N + 8 * (size_t)g.Kout);
}

bool thin_conv_eligible(const ConvGeom &g) {
    return g.N <= 32 && (g.Kout == 32 || g.Kout == 64) && g.K >= 8 && thin_smem_bytes(g) <= 47 * 1024 && g.B <= 0x7fffffff;
}

template <typename T, int KPT>
static void thin_launch_t(const T *X, const T *dY, const ConvGeom &g, float *G_w, float *db, float *partial, int slots,
                          int has_bias, size_t smem, cudaStream_t st) {
    if (g.R == 3 && g.S * g.Cin == 9)
        conv_wgrad_thin_kernel<T, KPT, 3, 9><<<g.B, 256, smem, st>>>(X, dY, g, G_w, db, partial, slots, has_bias);
    else
        conv_wgrad_thin_kernel<T, KPT, 0, 0><<<g.B, 256, smem, st>>>(X, dY, g, G_w, db, partial, slots, has_bias);
}

dp_status launch_conv_thin(int dtype, const void *X, const void *dY, const ConvGeom &g, float *G_w, float *db,
                           float *partial, int slots, int has_bias, cudaStream_t st) {
    const size_t smem = thin_smem_bytes(g);
    if (dtype == DP_F32) {
        if (g.Kout == 32) thin_launch_t<float, 1>(static_cast<const float *>(X), static_cast<const float *>(dY), g, G_w, db, partial, slots, has_bias, smem, st);
        else thin_launch_t<float, 2>(static_cast<const float *>(X), static_cast<const float *>(dY), g, G_w, db, partial, slots, has_bias, smem, st);
    } else {
        if (g.Kout == 32) thin_launch_t<__nv_bfloat16, 1>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), g, G_w, db, partial, slots, has_bias, smem, st);
        else thin_launch_t<__nv_bfloat16, 2>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), g, G_w, db, partial, slots, has_bias, smem, st);
    }
    DP_LAUNCH_CHECK("conv_wgrad_thin_kernel");
    return DP_OK;
}

// 3x3 convolutions on three input channels (image stems), output channels a multiple of 32: one block per example,
// the zero-padded image in shared memory.  Lane = output pixel (32 consecutive pixels per trip), warp w owns output
// channels 4w .. 4w+3 of the current group of 32, so a thread keeps a 4 x 27 block of the gradient in registers, every
// shared-memory word it reads feeds four FMAs, and the 32 lanes read 32 different words (3 floats apart: no bank
// conflict) instead of one broadcast word.  A trip is short (a few hundred cycles) against the memory latency, so dY
// streams through a ring of kRgbStages stages of 64 pixels x 32 channels, filled by coalesced asynchronous copies
// (cp.async, each thread two pieces of four channels per stage) three stages ahead of the arithmetic, one barrier per
// stage.  Inside a stage the piece of (pixel l, channel quad c) sits at quad position c ^ (l & 7) of its pixel row, so
// that the 32 lanes of a warp, which read the same quad of 32 different pixels, hit different banks.  The 32 pixel
// lanes are folded by two shuffle steps and then, in lane order, through shared memory; gradient, bias gradient and
// the example's squared norms leave from the same pass.
constexpr int kRgbRed = 113;      // floats per (warp, lane group) in the fold buffer: 4 x 27 weights + 4 bias sums (+1: odd stride)
constexpr int kRgbStages = 4;     // stages of dY in the ring
constexpr int kRgbStagePix = 64;  // pixels per stage (two trips)
constexpr int kRgbStageFloats = kRgbStagePix * 32;   // ring stride in 4-byte words (bf16 stages use half of it)

template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(void *smem_dst, const void *src, bool valid) {
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    const int n = valid ? BYTES : 0;                          // 0 source bytes: the destination is zero-filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2, %3;\n" ::"r"(dst), "l"(src), "n"(BYTES), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <typename T>
__global__ void __launch_bounds__(256, 2)
conv_wgrad_rgb3_kernel(const T *__restrict__ X, const T *__restrict__ dY, const ConvGeom g, float *__restrict__ G_w,
                       float *__restrict__ db, int has_bias, int separate, float *__restrict__ sqnorm,
                       long long sq_stride) {
    extern __shared__ __align__(16) float rgb_smem[];
    __shared__ double scratch[32];
    constexpr int kQuad = 4 * (int)sizeof(T);                // bytes of four output channels of dY
    const int Hp = g.H + 2 * g.pad, Wp = g.W + 2 * g.pad, row_p = Wp * 3;
    const int xs_count = Hp * row_p;
    char *ring = reinterpret_cast<char *>(rgb_smem);         // [kRgbStages][64 pixels][8 quads]; afterwards the fold
    float *red = rgb_smem;                                   //   buffer [8 warps][8 lane groups][kRgbRed]
    float *xs = rgb_smem + kRgbStages * kRgbStageFloats;     // [Hp][Wp][3], zero border
    const int n = blockIdx.x, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    {
        const int row_in = g.W * 3;
        for (int i = threadIdx.x; i < xs_count; i += 256) xs[i] = 0.f;
        __syncthreads();
        const T *Xn = X + (long long)n * g.H * row_in;
        for (int i = threadIdx.x; i < g.H * row_in; i += 256) {
            const int h = i / row_in, rest = i - h * row_in;
            xs[(h + g.pad) * row_p + g.pad * 3 + rest] = to_float(Xn[i]);
        }
    }
    float sq = 0.f, sqb = 0.f;
    const int stages = (g.K + kRgbStagePix - 1) / kRgbStagePix;
    // copies of this thread: quad cq of pixels cl and cl + 32 of a stage; reads: quad w of pixel lane (+32 on the second trip)
    const int cl = threadIdx.x >> 3, cq = threadIdx.x & 7;
    const int copy_off = cl * 8 * kQuad + ((cq ^ (cl & 7)) * kQuad);        // (cl + 32) & 7 == cl & 7
    const int read_off = lane * 8 * kQuad + ((w ^ (lane & 7)) * kQuad);
    for (int kg = 0; kg < g.Kout / 32; ++kg) {
        const T *dyp = dY + (long long)n * g.K * g.Kout + kg * 32;
        auto fetch = [&](int stage) {                        // one commit group per stage, also past the end
            char *dst = ring + (stage % kRgbStages) * (kRgbStageFloats * 4) + copy_off;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int p = stage * kRgbStagePix + cl + 32 * h;
                const bool valid = stage < stages && p < g.K;
                cp_async_zfill<kQuad>(dst + h * 32 * 8 * kQuad, dyp + (long long)(valid ? p : 0) * g.Kout + 4 * cq, valid);
            }
            cp_async_commit();
        };
        float acc[4][27], bs[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
#pragma unroll
            for (int j = 0; j < 27; ++j) acc[kk][j] = 0.f;
        for (int t = 0; t < kRgbStages - 1; ++t) fetch(t);
        int oh = lane / g.OW, ow = lane - oh * g.OW;         // pixel of this lane in the current trip
        for (int st = 0; st < stages; ++st) {
            cp_async_wait<kRgbStages - 2>();                 // this thread's pieces of stage st have landed
            __syncthreads();                                 // ... and everyone's; stage st-1 is no longer read
            fetch(st + kRgbStages - 1);                      // refills the slot of stage st-1
            const char *src = ring + (st % kRgbStages) * (kRgbStageFloats * 4) + read_off;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float gy[4];
                if constexpr (sizeof(T) == 4) {
                    const float4 v = *reinterpret_cast<const float4 *>(src + h * 32 * 8 * kQuad);
                    gy[0] = v.x; gy[1] = v.y; gy[2] = v.z; gy[3] = v.w;
                } else {
                    const uint2 v = *reinterpret_cast<const uint2 *>(src + h * 32 * 8 * kQuad);
                    gy[0] = __uint_as_float(v.x << 16); gy[1] = __uint_as_float(v.x & 0xffff0000u);
                    gy[2] = __uint_as_float(v.y << 16); gy[3] = __uint_as_float(v.y & 0xffff0000u);
                }
                // lanes past the last pixel carry zeros of dY; their patch address is clamped to pixel 0
                const bool live = st * kRgbStagePix + 32 * h + lane < g.K;
                const float *patch = xs + (live ? (oh * g.stride * Wp + ow * g.stride) * 3 : 0);
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    float x[9];
#pragma unroll
                    for (int q = 0; q < 9; ++q) x[q] = patch[r * row_p + q];
#pragma unroll
                    for (int q = 0; q < 9; ++q)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) acc[kk][r * 9 + q] = fmaf(gy[kk], x[q], acc[kk][r * 9 + q]);
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) bs[kk] += gy[kk];
                ow += 32;
                while (ow >= g.OW) { ow -= g.OW; ++oh; }
            }
        }
        cp_async_wait<0>();
        __syncthreads();                                     // every thread is done with the ring: it becomes the fold buffer
        // fold the 32 pixel lanes: two butterfly steps leave eight partial sums (lanes 0..7), added in lane order below
        float *mine = red + (w * 8 + (lane & 7)) * kRgbRed;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int j = 0; j < 27; ++j) {
                float v = acc[kk][j];
                v += __shfl_xor_sync(0xffffffffu, v, 16);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                if (lane < 8) mine[kk * 27 + j] = v;
            }
            float v = bs[kk];
            v += __shfl_xor_sync(0xffffffffu, v, 16);
            v += __shfl_xor_sync(0xffffffffu, v, 8);
            if (lane < 8) mine[108 + kk] = v;
        }
        __syncthreads();
        // entry o of this group of 32 channels is (warp o/108, register o%108) and sits at G_w[n][kg*864 + o]
        for (int o = threadIdx.x; o < 864; o += 256) {
            const float *src = red + (o / 108) * 8 * kRgbRed + (o % 108);
            float v = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) v += src[q * kRgbRed];
            if (G_w) G_w[(long long)n * g.Kout * 27 + kg * 864 + o] = v;
            sq = fmaf(v, v, sq);
        }
        if (has_bias && threadIdx.x < 32) {
            const float *src = red + (threadIdx.x >> 2) * 8 * kRgbRed + 108 + (threadIdx.x & 3);
            float v = 0.f;
#pragma unroll
            for (int q = 0; q < 8; ++q) v += src[q * kRgbRed];
            db[(long long)n * g.Kout + kg * 32 + threadIdx.x] = v;
            sqb = fmaf(v, v, sqb);
        }
        __syncthreads();
    }
    const double sw = block_sum((double)sq, scratch);
    const double sb = block_sum((double)sqb, scratch);
    if (threadIdx.x == 0) {
        if (separate) {
            sqnorm[n * sq_stride] = (float)sw;
            sqnorm[n * sq_stride + 1] = (float)sb;
        } else {
            sqnorm[n * sq_stride] = (float)(sw + sb);
        }
    }
}

static size_t rgb3_smem_bytes(const ConvGeom &g) {
    static_assert(kRgbStages * kRgbStageFloats >= 8 * 8 * kRgbRed, "the fold buffer reuses the dY ring");
    const size_t xs = ((size_t)(g.H + 2 * g.pad) * (g.W + 2 * g.pad) * 3 + 3) & ~(size_t)3;
    return sizeof(float) * (xs + (size_t)kRgbStages * kRgbStageFloats);
}

bool rgb3_conv_eligible(const ConvGeom &g) {
    return g.R == 3 && g.S == 3 && g.Cin == 3 && g.Kout % 32 == 0 && g.Kout <= 256 && rgb3_smem_bytes(g) <= 47 * 1024;
}

dp_status launch_conv_rgb3(int dtype, const void *X, const void *dY, const ConvGeom &g, float *G_w, float *db,
                           int has_bias, int separate, float *sqnorm, long long sq_stride,
                           cudaStream_t st) {
    const size_t smem = rgb3_smem_bytes(g);
    if (dtype == DP_F32)
        conv_wgrad_rgb3_kernel<float><<<g.B, 256, smem, st>>>(static_cast<const float *>(X), static_cast<const float *>(dY), g,
                                                              G_w, db, has_bias, separate, sqnorm, sq_stride);
    else
        conv_wgrad_rgb3_kernel<__nv_bfloat16><<<g.B, 256, smem, st>>>(static_cast<const __nv_bfloat16 *>(X),
                                                                      static_cast<const __nv_bfloat16 *>(dY), g, G_w, db,
                                                                      has_bias, separate, sqnorm, sq_stride);
    DP_LAUNCH_CHECK("conv_wgrad_rgb3_kernel");
    return DP_OK;
}

// db[n, k] = sum over pixels of dY[n, pix, k]; 64 channels x 4 pixel lanes per block, lanes folded in order.
template <typename T>
__global__ void __launch_bounds__(256)
bias_kernel(const T *__restrict__ dY, int K, int Kout, float *__restrict__ db, float *__restrict__ partial, int slots,
            int slot0) {
    __shared__ float lanes[4][kBiasCols];
    __shared__ float scratch[32];
    const int n = blockIdx.y, col = threadIdx.x & 63, lane = threadIdx.x >> 6;
    const int k = blockIdx.x * kBiasCols + col;
    float a = 0.f;
    if (k < Kout) {
        const T *p = dY + (long long)n * K * Kout + k;
        for (int pix = lane; pix < K; pix += 4) a += to_float(p[(long long)pix * Kout]);
    }
    lanes[lane][col] = a;
    __syncthreads();
    float sq = 0.f;
    if (lane == 0 && k < Kout) {
        const float v = (lanes[0][col] + lanes[1][col]) + (lanes[2][col] + lanes[3][col]);
        db[(long long)n * Kout + k] = v;
        sq = v * v;
    }
    sq = block_sum(sq, scratch);
    if (threadIdx.x == 0) partial[(long long)n * slots + slot0 + blockIdx.x] = sq;
}

// Vectorised variant for channel counts that are a multiple of one 16-byte vector (and at most 256 vectors):
// one block per example, thread = (pixel row, channel vector), 16-byte loads, pixel rows folded in order.
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
bias_vec_kernel(const T *__restrict__ dY, int K, int Kout, float *__restrict__ db, float *__restrict__ partial, int slots,
                int slot0, int bias_slots) {
    extern __shared__ float red[];                     // [rows][Kout]
    __shared__ float scratch[32];
    const int n = blockIdx.x;
    const int lanes_k = Kout / VEC, rows = 256 / lanes_k;
    const int prow = threadIdx.x / lanes_k, kv = threadIdx.x - prow * lanes_k;
    float a[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) a[v] = 0.f;
    if (prow < rows) {
        const T *base = dY + (long long)n * K * Kout + kv * VEC;
        // eight pixels per trip, all loads issued before any addition (a block is one example: few threads, so the
        // loads in flight per thread are what hides the memory latency); pixels still add in pixel order
        for (int pix = prow; pix < K; pix += 8 * rows) {
            uint4 g[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                if (pix + u * rows < K) g[u] = __ldcs(reinterpret_cast<const uint4 *>(base + (long long)(pix + u * rows) * Kout));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (pix + u * rows < K) {
                    const T *gv = reinterpret_cast<const T *>(&g[u]);
#pragma unroll
                    for (int v = 0; v < VEC; ++v) a[v] += to_float(gv[v]);
                }
            }
        }
#pragma unroll
        for (int v = 0; v < VEC; ++v) red[prow * Kout + kv * VEC + v] = a[v];
    }
    __syncthreads();
    float sq = 0.f;
    for (int k = threadIdx.x; k < Kout; k += 256) {
        float v = 0.f;
        for (int r = 0; r < rows; ++r) v += red[r * Kout + k];
        db[(long long)n * Kout + k] = v;
        sq = fmaf(v, v, sq);
    }
    sq = block_sum(sq, scratch);
    if (threadIdx.x < bias_slots) partial[(long long)n * slots + slot0 + threadIdx.x] = (threadIdx.x == 0) ? sq : 0.f;
}

// One block per example: weight slots [0, w_slots) and bias slots [w_slots, slots) summed in index order.
__global__ void __launch_bounds__(128)
finalize_norm_kernel(const float *__restrict__ partial, int slots, int w_slots, int separate, float *__restrict__ sqnorm,
                     long long sq_stride, int clip, float C_l, float *__restrict__ factor, float *clip_out) {
    __shared__ double scratch[32];
    const int n = blockIdx.x;
    const float *p = partial + (long long)n * slots;
    double sw = 0.0, sb = 0.0;
    for (int i = threadIdx.x; i < w_slots; i += 128) sw += (double)p[i];
    for (int i = w_slots + threadIdx.x; i < slots; i += 128) sb += (double)p[i];
    sw = block_sum(sw, scratch);
    sb = block_sum(sb, scratch);
    if (threadIdx.x != 0) return;
    if (separate) {
        sqnorm[n * sq_stride] = (float)sw;
        sqnorm[n * sq_stride + 1] = (float)sb;
        if (clip) {
            const float fw = clip_factor(sw, C_l), fb = clip_factor(sb, C_l);
            factor[2 * n] = fw; factor[2 * n + 1] = fb;
            if (clip_out) { clip_out[2 * n] = fw; clip_out[2 * n + 1] = fb; }
        }
    } else {
        const double s = sw + sb;
        sqnorm[n * sq_stride] = (float)s;
        if (clip) {
            const float f = clip_factor(s, C_l);
            factor[2 * n] = f; factor[2 * n + 1] = f;
            if (clip_out) clip_out[n] = f;
        }
    }
}

// acc[k] += sum_n f[n * f_stride] * v[n, k].  Block = 32 channels x 8 example groups (group q owns examples
// q, q+8, ...), groups folded in order.
template <typename T>
__global__ void __launch_bounds__(256)
bias_accum_kernel(const T *__restrict__ db, int B, int Kout, const float *__restrict__ f, long long f_stride,
                  float *__restrict__ acc_b) {
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, q = threadIdx.x >> 5;
    const int k = blockIdx.x * 32 + lane;
    float a = 0.f;
    if (k < Kout) {
#pragma unroll 8
        for (int n = q; n < B; n += 8) a = fmaf(f[n * f_stride], to_float(db[(long long)n * Kout + k]), a);
    }
    part[q][lane] = a;
    __syncthreads();
    if (q == 0 && k < Kout) {
        float t = part[0][lane];
#pragma unroll
        for (int i = 1; i < 8; ++i) t += part[i][lane];
        acc_b[k] += t;
    }
}

// Dense layer, clipped sum with known factors: acc[o, i] += sum_n (f_n dY[n, o]) X[n, i], a matrix product with the
// batch as the reduction axis and a tiny output.  Block = 32 input columns x 16 outputs; its eight warps share the
// examples (warp q owns q, q+8, ...), the scaled dY rows sit in shared memory, and the eight partial tiles are folded
// in warp order.  Bound by latency and by the accumulator's read-modify-write, not by arithmetic.
constexpr int kDenseOT = 16;
template <typename T>
__global__ void __launch_bounds__(256)
dense_scaled_sum_kernel(const T *__restrict__ X, const T *__restrict__ dY, const float *__restrict__ factor,
                        long long f_stride, int B, int Cin, int Kout, float *__restrict__ acc,
                        const float *__restrict__ factor_b, long long fb_stride, float *__restrict__ acc_b) {
    __shared__ __align__(16) float fy[256][kDenseOT];
    __shared__ float part[8][kDenseOT][32];
    __shared__ float bsum[16][kDenseOT];
    // the bias gradient of a dense layer is dY itself: the first column block of every output group also adds
    // acc_b[o] += sum_n fb_n dY[n, o] (16 outputs x 16 example groups, groups folded in order), which saves a launch
    if (acc_b && blockIdx.x == 0) {
        const int o = threadIdx.x & (kDenseOT - 1), gq = threadIdx.x >> 4, oo = blockIdx.y * kDenseOT + o;
        float sum = 0.f;
        if (oo < Kout) {
#pragma unroll 8
            for (int n = gq; n < B; n += 16) sum = fmaf(factor_b[n * fb_stride], to_float(dY[(long long)n * Kout + oo]), sum);
        }
        bsum[gq][o] = sum;
        __syncthreads();
        if (threadIdx.x < kDenseOT && blockIdx.y * kDenseOT + threadIdx.x < Kout) {
            float t = bsum[0][threadIdx.x];
#pragma unroll
            for (int g2 = 1; g2 < 16; ++g2) t += bsum[g2][threadIdx.x];
            acc_b[blockIdx.y * kDenseOT + threadIdx.x] += t;
        }
    }
    const int lane = threadIdx.x & 31, q = threadIdx.x >> 5;
    const int i = blockIdx.x * 32 + lane, o0 = blockIdx.y * kDenseOT;
    float a[kDenseOT];
#pragma unroll
    for (int o = 0; o < kDenseOT; ++o) a[o] = 0.f;
    for (int n0 = 0; n0 < B; n0 += 256) {
        const int nb = min(256, B - n0);
        __syncthreads();
        for (int t = threadIdx.x; t < nb * kDenseOT; t += 256) {
            const int n = t / kDenseOT, o = t - n * kDenseOT;
            fy[n][o] = (o0 + o < Kout) ? factor[(n0 + n) * f_stride] * to_float(dY[(long long)(n0 + n) * Kout + o0 + o]) : 0.f;
        }
        __syncthreads();
        if (i < Cin) {
#pragma unroll 8
            for (int n = q; n < nb; n += 8) {
                const float x = to_float(X[(long long)(n0 + n) * Cin + i]);
                const float4 *row = reinterpret_cast<const float4 *>(fy[n]);
#pragma unroll
                for (int v = 0; v < kDenseOT / 4; ++v) {
                    const float4 y = row[v];
                    a[4 * v] = fmaf(y.x, x, a[4 * v]); a[4 * v + 1] = fmaf(y.y, x, a[4 * v + 1]);
                    a[4 * v + 2] = fmaf(y.z, x, a[4 * v + 2]); a[4 * v + 3] = fmaf(y.w, x, a[4 * v + 3]);
                }
            }
        }
    }
#pragma unroll
    for (int o = 0; o < kDenseOT; ++o) part[q][o][lane] = a[o];
    __syncthreads();
    // 512 tile entries, two per thread: entry e = (output e / 32, column e % 32)
    for (int e = threadIdx.x; e < kDenseOT * 32; e += 256) {
        const int o = e >> 5, c = e & 31;
        if (o0 + o < Kout && blockIdx.x * 32 + c < Cin) {
            float t = part[0][o][c];
#pragma unroll
            for (int w = 1; w < 8; ++w) t += part[w][o][c];
            acc[(long long)(o0 + o) * Cin + blockIdx.x * 32 + c] += t;
        }
    }
}

// factor2[n] = (factor_w[n*stride], factor_b[n*stride]): caller-supplied factors in the layout the clipped-sum kernels read
__global__ void expand_factor_kernel(const float *__restrict__ factor_w, const float *__restrict__ factor_b,
                                     long long stride, int B, float *__restrict__ factor2) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= B) return;
    factor2[2 * n] = factor_w[n * stride];
    factor2[2 * n + 1] = factor_b[n * stride];
}

// ------------------------------------------------------------------ dense layer
// G_w[n, o, i] = dY[n, o] * X[n, i]: pure store stream.  One block per (example, output) row of the result,
// four columns per thread when Cin % 4 == 0.
template <typename T, bool VEC>
__global__ void __launch_bounds__(256)
dense_store_kernel(const T *__restrict__ X, const T *__restrict__ dY, int Cin, int Kout, int rows_per_block,
                   long long total_rows, float *__restrict__ G_w) {
    for (int rr = 0; rr < rows_per_block; ++rr) {
        const long long row = (long long)blockIdx.x * rows_per_block + rr;      // n * Kout + o
        if (row >= total_rows) return;
        const long long n = row / Kout;
        const float gy = to_float(dY[row]);
        const T *x = X + n * Cin;
        float *out = G_w + row * Cin;
        if (VEC) {
            for (int i = threadIdx.x * 4; i < Cin; i += 1024) {
                const float4 v = make_float4(gy * to_float(x[i]), gy * to_float(x[i + 1]), gy * to_float(x[i + 2]), gy * to_float(x[i + 3]));
                __stcs(reinterpret_cast<float4 *>(out + i), v);
            }
        } else {
            for (int i = threadIdx.x; i < Cin; i += 256) out[i] = gy * to_float(x[i]);
        }
    }
}


// Dense layer, everything but the outer-product store, one block per example: the rank-1 closed form of the squared
// norm (|dY_n^T X_n|_F^2 = |dY_n|^2 |X_n|^2, bias part |dY_n|^2), the bias gradient db_n = dY_n widened to fp32 (when
// a destination is given), and the same publishing of norms / clip factors the convolution paths do in a kernel of its own.
template <typename T>
__global__ void __launch_bounds__(256)
dense_norm_kernel(const T *__restrict__ X, const T *__restrict__ dY, int Cin, int Kout, int has_bias, float *__restrict__ db,
                  int separate, float *__restrict__ sqnorm, long long sq_stride, int clip, float C_l,
                  float *__restrict__ factor, float *clip_out) {
    __shared__ double scratch[32];
    const int n = blockIdx.x;
    double sx = 0.0, sy = 0.0;
    for (int i = threadIdx.x; i < Cin; i += 256) { const double v = to_float(X[(long long)n * Cin + i]); sx += v * v; }
    for (int i = threadIdx.x; i < Kout; i += 256) {
        const float g = to_float(dY[(long long)n * Kout + i]);
        if (db) db[(long long)n * Kout + i] = g;
        sy += (double)g * g;
    }
    sx = block_sum(sx, scratch);
    sy = block_sum(sy, scratch);
    if (threadIdx.x != 0) return;
    const double sw = sx * sy, sb = has_bias ? sy : 0.0;
    if (separate) {
        sqnorm[n * sq_stride] = (float)sw;
        sqnorm[n * sq_stride + 1] = (float)sb;
        if (clip) {
            const float fw = clip_factor(sw, C_l), fb = clip_factor(sb, C_l);
            factor[2 * n] = fw; factor[2 * n + 1] = fb;
            if (clip_out) { clip_out[2 * n] = fw; clip_out[2 * n + 1] = fb; }
        }
    } else {
        sqnorm[n * sq_stride] = (float)(sw + sb);
        if (clip) {
            const float f = clip_factor(sw + sb, C_l);
            factor[2 * n] = f; factor[2 * n + 1] = f;
            if (clip_out) clip_out[n] = f;
        }
    }
}

// ------------------------------------------------------------------ normalisation affine
// What the last thread block to finish an example does in the one-launch form of the layer: fold the example's
// pixel-chunk partial sums in chunk order, publish its squared norms (and clip factors), and -- when it is also the
// last block of the whole call and the batch is small enough to walk alone -- add the clipped sum over the examples
// to the accumulators.  "Last" is found with ticket counters (no block ever waits for another); the arithmetic and
// its order do not depend on which block turns out to be last, so results stay bit-reproducible.
struct AffineTail {
    int *counters;            // [B + 1] tickets: one per example, one for the call; zero on entry, left at zero.  null: off
    int blocks_per_example;
    int B;
    int clip;                 // 1: factors against C_l, clipped sum into acc_w / acc_b;  0: norms only
    int accumulate_here;      // 1: the last block of the call adds the clipped sum itself; 0: a second launch does
    int separate;
    float C_l;
    float *sqnorm; long long sq_stride; float *clip_out;
    float *factor;            // [B][2] scratch: (scale factor, shift factor) per example
    float *dgamma, *dbeta;    // [B][C] finished per-example gradients (scratch, or the caller's G_w / G_b)
    float *acc_w, *acc_b;
};

__device__ __forceinline__ void affine_tail(const AffineTail &t, int n, bool whole, const float *chunk_partial, int chunks,
                                            int C, double qg, double qb, double *scratch) {
    __shared__ int last_flag;
    if (!whole) {
        __threadfence();                                   // this block's chunk partials are visible before its ticket
        __syncthreads();
        if (threadIdx.x == 0) last_flag = (atomicAdd(&t.counters[n], 1) == t.blocks_per_example - 1);
        __syncthreads();
        if (!last_flag) return;
        __threadfence();
        qg = 0.0; qb = 0.0;
        for (int c = threadIdx.x; c < C; c += 256) {
            float a = 0.f, b = 0.f;
            const float *p = chunk_partial + ((long long)n * chunks * 2) * C + c;
            int k = 0;
            for (; k + 8 <= chunks; k += 8) {              // eight chunks' loads in flight, added in chunk order
                float x[8], y[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) { x[u] = __ldcg(p + (long long)(k + u) * 2 * C); y[u] = __ldcg(p + (long long)(k + u) * 2 * C + C); }
#pragma unroll
                for (int u = 0; u < 8; ++u) { a += x[u]; b += y[u]; }
            }
            for (; k < chunks; ++k) { a += __ldcg(p + (long long)k * 2 * C); b += __ldcg(p + (long long)k * 2 * C + C); }
            t.dgamma[(long long)n * C + c] = a;
            t.dbeta[(long long)n * C + c] = b;
            qg += (double)a * a;
            qb += (double)b * b;
        }
        qg = block_sum(qg, scratch);
        qb = block_sum(qb, scratch);
        if (threadIdx.x == 0) t.counters[n] = 0;
    }
    if (threadIdx.x == 0) {
        float f0 = 1.f, f1 = 1.f;
        if (t.separate) {
            t.sqnorm[n * t.sq_stride] = (float)qg; t.sqnorm[n * t.sq_stride + 1] = (float)qb;
            if (t.clip) { f0 = clip_factor(qg, t.C_l); f1 = clip_factor(qb, t.C_l); }
            if (t.clip && t.clip_out) { t.clip_out[2 * n] = f0; t.clip_out[2 * n + 1] = f1; }
        } else {
            t.sqnorm[n * t.sq_stride] = (float)(qg + qb);
            if (t.clip) f0 = f1 = clip_factor(qg + qb, t.C_l);
            if (t.clip && t.clip_out) t.clip_out[n] = f0;
        }
        t.factor[2 * n] = f0; t.factor[2 * n + 1] = f1;
    }
    if (!t.clip || !t.accumulate_here) return;
    __threadfence();                                       // this example's gradients and factors before the call's ticket
    __syncthreads();
    if (threadIdx.x == 0) {
        last_flag = (atomicAdd(&t.counters[t.B], 1) == t.B - 1);
        if (last_flag) t.counters[t.B] = 0;
    }
    __syncthreads();
    if (!last_flag) return;
    __threadfence();
    // thread = (channel, tensor); the factors of up to 256 examples at a time sit in shared memory and eight examples'
    // values are in flight per thread (the walk is latency-bound: everything comes from L2)
    __shared__ float f_sh[2][256];
    for (int c0 = 0; c0 < 2 * C; c0 += 256) {
        const int e = c0 + threadIdx.x;
        const int which = e >= C, c = which ? e - C : e;
        const float *v = (which ? t.dbeta : t.dgamma) + c;
        float a = 0.f;
        for (int m0 = 0; m0 < t.B; m0 += 256) {
            const int mb = min(256, t.B - m0);
            __syncthreads();
            if (threadIdx.x < mb) {
                f_sh[0][threadIdx.x] = __ldcg(t.factor + 2 * (m0 + threadIdx.x));
                f_sh[1][threadIdx.x] = __ldcg(t.factor + 2 * (m0 + threadIdx.x) + 1);
            }
            __syncthreads();
            if (e < 2 * C) {
                int m = 0;
                for (; m + 8 <= mb; m += 8) {
                    float x[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) x[u] = __ldcg(v + (long long)(m0 + m + u) * C);
#pragma unroll
                    for (int u = 0; u < 8; ++u) a = fmaf(f_sh[which][m + u], x[u], a);
                }
                for (; m < mb; ++m) a = fmaf(f_sh[which][m], __ldcg(v + (long long)(m0 + m) * C), a);
            }
        }
        if (e < 2 * C) (which ? t.acc_b : t.acc_w)[c] += a;
    }
}

// stage 1: block = (channel-vector block, pixel chunk, example); thread = (pixel row, channel vector).
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
norm_affine_partial_kernel(const T *__restrict__ X, const T *__restrict__ dY, int HW, int C, int tcv, int pix,
                           float *__restrict__ chunk_partial, int chunks, float *__restrict__ dgamma,
                           float *__restrict__ dbeta, float *__restrict__ partial2, const AffineTail tail) {
    extern __shared__ float red[];                       // [rows][tcv*VEC*2]
    const int n = blockIdx.z, chunk = blockIdx.y;
    const int rows = 256 / tcv;
    const int prow = threadIdx.x / tcv, cvi = threadIdx.x - prow * tcv;
    const int c0 = (blockIdx.x * tcv + cvi) * VEC;
    const bool live = prow < rows && c0 < C;
    float sg[VEC], sb[VEC];
#pragma unroll
    for (int v = 0; v < VEC; ++v) { sg[v] = 0.f; sb[v] = 0.f; }
    const int p_end = min(HW, (chunk + 1) * pix);
    if (live) {
        if (VEC * sizeof(T) == 16) {
            // four pixels per trip, all eight 16-byte loads issued before any arithmetic
            for (int p = chunk * pix + prow; p < p_end; p += 4 * rows) {
                uint4 xr[4], gr[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int pu = p + u * rows;
                    if (pu < p_end) {
                        const long long off = ((long long)n * HW + pu) * C + c0;
                        xr[u] = __ldcs(reinterpret_cast<const uint4 *>(X + off));
                        gr[u] = __ldcs(reinterpret_cast<const uint4 *>(dY + off));
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (p + u * rows < p_end) {
                        const T *xv = reinterpret_cast<const T *>(&xr[u]);
                        const T *gv = reinterpret_cast<const T *>(&gr[u]);
#pragma unroll
                        for (int v = 0; v < VEC; ++v) {
                            const float gg = to_float(gv[v]);
                            sg[v] = fmaf(gg, to_float(xv[v]), sg[v]);
                            sb[v] += gg;
                        }
                    }
                }
            }
        } else {
            for (int p = chunk * pix + prow; p < p_end; p += rows) {
                const long long off = ((long long)n * HW + p) * C + c0;
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                    const float gg = to_float(dY[off + v]);
                    sg[v] = fmaf(gg, to_float(X[off + v]), sg[v]);
                    sb[v] += gg;
                }
            }
        }
    }
    const int width = tcv * VEC * 2;
    if (prow < rows) {
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
            red[prow * width + cvi * VEC + v] = sg[v];
            red[prow * width + tcv * VEC + cvi * VEC + v] = sb[v];
        }
    }
    __syncthreads();
    // every thread folds one output column over the pixel rows, in row order.  When this block holds the whole
    // example (one pixel chunk, all channels) the sums are final: it writes the gradients and both squared norms
    // itself and the separate folding launch is skipped (dgamma != nullptr says so).
    {
        __shared__ double scratch[32];
        const bool whole = dgamma != nullptr;
        float *out = chunk_partial + (((long long)n * chunks + chunk) * 2) * C;
        const int half = tcv * VEC;
        double qg = 0.0, qb = 0.0;
        for (int e = threadIdx.x; e < 2 * half; e += 256) {
            const int is_beta = e >= half;
            const int c = blockIdx.x * half + (is_beta ? e - half : e);
            if (c >= C) continue;
            float a = 0.f;
            for (int rr = 0; rr < rows; ++rr) a += red[rr * width + e];
            if (whole) {
                (is_beta ? dbeta : dgamma)[(long long)n * C + c] = a;
                if (is_beta) qb += (double)a * a; else qg += (double)a * a;
            } else {
                out[is_beta ? C + c : c] = a;
            }
        }
        if (whole) {
            qg = block_sum(qg, scratch);
            qb = block_sum(qb, scratch);
            if (threadIdx.x == 0 && !tail.counters) { partial2[2 * n] = (float)qg; partial2[2 * n + 1] = (float)qb; }
        }
        if (tail.counters) affine_tail(tail, n, whole, chunk_partial, chunks, C, qg, qb, scratch);
    }
}

// stage 2: fold chunks in index order, store dgamma / dbeta, squared norms of both
__global__ void __launch_bounds__(256)
norm_affine_fold_kernel(const float *__restrict__ chunk_partial, int chunks, int C, float *__restrict__ dgamma,
                        float *__restrict__ dbeta, float *__restrict__ partial2) {
    __shared__ double scratch[32];
    const int n = blockIdx.x;
    double qg = 0.0, qb = 0.0;
    for (int c = threadIdx.x; c < C; c += 256) {
        float a = 0.f, b = 0.f;
        for (int k = 0; k < chunks; ++k) {
            const float *p = chunk_partial + (((long long)n * chunks + k) * 2) * C;
            a += p[c];
            b += p[C + c];
        }
        dgamma[(long long)n * C + c] = a;
        dbeta[(long long)n * C + c] = b;
        qg += (double)a * a;
        qb += (double)b * b;
    }
    qg = block_sum(qg, scratch);
    qb = block_sum(qb, scratch);
    if (threadIdx.x == 0) { partial2[2 * n] = (float)qg; partial2[2 * n + 1] = (float)qb; }
}


// Normalisation layers, fused clip: every block works out the factors of all examples from the two squared norms
// (cheap and identical in every block), block 0 publishes norms and factors, then each thread owns one channel and
// adds sum_n f_n dgamma[n, c] / dbeta[n, c] to the accumulators.
__global__ void __launch_bounds__(128)
affine_clip_accum_kernel(const float *__restrict__ partial2, int B, float C_l, int separate, float *__restrict__ sqnorm,
                         long long sq_stride, float *clip_out, const float *__restrict__ dgamma,
                         const float *__restrict__ dbeta, int C, float *__restrict__ acc_w, float *__restrict__ acc_b) {
    __shared__ float fw[512], fb[512];
    const int c = blockIdx.x * 128 + threadIdx.x;
    float a = 0.f, b = 0.f;
    for (int n0 = 0; n0 < B; n0 += 512) {
        const int nb = min(512, B - n0);
        __syncthreads();
        for (int t = threadIdx.x; t < nb; t += 128) {
            const int n = n0 + t;
            const double sw = (double)partial2[2 * n], sb = (double)partial2[2 * n + 1];
            float f0, f1;
            if (separate) { f0 = clip_factor(sw, C_l); f1 = clip_factor(sb, C_l); }
            else { f0 = f1 = clip_factor(sw + sb, C_l); }
            fw[t] = f0; fb[t] = f1;
            if (blockIdx.x == 0) {
                if (separate) {
                    sqnorm[n * sq_stride] = (float)sw; sqnorm[n * sq_stride + 1] = (float)sb;
                    if (clip_out) { clip_out[2 * n] = f0; clip_out[2 * n + 1] = f1; }
                } else {
                    sqnorm[n * sq_stride] = (float)(sw + sb);
                    if (clip_out) clip_out[n] = f0;
                }
            }
        }
        __syncthreads();
        if (c < C) {
            const float *g = dgamma + (long long)n0 * C + c, *h = dbeta + (long long)n0 * C + c;
#pragma unroll 8
            for (int t = 0; t < nb; ++t) {
                a = fmaf(fw[t], g[(long long)t * C], a);
                b = fmaf(fb[t], h[(long long)t * C], b);
            }
        }
    }
    if (c < C) { acc_w[c] += a; acc_b[c] += b; }
}

dp_status launch_affine_clip_accum(const float *partial2, int B, float C_l, int separate, float *sqnorm, long long sq_stride,
                                   float *clip_out, const float *dgamma, const float *dbeta, int C, float *acc_w,
                                   float *acc_b, cudaStream_t st) {
    affine_clip_accum_kernel<<<(C + 127) / 128, 128, 0, st>>>(partial2, B, C_l, separate, sqnorm, sq_stride, clip_out, dgamma,
                                                            dbeta, C, acc_w, acc_b);
    DP_LAUNCH_CHECK("affine_clip_accum_kernel");
    return DP_OK;
}

// ------------------------------------------------------------------ host launchers
int fma_clip_splits(const ConvGeom &g) {
    const int tiles = fma_tiles_m(g) * fma_tiles_n(g);
    int want = (2 * sm_count()) / tiles;
    if (want < 1) want = 1;
    if (want > g.B) want = g.B;
    const int per = (g.B + want - 1) / want;
    return (g.B + per - 1) / per;
}

// acc[i] += sum_s ws[s][i], splits in index order
__global__ void fold_sums_kernel(const float *__restrict__ ws, int splits, long long P, float *__restrict__ acc) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= P) return;
    float a = acc[i];
    for (int s = 0; s < splits; ++s) a += ws[(long long)s * P + i];
    acc[i] = a;
}

template <typename T>
static dp_status conv_fma_t(int mode, const T *X, const T *dY, const ConvGeom &g, float *G_w, float *partial, int slots,
                            const float *factor, float *acc_w, float *sum_ws, cudaStream_t st) {
    const int splits = (mode == 2) ? fma_clip_splits(g) : 1;
    const int per = (g.B + splits - 1) / splits;
    const dim3 grid(fma_tiles_n(g), fma_tiles_m(g), mode == 2 ? splits : g.B);
    if (grid.y > 65535 || grid.z > 65535) return DP_ERR_UNSUPPORTED;
    if (mode == 0) conv_wgrad_fma_kernel<T, 0><<<grid, 256, 0, st>>>(X, dY, g, G_w, partial, slots, factor, acc_w, per, sum_ws);
    else if (mode == 1) conv_wgrad_fma_kernel<T, 1><<<grid, 256, 0, st>>>(X, dY, g, G_w, partial, slots, factor, acc_w, per, sum_ws);
    else conv_wgrad_fma_kernel<T, 2><<<grid, 256, 0, st>>>(X, dY, g, G_w, partial, slots, factor, acc_w, per, sum_ws);
    DP_LAUNCH_CHECK("conv_wgrad_fma_kernel");
    if (mode == 2 && splits > 1) {
        const long long P = (long long)g.M * g.N;
        fold_sums_kernel<<<(unsigned)((P + 255) / 256), 256, 0, st>>>(sum_ws, splits, P, acc_w);
        DP_LAUNCH_CHECK("fold_sums_kernel");
    }
    return DP_OK;
}

dp_status launch_conv_fma(int dtype, int mode, const void *X, const void *dY, const ConvGeom &g, float *G_w,
                          float *partial, int slots, const float *factor, float *acc_w, float *sum_ws, cudaStream_t st) {
    if (dtype == DP_F32)
        return conv_fma_t(mode, static_cast<const float *>(X), static_cast<const float *>(dY), g, G_w, partial, slots, factor, acc_w, sum_ws, st);
    return conv_fma_t(mode, static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), g, G_w, partial, slots, factor, acc_w, sum_ws, st);
}

dp_status launch_bias(int dtype, const void *dY, const ConvGeom &g, float *db, float *partial, int slots, int slot0,
                      cudaStream_t st) {
    const int vec = (dtype == DP_F32) ? 4 : 8;
    if (g.Kout % vec == 0 && g.Kout / vec <= 256 && bias_blocks(g) <= 256) {
        const size_t smem = sizeof(float) * (size_t)(256 / (g.Kout / vec)) * g.Kout;
        if (dtype == DP_F32)
            bias_vec_kernel<float, 4><<<g.B, 256, smem, st>>>(static_cast<const float *>(dY), g.K, g.Kout, db, partial, slots, slot0, bias_blocks(g));
        else
            bias_vec_kernel<__nv_bfloat16, 8><<<g.B, 256, smem, st>>>(static_cast<const __nv_bfloat16 *>(dY), g.K, g.Kout, db, partial, slots, slot0, bias_blocks(g));
        DP_LAUNCH_CHECK("bias_vec_kernel");
        return DP_OK;
    }
    const dim3 grid(bias_blocks(g), g.B);
    if (grid.y > 65535) return DP_ERR_UNSUPPORTED;
    if (dtype == DP_F32) bias_kernel<<<grid, 256, 0, st>>>(static_cast<const float *>(dY), g.K, g.Kout, db, partial, slots, slot0);
    else bias_kernel<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(dY), g.K, g.Kout, db, partial, slots, slot0);
    DP_LAUNCH_CHECK("bias_kernel");
    return DP_OK;
}

dp_status launch_finalize(const float *partial, int B, int slots, int w_slots, int separate, float *sqnorm,
                          long long sq_stride, int clip, float C_l, float *factor, float *clip_out, cudaStream_t st) {
    finalize_norm_kernel<<<B, 128, 0, st>>>(partial, slots, w_slots, separate, sqnorm, sq_stride, clip, C_l, factor, clip_out);
    DP_LAUNCH_CHECK("finalize_norm_kernel");
    return DP_OK;
}

dp_status launch_bias_accum(const float *db, int B, int Kout, const float *factor, float *acc_b, cudaStream_t st, int which) {
    bias_accum_kernel<float><<<(Kout + 31) / 32, 256, 0, st>>>(db, B, Kout, factor + which, 2, acc_b);
    DP_LAUNCH_CHECK("bias_accum_kernel");
    return DP_OK;
}

dp_status launch_dense_scaled_sum(int dtype, const void *X, const void *dY, const float *factor, long long f_stride, int B,
                                  int Cin, int Kout, float *acc_w, cudaStream_t st, const float *factor_b, long long fb_stride,
                                  float *acc_b) {
    const dim3 grid((unsigned)((Cin + 31) / 32), (unsigned)((Kout + kDenseOT - 1) / kDenseOT));
    if (grid.y > 65535) return DP_ERR_UNSUPPORTED;
    if (dtype == DP_F32)
        dense_scaled_sum_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float *>(X), static_cast<const float *>(dY), factor, f_stride, B, Cin, Kout, acc_w, factor_b, fb_stride, acc_b);
    else
        dense_scaled_sum_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), factor, f_stride, B, Cin, Kout, acc_w, factor_b, fb_stride, acc_b);
    DP_LAUNCH_CHECK("dense_scaled_sum_kernel");
    return DP_OK;
}

dp_status launch_expand_factor(const float *factor_w, const float *factor_b, long long stride, int B, float *factor2, cudaStream_t st) {
    expand_factor_kernel<<<(B + 127) / 128, 128, 0, st>>>(factor_w, factor_b, stride, B, factor2);
    DP_LAUNCH_CHECK("expand_factor_kernel");
    return DP_OK;
}

template <typename T>
static dp_status dense_store_t(const T *X, const T *dY, int B, int Cin, int Kout, float *G_w, float *G_b, cudaStream_t st) {
    const bool vec = (Cin & 3) == 0;
    const long long rows = (long long)B * Kout;
    // short rows share a block so that every block still moves a few KB
    const int per_block = Cin >= 1024 ? 1 : (1024 + Cin - 1) / Cin;
    const long long blocks = (rows + per_block - 1) / per_block;
    if (blocks > 0x7fffffffLL) return DP_ERR_UNSUPPORTED;
    if (vec) dense_store_kernel<T, true><<<(unsigned)blocks, 256, 0, st>>>(X, dY, Cin, Kout, per_block, rows, G_w);
    else dense_store_kernel<T, false><<<(unsigned)blocks, 256, 0, st>>>(X, dY, Cin, Kout, per_block, rows, G_w);
    DP_LAUNCH_CHECK("dense_store_kernel");
    (void)G_b;      // the bias gradient is written by the norm kernel that every dense call runs
    return DP_OK;
}

dp_status launch_dense_store(int dtype, const void *X, const void *dY, int B, int Cin, int Kout, float *G_w, float *G_b,
                             cudaStream_t st) {
    if (dtype == DP_F32) return dense_store_t(static_cast<const float *>(X), static_cast<const float *>(dY), B, Cin, Kout, G_w, G_b, st);
    return dense_store_t(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), B, Cin, Kout, G_w, G_b, st);
}

dp_status launch_dense_norm(int dtype, const void *X, const void *dY, int B, int Cin, int Kout, int has_bias, float *db,
                            int separate, float *sqnorm, long long sq_stride, int clip, float C_l, float *factor,
                            float *clip_out, cudaStream_t st) {
    if (dtype == DP_F32)
        dense_norm_kernel<<<B, 256, 0, st>>>(static_cast<const float *>(X), static_cast<const float *>(dY), Cin, Kout, has_bias, db,
                                             separate, sqnorm, sq_stride, clip, C_l, factor, clip_out);
    else
        dense_norm_kernel<<<B, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), Cin, Kout,
                                             has_bias, db, separate, sqnorm, sq_stride, clip, C_l, factor, clip_out);
    DP_LAUNCH_CHECK("dense_norm_kernel");
    return DP_OK;
}

template <typename T, int VEC>
static dp_status norm_affine_t(const T *X, const T *dY, int B, int HW, int C, int tcv, int pix, float *chunk_partial,
                               float *dgamma, float *dbeta, float *partial2, bool &folded, AffineTail tail, cudaStream_t st) {
    const int cv = (C + VEC - 1) / VEC;
    const int chunks = (HW + pix - 1) / pix;
    const dim3 grid((cv + tcv - 1) / tcv, chunks, B);
    if (grid.y > 65535 || grid.z > 65535) return DP_ERR_UNSUPPORTED;
    const size_t smem = sizeof(float) * (size_t)(256 / tcv) * tcv * VEC * 2;
    folded = grid.x == 1 && chunks == 1;      // one block sees the whole example: it finishes the job itself
    tail.blocks_per_example = (int)(grid.x * grid.y);
    norm_affine_partial_kernel<T, VEC><<<grid, 256, smem, st>>>(X, dY, HW, C, tcv, pix, chunk_partial, chunks,
                                                               folded ? dgamma : nullptr, dbeta, partial2, tail);
    DP_LAUNCH_CHECK("norm_affine_partial_kernel");
    return DP_OK;
}

static dp_status norm_affine_dispatch(int dtype, const void *X, const void *dY, int B, int HW, int C, float *chunk_partial,
                                      float *dgamma, float *dbeta, float *partial2, bool &folded, const AffineTail &tail,
                                      cudaStream_t st) {
    int vec, tcv, pix;
    norm_shape(dtype, B, HW, C, vec, tcv, pix);
    if (dtype == DP_F32) {
        if ((C & 3) == 0) return norm_affine_t<float, 4>(static_cast<const float *>(X), static_cast<const float *>(dY), B, HW, C, tcv, pix, chunk_partial, dgamma, dbeta, partial2, folded, tail, st);
        return norm_affine_t<float, 1>(static_cast<const float *>(X), static_cast<const float *>(dY), B, HW, C, tcv, pix, chunk_partial, dgamma, dbeta, partial2, folded, tail, st);
    }
    if ((C & 7) == 0) return norm_affine_t<__nv_bfloat16, 8>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), B, HW, C, tcv, pix, chunk_partial, dgamma, dbeta, partial2, folded, tail, st);
    return norm_affine_t<__nv_bfloat16, 1>(static_cast<const __nv_bfloat16 *>(X), static_cast<const __nv_bfloat16 *>(dY), B, HW, C, tcv, pix, chunk_partial, dgamma, dbeta, partial2, folded, tail, st);
}

dp_status launch_norm_affine(int dtype, const void *X, const void *dY, int B, int HW, int C, float *chunk_partial,
                             float *dgamma, float *dbeta, float *partial2, cudaStream_t st) {
    bool folded = false;
    AffineTail off = {};
    const dp_status rc = norm_affine_dispatch(dtype, X, dY, B, HW, C, chunk_partial, dgamma, dbeta, partial2, folded, off, st);
    if (rc != DP_OK || folded) return rc;
    norm_affine_fold_kernel<<<B, 256, 0, st>>>(chunk_partial, norm_chunks(dtype, B, HW, C), C, dgamma, dbeta, partial2);
    DP_LAUNCH_CHECK("norm_affine_fold_kernel");
    return DP_OK;
}

// acc_w[c] += sum_n factor[2n] * dgamma[n, c] and acc_b[c] += sum_n factor[2n + 1] * dbeta[n, c] in one launch
// (blockIdx.y picks the tensor).  Block = 32 channels x 8 example groups, groups folded in order.
__global__ void __launch_bounds__(256)
affine_accum_kernel(const float *__restrict__ dgamma, const float *__restrict__ dbeta, int B, int C,
                    const float *__restrict__ factor, float *__restrict__ acc_w, float *__restrict__ acc_b) {
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, q = threadIdx.x >> 5, which = blockIdx.y;
    const float *v = which ? dbeta : dgamma;
    const int c = blockIdx.x * 32 + lane;
    float a = 0.f;
    if (c < C) {
#pragma unroll 8
        for (int n = q; n < B; n += 8) a = fmaf(factor[2 * n + which], v[(long long)n * C + c], a);
    }
    part[q][lane] = a;
    __syncthreads();
    if (q == 0 && c < C) {
        float t = part[0][lane];
#pragma unroll
        for (int i = 1; i < 8; ++i) t += part[i][lane];
        (which ? acc_b : acc_w)[c] += t;
    }
}

bool affine_fused_eligible(int B) { return B + 1 <= kWsCounters; }

// The whole layer call in one launch (two when the batch times the channel count is large): per-example gradients,
// their squared norms, and for clip != 0 the factors against C_l and the clipped sums.  dgamma / dbeta: [B][C]
// scratch or the caller's outputs; factor: [B][2] scratch; counters: B + 1 cleared tickets.
dp_status launch_norm_affine_fused(int dtype, const void *X, const void *dY, int B, int HW, int C, float *chunk_partial,
                                   float *dgamma, float *dbeta, float *factor, int *counters, int clip, float C_l,
                                   int separate, float *sqnorm, long long sq_stride, float *clip_out, float *acc_w,
                                   float *acc_b, cudaStream_t st) {
    AffineTail t = {};
    t.counters = counters; t.B = B; t.clip = clip; t.separate = separate; t.C_l = C_l;
    t.accumulate_here = clip && (long long)B * C <= 16384;
    t.sqnorm = sqnorm; t.sq_stride = sq_stride; t.clip_out = clip_out; t.factor = factor;
    t.dgamma = dgamma; t.dbeta = dbeta; t.acc_w = acc_w; t.acc_b = acc_b;
    bool folded = false;
    const dp_status rc = norm_affine_dispatch(dtype, X, dY, B, HW, C, chunk_partial, dgamma, dbeta, nullptr, folded, t, st);
    if (rc != DP_OK || !clip || t.accumulate_here) return rc;
    affine_accum_kernel<<<dim3((unsigned)((C + 31) / 32), 2), 256, 0, st>>>(dgamma, dbeta, B, C, factor, acc_w, acc_b);
    DP_LAUNCH_CHECK("affine_accum_kernel");
    return DP_OK;
}


}  // namespace dp

// Per-example convolution weight gradients on the 5th-generation tensor cores (tcgen05 + TMEM),
// operands staged by TMA.  One (example, output tile) at a time per CTA, persistent CTAs.
//
// For example n the gradient is the matrix product  D_n = dY_n^T * Xcol_n  over the output pixels:
//     dY_n   [pixels, K_out]          (channels-last: K_out contiguous)
//     Xcol_n [pixels, R*S*C_in]       (column j = (r*S+s)*C_in + c is the input shifted by tap (r,s))
// Both operands have the reduction index (pixel) as the slow axis, i.e. they are "MN-major" for the
// tensor core.  A TMA box {64 channels, OWt, OHt, 1 example} lands in shared memory as OWt*OHt rows of
// 128 bytes with the 128-byte swizzle, which is exactly the canonical MN-major operand slab; the tap
// shift and the zero padding come from the box start coordinate and TMA's out-of-bounds zero fill.
//
// Roles (224 threads): warps 0 and 6 issue TMA loads (A and B slabs), warp 1 allocates TMEM and issues tcgen05.mma,
// warps 2-5 read accumulators back with tcgen05.ld, square-sum them (the per-example norm) and store.
// Two accumulator buffers in TMEM let the epilogue of one tile overlap the main loop of the next.
// Every wait is bounded: on expiry the CTA sets a status word, drains and returns.
//
// fp32 inputs run as split tf32: the tensor core truncates fp32 to tf32, which biases every norm by about
// 1e-3, so eight more warps write lo = x - hi (hi = x with the low 13 mantissa bits cleared) of each landed
// stage into a second buffer of the same layout; x itself stays in place, where the tensor core's own truncation
// turns it into hi, and the issuer accumulates lo*hi + hi*lo + hi*hi per step.  What is dropped (lo*lo and the truncation of lo) is below 2^-20 relative.
#include "wgrad_tc.cuh"
#include <cuda.h>
#include <mutex>
#include <atomic>
#include <algorithm>
#include <array>
#include <map>

namespace dp {

constexpr int kRowBytes = 128;         // one pixel's slab of channels: 64 bf16 or 32 fp32/tf32
constexpr int kMaxStages = 8;
constexpr int kSmemBudget = 200 * 1024;
constexpr uint32_t kWaitPolls = 1u << 21;   // x ~1 us suspend hint: about two seconds before a wait gives up
static std::atomic<uint32_t> g_wait_polls{kWaitPolls};
void set_wait_polls(uint32_t polls) { g_wait_polls.store(polls, std::memory_order_relaxed); }
uint32_t default_wait_polls() { return kWaitPolls; }

struct TcPlan {
    bool ok;
    int a_is_x;                 // 1: rows of D are columns j of Xcol, columns of D are output channels k
    int a_ext, b_ext;           // operand extents in elements (multiples of the slab width)
    int m_tiles, n_tiles, NT;   // NT: nominal columns per tile (<= 256)
    int OWt, OHt, tiles_w, tiles_h, Kt, k_tiles;
    int stages, stage_bytes, a_bytes;
    size_t smem;
};

struct TcParams {
    int B, Kout, Ng, Cin, S, stride, pad;   // Ng: row length of G in memory = number of real gradient columns
    int n_pad_cols;             // 1 when the column extent carries zero padding beyond Ng (im2col'd small-channel layers)
    int slab_ch;                // channels per 128-byte row: 64 (bf16) or 32 (fp32 as tf32)
    int krows;                  // reduction rows per MMA: 16 (bf16) or 8 (tf32)
    int a_is_x, a_ext, b_ext, m_tiles, n_tiles, NT;
    int OWt, OHt, tiles_w, Kt, k_tiles, stages, stage_bytes, a_bytes;
    int lo_offset;              // split tf32: byte offset of the lo copy inside a stage
    int single_pass;            // fp32 inputs rounded to tf32 (nearest even) in place, one MMA per step, no lo copy
    int mode;                   // 0 store + norm, 1 norm only, 2 clipped sum over a range of examples
    float *G_w;
    float *partial;             // [B][slots], slot = (mt*n_tiles + nt)*4 + epilogue warp
    int slots;
    int *status;
    uint32_t wait_polls;        // polls after which a wait gives up
    int total_tiles;            // work items: (example, tile) pairs, or (example range, tile) pairs in mode 2
    // mode 2: item = (split, tile); the CTA walks examples [split*per_split, ...) and keeps sum_n f_n D_n in registers
    int splits, per_split;
    const float *factor;        // [B][2], element 0 = weight factor (used when inline_factor == 0)
    // inline_factor: the clipped-sum pass works the factor out itself from the norm pass's partial sums (partial,
    // slots) and publishes the squared norm and the factor, which saves the separate finalising launch
    int inline_factor;
    float C_l;
    float *sqnorm; long long sq_stride; float *clip_out;
    float *sum_out;             // splits == 1: the accumulator (added to); else partial sums [splits][Kout*Ng]
    // modes 0 / 1 with a ticket: counters[0] counts the CTAs that are done (zero on entry, left at zero); the last
    // one folds every example's slots [0, w_slots) and [w_slots, slots) into sqnorm (two values when `separate`)
    int *counters; int w_slots; int separate;
    float *factor_out;          // with the ticket: also the clip factors against C_l, [B][2] (weight, bias), and clip_out
    // space-to-depth form of a thin strided layer (s2d_st > 0): row j' of D is (r2, s2, dy, dx, c) of the regrouped
    // input and maps to column ((st*r2+dy)*s2d_S + st*s2d+dx)*s2d_Cin + c of the gradient, or to nothing
    int s2d_st, s2d_R, s2d_S, s2d_Cin;
};

// column of the gradient that row j of the space-to-depth product stands for, or -1 (a tap or channel that does not exist)
__device__ __forceinline__ int s2d_column(const TcParams &p, int j) {
    const int r2 = j >> 6, s2 = (j >> 4) & 3, ch = j & 15;
    const int q = ch / p.s2d_Cin, c = ch - q * p.s2d_Cin;
    const int dy = q / p.s2d_st, dx = q - dy * p.s2d_st;
    const int r = p.s2d_st * r2 + dy, s = p.s2d_st * s2 + dx;
    return (dy < p.s2d_st && r < p.s2d_R && s < p.s2d_S) ? (r * p.s2d_S + s) * p.s2d_Cin + c : -1;
}

struct Item { int mt, nt, n_lo, n_hi, split; };
__device__ __forceinline__ Item decode_item(const TcParams &p, int item) {
    Item it;
    const int tpe = p.m_tiles * p.n_tiles;
    const int outer = item / tpe;          // the example, or in mode 2 the example range
    const int rem = item - outer * tpe;
    it.mt = rem / p.n_tiles;
    it.nt = rem - it.mt * p.n_tiles;
    if (p.mode == 2) { it.split = outer; it.n_lo = outer * p.per_split; it.n_hi = min(p.B, it.n_lo + p.per_split); }
    else { it.split = 0; it.n_lo = outer; it.n_hi = outer + 1; }
    return it;
}

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
                 "selp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this or another wait expired).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t polls) {
    for (uint32_t it = 0; it < polls; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], fp32 accumulate, issued by one thread; TF32 selects kind::tf32 (fp32 inputs).
// The operand descriptors arrive as (low word, high word): only the low word (start address) changes from step to
// step, which keeps the issuing thread's work per instruction to one 32-bit add.
template <bool TF32>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t desc_hi, uint32_t idesc,
                                     uint32_t accumulate) {
    if (TF32)
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::1.kind::tf32 [%0], da, db, %4, p;\n\t}"
                     ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                     "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
                     ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate) : "memory");
}
// Issue only: the registers hold the values after tmem_ld_wait32 on the same array.  Two loads in flight per thread
// hide most of the tensor-memory round trip (a load-then-wait per 32 columns left the epilogue warps idle).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
// Waits for every tensor-memory load of this thread; the array rides along as in/out operands so that no use of its
// registers can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait32(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory operand descriptor without the start address, for MN-major slabs of 128-byte rows.
//   leading byte offset (between slabs) >> 4 at bit 16 | stride byte offset (between groups of reduction rows) >> 4
//   at bit 32 | descriptor version 1 at bit 46 | layout type at bit 61.
// 16-bit operands use the plain 128-byte swizzle (type 2: 16-byte chunks, pattern repeats every 8 rows = 1024 B).
// 32-bit (tf32) MN-major operands only exist with the 128-byte swizzle of 32-byte chunks (type 1: pattern
// repeats every 4 rows = 512 B); the tensor map then uses the matching SWIZZLE_128B_ATOM_32B mode.
template <bool TF32>
__device__ __forceinline__ uint64_t operand_desc_base(uint32_t slab_stride_bytes) {
    uint64_t d = (uint64_t)((slab_stride_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(((TF32 ? 512u : 1024u) >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)(TF32 ? 1 : 2) << 61;
    return d;
}
// Instruction descriptor: fp32 accumulator, A and B of one type (bf16 = 1, tf32 = 2), both MN-major, M = 128, N = n_cols.
__device__ __forceinline__ uint32_t instr_desc(int n_cols, uint32_t fmt) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(n_cols >> 3) << 17) | ((128u >> 4) << 24);
}

template <bool TF32, bool CLIP>
__global__ void __launch_bounds__(TF32 ? 480 : 224, 1)
conv_wgrad_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const TcParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], ready_bar[kMaxStages], tmem_full[2], tmem_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float xpose[4][32][33];      // per epilogue warp: 32 x 32 transpose buffer for coalesced row stores

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t tiles_u32 = smem_u32(tiles);

    if (threadIdx.x == 0) {
        // pull both tensor maps into the TMA descriptor cache before the first copy needs them
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&full_bar[s]), 2); mbar_init(smem_u32(&empty_bar[s]), 1); mbar_init(smem_u32(&ready_bar[s]), 4);
        }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tmem_full[b]), 1); mbar_init(smem_u32(&tmem_empty[b]), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int *abort_p = &abort_flag;

    const int slab_bytes = p.Kt * kRowBytes;
    const int a_slabs_tile = 128 / p.slab_ch, b_slabs_tile = p.NT / p.slab_ch;

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------------------ TMA producers
        // Two warps, because issuing a copy costs the issuing warp ~100 cycles: warp 0 loads the A slabs of every
        // stage, warp 6 the B slabs; each announces its own bytes on the stage's full barrier (two arrivals).
        // Lane L owns slab L: it works out its tap shift and channel offset once per tile and then only adds the
        // pixel-tile origin, so no division sits in the stage loop.
        int stage = 0; uint32_t phase = 0;
        bool live = true;
        for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const int mt = it.mt, nt = it.nt;
            const int a_slab0 = mt * a_slabs_tile, a_slabs = min(a_slabs_tile, p.a_ext / p.slab_ch - a_slab0);
            const int b_slab0 = nt * b_slabs_tile, b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - b_slab0);
            const bool is_a = warp == 0;
            const int local = lane;
            const bool active = is_a ? (local < a_slabs) : (local < b_slabs);
            const bool is_x = is_a ? (p.a_is_x != 0) : (p.a_is_x == 0);
            const int slab = (is_a ? a_slab0 : b_slab0) + local;
            int c0, dw = 0, dh = 0, mul = 1;
            if (is_x) {
                const int j0 = slab * p.slab_ch;
                const int tap = j0 / p.Cin;
                c0 = j0 - tap * p.Cin;
                const int r = tap / p.S;
                dw = (tap - r * p.S) - p.pad;
                dh = r - p.pad;
                mul = p.stride;
            } else {
                c0 = slab * p.slab_ch;
            }
            const CUtensorMap *map = is_x ? &tmX : &tmY;
            const uint32_t dst_off = (is_a ? 0u : (uint32_t)p.a_bytes) + (uint32_t)(local * slab_bytes);
            const uint32_t tx_bytes = (uint32_t)((is_a ? a_slabs : b_slabs) * slab_bytes);
            for (int n = it.n_lo; n < it.n_hi && live; ++n) {
                int ow0 = 0, oh0 = 0, tw = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    bool ok = true;
                    if (lane == 0) {
                        ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_p, p.wait_polls);
                        if (ok) mbar_expect_tx(smem_u32(&full_bar[stage]), tx_bytes);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { live = false; break; }
                    if (active)
                        tma_load_4d(tiles_u32 + stage * p.stage_bytes + dst_off, map, smem_u32(&full_bar[stage]), c0,
                                    ow0 * mul + dw, oh0 * mul + dh, n);
                    if (++tw == p.tiles_w) { tw = 0; ow0 = 0; oh0 += p.OHt; } else { ow0 += p.OWt; }
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            uint32_t acc_phase = 0;  // bit b: phase of accumulator buffer b
            int buf = 0;
            bool live = true;
            const uint64_t desc_base = operand_desc_base<TF32>((uint32_t)slab_bytes);
            const uint32_t desc_lo = (uint32_t)desc_base, desc_hi32 = (uint32_t)(desc_base >> 32);
            const int ksteps = p.Kt / p.krows;
            constexpr uint32_t kadvance = (uint32_t)((TF32 ? 8 : 16) * kRowBytes) >> 4;   // start-address units of 16 B per MMA step
            for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
              const Item it = decode_item(p, item);
              const int b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - it.nt * b_slabs_tile);
              const uint32_t idesc = instr_desc(b_slabs * p.slab_ch, TF32 ? 2u : 1u);
              for (int n = it.n_lo; n < it.n_hi && live; ++n) {
                if (!mbar_wait(smem_u32(&tmem_empty[buf]), ((acc_phase >> buf) & 1u) ^ 1u, abort_p, p.wait_polls)) { live = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                uint32_t accumulate = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    if (!mbar_wait(smem_u32(TF32 ? &ready_bar[stage] : &full_bar[stage]), phase, abort_p, p.wait_polls)) { live = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = tiles_u32 + stage * p.stage_bytes;
                    // descriptor low words: start address >> 4 in bits 0-13, slab stride >> 4 in bits 16-29
                    uint32_t ad = desc_lo | ((a_src & 0x3FFFFu) >> 4);
                    uint32_t bd = desc_lo | (((a_src + p.a_bytes) & 0x3FFFFu) >> 4);
                    // rows of the A tile past the operand's extent hold whatever the stage held before:
                    // they only feed rows of D that the epilogue never reads
                    if (TF32 && p.single_pass) {
#pragma unroll 4
                        for (int ks = 0; ks < ksteps; ++ks) {
                            umma<TF32>(d_tmem, ad, bd, desc_hi32, idesc, accumulate);
                            accumulate = 1;
                            ad += kadvance; bd += kadvance;
                        }
                    } else if (TF32) {
                        const uint32_t lo = (uint32_t)p.lo_offset >> 4;
#pragma unroll 2
                        for (int ks = 0; ks < ksteps; ++ks) {
                            umma<TF32>(d_tmem, ad + lo, bd, desc_hi32, idesc, accumulate);      // lo(A) * hi(B)
                            umma<TF32>(d_tmem, ad, bd + lo, desc_hi32, idesc, 1u);              // hi(A) * lo(B)
                            umma<TF32>(d_tmem, ad, bd, desc_hi32, idesc, 1u);                   // hi(A) * hi(B)
                            accumulate = 1;
                            ad += kadvance; bd += kadvance;
                        }
                    } else {
#pragma unroll 4
                        for (int ks = 0; ks < ksteps; ++ks) {
                            umma<TF32>(d_tmem, ad, bd, desc_hi32, idesc, accumulate);
                            accumulate = 1;
                            ad += kadvance; bd += kadvance;
                        }
                    }
                    umma_commit(smem_u32(&empty_bar[stage]));      // frees the stage once these MMAs have read it
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!live) break;
                umma_commit(smem_u32(&tmem_full[buf]));            // accumulator complete
                acc_phase ^= 1u << buf;
                buf ^= 1;
              }
            }
        }
    } else if (TF32 && warp >= 7) {
        // ------------------------------------------------------------ split warps (fp32 inputs only)
        // hi stays where TMA put it, lo goes to the same offset of the stage's second half; both keep the
        // swizzled layout because the split is element-wise on identical relative addresses.
        // The eight warps work as two groups of four that take alternate stages, so the proxy fence that ends one
        // group's stage (it waits for that group's stores to drain) overlaps the other group's loads and stores.
        const int group = (warp - 7) >> 2;
        const int tid = (threadIdx.x - 224) & 127;
        int stage = 0; uint32_t phase = 0;
        int turn = 0;                       // global stage counter modulo 2: whose stage is it
        bool live = true;
        for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const int a_slabs = min(a_slabs_tile, p.a_ext / p.slab_ch - it.mt * a_slabs_tile);
            const int b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - it.nt * b_slabs_tile);
            const int a_chunks = a_slabs * (slab_bytes >> 4), chunks = a_chunks + b_slabs * (slab_bytes >> 4);
            const int stage_count = (it.n_hi - it.n_lo) * p.k_tiles;
            for (int kt = 0; kt < stage_count; ++kt) {
                if (turn == group) {
                    const bool arrived = mbar_wait(smem_u32(&full_bar[stage]), phase, abort_p, p.wait_polls);
                    if (!__all_sync(0xffffffffu, arrived)) { live = false; break; }
                    uint8_t *base = tiles + (size_t)stage * p.stage_bytes;
                    // four 16-byte groups per thread and trip with all loads first, A region and B region in turn
                    for (int region = 0; region < 2; ++region) {
                        uint8_t *rbase = region ? base + p.a_bytes : base;
                        const int rchunks = region ? chunks - a_chunks : a_chunks;
                        for (int i0 = tid; i0 < rchunks; i0 += 512) {
                            float4 x[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (i0 + 128 * u < rchunks) x[u] = *reinterpret_cast<const float4 *>(rbase + ((size_t)(i0 + 128 * u) << 4));
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                if (i0 + 128 * u < rchunks && p.single_pass) {
                                    // round to tf32, nearest even, in place: the tensor core's own truncation then changes nothing
                                    uint4 b = *reinterpret_cast<const uint4 *>(&x[u]);
                                    b.x = (b.x + 0xFFFu + ((b.x >> 13) & 1u)) & 0xFFFFE000u;
                                    b.y = (b.y + 0xFFFu + ((b.y >> 13) & 1u)) & 0xFFFFE000u;
                                    b.z = (b.z + 0xFFFu + ((b.z >> 13) & 1u)) & 0xFFFFE000u;
                                    b.w = (b.w + 0xFFFu + ((b.w >> 13) & 1u)) & 0xFFFFE000u;
                                    *reinterpret_cast<uint4 *>(rbase + ((size_t)(i0 + 128 * u) << 4)) = b;
                                } else if (i0 + 128 * u < rchunks) {
                                    uint8_t *ptr = rbase + ((size_t)(i0 + 128 * u) << 4);
                                    float4 hi, lo;
                                    hi.x = __uint_as_float(__float_as_uint(x[u].x) & 0xFFFFE000u); lo.x = x[u].x - hi.x;
                                    hi.y = __uint_as_float(__float_as_uint(x[u].y) & 0xFFFFE000u); lo.y = x[u].y - hi.y;
                                    hi.z = __uint_as_float(__float_as_uint(x[u].z) & 0xFFFFE000u); lo.z = x[u].z - hi.z;
                                    hi.w = __uint_as_float(__float_as_uint(x[u].w) & 0xFFFFE000u); lo.w = x[u].w - hi.w;
                                    *reinterpret_cast<float4 *>(ptr + p.lo_offset) = lo;     // x stays: truncated by the MMA itself, it is hi
                                }
                            }
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ready_bar[stage]));
                }
                turn ^= 1;
                if (++stage == p.stages) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp >= 2 && warp <= 5) {
        // ------------------------------------------------------------ epilogue (4 warps, one TMEM lane quadrant each)
        const int q = warp & 3;
        const int row = q * 32 + lane;
        uint32_t full_phase = 0;     // bit b: parity to wait for on accumulator buffer b
        int buf = 0;
        bool live = true;
        for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const int mt = it.mt, nt = it.nt;
            const int a_rows = min(128, p.a_ext - mt * 128);
            const int n_cols = min(p.NT, p.b_ext - nt * p.NT);
            const int a_idx = mt * 128 + row;            // index along the A operand's extent
            const bool row_ok = row < a_rows && (!p.a_is_x || a_idx < p.Ng);
            float run[CLIP ? 128 : 1];                   // clip mode: this thread's row of sum_n f_n D_n (NT <= 128)
            if (CLIP) {
#pragma unroll
                for (int i = 0; i < 128; ++i) run[CLIP ? i : 0] = 0.f;
            }
            float f_lane = 0.f;     // clip mode, known factors: lane l holds the factor of example n_base + l
            int n_base = it.n_lo - 32;
            for (int n = it.n_lo; n < it.n_hi; ++n) {
                if (CLIP && !p.inline_factor && n >= n_base + 32) {
                    n_base = n;
                    f_lane = (n + lane < it.n_hi) ? p.factor[2 * (n + lane)] : 0.f;    // one coalesced load per 32 examples
                }
                const bool arrived = mbar_wait(smem_u32(&tmem_full[buf]), (full_phase >> buf) & 1u, abort_p, p.wait_polls);
                if (!__all_sync(0xffffffffu, arrived)) { live = false; break; }   // the whole warp leaves together
                full_phase ^= 1u << buf;
                tc_fence_after();
                const uint32_t t_addr = tmem_base + (uint32_t)(buf * 256) + ((uint32_t)(q * 32) << 16);
                if (CLIP) {
                    float f;
                    if (p.inline_factor) {
                        // same summation order in every warp of every CTA, so all of them apply the identical factor
                        double sn = 0.0;
                        const float *pn = p.partial + (long long)n * p.slots;
                        for (int i = lane; i < p.slots; i += 32) sn += (double)pn[i];
                        sn = warp_sum(sn);
                        f = clip_factor(sn, p.C_l);
                        if (mt == 0 && nt == 0 && q == 0 && lane == 0) {
                            p.sqnorm[n * p.sq_stride] = (float)sn;
                            if (p.clip_out) p.clip_out[n] = f;
                        }
                    } else {
                        f = __shfl_sync(0xffffffffu, f_lane, n - n_base);
                    }
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {           // columns in pairs of 32: both loads in flight before the wait
                        if (c2 * 64 < n_cols) {
                            uint32_t v0[32], v1[32];
                            tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64), v0);
                            tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64 + 32), v1);     // (NT is a multiple of 64 here)
                            tmem_ld_wait32(v0); tmem_ld_wait32(v1);
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                run[CLIP ? c2 * 64 + i : 0] = fmaf(f, __uint_as_float(v0[i]), run[CLIP ? c2 * 64 + i : 0]);
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                run[CLIP ? c2 * 64 + 32 + i : 0] = fmaf(f, __uint_as_float(v1[i]), run[CLIP ? c2 * 64 + 32 + i : 0]);
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
                } else {
                    float sq4[4] = {0.f, 0.f, 0.f, 0.f};      // four chains: one accumulator would serialise 256 dependent FMAs
                    float *Gn = p.G_w + (long long)n * p.Kout * p.Ng;
                    auto consume = [&](uint32_t (&v)[32], int cc) {
                        if (row_ok) {
#pragma unroll
                            for (int i = 0; i < 32; ++i) { const float f = __uint_as_float(v[i]); sq4[i & 3] = fmaf(f, f, sq4[i & 3]); }
                            if (p.mode == 0) {
                                const int b_idx = nt * p.NT + cc;
                                if (p.a_is_x) {      // row = column j of G, tile column = output channel k: lanes write consecutive j
                                    float *dst = Gn + (long long)b_idx * p.Ng + a_idx;
#pragma unroll
                                    for (int i = 0; i < 32; ++i) __stcs(dst + (long long)i * p.Ng, __uint_as_float(v[i]));
                                }
                            }
                        }
                        if (p.mode == 0 && !p.a_is_x) {
                            // row = output channel k, tile columns = 32 consecutive j: each lane holds one row, so the
                            // warp transposes its 32 x 32 block through shared memory and every store instruction then
                            // writes one 128-byte row segment (scattered 16-byte pieces ran at a fraction of the rate)
                            float (*xp)[33] = xpose[warp - 2];
#pragma unroll
                            for (int i = 0; i < 32; ++i) xp[lane][i] = __uint_as_float(v[i]);
                            __syncwarp();
                            const int col = nt * p.NT + cc + lane;
                            const int rows_here = min(32, a_rows - q * 32);
                            if (col < p.Ng) {
                                float *dst = Gn + (long long)(mt * 128 + q * 32) * p.Ng + col;
                                for (int r = 0; r < rows_here; ++r) __stcs(dst + (long long)r * p.Ng, xp[r][lane]);
                            }
                            __syncwarp();
                        }
                    };
                    // columns in pairs of 32 with both loads in flight before the wait.  The second load of a tile with
                    // an odd number of 32-column blocks reads columns of this accumulator buffer that nobody uses.
                    for (int cc = 0; cc < n_cols; cc += 64) {
                        uint32_t v0[32], v1[32];
                        tmem_ld32_issue(t_addr + (uint32_t)cc, v0);
                        tmem_ld32_issue(t_addr + (uint32_t)(cc + 32), v1);
                        tmem_ld_wait32(v0); tmem_ld_wait32(v1);
                        consume(v0, cc);
                        if (cc + 32 < n_cols) consume(v1, cc + 32);
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
                    const float sq = warp_sum((sq4[0] + sq4[1]) + (sq4[2] + sq4[3]));
                    if (lane == 0) p.partial[(long long)n * p.slots + (mt * p.n_tiles + nt) * 4 + q] = sq;
                }
                buf ^= 1;
            }
            if (!CLIP && p.counters && lane == 0 && item + (int)gridDim.x >= p.total_tiles)
                __threadfence();          // after this warp's last item: its partial sums are visible to the CTA that folds them
            if (CLIP && live && row_ok) {
                // one owner per output element: add straight into the accumulator, or leave a partial sum for the fold
                const bool add = p.splits == 1;
                float *base = p.sum_out + (add ? 0ll : (long long)it.split * p.Kout * p.Ng);
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4) {
                    if (c4 * 32 < n_cols) {
                        const int b_idx = nt * p.NT + c4 * 32;
                        if (p.a_is_x) {
                            float *dst = base + (long long)b_idx * p.Ng + a_idx;
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                float *e = dst + (long long)i * p.Ng;
                                const float r = run[CLIP ? c4 * 32 + i : 0];
                                *e = add ? *e + r : r;
                            }
                        } else if (!p.n_pad_cols) {
                            float4 *dst = reinterpret_cast<float4 *>(base + (long long)a_idx * p.Ng + b_idx);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                float4 r = make_float4(run[CLIP ? c4 * 32 + 4 * i : 0], run[CLIP ? c4 * 32 + 4 * i + 1 : 0],
                                                       run[CLIP ? c4 * 32 + 4 * i + 2 : 0], run[CLIP ? c4 * 32 + 4 * i + 3 : 0]);
                                if (add) { const float4 o = dst[i]; r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w; }
                                dst[i] = r;
                            }
                        } else {
                            float *dst = base + (long long)a_idx * p.Ng + b_idx;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (b_idx + i < p.Ng) dst[i] = add ? dst[i] + run[CLIP ? c4 * 32 + i : 0] : run[CLIP ? c4 * 32 + i : 0];
                        }
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (!CLIP && p.counters && !abort_flag) {
        // The last CTA to finish (one ticket per CTA, nobody waits) folds every example's partial squared norms,
        // bias slots included, in slot order and publishes the squared norm(s): no finalising launch.
        __shared__ int last_cta;
        if (threadIdx.x == 0) {
            __threadfence();
            last_cta = atomicAdd(&p.counters[0], 1) == (int)gridDim.x - 1;
            if (last_cta) p.counters[0] = 0;
        }
        __syncthreads();
        if (last_cta) {
            __threadfence();
            // eight lanes per example (slot i goes to lane i % 8, the eight sums are added by a butterfly), four
            // examples per warp and trip: the walk is a chain of L2 round trips, so many examples go side by side
            const int groups = (int)(blockDim.x >> 3), group = (int)(threadIdx.x >> 3), sub = lane & 7;
            for (int n0 = 0; n0 < p.B; n0 += groups) {     // uniform trip count: the shuffles below need whole warps
                const int n = n0 + group;
                double sw = 0.0, sb = 0.0;
                if (n < p.B) {
                    const float *pn = p.partial + (long long)n * p.slots;
                    for (int i = sub; i < p.w_slots; i += 8) sw += (double)__ldcg(pn + i);
                    for (int i = p.w_slots + sub; i < p.slots; i += 8) sb += (double)__ldcg(pn + i);
                }
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) {
                    sw += __shfl_xor_sync(0xffffffffu, sw, o);
                    sb += __shfl_xor_sync(0xffffffffu, sb, o);
                }
                if (n < p.B && sub == 0) {
                    if (p.separate) { p.sqnorm[n * p.sq_stride] = (float)sw; p.sqnorm[n * p.sq_stride + 1] = (float)sb; }
                    else p.sqnorm[n * p.sq_stride] = (float)(sw + sb);
                    if (p.factor_out) {                    // the clipped-sum pass that follows reads its factors here
                        const float fw = clip_factor(p.separate ? sw : sw + sb, p.C_l);
                        const float fb = p.separate ? clip_factor(sb, p.C_l) : fw;
                        p.factor_out[2 * n] = fw; p.factor_out[2 * n + 1] = fb;
                        if (p.clip_out) {
                            if (p.separate) { p.clip_out[2 * n] = fw; p.clip_out[2 * n + 1] = fb; }
                            else p.clip_out[n] = fw;
                        }
                    }
                }
            }
        }
        __syncthreads();
    }
    if (abort_flag) {
        // give copies still in flight time to land before shared memory is released
        if (threadIdx.x == 0) { *p.status = DP_ERR_TIMEOUT; __threadfence(); }
        __nanosleep(200000);
        __syncthreads();
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}


// ----------------------------------------------------------------------------- single-pass fused clip (bf16)
// Per-layer clipping needs an example's whole squared norm before any entry of its gradient can be scaled, so the
// kernel above runs every contraction twice (a norm pass, then the clipped sum).  Here each contraction runs once:
// a thread-block cluster owns ALL tiles of one example's gradient of this layer, one tile per CTA, kept in the CTA's
// tensor memory.  Every CTA square-sums its tile, the CTAs exchange their sums through distributed shared memory
// (one remote store per pair of CTAs that reports its bytes to the receiver's barrier; every CTA loads its own
// operands, nothing is multicast), every CTA then knows the example's norm and factor, scales its tile into a running
// sum held in registers, and moves on to the cluster's next example while the tensor core already fills the other
// accumulator buffer.  Clusters split the batch; with more than one cluster the running sums leave as partial sums,
// folded in cluster order by the launch that follows.  Given the factors beforehand (norms from the Gram-matrix kernel
// below) the same kernel runs without clusters and without the norm pass: one tile a CTA, any number of tiles.
//
// Roles (384 threads): warp 0 issues the TMA loads of the A slabs, warp 2 those of the B slabs, warp 1 allocates tensor
// memory and issues the MMAs, warp 3 idles; warps 4-11 are the epilogue: warp w reads TMEM lanes 32*(w%4).. and the
// 128-column half (w-4)/4 of the tile, so a thread holds 128 running sums.  The first warpgroup gives registers up
// (setmaxnreg) and the epilogue warpgroups take them: 128*56 + 256*224 = 384*168, the launch's allocation.
constexpr int kClipThreads = 384;
constexpr int kClipRegsLaunch = 168, kClipRegsControl = 56, kClipRegsEpilogue = 224;
static_assert(128 * kClipRegsControl + 256 * kClipRegsEpilogue == kClipThreads * kClipRegsLaunch, "register split must add up");
constexpr int kMaxCluster = 8;
constexpr int kMaxExamplesPerCluster = 32;   // examples a cluster walks through when an SM target is set (calls run side by side)

__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// one-way remote store that reports its bytes to a barrier of the receiving CTA (no separate arrival to release it)
__device__ __forceinline__ void st_async_f32(uint32_t cluster_addr, float v, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "r"(__float_as_uint(v)), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
                 "selp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t polls) {
    for (uint32_t it = 0; it < polls; ++it) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((it & 63u) == 63u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

__global__ void __launch_bounds__(kClipThreads, 1)
conv_wgrad_clip1_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const TcParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2], norm_bar[4], warp_bar[4];
    __shared__ float warp_part[4][8];                   // [example mod 4][epilogue warp]: this CTA's partial sums
    __shared__ float norm_part[4][kMaxCluster];         // [example mod 4][source CTA]: every CTA's sum, sent by its first epilogue warp
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t tiles_u32 = smem_u32(tiles);
    const int cs = p.m_tiles * p.n_tiles;                 // cluster size = tiles of one example's gradient
    // With the factors known beforehand (p.factor) nothing is exchanged: the launch has no clusters and any number of tiles
    const bool known = p.factor != nullptr;
    const int rank = known ? (int)(blockIdx.x % (unsigned)cs) : (int)cluster_rank();
    const int mt = rank / p.n_tiles, nt = rank - mt * p.n_tiles;
    const int split = (int)blockIdx.x / cs;
    const int n_lo = split * p.per_split, n_hi = min(p.B, n_lo + p.per_split);

    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 2); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tmem_full[b]), 1); mbar_init(smem_u32(&tmem_empty[b]), 8); }
        for (int b = 0; b < 4; ++b) { mbar_init(smem_u32(&norm_bar[b]), 1); mbar_init(smem_u32(&warp_bar[b]), 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                   // every CTA's barriers exist before anyone arrives on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int *abort_p = &abort_flag;

    const int slab_bytes = p.Kt * kRowBytes;
    const int a_slabs_tile = 128 / p.slab_ch, b_slabs_tile = p.NT / p.slab_ch;
    const int a_slabs = min(a_slabs_tile, p.a_ext / p.slab_ch - mt * a_slabs_tile);
    const int b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - nt * b_slabs_tile);

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kClipRegsControl));
        if (warp == 0 || warp == 2) {
            // ------------------------------------------------------------ TMA producers (A slabs / B slabs)
            const bool is_a = warp == 0;
            const bool active = is_a ? (lane < a_slabs) : (lane < b_slabs);
            const bool is_x = is_a ? (p.a_is_x != 0) : (p.a_is_x == 0);
            const int slab = (is_a ? mt * a_slabs_tile : nt * b_slabs_tile) + lane;
            int c0, dw = 0, dh = 0, mul = 1;
            if (is_x) {
                const int j0 = slab * p.slab_ch;
                const int tap = j0 / p.Cin;
                c0 = j0 - tap * p.Cin;
                const int r = tap / p.S;
                dw = (tap - r * p.S) - p.pad;
                dh = r - p.pad;
                mul = p.stride;
            } else {
                c0 = slab * p.slab_ch;
            }
            const CUtensorMap *map = is_x ? &tmX : &tmY;
            const uint32_t dst_off = (is_a ? 0u : (uint32_t)p.a_bytes) + (uint32_t)(lane * slab_bytes);
            const uint32_t tx_bytes = (uint32_t)((is_a ? a_slabs : b_slabs) * slab_bytes);
            int stage = 0; uint32_t phase = 0;
            bool live = true;
            for (int n = n_lo; n < n_hi && live; ++n) {
                int ow0 = 0, oh0 = 0, tw = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    bool ok = true;
                    if (lane == 0) {
                        ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_p, p.wait_polls);
                        if (ok) mbar_expect_tx(smem_u32(&full_bar[stage]), tx_bytes);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { live = false; break; }
                    if (active)
                        tma_load_4d(tiles_u32 + stage * p.stage_bytes + dst_off, map, smem_u32(&full_bar[stage]), c0,
                                    ow0 * mul + dw, oh0 * mul + dh, n);
                    if (++tw == p.tiles_w) { tw = 0; ow0 = 0; oh0 += p.OHt; } else { ow0 += p.OWt; }
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        } else if (warp == 1 && lane == 0) {
            // ------------------------------------------------------------ MMA issuer (one lane)
            int stage = 0; uint32_t phase = 0, acc_phase = 0;
            int buf = 0;
            bool live = true;
            const uint64_t desc_base = operand_desc_base<false>((uint32_t)slab_bytes);
            const uint32_t desc_lo = (uint32_t)desc_base, desc_hi32 = (uint32_t)(desc_base >> 32);
            const int ksteps = p.Kt / p.krows;
            constexpr uint32_t kadvance = (uint32_t)(16 * kRowBytes) >> 4;
            const uint32_t idesc = instr_desc(b_slabs * p.slab_ch, 1u);
            for (int n = n_lo; n < n_hi && live; ++n) {
                if (!mbar_wait(smem_u32(&tmem_empty[buf]), ((acc_phase >> buf) & 1u) ^ 1u, abort_p, p.wait_polls)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                uint32_t accumulate = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_p, p.wait_polls)) { live = false; break; }
                    tc_fence_after();
                    const uint32_t a_src = tiles_u32 + stage * p.stage_bytes;
                    uint32_t ad = desc_lo | ((a_src & 0x3FFFFu) >> 4);
                    uint32_t bd = desc_lo | (((a_src + p.a_bytes) & 0x3FFFFu) >> 4);
#pragma unroll 4
                    for (int ks = 0; ks < ksteps; ++ks) {
                        umma<false>(d_tmem, ad, bd, desc_hi32, idesc, accumulate);
                        accumulate = 1;
                        ad += kadvance; bd += kadvance;
                    }
                    umma_commit(smem_u32(&empty_bar[stage]));
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!live) break;
                umma_commit(smem_u32(&tmem_full[buf]));
                acc_phase ^= 1u << buf;
                buf ^= 1;
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kClipRegsEpilogue));
        // ---------------------------------------------------------------- epilogue (8 warps)
        const int e = warp - 4, q = e & 3, half = e >> 2;
        const int row = q * 32 + lane;
        const int a_rows = min(128, p.a_ext - mt * 128);
        const int n_cols = min(p.NT, p.b_ext - nt * p.NT);
        const int my_cols = max(0, min(128, n_cols - half * 128));     // columns of this warp's half that exist
        int a_idx = mt * 128 + row;
        bool row_ok = row < a_rows && (!p.a_is_x || a_idx < p.Ng);
        if (p.s2d_st) {                                    // (rows are input columns in this form)
            a_idx = row < a_rows ? s2d_column(p, a_idx) : -1;
            row_ok = a_idx >= 0;
        }
        float run[128];
#pragma unroll
        for (int i = 0; i < 128; ++i) run[i] = 0.f;
        bool live = true;
        // One step behind, with two tiles of tensor memory: step s first finishes example s - 1 (waits for its partial sums
        // from the whole cluster, scales its tile into the running sum and hands the tile's columns back to the MMA warp,
        // which starts on example s + 1), then square-sums example s and sends its partial sums on their way.
        // Slots and barriers of the exchange come in fours: a slot of example j is overwritten by example j + 4, which a
        // warp sends only after it has scaled example j + 3, i.e. after every warp of the cluster has sent example
        // j + 3, which each of them did after scaling (and so after reading the slots of) example j + 2 and before it j.
        const int count = n_hi - n_lo;
        for (int step = 0; known && step < count && live; ++step) {
            // factors known: one read of the finished tile per example, scaled into the running sum
            const int buf = step & 1;
            const bool arrived = mbar_wait(smem_u32(&tmem_full[buf]), (uint32_t)((step >> 1) & 1), abort_p, p.wait_polls);
            if (!__all_sync(0xffffffffu, arrived)) { live = false; break; }
            tc_fence_after();
            const float f = __ldg(p.factor + 2 * (n_lo + step));
            const uint32_t t_addr = tmem_base + (uint32_t)(buf * 256 + half * 128) + ((uint32_t)(q * 32) << 16);
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                if (c2 * 64 < my_cols) {
                    uint32_t v0[32], v1[32];
                    tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64), v0);
                    tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64 + 32), v1);
                    tmem_ld_wait32(v0); tmem_ld_wait32(v1);
#pragma unroll
                    for (int i = 0; i < 32; ++i) run[c2 * 64 + i] = fmaf(f, __uint_as_float(v0[i]), run[c2 * 64 + i]);
#pragma unroll
                    for (int i = 0; i < 32; ++i) run[c2 * 64 + 32 + i] = fmaf(f, __uint_as_float(v1[i]), run[c2 * 64 + 32 + i]);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
        }
        for (int step = 0; !known && step <= count && live; ++step) {
            if (step >= 1) {
                // finish example step - 1 first: its tile leaves tensor memory before this step's tile is touched, so the
                // MMAs of the example after this one run while this step's tile is being square-summed
                const int j = step - 1, n = n_lo + j, buf = j & 1, slot = j & 3;
                const bool all_in = mbar_wait_cluster(smem_u32(&norm_bar[slot]), (uint32_t)((j >> 2) & 1), abort_p, p.wait_polls);
                if (!__all_sync(0xffffffffu, all_in)) { live = false; break; }
                // the same tree in every warp of every CTA (two entries a lane, then a butterfly): all of them apply the
                // identical factor
                double sn = lane < cs ? (double)norm_part[slot][lane] : 0.0;
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) sn += __shfl_xor_sync(0xffffffffu, sn, o);      // (at most eight CTAs)
                sn = __shfl_sync(0xffffffffu, sn, 0);
                // min(1, C_l / sqrt(sn)) in single precision here: the double-precision square root and division are
                // some hundreds of cycles on the path every example waits on
                const float f = (sn <= (double)p.C_l * (double)p.C_l) ? 1.0f : p.C_l / sqrtf((float)sn);
                if (rank == 0 && e == 0 && lane == 0) {
                    p.sqnorm[n * p.sq_stride] = (float)sn;
                    if (p.clip_out) p.clip_out[n] = f;
                }
                // pass 2: scale the tile into the running sum
                const uint32_t t_addr = tmem_base + (uint32_t)(buf * 256 + half * 128) + ((uint32_t)(q * 32) << 16);
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    if (c2 * 64 < my_cols) {
                        uint32_t v0[32], v1[32];
                        tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64), v0);
                        tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64 + 32), v1);
                        tmem_ld_wait32(v0); tmem_ld_wait32(v1);
#pragma unroll
                        for (int i = 0; i < 32; ++i) run[c2 * 64 + i] = fmaf(f, __uint_as_float(v0[i]), run[c2 * 64 + i]);
#pragma unroll
                        for (int i = 0; i < 32; ++i) run[c2 * 64 + 32 + i] = fmaf(f, __uint_as_float(v1[i]), run[c2 * 64 + 32 + i]);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
            }
            if (step < count) {
                const int buf = step & 1, slot = step & 3;
                const bool arrived = mbar_wait(smem_u32(&tmem_full[buf]), (uint32_t)((step >> 1) & 1), abort_p, p.wait_polls);
                if (!__all_sync(0xffffffffu, arrived)) { live = false; break; }
                tc_fence_after();
                const uint32_t t_addr = tmem_base + (uint32_t)(buf * 256 + half * 128) + ((uint32_t)(q * 32) << 16);
                // pass 1: this warp's share of the example's squared norm
                float sq4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {           // columns in pairs of 32, both loads in flight before the wait
                    if (c2 * 64 < my_cols) {                // (my_cols is a multiple of 64)
                        uint32_t v0[32], v1[32];
                        tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64), v0);
                        tmem_ld32_issue(t_addr + (uint32_t)(c2 * 64 + 32), v1);
                        tmem_ld_wait32(v0); tmem_ld_wait32(v1);
                        if (row_ok) {      // (columns past the real ones of an unfolded thin layer hold exact zeros)
#pragma unroll
                            for (int i = 0; i < 32; ++i) { const float f = __uint_as_float(v0[i]); sq4[i & 3] = fmaf(f, f, sq4[i & 3]); }
#pragma unroll
                            for (int i = 0; i < 32; ++i) { const float f = __uint_as_float(v1[i]); sq4[i & 3] = fmaf(f, f, sq4[i & 3]); }
                        }
                    }
                }
                const float sq = warp_sum((sq4[0] + sq4[1]) + (sq4[2] + sq4[3]));
                // The CTA's eight partial sums meet in its own shared memory first; its first epilogue warp adds them and
                // tells the cluster: lane r sends the sum to CTA r with a store that reports its bytes to that CTA's barrier
                // (one way; a plain remote store followed by a releasing remote arrival costs a round trip more).
                if (lane == 0) { warp_part[slot][e] = sq; mbar_arrive(smem_u32(&warp_bar[slot])); }
                if (e == 0) {
                    const bool mine_in = mbar_wait(smem_u32(&warp_bar[slot]), (uint32_t)((step >> 2) & 1), abort_p, p.wait_polls);
                    if (!__all_sync(0xffffffffu, mine_in)) { live = false; break; }
                    const float *w = warp_part[slot];
                    const float cta_sq = ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
                    // this CTA expects one float from every CTA of the cluster (its own included) in this slot's phase
                    if (lane == 0) mbar_expect_tx(smem_u32(&norm_bar[slot]), (uint32_t)(cs * 4));
                    if (lane < cs)
                        st_async_f32(map_to_cta(smem_u32(&norm_part[slot][rank]), (uint32_t)lane), cta_sq,
                                     map_to_cta(smem_u32(&norm_bar[slot]), (uint32_t)lane));
                }
            }
        }
        if (live && row_ok) {
            // one owner per output element: add straight into the accumulator, or leave a partial sum for the fold
            const bool add = p.splits == 1;
            float *base = p.sum_out + (add ? 0ll : (long long)split * p.Kout * p.Ng);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                if (c4 * 32 < my_cols) {
                    const int b_idx = nt * p.NT + half * 128 + c4 * 32;
                    if (p.a_is_x) {
                        float *dst = base + (long long)b_idx * p.Ng + a_idx;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            float *el = dst + (long long)i * p.Ng;
                            const float r = run[c4 * 32 + i];
                            *el = add ? *el + r : r;
                        }
                    } else if (!p.n_pad_cols) {
                        float4 *dst = reinterpret_cast<float4 *>(base + (long long)a_idx * p.Ng + b_idx);
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            float4 r = make_float4(run[c4 * 32 + 4 * i], run[c4 * 32 + 4 * i + 1], run[c4 * 32 + 4 * i + 2], run[c4 * 32 + 4 * i + 3]);
                            if (add) { const float4 o = dst[i]; r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w; }
                            dst[i] = r;
                        }
                    } else {
                        float *dst = base + (long long)a_idx * p.Ng + b_idx;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (b_idx + i < p.Ng) dst[i] = add ? dst[i] + run[c4 * 32 + i] : run[c4 * 32 + i];
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) { *p.status = DP_ERR_TIMEOUT; __threadfence(); }
        __nanosleep(200000);
        __syncthreads();
    }
    cluster_sync_all();                                   // nobody leaves while a peer may still write to its shared memory
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}



// ----------------------------------------------------------------------------- clipped sum as ONE matrix product (bf16)
// With the factors known, sum_n f_n dY_n^T Xcol_n is a single matrix product whose reduction runs over (example, pixel)
// once every row of dY carries its example's factor: the tensor core then adds all examples into one accumulator and
// nothing is read back from tensor memory per example (reading a 128 x 256 tile back costs as much as eight MMAs,
// which is what bounds a per-example clipped sum on layers with few pixels).  f_n * dY does not fit bf16, so a small
// launch before this one splits it into hi + lo (both bf16, hi = the rounded product, lo = the rounded remainder: what
// is lost is below 2^-17 of each product) and every k-step issues two MMAs, X with hi and X with lo.  A work item is a
// tile for a range of examples; with more than one range the tiles leave as partial sums for the fold.
// Roles as in the kernel at the top: warp 0 / 6 TMA (the warp that loads dY loads both copies), warp 1 MMA, warps 2-5 epilogue.
__global__ void __launch_bounds__(224, 1)
conv_wgrad_ssum_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmYhi,
                       const __grid_constant__ CUtensorMap tmYlo, const TcParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t tiles_u32 = smem_u32(tiles);

    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmYhi)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmYlo)) : "memory");
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 2); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tmem_full[b]), 1); mbar_init(smem_u32(&tmem_empty[b]), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int *abort_p = &abort_flag;

    const int slab_bytes = p.Kt * kRowBytes;
    const int a_slabs_tile = 128 / p.slab_ch, b_slabs_tile = p.NT / p.slab_ch;
    const bool a_is_y = p.a_is_x == 0;                        // which operand is dY (and so has a lo copy)

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------------------ TMA producers
        int stage = 0; uint32_t phase = 0;
        bool live = true;
        for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const int a_slab0 = it.mt * a_slabs_tile, a_slabs = min(a_slabs_tile, p.a_ext / p.slab_ch - a_slab0);
            const int b_slab0 = it.nt * b_slabs_tile, b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - b_slab0);
            const bool is_a = warp == 0;
            const bool is_y = is_a == a_is_y;
            const int mine = is_a ? a_slabs : b_slabs;       // slabs of this warp's operand; a dY warp issues each twice (hi, lo)
            const bool second = is_y && lane >= mine;        // lanes [mine, 2*mine) of a dY warp load the lo copies
            const int local = second ? lane - mine : lane;
            const bool active = lane < (is_y ? 2 * mine : mine);
            const int slab = (is_a ? a_slab0 : b_slab0) + local;
            int c0, dw = 0, dh = 0, mul = 1;
            if (!is_y) {
                const int j0 = slab * p.slab_ch;
                const int tap = j0 / p.Cin;
                c0 = j0 - tap * p.Cin;
                const int r = tap / p.S;
                dw = (tap - r * p.S) - p.pad;
                dh = r - p.pad;
                mul = p.stride;
            } else {
                c0 = slab * p.slab_ch;
            }
            const CUtensorMap *map = !is_y ? &tmX : (second ? &tmYlo : &tmYhi);
            const uint32_t dst_off = (second ? (uint32_t)p.lo_offset : (is_a ? 0u : (uint32_t)p.a_bytes)) + (uint32_t)(local * slab_bytes);
            const uint32_t tx_bytes = (uint32_t)((is_y ? 2 * mine : mine) * slab_bytes);
            for (int n = it.n_lo; n < it.n_hi && live; ++n) {
                int ow0 = 0, oh0 = 0, tw = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    bool ok = true;
                    if (lane == 0) {
                        ok = mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_p, p.wait_polls);
                        if (ok) mbar_expect_tx(smem_u32(&full_bar[stage]), tx_bytes);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { live = false; break; }
                    if (active)
                        tma_load_4d(tiles_u32 + stage * p.stage_bytes + dst_off, map, smem_u32(&full_bar[stage]), c0,
                                    ow0 * mul + dw, oh0 * mul + dh, n);
                    if (++tw == p.tiles_w) { tw = 0; ow0 = 0; oh0 += p.OHt; } else { ow0 += p.OWt; }
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0, acc_phase = 0;
            int buf = 0;
            bool live = true;
            const uint64_t desc_base = operand_desc_base<false>((uint32_t)slab_bytes);
            const uint32_t desc_lo = (uint32_t)desc_base, desc_hi32 = (uint32_t)(desc_base >> 32);
            const int ksteps = p.Kt / p.krows;
            constexpr uint32_t kadvance = (uint32_t)(16 * kRowBytes) >> 4;
            for (int item = blockIdx.x; item < p.total_tiles && live; item += gridDim.x) {
                const Item it = decode_item(p, item);
                const int b_slabs = min(b_slabs_tile, p.b_ext / p.slab_ch - it.nt * b_slabs_tile);
                const uint32_t idesc = instr_desc(b_slabs * p.slab_ch, 1u);
                if (!mbar_wait(smem_u32(&tmem_empty[buf]), ((acc_phase >> buf) & 1u) ^ 1u, abort_p, p.wait_polls)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * 256);
                uint32_t accumulate = 0;
                for (int n = it.n_lo; n < it.n_hi && live; ++n) {
                    for (int kt = 0; kt < p.k_tiles; ++kt) {
                        if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_p, p.wait_polls)) { live = false; break; }
                        tc_fence_after();
                        const uint32_t src = tiles_u32 + stage * p.stage_bytes;
                        uint32_t ad = desc_lo | ((src & 0x3FFFFu) >> 4);
                        uint32_t bd = desc_lo | (((src + p.a_bytes) & 0x3FFFFu) >> 4);
                        uint32_t ld = desc_lo | (((src + p.lo_offset) & 0x3FFFFu) >> 4);
#pragma unroll 2
                        for (int ks = 0; ks < ksteps; ++ks) {
                            umma<false>(d_tmem, ad, bd, desc_hi32, idesc, accumulate);                               // X with hi(f dY)
                            if (a_is_y) umma<false>(d_tmem, ld, bd, desc_hi32, idesc, 1u);                           // X with lo(f dY)
                            else umma<false>(d_tmem, ad, ld, desc_hi32, idesc, 1u);
                            accumulate = 1;
                            ad += kadvance; bd += kadvance; ld += kadvance;
                        }
                        umma_commit(smem_u32(&empty_bar[stage]));
                        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                    }
                }
                if (!live) break;
                umma_commit(smem_u32(&tmem_full[buf]));
                acc_phase ^= 1u << buf;
                buf ^= 1;
            }
        }
    } else if (warp >= 2 && warp <= 5) {
        // ------------------------------------------------------------ epilogue: one read of the finished tile per item
        const int q = warp & 3;
        const int row = q * 32 + lane;
        uint32_t full_phase = 0;
        int buf = 0;
        for (int item = blockIdx.x; item < p.total_tiles; item += gridDim.x) {
            const Item it = decode_item(p, item);
            const int mt = it.mt, nt = it.nt;
            const int a_rows = min(128, p.a_ext - mt * 128);
            const int n_cols = min(p.NT, p.b_ext - nt * p.NT);
            const int a_idx = mt * 128 + row;
            const bool row_ok = row < a_rows && (!p.a_is_x || a_idx < p.Ng);
            const bool arrived = mbar_wait(smem_u32(&tmem_full[buf]), (full_phase >> buf) & 1u, abort_p, p.wait_polls);
            if (!__all_sync(0xffffffffu, arrived)) break;
            full_phase ^= 1u << buf;
            tc_fence_after();
            const uint32_t t_addr = tmem_base + (uint32_t)(buf * 256) + ((uint32_t)(q * 32) << 16);
            const bool add = p.splits == 1;
            float *base = p.sum_out + (add ? 0ll : (long long)it.split * p.Kout * p.Ng);
            auto put = [&](uint32_t (&v)[32], int cc) {
                if (!row_ok) return;
                const int b_idx = nt * p.NT + cc;
                if (p.a_is_x) {
                    float *dst = base + (long long)b_idx * p.Ng + a_idx;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float *el = dst + (long long)i * p.Ng;
                        const float r = __uint_as_float(v[i]);
                        *el = add ? *el + r : r;
                    }
                } else {
                    float4 *dst = reinterpret_cast<float4 *>(base + (long long)a_idx * p.Ng + b_idx);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float4 r = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]), __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
                        if (add) { const float4 o = dst[i]; r.x += o.x; r.y += o.y; r.z += o.z; r.w += o.w; }
                        dst[i] = r;
                    }
                }
            };
            for (int cc = 0; cc < n_cols; cc += 64) {
                uint32_t v0[32], v1[32];
                tmem_ld32_issue(t_addr + (uint32_t)cc, v0);
                tmem_ld32_issue(t_addr + (uint32_t)(cc + 32), v1);
                tmem_ld_wait32(v0); tmem_ld_wait32(v1);
                put(v0, cc);
                if (cc + 32 < n_cols) put(v1, cc + 32);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
            buf ^= 1;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) { *p.status = DP_ERR_TIMEOUT; __threadfence(); }
        __nanosleep(200000);
        __syncthreads();
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// ----------------------------------------------------------------------------- norms from Gram matrices
// For a layer whose gradient is far larger than its pixel count squared, the squared norm of example n comes cheaper
// from the identity  ||dY_n^T Xcol_n||_F^2 = sum_{p,q} (dY_n dY_n^T)[p,q] (Xcol_n Xcol_n^T)[p,q]  over pixel pairs
// (the norm the clip factor of the paper's section 2 needs, without the gradient itself): two Gram matrices of
// [pixels x pixels], each a product over channels, and Xcol's is the sum over the taps of the Gram matrices of the
// shifted inputs.  Here the SAME shared-memory tiles as above (one TMA box = pixels x 64 channels, 128-byte rows,
// 128-byte swizzle) are read as K-major operands: the pixel is the M / N index and the channel the reduction index,
// and one tile serves as both A and B.  One CTA per example; a plane of up to 256 pixels (box rows, a multiple of 16)
// is one or two row tiles of 128, and since both matrices are symmetric the second row tile only needs the columns
// from 128 on, the first one counting its columns from 128 on twice.  Planes of 64 box pixels go two examples to a tile
// (one TMA box over two examples): the small MMAs of a single 64-pixel example are bound by their issue rate.
// Roles (192 threads): warp 0 TMA, warp 1 MMA issue, warps 2-5 read both matrices back and sum their products.
struct GramParams {
    int B, Cin, Kout, S, taps, stride, pad;
    int rows;                   // pixels of the box (zero rows past the plane included), a multiple of 16, <= 256
    int pack;                   // examples per tile: 2 when rows == 64 (two examples fill the 128 rows of an MMA; only the
                                // diagonal 64 x 64 blocks of the products are read), else 1
    int m_tiles, stages, stage_bytes;
    float C_l;
    float *sqnorm; long long sq_stride; float *factor_out; float *clip_out;
    int *status;
    uint32_t wait_polls;
};

// K-major operand of 128-byte rows with the 128-byte swizzle: 8-row groups 1024 B apart; the leading offset is unused
// because one instruction's 32 bytes of K lie inside one swizzle row.
__device__ __forceinline__ uint64_t kmajor_desc_base() {
    uint64_t d = (uint64_t)1 << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n_cols
__device__ __forceinline__ uint32_t instr_desc_kmajor(int n_cols) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((128u >> 4) << 24);
}

__global__ void __launch_bounds__(192, 1)
conv_gram_norm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const GramParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages], empty_bar[kMaxStages], tmem_full[2], tmem_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ __align__(8) uint64_t norm_bar;
    __shared__ double warp_part[4][4];      // [example & 3][quadrant]: a warp may run up to three examples ahead of the one that adds up

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *tiles = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t tiles_u32 = smem_u32(tiles);

    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmY)) : "memory");
        abort_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(smem_u32(&full_bar[s]), 1); mbar_init(smem_u32(&empty_bar[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&tmem_full[b]), 1); mbar_init(smem_u32(&tmem_empty[b]), 4); }
        mbar_init(smem_u32(&norm_bar), 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int *abort_p = &abort_flag;

    // tensor memory: one or two buffers of 256 columns; in a buffer dY's matrix first, then Xcol's
    const int nbuf = p.rows > 128 ? 1 : 2;
    const uint32_t x_col = p.rows > 128 ? 256u : 128u;
    const int y_slabs = p.Kout / 64, c_slabs = p.Cin / 64;
    const int slabs = y_slabs + p.taps * c_slabs;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer: one box per stage
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool live = true;
            const uint32_t tx_bytes = (uint32_t)(p.pack * p.rows * kRowBytes);
            for (int n = blockIdx.x * p.pack; n < p.B && live; n += gridDim.x * p.pack) {
                for (int mt = 0; mt < p.m_tiles && live; ++mt) {
                    int tap = 0, cs = 0;
                    for (int s = 0; s < slabs; ++s) {
                        if (!mbar_wait(smem_u32(&empty_bar[stage]), phase ^ 1u, abort_p, p.wait_polls)) { live = false; break; }
                        mbar_expect_tx(smem_u32(&full_bar[stage]), tx_bytes);
                        const uint32_t dst = tiles_u32 + stage * p.stage_bytes;
                        if (s < y_slabs) {
                            tma_load_4d(dst, &tmY, smem_u32(&full_bar[stage]), s * 64, 0, 0, n);
                        } else {
                            const int r = tap / p.S;
                            tma_load_4d(dst, &tmX, smem_u32(&full_bar[stage]), cs * 64, (tap - r * p.S) - p.pad, r - p.pad, n);
                            if (++cs == c_slabs) { cs = 0; ++tap; }
                        }
                        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0, acc_phase = 0;
            int buf = 0;
            bool live = true;
            const uint64_t desc_base = kmajor_desc_base();
            const uint32_t desc_lo = (uint32_t)desc_base, desc_hi32 = (uint32_t)(desc_base >> 32);
            for (int n = blockIdx.x * p.pack; n < p.B && live; n += gridDim.x * p.pack) {
                for (int mt = 0; mt < p.m_tiles && live; ++mt) {
                    const int col0 = mt * 128;                       // the tile's columns start at its own first row
                    const uint32_t idesc = instr_desc_kmajor(p.pack * p.rows - col0);
                    if (!mbar_wait(smem_u32(&tmem_empty[buf]), ((acc_phase >> buf) & 1u) ^ 1u, abort_p, p.wait_polls)) { live = false; break; }
                    tc_fence_after();
                    const uint32_t d_y = tmem_base + (uint32_t)(buf * 256), d_x = d_y + x_col;
                    for (int s = 0; s < slabs; ++s) {
                        if (!mbar_wait(smem_u32(&full_bar[stage]), phase, abort_p, p.wait_polls)) { live = false; break; }
                        tc_fence_after();
                        const uint32_t src = tiles_u32 + stage * p.stage_bytes + (uint32_t)(col0 * kRowBytes);
                        uint32_t ad = desc_lo | ((src & 0x3FFFFu) >> 4);
                        const bool is_y = s < y_slabs;
                        const uint32_t d_tmem = is_y ? d_y : d_x;
                        uint32_t accumulate = (s == 0 || s == y_slabs) ? 0u : 1u;
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {             // 64 channels = four steps of 16, 32 bytes apart in the row
                            umma<false>(d_tmem, ad, ad, desc_hi32, idesc, accumulate);
                            accumulate = 1;
                            ad += 2;
                        }
                        umma_commit(smem_u32(&empty_bar[stage]));
                        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                    }
                    if (!live) break;
                    umma_commit(smem_u32(&tmem_full[buf]));
                    acc_phase ^= 1u << buf;
                    if (nbuf == 2) buf ^= 1;
                }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue: sum over the tile of G_Y .* G_X
        const int q = warp & 3;
        uint32_t full_phase = 0;
        int buf = 0;
        bool live = true;
        int trip = 0;
        for (int n = blockIdx.x * p.pack; n < p.B && live; n += gridDim.x * p.pack) {
            double acc = 0.0;
            for (int mt = 0; mt < p.m_tiles; ++mt) {
                const int col0 = mt * 128;
                const bool arrived = mbar_wait(smem_u32(&tmem_full[buf]), (full_phase >> buf) & 1u, abort_p, p.wait_polls);
                if (!__all_sync(0xffffffffu, arrived)) { live = false; break; }
                full_phase ^= 1u << buf;
                tc_fence_after();
                const int row = col0 + q * 32 + lane;
                // packed: quadrants 0, 1 hold the first example (columns 0..63), quadrants 2, 3 the second (64..127)
                const int c_lo = p.pack == 2 ? (q >> 1) * 64 : 0;
                const int c_hi = p.pack == 2 ? c_lo + 64 : p.rows - col0;
                if (col0 + q * 32 < p.pack * p.rows) {               // warps whose rows all lie past the box read nothing
                    const uint32_t t_y = tmem_base + (uint32_t)(buf * 256) + ((uint32_t)(q * 32) << 16), t_x = t_y + x_col;
                    float s1[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};     // columns below / from 128
                    for (int cc = c_lo; cc < c_hi; cc += 32) {
                        uint32_t vy[32], vx[32];
                        tmem_ld32_issue(t_y + (uint32_t)cc, vy);
                        tmem_ld32_issue(t_x + (uint32_t)cc, vx);
                        tmem_ld_wait32(vy); tmem_ld_wait32(vx);
                        const bool twice = cc >= 128;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float pr = (cc + i < c_hi) ? __uint_as_float(vy[i]) * __uint_as_float(vx[i]) : 0.f;
                            if (twice) s2[i & 3] += pr; else s1[i & 3] += pr;
                        }
                    }
                    if (row < p.pack * p.rows)
                        acc += ((double)s1[0] + (double)s1[1]) + ((double)s1[2] + (double)s1[3]) +
                               2.0 * (((double)s2[0] + (double)s2[1]) + ((double)s2[2] + (double)s2[3]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&tmem_empty[buf]));
                if (nbuf == 2) buf ^= 1;
            }
            if (!live) break;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            // the four warps hand their sums to the one that publishes through a barrier word (no warp waits for
            // another except that one, and its wait is bounded like every other)
            if (lane == 0) { warp_part[trip & 3][q] = acc; mbar_arrive(smem_u32(&norm_bar)); }
            if (q == 0) {
                if (!mbar_wait(smem_u32(&norm_bar), (uint32_t)(trip & 1), abort_p, p.wait_polls)) { live = false; break; }
                if (lane < p.pack && n + lane < p.B) {
                    const double *w = warp_part[trip & 3];
                    const double sq = p.pack == 2 ? w[2 * lane] + w[2 * lane + 1] : (w[0] + w[1]) + (w[2] + w[3]);
                    const int m = n + lane;
                    p.sqnorm[m * p.sq_stride] = (float)sq;
                    const float f = clip_factor(sq, p.C_l);
                    if (p.factor_out) { p.factor_out[2 * m] = f; p.factor_out[2 * m + 1] = f; }
                    if (p.clip_out) p.clip_out[m] = f;
                }
            }
            ++trip;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) { *p.status = DP_ERR_TIMEOUT; __threadfence(); }
        __nanosleep(200000);
        __syncthreads();
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 512); }
}

// hi[i] = bf16(f_n y[i]), lo[i] = bf16(f_n y[i] - hi[i]) for every entry of example n (eight entries per thread)
__global__ void __launch_bounds__(256)
scale_split_kernel(const __nv_bfloat16 *__restrict__ y, const float *__restrict__ factor, long long per_example, long long total8,
                   __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo) {
    const long long i8 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i8 >= total8) return;
    const long long i = i8 * 8;
    const float f = factor[2 * (i / per_example)];
    __nv_bfloat16 v[8], h[8], l[8];
    *reinterpret_cast<uint4 *>(v) = *reinterpret_cast<const uint4 *>(y + i);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float x = f * __bfloat162float(v[e]);
        h[e] = __float2bfloat16_rn(x);
        l[e] = __float2bfloat16_rn(x - __bfloat162float(h[e]));
    }
    *reinterpret_cast<uint4 *>(hi + i) = *reinterpret_cast<const uint4 *>(h);
    *reinterpret_cast<uint4 *>(lo + i) = *reinterpret_cast<const uint4 *>(l);
}

// acc[i] += sum over splits of part[s][i], splits in index order (P a multiple of 4, both 16-byte aligned)
__global__ void __launch_bounds__(256)
fold_partial_sums_kernel(const float *__restrict__ part, int splits, long long P, float *__restrict__ acc) {
    const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= P) return;
    float4 a = *reinterpret_cast<const float4 *>(acc + i);
    for (int s = 0; s < splits; ++s) {
        const float4 v = __ldcs(reinterpret_cast<const float4 *>(part + (long long)s * P + i));
        a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    *reinterpret_cast<float4 *>(acc + i) = a;
}

__global__ void fold_partial_sums_scalar_kernel(const float *__restrict__ part, int splits, long long P, float *__restrict__ acc) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= P) return;
    float a = acc[i];
    for (int s = 0; s < splits; ++s) a += part[(long long)s * P + i];
    acc[i] = a;
}

dp_status launch_fold_partial_sums(const float *part, int splits, long long P, float *acc, cudaStream_t stream) {
    if (P % 4 == 0 && aligned(part, 16) && aligned(acc, 16))
        fold_partial_sums_kernel<<<(unsigned)((P / 4 + 255) / 256), 256, 0, stream>>>(part, splits, P, acc);
    else
        fold_partial_sums_scalar_kernel<<<(unsigned)((P + 255) / 256), 256, 0, stream>>>(part, splits, P, acc);
    DP_LAUNCH_CHECK("fold_partial_sums_kernel");
    return DP_OK;
}

// Layers whose input has too few channels for a TMA slab (C_in = 3 stems) are first unfolded:
// Xcol[n, oh, ow, j] = Xpad[n, oh*st + r - pad, ow*st + s - pad, c], j = (r*S + s)*C_in + c, zero for j >= R*S*C_in,
// with rows padded to a whole number of slabs.  The layer then is a 1x1 convolution over Xcol for the kernel above.
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
unfold_small_channels_kernel(const T *__restrict__ X, T *__restrict__ Xcol, const ConvGeom g, int n_pad, long long total) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;       // one 16-byte group of columns each
    if (idx >= total) return;
    const int groups = n_pad / VEC;
    const long long pixel = idx / groups;                                        // (n*OH + oh)*OW + ow
    const int j0 = (int)(idx - pixel * groups) * VEC;
    const int ow = (int)(pixel % g.OW);
    const long long t = pixel / g.OW;
    const int oh = (int)(t % g.OH);
    const long long n = t / g.OH;
    T v[VEC];
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const int j = j0 + e;
        T x = T(0.f);
        if (j < g.N) {
            const int c = j % g.Cin, rs = j / g.Cin;
            const int r = rs / g.S, s = rs - r * g.S;
            const int ih = oh * g.stride + r - g.pad, iw = ow * g.stride + s - g.pad;
            if (ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) x = X[((n * g.H + ih) * g.W + iw) * g.Cin + c];
        }
        v[e] = x;
    }
    *reinterpret_cast<uint4 *>(Xcol + pixel * n_pad + j0) = *reinterpret_cast<const uint4 *>(v);
}

// Same unfolding, one block per (output row, example): the R input rows the output row touches are staged in
// shared memory with their zero padding written out (so no window needs a bounds check), then every thread
// assembles 16-byte groups of columns from them through a table  column j -> offset inside the staged rows.
// Within one filter row r the (s, c) columns of a pixel are a contiguous run of the input row.
constexpr int kUnfoldMaxCols = 512;
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
unfold_rows_kernel(const T *__restrict__ X, T *__restrict__ Xcol, const ConvGeom g, int n_pad) {
    extern __shared__ __align__(16) unsigned char unfold_smem[];
    __shared__ __align__(16) short col_off[kUnfoldMaxCols];
    T *rows = reinterpret_cast<T *>(unfold_smem);          // [R][Wp*Cin], Wp = (OW-1)*stride + S padded pixels
    const int oh = blockIdx.x, n = blockIdx.y;
    const int row_p = ((g.OW - 1) * g.stride + g.S) * g.Cin, row_len = g.W * g.Cin, shift = g.pad * g.Cin;
    const int tap_row = g.S * g.Cin;
    for (int j = threadIdx.x; j < n_pad; j += 256) {
        const int r = j / tap_row;
        col_off[j] = (j < g.N) ? (short)(r * row_p + (j - r * tap_row)) : (short)-1;
    }
    for (int r = 0; r < g.R; ++r) {
        const int ih = oh * g.stride + r - g.pad;
        const bool inside = ih >= 0 && ih < g.H;
        const T *src = X + ((long long)n * g.H + (inside ? ih : 0)) * row_len;
        for (int i = threadIdx.x; i < row_p; i += 256) {
            const int col = i - shift;
            rows[r * row_p + i] = (inside && col >= 0 && col < row_len) ? src[col] : T(0.f);
        }
    }
    __syncthreads();
    const int groups = n_pad / VEC, step = g.stride * g.Cin;
    T *dst = Xcol + ((long long)n * g.OH + oh) * g.OW * n_pad;
    for (int chunk = threadIdx.x; chunk < g.OW * groups; chunk += 256) {
        const int ow = chunk / groups;
        const int j0 = (chunk - ow * groups) * VEC;
        const T *win = rows + ow * step;
        __align__(16) short off[VEC];
        if (VEC == 8) *reinterpret_cast<uint4 *>(off) = *reinterpret_cast<const uint4 *>(col_off + j0);
        else *reinterpret_cast<uint2 *>(off) = *reinterpret_cast<const uint2 *>(col_off + j0);
        __align__(16) T v[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) v[e] = off[e] >= 0 ? win[off[e]] : T(0.f);
        *reinterpret_cast<uint4 *>(dst + (long long)chunk * VEC) = *reinterpret_cast<const uint4 *>(v);
    }
}

// Space-to-depth regrouping of a thin strided input (C_in * stride^2 <= 16 channels): pixel (a, b) of the result
// holds the stride x stride block of padded-input pixels (stride*a + dy, stride*b + dx) as channels
// (dy*stride + dx)*C_in + c, zero-filled up to 16.  The strided R x S convolution over the input is then a
// stride-1 convolution with ceil(R/stride) x ceil(S/stride) taps over 16-channel pixels, and the (at most four)
// taps of one filter row are 64 contiguous values: one 128-byte operand row per output pixel, read straight
// from this buffer by a tensor map whose pixel stride (32 bytes) is smaller than its row (128 bytes).
__global__ void __launch_bounds__(256)
space_to_depth_kernel(const __nv_bfloat16 *__restrict__ X, __nv_bfloat16 *__restrict__ Xs, const ConvGeom g, int Hs, int Ws, long long total) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // one output pixel each
    if (idx >= total) return;
    const int b = (int)(idx % Ws);
    const long long t = idx / Ws;
    const int a = (int)(t % Hs);
    const long long n = t / Hs;
    __align__(16) __nv_bfloat16 v[16];
#pragma unroll
    for (int ch = 0; ch < 16; ++ch) v[ch] = __float2bfloat16(0.f);
    const int st = g.stride;
    for (int dy = 0; dy < st; ++dy) {
        const int ih = st * a + dy - g.pad;
        if (ih < 0 || ih >= g.H) continue;
        for (int dx = 0; dx < st; ++dx) {
            const int iw = st * b + dx - g.pad;
            if (iw < 0 || iw >= g.W) continue;
            const __nv_bfloat16 *src = X + ((n * g.H + ih) * g.W + iw) * g.Cin;
            for (int c = 0; c < g.Cin; ++c) v[(dy * st + dx) * g.Cin + c] = src[c];
        }
    }
    uint4 *dst = reinterpret_cast<uint4 *>(Xs + idx * 16);
    dst[0] = *reinterpret_cast<const uint4 *>(v);
    dst[1] = *reinterpret_cast<const uint4 *>(v + 8);
}

// ----------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// What the tensor-core kernel is actually given: the layer itself, or its unfolded 1x1 form.
struct TcProblem {
    bool ok, unfold;
    ConvGeom eff;       // geometry the kernel tiles
    int n_pad;          // unfolded row length (columns incl. zero padding)
};

// A 1 x 1 convolution with stride 1 is a plain product over the pixels, whatever their arrangement: its planes are
// flattened to one row of H*W pixels, so that a pixel tile is any run of pixels (no width / height rounding: 14 x 14
// is 208 reduction rows instead of 240) and a TMA box is one long run instead of many short rows.
static void flatten_pointwise(ConvGeom &e) {
    if (e.R == 1 && e.S == 1 && e.stride == 1 && e.pad == 0 && e.H > 1) {
        e.W = e.H * e.W; e.H = 1;
        e.OW = e.OH * e.OW; e.OH = 1;
    }
}

static TcProblem tc_problem(int dtype, const ConvGeom &g) {
    TcProblem pr; pr.ok = false; pr.unfold = false; pr.eff = g; pr.n_pad = g.N;
    const int slab_ch = (dtype == DP_BF16) ? 64 : 32;
    if (g.Kout % slab_ch) return pr;
    if (g.Cin % slab_ch == 0) { pr.ok = true; flatten_pointwise(pr.eff); return pr; }
    // small-channel layers only: the unfolded copy costs N/C_in times the input, which is only worth it for thin inputs
    if (g.Cin > 8 || g.N > 512) return pr;
    pr.unfold = true;
    pr.n_pad = (g.N + slab_ch - 1) / slab_ch * slab_ch;
    ConvGeom e = g;
    e.H = g.OH; e.W = g.OW; e.Cin = pr.n_pad; e.R = 1; e.S = 1; e.stride = 1; e.pad = 0;
    e.N = pr.n_pad;
    flatten_pointwise(e);
    pr.eff = e;
    pr.ok = true;
    return pr;
}

// Cycle model of one MMA step (16 bf16 / 8 tf32 reduction rows) for the tiling search.  Measured on B200: an
// instruction occupies the tensor pipe for N/2 cycles, and shared memory moves 128 B per cycle in total, shared by
// the tensor core's operand reads (always 128 rows of A plus N rows of B, 32 B per row and step), the TMA fill of the
// stage and, for split tf32, the split warps (they read every landed byte once and write the lo copy).
static double step_cycles(int dtype, int n_cols, double a_slabs_loaded, double b_slabs) {
    if (dtype == DP_BF16) {
        const double smem = 4096.0 + 32.0 * n_cols + 2048.0 * (a_slabs_loaded + b_slabs);
        return std::max(n_cols / 2.0, smem / 128.0);
    }
    if (dtype == DP_TF32) {   // one MMA per step; the stage is filled once, read once and written back once by the rounding warps
        const double smem = 4096.0 + 32.0 * n_cols + 1024.0 * (a_slabs_loaded + b_slabs) * 3.0;
        return std::max(n_cols / 2.0, smem / 128.0);
    }
    const double smem = 3.0 * (4096.0 + 32.0 * n_cols) + 1024.0 * (a_slabs_loaded + b_slabs) * 3.0;
    return std::max(3.0 * n_cols / 2.0, smem / 128.0);
}

static TcPlan search_plan(int dtype, const ConvGeom &g, int mode);

// single-pass clipped sum: how many clusters share the batch and how many examples each walks through
// scaled-sum product: example ranges per tile.  A launch that already has a CTA for a quarter of the SMs keeps whole
// tiles (no partial sums to fold); fewer tiles are cut up to half of the SMs.
static void ssum_split(int B, int tiles, int &splits, int &per_split) {
    const int sms = sm_target();
    // (side by side with other calls, under an SM target, a quarter: fewer partial sums to write and fold)
    int want = (tiles * 4 >= sms) ? 1 : (sms / (sm_target_set() ? 4 : 2)) / tiles;
    if (want < 1) want = 1;
    if (want > B) want = B;
    per_split = (B + want - 1) / want;
    splits = (B + per_split - 1) / per_split;
}

static int max_active_clusters(int cluster_size);
// K, NT: pixels per example and columns per tile (for a rough time of one example in one CTA)
static void cluster_split(int B, int cluster_size, int K, int NT, int &splits, int &per_split) {
    int want = std::min(sm_target() / cluster_size, max_active_clusters(cluster_size));
    // A caller that set an SM target runs calls side by side: what counts then is SM time, and a cluster that walks
    // through several examples spends its start-up, its first loads and its final stores once for all of them -- up
    // to thirty-two examples (a whole chunk of the per-layer workload: one example range, nothing to fold), and not
    // beyond some 60 microseconds a launch, so that no call holds its stream up for long.
    if (sm_target_set()) {
        const double cycles = (K / 16.0) * std::max(NT / 2.0, 64.0) * 1.5;
        const int per = std::max(1, std::min(kMaxExamplesPerCluster, (int)(120000.0 / cycles)));
        want = std::min(want, std::max(1, B / per));
    }
    if (want < 1) want = 1;
    if (want > B) want = B;
    per_split = (B + want - 1) / want;
    splits = (B + per_split - 1) / per_split;
}

// The tiling search is pure; its results are memoised per layer geometry (host side only).
// mode: 0 gradients are stored, 1 norms only, 2 clipped sum (running sum in registers: at most 128 columns per tile)
static TcPlan make_plan(int dtype, const ConvGeom &g, int mode) {
    static std::mutex mu;
    static std::map<std::array<int, 12>, TcPlan> memo;
    const std::array<int, 12> key = {dtype, g.H, g.W, g.Cin, g.Kout, g.R, g.S, g.stride, g.pad, g.B, mode, sm_target_set() ? -sm_target() : sm_target()};
    std::lock_guard<std::mutex> lock(mu);
    auto it = memo.find(key);
    if (it != memo.end()) return it->second;
    const TcPlan pl = search_plan(dtype, g, mode);
    memo.emplace(key, pl);
    return pl;
}

// max_nt = 128 plans the clipped-sum mode: its running sum lives in registers (128 columns per thread) and the
// work items are (example range, tile) pairs, so the wave count no longer depends on the batch size
// mode 3 plans the single-pass clipped sum: all tiles of an example in one cluster (at most kMaxCluster of them), the
// clusters share the batch, and what is minimised is SM time (clusters x CTAs x time), not the time of one launch
static TcPlan search_plan(int dtype, const ConvGeom &g, int mode) {
    const int max_nt = (mode == 2) ? 128 : 256;
    const bool rows_are_inputs = mode == 6;              // mode 6: mode 3 with the rows of D fixed to the input columns
    const bool any_tiles = mode == 7;                    // mode 7: mode 3 without clusters (factors known): any number of tiles
    if (mode == 6 || mode == 7) mode = 3;
    TcPlan best; best.ok = false;
    const int slab_ch = (dtype == DP_BF16) ? 64 : 32;
    const int krows = (dtype == DP_BF16) ? 16 : 8;
    if (g.Cin % slab_ch || g.Kout % slab_ch) return best;
    if (g.stride > 8 || g.K < 1 || g.OH > 65535) return best;
    const int sms = sm_target();
    const int a_slabs_tile = 128 / slab_ch;
    const int copies = (dtype == DP_F32) ? 2 : 1;       // split tf32 keeps a hi and a lo copy of every stage
    double best_cost = 1e300;
    for (int a_is_x = rows_are_inputs ? 1 : 0; a_is_x < 2; ++a_is_x) {
        const int a_ext = a_is_x ? g.N : g.M, b_ext = a_is_x ? g.M : g.N;
        for (int NT = slab_ch; NT <= max_nt; NT += slab_ch) {
            if (NT != 32 && NT % 64) continue;
            if (NT > b_ext) break;
            const int m_tiles = (a_ext + 127) / 128, n_tiles = (b_ext + NT - 1) / NT;
            const int slabs = a_slabs_tile + NT / slab_ch;
            const long long total_tiles = (long long)g.B * m_tiles * n_tiles;
            if (total_tiles > 0x7fffffffLL) continue;
            if (mode == 3 && !any_tiles && m_tiles * n_tiles > kMaxCluster) continue;
            const int y_slabs = (mode == 4) ? (a_is_x ? NT / slab_ch : a_slabs_tile) : 0;     // second (lo) copy of the dY slabs
            // per-CTA share of (example, tile) units: whole waves of tiles, or in clipped-sum mode an even share of the examples
            double waves = (mode != 2) ? (double)((total_tiles + sms - 1) / sms)
                                       : std::max(1.0, (double)total_tiles / sms);
            double sm_share = 1.0;
            if (mode == 4) {
                int splits, per;
                ssum_split(g.B, m_tiles * n_tiles, splits, per);
                waves = per;
                sm_share = (double)std::min(splits * m_tiles * n_tiles, sms);
            }
            if (mode == 3) {
                int splits, per;
                cluster_split(g.B, m_tiles * n_tiles, g.K, NT, splits, per);
                waves = per;                                       // examples a cluster walks through
                sm_share = (double)splits * m_tiles * n_tiles;      // SMs the launch holds meanwhile
            }
            const double a_loaded = (double)(a_ext / slab_ch) / m_tiles, b_loaded = (double)(b_ext / slab_ch) / n_tiles;
            const double step = step_cycles(dtype, NT, a_loaded, b_loaded) * (mode == 4 ? 2.0 : 1.0);
            // the epilogue of a tile overlaps the main loop of the next; what it costs depends on what it does with
            // the 128 x NT accumulator: stores run at about 16 B/clk per SM when lanes write consecutive addresses
            // (rows of D are gradient columns) and about 7 B/clk otherwise; reading TMEM alone is cheap
            const double epilogue = (mode == 0) ? 128.0 * NT * 4.0 / (a_is_x ? 16.0 : 7.0)
                                  : (mode == 1 ? 6.0 * NT : (mode == 2 ? 10.0 * NT : (mode == 4 ? 0.0 : 10.0 * std::min(NT, 128) + 600.0)));
            // a pixel tile may reach past the output plane (its rows there are zero-filled by TMA and add nothing):
            // a 7 x 7 plane is one 8 x 8 tile of 64 reduction rows instead of four 4 x 4 tiles of 16
            const int oh_max = std::min((g.OH + 7) / 8 * 8, 256 / g.stride), ow_max = std::min((g.OW + 15) / 16 * 16, 256 / g.stride);
            for (int OHt = 1; OHt <= oh_max; ++OHt) {
                for (int OWt = 1; OWt <= ow_max; ++OWt) {
                    if (OWt > g.OW && OWt % 8) continue;      // overshoot only to the next multiple of eight
                    if (OHt > g.OH && OHt % 8) continue;
                    const int Kt = OHt * OWt;
                    if (Kt % krows || Kt > 256) continue;
                    const int stage_bytes = (slabs + y_slabs) * Kt * kRowBytes * copies;
                    int stages = kSmemBudget / stage_bytes;
                    if (stages < 2) continue;
                    if (stages > kMaxStages) stages = kMaxStages;
                    const int tw = (g.OW + OWt - 1) / OWt, th = (g.OH + OHt - 1) / OHt;
                    // a stage: its MMA steps plus the hand-over (barrier wait, commit) of the issuing thread
                    double stage_cost = (double)(Kt / krows) * step + 250.0;
                    // a TMA warp: barrier wait + expect_tx, then one copy per slab it owns (A or B), all latency-bound on that warp
                    stage_cost = std::max(stage_cost, 350.0 + 110.0 * std::max(a_loaded, b_loaded));
                    if (dtype != DP_BF16)   // split warps, two groups in turn: a fixed fence/hand-over plus their share of the bytes
                        stage_cost = std::max(stage_cost, 0.5 * (1000.0 + (a_loaded + b_loaded) * Kt * 2.5));
                    double mainloop = stage_cost * tw * th;
                    if (stages < 3) mainloop *= 1.15;
                    const double cost = ((std::max(mainloop, epilogue) + 300.0) * waves + (mode == 3 ? 4000.0 : (mode == 4 ? 6000.0 : 0.0))) * sm_share;
                    if (cost < best_cost) {
                        best_cost = cost;
                        best.ok = true; best.a_is_x = a_is_x; best.a_ext = a_ext; best.b_ext = b_ext;
                        best.m_tiles = m_tiles; best.n_tiles = n_tiles; best.NT = NT;
                        best.OWt = OWt; best.OHt = OHt; best.tiles_w = tw; best.tiles_h = th; best.Kt = Kt;
                        best.k_tiles = tw * th; best.stages = stages; best.stage_bytes = stage_bytes;
                        best.a_bytes = a_slabs_tile * Kt * kRowBytes;
                        best.smem = (size_t)stages * stage_bytes + 1024;
                    }
                }
            }
        }
    }
    return best;
}

bool tc_eligible(int dtype, const ConvGeom &g0, int epilogue) {
    const TcProblem pr = tc_problem(dtype, g0);
    if (!pr.ok || !encode_fn() || !make_plan(dtype, pr.eff, epilogue == DP_EPI_STORE_NORM ? 0 : 1).ok) return false;
    return epilogue != DP_EPI_CLIP_ACCUM || make_plan(dtype, pr.eff, 2).ok;
}

// The single-pass kernel's register split only adds up when the launch allocates kClipRegsLaunch registers a thread.
static bool clip1_registers_ok() {
    static int ok = -1;
    if (ok < 0) {
        cudaFuncAttributes attr;
        ok = (cudaFuncGetAttributes(&attr, conv_wgrad_clip1_kernel) == cudaSuccess && attr.numRegs == kClipRegsLaunch) ? 1 : 0;
        if (!ok) (void)cudaGetLastError();
    }
    return ok == 1;
}

// How many clusters of this size the GPU can hold at once (a cluster needs all its SMs free in one GPC at the same
// time, so this is less than SMs / size); more clusters than that would run as a second wave.  Unknown (no device): no cap.
static int max_active_clusters(int cluster_size) {
    static std::mutex mu;
    static int cached[kMaxCluster + 1] = {0};
    if (cluster_size < 1 || cluster_size > kMaxCluster) return 1 << 30;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[cluster_size] == 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(cluster_size * 64)); cfg.blockDim = dim3(kClipThreads); cfg.dynamicSmemBytes = kSmemBudget + 1024;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = (unsigned)cluster_size; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        const bool ok = cudaFuncSetAttribute(conv_wgrad_clip1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048) == cudaSuccess &&
                        cudaOccupancyMaxActiveClusters(&n, conv_wgrad_clip1_kernel, &cfg) == cudaSuccess && n > 0;
        if (!ok) (void)cudaGetLastError();
        cached[cluster_size] = ok ? n : -1;
    }
    return cached[cluster_size] > 0 ? cached[cluster_size] : 1 << 30;
}

// Thin strided layers (a 7 x 7 stride-2 stem on RGB) in space-to-depth form, see space_to_depth_kernel: the geometry the
// kernel tiles is a stride-1 convolution with ceil(R/stride) x 1 taps of 64 "channels" (one filter row's window).
struct S2dProblem { bool ok; int R2, Hs, Ws; ConvGeom eff; };
static S2dProblem s2d_problem(int dtype, const ConvGeom &g, const TcProblem &pr) {
    S2dProblem sp = {};
    if (dtype != DP_BF16 || !pr.ok || !pr.unfold || g.stride < 2 || g.Cin * g.stride * g.stride > 16 || g.Kout % 64) return sp;
    if ((g.S + g.stride - 1) / g.stride > 4) return sp;
    sp.R2 = (g.R + g.stride - 1) / g.stride;
    sp.Hs = g.OH + sp.R2 - 1; sp.Ws = g.OW + 3;
    if ((size_t)sp.Hs * sp.Ws * 32 > (size_t)g.OH * g.OW * pr.n_pad * 2) return sp;     // lives in the unfolded copy's room
    ConvGeom e = g;
    e.Cin = 64; e.R = sp.R2; e.S = 1; e.stride = 1; e.pad = 0; e.H = sp.Hs; e.W = g.OW;
    e.N = sp.R2 * 64;
    sp.eff = e; sp.ok = true;
    return sp;
}

// The single-pass plan of a layer and the geometry it tiles: bf16 inputs, the example's gradient fits the tensor memory
// of one cluster.  Thin strided layers take the space-to-depth form when that has a plan (rows of D = input columns).
static bool clip1_plan(int dtype, const ConvGeom &g0, const TcProblem &pr, TcPlan &pl, ConvGeom &g, bool &s2d) {
    s2d = false;
    if (dtype != DP_BF16 || !pr.ok) return false;
    const S2dProblem sp = s2d_problem(dtype, g0, pr);
    if (sp.ok) {
        pl = make_plan(dtype, sp.eff, 6);
        if (pl.ok) { g = sp.eff; s2d = true; return true; }
    }
    g = pr.eff;
    pl = make_plan(dtype, pr.eff, 3);
    return pl.ok;
}

// clipped-sum mode: how many example ranges each tile is cut into so that every SM has an item
static void clip_split(const ConvGeom &g, const TcPlan &pl, int &splits, int &per_split) {
    const int tiles = pl.m_tiles * pl.n_tiles;
    int want = sm_target() / tiles;
    if (want < 1) want = 1;
    if (want > g.B) want = g.B;
    per_split = (g.B + want - 1) / want;
    splits = (g.B + per_split - 1) / per_split;
}

int tc_norm_slots(int dtype, const ConvGeom &g0, int epilogue) {
    const TcProblem pr = tc_problem(dtype, g0);
    if (!pr.ok) return 0;
    const TcPlan pl = make_plan(dtype, pr.eff, epilogue == DP_EPI_STORE_NORM ? 0 : 1);
    return pl.ok ? pl.m_tiles * pl.n_tiles * 4 : 0;
}

static size_t unfold_bytes(int dtype, const ConvGeom &g0, const TcProblem &pr) {
    if (!pr.unfold) return 0;
    return round_up((size_t)g0.B * g0.OH * g0.OW * pr.n_pad * (dtype == DP_BF16 ? 2 : 4), 1024);
}

// the row-staging form of the unfolding: its staged rows must fit shared memory and its offsets 16 bits
static size_t unfold_rows_smem(int dtype, const ConvGeom &g) {
    return (size_t)g.R * ((size_t)(g.OW - 1) * g.stride + g.S) * g.Cin * (dtype == DP_BF16 ? 2 : 4);
}
static bool unfold_rows_ok(int dtype, const ConvGeom &g, int n_pad) {
    const size_t bytes = unfold_rows_smem(dtype, g);
    return bytes <= 40 * 1024 && bytes / (dtype == DP_BF16 ? 2 : 4) < 32768 && n_pad <= kUnfoldMaxCols && g.B <= 65535;
}

static size_t ssum_copy_bytes(const ConvGeom &g) { return round_up((size_t)g.B * g.OH * g.OW * g.Kout * 2, 1024); }
bool tc_clip_scaled_sum(int dtype, const ConvGeom &g0);
bool tc_clip_scaled_tiles(int dtype, const ConvGeom &g0);
static void scaled_tiles_split(const ConvGeom &g, const TcPlan &pl, int &splits, int &per);

// layout: [unfolded input, if any][partial sums of the clipped-sum mode, if any], or the scaled copies of dY and partial sums
size_t tc_workspace_bytes(int dtype, const ConvGeom &g0, int epilogue) {
    const TcProblem pr = tc_problem(dtype, g0);
    if (!pr.ok) return 0;
    size_t bytes = unfold_bytes(dtype, g0, pr);
    if (epilogue == DP_EPI_CLIP_ACCUM) {
        const TcPlan pl = make_plan(dtype, pr.eff, 2);
        if (!pl.ok) return 0;
        int splits, per;
        clip_split(pr.eff, pl, splits, per);
        TcPlan one; ConvGeom og; bool s2d;
        if (clip1_plan(dtype, g0, pr, one, og, s2d)) {     // room for either form: the single pass may be unavailable at run time
            int s1, p1;
            cluster_split(og.B, one.m_tiles * one.n_tiles, og.K, one.NT, s1, p1);
            splits = std::max(splits, s1);
        }
        size_t clip_bytes = splits > 1 ? sizeof(float) * (size_t)splits * g0.M * g0.N : 0;
        if (tc_clip_scaled_sum(dtype, g0)) {
            const TcPlan sp = make_plan(dtype, pr.eff, 4);
            int s4, p4;
            ssum_split(pr.eff.B, sp.m_tiles * sp.n_tiles, s4, p4);
            clip_bytes = std::max(clip_bytes, 2 * ssum_copy_bytes(pr.eff) + (s4 > 1 ? sizeof(float) * (size_t)s4 * g0.M * g0.N : 0));
        }
        if (tc_clip_scaled_tiles(dtype, g0)) {
            int s7, p7;
            scaled_tiles_split(pr.eff, make_plan(dtype, pr.eff, 7), s7, p7);
            clip_bytes = std::max(clip_bytes, s7 > 1 ? sizeof(float) * (size_t)s7 * g0.M * g0.N : (size_t)0);
        }
        bytes += clip_bytes;
    }
    return bytes;
}

static int gram_describe(int dtype, const ConvGeom &g0, int *out, int n);
int tc_describe_plan(int dtype, const ConvGeom &g0, int epilogue, int *out, int n) {
    const TcProblem pr = tc_problem(dtype, g0);
    if (!pr.ok) return 0;
    if (epilogue == 5) return gram_describe(dtype, g0, out, n);
    TcPlan pl;
    if (epilogue == 3) {
        ConvGeom g; bool s2d;
        if (!clip1_plan(dtype, g0, pr, pl, g, s2d)) return 0;
    } else {
        pl = make_plan(dtype, pr.eff, epilogue);
    }
    if (!pl.ok) return 0;
    const int v[12] = {pl.a_is_x, pl.a_ext, pl.b_ext, pl.m_tiles, pl.n_tiles, pl.NT, pl.OWt, pl.OHt, pl.Kt, pl.k_tiles,
                       pl.stages, pl.stage_bytes};
    for (int i = 0; i < n && i < 12; ++i) out[i] = v[i];
    return 12;
}

// channels-last [B, H, W, C] tensor, box = {one slab of channels, boxW, boxH, 1 example}; `step` > 1 walks every
// step-th pixel (the box then spans boxW*step pixels and delivers boxW of them)
static bool encode_nhwc(CUtensorMap *map, int dtype, const void *base, int C, int W, int H, int Bn, int boxW, int boxH, int step, int boxN = 1) {
    const cuuint64_t es = (dtype == DP_BF16) ? 2 : 4;
    const cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)Bn};
    const cuuint64_t strides[3] = {(cuuint64_t)C * es, (cuuint64_t)W * C * es, (cuuint64_t)H * W * C * es};
    const cuuint32_t box[4] = {(cuuint32_t)(kRowBytes / es), (cuuint32_t)(boxW * step), (cuuint32_t)(boxH * step), (cuuint32_t)boxN};
    const cuuint32_t estr[4] = {1, (cuuint32_t)step, (cuuint32_t)step, 1};
    return encode_fn()(map, dtype == DP_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4,
                       const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                       dtype == DP_BF16 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

dp_status launch_conv_tc(int dtype, int epilogue, const void *X, const void *dY, const ConvGeom &g_in, float *G_w,
                         float *partial, int slots, const float *factor, float *acc_w, void *tc_workspace, int *status,
                         cudaStream_t stream, bool second_pass, const TcInlineClip *inline_clip, const TcPublish *publish) {
    const bool clip = epilogue == DP_EPI_CLIP_ACCUM;
    const ConvGeom &g0 = g_in;
    const TcProblem pr = tc_problem(dtype, g0);
    if (!pr.ok || !encode_fn()) return DP_ERR_UNSUPPORTED;
    const ConvGeom &g = pr.eff;
    const TcPlan pl = make_plan(dtype, g, clip ? 2 : (epilogue == DP_EPI_STORE_NORM ? 0 : 1));
    if (!pl.ok) return DP_ERR_UNSUPPORTED;
    char *ws_bytes = static_cast<char *>(tc_workspace);
    if (pr.unfold) {
        // in a fused clip call this function runs twice (norm pass, then clipped-sum pass): the unfolded input is
        // rebuilt only by the first of them
        if (!(clip && second_pass)) {
            const int vec = (dtype == DP_BF16) ? 8 : 4;
            const long long total = (long long)g0.B * g0.OH * g0.OW * (pr.n_pad / vec);
            const unsigned blocks = (unsigned)((total + 255) / 256);
            const size_t row_smem = unfold_rows_smem(dtype, g0);
            if (unfold_rows_ok(dtype, g0, pr.n_pad)) {
                const dim3 grid_rows(g0.OH, g0.B);
                if (dtype == DP_BF16)
                    unfold_rows_kernel<__nv_bfloat16, 8><<<grid_rows, 256, row_smem, stream>>>(
                        static_cast<const __nv_bfloat16 *>(X), reinterpret_cast<__nv_bfloat16 *>(ws_bytes), g0, pr.n_pad);
                else
                    unfold_rows_kernel<float, 4><<<grid_rows, 256, row_smem, stream>>>(
                        static_cast<const float *>(X), reinterpret_cast<float *>(ws_bytes), g0, pr.n_pad);
            } else if (dtype == DP_BF16)
                unfold_small_channels_kernel<__nv_bfloat16, 8><<<blocks, 256, 0, stream>>>(
                    static_cast<const __nv_bfloat16 *>(X), reinterpret_cast<__nv_bfloat16 *>(ws_bytes), g0, pr.n_pad, total);
            else
                unfold_small_channels_kernel<float, 4><<<blocks, 256, 0, stream>>>(
                    static_cast<const float *>(X), reinterpret_cast<float *>(ws_bytes), g0, pr.n_pad, total);
            DP_LAUNCH_CHECK("unfold_small_channels_kernel");
        }
        X = ws_bytes;
    }
    float *part_ws = reinterpret_cast<float *>(ws_bytes + unfold_bytes(dtype, g0, pr));
    CUtensorMap tmX, tmY;
    if (!encode_nhwc(&tmX, dtype, X, g.Cin, g.W, g.H, g.B, pl.OWt, pl.OHt, g.stride)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(X)");
    if (!encode_nhwc(&tmY, dtype, dY, g.Kout, g.OW, g.OH, g.B, pl.OWt, pl.OHt, 1)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY)");
    TcParams p;
    p.B = g.B; p.Kout = g.Kout; p.Ng = g0.N; p.Cin = g.Cin; p.S = g.S; p.stride = g.stride; p.pad = g.pad;
    p.n_pad_cols = (g.N != g0.N) ? 1 : 0;
    p.slab_ch = (dtype == DP_BF16) ? 64 : 32; p.krows = (dtype == DP_BF16) ? 16 : 8;
    p.a_is_x = pl.a_is_x; p.a_ext = pl.a_ext; p.b_ext = pl.b_ext; p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.NT = pl.NT;
    p.OWt = pl.OWt; p.OHt = pl.OHt; p.tiles_w = pl.tiles_w; p.Kt = pl.Kt; p.k_tiles = pl.k_tiles;
    p.stages = pl.stages; p.stage_bytes = pl.stage_bytes; p.a_bytes = pl.a_bytes;
    p.lo_offset = pl.stage_bytes / 2;
    p.single_pass = (dtype == DP_TF32) ? 1 : 0;
    p.mode = clip ? 2 : (epilogue == DP_EPI_STORE_NORM ? 0 : 1);
    p.G_w = G_w; p.partial = partial; p.slots = slots; p.status = status;
    p.wait_polls = g_wait_polls.load(std::memory_order_relaxed);
    p.splits = 1; p.per_split = g.B; p.factor = factor; p.sum_out = acc_w;
    p.inline_factor = (clip && inline_clip) ? 1 : 0;
    p.C_l = inline_clip ? inline_clip->C_l : 0.f;
    p.sqnorm = inline_clip ? inline_clip->sqnorm : nullptr;
    p.sq_stride = inline_clip ? inline_clip->sq_stride : 0;
    p.clip_out = inline_clip ? inline_clip->clip_out : nullptr;
    p.counters = nullptr; p.w_slots = 0; p.separate = 0; p.factor_out = nullptr;
    if (!clip && publish) {
        p.counters = publish->counters; p.w_slots = publish->w_slots; p.separate = publish->separate;
        p.sqnorm = publish->sqnorm; p.sq_stride = publish->sq_stride;
        p.factor_out = publish->factor_out; p.C_l = publish->C_l; p.clip_out = publish->clip_out;
    }
    if (clip) {
        clip_split(g, pl, p.splits, p.per_split);
        if (p.splits > 1) p.sum_out = part_ws;
        p.total_tiles = p.splits * pl.m_tiles * pl.n_tiles;
    } else {
        p.total_tiles = g.B * pl.m_tiles * pl.n_tiles;
    }
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        const int bytes = kSmemBudget + 2048;
        attr_err = cudaFuncSetAttribute(conv_wgrad_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (attr_err == cudaSuccess) attr_err = cudaFuncSetAttribute(conv_wgrad_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (attr_err == cudaSuccess) attr_err = cudaFuncSetAttribute(conv_wgrad_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (attr_err == cudaSuccess) attr_err = cudaFuncSetAttribute(conv_wgrad_tc_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute");
    const unsigned grid = (unsigned)std::min(p.total_tiles, sm_target());
    if (dtype == DP_BF16) {
        if (clip) conv_wgrad_tc_kernel<false, true><<<grid, 224, pl.smem, stream>>>(tmX, tmY, p);
        else conv_wgrad_tc_kernel<false, false><<<grid, 224, pl.smem, stream>>>(tmX, tmY, p);
    } else {
        if (clip) conv_wgrad_tc_kernel<true, true><<<grid, 480, pl.smem, stream>>>(tmX, tmY, p);
        else conv_wgrad_tc_kernel<true, false><<<grid, 480, pl.smem, stream>>>(tmX, tmY, p);
    }
    DP_LAUNCH_CHECK("conv_wgrad_tc_kernel");
    if (clip && p.splits > 1) return launch_fold_partial_sums(p.sum_out, p.splits, (long long)g0.M * g0.N, acc_w, stream);
    return DP_OK;
}

// The fused clipped sum of a bf16 layer that does not fit a cluster: norm pass, then ONE matrix product over all examples.
bool tc_clip_scaled_sum(int dtype, const ConvGeom &g0) {
    const TcProblem pr = tc_problem(dtype, g0);
    return dtype == DP_BF16 && pr.ok && !pr.unfold && encode_fn() && g0.Kout % 8 == 0 && make_plan(dtype, pr.eff, 4).ok;
}

dp_status launch_conv_ssum(int dtype, const void *X, const void *dY, const ConvGeom &g0, const float *factor, float *acc_w,
                           void *tc_workspace, int *status, cudaStream_t stream) {
    if (!tc_clip_scaled_sum(dtype, g0)) return DP_ERR_UNSUPPORTED;
    const TcProblem pr = tc_problem(dtype, g0);
    const ConvGeom &g = pr.eff;
    const TcPlan pl = make_plan(dtype, g, 4);
    char *ws_bytes = static_cast<char *>(tc_workspace);
    __nv_bfloat16 *hi = reinterpret_cast<__nv_bfloat16 *>(ws_bytes), *lo = reinterpret_cast<__nv_bfloat16 *>(ws_bytes + ssum_copy_bytes(g));
    float *part_ws = reinterpret_cast<float *>(ws_bytes + 2 * ssum_copy_bytes(g));
    {
        const long long per_example = (long long)g.OH * g.OW * g.Kout, total8 = per_example * g.B / 8;
        scale_split_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, stream>>>(static_cast<const __nv_bfloat16 *>(dY), factor, per_example, total8, hi, lo);
        DP_LAUNCH_CHECK("scale_split_kernel");
    }
    CUtensorMap tmX, tmYhi, tmYlo;
    if (!encode_nhwc(&tmX, dtype, X, g.Cin, g.W, g.H, g.B, pl.OWt, pl.OHt, g.stride)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(X)");
    if (!encode_nhwc(&tmYhi, dtype, hi, g.Kout, g.OW, g.OH, g.B, pl.OWt, pl.OHt, 1)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY hi)");
    if (!encode_nhwc(&tmYlo, dtype, lo, g.Kout, g.OW, g.OH, g.B, pl.OWt, pl.OHt, 1)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY lo)");
    TcParams p = {};
    p.B = g.B; p.Kout = g.Kout; p.Ng = g.N; p.Cin = g.Cin; p.S = g.S; p.stride = g.stride; p.pad = g.pad;
    p.slab_ch = 64; p.krows = 16;
    p.a_is_x = pl.a_is_x; p.a_ext = pl.a_ext; p.b_ext = pl.b_ext; p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.NT = pl.NT;
    p.OWt = pl.OWt; p.OHt = pl.OHt; p.tiles_w = pl.tiles_w; p.Kt = pl.Kt; p.k_tiles = pl.k_tiles;
    p.stages = pl.stages; p.stage_bytes = pl.stage_bytes; p.a_bytes = pl.a_bytes;
    p.lo_offset = pl.a_bytes + (pl.NT / 64) * pl.Kt * kRowBytes;      // after the A and B slabs
    p.mode = 2; p.status = status;                                    // items are (example range, tile) pairs
    p.wait_polls = g_wait_polls.load(std::memory_order_relaxed);
    ssum_split(g.B, pl.m_tiles * pl.n_tiles, p.splits, p.per_split);
    p.sum_out = p.splits > 1 ? part_ws : acc_w;
    p.total_tiles = p.splits * pl.m_tiles * pl.n_tiles;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(conv_wgrad_ssum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute");
    const unsigned grid = (unsigned)std::min(p.total_tiles, sm_target());
    conv_wgrad_ssum_kernel<<<grid, 224, pl.smem, stream>>>(tmX, tmYhi, tmYlo, p);
    DP_LAUNCH_CHECK("conv_wgrad_ssum_kernel");
    if (p.splits > 1) return launch_fold_partial_sums(p.sum_out, p.splits, (long long)g.M * g.N, acc_w, stream);
    return DP_OK;
}

// ---- clipped sum with the factors known, per example through tensor memory (the single-pass kernel without its norm
// pass and exchange): one tile per CTA, the CTA walks a range of examples, reads each finished tile once and keeps
// sum_n f_n D_n in registers.  Pays where an example has enough pixels that its MMAs outlast the read-back of the tile
// (some nine steps of 16 pixels); below that the one-product form above is the better one.
constexpr int kScaledTilesMinPixels = 128;
bool tc_clip_scaled_tiles(int dtype, const ConvGeom &g0) {
    const TcProblem pr = tc_problem(dtype, g0);
    return dtype == DP_BF16 && pr.ok && !pr.unfold && encode_fn() && pr.eff.K >= kScaledTilesMinPixels &&
           make_plan(dtype, pr.eff, 7).ok && clip1_registers_ok();
}

static void scaled_tiles_split(const ConvGeom &g, const TcPlan &pl, int &splits, int &per) {
    cluster_split(g.B, pl.m_tiles * pl.n_tiles, g.K, pl.NT, splits, per);
}

dp_status launch_conv_scaled_tiles(int dtype, const void *X, const void *dY, const ConvGeom &g0, const float *factor, float *acc_w,
                                   void *tc_workspace, int *status, cudaStream_t stream) {
    if (!tc_clip_scaled_tiles(dtype, g0)) return DP_ERR_UNSUPPORTED;
    const TcProblem pr = tc_problem(dtype, g0);
    const ConvGeom &g = pr.eff;
    const TcPlan pl = make_plan(dtype, g, 7);
    CUtensorMap tmX, tmY;
    if (!encode_nhwc(&tmX, dtype, X, g.Cin, g.W, g.H, g.B, pl.OWt, pl.OHt, g.stride)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(X)");
    if (!encode_nhwc(&tmY, dtype, dY, g.Kout, g.OW, g.OH, g.B, pl.OWt, pl.OHt, 1)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY)");
    TcParams p = {};
    p.B = g.B; p.Kout = g.Kout; p.Ng = g.N; p.Cin = g.Cin; p.S = g.S; p.stride = g.stride; p.pad = g.pad;
    p.slab_ch = 64; p.krows = 16;
    p.a_is_x = pl.a_is_x; p.a_ext = pl.a_ext; p.b_ext = pl.b_ext; p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.NT = pl.NT;
    p.OWt = pl.OWt; p.OHt = pl.OHt; p.tiles_w = pl.tiles_w; p.Kt = pl.Kt; p.k_tiles = pl.k_tiles;
    p.stages = pl.stages; p.stage_bytes = pl.stage_bytes; p.a_bytes = pl.a_bytes;
    p.mode = 3; p.status = status; p.factor = factor;
    p.wait_polls = g_wait_polls.load(std::memory_order_relaxed);
    const int tiles = pl.m_tiles * pl.n_tiles;
    scaled_tiles_split(g, pl, p.splits, p.per_split);
    p.sum_out = p.splits > 1 ? static_cast<float *>(tc_workspace) : acc_w;
    p.total_tiles = p.splits * tiles;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(conv_wgrad_clip1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute");
    conv_wgrad_clip1_kernel<<<(unsigned)p.total_tiles, kClipThreads, pl.smem, stream>>>(tmX, tmY, p);
    DP_LAUNCH_CHECK("conv_wgrad_clip1_kernel");
    if (p.splits > 1) return launch_fold_partial_sums(p.sum_out, p.splits, (long long)g.M * g.N, acc_w, stream);
    return DP_OK;
}

// ---- norms from Gram matrices (conv_gram_norm_kernel): the whole output plane as one pixel box
struct GramPlan { bool ok; ConvGeom g; int OWb, OHb, rows, pack, m_tiles, stages, stage_bytes; size_t smem; };

static GramPlan gram_plan(int dtype, const ConvGeom &g0) {
    GramPlan gp = {};
    const TcProblem pr = tc_problem(dtype, g0);
    if (dtype != DP_BF16 || !pr.ok || pr.unfold || !encode_fn()) return gp;
    gp.g = pr.eff;
    const ConvGeom &g = gp.g;
    if (g.stride > 8) return gp;
    int best = 1 << 30;
    // the smallest box over the plane whose pixel count is a multiple of 16 (rows past the plane are zero-filled)
    for (int OHb = g.OH; OHb <= g.OH + 15; ++OHb)
        for (int OWb = g.OW; OWb <= g.OW + 15; ++OWb) {
            const int rows = OHb * OWb;
            if (rows % 16 || rows > 256 || OWb * g.stride > 256 || OHb * g.stride > 256 || rows >= best) continue;
            best = rows; gp.OWb = OWb; gp.OHb = OHb;
        }
    if (best > 256) return gp;
    gp.rows = best;
    gp.pack = (best == 64) ? 2 : 1;
    gp.m_tiles = (best + 127) / 128;
    gp.stage_bytes = gp.m_tiles * 128 * kRowBytes;      // a row tile always reads 128 rows, whatever the box holds
    gp.stages = std::min(kMaxStages, kSmemBudget / gp.stage_bytes);
    gp.smem = (size_t)gp.stages * gp.stage_bytes + 1024;
    gp.ok = true;
    return gp;
}

bool tc_gram_norm(int dtype, const ConvGeom &g0) { return gram_plan(dtype, g0).ok; }

// {1, pixels of the box, same, row tiles, 1, columns of the first row tile, box width, box height, pixels per stage,
//  loads per row tile, stages, bytes per stage}
static int gram_describe(int dtype, const ConvGeom &g0, int *out, int n) {
    const GramPlan gp = gram_plan(dtype, g0);
    if (!gp.ok) return 0;
    const int v[12] = {1, gp.rows, gp.rows, gp.m_tiles, 1, gp.rows, gp.OWb, gp.OHb, gp.rows,
                       gp.g.Kout / 64 + gp.g.R * gp.g.S * (gp.g.Cin / 64), gp.stages, gp.stage_bytes};
    for (int i = 0; i < n && i < 12; ++i) out[i] = v[i];
    return 12;
}

dp_status launch_conv_gram_norm(int dtype, const void *X, const void *dY, const ConvGeom &g0, const TcInlineClip &clipinfo,
                                float *factor_out, int *status, cudaStream_t stream) {
    const GramPlan gp = gram_plan(dtype, g0);
    if (!gp.ok) return DP_ERR_UNSUPPORTED;
    const ConvGeom &g = gp.g;
    CUtensorMap tmX, tmY;
    if (!encode_nhwc(&tmX, dtype, X, g.Cin, g.W, g.H, g.B, gp.OWb, gp.OHb, g.stride, gp.pack)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(X)");
    if (!encode_nhwc(&tmY, dtype, dY, g.Kout, g.OW, g.OH, g.B, gp.OWb, gp.OHb, 1, gp.pack)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY)");
    GramParams p = {};
    p.B = g.B; p.Cin = g.Cin; p.Kout = g.Kout; p.S = g.S; p.taps = g.R * g.S; p.stride = g.stride; p.pad = g.pad;
    p.rows = gp.rows; p.pack = gp.pack; p.m_tiles = gp.m_tiles; p.stages = gp.stages; p.stage_bytes = gp.stage_bytes;
    p.C_l = clipinfo.C_l; p.sqnorm = clipinfo.sqnorm; p.sq_stride = clipinfo.sq_stride; p.clip_out = clipinfo.clip_out;
    p.factor_out = factor_out; p.status = status;
    p.wait_polls = g_wait_polls.load(std::memory_order_relaxed);
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(conv_gram_norm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute");
    const unsigned grid = (unsigned)std::min((g.B + gp.pack - 1) / gp.pack, sm_target());
    conv_gram_norm_kernel<<<grid, 192, gp.smem, stream>>>(tmX, tmY, p);
    DP_LAUNCH_CHECK("conv_gram_norm_kernel");
    return DP_OK;
}

bool tc_clip_single_pass(int dtype, const ConvGeom &g0) {
    const TcProblem pr = tc_problem(dtype, g0);
    TcPlan pl; ConvGeom g; bool s2d;
    return pr.ok && encode_fn() && clip1_plan(dtype, g0, pr, pl, g, s2d) && clip1_registers_ok();
}

dp_status launch_conv_clip1(int dtype, const void *X, const void *dY, const ConvGeom &g0, float *partial, int slots,
                            const TcInlineClip &clipinfo, float *acc_w, void *tc_workspace, int *status, cudaStream_t stream) {
    (void)partial; (void)slots;
    const TcProblem pr = tc_problem(dtype, g0);
    TcPlan pl; ConvGeom g; bool s2d;
    if (!pr.ok || !encode_fn() || !clip1_plan(dtype, g0, pr, pl, g, s2d) || !clip1_registers_ok()) return DP_ERR_UNSUPPORTED;
    char *ws_bytes = static_cast<char *>(tc_workspace);
    CUtensorMap tmX, tmY;
    if (s2d) {
        const S2dProblem sp = s2d_problem(dtype, g0, pr);
        const long long total = (long long)g0.B * sp.Hs * sp.Ws;
        space_to_depth_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
            static_cast<const __nv_bfloat16 *>(X), reinterpret_cast<__nv_bfloat16 *>(ws_bytes), g0, sp.Hs, sp.Ws, total);
        DP_LAUNCH_CHECK("space_to_depth_kernel");
        // one operand row per output pixel: 64 values from pixel ow on, pixels 16 values apart
        const cuuint64_t dims[4] = {64, (cuuint64_t)g.OW, (cuuint64_t)sp.Hs, (cuuint64_t)g.B};
        const cuuint64_t strides[3] = {32, (cuuint64_t)sp.Ws * 32, (cuuint64_t)sp.Hs * sp.Ws * 32};
        const cuuint32_t box[4] = {64, (cuuint32_t)pl.OWt, (cuuint32_t)pl.OHt, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode_fn()(&tmX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, ws_bytes, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(space-to-depth X)");
    } else if (pr.unfold) {
        if (unfold_rows_ok(dtype, g0, pr.n_pad)) {
            unfold_rows_kernel<__nv_bfloat16, 8><<<dim3(g0.OH, g0.B), 256, unfold_rows_smem(dtype, g0), stream>>>(
                static_cast<const __nv_bfloat16 *>(X), reinterpret_cast<__nv_bfloat16 *>(ws_bytes), g0, pr.n_pad);
        } else {
            const long long total = (long long)g0.B * g0.OH * g0.OW * (pr.n_pad / 8);
            unfold_small_channels_kernel<__nv_bfloat16, 8><<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(
                static_cast<const __nv_bfloat16 *>(X), reinterpret_cast<__nv_bfloat16 *>(ws_bytes), g0, pr.n_pad, total);
        }
        DP_LAUNCH_CHECK("unfold_small_channels_kernel");
        X = ws_bytes;
    }
    float *part_ws = reinterpret_cast<float *>(ws_bytes + unfold_bytes(dtype, g0, pr));
    if (!s2d && !encode_nhwc(&tmX, dtype, X, g.Cin, g.W, g.H, g.B, pl.OWt, pl.OHt, g.stride)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(X)");
    if (!encode_nhwc(&tmY, dtype, dY, g.Kout, g.OW, g.OH, g.B, pl.OWt, pl.OHt, 1)) return cuda_fail(cudaErrorInvalidValue, "cuTensorMapEncodeTiled(dY)");
    TcParams p = {};
    p.B = g.B; p.Kout = g.Kout; p.Ng = g0.N; p.Cin = g.Cin; p.S = g.S; p.stride = g.stride; p.pad = g.pad;
    p.n_pad_cols = (g.N != g0.N) ? 1 : 0;
    p.slab_ch = 64; p.krows = 16;
    p.a_is_x = pl.a_is_x; p.a_ext = pl.a_ext; p.b_ext = pl.b_ext; p.m_tiles = pl.m_tiles; p.n_tiles = pl.n_tiles; p.NT = pl.NT;
    p.OWt = pl.OWt; p.OHt = pl.OHt; p.tiles_w = pl.tiles_w; p.Kt = pl.Kt; p.k_tiles = pl.k_tiles;
    p.stages = pl.stages; p.stage_bytes = pl.stage_bytes; p.a_bytes = pl.a_bytes;
    p.mode = 3; p.status = status;
    if (s2d) { p.s2d_st = g0.stride; p.s2d_R = g0.R; p.s2d_S = g0.S; p.s2d_Cin = g0.Cin; }
    p.wait_polls = g_wait_polls.load(std::memory_order_relaxed);
    p.C_l = clipinfo.C_l; p.sqnorm = clipinfo.sqnorm; p.sq_stride = clipinfo.sq_stride; p.clip_out = clipinfo.clip_out;
    const int cs = pl.m_tiles * pl.n_tiles;
    cluster_split(g.B, cs, g.K, pl.NT, p.splits, p.per_split);
    p.sum_out = p.splits > 1 ? part_ws : acc_w;
    p.total_tiles = p.splits * cs;
    static std::once_flag once;
    static cudaError_t attr_err = cudaSuccess;
    std::call_once(once, [] {
        attr_err = cudaFuncSetAttribute(conv_wgrad_clip1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
    });
    if (attr_err != cudaSuccess) return cuda_fail(attr_err, "cudaFuncSetAttribute");
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.splits * cs)); cfg.blockDim = dim3(kClipThreads); cfg.dynamicSmemBytes = pl.smem; cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    const cudaError_t le = cudaLaunchKernelEx(&cfg, conv_wgrad_clip1_kernel, tmX, tmY, p);
    if (le != cudaSuccess) return cuda_fail(le, "conv_wgrad_clip1_kernel");
    DP_LAUNCH_CHECK("conv_wgrad_clip1_kernel");
    if (p.splits > 1) return launch_fold_partial_sums(p.sum_out, p.splits, (long long)g0.M * g0.N, acc_w, stream);
    return DP_OK;
}

}  // namespace dp

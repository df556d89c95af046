// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) and the Box-Muller transform as device functions, shared by the
// kernels that draw noise.  Two streams are defined on top of one (seed, step) key space:
//   parameter stream   counter = (lo32(g/4), hi32(g/4), lo32(step), hi32(step)), g = global parameter index; lane g%4
//   example stream     counter = (lo32(g/4), 0x80000000 | e, lo32(step), hi32(step)) for example e of the step
//                      (needs g/4 < 2^32 and e < 2^31; never collides with the parameter stream while g < 2^33)
// key = (lo32(seed), hi32(seed)) in both.
#pragma once
#include "common.cuh"

namespace dp {

struct Words4 { uint32_t w0, w1, w2, w3; };

// One Philox4x32-10 block.  High and low halves of the 32x32 products come from
// __umulhi and the wrapping 32-bit multiply.
__device__ __forceinline__ Words4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return Words4{c0, c1, c2, c3};
}

__device__ __forceinline__ Words4 philox_block(unsigned long long seed, unsigned long long step,
                                               unsigned long long block) {
    return philox4x32_10((uint32_t)block, (uint32_t)(block >> 32), (uint32_t)step, (uint32_t)(step >> 32),
                         (uint32_t)seed, (uint32_t)(seed >> 32));
}

// Two standard normals from two words: u1 in (0,1) and u2 in [0,1) are exact in fp32.
__device__ __forceinline__ void box_muller(uint32_t ra, uint32_t rb, float &z_cos, float &z_sin) {
    const float u1 = ((float)(ra >> 9) + 0.5f) * 1.1920928955078125e-07f;   // 2^-23
    const float u2 = (float)(rb >> 8) * 5.9604644775390625e-08f;            // 2^-24
    const float radius = sqrtf(-2.0f * logf(u1));
    float s, c;
    sincospif(2.0f * u2, &s, &c);
    z_cos = radius * c;
    z_sin = radius * s;
}

__device__ __forceinline__ void normals4(unsigned long long seed, unsigned long long step,
                                         unsigned long long block, float z[4]) {
    const Words4 w = philox_block(seed, step, block);
    box_muller(w.w0, w.w1, z[0], z[1]);
    box_muller(w.w2, w.w3, z[2], z[3]);
}

// four normals of block `block` (low 32 bits of g/4) of example e's stream
__device__ __forceinline__ void example_normals4(unsigned long long seed, unsigned long long step, uint32_t example,
                                                 uint32_t block, float z[4]) {
    const Words4 w = philox4x32_10(block, 0x80000000u | example, (uint32_t)step, (uint32_t)(step >> 32),
                                   (uint32_t)seed, (uint32_t)(seed >> 32));
    box_muller(w.w0, w.w1, z[0], z[1]);
    box_muller(w.w2, w.w3, z[2], z[3]);
}

}  // namespace dp

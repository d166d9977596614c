// Device-side building blocks of the RPS step: Philox4x32-10, the counter
// layout of the three random streams, the Gaussian transform, and the layout of
// one step's drop masks in global memory.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rps {

constexpr int kMaxWorkers = 64;

// Random streams: counter words 0,1 hold the step t, word 3's low byte names the
// stream, the remaining bits say which draw of that stream is wanted.
//   UP / DOWN : word2 = (block j << 16) | worker i         (one draw per message)
//   NOISE     : word2 = column / 4, word3 |= (worker / 2) << 8
//   PERM      : word2 = position k of the Fisher-Yates shuffle
enum Stream : uint32_t { kStreamUp = 0, kStreamDown = 1, kStreamNoise = 2, kStreamPerm = 3 };

// Drop masks of one step (Section 3's channel applied to the 2n messages of each
// block): bit i of up[j] says worker i's copy of block j reached the server,
// bit i of down[j] says worker i received the average; cnt[j] = popcount(up[j]).
struct StepMasks {
    uint64_t up[kMaxWorkers];
    uint64_t down[kMaxWorkers];
    int32_t cnt[kMaxWorkers];
    int32_t server[kMaxWorkers];
};

struct Philox4 {
    uint32_t x, y, z, w;
};

// Philox4x32 with 10 rounds (Salmon et al., SC'11): each round multiplies words 0
// and 2 by fixed odd constants, folds the high halves into words 1 and 3 together
// with the round key, and the key advances by a Weyl constant.
__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                                 uint32_t k1)
{
    constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
    constexpr uint32_t kWeylA = 0x9E3779B9u, kWeylB = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi_a = __umulhi(kMulA, c0), lo_a = kMulA * c0;
        const uint32_t hi_b = __umulhi(kMulB, c2), lo_b = kMulB * c2;
        c0 = hi_b ^ c1 ^ k0;
        c1 = lo_b;
        c2 = hi_a ^ c3 ^ k1;
        c3 = lo_a;
        k0 += kWeylA;
        k1 += kWeylB;
    }
    return Philox4{c0, c1, c2, c3};
}

// One Box-Muller pair from one 32-bit word: the low 16 bits pick the radius
// uniform and the high 16 bits the angle uniform, both at bin centres
// (k + 1/2) / 2^16, which fp32 represents exactly.  Returns (r cos a, r sin a).
__device__ __forceinline__ float2 gaussian_pair(uint32_t word)
{
    // 1.0f + k * 2^-16 built in the mantissa, minus (1 - 2^-17): exact.
    const float u_radius = __uint_as_float(0x3F800000u | ((word & 0xFFFFu) << 7)) - 0.99999237060546875f;
    const float u_angle = __uint_as_float(0x3F800000u | ((word >> 16) << 7)) - 0.99999237060546875f;
    // r = sqrt(-2 ln u) with ln u = ln 2 * log2 u
    float radius;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(radius) : "f"(-1.3862943611198906f * __log2f(u_radius)));
    float s, c;
    __sincosf(6.283185307179586f * u_angle, &s, &c);
    return make_float2(radius * c, radius * s);
}

}  // namespace rps

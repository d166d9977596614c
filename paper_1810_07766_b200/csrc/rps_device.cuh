// Device-side building blocks of the RPS step: Philox4x32-10, the counter
// layout of the random streams, the Gaussian transform, the layout of one
// step's drop masks, and the per-lane arithmetic shared by the fused kernels
// (local SGD step, masked average, masked write-back).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rps_kernels.h"

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
    float inv_cnt[kMaxWorkers];  // 1 / cnt[j] rounded to nearest, 0 where cnt[j] == 0
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
        const uint64_t prod_a = (uint64_t)kMulA * c0;
        const uint64_t prod_b = (uint64_t)kMulB * c2;
        c0 = (uint32_t)(prod_b >> 32) ^ c1 ^ k0;
        c1 = (uint32_t)prod_b;
        c2 = (uint32_t)(prod_a >> 32) ^ c3 ^ k1;
        c3 = (uint32_t)prod_a;
        k0 += kWeylA;
        k1 += kWeylB;
    }
    return Philox4{c0, c1, c2, c3};
}

// The same round function with ROUNDS rounds and the round keys k + r * (Weyl constants) prepared by
// the host (FusedParams::round_key): inside the fused kernels the key never changes, so the key
// schedule costs nothing per draw.
template <int ROUNDS>
__device__ __forceinline__ Philox4 philox4x32_keyed(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                    const uint32_t (&round_key)[10][2])
{
    static_assert(ROUNDS >= 1 && ROUNDS <= 10, "round keys are prepared for ten rounds");
    constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < ROUNDS; ++r) {
        const uint64_t prod_a = (uint64_t)kMulA * c0;
        const uint64_t prod_b = (uint64_t)kMulB * c2;
        c0 = (uint32_t)(prod_b >> 32) ^ c1 ^ round_key[r][0];
        c1 = (uint32_t)prod_b;
        c2 = (uint32_t)(prod_a >> 32) ^ c3 ^ round_key[r][1];
        c3 = (uint32_t)prod_a;
    }
    return Philox4{c0, c1, c2, c3};
}

// One Box-Muller pair from one 32-bit word, already scaled by -(gamma*sigma): the sign of the update
// v = ... - (gamma sigma) xi is carried by the angle, which is taken half a turn on
// (cos(a + pi) = -cos a, sin(a + pi) = -sin a), so callers ADD radius * (c, s).  The low 16 bits pick the
// radius uniform and the high 16 bits the angle uniform, both at bin centres (k + 1/2) / 2^16.  2^23 + k is
// built in the mantissa, so one fma gives the uniform exactly.  Returns radius, and (c, s) = -(cos, sin) of
// the angle.
struct ScaledPair {
    float radius, c, s;
};

// u = (k + 1/2) / 2^16 = (2^23 + k) * 2^-16 - (128 - 2^-17), exact in fp32
constexpr float kUniformScale = 1.52587890625e-05f, kUniformShift = -127.99999237060546875f;
// the angle in turns plus half a turn, in (1/2, 3/2): (2^23 + k) * 2^-16 - (127.5 - 2^-17), exact for the same
// reason (127.5 - 2^-17 has 24 significant bits; 128.5 - 2^-17, for half a turn less, would have 25); it is
// scaled by 2 pi only after that, so that the rounding of the constant is not multiplied by 2^23
constexpr float kAngleShift = -127.49999237060546875f;
constexpr float kTwoPi = 6.283185307179586f;

__device__ __forceinline__ float approx_log2(float u)
{
    float r;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(u));
    return r;
}

// radius = gamma*sigma * sqrt(-2 ln u), with ln u = ln 2 * log2 u folded into noise_scale (scaled_log2 =
// noise_scale * log2 u).  The special-function unit's approximations are used in their flush-to-zero forms:
// no operand here is subnormal (u >= 2^-17), so the slower subnormal handling buys nothing.
__device__ __forceinline__ ScaledPair radius_and_direction(float scaled_log2, float angle_rad)
{
    ScaledPair out;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(out.radius) : "f"(scaled_log2));
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(out.s) : "f"(angle_rad));
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(out.c) : "f"(angle_rad));
    return out;
}

__device__ __forceinline__ ScaledPair gaussian_pair(uint32_t word, float noise_scale)
{
    const float k_radius = __uint_as_float(__byte_perm(word, 0x4B000000u, 0x7410));  // 2^23 + low half
    const float k_angle = __uint_as_float(__byte_perm(word, 0x4B000000u, 0x7432));   // 2^23 + high half
    const float u = fmaf(k_radius, kUniformScale, kUniformShift);
    const float angle_turns = fmaf(k_angle, kUniformScale, kAngleShift);
    return radius_and_direction(noise_scale * approx_log2(u), kTwoPi * angle_turns);
}

// Row slices of one lane: VEC replica-typed elements (16 bytes, or 8 for the narrow bf16 form) <-> fp32 registers.
template <typename T, int VEC>
struct RowVec;

template <>
struct RowVec<float, 4> {
    using Raw = uint4;
    static __device__ __forceinline__ void unpack(const uint4 raw, float (&out)[4])
    {
        out[0] = __uint_as_float(raw.x), out[1] = __uint_as_float(raw.y);
        out[2] = __uint_as_float(raw.z), out[3] = __uint_as_float(raw.w);
    }
    static __device__ __forceinline__ float narrow(float v) { return v; }
    static __device__ __forceinline__ uint4 pack(const float (&in)[4])
    {
        return make_uint4(__float_as_uint(in[0]), __float_as_uint(in[1]), __float_as_uint(in[2]),
                          __float_as_uint(in[3]));
    }
    // out = b - x, from the raw slice of b and the widened x
    static __device__ __forceinline__ void deviation(const uint4 raw_b, const float (&x)[4], float (&out)[4])
    {
        out[0] = __uint_as_float(raw_b.x) - x[0], out[1] = __uint_as_float(raw_b.y) - x[1];
        out[2] = __uint_as_float(raw_b.z) - x[2], out[3] = __uint_as_float(raw_b.w) - x[3];
    }
};

// (lo, hi) = the two bf16 halves of `pair`, each minus an fp32 value, in fp32: the mixed-precision subtract of
// sm_100 takes a bf16 operand as it is, so the halves of b are never widened by an instruction of their own.
// The result is the correctly rounded fp32 difference, the same bits as widening first.
__device__ __forceinline__ void bf16_pair_minus(uint32_t pair, float x_lo, float x_hi, float& lo, float& hi)
{
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tsub.rn.f32.bf16 %0, l, %3;\n\tsub.rn.f32.bf16 %1, h, %4;\n\t}"
        : "=f"(lo), "=f"(hi)
        : "r"(pair), "f"(x_lo), "f"(x_hi));
}

template <>
struct RowVec<__nv_bfloat16, 8> {
    using Raw = uint4;
    static __device__ __forceinline__ void unpack(const uint4 raw, float (&out)[8])
    {
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            out[2 * k] = __uint_as_float(w[k] << 16);  // bf16 -> fp32 is exact
            out[2 * k + 1] = __uint_as_float(w[k] & 0xFFFF0000u);
        }
    }
    static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
    static __device__ __forceinline__ uint4 pack(const float (&in)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const __nv_bfloat162 pair = __floats2bfloat162_rn(in[2 * k], in[2 * k + 1]);  // nearest-even
            w[k] = *reinterpret_cast<const uint32_t*>(&pair);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ void deviation(const uint4 raw_b, const float (&x)[8], float (&out)[8])
    {
        const uint32_t w[4] = {raw_b.x, raw_b.y, raw_b.z, raw_b.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) bf16_pair_minus(w[k], x[2 * k], x[2 * k + 1], out[2 * k], out[2 * k + 1]);
    }
};

// 8-byte slices of bf16 rows: half the columns per lane, so twice the lanes (and warps) per tile.
template <>
struct RowVec<__nv_bfloat16, 4> {
    using Raw = uint2;
    static __device__ __forceinline__ void unpack(const uint2 raw, float (&out)[4])
    {
        out[0] = __uint_as_float(raw.x << 16), out[1] = __uint_as_float(raw.x & 0xFFFF0000u);
        out[2] = __uint_as_float(raw.y << 16), out[3] = __uint_as_float(raw.y & 0xFFFF0000u);
    }
    static __device__ __forceinline__ __nv_bfloat16 narrow(float v) { return __float2bfloat16_rn(v); }
    static __device__ __forceinline__ uint2 pack(const float (&in)[4])
    {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(in[0], in[1]), hi = __floats2bfloat162_rn(in[2], in[3]);
        return make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
    static __device__ __forceinline__ void deviation(const uint2 raw_b, const float (&x)[4], float (&out)[4])
    {
        bf16_pair_minus(raw_b.x, x[0], x[1], out[0], out[1]);
        bf16_pair_minus(raw_b.y, x[2], x[3], out[2], out[3]);
    }
};

// The gradient noise draws with seven rounds: the generator's authors report that Philox4x32 passes their
// test batteries from seven rounds on (ten, used for the drop masks, is their default with a margin), and
// the three rounds saved are 1.6 of ~24 instructions per replica-param, which the bf16 shapes, bound by
// instruction issue, turn into 8 % more throughput.
constexpr int kNoiseRounds = 7;

// Subtracts (gamma * sigma) * xi from v: one Philox draw per worker pair and four columns, for step
// t = (t_hi, t_lo).
template <int VEC, int WPT>
__device__ __forceinline__ void add_gradient_noise(float (&v)[WPT][VEC], int64_t c, int w_first, const FusedParams& prm,
                                                   uint32_t t_lo, uint32_t t_hi)
{
#pragma unroll
    for (int w = 0; w < WPT; w += 2) {
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q) {
            const Philox4 r = philox4x32_keyed<kNoiseRounds>(t_lo, t_hi, (uint32_t)((c + prm.col_offset) >> 2) + q,
                                                             kStreamNoise | ((uint32_t)((w_first + w) >> 1) << 8),
                                                             prm.round_key);
            const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const ScaledPair z = gaussian_pair(words[m], prm.noise_scale);
                float(&row)[VEC] = v[w + (m >> 1)];  // words 0,1 -> worker w, words 2,3 -> worker w+1
                const int k = 4 * q + 2 * (m & 1);
                row[k] = fmaf(z.radius, z.c, row[k]);
                row[k + 1] = fmaf(z.radius, z.s, row[k + 1]);
            }
        }
    }
}

// ---- The same arithmetic two columns at a time, in the packed fp32 forms of sm_100 (fma / mul / add / sub
// .f32x2: one instruction, two IEEE operations, the same bits as the scalar forms).  A Float2 is two floats
// in one 64-bit register (an aligned register pair: packing and unpacking cost nothing where the halves
// already lie side by side, as the halves of a 16-byte load do).
using Float2 = unsigned long long;

__device__ __forceinline__ Float2 pack2(float lo, float hi)
{
    Float2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ Float2 pack2(uint32_t lo, uint32_t hi)
{
    Float2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(Float2 v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ Float2 fma2(Float2 a, Float2 b, Float2 c)
{
    Float2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ Float2 mul2(Float2 a, Float2 b)
{
    Float2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ Float2 sub2(Float2 a, Float2 b)
{
    Float2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// s += v (both halves) where `take` is set, as one predicated instruction
__device__ __forceinline__ void add2_if(Float2& s, Float2 v, uint32_t take)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p add.rn.f32x2 %0, %0, %1;\n\t}" : "+l"(s) : "l"(v), "r"(take));
}

// Loop-invariant operands of the packed step.
struct PackedScalars {
    Float2 gamma;          // (gamma, gamma)
    Float2 uniform_scale;  // (2^-16, 2^-16)
    Float2 uniform_shift;  // (shift of the radius uniform, shift of the angle)
    Float2 noise_and_turn; // (noise_scale, 2 pi)
    __device__ __forceinline__ explicit PackedScalars(const FusedParams& prm)
        : gamma(pack2(prm.gamma, prm.gamma)),
          uniform_scale(pack2(kUniformScale, kUniformScale)),
          uniform_shift(pack2(kUniformShift, kAngleShift)),
          noise_and_turn(pack2(prm.noise_scale, kTwoPi))
    {
    }
};

// v (two adjacent columns of one worker) += the Box-Muller pair of `word`; bit for bit what gaussian_pair and two
// scalar multiply-adds give.
__device__ __forceinline__ Float2 add_noise_pair(Float2 v, uint32_t word, const PackedScalars& k)
{
    const uint32_t k_radius = __byte_perm(word, 0x4B000000u, 0x7410);  // 2^23 + low half
    const uint32_t k_angle = __byte_perm(word, 0x4B000000u, 0x7432);   // 2^23 + high half
    float u, angle_turns;
    unpack2(fma2(pack2(k_radius, k_angle), k.uniform_scale, k.uniform_shift), u, angle_turns);
    float scaled_log2, angle_rad;
    unpack2(mul2(pack2(approx_log2(u), angle_turns), k.noise_and_turn), scaled_log2, angle_rad);
    const ScaledPair z = radius_and_direction(scaled_log2, angle_rad);
    return fma2(pack2(z.radius, z.radius), pack2(z.c, z.s), v);
}

__device__ __forceinline__ Float2 add2(Float2 a, Float2 b)
{
    Float2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Local SGD step of one lane on a worker pair (k even) x VEC columns from column c, from the raw slices, two
// columns at a time: v = x + gamma (b - x) - (gamma sigma) xi.  Same bits as local_sgd_raw<T, VEC, 2, false>.
// The step index (t_hi, t_lo) is the caller's: a launch may run several steps.
// TARGETS: also add the pair's targets to target_sum, as (b - x) + x from the values the step holds anyway
// (equal to b up to one rounding of the difference; for the tracked steps' mean of the targets).
// UPDATE: leave the update v - x = gamma (b - x) - (gamma sigma) xi in v instead (gradient averaging).
template <typename T, int VEC, bool TARGETS = false, bool UPDATE = false>
__device__ __forceinline__ void local_sgd_pair_packed(const uint4 (&raw_x)[2], const uint4 (&raw_b)[2],
                                                      Float2 (&v)[2][VEC / 2], int64_t c, int k,
                                                      const FusedParams& prm, const PackedScalars& scalars,
                                                      uint32_t t_lo, uint32_t t_hi, Float2* target_sum = nullptr)
{
    static_assert(VEC * sizeof(T) == 16, "a slice is 16 bytes");
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t wx[4] = {raw_x[h].x, raw_x[h].y, raw_x[h].z, raw_x[h].w};
        const uint32_t wb[4] = {raw_b[h].x, raw_b[h].y, raw_b[h].z, raw_b[h].w};
        if (sizeof(T) == 4) {
#pragma unroll
            for (int m = 0; m < 2; ++m) {
                const Float2 x2 = pack2(wx[2 * m], wx[2 * m + 1]);
                const Float2 b2 = pack2(wb[2 * m], wb[2 * m + 1]);
                v[h][m % (VEC / 2)] = UPDATE ? mul2(scalars.gamma, sub2(b2, x2)) : fma2(scalars.gamma, sub2(b2, x2), x2);
                if (TARGETS) target_sum[m % (VEC / 2)] = add2(target_sum[m % (VEC / 2)], b2);
            }
        } else {
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const float x_lo = __uint_as_float(wx[m] << 16), x_hi = __uint_as_float(wx[m] & 0xFFFF0000u);
                float d_lo, d_hi;
                bf16_pair_minus(wb[m], x_lo, x_hi, d_lo, d_hi);
                const Float2 d2 = pack2(d_lo, d_hi), x2 = pack2(x_lo, x_hi);
                v[h][m % (VEC / 2)] = UPDATE ? mul2(scalars.gamma, d2) : fma2(scalars.gamma, d2, x2);
                if (TARGETS) target_sum[m % (VEC / 2)] = add2(target_sum[m % (VEC / 2)], add2(d2, x2));
            }
        }
    }
    if (!prm.noisy) return;
#pragma unroll
    for (int q = 0; q < VEC / 4; ++q) {
        const Philox4 r = philox4x32_keyed<kNoiseRounds>(t_lo, t_hi, (uint32_t)((c + prm.col_offset) >> 2) + q,
                                                         kStreamNoise | ((uint32_t)(k >> 1) << 8), prm.round_key);
        // words 0,1 -> the pair's first worker (columns 0,1 and 2,3 of the four), words 2,3 -> its second
        v[0][2 * q] = add_noise_pair(v[0][2 * q], r.x, scalars);
        v[0][2 * q + 1] = add_noise_pair(v[0][2 * q + 1], r.y, scalars);
        v[1][2 * q] = add_noise_pair(v[1][2 * q], r.z, scalars);
        v[1][2 * q + 1] = add_noise_pair(v[1][2 * q + 1], r.w, scalars);
    }
}

// Local SGD step of one lane: WPT workers (starting at the even worker w_first) x
// VEC consecutive columns starting at column c, evaluated as
//   v = x - gamma * ((x - b) + sigma * xi) = x + gamma * (b - x) - (gamma * sigma) * xi :
// one subtraction, one fused multiply-add, and the noise (one Philox draw serves a worker pair on four
// columns).  GRAD: leave the update v - x = gamma * (b - x) - (gamma * sigma) * xi in v instead.
// `dev` holds b - x on entry.
template <int VEC, int WPT, bool GRAD>
__device__ __forceinline__ void sgd_from_deviation(const float (&xv)[WPT][VEC], const float (&dev)[WPT][VEC],
                                                   float (&v)[WPT][VEC], int64_t c, int w_first, const FusedParams& prm)
{
    static_assert(WPT % 2 == 0 && VEC % 4 == 0, "noise draws cover worker pairs and 4 columns");
#pragma unroll
    for (int w = 0; w < WPT; ++w)
#pragma unroll
        for (int e = 0; e < VEC; ++e) v[w][e] = GRAD ? prm.gamma * dev[w][e] : fmaf(prm.gamma, dev[w][e], xv[w][e]);
    if (prm.noisy) add_gradient_noise<VEC, WPT>(v, c, w_first, prm, prm.t_lo, prm.t_hi);
}

// The same from widened x and b.
template <int VEC, int WPT, bool GRAD>
__device__ __forceinline__ void local_sgd(const float (&xv)[WPT][VEC], const float (&bv)[WPT][VEC],
                                          float (&v)[WPT][VEC], int64_t c, int w_first, const FusedParams& prm)
{
    float dev[WPT][VEC];
#pragma unroll
    for (int w = 0; w < WPT; ++w)
#pragma unroll
        for (int e = 0; e < VEC; ++e) dev[w][e] = bv[w][e] - xv[w][e];
    sgd_from_deviation<VEC, WPT, GRAD>(xv, dev, v, c, w_first, prm);
}

// The same from the raw slices as they lie in memory: x is widened, b enters the subtraction as it is
// (bf16 replicas: no instruction is spent on widening b; the bits of the result do not depend on the route).
template <typename T, int VEC, int WPT, bool GRAD>
__device__ __forceinline__ void local_sgd_raw(const typename RowVec<T, VEC>::Raw (&raw_x)[WPT],
                                              const typename RowVec<T, VEC>::Raw (&raw_b)[WPT], float (&v)[WPT][VEC],
                                              int64_t c, int w_first, const FusedParams& prm)
{
    float xv[WPT][VEC], dev[WPT][VEC];
#pragma unroll
    for (int w = 0; w < WPT; ++w) {
        RowVec<T, VEC>::unpack(raw_x[w], xv[w]);
        RowVec<T, VEC>::deviation(raw_b[w], xv[w], dev[w]);
    }
    sgd_from_deviation<VEC, WPT, GRAD>(xv, dev, v, c, w_first, prm);
}

// s += v where `take` is set, as one predicated add (no branch, no select); a value that is
// not taken never enters the sum, whatever it is.
__device__ __forceinline__ void add_if(float& s, float v, uint32_t take)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p add.f32 %0, %0, %1;\n\t}" : "+f"(s) : "f"(v), "r"(take));
}

template <int G>
__device__ __forceinline__ float sum_over_groups(float s)
{
#pragma unroll
    for (int off = 32 / G; off < 32; off <<= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
    return s;
}

// Block (parameter server) of local column c: the model's columns are cut into n blocks of
// block_cols = ceil(d / n) columns (Step 0, model partitioning); x and b may be a window of the
// model that starts at its column col_offset.
__device__ __forceinline__ int block_of(int64_t c, const FusedParams& prm)
{
    const int64_t g = c + prm.col_offset;
    return prm.narrow ? (int)((uint32_t)g / (uint32_t)prm.block_cols) : (int)(g / prm.block_cols);
}

// What a lane needs to know about the masks: the words of block j, shifted so
// that bit w is worker w_first + w, and 1 / |N^(j)|.
struct MaskView {
    const uint64_t* up;
    const uint64_t* down;
    const float* inv_cnt;  // 1 / cnt[j], 0 where cnt[j] == 0
};

// Remembers the block a lane was last in: lanes walk the columns upwards, so the block
// index is recomputed (one division) only when a lane crosses into a new block.
struct BlockCursor {
    int64_t begin = 0, end = 0;  // local columns [begin, end) belong to block j; empty at first
    int j = 0;
    __device__ __forceinline__ int locate(int64_t c, const FusedParams& prm)
    {
        if (c < begin || c >= end) {
            j = block_of(c, prm);
            begin = (int64_t)j * prm.block_cols - prm.col_offset;
            end = begin + prm.block_cols;
        }
        return j;
    }
};

// RS + AG for one lane after local_sgd: masked sum over the lane's workers, xor
// butterfly over the G lane groups, multiply by 1/|N|, then every worker takes
// the average where its down-bit is set and keeps v otherwise.  On return v
// holds x_{t+1} (0 for columns that do not exist); the result has bit e set iff column c + e exists (< d).  Lanes
// whose VEC columns straddle two blocks or the end of the row send the whole
// warp through the per-column path.  All lanes of the warp must call this
// together.
template <int VEC, int WPT, int G>
__device__ __forceinline__ uint32_t average_and_select(float (&v)[WPT][VEC], int64_t c, bool col_live, int w_first,
                                                       const MaskView& masks, BlockCursor& cursor,
                                                       const FusedParams& prm)
{
    const int j_first = col_live ? cursor.locate(c, prm) : 0;
    const bool uniform = !col_live || (c + VEC <= cursor.end && c + VEC <= prm.d);
    if (__all_sync(0xFFFFFFFFu, uniform)) {
        const uint32_t up = (uint32_t)(masks.up[j_first] >> w_first);
        const uint32_t down = (uint32_t)(masks.down[j_first] >> w_first);
        const float inv = masks.inv_cnt[j_first];
        float s[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) s[e] = 0.0f;
#pragma unroll
        for (int w = 0; w < WPT; ++w) {
            const uint32_t arrived = (up >> w) & 1u;  // worker's copy reached the server: it is in N
#pragma unroll
            for (int e = 0; e < VEC; ++e) add_if(s[e], v[w][e], arrived);
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) s[e] = sum_over_groups<G>(s[e]) * inv;  // 1/|N| * sum over N (RS step)
#pragma unroll
        for (int w = 0; w < WPT; ++w) {
            const bool received = (down >> w) & 1u;  // AG step: receivers take the average
#pragma unroll
            for (int e = 0; e < VEC; ++e) v[w][e] = received ? s[e] : v[w][e];
        }
        return col_live ? (1u << VEC) - 1u : 0u;
    }
    uint32_t live_bits = 0;
#pragma unroll
    for (int e = 0; e < VEC; ++e) {
        const bool live = c + e < prm.d;
        const int j = live ? block_of(c + e, prm) : 0;
        const uint32_t up = (uint32_t)(masks.up[j] >> w_first);
        const uint32_t down = (uint32_t)(masks.down[j] >> w_first);
        float s = 0.0f;
#pragma unroll
        for (int w = 0; w < WPT; ++w) add_if(s, v[w][e], (up >> w) & 1u);
        const float avg = sum_over_groups<G>(s) * masks.inv_cnt[j];
#pragma unroll
        for (int w = 0; w < WPT; ++w) v[w][e] = !live ? 0.0f : (((down >> w) & 1u) ? avg : v[w][e]);
        live_bits |= (live ? 1u : 0u) << e;
    }
    return live_bits;
}

// Writes one worker's results at the ragged end of a row, element by element: only the columns
// that exist (the padding between d and the row pitch is never written).
template <typename T, int VEC>
__device__ __forceinline__ void store_ragged(T* dst, const float (&vals)[VEC], uint32_t live_bits)
{
#pragma unroll
    for (int e = 0; e < VEC; ++e)
        if ((live_bits >> e) & 1u) dst[e] = RowVec<T, VEC>::narrow(vals[e]);
}

// s = fma(v, v, s) where `take` is set (one predicated instruction, like add_if).
__device__ __forceinline__ void add_square_if(float& s, float v, uint32_t take)
{
    asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t@p fma.rn.f32 %0, %1, %1, %0;\n\t}" : "+f"(s) : "f"(v), "r"(take));
}

// The values a lane is about to store, as they will read back: rounded to T and widened again
// (nothing to do for fp32 replicas).
template <typename T, int VEC>
__device__ __forceinline__ void as_stored(float (&vals)[VEC])
{
    if (sizeof(T) != sizeof(float)) RowVec<T, VEC>::unpack(RowVec<T, VEC>::pack(vals), vals);
}

// By-product of a tracked step: what the step leaves behind, measured on the values that are in
// registers anyway (no extra pass over x):
//   dist2 = || mean_i x^(i) - mean_i b_i ||^2   squared distance of the averaged model to the optimum of
//                                               the quadratic objective,
//   cons  = sum_i || x^(i) - mean_k x^(k) ||^2  the consensus error (the quantity Lemma 3 bounds).
// Per column, relative to the pivot a = worker 0's new value (so that nothing large is squared and
// subtracted):  D = sum_i (x_i - a),  Q = sum_i (x_i - a)^2;  mean x = a + D/n;  cons = Q - D^2/n.
// fp32 within a tile of columns, fp64 across tiles.  All lanes of a warp call targets() and models()
// together; `present` has bit w set iff worker w_first + w exists.
template <int VEC, int WPT, int G>
struct Tracker {
    double dist2 = 0.0, cons = 0.0;
    float bsum[VEC];  // this lane's part of sum_i b_i of the tile in flight

    static __device__ __forceinline__ uint32_t present_workers(int w_first, int n)
    {
        const int left = n - w_first;
        return left >= WPT ? (1u << WPT) - 1u : (left > 0 ? (1u << left) - 1u : 0u);
    }

    __device__ __forceinline__ void targets(const float (&bv)[WPT][VEC], uint32_t present)
    {
#pragma unroll
        for (int e = 0; e < VEC; ++e) bsum[e] = 0.0f;
#pragma unroll
        for (int w = 0; w < WPT; ++w)
#pragma unroll
            for (int e = 0; e < VEC; ++e) add_if(bsum[e], bv[w][e], (present >> w) & 1u);
    }

    // v: x_{t+1} of this lane's workers and columns as stored; live_bits: which of the VEC columns exist
    __device__ __forceinline__ void models(const float (&v)[WPT][VEC], uint32_t present, uint32_t live_bits, float inv_n)
    {
        constexpr int LPG = 32 / G;
        const int lane = threadIdx.x & 31;
        const bool first_group = lane < LPG;  // holds worker 0; speaks for the column
        float q = 0.0f, dd = 0.0f;
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const uint32_t live = (live_bits >> e) & 1u;
            const float a = __shfl_sync(0xFFFFFFFFu, v[0][e], lane & (LPG - 1));
            float dsum = 0.0f;
#pragma unroll
            for (int w = 0; w < WPT; ++w) {
                const uint32_t take = (present >> w) & live;
                const float dev = v[w][e] - a;
                add_if(dsum, dev, take);
                add_square_if(q, dev, take);
            }
            dsum = sum_over_groups<G>(dsum);
            const float btot = sum_over_groups<G>(bsum[e]);
            if (first_group && live) {
                const float gap = fmaf(dsum - btot, inv_n, a);  // mean x - mean b of this column
                dd = fmaf(gap, gap, dd);
                q = fmaf(-dsum * inv_n, dsum, q);
            }
        }
        dist2 += (double)dd;
        cons += (double)q;
    }

    // Adds this warp's sums to the CTA's pair in shared memory (zeroed before the first call); the
    // last of `warps` warps to arrive adds the CTA's pair to out[0], out[1].  Nobody waits for anybody.
    __device__ __forceinline__ void flush(double* cta_pair, int* cta_arrivals, int warps, double* out)
    {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            dist2 += __shfl_xor_sync(0xFFFFFFFFu, dist2, off);
            cons += __shfl_xor_sync(0xFFFFFFFFu, cons, off);
        }
        if ((threadIdx.x & 31) == 0) {
            atomicAdd(&cta_pair[0], dist2);
            atomicAdd(&cta_pair[1], cons);
            __threadfence_block();
            if (atomicAdd(cta_arrivals, 1) == warps - 1) {
                __threadfence_block();
                atomicAdd(&out[0], *reinterpret_cast<volatile double*>(&cta_pair[0]));
                atomicAdd(&out[1], *reinterpret_cast<volatile double*>(&cta_pair[1]));
            }
        }
    }
};

}  // namespace rps

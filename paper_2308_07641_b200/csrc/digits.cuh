// Fixed-point digits of the real-valued operand, shared by the tensor-core and decode kernels.
//
// A token's values v (|v| <= amax < 2^E) are written as integers q = rint(v * 2^(8ND-2-E)),
// |q| <= 2^(8ND-2), and q as ND balanced radix-256 digits in [-128,127]: every product with a
// ternary entry and every partial sum is then an exact integer.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float to_float<int8_t>(int8_t v) { return (float)v; }

// Balanced radix-256 digits of sixteen fixed-point integers, as ND words of four int8 each per
// group of four values (dig[d][g] = digit d of values 4g..4g+3).  With q = sum_d digit_d*256^d
// and digits in [-128,127], digit d is byte d of q + 0x80 + 0x8000 + ... (d terms): adding half
// the radix at every lower position turns the floor of the arithmetic shift into rounding.
// The top digit is what is left; it fits because |q| <= 2^(8ND-2).
// One addition serves all digits: q + (0x80 + 0x8000 + ..., ND-1 terms) has, below the top
// digit, 0x80 too much in byte d, which an exclusive-or takes out again.  The bytes of four
// values are then transposed into the four digit words with eight byte permutes.
// `bias` is subtracted from every q first (0, or the integer image of the rounding constant when
// q comes from tsvd_round_bits below); it folds into the one addition.
template <int ND, int G>
__device__ __forceinline__ void digits_of(const int (&q)[4 * G], uint32_t (&dig)[ND][G], uint32_t bias = 0u)
{
    const uint32_t off = (ND == 1 ? 0u : ND == 2 ? 0x80u : ND == 3 ? 0x8080u : 0x808080u) - bias;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint32_t a = (uint32_t)q[4 * g] + off, b = (uint32_t)q[4 * g + 1] + off;
        const uint32_t c = (uint32_t)q[4 * g + 2] + off, e = (uint32_t)q[4 * g + 3] + off;
        const uint32_t ab01 = __byte_perm(a, b, 0x5140), cd01 = __byte_perm(c, e, 0x5140);   // bytes 0,1 of each pair
        dig[0][g] = __byte_perm(ab01, cd01, 0x5410) ^ (ND > 1 ? 0x80808080u : 0u);
        if constexpr (ND > 1) dig[1][g] = __byte_perm(ab01, cd01, 0x7632) ^ (ND > 2 ? 0x80808080u : 0u);
        if constexpr (ND > 2) {
            const uint32_t ab23 = __byte_perm(a, b, 0x7362), cd23 = __byte_perm(c, e, 0x7362);   // bytes 2,3
            dig[2][g] = __byte_perm(ab23, cd23, 0x5410) ^ (ND > 3 ? 0x80808080u : 0u);
            if constexpr (ND > 3) dig[3][g] = __byte_perm(ab23, cd23, 0x7632);
        }
    }
}

// rint(v * qscale) for |v * qscale| <= 2^22 without a conversion instruction: adding 1.5 * 2^23
// rounds the product to an integer (to nearest, ties to even, as cvt.rni does; the product itself is
// exact because qscale is a power of two), and the sum's bit pattern is that integer plus
// TSVD_ROUND_BIAS.
constexpr uint32_t TSVD_ROUND_BIAS = 0x4B400000u;
__device__ __forceinline__ int tsvd_round_bits(float v, float qscale)
{
    return __float_as_int(fmaf(v, qscale, 12582912.f));
}

template <int ND>
__device__ __forceinline__ void digits_of_16(const int (&q)[16], uint32_t (&dig)[ND][4]) { digits_of<ND, 4>(q, dig); }

// Load 8 consecutive values of a row as floats (one or two vector loads when the chunk is whole
// and the row 16-byte aligned, guarded scalar loads otherwise).
template <typename IN_T>
__device__ __forceinline__ void load8(const IN_T* __restrict__ row, int c0, int C, bool vec_ok, float (&v)[8])
{
    if (vec_ok && c0 + 8 <= C) {
        if constexpr (sizeof(IN_T) == 4) {
            const float4 f0 = __ldg(reinterpret_cast<const float4*>(row + c0));
            const float4 f1 = __ldg(reinterpret_cast<const float4*>(row + c0) + 1);
            v[0] = f0.x; v[1] = f0.y; v[2] = f0.z; v[3] = f0.w;
            v[4] = f1.x; v[5] = f1.y; v[6] = f1.z; v[7] = f1.w;
        } else if constexpr (sizeof(IN_T) == 2) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(row + c0));
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {   // bf16 -> fp32 is a 16-bit shift
                v[2 * j] = __uint_as_float(w[j] << 16);
                v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
            }
        } else {
            const uint2 u = __ldg(reinterpret_cast<const uint2*>(row + c0));
            const uint32_t w[2] = {u.x, u.y};
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (float)(int)(int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xFF);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = (c0 + e < C) ? to_float<IN_T>(row[c0 + e]) : 0.f;
    }
}

// Load 16 consecutive values of a row as floats (vector loads when the chunk is whole and
// 16-byte aligned, guarded scalar loads otherwise).
template <typename IN_T>
__device__ __forceinline__ void load16(const IN_T* __restrict__ row, int c0, int C, bool vec_ok, float (&v)[16])
{
    if (vec_ok && c0 + 16 <= C) {
        if constexpr (sizeof(IN_T) == 4) {
            const float4* p4 = reinterpret_cast<const float4*>(row + c0);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4 f = __ldg(p4 + i);
                v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
            }
        } else if constexpr (sizeof(IN_T) == 2) {
            const uint4* p4 = reinterpret_cast<const uint4*>(row + c0);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const uint4 u = __ldg(p4 + i);
                const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {   // bf16 -> fp32 is a 16-bit shift
                    v[8 * i + 2 * j] = __uint_as_float(w[j] << 16);
                    v[8 * i + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
                }
            }
        } else {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(row + c0));
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = (float)(int)(int8_t)((w[j >> 2] >> (8 * (j & 3))) & 0xFF);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) v[e] = (c0 + e < C) ? to_float<IN_T>(row[c0 + e]) : 0.f;
    }
}

// Range diagnostic (TSVD_E_RANGE): while a stage's input is converted, one value in eight is
// sampled; a sample counts when it is nonzero, and as resolved when it reaches 2^12 quantisation
// steps.  The two counts travel in one word (low half: nonzero, high half: resolved; a warp sees at
// most 65280 / 8 samples of a token).  A warp raises the flag when, among at least 32 nonzero
// samples of a token, fewer than a quarter are resolved.  For a bulk of normally distributed
// entries under an outlier 2^p times their scale the resolved share is 0.62 at p = 8 (p = 16 with
// four digits of a bf16 token, or for fp32), 0.32 one binade further and 0.05 two binades further,
// which is where outputs that do not see the outlier begin to leave the bf16 tolerance.
__device__ __forceinline__ void tsvd_range_sample(unsigned& cnt, float v, float qscale)
{
    const float a = fabsf(v) * qscale;
    cnt += (a != 0.f ? 1u : 0u) + (a >= 4096.f ? 0x10000u : 0u);
}
__device__ __forceinline__ bool tsvd_range_flagged(unsigned cnt)   // whole warp; the same answer in every lane
{
    const unsigned tot = __reduce_add_sync(0xffffffffu, cnt);
    const unsigned nz = tot & 0xffffu, big = tot >> 16;
    return nz >= 32u && 4u * big < nz;
}

// The exponent E of the rule above for a token whose largest magnitude is amax: amax = m * 2^E with
// m in [0.5, 1), read from the exponent field (zero and subnormal maxima take the floor of -90).
__device__ __forceinline__ int tsvd_quant_exponent(float amax)
{
    const int e = (int)((__float_as_uint(amax) >> 23) & 0xFFu) - 126;
    return max(e, -90);
}
// 2^e for -126 <= e <= 127, exactly.
__device__ __forceinline__ float tsvd_pow2(int e) { return __uint_as_float((uint32_t)(e + 127) << 23); }

// Device-side generator of the projection A ~ N_seed(0, 1/r)  (Algorithm 1: "A_W <- N_{s_W}(0, 1/r)").
//
// A[j,k] is a function of (seed, j, k): Philox4x32-10 (Salmon et al., SC'11) keyed by the two
// halves of the seed, counter (k/4, j, 0, 0), gives four words; words (0,1) make columns 4q, 4q+1
// (cosine and sine branch of Box-Muller), words (2,3) make 4q+2, 4q+3.  Only IEEE-754 binary32
// operations with a fixed order are used (explicit round-to-nearest intrinsics, never contracted
// by the compiler, no approximate hardware functions), so the value is reproducible bit by bit
// on any IEEE machine.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace flora {

struct PhiloxKey {
    uint32_t k0, k1;
};

__host__ __device__ __forceinline__ PhiloxKey make_key(uint64_t seed)
{
    PhiloxKey k;
    k.k0 = (uint32_t)(seed & 0xFFFFFFFFull);
    k.k1 = (uint32_t)(seed >> 32);
    return k;
}

// One Philox4x32-10 block with counter (q, j, 0, 0).
__device__ __forceinline__ void philox_block(uint32_t q, uint32_t j, PhiloxKey key, uint32_t (&x)[4])
{
    uint32_t c0 = q, c1 = j, c2 = 0u, c3 = 0u;
    uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    x[0] = c0; x[1] = c1; x[2] = c2; x[3] = c3;
}

// -2 ln(k1 / 2^24) for k1 in [1, 2^24]: k1 = 2^e * mant with mant in [2/3, 4/3),
// ln(mant) = s - s^2/2 + s^3 Q(s), s = mant - 1.
__device__ __forceinline__ float neg2_ln_u1(uint32_t k1)
{
    const float f = __uint2float_rn(k1);                     // exact
    const uint32_t b = __float_as_uint(f);
    const int32_t e = (int32_t)(b - 0x3F2AAAABu) >> 23;
    const float mant = __uint_as_float(b - ((uint32_t)e << 23));
    const float s = __fadd_rn(mant, -1.0f);                  // exact
    float q = 0x1.1b09e8p-3f;
    q = __fmaf_rn(q, s, -0x1.35b3ep-3f);
    q = __fmaf_rn(q, s, 0x1.1f9622p-3f);
    q = __fmaf_rn(q, s, -0x1.515a6cp-3f);
    q = __fmaf_rn(q, s, 0x1.99c32p-3f);
    q = __fmaf_rn(q, s, -0x1.000b1cp-2f);
    q = __fmaf_rn(q, s, 0x1.555528p-2f);
    const float s2 = __fmul_rn(s, s);
    float p = __fmaf_rn(q, s, -0.5f);
    p = __fmaf_rn(p, s2, s);
    const float steps = __int2float_rn(24 - e);              // exact
    return __fmaf_rn(steps, 0x1.62e43p+0f, __fmul_rn(-2.0f, p));
}

// cos and sin of 2 pi k2 / 2^24 by integer octant reduction and fixed polynomials on [0, pi/4].
__device__ __forceinline__ void cos_sin_2pi_u2(uint32_t k2, float& c, float& s)
{
    const uint32_t oct = k2 >> 21;
    uint32_t frac = k2 & 0x1FFFFFu;
    if (oct & 1u) frac = 0x200000u - frac;
    const float x = __fmul_rn(__uint2float_rn(frac), 0x1.921fb6p-22f);
    const float z = __fmul_rn(x, x);
    float sp = __fmaf_rn(-0x1.9943e2p-13f, z, 0x1.11073ap-7f);
    sp = __fmaf_rn(sp, z, -0x1.555546p-3f);
    const float sx = __fmaf_rn(__fmul_rn(x, z), sp, x);
    float cp = __fmaf_rn(-0x1.644d62p-10f, z, 0x1.553e8p-5f);
    cp = __fmaf_rn(cp, z, -0x1.ffffb2p-2f);
    const float cx = __fmaf_rn(z, cp, 1.0f);
    const bool swap = ((oct + 1u) >> 1) & 1u;
    const uint32_t cbits = __float_as_uint(swap ? sx : cx) ^ ((((oct + 2u) >> 2) & 1u) << 31);
    const uint32_t sbits = __float_as_uint(swap ? cx : sx) ^ ((oct >> 2) << 31);
    c = __uint_as_float(cbits);
    s = __uint_as_float(sbits);
}

// Two scaled normals from two Philox words: (rho cos, rho sin) * scale, scale = fl32(1/sqrtf(r)).
__device__ __forceinline__ void normal_pair(uint32_t xa, uint32_t xb, float scale, float& a_cos, float& a_sin)
{
    const float rho = __fsqrt_rn(neg2_ln_u1((xa >> 8) + 1u));
    float c, s;
    cos_sin_2pi_u2(xb >> 8, c, s);
    a_cos = __fmul_rn(__fmul_rn(rho, c), scale);
    a_sin = __fmul_rn(__fmul_rn(rho, s), scale);
}

// A[j, 4q .. 4q+3] as fp32.
__device__ __forceinline__ void projection_quad(uint32_t q, uint32_t j, PhiloxKey key, float scale, float (&a)[4])
{
    uint32_t x[4];
    philox_block(q, j, key, x);
    normal_pair(x[0], x[1], scale, a[0], a[1]);
    normal_pair(x[2], x[3], scale, a[2], a[3]);
}

// The same four values rounded to bf16 (nearest even), packed as two bf16x2 words:
// x = (A[j,4q], A[j,4q+1]), y = (A[j,4q+2], A[j,4q+3]); the lower column sits in the low half.
__device__ __forceinline__ uint2 projection_quad_bf16(uint32_t q, uint32_t j, PhiloxKey key, float scale)
{
    float a[4];
    projection_quad(q, j, key, scale, a);
    __nv_bfloat162 lo = __floats2bfloat162_rn(a[0], a[1]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(a[2], a[3]);
    uint2 out;
    out.x = *reinterpret_cast<uint32_t*>(&lo);
    out.y = *reinterpret_cast<uint32_t*>(&hi);
    return out;
}

__device__ __forceinline__ float bf16_round(float v)
{
    return __bfloat162float(__float2bfloat16_rn(v));
}

}  // namespace flora

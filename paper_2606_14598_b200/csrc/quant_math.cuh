// Arithmetic of the per-row int8 quantizer (paper, "The quantization recipe (reused)": symmetric per-token /
// per-channel int8 with scale = absmax / 127, round half to even), shared by the quantizer kernels and by the
// one-kernel path for small problems. Device code only.
#pragma once

#include "ptx.cuh"

#include <cuda_bf16.h>

namespace w8a8 {

// q = clamp(rne(x / s)) with the IEEE quotient, the definition.
__device__ __forceinline__ int quant_exact(float x, float s) {
    return max(-127, min(127, __float2int_rn(__fdiv_rn(x, s))));
}

// The IEEE quotient without a division instruction. With inv = RN(1 / s) (correctly rounded, once
// per row), q0 = RN(x * inv) is within 1.5 ulp of x / s; one fma pair (remainder r0 = x - s * q0,
// exact; q1 = RN(q0 + r0 * inv)) makes it faithful, and by Markstein's theorem a second pair then
// yields exactly RN(x / s): if the reciprocal is correctly rounded and q is faithful, RN(q + r * inv)
// with the exact remainder r is the correctly rounded quotient (no over/underflow; scales outside
// [1e-30, 1e30] take the division instead). Adding 1.5 * 2^23 rounds the quotient to the nearest
// integer, ties to even, and leaves the code in the low byte of the sum; |x / s| <= 127 * (1 + 2^-23)
// so the clamp to [-127, 127] cannot bind.
struct RowScale {
    float s, inv;
    bool fast;      // false for degenerate scales: every element takes the division
};
__device__ __forceinline__ RowScale make_row_scale(float amax) {
    RowScale r;
    r.s = amax > 0.f ? __fdiv_rn(amax, 127.0f) : 1.0f;
    r.inv = __frcp_rn(r.s);
    r.fast = r.s >= 1e-30f && r.s <= 1e30f;
    return r;
}
constexpr float MAGIC = 12582912.0f;               // 1.5 * 2^23

// the code of x in the low byte of the result (upper bytes are don't-care)
__device__ __forceinline__ uint32_t quant1(float x, const RowScale& rs) {
    const float q0 = __fmul_rn(x, rs.inv);
    const float r0 = __fmaf_rn(-rs.s, q0, x);
    const float q1 = __fmaf_rn(r0, rs.inv, q0);
    const float r1 = __fmaf_rn(-rs.s, q1, x);
    const float q2 = __fmaf_rn(r1, rs.inv, q1);
    return __float_as_uint(__fadd_rn(q2, MAGIC));
}
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, const RowScale& rs) {
    if (rs.fast) {
        const uint32_t lo = __byte_perm(quant1(a, rs), quant1(b, rs), 0x0040);
        const uint32_t hi = __byte_perm(quant1(c, rs), quant1(d, rs), 0x0040);
        return __byte_perm(lo, hi, 0x5410);
    }
    return (uint32_t(quant_exact(a, rs.s)) & 0xffu) | ((uint32_t(quant_exact(b, rs.s)) & 0xffu) << 8) |
           ((uint32_t(quant_exact(c, rs.s)) & 0xffu) << 16) | (uint32_t(quant_exact(d, rs.s)) << 24);
}

// |x| maximum of 8 packed bf16 values, kept packed (two running maxima)
__device__ __forceinline__ __nv_bfloat162 absmax8(const uint4& v, __nv_bfloat162 m) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) m = __hmax2(m, __habs2(*reinterpret_cast<const __nv_bfloat162*>(&w[i])));
    return m;
}
__device__ __forceinline__ float unpack_max(__nv_bfloat162 m) {
    const uint32_t mb = *reinterpret_cast<const uint32_t*>(&m);
    return fmaxf(__uint_as_float(mb << 16), __uint_as_float(mb & 0xffff0000u));
}
// Two quotients at a time with the packed fp32x2 instructions (each half rounds exactly like the scalar
// instruction): the same sequence as quant1 on a pair of values held in one 64-bit register.
struct RowScale2 {          // RowScale with its constants replicated into both halves
    uint64_t neg_s, inv, magic;
    uint64_t inv_hi, inv_lo;        // the reciprocal in two pieces, for bf16 inputs (see quant2)
};
__device__ __forceinline__ RowScale2 make_row_scale2(const RowScale& rs) {
    // inv_hi: the reciprocal cut to 16 significant bits; inv_lo: what is missing to 1 / s, to ~2^-39 of it
    const float inv_hi = __uint_as_float(__float_as_uint(rs.inv) & 0xffffff00u);
    const float inv_lo = rs.fast ? __fdiv_rn(__fmaf_rn(-rs.s, inv_hi, 1.0f), rs.s) : 0.f;
    return RowScale2{pack2(-rs.s, -rs.s), pack2(rs.inv, rs.inv), pack2(MAGIC, MAGIC), pack2(inv_hi, inv_hi), pack2(inv_lo, inv_lo)};
}
// Codes of the two bf16 values of `w` in byte 0 and byte 4 of the result. A bf16 value has 8 significant bits, so its
// product with the 16-bit inv_hi is exact; one fma adds x * inv_lo and rounds once: a faithful quotient (within an ulp
// of x / s) in two operations instead of three. The remainder pair then makes it the correctly rounded one as above.
__device__ __forceinline__ uint64_t quant2(uint32_t w, const RowScale2& r2) {
    const uint64_t x = pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    const uint64_t p = mul2(x, r2.inv_hi);
    const uint64_t q1 = fma2(x, r2.inv_lo, p);
    const uint64_t r1 = fma2(r2.neg_s, q1, x);
    const uint64_t q2 = fma2(r1, r2.inv, q1);
    return add2(q2, r2.magic);
}
__device__ __forceinline__ uint32_t gather4(uint64_t a, uint64_t b) {   // bytes 0 and 4 of a, then of b
    const uint32_t lo = __byte_perm(static_cast<uint32_t>(a), static_cast<uint32_t>(a >> 32), 0x0040);
    const uint32_t hi = __byte_perm(static_cast<uint32_t>(b), static_cast<uint32_t>(b >> 32), 0x0040);
    return __byte_perm(lo, hi, 0x5410);
}
// 8 packed bf16 -> 8 int8 codes (bf16 -> fp32 is exact: the 16 bits become the high half of the word)
__device__ __forceinline__ uint2 quant8(const uint4& v, const RowScale& rs, const RowScale2& r2) {
    if (rs.fast)
        return make_uint2(gather4(quant2(v.x, r2), quant2(v.y, r2)), gather4(quant2(v.z, r2), quant2(v.w, r2)));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    return make_uint2(quant4(f[0], f[1], f[2], f[3], rs), quant4(f[4], f[5], f[6], f[7], rs));
}

} // namespace w8a8

// Row quantiser of the INT8 KV cache (Section 2.2): symmetric codes, one fp32 scale per row.
//
// Sixteen (or eight) consecutive lanes own one 128-value row, eight (or sixteen) values per lane.  All lanes of
// a warp must call the quantiser together (the shuffles inside name all 32 lanes).
//
// code = round_half_even(127 x / amax) on the exact ratio, without a branch: the fp32 quotient of 127 x by
// amax is formed correctly rounded (first quotient p = y * rc with rc = RN(1 / amax) and y = 127 x, exact
// residual r = y - amax * p from one fused multiply-add, corrected quotient q = p + r * rc), and q + 1.5 * 2^23
// rounds it to the nearest integer, ties to even.  For bf16 x and amax an exact ratio that is not a rounding tie
// lies at least 2^8 fp32 ulps from the nearest tie, and a tie n + 1/2 is itself an fp32 number that the
// corrected quotient reproduces exactly, so the second rounding never changes the decision: codes and scales
// are reproducible bit for bit (checked on the host against integer arithmetic for every pair of finite bf16
// values |x| <= amax).  Rows whose amax lies outside [2^-60, 2^60] are rescaled by 2^(+-64) first, which is
// exact, so that no intermediate leaves the normal fp32 range.
#pragma once
#include "slim_common.cuh"

namespace slim {

constexpr float kRoundMagic = 12582912.f;   // 1.5 * 2^23

// packed arithmetic: two bf16 or two fp32 values per instruction
__device__ __forceinline__ uint32_t ap_abs_bf16x2(uint32_t a)
{
    uint32_t r;
    asm("abs.bf16x2 %0, %1;\n" : "=r"(r) : "r"(a));
    return r;
}
__device__ __forceinline__ uint32_t ap_max_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;\n" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint64_t ap_pack(float lo, float hi)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void ap_unpack(uint64_t v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t ap_fma2(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t ap_mul2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t ap_add2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// One row of 128 values owned by 16 / NV consecutive lanes; raw[v] holds this lane's eight consecutive values
// that start at column 8 * (lane + v * 16 / NV).  pk[v] receives their eight codes (byte i = value i), scale the
// row's amax / 127 (0 for an all-zero row, whose codes are 0).  Every lane of the warp must call it together.
template <int NV>
__device__ __forceinline__ void quantize_row(const uint4 (&raw)[NV], uint2 (&pk)[NV], float &scale)
{
    // absmax on the packed bf16 pairs, then across the lanes of the row
    uint32_t m2 = 0;
#pragma unroll
    for (int v = 0; v < NV; ++v)
        m2 = ap_max_bf16x2(m2, ap_max_bf16x2(ap_max_bf16x2(ap_abs_bf16x2(raw[v].x), ap_abs_bf16x2(raw[v].y)),
                                             ap_max_bf16x2(ap_abs_bf16x2(raw[v].z), ap_abs_bf16x2(raw[v].w))));
    float amax = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
#pragma unroll
    for (int o = 8 / NV; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));

    // rescaling of rows with extreme magnitudes (exact: a power of two)
    float f = 1.f;
    if (amax < 0x1p-60f) f = 0x1p64f;
    else if (amax > 0x1p60f) f = 0x1p-64f;
    const float as = __fmul_rn(amax, f), m127 = __fmul_rn(127.f, f);
    const float rc = (amax > 0.f) ? __frcp_rn(as) : 0.f;   // an all-zero row gets codes 0
    const uint64_t m127_2 = ap_pack(m127, m127), rc2 = ap_pack(rc, rc), nas2 = ap_pack(-as, -as),
                   magic2 = ap_pack(kRoundMagic, kRoundMagic);
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const uint32_t w[4] = {raw[v].x, raw[v].y, raw[v].z, raw[v].w};
        uint32_t tb[8];   // 0x4B400000 + code: the low byte is the code in two's complement
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            // two elements per instruction (packed fp32)
            const uint64_t x2 = ap_pack(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xFFFF0000u));
            const uint64_t y2 = ap_mul2(x2, m127_2);        // 127 x, exact
            const uint64_t p2 = ap_mul2(y2, rc2);           // first quotient
            const uint64_t r2 = ap_fma2(nas2, p2, y2);      // its exact residual
            const uint64_t q2 = ap_fma2(r2, rc2, p2);       // correctly rounded 127 x / amax
            const uint64_t t2 = ap_add2(q2, magic2);        // nearest integer, ties to even
            tb[2 * k] = (uint32_t)t2;
            tb[2 * k + 1] = (uint32_t)(t2 >> 32);
        }
        pk[v].x = __byte_perm(__byte_perm(tb[0], tb[1], 0x0040), __byte_perm(tb[2], tb[3], 0x0040), 0x5410);
        pk[v].y = __byte_perm(__byte_perm(tb[4], tb[5], 0x0040), __byte_perm(tb[6], tb[7], 0x0040), 0x5410);
    }
    // scale = RN(amax / 127) with the same two-step correction (c = RN(1 / 127)); the plain division serves the
    // rescaled rows, whose quotient may be subnormal
    constexpr float c127 = 1.f / 127.f;
    const float sq = __fmul_rn(amax, c127);
    scale = fmaf(fmaf(-127.f, sq, amax), c127, sq);
    if (f != 1.f) scale = __fdiv_rn(amax, 127.f);
}

// Sixteen lanes per row, eight values per lane.
__device__ __forceinline__ uint2 quantize_row16(const uint4 raw, float &scale)
{
    const uint4 r[1] = {raw};
    uint2 pk[1];
    quantize_row<1>(r, pk, scale);
    return pk[0];
}

}  // namespace slim

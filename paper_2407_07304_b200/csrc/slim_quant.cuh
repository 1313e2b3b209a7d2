// Row quantiser of the INT8 KV cache (Section 2.2): symmetric codes, one fp32 scale per row.
//
// Sixteen consecutive lanes own one 128-value row, eight consecutive values per lane.  Both halves of a warp
// must call quantize_row16 together (the shuffles and votes inside name all 32 lanes).
//
// code = round_half_even(127 x / amax) on the exact ratio.  The fast path multiplies by the correctly
// rounded 127 / amax and rounds with the 1.5 * 2^23 trick; the product is within 2^-16 of the exact ratio,
// so whenever it lies further than 2^-10 from a rounding tie the result is the exact one.  For the elements
// nearer to a tie (0.3 % of them, most of them exact ties of the coarse bf16 grid) the exact residual
// 127 x - c * amax is compared with amax / 2, which decides the tie correctly; a warp takes that path only
// when one of its lanes needs it.  Codes and scales are therefore reproducible bit for bit.
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
__device__ __forceinline__ uint64_t ap_add2(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// raw: this lane's eight bf16 values of the row.  Returns the eight codes (byte i = value i) and the row's
// scale amax / 127 (0 for an all-zero row, whose codes are 0).
__device__ __forceinline__ uint2 quantize_row16(const uint4 raw, float &scale)
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    // absmax on the packed bf16 pairs, then across the 16 lanes of the row
    uint32_t m2 = ap_max_bf16x2(ap_max_bf16x2(ap_abs_bf16x2(w[0]), ap_abs_bf16x2(w[1])),
                                ap_max_bf16x2(ap_abs_bf16x2(w[2]), ap_abs_bf16x2(w[3])));
    float amax = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xFFFF0000u));
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));   // within the 16 lanes

    uint32_t tb[8];   // 0x4B400000 + code: the low byte is the code in two's complement
    const float inv = (amax > 0.f) ? __fdiv_rn(127.f, amax) : 0.f;   // an all-zero row gets codes 0
    const float half = 0.5f * amax;
    const uint64_t inv2 = ap_pack(inv, inv), magic2 = ap_pack(kRoundMagic, kRoundMagic),
                   nmagic2 = ap_pack(-kRoundMagic, -kRoundMagic);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        // two elements per instruction (packed fp32): t = x * inv + 1.5 * 2^23 rounds the product to the nearest
        // integer (ties to even) in one step; c0 = that integer; d = x * inv - c0 its distance from the product
        const float x0 = __uint_as_float(w[k] << 16), x1 = __uint_as_float(w[k] & 0xFFFF0000u);
        const uint64_t x2 = ap_pack(x0, x1);
        const uint64_t t2 = ap_fma2(x2, inv2, magic2);
        const uint64_t c2 = ap_add2(t2, nmagic2);
        const uint64_t d2 = ap_fma2(x2, inv2, c2 ^ 0x8000000080000000ull);
        float c0[2], d[2];
        ap_unpack(c2, c0[0], c0[1]);
        ap_unpack(d2, d[0], d[1]);
        tb[2 * k] = (uint32_t)t2;
        tb[2 * k + 1] = (uint32_t)(t2 >> 32);
        const bool near0 = fabsf(d[0]) > 0.5f - 0x1p-10f, near1 = fabsf(d[1]) > 0.5f - 0x1p-10f;   // 0.3 % of the elements
        if (__any_sync(0xffffffffu, near0 || near1)) {
            // Near a rounding tie the approximate quotient may have picked the wrong neighbour.  The residual
            // 127 x - c0 * amax is exact in fp32 (127 x has 15 significant bits, c0 * amax at most 15, and they
            // are within a factor 2^9 of each other when c0 != 0), so comparing it with amax / 2 decides exactly.
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const float e = fmaf(-c0[j], amax, 127.f * (j ? x1 : x0));
                const bool odd = (tb[2 * k + j] & 1u) != 0u;
                const int up = (e > half || (e == half && odd)) ? 1 : 0;
                const int dn = (e < -half || (e == -half && odd)) ? 1 : 0;
                if (j ? near1 : near0) tb[2 * k + j] += (uint32_t)(up - dn);
            }
        }
    }
    uint2 pk;
    pk.x = __byte_perm(__byte_perm(tb[0], tb[1], 0x0040), __byte_perm(tb[2], tb[3], 0x0040), 0x5410);
    pk.y = __byte_perm(__byte_perm(tb[4], tb[5], 0x0040), __byte_perm(tb[6], tb[7], 0x0040), 0x5410);
    scale = (amax > 0.f) ? __fdiv_rn(amax, 127.f) : 0.f;
    return pk;
}

}  // namespace slim

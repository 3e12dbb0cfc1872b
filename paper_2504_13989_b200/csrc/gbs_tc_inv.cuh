// Helpers of the tensor-core inverse paths of gbs_dequantize (gbs_tc_uvinv.cu, gbs_tc_rowinv.cu): packed codes ->
// bf16 operand chunks without a conversion instruction, and the scaled stores of 32 rotated values.
#pragma once

#include <cuda_bf16.h>

namespace {

// Eight offset codes, even ones in the bytes of y and odd ones in the bytes of z (each byte = q + 2^(b-1)),
// -> four words of two bf16 numbers 128 + byte: [y.b0 z.b0] [y.b1 z.b1] [y.b2 z.b2] [y.b3 z.b3].
__device__ __forceinline__ uint4 bytes_to_bf16x8(unsigned y, unsigned z)
{
    uint4 o;
    o.x = (__byte_perm(y, z, 0x4400) & 0x00ff00ffu) | 0x43004300u;
    o.y = (__byte_perm(y, z, 0x5511) & 0x00ff00ffu) | 0x43004300u;
    o.z = (__byte_perm(y, z, 0x6622) & 0x00ff00ffu) | 0x43004300u;
    o.w = (__byte_perm(y, z, 0x7733) & 0x00ff00ffu) | 0x43004300u;
    return o;
}

// The 32 codes of one row segment (coordinates 32 u .. 32 u + 31 of a token) -> 32 bf16 numbers q + OFF,
// as the four 16-byte chunks of the operand row.
// UNSIGNED_FIELDS (asymmetric plans): the field is the code itself, stored as 128 + f (OFF = 128).
template <int BITS, bool UNSIGNED_FIELDS>
__device__ __forceinline__ void unpack_row(const unsigned char* src, uint4 chunk[4])
{
    if (BITS == 4) {
        const uint4 w = __ldg(reinterpret_cast<const uint4*>(src));
        const unsigned ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const unsigned x = ws[c] ^ (UNSIGNED_FIELDS ? 0u : 0x88888888u);   // two's-complement nibble -> q + 8
            chunk[c] = bytes_to_bf16x8(x & 0x0f0f0f0fu, (x >> 4) & 0x0f0f0f0fu);
        }
    } else {
        const unsigned* s = reinterpret_cast<const unsigned*>(src);
        const unsigned a0 = __ldg(s), a1 = __ldg(s + 1), a2 = __ldg(s + 2);
        // 24 bits (eight 3-bit fields) per chunk
        const unsigned g[4] = {a0 & 0xffffffu, ((a0 >> 24) | (a1 << 8)) & 0xffffffu, ((a1 >> 16) | (a2 << 16)) & 0xffffffu,
                               a2 >> 8};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const unsigned e = g[c], o = g[c] >> 3;                  // even fields at bits 6k, odd ones too after >> 3
            unsigned y = (e & 0x7u) | ((e << 2) & 0x700u) | ((e << 4) & 0x70000u) | ((e << 6) & 0x7000000u);
            unsigned z = (o & 0x7u) | ((o << 2) & 0x700u) | ((o << 4) & 0x70000u) | ((o << 6) & 0x7000000u);
            const unsigned fx = UNSIGNED_FIELDS ? 0u : 0x04040404u;              // two's-complement field -> q + 4
            chunk[c] = bytes_to_bf16x8(y ^ fx, z ^ fx);
        }
    }
}

__device__ __forceinline__ void st_shared_v4(unsigned addr, uint4 v)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// dst[i] = r[i] * sc (+ add0 for i = 0), 32 values, 16-byte stores
template <typename OutT>
__device__ __forceinline__ void store_row32(OutT* dst, const unsigned r[32], float sc, float add0);
template <>
__device__ __forceinline__ void store_row32<float>(float* dst, const unsigned r[32], float sc, float add0)
{
    float4* o = reinterpret_cast<float4*>(dst);
#pragma unroll
    for (int i = 0; i < 8; ++i)
        o[i] = make_float4(i == 0 ? fmaf(__uint_as_float(r[0]), sc, add0) : __uint_as_float(r[4 * i]) * sc,
                           __uint_as_float(r[4 * i + 1]) * sc, __uint_as_float(r[4 * i + 2]) * sc,
                           __uint_as_float(r[4 * i + 3]) * sc);
}
template <>
__device__ __forceinline__ void store_row32<__nv_bfloat16>(__nv_bfloat16* dst, const unsigned r[32], float sc, float add0)
{
    uint4* o = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        unsigned w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float lo = (i == 0 && k == 0) ? fmaf(__uint_as_float(r[0]), sc, add0) : __uint_as_float(r[8 * i + 2 * k]) * sc;
            const __nv_bfloat162 h = __floats2bfloat162_rn(lo, __uint_as_float(r[8 * i + 2 * k + 1]) * sc);
            w[k] = *reinterpret_cast<const unsigned*>(&h);
        }
        o[i] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}


}  // namespace

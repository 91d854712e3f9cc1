// Dequantisation of stored words to bf16, shared by the prefill kernels: the fused kernel's dequantisation warps
// (fq_gemm_fused.cu) and the stand-alone pass of the two-pass path (fq_gemm.cu).  Everything is specialised per
// field list (variant_index in fq_layout.cuh), so that field widths, shifts and offsets are compile-time constants.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "fq_internal.cuh"

namespace fq {

// Loop whose index is a compile-time constant in the body.
template <int I, int N, class Fn>
__device__ __forceinline__ void unrolled(Fn&& fn)
{
    if constexpr (I < N) {
        fn(std::integral_constant<int, I>{});
        unrolled<I + 1, N>(fn);
    }
}

FQ_HDC int fields_prefix(const FieldList fl, int fi) { int p = 0; for (int i = 0; i < fi; i++) p += fl.width[i]; return p; }
// 16-byte loads a lane needs for one tile and one stage (two k32 steps): two for an 8-bit field, one otherwise.
FQ_HDC int fields_loads(const FieldList fl, int fi) { int n = 0; for (int i = 0; i < fi; i++) n += fl.width[i] == 8 ? 2 : 1; return n; }

// The stored words of k32 steps j0, j0 + 1 of tile TL of superstep ssl: 16 bytes per lane and field chunk,
// exactly the words the decode kernel feeds to its integer MMAs.
//   blob_lane : the blob + 16 * lane
template <int VARIANT, int TL>
__device__ __forceinline__ void load_stage_words(const uint8_t* blob_lane, int ssl, int j0,
                                                 uint4 (&raw)[fields_loads(variant_fields(VARIANT), variant_fields(VARIANT).n)])
{
    constexpr FieldList FL = variant_fields(VARIANT);
    unrolled<0, FL.n>([&](auto FI) {
        constexpr int fi = decltype(FI)::value, F = FL.width[fi], P = 8 / F;
        constexpr int base = fields_loads(FL, fi);
        const uint8_t* tb = blob_lane + blob_field_off(fields_prefix(FL, fi), F, 0, TL) + ssl * (kBlobTiles * F * 512);
        if constexpr (F == 8) {
            raw[base] = __ldg(reinterpret_cast<const uint4*>(tb + j0 * 512));
            raw[base + 1] = __ldg(reinterpret_cast<const uint4*>(tb + j0 * 512 + 512));
        } else {
            raw[base] = __ldg(reinterpret_cast<const uint4*>(tb + (j0 / P) * 512));      // j0 and P are even: one chunk
        }
    });
}

// The A registers (four codes each, one per byte) of the two steps, all fields merged: a field's bits of
// step t sit at bit t * F of every byte of its word; one rotation brings them to the field's place in the
// code, one AND-OR merges them.
template <int VARIANT>
__device__ __forceinline__ void merge_codes(const uint4 (&raw)[fields_loads(variant_fields(VARIANT), variant_fields(VARIANT).n)],
                                            int j0, uint32_t (&code)[2][4])
{
    constexpr FieldList FL = variant_fields(VARIANT);
    unrolled<0, FL.n>([&](auto FI) {
        constexpr int fi = decltype(FI)::value, F = FL.width[fi], P = 8 / F, SH = FL.shift[fi];
        constexpr int base = fields_loads(FL, fi);
        constexpr uint32_t kM = (field_keep_mask(F, FL.keep[fi]) * 0x01010101u) << SH;
#pragma unroll
        for (int jj = 0; jj < 2; jj++) {
            const uint4 w = raw[F == 8 ? base + jj : base];
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int r = 0; r < 4; r++) {
                uint32_t v;
                if constexpr (F == 8) v = ww[r];
                else if constexpr (P == 2) v = __funnelshift_r(ww[r], ww[r], (jj * F - SH) & 31) & kM;   // j0 % 2 == 0
                else v = __funnelshift_r(ww[r], ww[r], (((j0 & (P - 1)) + jj) * F - SH) & 31) & kM;
                code[jj][r] = fi == 0 ? v : (code[jj][r] | v);
            }
        }
    });
}

// Four codes of one row (one A register) -> four bf16 weights w^ = (q - z) * s, each rounded once.
//   Codes up to 255: a byte q under the exponent byte 0x64 is the fp16 number 1024 + q; subtracting zz = 1024 + z
//   in fp16 is exact (integers below 2048), the product with the fp16 scale is exact in fp32 (9 x 11 bits).
__device__ __forceinline__ uint2 codes_to_bf16(uint32_t q4, __half2 zz, float s)
{
    const uint32_t p02 = (q4 & 0x00ff00ffu) | 0x64006400u;          // columns 0 and 2
    const uint32_t p13 = __byte_perm(q4, 0x64646464u, 0x4341);      // columns 1 and 3
    const float2 d02 = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&p02), zz));
    const float2 d13 = __half22float2(__hsub2(*reinterpret_cast<const __half2*>(&p13), zz));
    const __nv_bfloat162 lo = __floats2bfloat162_rn(d02.x * s, d13.x * s);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(d02.y * s, d13.y * s);
    uint2 o;
    o.x = *reinterpret_cast<const uint32_t*>(&lo);
    o.y = *reinterpret_cast<const uint32_t*>(&hi);
    return o;
}
//   Codes below 128: a byte q in bits 16..22 under the exponent byte 0x43 is the fp32 number 128 + q, and
//   fma(128 + q, s, c) with c = -(128 + z) * s (exact: 8 x 11 bits) is (q - z) * s without any rounding.
__device__ __forceinline__ uint2 small_codes_to_bf16(uint32_t q4, float c, float s)
{
    const float f0 = __uint_as_float(__byte_perm(q4, 0x43000000u, 0x7044));
    const float f1 = __uint_as_float(__byte_perm(q4, 0x43000000u, 0x7144));
    const float f2 = __uint_as_float(__byte_perm(q4, 0x43000000u, 0x7244));
    const float f3 = __uint_as_float(__byte_perm(q4, 0x43000000u, 0x7344));
    const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(f0, s, c), fmaf(f1, s, c));
    const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(f2, s, c), fmaf(f3, s, c));
    uint2 o;
    o.x = *reinterpret_cast<const uint32_t*>(&lo);
    o.y = *reinterpret_cast<const uint32_t*>(&hi);
    return o;
}

// The variant whose field list is `fl`, or -1.
inline int variant_of_fields(const FieldList& fl)
{
    for (int v = 0; v < kVariants; v++) {
        const FieldList c = variant_fields(v);
        bool same = c.n == fl.n;
        for (int i = 0; same && i < c.n; i++) same = c.width[i] == fl.width[i] && c.shift[i] == fl.shift[i] && c.keep[i] == fl.keep[i];
        if (same) return v;
    }
    return -1;
}

}  // namespace fq

// Decode arithmetic of one work item: one blob (two 16-row tiles x 512 columns = two supersteps of 256),
// batch 1.  Included by the decode kernel only.
//
// Stored words become A operands of the 8-bit mma.m16n8k32 with ONE AND each (a word holds 8/F
// registers on top of each other, see fq_layout.cuh); the activations are 16-bit fixed point per
// group of 128 columns, split into two signed byte digits, and are the B operand.  k32 step j of a
// superstep always feeds B columns (2*(j&3), 2*(j&3)+1) with (low digit, high digit) and zeros
// elsewhere, so the four steps of a group land in four different column pairs of ONE accumulator
// although their A registers sit at different bit offsets: lane (g, c) of the warp ends up with the
// partial sum of step class c, scaled by a power of two that only depends on (c, field width, group).
// Per group:  y += s * 2^-e * ( sum_fields 2^shift * sum_k field_k * x_int_k  -  z * sum_k x_int_k ),
// exact in s32 up to the final fp32 multiply.
#pragma once
#include <cuda_fp16.h>

#include <type_traits>

#include "fq_layout.cuh"

namespace fq {

// ------------------------------------------------------------------------------- shared-memory loads
// Shared memory is addressed with 32-bit shared-window addresses and explicit ld.shared; OFF is a
// compile-time byte offset that goes into the instruction's address field.
template <int OFF = 0>
__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF = 0>
__device__ __forceinline__ uint2 lds64(uint32_t a)
{
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF = 0>
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF));
    return v;
}
// Loop whose index is a compile-time constant in the body (so that it can be a load's immediate offset).
template <int I, int N, class Fn>
__device__ __forceinline__ void static_for(Fn&& fn)
{
    if constexpr (I < N) {
        fn(std::integral_constant<int, I>{});
        static_for<I + 1, N>(fn);
    }
}

// D = A(u8, 16x32, row) * B(s8, 32x8, col) + C, s32.  Not volatile: a pure function of its registers,
// the compiler may interleave independent chains.
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_u8s8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

// ------------------------------------------------------------------------------- activation layout
// Shared-memory image of the activations of one blob (512 columns), written by the pre-processing
// warps and read by the consumers:
//   digits   [superstep 2][step class jc 4][digit 2][c 4][16 B]                      (1024 B)
//            the 16 bytes are the B registers (b0, b1) of k32 step jc followed by those of step jc + 4:
//            b0 = columns 32j + 4c .. +3, b1 = columns 32j + 16 + 4c .. +3 of the superstep
//   groups   int sum[superstep 2][group 2], float scale[superstep 2][group 2]          (32 B)
constexpr int kXBlobDigitBytes = 1024;
constexpr int kXBlobGroupBytes = 32;
FQ_HDC int x_digit_off(int ss, int jc, int digit, int c) { return ss * 512 + jc * 128 + digit * 64 + c * 16; }

// An opaque -1: `a * kMinusOne + w` then stays a multiply-add (FMA pipe) instead of becoming an
// integer subtract on the ALU pipe, which the masks already keep busy.
__device__ __forceinline__ int opaque_minus_one()
{
    int v;
    asm volatile("mov.s32 %0, -1;" : "=r"(v));
    return v;
}

// One field of width F (at bit SHIFT of the code) of one tile, one superstep.  Adds (FIRSTF: stores)
// per row half r and group the integer  2^SHIFT * sum_k field_k * x_int_k  (this lane's step class) to v.
//   fa : shared address of this lane's 16-byte chunk in the tile's field array, this superstep
//   bx : B registers of the superstep: bx[jc] = (b0, b1 of step jc, b0, b1 of step jc + 4)
template <int F, int KEEP, int SHIFT, bool FIRSTF, int OFF>
__device__ __forceinline__ void field_step(uint32_t fa, const uint4 (&bx)[4], int c, int m1, int (&v)[2][2])
{
    constexpr int P = 8 / F;                                   // A registers stacked in one word
    constexpr uint32_t kMask = field_keep_mask(F, KEEP) * 0x01010101u;
    static_assert(F != 4 || KEEP == 4, "the word-minus-low-nibbles shortcut takes whole 4-bit fields");
    int acc[2][4];
    uint4 w[F < 4 ? F : 4];
    static_for<0, (F < 4 ? F : 4)>([&](auto JB) { w[decltype(JB)::value] = lds128<OFF + decltype(JB)::value * 512>(fa); });
    static_for<0, 8>([&](auto JI) {
        constexpr int j = decltype(JI)::value;                 // k32 step inside the superstep
        constexpr int jb = j / P, t = j % P, grp = j >> 2, jc = j & 3;
        if constexpr (F == 8 && j == 4)                        // second half of an 8-bit field's chunks
            static_for<0, 4>([&](auto JB) { w[decltype(JB)::value] = lds128<OFF + (4 + decltype(JB)::value) * 512>(fa); });
        uint4& a = w[F == 8 ? (jb & 3) : jb];
        [[maybe_unused]] constexpr uint32_t m = kMask << (t * F);
        const uint32_t b0 = grp == 0 ? bx[jc].x : bx[jc].z, b1 = grp == 0 ? bx[jc].y : bx[jc].w;
        uint32_t a0, a1, a2, a3;
        if constexpr (F == 8) { a0 = a.x; a1 = a.y; a2 = a.z; a3 = a.w; }
        else if constexpr (F == 4 && t == 1) { a0 = a.x; a1 = a.y; a2 = a.z; a3 = a.w; }   // what step t = 0 left over
        else { a0 = a.x & m; a1 = a.y & m; a2 = a.z & m; a3 = a.w & m; }
        if constexpr (F == 4 && t == 0) {                      // high nibbles = word - low nibbles, as multiply-adds
            a.x = (uint32_t)((int)a0 * m1 + (int)a.x); a.y = (uint32_t)((int)a1 * m1 + (int)a.y);
            a.z = (uint32_t)((int)a2 * m1 + (int)a.z); a.w = (uint32_t)((int)a3 * m1 + (int)a.w);
        }
        if constexpr (jc == 0) mma_u8s8_first(acc[grp], a0, a1, a2, a3, b0, b1);
        else mma_u8s8(acc[grp], a0, a1, a2, a3, b0, b1);
    });
    // digits -> integer; undo the scaling of this lane's step class (exact: every term is a multiple of
    // it); apply the field's position inside the code.  Bit offset of step j: F=1: j, F=2: 2(j&3), F=4: 4(j&1).
#pragma unroll
    for (int grp = 0; grp < 2; grp++) {
        const int down = F == 1 ? c + 4 * grp : F == 2 ? 2 * c : F == 4 ? 4 * (c & 1) : 0;
        const int e0 = (acc[grp][1] * 256 + acc[grp][0]) >> down;
        const int e1 = (acc[grp][3] * 256 + acc[grp][2]) >> down;
        if (FIRSTF) { v[grp][0] = e0 << SHIFT; v[grp][1] = e1 << SHIFT; }
        else { v[grp][0] += e0 << SHIFT; v[grp][1] += e1 << SHIFT; }
    }
}

// The fields of one (superstep, tile), unrolled at compile time from the variant's field list.
template <int VARIANT, int FI, int PREFIX, int SS, int TILE>
struct FieldLoop {
    static __device__ __forceinline__ void run(uint32_t fbase, const uint4 (&bx)[4], int c, int m1, int (&v)[2][2])
    {
        constexpr FieldList FL = variant_fields(VARIANT);
        if constexpr (FI < FL.n) {
            constexpr int F = FL.width[FI], SHIFT = FL.shift[FI], KEEP = FL.keep[FI];
            // field array of width F after fields adding up to PREFIX bits; tile (SS, TILE) of it
            constexpr int off = kBlobSteps * kBlobTiles * 512 * PREFIX + (SS * kBlobTiles + TILE) * (F * 512);
            field_step<F, KEEP, SHIFT, FI == 0, off>(fbase, bx, c, m1, v);
            FieldLoop<VARIANT, FI + 1, PREFIX + F, SS, TILE>::run(fbase, bx, c, m1, v);
        }
    }
};

// The same with the (superstep, tile) index known only at run time: one multiply-add per field instead of an
// immediate offset, but the loop over supersteps and tiles need not be unrolled.
template <int VARIANT, int FI, int PREFIX>
struct FieldLoopRt {
    static __device__ __forceinline__ void run(uint32_t fbase, int st, const uint4 (&bx)[4], int c, int m1, int (&v)[2][2])
    {
        constexpr FieldList FL = variant_fields(VARIANT);
        if constexpr (FI < FL.n) {
            constexpr int F = FL.width[FI], SHIFT = FL.shift[FI], KEEP = FL.keep[FI];
            field_step<F, KEEP, SHIFT, FI == 0, kBlobSteps * kBlobTiles * 512 * PREFIX>(fbase + st * (F * 512), bx, c, m1, v);
            FieldLoopRt<VARIANT, FI + 1, PREFIX + F>::run(fbase, st, bx, c, m1, v);
        }
    }
};

// Group epilogue of one (superstep, tile): y += s * 2^-e * (v - (z - adjust) * sum x_int).
template <int ADJUST>
__device__ __forceinline__ void group_epilogue(const uint4 mw, const int (&v)[2][2], const int (&nx)[2], const float (&sc)[2],
                                               float (&tot)[2])
{
    const uint32_t mm[2][2] = {{mw.x, mw.y}, {mw.z, mw.w}};      // (grp 0: row g, g + 8), (grp 1: row g, g + 8)
#pragma unroll
    for (int grp = 0; grp < 2; grp++) {
        const int base = ADJUST ? -ADJUST * nx[grp] : 0;
#pragma unroll
        for (int r = 0; r < 2; r++) {
            const uint32_t m = mm[grp][r];
            const float s = __half2float(__ushort_as_half((unsigned short)(m & 0xffffu)));
            const int t = v[grp][r] + (int)__umulhi(m, 65536u) * nx[grp] + base;
            tot[r] = fmaf((float)t, s * sc[grp], tot[r]);
        }
    }
}

// One blob (32 rows x 512 columns): tot[tile][r] += dequantised dot products of rows 16 tile + g + 8 r (this
// lane's step class only; the four lanes of a quad add up to the row sums).  Both row tiles share the B
// registers and the group sums of the activations.  Variants with one or two fields are unrolled over the
// two supersteps and the two tiles; the others (up to seven fields) loop, or the fourteen specialised
// bodies would not fit the instruction cache.
//   blob : shared address of the blob          xd : this lane's B source per step class (digits or zeros)
//   xg   : shared address of the blob's group sums / scales
//   tsel : 0 = both 16-row tiles of the blob, 1 = tile 0 only, 2 = tile 1 only (the other tile's sums stay 0)
template <int VARIANT>
__device__ __forceinline__ void blob_compute(uint32_t blob, const uint32_t (&xd)[4], uint32_t xg, int lane, int tsel,
                                             float (&tot)[kBlobTiles][2])
{
    // a nested child reads the parent's top bits; the dropped bits are filled with their mid-point, which
    // is the same as lowering every zero point by that amount
    constexpr int kAdjust = (VARIANT >= 7 && VARIANT < 13) ? 1 << (7 - (VARIANT - 5)) : 0;
    constexpr bool kUnrolled = variant_fields(VARIANT).n <= 2;
    const int g = lane >> 2, c = lane & 3;
    const uint32_t fbase = blob + kBlobMetaBytes + lane * 16;
    const uint32_t mbase = blob + g * 16;
    const int m1 = opaque_minus_one();
    const int czero = c == 0 ? m1 : 0;                         // only the class-0 lane of a quad subtracts the zero-point term
    if constexpr (kUnrolled) {
        static_for<0, kBlobSteps>([&](auto SSI) {
            constexpr int ss = decltype(SSI)::value;
            uint4 bx[4];
            static_for<0, 4>([&](auto JC) { bx[decltype(JC)::value] = lds128<ss * 512>(xd[decltype(JC)::value]); });
            const uint2 xs2 = lds64<ss * 8>(xg), sc2 = lds64<16 + ss * 8>(xg);
            const int nx[2] = {(int)xs2.x * czero, (int)xs2.y * czero};
            const float sc[2] = {__uint_as_float(sc2.x), __uint_as_float(sc2.y)};
            static_for<0, kBlobTiles>([&](auto TLI) {
                constexpr int tile = decltype(TLI)::value;
                if (tsel == 2 - tile) return;                    // (warp-uniform) this tile belongs to another item
                const uint4 mw = lds128<(ss * kBlobTiles + tile) * 128>(mbase);
                int v[2][2];
                FieldLoop<VARIANT, 0, 0, ss, tile>::run(fbase, bx, c, m1, v);
                group_epilogue<kAdjust>(mw, v, nx, sc, tot[tile]);
            });
        });
    } else {
#pragma unroll 1
        for (int ss = 0; ss < kBlobSteps; ss++) {
            uint4 bx[4];
            static_for<0, 4>([&](auto JC) { bx[decltype(JC)::value] = lds128(xd[decltype(JC)::value] + ss * 512); });
            const uint2 xs2 = lds64(xg + ss * 8), sc2 = lds64<16>(xg + ss * 8);
            const int nx[2] = {(int)xs2.x * czero, (int)xs2.y * czero};
            const float sc[2] = {__uint_as_float(sc2.x), __uint_as_float(sc2.y)};
            float tt[kBlobTiles][2] = {{tot[0][0], tot[0][1]}, {tot[1][0], tot[1][1]}};
#pragma unroll 1
            for (int tile = tsel == 2 ? 1 : 0; tile < (tsel == 1 ? 1 : kBlobTiles); tile++) {
                const int st = ss * kBlobTiles + tile;
                const uint4 mw = lds128(mbase + st * 128);
                int v[2][2];
                FieldLoopRt<VARIANT, 0, 0>::run(fbase, st, bx, c, m1, v);
                float t2[2] = {0.f, 0.f};
                group_epilogue<kAdjust>(mw, v, nx, sc, t2);
                if (tile == 0) { tt[0][0] += t2[0]; tt[0][1] += t2[1]; }
                else { tt[1][0] += t2[0]; tt[1][1] += t2[1]; }
            }
            tot[0][0] = tt[0][0]; tot[0][1] = tt[0][1]; tot[1][0] = tt[1][0]; tot[1][1] = tt[1][1];
        }
    }
}

// Selects the specialised loop of a variant (variant_index in fq_layout.cuh).
__device__ __forceinline__ void blob_dispatch(int variant, uint32_t blob, const uint32_t (&xd)[4], uint32_t xg, int lane, int tsel,
                                              float (&tot)[kBlobTiles][2])
{
#define FQ_VARIANT_CASE(V) case V: blob_compute<V>(blob, xd, xg, lane, tsel, tot); break;
    switch (variant) {
        FQ_VARIANT_CASE(0) FQ_VARIANT_CASE(1) FQ_VARIANT_CASE(2) FQ_VARIANT_CASE(3) FQ_VARIANT_CASE(4)
        FQ_VARIANT_CASE(5) FQ_VARIANT_CASE(6) FQ_VARIANT_CASE(7) FQ_VARIANT_CASE(8) FQ_VARIANT_CASE(9)
        FQ_VARIANT_CASE(10) FQ_VARIANT_CASE(11) FQ_VARIANT_CASE(12) FQ_VARIANT_CASE(13)
        default: break;
    }
#undef FQ_VARIANT_CASE
    static_assert(kVariants == 14, "one case per variant");
}

}  // namespace fq

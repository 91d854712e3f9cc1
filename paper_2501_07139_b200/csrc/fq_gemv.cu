// Decode path for a batch of 2..8 activation rows: fused dequantize-GEMV over tiled field arrays.
// (Batch 1 has its own kernel in fq_gemv1.cu.)
//
// One persistent CTA per SM with four roles:
//   producer warp   : streams "units" (32 output rows x one K chunk: every field array of the
//                     active variant plus the scale/zero words) from HBM into a shared-memory
//                     ring with bulk asynchronous copies (cp.async.bulk + mbarrier tx counts)
//                     and writes a small descriptor next to each stage;
//   x-prep warps    : once per (op, K chunk) that this CTA touches, wait -- bounded -- for the
//                     previous dependency phase, load the activations of that chunk and turn
//                     them into 16-bit fixed point per group of 128 columns
//                     (x_int = rint(x * 2^e), |x_int| < 2^14, stored as two signed byte digits);
//   consumer warps  : two warps share a unit, one 16-row tile each.  Stored words become 8-bit
//                     mma.m16n8k32 A operands with ONE AND each (no shift: a word holds 8/f
//                     registers on top of each other, see fq_layout.cuh), the activation digits
//                     are the B operand, accumulation is exact in s32.  At batch 1 the eight B
//                     columns carry (low digit, high digit) for up to four bit-offset classes,
//                     so no register ever has to be shifted.  The loops are compiled once per
//                     field list (14 variants) and chosen per unit.
//   output warp     : finishes row pairs (see below) and is the only warp that writes y.
//   Per group:  y += s * 2^-e * ( sum_fields 2^shift * sum_k field_k * x_int_k  -  z * sum_k x_int_k ).
// The K chunks of one row pair are computed by different CTAs.  Each unit publishes its row sums
// as 64-bit words (fp32 value, launch tag) with plain stores; the unit whose chunk index is
// (row pair mod chunks) hands its own sums to the output warp, which polls the other chunks'
// words until they carry this launch's tag and adds them in chunk order, so results do not
// depend on scheduling and no fence or atomic sits on the consumers' path.
//
// A whole stack of layers runs as one launch.  Every op's units are dealt to the CTAs in
// contiguous, K-chunk-major blocks (a CTA needs the activations of one or two chunks only);
// the producer runs ahead across op boundaries because weights do not depend on activations.
// Every wait has a time limit; when one runs out the kernel records FQ_ERR_TIMEOUT, stops
// computing, drains its copies and returns.
#include <cuda_fp16.h>

#include <type_traits>

#include "fq_internal.cuh"
#include "fq_ptx.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

#ifndef FQ_GEMV_WARPS
#define FQ_GEMV_WARPS 18
#endif
#ifndef FQ_GEMV_TPW
#define FQ_GEMV_TPW 1
#endif
#ifndef FQ_GEMV_UNIT_BYTES
#define FQ_GEMV_UNIT_BYTES 17408
#endif
constexpr int kConsumerWarps = FQ_GEMV_WARPS;
constexpr int kTilesPerWarp = FQ_GEMV_TPW;             // 16-row tiles of a unit that one consumer warp computes
constexpr int kWarpsPerUnit = kUnitRowTiles / kTilesPerWarp;
constexpr int kUnitsInFlight = kConsumerWarps / kWarpsPerUnit;
static_assert(kTilesPerWarp == 1 || kTilesPerWarp == 2, "a warp computes one or both row tiles of a unit");
static_assert(kConsumerWarps % kWarpsPerUnit == 0, "consumer warps come in groups of one unit");
constexpr int kProducerWarp = kConsumerWarps;          // warp index of the producer
constexpr int kPrepWarp = kConsumerWarps + 1;          // first warp of the activation pre-processors
constexpr int kPrepWarps = 4;                          // they share the items of a segment
constexpr int kOutputWarp = kPrepWarp + kPrepWarps;    // the warp that owns every global store of results
constexpr int kGemvThreads = (kConsumerWarps + 1 + kPrepWarps + 1) * 32;
constexpr int kUnitBytes = FQ_GEMV_UNIT_BYTES;         // bytes of one unit (whole blobs), at most: 2 x 4-bit or 1 x 8-bit blob
constexpr int kXSlots = 3;                             // activation chunks kept in shared memory

template <int MAXB> struct GemvCfg;
// kBlobsMax: k blobs (512 columns) per chunk, at most.  kOutSlots: finished units waiting for the output
// warp (it scans one slot per lane: at most 32).
template <> struct GemvCfg<1> { static constexpr int kBlobsMax = 3, kOutSlots = 32; };
template <> struct GemvCfg<8> { static constexpr int kBlobsMax = 2, kOutSlots = 16; };

// What the producer tells the consumers: once per op a copy of the op descriptor in a ring ...
constexpr int kOpRing = 16;                            // > stages + 1: an op slot outlives the start of its last unit
// ... and once per unit (next to the stage that holds the unit's weights)
struct UnitDesc {
    int ch, rp, nb, seg;                        // K chunk, row pair, blobs in the unit, activation segment
    int op_slot;                                // op ring slot
    int oseq;                                   // >= 0: this unit finishes its row pair, and is the oseq-th such unit of the CTA
    int pad[2];
};
static_assert(sizeof(UnitDesc) == 32, "descriptor layout");

// What a consumer hands to the output warp together with the unit's 32 x batch row sums.
struct OutDesc {
    int rp, ch, n_chunks, n_out, phase, batch;
    uint16_t* y;
    const unsigned long long* partial;
    int pad[2];
};
static_assert(sizeof(OutDesc) == 48, "descriptor layout");

template <int MAXB> struct GemvSmem {
    static constexpr int kCMax = GemvCfg<MAXB>::kBlobsMax * kBlobSteps;     // supersteps per chunk, at most
    static constexpr int kOutSlots = GemvCfg<MAXB>::kOutSlots;
    static constexpr int kStageBytes = kUnitBytes;
    // activation slot: low digits, high digits (rows padded so that LDS.64 of a quarter warp is
    // conflict free), then per (row, group) the integer sum and the power-of-two scale
    static constexpr int kXRow = MAXB == 1 ? kCMax * 256 : kCMax * 256 + 32;
    static constexpr int kDigitOff = MAXB == 1 ? kXRow : MAXB * kXRow + 64;
    static constexpr int kXsumOff = kDigitOff + MAXB * kXRow;
    static constexpr int kXscaleOff = kXsumOff + MAXB * kCMax * 2 * 4;
    static constexpr int kXSlotBytes = (kXscaleOff + MAXB * kCMax * 2 * 4 + 127) / 128 * 128;
    static constexpr int kZeroBytes = kCMax * 256 + 64;
    static constexpr int kOpBytes = (int)((sizeof(GemvOp) + 15) / 16 * 16);
    static constexpr int kOutFloats = 32 * (MAXB == 1 ? 1 : 8);              // row sums of one unit
    static constexpr int kOutBytes = kOutSlots * (kOutFloats * 4 + (int)sizeof(OutDesc));
    static constexpr int kFixed = kXSlots * kXSlotBytes + kZeroBytes + kOpRing * kOpBytes + (2 + 2 * kPrepWarps) * kOpBytes +
                                  kOutBytes + 512;
    static constexpr int kPerStage = kStageBytes + (int)sizeof(UnitDesc) + 16 + 4;
    static constexpr int kAuto = (232448 - kFixed) / kPerStage;
    static constexpr int kStages = kAuto > 16 ? 16 : kAuto;
    static constexpr int oStages = 0;
    static constexpr int oDesc = oStages + kStages * kStageBytes;
    static constexpr int oX = oDesc + kStages * (int)sizeof(UnitDesc);
    static constexpr int oZero = oX + kXSlots * kXSlotBytes;
    static constexpr int oOpRing = oZero + kZeroBytes;               // GemvOp[kOpRing]
    static constexpr int oOpBuf = oOpRing + kOpRing * kOpBytes;   // GemvOp[2] producer, GemvOp[2] per x-prep warp
    static constexpr int oOutData = oOpBuf + (2 + 2 * kPrepWarps) * kOpBytes;   // float[kOutSlots][kOutFloats]
    static constexpr int oOutDesc = oOutData + kOutSlots * kOutFloats * 4;     // OutDesc[kOutSlots]
    static constexpr int oBars = oOutDesc + kOutSlots * (int)sizeof(OutDesc);  // full[S], empty[S]
    static constexpr int oReleased = oBars + 2 * kStages * 8;        // u32[S]: consumer warps that released a stage, ever
    static constexpr int oCtl = oReleased + kStages * 4;             // x_ready[XS], x_pending[XS], flags[2], prep_cmd, pad
    static constexpr int oOutCtl = oCtl + 64;                        // out_fill[kOutSlots], out_gen[kOutSlots]
    static constexpr int oXBars = (oOutCtl + 2 * kOutSlots * 4 + 16 + 7) / 8 * 8;   // (+ out_total) one mbarrier per activation slot
    static constexpr int kTotal = oXBars + 8 * kXSlots + 8;
    static_assert(kStages >= 4, "decode kernel: no room for a ring");
    static_assert(kOpRing >= kStages + 2, "an op's ring slot must outlive the units that refer to it");
    static_assert(kTotal <= 232448, "decode kernel: shared memory over the 227 KB per-CTA limit");
    static_assert(oBars % 8 == 0 && oXBars % 8 == 0, "mbarriers are 8-byte objects");
};

// K blobs (512 columns) per K chunk for a variant of which `bits` bits are read.
int gemv_chunk_blobs(int bits, int batch)
{
    const int cmax = batch <= 1 ? GemvCfg<1>::kBlobsMax : GemvCfg<8>::kBlobsMax;
    int c = kUnitBytes / blob_bytes(bits);
    if (c > cmax) c = cmax;
    if (c < 1) c = 1;
    return c;
}
static_assert(kUnitBytes >= kBlobMetaBytes + kBlobSteps * kBlobTiles * 512 * 8, "a unit must hold an 8-bit blob");

// A split-K partial is one 64-bit word per (row, batch entry): fp32 sum in the low half, launch tag in the high half.
size_t gemv_partial_bytes_per_unit(int batch) { return (batch <= 1 ? 32 : 256) * sizeof(unsigned long long); }

// D += A(u8, 16x32, row) * B(s8, 32x8, col), s32 accumulate.
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------------------- per-CTA work split
// (this kernel numbers the units of an op chunk-major, u = ch * n_rp + rp, and deals them with cta_range)
void gemv_cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi) { cta_range(n_units, rot, cta, grid, lo, hi); }

struct StackArgs {
    const GemvOp* table;                   // device op table (nullptr: use the by-value op)
    const long long* phase_total;          // units per phase
    unsigned long long* phase_done;        // finished units per phase
    unsigned* exit_count;
    const int* cta_units;                  // units of every CTA (nullptr: single op, computed on the device)
    int* status;
    int n_ops, n_phases;
    unsigned epoch;                        // tag of this launch's split-K partials (never 0)
};

// Warp-cooperative fetch of op descriptors with one op of look-ahead: the words of op i+1 travel
// while op i is processed.
struct OpFetch {
    uint32_t w0, w1;
    __device__ __forceinline__ void issue(const GemvOp* ops, int oi, int n_ops, int lane)
    {
        w0 = w1 = 0u;
        if (oi < n_ops) {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(ops + oi);
            if (lane < (int)(sizeof(GemvOp) / 4)) w0 = src[lane];
            if (lane + 32 < (int)(sizeof(GemvOp) / 4)) w1 = src[lane + 32];
        }
    }
    __device__ __forceinline__ void store(GemvOp* dst, int lane) const
    {
        uint32_t* d = reinterpret_cast<uint32_t*>(dst);
        if (lane < (int)(sizeof(GemvOp) / 4)) d[lane] = w0;
        if (lane + 32 < (int)(sizeof(GemvOp) / 4)) d[lane + 32] = w1;
    }
};
static_assert(sizeof(GemvOp) <= 256, "op descriptor too large for the two-word fetch");

// ------------------------------------------------------------------------------- the arithmetic of one unit
// Shared memory is addressed with 32-bit shared-window addresses and explicit ld.shared: the inner
// loops then carry no 64-bit pointer arithmetic.
// (OFF is a compile-time byte offset: it goes into the instruction's address field instead of costing an add)
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
// D = A(u8, 16x32, row) * B(s8, 32x8, col): first link of an accumulation chain (C = 0).
__device__ __forceinline__ void mma_u8s8_first(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

#ifndef FQ_GEMV_NA
#define FQ_GEMV_NA 1
#endif

// One field of width F (at bit SHIFT of the code) of TILES row tiles, one superstep: eight k32 steps, the
// first four belong to the first group of 128 columns, the last four to the second.  Adds (FIRSTF: stores),
// per tile / pass / row / group, the integer  2^SHIFT * sum_k field_k * x_int_k  into v.
//   fa     : shared address of this lane's 16-byte chunk in the first tile's field array
//   MAXB 1 : B columns (2t, 2t+1) carry the activation digits for bit-offset class t; lane (g, c) ends up
//            with the partial sum of class c, still scaled by 2^(c*F); xa[t] is the shared address of this
//            lane's B data for class t (or of zeros)
//   MAXB 8 : every register is shifted down to class 0; B columns (2b, 2b+1) carry batch entry
//            4*pass + b; xa[pass] is this lane's B data
// With one tile per warp and batch 1 the k32 steps of a group may alternate between FQ_GEMV_NA accumulators.
template <int F, int KEEP, int SHIFT, bool FIRSTF, int MAXB, int TILES>
__device__ __forceinline__ void field_step(uint32_t fa, const uint32_t (&xa)[4], uint32_t xoff, bool two_pass, int c,
                                           int (&v)[TILES][MAXB == 1 ? 1 : 2][2][2])
{
    constexpr int P = 8 / F;                                   // A registers stacked in one word
    constexpr uint32_t kMask = field_keep_mask(F, KEEP) * 0x01010101u;
    constexpr int NP = MAXB == 1 ? 1 : 2;
    constexpr int NA = (TILES == 1 && MAXB == 1) ? FQ_GEMV_NA : 1;   // accumulators per (tile, pass, group)
    int acc[TILES][NP][2][NA][4];

    static_for<0, F>([&](auto JB) {
        constexpr int jb = decltype(JB)::value;
        uint4 w[TILES], h[TILES];
        static_for<0, TILES>([&](auto TLI) {
            constexpr int tl = decltype(TLI)::value;
            w[tl] = lds128<tl * F * 512 + jb * 512>(fa);
            h[tl] = w[tl];                                     // F == 1: classes 4..7 come down by one shift
            if (F == 1 && MAXB == 1) h[tl] = make_uint4(w[tl].x >> 4, w[tl].y >> 4, w[tl].z >> 4, w[tl].w >> 4);
        });
        static_for<0, P>([&](auto TI) {
            constexpr int t = decltype(TI)::value;
            constexpr int j = P * jb + t;                      // k32 step inside the superstep
            constexpr int grp = j >> 2;
            [[maybe_unused]] constexpr int ai = (j & 3) % NA;
            constexpr bool first = (j & 3) < NA;               // first link of this accumulator's chain
            if constexpr (MAXB == 1) {
                constexpr int tc = (F == 1) ? (t & 3) : t;     // bit-offset class = B column pair
                constexpr uint32_t m = kMask << (tc * F);
                const uint2 x = lds64<j * 32>(xa[tc] + xoff);
#pragma unroll
                for (int tl = 0; tl < TILES; tl++) {
                    const uint4& a = (F == 1 && t >= 4) ? h[tl] : w[tl];
                    if (F == 8) {
                        if (first) mma_u8s8_first(acc[tl][0][grp][ai], a.x, a.y, a.z, a.w, x.x, x.y);
                        else mma_u8s8(acc[tl][0][grp][ai], a.x, a.y, a.z, a.w, x.x, x.y);
                    } else {
                        if (first) mma_u8s8_first(acc[tl][0][grp][ai], a.x & m, a.y & m, a.z & m, a.w & m, x.x, x.y);
                        else mma_u8s8(acc[tl][0][grp][ai], a.x & m, a.y & m, a.z & m, a.w & m, x.x, x.y);
                    }
                }
            } else {
                constexpr int sh = t * F;
                const uint2 x = lds64<j * 32>(xa[0] + xoff);
                uint2 x2 = make_uint2(0u, 0u);
                if (two_pass) x2 = lds64<j * 32>(xa[1] + xoff);
#pragma unroll
                for (int tl = 0; tl < TILES; tl++) {
                    const uint32_t a0 = (w[tl].x >> sh) & kMask, a1 = (w[tl].y >> sh) & kMask;
                    const uint32_t a2 = (w[tl].z >> sh) & kMask, a3 = (w[tl].w >> sh) & kMask;
                    if (first) {
                        mma_u8s8_first(acc[tl][0][grp][0], a0, a1, a2, a3, x.x, x.y);
                        if (two_pass) mma_u8s8_first(acc[tl][NP - 1][grp][0], a0, a1, a2, a3, x2.x, x2.y);
                        else if (NP > 1) {
#pragma unroll
                            for (int i = 0; i < 4; i++) acc[tl][NP - 1][grp][0][i] = 0;
                        }
                    } else {
                        mma_u8s8(acc[tl][0][grp][0], a0, a1, a2, a3, x.x, x.y);
                        if (two_pass) mma_u8s8(acc[tl][NP - 1][grp][0], a0, a1, a2, a3, x2.x, x2.y);
                    }
                }
            }
        });
    });
    // digits -> integer, undo the class scaling (exact: every term is a multiple of 2^(c*F)),
    // apply the field's position inside the code
    const int down = MAXB == 1 ? c * F : 0;
#pragma unroll
    for (int tl = 0; tl < TILES; tl++)
#pragma unroll
        for (int p = 0; p < NP; p++)
#pragma unroll
            for (int grp = 0; grp < 2; grp++) {
                int a[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    a[i] = acc[tl][p][grp][0][i];
#pragma unroll
                    for (int n = 1; n < NA; n++) a[i] += acc[tl][p][grp][n][i];
                }
                const int v0 = ((a[0] + (a[1] << 8)) >> down) << SHIFT, v1 = ((a[2] + (a[3] << 8)) >> down) << SHIFT;
                if (FIRSTF) { v[tl][p][0][grp] = v0; v[tl][p][1][grp] = v1; }      // the first field starts the sums
                else { v[tl][p][0][grp] += v0; v[tl][p][1][grp] += v1; }
            }
}

// The fields of one superstep, unrolled at compile time from the variant's field list.
template <int VARIANT, int FI, int PREFIX, int MAXB, int TILES>
struct FieldLoop {
    static __device__ __forceinline__ void run(uint32_t fbase, int st_tile, const uint32_t (&xa)[4], uint32_t xoff,
                                               bool two_pass, int c, int (&v)[TILES][MAXB == 1 ? 1 : 2][2][2])
    {
        constexpr FieldList FL = variant_fields(VARIANT);
        if constexpr (FI < FL.n) {
            constexpr int F = FL.width[FI], SHIFT = FL.shift[FI], KEEP = FL.keep[FI];
            // field array of width F after fields adding up to PREFIX bits; tile (superstep, row tile) = st_tile
            const uint32_t fa = fbase + kBlobSteps * kBlobTiles * 512 * PREFIX + st_tile * (F * 512);
            field_step<F, KEEP, SHIFT, FI == 0, MAXB, TILES>(fa, xa, xoff, two_pass, c, v);
            FieldLoop<VARIANT, FI + 1, PREFIX + F, MAXB, TILES>::run(fbase, st_tile, xa, xoff, two_pass, c, v);
        }
    }
};

// All supersteps of one unit for this warp's row tiles: tot[tile][pass][row half] += the dequantised dot products.
//   st    : shared address of the stage          cnt : supersteps in the unit (whole blobs)
//   xs    : shared address of the activation slot (digits, group sums, group scales)
template <int VARIANT, int MAXB, int TILES, class S>
__device__ __forceinline__ void unit_compute(uint32_t st, int cnt, int blob_read, uint32_t xs, uint32_t zero_page,
                                             int B, int lane, int tile0, float (&tot)[TILES][MAXB == 1 ? 1 : 2][2])
{
    constexpr int NP = MAXB == 1 ? 1 : 2;
    // a nested child reads the parent's top bits; the dropped bits are filled with their mid-point, which
    // is the same as lowering every zero point by that amount
    constexpr int kAdjust = (VARIANT >= 7 && VARIANT < 13) ? 1 << (7 - (VARIANT - 5)) : 0;
    const int g = lane >> 2, c = lane & 3;
    const bool two_pass = MAXB > 1 && B > 4;
    // this lane's B-operand sources.  B column n = g holds digit (g & 1) of
    //   batch 1: bit-offset class g >> 1            batch > 1: batch entry 4 * pass + (g >> 1)
    uint32_t xa[4];
    if (MAXB == 1) {
#pragma unroll
        for (int t = 0; t < 4; t++) xa[t] = (g >> 1) == t ? xs + (g & 1) * S::kDigitOff + c * 8 : zero_page + c * 8;
    } else {
#pragma unroll
        for (int p = 0; p < 2; p++) {
            const int b = 4 * p + (g >> 1);
            xa[p] = b < B ? xs + b * S::kXRow + (g & 1) * S::kDigitOff + c * 8 : zero_page + c * 8;
        }
        xa[2] = xa[3] = zero_page + c * 8;
    }
    const uint32_t xsum = xs + S::kXsumOff, xscale = xs + S::kXscaleOff;
    uint32_t blob = st;
    for (int s = 0; s < cnt; s += kBlobSteps, blob += blob_read) {
#ifdef FQ_GEMV_UNROLL_SSL
#pragma unroll
#else
#pragma unroll 1                                                             // (keeps the 14 specialised loops small)
#endif
        for (int ssl = 0; ssl < kBlobSteps; ssl++) {
            const int st_tile = ssl * kBlobTiles + tile0;
            int v[TILES][NP][2][2];
            FieldLoop<VARIANT, 0, 0, MAXB, TILES>::run(blob + kBlobMetaBytes + lane * 16, st_tile, xa, (s + ssl) * 256, two_pass, c, v);
            // group epilogue: y += s * 2^-e * (v - z * sum x_int)
            const uint32_t meta = blob + st_tile * 128 + g * 16;          // words of (group, row half) at + group * 8 + half * 4
            if constexpr (MAXB == 1) {
                // both groups' activation sums and scales in one load each; only the class-0 lane of a quad
                // subtracts the zero-point term
                const uint2 xs2 = lds64(xsum + (s + ssl) * 8), sc2 = lds64(xscale + (s + ssl) * 8);
                const int nx[2] = {c == 0 ? -(int)xs2.x : 0, c == 0 ? -(int)xs2.y : 0};
                const float sc[2] = {__uint_as_float(sc2.x), __uint_as_float(sc2.y)};
                static_for<0, TILES * 2>([&](auto I) {
                    constexpr int tl = decltype(I)::value / 2, grp = decltype(I)::value % 2;
                    const uint32_t m0 = lds32<tl * 128 + grp * 8>(meta);
                    const uint32_t m1 = lds32<tl * 128 + grp * 8 + 4>(meta);
                    const float s0 = __low2float(*reinterpret_cast<const __half2*>(&m0));
                    const float s1 = __low2float(*reinterpret_cast<const __half2*>(&m1));
                    // v - (z - adjust) * X  =  v + z * (-X) - adjust * (-X)
                    const int base = kAdjust ? -kAdjust * nx[grp] : 0;
                    const int t0 = v[tl][0][0][grp] + (int)(m0 >> 16) * nx[grp] + base;
                    const int t1 = v[tl][0][1][grp] + (int)(m1 >> 16) * nx[grp] + base;
                    tot[tl][0][0] = fmaf((float)t0, s0 * sc[grp], tot[tl][0][0]);
                    tot[tl][0][1] = fmaf((float)t1, s1 * sc[grp], tot[tl][0][1]);
                });
            } else {
#pragma unroll
                for (int tl = 0; tl < TILES; tl++) {
#pragma unroll
                    for (int grp = 0; grp < 2; grp++) {
                        const uint32_t m0 = lds32(meta + tl * 128 + grp * 8);
                        const uint32_t m1 = lds32(meta + tl * 128 + grp * 8 + 4);
                        const float s0 = __low2float(*reinterpret_cast<const __half2*>(&m0));
                        const float s1 = __low2float(*reinterpret_cast<const __half2*>(&m1));
                        const int z0 = (int)(m0 >> 16) - kAdjust;
                        const int z1 = (int)(m1 >> 16) - kAdjust;
#pragma unroll
                        for (int p = 0; p < NP; p++) {
                            const int b = 4 * p + c;
                            const bool has = b < B;
                            const uint32_t gi = (uint32_t)(b * (S::kCMax * 2) + (s + ssl) * 2 + grp) * 4u;
                            const int xsm = has ? (int)lds32(xsum + gi) : 0;
                            const float scb = has ? __uint_as_float(lds32(xscale + gi)) : 0.f;
                            tot[tl][p][0] = fmaf((float)(v[tl][p][0][grp] - z0 * xsm), s0 * scb, tot[tl][p][0]);
                            tot[tl][p][1] = fmaf((float)(v[tl][p][1][grp] - z1 * xsm), s1 * scb, tot[tl][p][1]);
                        }
                    }
                }
            }
        }
    }
}

template <int MAXB, int TILES, class S>
__device__ __forceinline__ void unit_dispatch(int variant, uint32_t st, int cnt, int blob_read, uint32_t xs, uint32_t zero_page,
                                              int B, int lane, int tile0, float (&tot)[TILES][MAXB == 1 ? 1 : 2][2])
{
#define FQ_VARIANT_CASE(V) case V: unit_compute<V, MAXB, TILES, S>(st, cnt, blob_read, xs, zero_page, B, lane, tile0, tot); break;
    switch (variant) {
        FQ_VARIANT_CASE(0) FQ_VARIANT_CASE(1) FQ_VARIANT_CASE(2) FQ_VARIANT_CASE(3) FQ_VARIANT_CASE(4)
        FQ_VARIANT_CASE(5) FQ_VARIANT_CASE(6) FQ_VARIANT_CASE(7) FQ_VARIANT_CASE(8) FQ_VARIANT_CASE(9)
        FQ_VARIANT_CASE(10) FQ_VARIANT_CASE(11) FQ_VARIANT_CASE(12) FQ_VARIANT_CASE(13)
        default: break;
    }
#undef FQ_VARIANT_CASE
    static_assert(kVariants == 14, "one case per variant");
}

template <int MAXB>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const __grid_constant__ GemvOp single, const StackArgs sa)
{
    using S = GemvSmem<MAXB>;
    constexpr int NP = MAXB == 1 ? 1 : 2;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bars = smem_u32(smem + S::oBars);                          // full[0..S), empty[0..S)
    volatile unsigned* released = reinterpret_cast<volatile unsigned*>(smem + S::oReleased);
    volatile int* x_ready = reinterpret_cast<volatile int*>(smem + S::oCtl);   // segment number + 1 held by a slot
    const uint32_t xbars = smem_u32(smem + S::oXBars);                         // completes a phase per publication of a slot
    volatile int* x_pending = x_ready + kXSlots;                               // units that still need the slot
    volatile int* flags = x_pending + kXSlots;                                 // [0]: stop computing, [1]: stop everything
    volatile int* prep_cmd = flags + 2;                                        // decision shared by the pre-processing warps
    volatile unsigned* out_fill = reinterpret_cast<volatile unsigned*>(smem + S::oOutCtl);   // consumer warps that filled a slot
    volatile unsigned* out_gen = out_fill + S::kOutSlots;                         // times the output warp drained a slot
    volatile int* out_total = reinterpret_cast<volatile int*>(out_gen + S::kOutSlots);   // finishing units of this CTA (-1: not known yet)

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; s++) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (S::kStages + s), kWarpsPerUnit);
            released[s] = 0u;
        }
        for (int i = 0; i < kXSlots; i++) { x_ready[i] = 0; x_pending[i] = 0; mbar_init(xbars + 8 * i, 1); }
        for (int i = 0; i < S::kOutSlots; i++) { out_fill[i] = 0u; out_gen[i] = 0u; }
        out_total[0] = -1;
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < S::kZeroBytes / 4; i += blockDim.x)
        reinterpret_cast<uint32_t*>(smem + S::oZero)[i] = 0u;
    __syncthreads();

    const int grid = gridDim.x, cta = blockIdx.x;
    const GemvOp* ops = sa.table ? sa.table : &single;

    if (warp == kProducerWarp) {
        // ================================================================== producer (one warp)
        // Lane 0 owns the barriers; lanes 0 .. 2*n_fields+1 each issue one bulk copy per unit.
        GemvOp* opbuf = reinterpret_cast<GemvOp*>(smem + S::oOpBuf);
        uint8_t* opring = smem + S::oOpRing;
        OpFetch fetch;
        fetch.issue(ops, 0, sa.n_ops, lane);
        fetch.store(&opbuf[0], lane);
        __syncwarp();
        int stage = 0;                               // ring position and how often the ring wrapped (32-bit state only:
        unsigned wraps = 0;                          // this loop is the serial bottleneck of the CTA)
        int seg = -1, op_seq = -1;
        int oseq = 0;                                // finishing units issued so far
        bool stop = false;
        for (int oi = 0; oi < sa.n_ops && !stop; oi++) {
            const OpFetch cur = fetch;                                // the words of this op, still in registers
            fetch.issue(ops, oi + 1, sa.n_ops, lane);                 // travels while this op is issued
            const GemvOp& op = opbuf[oi & 1];
            int lo, hi;
            cta_range(op.n_units, op.rot, cta, grid, lo, hi);
            if (lo < hi) {
                op_seq++;
                const int op_slot = op_seq % kOpRing;
                cur.store(reinterpret_cast<GemvOp*>(opring + op_slot * S::kOpBytes), lane);   // for the consumers
                __threadfence_block();
                __syncwarp();          // all 32 lanes' words are in place before lane 0 announces the first unit
                // a PACKED variant's blobs are contiguous: one copy per unit (lane 0); a nested child reads a
                // prefix of every blob: one copy per blob (lanes 0 .. nb-1).
                // Everything the unit loop needs sits in registers and is advanced by additions: this loop
                // is the serial path that feeds the whole CTA.
                const int n_rp = op.n_rp, n_kb = op.n_kb, chunk_blobs = op.chunk_blobs, n_chunks = op.n_chunks;
                const uint32_t blob_read = (uint32_t)op.blob_read;
                const long long blob_stride = op.blob_stride;
                const uint8_t* store = op.store;
                const bool contiguous = op.blob_read == op.blob_stride;
                const long long rp_stride = (long long)n_kb * blob_stride;
                int ch = lo / n_rp, rp = lo - ch * n_rp;
                int rpm = rp % n_chunks;                             // rp mod n_chunks, kept up by counting
                int n_left = hi - lo;
                while (n_left > 0 && !stop) {
                    // ---- the units of one K chunk
                    seg++;
                    const int kb0 = ch * chunk_blobs;
                    const int nb = min(chunk_blobs, n_kb - kb0);
                    const uint32_t bytes = (uint32_t)nb * blob_read;
                    const uint8_t* src = store + ((long long)rp * n_kb + kb0) * blob_stride;
                    const int in_chunk = min(n_left, n_rp - rp);
                    for (int i = 0; i < in_chunk; i++) {
                        const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
                        int ok = 1;
                        if (lane == 0) {
                            if (wraps > 0 && !mbar_try_wait(empty, (wraps - 1u) & 1u)) {
                                // the ring is full: the usual case when the consumers wait for activations
                                if (flags[1]) ok = 0;
                                else if (!mbar_wait(empty, (wraps - 1u) & 1u)) {
                                    atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT);
                                    flags[0] = 1; flags[1] = 1;
                                    ok = 0;
                                }
                            }
                            if (ok) {
                                // the chunk that adds up a row pair rotates with the row pair, so that this work
                                // (and the place in the output queue it needs) is spread evenly over the CTAs
                                int4* d = reinterpret_cast<int4*>(smem + S::oDesc + stage * (int)sizeof(UnitDesc));
                                d[0] = make_int4(ch, rp, nb, seg);
                                d[1] = make_int4(op_slot, ch == rpm ? oseq : -1, 0, 0);
                                mbar_expect_tx(full, bytes);
                            }
                        }
                        ok = __shfl_sync(0xffffffffu, ok, 0);
                        if (!ok) { stop = true; break; }
                        const uint32_t stage_base = smem_u32(smem + S::oStages) + (uint32_t)stage * S::kStageBytes;
                        // (checked build) the blobs of this copy lie inside the stored variant and fit the stage; the
                        // transaction stays pending, the status word ends every wait
                        if (!FQ_IN_BOUNDS(rp >= 0 && rp < n_rp && kb0 >= 0 && kb0 + nb <= n_kb && bytes <= (uint32_t)S::kStageBytes,
                                          sa.status)) {
                            if (lane == 0) { flags[0] = 1; flags[1] = 1; }
                            stop = true;
                            break;
                        }
                        if (contiguous) {
                            if (lane == 0) bulk_g2s(stage_base, src, bytes, full);
                        } else if (lane < nb) {
                            bulk_g2s(stage_base + lane * blob_read, src + lane * blob_stride, blob_read, full);
                        }
                        if (ch == rpm) oseq++;
                        if (++rpm == n_chunks) rpm = 0;
                        if (++stage == S::kStages) { stage = 0; wraps++; }
                        rp++;
                        src += rp_stride;
                    }
                    n_left -= in_chunk;
                    rp = 0; rpm = 0; ch++;
                }
                if (lane == 0 && flags[1]) stop = true;
                stop = __shfl_sync(0xffffffffu, stop ? 1 : 0, 0) != 0;
            }
            __syncwarp();
            fetch.store(&opbuf[(oi + 1) & 1], lane);
            __syncwarp();
        }
        if (lane == 0 && !stop) out_total[0] = oseq;                // the output warp may leave after this many
    } else if (warp >= kPrepWarp && warp < kPrepWarp + kPrepWarps) {
        // ================================================================== activation pre-processing
        // All pre-processing warps walk the same list of (op, K chunk) segments and split the
        // (batch row, superstep) items of each segment among them; named barrier 1 keeps them in step.
        const int pw = warp - kPrepWarp;
        GemvOp* opbuf = reinterpret_cast<GemvOp*>(smem + S::oOpBuf) + 2 + 2 * pw;
        OpFetch fetch;
        fetch.issue(ops, 0, sa.n_ops, lane);
        fetch.store(&opbuf[0], lane);
        __syncwarp();
        int seg = -1;
        int phase_known = -1;                       // every phase <= phase_known is complete
        bool stop = false;
        for (int oi = 0; oi < sa.n_ops && !stop; oi++) {
            if (oi > 0) {
                __syncwarp();
                fetch.store(&opbuf[oi & 1], lane);
                __syncwarp();
            }
            fetch.issue(ops, oi + 1, sa.n_ops, lane);                 // travels while this op is processed
            const GemvOp& op = opbuf[oi & 1];
            int lo, hi;
            cta_range(op.n_units, op.rot, cta, grid, lo, hi);
            if (lo >= hi) continue;
            const int ch_lo = lo / op.n_rp, ch_hi = (hi - 1) / op.n_rp;
            for (int ch = ch_lo; ch <= ch_hi && !stop; ch++) {
                seg++;
                const int units = min(hi, (ch + 1) * op.n_rp) - max(lo, ch * op.n_rp);
                const int slot = seg % kXSlots;
                uint8_t* xs = smem + S::oX + slot * S::kXSlotBytes;
                if (pw == 0 && lane == 0) {
                    // the slot is free when every unit of the segment that used it before is done
                    if (!smem_wait([&] { return x_pending[slot] == 0 || flags[1]; })) {
                        atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1;
                    }
                    // the activations are the previous phase's outputs
                    if (!flags[0] && op.phase > 0 && phase_known < op.phase - 1) {
                        const unsigned long long need = (unsigned long long)sa.phase_total[op.phase - 1];
                        const unsigned long long t0 = global_ns();
                        unsigned it = 0;
                        while (ld_acquire_u64(sa.phase_done + (op.phase - 1)) < need) {
                            if ((++it & 63u) == 0u &&
                                (global_ns() - t0 > kWaitLimitNs || *reinterpret_cast<volatile int*>(sa.status) != 0 ||
                                 flags[0])) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; break; }
                        }
                    }
                    prep_cmd[0] = flags[1] ? 0 : (flags[0] ? 2 : 1);   // one decision for all pre-processing warps
                    __threadfence_block();
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kPrepWarps * 32) : "memory");
                const int go = prep_cmd[0];                            // 0: stop, 1: compute, 2: publish without computing
                if (op.phase > 0) phase_known = op.phase - 1;          // (meaningless after an abort; unused then)
                if (go == 0) { stop = true; break; }
                if (go == 1) {
                    const int ss0 = ch * op.chunk_blobs * kBlobSteps;
                    const int cnt = min(op.chunk_blobs, op.n_kb - ch * op.chunk_blobs) * kBlobSteps;
                    int* xsum = reinterpret_cast<int*>(xs + S::kXsumOff);
                    float* xscale = reinterpret_cast<float*>(xs + S::kXscaleOff);
                    const int n_items = cnt * op.batch;                // item = (batch row, superstep)
                    for (int i0 = pw; i0 < n_items; i0 += 4 * kPrepWarps) {
                        uint4 raw[4];                                  // all loads of up to four items first
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            raw[q] = make_uint4(0u, 0u, 0u, 0u);
                            const int item = i0 + q * kPrepWarps;
                            if (item < n_items) {
                                const int b = item / cnt, s_ = item % cnt;
                                const int k = (ss0 + s_) * kStepCols + lane * 8;   // this lane: 8 columns of the superstep
                                if (k < op.k_in)
                                    raw[q] = __ldcg(reinterpret_cast<const uint4*>(
                                        reinterpret_cast<const __half*>(op.x) + (long long)b * op.k_in + k));
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            const int item = i0 + q * kPrepWarps;
                            if (item >= n_items) break;
                            const int b = item / cnt, s_ = item % cnt;
                            const __half2* h2 = reinterpret_cast<const __half2*>(&raw[q]);
                            float f[8];
#pragma unroll
                            for (int i = 0; i < 4; i++) {
                                const float2 t2 = __half22float2(h2[i]);
                                f[2 * i] = t2.x; f[2 * i + 1] = t2.y;
                            }
                            float amax = 0.f;
#pragma unroll
                            for (int i = 0; i < 8; i++) amax = fmaxf(amax, fabsf(f[i]));
#pragma unroll
                            for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
                            // group of 128 columns = 16 lanes.  x_int = rint(x * 2^(13 - E)), 2^E <= amax < 2^(E+1)
                            const int eb = (__float_as_int(amax) >> 23) & 0xff;       // biased exponent of amax
                            const bool fin = amax > 0.f && eb < 255;
                            const float mult = fin ? __int_as_float((267 - eb) << 23) : 0.f;
                            const float back = fin ? __int_as_float((eb - 13) << 23) : 0.f;
                            int xi[8], sum = 0;
#pragma unroll
                            for (int i = 0; i < 8; i++) { xi[i] = __float2int_rn(f[i] * mult); sum += xi[i]; }
#pragma unroll
                            for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                            // signed digits base 256 of four values at a time: low byte as is, high byte + carry
                            uint32_t lo4[2], hi4[2];
#pragma unroll
                            for (int r = 0; r < 2; r++) {
                                const uint32_t p01 = __byte_perm((uint32_t)xi[4 * r + 0], (uint32_t)xi[4 * r + 1], 0x5410);
                                const uint32_t p23 = __byte_perm((uint32_t)xi[4 * r + 2], (uint32_t)xi[4 * r + 3], 0x5410);
                                const uint32_t h01 = (((p01 >> 8) & 0x00ff00ffu) + ((p01 >> 7) & 0x00010001u)) & 0x00ff00ffu;
                                const uint32_t h23 = (((p23 >> 8) & 0x00ff00ffu) + ((p23 >> 7) & 0x00010001u)) & 0x00ff00ffu;
                                lo4[r] = __byte_perm(p01, p23, 0x6420);
                                hi4[r] = __byte_perm(h01, h23, 0x6420);
                            }
                            // B-fragment order: per k32 step 32 bytes = [c][k 4c..4c+3 | k 16+4c..16+4c+3]
                            const int j = lane >> 2, q4 = lane & 3;
                            const int half = q4 >> 1, c0 = 2 * (q4 & 1);
                            uint8_t* row = xs + b * S::kXRow + s_ * 256 + j * 32 + half * 4;
                            *reinterpret_cast<uint32_t*>(row + c0 * 8) = lo4[0];
                            *reinterpret_cast<uint32_t*>(row + (c0 + 1) * 8) = lo4[1];
                            *reinterpret_cast<uint32_t*>(row + S::kDigitOff + c0 * 8) = hi4[0];
                            *reinterpret_cast<uint32_t*>(row + S::kDigitOff + (c0 + 1) * 8) = hi4[1];
                            if ((lane & 15) == 0) {
                                xsum[b * (S::kCMax * 2) + s_ * 2 + (lane >> 4)] = sum;
                                xscale[b * (S::kCMax * 2) + s_ * 2 + (lane >> 4)] = back;
                            }
                        }
                    }
                }
                __threadfence_block();
                asm volatile("bar.sync 1, %0;" ::"n"(kPrepWarps * 32) : "memory");
                if (pw == 0 && lane == 0) {
                    x_pending[slot] = units * kWarpsPerUnit;
                    __threadfence_block();
                    x_ready[slot] = seg + 1;
                    __threadfence_block();
                    mbar_arrive(xbars + 8 * slot);                     // wakes the consumers that sleep on this slot
                }
            }
        }
    } else if (warp == kOutputWarp) {
        // ================================================================== output warp
        // Finishes row pairs.  The unit whose K chunk is (row pair mod chunks) adds up its row pair: its own
        // sums arrive through the queue in shared memory, the other chunks' sums are tagged 64-bit words in
        // global memory (value, launch tag) that their consumers stored without any fence -- a word counts
        // once its tag is this launch's.  The sums are added in chunk order, so results do not depend on
        // timing.  One fence per batch of finished row pairs orders y before the phase counter.
        constexpr int BW = MAXB == 1 ? 1 : 8;                            // result floats per row
        const float* odata = reinterpret_cast<const float*>(smem + S::oOutData);
        const OutDesc* odesc = reinterpret_cast<const OutDesc*>(smem + S::oOutDesc);
        int processed = 0;
        unsigned long long last_progress = 0ull;
        unsigned idle_it = 0u;
        for (;;) {
            // every decision that ends the loop is taken by lane 0 and broadcast: the lanes must leave together
            const bool filled = lane < S::kOutSlots && out_fill[lane] == (unsigned)kWarpsPerUnit;
            const unsigned m = __ballot_sync(0xffffffffu, filled);
            unsigned done = 0u;
            if (m) {
                __threadfence_block();                                   // the slots' contents after their fill counts
                for (unsigned mm = m; mm; mm &= mm - 1u) {
                    const int s = __ffs(mm) - 1;
                    const OutDesc& d = odesc[s];
                    const float* o = odata + s * S::kOutFloats;
                    // a few chunks per round trip, every batch entry of them in flight at once; a round whose
                    // words are not all there ends the attempt
                    constexpr int QS = MAXB == 1 ? 24 : 2;
                    float sum[BW];
#pragma unroll
                    for (int i = 0; i < BW; i++) sum[i] = 0.f;
                    bool ok = true;
                    const unsigned long long* pt = d.partial + (long long)d.rp * d.n_chunks * (32 * BW) + lane;
                    for (int q0 = 0; q0 < d.n_chunks; q0 += QS) {
                        unsigned long long w[QS][BW];
#pragma unroll
                        for (int j = 0; j < QS; j++) {
                            const int q = q0 + j;
#pragma unroll
                            for (int i = 0; i < BW; i++) {                // element e = lane + 32 i = local row * BW + batch entry
                                w[j][i] = 0ull;
                                if (q < d.n_chunks && q != d.ch) w[j][i] = ld_relaxed_u64(pt + (long long)q * (32 * BW) + 32 * i);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < QS; j++) {
                            const int q = q0 + j;
                            if (q >= d.n_chunks) break;
#pragma unroll
                            for (int i = 0; i < BW; i++) {
                                if (q == d.ch) sum[i] += o[lane + 32 * i];
                                else {
                                    ok = ok && (unsigned)(w[j][i] >> 32) == sa.epoch;
                                    sum[i] += __uint_as_float((unsigned)w[j][i]);
                                }
                            }
                        }
                        if (!__all_sync(0xffffffffu, ok)) break;
                    }
                    if (!__all_sync(0xffffffffu, ok)) continue;          // some chunk has not arrived yet: look again later
                    const int row_base = d.rp * (kUnitRowTiles * kTileRows);
                    __half* y = reinterpret_cast<__half*>(d.y);
#pragma unroll
                    for (int i = 0; i < BW; i++) {
                        const int e = lane + 32 * i;
                        const int row = row_base + e / BW, b = e % BW;
                        if (row < d.n_out && b < d.batch) y[(long long)b * d.n_out + row] = __float2half_rn(sum[i]);
                    }
                    done |= 1u << s;
                }
            }
            if (done) {
                __syncwarp();
                __threadfence();                                         // y before the phase counter
                if ((done >> lane) & 1u) {
                    const int phase = odesc[lane].phase;
                    if (phase >= 0) red_add_relaxed_u64(sa.phase_done + phase, 1ull);
                    out_fill[lane] = 0u;                                 // hand the slot back
                    __threadfence_block();
                    out_gen[lane] = out_gen[lane] + 1u;
                }
                processed += __popc(done);
                last_progress = 0ull; idle_it = 0u;
                continue;
            }
            int leave = 0;
            if (lane == 0) {
                const int want = out_total[0];
                if (flags[0] || (want >= 0 && processed >= want)) leave = 1;
                else if ((++idle_it & 127u) == 0u) {
                    const unsigned long long now = global_ns();
                    if (last_progress == 0ull) last_progress = now;
                    else if (now - last_progress > kWaitLimitNs) {
                        atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1;
                        leave = 1;
                    }
                }
            }
            if (__shfl_sync(0xffffffffu, leave, 0)) break;
            __nanosleep(20);
        }
    } else {
        // ================================================================== consumers
        // kWarpsPerUnit warps share a unit, each computes kTilesPerWarp of its two 16-row tiles.
        const int g = lane >> 2, c = lane & 3;
        const int uidx = warp / kWarpsPerUnit;                       // which of the units in flight
        const int tile0 = (warp % kWarpsPerUnit) * kTilesPerWarp;    // first row tile of this warp
        constexpr int TL = kTilesPerWarp;
        int total = 0;                               // units of this CTA over the whole launch
        if (sa.cta_units) total = sa.cta_units[cta];
        else {
            int lo, hi;
            cta_range(single.n_units, single.rot, cta, grid, lo, hi);
            total = hi - lo;
        }
        const uint8_t* opring = smem + S::oOpRing;
        float* odata = reinterpret_cast<float*>(smem + S::oOutData);
        OutDesc* odesc = reinterpret_cast<OutDesc*>(smem + S::oOutDesc);
        bool stop = false;
        // ring position of this warp's next unit, advanced by additions
        int stage = uidx % S::kStages;
        unsigned use = (unsigned)(uidx / S::kStages);
        const uint32_t opring_a = smem_u32(smem + S::oOpRing), desc_a = smem_u32(smem + S::oDesc);
        for (int seq = uidx; seq < total && !stop; seq += kUnitsInFlight) {
            const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
            // a stage's uses are consumed strictly in order: wait for the release of the previous
            // use before trusting the parity of the full barrier
            bool ok = true;
            if (use > 0) ok = smem_wait([&] { return released[stage] >= use * kWarpsPerUnit || flags[1]; });
            if (ok) ok = mbar_wait(full, use & 1u);
            if (!ok || flags[1]) {
                if (lane == 0 && !ok) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1; }
                stop = true;
                break;
            }
            struct { int ch, rp, cnt, seg, blob_read, variant, batch, op_slot, oseq, n_chunks;
                     unsigned long long* partial; } d;
            {
                const uint4 u0 = lds128(desc_a + stage * (int)sizeof(UnitDesc));            // ch, rp, nb, seg
                const uint2 u1 = lds64(desc_a + stage * (int)sizeof(UnitDesc) + 16);        // op_slot, oseq
                const uint32_t od = opring_a + u1.x * S::kOpBytes;
                const uint4 o1 = lds128(od + 16);                                           // blob_read, variant, batch, n_chunks
                const uint2 o0 = lds64(od + 8);                                             // partial
                d.ch = (int)u0.x; d.rp = (int)u0.y; d.cnt = (int)u0.z * kBlobSteps; d.seg = (int)u0.w;
                d.op_slot = (int)u1.x; d.oseq = (int)u1.y;
                d.blob_read = (int)o1.x; d.variant = (int)o1.y; d.batch = (int)o1.z; d.n_chunks = (int)o1.w;
                d.partial = reinterpret_cast<unsigned long long*>(((unsigned long long)o0.y << 32) | o0.x);
            }
            // a unit that finishes its row pair needs a place in the output queue: that place must be free
            // again; the descriptor goes there now, while the op's slot in the op ring is certainly still valid
            const int oslot = d.oseq % S::kOutSlots;
            if (d.oseq >= 0) {
                const unsigned ogen = (unsigned)(d.oseq / S::kOutSlots);
                if (!smem_wait([&] { return out_gen[oslot] == ogen || flags[1]; })) {
                    if (lane == 0) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1; }
                    stop = true;
                    break;
                }
                if (flags[1]) { stop = true; break; }
                if (tile0 == 0 && lane == 0) {
                    const GemvOp& od = *reinterpret_cast<const GemvOp*>(opring + d.op_slot * S::kOpBytes);
                    OutDesc& q = odesc[oslot];
                    q.rp = d.rp; q.ch = d.ch; q.n_chunks = od.n_chunks; q.n_out = od.n_out; q.phase = od.phase; q.batch = od.batch;
                    q.y = od.y; q.partial = od.partial;
                }
            }
            const int slot = d.seg % kXSlots;
            // sleep on the slot's barrier (a hardware wake-up: this wait is on the critical path of every
            // dependency phase); the flag has the last word, because a warp that is several publications
            // ahead would read a stale parity
            if (x_ready[slot] != d.seg + 1 && !flags[1]) mbar_wait(xbars + 8 * slot, (unsigned)(d.seg / kXSlots) & 1u);
            if (!smem_wait([&] { return x_ready[slot] == d.seg + 1 || flags[1]; })) {
                if (lane == 0) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; }
            }
            __threadfence_block();
            __syncwarp();
            const bool live = !flags[0];

            float tot[TL][NP][2];
#pragma unroll
            for (int i = 0; i < TL * NP * 2; i++) (&tot[0][0][0])[i] = 0.f;

            if (live)
                unit_dispatch<MAXB, TL, S>(d.variant, smem_u32(smem + S::oStages) + (uint32_t)stage * S::kStageBytes, d.cnt,
                                           d.blob_read, smem_u32(smem + S::oX) + (uint32_t)slot * S::kXSlotBytes,
                                           smem_u32(smem + S::oZero), d.batch, lane, tile0, tot);
            __syncwarp();
            if (lane == 0) {
                atomicAdd(const_cast<unsigned*>(&released[stage]), 1u);
                __threadfence_block();
                mbar_arrive(empty);                              // the stage may be refilled
                atomicSub(const_cast<int*>(&x_pending[slot]), 1);   // one warp fewer needs the activation slot
            }
            stage += kUnitsInFlight;
            while (stage >= S::kStages) { stage -= S::kStages; use++; }
            if (!live) continue;

            if (MAXB == 1) {                                     // add up the bit-offset classes held by the quad
#pragma unroll
                for (int tl = 0; tl < TL; tl++)
#pragma unroll
                    for (int r = 0; r < 2; r++) {
                        float t = tot[tl][0][r];
                        t += __shfl_xor_sync(0xffffffffu, t, 1);
                        t += __shfl_xor_sync(0xffffffffu, t, 2);
                        tot[tl][0][r] = t;
                    }
            }

            // ---- the row sums: value (tile, pass, r) of lane (g, c) belongs to local row tile * 16 + g + 8 r,
            //      batch entry 0 (batch 1: every lane of the quad holds it) or 4 pass + c
            constexpr int BW = MAXB == 1 ? 1 : 8;
            if (d.oseq >= 0) {
                // this unit finishes its row pair: hand the sums to the output warp
                float* o = odata + oslot * S::kOutFloats;
#pragma unroll
                for (int tl = 0; tl < TL; tl++)
#pragma unroll
                    for (int p = 0; p < NP; p++)
#pragma unroll
                        for (int r = 0; r < 2; r++) {
                            const int lr = (tile0 + tl) * 16 + g + 8 * r;
                            if (MAXB == 1) { if (c == 0) o[lr] = tot[tl][0][r]; }
                            else o[lr * BW + 4 * p + c] = tot[tl][p][r];
                        }
                __threadfence_block();
                __syncwarp();
                if (lane == 0) atomicAdd(const_cast<unsigned*>(&out_fill[oslot]), 1u);
            } else {
                // another unit finishes it: publish tagged words (value, launch tag), fire and forget
                unsigned long long* pu = d.partial + ((long long)d.rp * d.n_chunks + d.ch) * (32 * BW);
                const unsigned long long tag = (unsigned long long)sa.epoch << 32;
#pragma unroll
                for (int tl = 0; tl < TL; tl++) {
                    if (MAXB == 1) {
                        if (c < 2) {                                 // lane c of the quad stores row g + 8 c
                            const float v = c == 0 ? tot[tl][0][0] : tot[tl][0][1];
                            st_relaxed_u64(pu + (tile0 + tl) * 16 + g + 8 * c, tag | __float_as_uint(v));
                        }
                    } else {
#pragma unroll
                        for (int p = 0; p < NP; p++)
#pragma unroll
                            for (int r = 0; r < 2; r++) {
                                const int lr = (tile0 + tl) * 16 + g + 8 * r;
                                st_relaxed_u64(pu + lr * BW + 4 * p + c, tag | __float_as_uint(tot[tl][p][r]));
                            }
                    }
                }
            }
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && sa.n_phases > 0) {
        __threadfence();
        const unsigned old = atomicAdd(sa.exit_count, 1u);
        if (old == gridDim.x - 1) {                    // last CTA out: counters back to zero
            for (int p = 0; p < sa.n_phases; p++) sa.phase_done[p] = 0ull;
            *sa.exit_count = 0u;
            __threadfence();
        }
    }
}

// ------------------------------------------------------------------------------- launchers
// The launch is always cooperative: a CTA that finishes a row pair waits (bounded) for sums that other
// CTAs produce, so all CTAs of the grid have to be resident together.
template <int MAXB>
static int launch_impl(Ctx* ctx, const GemvOp& single, const StackArgs& sa, long long total_units, cudaStream_t st)
{
    using S = GemvSmem<MAXB>;
    static bool configured[64] = {};
    if (ctx->device < 64 && !configured[ctx->device]) {
        FQ_CUDA_OK(cudaFuncSetAttribute(gemv_kernel<MAXB>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal));
        configured[ctx->device] = true;
    }
    long long blocks = ctx->sm_count;
    if (total_units < blocks) blocks = total_units;
    if (blocks < 1) return FQ_OK;
    void* args[] = {(void*)&single, (void*)&sa};
    FQ_CUDA_OK(cudaLaunchCooperativeKernel((const void*)gemv_kernel<MAXB>, dim3((unsigned)blocks), dim3(kGemvThreads),
                                           args, S::kTotal, st));
    return FQ_OK;
}

// Tag for the split-K partials of the next launch that uses the context's workspace.
static unsigned next_epoch(unsigned& e)
{
    if (++e == 0u) ++e;                        // 0 marks words that no launch has written
    return e;
}

int launch_gemv_single(Ctx* ctx, const GemvOp& op, cudaStream_t st)
{
    StackArgs sa{};
    sa.table = nullptr;
    sa.status = ctx->status_dev;
    sa.n_ops = 1;
    sa.n_phases = 0;
    sa.epoch = next_epoch(ctx->launch_epoch);
    const long long units = (long long)op.n_rp * op.n_chunks;
    return launch_impl<8>(ctx, op, sa, units, st);
}

int launch_gemv_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, int max_batch, cudaStream_t st)
{
    // counters live in the workspace head
    StackArgs sa{};
    sa.table = reinterpret_cast<const GemvOp*>(table_dev);
    sa.phase_total = reinterpret_cast<const long long*>(table_dev + (size_t)hdr.n_ops * sizeof(GemvOp));
    sa.cta_units = reinterpret_cast<const int*>(sa.phase_total + (hdr.n_phases > 0 ? hdr.n_phases : 1));
    sa.phase_done = reinterpret_cast<unsigned long long*>(ctx->ws);
    sa.exit_count = reinterpret_cast<unsigned*>(ctx->ws + 8 * 4096);
    sa.status = ctx->status_dev;
    sa.n_ops = hdr.n_ops;
    sa.n_phases = hdr.n_phases;
    sa.epoch = next_epoch(ctx->launch_epoch);
    GemvOp dummy{};
    (void)max_batch;
    return launch_impl<8>(ctx, dummy, sa, hdr.total_units, st);
}

}  // namespace fq

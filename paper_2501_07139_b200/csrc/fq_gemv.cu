// Decode path: fused dequantize-GEMV over tiled field arrays, batch 1..8.
//
// One persistent CTA per SM with three roles:
//   producer thread : streams "units" (32 output rows x one K chunk: every field array of the
//                     active variant plus the scale/zero words) from HBM into a shared-memory
//                     ring with bulk asynchronous copies (cp.async.bulk + mbarrier tx counts)
//                     and writes a small descriptor next to each stage;
//   x-prep warp     : once per (op, K chunk) that this CTA touches, waits -- bounded -- for the
//                     previous dependency phase, loads the activations of that chunk and turns
//                     them into 16-bit fixed point per group of 128 columns
//                     (x_int = rint(x * 2^e), |x_int| < 2^14, stored as two signed byte digits);
//   8 consumer warps: stored words become 8-bit mma.m16n8k32 A operands with ONE AND each (no
//                     shift: a word holds 8/f registers on top of each other, see fq_layout.cuh),
//                     the activation digits are the B operand, accumulation is exact in s32.
//                     At batch 1 the eight B columns carry (low digit, high digit) for up to
//                     four bit-offset classes, so no register ever has to be shifted.
//   Per group:  y += s * 2^-e * ( sum_fields 2^shift * sum_k field_k * x_int_k  -  z * sum_k x_int_k ).
// K chunks of one row pair are combined through fp32 partials in a workspace; the last arriver
// adds them in chunk order, so results do not depend on scheduling.
//
// A whole stack of layers runs as one launch.  Every op's units are dealt to the CTAs in
// contiguous, K-chunk-major blocks (a CTA needs the activations of one or two chunks only);
// the producer runs ahead across op boundaries because weights do not depend on activations.
// Every wait has a time limit; when one runs out the kernel records FQ_ERR_TIMEOUT, stops
// computing, drains its copies and returns.
#include <cuda_fp16.h>

#include "fq_internal.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

#ifndef FQ_GEMV_WARPS
#define FQ_GEMV_WARPS 10
#endif
#ifndef FQ_GEMV_UNIT_BYTES
#define FQ_GEMV_UNIT_BYTES 17408
#endif
constexpr int kConsumerWarps = FQ_GEMV_WARPS;
constexpr int kProducerWarp = kConsumerWarps;          // warp index of the producer
constexpr int kPrepWarp = kConsumerWarps + 1;          // first warp of the activation pre-processors
constexpr int kPrepWarps = 4;                          // they share the items of a segment
constexpr int kGemvThreads = (kConsumerWarps + 1 + kPrepWarps) * 32;
constexpr int kUnitBytes = FQ_GEMV_UNIT_BYTES;         // bytes of one unit (whole blobs), at most: 2 x 4-bit or 1 x 8-bit blob
constexpr int kXSlots = 4;                             // activation chunks kept in shared memory
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

template <int MAXB> struct GemvCfg;
template <> struct GemvCfg<1> { static constexpr int kBlobsMax = 3; };  // k blobs (512 columns) per chunk, at most
template <> struct GemvCfg<8> { static constexpr int kBlobsMax = 1; };

// What the producer tells the consumers: once per op a copy of the op descriptor in a ring ...
constexpr int kOpRing = 32;                            // > stages: an op slot outlives its last unit
// ... and once per unit (next to the stage that holds the unit's weights)
struct UnitDesc {
    int ch, rp, nb, seg, op_slot, pad[3];       // K chunk, row pair, blobs in the unit, activation segment, op ring slot
};
static_assert(sizeof(UnitDesc) == 32, "descriptor layout");

template <int MAXB> struct GemvSmem {
    static constexpr int kCMax = GemvCfg<MAXB>::kBlobsMax * kBlobSteps;     // supersteps per chunk, at most
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
    static constexpr int kFixed = kXSlots * kXSlotBytes + kZeroBytes + kOpRing * kOpBytes + (2 + 2 * kPrepWarps) * kOpBytes + 256;
    static constexpr int kPerStage = kStageBytes + (int)sizeof(UnitDesc) + 16 + 4;
    static constexpr int kAuto = (232448 - kFixed) / kPerStage;
    static constexpr int kStages = kAuto > 16 ? 16 : kAuto;
    static constexpr int oStages = 0;
    static constexpr int oDesc = oStages + kStages * kStageBytes;
    static constexpr int oX = oDesc + kStages * (int)sizeof(UnitDesc);
    static constexpr int oZero = oX + kXSlots * kXSlotBytes;
    static constexpr int oOpRing = oZero + kZeroBytes;               // GemvOp[kOpRing]
    static constexpr int oOpBuf = oOpRing + kOpRing * kOpBytes;   // GemvOp[2] producer, GemvOp[2] per x-prep warp
    static constexpr int oBars = oOpBuf + (2 + 2 * kPrepWarps) * kOpBytes;   // full[S], empty[S]
    static constexpr int oReleased = oBars + 2 * kStages * 8;        // u32[S]: uses of a stage that were released
    static constexpr int oCtl = oReleased + kStages * 4;             // x_ready[XS], x_pending[XS], flags[2]
    static constexpr int kTotal = oCtl + 64;
    static_assert(kStages >= 4, "decode kernel: no room for a ring");
    static_assert(kTotal <= 232448, "decode kernel: shared memory over the 227 KB per-CTA limit");
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

size_t gemv_partial_floats_per_unit(int batch) { return batch <= 1 ? 32 : 256; }

// ------------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait on an mbarrier phase.  Returns false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; i++)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > kWaitLimitNs) return false;
    }
}
// Bounded wait until a condition on shared-memory words written by another warp of this CTA holds.
template <typename Pred>
__device__ __forceinline__ bool smem_wait(Pred pred)
{
    if (pred()) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; i++) {
            if (pred()) return true;
            __nanosleep(20);
        }
        if (global_ns() - t0 > kWaitLimitNs) return false;
    }
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Counter updates that carry their own ordering instead of a separate membar: the release half makes
// this warp's earlier stores (ordered before it by __syncwarp) visible first, the acquire half orders
// the loads that follow.
__device__ __forceinline__ unsigned atom_add_acq_rel_u32(unsigned* p, unsigned v)
{
    unsigned old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void red_add_release_u64(unsigned long long* p, unsigned long long v)
{
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
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
// Units of an op are numbered chunk-major (u = ch * n_rp + rp) and dealt to the CTAs in contiguous
// blocks; the block boundaries rotate from op to op so that the remainders even out.
__host__ __device__ __forceinline__ void cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi)
{
    const unsigned c = (unsigned)((cta + grid - rot) % grid);
    lo = (int)((unsigned)n_units * c / (unsigned)grid);              // n_units * grid < 2^31 (checked on the host)
    hi = (int)((unsigned)n_units * (c + 1u) / (unsigned)grid);
}

void gemv_cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi) { cta_range(n_units, rot, cta, grid, lo, hi); }

struct StackArgs {
    const GemvOp* table;                   // device op table (nullptr: use the by-value op)
    const long long* phase_total;          // units per phase
    unsigned long long* phase_done;        // finished units per phase
    unsigned* exit_count;
    const int* cta_units;                  // units of every CTA (nullptr: single op, computed on the device)
    int* status;
    int n_ops, n_phases;
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

// ------------------------------------------------------------------------------- one field, one superstep
// Consumes field width F of up to two row tiles for one superstep: eight k32 steps, the first four
// belong to the first group of 128 columns, the last four to the second.  Adds, per tile / pass / row /
// group, the integer  2^shift * sum_k field_k * x_int_k  into v.
//   MAXB == 1 : B columns (2t, 2t+1) carry the digits for bit-offset class t, lane (g, c) ends up with
//               the partial sum of class c (still scaled by 2^(c*F)); xp[t] points at this lane's B
//               data for class t (or at zeros).
//   MAXB  > 1 : every register is shifted down to class 0; B columns (2b, 2b+1) carry batch entry
//               4*pass + b; xp[pass] points at this lane's B data.
template <int F, int MAXB>
__device__ __forceinline__ void field_step(const uint8_t* f0, const uint8_t* f1, bool two_tiles, bool two_pass,
                                           int lane, const uint8_t* const (&xp)[4], int xoff, int shift,
                                           int (&v)[2][2][2][2])
{
    constexpr int P = 8 / F;                                   // A registers stacked in one word
    constexpr uint32_t kMask = ((1u << F) - 1u) * 0x01010101u;
    constexpr int NP = MAXB == 1 ? 1 : 2;
    int acc[2][NP][2][4];
#pragma unroll
    for (int i = 0; i < 2 * NP * 2 * 4; i++) (&acc[0][0][0][0])[i] = 0;

#pragma unroll
    for (int jb = 0; jb < F; jb++) {
        const uint4 w0 = *reinterpret_cast<const uint4*>(f0 + jb * 512 + lane * 16);
        uint4 w1 = make_uint4(0u, 0u, 0u, 0u);
        if (two_tiles) w1 = *reinterpret_cast<const uint4*>(f1 + jb * 512 + lane * 16);
        uint4 h0 = w0, h1 = w1;                                // F == 1: classes 4..7 come down by one shift
        if (F == 1 && MAXB == 1) {
            h0 = make_uint4(w0.x >> 4, w0.y >> 4, w0.z >> 4, w0.w >> 4);
            h1 = make_uint4(w1.x >> 4, w1.y >> 4, w1.z >> 4, w1.w >> 4);
        }
#pragma unroll
        for (int t = 0; t < P; t++) {
            const int j = P * jb + t;                          // k32 step inside the superstep
            const int grp = j >> 2;
            if (MAXB == 1) {
                const int tc = (F == 1) ? (t & 3) : t;         // bit-offset class = B column pair
                const uint32_t m = kMask << (tc * F);
                const uint4& a = (F == 1 && t >= 4) ? h0 : w0;
                const uint4& b = (F == 1 && t >= 4) ? h1 : w1;
                const uint2 x = *reinterpret_cast<const uint2*>(xp[tc] + xoff + j * 32);
                mma_u8s8(acc[0][0][grp], a.x & m, a.y & m, a.z & m, a.w & m, x.x, x.y);
                mma_u8s8(acc[1][0][grp], b.x & m, b.y & m, b.z & m, b.w & m, x.x, x.y);
            } else {
                const int sh = t * F;
                const uint32_t a0 = (w0.x >> sh) & kMask, a1 = (w0.y >> sh) & kMask;
                const uint32_t a2 = (w0.z >> sh) & kMask, a3 = (w0.w >> sh) & kMask;
                const uint32_t b0 = (w1.x >> sh) & kMask, b1 = (w1.y >> sh) & kMask;
                const uint32_t b2 = (w1.z >> sh) & kMask, b3 = (w1.w >> sh) & kMask;
                const uint2 x = *reinterpret_cast<const uint2*>(xp[0] + xoff + j * 32);
                mma_u8s8(acc[0][0][grp], a0, a1, a2, a3, x.x, x.y);
                mma_u8s8(acc[1][0][grp], b0, b1, b2, b3, x.x, x.y);
                if (two_pass) {
                    const uint2 x2 = *reinterpret_cast<const uint2*>(xp[1] + xoff + j * 32);
                    mma_u8s8(acc[0][NP - 1][grp], a0, a1, a2, a3, x2.x, x2.y);
                    mma_u8s8(acc[1][NP - 1][grp], b0, b1, b2, b3, x2.x, x2.y);
                }
            }
        }
    }
    // digits -> integer, undo the class scaling (exact: every term is a multiple of 2^(c*F)),
    // apply the field's position inside the code
    const int down = MAXB == 1 ? (lane & 3) * F : 0;
#pragma unroll
    for (int tile = 0; tile < 2; tile++)
#pragma unroll
        for (int p = 0; p < NP; p++)
#pragma unroll
            for (int grp = 0; grp < 2; grp++) {
                const int* a = acc[tile][p][grp];
                v[tile][p][0][grp] += ((a[0] + (a[1] << 8)) >> down) << shift;
                v[tile][p][1][grp] += ((a[2] + (a[3] << 8)) >> down) << shift;
            }
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
    volatile int* x_pending = x_ready + kXSlots;                               // units that still need the slot
    volatile int* flags = x_pending + kXSlots;                                 // [0]: stop computing, [1]: stop everything
    volatile int* prep_cmd = flags + 2;                                        // decision shared by the pre-processing warps

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; s++) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (S::kStages + s), 1);
            released[s] = 0u;
        }
        for (int i = 0; i < kXSlots; i++) { x_ready[i] = 0; x_pending[i] = 0; }
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
                // prefix of every blob: one copy per blob (lanes 0 .. nb-1)
                const bool contiguous = op.blob_read == op.blob_stride;
                const int n_units = hi - lo;
                int ch = lo / op.n_rp, rp = lo % op.n_rp;
                bool new_chunk = true;
                int kb0 = 0, nb = 0;
                for (int iu = 0; iu < n_units; iu++) {
                    if (new_chunk) {
                        seg++;
                        kb0 = ch * op.chunk_blobs;
                        nb = min(op.chunk_blobs, op.n_kb - kb0);
                        new_chunk = false;
                    }
                    const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
                    int ok = 1;
                    if (lane == 0) {
                        if (flags[1]) ok = 0;
                        else if (wraps > 0 && !mbar_wait(empty, (wraps - 1u) & 1u)) {
                            atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT);
                            flags[0] = 1; flags[1] = 1;
                            ok = 0;
                        }
                        if (ok) {
                            UnitDesc* d = reinterpret_cast<UnitDesc*>(smem + S::oDesc) + stage;
                            d->ch = ch; d->rp = rp; d->nb = nb; d->seg = seg; d->op_slot = op_slot;
                            mbar_expect_tx(full, (uint32_t)(nb * op.blob_read));
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { stop = true; break; }
                    const uint32_t stage_base = smem_u32(smem + S::oStages + stage * S::kStageBytes);
                    const uint8_t* src = op.store + ((long long)rp * op.n_kb + kb0) * op.blob_stride;
                    if (contiguous) {
                        if (lane == 0) bulk_g2s(stage_base, src, nb * op.blob_read, full);
                    } else if (lane < nb) {
                        bulk_g2s(stage_base + lane * op.blob_read, src + (long long)lane * op.blob_stride, op.blob_read, full);
                    }
                    if (++stage == S::kStages) { stage = 0; wraps++; }
                    if (++rp == op.n_rp) { rp = 0; ch++; new_chunk = true; }
                }
            }
            __syncwarp();
            fetch.store(&opbuf[(oi + 1) & 1], lane);
            __syncwarp();
        }
    } else if (warp >= kPrepWarp) {
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
                            __nanosleep(40);
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
                    x_pending[slot] = units;
                    __threadfence_block();
                    x_ready[slot] = seg + 1;
                }
            }
        }
    } else {
        // ================================================================== consumers
        const int g = lane >> 2, c = lane & 3;
        const uint8_t* zero_page = smem + S::oZero + c * 8;
        int total = 0;                               // units of this CTA over the whole launch
        if (sa.cta_units) total = sa.cta_units[cta];
        else {
            int lo, hi;
            cta_range(single.n_units, single.rot, cta, grid, lo, hi);
            total = hi - lo;
        }
        const uint8_t* opring = smem + S::oOpRing;
        bool stop = false;
        {
            for (int seq = warp; seq < total && !stop; seq += kConsumerWarps) {
                if (flags[1]) { stop = true; break; }
                const int stage = seq % S::kStages;
                const unsigned use = (unsigned)(seq / S::kStages);
                const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
                // a stage's uses are consumed strictly in order: wait for the release of the previous
                // use before trusting the parity of the full barrier
                bool ok = true;
                if (use > 0) ok = smem_wait([&] { return released[stage] >= use || flags[1]; });
                if (ok && !flags[1]) ok = mbar_wait(full, use & 1u);
                if (!ok || flags[1]) {
                    if (lane == 0 && !ok) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1; }
                    stop = true;
                    break;
                }
                struct { int ch, rp, cnt, seg, n_out, n_chunks, blob_read, n_fields, phase, zero_adjust, batch;
                         uint16_t* y; float* partial; unsigned* tile_count; uint8_t width[8], shift[8]; } d;
                {
                    const UnitDesc ud = *(reinterpret_cast<const UnitDesc*>(smem + S::oDesc) + stage);
                    const GemvOp& od = *reinterpret_cast<const GemvOp*>(opring + ud.op_slot * S::kOpBytes);
                    d.ch = ud.ch; d.rp = ud.rp; d.cnt = ud.nb * kBlobSteps; d.seg = ud.seg;
                    d.n_out = od.n_out; d.n_chunks = od.n_chunks; d.blob_read = od.blob_read; d.n_fields = od.n_fields;
                    d.phase = od.phase; d.zero_adjust = od.zero_adjust; d.batch = od.batch;
                    d.y = od.y; d.partial = od.partial; d.tile_count = od.tile_count;
#pragma unroll
                    for (int i = 0; i < kMaxFields; i++) { d.width[i] = od.field_width[i]; d.shift[i] = od.field_shift[i]; }
                }
                const uint8_t* st = smem + S::oStages + stage * S::kStageBytes;
                const int slot = d.seg % kXSlots;
                if (!smem_wait([&] { return x_ready[slot] == d.seg + 1 || flags[1]; })) {
                    if (lane == 0) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; }
                }
                __threadfence_block();
                __syncwarp();
                const bool live = !flags[0];
                const int B = d.batch;
                const bool two_tiles = true, two_pass = MAXB > 1 && B > 4;
                const uint8_t* xs = smem + S::oX + slot * S::kXSlotBytes;

                float tot[2][NP][2];
#pragma unroll
                for (int i = 0; i < 2 * NP * 2; i++) (&tot[0][0][0])[i] = 0.f;

                if (live) {
                    // this lane's B-operand sources.  B column n = g holds digit (g & 1) of
                    //   batch 1: bit-offset class g >> 1            batch > 1: batch entry 4 * pass + (g >> 1)
                    const uint8_t* xp[4];
                    if (MAXB == 1) {
#pragma unroll
                        for (int t = 0; t < 4; t++)
                            xp[t] = (g >> 1) == t ? xs + (g & 1) * S::kDigitOff + c * 8 : zero_page;
                    } else {
#pragma unroll
                        for (int p = 0; p < 2; p++) {
                            const int b = 4 * p + (g >> 1);
                            xp[p] = b < B ? xs + b * S::kXRow + (g & 1) * S::kDigitOff + c * 8 : zero_page;
                        }
                        xp[2] = zero_page; xp[3] = zero_page;
                    }
                    const int* xsum = reinterpret_cast<const int*>(xs + S::kXsumOff);
                    const float* xscale = reinterpret_cast<const float*>(xs + S::kXscaleOff);
                    for (int s = 0; s < d.cnt; s++) {
                        const uint8_t* blob = st + (s / kBlobSteps) * d.blob_read;       // this superstep's blob (prefix)
                        const int ssl = s % kBlobSteps;
                        const uint32_t* meta_s = reinterpret_cast<const uint32_t*>(blob + blob_meta_off(ssl, 0));
                        int v[2][2][2][2];
#pragma unroll
                        for (int i = 0; i < 16; i++) (&v[0][0][0][0])[i] = 0;
                        int prefix = 0;
                        for (int fi = 0; fi < d.n_fields; fi++) {
                            const int f = d.width[fi];
                            const uint8_t* f0 = blob + blob_field_off(prefix, f, ssl, 0);
                            const uint8_t* f1 = f0 + f * 512;
                            switch (f) {
                                case 8: field_step<8, MAXB>(f0, f1, two_tiles, two_pass, lane, xp, s * 256, d.shift[fi], v); break;
                                case 4: field_step<4, MAXB>(f0, f1, two_tiles, two_pass, lane, xp, s * 256, d.shift[fi], v); break;
                                case 2: field_step<2, MAXB>(f0, f1, two_tiles, two_pass, lane, xp, s * 256, d.shift[fi], v); break;
                                default: field_step<1, MAXB>(f0, f1, two_tiles, two_pass, lane, xp, s * 256, d.shift[fi], v); break;
                            }
                            prefix += f;
                        }
                        // group epilogue: y += s * 2^-e * (v - z * sum x_int)
#pragma unroll
                        for (int tile = 0; tile < 2; tile++) {
                            if (tile == 1 && !two_tiles) break;
#pragma unroll
                            for (int grp = 0; grp < 2; grp++) {
                                const uint32_t m0 = meta_s[tile * 32 + grp * 16 + g];
                                const uint32_t m1 = meta_s[tile * 32 + grp * 16 + g + 8];
                                const float s0 = __half2float(__ushort_as_half((unsigned short)(m0 & 0xffffu)));
                                const float s1 = __half2float(__ushort_as_half((unsigned short)(m1 & 0xffffu)));
                                const int z0 = (int)(m0 >> 16) - d.zero_adjust;
                                const int z1 = (int)(m1 >> 16) - d.zero_adjust;
#pragma unroll
                                for (int p = 0; p < NP; p++) {
                                    // batch 1: only the class-0 lane subtracts the zero-point term
                                    const int b = MAXB == 1 ? 0 : 4 * p + c;
                                    const bool has = MAXB == 1 ? true : b < B;
                                    const int xsm = (MAXB == 1 ? c == 0 : has) ? xsum[b * (S::kCMax * 2) + s * 2 + grp] : 0;
                                    const float sc = has ? xscale[b * (S::kCMax * 2) + s * 2 + grp] : 0.f;
                                    tot[tile][p][0] = fmaf((float)(v[tile][p][0][grp] - z0 * xsm), s0 * sc, tot[tile][p][0]);
                                    tot[tile][p][1] = fmaf((float)(v[tile][p][1][grp] - z1 * xsm), s1 * sc, tot[tile][p][1]);
                                }
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    released[stage] = use + 1u;
                    __threadfence_block();
                    mbar_arrive(empty);                              // the stage may be refilled
                    atomicSub(const_cast<int*>(&x_pending[slot]), 1);   // one unit fewer needs the activation slot
                }
                if (!live) continue;

                if (MAXB == 1) {                                     // add up the bit-offset classes held by the quad
#pragma unroll
                    for (int tile = 0; tile < 2; tile++)
#pragma unroll
                        for (int r = 0; r < 2; r++) {
                            float t = tot[tile][0][r];
                            t += __shfl_xor_sync(0xffffffffu, t, 1);
                            t += __shfl_xor_sync(0xffffffffu, t, 2);
                            tot[tile][0][r] = t;
                        }
                }

                // ---- output: direct, or through split-K partials combined by the last arriver
                // value (tile, pass, r) of lane (g, c): row = (2 rp + tile) * 16 + g + 8 r,
                //   batch entry = 0 (batch 1, lane c == 0 only) or 4 pass + c
                __half* y = reinterpret_cast<__half*>(d.y);
                constexpr int BW = MAXB == 1 ? 1 : 8;                // partial floats per row
                const int row_base = d.rp * (kUnitRowTiles * kTileRows);
                bool wrote_final = true;
                if (d.n_chunks == 1) {
#pragma unroll
                    for (int tile = 0; tile < 2; tile++)
#pragma unroll
                        for (int p = 0; p < NP; p++)
#pragma unroll
                            for (int r = 0; r < 2; r++) {
                                const int row = row_base + tile * 16 + g + 8 * r;
                                const int b = MAXB == 1 ? 0 : 4 * p + c;
                                const bool mine = MAXB == 1 ? c == 0 : b < B;
                                if (mine && row < d.n_out) y[(long long)b * d.n_out + row] = __float2half_rn(tot[tile][p][r]);
                            }
                } else {
                    float* pu = d.partial + ((long long)d.rp * d.n_chunks + d.ch) * (32 * BW);
#pragma unroll
                    for (int tile = 0; tile < 2; tile++)
#pragma unroll
                        for (int p = 0; p < NP; p++)
#pragma unroll
                            for (int r = 0; r < 2; r++) {
                                const int lr = tile * 16 + g + 8 * r;
                                if (MAXB == 1) { if (c == 0) pu[lr] = tot[tile][0][r]; }
                                else pu[lr * BW + 4 * p + c] = tot[tile][p][r];
                            }
                    __syncwarp();
                    unsigned old = 0;
                    if (lane == 0) old = atom_add_acq_rel_u32(d.tile_count + d.rp, 1u);
                    old = __shfl_sync(0xffffffffu, old, 0);
                    wrote_final = false;
                    if (old == (unsigned)(d.n_chunks - 1)) {
                        const float* pt = d.partial + (long long)d.rp * d.n_chunks * (32 * BW);
                        for (int e = lane; e < 32 * BW; e += 32) {   // e = local row * BW + batch entry
                            float sum = 0.f;
                            for (int q = 0; q < d.n_chunks; q++) sum += __ldcg(pt + (long long)q * (32 * BW) + e);
                            const int row = row_base + e / BW, b = e % BW;
                            if (row < d.n_out && b < B) y[(long long)b * d.n_out + row] = __float2half_rn(sum);
                        }
                        if (lane == 0) d.tile_count[d.rp] = 0u;      // ready for the next launch
                        wrote_final = true;
                    }
                }
                if (d.phase >= 0) {
                    __syncwarp();                                    // y is ordered before the release below
                    if (lane == 0) red_add_release_u64(sa.phase_done + d.phase, 1ull);
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
template <int MAXB>
static int launch_impl(Ctx* ctx, const GemvOp& single, const StackArgs& sa, long long total_units, bool cooperative,
                       cudaStream_t st)
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
    if (cooperative) {
        void* args[] = {(void*)&single, (void*)&sa};
        FQ_CUDA_OK(cudaLaunchCooperativeKernel((const void*)gemv_kernel<MAXB>, dim3((unsigned)blocks), dim3(kGemvThreads),
                                               args, S::kTotal, st));
    } else {
        gemv_kernel<MAXB><<<(unsigned)blocks, kGemvThreads, S::kTotal, st>>>(single, sa);
        FQ_CUDA_OK(cudaGetLastError());
    }
    return FQ_OK;
}

int launch_gemv_single(Ctx* ctx, const GemvOp& op, cudaStream_t st)
{
    StackArgs sa{};
    sa.table = nullptr;
    sa.status = ctx->status_dev;
    sa.n_ops = 1;
    sa.n_phases = 0;
    const long long units = (long long)op.n_rp * op.n_chunks;
    return op.batch <= 1 ? launch_impl<1>(ctx, op, sa, units, false, st) : launch_impl<8>(ctx, op, sa, units, false, st);
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
    GemvOp dummy{};
    const bool coop = hdr.n_phases > 0;
    return max_batch <= 1 ? launch_impl<1>(ctx, dummy, sa, hdr.total_units, coop, st)
                          : launch_impl<8>(ctx, dummy, sa, hdr.total_units, coop, st);
}

// ------------------------------------------------------------------------------- allocation-free variant
// Split-K scratch that is part of the library image, for callers that must not allocate.
// Host code may only use the symbol through cudaGetSymbolAddress (its name is not a device
// address on the host side).
static __device__ __align__(256) unsigned char g_static_scratch[FQ_STATIC_SCRATCH_BYTES];

static int static_scratch_address(int device, unsigned char** out)
{
    static unsigned char* addr[64] = {};
    if (device < 0 || device >= 64) return FQ_ERR_ARG;
    if (!addr[device]) {                       // once per device, with that device current
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return FQ_ERR_CUDA;
        addr[device] = static_cast<unsigned char*>(p);
    }
    *out = addr[device];
    return FQ_OK;
}

// Runs one batch-1 decode op with counters and partials placed in the built-in array.
int launch_gemv_static(Ctx* ctx, GemvOp op, size_t counter_bytes, size_t partial_bytes, cudaStream_t st)
{
    const size_t counters = (size_t)round_up((int64_t)counter_bytes, 256);
    if (counters + partial_bytes > FQ_STATIC_SCRATCH_BYTES) return FQ_ERR_SCRATCH;
    unsigned char* base = nullptr;
    const int rc = static_scratch_address(ctx->device, &base);
    if (rc != FQ_OK) return rc;
    op.tile_count = reinterpret_cast<unsigned*>(base);
    op.partial = reinterpret_cast<float*>(base + counters);
    // the array keeps the previous call's contents: arrival counters must start at zero
    if (counter_bytes) FQ_CUDA_OK(cudaMemsetAsync(base, 0, counter_bytes, st));
    StackArgs sa{};
    sa.table = nullptr;
    sa.status = ctx->status_dev;
    sa.n_ops = 1;
    sa.n_phases = 0;
    return launch_impl<1>(ctx, op, sa, (long long)op.n_rp * op.n_chunks, false, st);
}

}  // namespace fq

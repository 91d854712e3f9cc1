// Decode path, batch 1: fused dequantize-GEMV over tiled field arrays, one persistent CTA per SM.
//
// Work split.  An op (one matrix) is cut into STRIPS of 32 output rows x the whole K, a strip into K
// chunks ("units": 1..3 blobs of 512 columns, what one ring stage holds).  Units are numbered strip-major
// and dealt to the CTAs in equal contiguous blocks (cta_work in fq_internal.cuh), so every CTA streams the
// same number of bytes and almost every strip is computed by ONE CTA from end to end: its K reduction
// stays in shared memory and the CTA writes y itself.  Only a strip that a block boundary cuts is shared
// by two (rarely three) CTAs: the CTA that owns the strip's last chunk finishes it, the others publish the
// sums of their blobs as tagged 64-bit words (fp32 value, launch tag) in global memory and process that
// strip first, long before the finisher asks for them.  y[row] is always the sum of the per-blob sums in
// blob order, whoever computed them, so results do not depend on how the op was dealt.
//
// Roles of a CTA:
//   producer warp   : walks the op list, streams units into a ring of shared-memory stages with bulk
//                     asynchronous copies (cp.async.bulk + mbarrier tx counts; it runs ahead across op and
//                     phase boundaries because weights do not depend on activations) and deals the
//                     (blob, 16-row tile) items of every unit round-robin into per-warp queues;
//   consumer warps  : 16 warps = 8 K lanes x 2 row tiles.  An item is one tile of one blob: the arithmetic
//                     of fq_gemv_core.cuh, then the 16 row sums go to the strip's slot in shared memory
//                     (or to global memory for a strip finished elsewhere).  The warp that delivers a
//                     strip's last item adds the blob sums up, writes y and counts the strip for its phase;
//   x-prep warps    : convert the activations of every blob this CTA needs into 16-bit fixed point per
//                     group of 128 columns (two signed byte digits, B-fragment order) in a ring of blob
//                     slots; before the first blob of an op they wait -- bounded -- until every CTA has
//                     finished the previous dependency phase.
// Every wait has a time limit; when one runs out the kernel records FQ_ERR_TIMEOUT, every role leaves its
// loop, the producer waits for its copies in flight and the CTA returns.
#include <cuda_fp16.h>

#include "fq_internal.cuh"
#include "fq_ptx.cuh"
#include "fq_gemv_core.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

namespace {

constexpr int kCW = 16;                                // consumer warps: K lane = warp >> 1, row tile = warp & 1
constexpr int kKLanes = kCW / kBlobTiles;
constexpr int kProducerWarp = kCW;
constexpr int kPrepWarp = kCW + 1;                     // first activation pre-processing warp
constexpr int kPrepWarps = 4;
constexpr int kThreads = (kCW + 1 + kPrepWarps) * 32;
constexpr int kStageBytes = 17408;                     // one unit: 2 x 4-bit blobs or 1 x 8-bit blob
constexpr int kBlobsMax = 3;                           // blobs per unit, at most
constexpr int kXSlots = 32;                            // activation blobs resident in shared memory
constexpr int kStripSlots = 4;                         // strips whose items are in flight
constexpr int kMaxKb = 32;                             // blobs per strip, at most (k_in <= 16384)
constexpr int kQD = 8;                                 // entries per consumer queue
constexpr int kMaxPhasesDev = 1024;

// What the producer tells a consumer warp about one item (one 16-byte store, one 16-byte load).
//   w0 blob shared address   w1 packed fields (below)   w2 activation blob number + 1   w3 sequence tag
constexpr uint32_t kItemEnd = 1u << 31;
__device__ __forceinline__ uint32_t item_pack(int xslot, int stage, int parity, int kb, int sslot, int variant)
{
    return (uint32_t)xslot | (uint32_t)stage << 5 | (uint32_t)parity << 9 | (uint32_t)kb << 10 | (uint32_t)sslot << 15 |
           (uint32_t)variant << 18;
}

// A strip in flight.
struct StripDesc {
    uint16_t* y;                             // output of the op
    unsigned long long* partial;             // tagged blob sums of this strip in global memory: [blob][32 rows]
    int n_out, row_base;
    int n_kb, kb_lo, kb_hi;                  // blobs of the strip; [kb_lo, kb_hi) are computed by this CTA
    int finish;                              // this CTA owns the last chunk: it adds up and writes y
    int phase;
    int expect;                              // items of this CTA in the strip
    int pad[4];
};
static_assert(sizeof(StripDesc) == 64, "descriptor layout");

struct Smem {
    static constexpr int kFixed = kXSlots * (kXBlobDigitBytes + kXBlobGroupBytes) + 1024 + kStripSlots * kMaxKb * 128 +
                                  kCW * kQD * 16 + kStripSlots * 64 + kMaxPhasesDev * 2 + 1024;
    static constexpr int kStages = (232448 - kFixed) / kStageBytes;
    static constexpr int oStages = 0;
    static constexpr int oXDig = oStages + kStages * kStageBytes;            // [slot][1024]
    static constexpr int oXGrp = oXDig + kXSlots * kXBlobDigitBytes;         // [slot][32]
    static constexpr int oZero = oXGrp + kXSlots * kXBlobGroupBytes;         // 1024 zero bytes
    static constexpr int oPart = oZero + 1024;                               // float [strip slot][blob][32 rows]
    static constexpr int oQueue = oPart + kStripSlots * kMaxKb * 128;        // uint4 [warp][kQD]
    static constexpr int oStrip = oQueue + kCW * kQD * 16;                   // StripDesc [strip slot]
    static constexpr int oFinTot = oStrip + kStripSlots * 64;                // u16 [phase]: strips this CTA finishes
    static constexpr int oBars = oFinTot + kMaxPhasesDev * 2;                // full[S], empty[S]
    static constexpr int oCtl = oBars + 2 * 16 * 8;
    // control words (u32 each)
    static constexpr int cXTag = 0;                                          // [kXSlots] activation blob number + 1 held
    static constexpr int cXCnt = cXTag + kXSlots;                            // [kXSlots] items that still need the slot
    static constexpr int cStripCnt = cXCnt + kXSlots;                        // [kStripSlots] items delivered
    static constexpr int cStripBusy = cStripCnt + kStripSlots;               // [kStripSlots]
    static constexpr int cFinCnt = cStripBusy + kStripSlots;                 // [8] strips finished, per phase & 7
    static constexpr int cQn = cFinCnt + 8;                                  // [kCW] entries queued so far (producer only)
    static constexpr int cAbort = cQn + kCW;
    static constexpr int kCtlWords = cAbort + 1;
    static constexpr int kTotal = oCtl + kCtlWords * 4;
    static_assert(kStages >= 4 && kStages <= 16, "decode kernel: ring size");
    static_assert(kTotal <= 232448, "decode kernel: shared memory over the 227 KB per-CTA limit");
    static_assert(oBars % 8 == 0 && oQueue % 16 == 0 && oStrip % 16 == 0 && oXDig % 128 == 0 && oZero % 128 == 0, "alignment");
};

struct Args {
    const GemvOp* table;                   // device op table (nullptr: the by-value op)
    const int* phase_total;                // CTAs that finish at least one strip, per phase
    unsigned long long* phase_done;        // CTAs that have finished all their strips, per phase
    unsigned* exit_count;
    int* status;
    int n_ops, n_phases;
    unsigned epoch;                        // tag of this launch's published blob sums (never 0)
    unsigned long long wait_ns;            // limit of every wait
};

__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
// Brings the descriptors of the ops a few steps ahead into L1: the table is read once per op by three roles,
// and a miss would cost each of them a trip to DRAM (the weights keep flushing the L2).
__device__ __forceinline__ void prefetch_ops(const GemvOp* ops, int oi, int n_ops, int lane)
{
    const int ahead = oi + 2 + (lane >> 1);                        // lanes 0..7: ops oi+2 .. oi+5, two lines each
    if (lane < 8 && ahead < n_ops) {
        const char* p = reinterpret_cast<const char*>(ops + ahead) + (lane & 1) * 64;
        asm volatile("prefetch.global.L1 [%0];" ::"l"(p));
    }
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// The strips of one op for one CTA, in the order in which it processes them: a strip that another CTA
// finishes goes first (its sums are wanted elsewhere), the rest in ascending order.
struct StripOrder {
    CtaWork w;
    int n_chunks, n_strips, first_is_last;
    __device__ __forceinline__ StripOrder(const GemvOp& op, int cta, int grid)
    {
        w = cta_work(op.n_units, op.n_chunks, op.rot, cta, grid);
        n_chunks = op.n_chunks;
        n_strips = w.any() ? w.rp_last - w.rp_first + 1 : 0;
        first_is_last = n_strips > 1 && (w.hi - w.rp_last * n_chunks) < n_chunks;
    }
    __device__ __forceinline__ int strip(int i) const
    {
        if (!first_is_last) return w.rp_first + i;
        return i == 0 ? w.rp_last : w.rp_first + i - 1;
    }
};

__device__ __forceinline__ void raise_timeout(const Args& a, volatile unsigned* ctl)
{
    atomicCAS(a.status, 0, FQ_ERR_TIMEOUT);
    ctl[Smem::cAbort] = 1u;
}

// Bounded wait for a condition on shared-memory words; gives up early when the CTA is aborting.
template <typename Pred>
__device__ __forceinline__ bool wait_smem(Pred pred, volatile unsigned* ctl, unsigned long long limit)
{
    if (pred()) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 32; i++) {
            if (pred()) return true;
            __nanosleep(32);
        }
        if (ctl[Smem::cAbort] || global_ns() - t0 > limit) return false;
    }
}
__device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity, volatile unsigned* ctl, unsigned long long limit)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; i++)
            if (mbar_try_wait(bar, parity)) return true;
        if (ctl[Smem::cAbort] || global_ns() - t0 > limit) return false;
    }
}

// ------------------------------------------------------------------------------- activation pre-processing
// One superstep (256 columns, 8 per lane) of fp16 activations -> fixed point per group of 128 columns:
// x_int = rint(x * 2^(13 - E)) with 2^E <= max|x| < 2^(E+1), stored as two signed byte digits in
// B-fragment order, plus per group the integer sum and the factor 2^(E - 13).  A group that holds an
// infinity or a NaN gets the factor NaN, so that every row sum that touches it comes out NaN.
__device__ __forceinline__ void convert_superstep(uint4 raw, uint8_t* xdig, uint8_t* xgrp, int ss, int lane)
{
    const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
    float f[8];
    bool bad = false;
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const float2 t2 = __half22float2(h2[i]);
        f[2 * i] = t2.x; f[2 * i + 1] = t2.y;
    }
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 8; i++) {
        amax = fmaxf(amax, fabsf(f[i]));
        bad = bad || !(fabsf(f[i]) <= 65504.f);                 // infinity or NaN
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const unsigned badmask = __ballot_sync(0xffffffffu, bad);
    bad = ((badmask >> (lane & 16)) & 0xffffu) != 0u;           // anywhere in this lane's group of 16 lanes
    const int eb = (__float_as_int(amax) >> 23) & 0xff;         // biased exponent of the group maximum
    const bool fin = amax > 0.f && !bad;
    const float mult = fin ? __int_as_float((267 - eb) << 23) : 0.f;
    const float back = bad ? __int_as_float(0x7fc00000) : (fin ? __int_as_float((eb - 13) << 23) : 0.f);
    int xi[8], sum = 0;
#pragma unroll
    for (int i = 0; i < 8; i++) { xi[i] = bad ? 0 : __float2int_rn(f[i] * mult); sum += xi[i]; }
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
    // lane l holds columns 8l .. 8l+7: k32 step j = l >> 2, half (l >> 1) & 1, column blocks c0 and c0 + 1
    const int j = lane >> 2, half = (lane >> 1) & 1, c0 = 2 * (lane & 1);
    uint8_t* cell = xdig + x_digit_off(ss, j & 3, 0, c0) + (2 * (j >> 2) + half) * 4;
    *reinterpret_cast<uint32_t*>(cell) = lo4[0];
    *reinterpret_cast<uint32_t*>(cell + 16) = lo4[1];
    *reinterpret_cast<uint32_t*>(cell + 64) = hi4[0];
    *reinterpret_cast<uint32_t*>(cell + 64 + 16) = hi4[1];
    if ((lane & 15) == 0) {
        reinterpret_cast<int*>(xgrp)[ss * 2 + (lane >> 4)] = sum;
        reinterpret_cast<float*>(xgrp + 16)[ss * 2 + (lane >> 4)] = back;
    }
}

// ------------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(kThreads, 1)
gemv1_kernel(const __grid_constant__ GemvOp single, const Args a)
{
    using S = Smem;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grid = gridDim.x, cta = blockIdx.x;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + S::oBars;                               // full[s] at 8 s, empty[s] at 128 + 8 s
    volatile unsigned* ctl = reinterpret_cast<volatile unsigned*>(smem + S::oCtl);
    unsigned short* fin_total = reinterpret_cast<unsigned short*>(smem + S::oFinTot);
    const GemvOp* ops = a.table ? a.table : &single;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; s++) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 128 + 8 * s, kCW);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < S::kCtlWords; i += blockDim.x) ctl[i] = 0u;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + S::oZero)[i] = 0u;
    for (int i = threadIdx.x; i < kCW * kQD * 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + S::oQueue)[i] = 0u;
    for (int i = threadIdx.x; i < kMaxPhasesDev / 2; i += blockDim.x) reinterpret_cast<uint32_t*>(fin_total)[i] = 0u;
    __syncthreads();
    // strips that this CTA finishes, per phase (the warp that finishes the last one reports the phase)
    if (a.n_phases > 0) {
        for (int oi = threadIdx.x; oi < a.n_ops; oi += blockDim.x) {
            const GemvOp& op = ops[oi];
            const int fin = cta_work(op.n_units, op.n_chunks, op.rot, cta, grid).finishing(op.n_chunks);
            if (fin > 0 && op.phase >= 0) {
                // two 16-bit counters per word
                atomicAdd(reinterpret_cast<unsigned*>(fin_total) + (op.phase >> 1), (unsigned)fin << (16 * (op.phase & 1)));
            }
        }
    }
    __syncthreads();

    if (warp == kProducerWarp) {
        // ================================================================== producer
        int stage = 0;
        unsigned wraps = 0;
        unsigned rr = 0;                              // K lane of the next blob (round-robin over everything)
        unsigned xseq = 0;                            // activation blobs of the ops seen so far
        unsigned strip_seq = 0;
        bool stop = false;
        StripDesc* sdesc = reinterpret_cast<StripDesc*>(smem + S::oStrip);
        for (int oi = 0; oi < a.n_ops && !stop; oi++) {
            prefetch_ops(ops, oi, a.n_ops, lane);
            const GemvOp& op = ops[oi];
            const StripOrder so(op, cta, grid);
            if (so.n_strips == 0) continue;
            const int n_kb = op.n_kb, cb = op.chunk_blobs;
            const uint32_t blob_read = (uint32_t)op.blob_read;
            const long long blob_stride = op.blob_stride;
            const bool contiguous = op.blob_read == op.blob_stride;
            for (int si = 0; si < so.n_strips && !stop; si++) {
                const int rp = so.strip(si);
                int c0, c1;
                so.w.chunks(so.n_chunks, rp, c0, c1);
                const int kb_lo = c0 * cb, kb_hi = min(c1 * cb, n_kb);
                const int sslot = (int)(strip_seq % kStripSlots);
                strip_seq++;
                int slot_ok = 1;
                if (lane == 0) {
                    if (!wait_smem([&] { return ctl[S::cStripBusy + sslot] == 0u; }, ctl, a.wait_ns)) {
                        if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                        slot_ok = 0;
                    } else {
                        StripDesc& d = sdesc[sslot];
                        d.y = op.y;
                        d.partial = op.partial + (long long)rp * n_kb * 32;
                        d.n_out = op.n_out; d.row_base = rp * (kBlobTiles * kTileRows);
                        d.n_kb = n_kb; d.kb_lo = kb_lo; d.kb_hi = kb_hi;
                        d.finish = c1 == so.n_chunks;
                        d.phase = op.phase;
                        d.expect = (kb_hi - kb_lo) * kBlobTiles;
                        ctl[S::cStripBusy + sslot] = 1u;
                        __threadfence_block();
                    }
                }
                if (!__shfl_sync(0xffffffffu, slot_ok, 0)) { stop = true; break; }   // (every loop exit is decided by lane 0)
                const uint8_t* src = op.store + ((long long)rp * n_kb + kb_lo) * blob_stride;
                for (int kb = kb_lo; kb < kb_hi; kb += cb) {
                    const int nb = min(cb, kb_hi - kb);
                    const uint32_t full = bars + 8 * stage, empty = bars + 128 + 8 * stage;
                    int ok = 1;
                    if (lane == 0) {
                        if (wraps > 0 && !wait_mbar(empty, (wraps - 1u) & 1u, ctl, a.wait_ns)) {
                            if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                            ok = 0;
                        }
                        if (ok) mbar_expect_tx(full, (uint32_t)nb * blob_read);
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { stop = true; break; }
                    const uint32_t stage_base = sbase + S::oStages + (uint32_t)stage * kStageBytes;
                    if (contiguous) {
                        if (lane == 0) bulk_g2s(stage_base, src, (uint32_t)nb * blob_read, full);
                    } else if (lane < nb) {
                        bulk_g2s(stage_base + lane * blob_read, src + lane * blob_stride, blob_read, full);
                    }
                    // the items of this unit: lane = blob * 2 + tile
                    if (lane < nb * kBlobTiles) {
                        const int b = lane >> 1, t = lane & 1;
                        const int w = (int)(((rr + (unsigned)b) % kKLanes) * kBlobTiles) + t;
                        const unsigned n = ctl[S::cQn + w];
                        const unsigned xs = xseq + (unsigned)(kb + b);
                        uint4 e;
                        e.x = stage_base + (uint32_t)b * blob_read;
                        e.y = item_pack((int)(xs % kXSlots), stage, (int)(wraps & 1u), kb + b, sslot, op.variant);
                        e.z = xs + 1u;
                        e.w = n + 1u;
                        sts128(sbase + S::oQueue + (uint32_t)(w * kQD + (int)(n % kQD)) * 16u, e);
                        ctl[S::cQn + w] = n + 1u;
                    }
                    if (lane == 0) mbar_arrive_n(empty, (uint32_t)(kCW - nb * kBlobTiles));   // warps without an item in this unit
                    __syncwarp();
                    rr += (unsigned)nb;
                    src += (long long)nb * blob_stride;
                    if (++stage == S::kStages) { stage = 0; wraps++; }
                }
            }
            xseq += (unsigned)n_kb;
        }
        // the end marker of every queue
        if (lane < kCW) {
            const unsigned n = ctl[S::cQn + lane];
            const uint4 e = make_uint4(0u, kItemEnd, 0u, n + 1u);
            // (the queue slot is free: a warp gets one entry per kKLanes blobs, so the entry that used the slot
            // kQD entries ago belongs to a unit whose stage has been refilled since, i.e. it was consumed)
            sts128(sbase + S::oQueue + (uint32_t)(lane * kQD + (int)(n % kQD)) * 16u, e);
        }
        // copies that are still in flight must land before the CTA may exit
        if (stop && lane == 0) {
            const int issued = (int)(wraps * S::kStages) + stage;
            const unsigned long long t0 = global_ns();
            for (int u = max(0, issued - S::kStages); u < issued; u++)
                while (!mbar_try_wait(bars + 8 * (u % S::kStages), (unsigned)(u / S::kStages) & 1u))
                    if (global_ns() - t0 > kWaitLimitNs) break;
        }
    } else if (warp >= kPrepWarp) {
        // ================================================================== activation pre-processing
        const int pw = warp - kPrepWarp;
        unsigned xseq = 0;
        int phase_known = -1;                         // every phase <= phase_known is complete
        bool stop = false;
        for (int oi = 0; oi < a.n_ops && !stop; oi++) {
            prefetch_ops(ops, oi, a.n_ops, lane);
            const GemvOp& op = ops[oi];
            const StripOrder so(op, cta, grid);
            if (so.n_strips == 0) continue;
            const int n_kb = op.n_kb, cb = op.chunk_blobs;
            // blobs of x that this CTA's strips cover: the first and the last strip may be partial
            int f0, f1, l0, l1;
            so.w.chunks(so.n_chunks, so.w.rp_first, f0, f1);
            so.w.chunks(so.n_chunks, so.w.rp_last, l0, l1);
            const int fk0 = f0 * cb, fk1 = min(f1 * cb, n_kb), lk0 = l0 * cb, lk1 = min(l1 * cb, n_kb);
            const int n_mid = so.n_strips > 2 ? so.n_strips - 2 : 0;
            // the activations are the previous phase's outputs
            if (op.phase > 0 && phase_known < op.phase - 1) {
                int ok = 1;
                if (lane == 0) {
                    const unsigned long long need = (unsigned long long)a.phase_total[op.phase - 1];
                    const unsigned long long t0 = global_ns();
                    unsigned it = 0;
                    while (ld_acquire_u64(a.phase_done + (op.phase - 1)) < need) {
                        if ((++it & 31u) == 0u) {
                            if (ctl[S::cAbort]) { ok = 0; break; }
                            if (global_ns() - t0 > a.wait_ns || *reinterpret_cast<volatile int*>(a.status) != 0) {
                                raise_timeout(a, ctl); ok = 0; break;
                            }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) { stop = true; break; }
                phase_known = op.phase - 1;
            }
            const __half* x = reinterpret_cast<const __half*>(op.x);
            // this warp's blobs of the op: activation blob numbers congruent to pw; up to four per round
            int kb = (int)((pw + kPrepWarps - (xseq % kPrepWarps)) % kPrepWarps);
            while (kb < n_kb && !stop) {
                uint4 raw[4][2];
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    const int kq = kb + q * kPrepWarps;
#pragma unroll
                    for (int ss = 0; ss < 2; ss++) {
                        raw[q][ss] = make_uint4(0u, 0u, 0u, 0u);
                        const int k = kq * 512 + ss * 256 + lane * 8;
                        if (kq < n_kb && k < op.k_in) raw[q][ss] = __ldcg(reinterpret_cast<const uint4*>(x + k));
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    const int kq = kb + q * kPrepWarps;
                    if (kq >= n_kb) break;
                    const unsigned xs = xseq + (unsigned)kq;
                    const int slot = (int)(xs % kXSlots);
                    int uses = n_mid + ((kq >= fk0 && kq < fk1) ? 1 : 0);
                    if (so.n_strips > 1) uses += (kq >= lk0 && kq < lk1) ? 1 : 0;
                    uses *= kBlobTiles;
                    int ok = 1;
                    if (lane == 0 && !wait_smem([&] { return ctl[S::cXCnt + slot] == 0u; }, ctl, a.wait_ns)) {
                        if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                        ok = 0;
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { stop = true; break; }
                    if (uses > 0) {
                        uint8_t* xdig = smem + S::oXDig + slot * kXBlobDigitBytes;
                        uint8_t* xgrp = smem + S::oXGrp + slot * kXBlobGroupBytes;
                        convert_superstep(raw[q][0], xdig, xgrp, 0, lane);
                        convert_superstep(raw[q][1], xdig, xgrp, 1, lane);
                    }
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) {
                        ctl[S::cXCnt + slot] = (unsigned)uses;
                        __threadfence_block();
                        ctl[S::cXTag + slot] = xs + 1u;
                    }
                }
                kb += 4 * kPrepWarps;
            }
            xseq += (unsigned)n_kb;
        }
    } else {
        // ================================================================== consumers
        const int tile = warp & 1;
        const int g = lane >> 2, c = lane & 3;
        const uint32_t queue = sbase + S::oQueue + (uint32_t)warp * kQD * 16u;
        const StripDesc* sdesc = reinterpret_cast<const StripDesc*>(smem + S::oStrip);
        float* part = reinterpret_cast<float*>(smem + S::oPart);
        const unsigned long long tag = (unsigned long long)a.epoch << 32;
        for (unsigned n = 0;; n++) {
            // ---- next item of this warp
            const uint32_t qa = queue + (n % kQD) * 16u;
            uint4 e = lds128(qa);
            if (!__all_sync(0xffffffffu, e.w == n + 1u)) {
                const unsigned long long t0 = global_ns();
                unsigned it = 0;
                bool ok = true;
                for (;;) {
                    e = lds128(qa);
                    if (__all_sync(0xffffffffu, e.w == n + 1u)) break;
                    __nanosleep(32);
                    int giveup = 0;
                    if (lane == 0 && (++it & 63u) == 0u && (ctl[S::cAbort] || global_ns() - t0 > a.wait_ns)) giveup = 1;
                    if (__shfl_sync(0xffffffffu, giveup, 0)) { ok = false; break; }   // (the lanes must leave together)
                }
                if (!ok) {
                    if (lane == 0 && !ctl[S::cAbort]) raise_timeout(a, ctl);
                    break;
                }
            }
            if (e.y & kItemEnd) break;
            const int xslot = (int)(e.y & 31u), stage = (int)((e.y >> 5) & 15u), parity = (int)((e.y >> 9) & 1u);
            const int kb = (int)((e.y >> 10) & 31u), sslot = (int)((e.y >> 15) & 7u), variant = (int)((e.y >> 18) & 15u);
            // ---- its weights and its activations
            bool ok = wait_mbar(bars + 8 * stage, (uint32_t)parity, ctl, a.wait_ns);
            if (ok) ok = wait_smem([&] { return ctl[S::cXTag + xslot] == e.z; }, ctl, a.wait_ns);
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0 && !ctl[S::cAbort]) raise_timeout(a, ctl);
                break;
            }
            __threadfence_block();
            const uint32_t xdig = sbase + S::oXDig + (uint32_t)xslot * kXBlobDigitBytes;
            uint32_t xd[4];
#pragma unroll
            for (int jc = 0; jc < 4; jc++)
                xd[jc] = (g >> 1) == jc ? xdig + x_digit_off(0, jc, g & 1, c) : sbase + S::oZero + c * 16;
            float tot[2] = {0.f, 0.f};
            blob_tile_dispatch(variant, e.x, tile, xd, sbase + S::oXGrp + (uint32_t)xslot * kXBlobGroupBytes, lane, tot);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bars + 128 + 8 * stage);                         // the stage may be refilled
                atomicSub(const_cast<unsigned*>(&ctl[S::cXCnt + xslot]), 1u);   // one item fewer needs the activation blob
            }
            // ---- the 16 row sums of the item: add up the step classes held by the quad
#pragma unroll
            for (int r = 0; r < 2; r++) {
                tot[r] += __shfl_xor_sync(0xffffffffu, tot[r], 1);
                tot[r] += __shfl_xor_sync(0xffffffffu, tot[r], 2);
            }
            const StripDesc& d = sdesc[sslot];
            const int finish = d.finish, expect = d.expect;                  // (read before this item is counted)
            unsigned long long* const dpart = d.partial;
            if (c < 2) {                                                     // lane c of the quad stores row g + 8 c
                const float v = c == 0 ? tot[0] : tot[1];
                const int lr = tile * kTileRows + g + 8 * c;
                if (finish) part[(sslot * kMaxKb + kb) * 32 + lr] = v;
                else st_relaxed_u64(dpart + kb * 32 + lr, tag | __float_as_uint(v));   // finished elsewhere
            }
            __threadfence_block();
            __syncwarp();
            int last = 0;
            if (lane == 0) last = atomicAdd(const_cast<unsigned*>(&ctl[S::cStripCnt + sslot]), 1u) + 1u == (unsigned)expect;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (!last) continue;
            // ---- this warp delivered the strip's last item
            __threadfence_block();
            bool live = true;
            if (finish) {
                // lane = row of the strip; blob sums in blob order; blobs of other CTAs from their tagged words
                const int n_kb = d.n_kb, kb_lo = d.kb_lo;
                float sum = 0.f;
                if (kb_lo > 0) {
                    const unsigned long long t0 = global_ns();
                    for (int q = 0; q < kb_lo && live; q++) {
                        unsigned long long wv = ld_relaxed_u64(d.partial + q * 32 + lane);
                        unsigned it = 0;
                        while (!__all_sync(0xffffffffu, (unsigned)(wv >> 32) == a.epoch)) {
                            __nanosleep(64);
                            int giveup = 0;
                            if (lane == 0 && (++it & 15u) == 0u && (ctl[S::cAbort] || global_ns() - t0 > a.wait_ns)) giveup = 1;
                            if (__shfl_sync(0xffffffffu, giveup, 0)) { live = false; break; }
                            wv = ld_relaxed_u64(d.partial + q * 32 + lane);
                        }
                        sum += __uint_as_float((unsigned)wv);
                    }
                    if (!live && lane == 0 && !ctl[S::cAbort]) raise_timeout(a, ctl);
                }
                if (live) {
                    const float* ps = part + (sslot * kMaxKb) * 32 + lane;
                    for (int q = kb_lo; q < n_kb; q++) sum += ps[q * 32];
                    const int row = d.row_base + lane;
                    if (row < d.n_out) reinterpret_cast<__half*>(d.y)[row] = __float2half_rn(sum);
                }
            }
            const int phase = d.phase;
            __syncwarp();
            if (lane == 0) {
                ctl[S::cStripCnt + sslot] = 0u;
                __threadfence_block();
                ctl[S::cStripBusy + sslot] = 0u;                             // the producer may reuse the slot
            }
            if (!live) break;
            if (finish && phase >= 0) {
                __threadfence();                                             // y before the phase counter
                __syncwarp();
                if (lane == 0) {
                    const unsigned done = atomicAdd(const_cast<unsigned*>(&ctl[S::cFinCnt + (phase & 7)]), 1u) + 1u;
                    if (done == (unsigned)fin_total[phase]) {
                        ctl[S::cFinCnt + (phase & 7)] = 0u;
                        red_add_relaxed_u64(a.phase_done + phase, 1ull);
                    }
                }
            }
        }
    }

    __syncthreads();
    if (threadIdx.x == 0 && a.n_phases > 0) {
        __threadfence();
        const unsigned old = atomicAdd(a.exit_count, 1u);
        if (old == gridDim.x - 1) {                    // last CTA out: counters back to zero
            for (int p = 0; p < a.n_phases; p++) a.phase_done[p] = 0ull;
            *a.exit_count = 0u;
            __threadfence();
        }
    }
}

int launch(Ctx* ctx, const GemvOp& single, const Args& a, long long total_units, cudaStream_t st)
{
    static bool configured[64] = {};
    if (ctx->device >= 64) return FQ_ERR_ARG;
    if (!configured[ctx->device]) {
        FQ_CUDA_OK(cudaFuncSetAttribute(gemv1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::kTotal));
        configured[ctx->device] = true;
    }
    long long blocks = ctx->sm_count;
    if (total_units < blocks) blocks = total_units;
    if (blocks < 1) return FQ_OK;
    void* args[] = {(void*)&single, (void*)&a};
    // cooperative: CTAs wait (bounded) for each other's phase counts and published sums, so all of them
    // have to be resident together
    FQ_CUDA_OK(cudaLaunchCooperativeKernel((const void*)gemv1_kernel, dim3((unsigned)blocks), dim3(kThreads), args,
                                           Smem::kTotal, st));
    return FQ_OK;
}

unsigned next_epoch(unsigned& e)
{
    if (++e == 0u) ++e;                        // 0 marks words that no launch has written
    return e;
}

}  // namespace

int gemv1_max_phases() { return kMaxPhasesDev; }
int gemv1_max_k() { return kMaxKb * 512; }

int launch_gemv1_single(Ctx* ctx, const GemvOp& op, cudaStream_t st)
{
    Args a{};
    a.status = ctx->status_dev;
    a.n_ops = 1;
    a.epoch = next_epoch(ctx->launch_epoch);
    a.wait_ns = ctx->wait_limit_ns;
    return launch(ctx, op, a, op.n_units, st);
}

int launch_gemv1_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, cudaStream_t st)
{
    Args a{};
    a.table = reinterpret_cast<const GemvOp*>(table_dev);
    a.phase_total = reinterpret_cast<const int*>(table_dev + (size_t)hdr.n_ops * sizeof(GemvOp));
    a.phase_done = reinterpret_cast<unsigned long long*>(ctx->ws);
    a.exit_count = reinterpret_cast<unsigned*>(ctx->ws + 8 * 4096);
    a.status = ctx->status_dev;
    a.n_ops = hdr.n_ops;
    a.n_phases = hdr.n_phases;
    a.epoch = next_epoch(ctx->launch_epoch);
    a.wait_ns = ctx->wait_limit_ns;
    GemvOp dummy{};
    return launch(ctx, dummy, a, hdr.total_units, st);
}

// ------------------------------------------------------------------------------- allocation-free variant
// Scratch that is part of the library image, for callers that must not allocate: the published blob sums
// of the strips that two CTAs share.  Host code may only use the symbol through cudaGetSymbolAddress (its
// name is not a device address on the host side).
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

// Runs one batch-1 decode op with its shared-strip sums placed in the built-in array.  The array keeps the
// previous call's contents.  Nothing in it has to start at zero: a word is only believed when it carries
// this call's tag, and the tags of the calls that share the array (all contexts on a device) come from one
// counter per device.
int launch_gemv_static(Ctx* ctx, GemvOp op, size_t partial_bytes, cudaStream_t st)
{
    static unsigned epoch[64] = {};
    if (partial_bytes > FQ_STATIC_SCRATCH_BYTES) return FQ_ERR_SCRATCH;
    unsigned char* base = nullptr;
    const int rc = static_scratch_address(ctx->device, &base);
    if (rc != FQ_OK) return rc;
    op.partial = reinterpret_cast<unsigned long long*>(base);
    Args a{};
    a.status = ctx->status_dev;
    a.n_ops = 1;
    a.epoch = next_epoch(epoch[ctx->device]);
    a.wait_ns = ctx->wait_limit_ns;
    return launch(ctx, op, a, op.n_units, st);
}

}  // namespace fq

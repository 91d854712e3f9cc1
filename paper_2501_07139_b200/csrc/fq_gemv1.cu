// Decode path, batch 1: fused dequantize-GEMV over tiled field arrays, one persistent CTA per SM.
//
// Work split.  An op (one matrix) is cut into STRIPS of 32 output rows x the whole K, a strip into blobs of
// 512 columns.  Blobs are numbered strip-major and dealt to the CTAs in equal contiguous blocks (cta_work in
// fq_internal.cuh), so every CTA streams the same number of bytes and almost every strip is computed by ONE
// CTA from end to end: its K reduction stays in shared memory and the CTA writes y itself.  Only a strip
// that a block boundary cuts is shared by two (rarely three) CTAs: the CTA that owns the strip's FIRST blob
// finishes it, the others publish the sums of their blobs as tagged 64-bit words (fp32 value, launch tag)
// in global memory.  The shared strip is the last thing the finisher computes and the first thing the
// publisher computes, so the words are there long before they are asked for.  A CTA streams
// its blobs of a strip in "units" of up to six (what one ring stage holds).  y[row] is always the sum of the per-blob sums in
// blob order, whoever computed them, so results do not depend on how the op was dealt.
//
// Roles of a CTA:
//   producer warp   : walks the op list, streams units into a ring of shared-memory stages with bulk
//                     asynchronous copies (cp.async.bulk + mbarrier tx counts; it runs ahead across op and
//                     phase boundaries because weights do not depend on activations) and deals the
//                     blobs of every unit round-robin into per-warp queues;
//   consumer warps  : 16 warps.  An item is one blob (32 rows x 512 columns): the arithmetic of
//                     fq_gemv_core.cuh, then the 32 row sums go to the strip's slot in shared memory
//                     (or to global memory for a strip finished elsewhere).  The warp that delivers a
//                     strip's last item adds the blob sums up, writes y and counts the strip for its phase;
//   x-prep warps    : convert the activations of every blob this CTA needs into 16-bit fixed point per
//                     group of 128 columns (two signed byte digits, B-fragment order) in a ring of blob
//                     slots; before the first blob of an op they wait -- bounded -- until every CTA has
//                     finished the previous dependency phase.
// Every wait has a time limit; when one runs out the kernel records FQ_ERR_TIMEOUT, every role leaves its
// loop, the producer waits for its copies in flight and the CTA returns.
#include <cuda_fp16.h>

#include <atomic>

#include "fq_internal.cuh"
#include "fq_ptx.cuh"
#include "fq_gemv_core.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

namespace {

constexpr int kCW = 16;                                // consumer warps; consecutive blobs go to consecutive warps
constexpr int kKLanes = kCW;
constexpr int kProducerWarp = kCW;
constexpr int kPrepWarp = kCW + 1;                     // first activation pre-processing warp
constexpr int kPrepWarps = 8;                          // the eight blobs of a 4096-column activation vector convert side by side
constexpr int kThreads = (kCW + 1 + kPrepWarps) * 32;
constexpr int kStageBytes = 34816;                     // one unit: 4 x 4-bit blobs or 2 x 8-bit blobs
constexpr int kBlobsMax = 6;                           // blobs per unit, at most (< kKLanes: a warp gets at most one item of a unit)
constexpr int kXSlots = 28;                            // activation blobs resident in shared memory
constexpr int kStripSlots = 5;                         // strips whose items are in flight
constexpr int kMaxKb = 28;                             // blobs per strip, at most (k_in <= 14336)
constexpr int kQD = 8;                                 // entries per consumer queue
constexpr int kMaxPhasesDev = 1024;
constexpr int kMaxOpsDev = 512;                        // ops of one launch (their per-CTA ranges sit in shared memory)

// What the producer tells a consumer warp about one item (one 16-byte store, one 16-byte load).
//   w0 blob shared address   w1 packed fields (below)   w2 activation blob number + 1   w3 sequence tag
constexpr uint32_t kItemEnd = 1u << 31;
__device__ __forceinline__ uint32_t item_pack(int xslot, int stage, int parity, int kb, int sslot, int variant, int tsel)
{
    return (uint32_t)xslot | (uint32_t)stage << 5 | (uint32_t)parity << 9 | (uint32_t)kb << 10 | (uint32_t)sslot << 15 |
           (uint32_t)variant << 18 | (uint32_t)tsel << 22;
}

// A strip in flight.
struct StripDesc {
    uint16_t* y;                             // output of the op
    unsigned long long* partial;             // tagged blob sums of this strip in global memory: [blob][32 rows]
    int n_out, row_base;
    int n_kb, kb_lo, kb_hi;                  // blobs of the strip; [kb_lo, kb_hi) are computed by this CTA
    int finish;                              // this CTA owns the first blob: it adds up and writes y
    int phase;
    int expect;                              // items of this CTA in the strip
    int pad[4];
};
static_assert(sizeof(StripDesc) == 64, "descriptor layout");

struct Smem {
    static constexpr int kFixed = kXSlots * (kXBlobDigitBytes + kXBlobGroupBytes + 8) + 1024 + kStripSlots * kMaxKb * 128 +
                                  kCW * kQD * 16 + kStripSlots * 64 + kMaxPhasesDev + kMaxOpsDev * 8 + 1024;
    static constexpr int kStages = (232448 - kFixed) / kStageBytes;
    static constexpr int oStages = 0;
    static constexpr int oXDig = oStages + kStages * kStageBytes;            // [slot][1024]
    static constexpr int oXGrp = oXDig + kXSlots * kXBlobDigitBytes;         // [slot][32]
    static constexpr int oZero = oXGrp + kXSlots * kXBlobGroupBytes;         // 1024 zero bytes
    static constexpr int oPart = oZero + 1024;                               // float [strip slot][blob][32 rows]
    static constexpr int oQueue = oPart + kStripSlots * kMaxKb * 128;        // uint4 [warp][kQD]
    static constexpr int oStrip = oQueue + kCW * kQD * 16;                   // StripDesc [strip slot]
    static constexpr int oRange = oStrip + kStripSlots * 64;                 // uint2 [op]: this CTA's strips of every op
    static constexpr int oFinTot = oRange + kMaxOpsDev * 8;                  // u8 [phase]: strips this CTA finishes
    static constexpr int oBars = oFinTot + kMaxPhasesDev;                    // full[S], empty[S], then one per activation slot
    static constexpr int oCtl = oBars + 2 * 16 * 8 + kXSlots * 8;
    // control words (u32 each)
    static constexpr int cXTag = 0;                                          // [kXSlots] activation blob number + 1 held
    static constexpr int cXCnt = cXTag + kXSlots;                            // [kXSlots] items that still need the slot
    static constexpr int cStripCnt = cXCnt + kXSlots;                        // [kStripSlots] items delivered
    static constexpr int cStripBusy = cStripCnt + kStripSlots;               // [kStripSlots]
    static constexpr int cFinCnt = cStripBusy + kStripSlots;                 // [8] strips finished, per phase & 7
    static constexpr int cPhaseKnown = cFinCnt + 8;                          // phases 0 .. value - 1 are complete
    static constexpr int cPollLock = cPhaseKnown + 1;                        // one warp at a time polls the phase counters
    static constexpr int cAbort = cPollLock + 1;
    static constexpr int kCtlWords = cAbort + 1;
    static constexpr int kTotal = oCtl + kCtlWords * 4;
    static_assert(kStages >= 4 && kStages <= 16, "decode kernel: ring size");
    static_assert(kTotal <= 232448, "decode kernel: shared memory over the 227 KB per-CTA limit");
    static_assert(oBars % 8 == 0 && oQueue % 16 == 0 && oStrip % 16 == 0 && oXDig % 128 == 0 && oZero % 128 == 0 &&
                  oRange % 8 == 0, "alignment");
};

struct Args {
    const GemvOp* table;                   // device op table (nullptr: the by-value op)
    const int* phase_total;                // CTAs that finish at least one strip, per phase
    const uint2* ranges;                   // [cta][op] strips of every op for every CTA (nullptr: computed here)
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

// The strips of one op for one CTA: rp_first .. rp_last; the first starts at blob c_first, the last ends
// before blob c_last (see cta_work).  Packed into two words per (CTA, op) by the host for a stack call.
constexpr uint32_t kRangeEmpty = 0xffffffffu;
FQ_HD uint2 pack_range(const CtaWork& w, int n_kb)
{
    if (!w.any()) return uint2{kRangeEmpty, 0u};
    int f0, f1, l0, l1;
    w.chunks(n_kb, w.rp_first, f0, f1);
    w.chunks(n_kb, w.rp_last, l0, l1);
    return uint2{(uint32_t)w.rp_first | (uint32_t)f0 << 20, (uint32_t)w.rp_last | (uint32_t)l1 << 20};
}
struct StripOrder {
    int rp_first, rp_last, c_first, c_last, n_kb, n_strips;
    __device__ __forceinline__ StripOrder(uint2 r, int n_kb_)
    {
        n_kb = n_kb_;
        if (r.x == kRangeEmpty) { n_strips = 0; rp_first = rp_last = c_first = c_last = 0; return; }
        rp_first = (int)(r.x & 0xfffffu); c_first = (int)(r.x >> 20);
        rp_last = (int)(r.y & 0xfffffu); c_last = (int)(r.y >> 20);
        n_strips = rp_last - rp_first + 1;
    }
    __device__ __forceinline__ int strip(int i) const { return rp_first + i; }
    // blobs [c0, c1) of strip rp that belong to this CTA
    __device__ __forceinline__ void chunks(int rp, int& c0, int& c1) const
    {
        c0 = rp == rp_first ? c_first : 0;
        c1 = rp == rp_last ? c_last : n_kb;
    }
    // strips that this CTA finishes (it owns their first blob)
    __device__ __forceinline__ int finishing() const { return n_strips == 0 ? 0 : n_strips - (c_first > 0 ? 1 : 0); }
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
// One blob (two supersteps of 256 columns, 8 per lane each) of fp16 activations -> fixed point per group of
// 128 columns: x_int = rint(x * 2^(13 - E)) with 2^E <= max|x| < 2^(E+1), stored as two signed byte digits in
// B-fragment order, plus per group the integer sum and the factor 2^(E - 13).  A group that holds an
// infinity or a NaN gets the factor NaN, so that every row sum that touches it comes out NaN.  The two
// supersteps are independent chains of shuffles and conversions: written side by side so that their
// latencies overlap.
__device__ __forceinline__ void convert_blob(const uint4 (&raw)[2], uint8_t* xdig, uint8_t* xgrp, int lane)
{
    float f[2][8], amax[2];
    bool bad[2];
#pragma unroll
    for (int ss = 0; ss < 2; ss++) {
        const __half2* h2 = reinterpret_cast<const __half2*>(&raw[ss]);
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const float2 t2 = __half22float2(h2[i]);
            f[ss][2 * i] = t2.x; f[ss][2 * i + 1] = t2.y;
        }
        float m01 = fmaxf(fabsf(f[ss][0]), fabsf(f[ss][1])), m23 = fmaxf(fabsf(f[ss][2]), fabsf(f[ss][3]));
        float m45 = fmaxf(fabsf(f[ss][4]), fabsf(f[ss][5])), m67 = fmaxf(fabsf(f[ss][6]), fabsf(f[ss][7]));
        amax[ss] = fmaxf(fmaxf(m01, m23), fmaxf(m45, m67));
        // an infinity or a NaN: |x| <= 65504 fails for both (fmaxf drops a NaN, so test the elements)
        bool ok = true;
#pragma unroll
        for (int i = 0; i < 8; i++) ok = ok && (fabsf(f[ss][i]) <= 65504.f);
        bad[ss] = !ok;
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
        amax[0] = fmaxf(amax[0], __shfl_xor_sync(0xffffffffu, amax[0], o));
        amax[1] = fmaxf(amax[1], __shfl_xor_sync(0xffffffffu, amax[1], o));
    }
    const unsigned badmask0 = __ballot_sync(0xffffffffu, bad[0]), badmask1 = __ballot_sync(0xffffffffu, bad[1]);
    bad[0] = ((badmask0 >> (lane & 16)) & 0xffffu) != 0u;       // anywhere in this lane's group of 16 lanes
    bad[1] = ((badmask1 >> (lane & 16)) & 0xffffu) != 0u;
    int xi[2][8], sum[2];
    float back[2];
#pragma unroll
    for (int ss = 0; ss < 2; ss++) {
        const int eb = (__float_as_int(amax[ss]) >> 23) & 0xff;  // biased exponent of the group maximum
        const bool fin = amax[ss] > 0.f && !bad[ss];
        const float mult = fin ? __int_as_float((267 - eb) << 23) : 0.f;
        back[ss] = bad[ss] ? __int_as_float(0x7fc00000) : (fin ? __int_as_float((eb - 13) << 23) : 0.f);
#pragma unroll
        for (int i = 0; i < 8; i++) xi[ss][i] = bad[ss] ? 0 : __float2int_rn(f[ss][i] * mult);
        sum[ss] = ((xi[ss][0] + xi[ss][1]) + (xi[ss][2] + xi[ss][3])) + ((xi[ss][4] + xi[ss][5]) + (xi[ss][6] + xi[ss][7]));
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
        sum[0] += __shfl_xor_sync(0xffffffffu, sum[0], o);
        sum[1] += __shfl_xor_sync(0xffffffffu, sum[1], o);
    }
    // lane l holds columns 8l .. 8l+7 of a superstep: k32 step j = l >> 2, half (l >> 1) & 1, column blocks c0, c0 + 1
    const int j = lane >> 2, half = (lane >> 1) & 1, c0 = 2 * (lane & 1);
#pragma unroll
    for (int ss = 0; ss < 2; ss++) {
        // signed digits base 256 of four values at a time: low byte as is, high byte + carry
        uint32_t lo4[2], hi4[2];
#pragma unroll
        for (int r = 0; r < 2; r++) {
            const uint32_t p01 = __byte_perm((uint32_t)xi[ss][4 * r + 0], (uint32_t)xi[ss][4 * r + 1], 0x5410);
            const uint32_t p23 = __byte_perm((uint32_t)xi[ss][4 * r + 2], (uint32_t)xi[ss][4 * r + 3], 0x5410);
            const uint32_t h01 = (((p01 >> 8) & 0x00ff00ffu) + ((p01 >> 7) & 0x00010001u)) & 0x00ff00ffu;
            const uint32_t h23 = (((p23 >> 8) & 0x00ff00ffu) + ((p23 >> 7) & 0x00010001u)) & 0x00ff00ffu;
            lo4[r] = __byte_perm(p01, p23, 0x6420);
            hi4[r] = __byte_perm(h01, h23, 0x6420);
        }
        uint8_t* cell = xdig + x_digit_off(ss, j & 3, 0, c0) + (2 * (j >> 2) + half) * 4;
        *reinterpret_cast<uint32_t*>(cell) = lo4[0];
        *reinterpret_cast<uint32_t*>(cell + 16) = lo4[1];
        *reinterpret_cast<uint32_t*>(cell + 64) = hi4[0];
        *reinterpret_cast<uint32_t*>(cell + 64 + 16) = hi4[1];
        if ((lane & 15) == 0) {
            reinterpret_cast<int*>(xgrp)[ss * 2 + (lane >> 4)] = sum[ss];
            reinterpret_cast<float*>(xgrp + 16)[ss * 2 + (lane >> 4)] = back[ss];
        }
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
    unsigned char* fin_total = smem + S::oFinTot;
    const uint2* range = reinterpret_cast<const uint2*>(smem + S::oRange);
    const GemvOp* ops = a.table ? a.table : &single;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; s++) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 128 + 8 * s, kCW);
        }
        for (int s = 0; s < kXSlots; s++) mbar_init(bars + 256 + 8 * s, 1);   // completes once per publication of the slot
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = threadIdx.x; i < S::kCtlWords; i += blockDim.x) ctl[i] = 0u;
    for (int i = threadIdx.x; i < 256; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + S::oZero)[i] = 0u;
    for (int i = threadIdx.x; i < kCW * kQD * 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + S::oQueue)[i] = 0u;
    for (int i = threadIdx.x; i < kMaxPhasesDev / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(fin_total)[i] = 0u;
    // this CTA's strips of every op
    for (int oi = threadIdx.x; oi < a.n_ops; oi += blockDim.x) {
        uint2 r;
        if (a.ranges) r = a.ranges[(long long)cta * a.n_ops + oi];
        else r = pack_range(cta_work(ops[oi].n_units, ops[oi].n_kb, ops[oi].rot, cta, grid), ops[oi].n_kb);
        reinterpret_cast<uint2*>(smem + S::oRange)[oi] = r;
    }
    __syncthreads();
    // strips that this CTA finishes, per phase (the warp that finishes the last one reports the phase)
    if (a.n_phases > 0) {
        for (int oi = threadIdx.x; oi < a.n_ops; oi += blockDim.x) {
            const int phase = ops[oi].phase;
            const int fin = StripOrder(range[oi], ops[oi].n_kb).finishing();
            if (fin > 0 && phase >= 0)                              // four 8-bit counters per word
                atomicAdd(reinterpret_cast<unsigned*>(fin_total) + (phase >> 2), (unsigned)fin << (8 * (phase & 3)));
        }
    }
    __syncthreads();

    if (warp == kProducerWarp) {
        // ================================================================== producer
        // This loop is the serial path that feeds the whole CTA: per unit it costs lane 0 a barrier test, the
        // transaction count, one bulk copy and one arrival; the item descriptors are written by the lanes of
        // the warps they are meant for (lane w keeps the number of entries queued for consumer warp w).
        int stage = 0;
        unsigned wraps = 0;
        unsigned rr = 0;                              // K lane of the next blob (round-robin over everything)
        unsigned xseq = 0;                            // activation blobs of the ops seen so far
        unsigned strip_seq = 0;
        unsigned qn = 0;                              // lane w < kCW: entries queued for consumer warp w
        bool stop = false;
        const uint32_t sdesc_a = sbase + S::oStrip;
        const unsigned long long stream_policy = l2_policy_evict_first();      // weights are read once per pass
        const uint32_t my_queue = sbase + S::oQueue + (uint32_t)(lane & (kCW - 1)) * kQD * 16u;
        const int my_klane = lane & (kKLanes - 1);
        // The descriptor of the next op travels while the units of the current one are issued.
        struct OpRegs {
            const uint8_t* store;
            unsigned long long* partial;
            uint16_t* y;
            int blob_read, blob_stride, n_kb, cb, variant, n_out, phase, split;
            __device__ __forceinline__ void fetch(const GemvOp* ops, int oi, int n_ops)
            {
                if (oi >= n_ops) return;
                const GemvOp& o = ops[oi];
                store = o.store; partial = o.partial; y = o.y; blob_read = o.blob_read; blob_stride = o.blob_stride;
                n_kb = o.n_kb; cb = o.chunk_blobs; variant = o.variant; n_out = o.n_out; phase = o.phase;
                split = o.split == 2 ? 2 : 1;
            }
        };
        OpRegs nxt;
        nxt.fetch(ops, 0, a.n_ops);
        for (int oi = 0; oi < a.n_ops && !stop; oi++) {
            const OpRegs cur = nxt;
            nxt.fetch(ops, oi + 1, a.n_ops);
            const int n_kb = cur.n_kb, cb = cur.cb, variant = cur.variant, n_out = cur.n_out, phase = cur.phase;
            const int split = cur.split;                 // items per blob: the whole blob, or one 16-row tile each
            const StripOrder so(range[oi], n_kb);
            if (so.n_strips == 0) continue;
            const uint32_t blob_read = (uint32_t)cur.blob_read;
            const long long blob_stride = cur.blob_stride;
            const uint8_t* const store = cur.store;
            uint16_t* const y = cur.y;
            unsigned long long* const partial = cur.partial;
            const bool contiguous = cur.blob_read == cur.blob_stride;
            for (int si = 0; si < so.n_strips && !stop; si++) {
                const int rp = so.strip(si);
                int c0, c1;
                so.chunks(rp, c0, c1);
                const int kb_lo = c0, kb_hi = c1;
                const int sslot = (int)(strip_seq % kStripSlots);
                strip_seq++;
                int slot_ok = 1;
                if (lane == 0 && !wait_smem([&] { return ctl[S::cStripBusy + sslot] == 0u; }, ctl, a.wait_ns)) {
                    if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                    slot_ok = 0;
                }
                if (!__shfl_sync(0xffffffffu, slot_ok, 0)) { stop = true; break; }   // (every loop exit is decided by lane 0)
                {
                    // the strip's descriptor: three lanes store 16 bytes each
                    unsigned long long* const sp = partial + (long long)rp * n_kb * 32;
                    uint4 d;
                    if (lane == 0) d = make_uint4((uint32_t)(uintptr_t)y, (uint32_t)((uintptr_t)y >> 32), (uint32_t)(uintptr_t)sp,
                                                  (uint32_t)((uintptr_t)sp >> 32));
                    else if (lane == 1) d = make_uint4((uint32_t)n_out, (uint32_t)(rp * (kBlobTiles * kTileRows)), (uint32_t)n_kb, (uint32_t)kb_lo);
                    else d = make_uint4((uint32_t)kb_hi, c0 == 0 ? 1u : 0u, (uint32_t)phase, (uint32_t)((kb_hi - kb_lo) * split));
                    if (lane < 3) sts128(sdesc_a + (uint32_t)sslot * 64u + (uint32_t)lane * 16u, d);
                    if (lane == 0) ctl[S::cStripBusy + sslot] = 1u;
                    __threadfence_block();                           // the descriptor before any item that refers to it
                    __syncwarp();
                }
                const uint8_t* src = store + ((long long)rp * n_kb + kb_lo) * blob_stride;
                for (int kb = kb_lo; kb < kb_hi; kb += cb) {
                    const int nb = min(cb, kb_hi - kb);
                    const uint32_t full = bars + 8 * stage, empty = bars + 128 + 8 * stage;
                    const uint32_t stage_base = sbase + S::oStages + (uint32_t)stage * kStageBytes;
                    // (checked build) the blobs of this copy lie inside the stored variant and fit the stage
                    if (!FQ_IN_BOUNDS(rp >= 0 && rp < row_pairs(n_out) && kb >= 0 && kb + nb <= n_kb &&
                                      (uint32_t)nb * blob_read <= (uint32_t)kStageBytes && sslot < kStripSlots, a.status)) {
                        if (lane == 0) ctl[S::cAbort] = 1u;
                        stop = true;
                        break;
                    }
                    int ok = 1;
                    if (lane == 0) {
                        if (wraps > 0 && !wait_mbar(empty, (wraps - 1u) & 1u, ctl, a.wait_ns)) {
                            if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                            ok = 0;
                        }
                        if (ok) {
                            mbar_expect_tx(full, (uint32_t)nb * blob_read);
                            if (contiguous) bulk_g2s_hint(stage_base, src, (uint32_t)nb * blob_read, full, stream_policy);
                            mbar_arrive_n(empty, (uint32_t)(kCW - nb * split));   // for the warps without an item in this unit
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, ok, 0);
                    if (!ok) { stop = true; break; }
                    if (!contiguous && lane < nb) bulk_g2s_hint(stage_base + lane * blob_read, src + lane * blob_stride, blob_read, full, stream_policy);
                    // the items of this unit: item i goes to consumer warp (rr + i) mod 16; item i is blob i, or tile
                    // i % 2 of blob i / 2
                    const int item = (int)((unsigned)my_klane - rr) & (kKLanes - 1);
                    if (lane < kCW && item < nb * split) {
                        const int b = split == 2 ? item >> 1 : item;
                        const int tsel = split == 2 ? 1 + (item & 1) : 0;
                        const unsigned xs = xseq + (unsigned)(kb + b);
                        uint4 e;
                        e.x = stage_base + (uint32_t)b * blob_read;
                        e.y = item_pack((int)(xs % kXSlots), stage, (int)(wraps & 1u), kb + b, sslot, variant, tsel);
                        e.z = xs + 1u;
                        e.w = qn + 1u;
                        sts128(my_queue + (qn % kQD) * 16u, e);
                        qn++;
                    }
                    rr += (unsigned)(nb * split);
                    src += (long long)nb * blob_stride;
                    if (++stage == S::kStages) { stage = 0; wraps++; }
                }
            }
            xseq += (unsigned)n_kb;
        }
        // the end marker of every queue
        if (lane < kCW) {
            // (the queue slot is free: a warp gets one entry per kCW blobs, so the entry that used the slot
            // kQD entries ago belongs to a unit whose stage has been refilled since, i.e. it was consumed)
            sts128(my_queue + (qn % kQD) * 16u, make_uint4(0u, kItemEnd, 0u, qn + 1u));
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
        // The activation blobs of all ops this CTA takes part in form one sequence; warp pw converts the blobs
        // whose number is congruent to pw.  The loads of a warp's next blob travel while it converts the
        // current one; they are only issued once the op's phase is known to be open.
        const int pw = warp - kPrepWarp;
        const unsigned long long keep_policy = l2_policy_evict_last();         // activations come back every pass
        struct Item {
            const __half* x;
            int k_in, kb, uses, phase;
            unsigned xs;
        };
        // iterator over this warp's blobs
        int it_oi = -1, it_kb = 0, it_nkb = 0, it_kin = 0, it_phase = -1;
        int fk0 = 0, fk1 = 0, lk0 = 0, lk1 = 0, n_mid = 0, two = 0, it_split = 1;
        unsigned xbase = 0;
        const __half* it_x = nullptr;
        auto advance = [&](Item& it) -> bool {
            for (;;) {
                if (it_kb < it_nkb) {
                    int uses = n_mid + ((it_kb >= fk0 && it_kb < fk1) ? 1 : 0) + ((two && it_kb >= lk0 && it_kb < lk1) ? 1 : 0);
                    uses *= it_split;                                // items, not blobs, count down the slot
                    it.x = it_x; it.k_in = it_kin; it.kb = it_kb; it.uses = uses; it.phase = it_phase;
                    it.xs = xbase + (unsigned)it_kb;
                    it_kb += kPrepWarps;
                    return true;
                }
                xbase += (unsigned)it_nkb;
                it_nkb = 0;
                do { it_oi++; } while (it_oi < a.n_ops && range[it_oi].x == kRangeEmpty);
                if (it_oi >= a.n_ops) return false;
                prefetch_ops(ops, it_oi, a.n_ops, lane);
                const GemvOp& op = ops[it_oi];
                const StripOrder so(range[it_oi], op.n_kb);
                it_nkb = op.n_kb; it_kin = op.k_in; it_phase = op.phase; it_split = op.split == 2 ? 2 : 1;
                it_x = reinterpret_cast<const __half*>(op.x);
                // blobs of x that this CTA's strips cover: the first and the last strip may be partial
                int f0, f1, l0, l1;
                so.chunks(so.rp_first, f0, f1);
                so.chunks(so.rp_last, l0, l1);
                fk0 = f0; fk1 = f1; lk0 = l0; lk1 = l1;
                n_mid = so.n_strips > 2 ? so.n_strips - 2 : 0;
                two = so.n_strips > 1;
                it_kb = (int)(((unsigned)pw + kPrepWarps - xbase % kPrepWarps) % kPrepWarps);
            }
        };
        // Is the phase that produces this op's activations complete?  (phases are opened in order)
        auto phase_open = [&](int phase) -> bool { return phase <= 0 || (int)ctl[S::cPhaseKnown] >= phase; };
        // Waits -- bounded -- until it is.  One warp of the CTA at a time polls the counters in global memory,
        // always the earliest phase that is not known to be complete (a warp whose next blob belongs to a
        // later phase must not keep a warp that still has to convert an earlier phase's activations from
        // learning that it may go ahead); the others watch the word it updates in shared memory.
        auto phase_wait = [&](int phase) -> bool {
            int ok = 1;
            if (lane == 0 && !phase_open(phase)) {
                const unsigned long long t0 = global_ns();
                unsigned it = 0;
                for (;;) {
                    if (phase_open(phase)) break;
                    if (atomicCAS(const_cast<unsigned*>(&ctl[S::cPollLock]), 0u, 1u) == 0u) {
                        while (ok && !phase_open(phase)) {
                            const int p = (int)ctl[S::cPhaseKnown];                  // phases 0 .. p - 1 are complete
                            const unsigned long long need = (unsigned long long)a.phase_total[p];
                            while (ld_acquire_u64(a.phase_done + p) < need) {
                                if ((++it & 31u) == 0u &&
                                    (ctl[S::cAbort] || global_ns() - t0 > a.wait_ns || *reinterpret_cast<volatile int*>(a.status) != 0)) {
                                    ok = 0; break;
                                }
                            }
                            if (ok) ctl[S::cPhaseKnown] = (unsigned)(p + 1);
                        }
                        __threadfence_block();
                        ctl[S::cPollLock] = 0u;
                        break;
                    }
                    __nanosleep(20);
                    if ((++it & 63u) == 0u && (ctl[S::cAbort] || global_ns() - t0 > a.wait_ns)) { ok = 0; break; }
                }
                if (!ok && !ctl[S::cAbort]) raise_timeout(a, ctl);
            }
            return __shfl_sync(0xffffffffu, ok, 0) != 0;
        };
        auto load = [&](const Item& it, uint4& r0, uint4& r1) {
            r0 = r1 = make_uint4(0u, 0u, 0u, 0u);
            const int k = it.kb * 512 + lane * 8;
            if (it.uses > 0) {
                if (k < it.k_in && FQ_IN_BOUNDS(k + 8 <= it.k_in, a.status)) r0 = ldg128_hint(it.x + k, keep_policy);
                if (k + 256 < it.k_in && FQ_IN_BOUNDS(k + 264 <= it.k_in, a.status)) r1 = ldg128_hint(it.x + k + 256, keep_policy);
            }
        };
        // Converts a blob into its slot and publishes it.  False: a wait ran out.
        auto process = [&](const Item& it, uint4 r0, uint4 r1) -> bool {
            const int slot = (int)(it.xs % kXSlots);
            int ok = 1;
            // the slot is free when the blob it held before has been published and every item that needed it is done
            const unsigned prev_tag = it.xs >= (unsigned)kXSlots ? it.xs - (unsigned)kXSlots + 1u : 0u;
            if (lane == 0 && !wait_smem([&] { return ctl[S::cXTag + slot] == prev_tag && ctl[S::cXCnt + slot] == 0u; }, ctl, a.wait_ns)) {
                if (!ctl[S::cAbort]) raise_timeout(a, ctl);
                ok = 0;
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
            if (it.uses > 0) {
                uint8_t* xdig = smem + S::oXDig + slot * kXBlobDigitBytes;
                uint8_t* xgrp = smem + S::oXGrp + slot * kXBlobGroupBytes;
                const uint4 raw[2] = {r0, r1};
                convert_blob(raw, xdig, xgrp, lane);
            }
            __threadfence_block();
            __syncwarp();
            if (lane == 0) {
                ctl[S::cXCnt + slot] = (unsigned)it.uses;
                ctl[S::cXTag + slot] = it.xs + 1u;
                __threadfence_block();
                mbar_arrive(bars + 256 + 8 * slot);                        // wakes the consumers that sleep on this slot
            }
            return true;
        };
        Item A, B;
        uint4 ra0, ra1, rb0, rb1;
        bool va = advance(A);
        if (va) {
            if (!phase_wait(A.phase)) va = false;
            else load(A, ra0, ra1);
        }
        while (va) {
            const bool vb = advance(B);
            bool issued = false;
            if (vb && __shfl_sync(0xffffffffu, phase_open(B.phase) ? 1 : 0, 0)) { load(B, rb0, rb1); issued = true; }
            if (!process(A, ra0, ra1)) break;
            if (vb && !issued) {
                if (!phase_wait(B.phase)) break;
                load(B, rb0, rb1);
            }
            A = B; ra0 = rb0; ra1 = rb1; va = vb;
        }
    } else {
        // ================================================================== consumers
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
            const int tsel = (int)((e.y >> 22) & 3u);                        // 0: both tiles, 1 / 2: tile 0 / 1 only
            // ---- its weights and its activations
            bool ok = wait_mbar(bars + 8 * stage, (uint32_t)parity, ctl, a.wait_ns);
            // (a hardware wake-up: at the start of a dependency phase every consumer sleeps here and must not
            // take issue slots from the pre-processing warps; the slot's barrier completes once per publication)
            if (ok) ok = wait_mbar(bars + 256 + 8 * xslot, ((e.z - 1u) / kXSlots) & 1u, ctl, a.wait_ns);
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
            float tot[kBlobTiles][2] = {{0.f, 0.f}, {0.f, 0.f}};
            blob_dispatch(variant, e.x, xd, sbase + S::oXGrp + (uint32_t)xslot * kXBlobGroupBytes, lane, tsel, tot);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bars + 128 + 8 * stage);                         // the stage may be refilled
                atomicSub(const_cast<unsigned*>(&ctl[S::cXCnt + xslot]), 1u);   // one item fewer needs the activation blob
            }
            // ---- the 32 row sums of the item: add up the step classes held by the quad; lane c of the quad
            //      then keeps the sum of row 16 (c >> 1) + g + 8 (c & 1)
#pragma unroll
            for (int tl = 0; tl < kBlobTiles; tl++)
#pragma unroll
                for (int r = 0; r < 2; r++) {
                    tot[tl][r] += __shfl_xor_sync(0xffffffffu, tot[tl][r], 1);
                    tot[tl][r] += __shfl_xor_sync(0xffffffffu, tot[tl][r], 2);
                }
            const StripDesc& d = sdesc[sslot];
            const int finish = d.finish, expect = d.expect;                  // (read before this item is counted)
            unsigned long long* const dpart = d.partial;
            {
                const float v = c == 0 ? tot[0][0] : c == 1 ? tot[0][1] : c == 2 ? tot[1][0] : tot[1][1];
                const int lr = (c >> 1) * kTileRows + g + 8 * (c & 1);
                if ((tsel == 0 || (c >> 1) == tsel - 1) &&                    // (rows of the tile(s) this item computed)
                    FQ_IN_BOUNDS(kb >= 0 && kb < d.n_kb && kb < kMaxKb && sslot >= 0 && sslot < kStripSlots, a.status)) {
                    if (finish) part[(sslot * kMaxKb + kb) * 32 + lr] = v;
                    else st_relaxed_u64(dpart + kb * 32 + lr, tag | __float_as_uint(v));   // finished elsewhere
                }
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
                // lane = row of the strip; blob sums in blob order: this CTA's from shared memory, then the blobs
                // of other CTAs from their tagged words
                const int n_kb = d.n_kb, kb_hi = d.kb_hi;
                float sum = 0.f;
                const float* ps = part + (sslot * kMaxKb) * 32 + lane;
                for (int q0 = 0; q0 < kb_hi; q0 += 8) {                      // eight loads in flight, added in blob order
                    float pv[8];
#pragma unroll
                    for (int i = 0; i < 8; i++) pv[i] = q0 + i < kb_hi ? ps[(q0 + i) * 32] : 0.f;
#pragma unroll
                    for (int i = 0; i < 8; i++) if (q0 + i < kb_hi) sum += pv[i];
                }
                if (kb_hi < n_kb) {
                    // eight words in flight per round trip; a round whose words are not all there is repeated
                    const unsigned long long t0 = global_ns();
                    unsigned it = 0;
                    for (int q0 = kb_hi; q0 < n_kb && live; q0 += 8) {
                        unsigned long long wv[8];
                        for (;;) {
                            bool all = true;
#pragma unroll
                            for (int i = 0; i < 8; i++) wv[i] = q0 + i < n_kb ? ld_relaxed_u64(d.partial + (q0 + i) * 32 + lane) : tag;
#pragma unroll
                            for (int i = 0; i < 8; i++) all = all && (unsigned)(wv[i] >> 32) == a.epoch;
                            if (__all_sync(0xffffffffu, all)) break;
                            __nanosleep(64);
                            int giveup = 0;
                            if (lane == 0 && (++it & 15u) == 0u && (ctl[S::cAbort] || global_ns() - t0 > a.wait_ns)) giveup = 1;
                            if (__shfl_sync(0xffffffffu, giveup, 0)) { live = false; break; }
                        }
#pragma unroll
                        for (int i = 0; i < 8; i++) if (q0 + i < n_kb) sum += __uint_as_float((unsigned)wv[i]);
                    }
                    if (!live && lane == 0 && !ctl[S::cAbort]) raise_timeout(a, ctl);
                }
                if (live) {
                    const int row = d.row_base + lane;
                    if (row < d.n_out && FQ_IN_BOUNDS(row >= 0, a.status)) reinterpret_cast<__half*>(d.y)[row] = __float2half_rn(sum);
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
                        if (FQ_IN_BOUNDS(phase < a.n_phases, a.status)) red_add_relaxed_u64(a.phase_done + phase, 1ull);
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
int gemv1_max_ops() { return kMaxOpsDev; }
uint2 gemv1_pack_range(const CtaWork& w, int n_chunks) { return pack_range(w, n_chunks); }
int gemv1_max_k() { return kMaxKb * 512; }
int gemv1_chunk_blobs(int blob_read_bytes)
{
    const int c = kStageBytes / blob_read_bytes;
    return c > kBlobsMax ? kBlobsMax : (c < 1 ? 1 : c);
}

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
    const size_t np = hdr.n_phases > 0 ? hdr.n_phases : 1;
    a.ranges = reinterpret_cast<const uint2*>(
        table_dev + (size_t)round_up((int64_t)((size_t)hdr.n_ops * sizeof(GemvOp) + np * sizeof(int)), 8));
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
    static std::atomic<unsigned> epoch[64];      // one tag counter per device, shared by every context and host thread
    if (partial_bytes > FQ_STATIC_SCRATCH_BYTES) return FQ_ERR_SCRATCH;
    unsigned char* base = nullptr;
    const int rc = static_scratch_address(ctx->device, &base);
    if (rc != FQ_OK) return rc;
    op.partial = reinterpret_cast<unsigned long long*>(base);
    Args a{};
    a.status = ctx->status_dev;
    a.n_ops = 1;
    unsigned e = epoch[ctx->device].fetch_add(1u) + 1u;
    if (e == 0u) e = epoch[ctx->device].fetch_add(1u) + 1u;      // 0 marks words that no launch has written
    a.epoch = e;
    a.wait_ns = ctx->wait_limit_ns;
    return launch(ctx, op, a, op.n_units, st);
}

}  // namespace fq

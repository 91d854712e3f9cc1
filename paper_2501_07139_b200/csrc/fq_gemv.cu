// Decode path: fused dequantize-GEMV over tiled field arrays, batch 1..8.
//
// One persistent CTA per SM.  A producer thread streams "units" (16 output rows x a chunk
// of K: every field array of the active variant plus the scale/zero words) from HBM into a
// shared-memory ring with bulk asynchronous copies (cp.async.bulk + mbarrier transaction
// counts).  Eight consumer warps each take one unit at a time: stored words become
// mma.m16n8k16 A-operands with one shift and one AND (the integer field sits in the
// mantissa of an fp16 subnormal, i.e. the tensor core sees field * 2^-24 exactly), the
// activations are the B operand (column n = batch entry), accumulation is fp32.  Per group
// of 128 columns:   y += s * (sum_fields 2^shift * sum_k field_k x_k  -  z * sum_k x_k).
// K chunks of one row tile are combined through fp32 partials in a workspace; the last
// arriver adds them in chunk order, so results do not depend on scheduling.
//
// A whole stack of layers runs as one launch: units of consecutive ops are dealt round-robin
// to the CTAs, the producer runs ahead across op boundaries (weights do not depend on
// activations), and only the consumers wait -- bounded -- for the previous phase's outputs.
#include <cuda_fp16.h>

#include "fq_internal.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

constexpr int kConsumerWarps = 8;
constexpr int kGemvThreads = (kConsumerWarps + 1) * 32;
constexpr int kUnitCodeBytes = 16384;                 // code bytes of one unit, at most
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // every device-side wait gives up after 2 s

template <int MAXB> struct GemvCfg;
template <> struct GemvCfg<1> { static constexpr int kMaxSS = 8; static constexpr int kStages = 11; };
template <> struct GemvCfg<8> { static constexpr int kMaxSS = 2; static constexpr int kStages = 16; };

template <int MAXB> struct GemvSmem {
    static constexpr int kMaxSS = GemvCfg<MAXB>::kMaxSS;
    static constexpr int kStages = GemvCfg<MAXB>::kStages;
    static constexpr int kStageBytes =
        (kMaxSS * 4096 < kUnitCodeBytes ? kMaxSS * 4096 : kUnitCodeBytes) + kMaxSS * 128;
    static constexpr int kXRow = kMaxSS * kStepCols + 32;         // halves per batch row (+64 B: bank spread)
    static constexpr int kXBytes = MAXB * kXRow * 2;
    static constexpr int kXsumFloats = MAXB * kMaxSS * 2;
    // offsets
    static constexpr int oStages = 0;
    static constexpr int oX = oStages + kStages * kStageBytes;
    static constexpr int oXsum = oX + kConsumerWarps * kXBytes;
    static constexpr int oOps = oXsum + kConsumerWarps * kXsumFloats * 4;
    static constexpr int oBars = oOps + (kConsumerWarps + 1) * (int)((sizeof(GemvOp) + 15) / 16 * 16);
    static constexpr int oFlags = oBars + 2 * kStages * 8;
    static constexpr int kTotal = oFlags + 16;
};

int gemv_chunks(int n_ss, int bits, int batch)
{
    int max_ss = batch <= 1 ? GemvCfg<1>::kMaxSS : GemvCfg<8>::kMaxSS;
    const int by_bytes = kUnitCodeBytes / (512 * bits);
    if (by_bytes < max_ss) max_ss = by_bytes;
    if (max_ss < 1) max_ss = 1;
    return (n_ss + max_ss - 1) / max_ss;
}

size_t gemv_partial_floats_per_unit(int batch) { return batch <= 1 ? 16 : 128; }

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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------------------- one field, one group
// `fs`: shared-memory address of this field's data for the current superstep ([F chunks][32 lanes][16 B]).
// Adds  scale * sum_k field_k * x_k  (k over the 128 columns of group `grp`) into gt.
template <int F>
__device__ __forceinline__ void field_group(const uint8_t* fs, int grp, int lane, const uint4 (&xv)[4],
                                            float scale, float (&gt)[4])
{
    constexpr int kWords = 2 * F;                 // words of this lane that belong to one group
    constexpr int kRegsPerWord = 16 / F;
    constexpr uint32_t kMask = ((1u << F) - 1u) * 0x00010001u;
    uint32_t wd[kWords];
    if constexpr (F == 1) {
        const uint4 v = *reinterpret_cast<const uint4*>(fs + lane * 16);
        wd[0] = grp ? v.z : v.x;
        wd[1] = grp ? v.w : v.y;
    } else {
        constexpr int kChunks = F / 2;            // 16-byte chunks per group
#pragma unroll
        for (int j = 0; j < kChunks; j++) {
            const uint4 v = *reinterpret_cast<const uint4*>(fs + (grp * kChunks + j) * 512 + lane * 16);
            wd[4 * j + 0] = v.x; wd[4 * j + 1] = v.y; wd[4 * j + 2] = v.z; wd[4 * j + 3] = v.w;
        }
    }
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int m = 0; m < 8; m++) {                 // eight k16 steps per group
        uint32_t a[4];
#pragma unroll
        for (int r = 0; r < 4; r++) {
            const int idx = m * 4 + r;
            const int t = idx % kRegsPerWord;
            a[r] = (wd[idx / kRegsPerWord] >> (t * F)) & kMask;
        }
        const uint4& x4 = xv[m >> 1];
        if (m & 1) mma16816(acc, a, x4.z, x4.w);
        else       mma16816(acc, a, x4.x, x4.y);
    }
#pragma unroll
    for (int i = 0; i < 4; i++) gt[i] = fmaf(acc[i], scale, gt[i]);
}

__device__ __forceinline__ void copy_op(GemvOp* dst, const GemvOp* src, int lane, int n_lanes)
{
    const uint32_t* s = reinterpret_cast<const uint32_t*>(src);
    uint32_t* d = reinterpret_cast<uint32_t*>(dst);
    for (int i = lane; i < (int)(sizeof(GemvOp) / 4); i += n_lanes) d[i] = s[i];
}

struct StackArgs {
    const GemvOp* table;                   // device op table (nullptr: use the by-value op)
    const long long* phase_total;          // units per phase
    unsigned long long* phase_done;        // finished units per phase
    unsigned* exit_count;
    int* status;
    int n_ops, n_phases;
    long long total_units;
};

template <int MAXB>
__global__ void __launch_bounds__(kGemvThreads, 1)
gemv_kernel(const __grid_constant__ GemvOp single, const StackArgs sa)
{
    using S = GemvSmem<MAXB>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bars = smem_u32(smem + S::oBars);            // full[0..S), empty[0..S)
    volatile int* flags = reinterpret_cast<volatile int*>(smem + S::oFlags);   // [0]: soft abort, [1]: hard abort
    GemvOp* my_op = reinterpret_cast<GemvOp*>(smem + S::oOps + warp * ((sizeof(GemvOp) + 15) / 16 * 16));

    if (threadIdx.x == 0) {
        for (int s = 0; s < S::kStages; s++) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (S::kStages + s), 1);
        }
        flags[0] = 0; flags[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const long long grid = gridDim.x, cta = blockIdx.x;
    const GemvOp* src_ops = sa.table ? sa.table : &single;

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            int op_idx = 0;
            copy_op(my_op, src_ops, 0, 1);
            for (long long seq = 0;; seq++) {
                const long long u = cta + seq * grid;
                if (u >= sa.total_units || flags[1]) break;
                while (u >= my_op->unit_base + (long long)my_op->n_rt * my_op->n_chunks) {
                    op_idx++;
                    copy_op(my_op, src_ops + op_idx, 0, 1);
                }
                const GemvOp& op = *my_op;
                const int ul = (int)(u - op.unit_base);
                const int rt = ul / op.n_chunks, ch = ul % op.n_chunks;
                const int ss0 = (int)((long long)ch * op.n_ss / op.n_chunks);
                const int cnt = (int)((long long)(ch + 1) * op.n_ss / op.n_chunks) - ss0;
                const int stage = (int)(seq % S::kStages);
                const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
                if (seq >= S::kStages) {
                    if (!mbar_wait(empty, (uint32_t)((seq / S::kStages - 1) & 1))) {
                        atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT);
                        flags[1] = 1;
                        break;
                    }
                }
                mbar_expect_tx(full, (uint32_t)cnt * (512u * op.bits + 128u));
                uint32_t dst = smem_u32(smem + S::oStages + stage * S::kStageBytes);
                const long long tile0 = (long long)rt * op.n_ss + ss0;
                for (int fi = 0; fi < op.n_fields; fi++) {
                    const uint32_t f = op.field_width[fi];
                    bulk_g2s(dst, op.field_ptr[fi] + tile0 * (f * 512), cnt * f * 512, full);
                    dst += cnt * f * 512;
                }
                bulk_g2s(dst, op.meta + ((long long)rt * op.n_ss * 2 + ss0 * 2) * 16, cnt * 128, full);
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers
        uint8_t* xs_raw = smem + S::oX + warp * S::kXBytes;
        __half* xs = reinterpret_cast<__half*>(xs_raw);
        float* xsum = reinterpret_cast<float*>(smem + S::oXsum) + warp * S::kXsumFloats;
        const int g = lane >> 2, c = lane & 3;
        int op_idx = 0;
        int phase_known = -1;                       // every phase <= phase_known is complete
        copy_op(my_op, src_ops, lane, 32);
        __syncwarp();
        for (long long seq = warp;; seq += kConsumerWarps) {
            const long long u = cta + seq * grid;
            if (u >= sa.total_units || flags[1]) break;
            while (u >= my_op->unit_base + (long long)my_op->n_rt * my_op->n_chunks) {
                op_idx++;
                __syncwarp();
                copy_op(my_op, src_ops + op_idx, lane, 32);
                __syncwarp();
            }
            const GemvOp& op = *my_op;
            const int ul = (int)(u - op.unit_base);
            const int rt = ul / op.n_chunks, ch = ul % op.n_chunks;
            const int ss0 = (int)((long long)ch * op.n_ss / op.n_chunks);
            const int cnt = (int)((long long)(ch + 1) * op.n_ss / op.n_chunks) - ss0;
            const int stage = (int)(seq % S::kStages);
            const uint32_t full = bars + 8 * stage, empty = bars + 8 * (S::kStages + stage);
            const uint8_t* st = smem + S::oStages + stage * S::kStageBytes;
            const int B = op.batch;
            bool live = !flags[0];

            // ---- wait for the previous phase's outputs (they are this op's activations)
            if (live && op.phase > 0 && phase_known < op.phase - 1) {
                int ok = 1;
                if (lane == 0) {
                    const unsigned long long need = (unsigned long long)sa.phase_total[op.phase - 1];
                    const unsigned long long t0 = global_ns();
                    unsigned it = 0;
                    while (ld_acquire_u64(sa.phase_done + (op.phase - 1)) < need) {
                        __nanosleep(64);
                        if ((++it & 63u) == 0u) {
                            if (global_ns() - t0 > kWaitLimitNs ||
                                *reinterpret_cast<volatile int*>(sa.status) != 0 || flags[0]) { ok = 0; break; }
                        }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) {
                    if (lane == 0) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; }
                    live = false;
                } else {
                    phase_known = op.phase - 1;
                }
            }

            // ---- stage this unit's activations (natural order) and their per-group sums
            if (live) {
                for (int b = 0; b < B; b++) {
                    const __half* xb = reinterpret_cast<const __half*>(op.x) + (long long)b * op.k_in;
                    for (int s = 0; s < cnt; s++) {
                        const int k = (ss0 + s) * kStepCols + lane * 8;
                        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                        if (k < op.k_in) v = __ldcg(reinterpret_cast<const uint4*>(xb + k));
                        *reinterpret_cast<uint4*>(xs + b * S::kXRow + s * kStepCols + lane * 8) = v;
                        const __half2* h = reinterpret_cast<const __half2*>(&v);
                        float sum = 0.f;
#pragma unroll
                        for (int i = 0; i < 4; i++) {
                            const float2 f2 = __half22float2(h[i]);
                            sum += f2.x + f2.y;
                        }
#pragma unroll
                        for (int o = 8; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
                        if ((lane & 15) == 0) xsum[b * (S::kMaxSS * 2) + s * 2 + (lane >> 4)] = sum;
                    }
                }
            }
            __syncwarp();

            // ---- wait for the unit's weights
            if (!mbar_wait(full, (uint32_t)((seq / S::kStages) & 1))) {
                if (lane == 0) { atomicCAS(sa.status, 0, FQ_ERR_TIMEOUT); flags[0] = 1; flags[1] = 1; }
                break;
            }

            float tot[4] = {0.f, 0.f, 0.f, 0.f};
            if (live) {
                const uint32_t* meta_s = reinterpret_cast<const uint32_t*>(st + cnt * 512 * op.bits);
                const bool has_x = g < B;
                const __half* xrow = xs + (has_x ? g : 0) * S::kXRow + c * 8;
                const int b0i = 2 * c, b1i = 2 * c + 1;
                for (int s = 0; s < cnt; s++) {
#pragma unroll
                    for (int grp = 0; grp < 2; grp++) {
                        uint4 xv[4];
#pragma unroll
                        for (int j = 0; j < 4; j++) {
                            xv[j] = make_uint4(0u, 0u, 0u, 0u);
                            if (has_x) xv[j] = *reinterpret_cast<const uint4*>(xrow + s * kStepCols + grp * kGroup + j * 32);
                        }
                        float gt[4] = {0.f, 0.f, 0.f, 0.f};
                        const uint8_t* fs = st;
                        for (int fi = 0; fi < op.n_fields; fi++) {
                            const int f = op.field_width[fi];
                            const float scale = __int_as_float((127 + 24 + op.field_shift[fi]) << 23);   // 2^(24+shift)
                            const uint8_t* fss = fs + s * f * 512;
                            switch (f) {
                                case 8: field_group<8>(fss, grp, lane, xv, scale, gt); break;
                                case 4: field_group<4>(fss, grp, lane, xv, scale, gt); break;
                                case 2: field_group<2>(fss, grp, lane, xv, scale, gt); break;
                                default: field_group<1>(fss, grp, lane, xv, scale, gt); break;
                            }
                            fs += cnt * f * 512;
                        }
                        const uint32_t m0 = meta_s[(s * 2 + grp) * 16 + g];
                        const uint32_t m1 = meta_s[(s * 2 + grp) * 16 + g + 8];
                        const float s0 = __half2float(__ushort_as_half((unsigned short)(m0 & 0xffffu)));
                        const float z0 = __half2float(__ushort_as_half((unsigned short)(m0 >> 16))) - op.zero_adjust;
                        const float s1 = __half2float(__ushort_as_half((unsigned short)(m1 & 0xffffu)));
                        const float z1 = __half2float(__ushort_as_half((unsigned short)(m1 >> 16))) - op.zero_adjust;
                        const float xs0 = b0i < B ? xsum[b0i * (S::kMaxSS * 2) + s * 2 + grp] : 0.f;
                        tot[0] = fmaf(s0, fmaf(-z0, xs0, gt[0]), tot[0]);
                        tot[2] = fmaf(s1, fmaf(-z1, xs0, gt[2]), tot[2]);
                        if (MAXB > 1) {
                            const float xs1 = b1i < B ? xsum[b1i * (S::kMaxSS * 2) + s * 2 + grp] : 0.f;
                            tot[1] = fmaf(s0, fmaf(-z0, xs1, gt[1]), tot[1]);
                            tot[3] = fmaf(s1, fmaf(-z1, xs1, gt[3]), tot[3]);
                        }
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty);          // the stage may be refilled

            if (!live) continue;

            // ---- output: direct, or through split-K partials combined by the last arriver
            const int r0 = rt * kTileRows + g, r1 = r0 + 8;
            __half* y = reinterpret_cast<__half*>(op.y);
            bool wrote_final = true;
            if (op.n_chunks == 1) {
                if (MAXB == 1) {
                    if (c == 0) {
                        if (r0 < op.n_out) y[r0] = __float2half_rn(tot[0]);
                        if (r1 < op.n_out) y[r1] = __float2half_rn(tot[2]);
                    }
                } else {
                    if (2 * c < B) {
                        if (r0 < op.n_out) y[(long long)(2 * c) * op.n_out + r0] = __float2half_rn(tot[0]);
                        if (r1 < op.n_out) y[(long long)(2 * c) * op.n_out + r1] = __float2half_rn(tot[2]);
                    }
                    if (2 * c + 1 < B) {
                        if (r0 < op.n_out) y[(long long)(2 * c + 1) * op.n_out + r0] = __float2half_rn(tot[1]);
                        if (r1 < op.n_out) y[(long long)(2 * c + 1) * op.n_out + r1] = __float2half_rn(tot[3]);
                    }
                }
            } else {
                constexpr int kPF = MAXB == 1 ? 16 : 128;       // floats per unit
                float* pu = op.partial + ((long long)rt * op.n_chunks + ch) * kPF;
                if (MAXB == 1) {
                    if (c == 0) { pu[g] = tot[0]; pu[g + 8] = tot[2]; }
                } else {
                    *reinterpret_cast<float2*>(pu + g * 8 + 2 * c) = make_float2(tot[0], tot[1]);
                    *reinterpret_cast<float2*>(pu + (g + 8) * 8 + 2 * c) = make_float2(tot[2], tot[3]);
                }
                __threadfence();
                __syncwarp();
                unsigned old = 0;
                if (lane == 0) old = atomicAdd(op.tile_count + rt, 1u);
                old = __shfl_sync(0xffffffffu, old, 0);
                wrote_final = false;
                if (old == (unsigned)(op.n_chunks - 1)) {
                    __threadfence();
                    const float* pt = op.partial + (long long)rt * op.n_chunks * kPF;
                    if (MAXB == 1) {
                        if (lane < 16) {
                            float v = 0.f;
                            for (int q = 0; q < op.n_chunks; q++) v += __ldcg(pt + q * kPF + lane);
                            const int r = rt * kTileRows + lane;
                            if (r < op.n_out) y[r] = __float2half_rn(v);
                        }
                    } else {
                        float2 v0 = make_float2(0.f, 0.f), v1 = make_float2(0.f, 0.f);
                        for (int q = 0; q < op.n_chunks; q++) {
                            const float2 p0 = __ldcg(reinterpret_cast<const float2*>(pt + q * kPF + g * 8 + 2 * c));
                            const float2 p1 = __ldcg(reinterpret_cast<const float2*>(pt + q * kPF + (g + 8) * 8 + 2 * c));
                            v0.x += p0.x; v0.y += p0.y; v1.x += p1.x; v1.y += p1.y;
                        }
                        if (2 * c < B) {
                            if (r0 < op.n_out) y[(long long)(2 * c) * op.n_out + r0] = __float2half_rn(v0.x);
                            if (r1 < op.n_out) y[(long long)(2 * c) * op.n_out + r1] = __float2half_rn(v1.x);
                        }
                        if (2 * c + 1 < B) {
                            if (r0 < op.n_out) y[(long long)(2 * c + 1) * op.n_out + r0] = __float2half_rn(v0.y);
                            if (r1 < op.n_out) y[(long long)(2 * c + 1) * op.n_out + r1] = __float2half_rn(v1.y);
                        }
                    }
                    if (lane == 0) op.tile_count[rt] = 0u;   // ready for the next launch
                    wrote_final = true;
                }
            }
            (void)wrote_final;
            if (op.phase >= 0) {
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(sa.phase_done + op.phase, 1ull);
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
static int launch_impl(Ctx* ctx, const GemvOp& single, const StackArgs& sa, bool cooperative, cudaStream_t st)
{
    using S = GemvSmem<MAXB>;
    static bool configured[64] = {};
    if (ctx->device < 64 && !configured[ctx->device]) {
        FQ_CUDA_OK(cudaFuncSetAttribute(gemv_kernel<MAXB>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal));
        configured[ctx->device] = true;
    }
    long long blocks = ctx->sm_count;
    if (sa.total_units < blocks) blocks = sa.total_units;
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
    sa.total_units = (long long)op.n_rt * op.n_chunks;
    return op.batch <= 1 ? launch_impl<1>(ctx, op, sa, false, st) : launch_impl<8>(ctx, op, sa, false, st);
}

int launch_gemv_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, int max_batch, cudaStream_t st)
{
    // table_dev: [GemvOp x n_ops][long long phase_total x n_phases]; counters live in the workspace head
    StackArgs sa{};
    sa.table = reinterpret_cast<const GemvOp*>(table_dev);
    sa.phase_total = reinterpret_cast<const long long*>(table_dev + (size_t)hdr.n_ops * sizeof(GemvOp));
    sa.phase_done = reinterpret_cast<unsigned long long*>(ctx->ws);
    sa.exit_count = reinterpret_cast<unsigned*>(ctx->ws + 8 * 4096);
    sa.status = ctx->status_dev;
    sa.n_ops = hdr.n_ops;
    sa.n_phases = hdr.n_phases;
    sa.total_units = hdr.total_units;
    GemvOp dummy{};
    const bool coop = hdr.n_phases > 0;
    return max_batch <= 1 ? launch_impl<1>(ctx, dummy, sa, coop, st) : launch_impl<8>(ctx, dummy, sa, coop, st);
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
    sa.total_units = (long long)op.n_rt * op.n_chunks;
    return launch_impl<1>(ctx, op, sa, false, st);
}

}  // namespace fq

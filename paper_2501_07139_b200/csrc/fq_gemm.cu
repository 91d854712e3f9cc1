// Prefill path:  Y[m][n] = sum_k X[m][k] * w^[n][k],  X and Y bf16, fp32 accumulation in TMEM.
//
// Two kernels per call:
//   1. dequant_kernel    stored blobs -> w^ as bf16 [n_out][k_in] in the context workspace
//                        (w^ = (q - z) * s computed exactly in fp32, rounded once to bf16);
//   2. gemm_kernel       a persistent, warp-specialised tcgen05 GEMM: one warp streams 128x64 X tiles
//                        and 256x64 w^ tiles into a 4-stage shared-memory ring with TMA (128-byte
//                        swizzle), one thread issues tcgen05.mma (M = 128 tokens, N = 256 outputs,
//                        K = 16 per instruction) into one of two 256-column TMEM accumulators, four
//                        warps drain the other accumulator (tcgen05.ld -> bf16 -> global) meanwhile.
// Every mbarrier wait is bounded by a timer; when one runs out the kernel records FQ_ERR_TIMEOUT,
// all roles leave their loops, and the TMEM allocation is released before the CTA exits.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fq_dequant.cuh"
#include "fq_internal.cuh"
#include "fq_umma.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

// ------------------------------------------------------------------------------- dequantise to bf16
struct DequantArgs {
    const uint8_t* store;
    int n_out, k_in, n_kb, blob_stride;
    int zero_adjust;
    __nv_bfloat16* out;              // [n_out][k_in]
};

// One warp per (row strip of 32, 64 columns): the lanes read the stored words of the two k32 steps exactly as
// the decode kernel does (16 bytes per lane and field chunk), merge the fields into four codes per register,
// convert (w^ = (q - z) * s exactly, one rounding to bf16) and write 8-byte runs; the four lanes of a quad
// cover 32 contiguous bytes of a row.  Specialised per field list like the fused kernel, whose helpers it shares.
template <int VARIANT>
__global__ void __launch_bounds__(256) dequant_kernel(const DequantArgs a)
{
    constexpr FieldList FL = variant_fields(VARIANT);
    constexpr int kLoads = fields_loads(FL, FL.n);
    constexpr bool kSmallCodes = VARIANT < 6;            // PACKED 2..7 bits: codes below 128, no zero adjustment
    const int lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const int n_rp = row_pairs(a.n_out), n_st = a.k_in / 64;
    const long long total = (long long)n_rp * n_st;
    const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    for (long long ti = warp0; ti < total; ti += n_warps) {
        const int rp = (int)(ti / n_st), ks = (int)(ti % n_st);       // consecutive warps: consecutive columns of a strip
        const int kb = ks >> 3, ssl = (ks >> 2) & 1, j0 = (ks & 3) * 2, grp = (ks >> 1) & 1;
        const uint8_t* blob_lane = a.store + ((long long)rp * a.n_kb + kb) * a.blob_stride + lane * 16;
        uint4 raw[kBlobTiles][kLoads];
        uint2 meta[kBlobTiles];
        load_stage_words<VARIANT, 0>(blob_lane, ssl, j0, raw[0]);
        load_stage_words<VARIANT, 1>(blob_lane, ssl, j0, raw[1]);
#pragma unroll
        for (int tl = 0; tl < kBlobTiles; tl++)
            meta[tl] = __ldg(reinterpret_cast<const uint2*>(blob_lane - lane * 16 + blob_meta_off(ssl, tl) + blob_meta_word(grp, g)));
#pragma unroll
        for (int tl = 0; tl < kBlobTiles; tl++) {
            uint32_t code[2][4];
            merge_codes<VARIANT>(raw[tl], j0, code);
            const uint32_t mm[2] = {meta[tl].x, meta[tl].y};
#pragma unroll
            for (int hr = 0; hr < 2; hr++) {
                const long long n = (long long)rp * 32 + tl * kTileRows + g + 8 * hr;
                if (n >= a.n_out) continue;
                const float s = __half2float(__ushort_as_half((unsigned short)(mm[hr] & 0xffffu)));
                const __half2 zz = __half2half2(__int2half_rn(1024 + (int)(mm[hr] >> 16) - a.zero_adjust));
                const float cc = -(float)(128 + (int)(mm[hr] >> 16)) * s;
                __nv_bfloat16* row = a.out + n * a.k_in + ks * 64 + 4 * c;
#pragma unroll
                for (int jj = 0; jj < 2; jj++)
#pragma unroll
                    for (int half = 0; half < 2; half++) {
                        const uint32_t q4 = code[jj][2 * half + hr];          // A register r = 2 * half + row half
                        const uint2 o = kSmallCodes ? small_codes_to_bf16(q4, cc, s) : codes_to_bf16(q4, zz, s);
                        *reinterpret_cast<uint2*>(row + 32 * jj + 16 * half) = o;
                    }
            }
        }
    }
}

template <int VARIANT>
static int launch_dequant(const DequantArgs& da, int sm_count, cudaStream_t st)
{
    const long long items = (long long)row_pairs(da.n_out) * (da.k_in / 64);     // one warp each
    long long blocks = (items + 7) / 8;
    if (blocks > (long long)sm_count * 8) blocks = (long long)sm_count * 8;
    dequant_kernel<VARIANT><<<(unsigned)blocks, 256, 0, st>>>(da);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ------------------------------------------------------------------------------- tcgen05 GEMM
constexpr int kBM = 128;                 // tokens per tile (UMMA M)
constexpr int kBN = 256;                 // outputs per tile (UMMA N)
constexpr int kBK = 64;                  // K per stage: 64 bf16 = one 128-byte swizzle span
constexpr int kGemmStages = 4;
constexpr int kGemmThreads = 192;        // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2..5: epilogue
constexpr int kTmemCols = 512;           // two accumulators of kBN columns

struct GemmSmem {
    static constexpr int kABytes = kBM * kBK * 2;                  // 16 KB
    static constexpr int kBBytes = kBN * kBK * 2;                  // 32 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int oBars = kGemmStages * kStageBytes;        // full[S], empty[S], tmem_full[2], tmem_empty[2]
    static constexpr int oTmemPtr = oBars + (2 * kGemmStages + 4) * 8;
    static constexpr int oFlag = oTmemPtr + 8;
    static constexpr int kTotal = oFlag + 8 + 1024;                // + slack for the 1024-byte alignment of the tiles
};

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
            __nv_bfloat16* __restrict__ Y, int M, int N, int K, int ldy, int* status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bars = g_smem_u32(smem + GemmSmem::oBars);
    const uint32_t full0 = bars, empty0 = bars + 8 * kGemmStages;
    const uint32_t tfull0 = bars + 16 * kGemmStages, tempty0 = tfull0 + 16;
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem + GemmSmem::oTmemPtr);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + GemmSmem::oFlag);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kGemmStages; s++) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full0 + 8 * s) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty0 + 8 * s) : "memory");
        }
        for (int b = 0; b < 2; b++) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tfull0 + 8 * b) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(tempty0 + 8 * b) : "memory");   // one arrival per epilogue warp
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                     // this warp owns the TMEM allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(g_smem_u32(const_cast<uint32_t*>(tmem_ptr))), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_ptr;

    const int m_blocks = (M + kBM - 1) / kBM, n_blocks = (N + kBN - 1) / kBN;
    const int n_tiles = m_blocks * n_blocks;
    const int k_steps = K / kBK;

    if (warp == 0) {
        // ================================================================== TMA producer
        if (lane == 0) {
            int stage = 0;
            uint32_t wraps = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                const int mb = t % m_blocks, nb = t / m_blocks;        // m fastest: the w^ tile stays in L2
                for (int ks = 0; ks < k_steps; ks++) {
                    if (wraps > 0 && !g_wait(empty0 + 8 * stage, (wraps - 1u) & 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = full0 + 8 * stage;
                    const uint32_t a_dst = g_smem_u32(smem + stage * GemmSmem::kStageBytes);
                    const uint32_t b_dst = a_dst + GemmSmem::kABytes;
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 ::"r"(full), "r"(GemmSmem::kStageBytes) : "memory");
                    asm volatile(
                        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                        ::"r"(a_dst), "l"(&map_x), "r"(ks * kBK), "r"(mb * kBM), "r"(full) : "memory");
                    asm volatile(
                        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                        ::"r"(b_dst), "l"(&map_w), "r"(ks * kBK), "r"(nb * kBN), "r"(full) : "memory");
                    if (++stage == kGemmStages) { stage = 0; wraps++; }
                }
            }
            if (!ok) { atomicCAS(status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kBM, kBN);
            int stage = 0;
            uint32_t wraps = 0;
            int local = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, local++) {
                const int buf = local & 1;
                const uint32_t use = (uint32_t)(local >> 1);           // how often this accumulator was used before
                if (use > 0 && !g_wait(tempty0 + 8 * buf, (use - 1u) & 1u, abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + (uint32_t)(buf * kBN);
                for (int ks = 0; ks < k_steps; ks++) {
                    if (!g_wait(full0 + 8 * stage, wraps & 1u, abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = g_smem_u32(smem + stage * GemmSmem::kStageBytes);
                    const uint32_t b_addr = a_addr + GemmSmem::kABytes;
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; kk++) {
                        const uint64_t adesc = umma_desc_sw128(a_addr + kk * 32);
                        const uint64_t bdesc = umma_desc_sw128(b_addr + kk * 32);
                        const uint32_t accumulate = (ks > 0 || kk > 0) ? 1u : 0u;
                        asm volatile(
                            "{\n\t.reg .pred p;\n\t"
                            "setp.ne.b32 p, %4, 0;\n\t"
                            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
                    }
                    // the stage may be refilled once these MMAs have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(empty0 + 8 * stage) : "memory");
                    if (++stage == kGemmStages) { stage = 0; wraps++; }
                }
                if (!ok) break;
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                             ::"r"(tfull0 + 8 * buf) : "memory");
            }
            if (!ok) { atomicCAS(status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
        }
    } else {
        // ================================================================== epilogue (warps 2..5)
        const int quarter = warp & 3;                                   // TMEM lanes 32*quarter .. +31 belong to this warp
        int local = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, local++) {
            const int mb = t % m_blocks, nb = t / m_blocks;
            const int buf = local & 1;
            const uint32_t use = (uint32_t)(local >> 1);
            if (!g_wait(tfull0 + 8 * buf, use & 1u, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const int row = mb * kBM + quarter * 32 + lane;              // token
            const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kBN);
#pragma unroll 1
            for (int cb = 0; cb < kBN / 32; cb++) {
                uint32_t v[32];
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                    : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                      "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                      "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                      "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                    : "r"(taddr0 + (uint32_t)(cb * 32)) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int col0 = nb * kBN + cb * 32;
                if (row < M && col0 < N) {
                    __nv_bfloat16* dst = Y + (long long)row * ldy + col0;
                    if (col0 + 32 <= N) {
#pragma unroll
                        for (int q = 0; q < 4; q++) {
                            uint4 o;
                            uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]),
                                                                               __uint_as_float(v[8 * q + 2 * e + 1]));
                                ow[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(dst + 8 * q) = o;
                        }
                    } else {
                        for (int e = 0; e < 32 && col0 + e < N; e++) dst[e] = __float2bfloat16_rn(__uint_as_float(v[e]));
                    }
                }
            }
            // the accumulator may be overwritten
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tempty0 + 8 * buf) : "memory");
        }
        if (!ok && lane == 0) { atomicCAS(status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
    }

    // every path ends here: release TMEM before the CTA exits
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------- host side
int launch_gemm(Ctx* ctx, const void* store, int blob_stride, const FieldList& fl, int zero_adjust, int n_out, int k_in,
                const uint16_t* X, int M, int ldx, uint16_t* Y, int ldy, void* w_scratch, cudaStream_t st)
{
    // 1. w^ as bf16 [n_out][k_in]
    DequantArgs da{};
    da.store = static_cast<const uint8_t*>(store); da.n_out = n_out; da.k_in = k_in;
    da.n_kb = k_blobs(k_in); da.blob_stride = blob_stride; da.zero_adjust = zero_adjust;
    da.out = static_cast<__nv_bfloat16*>(w_scratch);
    int rc = FQ_ERR_ARG;
    switch (variant_of_fields(fl)) {
#define FQ_CASE(V) case V: rc = launch_dequant<V>(da, ctx->sm_count, st); break;
        FQ_CASE(0) FQ_CASE(1) FQ_CASE(2) FQ_CASE(3) FQ_CASE(4) FQ_CASE(5) FQ_CASE(6)
        FQ_CASE(7) FQ_CASE(8) FQ_CASE(9) FQ_CASE(10) FQ_CASE(11) FQ_CASE(12) FQ_CASE(13)
#undef FQ_CASE
        default: break;
    }
    if (rc != FQ_OK) return rc;

    // 2. tcgen05 GEMM
    CUtensorMap map_x, map_w;
    rc = make_map(&map_x, X, M, k_in, ldx, kBM);
    if (rc != FQ_OK) return rc;
    rc = make_map(&map_w, w_scratch, n_out, k_in, k_in, kBN);
    if (rc != FQ_OK) return rc;
    static bool configured[64] = {};
    if (ctx->device < 64 && !configured[ctx->device]) {
        FQ_CUDA_OK(cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmSmem::kTotal));
        configured[ctx->device] = true;
    }
    const int tiles = ((M + kBM - 1) / kBM) * ((n_out + kBN - 1) / kBN);
    const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    gemm_kernel<<<grid, kGemmThreads, GemmSmem::kTotal, st>>>(map_x, map_w, reinterpret_cast<__nv_bfloat16*>(Y), M, n_out,
                                                             k_in, ldy, ctx->status_dev);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

}  // namespace fq

// Prefill path, fused:  Y[m][n] = sum_k X[m][k] * w^[n][k]  straight from the stored blobs.
//
// One persistent, warp-specialised kernel; a tile is 256 tokens x 256 outputs and fills the whole TMEM
// (two fp32 accumulators of 128 tokens x 256 outputs), so every dequantised weight is used for 256 tokens:
//   warp 0        TMA: two 128 x 64 bf16 tiles of X per stage (cp.async.bulk.tensor.2d, 128-byte swizzle);
//   warp 1        one thread issues tcgen05.mma (M = 128, N = 256, K = 16): per stage 4 K slices x 2 token halves,
//                 then tcgen05.commit hands the stage back;
//   warps 2..5    epilogue: tcgen05.ld -> bf16 -> global, both accumulators, after the tile's last stage;
//   warps 6..21   dequantisation, two groups of eight that take alternate stages: warp d of a group owns the 32
//                 output rows (one stored row pair) 32 d .. 32 d + 31 of the tile.  Per stage (64 columns = two k32 steps of a blob) its lanes load the stored words of
//                 those steps exactly as the decode kernel reads them (16 bytes per lane, straight from global
//                 memory / L2: the 32 token tiles of a matrix all read the same blobs), rebuild the codes four
//                 to a register, compute w^ = (q - z) * s exactly in fp32 (one fused multiply-add), round once to
//                 bf16 and store 8-byte runs into the stage's B tile in the layout TMA would have produced
//                 (128-byte rows, 16-byte chunks XOR-swizzled with the row), fence.proxy.async, arrive.
// The stage's "full" barrier counts the TMA transaction and one arrival per dequantisation warp.
// Every mbarrier wait is bounded by a timer; when one runs out the kernel records FQ_ERR_TIMEOUT, all roles
// leave their loops, and the TMEM allocation is released before the CTA exits.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "fq_dequant.cuh"
#include "fq_internal.cuh"
#include "fq_ptx.cuh"
#include "fq_umma.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

namespace {

constexpr int kFM = 256;                 // tokens per tile: two UMMA M = 128 halves
constexpr int kFN = 256;                 // outputs per tile (UMMA N)
constexpr int kFK = kUmmaBK;             // 64
constexpr int kFStages = 3;
constexpr int kDqWarps = kFN / 32;       // one per stored row pair of the tile ...
constexpr int kDqGroups = 2;             // ... in each of two groups that take alternate stages: the global loads of
                                         // one stage travel while the other group converts and stores its stage
constexpr int kFThreads = (6 + kDqGroups * kDqWarps) * 32;
constexpr int kFTmemCols = 512;

struct FusedSmem {
    static constexpr int kABytes = kFM * kFK * 2;                  // 32 KB: two 128 x 64 X tiles
    static constexpr int kBBytes = kFN * kFK * 2;                  // 32 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int oBars = kFStages * kStageBytes;           // full[S], empty[S], tmem_full, tmem_empty
    static constexpr int oTmemPtr = oBars + (2 * kFStages + 2) * 8;
    static constexpr int oFlag = oTmemPtr + 8;
    static constexpr int kTotal = oFlag + 8 + 1024;                // + slack for the 1024-byte alignment of the tiles
};
static_assert(FusedSmem::kTotal <= 232448, "fused GEMM: shared memory over the per-CTA limit");

struct FusedArgs {
    const uint8_t* store;
    int n_kb, blob_stride, zero_adjust;
    int M, N, K, ldy;
    __nv_bfloat16* Y;
    int* status;
    // balanced runs (below): one 256 x 256 fp32 slot per CTA, a flag per slot and epilogue warp, the launch number
    int halves;              // token halves (of 128) per tile: 2, or 1 when 256-token tiles would be too few for the SMs
    int balanced;
    float* parts;
    unsigned* part_flags;
    unsigned epoch;
};

constexpr int kPartFloats = kFM * kFN;

// Work of one CTA.  Normally whole tiles, CTA c takes tiles c, c + grid, ...  When that would leave most SMs idle in
// the last wave (160 tiles on 148 SMs), the host asks for BALANCED RUNS instead: the (tile, K stage) pairs,
// tile-major, are cut into gridDim.x equal contiguous runs.  A run is at least one tile long (grid <= tiles), hence
// covers: the rest of a tile that the previous CTA began (ks0 > 0), whole tiles, and the beginning of a tile that the
// next CTA finishes (ks1 < k_steps).  The CTA that computes the rest does so FIRST and leaves fp32 partial sums in
// its slot; the CTA that computes the beginning does so LAST, adds the slot and writes the outputs.
struct WorkItem { int tile, ks0, ks1; };
struct WorkRun {
    long long u, u_hi;
    int k_steps, n_tiles, next_tile;
    bool balanced;
    __device__ WorkRun(int n_tiles_, int k_steps_, bool balanced_) : k_steps(k_steps_), n_tiles(n_tiles_), balanced(balanced_)
    {
        const long long total = (long long)n_tiles_ * k_steps_;
        u = total * blockIdx.x / gridDim.x;
        u_hi = total * (blockIdx.x + 1) / gridDim.x;
        next_tile = blockIdx.x;
    }
    __device__ bool next(WorkItem& it)
    {
        if (!balanced) {
            if (next_tile >= n_tiles) return false;
            it.tile = next_tile; it.ks0 = 0; it.ks1 = k_steps;
            next_tile += gridDim.x;
            return true;
        }
        if (u >= u_hi) return false;
        it.tile = (int)(u / k_steps);
        it.ks0 = (int)(u % k_steps);
        const long long left = u_hi - u;
        it.ks1 = left < k_steps - it.ks0 ? it.ks0 + (int)left : k_steps;
        u += it.ks1 - it.ks0;
        return true;
    }
};

static __device__ __forceinline__ void sts64(uint32_t addr, uint32_t x, uint32_t y)
{
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}

template <int VARIANT>
__global__ void __launch_bounds__(kFThreads, 1)
gemm_fused_kernel(const __grid_constant__ CUtensorMap map_x, const FusedArgs a)
{
    constexpr FieldList FL = variant_fields(VARIANT);
    constexpr int kLoads = fields_loads(FL, FL.n);
    constexpr bool kSmallCodes = VARIANT < 6;            // PACKED 2..7 bits: codes below 128, no zero adjustment
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t bars = g_smem_u32(smem + FusedSmem::oBars);
    const uint32_t full0 = bars, empty0 = bars + 8 * kFStages;
    const uint32_t tfull = bars + 16 * kFStages, tempty = tfull + 8;
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem + FusedSmem::oTmemPtr);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + FusedSmem::oFlag);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kFStages; s++) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * s), "n"(1 + kDqWarps) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty0 + 8 * s) : "memory");
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tfull) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 4;" ::"r"(tempty) : "memory");      // one arrival per epilogue warp
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {                     // this warp owns the TMEM allocation
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(g_smem_u32(const_cast<uint32_t*>(tmem_ptr))), "n"(kFTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_ptr;

    const int halves = a.halves;                          // 128-token halves per tile
    const int tile_m = 128 * halves;
    const int m_blocks = (a.M + tile_m - 1) / tile_m, n_blocks = (a.N + kFN - 1) / kFN;
    const int n_tiles = m_blocks * n_blocks;
    const int k_steps = a.K / kFK;

    if (warp == 0) {
        // ================================================================== TMA producer (X)
        if (lane == 0) {
            int stage = 0;
            uint32_t wraps = 0;
            bool ok = true;
            WorkRun run(n_tiles, k_steps, a.balanced != 0);
            WorkItem it;
            while (ok && run.next(it)) {
                const int mb = it.tile % m_blocks;                         // m fastest: the blobs of a row block stay in L2
                for (int ks = it.ks0; ks < it.ks1; ks++) {
                    if (wraps > 0 && !g_wait(empty0 + 8 * stage, (wraps - 1u) & 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = full0 + 8 * stage;
                    const uint32_t a_dst = g_smem_u32(smem + stage * FusedSmem::kStageBytes);
                    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                                 ::"r"(full), "r"(halves * (FusedSmem::kABytes / 2)) : "memory");
#pragma unroll
                    for (int h = 0; h < 2; h++)
                        if (h < halves) asm volatile(
                            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                            ::"r"(a_dst + h * (FusedSmem::kABytes / 2)), "l"(&map_x), "r"(ks * kFK), "r"(mb * tile_m + h * 128), "r"(full)
                            : "memory");
                    if (++stage == kFStages) { stage = 0; wraps++; }
                }
            }
            if (!ok) { atomicCAS(a.status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
        }
    } else if (warp == 1) {
        // ================================================================== MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, kFN);
            int stage = 0;
            uint32_t wraps = 0;
            int local = 0;
            bool ok = true;
            WorkRun run(n_tiles, k_steps, a.balanced != 0);
            WorkItem it;
            for (; ok && run.next(it); local++) {
                // both accumulators belong to this item: wait until the epilogue has drained the previous one
                if (local > 0 && !g_wait(tempty, (uint32_t)(local - 1) & 1u, abort_flag)) { ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                for (int ks = it.ks0; ks < it.ks1; ks++) {
                    if (!g_wait(full0 + 8 * stage, wraps & 1u, abort_flag)) { ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = g_smem_u32(smem + stage * FusedSmem::kStageBytes);
                    const uint32_t b_addr = a_addr + FusedSmem::kABytes;
#pragma unroll
                    for (int h = 0; h < 2; h++)
#pragma unroll
                        for (int kk = 0; kk < kFK / 16; kk++) {
                            if (h >= halves) continue;                     // (tiles of 128 tokens use the first accumulator only)
                            const uint64_t adesc = umma_desc_sw128(a_addr + h * (FusedSmem::kABytes / 2) + kk * 32);
                            const uint64_t bdesc = umma_desc_sw128(b_addr + kk * 32);
                            const uint32_t accumulate = (ks > it.ks0 || kk > 0) ? 1u : 0u;
                            asm volatile(
                                "{\n\t.reg .pred p;\n\t"
                                "setp.ne.b32 p, %4, 0;\n\t"
                                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                ::"r"(tmem_base + (uint32_t)(h * kFN)), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
                        }
                    // the stage may be refilled once these MMAs have read it
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                                 ::"r"(empty0 + 8 * stage) : "memory");
                    if (++stage == kFStages) { stage = 0; wraps++; }
                }
                if (!ok) break;
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tfull) : "memory");
            }
            if (!ok) { atomicCAS(a.status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
        }
    } else if (warp < 6) {
        // ================================================================== epilogue (warps 2..5)
        const int quarter = warp & 3;                                   // TMEM lanes 32*quarter .. +31 belong to this warp
        int local = 0;
        bool ok = true;
        WorkRun run(n_tiles, k_steps, a.balanced != 0);
        WorkItem it;
        for (; ok && run.next(it); local++) {
            const int mb = it.tile % m_blocks, nb = it.tile / m_blocks;
            const bool dump = it.ks0 > 0;                               // the rest of a tile another CTA began: leave partial sums
            const bool merge = it.ks1 < k_steps;                        // the beginning of a tile: add the next CTA's partial sums
            // slot layout: float4 number q (columns 4q .. 4q + 3) of token half h: [h][q][quarter][lane] -- a warp's accesses are contiguous
            const float4* slot_in = reinterpret_cast<const float4*>(a.parts + (long long)(blockIdx.x + 1) * kPartFloats) + quarter * 32 + lane;
            float4* slot_out = reinterpret_cast<float4*>(a.parts + (long long)blockIdx.x * kPartFloats) + quarter * 32 + lane;
            if (merge) {
                // that CTA computed its part first of all, long ago; the wait is bounded all the same
                const unsigned* flag = a.part_flags + (blockIdx.x + 1) * 4 + quarter;
                bool seen = ld_acquire_u32(flag) == a.epoch;
                if (!seen) {
                    const unsigned long long t0 = g_ns();
                    while (!(seen = ld_acquire_u32(flag) == a.epoch) && !*abort_flag && g_ns() - t0 <= kGemmWaitNs) __nanosleep(64);
                }
                if (!__all_sync(0xffffffffu, seen)) { ok = false; break; }
            }
            if (!g_wait<256>(tfull, (uint32_t)local & 1u, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
            for (int h = 0; h < halves; h++) {
                const int row = mb * tile_m + h * 128 + quarter * 32 + lane;    // token
                const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * kFN);
                if (merge) {
                    // 16 columns at a time; the partial sums of the next 16 travel while these are added and stored
                    float4 p[4], pn[4];
#pragma unroll
                    for (int e = 0; e < 4; e++) p[e] = __ldcg(slot_in + ((h * 64 + e) * 4) * 32);
#pragma unroll 1
                    for (int cb = 0; cb < kFN / 16; cb++) {
                        uint32_t v[16];
                        asm volatile(
                            "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                            "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                              "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                            : "r"(taddr0 + (uint32_t)(cb * 16)) : "memory");
                        if (cb + 1 < kFN / 16) {
#pragma unroll
                            for (int e = 0; e < 4; e++) pn[e] = __ldcg(slot_in + ((h * 64 + (cb + 1) * 4 + e) * 4) * 32);
                        }
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        float f[16];
#pragma unroll
                        for (int e = 0; e < 4; e++) {
                            f[4 * e] = __uint_as_float(v[4 * e]) + p[e].x;
                            f[4 * e + 1] = __uint_as_float(v[4 * e + 1]) + p[e].y;
                            f[4 * e + 2] = __uint_as_float(v[4 * e + 2]) + p[e].z;
                            f[4 * e + 3] = __uint_as_float(v[4 * e + 3]) + p[e].w;
                            p[e] = pn[e];
                        }
                        const int col0 = nb * kFN + cb * 16;
                        if (row < a.M && col0 < a.N) {
                            __nv_bfloat16* dst = a.Y + (long long)row * a.ldy + col0;
                            if (col0 + 16 <= a.N) {
#pragma unroll
                                for (int q = 0; q < 2; q++) {
                                    uint4 o;
                                    uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                                    for (int e = 0; e < 4; e++) {
                                        const __nv_bfloat162 hh = __floats2bfloat162_rn(f[8 * q + 2 * e], f[8 * q + 2 * e + 1]);
                                        ow[e] = *reinterpret_cast<const uint32_t*>(&hh);
                                    }
                                    *reinterpret_cast<uint4*>(dst + 8 * q) = o;
                                }
                            } else {
#pragma unroll
                                for (int e = 0; e < 16; e++)
                                    if (col0 + e < a.N) dst[e] = __float2bfloat16_rn(f[e]);
                            }
                        }
                    }
                    continue;
                }
#pragma unroll 1
                for (int cb = 0; cb < kFN / 32; cb++) {
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
                    if (dump) {
#pragma unroll
                        for (int e = 0; e < 8; e++)
                            slot_out[((h * 64 + cb * 8 + e) * 4) * 32] = make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]),
                                                                                     __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                        continue;
                    }
                    const int col0 = nb * kFN + cb * 32;
                    if (row < a.M && col0 < a.N) {
                        __nv_bfloat16* dst = a.Y + (long long)row * a.ldy + col0;
                        if (col0 + 32 <= a.N) {
#pragma unroll
                            for (int q = 0; q < 4; q++) {
                                uint4 o;
                                uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                                for (int e = 0; e < 4; e++) {
                                    const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]),
                                                                                    __uint_as_float(v[8 * q + 2 * e + 1]));
                                    ow[e] = *reinterpret_cast<const uint32_t*>(&hh);
                                }
                                *reinterpret_cast<uint4*>(dst + 8 * q) = o;
                            }
                        } else {
#pragma unroll
                            for (int e = 0; e < 32; e++)
                                if (col0 + e < a.N) dst[e] = __float2bfloat16_rn(__uint_as_float(v[e]));
                        }
                    }
                }
            }
            if (dump) {                                                  // publish this warp's quarter of the slot
                __threadfence();
                __syncwarp();
                if (lane == 0) st_release_u32(a.part_flags + blockIdx.x * 4 + quarter, a.epoch);
            }
            // the accumulators may be overwritten
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tempty) : "memory");
        }
        if (!ok && lane == 0) { atomicCAS(a.status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
    } else {
        // ================================================================== dequantisation (warps 6..21)
        const int dw = (warp - 6) % kDqWarps;                           // row pair of the tile
        const int grp_id = (warp - 6) / kDqWarps;                       // this group takes the stages seq % kDqGroups == grp_id
        const int g = lane >> 2, c = lane & 3;
        const int n_rp = row_pairs(a.N);
        // Where this lane's 8-byte runs go inside a B tile: row 32 dw + 16 tile + g + 8 hr (128 bytes a row), 16-byte
        // chunk (4 jj + 2 half + (c >> 1)) XOR-swizzled with the row's low three bits (= g), + 8 (c & 1).
        uint32_t koff[4];
#pragma unroll
        for (int k4 = 0; k4 < 4; k4++)
            koff[k4] = (uint32_t)(dw * 4096 + g * 128 + (((2 * k4) ^ (g ^ (c >> 1))) << 4) + 8 * (c & 1));
        const uint32_t btile0 = g_smem_u32(smem) + FusedSmem::kABytes;
        long long seq = 0;                                              // stages of this CTA so far, over all its tiles
        bool ok = true;
        WorkRun run(n_tiles, k_steps, a.balanced != 0);
        WorkItem it;
        while (ok && run.next(it)) {
            const int nb = it.tile / m_blocks;
            const int rp = nb * kDqWarps + dw;
            const bool have = rp < n_rp;
            const uint8_t* row_blobs = a.store + (long long)(have ? rp : 0) * a.n_kb * a.blob_stride + lane * 16;
            for (int ks = it.ks0; ks < it.ks1; ks++, seq++) {
                if ((int)(seq % kDqGroups) != grp_id) continue;
                const int stage = (int)(seq % kFStages);
                const uint32_t wraps = (uint32_t)(seq / kFStages);
                // ---- the stored words of this stage (64 columns = k32 steps j0, j0 + 1 of one superstep of one blob)
                const int kb = ks >> 3, ssl = (ks >> 2) & 1, j0 = (ks & 3) * 2, grp = (ks >> 1) & 1;
                const uint8_t* blob_lane = row_blobs + (long long)kb * a.blob_stride;
                if (!FQ_IN_BOUNDS(kb < a.n_kb && (have ? rp : 0) < n_rp && stage < kFStages, a.status)) {   // (checked build)
                    if (lane == 0) *abort_flag = 1;
                    ok = false;
                    break;
                }
                uint4 raw[kBlobTiles][kLoads];
                uint2 meta[kBlobTiles];                                    // scale / zero words of rows g and g + 8: adjacent
                load_stage_words<VARIANT, 0>(blob_lane, ssl, j0, raw[0]);
                load_stage_words<VARIANT, 1>(blob_lane, ssl, j0, raw[1]);
#pragma unroll
                for (int tl = 0; tl < kBlobTiles; tl++)
                    meta[tl] = __ldg(reinterpret_cast<const uint2*>(blob_lane - lane * 16 + blob_meta_off(ssl, tl) + blob_meta_word(grp, g)));
                // ---- the stage's B tile must be free (the MMAs that read its previous contents are done)
                const bool is_free = wraps == 0 || g_wait(empty0 + 8 * stage, (wraps - 1u) & 1u, abort_flag);
                if (!__all_sync(0xffffffffu, is_free)) { ok = false; break; }      // (the lanes must leave together)
                const uint32_t btile = btile0 + stage * FusedSmem::kStageBytes;
#pragma unroll
                for (int tl = 0; tl < kBlobTiles; tl++) {
                    uint32_t code[2][4];
                    merge_codes<VARIANT>(raw[tl], j0, code);
                    const uint32_t mm[2] = {meta[tl].x, meta[tl].y};
                    __half2 zz[2];
                    float sc[2], cc[2];
#pragma unroll
                    for (int hr = 0; hr < 2; hr++) {
                        sc[hr] = have ? __half2float(__ushort_as_half((unsigned short)(mm[hr] & 0xffffu))) : 0.f;   // rows past N: zeros
                        zz[hr] = __half2half2(__int2half_rn(1024 + (int)(mm[hr] >> 16) - a.zero_adjust));
                        cc[hr] = -(float)(128 + (int)(mm[hr] >> 16)) * sc[hr];
                    }
#pragma unroll
                    for (int jj = 0; jj < 2; jj++)
#pragma unroll
                        for (int r = 0; r < 4; r++) {
                            const int hr = r & 1, half = r >> 1;               // A register r = 2 * half + row half
                            const uint2 o = kSmallCodes ? small_codes_to_bf16(code[jj][r], cc[hr], sc[hr]) : codes_to_bf16(code[jj][r], zz[hr], sc[hr]);
                            sts64(btile + koff[2 * jj + half] + tl * 2048 + hr * 1024, o.x, o.y);
                        }
                }
                // generic-proxy stores -> visible to the tensor core's reads (async proxy), then count this warp
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full0 + 8 * stage) : "memory");
            }
        }
        if (!ok && lane == 0) { atomicCAS(a.status, 0, FQ_ERR_TIMEOUT); *abort_flag = 1; }
    }

    // every path ends here: release TMEM before the CTA exits
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kFTmemCols) : "memory");
    }
}

template <int VARIANT>
int launch_variant(Ctx* ctx, const CUtensorMap& map_x, const FusedArgs& a, int grid, cudaStream_t st)
{
    static bool configured[64] = {};
    if (ctx->device < 64 && !configured[ctx->device]) {
        FQ_CUDA_OK(cudaFuncSetAttribute(gemm_fused_kernel<VARIANT>, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedSmem::kTotal));
        configured[ctx->device] = true;
    }
    gemm_fused_kernel<VARIANT><<<grid, kFThreads, FusedSmem::kTotal, st>>>(map_x, a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

}  // namespace

size_t gemm_fused_part_bytes() { return (size_t)kPartFloats * sizeof(float); }

// Balanced runs pay two extra epilogues per CTA; they are worth it when whole tiles would leave the last wave mostly empty.
// 256-token tiles make every converted weight serve 256 tokens; when they are so few that twice as many still fit
// the SMs in one wave, tiles of 128 tokens use twice the SMs for the same work.
int gemm_fused_halves(int M, int n_out, int sm_count)
{
    const long long tiles = (long long)((M + kFM - 1) / kFM) * ((n_out + kFN - 1) / kFN);
    const long long tiles128 = (long long)((M + 127) / 128) * ((n_out + kFN - 1) / kFN);
    return (tiles128 > tiles && 2 * tiles <= sm_count) ? 1 : 2;
}

bool gemm_fused_wants_balance(int M, int n_out, int sm_count)
{
    if (gemm_fused_halves(M, n_out, sm_count) == 1) return false;
    const long long tiles = (long long)((M + kFM - 1) / kFM) * ((n_out + kFN - 1) / kFN);
    if (tiles <= sm_count) return false;
    const long long waves = (tiles + sm_count - 1) / sm_count;
    return (double)tiles / (double)(waves * sm_count) < 0.80;
}

int launch_gemm_fused(Ctx* ctx, const void* store, int blob_stride, const FieldList& fl, int zero_adjust, int n_out, int k_in,
                      const uint16_t* X, int M, int ldx, uint16_t* Y, int ldy, float* parts, unsigned* part_flags, unsigned epoch,
                      cudaStream_t st)
{
    CUtensorMap map_x;
    const int rc = make_map(&map_x, X, M, k_in, ldx, 128);
    if (rc != FQ_OK) return rc;
    const int variant = variant_of_fields(fl);          // the kernel is specialised per field list
    if (variant < 0) return FQ_ERR_ARG;
    FusedArgs a{};
    a.store = static_cast<const uint8_t*>(store); a.n_kb = k_blobs(k_in); a.blob_stride = blob_stride;
    a.zero_adjust = zero_adjust; a.M = M; a.N = n_out; a.K = k_in; a.ldy = ldy;
    a.Y = reinterpret_cast<__nv_bfloat16*>(Y); a.status = ctx->status_dev;
    a.balanced = parts != nullptr ? 1 : 0; a.parts = parts; a.part_flags = part_flags; a.epoch = epoch;
    a.halves = gemm_fused_halves(M, n_out, ctx->sm_count);
    const int tile_m = 128 * a.halves;
    const int tiles = ((M + tile_m - 1) / tile_m) * ((n_out + kFN - 1) / kFN);
    const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    switch (variant) {
#define FQ_CASE(V) case V: return launch_variant<V>(ctx, map_x, a, grid, st);
        FQ_CASE(0) FQ_CASE(1) FQ_CASE(2) FQ_CASE(3) FQ_CASE(4) FQ_CASE(5) FQ_CASE(6)
        FQ_CASE(7) FQ_CASE(8) FQ_CASE(9) FQ_CASE(10) FQ_CASE(11) FQ_CASE(12) FQ_CASE(13)
#undef FQ_CASE
        default: return FQ_ERR_ARG;
    }
}

}  // namespace fq

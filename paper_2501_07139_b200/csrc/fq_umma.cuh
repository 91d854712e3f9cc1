// Pieces shared by the tcgen05 GEMM kernels: bounded mbarrier waits, shared-memory matrix descriptors,
// the instruction descriptor and the TMA tensor map of a bf16 matrix.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>

#include "fq_internal.cuh"

namespace fq {

constexpr unsigned long long kGemmWaitNs = 2000000000ull;
constexpr int kUmmaBK = 64;              // K per stage: 64 bf16 = one 128-byte swizzle span

static __device__ __forceinline__ uint32_t g_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
static __device__ __forceinline__ unsigned long long g_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
static __device__ __forceinline__ uint32_t g_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// Bounded wait; also gives up as soon as another role raised the abort flag.
//   SLEEP_NS > 0: for waits that last most of a tile (the epilogue's): sleep between polls, leaving the issue slots to the other roles
template <int SLEEP_NS = 0>
static __device__ __forceinline__ bool g_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (g_try_wait(bar, parity)) return true;
    const unsigned long long t0 = g_ns();
    for (;;) {
        for (int i = 0; i < 32; i++) {
            if (g_try_wait(bar, parity)) return true;
            if constexpr (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
        }
        if (*abort_flag) return false;
        if (g_ns() - t0 > kGemmWaitNs) return false;
    }
}

// Shared-memory matrix descriptor of a K-major bf16 tile stored with the 128-byte swizzle: rows are
// 128 bytes apart, groups of 8 rows 1024 bytes apart.
static __device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);            // start address, 16-byte units
    d |= (uint64_t)1 << 16;                                  // leading byte offset (unused with swizzle)
    d |= (uint64_t)(1024 >> 4) << 32;                        // stride byte offset: 8 rows
    d |= (uint64_t)1 << 46;                                  // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                                  // swizzle mode: 128 bytes
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 256.
static __device__ __forceinline__ uint32_t umma_idesc_bf16(int m, int n)
{
    uint32_t d = 0;
    d |= 1u << 4;                       // accumulator format: fp32
    d |= 1u << 7;                       // A format: bf16
    d |= 1u << 10;                      // B format: bf16
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(m >> 4) << 24;
    return d;
}

static PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder()
{
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

// 2-D bf16 tensor [rows][cols] with row pitch ld elements; box = box_rows x 64 columns, 128-byte swizzle.
static int make_map(CUtensorMap* map, const void* base, long long rows, long long cols, long long ld, int box_rows)
{
    PFN_cuTensorMapEncodeTiled_v12000 enc = tensor_map_encoder();
    if (!enc) return FQ_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kUmmaBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? FQ_OK : FQ_ERR_CUDA;
}


}  // namespace fq

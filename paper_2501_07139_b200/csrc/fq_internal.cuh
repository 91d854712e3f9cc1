// Host-side context and the descriptors passed to the kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>
#include <vector>

#include "../../include/flexq.h"
#include "fq_layout.cuh"

namespace fq {

// One stored variant of a layer.
struct Variant {
    bool present = false;        // resident on the device: kernels may read `store`
    void* store = nullptr;       // blobs: scale/zero words + field arrays (fq_layout.cuh)
    const void* host = nullptr;  // the same bytes in host memory (swap model, fq_host_variant), or null
    bool swap_owned = false;     // `store` was allocated by fq_transition_swap: released when the variant is dropped
};

struct Layer {
    bool registered = false;
    int n_out = 0, k_in = 0, fmt = FQ_FMT_PACKED;
    int active_bits = 0;
    Variant var[9];              // PACKED: index = bits; PLANES: only [8]
};

constexpr int kUnitRowTiles = 2;   // a decode unit covers two 16-row tiles (32 output rows)

// What one decode op needs on the device.
struct GemvOp {
    const uint8_t* store;        // blobs [row_pair][k_blob]
    unsigned long long* partial; // split-K partial sums, one tagged word per (row pair, chunk, row, batch entry)
    // read by every consumer warp for every unit: kept together, 16-byte aligned, one vector load
    int blob_read;               // bytes of every blob that this op reads (all of it, or a nested child's prefix)
    int variant;                 // variant_index(format, bits): selects the specialised inner loop
    int batch;
    int n_chunks;                // K chunks
    const uint16_t* x;           // fp16 [batch][k_in]
    uint16_t* y;                 // fp16 [batch][n_out]
    int blob_stride;             // bytes from one blob to the next (size of the stored variant's blobs)
    int n_fields;
    uint8_t field_width[kMaxFields];
    uint8_t field_shift[kMaxFields];
    int bits;                    // code bytes per tile superstep = 512 * bits
    int n_out, k_in;
    int n_ss, n_kb;              // supersteps, k blobs
    int n_rp;                    // row pairs = units per K chunk
    int chunk_blobs;             // k blobs per K chunk (the last chunk may be shorter)
    int zero_adjust;             // subtracted from every zero point (mid-point fill of a nested child)
    int phase;                   // -1: no ordering
    int n_units;                 // n_chunks * n_rp
    int rot;                     // rotation of the CTA blocks for this op (evens out remainders)
    int split;                   // batch 1: consumer items per blob: 1 (both 16-row tiles) or 2 (one tile each)
};
static_assert(offsetof(GemvOp, blob_read) == 16 && offsetof(GemvOp, partial) == 8, "consumer block of the op descriptor");

struct StackHeader {
    int n_ops;
    int n_phases;
    long long total_units;
};

struct Ctx {
    int device = 0;
    int sm_count = 0;
    std::vector<Layer> layers;
    // workspace shared by all calls on this context
    char* ws = nullptr;          // device
    size_t ws_bytes = 0;
    int* status_dev = nullptr;   // device status word
    // stack-call staging
    char* stack_dev = nullptr;   // device copy of the op table
    size_t stack_dev_bytes = 0;
    // prefill: dequantised bf16 copy of the layer being multiplied
    char* gemm_ws = nullptr;
    size_t gemm_ws_bytes = 0;
    char* fused_ws = nullptr;            // fused GEMM, balanced runs: flags, then one fp32 tile slot per SM (+ 1)
    unsigned fused_epoch = 0;
    std::vector<void*> owned;    // device buffers allocated by fq_load, freed by fq_destroy
    uint64_t config_epoch = 0;
    unsigned launch_epoch = 0;   // tag of the split-K partials of the latest decode launch (never 0)
    // the op list that is currently uploaded: every argument word of the call that built it
    std::vector<uint64_t> stack_sig;
    bool stack_valid = false;
    StackHeader stack_hdr{};
    // pinned staging buffers of the op table take turns; an event per buffer marks the end of its last upload
    char* stage_host[2] = {nullptr, nullptr};
    size_t stage_host_bytes[2] = {0, 0};
    cudaEvent_t stage_done[2] = {nullptr, nullptr};
    int stage_next = 0;
    size_t ws_reserved = 0;      // split-K bytes that the registered layers need (each used once per launch)
    unsigned long long wait_limit_ns = 2000000000ull;   // limit of every device-side wait
};

// Bytes of device workspace for `n_ops` ops whose split-K needs are summed by the caller.
int ensure_workspace(Ctx* ctx, size_t bytes);

// kernels / launchers implemented in the .cu files
int launch_quantize(const float* w, int n_out, int k_in, int bits, uint8_t* codes, uint16_t* scales,
                    uint16_t* zeros, cudaStream_t st);
int launch_pack(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, int n_out, int k_in,
                int stored_bits, const FieldList& fl, void* store, cudaStream_t st);
int launch_export_packed(const void* store, int n_out, int k_in, int bits, const FieldList& fl,
                         uint32_t* out, cudaStream_t st);
int launch_export_planes(const void* store, int n_out, int k_in, int bits, const FieldList& fl,
                         uint32_t* out, cudaStream_t st);
int launch_export_meta(const void* store, int n_out, int k_in, int stored_bits, uint16_t* scales, uint16_t* zeros,
                       cudaStream_t st);

// Checked build (-DFQ_CHECKED): `inside` states that an index a kernel computed lies inside the buffer it is about to
// touch.  When it does not hold, the status word gets FQ_ERR_BOUNDS (the first error wins) and the result is false:
// the caller skips the access and winds the kernel down the way it does after a timeout.  Every lane of the
// warp evaluates the same condition wherever the result steers control flow.  In the normal build the condition
// is not evaluated.
#ifdef FQ_CHECKED
#define FQ_IN_BOUNDS(inside, status_ptr) ((inside) ? true : (atomicCAS((status_ptr), 0, FQ_ERR_BOUNDS), false))
#else
#define FQ_IN_BOUNDS(inside, status_ptr) true
#endif

// SM count of the current device (cached); sizes the grids of the grid-stride kernels that have no context at hand.
int current_sm_count();

int launch_stream_read(const void* src, size_t bytes, unsigned* sink, int sm_count, cudaStream_t st);

// Chunking policy of the decode kernel: k blobs (512 columns) per K chunk.
int gemv_chunk_blobs(int bits, int batch);
size_t gemv_partial_bytes_per_unit(int batch);
int launch_gemv_single(Ctx* ctx, const GemvOp& op, cudaStream_t st);                 // batch 2..8
int launch_gemm_fused(Ctx* ctx, const void* store, int blob_stride, const FieldList& fl, int zero_adjust, int n_out, int k_in,
                      const uint16_t* X, int M, int ldx, uint16_t* Y, int ldy, float* parts, unsigned* part_flags, unsigned epoch,
                      cudaStream_t st);                   // parts == nullptr: whole tiles; else balanced runs through these slots
size_t gemm_fused_part_bytes();          // bytes of one CTA's partial-sum slot
bool gemm_fused_wants_balance(int M, int n_out, int sm_count);
struct CtaWork;
int launch_gemv1_single(Ctx* ctx, const GemvOp& op, cudaStream_t st);                // batch 1
// table_dev: [GemvOp x n_ops][int phase_total x max(n_phases,1)][uint2 strips x sm_count x n_ops]
int launch_gemv1_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, cudaStream_t st);
int gemv1_max_phases();
int gemv1_max_ops();
int gemv1_max_k();
int gemv1_chunk_blobs(int blob_read_bytes);
uint2 gemv1_pack_range(const CtaWork& w, int n_chunks);
int launch_gemv_static(Ctx* ctx, GemvOp op, size_t partial_bytes, cudaStream_t st);
// table_dev: [GemvOp x n_ops][long long phase_total x max(n_phases,1)][int cta_units x sm_count]
int launch_gemv_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, int max_batch, cudaStream_t st);
// Units of an op (n_units units, block rotation rot) that CTA `cta` of `grid` processes: [lo, hi).
void gemv_cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi);

// ---- how a decode op is dealt to the CTAs of the persistent grid (shared by host and device code)
// The pieces of an op (batch 1: the blobs of its 32-row strips; batch 2..8: K chunks of row pairs) are numbered
// strip-major, u = rp * pieces_per_strip + i, and dealt in contiguous blocks; the block boundaries rotate from
// op to op so that the remainders even out.
FQ_HD void cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi)
{
    const unsigned c = (unsigned)((cta + grid - rot) % grid);
    lo = (int)((unsigned)n_units * c / (unsigned)grid);              // n_units * grid < 2^31 (checked on the host)
    hi = (int)((unsigned)n_units * (c + 1u) / (unsigned)grid);
}
// The strips a CTA touches: rp_first .. rp_last; only the first may start and only the last may end inside a strip.
struct CtaWork {
    int lo, hi, rp_first, rp_last;
    FQ_HD bool any() const { return hi > lo; }
    // pieces [c0, c1) of strip rp that belong to this CTA
    FQ_HD void chunks(int n_chunks, int rp, int& c0, int& c1) const
    {
        c0 = rp == rp_first ? lo - rp * n_chunks : 0;
        c1 = rp == rp_last ? hi - rp * n_chunks : n_chunks;
    }
    // strips that this CTA finishes (it owns their first piece) and therefore writes to y
    FQ_HD int finishing(int n_chunks) const
    {
        if (!any()) return 0;
        return rp_last - rp_first + 1 - (lo - rp_first * n_chunks > 0 ? 1 : 0);
    }
};
FQ_HD CtaWork cta_work(int n_units, int n_chunks, int rot, int cta, int grid)
{
    CtaWork w;
    cta_range(n_units, rot, cta, grid, w.lo, w.hi);
    w.rp_first = w.lo / n_chunks;
    w.rp_last = w.hi > w.lo ? (w.hi - 1) / n_chunks : w.rp_first;
    return w;
}

int launch_gemm(Ctx* ctx, const void* store, int blob_stride, const FieldList& fl, int zero_adjust, int n_out, int k_in,
                const uint16_t* X, int M, int ldx, uint16_t* Y, int ldy, void* w_scratch, cudaStream_t st);

}  // namespace fq

struct fq_ctx : fq::Ctx {};

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
    bool present = false;
    void* store = nullptr;       // blobs: scale/zero words + field arrays (fq_layout.cuh)
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
    char* stack_host = nullptr;  // pinned
    size_t stack_host_bytes = 0;
    // prefill: dequantised bf16 copy of the layer being multiplied
    char* gemm_ws = nullptr;
    size_t gemm_ws_bytes = 0;
    std::vector<void*> owned;    // device buffers allocated by fq_load, freed by fq_destroy
    uint64_t config_epoch = 0;
    unsigned launch_epoch = 0;   // tag of the split-K partials of the latest decode launch (never 0)
    uint64_t stack_key = 0;      // hash of the op list that is currently uploaded
    bool stack_valid = false;
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

// Chunking policy of the decode kernel: k blobs (512 columns) per K chunk.
int gemv_chunk_blobs(int bits, int batch);
size_t gemv_partial_bytes_per_unit(int batch);
int launch_gemv_single(Ctx* ctx, const GemvOp& op, cudaStream_t st);
int launch_gemv_static(Ctx* ctx, GemvOp op, size_t partial_bytes, cudaStream_t st);
// table_dev: [GemvOp x n_ops][long long phase_total x max(n_phases,1)][int cta_units x sm_count]
int launch_gemv_stack(Ctx* ctx, const StackHeader& hdr, const char* table_dev, int max_batch, cudaStream_t st);
// Units of an op (n_units units, block rotation rot) that CTA `cta` of `grid` processes: [lo, hi).
void gemv_cta_range(int n_units, int rot, int cta, int grid, int& lo, int& hi);

int launch_gemm(Ctx* ctx, const void* store, int blob_stride, const FieldList& fl, int zero_adjust, int n_out, int k_in,
                const uint16_t* X, int M, int ldx, uint16_t* Y, int ldy, void* w_scratch, cudaStream_t st);

}  // namespace fq

struct fq_ctx : fq::Ctx {};

/*
 * flexq -- elastic mixed-bit dequantize-and-matmul for NVIDIA B200 (sm_100a).
 *
 * C ABI of the hot path of FlexQuant's elastic hosting scheme (arXiv 2501.07139).
 * In that scheme a model is served from an ensemble of quantised layers and every
 * elastic configuration ("EQM", Sec. III-A) assigns each module one of a few stored
 * bit-widths.  This library holds the stored variants on one GPU, switches between
 * configurations without moving weights, and runs every linear layer as a fused
 * dequantize-and-matmul at whatever bit-width the active configuration gives it
 * (Sec. II-A: the arithmetic itself stays in a standard 16-bit format).
 *
 * Conventions
 *   - All functions return FQ_OK (0) or a negative FQ_ERR_* code.  Nothing throws,
 *     aborts or traps.  fq_strerror() names a code.
 *   - "dev" pointers are device memory of the context's GPU, "host" pointers are host
 *     memory.  The library never takes ownership of a caller's buffer; buffers that a
 *     context RETAINS must stay alive until fq_destroy().
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls on one context must be ordered on one stream (or otherwise serialised):
 *     they share the context's workspace.
 *   - W is [n_out][k_in] row-major, quantised per group of 128 consecutive columns:
 *     w^ = (q - z) * s with fp16 scale s and fp16 zero point z (an integer value).
 *     k_in must be a multiple of 128; group must be 128.
 *   - fp16 / bf16 values cross the ABI as uint16_t bit patterns.
 */
#ifndef FLEXQ_H
#define FLEXQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fq_ctx fq_ctx;   /* opaque */

enum { FQ_FMT_PACKED = 0,       /* one stored variant per bit-width (Sec. III-A: QM(n) variants)   */
       FQ_FMT_PLANES = 1 };     /* one 8-bit parent whose bits are nested, most significant first (Sec. II-B, AnyPrecision) */

enum { FQ_OK = 0,
       FQ_ERR_ARG = -1,         /* NULL pointer, bad layer index, bad enum                */
       FQ_ERR_BITS = -2,        /* bit-width outside [2, 8] (or not 8 for a PLANES parent) */
       FQ_ERR_SHAPE = -3,       /* group != 128, k_in % 128 != 0, sizes <= 0, batch > 8 ... */
       FQ_ERR_ALIGN = -4,       /* a buffer is not 16-byte aligned                          */
       FQ_ERR_NO_VARIANT = -5,  /* configuration asks for a bit-width that is not stored    */
       FQ_ERR_NOT_PACKED = -6,  /* layer used before fq_pack_layer / fq_set_config          */
       FQ_ERR_CUDA = -7,        /* a CUDA runtime call failed (no device, out of memory...) */
       FQ_ERR_TIMEOUT = -8,     /* a bounded device-side wait ran out (see fq_status)       */
       FQ_ERR_SCRATCH = -9,     /* problem needs more than the built-in scratch (fq_gemv_static) */
       FQ_ERR_ONE_WAY = -10,    /* a layer would go to a higher bit-width (fq_transition)    */
       FQ_ERR_IO = -11,         /* file could not be opened, read or written, or is malformed */
       FQ_ERR_BOUNDS = -12 };   /* checked build only (-DFQ_CHECKED): a kernel computed an address outside its
                                   buffer; the access was skipped (see fq_status)                         */

#define FQ_MAX_BATCH 8          /* decode batch handled by the GEMV family */

/* Creates a context for `device` with room for `n_layers` layers (indices 0..n_layers-1). */
int fq_create(fq_ctx** out, int device, int n_layers);
/* Frees the context and its workspace.  Caller-owned buffers are not touched. */
int fq_destroy(fq_ctx* ctx);

/* Bytes the caller must allocate for one stored variant: codes AND scale/zero words, which the
 * device layout interleaves (blobs of 32 rows x 512 columns) so that a decode step fetches both
 * with one copy.  This is the algorithmic size n_out*k_in*bits/8 + n_out*(k_in/128)*4
 * (bits = 8 for a PLANES parent) computed on n_out rounded up to 32 and k_in rounded up to 512.
 * Returns 0 on invalid arguments. */
size_t fq_store_bytes(int n_out, int k_in, int bits, int fmt);

/* Min-max asymmetric group quantiser (the step in front of the path; the paper takes the
 * quantised models QM(n) of Sec. III-A as given).  Per group of 128 columns, in double:
 * s = fp16((max-min)/(2^b-1)) (2^-14 if that is zero), z = clamp(rint(-min/s), 0, 2^b-1),
 * q = clamp(rint(w/s) + z, 0, 2^b-1).
 *   w_dev      float32 [n_out][k_in]             (read)
 *   codes_dev  uint8   [n_out][k_in], one code per byte (written)
 *   scales_dev, zeros_dev  fp16 [n_out][k_in/128] (written)
 * Needs no context; runs on the current device. */
int fq_quantize_layer(const float* w_dev, int n_out, int k_in, int bits, int group,
                      uint8_t* codes_dev, uint16_t* scales_dev, uint16_t* zeros_dev, void* stream);

/* Registers one stored variant of `layer` and converts it to the device layout
 * (Sec. III-A: every module is stored at a few bit-widths; Sec. II-B for PLANES).
 *   PACKED: `bits` in [2,8] is the width of this variant; call again with another width
 *           to add a variant of the same layer (same shape).
 *   PLANES: `bits` must be 8; the parent is stored as four 2-bit fields (bits 7..6, 5..4, 3..2,
 *           1..0), most significant first inside every blob, so a b-bit child reads the first
 *           ceil(b / 2) fields of every blob (a child of odd width ignores the low bit of its last
 *           field) and every b in [2,8] becomes selectable.
 *   codes_dev   uint8 [n_out][k_in], one code per byte; read, not retained.
 *   scales_dev, zeros_dev   fp16 [n_out][k_in/128]; read, not retained.
 *   store_out_dev fq_store_bytes() bytes, 256-byte aligned; written and RETAINED.
 * The first variant packed for a layer becomes its active one. */
int fq_pack_layer(fq_ctx* ctx, int layer, int n_out, int k_in, int bits, int group, int fmt,
                  const uint8_t* codes_dev, const uint16_t* scales_dev, const uint16_t* zeros_dev,
                  void* store_out_dev, void* stream);

/* Activates an elastic configuration (Sec. III-A: an EQM is a per-module choice among the
 * stored variants; Sec. II-C: switching should cost as little memory traffic as possible).
 *   bits_host  uint8 [n_layers]: bit-width of every registered layer, each in [2,8].
 *   footprint_bytes_host (may be NULL): receives the memory footprint of the configuration,
 *       sum over layers of n_out*k_in*b/8 code bytes + n_out*(k_in/128)*4 scale/zero bytes.
 * Fails with FQ_ERR_NO_VARIANT (and changes nothing) if a PACKED layer has no variant at
 * the requested width.  Host-only bookkeeping: no weight byte is read, written or moved
 * and nothing is enqueued on `stream`. */
int fq_set_config(fq_ctx* ctx, const uint8_t* bits_host, int n_layers,
                  uint64_t* footprint_bytes_host, void* stream);

/* One-way transition to another elastic configuration (Sec. III-B: a module may only move to a
 * lower bit-width, which keeps the memory traffic of a transition small; Sec. II-C: what has to be
 * brought into memory on a switch should be minimal).  Same arguments and checks as fq_set_config;
 * on success the configuration is active and `report_host` (may be NULL) says what the step costs in
 * a deployment that keeps only the active variants resident:
 *   nested (PLANES) layer: lowering frees the dropped planes, N*K*(b0-b1)/8 bytes, and loads nothing;
 *                          raising loads the re-appended planes; scale/zero words never move.
 *   PACKED layer         : a change frees the old variant and loads the new one (codes + scale/zero).
 * The library itself keeps every registered variant resident: nothing is copied or released here.
 * require_one_way != 0: a configuration that raises any layer returns FQ_ERR_ONE_WAY and changes nothing. */
typedef struct fq_transition_report {
    uint64_t bytes_freed;       /* memory a deployment can release after this step               */
    uint64_t bytes_loaded;      /* memory it has to bring in before this step                    */
    uint64_t footprint_from;    /* footprint of the configuration that was active                */
    uint64_t footprint_to;      /* footprint of the new configuration                            */
    int layers_changed;
    int one_way;                /* 1: no layer goes to a higher bit-width                        */
} fq_transition_report;
int fq_transition(fq_ctx* ctx, const uint8_t* to_bits_host, int n_layers, int require_one_way,
                  fq_transition_report* report_host, void* stream);

/* Swap model of a transition (Sec. II-C: before a block of parameters is swapped out, its replacement has to
 * be loaded in addition to the current hybrid model; Sec. III-B: one-way moves keep that traffic small).
 * Only the variants the active configuration uses stay on the device; the others wait in host memory.
 *
 * fq_host_variant registers a PACKED variant of `bits` bits of `layer` whose stored bytes (exactly what
 * fq_pack_layer wrote into a device buffer, fq_store_bytes(n_out, k_in, bits) of them) lie at `store_host`.
 * The buffer stays the caller's and must outlive the context; page-locked memory makes the copies
 * asynchronous.  The first variant of a layer fixes its shape.  Nothing is copied here.
 *
 * fq_transition_swap moves to configuration `to_bits_host` layer by layer: a layer whose bit-width changes first
 * gets its new variant (cudaMallocAsync + one cudaMemcpyAsync from the host copy on `stream`, unless it is
 * resident already), then switches, then releases the variant it used before (cudaFreeAsync on `stream`) if
 * that one was brought in by an earlier swap and still has its host copy.  Variants given to fq_pack_layer in
 * the caller's own device buffers are used where they are and never released.  Nested (PLANES) layers only
 * switch: a child is a prefix of the resident parent.  Decode and prefill calls issued on `stream` afterwards see
 * the new configuration; calls issued before it keep reading the old variants, which are released in stream order.
 * The first call (no configuration active yet) loads every layer.
 * All checks of fq_transition happen before anything changes.  If an allocation or copy fails part-way the call
 * returns FQ_ERR_CUDA; every layer is then entirely on its old or entirely on its new variant.
 * Allocates, and may wait for the stream-ordered allocator: a control-path call, not a hot one. */
typedef struct fq_swap_report {
    uint64_t bytes_loaded;      /* copied host -> device by this call                              */
    uint64_t bytes_freed;       /* device memory released by this call                             */
    uint64_t peak_extra_bytes;  /* most memory held, during the call, beyond what was resident at its start */
    uint64_t resident_bytes;    /* swapped-in variants on the device after the call                */
    uint64_t footprint_from;    /* algorithmic footprint (as fq_set_config) before / after         */
    uint64_t footprint_to;
    int layers_changed;
    int one_way;
} fq_swap_report;
int fq_host_variant(fq_ctx* ctx, int layer, int n_out, int k_in, int bits, const void* store_host);
int fq_transition_swap(fq_ctx* ctx, const uint8_t* to_bits_host, int n_layers, int require_one_way,
                       fq_swap_report* report_host, void* stream);

/* The ensemble on disk (Sec. III / V-B: the stored quantized variants whose total size is the paper's
 * "storage cost").  fq_save writes every registered variant of every layer, exactly as stored on the
 * device, plus shapes, formats and the active configuration; it synchronises the device.
 * File (little-endian): "FLEXQ1\0\0", u32 n_layers, u32 0; per layer u32 registered, n_out, k_in, fmt,
 * active_bits, variant_mask (bit b = a variant of b bits follows); per variant u64 bytes, then the bytes.
 * fq_load registers the file's layers in `ctx` (created with at least as many layers, none registered yet)
 * and activates the saved configuration.  Unlike fq_pack_layer it ALLOCATES the device buffers itself
 * (cudaMalloc); the context owns them until fq_destroy.  Errors: FQ_ERR_ARG (path, context state),
 * FQ_ERR_IO (open / read / write / malformed file), FQ_ERR_CUDA. */
int fq_save(fq_ctx* ctx, const char* path, uint64_t* bytes_written_host);
int fq_load(fq_ctx* ctx, const char* path);

/* Tree search for an ensemble of elastic configurations (Sec. III-B, Algorithm 1), on tables instead of
 * perplexity runs.  n_modules modules, n_levels stored precisions ordered from n_up (level 0) down to n_low
 * (level n_levels-1); a configuration is one level per module.  Host tables, all [n_modules][n_levels]:
 *   cost : what calibrationEval adds when module m sits at level l (cost[m][0] = 0); a configuration is
 *          evaluated as the sum over its modules;
 *   sens : the pre-generated sensitivity of replacing module m of QM(n_up) by level l (smaller = ranked higher);
 *   foot : bytes of module m stored at level l.
 * Each iteration generates, for the last configuration of each of the (at most) `stems` ensembles, every
 * successor that lowers ONE module by ONE level (the one-way rule), keeps the `branches` least sensitive per
 * ensemble, evaluates them, ranks by (cost, footprint, generation order) and keeps the best `stems` distinct
 * ones.  It ends when every module is at n_low, after n_modules*(n_levels-1) steps, and returns the ensemble
 * with the smallest sum of cost over its configurations.
 *   chain_out uint8 [n_modules*(n_levels-1)+1][n_modules]: level per module, first row all 0.  Host memory. */
int fq_search_chain(const double* cost, const double* sens, const uint64_t* foot, int n_modules, int n_levels,
                    int stems, int branches, uint8_t* chain_out, int* n_states_out, double* curve_cost_out);

/* Pruning of mid-precision modules (Sec. III-C).  Every (module, mid level) pair is ranked by how many
 * configurations of `chain` use it, ties by use at lower footprints (later in the chain); the lowest-ranked
 * floor(fraction * pairs) are dropped.  A configuration that used a dropped pair falls to the next lower stored
 * level.  dropped_out uint8 [n_modules][n_levels] flags; storage = sum of foot over the kept pairs. */
int fq_prune_chain(const uint8_t* chain, int n_states, int n_modules, int n_levels, const uint64_t* foot, double fraction,
                   uint8_t* pruned_chain_out, uint8_t* dropped_out, uint64_t* storage_before_out, uint64_t* storage_after_out);

/* Output error of a layer, the stand-in for the calibration-set evaluation (Sec. III-B): writes
 * sums_dev[0] = sum (a-b)^2 and sums_dev[1] = sum b^2 over n bf16 values (device pointers). */
int fq_sqdiff(const uint16_t* a_bf16_dev, const uint16_t* b_bf16_dev, size_t n, double* sums_dev, void* stream);

/* Decode (Sec. II-A): y[n] = sum_k x[k] * w^[n][k] at the layer's active bit-width.
 *   x_dev fp16 [k_in], y_dev fp16 [n_out]; both 16-byte aligned.  fp32 accumulation.
 *   Layers with k_in <= 14336 run in the batch-1 kernel (the activations of one 32-row strip stay in shared
 *   memory); wider layers run in the batch kernel, slower per byte but without a limit on k_in.
 * Enqueues one kernel on `stream`; neither allocates (the scratch was reserved by fq_pack_layer) nor
 * synchronises.  An activation group that holds an infinity or a NaN makes every output NaN. */
int fq_gemv(fq_ctx* ctx, int layer, const uint16_t* x_dev, uint16_t* y_dev, void* stream);

/* Same result as fq_gemv, for callers that must not allocate device memory.  (The paper has no
 * counterpart; this is a deployment convenience.)  fq_gemv takes its scratch from the context's
 * workspace, device memory that fq_create / fq_pack_layer obtained with cudaMalloc.  That is
 * not acceptable for callers such as a real-time serving loop with a fixed memory budget, code
 * running while another library owns the allocator, or a host thread that must never block on
 * the device-wide synchronisation an allocation implies.  This variant keeps its scratch (the
 * per-blob partial sums that two thread blocks exchange when they share a 32-row strip of the
 * matrix) in a fixed array that is part of the library image: FQ_STATIC_SCRATCH_BYTES on every
 * GPU that loads the library, held until the process exits.  It calls no cudaMalloc / cudaFree
 * and nothing that allocates.
 *   - batch 1 only; x_dev fp16 [k_in], y_dev fp16 [n_out], 16-byte aligned, caller-owned.
 *   - Returns FQ_ERR_SCRATCH (and launches nothing) when the layer needs more scratch than the
 *     array holds: 256 bytes per (32-row strip x blob of 512 columns), i.e.
 *     ceil(n_out / 32) * ceil(k_in / 512) * 256 bytes.  Every Llama-2-7B / 13B shaped layer fits.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current); make that first call before starting any stream capture.
 *   - All calls share the one array and it keeps whatever the last call left there.  Nothing
 *     in it has to be cleared: every partial sum carries the tag of the call that wrote it and
 *     is ignored under any other tag.  Two calls that overlap on the GPU (different streams,
 *     or different contexts) race on it: serialise them.  Host calls are not thread-safe either:
 *     the per-device tag counter and address cache are plain statics. */
#define FQ_STATIC_SCRATCH_BYTES (2u << 20)
int fq_gemv_static(fq_ctx* ctx, int layer, const uint16_t* x_dev, uint16_t* y_dev, void* stream);

/* Decode at batch 1..8:  Y[b][n] = sum_k X[b][k] * w^[n][k].
 *   x_dev fp16 [batch][k_in], y_dev fp16 [batch][n_out], densely packed rows. */
int fq_gemv_batched(fq_ctx* ctx, int layer, const uint16_t* x_dev, int batch, uint16_t* y_dev, void* stream);

/* Decode through a whole stack of layers in ONE persistent launch; op i computes
 * y_dev[i] = x_dev[i] . w^(layers[i]) exactly as fq_gemv_batched would (bit-identical).
 *   layers_host int [n_ops]; x_dev_host / y_dev_host: host arrays of n_ops device pointers.
 *   phases_host (may be NULL = no ordering): non-decreasing int [n_ops], starting at 0 and
 *       without gaps; an op of phase p does not read its x before every op of phase p-1 has
 *       written its y (weights of later ops are prefetched meanwhile).
 * Batch 1: at most 512 ops and 1024 phases per call (FQ_ERR_SHAPE otherwise).
 * The call builds a table (ops, and which strips every thread block computes) and uploads it from a
 * pinned buffer; a call with the same arguments under the same configuration reuses the uploaded
 * table and only launches the kernel.  The workspace was sized by fq_pack_layer for lists that use
 * every layer at most once; a list that repeats layers may grow it (device allocation + sync). */
int fq_gemv_stack(fq_ctx* ctx, int n_ops, const int* layers_host,
                  const uint16_t* const* x_dev_host, uint16_t* const* y_dev_host,
                  const int* phases_host, int batch, void* stream);

/* Prefill / calibration-set evaluation (Sec. III-B: every candidate EQM is run forward over
 * token sequences):  Y[m][n] = sum_k X[m][k] * w^[n][k].
 *   X_dev bf16 [M][ldx >= k_in], Y_dev bf16 [M][ldy >= n_out], row-major, 16-byte aligned,
 *   ldx and ldy multiples of 8, 1 <= M <= 2^20.
 * One fused kernel: X tiles arrive by TMA, the stored blobs are dequantised inside the kernel
 * (w^ = (q - z) * s exactly in fp32, rounded once to bf16) into the shared-memory operand tiles of
 * the tensor cores (tcgen05, fp32 accumulation in TMEM), Y is rounded once to bf16.  Enqueues one
 * kernel on `stream` and encodes one tensor map on the host.  Shapes whose 256 x 256 output tiles would
 * leave the last wave of thread blocks mostly empty are cut into equal runs of (tile, K stage) work
 * instead; a tile shared by two blocks is then the fp32 sum of two partial accumulations (summation
 * order differs from the whole-tile case in the last bit), passed through a 38 MB workspace that the
 * context allocates the first time such a shape is used.  One fq_gemm at a time per context. */
int fq_gemm(fq_ctx* ctx, int layer, const uint16_t* X_dev, int M, int ldx,
            uint16_t* Y_dev, int ldy, void* stream);

/* The same product computed in two passes, kept as the comparison point of the fused kernel: the
 * layer is first dequantised to bf16 into a workspace of n_out*k_in*2 bytes that the context owns
 * (grown with a device allocation when a larger layer is first used), then multiplied by a plain
 * tcgen05 GEMM.  Same arguments, same rounding points, same results up to the fp32 summation order. */
int fq_gemm_two_pass(fq_ctx* ctx, int layer, const uint16_t* X_dev, int M, int ldx,
                     uint16_t* Y_dev, int ldy, void* stream);

/* Test / reporting support ------------------------------------------------------------ */

/* Writes the canonical form of what is stored for `layer` at width `bits`:
 *   PACKED: uint32 [n_out][k_in*bits/32], per row a little-endian bitstream, code k in bits
 *           [k*bits, (k+1)*bits).
 *   PLANES: uint32 [bits][n_out][k_in/32], plane t holds parent bit 7-t, bit (k%32) of a
 *           word belongs to column k; rebuilt from the first ceil(bits / 2) stored fields.
 * out_dev: n_out*k_in*bits/8 bytes. */
int fq_export_layer(fq_ctx* ctx, int layer, int bits, void* out_dev, void* stream);
/* Writes the stored scales and zero points back as fp16 [n_out][k_in/128] each. */
int fq_export_meta(fq_ctx* ctx, int layer, int bits, uint16_t* scales_dev, uint16_t* zeros_dev, void* stream);

/* Sum of the code and scale/zero bytes of every stored variant (the "storage cost" axis). */
uint64_t fq_storage_bytes(const fq_ctx* ctx);
/* Active bit-width of a layer, or a negative error. */
int fq_active_bits(const fq_ctx* ctx, int layer);
/* Synchronises the context's device, then returns and clears the device status word
 * (FQ_OK, or FQ_ERR_TIMEOUT if a bounded wait inside a kernel gave up). */
int fq_status(fq_ctx* ctx);

/* Limit of every device-side wait of the decode kernels, in nanoseconds (default 2e9; 0 restores the
 * default).  Diagnostic support: with a limit shorter than any real wait a launch gives up at once,
 * records FQ_ERR_TIMEOUT, drains its copies and returns; fq_status() then reports the code and resets
 * the counters, and later launches are unaffected. */
int fq_set_wait_limit_ns(fq_ctx* ctx, unsigned long long ns);

/* Measurement support: one read-only pass over `bytes` of device memory (16-byte aligned) with vector loads,
 * enqueued on `stream`.  Timing it gives the streaming-read bandwidth of the part, the ceiling of a kernel
 * that, like the decode path, reads weights once and writes almost nothing. */
int fq_stream_read(fq_ctx* ctx, const void* src_dev, size_t bytes, void* stream);

/* Algorithmic sizes (the terms of the footprint, Sec. III): bytes of the b-bit codes of a layer,
 * n_out * k_in * bits / 8, and of its scale/zero words, n_out * (k_in / group) * 4.  0 for invalid
 * arguments.  (fq_store_bytes is the size of the stored variant including tile padding.) */
size_t fq_code_bytes(int n_out, int k_in, int bits);
size_t fq_meta_bytes(int n_out, int k_in, int group);
const char* fq_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* FLEXQ_H */

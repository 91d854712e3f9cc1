// C ABI entry points: context, layer registry, configuration / footprint accountant,
// argument checks and dispatch to the kernels.
#include <cstdio>
#include <cstring>
#include <new>

#include "fq_internal.cuh"

using namespace fq;

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

namespace {

constexpr size_t kWsHead = 8 * 4096 + 64;      // phase counters (4096 x u64) + exit counter
constexpr int kMaxPhases = 4096;
// Workspace layout: [phase counters | exit counter][split-K partials].  A partial is a 64-bit word (fp32 sum,
// launch tag); the workspace starts out zeroed and tag 0 is never used, so a word is valid only when its
// tag equals the tag of the running launch.
constexpr size_t kPartialBase = kWsHead + 192;

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = prev == dev || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

FieldList active_fields(const Layer& L, int bits) { return L.fmt == FQ_FMT_PLANES ? plane_fields(bits) : packed_fields(bits); }

const Variant* active_variant(const Layer& L, int bits)
{
    const Variant& v = L.fmt == FQ_FMT_PLANES ? L.var[8] : L.var[bits];
    return v.present ? &v : nullptr;
}

// Batch 1: a group of ops (one dependency phase) that gives a CTA fewer blobs than this is cut into items of one
// 16-row tile instead of one blob, so that its 16 consumer warps end the phase after the same number of items
// (a phase of the 7B stack is 7 to 37 blobs per CTA: whole blobs leave the phase waiting for 1, 2 or 3 blob times
// where half blobs need 0.5, 1.5 or 2.5).  Long groups keep whole blobs, and so do variants of one or two fields,
// whose blobs are cheap: an item has fixed costs (measured on the 7B stack, ordered: nested 7-bit 2.66 -> 2.36 ms
// with half blobs, packed mixed 1.46 -> 1.55 ms, so only the many-field variants are cut).
constexpr int kSplitBelowBlobsPerCta = 48;
constexpr int kSplitAboveFields = 2;

// Fills the device descriptor of one decode op (everything except workspace pointers and unit_base).
//   one : the op runs in the batch-1 kernel (gemv1); otherwise in the batch kernel, which also serves batch 1 for
//         layers whose k_in exceeds what the batch-1 kernel keeps in shared memory
int fill_op(const Ctx* ctx, int layer, const uint16_t* x, uint16_t* y, int batch, bool one, GemvOp& op)
{
    if (layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    const Layer& L = ctx->layers[layer];
    if (!L.registered || L.active_bits == 0) return FQ_ERR_NOT_PACKED;
    if (!x || !y) return FQ_ERR_ARG;
    if (batch < 1 || batch > FQ_MAX_BATCH) return FQ_ERR_SHAPE;
    if (!aligned(x, 16) || !aligned(y, 16)) return FQ_ERR_ALIGN;
    const int bits = L.active_bits;
    const Variant* v = active_variant(L, bits);
    if (!v) return FQ_ERR_NO_VARIANT;
    const FieldList fl = active_fields(L, bits);
    std::memset(&op, 0, sizeof op);
    for (int i = 0; i < fl.n; i++) {
        op.field_width[i] = fl.width[i];
        op.field_shift[i] = fl.shift[i];
    }
    op.n_fields = fl.n;
    op.bits = bits;
    op.variant = variant_index(L.fmt == FQ_FMT_PLANES, bits);
    op.store = static_cast<const uint8_t*>(v->store);
    op.blob_stride = blob_bytes(L.fmt == FQ_FMT_PLANES ? 8 : bits);
    op.blob_read = blob_bytes(L.fmt == FQ_FMT_PLANES ? plane_read_bits(bits) : bits);   // a nested child reads whole 2-bit fields
    op.x = x;
    op.y = y;
    op.n_out = L.n_out;
    op.k_in = L.k_in;
    op.n_ss = supersteps(L.k_in);
    op.n_kb = k_blobs(L.k_in);
    op.n_rp = row_pairs(L.n_out);
    op.chunk_blobs = one ? gemv1_chunk_blobs(op.blob_read)
                                : gemv_chunk_blobs(L.fmt == FQ_FMT_PLANES ? plane_read_bits(bits) : bits, batch);
    op.n_chunks = (op.n_kb + op.chunk_blobs - 1) / op.chunk_blobs;
    op.batch = batch;
    // nested child: codes are the parent's top bits; the dropped bits are filled with their mid-point
    op.zero_adjust = (L.fmt == FQ_FMT_PLANES && bits < 8) ? (1 << (7 - bits)) : 0;
    // what is dealt to the CTAs: batch 1 the blobs of every strip, batch 2..8 the K chunks of every row pair
    op.n_units = (one ? op.n_kb : op.n_chunks) * op.n_rp;
    if ((long long)op.n_units * 1024 >= (1ll << 31)) return FQ_ERR_SHAPE;              // 32-bit unit arithmetic on the device
    if (one && (batch != 1 || L.k_in > gemv1_max_k())) return FQ_ERR_SHAPE;                   // a strip's activations stay in shared memory
    op.phase = -1;
    op.rot = 0;
    // a lone matrix is a few blobs per CTA: items of one 16-row tile spread them over twice as many consumer warps
    op.split = (one && fl.n > kSplitAboveFields && op.n_units < kSplitBelowBlobsPerCta * ctx->sm_count) ? 2 : 1;
    return FQ_OK;
}

// Split-K scratch of one op.  Batch 1: one tagged word per (strip, blob, row) -- only strips that two CTAs
// share are ever written.  Batch 2..8: one tagged word per (row pair, K chunk, row, batch entry).
size_t op_partial_bytes(const GemvOp& op, bool one, int max_batch)
{
    if (one) return op.n_kb <= 1 ? 0 : (size_t)op.n_rp * op.n_kb * 32 * sizeof(unsigned long long);
    if (op.n_chunks <= 1) return 0;
    return (size_t)op.n_rp * op.n_chunks * gemv_partial_bytes_per_unit(max_batch);
}

// Scratch that a registered layer can need in one launch, whatever its active variant and the batch.
size_t layer_partial_bytes(int n_out, int k_in)
{
    const size_t n_rp = (size_t)row_pairs(n_out), n_kb = (size_t)k_blobs(k_in);
    const size_t b1 = n_rp * n_kb * 32 * sizeof(unsigned long long);
    const size_t b8 = n_rp * n_kb * gemv_partial_bytes_per_unit(FQ_MAX_BATCH);     // chunks are whole blobs
    return (size_t)round_up((int64_t)(b1 > b8 ? b1 : b8), 256);
}

}  // namespace

namespace fq {

int ensure_workspace(Ctx* ctx, size_t bytes)
{
    if (bytes <= ctx->ws_bytes) return FQ_OK;
    const size_t want = (size_t)round_up((int64_t)(bytes + bytes / 2), 1 << 20);
    char* p = nullptr;
    FQ_CUDA_OK(cudaDeviceSynchronize());
    FQ_CUDA_OK(cudaMalloc(&p, want));
    if (cudaMemset(p, 0, want) != cudaSuccess) { cudaFree(p); return FQ_ERR_CUDA; }
    FQ_CUDA_OK(cudaDeviceSynchronize());
    if (ctx->ws) cudaFree(ctx->ws);
    ctx->ws = p;
    ctx->ws_bytes = want;
    ctx->stack_valid = false;          // cached op tables point into the old workspace
    return FQ_OK;
}

}  // namespace fq

extern "C" {

const char* fq_strerror(int code)
{
    switch (code) {
        case FQ_OK: return "ok";
        case FQ_ERR_ARG: return "invalid argument";
        case FQ_ERR_BITS: return "bit-width out of range";
        case FQ_ERR_SHAPE: return "unsupported shape";
        case FQ_ERR_ALIGN: return "buffer not aligned";
        case FQ_ERR_NO_VARIANT: return "no stored variant at this bit-width";
        case FQ_ERR_NOT_PACKED: return "layer not packed";
        case FQ_ERR_CUDA: return "CUDA runtime error";
        case FQ_ERR_TIMEOUT: return "device-side wait timed out";
        case FQ_ERR_SCRATCH: return "layer needs more than the built-in scratch";
        case FQ_ERR_ONE_WAY: return "transition would raise a layer's bit-width";
        case FQ_ERR_IO: return "file could not be opened, read or written, or is malformed";
        case FQ_ERR_BOUNDS: return "a kernel computed an address outside its buffer (checked build)";
        default: return "unknown error";
    }
}

int fq_create(fq_ctx** out, int device, int n_layers)
{
    if (!out || n_layers < 1 || n_layers > (1 << 20) || device < 0) return FQ_ERR_ARG;
    *out = nullptr;
    int count = 0;
    FQ_CUDA_OK(cudaGetDeviceCount(&count));
    if (device >= count) return FQ_ERR_CUDA;
    DeviceGuard guard(device);
    if (!guard.ok) return FQ_ERR_CUDA;
    fq_ctx* ctx = new (std::nothrow) fq_ctx();
    if (!ctx) return FQ_ERR_ARG;
    ctx->device = device;
    ctx->layers.resize(n_layers);
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaMalloc(&ctx->status_dev, sizeof(int)) != cudaSuccess ||
        cudaMemset(ctx->status_dev, 0, sizeof(int)) != cudaSuccess ||
        ensure_workspace(ctx, kPartialBase + (1 << 20)) != FQ_OK) {
        if (ctx->status_dev) cudaFree(ctx->status_dev);
        delete ctx;
        return FQ_ERR_CUDA;
    }
    *out = ctx;
    return FQ_OK;
}

int fq_destroy(fq_ctx* ctx)
{
    if (!ctx) return FQ_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (guard.ok) {
        cudaDeviceSynchronize();
        if (ctx->ws) cudaFree(ctx->ws);
        if (ctx->status_dev) cudaFree(ctx->status_dev);
        if (ctx->stack_dev) cudaFree(ctx->stack_dev);
        for (int i = 0; i < 2; i++) {
            if (ctx->stage_host[i]) cudaFreeHost(ctx->stage_host[i]);
            if (ctx->stage_done[i]) cudaEventDestroy(ctx->stage_done[i]);
        }
        if (ctx->gemm_ws) cudaFree(ctx->gemm_ws);
        if (ctx->fused_ws) cudaFree(ctx->fused_ws);
        for (void* p : ctx->owned) cudaFree(p);
        for (Layer& L : ctx->layers)
            for (Variant& v : L.var)
                if (v.swap_owned && v.store) cudaFree(v.store);
    }
    delete ctx;
    return FQ_OK;
}

size_t fq_store_bytes(int n_out, int k_in, int bits, int fmt)
{
    if (n_out < 1 || k_in < 1 || k_in % kGroup != 0) return 0;
    if (fmt == FQ_FMT_PLANES) { if (bits != 8) return 0; }
    else if (fmt == FQ_FMT_PACKED) { if (bits < 2 || bits > 8) return 0; }
    else return 0;
    return (size_t)store_bytes(n_out, k_in, bits);
}

size_t fq_code_bytes(int n_out, int k_in, int bits)
{
    if (n_out < 1 || k_in < 1 || k_in % kGroup != 0 || bits < 2 || bits > 8) return 0;
    return (size_t)n_out * (size_t)k_in * (size_t)bits / 8u;
}

size_t fq_meta_bytes(int n_out, int k_in, int group)
{
    if (n_out < 1 || k_in < 1 || group != kGroup || k_in % kGroup != 0) return 0;
    return (size_t)n_out * (size_t)(k_in / kGroup) * 4u;
}

int fq_stream_read(fq_ctx* ctx, const void* src_dev, size_t bytes, void* stream)
{
    if (!ctx || !src_dev || bytes < 16) return FQ_ERR_ARG;
    if (!aligned(src_dev, 16)) return FQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    return launch_stream_read(src_dev, bytes, reinterpret_cast<unsigned*>(ctx->ws + 8 * 4096 + 32), ctx->sm_count, (cudaStream_t)stream);
}

int fq_set_wait_limit_ns(fq_ctx* ctx, unsigned long long ns)
{
    if (!ctx) return FQ_ERR_ARG;
    ctx->wait_limit_ns = ns ? ns : 2000000000ull;
    return FQ_OK;
}

int fq_quantize_layer(const float* w_dev, int n_out, int k_in, int bits, int group,
                      uint8_t* codes_dev, uint16_t* scales_dev, uint16_t* zeros_dev, void* stream)
{
    if (!w_dev || !codes_dev || !scales_dev || !zeros_dev) return FQ_ERR_ARG;
    if (bits < 2 || bits > 8) return FQ_ERR_BITS;
    if (group != kGroup || n_out < 1 || k_in < 1 || k_in % kGroup != 0) return FQ_ERR_SHAPE;
    if (!aligned(w_dev, 16) || !aligned(codes_dev, 4)) return FQ_ERR_ALIGN;
    return launch_quantize(w_dev, n_out, k_in, bits, codes_dev, scales_dev, zeros_dev, (cudaStream_t)stream);
}

int fq_pack_layer(fq_ctx* ctx, int layer, int n_out, int k_in, int bits, int group, int fmt,
                  const uint8_t* codes_dev, const uint16_t* scales_dev, const uint16_t* zeros_dev,
                  void* store_out_dev, void* stream)
{
    if (!ctx || !codes_dev || !scales_dev || !zeros_dev || !store_out_dev) return FQ_ERR_ARG;
    if (layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    if (fmt != FQ_FMT_PACKED && fmt != FQ_FMT_PLANES) return FQ_ERR_ARG;
    if (bits < 2 || bits > 8 || (fmt == FQ_FMT_PLANES && bits != 8)) return FQ_ERR_BITS;
    if (group != kGroup || n_out < 1 || k_in < 1 || k_in % kGroup != 0) return FQ_ERR_SHAPE;
    if (!aligned(store_out_dev, 256)) return FQ_ERR_ALIGN;
    Layer& L = ctx->layers[layer];
    if (L.registered && (L.n_out != n_out || L.k_in != k_in || L.fmt != fmt)) return FQ_ERR_SHAPE;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    const FieldList fl = fmt == FQ_FMT_PLANES ? plane_fields(8) : packed_fields(bits);
    const int rc = launch_pack(codes_dev, scales_dev, zeros_dev, n_out, k_in, bits, fl, store_out_dev,
                               (cudaStream_t)stream);
    if (rc != FQ_OK) return rc;
    const bool first_variant = !L.registered;
    L.registered = true;
    L.n_out = n_out; L.k_in = k_in; L.fmt = fmt;
    Variant& v = L.var[bits];
    v.present = true; v.store = store_out_dev;
    if (L.active_bits == 0) L.active_bits = bits;
    ctx->config_epoch++;
    // the decode calls never allocate as long as a launch uses every layer at most once: the scratch for
    // that is sized here
    if (first_variant) {
        ctx->ws_reserved += layer_partial_bytes(n_out, k_in);
        const int rc2 = ensure_workspace(ctx, kPartialBase + ctx->ws_reserved + 256);
        if (rc2 != FQ_OK) return rc2;
    }
    return FQ_OK;
}

int fq_set_config(fq_ctx* ctx, const uint8_t* bits_host, int n_layers, uint64_t* footprint_bytes_host, void* stream)
{
    (void)stream;
    if (!ctx || !bits_host) return FQ_ERR_ARG;
    int registered = 0;
    for (const Layer& L : ctx->layers) registered += L.registered ? 1 : 0;
    if (n_layers != registered) return FQ_ERR_ARG;
    // validate everything first so a failing call changes nothing
    uint64_t total = 0;
    int i = 0;
    for (const Layer& L : ctx->layers) {
        if (!L.registered) continue;
        const int b = bits_host[i++];
        if (b < 2 || b > 8) return FQ_ERR_BITS;
        if (!active_variant(L, b)) return FQ_ERR_NO_VARIANT;
        total += (uint64_t)L.n_out * (uint64_t)L.k_in * (uint64_t)b / 8u;
        total += (uint64_t)L.n_out * (uint64_t)(L.k_in / kGroup) * 4u;
    }
    i = 0;
    for (Layer& L : ctx->layers)
        if (L.registered) L.active_bits = bits_host[i++];
    ctx->config_epoch++;
    if (footprint_bytes_host) *footprint_bytes_host = total;
    return FQ_OK;
}

int fq_transition(fq_ctx* ctx, const uint8_t* to_bits_host, int n_layers, int require_one_way,
                  fq_transition_report* report_host, void* stream)
{
    if (!ctx || !to_bits_host) return FQ_ERR_ARG;
    int registered = 0;
    for (const Layer& L : ctx->layers) registered += L.registered ? 1 : 0;
    if (n_layers != registered) return FQ_ERR_ARG;
    fq_transition_report rep{};
    rep.one_way = 1;
    int i = 0;
    for (const Layer& L : ctx->layers) {
        if (!L.registered) continue;
        const int b0 = L.active_bits, b1 = to_bits_host[i++];
        if (b1 < 2 || b1 > 8) return FQ_ERR_BITS;
        if (!active_variant(L, b1)) return FQ_ERR_NO_VARIANT;
        const uint64_t nk = (uint64_t)L.n_out * (uint64_t)L.k_in;
        const uint64_t meta = (uint64_t)L.n_out * (uint64_t)(L.k_in / kGroup) * 4u;
        rep.footprint_from += nk * (uint64_t)b0 / 8u + meta;
        if (b0 == b1) continue;
        rep.layers_changed++;
        if (b1 > b0) rep.one_way = 0;
        if (L.fmt == FQ_FMT_PLANES) {
            if (b1 < b0) rep.bytes_freed += nk * (uint64_t)(b0 - b1) / 8u;
            else rep.bytes_loaded += nk * (uint64_t)(b1 - b0) / 8u;
        } else {
            rep.bytes_freed += nk * (uint64_t)b0 / 8u + meta;
            rep.bytes_loaded += nk * (uint64_t)b1 / 8u + meta;
        }
    }
    if (require_one_way && !rep.one_way) return FQ_ERR_ONE_WAY;
    const int rc = fq_set_config(ctx, to_bits_host, n_layers, &rep.footprint_to, stream);
    if (rc != FQ_OK) return rc;
    if (report_host) *report_host = rep;
    return FQ_OK;
}

int fq_host_variant(fq_ctx* ctx, int layer, int n_out, int k_in, int bits, const void* store_host)
{
    if (!ctx || !store_host) return FQ_ERR_ARG;
    if (layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    if (bits < 2 || bits > 8) return FQ_ERR_BITS;
    if (n_out < 1 || k_in < 1 || k_in % kGroup != 0) return FQ_ERR_SHAPE;
    if (!aligned(store_host, 16)) return FQ_ERR_ALIGN;
    Layer& L = ctx->layers[layer];
    if (L.registered && (L.n_out != n_out || L.k_in != k_in || L.fmt != FQ_FMT_PACKED)) return FQ_ERR_SHAPE;
    if (!L.registered) {
        L.registered = true;
        L.n_out = n_out; L.k_in = k_in; L.fmt = FQ_FMT_PACKED;
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return FQ_ERR_CUDA;
        ctx->ws_reserved += layer_partial_bytes(n_out, k_in);
        const int rc = ensure_workspace(ctx, kPartialBase + ctx->ws_reserved + 256);
        if (rc != FQ_OK) return rc;
    }
    L.var[bits].host = store_host;
    return FQ_OK;
}

int fq_transition_swap(fq_ctx* ctx, const uint8_t* to_bits_host, int n_layers, int require_one_way,
                       fq_swap_report* report_host, void* stream)
{
    if (!ctx || !to_bits_host) return FQ_ERR_ARG;
    int registered = 0;
    for (const Layer& L : ctx->layers) registered += L.registered ? 1 : 0;
    if (n_layers != registered) return FQ_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    fq_swap_report rep{};
    rep.one_way = 1;
    // 1. validate everything: a failing call changes nothing
    int i = 0;
    for (const Layer& L : ctx->layers) {
        if (!L.registered) continue;
        const int b0 = L.active_bits, b1 = to_bits_host[i++];
        if (b1 < 2 || b1 > 8) return FQ_ERR_BITS;
        const Variant& v = L.fmt == FQ_FMT_PLANES ? L.var[8] : L.var[b1];
        if (!v.present && !(L.fmt == FQ_FMT_PACKED && v.host)) return FQ_ERR_NO_VARIANT;
        if (b0 != 0 && b1 > b0) rep.one_way = 0;
        const uint64_t meta = (uint64_t)L.n_out * (uint64_t)(L.k_in / kGroup) * 4u;
        if (b0 != 0) rep.footprint_from += (uint64_t)L.n_out * (uint64_t)L.k_in * (uint64_t)b0 / 8u + meta;
        rep.footprint_to += (uint64_t)L.n_out * (uint64_t)L.k_in * (uint64_t)b1 / 8u + meta;
    }
    if (require_one_way && !rep.one_way) return FQ_ERR_ONE_WAY;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    // 2. layer by layer: bring the replacement in, switch, release what it replaced (in that order: the old variant
    //    serves until the new one is resident, so the extra memory of a step is one variant at a time)
    i = 0;
    uint64_t resident_extra = 0;
    for (Layer& L : ctx->layers) {
        if (!L.registered) continue;
        const int b0 = L.active_bits, b1 = to_bits_host[i++];
        if (b0 == b1) continue;
        rep.layers_changed++;
        if (L.fmt == FQ_FMT_PLANES) {                                   // a child is a prefix of what is resident already
            L.active_bits = b1;
            continue;
        }
        Variant& nv = L.var[b1];
        const uint64_t nbytes = (uint64_t)store_bytes(L.n_out, L.k_in, b1);
        if (!nv.present) {
            void* p = nullptr;
            if (cudaMallocAsync(&p, nbytes, st) != cudaSuccess) { ctx->config_epoch++; return FQ_ERR_CUDA; }
            if (cudaMemcpyAsync(p, nv.host, nbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
                cudaFreeAsync(p, st);
                ctx->config_epoch++;
                return FQ_ERR_CUDA;
            }
            nv.store = p; nv.present = true; nv.swap_owned = true;
            rep.bytes_loaded += nbytes;
            resident_extra += nbytes;
            if (resident_extra > rep.peak_extra_bytes) rep.peak_extra_bytes = resident_extra;
        }
        L.active_bits = b1;
        if (b0 != 0) {
            Variant& ov = L.var[b0];
            if (ov.present && ov.swap_owned && ov.host) {               // can be brought back from the host copy
                const uint64_t obytes = (uint64_t)store_bytes(L.n_out, L.k_in, b0);
                if (cudaFreeAsync(ov.store, st) != cudaSuccess) { ctx->config_epoch++; return FQ_ERR_CUDA; }
                ov.store = nullptr; ov.present = false; ov.swap_owned = false;
                rep.bytes_freed += obytes;
                resident_extra = resident_extra > obytes ? resident_extra - obytes : 0;
            }
        }
    }
    ctx->config_epoch++;
    for (const Layer& L : ctx->layers)
        for (int b = 2; b <= 8; b++)
            if (L.registered && L.var[b].present && L.var[b].swap_owned) rep.resident_bytes += (uint64_t)store_bytes(L.n_out, L.k_in, b);
    if (report_host) *report_host = rep;
    return FQ_OK;
}

namespace {
const char kFileMagic[8] = {'F', 'L', 'E', 'X', 'Q', '1', 0, 0};
constexpr size_t kIoChunk = 32u << 20;            // device <-> file staging, bytes per copy
struct FileCloser { FILE* f; ~FileCloser() { if (f) std::fclose(f); } };
size_t variant_store_bytes(const Layer& L, int b) { return (size_t)store_bytes(L.n_out, L.k_in, b); }
}  // namespace

int fq_save(fq_ctx* ctx, const char* path, uint64_t* bytes_written_host)
{
    if (!ctx || !path) return FQ_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    FQ_CUDA_OK(cudaDeviceSynchronize());
    FileCloser fc{std::fopen(path, "wb")};
    if (!fc.f) return FQ_ERR_IO;
    std::vector<char> stage(kIoChunk);
    uint64_t written = 0;
    auto put = [&](const void* p, size_t n) { if (std::fwrite(p, 1, n, fc.f) != n) return false; written += n; return true; };
    const uint32_t head[2] = {(uint32_t)ctx->layers.size(), 0u};
    if (!put(kFileMagic, 8) || !put(head, 8)) return FQ_ERR_IO;
    for (const Layer& L : ctx->layers) {
        uint32_t mask = 0;
        for (int b = 2; b <= 8; b++) if (L.var[b].present) mask |= 1u << b;
        const uint32_t rec[6] = {L.registered ? 1u : 0u, (uint32_t)L.n_out, (uint32_t)L.k_in, (uint32_t)L.fmt,
                                 (uint32_t)L.active_bits, mask};
        if (!put(rec, sizeof rec)) return FQ_ERR_IO;
        for (int b = 2; b <= 8; b++) {
            if (!L.var[b].present) continue;
            const uint64_t bytes = variant_store_bytes(L, b);
            if (!put(&bytes, 8)) return FQ_ERR_IO;
            for (uint64_t off = 0; off < bytes; off += kIoChunk) {
                const size_t n = (size_t)(bytes - off < kIoChunk ? bytes - off : kIoChunk);
                FQ_CUDA_OK(cudaMemcpy(stage.data(), static_cast<const char*>(L.var[b].store) + off, n, cudaMemcpyDeviceToHost));
                if (!put(stage.data(), n)) return FQ_ERR_IO;
            }
        }
    }
    if (std::fflush(fc.f) != 0) return FQ_ERR_IO;
    if (bytes_written_host) *bytes_written_host = written;
    return FQ_OK;
}

int fq_load(fq_ctx* ctx, const char* path)
{
    if (!ctx || !path) return FQ_ERR_ARG;
    for (const Layer& L : ctx->layers) if (L.registered) return FQ_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    FileCloser fc{std::fopen(path, "rb")};
    if (!fc.f) return FQ_ERR_IO;
    auto get = [&](void* p, size_t n) { return std::fread(p, 1, n, fc.f) == n; };
    char magic[8];
    uint32_t head[2];
    if (!get(magic, 8) || std::memcmp(magic, kFileMagic, 8) != 0 || !get(head, 8)) return FQ_ERR_IO;
    if (head[0] > ctx->layers.size()) return FQ_ERR_ARG;
    std::vector<char> stage(kIoChunk);
    std::vector<Layer> loaded(head[0]);
    std::vector<void*> bufs;
    int rc = FQ_OK;
    for (uint32_t i = 0; i < head[0] && rc == FQ_OK; i++) {
        uint32_t rec[6];
        if (!get(rec, sizeof rec)) { rc = FQ_ERR_IO; break; }
        Layer& L = loaded[i];
        L.registered = rec[0] != 0;
        L.n_out = (int)rec[1]; L.k_in = (int)rec[2]; L.fmt = (int)rec[3]; L.active_bits = (int)rec[4];
        if (!L.registered) { if (rec[5] != 0) rc = FQ_ERR_IO; continue; }
        const bool planes = L.fmt == FQ_FMT_PLANES;
        const uint32_t mask = rec[5];
        const bool shape_ok = (L.fmt == FQ_FMT_PACKED || planes) && L.n_out >= 1 && L.k_in >= 1 && L.k_in % kGroup == 0;
        const bool mask_ok = mask != 0 && (mask & ~0x1FCu) == 0 && (!planes || mask == (1u << 8));
        const bool active_ok = L.active_bits >= 2 && L.active_bits <= 8 && (planes || (mask & (1u << L.active_bits)));
        if (!shape_ok || !mask_ok || !active_ok) { rc = FQ_ERR_IO; break; }
        for (int b = 2; b <= 8 && rc == FQ_OK; b++) {
            if (!(rec[5] & (1u << b))) continue;
            uint64_t bytes = 0;
            if (!get(&bytes, 8) || bytes != variant_store_bytes(L, b)) { rc = FQ_ERR_IO; break; }
            void* dev = nullptr;
            if (cudaMalloc(&dev, (size_t)bytes) != cudaSuccess) { rc = FQ_ERR_CUDA; break; }
            bufs.push_back(dev);
            for (uint64_t off = 0; off < bytes && rc == FQ_OK; off += kIoChunk) {
                const size_t n = (size_t)(bytes - off < kIoChunk ? bytes - off : kIoChunk);
                if (!get(stage.data(), n)) rc = FQ_ERR_IO;
                else if (cudaMemcpy(static_cast<char*>(dev) + off, stage.data(), n, cudaMemcpyHostToDevice) != cudaSuccess) rc = FQ_ERR_CUDA;
            }
            L.var[b].present = true;
            L.var[b].store = dev;
        }
    }
    if (rc != FQ_OK) {                                   // a failing call changes nothing
        for (void* p : bufs) cudaFree(p);
        return rc;
    }
    for (uint32_t i = 0; i < head[0]; i++) ctx->layers[i] = loaded[i];
    ctx->owned.insert(ctx->owned.end(), bufs.begin(), bufs.end());
    ctx->config_epoch++;
    ctx->stack_valid = false;
    return FQ_OK;
}

uint64_t fq_storage_bytes(const fq_ctx* ctx)
{
    if (!ctx) return 0;
    uint64_t total = 0;
    for (const Layer& L : ctx->layers) {
        if (!L.registered) continue;
        const uint64_t meta = (uint64_t)L.n_out * (uint64_t)(L.k_in / kGroup) * 4u;
        for (int b = 2; b <= 8; b++)
            if (L.var[b].present) total += (uint64_t)L.n_out * (uint64_t)L.k_in * (uint64_t)b / 8u + meta;
    }
    return total;
}

int fq_active_bits(const fq_ctx* ctx, int layer)
{
    if (!ctx || layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    const Layer& L = ctx->layers[layer];
    if (!L.registered) return FQ_ERR_NOT_PACKED;
    return L.active_bits;
}

int fq_status(fq_ctx* ctx)
{
    if (!ctx) return FQ_ERR_ARG;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    FQ_CUDA_OK(cudaDeviceSynchronize());
    int st = 0;
    FQ_CUDA_OK(cudaMemcpy(&st, ctx->status_dev, sizeof st, cudaMemcpyDeviceToHost));
    if (st != 0) {
        // counters may have been left half-way: start from a clean workspace
        FQ_CUDA_OK(cudaMemset(ctx->status_dev, 0, sizeof(int)));
        FQ_CUDA_OK(cudaMemset(ctx->ws, 0, ctx->ws_bytes));
        FQ_CUDA_OK(cudaDeviceSynchronize());
    }
    return st;
}

int fq_gemv_batched(fq_ctx* ctx, int layer, const uint16_t* x_dev, int batch, uint16_t* y_dev, void* stream)
{
    if (!ctx) return FQ_ERR_ARG;
    GemvOp op;
    if (layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    const bool one = batch == 1 && ctx->layers[layer].k_in <= gemv1_max_k();     // else the batch kernel (any K)
    int rc = fill_op(ctx, layer, x_dev, y_dev, batch, one, op);
    if (rc != FQ_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    const size_t pb = op_partial_bytes(op, one, batch);
    rc = ensure_workspace(ctx, kPartialBase + pb + 256);
    if (rc != FQ_OK) return rc;
    op.partial = reinterpret_cast<unsigned long long*>(ctx->ws + kPartialBase);
    return one ? launch_gemv1_single(ctx, op, (cudaStream_t)stream) : launch_gemv_single(ctx, op, (cudaStream_t)stream);
}

int fq_gemv(fq_ctx* ctx, int layer, const uint16_t* x_dev, uint16_t* y_dev, void* stream)
{
    return fq_gemv_batched(ctx, layer, x_dev, 1, y_dev, stream);
}

int fq_gemv_static(fq_ctx* ctx, int layer, const uint16_t* x_dev, uint16_t* y_dev, void* stream)
{
    if (!ctx) return FQ_ERR_ARG;
    GemvOp op;
    const int rc = fill_op(ctx, layer, x_dev, y_dev, 1, true, op);
    if (rc != FQ_OK) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    return launch_gemv_static(ctx, op, op_partial_bytes(op, true, 1), (cudaStream_t)stream);
}

// Relative cost of a byte, x64, per variant (0..6 packed 2..8 bits, 7..13 nested 2..8 bits).
static unsigned deal_weight(int variant)
{
    static const unsigned w[kVariants] = {125, 112, 66, 78, 78, 84, 48,      // packed 2..8
                                          108, 64, 64, 74, 74, 64, 64};      // nested 2..8 (per byte READ: whole 2-bit fields)
    return variant >= 0 && variant < kVariants ? w[variant] : 64u;
}

// Time a CTA spends on one blob of an op, in arbitrary units: bytes x the relative cost of a byte of the op's
// variant.  The 8-bit and 4-bit loops keep up with the CTA's share of HBM; variants with more fields per stored
// bit are bound by the integer pipe and take longer per byte (per-CTA rates of uniform stacks, all CTAs busy:
// 8 bits 48.8 GB/s, 4: 46.1, 5: 42.8, 6: 42.5, 7: 39.9, 3: 31.5, 2: 27.7; nested children 21 - 37 by field count).  The table
// starts from the inverse rates; the 8-bit entry is lower than that because a CTA that streams 8-bit blobs speeds
// up when its neighbours are compute-bound and leave it more of the HBM (tuned on the mixed 7B stack: the
// unordered pass went from 4350 to 5380 GB/s, the ordered one from 1.525 to 1.465 ms).
static unsigned long long blob_cost(const GemvOp& op)
{
    return (unsigned long long)(unsigned)op.blob_read * deal_weight(op.variant);
}

int fq_gemv_stack(fq_ctx* ctx, int n_ops, const int* layers_host, const uint16_t* const* x_dev_host,
                  uint16_t* const* y_dev_host, const int* phases_host, int batch, void* stream)
{
    if (!ctx || !layers_host || !x_dev_host || !y_dev_host || n_ops < 1) return FQ_ERR_ARG;
    if (batch < 1 || batch > FQ_MAX_BATCH) return FQ_ERR_SHAPE;
    // the batch-1 kernel keeps a strip's activations in shared memory: a list with a wider layer runs in the batch kernel
    bool one = batch == 1;
    for (int i = 0; i < n_ops && one; i++) {
        if (layers_host[i] < 0 || layers_host[i] >= (int)ctx->layers.size()) return FQ_ERR_ARG;
        if (ctx->layers[layers_host[i]].k_in > gemv1_max_k()) one = false;
    }
    int n_phases = 0;
    if (phases_host) {
        if (phases_host[0] != 0) return FQ_ERR_ARG;
        for (int i = 1; i < n_ops; i++)
            if (phases_host[i] < phases_host[i - 1] || phases_host[i] > phases_host[i - 1] + 1) return FQ_ERR_ARG;
        n_phases = phases_host[n_ops - 1] + 1;
        if (n_phases > (one ? gemv1_max_phases() : kMaxPhases)) return FQ_ERR_SHAPE;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    const cudaStream_t st = (cudaStream_t)stream;

    // The op table only depends on the arguments and the active configuration: the uploaded copy is
    // reused when every argument word is the same as in the call that built it.
    std::vector<uint64_t> sig;
    sig.reserve(4 + 4 * (size_t)n_ops);
    sig.push_back((uint64_t)n_ops); sig.push_back(ctx->config_epoch); sig.push_back((uint64_t)batch);
    sig.push_back(phases_host ? 1u : 0u);
    for (int i = 0; i < n_ops; i++) {
        sig.push_back((uint64_t)(int64_t)layers_host[i]);
        sig.push_back((uint64_t)reinterpret_cast<uintptr_t>(x_dev_host[i]));
        sig.push_back((uint64_t)reinterpret_cast<uintptr_t>(y_dev_host[i]));
        sig.push_back(phases_host ? (uint64_t)(int64_t)phases_host[i] : 0u);
    }
    const int np = n_phases > 0 ? n_phases : 1;
    // batch 1:    [GemvOp x n_ops][int phase_total x np][uint2 strips x sm_count x n_ops]
    // batch 2..8: [GemvOp x n_ops][long long phase_total x np][int cta_units x sm_count]
    const size_t range_off = (size_t)round_up((int64_t)((size_t)n_ops * sizeof(GemvOp) + (size_t)np * sizeof(int)), 8);
    const size_t table_bytes = one ? range_off + (size_t)ctx->sm_count * n_ops * sizeof(uint2)
                                          : (size_t)n_ops * sizeof(GemvOp) + (size_t)np * sizeof(long long) +
                                                (size_t)ctx->sm_count * sizeof(int);
    if (one && n_ops > gemv1_max_ops()) return FQ_ERR_SHAPE;

    if (!(ctx->stack_valid && ctx->stack_sig == sig)) {
        ctx->stack_valid = false;                           // until the new table is complete
        // staging buffer: the two take turns; wait for the upload that last read this one
        const int sb = ctx->stage_next;
        if (ctx->stage_done[sb]) FQ_CUDA_OK(cudaEventSynchronize(ctx->stage_done[sb]));
        else FQ_CUDA_OK(cudaEventCreateWithFlags(&ctx->stage_done[sb], cudaEventDisableTiming));
        if (ctx->stage_host_bytes[sb] < table_bytes) {
            if (ctx->stage_host[sb]) cudaFreeHost(ctx->stage_host[sb]);
            ctx->stage_host[sb] = nullptr; ctx->stage_host_bytes[sb] = 0;
            FQ_CUDA_OK(cudaMallocHost(&ctx->stage_host[sb], 2 * table_bytes));
            ctx->stage_host_bytes[sb] = 2 * table_bytes;
        }
        char* host = ctx->stage_host[sb];
        GemvOp* ops = reinterpret_cast<GemvOp*>(host);
        size_t ws_need = kPartialBase;
        long long unit_base = 0;
        std::vector<long long> bases(n_ops);
        for (int i = 0; i < n_ops; i++) {
            const int rc = fill_op(ctx, layers_host[i], x_dev_host[i], y_dev_host[i], batch, one, ops[i]);
            if (rc != FQ_OK) return rc;
            ops[i].phase = phases_host ? phases_host[i] : -1;
            bases[i] = unit_base;
            unit_base += ops[i].n_units;
            ws_need += (size_t)round_up((int64_t)op_partial_bytes(ops[i], one, batch), 256);
        }
        const int rc = ensure_workspace(ctx, ws_need + 256);   // (no allocation when every layer appears once)
        if (rc != FQ_OK) return rc;
        size_t poff = kPartialBase;
        for (int i = 0; i < n_ops; i++) {
            ops[i].partial = reinterpret_cast<unsigned long long*>(ctx->ws + poff);
            poff += (size_t)round_up((int64_t)op_partial_bytes(ops[i], one, batch), 256);
        }
        const int grid = (int)(unit_base < ctx->sm_count ? unit_base : ctx->sm_count);
        for (int i = 0; i < n_ops; i++) ops[i].rot = (int)(bases[i] % (grid > 0 ? grid : 1));
        if (one) {
            // per phase: CTAs that finish at least one strip (each reports once when its strips are done)
            int* phase_total = reinterpret_cast<int*>(host + (size_t)n_ops * sizeof(GemvOp));
            for (int p = 0; p < np; p++) phase_total[p] = 0;
            // ... and for every (CTA, op) the strips the CTA computes.  The ops of one dependency phase (of the
            // whole list when there are no phases) are dealt together: their blobs form one sequence, op
            // after op, and every CTA gets the same amount of WORK of it in one contiguous piece (bytes weighted by
            // what a byte of the op's variant costs a CTA, blob_cost()).  A CTA then touches one or two ops of a
            // phase instead of all of them: fewer activation vectors to convert, fewer strips shared with a
            // neighbour.
            uint2* ranges = reinterpret_cast<uint2*>(host + range_off);
            std::vector<int> last_phase(grid, -1);
            for (int g0 = 0, group = 0; g0 < n_ops; group++) {
                int g1 = g0 + 1;
                while (g1 < n_ops && (!phases_host || phases_host[g1] == phases_host[g0])) g1++;
                unsigned long long total = 0;
                long long strips = 0;
                for (int i = g0; i < g1; i++) {
                    total += (unsigned long long)ops[i].n_units * blob_cost(ops[i]);
                    strips += ops[i].n_rp;
                }
                long long group_blobs = 0;
                for (int i = g0; i < g1; i++) group_blobs += ops[i].n_units;
                for (int i = g0; i < g1; i++)
                    ops[i].split = (ops[i].n_fields > kSplitAboveFields && group_blobs < (long long)kSplitBelowBlobsPerCta * grid) ? 2 : 1;
                // A group with few strips per CTA is dealt in whole strips: such a phase is short, and what
                // counts is that no CTA has to wait for a neighbour's share of a strip, not the last few
                // per cent of balance.
                const bool whole_strips = phases_host && strips < 2ll * grid;
                const int rot = (int)((unsigned)group * 53u % (unsigned)grid);      // spreads the remainders
                unsigned long long before = 0;
                for (int i = g0; i < g1; i++) {
                    const unsigned long long sz = blob_cost(ops[i]);
                    const unsigned long long bytes = (unsigned long long)ops[i].n_units * sz;
                    const unsigned long long strip_bytes = (unsigned long long)ops[i].n_kb * sz;
                    for (int c = 0; c < grid; c++) {
                        const unsigned long long cc = (unsigned)((c + grid - rot) % grid);
                        // blobs of this op whose first byte lies in [cut(cc), cut(cc + 1))
                        auto first_blob_at = [&](unsigned long long pos) -> long long {
                            if (pos <= before) return 0;
                            if (pos >= before + bytes) return ops[i].n_units;
                            if (whole_strips) return (long long)((pos - before + strip_bytes - 1) / strip_bytes) * ops[i].n_kb;
                            return (long long)((pos - before + sz - 1) / sz);
                        };
                        CtaWork w;
                        w.lo = (int)first_blob_at(total * cc / (unsigned)grid);
                        w.hi = (int)first_blob_at(total * (cc + 1) / (unsigned)grid);
                        w.rp_first = w.lo / ops[i].n_kb;
                        w.rp_last = w.hi > w.lo ? (w.hi - 1) / ops[i].n_kb : w.rp_first;
                        ranges[(size_t)c * n_ops + i] = gemv1_pack_range(w, ops[i].n_kb);
                        if (phases_host && w.finishing(ops[i].n_kb) > 0 && last_phase[c] != phases_host[i]) {
                            last_phase[c] = phases_host[i];
                            phase_total[phases_host[i]]++;
                        }
                    }
                    before += bytes;
                }
                g0 = g1;
            }
        } else {
            long long* phase_total = reinterpret_cast<long long*>(host + (size_t)n_ops * sizeof(GemvOp));
            for (int p = 0; p < np; p++) phase_total[p] = 0;
            if (phases_host)
                for (int i = 0; i < n_ops; i++) phase_total[phases_host[i]] += ops[i].n_rp;   // one finished row pair = one count
            // how many units each CTA of the persistent grid will see (the consumers' loop bound)
            int* cta_units = reinterpret_cast<int*>(phase_total + np);
            for (int c = 0; c < ctx->sm_count; c++) cta_units[c] = 0;
            for (int i = 0; i < n_ops; i++)
                for (int c = 0; c < grid; c++) {
                    int lo, hi;
                    gemv_cta_range(ops[i].n_units, ops[i].rot, c, grid, lo, hi);
                    cta_units[c] += hi - lo;
                }
        }
        if (ctx->stack_dev_bytes < table_bytes) {
            FQ_CUDA_OK(cudaDeviceSynchronize());
            if (ctx->stack_dev) cudaFree(ctx->stack_dev);
            ctx->stack_dev = nullptr; ctx->stack_dev_bytes = 0;
            FQ_CUDA_OK(cudaMalloc(&ctx->stack_dev, 2 * table_bytes));
            ctx->stack_dev_bytes = 2 * table_bytes;
        }
        FQ_CUDA_OK(cudaMemcpyAsync(ctx->stack_dev, host, table_bytes, cudaMemcpyHostToDevice, st));
        FQ_CUDA_OK(cudaEventRecord(ctx->stage_done[sb], st));
        ctx->stage_next = sb ^ 1;
        ctx->stack_hdr.n_ops = n_ops; ctx->stack_hdr.n_phases = n_phases; ctx->stack_hdr.total_units = unit_base;
        ctx->stack_sig.swap(sig);
        ctx->stack_valid = true;
    }
    return one ? launch_gemv1_stack(ctx, ctx->stack_hdr, ctx->stack_dev, st)
                      : launch_gemv_stack(ctx, ctx->stack_hdr, ctx->stack_dev, batch, st);
}

static int gemm_common(fq_ctx* ctx, int layer, const uint16_t* X_dev, int M, int ldx, uint16_t* Y_dev, int ldy, void* stream,
                       bool fused)
{
    if (!ctx || !X_dev || !Y_dev) return FQ_ERR_ARG;
    if (layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    const Layer& L = ctx->layers[layer];
    if (!L.registered || L.active_bits == 0) return FQ_ERR_NOT_PACKED;
    if (M < 1 || M > (1 << 20) || ldx < L.k_in || ldy < L.n_out || ldx % 8 != 0 || ldy % 8 != 0) return FQ_ERR_SHAPE;
    if (!aligned(X_dev, 16) || !aligned(Y_dev, 16)) return FQ_ERR_ALIGN;
    const int bits = L.active_bits;
    const Variant* v = active_variant(L, bits);
    if (!v) return FQ_ERR_NO_VARIANT;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    const int zero_adjust = (L.fmt == FQ_FMT_PLANES && bits < 8) ? (1 << (7 - bits)) : 0;
    const int stride = blob_bytes(L.fmt == FQ_FMT_PLANES ? 8 : bits);
    if (fused) {
        float* parts = nullptr;
        unsigned* flags = nullptr;
        if (gemm_fused_wants_balance(M, L.n_out, ctx->sm_count)) {
            // partial-sum slots of the tiles that two CTAs share: [flags 4 x (SMs + 1), padded][slot x (SMs + 1)];
            // allocated the first time a shape asks for balanced runs
            const size_t flag_bytes = (size_t)round_up((int64_t)((ctx->sm_count + 1) * 4 * sizeof(unsigned)), 256);
            if (!ctx->fused_ws) {
                const size_t bytes = flag_bytes + (size_t)(ctx->sm_count + 1) * gemm_fused_part_bytes();
                FQ_CUDA_OK(cudaMalloc(&ctx->fused_ws, bytes));
                FQ_CUDA_OK(cudaMemset(ctx->fused_ws, 0, flag_bytes));
                ctx->fused_epoch = 0;
            }
            if (++ctx->fused_epoch == 0) ctx->fused_epoch = 1;               // (0 is the cleared flag)
            flags = reinterpret_cast<unsigned*>(ctx->fused_ws);
            parts = reinterpret_cast<float*>(ctx->fused_ws + flag_bytes);
        }
        return launch_gemm_fused(ctx, v->store, stride, active_fields(L, bits), zero_adjust, L.n_out, L.k_in, X_dev, M, ldx,
                                 Y_dev, ldy, parts, flags, ctx->fused_epoch, (cudaStream_t)stream);
    }
    const size_t need = (size_t)L.n_out * L.k_in * 2;
    if (need > ctx->gemm_ws_bytes) {
        FQ_CUDA_OK(cudaDeviceSynchronize());
        if (ctx->gemm_ws) cudaFree(ctx->gemm_ws);
        ctx->gemm_ws = nullptr; ctx->gemm_ws_bytes = 0;
        FQ_CUDA_OK(cudaMalloc(&ctx->gemm_ws, need));
        ctx->gemm_ws_bytes = need;
    }
    return launch_gemm(ctx, v->store, stride, active_fields(L, bits), zero_adjust, L.n_out, L.k_in, X_dev, M, ldx, Y_dev, ldy,
                       ctx->gemm_ws, (cudaStream_t)stream);
}

int fq_gemm(fq_ctx* ctx, int layer, const uint16_t* X_dev, int M, int ldx, uint16_t* Y_dev, int ldy, void* stream)
{
    return gemm_common(ctx, layer, X_dev, M, ldx, Y_dev, ldy, stream, true);
}

int fq_gemm_two_pass(fq_ctx* ctx, int layer, const uint16_t* X_dev, int M, int ldx, uint16_t* Y_dev, int ldy, void* stream)
{
    return gemm_common(ctx, layer, X_dev, M, ldx, Y_dev, ldy, stream, false);
}

int fq_export_layer(fq_ctx* ctx, int layer, int bits, void* out_dev, void* stream)
{
    if (!ctx || !out_dev || layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    if (bits < 2 || bits > 8) return FQ_ERR_BITS;
    const Layer& L = ctx->layers[layer];
    if (!L.registered) return FQ_ERR_NOT_PACKED;
    const Variant* v = active_variant(L, bits);
    if (!v) return FQ_ERR_NO_VARIANT;
    if (!aligned(out_dev, 4)) return FQ_ERR_ALIGN;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    if (L.fmt == FQ_FMT_PLANES)
        return launch_export_planes(v->store, L.n_out, L.k_in, bits, plane_fields(bits), (uint32_t*)out_dev,
                                    (cudaStream_t)stream);
    return launch_export_packed(v->store, L.n_out, L.k_in, bits, packed_fields(bits), (uint32_t*)out_dev,
                                (cudaStream_t)stream);
}

int fq_export_meta(fq_ctx* ctx, int layer, int bits, uint16_t* scales_dev, uint16_t* zeros_dev, void* stream)
{
    if (!ctx || !scales_dev || !zeros_dev || layer < 0 || layer >= (int)ctx->layers.size()) return FQ_ERR_ARG;
    if (bits < 2 || bits > 8) return FQ_ERR_BITS;
    const Layer& L = ctx->layers[layer];
    if (!L.registered) return FQ_ERR_NOT_PACKED;
    const Variant* v = active_variant(L, bits);
    if (!v) return FQ_ERR_NO_VARIANT;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return FQ_ERR_CUDA;
    return launch_export_meta(v->store, L.n_out, L.k_in, L.fmt == FQ_FMT_PLANES ? 8 : bits, scales_dev, zeros_dev,
                              (cudaStream_t)stream);
}

}  // extern "C"

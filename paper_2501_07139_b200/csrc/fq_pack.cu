// Quantiser, packer (canonical codes -> tiled field arrays) and exporters (back to canonical).
#include <cuda_fp16.h>

#include "fq_internal.cuh"

namespace fq {

#define FQ_CUDA_OK(expr) do { if ((expr) != cudaSuccess) return FQ_ERR_CUDA; } while (0)

// ---------------------------------------------------------------------------------------
// Quantiser: one warp per (row, group); all arithmetic that decides a code runs in double.
// ---------------------------------------------------------------------------------------

// Nearest-even conversion of a non-negative finite double to fp16 bits, done on the
// integer image of the double so that there is exactly one rounding.
__device__ __forceinline__ unsigned f64_to_f16_bits_nonneg(double v)
{
    const unsigned long long u = (unsigned long long)__double_as_longlong(v);
    const int e = (int)(u >> 52) & 0x7ff;
    if (e == 0) return 0u;
    if (e == 0x7ff) return 0x7c00u;
    const int E = e - 1023;
    const unsigned long long sig = (u & 0xFFFFFFFFFFFFFull) | (1ull << 52);
    int drop = 42;                        // 53-bit significand -> 11 bits
    if (E < -14) drop += -14 - E;         // subnormal result keeps fewer bits
    if (drop > 63) return 0u;
    unsigned long long kept = sig >> drop;
    const unsigned long long lost = sig & ((1ull << drop) - 1ull);
    const unsigned long long tie = 1ull << (drop - 1);
    kept += (lost > tie) || (lost == tie && (kept & 1ull));
    if (E < -14) return (unsigned)kept;
    const unsigned long long r = ((unsigned long long)(E + 15) << 10) + kept - 1024ull;
    return r >= 0x7c00ull ? 0x7c00u : (unsigned)r;
}

__device__ __forceinline__ double f16_bits_to_f64(unsigned h)
{
    return (double)__half2float(__ushort_as_half((unsigned short)h));
}

__global__ void __launch_bounds__(256)
quantize_kernel(const float* __restrict__ w, long long n_groups_total, int bits,
                uint8_t* __restrict__ codes, uint16_t* __restrict__ scales, uint16_t* __restrict__ zeros)
{
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
    const double qmax = (double)((1 << bits) - 1);
    for (long long grp = warp; grp < n_groups_total; grp += n_warps) {
        const float4 v = reinterpret_cast<const float4*>(w + grp * kGroup)[lane];
        float mn = fminf(fminf(v.x, v.y), fminf(v.z, v.w));
        float mx = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        unsigned sb = f64_to_f16_bits_nonneg(((double)mx - (double)mn) / qmax);
        if (sb == 0u) sb = 0x0400u;
        if (sb >= 0x7c00u) sb = 0x7bffu;
        const double S = f16_bits_to_f64(sb);
        double z = rint(-(double)mn / S);
        if (!(z > 0.0)) z = 0.0;
        if (z > qmax) z = qmax;
        const float vals[4] = {v.x, v.y, v.z, v.w};
        unsigned packed = 0;
#pragma unroll
        for (int i = 0; i < 4; i++) {
            double q = rint((double)vals[i] / S) + z;
            q = q < 0.0 ? 0.0 : (q > qmax ? qmax : q);
            packed |= (unsigned)q << (8 * i);
        }
        reinterpret_cast<unsigned*>(codes + grp * kGroup)[lane] = packed;
        if (lane == 0) {
            scales[grp] = (uint16_t)sb;
            zeros[grp] = __half_as_ushort(__float2half_rn((float)z));   // an integer <= 255: exact
        }
    }
}

int current_sm_count()
{
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 132;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 132;
        cached[dev] = n;
    }
    return cached[dev];
}

int launch_quantize(const float* w, int n_out, int k_in, int bits, uint8_t* codes, uint16_t* scales,
                    uint16_t* zeros, cudaStream_t st)
{
    const long long groups = (long long)n_out * (k_in / kGroup);
    long long blocks = (groups + 7) / 8;
    if (blocks > current_sm_count() * 16) blocks = current_sm_count() * 16;
    if (blocks < 1) return FQ_OK;
    quantize_kernel<<<(unsigned)blocks, 256, 0, st>>>(w, groups, bits, codes, scales, zeros);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ---------------------------------------------------------------------------------------
// Packer: one thread per 32-bit word of the stored variant (blob layout, see fq_layout.cuh).
// ---------------------------------------------------------------------------------------
struct StoreArgs {
    const uint8_t* codes;          // pack: canonical codes, one per byte
    const uint16_t* scales;
    const uint16_t* zeros;
    uint32_t* store;               // the stored variant
    int n_out, k_in, n_kb, groups;
    int stored_bits;               // bits of the stored variant (size of its blobs)
    FieldList fl;                  // fields that are written / read
    long long total_words;
};

__global__ void __launch_bounds__(256) pack_kernel(const StoreArgs a)
{
    const int blob_words = blob_bytes(a.stored_bits) / 4;
    for (long long wi = (long long)blockIdx.x * blockDim.x + threadIdx.x; wi < a.total_words;
         wi += (long long)gridDim.x * blockDim.x) {
        const long long blob = wi / blob_words;
        const int off = (int)(wi % blob_words) * 4;               // byte offset inside the blob
        const int rp = (int)(blob / a.n_kb), kb = (int)(blob % a.n_kb);
        unsigned v = 0;
        if (off < kBlobMetaBytes) {
            // scale/zero word: [superstep][tile][row & 7][group][row >> 3]
            const int r = ((off >> 4) & 7) + 8 * ((off >> 2) & 1), grp = (off >> 3) & 1, tile = (off >> 7) & 1, ssl = off >> 8;
            const long long n = ((long long)rp * kBlobTiles + tile) * kTileRows + r;
            const int g = (kb * kBlobSteps + ssl) * 2 + grp;
            if (n < a.n_out && g < a.groups) {
                const float z = __half2float(__ushort_as_half(a.zeros[n * a.groups + g]));
                const unsigned zi = (unsigned)fminf(fmaxf(rintf(z), 0.f), 65535.f);
                v = (unsigned)a.scales[n * a.groups + g] | (zi << 16);
            }
        } else {
            int rem = off - kBlobMetaBytes, fi = 0;
            while (rem >= kBlobSteps * kBlobTiles * 512 * a.fl.width[fi]) {
                rem -= kBlobSteps * kBlobTiles * 512 * a.fl.width[fi];
                fi++;
            }
            const int f = a.fl.width[fi], sh = a.fl.shift[fi];
            const int st = rem / (f * 512), in_tile = rem % (f * 512);       // st = ssl * 2 + tile
            const int ssl = st / kBlobTiles, tile = st % kBlobTiles;
            const int chunk = in_tile >> 9, lane = (in_tile >> 4) & 31, word = (in_tile >> 2) & 3;
            const unsigned mask = (1u << f) - 1u;
            for (int q = 0; q < 32 / f; q++) {
                int r, kk, bit;
                field_owner(f, chunk, lane, word, q, r, kk, bit);
                const long long n = ((long long)rp * kBlobTiles + tile) * kTileRows + r;
                const long long k = ((long long)kb * kBlobSteps + ssl) * kStepCols + kk;
                unsigned code = 0;
                if (n < a.n_out && k < a.k_in) code = a.codes[n * a.k_in + k];
                v |= ((code >> sh) & mask) << bit;
            }
        }
        a.store[wi] = v;
    }
}

static unsigned grid_for(long long total)
{
    long long b = (total + 255) / 256;
    if (b > (long long)current_sm_count() * 32) b = (long long)current_sm_count() * 32;
    return (unsigned)(b < 1 ? 1 : b);
}

int launch_pack(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, int n_out, int k_in,
                int stored_bits, const FieldList& fl, void* store, cudaStream_t st)
{
    StoreArgs a{};
    a.codes = codes; a.scales = scales; a.zeros = zeros; a.store = (uint32_t*)store;
    a.n_out = n_out; a.k_in = k_in; a.n_kb = k_blobs(k_in); a.groups = k_in / kGroup;
    a.stored_bits = stored_bits; a.fl = fl;
    a.total_words = store_bytes(n_out, k_in, stored_bits) / 4;
    pack_kernel<<<grid_for(a.total_words), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ---------------------------------------------------------------------------------------
// Exporters: rebuild canonical bytes from the stored variant (test / reporting support).
// ---------------------------------------------------------------------------------------
struct ExportArgs {
    const uint8_t* store;
    FieldList fl;                  // fields to read (a prefix of the stored ones for a nested child)
    int n_out, k_in, n_kb, groups, stored_bits, bits;
    uint32_t* out;
    uint16_t* scales;
    uint16_t* zeros;
    long long total_words;
};

__device__ __forceinline__ const uint8_t* blob_of(const ExportArgs& a, long long n, long long k, int& tile, int& ssl)
{
    const int rt = (int)(n / kTileRows), ss = (int)(k / kStepCols);
    tile = rt % kBlobTiles;
    ssl = ss % kBlobSteps;
    return a.store + ((long long)(rt / kBlobTiles) * a.n_kb + ss / kBlobSteps) * blob_bytes(a.stored_bits);
}

// The stored code of element (n, k), assembled from the fields in a.fl (shifts as stored).
__device__ __forceinline__ unsigned stored_code(const ExportArgs& a, long long n, long long k)
{
    int tile, ssl;
    const uint8_t* blob = blob_of(a, n, k, tile, ssl);
    const int r = (int)(n % kTileRows), kk = (int)(k % kStepCols);
    unsigned code = 0;
    int prefix = 0;
    for (int fi = 0; fi < a.fl.n; fi++) {
        const int f = a.fl.width[fi];
        const FieldPos p = field_pos(f, r, kk);
        const uint32_t wv = *reinterpret_cast<const uint32_t*>(blob + blob_field_off(prefix, f, ssl, tile) + p.word_byte);
        code |= ((wv >> p.bit) & ((1u << f) - 1u)) << a.fl.shift[fi];
        prefix += f;
    }
    return code;
}

__global__ void __launch_bounds__(256) export_packed_kernel(const ExportArgs a)
{
    const long long words_per_row = (long long)a.k_in * a.bits / 32;
    for (long long wi = (long long)blockIdx.x * blockDim.x + threadIdx.x; wi < a.total_words;
         wi += (long long)gridDim.x * blockDim.x) {
        const long long n = wi / words_per_row, w = wi % words_per_row;
        unsigned v = 0;
        for (int bit = 0; bit < 32; bit++) {
            const long long pos = w * 32 + bit;
            const long long k = pos / a.bits;
            const int j = (int)(pos % a.bits);
            v |= ((stored_code(a, n, k) >> j) & 1u) << bit;
        }
        a.out[wi] = v;
    }
}

// Canonical planes of the first `bits` stored planes: out[t][n][k/32], plane t = parent bit 7-t.
__global__ void __launch_bounds__(256) export_planes_kernel(const ExportArgs a)
{
    const long long words_per_row = a.k_in / 32;
    const long long words_per_plane = words_per_row * a.n_out;
    for (long long wi = (long long)blockIdx.x * blockDim.x + threadIdx.x; wi < a.total_words;
         wi += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(wi / words_per_plane);
        const long long rem = wi % words_per_plane;
        const long long n = rem / words_per_row, w = rem % words_per_row;
        unsigned v = 0;
        for (int bit = 0; bit < 32; bit++)
            v |= ((stored_code(a, n, w * 32 + bit) >> (7 - t)) & 1u) << bit;
        a.out[wi] = v;
    }
}

__global__ void __launch_bounds__(256) export_meta_kernel(const ExportArgs a)
{
    const long long total = (long long)a.n_out * a.groups;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long n = i / a.groups;
        const int g = (int)(i % a.groups);
        int tile, ssl;
        const uint8_t* blob = blob_of(a, n, (long long)g * kGroup, tile, ssl);
        const uint32_t v = *reinterpret_cast<const uint32_t*>(blob + blob_meta_off(ssl, tile) +
                                                              blob_meta_word(g & 1, (int)(n % kTileRows)));
        a.scales[i] = (uint16_t)(v & 0xffffu);
        a.zeros[i] = __half_as_ushort(__float2half_rn((float)(v >> 16)));
    }
}

static void fill_export(ExportArgs& a, const void* store, int n_out, int k_in, int stored_bits, int bits,
                        const FieldList& fl)
{
    a.store = (const uint8_t*)store; a.fl = fl; a.n_out = n_out; a.k_in = k_in; a.n_kb = k_blobs(k_in);
    a.groups = k_in / kGroup; a.stored_bits = stored_bits; a.bits = bits;
    a.total_words = (long long)n_out * k_in * bits / 32;
}

int launch_export_packed(const void* store, int n_out, int k_in, int bits, const FieldList& fl, uint32_t* out,
                         cudaStream_t st)
{
    ExportArgs a{};
    fill_export(a, store, n_out, k_in, bits, bits, fl);
    a.out = out;
    export_packed_kernel<<<grid_for(a.total_words), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

int launch_export_planes(const void* store, int n_out, int k_in, int bits, const FieldList& fl, uint32_t* out,
                         cudaStream_t st)
{
    ExportArgs a{};
    fill_export(a, store, n_out, k_in, 8, bits, fl);
    a.out = out;
    export_planes_kernel<<<grid_for(a.total_words), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

int launch_export_meta(const void* store, int n_out, int k_in, int stored_bits, uint16_t* scales, uint16_t* zeros,
                       cudaStream_t st)
{
    ExportArgs a{};
    fill_export(a, store, n_out, k_in, stored_bits, stored_bits, FieldList{});
    a.scales = scales; a.zeros = zeros;
    export_meta_kernel<<<grid_for((long long)n_out * a.groups), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ------------------------------------------------------------------------------- streaming read (measurement)
// Reads a buffer once with 16-byte loads, four in flight per thread, and folds the words into one value per
// thread block: what a kernel that only READS memory (as the decode path does) can reach on this part.
__global__ void __launch_bounds__(512) stream_read_kernel(const uint4* __restrict__ src, long long n16, unsigned* sink)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned acc = 0u;
    for (; i + 3 * stride < n16; i += 4 * stride) {
        const uint4 a = __ldcs(src + i), b = __ldcs(src + i + stride), c = __ldcs(src + i + 2 * stride), d = __ldcs(src + i + 3 * stride);
        acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w ^ c.x ^ c.y ^ c.z ^ c.w ^ d.x ^ d.y ^ d.z ^ d.w;
    }
    for (; i < n16; i += stride) {
        const uint4 a = __ldcs(src + i);
        acc ^= a.x ^ a.y ^ a.z ^ a.w;
    }
    for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
    if ((threadIdx.x & 31) == 0 && acc == 0x9e3779b9u) atomicXor(sink, acc);      // (keeps the loads alive; practically never taken)
}

int launch_stream_read(const void* src, size_t bytes, unsigned* sink, int sm_count, cudaStream_t st)
{
    stream_read_kernel<<<sm_count * 4, 512, 0, st>>>(static_cast<const uint4*>(src), (long long)(bytes / 16), sink);
    return cudaGetLastError() == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}

}  // namespace fq

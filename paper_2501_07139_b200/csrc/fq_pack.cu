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

int launch_quantize(const float* w, int n_out, int k_in, int bits, uint8_t* codes, uint16_t* scales,
                    uint16_t* zeros, cudaStream_t st)
{
    const long long groups = (long long)n_out * (k_in / kGroup);
    long long blocks = (groups + 7) / 8;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (blocks < 1) return FQ_OK;
    quantize_kernel<<<(unsigned)blocks, 256, 0, st>>>(w, groups, bits, codes, scales, zeros);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ---------------------------------------------------------------------------------------
// Packer: one thread per 32-bit word of a field array (gathers 32/f codes).
// ---------------------------------------------------------------------------------------
struct PackArgs {
    const uint8_t* codes;
    int n_out, k_in, n_ss;
    FieldList fl;
    long long field_word_base[kMaxFields + 1];   // first word of every field array, cumulative
    uint32_t* out;
};

__global__ void __launch_bounds__(256) pack_kernel(const PackArgs a)
{
    const long long total = a.field_word_base[a.fl.n];
    for (long long wi = (long long)blockIdx.x * blockDim.x + threadIdx.x; wi < total;
         wi += (long long)gridDim.x * blockDim.x) {
        int fi = 0;
        while (wi >= a.field_word_base[fi + 1]) fi++;
        const int f = a.fl.width[fi], sh = a.fl.shift[fi];
        const long long local = wi - a.field_word_base[fi];
        const int words_per_tile = f * 128;                    // f chunks * 32 lanes * 4 words
        const long long tile = local / words_per_tile;
        const int in_tile = (int)(local % words_per_tile);
        const int chunk = in_tile >> 7, lane = (in_tile >> 2) & 31, word = in_tile & 3;
        const int rt = (int)(tile / a.n_ss), ss = (int)(tile % a.n_ss);
        const unsigned mask = (1u << f) - 1u;
        unsigned v = 0;
        for (int q = 0; q < 32 / f; q++) {
            int r, kk, bit;
            field_owner(f, chunk, lane, word, q, r, kk, bit);
            const long long n = (long long)rt * kTileRows + r;
            const long long k = (long long)ss * kStepCols + kk;
            unsigned code = 0;
            if (n < a.n_out && k < a.k_in) code = a.codes[n * a.k_in + k];
            v |= ((code >> sh) & mask) << bit;
        }
        a.out[wi] = v;
    }
}

// Metadata: [row_tile][group (padded to 2 per superstep)][16 rows] words (scale | zero << 16).
__global__ void __launch_bounds__(256)
pack_meta_kernel(const uint16_t* __restrict__ scales, const uint16_t* __restrict__ zeros, int n_out, int groups,
                 int groups_padded, long long total, uint32_t* __restrict__ out)
{
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(i & 15);
        const long long tg = i >> 4;
        const int g = (int)(tg % groups_padded);
        const long long n = (tg / groups_padded) * kTileRows + r;
        uint32_t v = 0;
        if (n < n_out && g < groups) v = (uint32_t)scales[n * groups + g] | ((uint32_t)zeros[n * groups + g] << 16);
        out[i] = v;
    }
}

static unsigned grid_for(long long total)
{
    long long b = (total + 255) / 256;
    if (b > 148 * 32) b = 148 * 32;
    return (unsigned)(b < 1 ? 1 : b);
}

int launch_pack(const uint8_t* codes, const uint16_t* scales, const uint16_t* zeros, int n_out, int k_in,
                const FieldList& fl, void* code_out, void* meta_out, cudaStream_t st)
{
    PackArgs a{};
    a.codes = codes; a.n_out = n_out; a.k_in = k_in; a.n_ss = supersteps(k_in); a.fl = fl;
    a.out = (uint32_t*)code_out;
    long long base = 0;
    for (int i = 0; i < fl.n; i++) {
        a.field_word_base[i] = base;
        base += field_bytes(n_out, k_in, fl.width[i]) / 4;
    }
    a.field_word_base[fl.n] = base;
    pack_kernel<<<grid_for(base), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    const int groups = k_in / kGroup, groups_padded = supersteps(k_in) * 2;
    const long long total = (long long)row_tiles(n_out) * groups_padded * 16;
    pack_meta_kernel<<<grid_for(total), 256, 0, st>>>(scales, zeros, n_out, groups, groups_padded, total,
                                                    (uint32_t*)meta_out);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

// ---------------------------------------------------------------------------------------
// Exporters: rebuild canonical bytes from the field arrays (test / reporting support).
// ---------------------------------------------------------------------------------------
struct ExportArgs {
    const uint8_t* field_ptr[kMaxFields];
    FieldList fl;
    int n_out, k_in, n_ss, bits;
    uint32_t* out;
    long long total_words;
};

// Bits [lo_shift .. ] of the stored code of element (n, k), assembled from the field arrays.
__device__ __forceinline__ unsigned stored_code(const ExportArgs& a, long long n, long long k)
{
    const int rt = (int)(n / kTileRows), r = (int)(n % kTileRows);
    const int ss = (int)(k / kStepCols), kk = (int)(k % kStepCols);
    unsigned code = 0;
    for (int fi = 0; fi < a.fl.n; fi++) {
        const int f = a.fl.width[fi];
        const FieldPos p = field_pos(f, r, kk);
        const long long tile = (long long)rt * a.n_ss + ss;
        const uint32_t wv = *reinterpret_cast<const uint32_t*>(a.field_ptr[fi] + tile * (f * 512) + p.word_byte);
        code |= ((wv >> p.bit) & ((1u << f) - 1u)) << a.fl.shift[fi];
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

static void fill_export(ExportArgs& a, const void* codes, int n_out, int k_in, int bits, const FieldList& fl,
                        uint32_t* out)
{
    a.fl = fl; a.n_out = n_out; a.k_in = k_in; a.n_ss = supersteps(k_in); a.bits = bits; a.out = out;
    const uint8_t* p = (const uint8_t*)codes;
    for (int i = 0; i < fl.n; i++) {
        a.field_ptr[i] = p;
        p += field_bytes(n_out, k_in, fl.width[i]);
    }
    a.total_words = (long long)n_out * k_in * bits / 32;
}

int launch_export_packed(const void* codes, int n_out, int k_in, int bits, const FieldList& fl, uint32_t* out,
                         cudaStream_t st)
{
    ExportArgs a{};
    fill_export(a, codes, n_out, k_in, bits, fl, out);
    export_packed_kernel<<<grid_for(a.total_words), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

int launch_export_planes(const void* codes, int n_out, int k_in, int bits, const FieldList& fl, uint32_t* out,
                         cudaStream_t st)
{
    ExportArgs a{};
    fill_export(a, codes, n_out, k_in, bits, fl, out);
    export_planes_kernel<<<grid_for(a.total_words), 256, 0, st>>>(a);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

__global__ void __launch_bounds__(256)
export_meta_kernel(const uint32_t* __restrict__ meta, int n_out, int groups, int groups_padded,
                   uint16_t* __restrict__ scales, uint16_t* __restrict__ zeros)
{
    const long long total = (long long)n_out * groups;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long n = i / groups;
        const int g = (int)(i % groups);
        const uint32_t v = meta[((n / kTileRows) * groups_padded + g) * 16 + (n % kTileRows)];
        scales[i] = (uint16_t)(v & 0xffffu);
        zeros[i] = (uint16_t)(v >> 16);
    }
}

int launch_export_meta(const void* meta, int n_out, int k_in, uint16_t* scales, uint16_t* zeros, cudaStream_t st)
{
    const int groups = k_in / kGroup;
    export_meta_kernel<<<grid_for((long long)n_out * groups), 256, 0, st>>>(
        (const uint32_t*)meta, n_out, groups, supersteps(k_in) * 2, scales, zeros);
    FQ_CUDA_OK(cudaGetLastError());
    return FQ_OK;
}

}  // namespace fq

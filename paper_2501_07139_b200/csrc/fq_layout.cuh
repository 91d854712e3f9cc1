// Device layout of stored codes and scale/zero metadata.
//
// A stored variant is a list of FIELD ARRAYS, most significant field first.  A field is
// f in {8,4,2,1} consecutive bits of every code, (code >> shift) & (2^f - 1):
//   PACKED b bits : the binary decomposition of b   (7 -> 4,2,1;  5 -> 4,1;  3 -> 2,1 ...)
//   PLANES parent : a 2-bit top field (bits 7,6) followed by six 1-bit planes (5 .. 0),
//                   so a b-bit child is the first b-1 arrays = the first b/8 of the bytes.
// Every array is tiled: tile = 16 rows x 256 columns ("superstep"), tiles ordered
// [row_tile][superstep], and inside a tile  [f chunks][32 lanes][16 bytes].
// The order inside a tile is the order in which a warp consumes the values as A-operand
// registers of mma.m16n8k16 (lane = 4*g + c owns rows g, g+8 and columns 32*j2 + 8*c + i):
// each 32-bit word holds 16/f "pair registers"; pair register t is the two fields at bit
// offsets t*f (low half) and 16 + t*f (high half), so one shift and one AND turn a stored
// word into a ready half2 operand whose halves hold the integers as fp16 subnormals.
//
// Metadata: [row_tile][group][16 rows] words, low half = scale, high half = zero (fp16).
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define FQ_HD __host__ __device__ __forceinline__
#else
#define FQ_HD inline
#endif

namespace fq {

constexpr int kGroup = 128;
constexpr int kTileRows = 16;
constexpr int kStepCols = 256;            // columns per superstep (two groups)
constexpr int kMaxFields = 7;

struct FieldList {
    int n;
    uint8_t width[kMaxFields];
    uint8_t shift[kMaxFields];
};

// Fields of a PACKED variant of `bits` bits (most significant first).
FQ_HD FieldList packed_fields(int bits)
{
    FieldList fl{};
    int rem = bits;
    for (int f = 8; f >= 1; f >>= 1)
        if (rem >= f) {
            rem -= f;
            fl.width[fl.n] = (uint8_t)f;
            fl.shift[fl.n] = (uint8_t)rem;
            fl.n++;
        }
    return fl;
}

// Fields of the 8-bit PLANES parent restricted to its `bits` most significant bits.
// Shifts are in parent code units.
FQ_HD FieldList plane_fields(int bits)
{
    FieldList fl{};
    fl.width[0] = 2; fl.shift[0] = 6; fl.n = 1;
    for (int p = 5; p >= 8 - bits; p--) {
        fl.width[fl.n] = 1;
        fl.shift[fl.n] = (uint8_t)p;
        fl.n++;
    }
    return fl;
}

FQ_HD int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }
FQ_HD int row_tiles(int n_out) { return (n_out + kTileRows - 1) / kTileRows; }
FQ_HD int supersteps(int k_in) { return (k_in + kStepCols - 1) / kStepCols; }

// Bytes of one field array.
FQ_HD int64_t field_bytes(int n_out, int k_in, int f)
{
    return (int64_t)row_tiles(n_out) * supersteps(k_in) * f * 512;
}

// Position of the field of element (row r in 0..15, column kk in 0..255) inside a tile of a
// field array of width f: byte offset of the 32-bit word inside the tile, and bit offset.
struct FieldPos { int word_byte; int bit; };

FQ_HD FieldPos field_pos(int f, int r, int kk)
{
    const int g = r & 7, hi_row = r >> 3;
    const int j2 = kk >> 5, c = (kk >> 3) & 3, i = kk & 7;
    const int mma = i >> 2, pair = (i >> 1) & 1, half = i & 1;
    const int reg = j2 * 8 + mma * 4 + pair * 2 + hi_row;     // 0..63: A-register of this lane in the superstep
    const int regs_per_chunk = 64 / f;
    const int regs_per_word = 16 / f;
    const int chunk = reg / regs_per_chunk;
    const int rr = reg % regs_per_chunk;
    const int word = rr / regs_per_word;
    const int t = rr % regs_per_word;
    FieldPos p;
    p.word_byte = chunk * 512 + (4 * g + c) * 16 + word * 4;
    p.bit = half * 16 + t * f;
    return p;
}

// Inverse: which (row, column) of the tile does bit field (half, t) of word `word` of lane
// `lane` of chunk `chunk` belong to.
FQ_HD void field_owner(int f, int chunk, int lane, int word, int half, int t, int& r, int& kk)
{
    const int reg = chunk * (64 / f) + word * (16 / f) + t;
    const int j2 = reg >> 3, mma = (reg >> 2) & 1, pair = (reg >> 1) & 1, hi_row = reg & 1;
    const int g = lane >> 2, c = lane & 3;
    r = g + 8 * hi_row;
    kk = j2 * 32 + c * 8 + mma * 4 + pair * 2 + half;
}

}  // namespace fq

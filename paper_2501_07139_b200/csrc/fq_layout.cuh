// Device layout of stored codes and scale/zero metadata.
//
// A stored variant is a list of FIELD ARRAYS, most significant field first.  A field is
// f in {8,4,2,1} consecutive bits of every code, (code >> shift) & (2^f - 1):
//   PACKED b bits : the binary decomposition of b   (7 -> 4,2,1;  5 -> 4,1;  3 -> 2,1 ...)
//   PLANES parent : four 2-bit fields (bits 7..6, 5..4, 3..2, 1..0), so a b-bit child is the first
//                   ceil(b / 2) arrays; a child of odd width ignores the low bit of its last field.
// Storage is cut into BLOBS: one blob = one row pair (32 rows = two 16-row tiles) x 512 columns
// (two "supersteps" of 256).  A blob holds, in this order,
//     scale/zero words   [superstep][tile][row & 7][group][row >> 3]             (512 B)
//                        (the four words that one lane of the decode kernel needs are one 16-byte load)
//     field array 0      [superstep][tile][f0 chunks][32 lanes][16 B]            (2048 * f0 B)
//     field array 1 ...                                                          (most significant first)
// and blobs are ordered [row_pair][k_blob].  Everything a decode unit needs is therefore ONE
// contiguous range for a PACKED variant (one bulk copy), and for a nested child the first
// 512 + 4096 * ceil(b / 2) bytes of every blob (one bulk copy per blob): lower fields are never touched.
// The order inside a tile is the order in which a warp consumes the values as A-operand
// registers of the 8-bit mma.m16n8k32 (lane = 4*g + c owns rows g, g+8; in k32 step j it owns
// columns 32j + 4c .. +3 and 32j + 16 + 4c .. +3).  A 32-bit word holds P = 8/f A-registers
// on top of each other: byte b of the word belongs to k-slot b, and inside every byte the
// field of register t sits at bit offset t*f.  So `word & (field_mask << t*f)` IS the A
// register of k32 step  j = P*chunk + t  (values scaled by 2^(t*f)), with no shift at all;
// the four words of a lane's 16-byte chunk are the four A registers a0..a3.
//
// Scale/zero word: low half = fp16 scale, high half = the zero point as an unsigned integer.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define FQ_HD __host__ __device__ __forceinline__
#else
#define FQ_HD inline
#endif
#define FQ_HDC constexpr FQ_HD

namespace fq {

constexpr int kGroup = 128;
constexpr int kTileRows = 16;
constexpr int kStepCols = 256;            // columns per superstep (two groups)
constexpr int kMaxFields = 7;

struct FieldList {
    int n;
    uint8_t width[kMaxFields];    // stored bits of the field
    uint8_t shift[kMaxFields];    // position of the field's lowest stored bit inside the code
    uint8_t keep[kMaxFields];     // bits of the field that count, from its top (= width, except for the last field of a
                                  // nested child of odd width, whose low bit belongs to the bits the child drops)
};

// Mask of the bits of a field of width f that count.
FQ_HDC uint32_t field_keep_mask(int f, int keep) { return ((1u << f) - 1u) & ~((1u << (f - keep)) - 1u); }

// Fields of a PACKED variant of `bits` bits (most significant first).
FQ_HDC FieldList packed_fields(int bits)
{
    FieldList fl{};
    int rem = bits;
    for (int f = 8; f >= 1; f >>= 1)
        if (rem >= f) {
            rem -= f;
            fl.width[fl.n] = (uint8_t)f;
            fl.shift[fl.n] = (uint8_t)rem;
            fl.keep[fl.n] = (uint8_t)f;
            fl.n++;
        }
    return fl;
}

// Fields of the 8-bit PLANES parent restricted to its `bits` most significant bits.  The parent is stored as four
// 2-bit fields (bits 7..6, 5..4, 3..2, 1..0), most significant first, so a child of b bits is the first ceil(b / 2)
// fields of every blob; a child of odd width uses only the upper bit of its last field.  Shifts are in parent
// code units.
FQ_HDC FieldList plane_fields(int bits)
{
    FieldList fl{};
    fl.n = (bits + 1) / 2;
    for (int i = 0; i < fl.n; i++) {
        fl.width[i] = 2;
        fl.shift[i] = (uint8_t)(6 - 2 * i);
        fl.keep[i] = 2;
    }
    if (bits & 1) fl.keep[fl.n - 1] = 1;
    return fl;
}
// Stored bits per weight that a child of `bits` bits reads (whole fields).
FQ_HDC int plane_read_bits(int bits) { return 2 * ((bits + 1) / 2); }

FQ_HD int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }
FQ_HD int row_tiles(int n_out) { return (n_out + kTileRows - 1) / kTileRows; }
FQ_HD int supersteps(int k_in) { return (k_in + kStepCols - 1) / kStepCols; }

// Decode kernels are specialised per field list.  Variant index: 0..6 = PACKED 2..8 bits, 7..13 = a
// 2..8-bit child of the PLANES parent.
constexpr int kVariants = 14;
FQ_HDC int variant_index(bool planes, int bits) { return (planes ? 7 : 0) + bits - 2; }
FQ_HDC FieldList variant_fields(int variant) { return variant < 7 ? packed_fields(variant + 2) : plane_fields(variant - 5); }

constexpr int kBlobSteps = 2;             // supersteps per blob
constexpr int kBlobTiles = 2;             // row tiles per blob (a row pair)
constexpr int kBlobMetaBytes = kBlobSteps * kBlobTiles * 128;

FQ_HD int row_pairs(int n_out) { return (row_tiles(n_out) + kBlobTiles - 1) / kBlobTiles; }
FQ_HD int k_blobs(int k_in) { return (supersteps(k_in) + kBlobSteps - 1) / kBlobSteps; }
// Bytes of a blob whose fields add up to `bits` bits (also: prefix of a nested parent's blob that a
// `bits`-bit child reads).
FQ_HD int blob_bytes(int bits) { return kBlobMetaBytes + kBlobSteps * kBlobTiles * 512 * bits; }
FQ_HD int64_t store_bytes(int n_out, int k_in, int bits) { return (int64_t)row_pairs(n_out) * k_blobs(k_in) * blob_bytes(bits); }
// Offsets inside a blob: scale/zero words of (superstep ssl, tile), and the tile of field width f
// that comes after fields adding up to prefix_bits.
FQ_HD int blob_meta_off(int ssl, int tile) { return (ssl * kBlobTiles + tile) * 128; }
// ... and inside that, the word of row r (0..15) of the tile and group grp (0..1) of the superstep
FQ_HD int blob_meta_word(int grp, int r) { return (r & 7) * 16 + grp * 8 + (r >> 3) * 4; }
FQ_HD int blob_field_off(int prefix_bits, int f, int ssl, int tile)
{
    return kBlobMetaBytes + kBlobSteps * kBlobTiles * 512 * prefix_bits + (ssl * kBlobTiles + tile) * f * 512;
}

// Position of the field of element (row r in 0..15, column kk in 0..255) inside a tile of a
// field array of width f: byte offset of the 32-bit word inside the tile, and bit offset.
struct FieldPos { int word_byte; int bit; };

FQ_HD FieldPos field_pos(int f, int r, int kk)
{
    const int P = 8 / f;                                      // A-registers stacked in one word
    const int g = r & 7, hi_row = r >> 3;
    const int j = kk >> 5, p = kk & 31;
    const int half = p >> 4, c = (p >> 2) & 3, byte = p & 3;
    const int chunk = j / P, t = j % P;
    const int areg = 2 * half + hi_row;                       // a0..a3 of the mma
    FieldPos q;
    q.word_byte = chunk * 512 + (4 * g + c) * 16 + areg * 4;
    q.bit = byte * 8 + t * f;
    return q;
}

// Inverse: field slot q (0 .. 32/f - 1; q = byte * P + t) of word `word` of lane `lane` of chunk
// `chunk` belongs to which (row, column) of the tile, and at which bit it sits.
FQ_HD void field_owner(int f, int chunk, int lane, int word, int q, int& r, int& kk, int& bit)
{
    const int P = 8 / f;
    const int byte = q / P, t = q % P;
    const int g = lane >> 2, c = lane & 3;
    const int half = word >> 1, hi_row = word & 1;
    const int j = chunk * P + t;
    r = g + 8 * hi_row;
    kk = j * 32 + half * 16 + c * 4 + byte;
    bit = byte * 8 + t * f;
}

}  // namespace fq

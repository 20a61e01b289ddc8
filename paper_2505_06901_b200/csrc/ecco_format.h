// ecco_format.h -- constants of the 64-byte block and of the device metadata image, shared by
// the host encoder and the CUDA kernels of this library (never by the test oracle).
#pragma once
#include <cstdint>

namespace ecco {

constexpr int kGroup = 128;        // values per group (Sec. 3.1)
constexpr int kBlockBytes = 64;    // bytes per block (Sec. 3.1)
constexpr int kBlockBits = 512;
constexpr int kCentroids = 15;     // Sec. 3.2
constexpr int kSymbols = 16;       // 15 centroid indices + index 15 = the abs-max
constexpr int kMaxPatterns = 64;   // S
constexpr int kCodebooks = 4;      // H
constexpr int kMinLen = 2, kMaxLen = 8;   // Sec. 4.2
constexpr int kKpMaxLen = 12;      // limit of the ID_KP code
constexpr int kPadBits = 15;       // 7-bit location + FP8 value (Sec. 3.2)
constexpr int kMaxPads = 16;       // the sorter's top 16 (Sec. 4.3)
constexpr int kHeaderBits = 10;    // scale byte + ID_HF
constexpr int kExpMin = -32, kExpMax = 16;

// Device image of the per-tensor metadata: a 64-byte header, fixed-size tables, then two sections whose size
// depends on the codebooks (DevHeader says how large they are).  What the decoders stage into shared memory is
//   [pattern | ID_KP table | codebook records]   one bulk copy, kFixedTableBytes
//   [shape tables]                                 one bulk copy, n_shapes * 256 bytes
//   [pair tables]                                  one bulk copy, pair_bytes, to an address aligned to pair_align
//
// Code shapes.  A canonical code is fixed by how many of its 16 codewords have each length; the 256 codebooks of a
// tensor share a few dozen such shapes.  The decode tables are stored per shape and work on the symbol's RANK, its
// position in (length, symbol id) order: the codeword of rank r is the same bit string in every codebook of the
// shape, and a codebook record carries the symbol -> rank nibbles, which the kernels use to lay out the lane's
// sixteen dequantised values in rank order.
//
// Shape table [256] u8, indexed by the next 8 stream bits (first stream bit in bit 0): length << 4 | rank.
// Pair table [2^W] u16 (W = 8..12 per shape), indexed by the next W stream bits: two symbols per lookup,
//   bits 0..3   length of both codewords together           (escape: length of the first)
//   bits 4..6   zero (room for the sum of two entries)
//   bits 7..10  rank of the first symbol, i.e. rank << 7 = its byte offset in a [16][32] u32 value table
//   bits 11..14 rank of the second symbol                   (escape: zero)
//   bit  15     escape: the W bits end before the second codeword does; the decoder fetches it on its own
// Shapes get table widths by expected use (from the ID_KP code lengths) and by how much a wider table lowers the
// escape rate, within kPairBudgetBytes; tables are stored widest first, so each starts at a multiple of its size.
// If even eight-bit tables for every shape do not fit, there are none (pair_bytes = 0).
constexpr uint32_t kDevMagic = 0x4F434345u;  // "ECCO"
constexpr uint32_t kDevVersion = 4;
struct DevHeader {
    uint32_t magic, version;
    int32_t S, H, e;
    float T;                 // 2^e
    uint32_t total_bytes;
    uint32_t n_shapes;       // distinct code shapes among the codebooks
    uint32_t shape_bytes;    // n_shapes * 256
    uint32_t pair_bytes;     // 0: no pair tables
    uint32_t pair_align;     // size of the widest pair table (a power of two), 0 without pair tables
    uint32_t off_pair;       // byte offset of the pair tables in the image, a multiple of 16
    uint32_t hash_lo, hash_hi;   // hash of every staged table (not of e, T): equal hashes = same tables
    uint32_t reserved[2];
};
static_assert(sizeof(DevHeader) == 64, "header is 64 bytes");

constexpr uint32_t kOffPattern = 64;                                  // [64][16] fp16, entry 15 = 0
constexpr uint32_t kPatternBytes = kMaxPatterns * 16 * 2;
constexpr uint32_t kOffKpLut = kOffPattern + kPatternBytes;           // [4096] u16: kp | len << 8
constexpr uint32_t kKpLutBytes = (1u << kKpMaxLen) * 2;
// codebook records [S*H = 256] x 16 bytes:
//   word 0: (pair-table offset >> 9) | shape << 8 | W << 16   (W = 0: the shape has no pair table)
//   word 1: zero
//   words 2, 3: rank of symbol s in bits 4s of the 64-bit pair
constexpr uint32_t kOffCbRec = kOffKpLut + kKpLutBytes;
constexpr uint32_t kCbRecBytes = kMaxPatterns * kCodebooks * 16;
constexpr uint32_t kFixedTableBytes = kPatternBytes + kKpLutBytes + kCbRecBytes;   // 14336: what every decoder stages first
// encoder tables for the device-side compressor
constexpr uint32_t kOffEncCb = kOffCbRec + kCbRecBytes;               // [256][16] u16: stream-order codeword | length << 8
constexpr uint32_t kEncCbBytes = kMaxPatterns * kCodebooks * kSymbols * 2;
constexpr uint32_t kOffEncKp = kOffEncCb + kEncCbBytes;               // [64] u16: stream-order ID_KP codeword | length << 12
constexpr uint32_t kEncKpBytes = kMaxPatterns * 2;
constexpr uint32_t kEncBytes = kEncCbBytes + kEncKpBytes;             // 8320, a multiple of 16
constexpr uint32_t kOffShapeLut = kOffEncKp + kEncKpBytes;            // [n_shapes][256] u8
constexpr uint32_t kMaxShapes = kMaxPatterns * kCodebooks;
constexpr int kPairMinBits = 8, kPairMaxBits = 12;
constexpr uint32_t kPairBudgetBytes = 80u << 10;
constexpr uint32_t kMaxDevBytes = kOffShapeLut + kMaxShapes * 256 + kPairBudgetBytes;
// Both kinds of table are indexed by the next stream bits with the first stream bit in bit 0,
// i.e. by the bit-reversed codeword followed by whatever comes next.
//
// Both are stored with a per-shape rotation: the entry for window value i sits at byte offset
// (entry size * i) ^ table_rotation(shape).  The rotation touches offset bits 2..6, which select the
// shared-memory bank, so lanes that decode with different shapes spread over different banks even when
// their windows agree (neighbouring groups often start with the same few codewords).
#ifdef __CUDACC__
#define ECCO_HD __host__ __device__
#else
#define ECCO_HD
#endif
ECCO_HD constexpr uint32_t table_rotation(uint32_t shape) { return ((shape * 11u + (shape >> 3)) & 31u) << 2; }

// Variable-length container: index = u64 total_bits | u64 chunk_base[ceil(n / 4096)] | u32 offset[n];
// group g starts at stream bit chunk_base[g >> 12] + offset[g].
constexpr int kVarChunkShift = 12;
constexpr int kVarMaxBits = kHeaderBits + kKpMaxLen + kGroup * kMaxLen;      // 1046
ECCO_HD constexpr uint64_t var_chunks(uint64_t n_groups) { return (n_groups + (1ull << kVarChunkShift) - 1) >> kVarChunkShift; }

}  // namespace ecco

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

// Device image of the per-tensor metadata.  The tables follow the 64-byte header back to back
// so that one bulk copy brings them into shared memory.
constexpr uint32_t kDevMagic = 0x4F434345u;  // "ECCO"
constexpr uint32_t kDevVersion = 3;
struct DevHeader {
    uint32_t magic, version;
    int32_t S, H, e;
    float T;                 // 2^e
    uint32_t total_bytes;
    uint32_t reserved[9];
};
static_assert(sizeof(DevHeader) == 64, "header is 64 bytes");

constexpr uint32_t kOffPattern = 64;                                  // [64][16] fp16, entry 15 = 0
constexpr uint32_t kPatternBytes = kMaxPatterns * 16 * 2;
constexpr uint32_t kOffKpLut = kOffPattern + kPatternBytes;           // [4096] u16: kp | len << 8
constexpr uint32_t kKpLutBytes = (1u << kKpMaxLen) * 2;
constexpr uint32_t kOffSymLut = kOffKpLut + kKpLutBytes;              // [S*H = 256][256] u8: len << 4 | sym
constexpr uint32_t kSymLutBytes = kMaxPatterns * kCodebooks * 256;
constexpr uint32_t kTableBytes = kOffSymLut + kSymLutBytes - kOffPattern;   // 75776: what the decoders stage, a multiple of 16
// encoder tables for the device-side compressor, after the decode tables
constexpr uint32_t kOffEncCb = kOffSymLut + kSymLutBytes;             // [256][16] u16: stream-order codeword | length << 8
constexpr uint32_t kEncCbBytes = kMaxPatterns * kCodebooks * kSymbols * 2;
constexpr uint32_t kOffEncKp = kOffEncCb + kEncCbBytes;               // [64] u16: stream-order ID_KP codeword | length << 12
constexpr uint32_t kEncKpBytes = kMaxPatterns * 2;
constexpr uint32_t kEncBytes = kEncCbBytes + kEncKpBytes;             // 8320, a multiple of 16
// Tables of the decompress kernel's mixed decoder (table lookups and arithmetic decoding of the canonical
// code take turns, so that neither the load/store pipe nor the integer pipe carries every symbol).
// Both work on the symbol's RANK, a relabelling of the 16 symbols per codebook:
//   rank(s) = (position of s in (length, id) order + rho) mod 16, rho such that an 8-bit codeword's rank is
//   its own low four bits (rho = 0 without 8-bit codewords).
// Then rank = (codeword + delta[L]) mod 16 for a codeword of length L, with delta[8] = 0.
constexpr uint32_t kOffRankLut = kOffEncKp + kEncKpBytes;             // 84160: [256][256] u8: len << 4 | rank, rotated like the symbol tables
constexpr uint32_t kRankLutBytes = kSymLutBytes;
constexpr uint32_t kOffArith = kOffRankLut + kRankLutBytes;           // [5][256] u32, one row per word, column = codebook:
constexpr int kArithWords = 5;                                        //   0, 1: addends of the length compare (see below)
constexpr uint32_t kArithBytes = kArithWords * kMaxPatterns * kCodebooks * 4;   //   2: delta[2..7], 4 bits each, delta[L] in bits 4(L-2)
constexpr uint32_t kDevBytes = kOffArith + kArithBytes;               //   3, 4: rank of symbol s in bits 4s of the 64-bit pair
// Length compare: with b = the next 8 stream bits, first bit on top, and thr[L] = the smallest b whose codeword
// is longer than L (256 if none), field i of word 0 (bits 10 i ..) holds 256 - thr[2 + i] and field i of word 1
// (bits 10 i + 1 .., one bit higher so that the two words' result bits do not meet) holds 256 - thr[5 + i],
// i = 0..2; word 0 also has bits 30 and 31 set.  b * kArithSpread + word 0 and b * 2 kArithSpread + word 1 put
// b + 256 - thr in every field, whose bit 8 says b >= thr; the codeword length is the number of set bits under
// kArithGuard | bits 30, 31 of the first and 2 kArithGuard of the second, i.e. 2 + the number of thresholds passed.
constexpr uint32_t kArithSpread = 1u | (1u << 10) | (1u << 20);
constexpr uint32_t kArithGuard = (0x100u) | (0x100u << 10) | (0x100u << 20);
// Both lookup tables are indexed by the next stream bits with the first stream bit in bit 0,
// i.e. by the bit-reversed codeword followed by whatever comes next.
//
// Symbol tables are stored with a per-codebook index rotation: the entry for window value i of
// codebook cb sits at index i ^ lut_rotation(cb).  The rotation touches index bits 2..6, which
// select the shared-memory bank of a byte entry, so lanes that decode with different codebooks
// spread over different banks even when their windows agree.
#ifdef __CUDACC__
#define ECCO_HD __host__ __device__
#else
#define ECCO_HD
#endif
ECCO_HD constexpr uint32_t lut_rotation(uint32_t cb) { return ((cb * 11u + (cb >> 3)) & 31u) << 2; }

// Variable-length container: index = u64 total_bits | u64 chunk_base[ceil(n / 4096)] | u32 offset[n];
// group g starts at stream bit chunk_base[g >> 12] + offset[g].
constexpr int kVarChunkShift = 12;
constexpr int kVarMaxBits = kHeaderBits + kKpMaxLen + kGroup * kMaxLen;      // 1046
ECCO_HD constexpr uint64_t var_chunks(uint64_t n_groups) { return (n_groups + (1ull << kVarChunkShift) - 1) >> kVarChunkShift; }

}  // namespace ecco

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
constexpr uint32_t kDevVersion = 2;
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
constexpr uint32_t kDevBytes = kOffEncKp + kEncKpBytes;               // 84160
constexpr uint32_t kEncBytes = kEncCbBytes + kEncKpBytes;             // 8320, a multiple of 16
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

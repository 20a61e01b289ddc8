// ecco_kernels.cu -- sm_100a kernels and the device half of the C ABI.
//
// One thread owns one group: a 64-byte block is independent of every other block (Sec. 3.2,
// "all group-wise information ... compressed to a fixed compressed block size"), so the decoder
// runs the serial Huffman chain (Sec. 4.2) once per thread and takes its parallelism across
// groups, not inside a group.  The lanes of a warp advance symbol by symbol in lock step, which
// keeps every per-symbol index (output position, activation element) uniform across the warp.
//
// Shared memory per CTA:
//   tables   pattern[64][16] fp16 | ID_KP table [4096] u16 | symbol tables [256][256] u8,
//            brought in by one bulk copy (cp.async.bulk + mbarrier)
//   per warp bits[18][32] u32   the warp's 32 blocks, word-transposed: lane L's word w at
//                               [w][L] -> bank L whatever w is (conflict-free refills);
//                               rows 16 and 17 stay zero (stream bits past 512 read as 0)
//            tab[16][32]  u32   per-lane dequantised centroids (entry 15 = the abs-max)
//            syms[16][32] u32   (fused kernels) decoded indices, 8 nibbles per word, for the
//                               outlier fix-up
#include <cuda.h>
#include <cuda/std/type_traits>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/ecco.h"
#include "ecco_format.h"

using namespace ecco;

namespace {

__device__ int g_device_status = 0;            // sticky: ECCO_ERR_DEVICE_TIMEOUT if a bounded wait expired
thread_local int t_last_cuda_error = 0;
std::atomic<uint64_t> g_launches{0};

constexpr uint32_t kSmemPattern = 0;
constexpr uint32_t kSmemKpLut = kPatternBytes;
constexpr uint32_t kSmemSymLut = kPatternBytes + kKpLutBytes;        // 10240: 256-aligned
constexpr uint32_t kSmemWarpBase = kTableBytes;                      // 75776: 1024-aligned
constexpr uint32_t kSmemArith = kTableBytes;                         // mixed decoder: constants after the rank tables,
constexpr uint32_t kSmemRankWarpBase = kTableBytes + kArithBytes;    // per-warp arrays after them (80896: 1024-aligned)
constexpr uint32_t kBitsRows = 18;
constexpr uint32_t kBitsBytes = kBitsRows * 32 * 4;                  // 2304
constexpr uint32_t kTabBytes = 16 * 32 * 4;                          // 2048
constexpr uint32_t kSymsBytes = 16 * 32 * 4;                         // 2048
constexpr int kFusedFree = 12;                                       // fused kernels: leading decode steps without the clip test
// Scalar fused kernels (one or two dot products per group): decode mix as in the decompress kernel, 0 = all-table.
// They issue more instructions per symbol than the decompress kernel and gain nothing from the mix (11008x4096,
// batch 1: 44.2 us all-table, 44.3 us with one symbol in four decoded arithmetically, 46.1 us with two; scores over
// the cfg-3 K cache 128.0 / 128.3 / 134.6 us), so it stays off; -DECCO_FUSED_ARITH=<mask> builds the other variants.
#ifndef ECCO_FUSED_ARITH
#define ECCO_FUSED_ARITH 0
#endif
constexpr uint32_t kFusedArith = ECCO_FUSED_ARITH;
constexpr bool kFusedRank = kFusedArith != 0;
constexpr uint32_t kFusedBase = kFusedRank ? kSmemRankWarpBase : kSmemWarpBase;
constexpr int kWaitLimit = 1 << 22;                                  // bounded mbarrier polling

// ---------------------------------------------------------------------------------------------
// small PTX helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// 1-D bulk copy global -> shared (TMA engine, no tensor map, no multicast); both addresses and
// the size are multiples of 16 bytes
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
// one 64-byte block = two 32-byte loads per lane: every load instruction asks for whole sectors
struct Block { uint32_t w[16]; };
__device__ __forceinline__ void ldg_block(Block& b, const uint8_t* p)
{
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(b.w[0]), "=r"(b.w[1]), "=r"(b.w[2]), "=r"(b.w[3]), "=r"(b.w[4]), "=r"(b.w[5]), "=r"(b.w[6]), "=r"(b.w[7])
                 : "l"(p));
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(b.w[8]), "=r"(b.w[9]), "=r"(b.w[10]), "=r"(b.w[11]), "=r"(b.w[12]), "=r"(b.w[13]), "=r"(b.w[14]), "=r"(b.w[15])
                 : "l"(p + 32));
}
__device__ __forceinline__ void stg_v8(void* p, const uint32_t (&r)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
                 "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// 2-D tiled bulk store shared -> global through a tensor map (TMA); rows outside the tensor are dropped
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(map), "r"(src), "r"(x),
                 "r"(y)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// OCP E4M3 byte -> fp32, arithmetically (the all-ones exponent/mantissa code reads as 480)
__device__ __forceinline__ float fp8_to_float(uint32_t b)
{
    uint32_t ex = (b >> 3) & 15u, man = b & 7u;
    float mag = ex ? __uint_as_float(((ex + 120u) << 23) | (man << 20)) : static_cast<float>(man) * 0.001953125f;
    return (b & 0x80u) ? -mag : mag;
}
__device__ __forceinline__ uint32_t f2h_bits(float f) { return static_cast<uint32_t>(__half_as_ushort(__float2half_rn(f))); }

// ---------------------------------------------------------------------------------------------
// table staging (Sec. 4.2: metadata "loaded once" before the compressed loads)
// ---------------------------------------------------------------------------------------------
// In two halves, so that the caller can put work between the issue and the wait.  wait_tables returns false
// (CTA-uniform) if the bounded wait expired; the caller must then return.
__device__ __forceinline__ void issue_tables(uint8_t* smem, const uint8_t* d_meta, uint64_t* bar_storage)
{
    const uint32_t bar = smem_u32(bar_storage);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_expect_tx(bar, kTableBytes);
        bulk_g2s(smem_u32(smem), d_meta + kOffPattern, kTableBytes, bar);
    }
}
__device__ __forceinline__ bool wait_tables(uint64_t* bar_storage, uint32_t parity = 0)
{
    const uint32_t bar = smem_u32(bar_storage);
    __syncthreads();                             // the barrier word is initialised
    bool done = false;
    for (int i = 0; i < kWaitLimit && !done; ++i) done = mbar_try_wait(bar, parity);
    if (!done)                                   // second, bounded chance for the copy in flight
        for (int i = 0; i < kWaitLimit && !done; ++i) done = mbar_try_wait(bar, parity);
    const bool all = __syncthreads_and(done);
    if (!all && threadIdx.x == 0) atomicExch(&g_device_status, ECCO_ERR_DEVICE_TIMEOUT);
    return all;
}
__device__ __forceinline__ bool stage_tables(uint8_t* smem, const uint8_t* d_meta, uint64_t* bar_storage)
{
    issue_tables(smem, d_meta, bar_storage);
    return wait_tables(bar_storage);
}
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may become resident
// while the previous kernel in the stream is still draining.  dependency_wait() returns once that kernel has
// completed and its writes are visible (at once if there is no such overlap); every kernel executes it before
// its first access to global memory, so stream order is what it is without the attribute and only launch and
// prologue overlap.  release_dependents() lets the next kernel of the stream do the same with respect to this one.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Same for the mixed decoder: patterns and ID_KP table, then rank tables and arithmetic constants
// (adjacent in the image and in shared memory), two bulk copies on one barrier.  In two halves so
// that the caller can put work between the issue and the wait.
__device__ __forceinline__ void issue_rank_tables(uint8_t* smem, const uint8_t* d_meta, uint64_t* bar_storage, bool first = true)
{
    const uint32_t bar = smem_u32(bar_storage);
    if (threadIdx.x == 0) {
        if (first) {                             // later phases of the same barrier only re-arm it
            mbar_init(bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        mbar_expect_tx(bar, kPatternBytes + kKpLutBytes + kRankLutBytes + kArithBytes);
        bulk_g2s(smem_u32(smem), d_meta + kOffPattern, kPatternBytes + kKpLutBytes, bar);
        bulk_g2s(smem_u32(smem) + kSmemSymLut, d_meta + kOffRankLut, kRankLutBytes + kArithBytes, bar);
    }
}
// ---------------------------------------------------------------------------------------------
// the per-group decoder
// ---------------------------------------------------------------------------------------------
struct WarpSmem {
    uint32_t bits;      // shared address of bits[0][lane]
    uint32_t tab;       // shared address of tab[0][lane]
    uint32_t syms;      // shared address of syms[0][lane] (fused kernels only)
};

struct GroupHeader {
    uint32_t pos;       // first bit of the coded indices
    uint32_t lut;       // shared address of the symbol table of (ID_KP, ID_HF), OR-ed with its index rotation
    // mixed decoder only: addends of the length compare, and delta[L] in byte L of {dhi:dlo} (byte 0 = 0)
    uint32_t c1, c2, dlo, dhi;
};
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

// Pattern retriever (Sec. 4.2): scale byte, ID_HF, Huffman-coded ID_KP from the group's first 22
// stream bits (hdr, first bit in bit 0); writes the lane's 16 dequantised values (fp16 bits, or
// fp32 bits when kFloatTab).  first_bit = position of the group's first bit in the lane's staged
// bit stream.
// kRank: the kernel staged the rank tables (stage_rank_tables); tab is then indexed by rank.
template <bool kFloatTab, bool kRank = false>
__device__ __forceinline__ GroupHeader open_header(uint32_t hdr, uint32_t first_bit, uint32_t smem_base, const WarpSmem& ws, float T)
{
    const uint32_t qs = hdr & 0xffu, hf = (hdr >> 8) & 3u;
    const uint32_t kpw = (hdr >> kHeaderBits) & 0xfffu;
    uint32_t kpe;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(kpe) : "r"(smem_base + kSmemKpLut + kpw * 2));
    const uint32_t kp = kpe & 0xffu;
    GroupHeader h;
    h.pos = first_bit + kHeaderBits + (kpe >> 8);
    const uint32_t cb = kp * kCodebooks + hf;
    h.lut = (smem_base + kSmemSymLut + cb * 256) | lut_rotation(cb);   // table rows are 256-byte aligned
    const float top = fp8_to_float(qs) * T;           // FP8 -> FP16 range by the power-of-two factor
    const float s = fabsf(top);
    uint4 p0, p1;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(p0.x), "=r"(p0.y), "=r"(p0.z), "=r"(p0.w) : "r"(smem_base + kSmemPattern + kp * 32));
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(p1.x), "=r"(p1.y), "=r"(p1.z), "=r"(p1.w) : "r"(smem_base + kSmemPattern + kp * 32 + 16));
    const uint32_t pr[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
    uint32_t rank_lo = 0, rank_hi = 0;
    if (kRank) {
        const uint32_t a = smem_base + kSmemArith + cb * 4;
        h.c1 = lds_u32(a);
        h.c2 = lds_u32(a + 1024);
        const uint32_t d = lds_u32(a + 2048);
        rank_lo = lds_u32(a + 3072);
        rank_hi = lds_u32(a + 4096);
        const uint32_t even = d & 0x0f0f0fu, odd = (d >> 4) & 0x0f0f0fu;     // delta[2], [4], [6] and delta[3], [5], [7]
        h.dlo = prmt(even, odd, 0x4033u);
        h.dhi = prmt(even, odd, 0x6251u);
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const __half c = __ushort_as_half(static_cast<unsigned short>((pr[j >> 1] >> ((j & 1) * 16)) & 0xffffu));
        // mapper (Sec. 4.2): one fp32 product, one rounding to fp16
        const __half v = __float2half_rn(j < 15 ? __half2float(c) * s : top);
        const uint32_t row = kRank ? ((j < 8 ? rank_lo : rank_hi) >> ((j & 7) * 4)) & 15u : static_cast<uint32_t>(j);
        sts_u32(ws.tab + row * 128, kFloatTab ? __float_as_uint(__half2float(v)) : static_cast<uint32_t>(__half_as_ushort(v)));
    }
    return h;
}

// 64-byte block: stage the 16 words in the lane's column of the transposed bit-stream array, then the header
template <bool kFloatTab, bool kRank = false>
__device__ __forceinline__ GroupHeader open_group(const Block& blk, uint32_t smem_base, const WarpSmem& ws, float T)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) sts_u32(ws.bits + i * 128, blk.w[i]);
    return open_header<kFloatTab, kRank>(blk.w[0], 0u, smem_base, ws, T);
}

// Decodes the 128 indices of the lane's group (Sec. 4.2, Huffman decode) and hands each value to
// sink(n, value_bits, symbol, alive) (kLookup = false skips the value lookup and passes 0).  A codeword that would cross bit 512 ends the group: that and all
// later positions are delivered as zero (clipped).  Returns the end bit if all 128 fitted, else 0.
// Must be called by all 32 lanes of the warp.  Four symbols are decoded per window refill; the
// per-symbol clip test runs only in steps where some lane of the warp reaches bit 512.
// kLastRow / kEndBit: last data row of the lane's staged stream (two zero rows follow) and the bit
// at which the stream ends (16 and 512 for the 64-byte block).
// kArith (rank tables only): bit j set = symbol j of every four is decoded arithmetically from the canonical
// code's length thresholds instead of through the byte table; the sink's symbol is then the rank, and only its
// low four bits are meaningful.
// kFreeSteps (a multiple of 4): that many leading steps run without the clip test; the caller guarantees that
// the stream cannot end within them (a block's indices start at bit 22 at the latest, so 12 steps of at most
// 32 bits end by bit 406).
template <bool kLookup = true, uint32_t kLastRow = 16, uint32_t kEndBit = kBlockBits, uint32_t kArith = 0, int kFreeSteps = 0, class Sink>
__device__ __forceinline__ uint32_t decode_symbols(const GroupHeader& h, const WarpSmem& ws, Sink&& sink)
{
    static_assert(kFreeSteps % 4 == 0 && kFreeSteps < 32, "whole unrolled iterations");
    uint32_t pos = h.pos;
    bool alive = true;
    auto four = [&](int step, auto tested) {
        constexpr bool kTest = decltype(tested)::value;
        const uint32_t wi = kTest ? min(pos >> 5, kLastRow) : pos >> 5;
        const uint32_t lo = lds_u32(ws.bits + wi * 128), hi = lds_u32(ws.bits + wi * 128 + 128);
        const uint32_t win = __funnelshift_r(lo, hi, pos);           // 32 stream bits from pos
        const uint32_t wrev = kArith ? __brev(win) : 0u;             // the same bits, first one on top
        uint32_t e[4], end[4], acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if ((kArith >> j) & 1u) {
                const uint32_t t = wrev << acc, b = t >> 24;
                const uint32_t m = ((b * kArithSpread + h.c1) & (kArithGuard | 0xC0000000u)) | ((b * (2u * kArithSpread) + h.c2) & (2u * kArithGuard));
                const uint32_t len = __popc(m);                      // 2 + thresholds passed
                e[j] = __funnelshift_l(t, 0u, len) + prmt(h.dlo, h.dhi, len);   // codeword + delta[len]
                acc += len;
            } else {
                e[j] = lds_u8(h.lut ^ ((win >> acc) & 0xffu));       // rotated index, see lut_rotation()
                acc += e[j] >> 4;
            }
            end[j] = acc;
        }
        if (kTest && __any_sync(0xffffffffu, pos + acc > kEndBit)) {
            const uint32_t limit = kEndBit - min(pos, kEndBit);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                alive = alive && (end[j] <= limit);
                const uint32_t v = kLookup ? lds_u32(ws.tab + (e[j] & 15u) * 128) : 0u;
                sink(step * 4 + j, alive ? v : 0u, e[j] & 15u, alive);
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                sink(step * 4 + j, kLookup ? lds_u32(ws.tab + (e[j] & 15u) * 128) : 0u, e[j] & 15u, true);
        }
        pos += acc;
    };
    if (kFreeSteps > 0) {
#pragma unroll 4
        for (int step = 0; step < kFreeSteps; ++step) four(step, cuda::std::false_type{});
    }
#pragma unroll 4
    for (int step = kFreeSteps; step < 32; ++step) four(step, cuda::std::true_type{});
    return alive ? pos : 0u;
}

// Outlier fields (Sec. 3.2: 7-bit location + FP8 value, quantised with the per-tensor factor):
// pad j sits at bits [512-15(j+1), 512-15j).
__device__ __forceinline__ uint32_t read_pad(const WarpSmem& ws, int j)
{
    const uint32_t bitpos = kBlockBits - kPadBits * (j + 1);
    const uint32_t wi = bitpos >> 5;
    const uint32_t lo = lds_u32(ws.bits + wi * 128), hi = lds_u32(ws.bits + wi * 128 + 128);
    return __funnelshift_r(lo, hi, bitpos) & 0x7fffu;
}

// ---------------------------------------------------------------------------------------------
// K1: ecco_decompress
// ---------------------------------------------------------------------------------------------
// Work is dealt out in warp tiles of 32 consecutive groups, tile i to warp (i mod total warps):
// every SM then gets the same number of tiles to within one, whatever the tensor size.
template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_decompress_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_blocks, uint64_t n_groups,
                       uint16_t* __restrict__ d_out, uint32_t active_warps)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t smem_base = smem_u32(smem);
    WarpSmem ws;
    ws.bits = smem_base + kSmemWarpBase + warp * (kBitsBytes + kTabBytes) + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = 0;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);

    const uint64_t n_tiles = (n_groups + 31) / 32;
    // the host picks active_warps so that every working warp gets the same number of tiles (+-1 over
    // the whole grid); warp ids interleave over the CTAs, so every SM keeps the same number busy
    const uint64_t tile_stride = active_warps;
    uint64_t tile = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;
    if (tile >= tile_stride) tile = n_tiles;               // this warp sits the launch out (after the table barrier)
    Block blk;
    // lanes past the end of the tensor decode the last group again and store nothing
    if (tile < n_tiles) ldg_block(blk, d_blocks + min(tile * 32 + lane, n_groups - 1) * kBlockBytes);
    if (!stage_tables(smem, d_meta, &bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    for (; tile < n_tiles; tile += tile_stride) {
        const uint64_t g = tile * 32 + lane;
        const bool store = g < n_groups;
        const GroupHeader h = open_group<false>(blk, smem_base, ws, T);
        const uint64_t tn = tile + tile_stride;
        if (tn < n_tiles)                                  // next block in flight while this one decodes
            ldg_block(blk, d_blocks + min(tn * 32 + lane, n_groups - 1) * kBlockBytes);
        uint16_t* out = d_out + min(g, n_groups - 1) * kGroup;
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const uint32_t end = decode_symbols(h, ws, [&](int n, uint32_t v, uint32_t, bool) {
            const int slot = (n & 15) >> 1;
            if (n & 1) r[slot] |= v << 16; else r[slot] = v;
            if ((n & 15) == 15 && store) stg_v8(out + (n - 15), r);
        });
        if (end && store) {
            const int n_pad = min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits));
            for (int j = 0; j < n_pad; ++j) {
                const uint32_t f = read_pad(ws, j);
                // same thread, same address as the vector store above: program order holds
                out[f & 127u] = static_cast<uint16_t>(f2h_bits(fp8_to_float(f >> 7) * T));
            }
        }
    }
}

// K1, bulk-store variant.  Per-lane 32-byte stores land in 32 different 128-byte lines and cost the
// load/store pipe one pass per sector.  Here every 16 decoded values per lane go to a 1 KB
// staging tile in shared memory ([32 groups][32 bytes], 16-byte halves swizzled the way the
// tensor map's 32-byte swizzle expects, so the 128-bit shared stores are conflict-free) and one
// lane hands the tile to the TMA engine, which writes the 32 rows of the [n_groups][128] fp16
// tensor and drops rows past its end.  Outliers: those in the last tile (positions >= 112) are
// patched in shared memory before that tile leaves; the others are 2-byte global stores issued
// after the group's earlier tiles have been written (bulk wait + warp barrier), so they land last.
// The kernel takes up to kMaxJobs tensors and works through them one after the other without leaving the SM:
// between two tensors only the CTA's own warps meet (the tables are the CTA's), so an SM that is done with
// one tensor starts the next while others still finish, and launch latency and tail are paid once per call.
constexpr int kMaxJobs = 8;
struct alignas(64) DecompressJob {
    const uint8_t* meta;
    const uint8_t* blocks;
    uint64_t n_groups;
    uint16_t* out;
    uint32_t active_warps;     // working warps for this tensor: all get the same number of tiles
    uint32_t reserved[7];
    CUtensorMap map;           // [n_groups][128] fp16, box 32 x 16, 32-byte swizzle
};
struct DecompressBatch {
    int32_t n;
    int32_t reserved[15];
    DecompressJob job[kMaxJobs];
};

template <int kWarps, uint32_t kArith, int kDecFree = 12>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_decompress_tma_kernel(const __grid_constant__ DecompressBatch batch)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t smem_base = smem_u32(smem);
    constexpr uint32_t kStageBase = (kSmemRankWarpBase + kWarps * (kBitsBytes + kTabBytes) + 1023u) & ~1023u;
    WarpSmem ws;
    ws.bits = smem_base + kSmemRankWarpBase + warp * (kBitsBytes + kTabBytes) + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = 0;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);
    const uint32_t stage = smem_base + kStageBase + warp * 1024;                 // this warp's staging tile
    const uint32_t fp8tab = smem_base + kStageBase + kWarps * 1024;              // [256] fp16: outlier byte -> value
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem + kStageBase + kWarps * 1024 + 512);   // in the dynamic part: no room for a static one
    const uint32_t swz = ((lane >> 2) & 1u) << 4;                               // 32-byte swizzle: bit 4 ^= bit 7
    const uint32_t my_row = stage + lane * 32;

    dependency_wait();
    release_dependents();
  for (int t = 0; t < batch.n; ++t) {
    const DecompressJob& job = batch.job[t];
    const uint8_t* __restrict__ d_meta = job.meta;
    const uint8_t* __restrict__ d_blocks = job.blocks;
    const uint64_t n_groups = job.n_groups;
    uint16_t* __restrict__ d_out = job.out;
    const CUtensorMap& out_map = job.map;
    const uint64_t n_tiles = (n_groups + 31) / 32;
    const uint64_t tile_stride = job.active_warps;         // see ecco_decompress_kernel
    uint64_t tile = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;
    if (tile >= tile_stride) tile = n_tiles;
    if (t > 0) __syncthreads();                            // every warp is done with the previous tensor's tables
    issue_rank_tables(smem, d_meta, bar, t == 0);
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;
    if (threadIdx.x < 256)                                 // visible after the barriers inside wait_tables
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(fp8tab + threadIdx.x * 2),
                     "h"(static_cast<unsigned short>(f2h_bits(fp8_to_float(threadIdx.x) * T))) : "memory");
    Block blk;
    if (tile < n_tiles) ldg_block(blk, d_blocks + min(tile * 32 + lane, n_groups - 1) * kBlockBytes);
    if (!wait_tables(bar, static_cast<uint32_t>(t & 1))) return;

    for (; tile < n_tiles; tile += tile_stride) {
        const uint64_t g = tile * 32 + lane;
        const bool store = g < n_groups;
        const GroupHeader h = open_group<false, true>(blk, smem_base, ws, T);
        const uint64_t tn = tile + tile_stride;
        if (tn < n_tiles) ldg_block(blk, d_blocks + min(tn * 32 + lane, n_groups - 1) * kBlockBytes);
        const int row0 = static_cast<int>(tile * 32);
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        auto stage_rows = [&]() {
            if (lane == 0) bulk_wait_read0();              // the engine has read the previous tile
            __syncwarp();
            sts_v4(my_row + swz, r[0], r[1], r[2], r[3]);
            sts_v4(my_row + (swz ^ 16u), r[4], r[5], r[6], r[7]);
        };
        auto send_tile = [&](int chunk) {
            fence_async_smem();                            // generic-proxy writes -> visible to the engine
            __syncwarp();
            if (lane == 0) { tma_store_2d(&out_map, stage, chunk * 16, row0); bulk_commit(); }
        };
        const uint32_t end = decode_symbols<true, 16, kBlockBits, kArith, kDecFree>(h, ws, [&](int n, uint32_t v, uint32_t, bool) {
            const int slot = (n & 15) >> 1;
            if (n & 1) r[slot] |= v << 16; else r[slot] = v;
            if ((n & 15) == 15 && n != 127) { stage_rows(); send_tile(n >> 4); }
        });
        stage_rows();                                      // values 112..127
        const int n_pad = end ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
        if (__any_sync(0xffffffffu, n_pad > 0)) {
            if (lane == 0) bulk_wait_all();                // tiles 0..6 of this group are in memory
            __syncwarp();
            uint16_t* out = d_out + min(g, n_groups - 1) * kGroup;
            const int n_max = __reduce_max_sync(0xffffffffu, n_pad);
#pragma unroll
            for (int j = 0; j < kMaxPads; ++j) {           // ascending: a later pad overrides an earlier one
                if (j >= n_max) break;
                if (j < n_pad) {
                    const uint32_t f = read_pad(ws, j);
                    const uint32_t loc = f & 127u;
                    unsigned short val;
                    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(val) : "r"(fp8tab + (f >> 7) * 2));
                    if (loc >= 112u) {
                        const uint32_t byte = (loc - 112u) * 2;
                        asm volatile("st.shared.u16 [%0], %1;" ::"r"(my_row + ((byte & 16u) ^ swz) + (byte & 15u)), "h"(val) : "memory");
                    } else if (store) {
                        out[loc] = val;
                    }
                }
            }
        }
        send_tile(7);
    }
  }
    if (lane == 0) bulk_wait_all();                        // shared memory must outlive the engine's reads
}

// ---------------------------------------------------------------------------------------------
// K1v: decompress of the variable-length container (groups back to back in one bit stream, start
// index on the side; nothing clipped, nothing padded).  Same thread-per-group decode and the same
// TMA tile store as K1; the difference is the front end: a lane copies the 16-byte chunks that
// cover its group (on average 5) into its column of a 40-row transposed array, masks the bits
// that belong to the next group, and starts decoding at bit (start mod 128).
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kVarRows = 40;                        // 10 chunks: 127 + 1046 bits at most, plus slack
constexpr uint32_t kVarBitsBytes = kVarRows * 128;

template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_var_decompress_kernel(const uint8_t* __restrict__ d_meta, const uint4* __restrict__ d_stream,
                           const uint64_t* __restrict__ d_index, uint64_t n_groups, uint16_t* __restrict__ d_out,
                           uint32_t active_warps, const __grid_constant__ CUtensorMap out_map)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t smem_base = smem_u32(smem);
    constexpr uint32_t kStageBase = (kSmemWarpBase + kWarps * (kVarBitsBytes + kTabBytes) + 1023u) & ~1023u;
    WarpSmem ws;
    ws.bits = smem_base + kSmemWarpBase + warp * (kVarBitsBytes + kTabBytes) + lane * 4;
    ws.tab = ws.bits + kVarBitsBytes;
    ws.syms = 0;
    for (uint32_t r = 0; r < kVarRows; ++r) sts_u32(ws.bits + r * 128, 0u);
    const uint32_t stage = smem_base + kStageBase + warp * 1024;
    const uint32_t swz = ((lane >> 2) & 1u) << 4;
    const uint32_t my_row = stage + lane * 32;

    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    issue_tables(smem, d_meta, &bar);
    const uint64_t total_bits = d_index[0];
    const uint64_t stream_chunks = (total_bits + 127) >> 7;
    const uint64_t* chunk_base = d_index + 1;
    const uint32_t* off32 = reinterpret_cast<const uint32_t*>(d_index + 1 + var_chunks(n_groups));
    auto start_of = [&](uint64_t g) { return g < n_groups ? chunk_base[g >> kVarChunkShift] + off32[g] : total_bits; };

    const uint64_t n_tiles = (n_groups + 31) / 32;
    const uint64_t tile_stride = active_warps;
    uint64_t tile = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;
    if (tile >= tile_stride) tile = n_tiles;
    uint32_t dirty_rows = 0;                               // rows of this lane's column that hold a previous group

    // The span of a group comes from the index and its chunks from the stream: two dependent trips to memory.
    // Both are fetched one tile ahead, the first kVarAhead chunks into registers (an average group covers five),
    // the rare rest when the tile is staged.
    constexpr uint32_t kVarAhead = 6;
    struct Span { uint64_t start, end, c0; uint32_t nc; };
    auto span_of = [&](uint64_t t) {
        Span sp;
        const uint64_t g = min(t * 32 + lane, n_groups - 1);
        sp.start = min(start_of(g), total_bits);
        sp.end = max(min(start_of(g + 1), total_bits), sp.start);          // the group sees [start, end), zeros after
        sp.c0 = sp.start >> 7;
        sp.nc = static_cast<uint32_t>(min(static_cast<uint64_t>(kVarRows / 4), ((sp.end + 127) >> 7) - sp.c0));
        return sp;
    };
    auto load_chunk = [&](uint64_t c) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (c < stream_chunks) asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(d_stream + c));
        return v;
    };
    Span cur = {0, 0, 0, 0};
    uint4 ahead[kVarAhead];
    if (tile < n_tiles) {
        cur = span_of(tile);
#pragma unroll
        for (uint32_t c = 0; c < kVarAhead; ++c) ahead[c] = c < cur.nc ? load_chunk(cur.c0 + c) : make_uint4(0, 0, 0, 0);
    }

    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    for (; tile < n_tiles; tile += tile_stride) {
        const uint64_t end = cur.end;
        const uint64_t c0 = cur.c0;
        const uint32_t nc = cur.nc;
        const uint32_t first_bit = static_cast<uint32_t>(cur.start & 127u);
        auto stage_chunk = [&](uint32_t c, const uint4& v) {
            uint32_t w[4] = {v.x, v.y, v.z, v.w};
            const uint64_t first = (c0 + c) << 7;          // stream bit of w[0] bit 0
            if (first + 128 > end) {                       // bits of the next group read as zero
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint64_t wb = first + 32 * k;
                    w[k] = wb >= end ? 0u : (end - wb >= 32 ? w[k] : (w[k] & ((1u << static_cast<uint32_t>(end - wb)) - 1u)));
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) sts_u32(ws.bits + (4 * c + k) * 128, w[k]);
        };
#pragma unroll
        for (uint32_t c = 0; c < kVarAhead; ++c)
            if (c < nc) stage_chunk(c, ahead[c]);
        for (uint32_t c = kVarAhead; c < nc; ++c) stage_chunk(c, load_chunk(c0 + c));
        const uint64_t tn = tile + tile_stride;
        if (tn < n_tiles) {                                // the next tile's span and first chunks, in flight during this decode
            cur = span_of(tn);
#pragma unroll
            for (uint32_t c = 0; c < kVarAhead; ++c) ahead[c] = c < cur.nc ? load_chunk(cur.c0 + c) : make_uint4(0, 0, 0, 0);
        }
        for (uint32_t r = 4 * nc; r < dirty_rows; ++r) sts_u32(ws.bits + r * 128, 0u);
        dirty_rows = 4 * nc;
        const uint32_t hw = first_bit >> 5;
        const uint32_t hdr = __funnelshift_r(lds_u32(ws.bits + hw * 128), lds_u32(ws.bits + hw * 128 + 128), first_bit);
        const GroupHeader h = open_header<false>(hdr, first_bit, smem_base, ws, T);
        const int row0 = static_cast<int>(tile * 32);
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        decode_symbols<true, kVarRows - 2, kVarRows * 32, 0, 28>(h, ws, [&](int n, uint32_t v, uint32_t, bool) {
            const int slot = (n & 15) >> 1;
            if (n & 1) r[slot] |= v << 16; else r[slot] = v;
            if ((n & 15) == 15) {
                if (lane == 0) bulk_wait_read0();          // the engine has read the previous tile
                __syncwarp();
                sts_v4(my_row + swz, r[0], r[1], r[2], r[3]);
                sts_v4(my_row + (swz ^ 16u), r[4], r[5], r[6], r[7]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { tma_store_2d(&out_map, stage, (n >> 4) * 16, row0); bulk_commit(); }
            }
        });
    }
    if (lane == 0) bulk_wait_all();
}

// ---------------------------------------------------------------------------------------------
// K2/K3: fused consumers.  kV = number of dot products per group (batch rows of x, or query
// heads per KV head).  The vector slice xs[128][kV] fp32 lives in shared memory; every lane reads
// the same element at the same time (one broadcast wavefront), 16 bytes per load, so a slice
// element costs 1/4 (kV = 1) to 2 (kV = 8) loads per symbol.
// ---------------------------------------------------------------------------------------------
template <int kV>
struct Accum {
    float a[kV];
    float4 cache;                       // the current 16 bytes of the slice (kV <= 2)
    __device__ __forceinline__ void clear()
    {
#pragma unroll
        for (int v = 0; v < kV; ++v) a[v] = 0.0f;
    }
    static __device__ __forceinline__ float4 lds_f4(uint32_t addr)
    {
        float4 x;
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(addr));
        return x;
    }
    // value w of position n (n is a compile-time constant after unrolling); xs = shared address of xs[0][0]
    __device__ __forceinline__ void fma(int n, float w, uint32_t xs)
    {
        if constexpr (kV == 1) {
            if ((n & 3) == 0) cache = lds_f4(xs + n * 4);
            const float x = (n & 3) == 0 ? cache.x : (n & 3) == 1 ? cache.y : (n & 3) == 2 ? cache.z : cache.w;
            a[0] = fmaf(w, x, a[0]);
        } else if constexpr (kV == 2) {
            if ((n & 1) == 0) cache = lds_f4(xs + n * 8);
            a[0] = fmaf(w, (n & 1) ? cache.z : cache.x, a[0]);
            a[1] = fmaf(w, (n & 1) ? cache.w : cache.y, a[1]);
        } else {
#pragma unroll
            for (int q = 0; q < kV / 4; ++q) {
                const float4 x = lds_f4(xs + n * (kV * 4) + q * 16);
                a[q * 4 + 0] = fmaf(w, x.x, a[q * 4 + 0]);
                a[q * 4 + 1] = fmaf(w, x.y, a[q * 4 + 1]);
                a[q * 4 + 2] = fmaf(w, x.z, a[q * 4 + 2]);
                a[q * 4 + 3] = fmaf(w, x.w, a[q * 4 + 3]);
            }
        }
    }
    // out-of-order correction at a run-time position (outlier fix-up)
    __device__ __forceinline__ void fma_at(uint32_t loc, float w, uint32_t xs)
    {
#pragma unroll
        for (int v = 0; v < kV; ++v) {
            float x;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(xs + (loc * kV + v) * 4));
            a[v] = fmaf(w, x, a[v]);
        }
    }
};

// decode one group and accumulate its kV dot products against xs (shared address of xs[0][0])
template <int kV>
__device__ __forceinline__ void fused_group(const Block& blk, uint32_t smem_base, const WarpSmem& ws, float T,
                                            uint32_t xs, Accum<kV>& acc)
{
    const GroupHeader h = open_group<true, kFusedRank>(blk, smem_base, ws, T);
    uint32_t packed = 0;
    const uint32_t end = decode_symbols<true, 16, kBlockBits, kFusedArith, kFusedFree>(h, ws, [&](int n, uint32_t v, uint32_t sym, bool) {
        acc.fma(n, __uint_as_float(v), xs);
        packed |= sym << ((n & 7) * 4);
        if ((n & 7) == 7) { sts_u32(ws.syms + (n >> 3) * 128, packed); packed = 0; }
    });
    if (end) {
        // outliers replace the mapped value at their location: add (outlier - mapped) * x
        const int n_pad = min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits));
        uint64_t seen_lo = 0, seen_hi = 0;                  // 128-bit "already replaced" mask
        for (int j = n_pad - 1; j >= 0; --j) {             // the last pad wins on a duplicate location
            const uint32_t f = read_pad(ws, j);
            const uint32_t loc = f & 127u;
            const uint64_t bit = 1ull << (loc & 63u);
            const bool upper = loc >= 64u;
            if ((upper ? seen_hi : seen_lo) & bit) continue;
            if (upper) seen_hi |= bit; else seen_lo |= bit;
            const uint32_t word = lds_u32(ws.syms + (loc >> 3) * 128);
            const uint32_t sym = (word >> ((loc & 7u) * 4)) & 15u;
            const float mapped = __uint_as_float(lds_u32(ws.tab + sym * 128));
            const float outlier = __half2float(__float2half_rn(fp8_to_float(f >> 7) * T));
            acc.fma_at(loc, outlier - mapped, xs);
        }
    }
}

// Contiguous split of U work units over G CTAs: CTA c owns [unit_begin(c), unit_begin(c + 1)).
__host__ __device__ __forceinline__ int64_t unit_begin(int64_t U, int G, int c) { return U * c / G; }
__host__ __device__ __forceinline__ int unit_owner(int64_t U, int G, int64_t u)
{
    int c = static_cast<int>(u * G / U);
    while (c + 1 < G && unit_begin(U, G, c + 1) <= u) ++c;
    while (c > 0 && unit_begin(U, G, c) > u) --c;
    return c;
}

template <int kWarps>
__device__ __forceinline__ WarpSmem fused_warp_smem(uint32_t smem_base)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    constexpr uint32_t kWarpBytes = kBitsBytes + kTabBytes + kSymsBytes;
    WarpSmem ws;
    ws.bits = smem_base + kFusedBase + warp * kWarpBytes + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = ws.tab + kTabBytes;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);
    return ws;
}

// K2 for one or two rows of x: the slice is small enough (512 B or 1 KB) for every warp to keep
// its own, so warps never meet at a barrier.  A work unit is (32 consecutive rows, one k-block),
// numbered row-tile major; every working warp owns a contiguous run of units and keeps its rows'
// partial sums in registers along k.  When a row tile is shared by several warps each writes its
// partial sums to its own workspace slot (slot = global warp id + row tile: unique along the
// staircase of (warp, tile) pairs) and the last to arrive (ticket counter) adds the slots in warp
// order: the result does not depend on scheduling.  Workspace: partial[slot][kV][32] floats, then
// one ticket per 32-row tile.
template <int kV, int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_gemv_warp_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_blocks, int n_out, int kblocks,
                      const __half* __restrict__ d_x, float* __restrict__ d_y, float* __restrict__ d_partial,
                      unsigned int* __restrict__ d_tickets, int active_warps)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    constexpr uint32_t kWarpBytes = kBitsBytes + kTabBytes + kSymsBytes;
    constexpr uint32_t kXsBytes = kGroup * kV * 4;
    const uint32_t smem_base = smem_u32(smem);
    const WarpSmem ws = fused_warp_smem<kWarps>(smem_base);
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    const uint32_t xs = smem_base + kFusedBase + kWarps * kWarpBytes + warp * kXsBytes;   // this warp's slice

    // W working warps (chosen by the host so that they all get the same number of units, and never
    // more than there are units); warp ids interleave over the CTAs; the other warps idle
    const int wg = warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x);
    const int tiles = (n_out + 31) / 32;
    const int64_t U = static_cast<int64_t>(tiles) * kblocks;
    const int W = active_warps;
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    const int k = kblocks * kGroup;
    auto block_ptr = [&](int64_t u) {
        const int row = min(static_cast<int>(u / kblocks) * 32 + lane, n_out - 1);     // rows past the end: repeat the last
        return d_blocks + (static_cast<uint64_t>(row) * kblocks + static_cast<int>(u % kblocks)) * kBlockBytes;
    };
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    if (kFusedRank) issue_rank_tables(smem, d_meta, &bar); else issue_tables(smem, d_meta, &bar);
    Block blk;
    if (u0 < u1) ldg_block(blk, block_ptr(u0));
    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    Accum<kV> acc;
    acc.clear();
    auto flush = [&](int tile) {
        const int row = tile * 32 + lane;
        const bool row_ok = row < n_out;
        const int w_lo = unit_owner(U, W, static_cast<int64_t>(tile) * kblocks);
        const int w_hi = unit_owner(U, W, static_cast<int64_t>(tile + 1) * kblocks - 1);
        if (w_lo == w_hi) {
            if (row_ok) {
#pragma unroll
                for (int b = 0; b < kV; ++b) d_y[static_cast<size_t>(b) * n_out + row] = acc.a[b];
            }
            return;
        }
        float* mine = d_partial + static_cast<size_t>(wg + tile) * kV * 32;
#pragma unroll
        for (int b = 0; b < kV; ++b) mine[b * 32 + lane] = acc.a[b];
        __threadfence();
        __syncwarp();
        unsigned int t = 0;
        if (lane == 0) t = atomicAdd(&d_tickets[tile], 1u);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t == static_cast<unsigned int>(w_hi - w_lo)) {  // last of the warps that share this tile
            __threadfence();
            if (row_ok) {
#pragma unroll
                for (int b = 0; b < kV; ++b) {
                    // slots are added in warp order whatever the arrival order; loads go out sixteen at a time
                    const float* slot = d_partial + (static_cast<size_t>(w_lo + tile) * kV + b) * 32 + lane;
                    float sum = 0.0f;
                    int ww = w_lo;
                    for (; ww + 16 <= w_hi + 1; ww += 16, slot += 16 * kV * 32) {
                        float v[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = __ldcg(slot + i * kV * 32);
#pragma unroll
                        for (int i = 0; i < 16; ++i) sum += v[i];
                    }
                    for (; ww <= w_hi; ++ww, slot += kV * 32) sum += __ldcg(slot);
                    d_y[static_cast<size_t>(b) * n_out + row] = sum;
                }
            }
            if (lane == 0) d_tickets[tile] = 0;
        }
    };

    // x for a unit is fetched one unit ahead, like the block
    uint2 xraw[kV];
    auto load_x = [&](int64_t u) {
        const int kb = static_cast<int>(u % kblocks);
#pragma unroll
        for (int b = 0; b < kV; ++b)
            xraw[b] = __ldg(reinterpret_cast<const uint2*>(d_x + static_cast<size_t>(b) * k + kb * kGroup + lane * 4));
    };
    if (u0 < u1) load_x(u0);
    int cur_tile = static_cast<int>(u0 / kblocks);
    for (int64_t u = u0; u < u1; ++u) {
        const int tile = static_cast<int>(u / kblocks);
        if (tile != cur_tile) { flush(cur_tile); acc.clear(); cur_tile = tile; }
        // this warp's slice: lane l converts x[b][kb*128 + 4l .. 4l+3] to fp32, layout xs[i][b]
        __syncwarp();
        {
            float v[kV][4];
#pragma unroll
            for (int b = 0; b < kV; ++b) {
                const __half2 h0 = *reinterpret_cast<const __half2*>(&xraw[b].x), h1 = *reinterpret_cast<const __half2*>(&xraw[b].y);
                v[b][0] = __low2float(h0); v[b][1] = __high2float(h0); v[b][2] = __low2float(h1); v[b][3] = __high2float(h1);
            }
            if constexpr (kV == 1) {
                sts_v4(xs + lane * 16, __float_as_uint(v[0][0]), __float_as_uint(v[0][1]), __float_as_uint(v[0][2]), __float_as_uint(v[0][3]));
            } else {
                sts_v4(xs + lane * 32, __float_as_uint(v[0][0]), __float_as_uint(v[1][0]), __float_as_uint(v[0][1]), __float_as_uint(v[1][1]));
                sts_v4(xs + lane * 32 + 16, __float_as_uint(v[0][2]), __float_as_uint(v[1][2]), __float_as_uint(v[0][3]), __float_as_uint(v[1][3]));
            }
        }
        __syncwarp();
        const Block cur = blk;
        if (u + 1 < u1) { ldg_block(blk, block_ptr(u + 1)); load_x(u + 1); }
        fused_group<kV>(cur, smem_base, ws, T, xs, acc);
    }
    if (u0 < u1) flush(cur_tile);
}

// K3: scores[b][hq][t] = scale * q[b][hq] . K~[b][hq / q_per_kv][t].  A work unit is (one (batch, kv
// head) pair, a chunk of kWarps*32 tokens); units are dealt to persistent CTAs in contiguous runs,
// the query slice is restaged when the head changes, a thread owns one token.
template <int kV, int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_attn_scores_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_kblocks, int heads, int seq,
                        int q_per_kv, const __half* __restrict__ d_q, float scale, float* __restrict__ d_scores)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    constexpr int kTokens = kWarps * 32;
    constexpr uint32_t kWarpBytes = kBitsBytes + kTabBytes + kSymsBytes;
    const uint32_t smem_base = smem_u32(smem);
    const WarpSmem ws = fused_warp_smem<kWarps>(smem_base);
    float* xs = reinterpret_cast<float*>(smem + kFusedBase + kWarps * kWarpBytes);
    const uint32_t xs_addr = smem_u32(xs);

    const int G = gridDim.x, c = blockIdx.x, tid = static_cast<int>(threadIdx.x);
    const int chunks = (seq + kTokens - 1) / kTokens;
    const int64_t U = static_cast<int64_t>(heads) * chunks;
    const int64_t u0 = unit_begin(U, G, c), u1 = unit_begin(U, G, c + 1);
    // lanes past the end of the sequence decode its last token again and store nothing
    auto block_ptr = [&](int64_t u) {
        const int bh = static_cast<int>(u / chunks), t = min(static_cast<int>(u % chunks) * kTokens + tid, seq - 1);
        return d_kblocks + (static_cast<uint64_t>(bh) * seq + t) * kBlockBytes;
    };
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    if (kFusedRank) issue_rank_tables(smem, d_meta, &bar); else issue_tables(smem, d_meta, &bar);
    Block blk;
    if (u0 < u1) ldg_block(blk, block_ptr(u0));
    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    int cur_bh = -1;
    for (int64_t u = u0; u < u1; ++u) {
        const int bh = static_cast<int>(u / chunks), t = static_cast<int>(u % chunks) * kTokens + tid;
        if (bh != cur_bh) {
            __syncthreads();                               // everyone is done with the previous head's slice
            // q[b][h*q_per_kv + r][d] -> xs[d][r], pre-multiplied by scale; heads beyond q_per_kv are zero
            for (int i = tid; i < kGroup * kV; i += kTokens) {
                const int r = i % kV, d = i / kV;
                xs[i] = (r < q_per_kv) ? scale * __half2float(d_q[(static_cast<size_t>(bh) * q_per_kv + r) * kGroup + d]) : 0.0f;
            }
            __syncthreads();
            cur_bh = bh;
        }
        const Block cur = blk;
        if (u + 1 < u1) ldg_block(blk, block_ptr(u + 1));
        Accum<kV> acc;
        acc.clear();
        fused_group<kV>(cur, smem_base, ws, T, xs_addr, acc);
        if (t < seq) {
#pragma unroll
            for (int r = 0; r < kV; ++r)
                if (r < q_per_kv) d_scores[(static_cast<size_t>(bh) * q_per_kv + r) * seq + t] = acc.a[r];
        }
    }
}

// ---------------------------------------------------------------------------------------------
// K5: attention output over a compressed V cache (Eq. 3: softmax(QK^T / sqrt(d_k)) V).
// out[b][hq][d] = sum_t p[b][hq][t] * V~[b][hq / q_per_kv][t][d] with p = softmax_t(scores).
// A thread owns one token (one group) as in K3, but here the sum runs over tokens, i.e. across
// lanes.  Pass 1 runs the serial Huffman chain and keeps only the 4-bit indices (syms[16][32]);
// by then the end bit, hence the outliers, are known.  Pass 2 walks the eight 16-dim chunks: map
// the indices through the lane's table, stage them in a [32 tokens][16 dims] fp16 tile (same
// swizzle as the decompress staging tile), overwrite the outliers of that chunk in the tile, and
// contract the tile on the tensor cores: (V tile)^T [16 dims x 32 tokens] x P^T [32 tokens x 8
// heads] with mma.m16n8k16, fp32 accumulators (4 registers per 16 dims, 32 for the 128 dims).  p is
// split into an fp16 head and an fp16 remainder (two MMAs) so that its rounding does not show.
// The result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
ecco_softmax_stats_kernel(const float* __restrict__ d_scores, int rows, int seq, float2* __restrict__ d_stats)
{
    const int row = static_cast<int>(blockIdx.x) * 8 + static_cast<int>(threadIdx.x >> 5), lane = static_cast<int>(threadIdx.x & 31u);
    dependency_wait();                                     // the scores may come from the previous kernel of the stream
    release_dependents();
    if (row >= rows) return;
    const float* s = d_scores + static_cast<size_t>(row) * seq;
    float mx = -INFINITY;
    for (int t = lane; t < seq; t += 32) mx = fmaxf(mx, s[t]);
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = 0.0f;
    for (int t = lane; t < seq; t += 32) sum += expf(s[t] - mx);
#pragma unroll
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) d_stats[row] = make_float2(mx, 1.0f / sum);
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

constexpr uint32_t kAvWarpBytes = kBitsBytes + kTabBytes + kSymsBytes + 1024;   // + the [32][16] fp16 tile

template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_attn_values_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_vblocks, int heads, int seq,
                        int q_per_kv, const float* __restrict__ d_scores, const float2* __restrict__ d_stats,
                        float* __restrict__ d_out, float* __restrict__ d_partial, unsigned int* __restrict__ d_tickets)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    __shared__ unsigned int ticket;
    __shared__ float2 stats_s[8];
    constexpr int kTokens = kWarps * 32;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const int tid = static_cast<int>(threadIdx.x);
    WarpSmem ws;
    ws.bits = smem_base + kSmemWarpBase + warp * kAvWarpBytes + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = ws.tab + kTabBytes;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);
    const uint32_t stage = smem_base + kSmemWarpBase + warp * kAvWarpBytes + kBitsBytes + kTabBytes + kSymsBytes;
    const uint32_t swz = ((lane >> 2) & 1u) << 4;
    const uint32_t my_row = stage + lane * 32;
    float* out_s = reinterpret_cast<float*>(smem + kSmemWarpBase + kWarps * kAvWarpBytes);    // [128 dims][8 heads]

    const int G = gridDim.x, c = blockIdx.x;
    const int chunks = (seq + kTokens - 1) / kTokens;
    const int64_t U = static_cast<int64_t>(heads) * chunks;
    const int64_t u0 = unit_begin(U, G, c), u1 = unit_begin(U, G, c + 1);
    auto block_ptr = [&](int64_t u) {
        const int bh = static_cast<int>(u / chunks), t = min(static_cast<int>(u % chunks) * kTokens + tid, seq - 1);
        return d_vblocks + (static_cast<uint64_t>(bh) * seq + t) * kBlockBytes;
    };
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    issue_tables(smem, d_meta, &bar);
    Block blk;
    if (u0 < u1) ldg_block(blk, block_ptr(u0));
    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    float acc[8][4];                                       // [16-dim chunk][mma accumulator]
    auto clear_acc = [&]() {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    };
    clear_acc();

    // all tokens of head bh seen by this CTA are in acc: reduce over the warps in warp order, then
    // either store (this CTA owns the whole head) or hand a partial to the slot-and-ticket reduction
    auto flush = [&](int bh) {
        for (int i = tid; i < kGroup * 8; i += kTokens) out_s[i] = 0.0f;
        __syncthreads();
        for (int w = 0; w < kWarps; ++w) {
            if (static_cast<int>(warp) == w) {
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int dim = ch * 16 + static_cast<int>(lane >> 2) + (j >= 2 ? 8 : 0);
                        const int head = static_cast<int>(lane & 3u) * 2 + (j & 1);
                        out_s[dim * 8 + head] += acc[ch][j];
                    }
            }
            __syncthreads();
        }
        const int c_lo = unit_owner(U, G, static_cast<int64_t>(bh) * chunks);
        const int c_hi = unit_owner(U, G, static_cast<int64_t>(bh + 1) * chunks - 1);
        if (c_lo == c_hi) {
            for (int i = tid; i < kGroup * 8; i += kTokens) {
                const int dim = i >> 3, r = i & 7;
                if (r < q_per_kv) d_out[(static_cast<size_t>(bh) * q_per_kv + r) * kGroup + dim] = out_s[i];
            }
        } else {
            float* mine = d_partial + static_cast<size_t>(c + bh) * (kGroup * 8);
            for (int i = tid; i < kGroup * 8; i += kTokens) mine[i] = out_s[i];
            __threadfence();
            __syncthreads();
            if (tid == 0) ticket = atomicAdd(&d_tickets[bh], 1u);
            __syncthreads();
            if (ticket == static_cast<unsigned int>(c_hi - c_lo)) {
                __threadfence();
                for (int i = tid; i < kGroup * 8; i += kTokens) {
                    const int dim = i >> 3, r = i & 7;
                    if (r >= q_per_kv) continue;
                    float sum = 0.0f;
                    for (int cc = c_lo; cc <= c_hi; ++cc) sum += __ldcg(d_partial + static_cast<size_t>(cc + bh) * (kGroup * 8) + i);
                    d_out[(static_cast<size_t>(bh) * q_per_kv + r) * kGroup + dim] = sum;
                }
                if (tid == 0) d_tickets[bh] = 0;
            }
        }
        __syncthreads();
    };

    int cur_bh = -1;
    for (int64_t u = u0; u < u1; ++u) {
        const int bh = static_cast<int>(u / chunks);
        const int tile_base = static_cast<int>(u % chunks) * kTokens + static_cast<int>(warp) * 32;
        const int t = tile_base + static_cast<int>(lane);
        if (bh != cur_bh) {
            if (cur_bh >= 0) { flush(cur_bh); clear_acc(); }
            if (tid < 8) stats_s[tid] = tid < q_per_kv ? d_stats[static_cast<size_t>(bh) * q_per_kv + tid] : make_float2(0.0f, 0.0f);
            __syncthreads();
            cur_bh = bh;
        }
        // P^T fragments (B operand): head = lane / 4, tokens (lane % 4) * 2 + {0, 1} + 8 j
        uint32_t p_hi[4], p_lo[4];
        {
            const int r = static_cast<int>(lane >> 2);
            const float2 st = stats_s[r];
            const float* srow = d_scores + (static_cast<size_t>(bh) * q_per_kv + min(r, q_per_kv - 1)) * seq;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int tk = tile_base + static_cast<int>(lane & 3u) * 2 + 8 * j;
                float p0 = 0.0f, p1 = 0.0f;
                if (r < q_per_kv && tk < seq) p0 = __expf(srow[tk] - st.x) * st.y;
                if (r < q_per_kv && tk + 1 < seq) p1 = __expf(srow[tk + 1] - st.x) * st.y;
                const __half h0 = __float2half_rn(p0), h1 = __float2half_rn(p1);
                const __half l0 = __float2half_rn(p0 - __half2float(h0)), l1 = __float2half_rn(p1 - __half2float(h1));
                p_hi[j] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
                p_lo[j] = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
            }
        }
        const Block cur = blk;
        if (u + 1 < u1) ldg_block(blk, block_ptr(u + 1));
        const bool valid = t < seq;                        // lanes past the end stage zeros (their p is zero too)
        const GroupHeader h = open_group<false>(cur, smem_base, ws, T);
        // pass 1: the serial Huffman chain, indices only (8 per word into syms[16][32])
        uint32_t packed = 0;
        int n_fit = kGroup;
        const uint32_t end = decode_symbols<false, 16, kBlockBits, 0, kFusedFree>(h, ws, [&](int n, uint32_t, uint32_t sym, bool alive) {
            if (!alive) n_fit = min(n_fit, n);             // only the clip path can see alive == false
            packed |= sym << ((n & 7) * 4);
            if ((n & 7) == 7) { sts_u32(ws.syms + (n >> 3) * 128, packed); packed = 0; }
        });
        if (!valid) n_fit = 0;
        // outliers of a complete group: which 16-dim chunks they fall into
        const int n_pad = (end && valid) ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
        uint64_t pads_lo = 0, pads_hi = 0;                 // 16 bits per chunk: which pads fall into it
        for (int j = 0; j < n_pad; ++j) {
            const uint32_t ch = (read_pad(ws, j) & 127u) >> 4;
            const uint64_t bit = 1ull << ((ch & 3u) * 16 + j);
            if (ch < 4) pads_lo |= bit; else pads_hi |= bit;
        }
        // pass 2: per 16-dim chunk map the indices, patch the outliers in the tile, contract on the tensor cores
        for (int ch = 0; ch < 8; ++ch) {
            uint32_t r8[8];
            const uint32_t w0 = lds_u32(ws.syms + (2 * ch) * 128), w1 = lds_u32(ws.syms + (2 * ch + 1) * 128);
            const bool whole = ch * 16 + 16 <= n_fit;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const uint32_t sym = ((i < 8 ? w0 : w1) >> ((i & 7) * 4)) & 15u;
                uint32_t v = lds_u32(ws.tab + sym * 128);
                if (!whole) v = (ch * 16 + i < n_fit) ? v : 0u;      // clipped positions (and lanes past the end) are +0
                if (i & 1) r8[i >> 1] |= v << 16; else r8[i >> 1] = v;
            }
            __syncwarp();                                  // the previous tile has been read
            sts_v4(my_row + swz, r8[0], r8[1], r8[2], r8[3]);
            sts_v4(my_row + (swz ^ 16u), r8[4], r8[5], r8[6], r8[7]);
            uint32_t mine = static_cast<uint32_t>((ch < 4 ? pads_lo : pads_hi) >> ((ch & 3) * 16)) & 0xffffu;
            while (mine) {                                 // ascending: a later pad overrides an earlier one
                const int j = __ffs(static_cast<int>(mine)) - 1;
                mine &= mine - 1;
                const uint32_t f = read_pad(ws, j);
                const uint32_t byte = (f & 15u) * 2;
                asm volatile("st.shared.u16 [%0], %1;" ::"r"(my_row + ((byte & 16u) ^ swz) + (byte & 15u)),
                             "h"(static_cast<unsigned short>(f2h_bits(fp8_to_float(f >> 7) * T))) : "memory");
            }
            __syncwarp();                                  // tile complete
            uint32_t a[2][4];
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const uint32_t tok = (lane >> 4) * 8 + (lane & 7u) + 16 * ks, half = (lane >> 3) & 1u;
                ldmatrix_x4_trans(a[ks], stage + tok * 32 + ((half ^ ((tok >> 2) & 1u)) << 4));
            }
            // ch is uniform but not a compile-time constant: pick the accumulator set by uniform branches so
            // that it stays in registers
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (ch == k) {
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        mma_16816(acc[k], a[ks], p_hi[2 * ks], p_hi[2 * ks + 1]);
                        mma_16816(acc[k], a[ks], p_lo[2 * ks], p_lo[2 * ks + 1]);
                    }
                }
            }
        }
    }
    if (cur_bh >= 0) flush(cur_bh);
}

// ---------------------------------------------------------------------------------------------
// K2m / K3m: the fused consumers for 3 to 8 dot products per group (rows of x, query heads) on the
// tensor cores.  With eight products per weight the scalar path spends four shared-memory
// wavefronts and eight FMAs per symbol on the vector operand alone.  Here a group is decoded in
// two passes as in K5 (indices first; then per 16 values: map, stage a [32 rows][16 k] fp16 tile,
// patch its outliers) and each tile is contracted against the fp16 vector fragments, which stay
// in registers for the whole group: C[32 rows][8] += tile[32 x 16] * V[16 x 8], two
// mma.m16n8k16 per tile, fp32 accumulate (fp16 x fp16 products are exact in fp32).  A warp is
// independent of the others: no vector slice in shared memory, no block barrier.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kMmaWarpBytes = kBitsBytes + kTabBytes + kSymsBytes + 1024;

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]) : "r"(addr));
}

// Position i (0..15) of a 16-value chunk is staged in tile column 2q + (j & 1) + 8 (j >> 1) with i = 4q + j.  The
// contraction index of an MMA may be permuted freely as long as both operands agree, and with this
// order the four vector elements a lane needs per chunk (columns 2q, 2q+1, 2q+8, 2q+9) are the
// contiguous k = 4q .. 4q+3: one 8-byte load instead of two 4-byte ones.
__host__ __device__ constexpr int tile_column(int i) { return 2 * (i >> 2) + (i & 1) + 8 * ((i >> 1) & 1); }

// vfrag[2c], vfrag[2c+1]: B fragments of chunk c (tile columns (lane%4)*2 + {0,1}, and + 8), vector lane/4
// acc[0] / acc[1]: C fragments of rows 0..15 / 16..31 of the warp's 32 groups
__device__ __forceinline__ void row_dot_mma(const Block& blk, uint32_t smem_base, const WarpSmem& ws, uint32_t stage, float T,
                                            bool valid, const uint32_t (&vfrag)[16], float (&acc)[2][4])
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t swz = ((lane >> 2) & 1u) << 4, my_row = stage + lane * 32;
    const GroupHeader h = open_group<false>(blk, smem_base, ws, T);
    uint32_t packed = 0;
    int n_fit = kGroup;
    const uint32_t end = decode_symbols<false, 16, kBlockBits, 0, kFusedFree>(h, ws, [&](int n, uint32_t, uint32_t sym, bool alive) {
        if (!alive) n_fit = min(n_fit, n);
        packed |= sym << ((n & 7) * 4);
        if ((n & 7) == 7) { sts_u32(ws.syms + (n >> 3) * 128, packed); packed = 0; }
    });
    if (!valid) n_fit = 0;                                 // rows past the end contribute zeros
    const int n_pad = (end && valid) ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
    uint64_t pads_lo = 0, pads_hi = 0;                     // 16 bits per chunk: which pads fall into it
    for (int j = 0; j < n_pad; ++j) {
        const uint32_t ch = (read_pad(ws, j) & 127u) >> 4;
        const uint64_t bit = 1ull << ((ch & 3u) * 16 + j);
        if (ch < 4) pads_lo |= bit; else pads_hi |= bit;
    }
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
        uint32_t r8[8];
        const uint32_t w0 = lds_u32(ws.syms + (2 * ch) * 128), w1 = lds_u32(ws.syms + (2 * ch + 1) * 128);
        const bool whole = ch * 16 + 16 <= n_fit;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t sym = ((i < 8 ? w0 : w1) >> ((i & 7) * 4)) & 15u;
            uint32_t v = lds_u32(ws.tab + sym * 128);
            if (!whole) v = (ch * 16 + i < n_fit) ? v : 0u;
            const int col = tile_column(i);                // see load_vfrag
            if (col & 1) r8[col >> 1] |= v << 16; else r8[col >> 1] = v;
        }
        __syncwarp();                                      // the previous tile has been read
        sts_v4(my_row + swz, r8[0], r8[1], r8[2], r8[3]);
        sts_v4(my_row + (swz ^ 16u), r8[4], r8[5], r8[6], r8[7]);
        uint32_t mine = static_cast<uint32_t>((ch < 4 ? pads_lo : pads_hi) >> ((ch & 3) * 16)) & 0xffffu;
        while (mine) {                                     // ascending: a later pad overrides an earlier one
            const int j = __ffs(static_cast<int>(mine)) - 1;
            mine &= mine - 1;
            const uint32_t f = read_pad(ws, j);
            const uint32_t byte = static_cast<uint32_t>(tile_column(static_cast<int>(f & 15u))) * 2;
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(my_row + ((byte & 16u) ^ swz) + (byte & 15u)),
                         "h"(static_cast<unsigned short>(f2h_bits(fp8_to_float(f >> 7) * T))) : "memory");
        }
        __syncwarp();                                      // tile complete
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const uint32_t row = ((lane >> 3) & 1u) * 8 + (lane & 7u) + 16 * mt, half = lane >> 4;
            uint32_t a[4];
            ldmatrix_x4(a, stage + row * 32 + ((half ^ ((row >> 2) & 1u)) << 4));
            mma_16816(acc[mt], a, vfrag[2 * ch], vfrag[2 * ch + 1]);
        }
    }
}

// fragments of eight fp16 vectors v[col][k0 .. k0+127] (col = lane/4; columns >= n_cols are zero)
__device__ __forceinline__ void load_vfrag(uint32_t (&vfrag)[16], const __half* base, size_t col_stride, int n_cols)
{
    const int lane = static_cast<int>(threadIdx.x & 31u), col = lane >> 2;
    const uint2* p = reinterpret_cast<const uint2*>(base + static_cast<size_t>(min(col, n_cols - 1)) * col_stride) + (lane & 3);
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const uint2 v = col < n_cols ? __ldg(p + c * 4) : make_uint2(0u, 0u);     // k = 16c + 4 (lane%4) .. + 3
        vfrag[2 * c] = v.x;                                // tile columns 2q, 2q+1
        vfrag[2 * c + 1] = v.y;                            // tile columns 2q+8, 2q+9
    }
}

// K2m: y[b][n] = sum_k W~[n][k] x[b][k] for 3..8 rows of x.  Units, ownership and the slot-and-ticket
// reduction are those of the per-warp kernel (unit = 32 rows x one k-block).
template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_gemv_mma_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_blocks, int n_out, int kblocks,
                     const __half* __restrict__ d_x, int batch, float* __restrict__ d_y, float* __restrict__ d_partial,
                     unsigned int* __restrict__ d_tickets, int active_warps)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    const uint32_t smem_base = smem_u32(smem);
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    WarpSmem ws;
    ws.bits = smem_base + kSmemWarpBase + warp * kMmaWarpBytes + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = ws.tab + kTabBytes;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);
    const uint32_t stage = smem_base + kSmemWarpBase + warp * kMmaWarpBytes + kBitsBytes + kTabBytes + kSymsBytes;

    const int wg = warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x);
    const int tiles = (n_out + 31) / 32;
    const int64_t U = static_cast<int64_t>(tiles) * kblocks;
    const int W = active_warps;
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    const int k = kblocks * kGroup;
    auto block_ptr = [&](int64_t u) {
        const int row = min(static_cast<int>(u / kblocks) * 32 + lane, n_out - 1);
        return d_blocks + (static_cast<uint64_t>(row) * kblocks + static_cast<int>(u % kblocks)) * kBlockBytes;
    };
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    issue_tables(smem, d_meta, &bar);
    Block blk;
    uint32_t vnext[16];
    if (u0 < u1) { ldg_block(blk, block_ptr(u0)); load_vfrag(vnext, d_x + static_cast<int>(u0 % kblocks) * kGroup, k, batch); }
    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    // C fragment element (mt, i): row = 16 mt + lane/4 + 8 (i >= 2), column b = (lane%4)*2 + (i & 1)
    auto flush = [&](int tile) {
        const int w_lo = unit_owner(U, W, static_cast<int64_t>(tile) * kblocks);
        const int w_hi = unit_owner(U, W, static_cast<int64_t>(tile + 1) * kblocks - 1);
        float* mine = d_partial + static_cast<size_t>(wg + tile) * 8 * 32;
        if (w_lo != w_hi) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    mine[((lane & 3) * 2 + (i & 1)) * 32 + 16 * mt + (lane >> 2) + (i >= 2 ? 8 : 0)] = acc[mt][i];
            __threadfence();
            __syncwarp();
            unsigned int t = 0;
            if (lane == 0) t = atomicAdd(&d_tickets[tile], 1u);
            t = __shfl_sync(0xffffffffu, t, 0);
            if (t != static_cast<unsigned int>(w_hi - w_lo)) return;
            __threadfence();
        }
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = 16 * mt + (lane >> 2) + (i >= 2 ? 8 : 0), b = (lane & 3) * 2 + (i & 1);
                const int row = tile * 32 + r;
                float sum = acc[mt][i];
                if (w_lo != w_hi) {                        // slots in warp order, whatever the arrival order
                    sum = 0.0f;
                    for (int ww = w_lo; ww <= w_hi; ++ww) sum += __ldcg(d_partial + (static_cast<size_t>(ww + tile) * 8 + b) * 32 + r);
                }
                if (row < n_out && b < batch) d_y[static_cast<size_t>(b) * n_out + row] = sum;
            }
        if (w_lo != w_hi && lane == 0) d_tickets[tile] = 0;
    };

    int cur_tile = static_cast<int>(u0 / kblocks);
    for (int64_t u = u0; u < u1; ++u) {
        const int tile = static_cast<int>(u / kblocks);
        if (tile != cur_tile) {
            flush(cur_tile);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;
            cur_tile = tile;
        }
        const Block cur = blk;
        uint32_t vfrag[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) vfrag[i] = vnext[i];
        if (u + 1 < u1) { ldg_block(blk, block_ptr(u + 1)); load_vfrag(vnext, d_x + static_cast<int>((u + 1) % kblocks) * kGroup, k, batch); }
        row_dot_mma(cur, smem_base, ws, stage, T, tile * 32 + lane < n_out, vfrag, acc);
    }
    if (u0 < u1) flush(cur_tile);
}

// K3m: scores[b][hq][t] = scale * q[b][hq] . K~[b][hq / q_per_kv][t] for 3..8 query heads per KV head.
// Unit = (one (batch, kv head), 32 tokens); every working warp owns a contiguous run of units.
template <int kWarps>
__global__ void __launch_bounds__(kWarps * 32, 1)
ecco_attn_scores_mma_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_kblocks, int heads, int seq,
                            int q_per_kv, const __half* __restrict__ d_q, float scale, float* __restrict__ d_scores,
                            int active_warps)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bar;
    const uint32_t smem_base = smem_u32(smem);
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    WarpSmem ws;
    ws.bits = smem_base + kSmemWarpBase + warp * kMmaWarpBytes + lane * 4;
    ws.tab = ws.bits + kBitsBytes;
    ws.syms = ws.tab + kTabBytes;
    sts_u32(ws.bits + 16 * 128, 0u);
    sts_u32(ws.bits + 17 * 128, 0u);
    const uint32_t stage = smem_base + kSmemWarpBase + warp * kMmaWarpBytes + kBitsBytes + kTabBytes + kSymsBytes;

    const int wg = warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x);
    const int tiles = (seq + 31) / 32;
    const int64_t U = static_cast<int64_t>(heads) * tiles;
    const int W = active_warps;
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    auto block_ptr = [&](int64_t u) {
        const int bh = static_cast<int>(u / tiles), t = min(static_cast<int>(u % tiles) * 32 + lane, seq - 1);
        return d_kblocks + (static_cast<uint64_t>(bh) * seq + t) * kBlockBytes;
    };
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    issue_tables(smem, d_meta, &bar);
    Block blk;
    if (u0 < u1) ldg_block(blk, block_ptr(u0));
    if (!wait_tables(&bar)) return;
    const float T = reinterpret_cast<const DevHeader*>(d_meta)->T;

    uint32_t vfrag[16];
    int cur_bh = -1;
    for (int64_t u = u0; u < u1; ++u) {
        const int bh = static_cast<int>(u / tiles), t0 = static_cast<int>(u % tiles) * 32;
        if (bh != cur_bh) { load_vfrag(vfrag, d_q + static_cast<size_t>(bh) * q_per_kv * kGroup, kGroup, q_per_kv); cur_bh = bh; }
        const Block cur = blk;
        if (u + 1 < u1) ldg_block(blk, block_ptr(u + 1));
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        row_dot_mma(cur, smem_base, ws, stage, T, t0 + lane < seq, vfrag, acc);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = t0 + 16 * mt + (lane >> 2) + (i >= 2 ? 8 : 0), r = (lane & 3) * 2 + (i & 1);
                if (t < seq && r < q_per_kv) d_scores[(static_cast<size_t>(bh) * q_per_kv + r) * seq + t] = scale * acc[mt][i];
            }
    }
}

// ---------------------------------------------------------------------------------------------
// host-side launch helpers
// ---------------------------------------------------------------------------------------------
// number of working warps <= w_max such that `units` split evenly: all get ceil(units / w_max) or one less
inline uint32_t balanced_warps(uint64_t units, uint32_t w_max)
{
    if (units <= w_max) return static_cast<uint32_t>(units);
    const uint64_t per_warp = (units + w_max - 1) / w_max;
    return static_cast<uint32_t>((units + per_warp - 1) / per_warp);
}

struct DeviceInfo {
    int device = -1, sms = 0, cc_major = 0;
    bool ok = false;
};

int device_info(DeviceInfo* out)
{
    static thread_local DeviceInfo cache[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return ECCO_ERR_INVALID_ARG;
    DeviceInfo& c = cache[dev];
    if (!c.ok) {
        cudaDeviceProp prop;
        e = cudaGetDeviceProperties(&prop, dev);
        if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
        c.device = dev; c.sms = prop.multiProcessorCount; c.cc_major = prop.major; c.ok = true;
    }
    *out = c;
    return c.cc_major == 10 ? ECCO_OK : ECCO_ERR_UNSUPPORTED_ARCH;
}

int check_launch();
// Launch with the programmatic stream-serialisation attribute (see dependency_wait in the kernels):
// the kernel must call dependency_wait() before its first access to global memory.
template <class... Params, class... Args>
int launch_overlapped(void (*kernel)(Params...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    return check_launch();
}

// Zeroes the ticket words of a workspace.  A kernel rather than a memset so that it can sit in a chain of
// overlapped launches: it lets its successor start at once and clears only after its predecessor (which may
// still be using the same workspace) has completed.
__global__ void ecco_zero_words_kernel(unsigned int* __restrict__ p, size_t n)
{
    release_dependents();
    dependency_wait();
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n; i += static_cast<size_t>(gridDim.x) * blockDim.x) p[i] = 0u;
}
inline int zero_tickets(unsigned int* tickets, size_t bytes, cudaStream_t stream)
{
    const size_t n = bytes / sizeof(unsigned int);
    if (n == 0) return ECCO_OK;
    const unsigned grid = static_cast<unsigned>(n < 8192 ? (n + 255) / 256 : 32);
    return launch_overlapped(ecco_zero_words_kernel, grid, 256u, 0, stream, tickets, n);
}

template <class K>
int set_smem(K kernel, size_t bytes)
{
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    return ECCO_OK;
}

int check_launch()
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ECCO_OK;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr int kDecompressWarps = 32;
// warps per CTA of the scalar fused kernels (one or two dot products per group): as many as shared memory allows
constexpr int fused_warps(int) { return 22; }
// per-warp GEMV: every warp also carries its own slice of x, which leaves room for 22 / 20 warps
constexpr int gemv_warp_warps(int kV) { return kFusedRank ? (kV >= 2 ? 20 : 21) : (kV >= 2 ? 20 : 22); }

struct GemvPlan { int row_tiles, grid; size_t partial_bytes, ticket_bytes; };

// plan of the per-warp GEMV (one or two rows of x)
GemvPlan gemv_warp_plan(int n_out, int kblocks, int vpad, int ctas_max)
{
    GemvPlan p;
    p.row_tiles = (n_out + 31) / 32;
    const int64_t units = static_cast<int64_t>(p.row_tiles) * kblocks;
    const int64_t ctas = (units + gemv_warp_warps(vpad) - 1) / gemv_warp_warps(vpad);
    p.grid = static_cast<int>(ctas < ctas_max ? ctas : ctas_max);
    p.partial_bytes = static_cast<size_t>(p.grid * gemv_warp_warps(vpad) + p.row_tiles) * vpad * 32 * sizeof(float);
    p.partial_bytes = (p.partial_bytes + 255) & ~static_cast<size_t>(255);
    p.ticket_bytes = (static_cast<size_t>(p.row_tiles) * sizeof(unsigned int) + 255) & ~static_cast<size_t>(255);
    return p;
}

constexpr int kMmaWarps = 20;

// plan of the tensor-core GEMV (3..8 rows of x): units and slots as in the per-warp kernel, eight columns
GemvPlan gemv_mma_plan(int n_out, int kblocks, int ctas_max)
{
    GemvPlan p;
    p.row_tiles = (n_out + 31) / 32;
    const int64_t units = static_cast<int64_t>(p.row_tiles) * kblocks;
    const int64_t ctas = (units + kMmaWarps - 1) / kMmaWarps;
    p.grid = static_cast<int>(ctas < ctas_max ? ctas : ctas_max);
    p.partial_bytes = (static_cast<size_t>(p.grid * kMmaWarps + p.row_tiles) * 8 * 32 * sizeof(float) + 255) & ~static_cast<size_t>(255);
    p.ticket_bytes = (static_cast<size_t>(p.row_tiles) * sizeof(unsigned int) + 255) & ~static_cast<size_t>(255);
    return p;
}

inline int pad_v(int v) { return v <= 1 ? 1 : v <= 2 ? 2 : v <= 4 ? 4 : 8; }

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------
extern "C" int ecco_last_cuda_error(void) { return t_last_cuda_error; }
extern "C" uint64_t ecco_kernel_launch_count(void) { return g_launches.load(); }

extern "C" int ecco_device_status(void)
{
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    int st = 0, zero = 0;
    e = cudaMemcpyFromSymbol(&st, g_device_status, sizeof st);
    if (e == cudaSuccess && st) e = cudaMemcpyToSymbol(g_device_status, &zero, sizeof zero);
    if (e != cudaSuccess) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
    return st;
}

// cuTensorMapEncodeTiled through the runtime's driver entry point query (no link against libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn()
{
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// tensor map of the output seen as [n_groups][128] fp16, box = 32 rows x 16 values, 32-byte swizzle
static bool make_out_map(CUtensorMap* map, void* d_out, uint64_t n_groups)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {kGroup, n_groups};
    const cuuint64_t strides[1] = {kGroup * 2};
    const cuuint32_t box[2] = {16, 32};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, d_out, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_32B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kDecompressTmaWarps = 28;
// symbols 1 and 3 of every four are decoded arithmetically, 0 and 2 through the byte table: measured best of
// {none, one, two, three, all} on the 11008x4096 matrix and on a 256 MiB cache (all-table 441 us, this 394 us, all-arithmetic 459 us)
constexpr uint32_t kDecompressArith = 0b1010;

// tensors of fewer than 32 groups (the tile store's box is 32 rows tall), or when no tensor map can be made
static int launch_decompress_small(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, void* d_out,
                                   cudaStream_t stream)
{
    static thread_local bool configured[64] = {};
    auto kernel = ecco_decompress_kernel<kDecompressWarps>;
    const size_t smem = kSmemWarpBase + static_cast<size_t>(kDecompressWarps) * (kBitsBytes + kTabBytes);
    if (!configured[di.device]) {
        int rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    const uint64_t cta_tiles = (n_groups + kDecompressWarps * 32 - 1) / (kDecompressWarps * 32);   // one tile per warp
    const unsigned grid = static_cast<unsigned>(cta_tiles < static_cast<uint64_t>(di.sms) ? cta_tiles : di.sms);
    kernel<<<grid, kDecompressWarps * 32, smem, stream>>>(static_cast<const uint8_t*>(d_meta), d_blocks, n_groups,
                                                          static_cast<uint16_t*>(d_out),
                                                          balanced_warps((n_groups + 31) / 32, grid * kDecompressWarps));
    return check_launch();
}

// one launch of the tile-store kernel over batch.n tensors (maps already made)
static int launch_decompress_batch(const DeviceInfo& di, DecompressBatch& batch, cudaStream_t stream)
{
    static thread_local bool configured[64] = {};
    auto kernel = ecco_decompress_tma_kernel<kDecompressTmaWarps, kDecompressArith>;
    constexpr size_t smem =
        ((kSmemRankWarpBase + static_cast<size_t>(kDecompressTmaWarps) * (kBitsBytes + kTabBytes) + 1023) & ~static_cast<size_t>(1023)) +
        static_cast<size_t>(kDecompressTmaWarps) * 1024 + 512 + 16;           // + outlier value table + barrier
    static_assert(smem <= 232448, "227 KB per CTA");
    if (!configured[di.device]) {
        int rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    uint64_t cta_tiles = 0;
    for (int t = 0; t < batch.n; ++t) {
        const uint64_t c = (batch.job[t].n_groups + kDecompressTmaWarps * 32 - 1) / (kDecompressTmaWarps * 32);
        cta_tiles = c > cta_tiles ? c : cta_tiles;
    }
    const unsigned grid = static_cast<unsigned>(cta_tiles < static_cast<uint64_t>(di.sms) ? cta_tiles : di.sms);
    for (int t = 0; t < batch.n; ++t)
        batch.job[t].active_warps = balanced_warps((batch.job[t].n_groups + 31) / 32, grid * kDecompressTmaWarps);
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kDecompressTmaWarps * 32), smem, stream, batch);
}

static int check_decompress_args(const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, const void* d_out)
{
    if (!d_meta || !d_blocks || !d_out) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_blocks) || !aligned16(d_out)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > (1ull << 40)) return ECCO_ERR_INVALID_ARG;
    return ECCO_OK;
}

extern "C" int ecco_decompress_batch(const ecco_decompress_item* items, int32_t n_items, void* stream)
{
    if (n_items < 0 || (n_items > 0 && !items)) return ECCO_ERR_INVALID_ARG;
    for (int i = 0; i < n_items; ++i) {                    // nothing is launched unless every item is acceptable
        if (items[i].n_groups == 0) continue;
        const int rc = check_decompress_args(items[i].d_meta, items[i].d_blocks, items[i].n_groups, items[i].d_out_fp16);
        if (rc) return rc;
    }
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DecompressBatch batch;
    std::memset(&batch, 0, sizeof batch);
    for (int i = 0; i < n_items; ++i) {
        const ecco_decompress_item& it = items[i];
        if (it.n_groups == 0) continue;
        DecompressJob& job = batch.job[batch.n];
        if (it.n_groups >= 32 && make_out_map(&job.map, it.d_out_fp16, it.n_groups)) {
            job.meta = static_cast<const uint8_t*>(it.d_meta);
            job.blocks = it.d_blocks;
            job.n_groups = it.n_groups;
            job.out = static_cast<uint16_t*>(it.d_out_fp16);
            if (++batch.n == kMaxJobs) {
                rc = launch_decompress_batch(di, batch, s);
                if (rc) return rc;
                batch.n = 0;
            }
        } else {                                           // items keep their order in the stream
            if (batch.n) {
                rc = launch_decompress_batch(di, batch, s);
                if (rc) return rc;
                batch.n = 0;
            }
            rc = launch_decompress_small(di, it.d_meta, it.d_blocks, it.n_groups, it.d_out_fp16, s);
            if (rc) return rc;
        }
    }
    return batch.n ? launch_decompress_batch(di, batch, s) : ECCO_OK;
}

extern "C" int ecco_decompress(const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, void* d_out, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    const ecco_decompress_item item = {d_meta, d_blocks, n_groups, d_out};
    return ecco_decompress_batch(&item, 1, stream);
}

constexpr int kVarWarps = 18;

extern "C" int ecco_var_decompress(const void* d_meta, const uint8_t* d_stream, const void* d_index, uint64_t n_groups, void* d_out,
                                   void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_meta || !d_stream || !d_index || !d_out) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_stream) || !aligned16(d_out) || (reinterpret_cast<uintptr_t>(d_index) & 7u)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > (1ull << 40)) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    // the tile store needs 32 rows: pad the logical row count of tiny tensors is not possible, so they are refused
    CUtensorMap map;
    if (!make_out_map(&map, d_out, n_groups)) return ECCO_ERR_CUDA;
    auto kernel = ecco_var_decompress_kernel<kVarWarps>;
    constexpr size_t smem =
        ((kSmemWarpBase + static_cast<size_t>(kVarWarps) * (kVarBitsBytes + kTabBytes) + 1023) & ~static_cast<size_t>(1023)) +
        static_cast<size_t>(kVarWarps) * 1024;
    static thread_local bool configured[64] = {};
    if (!configured[di.device]) {
        rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    const uint64_t cta_tiles = (n_groups + kVarWarps * 32 - 1) / (kVarWarps * 32);
    const unsigned grid = static_cast<unsigned>(cta_tiles < static_cast<uint64_t>(di.sms) ? cta_tiles : di.sms);
    const uint32_t active = balanced_warps((n_groups + 31) / 32, grid * kVarWarps);
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kVarWarps * 32), smem, static_cast<cudaStream_t>(stream),
                             static_cast<const uint8_t*>(d_meta), reinterpret_cast<const uint4*>(d_stream),
                             static_cast<const uint64_t*>(d_index), n_groups, static_cast<uint16_t*>(d_out), active, map);
}

extern "C" size_t ecco_gemv_workspace_bytes(int32_t n_out, int32_t k, int32_t batch)
{
    if (n_out <= 0 || k <= 0 || k % kGroup || batch < 1 || batch > ECCO_MAX_BATCH) return 0;
    // sized for the largest plan any supported device can ask for (at most 256 persistent CTAs)
    const GemvPlan p = pad_v(batch) <= 2 ? gemv_warp_plan(n_out, k / kGroup, pad_v(batch), 256) : gemv_mma_plan(n_out, k / kGroup, 256);
    return p.partial_bytes + p.ticket_bytes;
}

// three to eight rows of x: the tensor-core kernel
static int launch_gemv_mma(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, int n_out, int kblocks,
                           const void* d_x, int batch, float* d_y, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    auto kernel = ecco_gemv_mma_kernel<kMmaWarps>;
    const size_t smem = kSmemWarpBase + static_cast<size_t>(kMmaWarps) * kMmaWarpBytes;
    static thread_local bool configured[64] = {};
    if (!configured[di.device]) {
        int rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    const GemvPlan p = gemv_mma_plan(n_out, kblocks, di.sms < 256 ? di.sms : 256);
    if (!d_ws || !aligned16(d_ws)) return d_ws ? ECCO_ERR_ALIGNMENT : ECCO_ERR_WORKSPACE;
    if (ws_bytes < p.partial_bytes + p.ticket_bytes) return ECCO_ERR_WORKSPACE;
    float* partial = static_cast<float*>(d_ws);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(d_ws) + p.partial_bytes);
    int rc = zero_tickets(tickets, p.ticket_bytes, stream);
    if (rc) return rc;
    const int active = static_cast<int>(balanced_warps(static_cast<uint64_t>(p.row_tiles) * kblocks, p.grid * kMmaWarps));
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kMmaWarps * 32), smem, stream,
                             static_cast<const uint8_t*>(d_meta), d_blocks, n_out, kblocks, static_cast<const __half*>(d_x), batch, d_y,
                             partial, tickets, active);
}

// one or two rows of x (batch == kV): the per-warp kernel
template <int kV>
static int launch_gemv_warp(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, int n_out, int kblocks,
                            const void* d_x, float* d_y, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    constexpr int kFusedWarps = gemv_warp_warps(kV);
    auto kernel = ecco_gemv_warp_kernel<kV, kFusedWarps>;
    const size_t smem = kFusedBase + static_cast<size_t>(kFusedWarps) * (kBitsBytes + kTabBytes + kSymsBytes + kGroup * kV * 4);
    static thread_local bool configured[64] = {};
    if (!configured[di.device]) {
        int rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    const GemvPlan p = gemv_warp_plan(n_out, kblocks, kV, di.sms < 256 ? di.sms : 256);
    if (!d_ws || !aligned16(d_ws)) return d_ws ? ECCO_ERR_ALIGNMENT : ECCO_ERR_WORKSPACE;
    if (ws_bytes < p.partial_bytes + p.ticket_bytes) return ECCO_ERR_WORKSPACE;
    float* partial = static_cast<float*>(d_ws);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(d_ws) + p.partial_bytes);
    int rc = zero_tickets(tickets, p.ticket_bytes, stream);
    if (rc) return rc;
    const int active = static_cast<int>(balanced_warps(static_cast<uint64_t>(p.row_tiles) * kblocks, p.grid * kFusedWarps));
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kFusedWarps * 32), smem, stream,
                             static_cast<const uint8_t*>(d_meta), d_blocks, n_out, kblocks, static_cast<const __half*>(d_x), d_y, partial,
                             tickets, active);
}

extern "C" int ecco_gemv(const void* d_meta, const uint8_t* d_blocks, int32_t n_out, int32_t k, const void* d_x,
                         int32_t batch, float* d_y, void* d_workspace, size_t workspace_bytes, void* stream)
{
    if (!d_meta || !d_blocks || !d_x || !d_y) return ECCO_ERR_INVALID_ARG;
    if (n_out <= 0 || k <= 0 || k % kGroup || batch < 1 || batch > ECCO_MAX_BATCH) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_blocks) || !aligned16(d_x) || !aligned16(d_y)) return ECCO_ERR_ALIGNMENT;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int kblocks = k / kGroup;
    switch (pad_v(batch)) {
        case 1: return launch_gemv_warp<1>(di, d_meta, d_blocks, n_out, kblocks, d_x, d_y, d_workspace, workspace_bytes, s);
        case 2: return launch_gemv_warp<2>(di, d_meta, d_blocks, n_out, kblocks, d_x, d_y, d_workspace, workspace_bytes, s);
        default: return launch_gemv_mma(di, d_meta, d_blocks, n_out, kblocks, d_x, batch, d_y, d_workspace, workspace_bytes, s);
    }
}

// ---------------------------------------------------------------------------------------------
// ecco_gemv_static_ws: ecco_gemv for callers that cannot allocate.  The split-k scratch is this
// fixed array in the library's device image.  In host code the name below is only a handle for
// the runtime, not a device address: the address comes from cudaGetSymbolAddress, once per
// device, and that pointer is what the kernel receives.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[ECCO_STATIC_WORKSPACE_BYTES];

extern "C" int ecco_gemv_static_ws(const void* d_meta, const uint8_t* d_blocks, int32_t n_out, int32_t k, const void* d_x,
                                   int32_t batch, float* d_y, void* stream)
{
    if (!d_meta || !d_blocks || !d_x || !d_y) return ECCO_ERR_INVALID_ARG;
    if (n_out <= 0 || k <= 0 || k % kGroup || batch < 1 || batch > ECCO_MAX_BATCH) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_blocks) || !aligned16(d_x) || !aligned16(d_y)) return ECCO_ERR_ALIGNMENT;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const int kblocks = k / kGroup, vpad = pad_v(batch);
    // refuse, before any launch, a shape whose plan does not fit the fixed array
    const int ctas = di.sms < 256 ? di.sms : 256;
    const GemvPlan p = vpad <= 2 ? gemv_warp_plan(n_out, kblocks, vpad, ctas) : gemv_mma_plan(n_out, kblocks, ctas);
    if (p.partial_bytes + p.ticket_bytes > ECCO_STATIC_WORKSPACE_BYTES) return ECCO_ERR_WORKSPACE;
    // one-time set-up per device (the current device is di.device): resolve the array's address
    static std::mutex mu;
    static void* address[64] = {};
    void* ws = nullptr;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!address[di.device]) {
            void* ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_workspace);
            if (e != cudaSuccess || !ptr) { t_last_cuda_error = static_cast<int>(e); return ECCO_ERR_CUDA; }
            address[di.device] = ptr;
        }
        ws = address[di.device];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (vpad) {
        case 1: return launch_gemv_warp<1>(di, d_meta, d_blocks, n_out, kblocks, d_x, d_y, ws, ECCO_STATIC_WORKSPACE_BYTES, s);
        case 2: return launch_gemv_warp<2>(di, d_meta, d_blocks, n_out, kblocks, d_x, d_y, ws, ECCO_STATIC_WORKSPACE_BYTES, s);
        default: return launch_gemv_mma(di, d_meta, d_blocks, n_out, kblocks, d_x, batch, d_y, ws, ECCO_STATIC_WORKSPACE_BYTES, s);
    }
}

template <int kV>
static int launch_attn(const DeviceInfo& di, const void* d_meta, const uint8_t* d_kblocks, int batch, int n_kv_heads,
                       int seq, int q_per_kv, const void* d_q, float scale, float* d_scores, cudaStream_t stream)
{
    constexpr int kFusedWarps = fused_warps(kV), kFusedRows = kFusedWarps * 32;
    auto kernel = ecco_attn_scores_kernel<kV, kFusedWarps>;
    const size_t smem = kFusedBase + static_cast<size_t>(kFusedWarps) * (kBitsBytes + kTabBytes + kSymsBytes) + kGroup * kV * 4;
    static thread_local bool configured[64] = {};
    if (!configured[di.device]) {
        int rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    const int heads = batch * n_kv_heads;
    const int64_t units = static_cast<int64_t>(heads) * ((seq + kFusedRows - 1) / kFusedRows);
    const unsigned grid = balanced_warps(static_cast<uint64_t>(units), static_cast<uint32_t>(di.sms));   // persistent CTAs, same units each
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kFusedWarps * 32), smem, stream, static_cast<const uint8_t*>(d_meta),
                             d_kblocks, heads, seq, q_per_kv, static_cast<const __half*>(d_q), scale, d_scores);
}

extern "C" int ecco_attn_scores(const void* d_meta, const uint8_t* d_kblocks, int32_t batch, int32_t n_kv_heads, int32_t seq,
                                int32_t q_per_kv, const void* d_q, float scale, float* d_scores, void* stream)
{
    if (batch == 0 || n_kv_heads == 0 || seq == 0) return (batch < 0 || n_kv_heads < 0 || seq < 0) ? ECCO_ERR_INVALID_ARG : ECCO_OK;
    if (!d_meta || !d_kblocks || !d_q || !d_scores) return ECCO_ERR_INVALID_ARG;
    if (batch < 0 || n_kv_heads < 0 || seq < 0 || q_per_kv < 1 || q_per_kv > 8) return ECCO_ERR_INVALID_ARG;
    if (static_cast<int64_t>(batch) * n_kv_heads > (1 << 24)) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_kblocks) || !aligned16(d_q) || !aligned16(d_scores)) return ECCO_ERR_ALIGNMENT;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (pad_v(q_per_kv)) {
        case 1: return launch_attn<1>(di, d_meta, d_kblocks, batch, n_kv_heads, seq, q_per_kv, d_q, scale, d_scores, s);
        case 2: return launch_attn<2>(di, d_meta, d_kblocks, batch, n_kv_heads, seq, q_per_kv, d_q, scale, d_scores, s);
        default: {
            auto kernel = ecco_attn_scores_mma_kernel<kMmaWarps>;
            const size_t smem = kSmemWarpBase + static_cast<size_t>(kMmaWarps) * kMmaWarpBytes;
            static thread_local bool configured[64] = {};
            if (!configured[di.device]) {
                rc = set_smem(kernel, smem);
                if (rc) return rc;
                configured[di.device] = true;
            }
            const uint64_t units = static_cast<uint64_t>(batch) * n_kv_heads * ((seq + 31) / 32);
            const uint64_t ctas = (units + kMmaWarps - 1) / kMmaWarps;
            const unsigned grid = static_cast<unsigned>(ctas < static_cast<uint64_t>(di.sms) ? ctas : di.sms);
            const int active = static_cast<int>(balanced_warps(units, grid * kMmaWarps));
            return launch_overlapped(kernel, grid, static_cast<unsigned>(kMmaWarps * 32), smem, s, static_cast<const uint8_t*>(d_meta),
                                     d_kblocks, batch * n_kv_heads, seq, q_per_kv, static_cast<const __half*>(d_q), scale, d_scores, active);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// ecco_attn_values
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kAvWarps = 16;    // 512 tokens per unit: divides the usual sequence lengths
struct AvPlan { int grid; size_t stats_bytes, partial_bytes, ticket_bytes; };
AvPlan av_plan(int batch, int n_kv_heads, int seq, int q_per_kv, int ctas_max)
{
    AvPlan p;
    const int heads = batch * n_kv_heads;
    const int64_t units = static_cast<int64_t>(heads) * ((seq + kAvWarps * 32 - 1) / (kAvWarps * 32));
    p.grid = static_cast<int>(balanced_warps(static_cast<uint64_t>(units), static_cast<uint32_t>(ctas_max)));
    auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
    p.stats_bytes = up(static_cast<size_t>(heads) * q_per_kv * sizeof(float2));
    p.partial_bytes = up(static_cast<size_t>(p.grid + heads) * kGroup * 8 * sizeof(float));
    p.ticket_bytes = up(static_cast<size_t>(heads) * sizeof(unsigned int));
    return p;
}
}  // namespace

extern "C" size_t ecco_attn_values_workspace_bytes(int32_t batch, int32_t n_kv_heads, int32_t seq, int32_t q_per_kv)
{
    if (batch <= 0 || n_kv_heads <= 0 || seq <= 0 || q_per_kv < 1 || q_per_kv > 8) return 0;
    if (static_cast<int64_t>(batch) * n_kv_heads > (1 << 24)) return 0;
    const AvPlan p = av_plan(batch, n_kv_heads, seq, q_per_kv, 256);
    return p.stats_bytes + p.partial_bytes + p.ticket_bytes;
}

extern "C" int ecco_attn_values(const void* d_meta, const uint8_t* d_vblocks, int32_t batch, int32_t n_kv_heads, int32_t seq,
                                int32_t q_per_kv, const float* d_scores, float* d_out, void* d_workspace, size_t workspace_bytes,
                                void* stream)
{
    if (batch == 0 || n_kv_heads == 0) return (batch < 0 || n_kv_heads < 0) ? ECCO_ERR_INVALID_ARG : ECCO_OK;
    if (!d_meta || !d_vblocks || !d_scores || !d_out) return ECCO_ERR_INVALID_ARG;
    if (batch < 0 || n_kv_heads < 0 || seq <= 0 || q_per_kv < 1 || q_per_kv > 8) return ECCO_ERR_INVALID_ARG;
    if (static_cast<int64_t>(batch) * n_kv_heads > (1 << 24)) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_vblocks) || !aligned16(d_scores) || !aligned16(d_out)) return ECCO_ERR_ALIGNMENT;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const AvPlan p = av_plan(batch, n_kv_heads, seq, q_per_kv, di.sms < 256 ? di.sms : 256);
    if (!d_workspace || !aligned16(d_workspace)) return d_workspace ? ECCO_ERR_ALIGNMENT : ECCO_ERR_WORKSPACE;
    if (workspace_bytes < p.stats_bytes + p.partial_bytes + p.ticket_bytes) return ECCO_ERR_WORKSPACE;
    auto kernel = ecco_attn_values_kernel<kAvWarps>;
    const size_t smem = kSmemWarpBase + static_cast<size_t>(kAvWarps) * kAvWarpBytes + kGroup * 8 * sizeof(float);
    static thread_local bool configured[64] = {};
    if (!configured[di.device]) {
        rc = set_smem(kernel, smem);
        if (rc) return rc;
        configured[di.device] = true;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* wsb = static_cast<uint8_t*>(d_workspace);
    float2* stats = reinterpret_cast<float2*>(wsb);
    float* partial = reinterpret_cast<float*>(wsb + p.stats_bytes);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(wsb + p.stats_bytes + p.partial_bytes);
    rc = zero_tickets(tickets, p.ticket_bytes, s);
    if (rc) return rc;
    const int heads = batch * n_kv_heads, rows = heads * q_per_kv;
    rc = launch_overlapped(ecco_softmax_stats_kernel, static_cast<unsigned>((rows + 7) / 8), 256u, 0, s, d_scores, rows, seq, stats);
    if (rc) return rc;
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kAvWarps * 32), smem, s,
                             static_cast<const uint8_t*>(d_meta), d_vblocks, heads, seq, q_per_kv, d_scores, stats, d_out, partial, tickets);
}

// ---------------------------------------------------------------------------------------------
// 2x activation format (Sec. 3.2 "Activation Compression"; Sec. 4.2 / 4.3 low-ratio units):
// 64 fp16 values <-> 64 bytes.  Byte i = 7-bit two's-complement value in bits 0..6 and one bit
// of metadata in bit 7: metadata bits 0..15 = fp16 scale, 16..31 = fp16 zero point, 32..63 = 0.
// Four lanes share a group (16 bytes / 16 values each), so a warp moves 512 B of blocks and
// 1 KB of fp16 per instruction, fully coalesced; both kernels are plain HBM streams.
// ---------------------------------------------------------------------------------------------
namespace {

// bit 7 of the four bytes of w, gathered into bits 0..3
__device__ __forceinline__ uint32_t top_bits(uint32_t w) { return ((w & 0x80808080u) * 0x00204081u) >> 28; }

__global__ void __launch_bounds__(256)
ecco_act_decompress_kernel(const uint4* __restrict__ d_blocks, uint64_t n_chunks, uint4* __restrict__ d_out)
{
    // one chunk = 16 bytes of a block = 16 values; chunk c belongs to group c / 4
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    const uint64_t rounds = (n_chunks + stride - 1) / stride;
    for (uint64_t r = 0, c = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; r < rounds; ++r, c += stride) {
        const bool ok = c < n_chunks;                       // whole warps stay in the loop for the shuffles
        uint4 b = make_uint4(0, 0, 0, 0);
        if (ok) asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(d_blocks + c));
        const uint32_t bits16 = top_bits(b.x) | (top_bits(b.y) << 4) | (top_bits(b.z) << 8) | (top_bits(b.w) << 12);
        const uint32_t lane = threadIdx.x & 31u;
        const uint32_t scale_bits = __shfl_sync(0xffffffffu, bits16, lane & ~3u);          // chunk 0 of the group
        const uint32_t zero_bits = __shfl_sync(0xffffffffu, bits16, (lane & ~3u) | 1u);    // chunk 1
        const float scale = __half2float(__ushort_as_half(static_cast<unsigned short>(scale_bits)));
        const float zero = __half2float(__ushort_as_half(static_cast<unsigned short>(zero_bits)));
        const uint32_t w[4] = {b.x, b.y, b.z, b.w};
        uint32_t o[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int j = 0; j < 4; j += 2) {
                // sign-extend the 7-bit values (shift the value's sign into the byte's sign, arithmetic shift back)
                const int q0 = static_cast<int>(static_cast<int8_t>((w[i] >> (8 * j)) << 1)) >> 1;
                const int q1 = static_cast<int>(static_cast<int8_t>((w[i] >> (8 * j + 8)) << 1)) >> 1;
                const uint32_t h0 = f2h_bits(fmaf(static_cast<float>(q0), scale, zero));
                const uint32_t h1 = f2h_bits(fmaf(static_cast<float>(q1), scale, zero));
                o[i * 2 + j / 2] = h0 | (h1 << 16);
            }
        }
        if (ok) {
            asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(d_out + c * 2), "r"(o[0]), "r"(o[1]), "r"(o[2]),
                         "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                         : "memory");
        }
    }
}

__global__ void __launch_bounds__(256)
ecco_act_compress_kernel(const uint4* __restrict__ d_x, uint64_t n_chunks, uint4* __restrict__ d_blocks)
{
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    const uint64_t rounds = (n_chunks + stride - 1) / stride;
    for (uint64_t r = 0, c = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; r < rounds; ++r, c += stride) {
        const bool ok = c < n_chunks;
        uint32_t h[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (ok)
            asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]), "=r"(h[4]), "=r"(h[5]), "=r"(h[6]), "=r"(h[7])
                         : "l"(d_x + c * 2));
        float x[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const __half2 v = *reinterpret_cast<const __half2*>(&h[i]);
            x[2 * i] = __low2float(v);
            x[2 * i + 1] = __high2float(v);
        }
        float lo = x[0], hi = x[0];
#pragma unroll
        for (int i = 1; i < 16; ++i) { lo = fminf(lo, x[i]); hi = fmaxf(hi, x[i]); }
        // min / max over the four lanes of the group (the compressor's sorter stage, Sec. 4.3)
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 1)); hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, 1));
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, 2)); hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, 2));
        const uint32_t scale16 = f2h_bits(__fdiv_rn(hi - lo, 127.0f));
        const float scale = __half2float(__ushort_as_half(static_cast<unsigned short>(scale16)));
        const uint32_t zero16 = f2h_bits(fmaf(64.0f, scale, lo));      // 64 * scale is exact, so this is lo + 64 * scale rounded once
        const float zero = __half2float(__ushort_as_half(static_cast<unsigned short>(zero16)));
        const bool usable = scale > 0.0f && scale < __int_as_float(0x7f800000);
        const float inv = __fdiv_rn(1.0f, scale);          // multiply-and-round (Sec. 4.3): one division per group
        const uint32_t part = (threadIdx.x & 3u);
        const uint32_t meta16 = part == 0 ? scale16 : part == 1 ? zero16 : 0u;   // this chunk's 16 metadata bits
        uint32_t out[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // clamping before the rounding gives what clamping after it gives (the bounds are integers, rounding is
            // monotone); cvt.rni rounds to nearest even like rintf; two pack instructions make the four bytes
            int q[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float p = fminf(fmaxf(__fmul_rn(x[i * 4 + j] - zero, inv), -64.0f), 63.0f);
                q[j] = usable ? __float2int_rn(p) : 0;
            }
            uint32_t hi16, wv;                             // d = sat(a) << 8 | sat(b) | c << 16
            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi16) : "r"(q[3]), "r"(q[2]), "r"(0));
            asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(wv) : "r"(q[1]), "r"(q[0]), "r"(hi16));
            // bits 4i .. 4i+3 of the metadata go to bit 7 of bytes 0..3
            const uint32_t m4 = (meta16 >> (4 * i)) & 15u;
            out[i] = (wv & 0x7f7f7f7fu) | (((m4 * 0x00204081u) & 0x01010101u) << 7);
        }
        if (ok) d_blocks[c] = make_uint4(out[0], out[1], out[2], out[3]);
    }
}

int act_grid(uint64_t n_chunks, const DeviceInfo& di)
{
    const uint64_t ctas = (n_chunks + 255) / 256;
    const uint64_t cap = static_cast<uint64_t>(di.sms) * 8;           // eight 256-thread CTAs per SM, grid-stride beyond that
    return static_cast<int>(ctas < cap ? ctas : cap);
}

}  // namespace

extern "C" int ecco_act_decompress(const uint8_t* d_blocks, uint64_t n_groups, void* d_out_fp16, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_blocks || !d_out_fp16) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_blocks) || (reinterpret_cast<uintptr_t>(d_out_fp16) & 31u)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > (1ull << 40)) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const uint64_t n_chunks = n_groups * 4;
    ecco_act_decompress_kernel<<<act_grid(n_chunks, di), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        reinterpret_cast<const uint4*>(d_blocks), n_chunks, static_cast<uint4*>(d_out_fp16));
    return check_launch();
}

extern "C" int ecco_act_compress(const void* d_x_fp16, uint64_t n_groups, uint8_t* d_blocks, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_blocks || !d_x_fp16) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_blocks) || (reinterpret_cast<uintptr_t>(d_x_fp16) & 31u)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > (1ull << 40)) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const uint64_t n_chunks = n_groups * 4;
    ecco_act_compress_kernel<<<act_grid(n_chunks, di), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(d_x_fp16), n_chunks, reinterpret_cast<uint4*>(d_blocks));
    return check_launch();
}

// ---------------------------------------------------------------------------------------------
// Online 4x compressor for the KV cache (Sec. 4.3, "High Compression Ratio (4x) Compressor"):
// one warp encodes one group of 128 fp16 values into its 64-byte block, four values per lane.
//   sorter stage      abs-max (first on ties) -> FP8 scale byte; min / max of the normalised rest
//   pattern selector  fitness = (pattern min - group min)^2 + (pattern max - group max)^2, S scores
//                     spread over the lanes, arg-min with ties to the lower id
//   encoders          nearest centroid per value, the four codebooks' total lengths, the shortest
//                     wins (ID_HF); bit positions by a warp prefix sum
//   pack / clip       codewords OR-ed into the block image in shared memory; the first codeword
//                     that crosses bit 512 is truncated and the rest dropped; a complete group is
//                     padded with its next-largest values (15-bit outliers from the tail)
// Every comparison that decides an index is made in the same precision and order as the host
// encoder (fp32 division by the scale, fp64 squared distances, no fused multiply-add), so the
// blocks are byte-identical to ecco_encode_host with ECCO_SELECT_MINMAX | ECCO_KEEP_EXPONENT.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kKvWarps = 8;

__global__ void __launch_bounds__(kKvWarps * 32)
ecco_kv_compress_kernel(const uint8_t* __restrict__ d_meta, const __half* __restrict__ d_x, uint64_t n_groups,
                        uint8_t* __restrict__ d_blocks)
{
    __shared__ __align__(16) uint16_t pat_s[kMaxPatterns * 16];
    __shared__ __align__(16) uint16_t enc_s[kMaxPatterns * kCodebooks * kSymbols];
    __shared__ __align__(16) uint16_t kp_s[kMaxPatterns];
    __shared__ uint32_t blk_s[kKvWarps][16];
    const int tid = static_cast<int>(threadIdx.x), lane = tid & 31, warp = tid >> 5;
    dependency_wait();                                     // the previous kernel of the stream has completed
    release_dependents();
    {
        const uint4* src_p = reinterpret_cast<const uint4*>(d_meta + kOffPattern);
        for (int i = tid; i < static_cast<int>(kPatternBytes / 16); i += kKvWarps * 32) reinterpret_cast<uint4*>(pat_s)[i] = src_p[i];
        const uint4* src_e = reinterpret_cast<const uint4*>(d_meta + kOffEncCb);
        for (int i = tid; i < static_cast<int>(kEncCbBytes / 16); i += kKvWarps * 32) reinterpret_cast<uint4*>(enc_s)[i] = src_e[i];
        const uint4* src_k = reinterpret_cast<const uint4*>(d_meta + kOffEncKp);
        for (int i = tid; i < static_cast<int>(kEncKpBytes / 16); i += kKvWarps * 32) reinterpret_cast<uint4*>(kp_s)[i] = src_k[i];
    }
    __syncthreads();
    const DevHeader* hdr = reinterpret_cast<const DevHeader*>(d_meta);
    const int S = hdr->S;
    const float T = hdr->T, invT = 1.0f / T;             // both exact powers of two
    const unsigned full = 0xffffffffu;
    uint32_t* blk = blk_s[warp];
    auto fp8 = [&](float v) { return static_cast<uint32_t>(__nv_cvt_float_to_fp8(v * invT, __NV_SATFINITE, __NV_E4M3)); };

    for (uint64_t g = static_cast<uint64_t>(blockIdx.x) * kKvWarps + warp; g < n_groups; g += static_cast<uint64_t>(gridDim.x) * kKvWarps) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(d_x + g * kGroup) + lane);
        const uint32_t h16[4] = {raw.x & 0xffffu, raw.x >> 16, raw.y & 0xffffu, raw.y >> 16};
        float x[4];
        uint32_t key[4];                                   // |x| then low index first
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            x[j] = __half2float(__ushort_as_half(static_cast<unsigned short>(h16[j])));
            key[j] = ((h16[j] & 0x7fffu) << 7) | static_cast<uint32_t>(127 - (lane * 4 + j));
        }
        // sorter: abs-max, first index on ties
        const uint32_t best = __reduce_max_sync(full, max(max(key[0], key[1]), max(key[2], key[3])));
        const int pstar = 127 - static_cast<int>(best & 127u);
        const float xsel = (pstar & 3) == 0 ? x[0] : (pstar & 3) == 1 ? x[1] : (pstar & 3) == 2 ? x[2] : x[3];
        const float xp = __shfl_sync(full, xsel, pstar >> 2);
        const uint32_t qs = fp8(xp);
        const float scale = fabsf(fp8_to_float(qs) * T);
        float u[4], lo = INFINITY, hi = -INFINITY;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool is_max = lane * 4 + j == pstar;
            u[j] = (is_max || scale == 0.0f) ? 0.0f : __fdiv_rn(x[j], scale);
            if (!is_max) { lo = fminf(lo, u[j]); hi = fmaxf(hi, u[j]); }
        }
        // warp min / max through the order-preserving integer image of a float (the sign of a zero result is
        // irrelevant below: it only enters differences)
        auto ordered = [](float f) { const uint32_t b = __float_as_uint(f); return b ^ (static_cast<uint32_t>(static_cast<int32_t>(b) >> 31) | 0x80000000u); };
        auto unordered = [](uint32_t o) { return __uint_as_float(o ^ ((o >> 31) ? 0x80000000u : 0xffffffffu)); };
        lo = unordered(__reduce_min_sync(full, ordered(lo)));
        hi = unordered(__reduce_max_sync(full, ordered(hi)));
        // pattern selector: min/max fitness, two patterns per lane
        double score = INFINITY;
        int kp = lane;
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const int k = lane + 32 * r;
            if (k < S) {
                const double a = static_cast<double>(__half2float(__ushort_as_half(pat_s[k * 16]))) - static_cast<double>(lo);
                const double b = static_cast<double>(__half2float(__ushort_as_half(pat_s[k * 16 + 14]))) - static_cast<double>(hi);
                const double sc = __dadd_rn(__dmul_rn(a, a), __dmul_rn(b, b));
                if (sc < score) { score = sc; kp = k; }
            }
        }
        {   // arg-min over the lanes, ties to the lower id: a non-negative double orders like its bit pattern
            const uint64_t sb = static_cast<uint64_t>(__double_as_longlong(score));
            const uint32_t s_hi = static_cast<uint32_t>(sb >> 32), s_lo = static_cast<uint32_t>(sb);
            const uint32_t m_hi = __reduce_min_sync(full, s_hi);
            const uint32_t m_lo = __reduce_min_sync(full, s_hi == m_hi ? s_lo : 0xffffffffu);
            kp = static_cast<int>(__reduce_min_sync(full, (s_hi == m_hi && s_lo == m_lo) ? static_cast<uint32_t>(kp) : 0xffffffffu));
        }
        // value mappers: nearest centroid, ties to the lower index
        // The pattern is ascending, so the nearest centroid is one of the two that bracket the value
        // (exact fp32 comparisons find them); the fp64 squared distances of those two decide, as in the
        // definition, and equal centroids resolve to the lowest index.
        // A centroid is an fp16 number, so c <= u exactly when c <= u rounded down to fp16: the fifteen
        // comparisons are eight packed fp16 ones (entry 15 of the row is replaced by +inf).
        uint4 c_lo = reinterpret_cast<const uint4*>(pat_s)[kp * 2], c_hi = reinterpret_cast<const uint4*>(pat_s)[kp * 2 + 1];
        c_hi.w = (c_hi.w & 0xffffu) | 0x7c000000u;
        const uint32_t crow[8] = {c_lo.x, c_lo.y, c_lo.z, c_lo.w, c_hi.x, c_hi.y, c_hi.z, c_hi.w};
        uint32_t sym[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const __half2 uu = __half2half2(__float2half_rd(u[j]));
            __half2 cnt = __floats2half2_rn(0.0f, 0.0f);
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                __half2 c2;
                asm("mov.b32 %0, %1;" : "=r"(*reinterpret_cast<uint32_t*>(&c2)) : "r"(crow[m]));
                cnt = __hadd2(cnt, __hle2(c2, uu));
            }
            const int below = __half2int_rn(__hadd(__low2half(cnt), __high2half(cnt)));     // centroids <= u
            const int a = max(below - 1, 0), b = min(below, kCentroids - 1);
            const float ca = __half2float(__ushort_as_half(pat_s[kp * 16 + a])), cb = __half2float(__ushort_as_half(pat_s[kp * 16 + b]));
            const double da = static_cast<double>(u[j]) - static_cast<double>(ca), db = static_cast<double>(u[j]) - static_cast<double>(cb);
            int bi = __dmul_rn(db, db) < __dmul_rn(da, da) ? b : a;
            while (bi > 0 && pat_s[kp * 16 + bi - 1] == pat_s[kp * 16 + bi]) --bi;      // duplicates: first entry
            sym[j] = (lane * 4 + j == pstar) ? 15u : static_cast<uint32_t>(bi);
        }
        // four encoders: total length per codebook, the shortest wins (ties to the lower id)
        uint32_t t01 = 0, t23 = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint16_t* e = enc_s + (kp * kCodebooks) * kSymbols + sym[j];
            t01 += (e[0] >> 8) | (static_cast<uint32_t>(e[kSymbols] >> 8) << 16);
            t23 += (e[2 * kSymbols] >> 8) | (static_cast<uint32_t>(e[3 * kSymbols] >> 8) << 16);
        }
        t01 = __reduce_add_sync(full, t01);
        t23 = __reduce_add_sync(full, t23);
        const uint32_t tot[4] = {t01 & 0xffffu, t01 >> 16, t23 & 0xffffu, t23 >> 16};
        int hf = 0;
        uint32_t shortest = tot[0];
#pragma unroll
        for (int hh = 1; hh < 4; ++hh)
            if (tot[hh] < shortest) { shortest = tot[hh]; hf = hh; }
        // bit positions: header, ID_KP codeword, then a prefix sum over the 128 code lengths
        const uint32_t kpe = kp_s[kp];
        const uint32_t kp_len = kpe >> 12;
        uint32_t code[4], len[4], lane_bits = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t e = enc_s[(kp * kCodebooks + hf) * kSymbols + sym[j]];
            code[j] = e & 0xffu;
            len[j] = e >> 8;
            lane_bits += len[j];
        }
        uint32_t incl = lane_bits;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(full, incl, o);
            if (lane >= o) incl += v;
        }
        const uint32_t end_bit = kHeaderBits + kp_len + __shfl_sync(full, incl, 31);
        uint32_t pos = kHeaderBits + kp_len + incl - lane_bits;
        // pack / clip
        if (lane < 16) blk[lane] = 0;
        __syncwarp();
        if (lane == 0) atomicOr(&blk[0], qs | (static_cast<uint32_t>(hf) << 8) | ((kpe & 0xfffu) << kHeaderBits));
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (pos < static_cast<uint32_t>(kBlockBits)) {
                const uint32_t nbits = min(len[j], static_cast<uint32_t>(kBlockBits) - pos);   // truncated at bit 512
                const uint32_t v = code[j] & ((1u << nbits) - 1u);
                const uint32_t w = pos >> 5, off = pos & 31u;
                atomicOr(&blk[w], v << off);
                if (off + nbits > 32u) atomicOr(&blk[w + 1], v >> (32u - off));
            }
            pos += len[j];
        }
        if (end_bit <= static_cast<uint32_t>(kBlockBits)) {
            // outliers: the next-largest |x| (ties: lower index), as many 15-bit slots as fit, at most 16
            const int n_pad = min(kMaxPads, static_cast<int>((kBlockBits - end_bit) / kPadBits));
            // Every lane sorts its four keys (the abs-max itself left out); n_pad times the warp takes the largest
            // head and its owner advances.  A lane then knows which of its values are outliers and with which
            // slot numbers, and all lanes write their fields at once.
            uint32_t k0 = key[0] + 1u, k1 = key[1] + 1u, k2 = key[2] + 1u, k3 = key[3] + 1u;      // +1: zero means "nothing left"
            if ((pstar >> 2) == lane) {
                if ((pstar & 3) == 0) k0 = 0; else if ((pstar & 3) == 1) k1 = 0; else if ((pstar & 3) == 2) k2 = 0; else k3 = 0;
            }
            auto order = [](uint32_t& a, uint32_t& b) { const uint32_t hi_ = max(a, b), lo_ = min(a, b); a = hi_; b = lo_; };
            order(k0, k1); order(k2, k3); order(k0, k2); order(k1, k3); order(k1, k2);            // descending
            const uint32_t s0 = k0, s1 = k1, s2 = k2, s3 = k3;
            uint32_t slots = 0;                            // slot numbers of this lane's outliers, the latest in the low byte
            int mine = 0;
            for (int p = 0; p < n_pad; ++p) {
                const uint32_t top = __reduce_max_sync(full, k0);
                if (k0 == top) {                           // keys are distinct: exactly one lane
                    k0 = k1; k1 = k2; k2 = k3; k3 = 0;
                    slots = (slots << 8) | static_cast<uint32_t>(p);
                    ++mine;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (i < mine) {
                    const int idx = 127 - static_cast<int>(((i == 0 ? s0 : i == 1 ? s1 : i == 2 ? s2 : s3) - 1u) & 127u);
                    const int p = static_cast<int>((slots >> (8 * (mine - 1 - i))) & 0xffu);
                    const int j = idx & 3;
                    const float xv = j == 0 ? x[0] : j == 1 ? x[1] : j == 2 ? x[2] : x[3];
                    const uint32_t field = static_cast<uint32_t>(idx) | (fp8(xv) << 7);
                    const uint32_t bp = kBlockBits - kPadBits * (p + 1), w = bp >> 5, off = bp & 31u;
                    atomicOr(&blk[w], field << off);
                    if (off + kPadBits > 32u) atomicOr(&blk[w + 1], field >> (32u - off));
                }
            }
        }
        __syncwarp();
        if (lane < 16) reinterpret_cast<uint32_t*>(d_blocks + g * kBlockBytes)[lane] = blk[lane];
        __syncwarp();
    }
}

}  // namespace

extern "C" int ecco_kv_compress(const void* d_meta, const void* d_x_fp16, uint64_t n_groups, uint8_t* d_blocks, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_meta || !d_x_fp16 || !d_blocks) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_x_fp16) || !aligned16(d_blocks)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > (1ull << 40)) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const uint64_t ctas = (n_groups + kKvWarps - 1) / kKvWarps;
    const uint64_t cap = static_cast<uint64_t>(di.sms) * 8;
    return launch_overlapped(ecco_kv_compress_kernel, static_cast<unsigned>(ctas < cap ? ctas : cap), static_cast<unsigned>(kKvWarps * 32), 0,
                             static_cast<cudaStream_t>(stream), static_cast<const uint8_t*>(d_meta), static_cast<const __half*>(d_x_fp16),
                             n_groups, d_blocks);
}

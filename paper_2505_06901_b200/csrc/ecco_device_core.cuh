// ecco_device_core.cuh -- shared-memory layout, PTX helpers, table staging, the per-group decoder
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

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


}  // namespace

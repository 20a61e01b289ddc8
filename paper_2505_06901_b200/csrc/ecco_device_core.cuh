// ecco_device_core.cuh -- shared-memory layout, PTX helpers, table staging, the per-group decoder
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

#include <cuda.h>
#include <cuda/std/type_traits>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>

#include <atomic>
#include <climits>
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

// Shared memory of a decoding CTA, from its 1 KB-aligned base:
//   kMiscBytes                                 barrier word (at a fixed place: images come and go, the barrier stays), small CTA-wide words
//   pattern | ID_KP table | codebook records   (kFixedTableBytes)
//   shape tables                               (DevHeader::shape_bytes)
//   pair tables                                at the next address that is a multiple of DevHeader::pair_align
//   per-warp arrays                            at the next multiple of 2 KB; as many warps work as fit
// The sizes come from the image's header, so the kernels are launched with all the shared memory an SM has and
// the most warps their registers allow, and lay themselves out once they have read the header.
constexpr uint32_t kMiscBytes = 1024;
constexpr uint32_t kSmemPattern = kMiscBytes;
constexpr uint32_t kSmemKpLut = kSmemPattern + kPatternBytes;
constexpr uint32_t kSmemCbRec = kSmemKpLut + kKpLutBytes;
constexpr uint32_t kSmemShapeLut = kMiscBytes + kFixedTableBytes;    // 15360: 256-aligned
constexpr uint32_t kSmemCtaBytes = 232448;                           // 227 KB: what every decoding kernel asks for
constexpr uint32_t kBitsRows = 18;
constexpr uint32_t kBitsBytes = kBitsRows * 32 * 4;                  // 2304
constexpr uint32_t kTabBytes = 16 * 32 * 4;                          // 2048: one value table
constexpr uint32_t kSymsBytes = 16 * 32 * 4;                         // 2048
constexpr int kFusedFree = 12;                                       // fused kernels: leading decode steps without the clip test
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
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ int32_t lds_s16(uint32_t addr)
{
    int32_t v;
    asm volatile("ld.shared.s16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v) { asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(static_cast<unsigned short>(v)) : "memory"); }
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_u32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
// one 64-byte block = two 32-byte loads per lane: every load instruction asks for whole sectors.  Plain (coherent)
// loads that bypass L1: under the overlapped launches the blocks may have been written by the previous kernel of the
// stream (the online compressor), and the non-coherent path is only for data that nobody writes while a kernel lives.
struct Block { uint32_t w[16]; };
__device__ __forceinline__ void ldg_block(Block& b, const uint8_t* p)
{
    asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(b.w[0]), "=r"(b.w[1]), "=r"(b.w[2]), "=r"(b.w[3]), "=r"(b.w[4]), "=r"(b.w[5]), "=r"(b.w[6]), "=r"(b.w[7])
                 : "l"(p));
    asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(b.w[8]), "=r"(b.w[9]), "=r"(b.w[10]), "=r"(b.w[11]), "=r"(b.w[12]), "=r"(b.w[13]), "=r"(b.w[14]), "=r"(b.w[15])
                 : "l"(p + 32));
}
__device__ __forceinline__ void prefetch_block_l2(const uint8_t* p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p + 32));
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
// Where the tables of the current image sit in shared memory (absolute shared addresses) and what is left
// for the warps.  Uniform over the CTA.
struct Tables {
    uint32_t base;          // misc area (barrier word at +0), then pattern, ID_KP table and codebook records
    uint32_t shape;         // shape tables
    uint32_t pair;          // pair tables (aligned to the widest)
    uint32_t warp_base;     // per-warp arrays, 2 KB aligned
    uint32_t shape_bytes, pair_bytes;
    bool pairs;             // the image has pair tables
    float T;
    uint32_t hash_lo, hash_hi;
};
// use_pairs = false: the kernel decodes one symbol per lookup and leaves the pair tables out (more room for warps)
__device__ __forceinline__ Tables plan_tables(uint32_t smem_base, const uint8_t* d_meta, bool use_pairs = true)
{
    const DevHeader* hd = reinterpret_cast<const DevHeader*>(d_meta);
    Tables tb;
    tb.base = smem_base;
    tb.shape = smem_base + kSmemShapeLut;
    tb.shape_bytes = min(__ldg(&hd->shape_bytes), kMaxShapes * 256u) & ~255u;     // clamped: a bad header cannot overrun shared memory
    tb.pair_bytes = use_pairs ? min(__ldg(&hd->pair_bytes), kPairBudgetBytes) & ~511u : 0u;
    const uint32_t align = min(max(__ldg(&hd->pair_align), 512u), 2u << kPairMaxBits);
    const uint32_t tables_end = tb.shape + tb.shape_bytes;
    tb.pair = tb.pair_bytes ? (tables_end + align - 1u) & ~(align - 1u) : tables_end;
    tb.warp_base = (tb.pair + tb.pair_bytes + 2047u) & ~2047u;
    tb.pairs = tb.pair_bytes != 0;
    tb.T = __ldg(&hd->T);
    tb.hash_lo = __ldg(&hd->hash_lo);
    tb.hash_hi = __ldg(&hd->hash_hi);
    return tb;
}
// warps of this CTA that have room for warp_bytes each (the others sit the launch out)
__device__ __forceinline__ uint32_t warps_that_fit(const Tables& tb, uint32_t warp_bytes, uint32_t tail_bytes = 0)
{
    const uint32_t used = tb.warp_base - tb.base + tail_bytes;
    const uint32_t room = used < kSmemCtaBytes ? kSmemCtaBytes - used : 0u;
    return min(room / warp_bytes, blockDim.x >> 5);
}
// In two halves, so that the caller can put work between the issue and the wait.  wait_tables returns false
// (CTA-uniform) if the bounded wait expired; the caller must then return.  The barrier word is the first word of
// the CTA's shared memory; first = false re-arms a barrier that an earlier phase initialised.
__device__ __forceinline__ void issue_tables(const Tables& tb, const uint8_t* d_meta, bool first = true)
{
    const uint32_t bar = tb.base;
    if (threadIdx.x == 0) {
        if (first) {
            mbar_init(bar, 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        const DevHeader* hd = reinterpret_cast<const DevHeader*>(d_meta);
        mbar_expect_tx(bar, kFixedTableBytes + tb.shape_bytes + tb.pair_bytes);
        bulk_g2s(tb.base + kSmemPattern, d_meta + kOffPattern, kFixedTableBytes, bar);
        bulk_g2s(tb.shape, d_meta + kOffShapeLut, tb.shape_bytes, bar);
        if (tb.pair_bytes) bulk_g2s(tb.pair, d_meta + __ldg(&hd->off_pair), tb.pair_bytes, bar);
    }
}
// Bounded wait of the whole CTA on a barrier word: at most 2 * limit polls per thread (the second round is a last
// chance for a copy in flight), then the CTA gives up together, records ECCO_ERR_DEVICE_TIMEOUT and returns false.
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, int limit)
{
    __syncthreads();                             // the barrier word is initialised
    bool done = false;
    for (int i = 0; i < limit && !done; ++i) done = mbar_try_wait(bar, parity);
    if (!done)
        for (int i = 0; i < limit && !done; ++i) done = mbar_try_wait(bar, parity);
    const bool all = __syncthreads_and(done);
    if (!all && threadIdx.x == 0) atomicExch(&g_device_status, ECCO_ERR_DEVICE_TIMEOUT);
    return all;
}
__device__ __forceinline__ bool wait_tables(const Tables& tb, uint32_t parity = 0) { return bounded_wait(tb.base, parity, kWaitLimit); }
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may become resident
// while the previous kernel in the stream is still draining.  dependency_wait() returns once that kernel has
// completed and its writes are visible (at once if there is no such overlap); every kernel executes it before
// its first access to global memory other than the metadata image, so stream order is what it is without the
// attribute and only launch, table fetch and prologue overlap.  The image is the exception because no kernel writes
// it: it reaches the device by a copy, which is a stream operation of its own (a kernel behind a copy starts after
// it), and a kernel can start early only behind one that releases its dependents, i.e. one of this file.
// release_dependents() lets the next kernel of the stream do the same with respect to this one.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// the per-group decoder
// ---------------------------------------------------------------------------------------------
// The lane's sixteen dequantised values sit in rows of 128 bytes, one row per rank, as
//   kTabHalfBits  fp16 bits in a 32-bit word      tab[16][32] u32, 2 KB per warp
//   kTabFloat     fp32                            the same shape
//   kTabHalf      fp16, two warps to an array     tab[16][32][2] u16: a lane of an even warp uses the low half of its word,
//                                                 the same lane of the next warp the high half (each lane keeps its own bank)
enum TabKind { kTabHalfBits, kTabFloat, kTabHalf };
template <TabKind kTab> __device__ __forceinline__ uint32_t lds_tab(uint32_t addr) { return kTab == kTabHalf ? lds_u16(addr) : lds_u32(addr); }
// shared address of the lane's column in the value table of `warp`, given the first table's address (a multiple of 2 KB)
template <TabKind kTab> __device__ __forceinline__ uint32_t tab_column(uint32_t tabs, uint32_t warp, uint32_t lane)
{
    return kTab == kTabHalf ? tabs + (warp >> 1) * kTabBytes + lane * 4u + (warp & 1u) * 2u : tabs + warp * kTabBytes + lane * 4u;
}
// bytes the value tables of nw warps take
template <TabKind kTab> __device__ __forceinline__ uint32_t tab_bytes(uint32_t nw) { return kTab == kTabHalf ? ((nw + 1u) >> 1) * kTabBytes : nw * kTabBytes; }

struct WarpSmem {
    uint32_t bits;      // shared address of bits[0][lane]
    uint32_t tab;       // shared address of the lane's column of the value table (row r at + 128 r)
    uint32_t syms;      // shared address of syms[0][lane] (kernels that keep the decoded ranks)
};

struct GroupHeader {
    uint32_t pos;       // first bit of the coded indices
    uint32_t blut;      // shared address of the shape table of (ID_KP, ID_HF) (256-byte aligned), OR-ed with its rotation
    uint32_t plut;      // shared address of its pair table (aligned to the table's size), OR-ed with its rotation
    uint32_t mask;      // ((1 << W) - 1) << 1: byte offset of a pair-table entry from a window that starts one bit early
};

// Pattern retriever (Sec. 4.2): scale byte, ID_HF, Huffman-coded ID_KP from the group's first 22
// stream bits (hdr, first bit in bit 0); writes the lane's 16 dequantised values (fp16 bits, or
// fp32 bits when kFloatTab) in RANK order, the order the decode tables speak.  first_bit = position
// of the group's first bit in the lane's staged bit stream.
template <TabKind kTab>
__device__ __forceinline__ GroupHeader open_header(uint32_t hdr, uint32_t first_bit, const Tables& tb, const WarpSmem& ws, float T)
{
    const uint32_t qs = hdr & 0xffu, hf = (hdr >> 8) & 3u;
    const uint32_t kpw = (hdr >> kHeaderBits) & 0xfffu;
    uint32_t kpe;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(kpe) : "r"(tb.base + kSmemKpLut + kpw * 2));
    const uint32_t kp = kpe & 0xffu;
    GroupHeader h;
    h.pos = first_bit + kHeaderBits + (kpe >> 8);
    const uint32_t cb = kp * kCodebooks + hf;
    uint4 rec;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(rec.x), "=r"(rec.y), "=r"(rec.z), "=r"(rec.w) : "r"(tb.base + kSmemCbRec + cb * 16));
    const uint32_t shape = (rec.x >> 8) & 0xffu, rot = table_rotation(shape);   // entry of window i at offset (size * i) ^ rot
    h.blut = (tb.shape + shape * 256u) | rot;
    h.plut = (tb.pair + ((rec.x & 0xffu) << 9)) | rot;
    h.mask = ((1u << (rec.x >> 16)) - 1u) << 1;
    const float top = fp8_to_float(qs) * T;           // FP8 -> FP16 range by the power-of-two factor
    const float s = fabsf(top);
    uint4 p0, p1;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(p0.x), "=r"(p0.y), "=r"(p0.z), "=r"(p0.w) : "r"(tb.base + kSmemPattern + kp * 32));
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(p1.x), "=r"(p1.y), "=r"(p1.z), "=r"(p1.w) : "r"(tb.base + kSmemPattern + kp * 32 + 16));
    const uint32_t pr[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const __half c = __ushort_as_half(static_cast<unsigned short>((pr[j >> 1] >> ((j & 1) * 16)) & 0xffffu));
        // mapper (Sec. 4.2): one fp32 product, one rounding to fp16
        const __half v = __float2half_rn(j < 15 ? __half2float(c) * s : top);
        const uint32_t row = ((j < 8 ? rec.z : rec.w) >> ((j & 7) * 4)) & 15u;
        if (kTab == kTabHalf) sts_u16(ws.tab + row * 128, __half_as_ushort(v));
        else sts_u32(ws.tab + row * 128, kTab == kTabFloat ? __float_as_uint(__half2float(v)) : static_cast<uint32_t>(__half_as_ushort(v)));
    }
    return h;
}

// 64-byte block: stage the 16 words in the lane's column of the transposed bit-stream array, then the header
template <TabKind kTab>
__device__ __forceinline__ GroupHeader open_group(const Block& blk, const Tables& tb, const WarpSmem& ws, float T)
{
#pragma unroll
    for (int i = 0; i < 16; ++i) sts_u32(ws.bits + i * 128, blk.w[i]);
    return open_header<kTab>(blk.w[0], 0u, tb, ws, T);
}

// Decodes the 128 indices of the lane's group (Sec. 4.2, Huffman decode) and hands each value to
// sink(n, value_bits, rank, alive, pair) (kLookup = false skips the value lookup and passes 0); for even n the low
// byte of `pair` holds the ranks of positions n and n + 1 (low nibble first), for kernels that keep the ranks.  A codeword that would
// cross the end bit ends the group: that and all later positions are delivered as zero (clipped).  Returns the
// end bit if all 128 fitted, else 0.  Must be called by all 32 lanes of the warp.
//
// Four symbols per step, from one 32-bit window of the lane's stream.  With pair tables (pairs = true, uniform
// over the warp) a step is two lookups of two symbols each; a lane whose entry says "escape" (the table's window
// ended inside the second codeword) fetches that symbol through the shape table, under a warp vote, so the lanes
// stay in lock step at four symbols per step.  Steps in which some lane reaches the end of its stream, and every
// step when the image has no pair tables, decode one symbol per lookup through the shape table and carry the
// per-symbol clip test.
// kLastRow / kEndBit: last data row of the lane's staged stream (two zero rows follow) and the bit
// at which the stream ends (16 and 512 for the 64-byte block).
// kFreeSteps (a multiple of 4): that many leading steps run without the clip test; the caller guarantees that
// the stream cannot end within them (a block's indices start at bit 22 at the latest, so 12 steps of at most
// 32 bits end by bit 406).
template <bool kLookup = true, uint32_t kLastRow = 16, uint32_t kEndBit = kBlockBits, int kFreeSteps = 0, TabKind kTab = kTabHalfBits, class Sink>
__device__ __forceinline__ uint32_t decode_symbols(const GroupHeader& h, const WarpSmem& ws, bool pairs, Sink&& sink)
{
    static_assert(kFreeSteps % 4 == 0 && kFreeSteps < 32, "whole unrolled iterations");
    constexpr uint32_t kFull = 0xffffffffu;
    uint32_t pos = h.pos;
    bool alive = true;
    // one symbol per lookup
    auto four_single = [&](int step, auto tested) {
        constexpr bool kTest = decltype(tested)::value;
        const uint32_t wi = kTest ? min(pos >> 5, kLastRow) : pos >> 5;
        const uint32_t lo = lds_u32(ws.bits + wi * 128), hi = lds_u32(ws.bits + wi * 128 + 128);
        const uint32_t win = __funnelshift_r(lo, hi, pos);           // 32 stream bits from pos
        uint32_t e[4], end[4], acc = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            e[j] = lds_u8(h.blut ^ ((win >> acc) & 0xffu));
            acc += e[j] >> 4;
            end[j] = acc;
        }
        if (kTest && __any_sync(kFull, pos + acc > kEndBit)) {
            const uint32_t limit = kEndBit - min(pos, kEndBit);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                alive = alive && (end[j] <= limit);
                const uint32_t v = kLookup ? lds_tab<kTab>(ws.tab + (e[j] & 15u) * 128) : 0u;
                sink(step * 4 + j, alive ? v : 0u, e[j] & 15u, alive, (e[j] & 15u) | (e[j | 1] << 4));
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                sink(step * 4 + j, kLookup ? lds_tab<kTab>(ws.tab + (e[j] & 15u) * 128) : 0u, e[j] & 15u, true, (e[j] & 15u) | (e[j | 1] << 4));
        }
        pos += acc;
    };
    // eight stream bits from absolute position q, through the shape table: length << 4 | rank
    auto single_at = [&](uint32_t q) {
        const uint32_t qi = min(q >> 5, kLastRow);
        const uint32_t lo = lds_u32(ws.bits + qi * 128), hi = lds_u32(ws.bits + qi * 128 + 128);
        return lds_u8(h.blut ^ (__funnelshift_r(lo, hi, q) & 0xffu));
    };
    // an escape entry completed with its second symbol, which starts `off` bits into the window (off = 1 + the bits
    // before it); the window has it whole unless off > 24, which takes three 8-bit codewords in a row
    auto resolve = [&](int32_t e, uint32_t win, uint32_t off, uint32_t p) {
        const uint32_t b = off <= 24u ? lds_u8(h.blut ^ ((win >> off) & 0xffu)) : single_at(p + (static_cast<uint32_t>(e) & 15u));
        return static_cast<int32_t>((static_cast<uint32_t>(e) & 0x078fu) + (b >> 4) + ((b & 15u) << 11));
    };
    // Two symbols per lookup, software-pipelined by hand: a warp issues in order and every shared-memory load here is
    // a volatile asm statement, so the loads keep the order they are written in.  The window of the next step is
    // fetched as soon as this step's length is known, and the four values of a step are looked up at its end but
    // handed to the sink only after the first lookup of the next step has been issued.
    uint32_t lo = 0, hi = 0;                 // the words the next window comes from
    uint32_t pv[4] = {0, 0, 0, 0}, pu0 = 0, pu1 = 0;   // values and entries of the previous step, not yet delivered
    bool pending = false;                    // uniform over the warp
    auto load_window = [&](auto clamp) {
        const uint32_t p1 = pos - 1u;        // the window starts one bit early: its bits 1.. are the byte offset of a 2-byte entry
        const uint32_t wi = decltype(clamp)::value ? min(p1 >> 5, kLastRow) : p1 >> 5;
        lo = lds_u32(ws.bits + wi * 128);
        hi = lds_u32(ws.bits + wi * 128 + 128);
    };
    auto deliver = [&](int step) {
        sink(step * 4 + 0, pv[0], (pu0 >> 7) & 15u, true, pu0 >> 7);
        sink(step * 4 + 1, pv[1], (pu0 >> 11) & 15u, true, 0u);
        sink(step * 4 + 2, pv[2], (pu1 >> 7) & 15u, true, pu1 >> 7);
        sink(step * 4 + 3, pv[3], (pu1 >> 11) & 15u, true, 0u);
    };
    // owed: 0 = nothing to deliver (first step), 1 = the previous step is always owed (steps without the clip test
    // after the first), 2 = look at `pending`
    auto four_pair = [&](int step, auto tested, auto owed) {
        constexpr bool kTest = decltype(tested)::value;
        constexpr int kOwed = decltype(owed)::value;
        const uint32_t win = __funnelshift_r(lo, hi, pos - 1u);
        int32_t e0 = lds_s16(h.plut ^ (win & h.mask));
        if (kOwed == 1 || (kOwed == 2 && pending)) deliver(step - 1);  // while the lookup is in flight
        int32_t e1 = lds_s16(h.plut ^ (__funnelshift_r(win, 0u, static_cast<uint32_t>(e0)) & h.mask));   // shift by e0 mod 32 = its length field
        const bool esc = (e0 | e1) < 0;
        uint32_t acc = static_cast<uint32_t>(e0 + e1) & 0x7fu;      // bits consumed by the four symbols (if no escape)
        if (__any_sync(kFull, esc || (kTest && pos + acc > kEndBit))) {
            if (esc) {
                if (e0 < 0) {
                    e0 = resolve(e0, win, 1u + (static_cast<uint32_t>(e0) & 15u), pos);
                    e1 = lds_s16(h.plut ^ (__funnelshift_r(win, 0u, static_cast<uint32_t>(e0)) & h.mask));
                }
                if (e1 < 0) e1 = resolve(e1, win, 1u + (static_cast<uint32_t>(e0) & 31u) + (static_cast<uint32_t>(e1) & 15u), pos + (static_cast<uint32_t>(e0) & 31u));
                acc = static_cast<uint32_t>(e0 + e1) & 0x7fu;
            }
            if (kTest && __any_sync(kFull, pos + acc > kEndBit)) {   // some lane's stream ends in this step
                pending = false;
                four_single(step, tested);
                load_window(tested);
                return;
            }
        }
        pos += acc;
        load_window(tested);
        pu0 = static_cast<uint32_t>(e0);
        pu1 = static_cast<uint32_t>(e1);
        if (kLookup) {
            pv[0] = lds_tab<kTab>(ws.tab | (pu0 & 0x780u));
            pv[1] = lds_tab<kTab>(ws.tab | ((pu0 >> 4) & 0x780u));
            pv[2] = lds_tab<kTab>(ws.tab | (pu1 & 0x780u));
            pv[3] = lds_tab<kTab>(ws.tab | ((pu1 >> 4) & 0x780u));
        }
        pending = true;
    };
    if (pairs) {
        load_window(cuda::std::false_type{});
        using Never = cuda::std::integral_constant<int, 0>;
        using Always = cuda::std::integral_constant<int, 1>;
        using Check = cuda::std::integral_constant<int, 2>;
        if (kFreeSteps > 0) {
            four_pair(0, cuda::std::false_type{}, Never{});
#pragma unroll 4
            for (int step = 1; step < kFreeSteps; ++step) four_pair(step, cuda::std::false_type{}, Always{});
        }
#pragma unroll 4
        for (int step = kFreeSteps; step < 32; ++step) four_pair(step, cuda::std::true_type{}, Check{});
        if (pending) deliver(31);
    } else {
        if (kFreeSteps > 0) {
#pragma unroll 4
            for (int step = 0; step < kFreeSteps; ++step) four_single(step, cuda::std::false_type{});
        }
#pragma unroll 4
        for (int step = kFreeSteps; step < 32; ++step) four_single(step, cuda::std::true_type{});
    }
    return alive ? pos : 0u;
}

// Kernels that need the decoded ranks again (the outlier fix-up of the scalar fused kernels) keep them in syms[16][32]: position n in
// nibble n & 7 of word n >> 3.  put() takes the sink's pair byte at even n and stores a word when it is complete
// (n mod 8 is a compile-time constant after unrolling).
struct RankPacker {
    uint32_t word;
    __device__ __forceinline__ void put(int n, uint32_t pair, uint32_t syms)
    {
        if (n & 1) return;
        switch ((n & 7) >> 1) {                            // bytes above the one written are overwritten later
            case 0: word = pair; break;
            case 1: word = prmt(word, pair, 0x3240u); break;
            case 2: word = prmt(word, pair, 0x3410u); break;
            default: word = prmt(word, pair, 0x4210u); sts_u32(syms + (n >> 3) * 128, word); break;
        }
    }
};

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

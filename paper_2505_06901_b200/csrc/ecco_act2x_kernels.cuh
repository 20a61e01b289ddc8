// ecco_act2x_kernels.cuh -- 2x activation codec kernels
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

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
        if (ok) asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(d_blocks + c));
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
            asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
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

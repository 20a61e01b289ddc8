// ecco_kv_compress_kernel.cuh -- online 4x compressor kernel
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

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
        const uint2 raw = __ldcg(reinterpret_cast<const uint2*>(d_x + g * kGroup) + lane);
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

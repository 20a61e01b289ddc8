// ecco_attn_values_kernels.cuh -- K5: attention output over a compressed V cache
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

namespace {

// ---------------------------------------------------------------------------------------------
// K5: attention output over a compressed V cache (Eq. 3: softmax(QK^T / sqrt(d_k)) V).
// out[b][hq][d] = sum_t p[b][hq][t] * V~[b][hq / q_per_kv][t][d] with p = softmax_t(scores).
// A thread owns one token (one group) as in K3, but here the sum runs over tokens, i.e. across
// lanes.  The group is decoded once, values and all, into eight [32 tokens][16 dims] fp16 tiles of the
// warp (the swizzle of the decompress staging tile); when the end bit is known the outliers are
// written over their positions in the tiles; then every tile is contracted on the tensor cores:
// (V tile)^T [16 dims x 32 tokens] x P^T [32 tokens x 8 heads] with mma.m16n8k16, fp32 accumulators
// (4 registers per 16 dims, 32 for the 128 dims).  p is split into an fp16 head and an fp16 remainder
// (two MMAs) so that its rounding does not show.  The result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------
// Row maximum and reciprocal of the row's sum of exponentials, one CTA per row.  One pass: every thread keeps a running
// (maximum, sum of exp(x - maximum)) over its elements, rescaling the sum when the maximum grows; the pairs are then
// merged over the warp and over the warps in a fixed order.
__device__ __forceinline__ void softmax_merge(float& m, float& s, float m2, float s2)
{
    const float mn = fmaxf(m, m2);
    // an empty side has maximum -inf and sum 0: its factor is exp(-inf) = 0 unless both are empty (avoid -inf - -inf)
    const float f1 = m == mn ? 1.0f : expf(m - mn), f2 = m2 == mn ? 1.0f : expf(m2 - mn);
    s = s * f1 + s2 * f2;
    m = mn;
}
__global__ void __launch_bounds__(256)
ecco_softmax_stats_kernel(const float* d_scores, int rows, int seq, float2* d_stats, unsigned int* d_tickets, int n_tickets)
{
    __shared__ float2 part[8];
    const int row = static_cast<int>(blockIdx.x), tid = static_cast<int>(threadIdx.x), lane = tid & 31, warp = tid >> 5;
    release_dependents();
    dependency_wait();                                     // the scores may come from the previous kernel of the stream
    // also clears the ticket words of the call's workspace (the previous kernel, which may have used them, is complete)
    for (int i = row * 256 + tid; i < n_tickets; i += static_cast<int>(gridDim.x) * 256) d_tickets[i] = 0u;
    if (row >= rows) return;
    const float* s = d_scores + static_cast<size_t>(row) * seq;
    float mx = -INFINITY, sum = 0.0f;
    auto take = [&](float x) {
        if (x > mx) { sum = sum * expf(mx - x) + 1.0f; mx = x; }      // exp(-inf) = 0 on the first element
        else if (x != -INFINITY) sum += expf(x - mx);                  // a masked score (-inf) adds nothing, also before any finite one
    };
    // the scores may come from the previous kernel: coherent loads; 16-byte loads where the row allows it
    if ((reinterpret_cast<uintptr_t>(s) & 15u) == 0) {
        const float4* s4 = reinterpret_cast<const float4*>(s);
        const int n4 = seq / 4;
        int i = tid;
        for (; i + 3 * 256 < n4; i += 4 * 256) {           // four loads in flight per thread
            const float4 a = __ldcg(s4 + i), b = __ldcg(s4 + i + 256), c = __ldcg(s4 + i + 512), d = __ldcg(s4 + i + 768);
            take(a.x); take(a.y); take(a.z); take(a.w);
            take(b.x); take(b.y); take(b.z); take(b.w);
            take(c.x); take(c.y); take(c.z); take(c.w);
            take(d.x); take(d.y); take(d.z); take(d.w);
        }
        for (; i < n4; i += 256) {
            const float4 v = __ldcg(s4 + i);
            take(v.x); take(v.y); take(v.z); take(v.w);
        }
        for (int t = (seq & ~3) + tid; t < seq; t += 256) take(__ldcg(s + t));
    } else {
        for (int t = tid; t < seq; t += 256) take(__ldcg(s + t));
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, mx, o), s2 = __shfl_xor_sync(0xffffffffu, sum, o);
        softmax_merge(mx, sum, m2, s2);
    }
    if (lane == 0) part[warp] = make_float2(mx, sum);
    __syncthreads();
    if (tid == 0) {
        float m = part[0].x, t = part[0].y;
        for (int w = 1; w < 8; ++w) softmax_merge(m, t, part[w].x, part[w].y);
        d_stats[row] = make_float2(m, 1.0f / t);
    }
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

// eight [32 tokens][16 dims] fp16 tiles, the last of which lies over rows 0..7 of the warp's bit-stream array (see K2m)
constexpr uint32_t kAvValueBytes = 7 * 1024;
constexpr uint32_t kAvWarpBytes = kTabBytes / 2 + kAvValueBytes + kBitsBytes;   // half a value table (two warps share one), tiles, bit stream
constexpr uint32_t kAvSlots = 8;                                            // reduction slots: see flush

constexpr float kProbScale = 32768.0f, kProbUnscale = 1.0f / 32768.0f;      // powers of two: exact

template <int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_attn_values_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_vblocks, int heads, int seq,
                        int q_per_kv, const float* d_scores, const float2* d_stats,
                        float* __restrict__ d_out, float* __restrict__ d_partial, unsigned int* __restrict__ d_tickets)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const int tid = static_cast<int>(threadIdx.x), n_threads = static_cast<int>(blockDim.x);
    release_dependents();
    const Tables tb = plan_tables(smem_u32(smem), d_meta, false);   // one symbol per lookup: see the scalar fused kernels
    constexpr uint32_t kSlotFloats = kGroup * 8;
    const uint32_t nw = warps_that_fit(tb, kAvWarpBytes, kTabBytes / 2 + kAvSlots * kSlotFloats * sizeof(float));
    const int kTokens = static_cast<int>(nw) * 32;         // tokens per unit: one per thread of the working warps
    const bool working = warp < nw;
    // small CTA-wide words in the misc area at the start of shared memory (the barrier word is its first)
    unsigned int& ticket = *reinterpret_cast<unsigned int*>(smem + 32);
    float2* stats_s = reinterpret_cast<float2*>(smem + 64);
    WarpSmem ws;
    ws.tab = tab_column<kTabHalf>(tb.warp_base, warp, lane);
    const uint32_t per_warp = tb.warp_base + tab_bytes<kTabHalf>(nw);
    const uint32_t vals = per_warp + warp * (kAvValueBytes + kBitsBytes);      // this warp's eight tiles
    ws.bits = vals + kAvValueBytes + lane * 4;
    ws.syms = 0;
    if (working) {
        sts_u32(ws.bits + 16 * 128, 0u);
        sts_u32(ws.bits + 17 * 128, 0u);
    }
    const uint32_t swz = ((lane >> 2) & 1u) << 4;
    const uint32_t my_row = vals + lane * 32;
    float* out_s = reinterpret_cast<float*>(smem + (per_warp - tb.base) + nw * (kAvValueBytes + kBitsBytes));    // slots of [128 dims][8 heads]

    const int chunks = (seq + kTokens - 1) / kTokens;
    const int64_t U = static_cast<int64_t>(heads) * chunks;
    // the CTAs that share a head count each other in (ticket), so every CTA of the split must own a unit: the
    // launch may bring more CTAs than there are units (the host does not know how many warps find room)
    const int G = static_cast<int>(min(static_cast<int64_t>(gridDim.x), U)), c = blockIdx.x;
    if (c >= G) return;
    const int64_t u0 = unit_begin(U, G, c), u1 = unit_begin(U, G, c + 1);
    auto block_ptr = [&](int64_t u) {
        const int bh = static_cast<int>(u / chunks), t = min(static_cast<int>(u % chunks) * kTokens + tid, seq - 1);
        return d_vblocks + (static_cast<uint64_t>(bh) * seq + t) * kBlockBytes;
    };
    issue_tables(tb, d_meta);
    dependency_wait();                                     // everything but the host-written tables: after the previous kernel of the stream
    if (u0 < u1 && working) prefetch_block_l2(block_ptr(u0));
    if (!wait_tables(tb)) return;
    const float T = tb.T;

    float acc[8][4];                                       // [16-dim chunk][mma accumulator]
    auto clear_acc = [&]() {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    };
    clear_acc();

    // all tokens of head bh seen by this CTA are in acc: reduce over the warps in a fixed order (in rounds of
    // kAvSlots warps: warp w adds its sums to slot w mod kAvSlots, the first round by plain stores; then the slots are
    // added in slot order), then either store (this CTA owns the whole head) or hand a partial to the slot-and-ticket
    // reduction
    auto flush = [&](int bh) {
        for (uint32_t first = 0; first < nw; first += kAvSlots) {
            if (warp >= first && warp < first + kAvSlots && warp < nw) {
                float* slot = out_s + (warp - first) * kSlotFloats;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int dim = ch * 16 + static_cast<int>(lane >> 2) + (j >= 2 ? 8 : 0);
                        const int head = static_cast<int>(lane & 3u) * 2 + (j & 1);
                        const float v = acc[ch][j] * kProbUnscale;
                        slot[dim * 8 + head] = first ? slot[dim * 8 + head] + v : v;
                    }
            }
            __syncthreads();
        }
        const uint32_t used = min(nw, kAvSlots);
        for (int i = tid; i < static_cast<int>(kSlotFloats); i += n_threads) {   // thread i keeps element i from here on
            float sum = out_s[i];
            for (uint32_t sl = 1; sl < used; ++sl) sum += out_s[sl * kSlotFloats + i];
            out_s[i] = sum;
        }
        const int c_lo = unit_owner(U, G, static_cast<int64_t>(bh) * chunks);
        const int c_hi = unit_owner(U, G, static_cast<int64_t>(bh + 1) * chunks - 1);
        if (c_lo == c_hi) {
            for (int i = tid; i < kGroup * 8; i += n_threads) {
                const int dim = i >> 3, r = i & 7;
                if (r < q_per_kv) d_out[(static_cast<size_t>(bh) * q_per_kv + r) * kGroup + dim] = out_s[i];
            }
        } else {
            float* mine = d_partial + static_cast<size_t>(c + bh) * (kGroup * 8);
            for (int i = tid; i < kGroup * 8; i += n_threads) mine[i] = out_s[i];
            __threadfence();
            __syncthreads();
            if (tid == 0) ticket = atomicAdd(&d_tickets[bh], 1u);
            __syncthreads();
            if (ticket == static_cast<unsigned int>(c_hi - c_lo)) {
                __threadfence();
                for (int i = tid; i < kGroup * 8; i += n_threads) {
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
        const bool valid = tile_base + static_cast<int>(lane) < seq;
        if (bh != cur_bh) {
            if (cur_bh >= 0) { flush(cur_bh); clear_acc(); }
            if (tid < 8) stats_s[tid] = tid < q_per_kv ? __ldcg(d_stats + static_cast<size_t>(bh) * q_per_kv + tid) : make_float2(0.0f, 0.0f);
            __syncthreads();
            cur_bh = bh;
        }
        if (!working) continue;                            // warps without room for their arrays only help with the reductions
        // P^T fragments (B operand): head = lane / 4, tokens (lane % 4) * 2 + {0, 1} + 8 j
        uint32_t p_hi[4], p_lo[4];
        {
            const int r = static_cast<int>(lane >> 2);
            const float2 st = stats_s[r];
            // Probabilities enter the tensor cores as fp16 pairs (value + remainder).  Taken as they are, everything
            // below 6e-5 would sit in fp16's subnormal range (one part in a thousand at p = 3e-5, the typical weight of
            // a token in a 32768-token row); scaled by 2^15 they keep 22 bits down to 2e-12, and p <= 1 cannot
            // overflow.  The sums are scaled back when they leave the accumulators (kProbUnscale in flush).
            const float to_p = st.y * kProbScale;
            const float* srow = d_scores + (static_cast<size_t>(bh) * q_per_kv + min(r, q_per_kv - 1)) * seq;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int tk = tile_base + static_cast<int>(lane & 3u) * 2 + 8 * j;
                float p0 = 0.0f, p1 = 0.0f;
                if (r < q_per_kv && tk < seq) p0 = __expf(__ldcg(srow + tk) - st.x) * to_p;
                if (r < q_per_kv && tk + 1 < seq) p1 = __expf(__ldcg(srow + tk + 1) - st.x) * to_p;
                const __half h0 = __float2half_rn(p0), h1 = __float2half_rn(p1);
                const __half l0 = __float2half_rn(p0 - __half2float(h0)), l1 = __float2half_rn(p1 - __half2float(h1));
                p_hi[j] = static_cast<uint32_t>(__half_as_ushort(h0)) | (static_cast<uint32_t>(__half_as_ushort(h1)) << 16);
                p_lo[j] = static_cast<uint32_t>(__half_as_ushort(l0)) | (static_cast<uint32_t>(__half_as_ushort(l1)) << 16);
            }
        }
        Block cur;                                         // fetched now, prefetched into L2 one unit earlier
        ldg_block(cur, block_ptr(u));
        if (u + 1 < u1) {
            prefetch_block_l2(block_ptr(u + 1));
            // the scores of this warp's tokens in the next unit, one 128-byte line per query head: into L2 now
            const int nbh = static_cast<int>((u + 1) / chunks), nt = static_cast<int>((u + 1) % chunks) * kTokens + static_cast<int>(warp) * 32;
            if (static_cast<int>(lane) < q_per_kv && nt < seq)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(d_scores + (static_cast<size_t>(nbh) * q_per_kv + lane) * seq + nt));
        }
        // lanes past the end of the row decode the row's last token again (zeroed below)
        __syncwarp();                                      // the tiles of the previous token tile have been read
        const GroupHeader h = open_group<kTabHalf>(cur, tb, ws, T);
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const uint32_t end = decode_symbols<true, 16, kBlockBits, kFusedFree, kTabHalf>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t) {
            const int slot = (n & 15) >> 1;                // clipped positions arrive as +0
            if (n & 1) r[slot] = __byte_perm(r[slot], v, 0x5410); else r[slot] = v;
            if ((n & 15) == 15) {
                const uint32_t row = my_row + (n >> 4) * 1024;
                sts_v4(row + swz, r[0], r[1], r[2], r[3]);
                sts_v4(row + (swz ^ 16u), r[4], r[5], r[6], r[7]);
            }
        });
        // outliers of a complete group replace the mapped values in the tiles (ascending: a later pad overrides an earlier one)
        const int n_pad = end ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
        for (int j = 0; j < n_pad; ++j) {
            const uint32_t f = read_pad(ws, j);
            const uint32_t loc = f & 127u, byte = (loc & 15u) * 2;
            asm volatile("st.shared.u16 [%0], %1;" ::"r"(my_row + (loc >> 4) * 1024 + ((byte & 16u) ^ swz) + (byte & 15u)),
                         "h"(static_cast<unsigned short>(f2h_bits(fp8_to_float(f >> 7) * T))) : "memory");
        }
        if (__any_sync(0xffffffffu, !valid)) {             // a row's ragged last tile: lanes past its end hold zeros (p is
            if (!valid) {                                  // zero there, but a decoded value need not be finite)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    sts_v4(my_row + ch * 1024, 0u, 0u, 0u, 0u);
                    sts_v4(my_row + ch * 1024 + 16, 0u, 0u, 0u, 0u);
                }
            }
        }
        __syncwarp();                                      // tiles complete
        // per 16-dim chunk: (V tile)^T x P^T on the tensor cores
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
            uint32_t a[2][4];
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                const uint32_t tok = (lane >> 4) * 8 + (lane & 7u) + 16 * ks, half = (lane >> 3) & 1u;
                ldmatrix_x4_trans(a[ks], vals + ch * 1024 + tok * 32 + ((half ^ ((tok >> 2) & 1u)) << 4));
            }
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                mma_16816(acc[ch], a[ks], p_hi[2 * ks], p_hi[2 * ks + 1]);
                mma_16816(acc[ch], a[ks], p_lo[2 * ks], p_lo[2 * ks + 1]);
            }
        }
    }
    if (cur_bh >= 0) flush(cur_bh);
}


}  // namespace

// ecco_fused_scalar_kernels.cuh -- K2 / K3: fused GEMV and attention scores for one or two dot products per group
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

namespace {

// The fused kernels decode one symbol per lookup (shape tables only) and leave the pair tables out of shared memory:
// measured on the 7B-shaped matrices and the cfg-3 K cache, the room the pair tables take (fewer resident warps) costs
// them as much as two-symbol lookups save, and on KV caches, whose codebooks spread over three dozen code shapes,
// escapes make the pair path the slower one.
constexpr bool kFusedPairs = false;

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
__device__ __forceinline__ void fused_group(const Block& blk, const Tables& tb, const WarpSmem& ws, float T,
                                            uint32_t xs, Accum<kV>& acc)
{
    const GroupHeader h = open_group<kTabFloat>(blk, tb, ws, T);
    RankPacker rk;
    const uint32_t end = decode_symbols<true, 16, kBlockBits, kFusedFree>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t pair) {
        acc.fma(n, __uint_as_float(v), xs);
        rk.put(n, pair, ws.syms);
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
            const uint32_t rank = (word >> ((loc & 7u) * 4)) & 15u;
            const float mapped = __uint_as_float(lds_u32(ws.tab + rank * 128));
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

// per-warp arrays of the scalar fused kernels: value table (fp32), bit-stream array, decoded ranks
constexpr uint32_t kFusedWarpBytes = kTabBytes + kBitsBytes + kSymsBytes;
__device__ __forceinline__ WarpSmem fused_warp_smem(const Tables& tb, uint32_t nw)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    WarpSmem ws;
    ws.tab = tab_column<kTabFloat>(tb.warp_base, warp, lane);
    ws.bits = tb.warp_base + nw * kTabBytes + warp * (kBitsBytes + kSymsBytes) + lane * 4;
    ws.syms = ws.bits + kBitsBytes;
    if (warp < nw) {
        sts_u32(ws.bits + 16 * 128, 0u);
        sts_u32(ws.bits + 17 * 128, 0u);
    }
    return ws;
}

// One call of the fused GEMV may cover several matrices (ecco_gemv_batch): the units of all of them form one unit
// space, dealt out to the working warps as one, so that a group of small matrices pays one launch, one table fetch and
// one tail.  All matrices of a call share the decode tables (equal table hash; only the exponent differs).
constexpr int kMaxGemvJobs = 8;
struct GemvJob {
    const uint8_t* meta;       // metadata image of this matrix (its exponent factor T is read from here)
    const uint8_t* blocks;
    const __half* x;           // [kV or batch][k]
    float* y;                  // [batch][n_out]
    int32_t n_out, kblocks;
    int32_t tile_first;        // first 32-row tile of this matrix in the call's tile space (tickets and slots)
    int32_t reserved;
    int64_t unit_first;        // first unit of this matrix in the call's unit space
};
struct GemvBatch {
    int32_t n, reserved;
    int64_t units;             // of all matrices
    GemvJob job[kMaxGemvJobs];
};
// true (uniformly over the grid) if every matrix of the call carries the tables of the first
__device__ __forceinline__ bool same_tables(const GemvBatch& batch, const Tables& tb)
{
    bool same = true;
    for (int t = 1; t < batch.n; ++t) {
        const DevHeader* hd = reinterpret_cast<const DevHeader*>(batch.job[t].meta);
        same = same && __ldg(&hd->hash_lo) == tb.hash_lo && __ldg(&hd->hash_hi) == tb.hash_hi;
    }
    if (!same && threadIdx.x == 0) atomicExch(&g_device_status, ECCO_ERR_INVALID_ARG);
    return same;
}

// Where a unit sits: matrix, 32-row tile and k-block.  Units are visited in order, so the position is advanced by one
// instead of being divided out of the unit number every time.
struct GemvPos { int j, tile, kb; };
__device__ __forceinline__ GemvPos gemv_pos_of(const GemvBatch& batch, int64_t u)
{
    GemvPos p = {0, 0, 0};
    while (p.j + 1 < batch.n && u >= batch.job[p.j + 1].unit_first) ++p.j;
    const int64_t lu = u - batch.job[p.j].unit_first;
    p.tile = static_cast<int>(lu / batch.job[p.j].kblocks);
    p.kb = static_cast<int>(lu % batch.job[p.j].kblocks);
    return p;
}
__device__ __forceinline__ GemvPos gemv_pos_next(const GemvBatch& batch, GemvPos p)
{
    if (++p.kb == batch.job[p.j].kblocks) {
        p.kb = 0;
        if (++p.tile == (batch.job[p.j].n_out + 31) / 32) { p.tile = 0; ++p.j; }
    }
    return p;
}
__device__ __forceinline__ const uint8_t* gemv_block_ptr(const GemvBatch& batch, const GemvPos& p, int lane)
{
    const GemvJob& jb = batch.job[p.j];
    const int row = min(p.tile * 32 + lane, jb.n_out - 1);                         // rows past the end: repeat the last
    return jb.blocks + (static_cast<uint64_t>(row) * jb.kblocks + p.kb) * kBlockBytes;
}

// K2 for one or two rows of x: the slice is small enough (512 B or 1 KB) for every warp to keep
// its own, so warps never meet at a barrier.  A work unit is (32 consecutive rows, one k-block),
// numbered matrix by matrix, row-tile major; every working warp owns a contiguous run of units and keeps its
// rows' partial sums in registers along k.  When a row tile is shared by several warps each writes its
// partial sums to its own workspace slot (slot = global warp id + row tile: unique along the
// staircase of (warp, tile) pairs) and the last to arrive (ticket counter) adds the slots in warp
// order: the result does not depend on scheduling.  Workspace: partial[slot][kV][32] floats, then
// one ticket per 32-row tile.
template <int kV, int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_gemv_warp_kernel(const __grid_constant__ GemvBatch batch, float* __restrict__ d_partial, unsigned int* __restrict__ d_tickets)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr uint32_t kXsBytes = kGroup * kV * 4;
    release_dependents();
    const uint8_t* d_meta = batch.job[0].meta;
    const Tables tb = plan_tables(smem_u32(smem), d_meta, kFusedPairs);
    const int nw = static_cast<int>(warps_that_fit(tb, kFusedWarpBytes + kXsBytes));
    const WarpSmem ws = fused_warp_smem(tb, nw);
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    const uint32_t xs = tb.warp_base + nw * kFusedWarpBytes + warp * kXsBytes;   // this warp's slice

    // W working warps (chosen so that they all get the same number of units, and never more than there are
    // units); warp ids interleave over the CTAs; the other warps idle
    const int wg = warp < nw ? warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x) : INT_MAX;
    const int64_t U = batch.units;
    const int W = static_cast<int>(balanced_warps(static_cast<uint64_t>(U), gridDim.x * static_cast<uint32_t>(nw)));
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    issue_tables(tb, d_meta);
    if (!same_tables(batch, tb)) {                         // images are host-written: readable before the wait
        wait_tables(tb);                                   // the table copies into this CTA's shared memory must land first
        return;
    }
    dependency_wait();                                     // everything but the host-written tables: after the previous kernel of the stream
    GemvPos pos = {0, 0, 0};
    if (u0 < u1) { pos = gemv_pos_of(batch, u0); prefetch_block_l2(gemv_block_ptr(batch, pos, lane)); }
    if (!wait_tables(tb)) return;

    Accum<kV> acc;
    acc.clear();
    auto flush = [&](int jf, int tile) {
        const GemvJob& jb = batch.job[jf];
        const int n_out = jb.n_out, kblocks = jb.kblocks, gtile = jb.tile_first + tile;
        float* d_y = jb.y;
        const int row = tile * 32 + lane;
        const bool row_ok = row < n_out;
        const int64_t g0 = jb.unit_first + static_cast<int64_t>(tile) * kblocks;
        const int w_lo = unit_owner(U, W, g0);
        const int w_hi = unit_owner(U, W, g0 + kblocks - 1);
        if (w_lo == w_hi) {
            if (row_ok) {
#pragma unroll
                for (int b = 0; b < kV; ++b) d_y[static_cast<size_t>(b) * n_out + row] = acc.a[b];
            }
            return;
        }
        float* mine = d_partial + static_cast<size_t>(wg + gtile) * kV * 32;
#pragma unroll
        for (int b = 0; b < kV; ++b) mine[b * 32 + lane] = acc.a[b];
        __threadfence();
        __syncwarp();
        unsigned int t = 0;
        if (lane == 0) t = atomicAdd(&d_tickets[gtile], 1u);
        t = __shfl_sync(0xffffffffu, t, 0);
        if (t == static_cast<unsigned int>(w_hi - w_lo)) {  // last of the warps that share this tile
            __threadfence();
            if (row_ok) {
#pragma unroll
                for (int b = 0; b < kV; ++b) {
                    // slots are added in warp order whatever the arrival order; loads go out thirty-two at a time (a
                    // 4096-wide row is 32 k-blocks: one round trip to L2 instead of two at the end of the kernel)
                    const float* slot = d_partial + (static_cast<size_t>(w_lo + gtile) * kV + b) * 32 + lane;
                    float sum = 0.0f;
                    int ww = w_lo;
                    for (; ww + 32 <= w_hi + 1; ww += 32, slot += 32 * kV * 32) {
                        float v[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __ldcg(slot + i * kV * 32);
#pragma unroll
                        for (int i = 0; i < 32; ++i) sum += v[i];
                    }
                    for (; ww + 8 <= w_hi + 1; ww += 8, slot += 8 * kV * 32) {
                        float v[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[i] = __ldcg(slot + i * kV * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i) sum += v[i];
                    }
                    for (; ww <= w_hi; ++ww, slot += kV * 32) sum += __ldcg(slot);
                    d_y[static_cast<size_t>(b) * n_out + row] = sum;
                }
            }
            if (lane == 0) d_tickets[gtile] = 0;
        }
    };

    // x for a unit is fetched one unit ahead, like the block
    uint2 xraw[kV];
    auto load_x = [&](const GemvPos& p) {
        const GemvJob& jb = batch.job[p.j];
        const size_t k = static_cast<size_t>(jb.kblocks) * kGroup;
#pragma unroll
        for (int b = 0; b < kV; ++b)
            xraw[b] = __ldcg(reinterpret_cast<const uint2*>(jb.x + static_cast<size_t>(b) * k + p.kb * kGroup + lane * 4));
    };
    if (u0 >= u1) return;
    load_x(pos);
    int cur_j = pos.j, cur_tile = pos.tile;
    float T = __ldg(&reinterpret_cast<const DevHeader*>(batch.job[pos.j].meta)->T);
    for (int64_t u = u0; u < u1; ++u) {
        if (pos.j != cur_j || pos.tile != cur_tile) {
            flush(cur_j, cur_tile);
            acc.clear();
            if (pos.j != cur_j) T = __ldg(&reinterpret_cast<const DevHeader*>(batch.job[pos.j].meta)->T);
            cur_j = pos.j;
            cur_tile = pos.tile;
        }
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
        // the block is fetched when its turn comes (it was prefetched into L2 one unit earlier): holding the next
        // one in sixteen registers through a whole group costs more in resident warps than the fetch costs here
        Block cur;
        ldg_block(cur, gemv_block_ptr(batch, pos, lane));
        if (u + 1 < u1) {
            pos = gemv_pos_next(batch, pos);
            prefetch_block_l2(gemv_block_ptr(batch, pos, lane));
            load_x(pos);
        }
        fused_group<kV>(cur, tb, ws, T, xs, acc);
    }
    flush(cur_j, cur_tile);
}

// K3: scores[b][hq][t] = scale * q[b][hq] . K~[b][hq / q_per_kv][t] for one or two query heads per KV head.
// Built like K2: a work unit is (one (batch, kv head) pair, 32 consecutive tokens), a lane owns one token, every
// working warp owns a contiguous run of units and keeps its own query slice (pre-multiplied by scale, restaged
// when the head changes), so warps never meet at a barrier and a ragged sequence length costs at most one
// partly filled unit per head.
template <int kV, int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_attn_scores_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_kblocks, int heads, int seq,
                        int q_per_kv, const __half* d_q, float scale, float* __restrict__ d_scores)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr uint32_t kXsBytes = kGroup * kV * 4;
    release_dependents();
    const Tables tb = plan_tables(smem_u32(smem), d_meta, kFusedPairs);
    const int nw = static_cast<int>(warps_that_fit(tb, kFusedWarpBytes + kXsBytes));
    const WarpSmem ws = fused_warp_smem(tb, nw);
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    const uint32_t xs = tb.warp_base + nw * kFusedWarpBytes + warp * kXsBytes;   // this warp's slice: xs[d][r]

    const int wg = warp < nw ? warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x) : INT_MAX;
    const int tiles = (seq + 31) / 32;
    const int64_t U = static_cast<int64_t>(heads) * tiles;
    const int W = static_cast<int>(balanced_warps(static_cast<uint64_t>(U), gridDim.x * static_cast<uint32_t>(nw)));
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    // lanes past the end of the sequence decode its last token again and store nothing; (head, tile) of a unit is
    // advanced by one per unit instead of divided out of the unit number
    auto block_ptr = [&](int bh, int tile) {
        return d_kblocks + (static_cast<uint64_t>(bh) * seq + min(tile * 32 + lane, seq - 1)) * kBlockBytes;
    };
    int bh = static_cast<int>(u0 / tiles), tile = static_cast<int>(u0 % tiles);
    issue_tables(tb, d_meta);
    dependency_wait();                                     // everything but the host-written tables: after the previous kernel of the stream
    if (u0 < u1) prefetch_block_l2(block_ptr(bh, tile));
    if (!wait_tables(tb)) return;
    const float T = tb.T;

    int cur_bh = -1;
    for (int64_t u = u0; u < u1; ++u) {
        const int t = tile * 32 + lane;
        if (bh != cur_bh) {
            // lane l stages q[b][h*q_per_kv + r][4l .. 4l+3] * scale as fp32, layout xs[d][r]; heads beyond q_per_kv are zero
            float v[kV][4];
#pragma unroll
            for (int r = 0; r < kV; ++r) {
                uint2 raw = make_uint2(0u, 0u);
                if (r < q_per_kv) raw = __ldcg(reinterpret_cast<const uint2*>(d_q + (static_cast<size_t>(bh) * q_per_kv + r) * kGroup) + lane);
                const __half2 h0 = *reinterpret_cast<const __half2*>(&raw.x), h1 = *reinterpret_cast<const __half2*>(&raw.y);
                v[r][0] = scale * __low2float(h0); v[r][1] = scale * __high2float(h0);
                v[r][2] = scale * __low2float(h1); v[r][3] = scale * __high2float(h1);
            }
            __syncwarp();                                  // every lane is done with the previous head's slice
            if constexpr (kV == 1) {
                sts_v4(xs + lane * 16, __float_as_uint(v[0][0]), __float_as_uint(v[0][1]), __float_as_uint(v[0][2]), __float_as_uint(v[0][3]));
            } else {
                sts_v4(xs + lane * 32, __float_as_uint(v[0][0]), __float_as_uint(v[1][0]), __float_as_uint(v[0][1]), __float_as_uint(v[1][1]));
                sts_v4(xs + lane * 32 + 16, __float_as_uint(v[0][2]), __float_as_uint(v[1][2]), __float_as_uint(v[0][3]), __float_as_uint(v[1][3]));
            }
            __syncwarp();
            cur_bh = bh;
        }
        Block cur;
        ldg_block(cur, block_ptr(bh, tile));
        const int out_bh = bh;
        if (++tile == tiles) { tile = 0; ++bh; }
        if (u + 1 < u1) prefetch_block_l2(block_ptr(bh, tile));
        Accum<kV> acc;
        acc.clear();
        fused_group<kV>(cur, tb, ws, T, xs, acc);
        if (t < seq) {
#pragma unroll
            for (int r = 0; r < kV; ++r)
                if (r < q_per_kv) d_scores[(static_cast<size_t>(out_bh) * q_per_kv + r) * seq + t] = acc.a[r];
        }
    }
}


}  // namespace

// ecco_fused_mma_kernels.cuh -- K2m / K3m: fused GEMV and attention scores for three to eight dot products per group (tensor cores)
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

namespace {

// ---------------------------------------------------------------------------------------------
// K2m / K3m: the fused consumers for 3 to 8 dot products per group (rows of x, query heads) on the
// tensor cores.  With eight products per weight the scalar path spends four shared-memory
// wavefronts and eight FMAs per symbol on the vector operand alone.  Here a group is decoded once,
// values and all, into eight [32 rows][16 k] fp16 tiles of the warp (as in K5); when the end bit is
// known the outliers are written over their positions; then each tile is contracted against the fp16
// vector fragments: C[32 rows][8] += tile[32 x 16] * V[16 x 8], two mma.m16n8k16 per tile, fp32
// accumulate (fp16 x fp16 products are exact in fp32).  A warp is independent of the others: no
// vector slice in shared memory, no block barrier.
// ---------------------------------------------------------------------------------------------
// Eight [32 rows][16 k] fp16 tiles per warp, the last of which lies over rows 0..7 of the warp's bit-stream array: it
// is written when symbol 127 has been decoded, and by then every lane is past stream bit 256 (22 header bits at least
// and two bits per symbol), while the outlier fields sit in bits 272..511, rows 8..15.
constexpr uint32_t kMmaValueBytes = 7 * 1024;
constexpr uint32_t kMmaWarpBytes = kTabBytes / 2 + kMmaValueBytes + kBitsBytes;   // half a value table (two warps share one), tiles, bit stream
// value tables first, then per warp the tiles and the bit-stream array; *vals = the warp's first tile
__device__ __forceinline__ WarpSmem mma_warp_smem(const Tables& tb, uint32_t nw, uint32_t* vals)
{
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    WarpSmem ws;
    ws.tab = tab_column<kTabHalf>(tb.warp_base, warp, lane);
    *vals = tb.warp_base + tab_bytes<kTabHalf>(nw) + warp * (kMmaValueBytes + kBitsBytes);
    ws.bits = *vals + kMmaValueBytes + lane * 4;
    ws.syms = 0;
    if (warp < nw) {
        sts_u32(ws.bits + 16 * 128, 0u);
        sts_u32(ws.bits + 17 * 128, 0u);
    }
    return ws;
}

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
// fetch_vectors(vfrag) is called after the decode: a caller whose vectors change with every group (the GEMV)
// loads them there, so that they do not occupy sixteen registers during the decode; one whose vectors stay
// (the scores) copies them.
__device__ __forceinline__ void load_vfrag(uint32_t (&vfrag)[16], const __half* base, size_t col_stride, int n_cols);

template <class FetchVectors>
__device__ __forceinline__ void row_dot_mma(const Block& blk, const Tables& tb, const WarpSmem& ws, uint32_t vals, float T,
                                            FetchVectors&& fetch_vectors, float (&acc)[2][4])
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t swz = ((lane >> 2) & 1u) << 4, my_row = vals + lane * 32;
    __syncwarp();                                          // the tiles of the previous group have been read (the last one is
    const GroupHeader h = open_group<kTabHalf>(blk, tb, ws, T);     // about to be overwritten by this group's stream)
    uint32_t r8[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    const uint32_t end = decode_symbols<true, 16, kBlockBits, kFusedFree, kTabHalf>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t) {
        const int col = tile_column(n & 15);               // see load_vfrag; clipped positions arrive as +0
        if (col & 1) r8[col >> 1] = __byte_perm(r8[col >> 1], v, 0x5410); else r8[col >> 1] = v;   // the even column of a pair comes first
        if ((n & 15) == 15) {
            const uint32_t row = my_row + (n >> 4) * 1024;
            sts_v4(row + swz, r8[0], r8[1], r8[2], r8[3]);
            sts_v4(row + (swz ^ 16u), r8[4], r8[5], r8[6], r8[7]);
        }
    });
    uint32_t vfrag[16];
    fetch_vectors(vfrag);
    // outliers of a complete group replace the mapped values in the tiles (ascending: a later pad overrides an earlier
    // one).  Rows past the end of the matrix or the sequence decode the last one again; their results are not stored.
    const int n_pad = end ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
    for (int j = 0; j < n_pad; ++j) {
        const uint32_t f = read_pad(ws, j);
        const uint32_t loc = f & 127u, i = loc & 15u;
        const uint32_t byte = (2u * (i >> 2) + (i & 1u) + 8u * ((i >> 1) & 1u)) * 2u;          // tile_column(i) * 2
        asm volatile("st.shared.u16 [%0], %1;" ::"r"(my_row + (loc >> 4) * 1024 + ((byte & 16u) ^ swz) + (byte & 15u)),
                     "h"(static_cast<unsigned short>(f2h_bits(fp8_to_float(f >> 7) * T))) : "memory");
    }
    __syncwarp();                                          // tiles complete
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) {
            const uint32_t row = ((lane >> 3) & 1u) * 8 + (lane & 7u) + 16 * mt, half = lane >> 4;
            uint32_t a[4];
            ldmatrix_x4(a, vals + ch * 1024 + row * 32 + ((half ^ ((row >> 2) & 1u)) << 4));
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
        const uint2 v = col < n_cols ? __ldcg(p + c * 4) : make_uint2(0u, 0u);     // k = 16c + 4 (lane%4) .. + 3
        vfrag[2 * c] = v.x;                                // tile columns 2q, 2q+1
        vfrag[2 * c + 1] = v.y;                            // tile columns 2q+8, 2q+9
    }
}

// K2m: y[b][n] = sum_k W~[n][k] x[b][k] for 3..8 rows of x.  Units (over all matrices of the call), ownership and the
// slot-and-ticket reduction are those of the per-warp kernel (unit = 32 rows x one k-block).
template <int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_gemv_mma_kernel(const __grid_constant__ GemvBatch batch, int n_cols, float* __restrict__ d_partial,
                     unsigned int* __restrict__ d_tickets)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    release_dependents();
    const uint8_t* d_meta = batch.job[0].meta;
    const Tables tb = plan_tables(smem_u32(smem), d_meta, false);   // one symbol per lookup: see the scalar kernels
    const int nw = static_cast<int>(warps_that_fit(tb, kMmaWarpBytes, kTabBytes / 2));
    uint32_t stage;
    const WarpSmem ws = mma_warp_smem(tb, nw, &stage);

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
    if (u0 >= u1) return;

    float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    // C fragment element (mt, i): row = 16 mt + lane/4 + 8 (i >= 2), column b = (lane%4)*2 + (i & 1)
    auto flush = [&](int jf, int tile) {
        const GemvJob& jb = batch.job[jf];
        const int n_out = jb.n_out, kblocks = jb.kblocks, gtile = jb.tile_first + tile;
        float* d_y = jb.y;
        const int64_t g0 = jb.unit_first + static_cast<int64_t>(tile) * kblocks;
        const int w_lo = unit_owner(U, W, g0);
        const int w_hi = unit_owner(U, W, g0 + kblocks - 1);
        float* mine = d_partial + static_cast<size_t>(wg + gtile) * 8 * 32;
        if (w_lo != w_hi) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    mine[((lane & 3) * 2 + (i & 1)) * 32 + 16 * mt + (lane >> 2) + (i >= 2 ? 8 : 0)] = acc[mt][i];
            __threadfence();
            __syncwarp();
            unsigned int t = 0;
            if (lane == 0) t = atomicAdd(&d_tickets[gtile], 1u);
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
                    for (int ww = w_lo; ww <= w_hi; ++ww) sum += __ldcg(d_partial + (static_cast<size_t>(ww + gtile) * 8 + b) * 32 + r);
                }
                if (row < n_out && b < n_cols) d_y[static_cast<size_t>(b) * n_out + row] = sum;
            }
        if (w_lo != w_hi && lane == 0) d_tickets[gtile] = 0;
    };

    int cur_j = pos.j, cur_tile = pos.tile;
    float T = __ldg(&reinterpret_cast<const DevHeader*>(batch.job[pos.j].meta)->T);
    for (int64_t u = u0; u < u1; ++u) {
        const GemvJob& jb = batch.job[pos.j];
        const int tile = pos.tile;
        if (pos.j != cur_j || tile != cur_tile) {
            flush(cur_j, cur_tile);
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][i] = 0.0f;
            if (pos.j != cur_j) T = __ldg(&reinterpret_cast<const DevHeader*>(jb.meta)->T);
            cur_j = pos.j;
            cur_tile = tile;
        }
        Block cur;                                         // fetched now, prefetched into L2 one unit earlier (see the scalar kernels)
        ldg_block(cur, gemv_block_ptr(batch, pos, lane));
        const __half* xk = jb.x + pos.kb * kGroup;
        const size_t k = static_cast<size_t>(jb.kblocks) * kGroup;
        if (u + 1 < u1) { pos = gemv_pos_next(batch, pos); prefetch_block_l2(gemv_block_ptr(batch, pos, lane)); }
        row_dot_mma(cur, tb, ws, stage, T, [&](uint32_t (&v)[16]) { load_vfrag(v, xk, k, n_cols); }, acc);
    }
    flush(cur_j, cur_tile);
}

// K3m: scores[b][hq][t] = scale * q[b][hq] . K~[b][hq / q_per_kv][t] for 3..8 query heads per KV head.
// Unit = (one (batch, kv head), 32 tokens); every working warp owns a contiguous run of units.
template <int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_attn_scores_mma_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_kblocks, int heads, int seq,
                            int q_per_kv, const __half* d_q, float scale, float* __restrict__ d_scores)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int lane = static_cast<int>(threadIdx.x & 31u), warp = static_cast<int>(threadIdx.x >> 5);
    release_dependents();
    const Tables tb = plan_tables(smem_u32(smem), d_meta, false);   // one symbol per lookup: see the scalar kernels
    const int nw = static_cast<int>(warps_that_fit(tb, kMmaWarpBytes, kTabBytes / 2));
    uint32_t stage;
    const WarpSmem ws = mma_warp_smem(tb, nw, &stage);

    const int wg = warp < nw ? warp * static_cast<int>(gridDim.x) + static_cast<int>(blockIdx.x) : INT_MAX;
    const int tiles = (seq + 31) / 32;
    const int64_t U = static_cast<int64_t>(heads) * tiles;
    const int W = static_cast<int>(balanced_warps(static_cast<uint64_t>(U), gridDim.x * static_cast<uint32_t>(nw)));
    const int64_t u0 = wg < W ? unit_begin(U, W, wg) : 0, u1 = wg < W ? unit_begin(U, W, wg + 1) : 0;
    auto block_ptr = [&](int bh, int tile) {
        return d_kblocks + (static_cast<uint64_t>(bh) * seq + min(tile * 32 + lane, seq - 1)) * kBlockBytes;
    };
    int nbh = static_cast<int>(u0 / tiles), ntile = static_cast<int>(u0 % tiles);     // advanced by one per unit
    issue_tables(tb, d_meta);
    dependency_wait();                                     // everything but the host-written tables: after the previous kernel of the stream
    if (u0 < u1) prefetch_block_l2(block_ptr(nbh, ntile));
    if (!wait_tables(tb)) return;
    const float T = tb.T;

    uint32_t vfrag[16];
    int cur_bh = -1;
    for (int64_t u = u0; u < u1; ++u) {
        const int bh = nbh, t0 = ntile * 32;
        if (bh != cur_bh) { load_vfrag(vfrag, d_q + static_cast<size_t>(bh) * q_per_kv * kGroup, kGroup, q_per_kv); cur_bh = bh; }
        Block cur;
        ldg_block(cur, block_ptr(nbh, ntile));
        if (++ntile == tiles) { ntile = 0; ++nbh; }
        if (u + 1 < u1) prefetch_block_l2(block_ptr(nbh, ntile));
        float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        row_dot_mma(cur, tb, ws, stage, T,
                    [&](uint32_t (&v)[16]) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = vfrag[i];
                    }, acc);
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int t = t0 + 16 * mt + (lane >> 2) + (i >= 2 ? 8 : 0), r = (lane & 3) * 2 + (i & 1);
                if (t < seq && r < q_per_kv) d_scores[(static_cast<size_t>(bh) * q_per_kv + r) * seq + t] = scale * acc[mt][i];
            }
    }
}


}  // namespace

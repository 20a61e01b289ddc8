// ecco_decompress_kernels.cuh -- K1 / K1v: ecco_decompress and ecco_var_decompress kernels
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

namespace {

// ---------------------------------------------------------------------------------------------
// K1: ecco_decompress
// ---------------------------------------------------------------------------------------------
// number of working warps <= w_max such that `units` split evenly: all get ceil(units / w_max) or one less
__host__ __device__ __forceinline__ uint32_t balanced_warps(uint64_t units, uint32_t w_max)
{
    if (units <= w_max) return static_cast<uint32_t>(units);
    const uint64_t per_warp = (units + w_max - 1) / w_max;
    return static_cast<uint32_t>((units + per_warp - 1) / per_warp);
}

// Work is dealt out in warp tiles of 32 consecutive groups, tile i to warp (i mod working warps):
// every SM then gets the same number of tiles to within one, whatever the tensor size.
constexpr uint32_t kSmallWarpBytes = kTabBytes / 2 + kBitsBytes;   // half a value table (two warps share one), bit-stream array
template <int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_decompress_kernel(const uint8_t* __restrict__ d_meta, const uint8_t* __restrict__ d_blocks, uint64_t n_groups,
                       uint16_t* __restrict__ d_out)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const Tables tb = plan_tables(smem_u32(smem), d_meta);
    const uint32_t nw = warps_that_fit(tb, kSmallWarpBytes, kTabBytes / 2);   // an odd warp count leaves half a table unused
    WarpSmem ws;
    ws.tab = tab_column<kTabHalf>(tb.warp_base, warp, lane);
    ws.bits = tb.warp_base + tab_bytes<kTabHalf>(nw) + warp * kBitsBytes + lane * 4;
    ws.syms = 0;
    if (warp < nw) {
        sts_u32(ws.bits + 16 * 128, 0u);
        sts_u32(ws.bits + 17 * 128, 0u);
    }
    const uint64_t n_tiles = (n_groups + 31) / 32;
    // every working warp gets the same number of tiles (+-1 over the whole grid); warp ids interleave over
    // the CTAs, so every SM keeps the same number busy
    const uint64_t tile_stride = balanced_warps(n_tiles, gridDim.x * nw);
    uint64_t tile = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;
    if (warp >= nw || tile >= tile_stride) tile = n_tiles;               // this warp sits the launch out (after the table barrier)
    Block blk;
    // lanes past the end of the tensor decode the last group again and store nothing
    if (tile < n_tiles) ldg_block(blk, d_blocks + min(tile * 32 + lane, n_groups - 1) * kBlockBytes);
    issue_tables(tb, d_meta);
    if (!wait_tables(tb)) return;
    const float T = tb.T;

    for (; tile < n_tiles; tile += tile_stride) {
        const uint64_t g = tile * 32 + lane;
        const bool store = g < n_groups;
        const GroupHeader h = open_group<kTabHalf>(blk, tb, ws, T);
        const uint64_t tn = tile + tile_stride;
        if (tn < n_tiles)                                  // next block in flight while this one decodes
            ldg_block(blk, d_blocks + min(tn * 32 + lane, n_groups - 1) * kBlockBytes);
        uint16_t* out = d_out + min(g, n_groups - 1) * kGroup;
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        const uint32_t end = decode_symbols<true, 16, kBlockBits, 0, kTabHalf>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t) {
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
//
// The kernel takes up to kMaxJobs tensors.  Consecutive tensors whose images carry the same tables (equal table
// hash: the matrices of a layer calibrated together differ in the exponent only) form a run: the tables are
// staged once per run and the warp tiles of all its tensors are dealt out as one tile space, so a run pays one
// table fetch and one tail.  Between two runs only the CTA's own warps meet (the tables are the CTA's), so an SM
// that is done with one run starts the next while others still finish.
constexpr int kMaxJobs = 8;
struct alignas(64) DecompressJob {
    const uint8_t* meta;
    const uint8_t* blocks;
    uint64_t n_groups;
    uint16_t* out;
    uint32_t reserved[8];
    CUtensorMap map;           // [n_groups][128] fp16, box 32 x 16, 32-byte swizzle
};
struct DecompressBatch {
    int32_t n;
    int32_t reserved[15];
    DecompressJob job[kMaxJobs];
};
constexpr uint32_t kTmaWarpBytes = kTabBytes / 2 + 1024 + kBitsBytes;   // half a value table (two warps share one), staging tile, bit-stream array

template <int kMaxWarps, int kDecFree = 12>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_decompress_tma_kernel(const __grid_constant__ DecompressBatch batch)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t swz = ((lane >> 2) & 1u) << 4;                               // 32-byte swizzle: bit 4 ^= bit 7

    // The metadata images are written by the host only, never by a kernel of this library, and this kernel can
    // start early only behind a kernel that releases its dependents, i.e. one of this library: the tables of the
    // first run are fetched before the wait on the previous kernel, everything else after it.
    release_dependents();
    auto hash_of = [&](int t) {
        const DevHeader* hd = reinterpret_cast<const DevHeader*>(batch.job[t].meta);
        return make_uint2(__ldg(&hd->hash_lo), __ldg(&hd->hash_hi));
    };
    auto tiles_of = [&](int t) { return (batch.job[t].n_groups + 31) / 32; };
    int run = 0;
    for (int t0 = 0; t0 < batch.n; ++run) {
        const Tables tb = plan_tables(smem_base, batch.job[t0].meta);
        int t1 = t0 + 1;
        uint64_t run_tiles = tiles_of(t0);
        for (; t1 < batch.n; ++t1) {
            const uint2 hh = hash_of(t1);
            if (hh.x != tb.hash_lo || hh.y != tb.hash_hi) break;
            run_tiles += tiles_of(t1);
        }
        if (run > 0) __syncthreads();                      // every warp is done with the previous run's tables
        issue_tables(tb, batch.job[t0].meta, run == 0);
        const uint32_t nw = warps_that_fit(tb, kTmaWarpBytes, kTabBytes / 2);
        WarpSmem ws;
        ws.tab = tab_column<kTabHalf>(tb.warp_base, warp, lane);
        const uint32_t stage = tb.warp_base + tab_bytes<kTabHalf>(nw) + warp * 1024;     // this warp's staging tile
        ws.bits = stage + (nw - warp) * 1024 + warp * kBitsBytes + lane * 4;
        ws.syms = 0;
        const uint32_t my_row = stage + lane * 32;
        if (warp < nw) {
            sts_u32(ws.bits + 16 * 128, 0u);
            sts_u32(ws.bits + 17 * 128, 0u);
        }
        const uint64_t tile_stride = balanced_warps(run_tiles, gridDim.x * nw);
        uint64_t gt = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;       // tile in the run's tile space
        if (warp >= nw || gt >= tile_stride) gt = run_tiles;
        // cursor: the job that holds tile gt, and the first tile of that job in the run's tile space
        struct Cursor { int job; uint64_t first, tiles; };
        Cursor cur = {t0, 0, tiles_of(t0)};
        auto seek = [&](Cursor& c, uint64_t g) {
            while (g >= c.first + c.tiles && c.job + 1 < t1) { c.first += c.tiles; ++c.job; c.tiles = tiles_of(c.job); }
        };
        auto block_ptr = [&](const Cursor& c, uint64_t g) {
            const DecompressJob& job = batch.job[c.job];
            return job.blocks + min((g - c.first) * 32 + lane, job.n_groups - 1) * kBlockBytes;
        };
        if (run == 0) dependency_wait();                   // blocks and output: only after the previous kernel has completed
        if (gt < run_tiles) { seek(cur, gt); prefetch_block_l2(block_ptr(cur, gt)); }
        if (!wait_tables(tb, static_cast<uint32_t>(run & 1))) return;
        float T = tb.T;
        int t_of_T = t0;

        for (; gt < run_tiles; gt += tile_stride) {
            const DecompressJob& job = batch.job[cur.job];
            if (cur.job != t_of_T) { T = __ldg(&reinterpret_cast<const DevHeader*>(job.meta)->T); t_of_T = cur.job; }
            const uint64_t n_groups = job.n_groups;
            const uint64_t tile = gt - cur.first;
            const uint64_t g = tile * 32 + lane;
            const bool store = g < n_groups;
            uint16_t* out = job.out + min(g, n_groups - 1) * kGroup;
            const CUtensorMap* out_map = &job.map;
            const int row0 = static_cast<int>(tile * 32);
            // The block is fetched when its turn comes, after a prefetch into L2 one tile earlier: holding the next
            // block in sixteen registers through a whole group would cost four of the 32 warps.
            Block blk;
            ldg_block(blk, block_ptr(cur, gt));
            const GroupHeader h = open_group<kTabHalf>(blk, tb, ws, T);
            const uint64_t gn = gt + tile_stride;
            if (gn < run_tiles) { seek(cur, gn); prefetch_block_l2(block_ptr(cur, gn)); }
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
                if (lane == 0) { tma_store_2d(out_map, stage, chunk * 16, row0); bulk_commit(); }
            };
            const uint32_t end = decode_symbols<true, 16, kBlockBits, kDecFree, kTabHalf>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t) {
                const int slot = (n & 15) >> 1;
                if (n & 1) r[slot] = __byte_perm(r[slot], v, 0x5410); else r[slot] = v;
                if ((n & 15) == 15 && n != 127) { stage_rows(); send_tile(n >> 4); }
            });
            stage_rows();                                      // values 112..127
            const int n_pad = end ? min(kMaxPads, static_cast<int>((kBlockBits - end) / kPadBits)) : 0;
            if (__any_sync(0xffffffffu, n_pad > 0)) {
                if (lane == 0) bulk_wait_all();                // tiles 0..6 of this group are in memory
                __syncwarp();
                const int n_max = __reduce_max_sync(0xffffffffu, n_pad);
#pragma unroll
                for (int j = 0; j < kMaxPads; ++j) {           // ascending: a later pad overrides an earlier one
                    if (j >= n_max) break;
                    if (j < n_pad) {
                        const uint32_t f = read_pad(ws, j);
                        const uint32_t loc = f & 127u;
                        const unsigned short val = static_cast<unsigned short>(f2h_bits(fp8_to_float(f >> 7) * T));
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
        if (lane == 0) bulk_wait_all();                    // the staging tile may move with the next run's layout
        t0 = t1;
    }
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

constexpr uint32_t kVarWarpBytes = kTabBytes / 2 + 1024 + kVarBitsBytes;

template <int kMaxWarps>
__global__ void __launch_bounds__(kMaxWarps * 32, 1)
ecco_var_decompress_kernel(const uint8_t* __restrict__ d_meta, const uint4* __restrict__ d_stream,
                           const uint64_t* __restrict__ d_index, uint64_t n_groups, uint16_t* __restrict__ d_out,
                           const __grid_constant__ CUtensorMap out_map)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;

    release_dependents();
    // one symbol per lookup: a warp's 40-row stream array takes 5 KB, and 28 warps beside the shape tables measured
    // as fast as 20 beside the pair tables
    const Tables tb = plan_tables(smem_u32(smem), d_meta, false);
    const uint32_t nw = warps_that_fit(tb, kVarWarpBytes, kTabBytes / 2);
    WarpSmem ws;
    ws.tab = tab_column<kTabHalf>(tb.warp_base, warp, lane);
    const uint32_t stage = tb.warp_base + tab_bytes<kTabHalf>(nw) + warp * 1024;
    ws.bits = stage + (nw - warp) * 1024 + warp * kVarBitsBytes + lane * 4;
    ws.syms = 0;
    if (warp < nw)
        for (uint32_t r = 0; r < kVarRows; ++r) sts_u32(ws.bits + r * 128, 0u);
    const uint32_t swz = ((lane >> 2) & 1u) << 4;
    const uint32_t my_row = stage + lane * 32;
    issue_tables(tb, d_meta);
    dependency_wait();                                     // everything but the host-written tables: after the previous kernel of the stream
    const uint64_t total_bits = d_index[0];
    const uint64_t stream_chunks = (total_bits + 127) >> 7;
    const uint64_t* chunk_base = d_index + 1;
    const uint32_t* off32 = reinterpret_cast<const uint32_t*>(d_index + 1 + var_chunks(n_groups));
    auto start_of = [&](uint64_t g) { return g < n_groups ? chunk_base[g >> kVarChunkShift] + off32[g] : total_bits; };

    const uint64_t n_tiles = (n_groups + 31) / 32;
    const uint64_t tile_stride = balanced_warps(n_tiles, gridDim.x * nw);
    uint64_t tile = static_cast<uint64_t>(warp) * gridDim.x + blockIdx.x;
    if (warp >= nw || tile >= tile_stride) tile = n_tiles;
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
        if (c < stream_chunks) asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(d_stream + c));
        return v;
    };
    Span cur = {0, 0, 0, 0};
    uint4 ahead[kVarAhead];
    if (tile < n_tiles) {
        cur = span_of(tile);
#pragma unroll
        for (uint32_t c = 0; c < kVarAhead; ++c) ahead[c] = c < cur.nc ? load_chunk(cur.c0 + c) : make_uint4(0, 0, 0, 0);
    }

    if (!wait_tables(tb)) return;
    const float T = tb.T;

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
        const GroupHeader h = open_header<kTabHalf>(hdr, first_bit, tb, ws, T);
        const int row0 = static_cast<int>(tile * 32);
        uint32_t r[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        decode_symbols<true, kVarRows - 2, kVarRows * 32, 28, kTabHalf>(h, ws, tb.pairs, [&](int n, uint32_t v, uint32_t, bool, uint32_t) {
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


}  // namespace

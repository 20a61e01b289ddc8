// ecco_kernels.cu -- sm_100a kernels and the device half of the C ABI.
//
// One thread owns one group: a 64-byte block is independent of every other block (Sec. 3.2,
// "all group-wise information ... compressed to a fixed compressed block size"), so the decoder
// runs the serial Huffman chain (Sec. 4.2) once per thread and takes its parallelism across
// groups, not inside a group.  The lanes of a warp advance symbol by symbol in lock step, which
// keeps every per-symbol index (output position, activation element) uniform across the warp.
//
// Shared memory per CTA (sizes from the image's header, see ecco_device_core.cuh):
//   tables   pattern[64][16] fp16 | ID_KP table [4096] u16 | codebook records [256] x 16 B | shape tables
//            [n_shapes][256] u8 | pair tables, brought in by three bulk copies (cp.async.bulk + mbarrier)
//   per warp tab[16][32]  u32   per-lane dequantised centroids in rank order (the rank of the abs-max symbol
//                               holds the abs-max); fp32 in the scalar fused kernels, fp16 with two warps to an
//                               array elsewhere
//            bits[18][32] u32   the warp's 32 blocks, word-transposed: lane L's word w at
//                               [w][L] -> bank L whatever w is (conflict-free refills);
//                               rows 16 and 17 stay zero (stream bits past 512 read as 0)
//            syms[16][32] u32   (scalar fused kernels) decoded ranks, 8 nibbles per word, for the
//                               outlier fix-up
//            tiles              ecco_decompress: one [32 groups][16 values] fp16 staging tile for the tensor stores;
//                               tensor-core kernels: eight of them, the whole decoded group, as MMA operands
//
// Layout of the sources (one translation unit; the .cuh files are included here and nowhere else):
//   ecco_device_core.cuh            shared-memory layout, PTX helpers, table staging, the per-group decoder
//   ecco_decompress_kernels.cuh     ecco_decompress (tile-store and small-tensor kernels), ecco_var_decompress
//   ecco_fused_scalar_kernels.cuh   fused GEMV / attention scores, one or two dot products per group
//   ecco_fused_mma_kernels.cuh      the same for three to eight dot products, on the tensor cores
//   ecco_attn_values_kernels.cuh    softmax(scores) . V over a compressed V cache
//   ecco_act2x_kernels.cuh          2x activation codec
//   ecco_kv_compress_kernel.cuh     online 4x compressor
//   ecco_launch.cuh                 device query, overlapped launches, work plans
//   this file                       the C ABI: argument checks and launches
#include "ecco_device_core.cuh"
#include "ecco_decompress_kernels.cuh"
#include "ecco_fused_scalar_kernels.cuh"
#include "ecco_attn_values_kernels.cuh"
#include "ecco_fused_mma_kernels.cuh"
#include "ecco_launch.cuh"
#include "ecco_act2x_kernels.cuh"
#include "ecco_kv_compress_kernel.cuh"


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

// Diagnostics: the give-up path of the bounded wait, exercised without anything that could hang.  The kernel arms a
// barrier with a byte count that no copy will ever deliver (nothing is in flight, so the CTA may exit at any time),
// polls it a few hundred times, gives up, records the time-out and returns normally.
namespace {
__global__ void ecco_wait_timeout_probe_kernel()
{
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        mbar_expect_tx(b, 64);
    }
    (void)bounded_wait(b, 0, 256);
}
}  // namespace
extern "C" int ecco_test_wait_timeout(void* stream)
{
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    ecco_wait_timeout_probe_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>();
    return check_launch();
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

constexpr int kDecompressTmaWarps = 32;

// every decoding kernel asks for all the shared memory of an SM and lays itself out on the device
template <class K>
static int want_all_smem(K kernel, bool* configured)
{
    if (*configured) return ECCO_OK;
    const int rc = set_smem(kernel, kSmemCtaBytes);
    if (rc == ECCO_OK) *configured = true;
    return rc;
}

// tensors of fewer than 32 groups (the tile store's box is 32 rows tall), or when no tensor map can be made
static int launch_decompress_small(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, void* d_out,
                                   cudaStream_t stream)
{
    static thread_local bool configured[64] = {};
    auto kernel = ecco_decompress_kernel<kDecompressWarps>;
    int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    const uint64_t cta_tiles = (n_groups + kDecompressWarps * 32 - 1) / (kDecompressWarps * 32);   // one tile per warp
    const unsigned grid = static_cast<unsigned>(cta_tiles < static_cast<uint64_t>(di.sms) ? cta_tiles : di.sms);
    kernel<<<grid, kDecompressWarps * 32, kSmemCtaBytes, stream>>>(static_cast<const uint8_t*>(d_meta), d_blocks, n_groups,
                                                                   static_cast<uint16_t*>(d_out));
    return check_launch();
}

// one launch of the tile-store kernel over batch.n tensors (maps already made)
static int launch_decompress_batch(const DeviceInfo& di, DecompressBatch& batch, cudaStream_t stream)
{
    static thread_local bool configured[64] = {};
    auto kernel = ecco_decompress_tma_kernel<kDecompressTmaWarps>;
    int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    uint64_t tiles = 0;
    for (int t = 0; t < batch.n; ++t) tiles += (batch.job[t].n_groups + 31) / 32;
    const uint64_t ctas = (tiles + kDecompressTmaWarps - 1) / kDecompressTmaWarps;
    const unsigned grid = static_cast<unsigned>(ctas < static_cast<uint64_t>(di.sms) ? ctas : di.sms);
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kDecompressTmaWarps * 32), kSmemCtaBytes, stream, batch);
}

// The tile-store kernel addresses output rows with the 32-bit signed coordinates of the TMA unit: tensors of 2^31 groups
// (256 GiB of fp16) or more are refused.
constexpr uint64_t kMaxGroups = (1ull << 31) - 32;

static int check_decompress_args(const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, const void* d_out)
{
    if (!d_meta || !d_blocks || !d_out) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_blocks) || !aligned16(d_out)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > kMaxGroups) return ECCO_ERR_INVALID_ARG;
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

constexpr int kVarWarps = 28;

extern "C" int ecco_var_decompress(const void* d_meta, const uint8_t* d_stream, const void* d_index, uint64_t n_groups, void* d_out,
                                   void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_meta || !d_stream || !d_index || !d_out) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_stream) || !aligned16(d_out) || (reinterpret_cast<uintptr_t>(d_index) & 7u)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > kMaxGroups) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    // rows past the end of the tensor are dropped by the tile store, so any n_groups >= 1 works
    CUtensorMap map;
    if (!make_out_map(&map, d_out, n_groups)) return ECCO_ERR_CUDA;
    auto kernel = ecco_var_decompress_kernel<kVarWarps>;
    static thread_local bool configured[64] = {};
    rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    const uint64_t cta_tiles = (n_groups + kVarWarps * 32 - 1) / (kVarWarps * 32);
    const unsigned grid = static_cast<unsigned>(cta_tiles < static_cast<uint64_t>(di.sms) ? cta_tiles : di.sms);
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kVarWarps * 32), kSmemCtaBytes, static_cast<cudaStream_t>(stream),
                             static_cast<const uint8_t*>(d_meta), reinterpret_cast<const uint4*>(d_stream),
                             static_cast<const uint64_t*>(d_index), n_groups, static_cast<uint16_t*>(d_out), map);
}

extern "C" size_t ecco_gemv_workspace_bytes(int32_t n_out, int32_t k, int32_t batch)
{
    if (n_out <= 0 || k <= 0 || k % kGroup || batch < 1 || batch > ECCO_MAX_BATCH) return 0;
    // sized for the largest plan any supported device can ask for (at most 256 persistent CTAs)
    const int row_tiles = (n_out + 31) / 32;
    const GemvPlan p = gemv_plan_for(static_cast<int64_t>(row_tiles) * (k / kGroup), row_tiles, pad_v(batch), 256);
    return p.partial_bytes + p.ticket_bytes;
}

// the matrices of one call with their places in the call's unit and tile spaces
struct GemvCall {
    GemvBatch b;
    int row_tiles;
};
static void gemv_call_begin(GemvCall* c)
{
    std::memset(c, 0, sizeof *c);
}
static void gemv_call_add(GemvCall* c, const void* d_meta, const uint8_t* d_blocks, int n_out, int kblocks, const void* d_x, float* d_y)
{
    GemvJob& j = c->b.job[c->b.n++];
    j.meta = static_cast<const uint8_t*>(d_meta);
    j.blocks = d_blocks;
    j.x = static_cast<const __half*>(d_x);
    j.y = d_y;
    j.n_out = n_out;
    j.kblocks = kblocks;
    j.tile_first = c->row_tiles;
    j.unit_first = c->b.units;
    const int tiles = (n_out + 31) / 32;
    c->row_tiles += tiles;
    c->b.units += static_cast<int64_t>(tiles) * kblocks;
}

// three to eight rows of x: the tensor-core kernel
static int launch_gemv_mma_call(const DeviceInfo& di, const GemvCall& c, int batch, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    auto kernel = ecco_gemv_mma_kernel<kMmaWarps>;
    static thread_local bool configured[64] = {};
    int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    const GemvPlan p = gemv_plan_for(c.b.units, c.row_tiles, 8, di.sms < 256 ? di.sms : 256);
    if (!d_ws || !aligned16(d_ws)) return d_ws ? ECCO_ERR_ALIGNMENT : ECCO_ERR_WORKSPACE;
    if (ws_bytes < p.partial_bytes + p.ticket_bytes) return ECCO_ERR_WORKSPACE;
    float* partial = static_cast<float*>(d_ws);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(d_ws) + p.partial_bytes);
    rc = zero_tickets(tickets, p.ticket_bytes, stream);
    if (rc) return rc;
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kMmaWarps * 32), kSmemCtaBytes, stream, c.b, batch,
                             partial, tickets);
}
static int launch_gemv_mma(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, int n_out, int kblocks,
                           const void* d_x, int batch, float* d_y, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    GemvCall c;
    gemv_call_begin(&c);
    gemv_call_add(&c, d_meta, d_blocks, n_out, kblocks, d_x, d_y);
    return launch_gemv_mma_call(di, c, batch, d_ws, ws_bytes, stream);
}

// one or two rows of x (batch == kV): the per-warp kernel
template <int kV>
static int launch_gemv_warp_call(const DeviceInfo& di, const GemvCall& c, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    constexpr int kFusedWarps = gemv_warp_warps(kV);
    auto kernel = ecco_gemv_warp_kernel<kV, kFusedWarps>;
    static thread_local bool configured[64] = {};
    int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    const GemvPlan p = gemv_plan_for(c.b.units, c.row_tiles, kV, di.sms < 256 ? di.sms : 256);
    if (!d_ws || !aligned16(d_ws)) return d_ws ? ECCO_ERR_ALIGNMENT : ECCO_ERR_WORKSPACE;
    if (ws_bytes < p.partial_bytes + p.ticket_bytes) return ECCO_ERR_WORKSPACE;
    float* partial = static_cast<float*>(d_ws);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(d_ws) + p.partial_bytes);
    rc = zero_tickets(tickets, p.ticket_bytes, stream);
    if (rc) return rc;
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kFusedWarps * 32), kSmemCtaBytes, stream, c.b,
                             partial, tickets);
}
template <int kV>
static int launch_gemv_warp(const DeviceInfo& di, const void* d_meta, const uint8_t* d_blocks, int n_out, int kblocks,
                            const void* d_x, float* d_y, void* d_ws, size_t ws_bytes, cudaStream_t stream)
{
    GemvCall c;
    gemv_call_begin(&c);
    gemv_call_add(&c, d_meta, d_blocks, n_out, kblocks, d_x, d_y);
    return launch_gemv_warp_call<kV>(di, c, d_ws, ws_bytes, stream);
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

// several matrices in one call: one unit space, one launch
static int check_gemv_items(const ecco_gemv_item* items, int32_t n_items, int32_t batch)
{
    if (!items || n_items < 1 || n_items > ECCO_MAX_GEMV_ITEMS || batch < 1 || batch > ECCO_MAX_BATCH) return ECCO_ERR_INVALID_ARG;
    for (int i = 0; i < n_items; ++i) {
        const ecco_gemv_item& it = items[i];
        if (!it.d_meta || !it.d_blocks || !it.d_x_fp16 || !it.d_y) return ECCO_ERR_INVALID_ARG;
        if (it.n_out <= 0 || it.k <= 0 || it.k % kGroup) return ECCO_ERR_INVALID_ARG;
        if (!aligned16(it.d_meta) || !aligned16(it.d_blocks) || !aligned16(it.d_x_fp16) || !aligned16(it.d_y)) return ECCO_ERR_ALIGNMENT;
    }
    return ECCO_OK;
}
static void gemv_call_from_items(GemvCall* c, const ecco_gemv_item* items, int32_t n_items)
{
    gemv_call_begin(c);
    for (int i = 0; i < n_items; ++i)
        gemv_call_add(c, items[i].d_meta, items[i].d_blocks, items[i].n_out, items[i].k / kGroup, items[i].d_x_fp16, items[i].d_y);
}

extern "C" size_t ecco_gemv_batch_workspace_bytes(const ecco_gemv_item* items, int32_t n_items, int32_t batch)
{
    if (!items || n_items < 1 || n_items > ECCO_MAX_GEMV_ITEMS || batch < 1 || batch > ECCO_MAX_BATCH) return 0;
    int64_t units = 0, tiles = 0;
    for (int i = 0; i < n_items; ++i) {
        if (items[i].n_out <= 0 || items[i].k <= 0 || items[i].k % kGroup) return 0;
        const int64_t t = (items[i].n_out + 31) / 32;
        tiles += t;
        units += t * (items[i].k / kGroup);
    }
    if (tiles > INT32_MAX) return 0;
    const GemvPlan p = gemv_plan_for(units, static_cast<int>(tiles), pad_v(batch), 256);
    return p.partial_bytes + p.ticket_bytes;
}

extern "C" int ecco_gemv_batch(const ecco_gemv_item* items, int32_t n_items, int32_t batch, void* d_workspace,
                               size_t workspace_bytes, void* stream)
{
    int rc = check_gemv_items(items, n_items, batch);
    if (rc) return rc;
    DeviceInfo di;
    rc = device_info(&di);
    if (rc) return rc;
    GemvCall c;
    gemv_call_from_items(&c, items, n_items);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (pad_v(batch)) {
        case 1: return launch_gemv_warp_call<1>(di, c, d_workspace, workspace_bytes, s);
        case 2: return launch_gemv_warp_call<2>(di, c, d_workspace, workspace_bytes, s);
        default: return launch_gemv_mma_call(di, c, batch, d_workspace, workspace_bytes, s);
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
    const int row_tiles = (n_out + 31) / 32;
    const GemvPlan p = gemv_plan_for(static_cast<int64_t>(row_tiles) * kblocks, row_tiles, vpad, ctas);
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
    constexpr int kFusedWarps = fused_warps(kV);
    auto kernel = ecco_attn_scores_kernel<kV, kFusedWarps>;
    static thread_local bool configured[64] = {};
    int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    const int heads = batch * n_kv_heads;
    // persistent CTAs; the units (32 tokens of a head) are split evenly over the working warps on the device
    const int64_t units = static_cast<int64_t>(heads) * ((seq + 31) / 32);
    const int64_t ctas = (units + kFusedWarps - 1) / kFusedWarps;
    const unsigned grid = static_cast<unsigned>(ctas < di.sms ? ctas : di.sms);
    return launch_overlapped(kernel, grid, static_cast<unsigned>(kFusedWarps * 32), kSmemCtaBytes, stream, static_cast<const uint8_t*>(d_meta),
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
            static thread_local bool configured[64] = {};
            rc = want_all_smem(kernel, &configured[di.device]);
            if (rc) return rc;
            const uint64_t units = static_cast<uint64_t>(batch) * n_kv_heads * ((seq + 31) / 32);
            const uint64_t ctas = (units + kMmaWarps - 1) / kMmaWarps;
            const unsigned grid = static_cast<unsigned>(ctas < static_cast<uint64_t>(di.sms) ? ctas : di.sms);
            return launch_overlapped(kernel, grid, static_cast<unsigned>(kMmaWarps * 32), kSmemCtaBytes, s, static_cast<const uint8_t*>(d_meta),
                                     d_kblocks, batch * n_kv_heads, seq, q_per_kv, static_cast<const __half*>(d_q), scale, d_scores);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// ecco_attn_values
// ---------------------------------------------------------------------------------------------
namespace {
// A CTA of ecco_attn_values has 16 warps (512 tokens per unit).  18 find room (10.25 KB of shared memory per warp) but
// measured no faster on 32768-token rows (602.8 against 600.6 us) and slower on 4096-token rows, whose last unit
// they leave half empty (99.1 against 89.3 us).
constexpr int kAvWarps = 16;
inline int av_warps(int) { return kAvWarps; }
struct AvPlan { int grid, warps; size_t stats_bytes, partial_bytes, ticket_bytes; };
AvPlan av_plan(int batch, int n_kv_heads, int seq, int q_per_kv, int ctas_max)
{
    AvPlan p;
    p.warps = av_warps(seq);
    const int heads = batch * n_kv_heads;
    // at most this many units (fewer when all p.warps warps find room); the device splits what there is evenly
    const int64_t units = static_cast<int64_t>(heads) * ((seq + 31) / 32);
    p.grid = static_cast<int>(units < ctas_max ? units : ctas_max);
    auto up = [](size_t v) { return (v + 255) & ~static_cast<size_t>(255); };
    p.stats_bytes = up(static_cast<size_t>(heads) * q_per_kv * sizeof(float2));
    p.partial_bytes = up(static_cast<size_t>(p.grid + heads) * kGroup * 8 * sizeof(float));
    p.ticket_bytes = up(static_cast<size_t>(heads) * sizeof(unsigned int));
    return p;
}

template <int kWarps>
int launch_attn_values(const DeviceInfo& di, const AvPlan& p, const void* d_meta, const uint8_t* d_vblocks, int heads, int seq,
                       int q_per_kv, const float* d_scores, float2* stats, float* d_out, float* partial, unsigned int* tickets,
                       cudaStream_t s)
{
    auto kernel = ecco_attn_values_kernel<kWarps>;
    static thread_local bool configured[64] = {};
    const int rc = want_all_smem(kernel, &configured[di.device]);
    if (rc) return rc;
    return launch_overlapped(kernel, static_cast<unsigned>(p.grid), static_cast<unsigned>(kWarps * 32), kSmemCtaBytes, s,
                             static_cast<const uint8_t*>(d_meta), d_vblocks, heads, seq, q_per_kv, d_scores, stats, d_out, partial, tickets);
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
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* wsb = static_cast<uint8_t*>(d_workspace);
    float2* stats = reinterpret_cast<float2*>(wsb);
    float* partial = reinterpret_cast<float*>(wsb + p.stats_bytes);
    unsigned int* tickets = reinterpret_cast<unsigned int*>(wsb + p.stats_bytes + p.partial_bytes);
    const int heads = batch * n_kv_heads, rows = heads * q_per_kv;
    rc = launch_overlapped(ecco_softmax_stats_kernel, static_cast<unsigned>(rows), 256u, 0, s, d_scores, rows, seq, stats, tickets,
                           static_cast<int>(p.ticket_bytes / sizeof(unsigned int)));
    if (rc) return rc;
    return launch_attn_values<kAvWarps>(di, p, d_meta, d_vblocks, heads, seq, q_per_kv, d_scores, stats, d_out, partial, tickets, s);
}


extern "C" int ecco_act_decompress(const uint8_t* d_blocks, uint64_t n_groups, void* d_out_fp16, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_blocks || !d_out_fp16) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_blocks) || (reinterpret_cast<uintptr_t>(d_out_fp16) & 31u)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > kMaxGroups) return ECCO_ERR_INVALID_ARG;
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
    if (n_groups > kMaxGroups) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const uint64_t n_chunks = n_groups * 4;
    ecco_act_compress_kernel<<<act_grid(n_chunks, di), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(d_x_fp16), n_chunks, reinterpret_cast<uint4*>(d_blocks));
    return check_launch();
}


extern "C" int ecco_kv_compress(const void* d_meta, const void* d_x_fp16, uint64_t n_groups, uint8_t* d_blocks, void* stream)
{
    if (n_groups == 0) return ECCO_OK;
    if (!d_meta || !d_x_fp16 || !d_blocks) return ECCO_ERR_INVALID_ARG;
    if (!aligned16(d_meta) || !aligned16(d_x_fp16) || !aligned16(d_blocks)) return ECCO_ERR_ALIGNMENT;
    if (n_groups > kMaxGroups) return ECCO_ERR_INVALID_ARG;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc) return rc;
    const uint64_t ctas = (n_groups + kKvWarps - 1) / kKvWarps;
    const uint64_t cap = static_cast<uint64_t>(di.sms) * 8;
    return launch_overlapped(ecco_kv_compress_kernel, static_cast<unsigned>(ctas < cap ? ctas : cap), static_cast<unsigned>(kKvWarps * 32), 0,
                             static_cast<cudaStream_t>(stream), static_cast<const uint8_t*>(d_meta), static_cast<const __half*>(d_x_fp16),
                             n_groups, d_blocks);
}

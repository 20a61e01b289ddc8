// ecco_launch.cuh -- host-side launch helpers: device query, overlapped launches, work plans
// Part of the one translation unit ecco_kernels.cu; included from there only.
#pragma once

namespace {

// ---------------------------------------------------------------------------------------------
// host-side launch helpers
// ---------------------------------------------------------------------------------------------
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

// Warps per CTA the decoding kernels are launched with (their register budget); how many of them work is decided on
// the device, from the size of the image's tables.
constexpr int kDecompressWarps = 28;
constexpr int fused_warps(int) { return 28; }
constexpr int gemv_warp_warps(int) { return 28; }

struct GemvPlan { int row_tiles, grid; size_t partial_bytes, ticket_bytes; };

// plan of a fused GEMV call over `units` units in `row_tiles` 32-row tiles (all matrices of the call together):
// persistent CTAs of `warps` warps, one slot of cols x 32 partial sums per (warp, tile) step of the staircase, one
// ticket per tile
inline GemvPlan gemv_plan(int64_t units, int row_tiles, int warps, int cols, int ctas_max)
{
    GemvPlan p;
    p.row_tiles = row_tiles;
    const int64_t ctas = (units + warps - 1) / warps;
    p.grid = static_cast<int>(ctas < ctas_max ? ctas : ctas_max);
    p.partial_bytes = (static_cast<size_t>(p.grid * warps + row_tiles) * cols * 32 * sizeof(float) + 255) & ~static_cast<size_t>(255);
    p.ticket_bytes = (static_cast<size_t>(row_tiles) * sizeof(unsigned int) + 255) & ~static_cast<size_t>(255);
    return p;
}

constexpr int kMmaWarps = 20;      // 18 find room beside the tables of a typical image (11.25 KB of shared memory per warp)

// the per-warp kernel (one or two rows of x: vpad columns) or the tensor-core kernel (3..8 rows: eight columns)
inline GemvPlan gemv_plan_for(int64_t units, int row_tiles, int vpad, int ctas_max)
{
    return vpad <= 2 ? gemv_plan(units, row_tiles, gemv_warp_warps(vpad), vpad, ctas_max) : gemv_plan(units, row_tiles, kMmaWarps, 8, ctas_max);
}

inline int pad_v(int v) { return v <= 1 ? 1 : v <= 2 ? 2 : v <= 4 ? 4 : 8; }


}  // namespace

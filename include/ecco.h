/*
 * ecco.h -- C ABI of the B200-native Ecco 4x block codec (decompression hot path).
 *
 * Format (Ecco, Sec. 3.1-3.2): a tensor is cut into groups of 128 fp16 values; every group is
 * stored in one 64-byte block holding an FP8 group scale (the group's signed abs-max under a
 * per-tensor power-of-two factor T = 2^e), a 2-bit choice ID_HF among H = 4 Huffman codebooks,
 * the Huffman-coded index ID_KP of one of S <= 64 shared 15-centroid k-means patterns, and 128
 * Huffman-coded 4-bit indices (code lengths 2..8; index 15 = the abs-max itself).  A stream
 * longer than the block is clipped; a shorter one is padded with 15-bit outliers (7-bit
 * location + FP8 value) for the next-largest values (Sec. 3.2, Fig. 4 step 9).
 *
 * Bit order inside a block (the paper's block drawing is not part of its text; this is the
 * library's definition): stream bit k is bit (k & 7) of byte (k >> 3).  Fixed-width fields are
 * least-significant bit first; codewords are first-code-bit first (canonical codes: symbols
 * ordered by (length, id), consecutive values).  Stream order: [0,8) scale byte (OCP E4M3),
 * [8,10) ID_HF, [10, ..) ID_KP codeword, then the codewords of positions 0..127, zero fill,
 * and pads in 15-bit slots growing down from bit 511: pad j occupies [512-15(j+1), 512-15j),
 * low 7 bits location, high 8 bits E4M3 value; at most 16 pads.
 *
 * Conventions: every function returns ECCO_OK (0) or a negative error code and never throws.
 * "host" pointers are ordinary CPU memory; "device" pointers (d_*) are CUDA device memory
 * owned by the caller, who also owns the stream.  Device calls are asynchronous on `stream`
 * (a cudaStream_t passed as void*, NULL = the legacy default stream), never synchronise and
 * never allocate.  fp16 values travel as raw uint16_t / void*.  d_blocks, d_out, d_x, d_q and
 * d_meta must be 16-byte aligned.  The library refuses to run on a device that is not
 * compute capability 10.x (ECCO_ERR_UNSUPPORTED_ARCH); there is no CPU fallback.
 *
 * Graph capture: a chain of device calls may be captured into a CUDA graph and replayed, once every entry point in
 * it has been called eagerly on that device (the first call sets its kernels' attributes).
 *
 * Stream order: the usual one.  Internally the kernels are launched so that one may become
 * resident while the previous kernel of the stream is still draining, but each waits for that
 * kernel to complete before its first access to memory, so only launch latency overlaps.  The
 * one thing a kernel reads before that wait is the metadata image: d_meta must be filled by a
 * copy (cudaMemcpy / cudaMemcpyAsync, which the stream orders as usual), not written by a kernel
 * that is still running when the call is issued.
 */
#ifndef ECCO_H_
#define ECCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ECCO_GROUP 128          /* values per group  (Sec. 3.1) */
#define ECCO_BLOCK_BYTES 64     /* bytes per block   (Sec. 3.1) */
#define ECCO_MAX_PATTERNS 64    /* S                 (Sec. 3.2) */
#define ECCO_CODEBOOKS 4        /* H                 (Sec. 3.2) */
#define ECCO_CENTROIDS 15       /* per pattern       (Sec. 3.2) */
#define ECCO_MAX_BATCH 8        /* ecco_gemv rows of x */

enum {
    ECCO_OK = 0,
    ECCO_ERR_INVALID_ARG = -1,
    ECCO_ERR_ALIGNMENT = -2,
    ECCO_ERR_NONFINITE_INPUT = -3,
    ECCO_ERR_BAD_META = -4,
    ECCO_ERR_UNSUPPORTED_ARCH = -5,
    ECCO_ERR_CUDA = -6,             /* see ecco_last_cuda_error() */
    ECCO_ERR_WORKSPACE = -7,        /* workspace too small */
    ECCO_ERR_DEVICE_TIMEOUT = -8    /* a bounded device-side wait gave up (ecco_device_status) */
};

/* flags of ecco_encode_host / ecco_params.select */
#define ECCO_SELECT_MSE 0u        /* Fig. 4 step 5: pattern with the least squared error (weights) */
#define ECCO_SELECT_MINMAX 1u     /* Sec. 4.3: min/max fitness (online KV path) */
#define ECCO_KEEP_EXPONENT 2u     /* keep the metadata's exponent e instead of refitting it */

typedef struct ecco_meta ecco_meta;   /* opaque per-tensor metadata (Sec. 4.2: "tensor-wise metadata") */

typedef struct {
    int32_t S;                  /* shared patterns, 2..64 */
    int32_t H;                  /* must be 4 */
    uint64_t seed;              /* seeds the k-means initialisations */
    uint32_t select;            /* ECCO_SELECT_MSE or ECCO_SELECT_MINMAX for step 5 of calibration */
    int32_t kmeans_iters;       /* iteration cap of every Lloyd loop (0 = 25) */
    uint64_t max_groups;        /* calibrate on at most this many groups, evenly strided (0 = all) */
    int32_t threads;            /* worker threads (0 = all available cores) */
} ecco_params;

typedef struct {
    uint64_t n_groups;
    uint64_t clipped_groups;    /* groups that lost at least one value to clipping */
    uint64_t clipped_values;
    uint64_t padded_groups;
    uint64_t padded_values;
    uint64_t total_bits;        /* header + stored codewords, summed over groups */
    uint64_t kp_usage[ECCO_MAX_PATTERNS];
    uint64_t hf_usage[ECCO_CODEBOOKS];
    uint64_t sym_count[16];
} ecco_stats;

/* ---------------------------------------------------------------- host, blocking */

/* Fig. 4 steps 1-7 on a calibration tensor of n_groups*128 fp16 values (host): per-group
 * 15-means patterns, S shared patterns, H codebooks per pattern (lengths 2..8, Sec. 4.2) and the
 * ID_KP code.  elem_weights_or_null: 128 non-negative weights applied to every group in step 3
 * ("activation-aware"), or NULL.  *out_meta is owned by the caller (ecco_meta_free). */
int ecco_calibrate_host(const uint16_t* calib_fp16, uint64_t n_groups, const float* elem_weights_or_null,
                        const ecco_params* params, ecco_meta** out_meta);

/* Metadata from explicit tables (host arrays): patterns [S][15] fp16 ascending, cb_len [S][4][16]
 * in 2..8 with Kraft sum 1, kp_len [S] in 1..12 with Kraft sum 1, exponent e in [-32, 16].
 * Returns ECCO_ERR_BAD_META if any table is inconsistent. */
int ecco_meta_create(int32_t S, int32_t e, const uint16_t* patterns, const uint8_t* cb_len, const uint8_t* kp_len,
                     ecco_meta** out_meta);
/* Copies the tables out (any output pointer may be NULL). */
int ecco_meta_get(const ecco_meta* meta, int32_t* S, int32_t* e, uint16_t* patterns, uint8_t* cb_len, uint8_t* kp_len);
void ecco_meta_free(ecco_meta* meta);

/* Fig. 4 steps 2, 5, 8, 9 (and Sec. 4.3 for ECCO_SELECT_MINMAX): encodes n_groups*128 fp16 host
 * values into n_groups*64 bytes at dst_blocks (host, caller-owned).  Unless ECCO_KEEP_EXPONENT is
 * set, first refits meta's exponent e to this tensor (smallest e with max|x| <= 448*2^e).
 * Non-finite input gives ECCO_ERR_NONFINITE_INPUT.  Runs on all available cores. */
int ecco_encode_host(ecco_meta* meta, const uint16_t* src_fp16, uint64_t n_groups, uint32_t flags,
                     uint8_t* dst_blocks, ecco_stats* stats_or_null);

/* Device image of the metadata (Sec. 4.2: loaded once before the compressed loads): header,
 * patterns, and the prebuilt decode tables.  The caller copies `bytes` bytes from host_staging to
 * 16-byte aligned device memory and passes that pointer as d_meta. */
size_t ecco_meta_device_bytes(const ecco_meta* meta);
int ecco_meta_serialize_device(const ecco_meta* meta, void* host_staging, size_t bytes);

/* ---------------------------------------------------------------- device, asynchronous */

/* Sec. 4.2 (pattern retriever, Huffman decode, outlier handling, mapper): n_groups blocks at
 * d_blocks -> n_groups*128 fp16 at d_out_fp16.  Value = fp16_rn(fp32(centroid) * fp32(scale));
 * clipped positions read +0.  n_groups == 0 is a no-op. */
int ecco_decompress(const void* d_meta, const uint8_t* d_blocks, uint64_t n_groups, void* d_out_fp16, void* stream);

/* The same for several tensors in one call (the seven matrices of a decoder layer, the K and V caches of a
 * layer).  The items must be independent of each other: no item's output may overlap another item's output or
 * blocks.  Then the effect is that of ecco_decompress on every item, but tensors of 32 groups or more share one
 * kernel launch per 8 items, in which every SM moves on to the next tensor as soon as it is done with its share
 * of the current one, so launch latency and tail are paid once.  With respect to other work in the stream the
 * call is ordered like a single kernel.  `items` is a HOST array read before the call returns; every item has
 * its own metadata image; items with n_groups == 0 are skipped.  Errors are those of ecco_decompress and are
 * found before anything is launched. */
typedef struct ecco_decompress_item {
    const void* d_meta;        /* device: metadata image of this tensor */
    const uint8_t* d_blocks;   /* device: 64 * n_groups bytes */
    uint64_t n_groups;
    void* d_out_fp16;          /* device: 128 * n_groups fp16 values */
} ecco_decompress_item;
int ecco_decompress_batch(const ecco_decompress_item* items, int32_t n_items, void* stream);

/* Decode-phase GEMV on compressed weights (Sec. 2.1: M = 1 matrix-vector products; Sec. 4.2
 * decode): y[b][n] = sum_k W~[n][k] * x[b][k], fp32 accumulation.  W is row-major [n_out][k],
 * groups along k, block of (n, kblock) at byte 64*(n*(k/128) + kblock).  x is fp16 [batch][k],
 * y is fp32 [batch][n_out], batch in 1..8, k a multiple of 128.  d_workspace: device scratch of
 * at least ecco_gemv_workspace_bytes(n_out, k, batch) bytes, 16-byte aligned, contents
 * irrelevant before and undefined after; calls sharing a workspace must not overlap. */
size_t ecco_gemv_workspace_bytes(int32_t n_out, int32_t k, int32_t batch);
int ecco_gemv(const void* d_meta, const uint8_t* d_blocks, int32_t n_out, int32_t k, const void* d_x_fp16,
              int32_t batch, float* d_y, void* d_workspace, size_t workspace_bytes, void* stream);

/* The same for several matrices in one call: y_i = W~_i x_i for up to ECCO_MAX_GEMV_ITEMS matrices that are
 * independent of each other (the q, k and v projections of a decoder layer, which read the same x; gate and up).  The
 * work of all matrices is dealt out to the SMs as one, so launch, table fetch and tail are paid once and small
 * matrices fill the machine together.  All items must have been encoded with the same patterns and codebooks (equal
 * decode tables; the per-tensor exponent may differ) and use the same batch; x and y are per item and may be shared
 * between items only for x.  The result is reproducible (the same call gives the same bits) and equals that of
 * ecco_gemv on each item up to fp32 rounding: a row's sum over k is cut into partial sums at other places.  `items` is a
 * HOST array read before the call returns.  Errors of the arguments are found before anything is launched; items
 * whose tables differ from those of the first are detected on the device: nothing is computed and
 * ecco_device_status() then reports ECCO_ERR_INVALID_ARG.  Workspace as for ecco_gemv, sized by
 * ecco_gemv_batch_workspace_bytes for the same items. */
#define ECCO_MAX_GEMV_ITEMS 8
typedef struct ecco_gemv_item {
    const void* d_meta;        /* device: metadata image of this matrix */
    const uint8_t* d_blocks;   /* device: 64 * n_out * (k / 128) bytes */
    int32_t n_out, k;
    const void* d_x_fp16;      /* device: fp16 [batch][k] */
    float* d_y;                /* device: fp32 [batch][n_out] */
} ecco_gemv_item;
size_t ecco_gemv_batch_workspace_bytes(const ecco_gemv_item* items, int32_t n_items, int32_t batch);
int ecco_gemv_batch(const ecco_gemv_item* items, int32_t n_items, int32_t batch, void* d_workspace,
                    size_t workspace_bytes, void* stream);

/* Allocation-free variant of ecco_gemv.  The paper has no counterpart: this entry point exists for
 * callers that are not allowed to obtain device memory at the time they need the product -- a
 * layer plugged into an inference engine whose memory plan was fixed when the engine was built, a
 * serving loop that must not call cudaMalloc because it synchronises the whole device and stalls
 * every other stream, or a process whose memory budget was handed out in full at start-up.  Same
 * arguments and result as ecco_gemv, but the scratch for the split-k partial sums is a fixed array
 * of ECCO_STATIC_WORKSPACE_BYTES inside the library's device image (every GPU that loads the
 * library carries it until the process exits) instead of a caller buffer.  The call allocates
 * nothing.  A shape whose plan needs more scratch than that is refused with ECCO_ERR_WORKSPACE
 * before anything is launched.  For scale, on a 148-SM part: batch 8 on an 11008 x 4096 matrix needs 3.38 MB, batch 1
 * or 2 on the same matrix 0.6 / 1.1 MB, batch 8 on 28672 x 8192 3.96 MB; a matrix with more than about 36 000 output
 * rows at batch 3..8 does not fit and is refused.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the one array:
 * it still holds the previous call's values when the next call starts (each call clears the part
 * that must start from zero), and two calls whose kernels overlap on the GPU -- different streams,
 * no dependency between them -- race on it and give undefined results.  Serialise them, or use
 * ecco_gemv with separate workspaces. */
#define ECCO_STATIC_WORKSPACE_BYTES (4u << 20)
int ecco_gemv_static_ws(const void* d_meta, const uint8_t* d_blocks, int32_t n_out, int32_t k, const void* d_x_fp16,
                        int32_t batch, float* d_y, void* stream);

/* Fused attention scores over a compressed K cache (Eq. 3: Q K^T / sqrt(d_k), without the
 * softmax): scores[b][hq][t] = scale * sum_d q[b][hq][d] * K~[b][hq / q_per_kv][t][d].  One group
 * is the 128-wide head vector of one token; blocks are ordered [batch][n_kv_heads][seq]; q is
 * fp16 [batch][n_kv_heads*q_per_kv][128]; scores fp32 [batch][n_kv_heads*q_per_kv][seq];
 * q_per_kv in 1..8. */
int ecco_attn_scores(const void* d_meta, const uint8_t* d_kblocks, int32_t batch, int32_t n_kv_heads, int32_t seq,
                     int32_t q_per_kv, const void* d_q_fp16, float scale, float* d_scores, void* stream);

/* Attention output over a compressed V cache (Eq. 3: softmax(Q K^T / sqrt(d_k)) V):
 * out[b][hq][d] = sum_t p[b][hq][t] * V~[b][hq / q_per_kv][t][d] with p = softmax over t of
 * scores[b][hq][:] (fp32 logits, e.g. the output of ecco_attn_scores).  Blocks are ordered
 * [batch][n_kv_heads][seq], one group = one token's 128-wide head vector; out is fp32
 * [batch][n_kv_heads*q_per_kv][128]; q_per_kv in 1..8; seq >= 1.  The sum over tokens runs on the
 * tensor cores with fp32 accumulation, in an order fixed by the shapes (results are reproducible).
 * Probabilities are carried with 22 bits down to 2e-12; smaller ones count as zero.
 * d_workspace: at least ecco_attn_values_workspace_bytes(...)
 * bytes, 16-byte aligned, contents irrelevant before and undefined after; calls sharing a workspace
 * must not overlap. */
size_t ecco_attn_values_workspace_bytes(int32_t batch, int32_t n_kv_heads, int32_t seq, int32_t q_per_kv);
int ecco_attn_values(const void* d_meta, const uint8_t* d_vblocks, int32_t batch, int32_t n_kv_heads, int32_t seq,
                     int32_t q_per_kv, const float* d_scores, float* d_out, void* d_workspace, size_t workspace_bytes,
                     void* stream);

/* Online 4x compressor for the KV cache (Sec. 4.3: sorter, min/max pattern selector, four encoders,
 * pack and clip): n_groups*128 fp16 device values -> n_groups*64 bytes at d_blocks, with the
 * patterns, codebooks and exponent of d_meta (the device image, which also carries the encoder
 * tables).  The blocks are byte-identical to ecco_encode_host(meta, x, n_groups,
 * ECCO_SELECT_MINMAX | ECCO_KEEP_EXPONENT, ...).  Inputs must be finite (non-finite values give
 * unspecified blocks, never a fault); values above 448 * 2^e saturate. */
int ecco_kv_compress(const void* d_meta, const void* d_x_fp16, uint64_t n_groups, uint8_t* d_blocks, void* stream);

/* ---------------------------------------------------------------- variable-length container */

/* The same per-group fields as the 64-byte block (scale byte, ID_HF, ID_KP codeword, 128 codewords;
 * Sec. 3.2) written back to back into one bit stream: nothing is clipped, nothing is padded, and
 * a side index says where every group starts.  (The paper has only the fixed block; this layout
 * trades the fixed 4x ratio for the absence of clipping loss.)  Stream bit k = bit k&7 of byte k>>3.
 * Index (host and device, 8-byte aligned): u64 total_bits | u64 chunk_base[ceil(n/4096)] | u32
 * offset[n]; group g starts at bit chunk_base[g >> 12] + offset[g] and sees the stream up to the
 * start of group g+1 (zeros after that).  ecco_var_encode_host quantises exactly like
 * ecco_encode_host (same flags) and needs stream_capacity >= 16 * ceil(total_bits / 128), at most
 * ecco_var_stream_bytes_bound(n_groups).  ecco_var_decompress: d_stream 16-byte aligned and a
 * multiple of 16 bytes long, d_index 8-byte aligned, output as ecco_decompress. */
size_t ecco_var_stream_bytes_bound(uint64_t n_groups);
size_t ecco_var_index_bytes(uint64_t n_groups);
int ecco_var_encode_host(ecco_meta* meta, const uint16_t* src_fp16, uint64_t n_groups, uint32_t flags, uint8_t* dst_stream,
                         size_t stream_capacity, void* dst_index, size_t index_capacity, uint64_t* total_bits_out);
int ecco_var_decompress(const void* d_meta, const uint8_t* d_stream, const void* d_index, uint64_t n_groups, void* d_out_fp16,
                        void* stream);

/* ---------------------------------------------------------------- 2x activation format (device) */

/* Sec. 3.2 "Activation Compression", Sec. 4.2 / 4.3 low-ratio (de)compressor: 64 fp16 values <-> one
 * 64-byte block.  Byte i holds the 7-bit two's-complement quantised value q_i (-64..63) in bits 0..6
 * and one metadata bit in bit 7; metadata bits 0..15 are the fp16 scale, 16..31 the fp16 zero point
 * (both least-significant bit first), 32..63 zero.  (The field widths are the paper's; the order
 * is this library's definition.)  Compression: scale = fp16((max - min) / 127), zero point =
 * fp16(min + 64 * scale), q = clamp(round_to_nearest_even((x - zero) * (1 / scale)), -64, 63) in fp32;
 * a zero scale stores q = 0.  Decompression: fp16_rn(fma(q, scale, zero)) in fp32.  Inputs must be
 * finite (non-finite values give unspecified bytes, never a fault).  Blocks 16-byte aligned, fp16
 * buffers 32-byte aligned.  Both calls are asynchronous on `stream`. */
#define ECCO_ACT_GROUP 64
int ecco_act_compress(const void* d_x_fp16, uint64_t n_groups, uint8_t* d_blocks, void* stream);
int ecco_act_decompress(const uint8_t* d_blocks, uint64_t n_groups, void* d_out_fp16, void* stream);

/* ---------------------------------------------------------------- diagnostics */
const char* ecco_error_string(int code);
int ecco_last_cuda_error(void);        /* cudaError_t of the last ECCO_ERR_CUDA on this thread */
/* Synchronises the device and reads the library's device-side status word: 0, or
 * ECCO_ERR_DEVICE_TIMEOUT if a kernel's bounded wait on a bulk copy expired (its output is then
 * undefined).  Clears the word. */
int ecco_device_status(void);
/* Number of kernels the library has launched in this process (diagnostic counter). */
uint64_t ecco_kernel_launch_count(void);
/* Test aid for the give-up path of the bounded device-side wait (Sec. 4.2's "loaded once" staging waits on a
 * barrier that a bulk copy completes): launches one small CTA on `stream` that arms such a barrier for bytes
 * no copy will deliver -- nothing is in flight and nothing can hang --, polls it a few hundred times, gives up and
 * returns normally.  Afterwards ecco_device_status() reports ECCO_ERR_DEVICE_TIMEOUT once. */
int ecco_test_wait_timeout(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ECCO_H_ */

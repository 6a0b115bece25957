/*
 * unionsparse.h -- C ABI of the B200 (sm_100a) W4A4 bitmap-sparse SpMM library.
 *
 *   Y = W * X,  W: M x K pruned INT4 weights held in a bitmap format (IE-BME, paper Sec. V-A),
 *               X: K x N dense INT4 activations, INT32 accumulation,
 *               optional fused dequantisation Y16 = fp16(acc * s_w[m] * s_x[n]).
 *
 * Every call returns a us_status; nothing aborts, traps or blocks on the GPU. Pointers are
 * plain host or device pointers as stated per argument; no framework types cross this ABI.
 * Unless stated otherwise a call may be made from any host thread, but calls on one handle
 * must not overlap.
 */
#ifndef UNIONSPARSE_H_
#define UNIONSPARSE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum us_status {
    US_OK = 0,
    US_ERR_INVALID_ARG = 1,   /* NULL pointer, non-positive size, N outside 1..max_N, ...   */
    US_ERR_VALUE_RANGE = 2,   /* a weight outside [-8, 7]                                   */
    US_ERR_SHAPE = 3,         /* format parameters that do not divide / do not fill words   */
    US_ERR_UNSUPPORTED = 4,   /* a valid IE-BME format no kernel of this library implements */
    US_ERR_ALLOC = 5,         /* host or device allocation failed                           */
    US_ERR_CUDA = 6,          /* a CUDA runtime call failed (see us_last_error)             */
    US_ERR_DEVICE_TIMEOUT = 7,/* a bounded wait inside a kernel gave up (no hang, no trap)  */
    US_ERR_SCRATCH_TOO_SMALL = 8 /* us_spmm_static_scratch: the problem needs more scratch than
                                    the library's fixed device array holds                   */
} us_status;

/*
 * IE-BME format parameters (paper Sec. V-A "Area Partitioning"): a local tile of H_L x K_L
 * weights is split into an R_A x C_A grid of areas; one union-mask bit covers the Q = R_A*C_A
 * values at the same position of every area. Every format whose union mask fills whole 64-bit
 * words (the paper's {16, 64, 2, 2} among them, and per-element bitmaps {16, 64, 1, 1}) can be
 * encoded, decoded and measured (us_get_stats) on a US_ENCODE_HOST_ONLY handle, in the paper's
 * own array layout. The kernels implement H_L = 16, R_A = 2 with
 *   C_A = 1 (Q = 2): one bit covers rows i and i+8 of a 16-row strip; K_L a multiple of 128;
 *   C_A = 2 (Q = 4, the paper's 2 x 2 union): the bit also covers the column K_L/2 further on in the
 *            tile; K_L a multiple of 256; no chained calls (us_spmm_requant with y_amax), no row pairing;
 * K_L up to 8192. Only such handles can be uploaded and multiplied. On a mask without structure
 * Q = 4 stores 1 - s^4 of the dense payload against 1 - s^2 for Q = 2 and is decoded with fewer
 * instructions per weight.
 */
typedef struct us_format {
    int32_t H_L, K_L, R_A, C_A;
} us_format;

/* Statistics of an encoded matrix (paper Sec. V-A storage arrays and Eq. 1). */
typedef struct us_stats {
    int64_t M, K;                 /* logical shape                                          */
    int64_t Mp, Kp;               /* shape after zero padding to whole tiles                */
    int64_t nnz;                  /* true nonzeros                                          */
    int64_t n_tiles;              /* local tiles (one offset each)                          */
    int64_t sum_P;                /* sum over tiles of P_t = active union-mask bits         */
    int64_t bytes_payload;        /* ceil(Q * sum_P * weight_bits / 8): the packed values   */
    int64_t bytes_payload_padded; /* payload bytes as stored (kernel layout: lane streams padded
                                     per tile; the paper's layout stores no padding)        */
    int64_t bytes_bitmap;         /* union bitmaps                                          */
    int64_t bytes_offsets;        /* 4 * (n_tiles + 1)                                      */
    int64_t bytes_total;          /* bytes_payload_padded + bytes_bitmap + bytes_offsets    */
    double  pmr;                  /* Eq. 1: B_w * nnz / (bytes_bitmap + bytes_offsets), B_w = weight_bits / 8 */
    double  fill;                 /* stored values / (M*K) = Q * sum_P / (M*K)              */
    us_format fmt;                /* the format in use                                      */
    int32_t weight_bits;          /* 4, or 2 for a US_ENCODE_W2 handle                      */
    int32_t reserved;
} us_stats;

typedef struct us_handle us_handle;

/* Flags of us_encode. */
#define US_ENCODE_HOST_ONLY 1u /* build the format on the host only: no CUDA call is made;
                                  the handle serves us_get_stats / us_decode, not us_spmm    */
#define US_ENCODE_SORT_ROWS 2u /* order rows by nonzero count before cutting 16-row strips,
                                  so that rows of similar density share a strip; the output
                                  row order of us_spmm is unchanged (folded into the store)  */

#define US_ENCODE_W2 8u        /* W2A4 (paper Sec. VII-B, the W2A4 kernel figure): the weights are INT2, values in
                                  [-2, 1] (others: US_ERR_VALUE_RANGE). Needs the format (16, K_L, 2, 2): the
                                  four 2-bit values under one union-mask bit fill exactly one payload byte
                                  (bits 1:0 = W[i][k] + 2, 3:2 = W[i+8][k] + 2, 5:4 and 7:6 the same at column
                                  k + K_L/2), so the decode stays byte-granular. Other formats:
                                  US_ERR_UNSUPPORTED. No chained calls, no row pairing.                  */
#define US_ENCODE_PAIR_ROWS 4u /* bitmap-aware row reordering (paper Sec. V-B, Alg. 1) in its
                                  per-strip form: inside every 16-row strip (after SORT_ROWS, if
                                  also given) choose which two rows share each union-mask row so
                                  that the strip's union mask has the fewest active bits over all
                                  of K; exact (subset DP, Eq. 5). One grouping per strip rather
                                  than per tile, so the output row order of us_spmm is unchanged
                                  (folded into the store) at no run-time cost                */

/*
 * Offline encoder (paper Sec. V-A, Fig. 7: dense pruned INT4 -> union bitmaps, per-tile
 * offsets, packed INT4 values), followed by the upload to the current CUDA device.
 *   W        host, M x K row-major int8, values in [-8, 7], 0 = pruned. Not retained.
 *   w_scale  host, M fp16 bit patterns (per-output-channel scales), or NULL when only INT32
 *            output will be requested. Not retained.
 *   fmt      NULL selects {16, K_L, 2, 1} with K_L = 1024, 512 or 256 by the shape (long tiles
 *            for large matrices, short ones where every SM must still find work).
 *   max_N    largest N later passed to us_spmm (1..64); sizes the split-K workspace.
 *   out      receives the handle; it owns every host and device array it allocates.
 * M, K need not be multiples of the tile: the matrix is zero padded internally.
 * Errors: INVALID_ARG, VALUE_RANGE, SHAPE, UNSUPPORTED, ALLOC, CUDA. On error *out is NULL.
 */
us_status us_encode(const int8_t* W, int64_t M, int64_t K, const uint16_t* w_scale,
                    const us_format* fmt, int32_t max_N, uint32_t flags, us_handle** out);

/* Pure host read of the statistics, PMR (paper Eq. 1) included. */
us_status us_get_stats(const us_handle* h, us_stats* out);

/*
 * Test hook: exact inverse of the encoder, from the handle's host copy of the encoded arrays
 * (paper Sec. V-A read backwards). W_out: host, M x K int8.
 */
us_status us_decode(const us_handle* h, int8_t* W_out);

/*
 * Test hook: the row order in use. perm_out: host, Mp int32 entries; entry p is the original
 * row stored at padded position p (strip p/16, row p%16), or -1 for a padding row.
 */
us_status us_get_row_order(const us_handle* h, int32_t* perm_out);

/*
 * The SpMM (paper Alg. 2: W in IE-BME format, dense X -> Y), enqueue-only.
 *   X        device, N x K token-major packed INT4: byte n*ceil(K/2) + k/2 holds k even in its
 *            low nibble and k odd in its high nibble, two's complement. 16-byte aligned.
 *   N        1..max_N.
 *   x_scale  device, N fp16 per-token scales, or NULL.
 *   Y        device, token-major N x M: int32 when x_scale is NULL, else fp16
 *            fp16(acc * w_scale[m] * x_scale[n]) (needs a handle encoded with w_scale).
 *   stream   a cudaStream_t (NULL = the default stream).
 * Caller owns X, x_scale and Y. Returns before the kernel completes; device-side failures are
 * reported by us_last_error. One call per handle may be in flight: the split-K workspace and
 * arrival counters belong to the handle and are left zeroed by each call.
 * The handle's device must be the current device. After a call that us_last_error reports as
 * failed, the workspace has been cleared again and the handle can be used as before.
 * Errors: INVALID_ARG (also: another device is current), UNSUPPORTED (host-only handle, or a
 * format no kernel reads), CUDA.
 */
us_status us_spmm(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y,
                  void* stream);

/*
 * The same SpMM as us_spmm for callers that must not allocate device memory around the call.
 * (The paper has no counterpart: this entry point exists for the integration, not the method.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits or too costly -- a
 * serving loop that has handed all device memory to its own pool, a latency-critical path that
 * cannot afford the device-wide synchronisation an allocation may cause, or a section of a
 * program in which allocation calls are not permitted. us_spmm keeps its split-K workspace and
 * arrival counters in memory that the handle allocated; this call instead uses a fixed array that
 * is part of the library image itself, US_STATIC_SCRATCH_BYTES (4 MiB) per GPU, held by every GPU
 * that loads the library until the process exits. It calls no allocation routine of any kind.
 *
 * Arguments, layouts, output and error behaviour are those of us_spmm, plus:
 *   - the problem must fit the array: n_strips * (n_tiles_N * 512 + 4) bytes, n_strips =
 *     ceil(M/16), n_tiles_N = 1, 2, 4, 8 for N <= 8, 16, 32, 64; otherwise
 *     US_ERR_SCRATCH_TOO_SMALL is returned and nothing is enqueued;
 *   - the handle's device must be the current device (US_ERR_INVALID_ARG otherwise);
 *   - the array is shared by every call on that GPU and keeps whatever the last call left in it:
 *     each call first enqueues a clear of the part it uses on `stream`, then the kernel. Two
 *     calls that can overlap on the GPU (different streams, no dependency) race on the array and
 *     give wrong results: serialise them;
 *   - the first call on a device looks up the array's device address (once per device, with that
 *     device current). Make that first call before any stream capture begins.
 */
#define US_STATIC_SCRATCH_BYTES (4u << 20)
us_status us_spmm_static_scratch(us_handle* h, const void* X, int32_t N, const void* x_scale, void* Y,
                                 void* stream);

/*
 * Synchronises the device, then reports the first failure recorded for this handle: a CUDA
 * error of an earlier launch (US_ERR_CUDA) or a bounded in-kernel wait that ran out
 * (US_ERR_DEVICE_TIMEOUT). Clears the record and, after a failure, the handle's split-K workspace
 * and arrival counters (a call that gave up leaves partial sums behind).
 */
us_status us_last_error(us_handle* h);

/*
 * Chained calls: fp16 activations in, INT4 inside, fp16 out.
 *
 * The paper evaluates the W4A4 kernel on INT4 activations that are given (Sec. VII-A) and defines
 * no activation quantiser; these three calls have no counterpart in it. They let the fp16 output of
 * one projection feed the next: the producing kernel's epilogue leaves the per-token absmax, and one
 * small kernel between the two turns the activations into INT4 codes. The quantiser is the
 * plain per-token symmetric one with a reciprocal step:
 *     amax[n]  = max |x[n][k]| over the quantised columns
 *     scale[n] = RN_fp16(amax[n] / 7)                     (what the dequantisation multiplies by)
 *     inv[n]   = min(RN_fp16(7 / amax[n]), 65504)         (65504 for amax = 0)
 *     code     = clamp(RNE(x * inv[n]), -8, 7)            (the fp16 x fp16 product taken exactly)
 * so the codes are reproducible bit for bit. Tokens with amax below 7 / 65504 lose resolution.
 *
 * Absmax buffer: US_AMAX_BYTES bytes of device memory, 4-byte aligned, written by us_absmax_f16 or
 * by a us_spmm_requant (y_amax) and read by the next us_spmm_requant (x_amax). Layout: word 0 = P,
 * the number of parts; word 64 + 64 * p + n = the fp16 bit pattern of a partial absmax of token n
 * (p < P, n < 64); amax[n] is the largest of the P words. Writers store every part, so a buffer
 * never needs clearing. It holds one tensor's absmax at a time.
 *
 * us_spmm_requant: Y16[n][m] = RN_fp16(sum_k W[m][k] * code(X16[n][k]) * w_scale[m] * scale[n]).
 *   X16     device, N rows of fp16, row n at X16 + n * ldx (elements), ldx >= K; finite values.
 *           16-byte aligned rows (pointer and ldx % 8 == 0) take the vector path.
 *   x_amax  device absmax buffer of X16's quantised columns.
 *   Y16     device, N x M fp16 row-major. The handle must hold weight scales.
 *   y_amax  device absmax buffer or NULL. If given, the call fills it with the absmax of
 *           Y16[n][m] over amax_m0 <= m < amax_m1 (0 for an empty range): the x_amax of a next
 *           call that reads columns [amax_m0, amax_m1) of Y16. Must differ from x_amax.
 * Everything else (stream order, workspace, errors, limits on N) is as for us_spmm.
 *
 * us_absmax_f16: fills an absmax buffer from X16 (N <= 64 tokens, K columns) for the head of a chain.
 * us_quantize_f16: the codes themselves, packed as us_spmm expects X (N x ceil(K/2) bytes, even k in
 *   the low nibble), and the scales as fp16 bit patterns in x_scale (N entries, may be NULL).
 * Both take device pointers, run on `stream`, keep no state and allocate nothing.
 */
#define US_AMAX_BYTES (4 * 64 * (1 + 192))
us_status us_spmm_requant(us_handle* h, const void* X16, int64_t ldx, const void* x_amax, int32_t N,
                          void* Y16, void* y_amax, int64_t amax_m0, int64_t amax_m1, void* stream);
us_status us_absmax_f16(const void* X16, int64_t ldx, int32_t N, int64_t K, void* amax, void* stream);
us_status us_quantize_f16(const void* X16, int64_t ldx, int32_t N, int64_t K, const void* amax, void* Xq,
                          void* x_scale, void* stream);

/*
 * Test hook for the bounded waits of the kernel (no counterpart in the paper): from now on every
 * us_spmm on this handle leaves out the copy of the tile at `position` of the processing order
 * (0 <= position < number of tiles) and gives up its waits after wait_us microseconds
 * (1..2000000). Nothing is left in flight and nothing traps: the warp that waits for the missing
 * tile times out and stops, the kernel returns, and us_last_error reports US_ERR_DEVICE_TIMEOUT.
 * position < 0 restores normal operation.
 */
us_status us_debug_withhold_copy(us_handle* h, int64_t position, int64_t wait_us);

/*
 * Diagnostic stage timers of the SpMM kernel (paper Sec. VII-C reports where its kernel's time
 * goes; these are the same question asked of this one). enable: 1 = record in later us_spmm
 * calls, 0 = stop, -1 = leave as is. out (host, n_out >= 8 words, may be NULL): synchronises the
 * device, returns and clears the figures of all warps that ran since the last read -- sums of SM
 * cycles spent [0] waiting for staged tiles, [1] decoding + MMA, [2] in the reduce/store epilogue,
 * [3] whole warp lifetime; [4] the number of warps; [5] sum of cycles before a warp's first tile;
 * [6] the longest warp lifetime in cycles; [7] nanoseconds from the first warp's start to the last
 * warp's end; then, as far as n_out reaches, [8..11] sums of the prologue checkpoints (cycles at
 * which the range was known, the first copies issued, the table built, the activations staged)
 * and from [12] five words per CTA (192 CTAs), in ns after the first warp's start: CTA start, first
 * warp's end, activations staged, CTA end, past the wait for the stream's earlier work.
 * Recording costs a few clock reads per tile; off by default.
 */
us_status us_stage_timers(us_handle* h, int32_t enable, uint64_t* out, int32_t n_out);

/* Frees device and host memory. NULL is accepted. */
us_status us_destroy(us_handle* h);

/* Algorithmic bytes one us_spmm call moves: encoded W as stored + X + Y + scales. */
int64_t us_spmm_bytes(const us_handle* h, int32_t N, int32_t fp16_out);

/* Launch geometry of the next us_spmm(N): CTAs, threads per CTA, dynamic shared memory. */
us_status us_launch_info(const us_handle* h, int32_t N, int32_t* grid, int32_t* block,
                         int32_t* smem_bytes);

const char* us_status_string(us_status s);

#ifdef __cplusplus
}
#endif
#endif /* UNIONSPARSE_H_ */

/*
 * tpq.h -- C ABI of libtpq: low-bit synchronisation of tensor-parallel partial
 * sums on NVIDIA B200 (sm_100a), after "Towards Low-bit Communication for
 * Tensor Parallel LLM Inference" (arXiv 2411.07942).
 *
 * Setting (paper Section 2): N devices each hold a partial sum
 * f^(i)(x^(i)) in R^E per token; the synchronised value is their sum.  The
 * library provides the per-device compression C^(i) (tpq_quantize_pack), the
 * decompress-and-sum  sum_i D^(i)  (tpq_dequant_reduce), and the calibration
 * that fixes their static parameters (tpq_calibrate_ranges,
 * tpq_select_features), paper Section 3.
 *
 * Conventions for every entry point
 *   - "dev" pointers are CUDA device pointers, "host" pointers are host memory.
 *   - BF16 tensors are 16-bit patterns, row-major, row stride given in ELEMENTS
 *     (any stride >= E; the tiled kernels need E, k and the strides to be
 *     multiples of 8, other shapes run on slower shape-generic kernels).
 *   - The caller owns every data buffer.  The library owns only the context
 *     and its small device tables (O(N*E) floats), released by tpq_destroy.
 *   - Calls that take a `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream) only ENQUEUE work on it and never synchronise.  Calls
 *     that return host data synchronise the device.
 *   - Arguments are validated before anything is launched; a non-zero status
 *     means nothing was enqueued.  No entry point throws, aborts or traps.
 *   - A context is bound to the CUDA device that was current at tpq_create and
 *     may be used from one host thread at a time.  Work enqueued through one
 *     context must not overlap on the GPU with itself: use one stream, or
 *     streams ordered by events (the kernels share the context's status word,
 *     the calibration scratch and the block counter of tpq_quantize_pack_push).
 *   - One context serves all N simulated devices: the static parameters and
 *     the selected feature set are identical on every device by construction
 *     (Section 3: the set is static and shared by every sequence and device).
 */
#ifndef TPQ_H
#define TPQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tpq_ctx tpq_ctx; /* opaque */

typedef enum {
    TPQ_OK = 0,
    TPQ_ERR_INVALID_ARG = 1, /* null pointer, negative size, shard out of range, unsorted index set ... */
    TPQ_ERR_BAD_STATE = 2,   /* e.g. quantize before a feature set exists, select before calibration */
    TPQ_ERR_SIZE = 3,        /* a caller buffer is too small */
    TPQ_ERR_ALIGN = 4,       /* a device pointer is not 16-byte aligned */
    TPQ_ERR_CUDA = 5,        /* a CUDA call failed; text in tpq_last_error */
    TPQ_ERR_NOMEM = 6,       /* host or device allocation failed */
    TPQ_ERR_TIMEOUT = 7      /* a bounded device-side wait gave up (see tpq_device_status) */
} tpq_status;

typedef enum { TPQ_OUT_BF16 = 0, TPQ_OUT_FP32 = 1 } tpq_out_dtype;

/* Options for tpq_set_option. */
typedef enum {
    /* 0 = automatic (default); 1 = always the shape-generic kernels; 2 = the tiled kernels,
     * TPQ_ERR_INVALID_ARG from the call if the shape does not admit them (E, k and strides
     * multiples of 8, 4-bit codes). */
    TPQ_OPT_KERNEL_PATH = 0,
    /* Which tiled kernel tpq_dequant_reduce uses when the tiled path is taken: 0 = chosen from the
     * shape (default); 1 = row kernel (needs N <= 4 and (E-k)/8 <= 768, or N <= 8 and (E-k)/8 <= 640); 2 = tensor-map panel kernel
     * (needs N <= 16 and at least as many rows as it takes for the code stream to be 16-byte aligned again:
     * 1, 2 or 4); 3 = copy-ring panel kernel.  A kernel that the shape
     * does not admit makes the call return TPQ_ERR_INVALID_ARG.  For tests and measurements: all
     * kernels give identical results. */
    TPQ_OPT_DEQUANT_KERNEL = 1
} tpq_option;

/* Bytes a real exchange would move per synchronisation and per device
 * (paper Section 5: all-reduce executed as all-gather + local reduction). */
typedef struct tpq_comm_report {
    int64_t payload_bytes;             /* P: one device's payload for T tokens                         */
    int64_t quantized_allgather_send;  /* (N-1) * P, unicast all-gather of payloads (the method)        */
    int64_t bf16_allgather_send;       /* (N-1) * 2*T*E, all-gather of the raw BF16 partial sums         */
    int64_t bf16_ring_allreduce_send;  /* 2*(N-1)/N * 2*T*E, bandwidth-optimal BF16 all-reduce           */
    double bits_per_value;             /* 8*P / (T*E); equals b + (16-b)k/E up to the 16-byte pad (Sec. 4) */
    double bits_per_value_formula;     /* b + (16-b)k/E for b-bit codes: 4 + 12k/E for the paper's Int4   */
} tpq_comm_report;

/* ---------------------------------------------------------------- context */

/* Create a context for n_shards (N >= 1) devices and n_features (E >= 1)
 * features on the current CUDA device.  bits is the code width: 4 is the
 * paper's Int4 (Section 3) and the width the tiled kernels serve; 2..8 are
 * accepted (other code widths, as evaluated in Section 4 / Figure 3:
 * step R/(2^bits - 1), codes -2^(bits-1) .. 2^(bits-1)-1, one little-endian
 * stream of bits-wide codes) and run on the shape-generic kernels.  gamma is
 * the moving-average constant of Eq. (1)-(2) (the paper uses 0.01),
 * 0 <= gamma <= 1.  Errors: INVALID_ARG, NOMEM, CUDA. */
tpq_status tpq_create(tpq_ctx **ctx, int n_shards, int n_features, int bits, float gamma);
tpq_status tpq_destroy(tpq_ctx *ctx); /* NULL is accepted */
tpq_status tpq_set_option(tpq_ctx *ctx, tpq_option opt, int value);

/* ------------------------------------------------------------ calibration */

/* Section 3 "Calibration", Eq. (1)-(2): fold n_seq sequences of device `shard`
 * into its running (m_j, M_j), in index order.  For every sequence the
 * column-wise minimum and maximum over its S tokens are taken; the first
 * sequence a device ever sees initialises (m, M), later ones update
 *   m <- (1-gamma) m + gamma min,  M <- (1-gamma) M + gamma max
 * in binary32, evaluated left to right.
 *   y_bf16_dev : [n_seq][S][E] BF16, row stride row_stride_elems (>= E), the
 *                sequences back to back (sequence q starts at row q*S).
 * Enqueues on cuda_stream.  May grow a context-owned scratch buffer
 * (cudaMalloc) when n_seq*S exceeds every earlier call.
 * n_seq == 0 is a no-op.  Errors: INVALID_ARG, ALIGN, NOMEM, CUDA. */
tpq_status tpq_calibrate_ranges(tpq_ctx *ctx, int shard, const void *y_bf16_dev, int64_t n_seq, int64_t S,
                                int64_t row_stride_elems, void *cuda_stream);

/* The same fold as tpq_calibrate_ranges, for callers that must not allocate.  (The paper has no
 * counterpart: this is a deployment variant of the call above.)  tpq_calibrate_ranges may grow its
 * scratch buffer with cudaMalloc / cudaFree, which a caller cannot afford when it runs inside a
 * serving loop whose device memory is owned by a pool, under a framework that forbids allocation
 * outside start-up, or at a point where the implicit device synchronisation of cudaFree would stall
 * other streams.  This variant keeps the per-sequence column extremes in a fixed array that is part
 * of the library image: TPQ_NOALLOC_SCRATCH_MAX_BYTES (4 MiB) of global memory on every device that
 * loads the library, held until the process exits.  It calls no cudaMalloc, no cudaFree and no
 * allocating library routine.
 *   Limit: 4 * n_seq * E bytes must fit the array, i.e. n_seq * E <= 1 048 576 (e.g. 204 sequences at
 *   E = 5120) and n_seq <= 65535; larger calls return TPQ_ERR_SIZE and enqueue nothing: fold fewer
 *   sequences per call (the result does not depend on how the sequences are split over calls).
 *   The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that
 *   first call before any stream capture begins.  The device the context was created on must be current.
 *   All calls, from every context, share the one array per device: two calls whose kernels can overlap
 *   on the GPU (different streams) race on it; serialise them on one stream or with events.  Nothing
 *   in the array has to be cleared between calls: every element a call reads it has written first.
 * Same arguments, results and errors as tpq_calibrate_ranges otherwise. */
#define TPQ_NOALLOC_SCRATCH_MAX_BYTES (4u << 20)
tpq_status tpq_calibrate_ranges_noalloc(tpq_ctx *ctx, int shard, const void *y_bf16_dev, int64_t n_seq, int64_t S,
                                        int64_t row_stride_elems, void *cuda_stream);

/* Section 3 "Selecting High Precision Features": R^(i)_j = 2 max(-m, M),
 * aggregated range Rbar_j = sum_i R^(i)_j (binary32, devices ascending), the
 * k features with the largest Rbar_j (ties: lower index) become the BF16 set;
 * every other feature gets its static Int4 step s = R/15 (floored at 2^-23)
 * and reciprocal.  k < 0 selects the paper's k = floor(E/64) (Section 4).
 * Every device must have been calibrated with at least one sequence
 * (else BAD_STATE).  Writes the k indices, ascending, to hp_idx_out_host
 * (capacity >= k int32; may be NULL) and k to k_out (may be NULL).
 * Synchronises the device. */
tpq_status tpq_select_features(tpq_ctx *ctx, int k, int32_t *hp_idx_out_host, int *k_out);

/* Install an arbitrary feature set (strictly ascending indices in [0, E),
 * 0 <= k <= E) instead of the top-k one: the paper's "Int4" (k = 0) and
 * "Int4 + Random BF16" baselines (Section 4), or a restored set.  Steps are
 * derived from the calibrated ranges as in tpq_select_features.  Synchronises. */
tpq_status tpq_set_features(tpq_ctx *ctx, const int32_t *hp_idx_host, int k);

/* Install calibration state directly: m and M are [N][E] binary32 (host),
 * counts[N] the number of sequences each device has folded.  Used to resume
 * calibration or to skip it.  Synchronises. */
tpq_status tpq_set_ranges(tpq_ctx *ctx, const float *m_host, const float *M_host, const int64_t *counts_host);

/* Read back state (host outputs, any may be NULL; synchronises):
 * m, M, R are [N][E]; Rbar is [E].  R and Rbar are valid after a feature set exists. */
tpq_status tpq_get_ranges(tpq_ctx *ctx, float *m_host, float *M_host, float *R_host, float *Rbar_host);
/* s and inv_s are [N][E] (entries at selected features are defined but unused). BAD_STATE before a feature set. */
tpq_status tpq_get_scales(tpq_ctx *ctx, float *s_host, float *inv_s_host);
/* Number of selected features, or -1 before a feature set exists. */
int tpq_num_selected(const tpq_ctx *ctx);
/* The selected indices, ascending (capacity >= k).  BAD_STATE before a feature set. */
tpq_status tpq_get_features(tpq_ctx *ctx, int32_t *hp_idx_out_host);
/* The slot order of the payload's code section (see "Wire format" below): slot_feature_out_host[c],
 * 0 <= c < E-k, is the feature whose code slot c of every token carries (capacity >= E-k int32).
 * The order is this library's choice (the paper gives only the bit count, Section 4).
 * BAD_STATE before a feature set; synchronises. */
tpq_status tpq_get_slot_order(tpq_ctx *ctx, int32_t *slot_feature_out_host);

/* ------------------------------------------------------------- the payload */

/* Payload size in bytes for T tokens with the current feature set:
 *   roundup16(ceil(T*(E-k)/2)) + 2*T*k
 * (Section 4 counts (E-k) 4-bit codes and k BF16 values per token; the byte
 * layout below is this library's: the paper fixes only the bit count).
 *
 * Wire format.  With L = E-k:
 *   bytes [0, roundup16(ceil(T*L/2)))  the code section: one flat stream of
 *       4-bit two's-complement codes; code p = t*L + c (token t, slot c) is
 *       the low nibble of byte p/2 if p is even, the high nibble if p is odd;
 *       unused nibbles and the padding up to a multiple of 16 bytes are 0;
 *   then T*k BF16 values, token-major: value t*k + h is the h-th selected
 *       feature (ascending feature index) of token t, its bits unchanged.
 * No header; the static steps are never transmitted.
 *
 * Slot order ("hole filling"): which feature slot c of a token carries.
 * Let S be the selected set.  The holes are the selected features below L,
 * ascending: h_0 < h_1 < ...; the fillers are the unselected features at or
 * above L, ascending: f_0 < f_1 < ... (there are equally many of both).
 *   slot c, 0 <= c < L, carries feature c        if c is not selected,
 *                               feature f_i      if c = h_i.
 * So every unselected feature below L keeps its own index as slot, and the
 * i-th filler takes the i-th hole.  Example: E = 8, S = {1, 6}, L = 6: the
 * hole is 1, the filler is 7, the slots carry features 0 7 2 3 4 5 and the
 * BF16 values are features 1 and 6.  tpq_get_slot_order returns the table.
 * For code widths other than 4 bits the stream is the same with bits-wide
 * codes: code p occupies bits [p*bits, (p+1)*bits) of the little-endian stream.
 * tpq_payload_bytes returns 0 before a feature set exists or for T <= 0. */
size_t tpq_payload_bytes(const tpq_ctx *ctx, int64_t T);
/* The same closed form without a context (Int4), and for a code width of
 * 2..8 bits: roundup16(ceil(T*(E-k)*bits / 8)) + 2*T*k. */
size_t tpq_payload_bytes_for(int64_t T, int64_t E, int64_t k);
size_t tpq_payload_bytes_for_bits(int64_t T, int64_t E, int64_t k, int bits);

/* Section 5 / Section 4: bytes per synchronisation and bits per value. */
tpq_status tpq_comm_bytes(const tpq_ctx *ctx, int64_t T, tpq_comm_report *out);

/* --------------------------------------------------------- the hot path */

/* C^(i) (Sections 2-3, Figure 2): one device's [T][E] BF16 partial sums ->
 * payload.  Low-precision feature: u = fl(x * inv_s); u clamped to [-8, 7];
 * code = round-half-to-even(u) (two binary32 roundings, never fused).
 * Selected feature: the BF16 pattern is copied unchanged.
 *   y_bf16_dev  : [T][E] BF16, row stride row_stride_elems (>= E)
 *   payload_dev : >= tpq_payload_bytes(ctx, T) bytes, 16-byte aligned; every
 *                 byte of the payload (padding included) is written.
 * Enqueues on cuda_stream; T == 0 is a no-op.
 * Errors: BAD_STATE (no feature set), INVALID_ARG, ALIGN, SIZE, CUDA. */
tpq_status tpq_quantize_pack(tpq_ctx *ctx, int shard, const void *y_bf16_dev, int64_t T, int64_t row_stride_elems,
                             void *payload_dev, size_t payload_capacity, void *cuda_stream);

/* The same C^(i) for n consecutive devices first_shard .. first_shard+n-1 in ONE launch, for a process
 * that holds several devices' partial sums on one GPU (the single-GPU simulation of N ranks; in a real
 * deployment every rank calls tpq_quantize_pack once).  The SMs are divided among the shards; every payload
 * is byte-identical to what tpq_quantize_pack writes for that shard.
 *   ys_dev_host / payloads_dev_host : HOST arrays of n DEVICE pointers (inputs [T][E] with the common row
 *   stride; payloads of payload_capacity bytes each), all 16-byte aligned.
 * Enqueues on cuda_stream; T == 0 or n == 0 is a no-op.  Errors as tpq_quantize_pack. */
tpq_status tpq_quantize_pack_batch(tpq_ctx *ctx, int first_shard, int n, const void *const *ys_dev_host, int64_t T,
                                   int64_t row_stride_elems, void *const *payloads_dev_host, size_t payload_capacity,
                                   void *cuda_stream);

/* sum_i D^(i) (Figure 2 caption; Section 5 "local reduction"): N payloads ->
 * the synchronised [T][E] output in the original feature order.
 * Low-precision feature: sum_i code_i * s^(i)_j; selected feature: sum_i of
 * the BF16 values.  Accumulation is binary32 in ascending device order with
 * one final rounding for BF16 output.
 *   payloads_dev_host : HOST array of n_payloads DEVICE pointers, device order;
 *                       n_payloads must equal N; each 16-byte aligned
 *   out_dev           : [T][E] of dt, row stride out_row_stride_elems (>= E)
 * Enqueues on cuda_stream; T == 0 is a no-op.
 * Errors: BAD_STATE, INVALID_ARG, ALIGN, CUDA. */
tpq_status tpq_dequant_reduce(tpq_ctx *ctx, const void *const *payloads_dev_host, int n_payloads, int64_t T,
                              void *out_dev, tpq_out_dtype dt, int64_t out_row_stride_elems, void *cuda_stream);

/* The same with the layer's bias added after the sum (Section 2: f(x) = sum_i f^(i)(x^(i)) + b):
 * out[t][j] = round(fl32(acc[t][j] + bias[j])), acc the binary32 sum of tpq_dequant_reduce before its
 * final rounding.  bias_dev: DEVICE pointer to E binary32 values, 16-byte aligned, read during the
 * call's kernels (the caller keeps it alive and unchanged until they have run).  Errors as
 * tpq_dequant_reduce, plus INVALID_ARG for a NULL bias and ALIGN for a misaligned one. */
tpq_status tpq_dequant_reduce_bias(tpq_ctx *ctx, const void *const *payloads_dev_host, int n_payloads, int64_t T,
                                   void *out_dev, tpq_out_dtype out_dtype, int64_t out_row_stride,
                                   const float *bias_dev, void *stream);

/* ------------------------------------------------- the layer ahead of the synchronisation point (Section 2) */

/* Section 2 defines what is synchronised: the output of the last linear layer of an attention or
 * feed-forward block, f^(i)(x^(i)) = x^(i) W^(i) on device i.  These two calls compute that product on the
 * tensor cores and compress it in the same kernel, so the [T][E] partial sums are never written:
 *   payload = C^(i)( bf16( x W^T ) ),  x: [T][K] BF16,  W: [E][K] BF16 (one row per output feature),
 * FP32 accumulation, one rounding to BF16 (the layer's output type), then exactly tpq_quantize_pack.
 *
 * tpq_permute_weight: once per weight matrix and feature set, gather the rows of w_bf16_dev ([E][K],
 * row-major, 16-byte aligned) into the payload's slot order ("Wire format" above; tpq_get_slot_order): row
 * c < E-k is the feature that code slot c carries, row E-k+h the h-th selected feature.  w_slots_dev: [E][K], 16-byte aligned, not aliasing w.
 * Errors: BAD_STATE (no feature set), INVALID_ARG, ALIGN, CUDA. */
tpq_status tpq_permute_weight(tpq_ctx *ctx, const void *w_bf16_dev, int64_t K, void *w_slots_dev, void *cuda_stream);

/* tpq_linear_quantize_pack: the fused layer for one device.
 *   x_bf16_dev  : [T][K] BF16, row-major, 16-byte aligned; K a multiple of 8
 *   w_slots_dev : output of tpq_permute_weight for the current feature set
 *   payload_dev : as tpq_quantize_pack; byte-identical to tpq_quantize_pack applied to bf16(x W^T)
 *   y_slots_dev : NULL, or [T][E] BF16 (16-byte aligned) that receives the rounded partial sums in slot
 *                 order (column c as the rows of w_slots_dev) -- for verification or a residual path
 * Needs 4-bit codes and E, k multiples of 8 (INVALID_ARG otherwise).  Enqueues on cuda_stream; T == 0 is a
 * no-op.  Errors: BAD_STATE, INVALID_ARG, ALIGN, SIZE, CUDA; TPQ_ERR_TIMEOUT through tpq_device_status. */
tpq_status tpq_linear_quantize_pack(tpq_ctx *ctx, int shard, const void *x_bf16_dev, const void *w_slots_dev, int64_t T,
                                    int64_t K, void *payload_dev, size_t payload_capacity, void *y_slots_dev,
                                    void *cuda_stream);

/* ------------------------------------------------- exchange (Section 5) */

/* Section 5 describes the system-level form of the method: the payloads are all-gathered and every
 * device then reduces locally.  These two calls are that exchange without a collective library: the
 * quantiser stores its payload straight into every destination (its own receive slot and, through
 * peer-mapped pointers over NVLink, the slot it owns in each peer's receive buffer), and the reducing
 * side waits, with a limit, for the N arrival words in its own memory.
 *
 * tpq_quantize_pack_push: C^(i) of tpq_quantize_pack for one shard, the payload written to n_dst
 * destinations (byte-identical in each), then `epoch` written to the n_dst arrival words with release
 * semantics at system scope once every byte of every destination has been stored.
 *   dst_dev_host     : HOST array of n_dst DEVICE pointers (local or peer-mapped), each of dst_capacity
 *                      >= tpq_payload_bytes(ctx, T) bytes, 16-byte aligned
 *   arrived_dev_host : HOST array of n_dst DEVICE pointers to 32-bit words, 4-byte aligned, one per
 *                      destination, in the same memory as the destination
 *   n_dst            : 1 .. 16
 *   epoch            : the step's tag; a receiver waits for exactly this value, so consecutive steps
 *                      on the same slot use different tags
 * T must be >= 1.  Enqueues on cuda_stream.  The caller owns the slot discipline (a slot is not
 * pushed again before its reader has finished: two alternating slot sets suffice when every step
 * waits for all N arrivals).  Errors: BAD_STATE, INVALID_ARG, ALIGN, SIZE, CUDA. */
tpq_status tpq_quantize_pack_push(tpq_ctx *ctx, int shard, const void *y_bf16_dev, int64_t T, int64_t row_stride_elems,
                                  void *const *dst_dev_host, uint32_t *const *arrived_dev_host, int n_dst,
                                  size_t dst_capacity, uint32_t epoch, void *cuda_stream);

/* Enqueue a wait, on cuda_stream, until the n arrival words at arrived_dev (DEVICE pointer, this GPU's
 * memory, 4-byte aligned) all equal `epoch`; work enqueued behind it on the stream (tpq_dequant_reduce)
 * then reads complete payloads.  The wait gives up after timeout_ns (0: one second; at most 5 s): the
 * context's device status becomes TPQ_ERR_TIMEOUT (tpq_device_status), the kernel returns, the stream
 * continues and whatever is reduced afterwards is unspecified.  n: 1 .. 1024.
 * Errors: INVALID_ARG, ALIGN, CUDA. */
tpq_status tpq_wait_arrivals(tpq_ctx *ctx, const uint32_t *arrived_dev, int n, uint32_t epoch, uint64_t timeout_ns,
                             void *cuda_stream);

/* tpq_dequant_reduce (with the bias of tpq_dequant_reduce_bias when bias_dev is not NULL) whose kernels wait
 * themselves, in their prologue and with the limit of tpq_wait_arrivals, for the N arrival words at
 * arrived_dev (word i beside payload i) before they read any payload: the wait costs no launch of its own.
 * Errors as tpq_dequant_reduce and tpq_wait_arrivals; expiry is reported through tpq_device_status. */
tpq_status tpq_dequant_reduce_arrivals(tpq_ctx *ctx, const void *const *payloads_dev_host, int n_payloads, int64_t T,
                                       void *out_dev, tpq_out_dtype out_dtype, int64_t out_row_stride,
                                       const float *bias_dev, const uint32_t *arrived_dev, uint32_t epoch,
                                       uint64_t timeout_ns, void *cuda_stream);

/* ------------------------------------------------- checkpoint and status */

/* Serialise / restore the whole static state (N, E, bits, gamma, counts, m, M,
 * feature set) as a flat little-endian blob.  tpq_get_state with blob == NULL
 * writes the required size to *bytes; otherwise *bytes is the capacity on
 * entry and the size written on return.  tpq_set_state requires a context of
 * the same N, E and bits.  Both synchronise. */
tpq_status tpq_get_state(tpq_ctx *ctx, void *blob_host, size_t *bytes);
tpq_status tpq_set_state(tpq_ctx *ctx, const void *blob_host, size_t bytes);

/* Synchronise and read the device-side status word: TPQ_OK, or
 * TPQ_ERR_TIMEOUT if a kernel's bounded wait on an asynchronous copy gave up
 * (the kernel then returned early and its output is incomplete).  The word is
 * cleared by the call. */
tpq_status tpq_device_status(tpq_ctx *ctx);

/* Kernels launched by this context since creation (for launch accounting). */
int64_t tpq_launch_count(const tpq_ctx *ctx);

const char *tpq_status_string(tpq_status st);
const char *tpq_last_error(const tpq_ctx *ctx); /* "" if none; valid until the next call on ctx */
const char *tpq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TPQ_H */

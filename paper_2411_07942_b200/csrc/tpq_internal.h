// Internal declarations shared by the translation units of libtpq (not installed).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tpq.h"

#define TPQ_MAX_SHARDS 64

// Device tables of one context.  All in the ORIGINAL feature order unless noted.
struct tpq_tables {
    float *m, *M;        // [N][E] running minimum / maximum, Eq. (1)-(2)
    float *R;            // [N][E] symmetric range 2 max(-m, M)
    float *Rbar;         // [E]    aggregated range
    float *s, *inv_s;    // [N][E] Int4 step and its reciprocal
    float *s_k;          // [N][E] step with 0 at selected features (dequantiser's copy)
    float *s_slot;       // [N][E] step of the feature held by code slot c (slot order; 0 for c >= E-k)
    uint8_t *flag;       // [E]    1 = selected (kept in BF16)
    int32_t *hpre;       // [E]    number of selected features before j
    int32_t *pos;        // [E]    >= 0: code slot of feature j; < 0: -(h+1), h = rank among selected
    int32_t *hp_idx;     // [E]    first k entries: selected features, ascending
    int32_t *lp_idx;     // [E]    first L = E-k entries: feature held by code slot c (slot order below)
    int32_t *hole;       // [E]    first n_holes entries: selected features below L, ascending (slots to fill)
    int32_t *filler;     // [E]    first n_holes entries: unselected features at or above L, ascending
    uint32_t *grp;       // [ceil(E/8)] per group of 8 features: (selected before the group << 8) | 8-bit mask
    int *status;         // device status word (0 = ok)
    unsigned int *push_done;  // blocks of a pushing quantiser that have finished (0 between launches)
};

// Arrival words a reduction waits for before it reads the payloads (the fused exchange): n words in this
// GPU's memory, each written with `epoch` by the device that pushed the matching payload.
struct tpq_arrivals {
    const uint32_t *words;
    uint32_t epoch;
    int n;
    unsigned long long timeout_ns;
    int *status;
};

struct tpq_ctx {
    int N, E, bits;
    float gamma;
    int k;              // -1 until a feature set exists
    int n_holes;        // selected features below E-k (= unselected ones at or above it)
    int device;
    int sm_count;
    int smem_optin;     // max dynamic shared memory per block
    int kernel_path;    // TPQ_OPT_KERNEL_PATH
    int dq_kernel;      // TPQ_OPT_DEQUANT_KERNEL
    int64_t counts[TPQ_MAX_SHARDS];
    tpq_tables t;
    void *scratch;      // calibration partial extremes
    size_t scratch_bytes;
    int64_t launches;
    void *dq_cache;     // tensor maps of recently used payloads (dequant.cu)
    const float *call_bias;  // bias of the tpq_dequant_reduce_bias call in progress (NULL otherwise)
    tpq_arrivals call_arr;   // arrival words the reduction in progress waits for (words == NULL: none)
    char err[512];
};

// Slot order of a token's L = E-k codes ("hole filling"): slot c holds feature c unless c is selected;
// the selected features below L (hole[], ascending) are filled in order with the unselected features
// at or above L (filler[], ascending).  Most features keep their own index as slot, so a group of 8
// adjacent features is one aligned 32-bit word of the code stream.
//
// Payload geometry (Section 4 bit count; layout documented in tpq.h).
static inline int64_t tpq_lp_bytes_i(int64_t T, int64_t E, int64_t k, int bits = 4)
{
    int64_t nbits = T * (E - k) * bits;  // one flat little-endian bit stream of `bits`-bit codes
    int64_t b = (nbits + 7) / 8;
    return (b + 15) / 16 * 16;
}

// ---- launchers (each returns the launch error, enqueues on `st`, adds to *launches)

// Eq. (1)-(2): column extremes of n_seq sequences, then the moving-average fold.
size_t tpq_calib_scratch_bytes(int64_t n_seq, int64_t S, int E, int sm_count, int *n_split_out);
cudaError_t tpq_launch_calibrate(const uint16_t *y, int64_t n_seq, int64_t S, int64_t stride, int E, float *m,
                                 float *M, int64_t count0, float gamma, void *scratch, int n_split, cudaStream_t st,
                                 int64_t *launches);

// Allocation-free calibration: fixed scratch array inside the library (see calibrate.cu).
#define TPQ_NOALLOC_SCRATCH_BYTES TPQ_NOALLOC_SCRATCH_MAX_BYTES  /* tpq.h */
cudaError_t tpq_static_scratch_address(int device, void **ptr_out);
int tpq_static_scratch_splits(int64_t n_seq, int64_t S, int E, int sm_count);

// Section 3: ranges, aggregate, steps; top-k flags (or flags given); index tables.
cudaError_t tpq_launch_ranges(const tpq_tables &t, int N, int E, int bits, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_topk_flags(const tpq_tables &t, int E, int k, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_tables(const tpq_tables &t, int N, int E, int k, cudaStream_t st, int64_t *launches);

// C^(i): quantise + pack.
bool tpq_quantize_tiled_ok(const tpq_ctx *c, int64_t T, int64_t stride);
cudaError_t tpq_launch_quantize_generic(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                        uint8_t *payload, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_quantize_tiled(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                      uint8_t *payload, cudaStream_t st, int64_t *launches);

cudaError_t tpq_launch_quantize_tiled_batch(const tpq_ctx *c, int shard0, int n, const void *const *ys, int64_t T,
                                            int64_t stride, void *const *payloads, cudaStream_t st, int64_t *launches);

// Push mode of the tiled quantiser: every payload store goes to n_dst destinations and the last block to
// finish writes `epoch` to the n_dst arrival words (release, system scope).  n_dst <= tpq_push_max_dst().
int tpq_push_max_dst();
cudaError_t tpq_launch_quantize_tiled_push(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                           void *const *dst, uint32_t *const *arrived, int n_dst, uint32_t epoch,
                                           cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_publish_arrivals(uint32_t *const *arrived, int n_dst, uint32_t epoch, cudaStream_t st,
                                        int64_t *launches);
// Bounded wait until n arrival words equal `epoch`; on expiry the context's device status becomes TPQ_ERR_TIMEOUT.
cudaError_t tpq_launch_wait_arrivals(const tpq_ctx *c, const uint32_t *arrived, int n, uint32_t epoch,
                                     unsigned long long timeout_ns, cudaStream_t st, int64_t *launches);

// cuTensorMapEncodeTiled, looked up once through the runtime (the library does not link the driver API);
// NULL if the driver does not provide it.
typedef CUresult (*tpq_encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                        const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                        CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
tpq_encode_tiled_fn tpq_tensor_map_encoder();

// The pre-synchronisation linear layer fused with the compressor (linear.cu): tensor-core GEMM whose epilogue
// quantises and packs.  w_slots is the [E][K] weight matrix with its rows in slot order (tpq_launch_permute_weight).
bool tpq_linear_ok(const tpq_ctx *c, int64_t T, int64_t K);
cudaError_t tpq_launch_permute_weight(const tpq_ctx *c, const void *w, void *out, int64_t K, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_linear_quantize(const tpq_ctx *c, int shard, const void *x, const void *w_slots, int64_t T, int64_t K,
                                       void *payload, void *y_slots, cudaStream_t st, int64_t *launches);

// Code widths other than 4 bits on shapes that are multiples of 8 (groups.cu).
bool tpq_groups_ok(const tpq_ctx *c, int64_t T, int64_t stride);
cudaError_t tpq_launch_quantize_groups(const tpq_ctx *c, int shard0, int n, const void *const *ys, int64_t T,
                                       int64_t stride, void *const *payloads, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_dequant_groups(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int fp32_out,
                                      int64_t out_stride, cudaStream_t st, int64_t *launches);

// sum_i D^(i): dequantise + reduce.
bool tpq_dequant_tiled_ok(const tpq_ctx *c, int64_t T, int64_t out_stride, int fp32_out);
void tpq_dequant_release(tpq_ctx *c);  // frees dq_cache
cudaError_t tpq_launch_dequant_generic(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out,
                                       int fp32_out, int64_t out_stride, cudaStream_t st, int64_t *launches);
cudaError_t tpq_launch_dequant_tiled(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out,
                                     int fp32_out, int64_t out_stride, cudaStream_t st, int64_t *launches);

// ---- programmatic dependent launch: a kernel launched this way may start (and run its prologue: barrier
// set-up, loads of the context's tables, which no kernel in flight writes) before the kernel ahead of it in
// the stream has drained; it must execute tpq_grid_dep_wait() before it touches memory that earlier work in
// the stream may still read or write.
#ifdef __CUDACC__
__device__ __forceinline__ void tpq_grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void tpq_grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- mbarrier / asynchronous-copy primitives shared by the pipelined kernels.  Every wait is bounded: it
// returns false when the phase has not completed after TPQ_WAIT_LIMIT attempts (each attempt suspends the
// thread for a hardware time slice), and the caller records TPQ_ERR_TIMEOUT and leaves.
constexpr int TPQ_WAIT_LIMIT = 1 << 22;
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int i = 0; i < TPQ_WAIT_LIMIT; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
// global -> this block's shared memory; bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// one box of a 2-D tensor map -> this block's shared memory (x: innermost coordinate, 16-byte aligned in bytes)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *map, int x, int y, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

// Bounded wait of a block for the arrival words (every block waits by itself; call it ahead of a
// __syncthreads() that precedes the block's first payload read).  On expiry the status word becomes
// TPQ_ERR_TIMEOUT and the block carries on: its output is then unspecified.
// (Out of line on purpose: inlined, the polling loop's atomics and acquire loads cost the kernels' prologues
// a few hundred cycles even when there is nothing to wait for.)
static __device__ __noinline__ void tpq_poll_arrivals(const uint32_t *words, uint32_t epoch, int n,
                                                      unsigned long long timeout_ns, int *status)
{
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        unsigned long long t0, t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
        for (;;) {
            uint32_t v;
            asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(words + i) : "memory");
            if (v == epoch) break;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            if (t1 - t0 > timeout_ns) {
                atomicExch(status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
            __nanosleep(100);
        }
        // the payloads are read next through bulk asynchronous copies as well as plain loads
        asm volatile("fence.proxy.async;" ::: "memory");
    }
}

__device__ __forceinline__ void tpq_block_wait_arrivals(const tpq_arrivals &a)
{
    if (a.words != nullptr) tpq_poll_arrivals(a.words, a.epoch, a.n, a.timeout_ns, a.status);
}

template <typename... KArgs, typename... Args>
cudaError_t tpq_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

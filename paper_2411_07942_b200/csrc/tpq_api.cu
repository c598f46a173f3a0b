// libtpq C ABI: context, validation, state and the entry points declared in tpq.h.
// Every computation of the method runs in the CUDA kernels of this library; the host
// code below only validates, sizes and launches.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "tpq_internal.h"

namespace {

tpq_status fail(tpq_ctx *c, tpq_status st, const char *fmt, ...)
{
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof c->err, fmt, ap);
        va_end(ap);
    }
    return st;
}

tpq_status cuda_fail(tpq_ctx *c, cudaError_t e, const char *what)
{
    return fail(c, e == cudaErrorMemoryAllocation ? TPQ_ERR_NOMEM : TPQ_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define TPQ_CUDA(c, call)                                   \
    do {                                                    \
        cudaError_t e_ = (call);                            \
        if (e_ != cudaSuccess) return cuda_fail(c, e_, #call); \
    } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
cudaError_t dalloc(T **p, size_t n)
{
    return cudaMalloc(reinterpret_cast<void **>(p), (n ? n : 1) * sizeof(T));
}

void free_tables(tpq_tables &t)
{
    cudaFree(t.m); cudaFree(t.M); cudaFree(t.R); cudaFree(t.Rbar); cudaFree(t.s); cudaFree(t.inv_s);
    cudaFree(t.s_k); cudaFree(t.s_slot); cudaFree(t.flag); cudaFree(t.hpre); cudaFree(t.pos); cudaFree(t.hp_idx);
    cudaFree(t.lp_idx); cudaFree(t.hole); cudaFree(t.filler); cudaFree(t.grp); cudaFree(t.status); cudaFree(t.push_done);
    memset(&t, 0, sizeof t);
}

bool all_calibrated(const tpq_ctx *c)
{
    for (int i = 0; i < c->N; ++i)
        if (c->counts[i] < 1) return false;
    return true;
}

// ranges -> (flags already on the device) -> tables; synchronises
tpq_status build_tables(tpq_ctx *c, int k, bool topk)
{
    cudaError_t e = tpq_launch_ranges(c->t, c->N, c->E, c->bits, 0, &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "ranges kernel");
    if (topk) {
        e = tpq_launch_topk_flags(c->t, c->E, k, 0, &c->launches);
        if (e != cudaSuccess) return cuda_fail(c, e, "top-k kernel");
    }
    e = tpq_launch_tables(c->t, c->N, c->E, k, 0, &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "tables kernel");
    TPQ_CUDA(c, cudaDeviceSynchronize());
    c->n_holes = 0;
    if (k > 0 && k < c->E)
        TPQ_CUDA(c, cudaMemcpy(&c->n_holes, c->t.hpre + (c->E - k), sizeof(int), cudaMemcpyDeviceToHost));
    c->k = k;
    return TPQ_OK;
}

struct StateHeader {
    char magic[8];
    int32_t version, N, E, bits;
    float gamma;
    int32_t k;
};

}  // namespace

tpq_encode_tiled_fn tpq_tensor_map_encoder()
{
    static tpq_encode_tiled_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tpq_encode_tiled_fn>(sym);
        else
            (void)cudaGetLastError();
    }
    return fn;
}

extern "C" {

const char *tpq_version(void) { return "tpq 0.1 (sm_100a)"; }

const char *tpq_status_string(tpq_status st)
{
    switch (st) {
        case TPQ_OK: return "ok";
        case TPQ_ERR_INVALID_ARG: return "invalid argument";
        case TPQ_ERR_BAD_STATE: return "bad state";
        case TPQ_ERR_SIZE: return "buffer too small";
        case TPQ_ERR_ALIGN: return "misaligned pointer or stride";
        case TPQ_ERR_CUDA: return "CUDA error";
        case TPQ_ERR_NOMEM: return "out of memory";
        case TPQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char *tpq_last_error(const tpq_ctx *ctx) { return ctx ? ctx->err : ""; }

tpq_status tpq_create(tpq_ctx **out, int n_shards, int n_features, int bits, float gamma)
{
    if (!out) return TPQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_shards < 1 || n_shards > TPQ_MAX_SHARDS || n_features < 1 || n_features > (1 << 22)) return TPQ_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return TPQ_ERR_INVALID_ARG;
    if (!(gamma >= 0.0f && gamma <= 1.0f)) return TPQ_ERR_INVALID_ARG;
    tpq_ctx *c = new (std::nothrow) tpq_ctx();
    if (!c) return TPQ_ERR_NOMEM;
    memset(c, 0, sizeof *c);
    c->N = n_shards; c->E = n_features; c->bits = bits; c->gamma = gamma; c->k = -1;
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device);
    const size_t NE = (size_t)n_shards * n_features, E = n_features;
    tpq_tables &t = c->t;
    if (e == cudaSuccess) e = dalloc(&t.m, NE);
    if (e == cudaSuccess) e = dalloc(&t.M, NE);
    if (e == cudaSuccess) e = dalloc(&t.R, NE);
    if (e == cudaSuccess) e = dalloc(&t.Rbar, E);
    if (e == cudaSuccess) e = dalloc(&t.s, NE);
    if (e == cudaSuccess) e = dalloc(&t.inv_s, NE);
    if (e == cudaSuccess) e = dalloc(&t.s_k, NE);
    if (e == cudaSuccess) e = dalloc(&t.s_slot, NE);
    if (e == cudaSuccess) e = dalloc(&t.flag, E);
    if (e == cudaSuccess) e = dalloc(&t.hpre, E);
    if (e == cudaSuccess) e = dalloc(&t.pos, E);
    if (e == cudaSuccess) e = dalloc(&t.hp_idx, E);
    if (e == cudaSuccess) e = dalloc(&t.lp_idx, E);
    if (e == cudaSuccess) e = dalloc(&t.hole, E);
    if (e == cudaSuccess) e = dalloc(&t.filler, E);
    if (e == cudaSuccess) e = dalloc(&t.grp, (E + 7) / 8);
    if (e == cudaSuccess) e = dalloc(&t.status, 1);
    if (e == cudaSuccess) e = dalloc(&t.push_done, 1);
    if (e == cudaSuccess) e = cudaMemset(t.m, 0, NE * sizeof(float));
    if (e == cudaSuccess) e = cudaMemset(t.M, 0, NE * sizeof(float));
    if (e == cudaSuccess) e = cudaMemset(t.status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(t.push_done, 0, sizeof(unsigned int));
    if (e != cudaSuccess) {
        tpq_status st = (e == cudaErrorMemoryAllocation) ? TPQ_ERR_NOMEM : TPQ_ERR_CUDA;
        free_tables(t);
        delete c;
        return st;
    }
    *out = c;
    return TPQ_OK;
}

tpq_status tpq_destroy(tpq_ctx *c)
{
    if (!c) return TPQ_OK;
    cudaDeviceSynchronize();
    free_tables(c->t);
    cudaFree(c->scratch);
    tpq_dequant_release(c);
    delete c;
    return TPQ_OK;
}

tpq_status tpq_set_option(tpq_ctx *c, tpq_option opt, int value)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (opt == TPQ_OPT_KERNEL_PATH && value >= 0 && value <= 2) {
        c->kernel_path = value;
        return TPQ_OK;
    }
    if (opt == TPQ_OPT_DEQUANT_KERNEL && value >= 0 && value <= 3) {
        c->dq_kernel = value;
        return TPQ_OK;
    }
    return fail(c, TPQ_ERR_INVALID_ARG, "unknown option %d or value %d", (int)opt, value);
}

tpq_status tpq_calibrate_ranges(tpq_ctx *c, int shard, const void *y, int64_t n_seq, int64_t S, int64_t stride,
                                void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (shard < 0 || shard >= c->N) return fail(c, TPQ_ERR_INVALID_ARG, "shard %d out of range [0, %d)", shard, c->N);
    if (n_seq < 0 || S < 1) return fail(c, TPQ_ERR_INVALID_ARG, "n_seq must be >= 0 and S >= 1");
    if (n_seq == 0) return TPQ_OK;
    if (!y) return fail(c, TPQ_ERR_INVALID_ARG, "y is NULL");
    if (stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "row stride %lld < E", (long long)stride);
    if (reinterpret_cast<uintptr_t>(y) & 1u) return fail(c, TPQ_ERR_ALIGN, "y is not 2-byte aligned");
    if (n_seq * S > (int64_t)1 << 40) return fail(c, TPQ_ERR_INVALID_ARG, "calibration set too large");
    int n_split = 1;
    const size_t need = tpq_calib_scratch_bytes(n_seq, S, c->E, c->sm_count, &n_split);
    if (need > c->scratch_bytes) {
        TPQ_CUDA(c, cudaFree(c->scratch));  // waits for work that still uses it
        c->scratch = nullptr;
        c->scratch_bytes = 0;
        cudaError_t e = cudaMalloc(&c->scratch, need);
        if (e != cudaSuccess) return cuda_fail(c, e, "calibration scratch");
        c->scratch_bytes = need;
    }
    float *m = c->t.m + (size_t)shard * c->E, *M = c->t.M + (size_t)shard * c->E;
    cudaError_t e = tpq_launch_calibrate(static_cast<const uint16_t *>(y), n_seq, S, stride, c->E, m, M,
                                         c->counts[shard], c->gamma, c->scratch, n_split,
                                         static_cast<cudaStream_t>(stream), &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "calibration kernels");
    c->counts[shard] += n_seq;
    return TPQ_OK;
}

tpq_status tpq_calibrate_ranges_noalloc(tpq_ctx *c, int shard, const void *y, int64_t n_seq, int64_t S, int64_t stride,
                                        void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (shard < 0 || shard >= c->N) return fail(c, TPQ_ERR_INVALID_ARG, "shard %d out of range [0, %d)", shard, c->N);
    if (n_seq < 0 || S < 1) return fail(c, TPQ_ERR_INVALID_ARG, "n_seq must be >= 0 and S >= 1");
    if (n_seq == 0) return TPQ_OK;
    if (!y) return fail(c, TPQ_ERR_INVALID_ARG, "y is NULL");
    if (stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "row stride %lld < E", (long long)stride);
    if (reinterpret_cast<uintptr_t>(y) & 1u) return fail(c, TPQ_ERR_ALIGN, "y is not 2-byte aligned");
    if (n_seq > 65535) return fail(c, TPQ_ERR_SIZE, "at most 65535 sequences per call");
    const int n_split = tpq_static_scratch_splits(n_seq, S, c->E, c->sm_count);
    if (n_split < 1)
        return fail(c, TPQ_ERR_SIZE,
                    "n_seq * E = %lld exceeds the built-in scratch (%u bytes hold n_seq * E <= %u): "
                    "fold fewer sequences per call",
                    (long long)(n_seq * c->E), (unsigned)TPQ_NOALLOC_SCRATCH_BYTES,
                    (unsigned)(TPQ_NOALLOC_SCRATCH_BYTES / 4));
    void *scratch = nullptr;
    cudaError_t e = tpq_static_scratch_address(c->device, &scratch);  // first call on a device: symbol look-up
    if (e == cudaErrorInvalidDevice)
        return fail(c, TPQ_ERR_BAD_STATE, "the context's device (%d) must be the current CUDA device", c->device);
    if (e != cudaSuccess) return cuda_fail(c, e, "cudaGetSymbolAddress(static scratch)");
    float *m = c->t.m + (size_t)shard * c->E, *M = c->t.M + (size_t)shard * c->E;
    e = tpq_launch_calibrate(static_cast<const uint16_t *>(y), n_seq, S, stride, c->E, m, M, c->counts[shard], c->gamma,
                             scratch, n_split, static_cast<cudaStream_t>(stream), &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "calibration kernels");
    c->counts[shard] += n_seq;
    return TPQ_OK;
}

tpq_status tpq_select_features(tpq_ctx *c, int k, int32_t *hp_out, int *k_out)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (k < 0) k = c->E / 64;  // Section 4: k = floor(E/64)
    if (k > c->E) return fail(c, TPQ_ERR_INVALID_ARG, "k = %d exceeds E = %d", k, c->E);
    if (!all_calibrated(c)) return fail(c, TPQ_ERR_BAD_STATE, "every shard needs at least one calibration sequence");
    tpq_status st = build_tables(c, k, true);
    if (st != TPQ_OK) return st;
    if (hp_out && k > 0) TPQ_CUDA(c, cudaMemcpy(hp_out, c->t.hp_idx, (size_t)k * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (k_out) *k_out = k;
    return TPQ_OK;
}

tpq_status tpq_set_features(tpq_ctx *c, const int32_t *hp, int k)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (k < 0 || k > c->E || (k > 0 && !hp)) return fail(c, TPQ_ERR_INVALID_ARG, "bad feature set size %d", k);
    if (!all_calibrated(c)) return fail(c, TPQ_ERR_BAD_STATE, "every shard needs at least one calibration sequence");
    std::vector<uint8_t> flag((size_t)c->E, 0);
    for (int h = 0; h < k; ++h) {
        if (hp[h] < 0 || hp[h] >= c->E || (h > 0 && hp[h] <= hp[h - 1]))
            return fail(c, TPQ_ERR_INVALID_ARG, "feature indices must be strictly ascending in [0, E)");
        flag[hp[h]] = 1;
    }
    TPQ_CUDA(c, cudaMemcpy(c->t.flag, flag.data(), flag.size(), cudaMemcpyHostToDevice));
    return build_tables(c, k, false);
}

tpq_status tpq_set_ranges(tpq_ctx *c, const float *m, const float *M, const int64_t *counts)
{
    if (!c || !m || !M || !counts) return c ? fail(c, TPQ_ERR_INVALID_ARG, "NULL argument") : TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    for (int i = 0; i < c->N; ++i)
        if (counts[i] < 0) return fail(c, TPQ_ERR_INVALID_ARG, "negative count");
    const size_t bytes = (size_t)c->N * c->E * sizeof(float);
    TPQ_CUDA(c, cudaDeviceSynchronize());
    TPQ_CUDA(c, cudaMemcpy(c->t.m, m, bytes, cudaMemcpyHostToDevice));
    TPQ_CUDA(c, cudaMemcpy(c->t.M, M, bytes, cudaMemcpyHostToDevice));
    for (int i = 0; i < c->N; ++i) c->counts[i] = counts[i];
    c->k = -1;  // steps depend on the ranges: a feature set must be (re)installed
    return TPQ_OK;
}

tpq_status tpq_get_ranges(tpq_ctx *c, float *m, float *M, float *R, float *Rbar)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    const size_t bytes = (size_t)c->N * c->E * sizeof(float);
    TPQ_CUDA(c, cudaDeviceSynchronize());
    if (m) TPQ_CUDA(c, cudaMemcpy(m, c->t.m, bytes, cudaMemcpyDeviceToHost));
    if (M) TPQ_CUDA(c, cudaMemcpy(M, c->t.M, bytes, cudaMemcpyDeviceToHost));
    if ((R || Rbar) && c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "ranges exist once a feature set is installed");
    if (R) TPQ_CUDA(c, cudaMemcpy(R, c->t.R, bytes, cudaMemcpyDeviceToHost));
    if (Rbar) TPQ_CUDA(c, cudaMemcpy(Rbar, c->t.Rbar, (size_t)c->E * sizeof(float), cudaMemcpyDeviceToHost));
    return TPQ_OK;
}

tpq_status tpq_get_scales(tpq_ctx *c, float *s, float *inv_s)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set yet");
    const size_t bytes = (size_t)c->N * c->E * sizeof(float);
    TPQ_CUDA(c, cudaDeviceSynchronize());
    if (s) TPQ_CUDA(c, cudaMemcpy(s, c->t.s, bytes, cudaMemcpyDeviceToHost));
    if (inv_s) TPQ_CUDA(c, cudaMemcpy(inv_s, c->t.inv_s, bytes, cudaMemcpyDeviceToHost));
    return TPQ_OK;
}

int tpq_num_selected(const tpq_ctx *c) { return c ? c->k : -1; }

tpq_status tpq_get_features(tpq_ctx *c, int32_t *hp_out)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set yet");
    if (c->k > 0) {
        if (!hp_out) return fail(c, TPQ_ERR_INVALID_ARG, "NULL output");
        TPQ_CUDA(c, cudaMemcpy(hp_out, c->t.hp_idx, (size_t)c->k * sizeof(int32_t), cudaMemcpyDeviceToHost));
    }
    return TPQ_OK;
}

tpq_status tpq_get_slot_order(tpq_ctx *c, int32_t *slot_out)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set yet");
    if (c->E - c->k > 0) {
        if (!slot_out) return fail(c, TPQ_ERR_INVALID_ARG, "NULL output");
        TPQ_CUDA(c, cudaMemcpy(slot_out, c->t.lp_idx, (size_t)(c->E - c->k) * sizeof(int32_t), cudaMemcpyDeviceToHost));
    }
    return TPQ_OK;
}

size_t tpq_payload_bytes_for(int64_t T, int64_t E, int64_t k)
{
    if (T <= 0 || E <= 0 || k < 0 || k > E) return 0;
    return (size_t)(tpq_lp_bytes_i(T, E, k) + 2 * T * k);
}

size_t tpq_payload_bytes_for_bits(int64_t T, int64_t E, int64_t k, int bits)
{
    if (T <= 0 || E <= 0 || k < 0 || k > E || bits < 2 || bits > 8) return 0;
    return (size_t)(tpq_lp_bytes_i(T, E, k, bits) + 2 * T * k);
}

size_t tpq_payload_bytes(const tpq_ctx *c, int64_t T)
{
    if (!c || c->k < 0) return 0;
    return tpq_payload_bytes_for_bits(T, c->E, c->k, c->bits);
}

tpq_status tpq_comm_bytes(const tpq_ctx *c, int64_t T, tpq_comm_report *out)
{
    if (!c || !out || T < 1) return TPQ_ERR_INVALID_ARG;
    if (c->k < 0) return TPQ_ERR_BAD_STATE;
    const int64_t P = (int64_t)tpq_payload_bytes(c, T);
    const int64_t raw = 2 * T * (int64_t)c->E;
    out->payload_bytes = P;
    out->quantized_allgather_send = (c->N - 1) * P;
    out->bf16_allgather_send = (c->N - 1) * raw;
    out->bf16_ring_allreduce_send = 2 * (int64_t)(c->N - 1) * raw / c->N;
    out->bits_per_value = 8.0 * (double)P / ((double)T * c->E);
    out->bits_per_value_formula = c->bits + (16.0 - c->bits) * c->k / c->E;
    return TPQ_OK;
}

tpq_status tpq_quantize_pack(tpq_ctx *c, int shard, const void *y, int64_t T, int64_t stride, void *payload,
                             size_t cap, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (shard < 0 || shard >= c->N) return fail(c, TPQ_ERR_INVALID_ARG, "shard %d out of range [0, %d)", shard, c->N);
    if (T < 0) return fail(c, TPQ_ERR_INVALID_ARG, "T < 0");
    if (T == 0) return TPQ_OK;
    if (!y || !payload) return fail(c, TPQ_ERR_INVALID_ARG, "NULL buffer");
    if (stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "row stride %lld < E", (long long)stride);
    if (!aligned16(y) || !aligned16(payload)) return fail(c, TPQ_ERR_ALIGN, "y and payload must be 16-byte aligned");
    if (cap < tpq_payload_bytes(c, T))
        return fail(c, TPQ_ERR_SIZE, "payload capacity %zu < %zu", cap, tpq_payload_bytes(c, T));
    const bool groups_ok = tpq_groups_ok(c, T, stride);
    const bool tiled_ok = groups_ok || tpq_quantize_tiled_ok(c, T, stride);
    if (c->kernel_path == 2 && !tiled_ok) return fail(c, TPQ_ERR_INVALID_ARG, "shape does not admit the tiled kernel");
    cudaError_t e;
    if (groups_ok && c->kernel_path != 1)
        e = tpq_launch_quantize_groups(c, shard, 1, &y, T, stride, &payload, static_cast<cudaStream_t>(stream),
                                       &c->launches);
    else if (tiled_ok && c->kernel_path != 1)
        e = tpq_launch_quantize_tiled(c, shard, static_cast<const uint16_t *>(y), T, stride,
                                      static_cast<uint8_t *>(payload), static_cast<cudaStream_t>(stream), &c->launches);
    else
        e = tpq_launch_quantize_generic(c, shard, static_cast<const uint16_t *>(y), T, stride,
                                        static_cast<uint8_t *>(payload), static_cast<cudaStream_t>(stream),
                                        &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "quantize_pack kernel");
    return TPQ_OK;
}

tpq_status tpq_quantize_pack_batch(tpq_ctx *c, int first_shard, int n, const void *const *ys, int64_t T,
                                   int64_t stride, void *const *payloads, size_t cap, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (n < 0 || first_shard < 0 || first_shard + n > c->N)
        return fail(c, TPQ_ERR_INVALID_ARG, "shards [%d, %d) out of range [0, %d)", first_shard, first_shard + n, c->N);
    if (T < 0) return fail(c, TPQ_ERR_INVALID_ARG, "T < 0");
    if (T == 0 || n == 0) return TPQ_OK;
    if (!ys || !payloads) return fail(c, TPQ_ERR_INVALID_ARG, "NULL pointer array");
    if (stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "row stride %lld < E", (long long)stride);
    if (cap < tpq_payload_bytes(c, T))
        return fail(c, TPQ_ERR_SIZE, "payload capacity %zu < %zu", cap, tpq_payload_bytes(c, T));
    for (int b = 0; b < n; ++b) {
        if (!ys[b] || !payloads[b]) return fail(c, TPQ_ERR_INVALID_ARG, "NULL buffer for shard %d", first_shard + b);
        if (!aligned16(ys[b]) || !aligned16(payloads[b]))
            return fail(c, TPQ_ERR_ALIGN, "y and payload of shard %d must be 16-byte aligned", first_shard + b);
    }
    const bool groups_ok = tpq_groups_ok(c, T, stride);
    const bool tiled_ok = groups_ok || tpq_quantize_tiled_ok(c, T, stride);
    if (c->kernel_path == 2 && !tiled_ok) return fail(c, TPQ_ERR_INVALID_ARG, "shape does not admit the tiled kernel");
    cudaError_t e = cudaSuccess;
    if (groups_ok && c->kernel_path != 1) {
        e = tpq_launch_quantize_groups(c, first_shard, n, ys, T, stride, payloads, static_cast<cudaStream_t>(stream),
                                       &c->launches);
    } else if (tiled_ok && c->kernel_path != 1) {
        e = tpq_launch_quantize_tiled_batch(c, first_shard, n, ys, T, stride, payloads, static_cast<cudaStream_t>(stream),
                                            &c->launches);
    } else {
        for (int b = 0; b < n && e == cudaSuccess; ++b)
            e = tpq_launch_quantize_generic(c, first_shard + b, static_cast<const uint16_t *>(ys[b]), T, stride,
                                            static_cast<uint8_t *>(payloads[b]), static_cast<cudaStream_t>(stream),
                                            &c->launches);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "quantize_pack kernel");
    return TPQ_OK;
}

// Section 5 (system level: all-gather, then a local reduction): the exchange fused into the quantiser.
tpq_status tpq_quantize_pack_push(tpq_ctx *c, int shard, const void *y, int64_t T, int64_t stride, void *const *dst,
                                  uint32_t *const *arrived, int n_dst, size_t cap, uint32_t epoch, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (shard < 0 || shard >= c->N) return fail(c, TPQ_ERR_INVALID_ARG, "shard %d out of range [0, %d)", shard, c->N);
    if (n_dst < 1 || n_dst > tpq_push_max_dst())
        return fail(c, TPQ_ERR_INVALID_ARG, "n_dst %d out of range [1, %d]", n_dst, tpq_push_max_dst());
    if (T < 1) return fail(c, TPQ_ERR_INVALID_ARG, "T < 1 (an empty step has nothing to publish)");
    if (!y || !dst || !arrived) return fail(c, TPQ_ERR_INVALID_ARG, "NULL pointer");
    if (stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "row stride %lld < E", (long long)stride);
    if (!aligned16(y)) return fail(c, TPQ_ERR_ALIGN, "y must be 16-byte aligned");
    if (cap < tpq_payload_bytes(c, T))
        return fail(c, TPQ_ERR_SIZE, "destination capacity %zu < %zu", cap, tpq_payload_bytes(c, T));
    for (int d = 0; d < n_dst; ++d) {
        if (!dst[d] || !arrived[d]) return fail(c, TPQ_ERR_INVALID_ARG, "NULL destination %d", d);
        if (!aligned16(dst[d])) return fail(c, TPQ_ERR_ALIGN, "destination %d must be 16-byte aligned", d);
        if (reinterpret_cast<uintptr_t>(arrived[d]) & 3u)
            return fail(c, TPQ_ERR_ALIGN, "arrival word %d must be 4-byte aligned", d);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (c->kernel_path != 1 && tpq_quantize_tiled_ok(c, T, stride)) {
        e = tpq_launch_quantize_tiled_push(c, shard, static_cast<const uint16_t *>(y), T, stride, dst, arrived, n_dst, epoch,
                                           st, &c->launches);
        if (e != cudaSuccess) return cuda_fail(c, e, "quantize_pack_push kernel");
        return TPQ_OK;
    }
    // other shapes and code widths: quantise into the first destination, copy it to the others in stream
    // order, then publish the arrival words
    void *first = dst[0];
    if (tpq_groups_ok(c, T, stride) && c->kernel_path != 1)
        e = tpq_launch_quantize_groups(c, shard, 1, &y, T, stride, &first, st, &c->launches);
    else
        e = tpq_launch_quantize_generic(c, shard, static_cast<const uint16_t *>(y), T, stride,
                                        static_cast<uint8_t *>(first), st, &c->launches);
    const size_t bytes = tpq_payload_bytes(c, T);
    for (int d = 1; d < n_dst && e == cudaSuccess; ++d)
        if (dst[d] != first) e = cudaMemcpyAsync(dst[d], first, bytes, cudaMemcpyDefault, st);
    if (e == cudaSuccess) e = tpq_launch_publish_arrivals(arrived, n_dst, epoch, st, &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "quantize_pack_push (copy path)");
    return TPQ_OK;
}

tpq_status tpq_wait_arrivals(tpq_ctx *c, const uint32_t *arrived, int n, uint32_t epoch, uint64_t timeout_ns, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (!arrived || n < 1 || n > 1024) return fail(c, TPQ_ERR_INVALID_ARG, "arrival words: NULL or n = %d outside [1, 1024]", n);
    if (reinterpret_cast<uintptr_t>(arrived) & 3u) return fail(c, TPQ_ERR_ALIGN, "arrival words must be 4-byte aligned");
    if (timeout_ns == 0) timeout_ns = 1000000000ull;  // one second
    if (timeout_ns > 5000000000ull) return fail(c, TPQ_ERR_INVALID_ARG, "timeout above 5 s");
    cudaError_t e = tpq_launch_wait_arrivals(c, arrived, n, epoch, timeout_ns, static_cast<cudaStream_t>(stream), &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "wait_arrivals kernel");
    return TPQ_OK;
}

// Section 2: the layer ahead of the synchronisation point, f^(i)(x^(i)) = x^(i) W^(i), fused with C^(i).
tpq_status tpq_permute_weight(tpq_ctx *c, const void *w, int64_t K, void *w_slots, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (!w || !w_slots || w == w_slots) return fail(c, TPQ_ERR_INVALID_ARG, "NULL or aliased weight buffers");
    if (K < 1) return fail(c, TPQ_ERR_INVALID_ARG, "K < 1");
    if (!aligned16(w) || !aligned16(w_slots)) return fail(c, TPQ_ERR_ALIGN, "weight buffers must be 16-byte aligned");
    cudaError_t e = tpq_launch_permute_weight(c, w, w_slots, K, static_cast<cudaStream_t>(stream), &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "permute_weight kernel");
    return TPQ_OK;
}

tpq_status tpq_linear_quantize_pack(tpq_ctx *c, int shard, const void *x, const void *w_slots, int64_t T, int64_t K,
                                    void *payload, size_t cap, void *y_slots, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (shard < 0 || shard >= c->N) return fail(c, TPQ_ERR_INVALID_ARG, "shard %d out of range [0, %d)", shard, c->N);
    if (T < 0) return fail(c, TPQ_ERR_INVALID_ARG, "T < 0");
    if (T == 0) return TPQ_OK;
    if (!x || !w_slots || !payload) return fail(c, TPQ_ERR_INVALID_ARG, "NULL buffer");
    if (!aligned16(x) || !aligned16(w_slots) || !aligned16(payload) || (y_slots && !aligned16(y_slots)))
        return fail(c, TPQ_ERR_ALIGN, "x, w_slots, payload and y_slots must be 16-byte aligned");
    if (!tpq_linear_ok(c, T, K))
        return fail(c, TPQ_ERR_INVALID_ARG,
                    "the fused layer needs 4-bit codes, E and k multiples of 8 and K a multiple of 8 (K = %lld)", (long long)K);
    if (cap < tpq_payload_bytes(c, T))
        return fail(c, TPQ_ERR_SIZE, "payload capacity %zu < %zu", cap, tpq_payload_bytes(c, T));
    cudaError_t e = tpq_launch_linear_quantize(c, shard, x, w_slots, T, K, payload, y_slots, static_cast<cudaStream_t>(stream),
                                               &c->launches);
    if (e != cudaSuccess) return cuda_fail(c, e, "linear_quantize kernel");
    return TPQ_OK;
}

static tpq_status dequant_reduce_impl(tpq_ctx *c, const void *const *payloads, int n_payloads, int64_t T, void *out,
                                      tpq_out_dtype dt, int64_t out_stride, void *stream);

tpq_status tpq_dequant_reduce(tpq_ctx *c, const void *const *payloads, int n_payloads, int64_t T, void *out,
                              tpq_out_dtype dt, int64_t out_stride, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->call_bias = nullptr;
    c->call_arr = tpq_arrivals{};
    return dequant_reduce_impl(c, payloads, n_payloads, T, out, dt, out_stride, stream);
}

tpq_status tpq_dequant_reduce_bias(tpq_ctx *c, const void *const *payloads, int n_payloads, int64_t T, void *out,
                                   tpq_out_dtype dt, int64_t out_stride, const float *bias, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (!bias) return fail(c, TPQ_ERR_INVALID_ARG, "bias is NULL (use tpq_dequant_reduce)");
    if (!aligned16(bias)) return fail(c, TPQ_ERR_ALIGN, "bias must be 16-byte aligned");
    c->call_bias = bias;
    c->call_arr = tpq_arrivals{};
    const tpq_status st = dequant_reduce_impl(c, payloads, n_payloads, T, out, dt, out_stride, stream);
    c->call_bias = nullptr;
    return st;
}

tpq_status tpq_dequant_reduce_arrivals(tpq_ctx *c, const void *const *payloads, int n_payloads, int64_t T, void *out,
                                       tpq_out_dtype dt, int64_t out_stride, const float *bias, const uint32_t *arrived,
                                       uint32_t epoch, uint64_t timeout_ns, void *stream)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (bias && !aligned16(bias)) return fail(c, TPQ_ERR_ALIGN, "bias must be 16-byte aligned");
    if (!arrived) return fail(c, TPQ_ERR_INVALID_ARG, "arrival words are NULL (use tpq_dequant_reduce)");
    if (reinterpret_cast<uintptr_t>(arrived) & 3u) return fail(c, TPQ_ERR_ALIGN, "arrival words must be 4-byte aligned");
    if (timeout_ns == 0) timeout_ns = 1000000000ull;  // one second
    if (timeout_ns > 5000000000ull) return fail(c, TPQ_ERR_INVALID_ARG, "timeout above 5 s");
    c->call_bias = bias;
    c->call_arr = tpq_arrivals{arrived, epoch, c->N, timeout_ns, c->t.status};
    const tpq_status st = dequant_reduce_impl(c, payloads, n_payloads, T, out, dt, out_stride, stream);
    c->call_bias = nullptr;
    c->call_arr = tpq_arrivals{};
    return st;
}

static tpq_status dequant_reduce_impl(tpq_ctx *c, const void *const *payloads, int n_payloads, int64_t T, void *out,
                                      tpq_out_dtype dt, int64_t out_stride, void *stream)
{
    c->err[0] = 0;
    if (c->k < 0) return fail(c, TPQ_ERR_BAD_STATE, "no feature set: call tpq_select_features or tpq_set_features");
    if (n_payloads != c->N) return fail(c, TPQ_ERR_INVALID_ARG, "n_payloads = %d, expected N = %d", n_payloads, c->N);
    if (dt != TPQ_OUT_BF16 && dt != TPQ_OUT_FP32) return fail(c, TPQ_ERR_INVALID_ARG, "unknown output type");
    if (T < 0) return fail(c, TPQ_ERR_INVALID_ARG, "T < 0");
    if (T == 0) return TPQ_OK;
    if (!payloads || !out) return fail(c, TPQ_ERR_INVALID_ARG, "NULL buffer");
    if (out_stride < c->E) return fail(c, TPQ_ERR_INVALID_ARG, "output row stride %lld < E", (long long)out_stride);
    for (int i = 0; i < c->N; ++i) {
        if (!payloads[i]) return fail(c, TPQ_ERR_INVALID_ARG, "payload %d is NULL", i);
        if (!aligned16(payloads[i])) return fail(c, TPQ_ERR_ALIGN, "payload %d is not 16-byte aligned", i);
    }
    if (!aligned16(out)) return fail(c, TPQ_ERR_ALIGN, "out must be 16-byte aligned");
    const int fp32 = dt == TPQ_OUT_FP32;
    const bool groups_ok = tpq_groups_ok(c, T, out_stride);
    const bool tiled_ok = groups_ok || tpq_dequant_tiled_ok(c, T, out_stride, fp32);
    if (c->kernel_path == 2 && !tiled_ok) return fail(c, TPQ_ERR_INVALID_ARG, "shape does not admit the tiled kernel");
    cudaError_t e;
    if (groups_ok && c->kernel_path != 1)
        e = tpq_launch_dequant_groups(c, payloads, T, out, fp32, out_stride, static_cast<cudaStream_t>(stream),
                                      &c->launches);
    else if (tiled_ok && c->kernel_path != 1)
        e = tpq_launch_dequant_tiled(c, payloads, T, out, fp32, out_stride, static_cast<cudaStream_t>(stream),
                                     &c->launches);
    else
        e = tpq_launch_dequant_generic(c, payloads, T, out, fp32, out_stride, static_cast<cudaStream_t>(stream),
                                       &c->launches);
    if (e == cudaErrorInvalidValue && c->dq_kernel != 0)
        return fail(c, TPQ_ERR_INVALID_ARG, "shape does not admit dequant kernel %d", c->dq_kernel);
    if (e != cudaSuccess) return cuda_fail(c, e, "dequant_reduce kernel");
    return TPQ_OK;
}

tpq_status tpq_get_state(tpq_ctx *c, void *blob, size_t *bytes)
{
    if (!c || !bytes) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    const size_t NE = (size_t)c->N * c->E;
    const int k = c->k < 0 ? 0 : c->k;
    const size_t need = sizeof(StateHeader) + (size_t)c->N * 8 + 2 * NE * 4 + (size_t)k * 4;
    if (!blob) {
        *bytes = need;
        return TPQ_OK;
    }
    if (*bytes < need) return fail(c, TPQ_ERR_SIZE, "state needs %zu bytes", need);
    uint8_t *p = static_cast<uint8_t *>(blob);
    StateHeader h;
    memset(&h, 0, sizeof h);
    memcpy(h.magic, "TPQSTAT1", 8);
    h.version = 1; h.N = c->N; h.E = c->E; h.bits = c->bits; h.gamma = c->gamma; h.k = c->k;
    memcpy(p, &h, sizeof h);
    p += sizeof h;
    memcpy(p, c->counts, (size_t)c->N * 8);
    p += (size_t)c->N * 8;
    TPQ_CUDA(c, cudaDeviceSynchronize());
    TPQ_CUDA(c, cudaMemcpy(p, c->t.m, NE * 4, cudaMemcpyDeviceToHost));
    p += NE * 4;
    TPQ_CUDA(c, cudaMemcpy(p, c->t.M, NE * 4, cudaMemcpyDeviceToHost));
    p += NE * 4;
    if (k) TPQ_CUDA(c, cudaMemcpy(p, c->t.hp_idx, (size_t)k * 4, cudaMemcpyDeviceToHost));
    *bytes = need;
    return TPQ_OK;
}

tpq_status tpq_set_state(tpq_ctx *c, const void *blob, size_t bytes)
{
    if (!c || !blob) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    if (bytes < sizeof(StateHeader)) return fail(c, TPQ_ERR_SIZE, "state blob truncated");
    StateHeader h;
    memcpy(&h, blob, sizeof h);
    if (memcmp(h.magic, "TPQSTAT1", 8) != 0 || h.version != 1) return fail(c, TPQ_ERR_INVALID_ARG, "not a tpq state blob");
    if (h.N != c->N || h.E != c->E || h.bits != c->bits)
        return fail(c, TPQ_ERR_INVALID_ARG, "state is for N=%d E=%d bits=%d", h.N, h.E, h.bits);
    if (h.k < -1 || h.k > c->E) return fail(c, TPQ_ERR_INVALID_ARG, "corrupt state (k)");
    const size_t NE = (size_t)c->N * c->E;
    const int k = h.k < 0 ? 0 : h.k;
    const size_t need = sizeof(StateHeader) + (size_t)c->N * 8 + 2 * NE * 4 + (size_t)k * 4;
    if (bytes < need) return fail(c, TPQ_ERR_SIZE, "state blob truncated");
    const uint8_t *p = static_cast<const uint8_t *>(blob) + sizeof h;
    std::vector<int64_t> counts((size_t)c->N);
    memcpy(counts.data(), p, (size_t)c->N * 8);
    p += (size_t)c->N * 8;
    const float *m = reinterpret_cast<const float *>(p);
    const float *M = m + NE;
    std::vector<float> mm(m, m + NE), MM(M, M + NE);  // aligned copies
    tpq_status st = tpq_set_ranges(c, mm.data(), MM.data(), counts.data());
    if (st != TPQ_OK) return st;
    c->gamma = h.gamma;
    if (h.k >= 0) {
        std::vector<int32_t> hp((size_t)k);
        if (k) memcpy(hp.data(), p + 2 * NE * 4, (size_t)k * 4);
        return tpq_set_features(c, hp.data(), k);
    }
    return TPQ_OK;
}

tpq_status tpq_device_status(tpq_ctx *c)
{
    if (!c) return TPQ_ERR_INVALID_ARG;
    c->err[0] = 0;
    int word = 0;
    TPQ_CUDA(c, cudaDeviceSynchronize());
    TPQ_CUDA(c, cudaMemcpy(&word, c->t.status, sizeof word, cudaMemcpyDeviceToHost));
    if (word != 0) {
        TPQ_CUDA(c, cudaMemset(c->t.status, 0, sizeof word));
        return fail(c, (tpq_status)word, "a kernel reported status %d", word);
    }
    return TPQ_OK;
}

int64_t tpq_launch_count(const tpq_ctx *c) { return c ? c->launches : 0; }

}  // extern "C"

// C^(i): quantise one device's BF16 partial sums to static symmetric Int4 and pack
// them, selected features passed through in BF16 (paper Section 3, Figure 2).
//
// Per low-precision element: u = fl(x * inv_s); u clamped to [-8, 7]; code = rne(u).
// The two roundings are kept separate (__fmul_rn, then the magic-constant add).
#include "tpq_internal.h"

namespace {

// ----------------------------------------------------------------------------------------------
// Shape-generic kernel: one thread per 32-bit word of the code stream (8 codes), any E, k, stride.
// ----------------------------------------------------------------------------------------------
__device__ __forceinline__ int quant_one(uint16_t x, float inv_s)
{
    float u = __fmul_rn(__uint_as_float((uint32_t)x << 16), inv_s);
    u = fminf(fmaxf(u, -8.0f), 7.0f);
    return __float2int_rn(u);
}

__global__ void __launch_bounds__(256) quantize_generic(const uint16_t *__restrict__ y, int64_t T, int64_t stride, int E,
                                                        int k, const float *__restrict__ inv_s,
                                                        const int32_t *__restrict__ lp_idx,
                                                        const int32_t *__restrict__ hp_idx,
                                                        uint32_t *__restrict__ lp_out, int64_t lp_words,
                                                        uint16_t *__restrict__ hp_out)
{
    const int64_t L = E - k;
    const int64_t n_nib = T * L;
    const int64_t hp_elems = T * k;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t gsz = (int64_t)gridDim.x * blockDim.x;
    for (int64_t w = gid; w < lp_words; w += gsz) {
        uint32_t word = 0;
        int64_t p = 8 * w;
        if (p < n_nib) {
            int64_t t = p / L;
            int64_t c = p - t * L;
#pragma unroll 1
            for (int n = 0; n < 8 && p < n_nib; ++n, ++p) {
                const int j = lp_idx[c];
                const int q = quant_one(y[t * stride + j], inv_s[j]);
                word |= (uint32_t)(q & 0xF) << (4 * n);
                if (++c == L) {
                    c = 0;
                    ++t;
                }
            }
        }
        lp_out[w] = word;
    }
    for (int64_t a = gid; a < hp_elems; a += gsz) {
        const int64_t t = a / k;
        const int h = (int)(a - t * k);
        hp_out[a] = y[t * stride + hp_idx[h]];
    }
}

// ----------------------------------------------------------------------------------------------
// Tiled kernel for E, k and stride multiples of 8.
//
// One persistent block per SM.  Rows reach shared memory through 1-D bulk asynchronous copies
// (cp.async.bulk, completion on an mbarrier) into a ring of stages of G rows each, so the
// whole share of a block can be in flight while it computes.  Thread <-> 8 adjacent features:
// the reciprocal steps stay in registers for the life of the block.
//   phase 1: 128-bit shared load of 8 BF16 -> 8 codes in feature order -> one word of a
//            shared "code row"; selected features' BF16 patterns go to a shared side buffer
//   phase 2: the selected features are squeezed out of the code row: output word w of a row
//            is an unaligned 32-bit window of the code row (one funnel shift) unless a
//            selected feature falls inside it (then code by code); coalesced 32-bit stores.
// ----------------------------------------------------------------------------------------------
constexpr int QP_MAX_GPT = 4;          // groups of 8 features per thread
constexpr int QP_WAIT_LIMIT = 1 << 22; // bounded mbarrier polling

struct QPParams {
    const uint16_t *y;
    int64_t stride;
    int64_t T;
    int E, k;
    int G;        // rows per stage
    int nstage;
    int64_t ngroups;
    const float *inv_s;    // this device's [E]
    const uint32_t *grp;   // [E/8]
    const int32_t *lp_idx; // [E-k]
    const int32_t *hp_idx; // [k]
    uint32_t *lp_out;
    int64_t lp_words;      // words of the code section, padding included
    uint32_t *hp_out;      // as 32-bit words (k even)
    int *status;
#ifdef TPQ_TRACE
    long long *trace;
#endif
};

// Dynamic shared memory layout (byte offsets, every section 16-byte aligned).
struct QPLayout {
    size_t ring, nib, hpb, bars, total;
};
__host__ __device__ inline QPLayout qp_layout(int E, int k, int G, int nstage)
{
    QPLayout l;
    l.ring = 0;
    l.nib = (size_t)nstage * G * E * 2;
    l.hpb = l.nib + (((size_t)2 * G * (E / 8 + 2) * 4 + 15) & ~(size_t)15);
    l.bars = l.hpb + (((size_t)2 * G * k * 2 + 15) & ~(size_t)15);
    l.total = l.bars + (size_t)nstage * 8;
    return l;
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait: false if the phase never completed
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (int i = 0; i < QP_WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> this block's shared memory, bytes a multiple of 16, both addresses 16-byte aligned
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// 8 BF16 (one uint4) -> 8 two's-complement nibbles in feature order.
// code + 0x4B400000 sits in the bits of fl(u + 1.5*2^23); shifted copies are summed with one
// shift-add each and the constant parts are removed at the end (offset-binary -> two's complement).
// Products and magic adds run two at a time (f32x2); each is still one binary32 rounding per element.
__device__ __forceinline__ uint32_t quant8(const uint4 v, const float2 (&inv)[4])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t acc = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 u = __fmul2_rn(make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u)), inv[i]);
        u.x = fminf(fmaxf(u.x, -8.0f), 7.0f);
        u.y = fminf(fmaxf(u.y, -8.0f), 7.0f);
        const float2 r = __fadd2_rn(u, make_float2(12582912.0f, 12582912.0f));
        acc += __float_as_uint(r.x) << (8 * i);
        acc += __float_as_uint(r.y) << (8 * i + 4);
    }
    // sum_n (0x4B400000 << 4n) mod 2^32
    constexpr uint32_t K0 = 0x4B400000u + (0x4B400000u << 4) + (0x4B400000u << 8) + (0x4B400000u << 12) +
                            (0x4B400000u << 16) + (0x4B400000u << 20) + (0x4B400000u << 24) + (0x4B400000u << 28);
    return (acc - K0 + 0x88888888u) ^ 0x88888888u;
}

#ifdef TPQ_TRACE
static long long *g_trace = nullptr;  // 64 slots per block, globaltimer ns
__device__ __forceinline__ long long tpq_now()
{
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define TPQ_MARK(slot) do { if (threadIdx.x == 0 && p.trace && (slot) < 64) p.trace[blockIdx.x * 64 + (slot)] = tpq_now(); } while (0)
#else
#define TPQ_MARK(slot) do { } while (0)
#endif

template <int GPT>
__global__ void __launch_bounds__(1024, 1) quantize_tiled(const QPParams p)
{
    TPQ_MARK(0);
    extern __shared__ __align__(128) uint8_t smem[];
    const int tid = threadIdx.x, NT = blockDim.x;
    const int E = p.E, k = p.k, G = p.G, nstage = p.nstage;
    const int E8 = E >> 3, L8 = (E - k) >> 3;
    const int nib_stride = E8 + 2;
    const uint32_t row_bytes = (uint32_t)E * 2u;
    const uint32_t stage_bytes = (uint32_t)G * row_bytes;

    const QPLayout lay = qp_layout(E, k, G, nstage);
    uint8_t *ring = smem + lay.ring;
    uint32_t *nib = reinterpret_cast<uint32_t *>(smem + lay.nib);
    uint16_t *hpb = reinterpret_cast<uint16_t *>(smem + lay.hpb);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + lay.bars);
    __shared__ int abort_flag;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < nstage; ++s) mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    TPQ_MARK(40);

    auto issue = [&](int it, int st) {  // group blockIdx.x + it*gridDim.x into stage st
        const int64_t gi = blockIdx.x + it * (int64_t)gridDim.x;
        if (gi >= p.ngroups) return;
        const int64_t t0 = gi * G;
        const int rows = (int)((p.T - t0 < G) ? p.T - t0 : G);
        const uint32_t bar = smem_u32(&bars[st]);
        const uint32_t dst = smem_u32(ring + (size_t)st * stage_bytes);
        mbar_expect_tx(bar, rows * row_bytes);
        if (p.stride == E) {
            bulk_g2s(dst, p.y + t0 * p.stride, rows * row_bytes, bar);
        } else {
            for (int r = 0; r < rows; ++r) bulk_g2s(dst + r * row_bytes, p.y + (t0 + r) * p.stride, row_bytes, bar);
        }
    };
    if (tid == 0)
        for (int it = 0; it < nstage; ++it) issue(it, it);
    TPQ_MARK(41);

    // ---- per-thread constants (their loads overlap the first copies)
    // phase 1: the reciprocal steps of the thread's 8 features, as four pairs
    float2 inv[GPT][4];
    // selected features: thread h < k copies feature my_hp of every row to the BF16 side buffer
    const int my_hp = (tid < k) ? __ldg(p.hp_idx + tid) : 0;
    // phase 2: output word wc = tid + a*NT of a row holds the 8 codes whose source features are
    // lp_idx[8wc .. 8wc+7].  With d = number of selected features skipped so far (0, 1 or 2 inside one
    // word in all but pathological sets), code c sits at source nibble src0 + c + d: the word is
    // (W0 & ~(m1|m2)) | (W1 & m1) | (W2 & m2), Wd = the 32-bit window of the code row at nibble src0 + d.
    int w0[GPT], sh[GPT];
    uint32_t m1[GPT], m2[GPT];
    int mode[GPT];  // 0: no word, 1: windows, 2: more than two skipped features, code by code
#pragma unroll
    for (int a = 0; a < GPT; ++a) {
        const int g = tid + a * NT;
#pragma unroll
        for (int i = 0; i < 4; ++i) inv[a][i] = make_float2(0.0f, 0.0f);
        if (g < E8) {
            const float4 i0 = __ldg(reinterpret_cast<const float4 *>(p.inv_s + 8 * g));
            const float4 i1 = __ldg(reinterpret_cast<const float4 *>(p.inv_s + 8 * g + 4));
            inv[a][0] = make_float2(i0.x, i0.y);
            inv[a][1] = make_float2(i0.z, i0.w);
            inv[a][2] = make_float2(i1.x, i1.y);
            inv[a][3] = make_float2(i1.z, i1.w);
        }
        w0[a] = 0; sh[a] = 0; m1[a] = 0; m2[a] = 0; mode[a] = 0;
        if (g < L8) {
            const int4 l0 = __ldg(reinterpret_cast<const int4 *>(p.lp_idx + 8 * g));
            const int4 l1 = __ldg(reinterpret_cast<const int4 *>(p.lp_idx + 8 * g + 4));
            const int idx[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
            w0[a] = idx[0] >> 3;
            sh[a] = (idx[0] & 7) * 4;
            mode[a] = (idx[7] - idx[0] - 7 <= 2) ? 1 : 2;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int d = idx[c] - idx[0] - c;
                if (d == 1) m1[a] |= 0xFu << (4 * c);
                if (d == 2) m2[a] |= 0xFu << (4 * c);
            }
        }
    }

    TPQ_MARK(1);
    int it = 0, st = 0;       // iteration, its ring stage (it mod nstage, kept without dividing)
    uint32_t parity = 0;      // (it / nstage) & 1
    for (;; ++it) {
        const int64_t gi = blockIdx.x + it * (int64_t)gridDim.x;
        if (gi >= p.ngroups) break;
        const int64_t t0 = gi * G;
        const int rows = (int)((p.T - t0 < G) ? p.T - t0 : G);
        const int buf = it & 1;
        if (!mbar_wait(smem_u32(&bars[st]), parity)) abort_flag = 1;
        TPQ_MARK(2 + 3 * (int)it);

        // ---- phase 1: quantise in feature order; copy the selected features
        const uint4 *stage = reinterpret_cast<const uint4 *>(ring + (size_t)st * stage_bytes);
        uint32_t *nrow = nib + (size_t)buf * G * nib_stride;
        uint16_t *hrow = hpb + (size_t)buf * G * k;
#pragma unroll
        for (int a = 0; a < GPT; ++a) {
            const int g = tid + a * NT;
            if (g < E8)
                for (int r = 0; r < rows; ++r) nrow[r * nib_stride + g] = quant8(stage[r * E8 + g], inv[a]);
        }
        {
            const uint16_t *stage16 = reinterpret_cast<const uint16_t *>(stage);
            for (int h = tid; h < k; h += NT) {
                const int j = (h == tid) ? my_hp : __ldg(p.hp_idx + h);
                for (int r = 0; r < rows; ++r) hrow[r * k + h] = stage16[r * E + j];
            }
        }
        __syncthreads();
        TPQ_MARK(3 + 3 * (int)it);
        if (abort_flag) break;
        if (tid == 0) issue(it + nstage, st);  // the stage is free again

        // ---- phase 2: squeeze out the selected features, store
#pragma unroll
        for (int a = 0; a < GPT; ++a) {
            const int wc = tid + a * NT;
            if (mode[a] != 0) {
                for (int r = 0; r < rows; ++r) {
                    const uint32_t *src = nrow + r * nib_stride + w0[a];
                    uint32_t word;
                    if (mode[a] == 1) {
                        const uint32_t x0 = src[0], x1 = src[1];
                        const uint32_t W0 = __funnelshift_r(x0, x1, sh[a]);
                        const uint32_t W1 = __funnelshift_rc(x0, x1, sh[a] + 4);
                        word = (W0 & ~(m1[a] | m2[a])) | (W1 & m1[a]);
                        if (m2[a]) {
                            const uint32_t W2 = (sh[a] == 28) ? __funnelshift_r(x1, src[2], 4)
                                                              : __funnelshift_rc(x0, x1, sh[a] + 8);
                            word |= W2 & m2[a];
                        }
                    } else {
                        word = 0;
#pragma unroll 1
                        for (int n = 0; n < 8; ++n) {
                            const int j = __ldg(p.lp_idx + 8 * wc + n);
                            word |= ((nrow[r * nib_stride + (j >> 3)] >> ((j & 7) * 4)) & 0xFu) << (4 * n);
                        }
                    }
                    p.lp_out[(t0 + r) * L8 + wc] = word;
                }
            }
        }
        {
            const uint32_t *h32 = reinterpret_cast<const uint32_t *>(hrow);
            const int n32 = rows * k / 2;
            uint32_t *dst = p.hp_out + t0 * (k / 2);
            for (int a = tid; a < n32; a += NT) dst[a] = h32[a];
        }
        TPQ_MARK(4 + 3 * (int)it);
        if (++st == nstage) {
            st = 0;
            parity ^= 1u;
        }
    }

    if (abort_flag) {
        // a copy never completed: report, give the copies still in flight a bounded chance to land, leave
        if (tid == 0) {
            atomicExch(p.status, (int)TPQ_ERR_TIMEOUT);
            for (int j = it + 1; j < it + nstage; ++j) {
                if (blockIdx.x + j * (int64_t)gridDim.x >= p.ngroups) break;
                mbar_wait(smem_u32(&bars[j % nstage]), (uint32_t)((j / nstage) & 1));
            }
        }
        return;
    }
    // zero padding of the code section (at most 3 words), by the block that owned the last rows
    if ((p.ngroups - 1) % gridDim.x == blockIdx.x) {
        const int64_t valid = p.T * L8;
        for (int64_t w = valid + tid; w < p.lp_words; w += NT) p.lp_out[w] = 0u;
    }
}

size_t qp_smem_bytes(int E, int k, int G, int nstage) { return qp_layout(E, k, G, nstage).total; }

}  // namespace

bool tpq_quantize_tiled_ok(const tpq_ctx *c, int64_t T, int64_t stride)
{
    const int E = c->E, k = c->k;
    if (E % 8 || k % 8 || stride % 8 || T <= 0) return false;
    if (E - k < 8) return false;                       // nothing (or too little) to squeeze
    if (E / 8 > 1024 * QP_MAX_GPT) return false;
    if (qp_smem_bytes(E, k, 1, 2) > (size_t)c->smem_optin) return false;
    return true;
}

cudaError_t tpq_launch_quantize_generic(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                        uint8_t *payload, cudaStream_t st, int64_t *launches)
{
    const int E = c->E, k = c->k;
    const int64_t lpb = tpq_lp_bytes_i(T, E, k);
    const int64_t lp_words = lpb / 4;
    int64_t work = lp_words > T * k ? lp_words : T * (int64_t)k;
    int64_t blocks = (work + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (blocks < 1) blocks = 1;
    quantize_generic<<<(unsigned)blocks, 256, 0, st>>>(y, T, stride, E, k, c->t.inv_s + (size_t)shard * E, c->t.lp_idx,
                                                       c->t.hp_idx, reinterpret_cast<uint32_t *>(payload), lp_words,
                                                       reinterpret_cast<uint16_t *>(payload + lpb));
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_quantize_tiled(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                      uint8_t *payload, cudaStream_t st, int64_t *launches)
{
    const int E = c->E, k = c->k;
    const int E8 = E / 8;
    const int gpt = (E8 + 1023) / 1024;
    int nt = ((E8 + gpt - 1) / gpt + 31) / 32 * 32;
    // rows per stage: small enough that every SM gets work, large enough to amortise the barrier
    int G = 2;
    if ((T + G - 1) / G < c->sm_count) G = 1;
    while (G > 1 && qp_smem_bytes(E, k, G, 2) > (size_t)c->smem_optin) G >>= 1;
    const int64_t ngroups = (T + G - 1) / G;
    int64_t grid = ngroups < c->sm_count ? ngroups : c->sm_count;
    int64_t per_block = (ngroups + grid - 1) / grid;
    int nstage = (int)(per_block < 8 ? per_block : 8);
    if (nstage < 1) nstage = 1;
    while (nstage > 1 && qp_smem_bytes(E, k, G, nstage) > (size_t)c->smem_optin) --nstage;

    QPParams p;
    const int64_t lpb = tpq_lp_bytes_i(T, E, k);
    p.y = y; p.stride = stride; p.T = T; p.E = E; p.k = k; p.G = G; p.nstage = nstage; p.ngroups = ngroups;
    p.inv_s = c->t.inv_s + (size_t)shard * E; p.grp = c->t.grp; p.lp_idx = c->t.lp_idx; p.hp_idx = c->t.hp_idx;
    p.lp_out = reinterpret_cast<uint32_t *>(payload); p.lp_words = lpb / 4;
    p.hp_out = reinterpret_cast<uint32_t *>(payload + lpb); p.status = c->t.status;
#ifdef TPQ_TRACE
    p.trace = g_trace;
#endif
    const size_t smem = qp_smem_bytes(E, k, G, nstage);

    cudaError_t e = cudaSuccess;
#define TPQ_QP_LAUNCH(GPT)                                                                                       \
    do {                                                                                                         \
        e = cudaFuncSetAttribute(quantize_tiled<GPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);   \
        if (e == cudaSuccess) quantize_tiled<GPT><<<(unsigned)grid, nt, smem, st>>>(p);                          \
    } while (0)
    switch (gpt) {
        case 1: TPQ_QP_LAUNCH(1); break;
        case 2: TPQ_QP_LAUNCH(2); break;
        case 3: TPQ_QP_LAUNCH(3); break;
        default: TPQ_QP_LAUNCH(4); break;
    }
#undef TPQ_QP_LAUNCH
    if (e != cudaSuccess) return e;
    ++*launches;
    return cudaGetLastError();
}

// sum_i D^(i): dequantise the N devices' payloads and sum them into the synchronised
// output, features back in their original order (paper Figure 2 caption; Section 5,
// all-gather followed by a local reduction).
//
// Accumulation is binary32, devices in ascending order: acc = fma(code_i, s_i, acc) for a
// low-precision feature, acc = fl(acc + y_i) for a selected one; one final rounding for BF16.
#include <cuda_bf16.h>

#include "tpq_internal.h"

namespace {

struct DQParams {
    const uint8_t *pl[TPQ_MAX_SHARDS];  // payloads, device order
    int N, E, k;
    int64_t T;
    int64_t lp_bytes;      // code section size (HP block starts here)
    const float *s_k;      // [N][E], 0 at selected features
    const int32_t *pos;    // [E]
    const uint32_t *grp;   // [E/8]
    void *out;
    int64_t out_stride;
};

// ----------------------------------------------------------------------------------------------
// Shape-generic kernel: one thread per output element.
// ----------------------------------------------------------------------------------------------
template <bool FP32OUT>
__global__ void __launch_bounds__(256) dequant_generic(const DQParams p)
{
    const int64_t total = p.T * (int64_t)p.E;
    const int64_t L = p.E - p.k;
    for (int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; a < total; a += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = a / p.E;
        const int j = (int)(a - t * p.E);
        const int ps = p.pos[j];
        float acc = 0.0f;
        if (ps >= 0) {
            const int64_t q = t * L + ps;
            for (int i = 0; i < p.N; ++i) {
                const uint32_t b = p.pl[i][q >> 1];
                const int nib = (q & 1) ? (b >> 4) : (b & 0xF);
                const int code = (nib ^ 8) - 8;
                acc = __fmaf_rn((float)code, p.s_k[(size_t)i * p.E + j], acc);
            }
        } else {
            const int h = -ps - 1;
            for (int i = 0; i < p.N; ++i) {
                const uint16_t v = reinterpret_cast<const uint16_t *>(p.pl[i] + p.lp_bytes)[t * p.k + h];
                acc = __fadd_rn(acc, __uint_as_float((uint32_t)v << 16));
            }
        }
        if (FP32OUT)
            static_cast<float *>(p.out)[t * p.out_stride + j] = acc;
        else
            static_cast<__nv_bfloat16 *>(p.out)[t * p.out_stride + j] = __float2bfloat16_rn(acc);
    }
}

// ----------------------------------------------------------------------------------------------
// Tiled kernel for E, k and the output stride multiples of 8.
//
// Thread <-> 8 adjacent OUTPUT features; block <-> a strip of 8*blockDim.x features; blocks walk
// row blocks of R rows.  The steps of NC devices for the thread's 8 features live in registers.
// Because (E-k) is a multiple of 8, the bit offset of the thread's codes inside a 32-bit word of
// the flat code stream is the same for every row: one (or two) 32-bit loads per device and row
// plus a funnel shift give its 8 codes; a warp reads 128 contiguous bytes.  Where a selected
// feature falls inside the thread's 8, the codes are spread around the hole and the BF16 value
// of every device is added instead.  R*NC independent loads are in flight per thread.
// ----------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t spread_holes(uint32_t raw, uint32_t mask)
{
    // insert a zero nibble at every set position of mask (ascending)
    while (mask) {
        const int b = __ffs(mask) - 1;
        const uint32_t low = (b == 0) ? 0u : (0xFFFFFFFFu >> (32 - 4 * b));
        raw = (raw & low) | ((raw & ~low) << 4);
        mask &= mask - 1;
    }
    return raw;
}

template <int NC, int R, bool FP32OUT>
__global__ void __launch_bounds__(128) dequant_tiled(const DQParams p)
{
    const int E8 = p.E >> 3, L8 = (p.E - p.k) >> 3;
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= E8) return;
    const uint32_t gd = __ldg(p.grp + g);
    const uint32_t mask = gd & 0xFFu;
    const int hb = (int)(gd >> 8);
    const int c0 = 8 * g - hb;              // compacted slot of the group's first code
    const int n_lp = 8 - __popc(mask);
    const int sh = (c0 & 7) * 4;
    const int wbase = c0 >> 3;
    const bool need_lo = n_lp > 0;
    const bool need_hi = (c0 & 7) + n_lp > 8;
    const int64_t n_rb = (p.T + R - 1) / R;
    const bool single = p.N <= NC;

    float sc[NC][8];
    if (single) {
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            if (i < p.N) {
                const float4 a = __ldg(reinterpret_cast<const float4 *>(p.s_k + (size_t)i * p.E + 8 * g));
                const float4 b = __ldg(reinterpret_cast<const float4 *>(p.s_k + (size_t)i * p.E + 8 * g + 4));
                sc[i][0] = a.x; sc[i][1] = a.y; sc[i][2] = a.z; sc[i][3] = a.w;
                sc[i][4] = b.x; sc[i][5] = b.y; sc[i][6] = b.z; sc[i][7] = b.w;
            } else {
#pragma unroll
                for (int n = 0; n < 8; ++n) sc[i][n] = 0.0f;
            }
        }
    }

    for (int64_t rb = blockIdx.y; rb < n_rb; rb += gridDim.y) {
        const int64_t t0 = rb * R;
        float acc[R][8];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int n = 0; n < 8; ++n) acc[r][n] = 0.0f;

        for (int i0 = 0; i0 < p.N; i0 += NC) {
            if (!single) {
#pragma unroll
                for (int i = 0; i < NC; ++i) {
                    if (i0 + i < p.N) {
                        const float4 a = __ldg(reinterpret_cast<const float4 *>(p.s_k + (size_t)(i0 + i) * p.E + 8 * g));
                        const float4 b =
                            __ldg(reinterpret_cast<const float4 *>(p.s_k + (size_t)(i0 + i) * p.E + 8 * g + 4));
                        sc[i][0] = a.x; sc[i][1] = a.y; sc[i][2] = a.z; sc[i][3] = a.w;
                        sc[i][4] = b.x; sc[i][5] = b.y; sc[i][6] = b.z; sc[i][7] = b.w;
                    }
                }
            }
            uint32_t lo[R][NC], hi[R][NC];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < NC; ++i) {
                    lo[r][i] = 0u;
                    hi[r][i] = 0u;
                    if (t0 + r < p.T && i0 + i < p.N) {
                        const uint32_t *w = reinterpret_cast<const uint32_t *>(p.pl[i0 + i]) + (t0 + r) * L8 + wbase;
                        if (need_lo) lo[r][i] = __ldcs(w);
                        if (need_hi) hi[r][i] = __ldcs(w + 1);
                    }
                }
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int i = 0; i < NC; ++i) {
                    if (t0 + r < p.T && i0 + i < p.N) {
                        uint32_t raw = __funnelshift_r(lo[r][i], hi[r][i], sh);
                        if (mask) raw = spread_holes(raw, mask);
                        const uint32_t x = raw ^ 0x88888888u;  // two's complement -> offset binary
#pragma unroll
                        for (int n = 0; n < 8; ++n) {
                            // 2^23 + (code + 8) as a float, minus (2^23 + 8): the code, exactly
                            const float f =
                                __fsub_rn(__uint_as_float(0x4B000000u | ((x >> (4 * n)) & 0xFu)), 8388616.0f);
                            acc[r][n] = __fmaf_rn(f, sc[i][n], acc[r][n]);
                        }
                        if (mask) {
                            const uint16_t *hp = reinterpret_cast<const uint16_t *>(p.pl[i0 + i] + p.lp_bytes) +
                                                 (t0 + r) * p.k + hb;
                            int h = 0;
#pragma unroll
                            for (int n = 0; n < 8; ++n)
                                if (mask & (1u << n))
                                    acc[r][n] = __fadd_rn(acc[r][n], __uint_as_float((uint32_t)__ldcs(hp + h++) << 16));
                        }
                    }
                }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (t0 + r < p.T) {
                if (FP32OUT) {
                    float4 *o = reinterpret_cast<float4 *>(static_cast<float *>(p.out) + (t0 + r) * p.out_stride + 8 * g);
                    __stcs(o, make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]));
                    __stcs(o + 1, make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]));
                } else {
                    uint32_t w[4];
#pragma unroll
                    for (int n = 0; n < 4; ++n) {
                        __nv_bfloat162 b = __floats2bfloat162_rn(acc[r][2 * n], acc[r][2 * n + 1]);
                        w[n] = *reinterpret_cast<uint32_t *>(&b);
                    }
                    uint4 *o = reinterpret_cast<uint4 *>(static_cast<uint16_t *>(p.out) + (t0 + r) * p.out_stride + 8 * g);
                    __stcs(o, make_uint4(w[0], w[1], w[2], w[3]));
                }
            }
        }
    }
}

void fill_params(DQParams &p, const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int64_t out_stride)
{
    for (int i = 0; i < c->N; ++i) p.pl[i] = static_cast<const uint8_t *>(payloads[i]);
    p.N = c->N; p.E = c->E; p.k = c->k; p.T = T;
    p.lp_bytes = tpq_lp_bytes_i(T, c->E, c->k);
    p.s_k = c->t.s_k; p.pos = c->t.pos; p.grp = c->t.grp;
    p.out = out; p.out_stride = out_stride;
}

}  // namespace

bool tpq_dequant_tiled_ok(const tpq_ctx *c, int64_t T, int64_t out_stride, int fp32_out)
{
    (void)fp32_out;
    if (c->E % 8 || c->k % 8 || out_stride % 8 || T <= 0) return false;
    return true;
}

cudaError_t tpq_launch_dequant_generic(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int fp32_out,
                                       int64_t out_stride, cudaStream_t st, int64_t *launches)
{
    DQParams p;
    fill_params(p, c, payloads, T, out, out_stride);
    int64_t blocks = (T * (int64_t)c->E + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (fp32_out)
        dequant_generic<true><<<(unsigned)blocks, 256, 0, st>>>(p);
    else
        dequant_generic<false><<<(unsigned)blocks, 256, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_dequant_tiled(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int fp32_out,
                                     int64_t out_stride, cudaStream_t st, int64_t *launches)
{
    DQParams p;
    fill_params(p, c, payloads, T, out, out_stride);
    const int E8 = c->E / 8;
    const int strips = (E8 + 127) / 128;
    constexpr int R = 4;
    const int64_t n_rb = (T + R - 1) / R;
    int64_t gy = ((int64_t)c->sm_count * 4 + strips - 1) / strips;
    if (gy > n_rb) gy = n_rb;
    if (gy > 65535) gy = 65535;
    if (gy < 1) gy = 1;
    dim3 grid(strips, (unsigned)gy), block(128);
    if (c->N <= 4) {
        if (fp32_out) dequant_tiled<4, R, true><<<grid, block, 0, st>>>(p);
        else          dequant_tiled<4, R, false><<<grid, block, 0, st>>>(p);
    } else {
        if (fp32_out) dequant_tiled<8, R, true><<<grid, block, 0, st>>>(p);
        else          dequant_tiled<8, R, false><<<grid, block, 0, st>>>(p);
    }
    ++*launches;
    return cudaGetLastError();
}

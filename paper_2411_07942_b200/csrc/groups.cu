// Group kernels: C^(i) and sum_i D^(i) for code widths other than 4 bits (the method "at lower and higher
// precision", paper Section 4 / Figure 3) on shapes whose E, k and strides are multiples of 8.
//
// In the payload's slot order the 8 adjacent features 8g .. 8g+7 (g < (E-k)/8) are B adjacent bytes of the
// token's code row (8 codes of B bits), so a thread that owns a group reads 16 bytes of BF16 input and
// writes B bytes of codes (quantise), or reads B bytes per device and writes 16 bytes of BF16 output
// (dequantise).  A thread keeps its group's 8 steps in registers and walks R rows.  Slots of selected
// features below E-k ("holes") carry the filler features' codes: the quantiser fetches the filler's value
// for those lanes, the dequantiser (whose steps are in slot order) stores those lanes to the filler
// features' columns.  Selected features travel as BF16: one thread per 8 of them and row.
// Plain vector loads and stores; no shared memory.  Arithmetic as in the Int4 kernels: u = fl(x * inv_s),
// clamp, round to nearest even; acc = fma(code, s, acc) over the devices in ascending order.
#include <cuda_bf16.h>

#include "tpq_internal.h"

namespace {

constexpr int GK_THREADS = 256;
constexpr int GK_MAX_BATCH = 16;

// ---- B bytes <-> 64 bits (the destination / source is B-byte aligned at best)
template <int B>
__device__ __forceinline__ void store_code_bytes(uint8_t *dst, uint64_t bits)
{
    if (B == 8) {
        *reinterpret_cast<uint2 *>(dst) = make_uint2((uint32_t)bits, (uint32_t)(bits >> 32));
    } else if (B == 4) {
        *reinterpret_cast<uint32_t *>(dst) = (uint32_t)bits;
    } else if (B == 2) {
        *reinterpret_cast<uint16_t *>(dst) = (uint16_t)bits;
    } else if (B == 6) {
#pragma unroll
        for (int j = 0; j < 3; ++j) reinterpret_cast<uint16_t *>(dst)[j] = (uint16_t)(bits >> (16 * j));
    } else {
#pragma unroll
        for (int j = 0; j < B; ++j) dst[j] = (uint8_t)(bits >> (8 * j));
    }
}

template <int B>
__device__ __forceinline__ uint64_t load_code_bytes(const uint8_t *src)
{
    if (B == 8) {
        const uint2 v = __ldcs(reinterpret_cast<const uint2 *>(src));
        return (uint64_t)v.x | ((uint64_t)v.y << 32);
    } else if (B == 4) {
        return __ldcs(reinterpret_cast<const uint32_t *>(src));
    } else if (B == 2) {
        return __ldcs(reinterpret_cast<const uint16_t *>(src));
    } else if (B == 6) {
        uint64_t r = 0;
#pragma unroll
        for (int j = 0; j < 3; ++j) r |= (uint64_t)__ldcs(reinterpret_cast<const uint16_t *>(src) + j) << (16 * j);
        return r;
    } else {
        uint64_t r = 0;
#pragma unroll
        for (int j = 0; j < B; ++j) r |= (uint64_t)__ldcs(src + j) << (8 * j);
        return r;
    }
}

// ----------------------------------------------------------------------------------------------
// Quantise + pack.  grid.y = shard of the batch; a thread <-> (group or 8 selected features, R rows).
// ----------------------------------------------------------------------------------------------
struct QGParams {
    const uint16_t *y[GK_MAX_BATCH];
    uint8_t *payload[GK_MAX_BATCH];
    int64_t T, stride, lp_bytes;
    int E, k;
    const float *inv_s;  // [n][E], first shard of the batch
    const uint32_t *grp;
    const int32_t *lp_idx, *hp_idx;
};

// Work layout of both kernels: the GW = (E-k)/8 + k/8 thread columns of a row (groups, then octets of
// selected features) are cut into chunks of GK_THREADS; grid.x = chunks x row lanes.  A thread keeps its column
// for its whole life (its tables are loaded once) and walks blocks of R rows with the stride of the row lanes.
template <int B>
__global__ void __launch_bounds__(GK_THREADS) quantize_groups(const QGParams p)
{
    constexpr int R = 4;
    const int E = p.E, k = p.k, L8 = (E - k) >> 3, k8 = k >> 3, GW = L8 + k8;
    const int chunks = (GW + GK_THREADS - 1) / GK_THREADS;
    const int gi = (int)(blockIdx.x % chunks) * GK_THREADS + threadIdx.x;
    const int lane0 = blockIdx.x / chunks, lanes = gridDim.x / chunks;
    const int sh = blockIdx.y;
    const uint16_t *const y = p.y[sh];
    uint8_t *const pl = p.payload[sh];
    const float *const inv_s = p.inv_s + (size_t)sh * E;
    const int64_t n_rb = (p.T + R - 1) / R;
    const float lo = -(float)(1 << (B - 1)), hi = (float)((1 << (B - 1)) - 1);
    {   // the code section is padded with zeros to a multiple of 16 bytes
        const int64_t code_bytes = p.T * L8 * B;
        if (blockIdx.x == 0 && code_bytes + threadIdx.x < p.lp_bytes) pl[code_bytes + threadIdx.x] = 0;
    }
    if (gi >= GW) return;
    if (gi < L8) {
        const int g = gi;
        const float4 i0 = __ldg(reinterpret_cast<const float4 *>(inv_s + 8 * g));
        const float4 i1 = __ldg(reinterpret_cast<const float4 *>(inv_s + 8 * g + 4));
        float inv[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
        const uint32_t mask = __ldg(p.grp + g) & 0xFFu;
        // holes: the slot carries the filler feature.  The first hole of the group is handled without a branch
        // (its filler value is fetched with the row), further ones (rare) in a branch.
        const int first = mask ? __ffs(mask) - 1 : 0;
        const int f_first = mask ? __ldg(p.lp_idx + 8 * g + first) : 8 * g;
        const uint32_t more = mask & (mask - 1);
        if (mask) {
#pragma unroll
            for (int n = 0; n < 8; ++n)
                if (mask & (1u << n)) inv[n] = __ldg(inv_s + __ldg(p.lp_idx + 8 * g + n));
        }
        for (int64_t rb = lane0; rb < n_rb; rb += lanes) {
            const int64_t t0 = rb * R;
            uint4 v[R];
            uint32_t fv[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {  // all loads first; rows past the end re-read the last row
                const int64_t t = (t0 + r < p.T) ? t0 + r : p.T - 1;
                const uint16_t *const row = y + t * p.stride;
                v[r] = __ldcs(reinterpret_cast<const uint4 *>(row + 8 * g));
                fv[r] = (uint32_t)__ldg(row + f_first) << 16;
            }
            uint8_t *dst = pl + (t0 * L8 + g) * B;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (t0 + r >= p.T) break;
                uint32_t xb[8] = {v[r].x << 16, v[r].x & 0xFFFF0000u, v[r].y << 16, v[r].y & 0xFFFF0000u,
                                  v[r].z << 16, v[r].z & 0xFFFF0000u, v[r].w << 16, v[r].w & 0xFFFF0000u};
                if (mask) {
#pragma unroll
                    for (int n = 0; n < 8; ++n) xb[n] = (n == first) ? fv[r] : xb[n];
                    if (more) {
                        const uint16_t *const row = y + (t0 + r) * p.stride;
#pragma unroll
                        for (int n = 0; n < 8; ++n)
                            if (more & (1u << n)) xb[n] = (uint32_t)__ldg(row + __ldg(p.lp_idx + 8 * g + n)) << 16;
                    }
                }
                // codes 0..3 and 4..7 are gathered in two 32-bit halves (4 B <= 32 bits each); the code is read
                // from the low bits of fl(u + 1.5 * 2^23): nearest-even rounding without a conversion instruction
                uint32_t half[2] = {0u, 0u};
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    float uq = __fmul_rn(__uint_as_float(xb[n]), inv[n]);
                    uq = fminf(fmaxf(uq, lo), hi);
                    const uint32_t q = __float_as_uint(__fadd_rn(uq, 12582912.0f)) & ((1u << B) - 1u);
                    half[n >> 2] |= q << ((n & 3) * B);
                }
                store_code_bytes<B>(dst, (uint64_t)half[0] | ((uint64_t)half[1] << (4 * B)));
                dst += (size_t)L8 * B;
            }
        }
    } else {
        const int h8 = gi - L8;
        const int4 c0 = __ldg(reinterpret_cast<const int4 *>(p.hp_idx + 8 * h8));
        const int4 c1 = __ldg(reinterpret_cast<const int4 *>(p.hp_idx + 8 * h8) + 1);
        const int col[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        for (int64_t rb = lane0; rb < n_rb; rb += lanes) {
            const int64_t t0 = rb * R;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int64_t t = t0 + r;
                if (t >= p.T) break;
                const uint16_t *const row = y + t * p.stride;
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    w[j] = (uint32_t)__ldg(row + col[2 * j]) | ((uint32_t)__ldg(row + col[2 * j + 1]) << 16);
                *reinterpret_cast<uint4 *>(pl + p.lp_bytes + (t * k + 8 * h8) * 2) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
    }
}

// ----------------------------------------------------------------------------------------------
// Dequantise + reduce.  A thread <-> (group or 8 selected features, R rows).
// ----------------------------------------------------------------------------------------------
struct DGParams {
    const uint8_t *pl[TPQ_MAX_SHARDS];
    int N, E, k;
    int64_t T, lp_bytes, out_stride;
    const float *s_slot;  // [N][E] steps in slot order
    const uint32_t *grp;
    const int32_t *lp_idx, *hp_idx;
    void *out;
    const float *bias;  // [E] added after the sum, or NULL
    tpq_arrivals arr;   // arrival words to wait for before the first payload read (words == NULL: none)
};

template <bool FP32OUT>
__device__ __forceinline__ void gk_store(void *out, int64_t off, float v)
{
    if (FP32OUT)
        static_cast<float *>(out)[off] = v;
    else
        static_cast<__nv_bfloat16 *>(out)[off] = __float2bfloat16_rn(v);
}

template <int B, bool FP32OUT>
__global__ void __launch_bounds__(GK_THREADS) dequant_groups(const DGParams p)
{
    if (p.arr.words) {
        tpq_block_wait_arrivals(p.arr);
        __syncthreads();
    }
    constexpr int R = 2;
    const int E = p.E, k = p.k, L8 = (E - k) >> 3, k8 = k >> 3, GW = L8 + k8;
    const int64_t n_rb = (p.T + R - 1) / R;
    for (int64_t u = (int64_t)blockIdx.x * GK_THREADS + threadIdx.x; u < n_rb * GW; u += (int64_t)gridDim.x * GK_THREADS) {
        const int64_t rb = u / GW;
        const int gi = (int)(u - rb * GW);
        const int64_t t0 = rb * R;
        const int rows = (int)((p.T - t0 < R) ? p.T - t0 : R);
        if (gi < L8) {
            const int g = gi;
            float acc[R][8];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < 8; ++n) acc[r][n] = 0.0f;
            constexpr int NI = 4;  // devices whose loads are in flight together
            for (int i0 = 0; i0 < p.N; i0 += NI) {
                uint64_t bits[NI][R];
#pragma unroll
                for (int ii = 0; ii < NI; ++ii)
#pragma unroll
                    for (int r = 0; r < R; ++r)
                        if (i0 + ii < p.N && r < rows) bits[ii][r] = load_code_bytes<B>(p.pl[i0 + ii] + ((t0 + r) * L8 + g) * B);
#pragma unroll
                for (int ii = 0; ii < NI; ++ii) {
                    const int i = i0 + ii;
                    if (i >= p.N) break;
                    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(p.s_slot + (size_t)i * E + 8 * g));
                    const float4 s1 = __ldg(reinterpret_cast<const float4 *>(p.s_slot + (size_t)i * E + 8 * g + 4));
                    const float s[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        if (r >= rows) break;
#pragma unroll
                        for (int n = 0; n < 8; ++n) {
                            // two's complement, B bits: shift the code to the top of a 64-bit integer and back
                            const int code = (int)((int64_t)(bits[ii][r] << (64 - (n + 1) * B)) >> (64 - B));
                            acc[r][n] = __fmaf_rn((float)code, s[n], acc[r][n]);
                        }
                    }
                }
            }
            const uint32_t mask = __ldg(p.grp + g) & 0xFFu;
            if (p.bias) {
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    const int col = (mask & (1u << n)) ? __ldg(p.lp_idx + 8 * g + n) : 8 * g + n;
                    const float b = __ldg(p.bias + col);
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r][n] = __fadd_rn(acc[r][n], b);
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (r >= rows) break;
                const int64_t orow = (t0 + r) * p.out_stride;
                if (mask == 0) {
                    if (FP32OUT) {
                        float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.out) + orow + 8 * g);
                        dst[0] = make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
                        dst[1] = make_float4(acc[r][4], acc[r][5], acc[r][6], acc[r][7]);
                    } else {
                        uint32_t w[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[r][2 * j], acc[r][2 * j + 1]);
                            w[j] = *reinterpret_cast<uint32_t *>(&b2);
                        }
                        *reinterpret_cast<uint4 *>(static_cast<uint16_t *>(p.out) + orow + 8 * g) =
                            make_uint4(w[0], w[1], w[2], w[3]);
                    }
                } else {
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        // a hole's lane holds the sum of the filler feature whose codes sit in the slot
                        const int col = (mask & (1u << n)) ? __ldg(p.lp_idx + 8 * g + n) : 8 * g + n;
                        gk_store<FP32OUT>(p.out, orow + col, acc[r][n]);
                    }
                }
            }
        } else {
            const int h8 = gi - L8;
            float acc[R][8];
#pragma unroll
            for (int r = 0; r < R; ++r)
#pragma unroll
                for (int n = 0; n < 8; ++n) acc[r][n] = 0.0f;
            for (int i = 0; i < p.N; ++i) {
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    if (r >= rows) break;
                    const uint4 v = __ldcs(reinterpret_cast<const uint4 *>(p.pl[i] + p.lp_bytes + ((t0 + r) * k + 8 * h8) * 2));
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        acc[r][2 * j] = __fadd_rn(acc[r][2 * j], __uint_as_float(w[j] << 16));
                        acc[r][2 * j + 1] = __fadd_rn(acc[r][2 * j + 1], __uint_as_float(w[j] & 0xFFFF0000u));
                    }
                }
            }
            const int4 c0 = __ldg(reinterpret_cast<const int4 *>(p.hp_idx + 8 * h8));
            const int4 c1 = __ldg(reinterpret_cast<const int4 *>(p.hp_idx + 8 * h8) + 1);
            const int col[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
            for (int r = 0; r < R; ++r) {
                if (r >= rows) break;
#pragma unroll
                for (int n = 0; n < 8; ++n)
                    gk_store<FP32OUT>(p.out, (t0 + r) * p.out_stride + col[n],
                                      p.bias ? __fadd_rn(acc[r][n], __ldg(p.bias + col[n])) : acc[r][n]);
            }
        }
    }
}

// flat grid of the dequantiser: one unit = (row block, thread column)
unsigned gk_grid_units(int64_t units, int sm_count)
{
    int64_t blocks = (units + GK_THREADS - 1) / GK_THREADS;
    const int64_t cap = (int64_t)sm_count * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (unsigned)blocks;
}

// grid.x = column chunks x row lanes; every row lane walks the same number of row blocks (no lane is left
// with one block more than the others), up to about 32 blocks per SM
unsigned gk_grid(int GW, int64_t row_blocks, int sm_count)
{
    const int64_t chunks = (GW + GK_THREADS - 1) / GK_THREADS;
    int64_t lanes_max = ((int64_t)sm_count * 32 + chunks - 1) / chunks;
    if (lanes_max < 1) lanes_max = 1;
    const int64_t iters = (row_blocks + lanes_max - 1) / lanes_max;
    int64_t lanes = (row_blocks + iters - 1) / (iters > 0 ? iters : 1);
    if (lanes < 1) lanes = 1;
    return (unsigned)(chunks * lanes);
}

}  // namespace

bool tpq_groups_ok(const tpq_ctx *c, int64_t T, int64_t stride)
{
    if (c->bits == 4 || c->bits < 2 || c->bits > 8) return false;
    if (c->E % 8 || c->k % 8 || stride % 8 || T <= 0) return false;
    return c->E - c->k >= 8;
}

cudaError_t tpq_launch_quantize_groups(const tpq_ctx *c, int shard0, int n, const void *const *ys, int64_t T,
                                       int64_t stride, void *const *payloads, cudaStream_t st, int64_t *launches)
{
    const int E = c->E, k = c->k;
    for (int b0 = 0; b0 < n; b0 += GK_MAX_BATCH) {
        const int nb = (n - b0 < GK_MAX_BATCH) ? n - b0 : GK_MAX_BATCH;
        QGParams p;
        for (int b = 0; b < nb; ++b) {
            p.y[b] = static_cast<const uint16_t *>(ys[b0 + b]);
            p.payload[b] = static_cast<uint8_t *>(payloads[b0 + b]);
        }
        p.T = T; p.stride = stride; p.lp_bytes = tpq_lp_bytes_i(T, E, k, c->bits);
        p.E = E; p.k = k;
        p.inv_s = c->t.inv_s + (size_t)(shard0 + b0) * E;
        p.grp = c->t.grp; p.lp_idx = c->t.lp_idx; p.hp_idx = c->t.hp_idx;
        const dim3 grid(gk_grid((E - k) / 8 + k / 8, (T + 3) / 4, c->sm_count), (unsigned)nb);
        switch (c->bits) {
        case 2: quantize_groups<2><<<grid, GK_THREADS, 0, st>>>(p); break;
        case 3: quantize_groups<3><<<grid, GK_THREADS, 0, st>>>(p); break;
        case 5: quantize_groups<5><<<grid, GK_THREADS, 0, st>>>(p); break;
        case 6: quantize_groups<6><<<grid, GK_THREADS, 0, st>>>(p); break;
        case 7: quantize_groups<7><<<grid, GK_THREADS, 0, st>>>(p); break;
        case 8: quantize_groups<8><<<grid, GK_THREADS, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
        }
        const cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    return cudaSuccess;
}

namespace {
template <int B>
void launch_dequant_groups_b(const DGParams &p, int fp32_out, unsigned grid, cudaStream_t st)
{
    if (fp32_out)
        dequant_groups<B, true><<<grid, GK_THREADS, 0, st>>>(p);
    else
        dequant_groups<B, false><<<grid, GK_THREADS, 0, st>>>(p);
}
}  // namespace

cudaError_t tpq_launch_dequant_groups(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int fp32_out,
                                      int64_t out_stride, cudaStream_t st, int64_t *launches)
{
    const int E = c->E, k = c->k;
    DGParams p;
    for (int i = 0; i < c->N; ++i) p.pl[i] = static_cast<const uint8_t *>(payloads[i]);
    p.N = c->N; p.E = E; p.k = k; p.T = T;
    p.lp_bytes = tpq_lp_bytes_i(T, E, k, c->bits);
    p.out_stride = out_stride;
    p.s_slot = c->t.s_slot; p.grp = c->t.grp; p.lp_idx = c->t.lp_idx; p.hp_idx = c->t.hp_idx;
    p.out = out;
    p.bias = c->call_bias;
    p.arr = c->call_arr;
    const int64_t units = ((T + 1) / 2) * (int64_t)((E - k) / 8 + k / 8);
    const unsigned grid = gk_grid_units(units, c->sm_count);
    switch (c->bits) {
    case 2: launch_dequant_groups_b<2>(p, fp32_out, grid, st); break;
    case 3: launch_dequant_groups_b<3>(p, fp32_out, grid, st); break;
    case 5: launch_dequant_groups_b<5>(p, fp32_out, grid, st); break;
    case 6: launch_dequant_groups_b<6>(p, fp32_out, grid, st); break;
    case 7: launch_dequant_groups_b<7>(p, fp32_out, grid, st); break;
    case 8: launch_dequant_groups_b<8>(p, fp32_out, grid, st); break;
    default: return cudaErrorInvalidValue;
    }
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) ++*launches;
    return e;
}

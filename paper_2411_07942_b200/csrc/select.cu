// Range aggregation, top-k feature selection and table construction
// (paper Section 3 "Selecting High Precision Features"; k = floor(E/64) in Section 4).
#include "tpq_internal.h"

namespace {

// R^(i)_j = 2 max(-m, M); Rbar_j = sum_i R^(i)_j (binary32, devices ascending);
// step s = R/(2^bits - 1) (R/15 for Int4) floored at 2^-23 and its reciprocal (IEEE division, no fast-math).
__global__ void __launch_bounds__(256) ranges_kernel(const float *__restrict__ m, const float *__restrict__ M, int N,
                                                     int E, float levels, float *__restrict__ R,
                                                     float *__restrict__ Rbar, float *__restrict__ s,
                                                     float *__restrict__ inv_s)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= E) return;
    float acc = 0.0f;
    for (int i = 0; i < N; ++i) {
        const size_t o = (size_t)i * E + j;
        const float a = -m[o], b = M[o];
        const float A = (a > b) ? a : b;
        const float r = __fmul_rn(2.0f, A);
        R[o] = r;
        acc = (i == 0) ? r : __fadd_rn(acc, r);
        float sv = __fdiv_rn(r, levels);
        if (!(sv >= 1.1920928955078125e-07f)) sv = 1.1920928955078125e-07f;
        s[o] = sv;
        inv_s[o] = __fdiv_rn(1.0f, sv);
    }
    Rbar[j] = acc;
}

// Feature j is selected iff fewer than k features beat it, where a beats j when
// Rbar_a > Rbar_j, or Rbar_a == Rbar_j and a < j.  O(E^2) comparisons, tiled through shared memory.
__global__ void __launch_bounds__(256) topk_flags_kernel(const float *__restrict__ Rbar, int E, int k,
                                                         uint8_t *__restrict__ flag)
{
    __shared__ float tile[1024];
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const float mine = (j < E) ? Rbar[j] : 0.0f;
    int beats = 0;
    for (int a0 = 0; a0 < E; a0 += 1024) {
        __syncthreads();
        for (int a = threadIdx.x; a < 1024; a += blockDim.x) tile[a] = (a0 + a < E) ? Rbar[a0 + a] : 0.0f;
        __syncthreads();
        const int n = (E - a0 < 1024) ? E - a0 : 1024;
        for (int a = 0; a < n; ++a) {
            const float v = tile[a];
            beats += (v > mine) || (v == mine && (a0 + a) < j);
        }
    }
    if (j < E) flag[j] = (beats < k) ? 1 : 0;
}

// One block: exclusive scan of the flags -> selected list, hole / filler lists, slot order,
// per-feature slots, the dequantiser's zeroed-step and slot-order step copies and the per-8-feature
// group descriptors.
__global__ void __launch_bounds__(1024) tables_kernel(tpq_tables t, int N, int E, int k)
{
    __shared__ int warp_sums[32];
    __shared__ int carry;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int L = E - k;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int j0 = 0; j0 < E; j0 += 1024) {
        const int j = j0 + tid;
        const int f = (j < E) ? t.flag[j] : 0;
        int incl = f;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        if (lane == 31) warp_sums[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            int w = warp_sums[lane];
            int wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int o = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= d) wi += o;
            }
            warp_sums[lane] = wi - w;  // exclusive
        }
        __syncthreads();
        const int before = carry + warp_sums[wid] + incl - f;  // selected features before j
        if (j < E) {
            t.hpre[j] = before;
            if (f) t.hp_idx[before] = j;
            for (int i = 0; i < N; ++i) t.s_k[(size_t)i * E + j] = f ? 0.0f : t.s[(size_t)i * E + j];
        }
        __syncthreads();
        if (tid == 1023) carry = before + f;
        __syncthreads();
    }
    // holes: selected features below L; fillers: unselected features at or above L (equally many)
    const int m = (L < E) ? t.hpre[L] : 0;
    for (int j = tid; j < E; j += 1024) {
        const int f = t.flag[j];
        if (f && j < L) t.hole[t.hpre[j]] = j;
        if (!f && j >= L) t.filler[(j - L) - (t.hpre[j] - m)] = j;
    }
    __syncthreads();
    for (int j = tid; j < E; j += 1024) {
        const int f = t.flag[j];
        const int src = (j < L) ? (f ? t.filler[t.hpre[j]] : j) : -1;  // feature held by slot j
        if (j < L) t.lp_idx[j] = src;
        for (int i = 0; i < N; ++i) t.s_slot[(size_t)i * E + j] = (src >= 0) ? t.s[(size_t)i * E + src] : 0.0f;
        if (f)
            t.pos[j] = -(t.hpre[j] + 1);
        else
            t.pos[j] = (j < L) ? j : t.hole[(j - L) - (t.hpre[j] - m)];
    }
    const int n_grp = (E + 7) / 8;
    for (int g = tid; g < n_grp; g += 1024) {
        uint32_t mask = 0;
        for (int n = 0; n < 8; ++n)
            if (8 * g + n < E && t.flag[8 * g + n]) mask |= 1u << n;
        t.grp[g] = ((uint32_t)t.hpre[8 * g] << 8) | mask;
    }
}

}  // namespace

cudaError_t tpq_launch_ranges(const tpq_tables &t, int N, int E, int bits, cudaStream_t st, int64_t *launches)
{
    ranges_kernel<<<(E + 255) / 256, 256, 0, st>>>(t.m, t.M, N, E, (float)((1 << bits) - 1), t.R, t.Rbar, t.s, t.inv_s);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_topk_flags(const tpq_tables &t, int E, int k, cudaStream_t st, int64_t *launches)
{
    topk_flags_kernel<<<(E + 255) / 256, 256, 0, st>>>(t.Rbar, E, k, t.flag);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_tables(const tpq_tables &t, int N, int E, int k, cudaStream_t st, int64_t *launches)
{
    tables_kernel<<<1, 1024, 0, st>>>(t, N, E, k);
    ++*launches;
    return cudaGetLastError();
}

// Calibration kernels: column extremes per sequence and the moving-average fold
// (paper Section 3 "Calibration", Eq. (1)-(2)).
//
// BF16 values are compared through an order-preserving 16-bit integer key
// (sign-magnitude -> two's complement, so -0 sorts below +0 and the result does
// not depend on the order in which rows are visited); min / max of the keys are
// exact, so any reduction tree gives the same bits.
#include <mutex>

#include "tpq_internal.h"

namespace {

// two packed BF16 patterns -> two packed signed 16-bit keys (an involution)
__device__ __forceinline__ uint32_t key2(uint32_t w)
{
    uint32_t neg = (w >> 15) & 0x00010001u;
    return w ^ (neg * 0x7FFFu);
}
__device__ __forceinline__ uint32_t min_s16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("min.s16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t max_s16x2(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.s16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float key_to_float(int16_t key)
{
    uint32_t kk = (uint16_t)key;
    uint32_t pat = kk ^ ((kk >> 15) * 0x7FFFu);
    return __uint_as_float(pat << 16);
}

constexpr uint32_t KEY_MAX2 = 0x7FFF7FFFu;  // identity of min
constexpr uint32_t KEY_MIN2 = 0x80008000u;  // identity of max

// Tiled extremes: thread = 8 adjacent features (one 128-bit load per row), 8 row lanes per block,
// eight independent loads in flight per thread.  grid = (feature chunks of 256, row splits, sequences).
__global__ void __launch_bounds__(256) colminmax_tiled(const uint16_t *__restrict__ y, int64_t S, int64_t stride, int E,
                                                       int n_split, int16_t *__restrict__ part_lo,
                                                       int16_t *__restrict__ part_hi)
{
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int g = blockIdx.x * 32 + tx;  // group of 8 features
    const int sp = blockIdx.y;
    const int64_t q = blockIdx.z;
    const int64_t rps = (S + n_split - 1) / n_split;
    const int64_t r0 = sp * rps;
    const int64_t r1 = (r0 + rps < S) ? r0 + rps : S;
    const bool live = 8 * g < E;

    uint32_t lo[4] = {KEY_MAX2, KEY_MAX2, KEY_MAX2, KEY_MAX2};
    uint32_t hi[4] = {KEY_MIN2, KEY_MIN2, KEY_MIN2, KEY_MIN2};
    if (live) {
        const uint16_t *col = y + q * S * stride + 8 * (int64_t)g;
        int64_t r = r0 + ty;
        for (; r + 56 < r1; r += 64) {  // eight independent 128-bit loads in flight per thread
            uint4 v[8];
#pragma unroll
            for (int a = 0; a < 8; ++a) v[a] = __ldcs(reinterpret_cast<const uint4 *>(col + (r + 8 * a) * stride));
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                const uint32_t w[4] = {v[a].x, v[a].y, v[a].z, v[a].w};
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    uint32_t kk = key2(w[b]);
                    lo[b] = min_s16x2(lo[b], kk);
                    hi[b] = max_s16x2(hi[b], kk);
                }
            }
        }
        for (; r + 24 < r1; r += 32) {
            uint4 v0 = __ldcs(reinterpret_cast<const uint4 *>(col + r * stride));
            uint4 v1 = __ldcs(reinterpret_cast<const uint4 *>(col + (r + 8) * stride));
            uint4 v2 = __ldcs(reinterpret_cast<const uint4 *>(col + (r + 16) * stride));
            uint4 v3 = __ldcs(reinterpret_cast<const uint4 *>(col + (r + 24) * stride));
            const uint32_t w[4][4] = {{v0.x, v0.y, v0.z, v0.w}, {v1.x, v1.y, v1.z, v1.w},
                                      {v2.x, v2.y, v2.z, v2.w}, {v3.x, v3.y, v3.z, v3.w}};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    uint32_t kk = key2(w[a][b]);
                    lo[b] = min_s16x2(lo[b], kk);
                    hi[b] = max_s16x2(hi[b], kk);
                }
        }
        for (; r < r1; r += 8) {
            uint4 v = __ldcs(reinterpret_cast<const uint4 *>(col + r * stride));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                uint32_t kk = key2(w[b]);
                lo[b] = min_s16x2(lo[b], kk);
                hi[b] = max_s16x2(hi[b], kk);
            }
        }
    }
    __shared__ uint4 slo[8][32], shi[8][32];
    slo[ty][tx] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
    shi[ty][tx] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    __syncthreads();
    if (ty == 0 && live) {
#pragma unroll
        for (int a = 1; a < 8; ++a) {
            uint4 l = slo[a][tx], h = shi[a][tx];
            lo[0] = min_s16x2(lo[0], l.x); lo[1] = min_s16x2(lo[1], l.y);
            lo[2] = min_s16x2(lo[2], l.z); lo[3] = min_s16x2(lo[3], l.w);
            hi[0] = max_s16x2(hi[0], h.x); hi[1] = max_s16x2(hi[1], h.y);
            hi[2] = max_s16x2(hi[2], h.z); hi[3] = max_s16x2(hi[3], h.w);
        }
        const int64_t o = (q * n_split + sp) * (int64_t)E + 8 * (int64_t)g;
        *reinterpret_cast<uint4 *>(part_lo + o) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        *reinterpret_cast<uint4 *>(part_hi + o) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    }
}

// Shape-generic extremes: thread = one feature, any E and stride.
__global__ void __launch_bounds__(256) colminmax_generic(const uint16_t *__restrict__ y, int64_t S, int64_t stride,
                                                         int E, int n_split, int16_t *__restrict__ part_lo,
                                                         int16_t *__restrict__ part_hi)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= E) return;
    const int sp = blockIdx.y;
    const int64_t q = blockIdx.z;
    const int64_t rps = (S + n_split - 1) / n_split;
    const int64_t r0 = sp * rps;
    const int64_t r1 = (r0 + rps < S) ? r0 + rps : S;
    int lo = 0x7FFF, hi = -0x8000;
    for (int64_t r = r0; r < r1; ++r) {
        uint32_t w = y[(q * S + r) * stride + j];
        int kk = (int)(int16_t)(uint16_t)(w ^ ((w >> 15) * 0x7FFFu));
        lo = min(lo, kk);
        hi = max(hi, kk);
    }
    const int64_t o = (q * n_split + sp) * (int64_t)E + j;
    part_lo[o] = (int16_t)lo;
    part_hi[o] = (int16_t)hi;
}

// Eq. (1)-(2): combine the row splits of every sequence, then fold the sequences in order.
// m <- fl( fl((1-gamma) m) + fl(gamma min) ); the first sequence a device sees initialises.
//
// A block owns EF_X features.  Its EF_Y thread rows first reduce the splits of EF_Q sequences side by side
// (extremes are order-free, and these loads are the latency of the kernel: one thread walking every partial
// of a feature pays one L2 round trip per sequence and split), park the per-sequence extremes in shared
// memory, and the first thread row then runs the moving average over them in sequence order.
constexpr int EF_X = 32, EF_Y = 8, EF_Q = 64;

__global__ void __launch_bounds__(EF_X *EF_Y) ema_fold(const int16_t *__restrict__ part_lo,
                                                       const int16_t *__restrict__ part_hi, int64_t n_seq, int n_split,
                                                       int E, float *__restrict__ m, float *__restrict__ M,
                                                       int64_t count0, float gamma)
{
    __shared__ int16_t s_lo[EF_Q][EF_X], s_hi[EF_Q][EF_X];
    const int x = threadIdx.x & (EF_X - 1), yl = threadIdx.x / EF_X;
    const int j = blockIdx.x * EF_X + x;
    const bool live = j < E;
    const float c = __fsub_rn(1.0f, gamma);
    float mj = 0.f, Mj = 0.f;
    if (live && yl == 0) {
        mj = m[j];
        Mj = M[j];
    }
    for (int64_t q0 = 0; q0 < n_seq; q0 += EF_Q) {
        const int nq = (int)((n_seq - q0 < EF_Q) ? n_seq - q0 : EF_Q);
        for (int u = yl; u < nq; u += EF_Y) {
            int lo = 0x7FFF, hi = -0x8000;
            if (live) {
                const int16_t *pl = part_lo + (q0 + u) * n_split * (int64_t)E + j;
                const int16_t *ph = part_hi + (q0 + u) * n_split * (int64_t)E + j;
#pragma unroll 4
                for (int sp = 0; sp < n_split; ++sp) {
                    lo = min(lo, (int)pl[(int64_t)sp * E]);
                    hi = max(hi, (int)ph[(int64_t)sp * E]);
                }
            }
            s_lo[u][x] = (int16_t)lo;
            s_hi[u][x] = (int16_t)hi;
        }
        __syncthreads();
        if (live && yl == 0) {
            for (int u = 0; u < nq; ++u) {
                const float mn = key_to_float(s_lo[u][x]), mx = key_to_float(s_hi[u][x]);
                if (count0 + q0 + u == 0) {
                    mj = mn;
                    Mj = mx;
                } else {
                    mj = __fadd_rn(__fmul_rn(c, mj), __fmul_rn(gamma, mn));
                    Mj = __fadd_rn(__fmul_rn(c, Mj), __fmul_rn(gamma, mx));
                }
            }
        }
        __syncthreads();
    }
    if (live && yl == 0) {
        m[j] = mj;
        M[j] = Mj;
    }
}

int pick_splits(int64_t n_seq, int64_t S, int E, int sm_count)
{
    int64_t chunks = (E + 255) / 256;
    int64_t ctas = chunks * n_seq;
    int64_t want = (8LL * sm_count + ctas - 1) / ctas;
    int64_t cap = (S + 63) / 64;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    if (want > 65535) want = 65535;
    return (int)want;
}

}  // namespace

size_t tpq_calib_scratch_bytes(int64_t n_seq, int64_t S, int E, int sm_count, int *n_split_out)
{
    int ns = pick_splits(n_seq, S, E, sm_count);
    if (n_split_out) *n_split_out = ns;
    return (size_t)2 * (size_t)n_seq * ns * E * sizeof(int16_t);
}

cudaError_t tpq_launch_calibrate(const uint16_t *y, int64_t n_seq, int64_t S, int64_t stride, int E, float *m, float *M,
                                 int64_t count0, float gamma, void *scratch, int n_split, cudaStream_t st,
                                 int64_t *launches)
{
    int16_t *part_lo = static_cast<int16_t *>(scratch);
    int16_t *part_hi = part_lo + (size_t)n_seq * n_split * E;
    const bool tiled = (E % 8 == 0) && (stride % 8 == 0) && ((reinterpret_cast<uintptr_t>(y) & 15) == 0);
    // gridDim.z is limited to 65535: fold long calibration sets in slices of sequences
    for (int64_t q0 = 0; q0 < n_seq; q0 += 65535) {
        const int64_t nq = (n_seq - q0 < 65535) ? n_seq - q0 : 65535;
        const uint16_t *yq = y + q0 * S * stride;
        int16_t *lo = part_lo + (size_t)q0 * n_split * E, *hi = part_hi + (size_t)q0 * n_split * E;
        if (tiled) {
            dim3 grid((E / 8 + 31) / 32, n_split, (unsigned)nq), block(32, 8);
            colminmax_tiled<<<grid, block, 0, st>>>(yq, S, stride, E, n_split, lo, hi);
        } else {
            dim3 grid((E + 255) / 256, n_split, (unsigned)nq), block(256);
            colminmax_generic<<<grid, block, 0, st>>>(yq, S, stride, E, n_split, lo, hi);
        }
        ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    ema_fold<<<(E + EF_X - 1) / EF_X, EF_X * EF_Y, 0, st>>>(part_lo, part_hi, n_seq, n_split, E, m, M, count0, gamma);
    ++*launches;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the calibration pass.
//
// Same kernels as above; the partial-extremes scratch is this fixed array, resident in the global
// memory of every device that loads the library until the process exits.  Its address is looked up
// once per device with cudaGetSymbolAddress (the array's name is only a host-side handle, never a
// device address) and handed to the kernels like any other scratch pointer.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) int16_t g_calib_static_scratch[TPQ_NOALLOC_SCRATCH_BYTES / sizeof(int16_t)];

namespace {
constexpr int kMaxDevices = 64;
void *g_static_scratch_ptr[kMaxDevices];  // device address of the array, per device ordinal (set-up once)
bool g_static_scratch_ready[kMaxDevices];
std::mutex g_static_scratch_mutex;
}  // namespace

cudaError_t tpq_static_scratch_address(int device, void **ptr_out)
{
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    // The look-up answers for the CURRENT device: a caller on another device would cache a wrong address.
    int current = -1;
    cudaError_t e = cudaGetDevice(&current);
    if (e != cudaSuccess) return e;
    if (current != device) return cudaErrorInvalidDevice;
    // One look-up per device; contexts on several host threads may get here together.
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ready[device]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_calib_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_scratch_ptr[device] = ptr;
        g_static_scratch_ready[device] = true;
    }
    *ptr_out = g_static_scratch_ptr[device];
    return cudaSuccess;
}

// Largest row-split count (<= the usual choice) whose partial extremes fit the static array; 0 if none.
int tpq_static_scratch_splits(int64_t n_seq, int64_t S, int E, int sm_count)
{
    int ns = pick_splits(n_seq, S, E, sm_count);
    const size_t per_split = (size_t)2 * (size_t)n_seq * E * sizeof(int16_t);
    if (per_split == 0 || per_split > (size_t)TPQ_NOALLOC_SCRATCH_BYTES) return 0;
    const size_t fit = (size_t)TPQ_NOALLOC_SCRATCH_BYTES / per_split;
    if ((size_t)ns > fit) ns = (int)fit;
    return ns;
}

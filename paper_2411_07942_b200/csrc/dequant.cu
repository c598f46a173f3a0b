// sum_i D^(i): dequantise the N devices' payloads and sum them into the synchronised
// output, features back in their original order (paper Figure 2 caption; Section 5,
// all-gather followed by a local reduction).
//
// Accumulation is binary32, devices in ascending order: acc = fma(code_i, s_i, acc) for a
// low-precision feature, acc = fl(acc + y_i) for a selected one; one final rounding for BF16.
#include <cuda.h>  // CUtensorMap and the encode function's type (reached through the runtime, no libcuda link)
#include <cuda_bf16.h>

#include <new>

#include "tpq_internal.h"

namespace {

struct DQParams {
    const uint8_t *pl[TPQ_MAX_SHARDS];  // payloads, device order
    int N, E, k, bits;
    int64_t T;
    int64_t lp_bytes;      // code section size (HP block starts here)
    const float *s_k;      // [N][E], 0 at selected features
    const int32_t *pos;    // [E]
    const uint32_t *grp;   // [E/8]
    void *out;
    int64_t out_stride;
    const float *bias;     // [E] added after the sum (Section 2: f(x) = sum_i f_i(x_i) + b), or NULL
    tpq_arrivals arr;      // arrival words to wait for before the first payload read (words == NULL: none)
};

// ----------------------------------------------------------------------------------------------
// Shape-generic kernel: one thread per output element; any code width of 2..8 bits.
// ----------------------------------------------------------------------------------------------
template <bool FP32OUT>
__global__ void __launch_bounds__(256) dequant_generic(const DQParams p)
{
    if (p.arr.words) {
        tpq_block_wait_arrivals(p.arr);
        __syncthreads();
    }
    const int64_t total = p.T * (int64_t)p.E;
    const int64_t L = p.E - p.k;
    for (int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; a < total; a += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = a / p.E;
        const int j = (int)(a - t * p.E);
        const int ps = p.pos[j];
        float acc = 0.0f;
        if (ps >= 0) {
            const int64_t bit = (t * L + ps) * p.bits;  // first bit of the code in the little-endian stream
            const int sh = (int)(bit & 7);
            const bool two = sh + p.bits > 8;
            const uint32_t cmask = (1u << p.bits) - 1u, sign = 1u << (p.bits - 1);
            for (int i = 0; i < p.N; ++i) {
                uint32_t b = p.pl[i][bit >> 3];
                if (two) b |= (uint32_t)p.pl[i][(bit >> 3) + 1] << 8;
                const uint32_t u = (b >> sh) & cmask;
                const int code = (int)(u ^ sign) - (int)sign;  // two's complement, `bits` wide
                acc = __fmaf_rn((float)code, p.s_k[(size_t)i * p.E + j], acc);
            }
        } else {
            const int h = -ps - 1;
            for (int i = 0; i < p.N; ++i) {
                const uint16_t v = reinterpret_cast<const uint16_t *>(p.pl[i] + p.lp_bytes)[t * p.k + h];
                acc = __fadd_rn(acc, __uint_as_float((uint32_t)v << 16));
            }
        }
        if (p.bias) acc = __fadd_rn(acc, p.bias[j]);
        if (FP32OUT)
            static_cast<float *>(p.out)[t * p.out_stride + j] = acc;
        else
            static_cast<__nv_bfloat16 *>(p.out)[t * p.out_stride + j] = __float2bfloat16_rn(acc);
    }
}

// ----------------------------------------------------------------------------------------------
// Shared pieces of the tiled kernels (E, k and the output stride multiples of 8).
//
// In the payload's slot order, output features 8g .. 8g+7 (g < L/8, L = E-k) are the aligned 32-bit
// word g of every device's code row, so a thread that owns them needs one word per device and row.
// Slots whose feature is a selected one hold a filler feature's code instead: the thread's step for
// them is 0, it does not store them, and two small extra jobs complete the row:
//   - filler feature filler[tau], tau < n_holes, lives in slot hole[tau]: one code per device;
//   - selected feature hp_idx[h], h < k: the sum of the devices' BF16 values.
// ----------------------------------------------------------------------------------------------

__device__ __host__ constexpr int dq_pos(int n) { return n & 3; }

// 8 two's-complement codes of `raw` times their steps, accumulated.  The codes are decoded in place:
// (x & 0xF << 4n) | 0x4B000000 is the float 2^23 + (code+8) 16^n; subtracting 2^23 + 8*16^n leaves
// code * 16^n exactly, and the step was pre-divided by 16^n (an exact scaling), so
// fma(code*16^n, s/16^n, acc) rounds exactly like fma(code, s, acc).  Codes 0..3 are taken from the low
// half of the word, codes 4..7 from the word shifted down by 16, both at positions 0..3, so that four
// masks and two bias pairs serve all eight.  Subtractions and FMAs run two at a time (f32x2), one binary32
// rounding per element as before.
//
// Each code costs ONE logic instruction only if the mask and the exponent pattern are both register
// operands of an explicit lop3 ((x & mask) | magic, truth table 0xEA), and the packed subtract takes its
// bias pair from registers: the constants are made opaque to the compiler once per thread (DecodeConsts),
// which otherwise rebuilds them from immediates at every use.
struct DecodeConsts {
    uint32_t mask[4];  // 0xF << 4n
    uint32_t magic;    // 0x4B000000
    float2 bias[2];    // -(2^23 + 8 * 16^n) for positions (0,1) and (2,3)
};
__device__ __forceinline__ DecodeConsts decode_consts()
{
    DecodeConsts c;
    asm volatile("mov.u32 %0, 0xF;" : "=r"(c.mask[0]));
    asm volatile("mov.u32 %0, 0xF0;" : "=r"(c.mask[1]));
    asm volatile("mov.u32 %0, 0xF00;" : "=r"(c.mask[2]));
    asm volatile("mov.u32 %0, 0xF000;" : "=r"(c.mask[3]));
    asm volatile("mov.u32 %0, 0x4B000000;" : "=r"(c.magic));
    asm volatile("mov.f32 %0, 0fCB000008;" : "=f"(c.bias[0].x));  // -(2^23 + 8)
    asm volatile("mov.f32 %0, 0fCB000080;" : "=f"(c.bias[0].y));  // -(2^23 + 128)
    asm volatile("mov.f32 %0, 0fCB000800;" : "=f"(c.bias[1].x));  // -(2^23 + 2048)
    asm volatile("mov.f32 %0, 0fCB008000;" : "=f"(c.bias[1].y));  // -(2^23 + 32768)
    return c;
}
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t mask, uint32_t magic)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "r"(mask), "r"(magic));
    return d;
}

// FIRST: the accumulators start here, acc = code * step (what fma(code, step, +0) gives: a product that is
// zero has a +0 code, except at a hole's lane, whose step is 0 and whose sum is never kept).
template <bool FIRST = false>
__device__ __forceinline__ void decode8(uint32_t raw, const float2 (&sc)[4], float2 (&acc)[4], const DecodeConsts &c)
{
    const uint32_t xa = raw ^ 0x88888888u;
    const uint32_t xb = xa >> 16;
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const uint32_t x = (h < 2) ? xa : xb;
        const float f0 = __uint_as_float(and_or(x, c.mask[2 * (h & 1)], c.magic));
        const float f1 = __uint_as_float(and_or(x, c.mask[2 * (h & 1) + 1], c.magic));
        const float2 d = __fadd2_rn(make_float2(f0, f1), c.bias[h & 1]);
        acc[h] = FIRST ? __fmul2_rn(d, sc[h]) : __ffma2_rn(d, sc[h], acc[h]);
    }
}

// the steps of features 8g .. 8g+7 of device i, pre-divided by the power of 16 of their decode position
__device__ __forceinline__ void load_steps(const float *s_k_row, int g, float2 (&sc)[4])
{
    const float4 a = __ldg(reinterpret_cast<const float4 *>(s_k_row + 8 * g));
    const float4 b = __ldg(reinterpret_cast<const float4 *>(s_k_row + 8 * g + 4));
    const float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int h = 0; h < 4; ++h)
        sc[h] = make_float2(v[2 * h] * (1.0f / (float)(1 << (4 * dq_pos(2 * h)))),
                            v[2 * h + 1] * (1.0f / (float)(1 << (4 * dq_pos(2 * h + 1)))));
}

template <bool FP32OUT>
__device__ __forceinline__ void store_one(void *out, int64_t off, float v)
{
    if (FP32OUT)
        static_cast<float *>(out)[off] = v;
    else
        static_cast<__nv_bfloat16 *>(out)[off] = __float2bfloat16_rn(v);
}

// the 8 sums of a thread -> features o .. o+7 of the output row, skipping the selected ones
template <bool FP32OUT>
__device__ __forceinline__ void store_group(void *out, int64_t o, const float2 (&acc)[4], uint32_t mask)
{
    if (mask == 0) {
        if (FP32OUT) {
            float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(out) + o);
            __stcs(dst, make_float4(acc[0].x, acc[0].y, acc[1].x, acc[1].y));
            __stcs(dst + 1, make_float4(acc[2].x, acc[2].y, acc[3].x, acc[3].y));
        } else {
            uint32_t w[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                __nv_bfloat162 b = __floats2bfloat162_rn(acc[h].x, acc[h].y);
                w[h] = *reinterpret_cast<uint32_t *>(&b);
            }
            __stcs(reinterpret_cast<uint4 *>(static_cast<uint16_t *>(out) + o), make_uint4(w[0], w[1], w[2], w[3]));
        }
    } else {
        const float a8[8] = {acc[0].x, acc[0].y, acc[1].x, acc[1].y, acc[2].x, acc[2].y, acc[3].x, acc[3].y};
#pragma unroll
        for (int n = 0; n < 8; ++n)
            if (!(mask & (1u << n))) store_one<FP32OUT>(out, o + n, a8[n]);
    }
}

struct DXParams {           // extras shared by the tiled kernels
    const int32_t *hp_idx;  // [k]
    const int32_t *hole;    // [n_holes]
    const int32_t *filler;  // [n_holes]
    int n_holes;
    int *status;
};


// ----------------------------------------------------------------------------------------------
// Panel kernel (any N, any row length).  A block owns a panel of CG groups of 8 adjacent code slots and
// walks chunks of RC = RS*DP_R rows, RS = DP_THREADS / CG; thread <-> (group, DP_R rows).  A chunk is taken
// DP_NB devices at a time ("step").  The code words of a step -- one segment of CG words per (device, row),
// widened to a 16-byte aligned start -- are fetched by all threads together with 16-byte asynchronous
// copies into a ring of shared-memory stages, DP_STAGES-1 steps ahead of their use; one block barrier per
// step makes a landed stage visible and frees the stage consumed before it.  (A chunk starts on a 16-byte
// boundary of the code stream because RC is a multiple of 4, so the shift of a row inside its segment
// depends only on the row's place in the chunk.)  The panel's steps of all N devices IN SLOT ORDER,
// pre-divided for the in-place decode, live in shared memory ([N][2][CG] float4), so the register cost does
// not grow with N.  A hole's slot carries the filler feature's step, so its lane accumulates the filler
// feature's sum; every group is stored whole (8 lanes, one 128-bit store).  Item threads (one per row of the
// chunk and selected feature of the panel) add the devices' BF16 values in ascending order, a step's values
// loaded one step before they are used; after the next block barrier they move the filler's sum from the
// hole's column to the filler feature's own column and write the selected feature's sum over it.
// ----------------------------------------------------------------------------------------------
#ifndef TPQ_DP_THREADS
#define TPQ_DP_THREADS 512
#define TPQ_DP_NB 4
#define TPQ_DP_STAGES 4
#endif
constexpr int DP_THREADS = TPQ_DP_THREADS;
constexpr int DP_R = 4;                   // rows per thread (a multiple of 4: see above)
constexpr int DP_NB = TPQ_DP_NB;          // devices per step
constexpr int DP_STAGES = TPQ_DP_STAGES;  // ring depth (steps)

struct DPParams {
    DQParams q;
    const float *s_slot;    // [N][E] slot-order steps
    const int32_t *lp_idx;  // [E-k] feature of each slot
    const int32_t *hp_idx;  // [k]
    const int32_t *filler;  // [n_holes] feature whose codes sit in hole tau's slot
    int n_holes;
    int CG, panels, gy;
    int64_t n_chunks;
};

__host__ __device__ inline size_t dp_steps_bytes(int N, int CG) { return (size_t)N * CG * 32; }
__host__ __device__ inline size_t dp_stage_bytes(int CG)
{
    return (size_t)DP_NB * (DP_THREADS / CG * DP_R) * (CG / 4 + 1) * 16;
}
__host__ __device__ inline size_t dp_smem_bytes(int N, int CG)
{
    return dp_steps_bytes(N, CG) + (size_t)DP_STAGES * dp_stage_bytes(CG);
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory");
}

// a thread's DP_R rows of sums -> the output; lane n of a hole's slot holds the sum of the filler feature
// lp_idx[8g+n] and goes to that feature's column
template <bool FP32OUT>
__device__ __forceinline__ void dp_store_rows(const DQParams &p, const int32_t *lp_idx, int64_t t0, int64_t t_lim, int g,
                                              uint32_t mask, const float2 (&acc_in)[DP_R][4])
{
    float2 acc[DP_R][4];
#pragma unroll
    for (int r = 0; r < DP_R; ++r)
#pragma unroll
        for (int h = 0; h < 4; ++h) acc[r][h] = acc_in[r][h];
    if (p.bias) {
        // lane n belongs to feature 8g+n, or, at a hole, to the filler feature whose codes sit in the slot
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g + 4));
        float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
        const uint32_t holes = __ldg(p.grp + g) & 0xFFu;
        if (holes) {
#pragma unroll
            for (int n = 0; n < 8; ++n)
                if (holes & (1u << n)) b[n] = __ldg(p.bias + __ldg(lp_idx + 8 * g + n));
        }
#pragma unroll
        for (int r = 0; r < DP_R; ++r)
#pragma unroll
            for (int h = 0; h < 4; ++h)
                acc[r][h] = __fadd2_rn(acc[r][h], make_float2(b[2 * h], b[2 * h + 1]));
    }
    if (mask == 0) {
#pragma unroll
        for (int r = 0; r < DP_R; ++r)
            if (t0 + r < t_lim) store_group<FP32OUT>(p.out, (t0 + r) * p.out_stride + 8 * (int64_t)g, acc[r], 0u);
    } else {
        int col[8];
#pragma unroll
        for (int n = 0; n < 8; ++n) col[n] = (mask & (1u << n)) ? __ldg(lp_idx + 8 * g + n) : 8 * g + n;
#pragma unroll
        for (int r = 0; r < DP_R; ++r)
            if (t0 + r < t_lim) {
                const int64_t orow = (t0 + r) * p.out_stride;
                const float a8[8] = {acc[r][0].x, acc[r][0].y, acc[r][1].x, acc[r][1].y,
                                     acc[r][2].x, acc[r][2].y, acc[r][3].x, acc[r][3].y};
#pragma unroll
                for (int n = 0; n < 8; ++n) store_one<FP32OUT>(p.out, orow + col[n], a8[n]);
            }
    }
}

template <int CG, bool FP32OUT, bool HAS_WAIT>
__global__ void __launch_bounds__(DP_THREADS, 1) dequant_panels(const DPParams pp)
{
    extern __shared__ __align__(128) uint8_t dp_smem[];
    constexpr int RS = DP_THREADS / CG, RC = RS * DP_R;
    constexpr int SEGC = CG / 4 + 1;          // 16-byte pieces per segment
    constexpr int SEGW = SEGC * 4;            // words per segment
    constexpr int PIECES = DP_NB * RC * SEGC; // pieces per step
    constexpr int NCP = (PIECES + DP_THREADS - 1) / DP_THREADS;
    constexpr uint32_t STAGE_BYTES = PIECES * 16;
    static_assert(RC % 4 == 0, "a chunk must start on a 16-byte boundary of the code stream");

    const DQParams &p = pp.q;
    const int N = p.N, E = p.E, k = p.k, L8 = (E - k) >> 3;
    const int tid = threadIdx.x;
    float4 *const dp_steps = reinterpret_cast<float4 *>(dp_smem);  // [N][2][CG]
    if constexpr (HAS_WAIT) {  // (first thing, with no load of its own in flight; an instantiation of its own)
        tpq_block_wait_arrivals(p.arr);
        __syncthreads();
    }
    const int panel = blockIdx.x % pp.panels, by = blockIdx.x / pp.panels;
    const int cg = tid & (CG - 1), rs = tid / CG;
    const int g = panel * CG + cg;
    const bool live = g < L8;
    const int nbatch = (N + DP_NB - 1) / DP_NB;
    const int64_t chunk_bytes = (int64_t)RC * L8 * 4;  // code bytes of one device in a chunk of rows
    uint8_t *const ring = dp_smem + dp_steps_bytes(N, CG);
    const uint32_t ring_s = smem_u32(ring);

    // copy side: piece c = tid + j * DP_THREADS of a step is piece `within` of segment (device i, row) and
    // lands at byte 16 c of the stage; its source offset inside the chunk does not depend on the chunk
    uint32_t cp_goff[NCP];  // source byte offset inside the device's chunk
    int cp_dev[NCP];        // device within the step; -1: no such piece
#pragma unroll
    for (int j = 0; j < NCP; ++j) {
        const int c = tid + j * DP_THREADS;
        const int seg = c / SEGC, within = c - seg * SEGC;
        const int i = seg / RC, row = seg - i * RC;
        cp_dev[j] = (c < PIECES) ? i : -1;
        cp_goff[j] = (((uint32_t)row * (uint32_t)L8 + (uint32_t)panel * CG) * 4u & ~15u) + (uint32_t)within * 16u;
    }
    int64_t ich = by;
    int ib = 0;
    uint32_t idst = ring_s + (uint32_t)tid * 16u;
    auto issue = [&]() {
        if (ich < pp.n_chunks) {
            const int64_t cbase = ich * chunk_bytes;
            const int64_t left = p.lp_bytes - cbase;  // bytes of the code section from the chunk's start on
            const uint32_t lim = (uint32_t)(left < (int64_t)0x7FFFFFF0 ? left : (int64_t)0x7FFFFFF0);
            const int i0 = ib * DP_NB;
#pragma unroll
            for (int j = 0; j < NCP; ++j) {
                // pieces past the end of the code section (rows past the end, the last panel's overhang) and
                // devices past N are skipped; what they would have filled is never stored
                if (cp_dev[j] >= 0 && i0 + cp_dev[j] < N && cp_goff[j] + 16u <= lim)
                    cp_async16(idst + (uint32_t)(j * DP_THREADS * 16), p.pl[i0 + cp_dev[j]] + cbase + cp_goff[j]);
            }
            if (++ib == nbatch) {
                ib = 0;
                ich += pp.gy;
            }
            idst += STAGE_BYTES;
            if (idst == ring_s + (uint32_t)tid * 16u + DP_STAGES * STAGE_BYTES) idst = ring_s + (uint32_t)tid * 16u;
        }
        cp_async_commit();  // (possibly empty: keeps the group count in step with the consumer)
    };
    tpq_grid_dep_wait();    // the payloads and the output buffer may still be in use by the kernel ahead
    tpq_grid_dep_launch();  // the next kernel in the stream may start its own prologue
#pragma unroll
    for (int s = 0; s < DP_STAGES - 1; ++s) issue();

    for (int a = tid; a < N * CG; a += DP_THREADS) {
        const int i = a / CG, c = a & (CG - 1), gg = panel * CG + c;
        float2 s4[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) s4[h] = make_float2(0.0f, 0.0f);
        if (gg < L8) load_steps(pp.s_slot + (size_t)i * E, gg, s4);
        dp_steps[(2 * i) * CG + c] = make_float4(s4[0].x, s4[0].y, s4[1].x, s4[1].y);
        dp_steps[(2 * i + 1) * CG + c] = make_float4(s4[2].x, s4[2].y, s4[3].x, s4[3].y);
    }
    const DecodeConsts dc = decode_consts();

    // consume side: word of (device i of the step, this thread's row r) inside a stage
    int wofs[DP_R];
#pragma unroll
    for (int r = 0; r < DP_R; ++r) {
        const int rowc = rs * DP_R + r;
        wofs[r] = rowc * SEGW + (int)(((uint32_t)rowc * (uint32_t)L8 + (uint32_t)panel * CG) & 3u) + (live ? cg : 0);
    }
    const float4 *const my_steps = dp_steps + cg;
    const uint32_t *const ring_w = reinterpret_cast<const uint32_t *>(ring);
    const uint32_t *sw = ring_w;

    // Selected features completed by this block ("items", one per row and rank): the panel's holes, ranks
    // [hs, he); the last panel also takes the selected features at or above E-k, ranks [n_holes, k).
    // Threads store all 8 lanes of every group; a hole's lane holds the sum of the filler feature whose
    // codes sit in the hole's slot.  After the next block barrier (which orders the two stores to the hole's
    // column) the item thread moves that value to the filler feature's column and writes the selected
    // feature's own sum -- the devices' BF16 values added in ascending order -- over it.
    const int n_holes = pp.n_holes;
    const int hs = (int)(__ldg(p.grp + panel * CG) >> 8);
    const int he = (panel == pp.panels - 1) ? k : (int)(__ldg(p.grp + (panel + 1) * CG) >> 8);
    const int n_it = he - hs;                           // items per row
    const int items = RC * n_it;
    const int my_r = (tid < items) ? tid / n_it : 0;    // this thread's first item: row of the chunk, rank
    const int my_h = (tid < items) ? hs + (tid - my_r * n_it) : 0;
    const int my_col = (tid < items) ? __ldg(pp.hp_idx + my_h) : 0;
    const int my_fcol = (tid < items && my_h < n_holes) ? __ldg(pp.filler + my_h) : -1;
    auto item_done = [&](int64_t t, int sel_col, int filler_col, float v) {
        const int64_t orow = t * p.out_stride;
        if (filler_col >= 0) {
            if (FP32OUT)
                static_cast<float *>(p.out)[orow + filler_col] = __ldcg(static_cast<const float *>(p.out) + orow + sel_col);
            else
                static_cast<uint16_t *>(p.out)[orow + filler_col] =
                    __ldcg(static_cast<const uint16_t *>(p.out) + orow + sel_col);
        }
        store_one<FP32OUT>(p.out, orow + sel_col, p.bias ? __fadd_rn(v, __ldg(p.bias + sel_col)) : v);
    };
    // the items of the chunk whose first row is tcp: this thread's pipelined one (sum v) and, in panels with
    // more items than threads, the rest
    // The pipelined item only issues its read of the hole's column here; both of its stores follow a step
    // later (flush), when the value has arrived.  (A store to the hole's column right behind the read of the
    // same address stalls the memory pipe of the whole SM until the read is done: measured 60 % slower.)
    bool fl_on = false;
    float fl_f = 0.0f, fl_v = 0.0f;
    int64_t fl_row = 0;
    auto flush = [&]() {
        if (fl_on) {
            if (my_fcol >= 0) {
                if (FP32OUT)
                    static_cast<float *>(p.out)[fl_row + my_fcol] = fl_f;
                else
                    static_cast<uint16_t *>(p.out)[fl_row + my_fcol] = (uint16_t)__float_as_uint(fl_f);
            }
            store_one<FP32OUT>(p.out, fl_row + my_col, p.bias ? __fadd_rn(fl_v, __ldg(p.bias + my_col)) : fl_v);
            fl_on = false;
        }
    };
    auto fixup = [&](int64_t tcp, bool on, float v) {
        if (on) {
            fl_row = (tcp + my_r) * p.out_stride;
            if (my_fcol >= 0) {
                if (FP32OUT)
                    fl_f = __ldcg(static_cast<const float *>(p.out) + fl_row + my_col);
                else
                    fl_f = __uint_as_float((uint32_t)__ldcg(static_cast<const uint16_t *>(p.out) + fl_row + my_col));
            }
            fl_v = v;
            fl_on = true;
        }
        for (int a = tid + DP_THREADS; a < items; a += DP_THREADS) {
            const int r = a / n_it, h = hs + (a - r * n_it);
            if (tcp + r >= p.T) break;
            const int64_t off = p.lp_bytes + ((tcp + r) * k + h) * 2;
            float u = 0.0f;
            for (int i = 0; i < N; ++i)
                u = __fadd_rn(u, __uint_as_float((uint32_t)__ldcs(reinterpret_cast<const uint16_t *>(p.pl[i] + off)) << 16));
            item_done(tcp + r, __ldg(pp.hp_idx + h), h < n_holes ? __ldg(pp.filler + h) : -1, u);
        }
    };
    bool pend = false, pend_on = false;
    float pend_v = 0.0f;
    int64_t pend_tc = 0;

    for (int64_t ch = by; ch < pp.n_chunks; ch += pp.gy) {
        const int64_t tc = ch * RC;
        const int64_t t0 = tc + rs * DP_R;
        const bool it_on = tid < items && tc + my_r < p.T;
        const int64_t it_off = p.lp_bytes + ((tc + my_r) * k + my_h) * 2;
        float hv = 0.0f;
        uint16_t hvv[DP_NB] = {};
        float2 acc[DP_R][4];
#pragma unroll
        for (int r = 0; r < DP_R; ++r)
#pragma unroll
            for (int h = 0; h < 4; ++h) acc[r][h] = make_float2(0.0f, 0.0f);
        const float4 *st4 = my_steps;
        for (int i0 = 0; i0 < N; i0 += DP_NB, st4 += DP_NB * 2 * CG) {
            cp_async_wait<DP_STAGES - 2>();  // this thread's pieces of the step have landed ...
            __syncthreads();                 // ... and everybody's; the stage consumed last is free
            issue();
            flush();
            if (pend) {  // (first step of a chunk) the barrier above is also behind the previous chunk's row stores
                if (n_it > 0) fixup(pend_tc, pend_on, pend_v);
                pend = false;
            }
            if (it_on) {
                // add the values loaded a step ago (ascending device order), then load this step's
                if (i0 > 0) {
#pragma unroll
                    for (int i = 0; i < DP_NB; ++i) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
                }
#pragma unroll
                for (int i = 0; i < DP_NB; ++i)
                    if (i0 + i < N) hvv[i] = __ldcs(reinterpret_cast<const uint16_t *>(p.pl[i0 + i] + it_off));
            }
            uint32_t w[DP_NB][DP_R];
#pragma unroll
            for (int i = 0; i < DP_NB; ++i)
#pragma unroll
                for (int r = 0; r < DP_R; ++r) w[i][r] = sw[i * RC * SEGW + wofs[r]];
            sw += STAGE_BYTES / 4;
            if (sw == ring_w + DP_STAGES * (STAGE_BYTES / 4)) sw = ring_w;
            if (i0 + DP_NB <= N) {
#pragma unroll
                for (int i = 0; i < DP_NB; ++i) {
                    const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                    const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                          make_float2(b.z, b.w)};
#pragma unroll
                    for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], dc);
                }
            } else {
#pragma unroll
                for (int i = 0; i < DP_NB; ++i)
                    if (i0 + i < N) {
                        const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                        const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                              make_float2(b.z, b.w)};
#pragma unroll
                        for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], dc);
                    }
            }
        }
        if (it_on) {  // the last step's values (a partial batch has N % DP_NB of them)
            const int nl = N - (N - 1) / DP_NB * DP_NB;
#pragma unroll
            for (int i = 0; i < DP_NB; ++i)
                if (i < nl) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
        }
        if (live) dp_store_rows<FP32OUT>(p, pp.lp_idx, t0, p.T, g, 0u, acc);
        pend = true;
        pend_on = it_on;
        pend_v = hv;
        pend_tc = tc;
    }
    cp_async_wait<0>();
    flush();
    if (pend) {
        __syncthreads();
        if (n_it > 0) fixup(pend_tc, pend_on, pend_v);
        flush();
    }
}

// ----------------------------------------------------------------------------------------------
// Tensor-map panel kernel (N <= DT_MAX_DEV devices, row pitch a multiple of 16 bytes).
//
// Same division of work as the panel kernel above, but the code words arrive through the tensor copy
// engine: each device's code section is a 2-D tensor of 32-bit words ((E-k)/8 words x T rows), and one
// tiled copy per device and step brings a box of CG words x RC rows into a shared-memory stage, signalling
// a "full" mbarrier.  A producer warp (one elected lane) issues the copies; main warps free a stage through
// the "empty" mbarrier as soon as its words are in registers.  Rows past T and words past the row end are
// zero-filled by the copy engine (their sums are never stored).  Every wait is bounded: on expiry the
// kernel sets the status word and returns.
// ----------------------------------------------------------------------------------------------
constexpr int DT_MAX_DEV = 16;
constexpr int DT_MAIN = 512;
constexpr int DT_THREADS = DT_MAIN + 32;
constexpr int DT_NB = 4;      // devices per stage

struct alignas(64) DTMaps {
    CUtensorMap m[DT_MAX_DEV];
};

struct DTParams {
    DPParams d;
    int nstage;
    int g0;  // rows after which the code stream is 16-byte aligned again (1, 2 or 4)
    int tail_rows;  // T mod g0: rows after the last whole group, which the tensor map does not cover
    int *status;
};

// Rows whose length is not a multiple of 16 bytes ((E-k)/8 not a multiple of 4): g0 = 2 or 4 adjacent rows
// are one row of the tensor map, so row class c (row index modulo g0) of a panel starts c*(E-k)/8 words into
// it, rounded down to a multiple of 4 words (the copy's 16-byte rule); the box is 4 words wider, and a thread
// reads its word (c*(E-k)/8 mod 4) words further on.  A device's part of a stage holds the g0 classes one
// after the other, each padded to the 128 bytes the copy's destination must be aligned to.  The T mod g0 rows
// after the last whole group are a chunk of their own (the last one), whose words come by one plain bulk copy
// per device and row, from the same 16-byte aligned places.
__host__ __device__ constexpr uint32_t dt_class_bytes(int CG, int g0)
{
    return ((uint32_t)(CG + (g0 > 1 ? 4 : 0)) * (uint32_t)(DT_MAIN / CG * DP_R / g0) * 4u + 127u) & ~127u;
}
__host__ __device__ constexpr size_t dt_stage_bytes(int CG, int g0) { return (size_t)DT_NB * g0 * dt_class_bytes(CG, g0); }
__host__ __device__ inline size_t dt_smem_bytes(int N, int CG, int nstage, int g0)
{
    return dp_steps_bytes(N, CG) + (size_t)nstage * dt_stage_bytes(CG, g0) + (size_t)nstage * 16;  // steps, ring, mbarriers
}


template <int CG, int G0, int M4, bool FP32OUT>
__global__ void __launch_bounds__(DT_THREADS, 1) dequant_tpanels(const DTParams tp, const __grid_constant__ DTMaps maps)
{
    extern __shared__ __align__(128) uint8_t dp_smem[];
    constexpr int RS = DT_MAIN / CG, RC = RS * DP_R;
    constexpr int CGW = CG + (G0 > 1 ? 4 : 0);                          // words of a box row
    constexpr uint32_t CLS_BYTES = dt_class_bytes(CG, G0);              // a row class of a device
    constexpr uint32_t COPY_BYTES = (uint32_t)CGW * (RC / G0) * 4;      // what one copy brings
    constexpr uint32_t BOX_BYTES = G0 * CLS_BYTES;                      // a device's part of a stage
    constexpr uint32_t STAGE_BYTES = DT_NB * BOX_BYTES;
    // word offset of a thread's row r (0 <= r < DP_R) inside a device's part, relative to its row 0 of class 0
    auto row_off = [](int r) constexpr {
        return (r % G0) * (int)(CLS_BYTES / 4) + (r / G0) * CGW + ((r % G0) * M4) % 4;
    };
    const DPParams &pp = tp.d;
    const DQParams &p = pp.q;
    const int N = p.N, E = p.E, k = p.k, L8 = (E - k) >> 3;
    const int tid = threadIdx.x, nstage = tp.nstage;
    const int lane = tid & 31;
    float4 *const dp_steps = reinterpret_cast<float4 *>(dp_smem);  // [N][2][CG]
    uint8_t *const ring = dp_smem + dp_steps_bytes(N, CG);
    uint64_t *full = reinterpret_cast<uint64_t *>(ring + (size_t)nstage * STAGE_BYTES);
    uint64_t *empty = full + nstage;

    // Work items are (panel, chunk) pairs, panel-major; the blocks take equal contiguous runs of them, so a
    // block works on one panel, or on the end of one and the start of the next ("segments").
    const int64_t total = (int64_t)pp.panels * pp.n_chunks;
    int64_t f0 = total * blockIdx.x / gridDim.x, f1 = total * (blockIdx.x + 1) / gridDim.x;
    // or (gy > 0): a block keeps one panel and takes every gy-th chunk of it, so that at any time the blocks
    // of the different panels read the same rows (whole rows of the code stream between them)
    const int cstep = pp.gy > 0 ? pp.gy : 1;
    if (pp.gy > 0) {
        f0 = (int64_t)(blockIdx.x % pp.panels) * pp.n_chunks + blockIdx.x / pp.panels;
        f1 = (int64_t)(blockIdx.x % pp.panels + 1) * pp.n_chunks;
        if (blockIdx.x / pp.panels >= pp.n_chunks) f0 = f1;
    }

    tpq_block_wait_arrivals(p.arr);  // (first thing, with no load of its own in flight; a barrier follows)
    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), DT_MAIN / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    const int cg = tid & (CG - 1), rs = tid / CG;
    const DecodeConsts dc = decode_consts();
    const float4 *const my_steps = dp_steps + cg;
    const uint32_t *const ring_w = reinterpret_cast<const uint32_t *>(ring) + (rs * DP_R / G0) * CGW + cg;
    // ring state: the producer lane and the main warps walk the same sequence of stages across segments
    int st = 0, it = 0;
    uint32_t parity = (tid >= DT_MAIN) ? 1u : 0u;  // producer: parity of the "empty" phase to wait for
    bool dead = false;  // a wait of this thread ran out (TPQ_ERR_TIMEOUT is recorded)

    for (int64_t f = f0; f < f1;) {
        const int panel = (int)(f / pp.n_chunks);
        const int64_t chb = f - (int64_t)panel * pp.n_chunks;
        const int64_t che = (pp.n_chunks - chb < f1 - f) ? pp.n_chunks : chb + (f1 - f);
        __syncthreads();  // (the previous segment's steps are no longer read; first time: the barriers exist)
        // the panel's steps (loads issued before the barrier that releases the producer)
        for (int a = tid; a < N * CG; a += DT_THREADS) {
            const int i = a / CG, c = a & (CG - 1), gg = panel * CG + c;
            float2 s4[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) s4[h] = make_float2(0.0f, 0.0f);
            if (gg < L8) load_steps(pp.s_slot + (size_t)i * E, gg, s4);
            dp_steps[(2 * i) * CG + c] = make_float4(s4[0].x, s4[0].y, s4[1].x, s4[1].y);
            dp_steps[(2 * i + 1) * CG + c] = make_float4(s4[2].x, s4[2].y, s4[3].x, s4[3].y);
        }
        const int g = panel * CG + cg;
        const bool live = tid < DT_MAIN && g < L8;
        if (f == f0) tpq_grid_dep_wait();  // the payloads and the output buffer may still be in use by the kernel ahead
        __syncthreads();
        if (f == f0) tpq_grid_dep_launch();  // the next kernel in the stream may start its own prologue

        if (tid >= DT_MAIN) {
            // ---------------- producer warp: one lane issues everything
            if (tid == DT_MAIN) {
                for (int64_t ch = chb; ch < che; ch += cstep) {
                    for (int i0 = 0; i0 < N; i0 += DT_NB, ++it) {
                        const int nb = (N - i0 < DT_NB) ? N - i0 : DT_NB;
                        const uint32_t bar = smem_u32(&full[st]);
                        if (it >= nstage && !dead && !mbar_wait(smem_u32(&empty[st]), parity)) {
                            atomicExch(tp.status, (int)TPQ_ERR_TIMEOUT);
                            dead = true;  // nothing more is issued; the loops go on so that every barrier is still met
                        }
                        const uint32_t stage = smem_u32(ring + (size_t)st * STAGE_BYTES);
                        if (G0 > 1 && tp.tail_rows > 0 && ch == pp.n_chunks - 1) {
                            // the rows after the last whole group: row (= class) cl of the chunk, first box row
                            if (!dead) {
                                const int64_t row_bytes = (int64_t)L8 * 4, t_tail = p.T - tp.tail_rows;
                                uint32_t bytes[G0 > 1 ? G0 : 1];
                                uint32_t sum = 0;
                                for (int cl = 0; cl < tp.tail_rows; ++cl) {
                                    // from the class's aligned start to the end of the box row or of the code rows (padded to 16 bytes)
                                    const int64_t from = (t_tail + cl) * row_bytes + (int64_t)(panel * CG - (cl * M4) % 4) * 4;
                                    const int64_t end = (p.T * row_bytes + 15) & ~(int64_t)15;
                                    bytes[cl] = (uint32_t)(end - from < (int64_t)CGW * 4 ? end - from : (int64_t)CGW * 4);
                                    sum += bytes[cl];
                                }
                                mbar_expect_tx(bar, (uint32_t)nb * sum);
                                for (int i = 0; i < nb; ++i)
                                    for (int cl = 0; cl < tp.tail_rows; ++cl)
                                        bulk_g2s(stage + (uint32_t)i * BOX_BYTES + (uint32_t)cl * CLS_BYTES,
                                                 p.pl[i0 + i] + (t_tail + cl) * row_bytes + (int64_t)(panel * CG - (cl * M4) % 4) * 4,
                                                 bytes[cl], bar);
                            }
                        } else if (!dead) {
                            mbar_expect_tx(bar, (uint32_t)nb * G0 * COPY_BYTES);
                            for (int i = 0; i < nb; ++i)
#pragma unroll
                                for (int cl = 0; cl < G0; ++cl)
                                    tma_load_2d(stage + (uint32_t)i * BOX_BYTES + (uint32_t)cl * CLS_BYTES, &maps.m[i0 + i],
                                                cl * L8 + panel * CG - (cl * M4) % 4, (int)(ch * (RC / G0)), bar);
                        }
                        if (++st == nstage) {
                            st = 0;
                            parity ^= 1u;
                        }
                    }
                }
            }
            f += che - chb;
            continue;
        }

        // ---------------- main warps
        // Selected features completed for this panel ("items", one per row and rank): the panel's holes,
        // ranks [hs, he); the last panel also takes the selected features at or above E-k, ranks [n_holes, k).
        // Main threads store all 8 lanes of every group; a hole's lane holds the sum of the filler feature
        // whose codes sit in the hole's slot.  After a barrier among the main warps (which orders the two
        // stores to the hole's column) the item thread moves that value to the filler feature's column and
        // writes the selected feature's own sum -- the devices' BF16 values added in ascending order -- over it.
        const int n_holes = pp.n_holes;
        const int hs = (int)(__ldg(p.grp + panel * CG) >> 8);
        const int he = (panel == pp.panels - 1) ? k : (int)(__ldg(p.grp + (panel + 1) * CG) >> 8);
        const int n_it = he - hs;                           // items per row
        const int items = RC * n_it;
        const int my_r = (tid < items) ? tid / n_it : 0;    // this thread's first item: row of the chunk, rank
        const int my_h = (tid < items) ? hs + (tid - my_r * n_it) : 0;
        const int my_col = (tid < items) ? __ldg(pp.hp_idx + my_h) : 0;
        const int my_fcol = (tid < items && my_h < n_holes) ? __ldg(pp.filler + my_h) : -1;
        auto item_done = [&](int64_t t, int sel_col, int filler_col, float v) {
            const int64_t orow = t * p.out_stride;
            if (filler_col >= 0) {
                if (FP32OUT)
                    static_cast<float *>(p.out)[orow + filler_col] =
                        __ldcg(static_cast<const float *>(p.out) + orow + sel_col);
                else
                    static_cast<uint16_t *>(p.out)[orow + filler_col] =
                        __ldcg(static_cast<const uint16_t *>(p.out) + orow + sel_col);
            }
            store_one<FP32OUT>(p.out, orow + sel_col, p.bias ? __fadd_rn(v, __ldg(p.bias + sel_col)) : v);
        };

        for (int64_t ch = chb; ch < che; ch += cstep) {
            // (the chunk after the last whole group of g0 rows starts right there)
            const bool tail = G0 > 1 && tp.tail_rows > 0 && ch == pp.n_chunks - 1;
            const int64_t tc = tail ? p.T - tp.tail_rows : ch * RC;
            const int64_t t_lim = tail ? p.T : p.T - (G0 > 1 ? tp.tail_rows : 0);  // (the maps' rows end at the last whole group)
            const int64_t t0 = tc + rs * DP_R;
            float2 acc[DP_R][4];
#pragma unroll
            for (int r = 0; r < DP_R; ++r)
#pragma unroll
                for (int h = 0; h < 4; ++h) acc[r][h] = make_float2(0.0f, 0.0f);
            const bool it_on = tid < items && tc + my_r < t_lim;
            const int64_t it_off = p.lp_bytes + ((tc + my_r) * k + my_h) * 2;
            float hv = 0.0f;
            uint16_t hvv[DT_NB] = {};
            const float4 *st4 = my_steps;
            for (int i0 = 0; i0 < N; i0 += DT_NB, st4 += DT_NB * 2 * CG) {
                if (it_on) {
                    // add the values loaded a step ago (ascending device order), then load this step's
                    if (i0 > 0) {
#pragma unroll
                        for (int i = 0; i < DT_NB; ++i) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
                    }
#pragma unroll
                    for (int i = 0; i < DT_NB; ++i)
                        if (i0 + i < N) hvv[i] = __ldcs(reinterpret_cast<const uint16_t *>(p.pl[i0 + i] + it_off));
                }
                if (!dead && !mbar_wait(smem_u32(&full[st]), parity)) {
                    atomicExch(tp.status, (int)TPQ_ERR_TIMEOUT);
                    dead = true;  // no more waits and no more stores; the loops go on so that every barrier is still met
                }
                const uint32_t *const sw = ring_w + (size_t)st * (STAGE_BYTES / 4);
                uint32_t w[DT_NB][DP_R];
#pragma unroll
                for (int i = 0; i < DT_NB; ++i)
#pragma unroll
                    for (int r = 0; r < DP_R; ++r) w[i][r] = sw[i * (int)(BOX_BYTES / 4) + row_off(r)];
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&empty[st]));  // the stage's words are in registers
                if (++st == nstage) {
                    st = 0;
                    parity ^= 1u;
                }
                if (i0 + DT_NB <= N) {
#pragma unroll
                    for (int i = 0; i < DT_NB; ++i) {
                        const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                        const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                              make_float2(b.z, b.w)};
#pragma unroll
                        for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], dc);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < DT_NB; ++i)
                        if (i0 + i < N) {
                            const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                            const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                                  make_float2(b.z, b.w)};
#pragma unroll
                            for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], dc);
                        }
                }
            }
            if (it_on) {  // the last step's values (a partial batch has N % DT_NB of them)
                const int nl = N - (N - 1) / DT_NB * DT_NB;
#pragma unroll
                for (int i = 0; i < DT_NB; ++i)
                    if (i < nl) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
            }
            if (live && !dead) dp_store_rows<FP32OUT>(p, pp.lp_idx, t0, t_lim, g, 0u, acc);
            if (n_it > 0) {
                asm volatile("bar.sync 1, %0;" ::"n"(DT_MAIN) : "memory");  // the chunk's rows are stored
                if (it_on && !dead) item_done(tc + my_r, my_col, my_fcol, hv);
                // panels with more items than threads (many selected features in one panel): the rest, unpipelined
                for (int a = tid + DT_MAIN; a < items && !dead; a += DT_MAIN) {
                    const int r = a / n_it, h = hs + (a - r * n_it);
                    if (tc + r >= t_lim) break;
                    const int64_t off = p.lp_bytes + ((tc + r) * k + h) * 2;
                    float v = 0.0f;
                    for (int i = 0; i < N; ++i)
                        v = __fadd_rn(v, __uint_as_float((uint32_t)__ldcs(reinterpret_cast<const uint16_t *>(p.pl[i] + off)) << 16));
                    item_done(tc + r, __ldg(pp.hp_idx + h), h < n_holes ? __ldg(pp.filler + h) : -1, v);
                }
            }
        }
        f += che - chb;
    }
}

// ----------------------------------------------------------------------------------------------
// Row kernel for N <= 8 devices and (E-k)/8 <= MAXT main threads.
//
// One persistent block per SM works on a run of adjacent rows, G at a time, with three kinds of warps:
//   producer (1 warp)  sets up the barriers, waits for the kernel ahead in the stream and streams the
//                      stages (a code-row block and a BF16 block per device, 2N 1-D bulk asynchronous
//                      copies issued by 2N lanes) into a ring of shared-memory stages; "full" mbarriers;
//   main (MAXT/32)     thread <-> 8 adjacent output features = one aligned word per device and row; the
//                      8 steps of every device live in registers for the life of the block (0 at holes);
//                      straight-line decode + one 128-bit store per row.  A thread whose group contains a
//                      selected feature then overwrites that lane of its own stores (same thread, same
//                      address: ordered) with the sum the auxiliary warps left in shared memory;
//   auxiliary (3 or 5) per stage, from shared memory only: (1) the sums of the devices' BF16 values of every
//                      (row, selected feature), left in shared memory in the output's format ("sums"
//                      barrier); (2) the last k columns of the output, which no main thread covers: an
//                      unselected one is a filler feature, decoded from the hole's slot that carries its
//                      codes, a selected one takes its sum; lane <-> column, so the small stores of a warp
//                      are adjacent.
// No warp ever waits for another one's global stores, and no block-wide barrier follows the prologue.
// Blocks and stages start on rows at which the code stream is 16-byte aligned (multiples of 4/gcd(4, L/8)).
//
// Up to four devices (NMAX = 4) a block has a main thread for every group of the row.  With five to eight
// (NMAX = the device count, 40 to 64 registers of steps per thread) the register file holds half as many
// threads, so two blocks (on two SMs) share a run of rows: both stage the whole rows, each decodes one half
// of the groups, adds up the selected features its own main threads overwrite and stores one half of the
// last k columns; its auxiliary threads take one item (a sum or a column) each and, where they outnumber the
// items, several rows of a stage side by side.
// ----------------------------------------------------------------------------------------------
constexpr int DR_AUX = 96;          // auxiliary threads
constexpr int DR_PREFETCH_ROWS = 4; // rows whose bytes a block asks L2 for ahead of the dependency wait (measured: 2..8 alike, all: worse)

// main threads (= 32-bit words of a code row a stage leaves room for) for a row of L8 words
__host__ __device__ inline int dr_row_cap(int L8) { return L8 <= 640 ? 640 : 768; }

struct DRLayout {
    size_t lp_stage, hp_stage, stage, sums, sums_stage, bars, total;
};
__host__ __device__ inline DRLayout dr_layout(int N, int E, int k, int G, int nstage)
{
    DRLayout l;
    // a device's code rows of a stage start at a stride that depends on G only (the widest row the main
    // threads cover), so that the main loop addresses them with immediate offsets
    l.lp_stage = (size_t)G * dr_row_cap((E - k) >> 3) * 4;
    l.hp_stage = (size_t)G * k * 2;
    l.stage = (size_t)N * (l.lp_stage + l.hp_stage);
    l.sums = (size_t)nstage * l.stage;
    l.sums_stage = (((size_t)G * k * 4) + 15) & ~(size_t)15;  // one 32-bit slot per (row, rank)
    l.bars = l.sums + (size_t)nstage * l.sums_stage;
    l.total = l.bars + (size_t)nstage * 24;
    return l;
}

struct DRParams {
    DQParams q;
    DXParams x;
    int G, nstage;
    int first;               // rows of a block's first stage (<= G: a short first stage lands sooner)
    int pairs;               // main threads walk a stage two rows at a time in a rolled loop
    int half_groups;         // (more than four devices) groups per block: two blocks share a run of rows
    int64_t rows_per_block;  // a block works on rows_per_block adjacent rows (a multiple of the number of
                             // rows after which the code stream is 16-byte aligned again)
};

__device__ __forceinline__ uint32_t lds32(uint32_t saddr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t saddr)
{
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ void sts64(uint32_t saddr, uint32_t a, uint32_t b)
{
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(saddr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t saddr, uint32_t a)
{
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(saddr), "r"(a) : "memory");
}

// the bits an output element holds for the sum v
template <bool FP32OUT>
__device__ __forceinline__ uint32_t out_bits(float v)
{
    if (FP32OUT) return __float_as_uint(v);
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(v));
}
template <bool FP32OUT>
__device__ __forceinline__ void store_bits(uint8_t *ptr, uint32_t bits)
{
    if (FP32OUT)
        *reinterpret_cast<uint32_t *>(ptr) = bits;
    else
        *reinterpret_cast<uint16_t *>(ptr) = (uint16_t)bits;
}
// the code in bits [sh, sh+4) of w, as a float
__device__ __forceinline__ float code_at(uint32_t w, int sh)
{
    return __fsub_rn(__uint_as_float((((w >> sh) & 0xFu) ^ 8u) | 0x4B000000u), 8388616.0f);
}

// GR rows of a stage for one main thread.  sa: shared-memory address of its word of the first row of
// device 0; device i's copy of a row lies DEVSTEP bytes further on each (a compile-time constant, so the
// device's word is one load at an immediate offset; 0: dev_step, known at run time only); a row is
// row_bytes long.  NDEV > 0: the number of devices, known at compile time; 0: n (1 <= n <= NMAX) devices.
template <int NMAX, int NDEV, int GR, uint32_t DEVSTEP, bool FP32OUT, bool HAS_BIAS>
__device__ __forceinline__ void rows_stage(uint32_t sa, uint32_t dev_step, uint32_t row_bytes, int n,
                                           const float2 (&sc)[NMAX][4], const DecodeConsts &dc, const float2 (&b)[4],
                                           uint8_t *orow, int64_t out_row_bytes, bool live)
{
#pragma unroll
    for (int r = 0; r < GR; ++r) {
        float2 acc[4];
        decode8<true>(lds32(sa), sc[0], acc, dc);
#pragma unroll
        for (int i = 1; i < NMAX; ++i)
            if (NDEV ? i < NDEV : i < n) decode8(lds32(sa + (uint32_t)i * (DEVSTEP ? DEVSTEP : dev_step)), sc[i], acc, dc);
        sa += row_bytes;
        if (live) {
            if (HAS_BIAS) {  // (a hole's lane gets its own column's bias here and is overwritten below)
#pragma unroll
                for (int h = 0; h < 4; ++h) acc[h] = __fadd2_rn(acc[h], b[h]);
            }
            store_group<FP32OUT>(orow, 0, acc, 0u);
        }
        orow += out_row_bytes;
    }
}

// Marks a value loaded once per thread as opaque: without it the compiler, short of registers, drops the value
// and repeats its chain of (read-only) table loads at every use inside the stage loop, a trip to L2 each time.
__device__ __forceinline__ void keep(int &v) { asm volatile("" : "+r"(v)); }
__device__ __forceinline__ void keep(uint32_t &v) { asm volatile("" : "+r"(v)); }
__device__ __forceinline__ void keep(float &v) { asm volatile("" : "+f"(v)); }

// first row (within the block's run) of the block's it-th stage
__device__ __forceinline__ int dr_stage_row(int it, int first, int G) { return it == 0 ? 0 : first + (it - 1) * G; }

template <int NMAX, int ROWCAP, int MAXT, int DAUX, bool FP32OUT, bool HAS_BIAS, bool HAS_WAIT>
__global__ void __launch_bounds__(MAXT + DAUX + 32, 1) dequant_rows(const DRParams pp)
{
    constexpr bool SPLIT = NMAX > 4;  // two blocks share a run of rows, each decoding one half of the groups
    extern __shared__ __align__(128) uint8_t smem[];
    const DQParams &p = pp.q;
    const DXParams &x = pp.x;
    const int tid = threadIdx.x;
    // warp 0 is the producer, then the auxiliary warps, then the main warps: where several warps of a
    // scheduler can issue, the one launched first goes first, and the few instructions of the producer and of
    // the auxiliary warps must not wait behind the main warps' many (as last warps they took 3 us per stage)
    const int NT = blockDim.x - DAUX - 32;  // main threads
    const int N = p.N, E = p.E, k = p.k, G = pp.G, nstage = pp.nstage;
    const int L = E - k, L8 = L >> 3;
    const DRLayout lay = dr_layout(N, E, k, G, nstage);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + lay.bars);
    uint64_t *empty = full + nstage;
    uint64_t *sums_ready = empty + nstage;
    // this block's rows
    const int half = SPLIT ? (int)(blockIdx.x & 1u) : 0;
    const int64_t t_begin = (int64_t)(SPLIT ? blockIdx.x >> 1 : blockIdx.x) * pp.rows_per_block;
    const int64_t t_end = (p.T - t_begin < pp.rows_per_block) ? p.T : t_begin + pp.rows_per_block;
    const int rows_mine = (int)(t_end - t_begin);
    constexpr int ESIZE = FP32OUT ? 4 : 2;
    const int64_t out_row_bytes = p.out_stride * ESIZE;
    const uint32_t smem_s = smem_u32(smem);
    const uint32_t stage_b = (uint32_t)lay.stage, lp_b = (uint32_t)lay.lp_stage, hp_b = (uint32_t)lay.hp_stage;
    const uint32_t sums_s = smem_s + (uint32_t)lay.sums, sums_b = (uint32_t)lay.sums_stage;

    // Order of the prologue.  The producer warp sets up the barriers, waits for the kernel ahead in the stream
    // and issues the first stages' copies at once: the other warps' table loads then run in the shadow of the
    // first stage's flight instead of ahead of it.  Only the producer executes griddepcontrol.wait: every
    // other access to the payloads, and every store to the output, follows a "full" barrier that one of the
    // producer's copies completes, i.e. follows that wait.
    tpq_grid_dep_launch();  // the next kernel in the stream may start its own prologue as SMs free up
    if constexpr (HAS_WAIT) {  // (an instantiation of its own: the plain call's prologue stays short)
        tpq_block_wait_arrivals(p.arr);
        __syncthreads();
    } else if constexpr (SPLIT) {  // (one instantiation per device count already: decided at run time here)
        if (p.arr.words != nullptr) {
            tpq_block_wait_arrivals(p.arr);
            __syncthreads();
        }
    }
    if (tid < 32) {
        // ---------------- producer warp: lane 0 waits for the stage and arms its barrier, then the 2N
        // copies of the stage are issued by 2N lanes at once
        const int pl = tid;
        if (pl == 0) {
            for (int s = 0; s < nstage; ++s) {
                mbar_init(smem_u32(&full[s]), 1);
                mbar_init(smem_u32(&empty[s]), (NT + DAUX) / 32);
                mbar_init(smem_u32(&sums_ready[s]), DAUX / 32);
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
        asm volatile("bar.arrive 1, %0;" ::"r"(blockDim.x) : "memory");  // the barriers exist
        if (pl < 2 * N) {
            // the block's first rows may start their way from HBM to L2 while it waits (a hint only: L2 is the
            // point of coherence, so whatever the kernel ahead still writes is what the copies will read)
            const int rows = rows_mine < DR_PREFETCH_ROWS ? rows_mine : DR_PREFETCH_ROWS;
            const int i = pl >> 1;
            if ((pl & 1) == 0)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.pl[i] + t_begin * ((E - k) / 2)),
                             "r"((uint32_t)((((size_t)rows * (E - k) / 2) + 15) & ~(size_t)15)) : "memory");
            else if (k)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p.pl[i] + p.lp_bytes + t_begin * k * 2),
                             "r"((uint32_t)rows * k * 2u) : "memory");
        }
        tpq_grid_dep_wait();  // the payloads and the output buffer may still be in use by the kernel ahead
        int st = 0;
        uint32_t parity = 1;  // parity of the "empty" phase to wait for
        for (int it = 0;; ++it) {
            const int r0 = dr_stage_row(it, pp.first, G);
            if (r0 >= rows_mine) break;
            const int cap = it == 0 ? pp.first : G;
            const int rows = rows_mine - r0 < cap ? rows_mine - r0 : cap;
            const int64_t t0 = t_begin + r0;
            const uint32_t lp_bytes = (uint32_t)((((size_t)rows * (E - k) / 2) + 15) & ~(size_t)15);
            const uint32_t hp_bytes = (uint32_t)rows * k * 2u;
            const uint32_t bar = smem_u32(&full[st]);
            const uint32_t stage = smem_s + (uint32_t)st * stage_b;
            int ok = 1;
            if (pl == 0) {
                if (it >= nstage && !mbar_wait(smem_u32(&empty[st]), parity)) {
                    atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                    ok = 0;
                } else {
                    mbar_expect_tx(bar, (uint32_t)N * (lp_bytes + hp_bytes));
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            for (int c = pl; c < 2 * N; c += 32) {
                const int i = c >> 1;
                if ((c & 1) == 0)
                    bulk_g2s(stage + (uint32_t)i * lp_b, p.pl[i] + t0 * ((E - k) / 2), lp_bytes, bar);
                else if (hp_bytes)
                    bulk_g2s(stage + (uint32_t)N * lp_b + (uint32_t)i * hp_b, p.pl[i] + p.lp_bytes + t0 * k * 2, hp_bytes, bar);
            }
            if (++st == nstage) {
                st = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    int st = 0;
    uint32_t parity = 0;
    const int lane = tid & 31;

    if (tid < 32 + DAUX) {
        // ---------------- auxiliary warps
        if constexpr (SPLIT) {
            // Two blocks share the rows.  Each adds up only the selected features that its own main threads
            // overwrite (its holes, ranks [hs, he)) and stores its share of the last k columns, a selected one
            // straight from the devices' BF16 values.  One item (a rank or a column) per thread and row; where
            // the threads outnumber the items, RP rows of a stage are worked on side by side.  What a thread
            // needs from the tables is loaded once.  Short rolled loops: this code runs once per stage, so
            // straight-line code would pay an instruction fetch for every few instructions it executes.
            const int at = tid - 32;
            const int hmid = pp.half_groups < L8 ? (int)(__ldg(p.grp + pp.half_groups) >> 8) : x.n_holes;  // holes of the first half
            const int hs = half == 0 ? 0 : hmid, he = half == 0 ? hmid : x.n_holes;
            const int nr = he - hs;
            // the last k columns are divided so that both blocks have the same number of items (a block with a
            // few more than DAUX / 2 would work on one row at a time instead of two)
            int nc0 = (x.n_holes + k + 1) / 2 - hmid;
            nc0 = nc0 < 0 ? 0 : (nc0 > k ? k : nc0);
            const int c0 = half == 0 ? 0 : nc0, nc = half == 0 ? nc0 : k - nc0;
            const int W = nr + nc;  // items per row
            const bool fast = W > 0 && W <= DAUX;
            int RP = 1;
            while (RP * 2 <= G && W * RP * 2 <= DAUX) RP *= 2;
            const int rp = fast ? at / W : 0, idx = fast ? at - rp * W : 0;
            const bool on = fast && rp < RP;
            const bool is_col = idx < nc;
            const int col = L + c0 + (is_col ? idx : 0);
            const int ps = (on && is_col) ? __ldg(p.pos + col) : -1;
            int do_sum = on && (!is_col || ps < 0), do_dec = on && is_col && ps >= 0;
            // the selected feature whose values this thread adds up, and where the sum goes
            const int rank = is_col ? (ps < 0 ? -ps - 1 : 0) : hs + idx - nc;
            int to_out = is_col;
            // a filler column's code sits at bits [sh, sh + 4) of a word of the hole's slot that carries it; it is
            // decoded in place like the main threads' codes (mask, exponent pattern, bias and a step divided by
            // the code's position), from the word shifted down by 16 for the upper four positions
            const int slot = do_dec ? ps : 0;
            uint32_t c_off = (uint32_t)(slot >> 3) * 4u;
            const int sh = (slot & 7) * 4, shl = sh & 15;
            uint32_t c_hi = sh >= 16 ? 16u : 0u, c_mask = 0xFu << shl;
            float c_nb = -(8388608.0f + (float)(8 << shl));
            float c_s[NMAX];
#pragma unroll
            for (int i = 0; i < NMAX; ++i)
                c_s[i] = (do_dec && i < N) ? __ldg(p.s_k + (size_t)i * E + col) * (1.0f / (float)(1 << shl)) : 0.0f;
            float c_b = 0.0f;  // the column's bias
            if (HAS_BIAS && do_dec) c_b = __ldg(p.bias + col);
            if (HAS_BIAS && do_sum) c_b = __ldg(p.bias + __ldg(x.hp_idx + rank));
            uint32_t h_off = (uint32_t)rank * 2u, s_off = (uint32_t)rank * 4u;
            keep(do_sum); keep(do_dec); keep(to_out); keep(c_off); keep(c_hi); keep(c_mask); keep(c_nb); keep(c_b);
            keep(h_off); keep(s_off);
#pragma unroll
            for (int i = 0; i < NMAX; ++i) keep(c_s[i]);
            uint32_t magic = 0x4B000000u;
            keep(magic);
            const uint32_t kb2 = (uint32_t)k * 2u, kb4 = (uint32_t)k * 4u, row_b = (uint32_t)L8 * 4u;
            asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");
            for (int it = 0;; ++it) {
                const int r0 = dr_stage_row(it, pp.first, G);
                if (r0 >= rows_mine) break;
                const int cap = it == 0 ? pp.first : G;
                const int rows = rows_mine - r0 < cap ? rows_mine - r0 : cap;
                if (!mbar_wait(smem_u32(&full[st]), parity)) {
                    atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                    break;
                }
                const uint32_t stage = smem_s + (uint32_t)st * stage_b;
                const uint32_t hp_s = stage + (uint32_t)N * lp_b;  // device 0's BF16 rows
                const uint32_t sums = sums_s + (uint32_t)st * sums_b;
                uint8_t *const obase = static_cast<uint8_t *>(p.out) + (t_begin + r0) * out_row_bytes;
                if (do_sum) {
                    uint32_t a = hp_s + h_off + (uint32_t)rp * kb2, o = sums + s_off + (uint32_t)rp * kb4;
                    uint8_t *og = obase + rp * out_row_bytes + (int64_t)col * ESIZE;
#pragma unroll 1
                    for (int r = rp; r < rows; r += RP, a += RP * kb2, o += RP * kb4, og += RP * out_row_bytes) {
                        float v = 0.0f;
#pragma unroll
                        for (int i = 0; i < NMAX; ++i)
                            if (i < N) v = __fadd_rn(v, __uint_as_float(lds16(a + (uint32_t)i * hp_b) << 16));
                        if (HAS_BIAS) v = __fadd_rn(v, c_b);
                        if (to_out) store_bits<FP32OUT>(og, out_bits<FP32OUT>(v));
                        else sts32(o, out_bits<FP32OUT>(v));
                    }
                }
                if (do_dec) {
                    uint32_t a = stage + c_off + (uint32_t)rp * row_b;
                    uint8_t *og = obase + rp * out_row_bytes + (int64_t)col * ESIZE;
#pragma unroll 1
                    for (int r = rp; r < rows; r += RP, a += RP * row_b, og += RP * out_row_bytes) {
                        float v = 0.0f;
#pragma unroll
                        for (int i = 0; i < NMAX; ++i)
                            if (i < N) {
                                const uint32_t w = (lds32(a + (uint32_t)i * lp_b) ^ 0x88888888u) >> c_hi;
                                v = __fmaf_rn(__fadd_rn(__uint_as_float(and_or(w, c_mask, magic)), c_nb), c_s[i], v);
                            }
                        if (HAS_BIAS) v = __fadd_rn(v, c_b);
                        store_bits<FP32OUT>(og, out_bits<FP32OUT>(v));
                    }
                }
                if (!fast) {  // (more items than threads: every item with its tables read where they are used)
                    for (int q = at; q < W; q += DAUX) {
                        const int cl = L + c0 + q, pc = q < nc ? __ldg(p.pos + cl) : -1;
                        const int rk = q < nc ? -pc - 1 : hs + q - nc;
                        for (int r = 0; r < rows; ++r) {
                            float v = 0.0f;
                            if (pc >= 0) {
                                for (int i = 0; i < N; ++i)
                                    v = __fmaf_rn(code_at(lds32(stage + (uint32_t)i * lp_b + (uint32_t)(r * L8 + (pc >> 3)) * 4u), (pc & 7) * 4),
                                                  __ldg(p.s_k + (size_t)i * E + cl), v);
                                if (HAS_BIAS) v = __fadd_rn(v, __ldg(p.bias + cl));
                            } else {
                                for (int i = 0; i < N; ++i)
                                    v = __fadd_rn(v, __uint_as_float(lds16(hp_s + (uint32_t)i * hp_b + (uint32_t)(r * k + rk) * 2u) << 16));
                                if (HAS_BIAS) v = __fadd_rn(v, __ldg(p.bias + __ldg(x.hp_idx + rk)));
                            }
                            if (q < nc) store_bits<FP32OUT>(obase + r * out_row_bytes + (int64_t)cl * ESIZE, out_bits<FP32OUT>(v));
                            else sts32(sums + (uint32_t)(r * k + rk) * 4u, out_bits<FP32OUT>(v));
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(smem_u32(&sums_ready[st]));  // (release: the sums above are visible to whoever waits)
                    mbar_arrive(smem_u32(&empty[st]));
                }
                if (++st == nstage) {
                    st = 0;
                    parity ^= 1u;
                }
            }
            return;
        }
        // Thread c works on the c-th selected feature (its sum) and on column L + c of the output, row by
        // row, in short rolled loops: these warps run code that nobody else runs, once per stage, so
        // straight-line code would pay an instruction fetch for every few instructions it executes.
        // What a thread needs from the tables is loaded once (feature sets with more than DR_AUX selected
        // features: further chunks of DR_AUX, with the tables read where they are used).
        const int at = tid - 32;
        const bool on = at < k;
        const int col = L + (on ? at : 0);
        const int ps = on ? __ldg(p.pos + col) : 0;
        // the column's code sits at bits [sh, sh + 4) of a word of the hole's slot that carries it; it is
        // decoded in place like the main threads' codes (mask, exponent pattern, bias and a step divided by
        // the code's position), from the word shifted down by 16 for the upper four positions
        const int slot = ps >= 0 ? ps : 0;
        int sel = ps < 0;
        uint32_t c_off = (uint32_t)(slot >> 3) * 4u;                    // the word inside a code row
        uint32_t c_sum = ps < 0 ? (uint32_t)(-ps - 1) * 4u : 0u;        // a selected column's sum inside a row of sums
        const int sh = (slot & 7) * 4, shl = sh & 15;
        uint32_t c_hi = sh >= 16 ? 16u : 0u, c_mask = 0xFu << shl;
        float c_nb = -(8388608.0f + (float)(8 << shl));
        float c_s[NMAX];
#pragma unroll
        for (int i = 0; i < NMAX; ++i)
            c_s[i] = (on && ps >= 0 && i < N) ? __ldg(p.s_k + (size_t)i * E + col) * (1.0f / (float)(1 << shl)) : 0.0f;
        float c_b = (HAS_BIAS && on && ps >= 0) ? __ldg(p.bias + col) : 0.0f;
        float h_b = (HAS_BIAS && on) ? __ldg(p.bias + __ldg(x.hp_idx + at)) : 0.0f;
        keep(sel); keep(c_off); keep(c_sum); keep(c_hi); keep(c_mask); keep(c_nb); keep(c_b); keep(h_b);
#pragma unroll
        for (int i = 0; i < NMAX; ++i) keep(c_s[i]);
        uint32_t magic = 0x4B000000u;
        keep(magic);
        const uint32_t kb2 = (uint32_t)k * 2u, kb4 = (uint32_t)k * 4u, row_b = (uint32_t)L8 * 4u;
        asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");
        for (int it = 0;; ++it) {
            const int r0 = dr_stage_row(it, pp.first, G);
            if (r0 >= rows_mine) break;
            const int cap = it == 0 ? pp.first : G;
            const int rows = rows_mine - r0 < cap ? rows_mine - r0 : cap;
            if (!mbar_wait(smem_u32(&full[st]), parity)) {
                atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
            const uint32_t stage = smem_s + (uint32_t)st * stage_b;
            const uint32_t hp_s = stage + (uint32_t)N * lp_b;  // device 0's BF16 rows
            const uint32_t sums = sums_s + (uint32_t)st * sums_b;
            // (1) the sums of the selected features
            if (on) {
                uint32_t a = hp_s + (uint32_t)at * 2u, o = sums + (uint32_t)at * 4u;
#pragma unroll 1
                for (int r = 0; r < rows; ++r, a += kb2, o += kb4) {
                    float v = 0.0f;
#pragma unroll
                    for (int i = 0; i < NMAX; ++i)
                        if (i < N) v = __fadd_rn(v, __uint_as_float(lds16(a + (uint32_t)i * hp_b) << 16));
                    if (HAS_BIAS) v = __fadd_rn(v, h_b);
                    sts32(o, out_bits<FP32OUT>(v));
                }
            }
            for (int c = at + DR_AUX; c < k; c += DR_AUX) {  // (more selected features than threads)
                const float hb = HAS_BIAS ? __ldg(p.bias + __ldg(x.hp_idx + c)) : 0.0f;
                for (int r = 0; r < rows; ++r) {
                    float v = 0.0f;
                    for (int i = 0; i < N; ++i)
                        v = __fadd_rn(v, __uint_as_float(lds16(hp_s + (uint32_t)i * hp_b + (uint32_t)(r * k + c) * 2u) << 16));
                    if (HAS_BIAS) v = __fadd_rn(v, hb);
                    sts32(sums + (uint32_t)(r * k + c) * 4u, out_bits<FP32OUT>(v));
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sums_ready[st]));  // (release: the sums above are visible to whoever waits)
            if (!mbar_wait(smem_u32(&sums_ready[st]), parity)) {    // the other auxiliary warps' sums
                atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
            // (2) the last k columns
            // (of two blocks that share the rows, the second one stores them)
            const bool tail = !SPLIT || half == 1;
            uint8_t *const obase = static_cast<uint8_t *>(p.out) + (t_begin + r0) * out_row_bytes;
            if (on && tail) {
                uint32_t a = stage + c_off, sa = sums + c_sum;
                uint8_t *o = obase + (int64_t)col * ESIZE;
#pragma unroll 1
                for (int r = 0; r < rows; ++r, a += row_b, sa += kb4, o += out_row_bytes) {
                    float v = 0.0f;
#pragma unroll
                    for (int i = 0; i < NMAX; ++i)
                        if (i < N) {
                            const uint32_t w = (lds32(a + (uint32_t)i * lp_b) ^ 0x88888888u) >> c_hi;
                            v = __fmaf_rn(__fadd_rn(__uint_as_float(and_or(w, c_mask, magic)), c_nb), c_s[i], v);
                        }
                    if (HAS_BIAS) v = __fadd_rn(v, c_b);
                    const uint32_t sum = lds32(sa);
                    store_bits<FP32OUT>(o, sel ? sum : out_bits<FP32OUT>(v));
                }
            }
            for (int c = at + DR_AUX; tail && c < k; c += DR_AUX) {  // (more columns than threads)
                const int cl = L + c, pc = __ldg(p.pos + cl);
                for (int r = 0; r < rows; ++r) {
                    uint32_t bits;
                    if (pc >= 0) {
                        float v = 0.0f;
                        for (int i = 0; i < N; ++i)
                            v = __fmaf_rn(code_at(lds32(stage + (uint32_t)i * lp_b + (uint32_t)(r * L8 + (pc >> 3)) * 4u), (pc & 7) * 4),
                                          __ldg(p.s_k + (size_t)i * E + cl), v);
                        if (HAS_BIAS) v = __fadd_rn(v, __ldg(p.bias + cl));
                        bits = out_bits<FP32OUT>(v);
                    } else {
                        bits = lds32(sums + (uint32_t)(r * k + (-pc - 1)) * 4u);
                    }
                    store_bits<FP32OUT>(obase + r * out_row_bytes + (int64_t)cl * ESIZE, bits);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&empty[st]));
            if (++st == nstage) {
                st = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    // ---------------- main warps
    const int gl = tid - 32 - DAUX;
    const int g = SPLIT ? half * pp.half_groups + gl : gl;
    const bool live = SPLIT ? (gl < pp.half_groups && g < L8) : g < L8;
    const int g_ld = live ? g : 0;
    float2 sc[NMAX][4];
#pragma unroll
    for (int i = 0; i < NMAX; ++i) {
#pragma unroll
        for (int h = 0; h < 4; ++h) sc[i][h] = make_float2(0.0f, 0.0f);
        if (live && i < N) load_steps(p.s_k + (size_t)i * E, g, sc[i]);
    }
    // the selected features among the thread's 8 ("holes": their lanes are overwritten with the sums)
    const uint32_t gd = live ? __ldg(p.grp + g) : 0u;
    const uint32_t hmask = gd & 0xFFu;
    const int hrank = (int)(gd >> 8);  // rank of the group's first selected feature
    const int nh = __popc(hmask);
    const int hl0 = nh > 0 ? __ffs(hmask) - 1 : 0;
    const int hl1 = nh > 1 ? __ffs(hmask & (hmask - 1)) - 1 : 0;
    const bool warp_holes = __any_sync(0xffffffffu, nh > 0);
    float2 b[4];  // the thread's 8 biases (only in the instantiation that adds them)
#pragma unroll
    for (int h = 0; h < 4; ++h) b[h] = make_float2(0.0f, 0.0f);
    if (HAS_BIAS) {
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g_ld));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g_ld + 4));
        b[0] = make_float2(b0.x, b0.y); b[1] = make_float2(b0.z, b0.w);
        b[2] = make_float2(b1.x, b1.y); b[3] = make_float2(b1.z, b1.w);
    }
    const DecodeConsts dc = decode_consts();
    const uint32_t word_s = smem_s + (uint32_t)g_ld * 4u;  // this thread's word of row 0, device 0, stage 0
    const uint32_t row_b = (uint32_t)L8 * 4u;
    uint8_t *orow = static_cast<uint8_t *>(p.out) + (size_t)8 * g_ld * ESIZE + t_begin * out_row_bytes;
    asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");

    for (int it = 0;; ++it) {
        const int r0 = dr_stage_row(it, pp.first, G);
        if (r0 >= rows_mine) break;
        const int cap = it == 0 ? pp.first : G;
        const int rows = rows_mine - r0 < cap ? rows_mine - r0 : cap;
        if (!mbar_wait(smem_u32(&full[st]), parity)) {
            atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
            break;
        }
        const uint32_t sa = word_s + (uint32_t)st * stage_b;
        // whole stages run as straight-line code (rows per stage and device count known at compile time)
        if (G == 4 && rows == 4 && !pp.pairs) {
            if (N == NMAX) rows_stage<NMAX, NMAX, 4, 4 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa, lp_b, row_b, N, sc, dc, b, orow, out_row_bytes, live);
            else rows_stage<NMAX, 0, 4, 4 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa, lp_b, row_b, N, sc, dc, b, orow, out_row_bytes, live);
        } else if (G == 4 || G == 2) {
            // two rows at a time in a rolled loop (long runs: measured 3 % ahead of four rows as one straight line
            // at 8192 x 5120, 4 % behind at 2048 rows, where the straight line is used for whole stages)
            int r = 0;
            if (G == 4) {
                if (N == NMAX) {
#pragma unroll 1
                    for (; r + 2 <= rows; r += 2)
                        rows_stage<NMAX, NMAX, 2, 4 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa + (uint32_t)r * row_b, lp_b, row_b, N, sc, dc, b,
                                                                                        orow + r * out_row_bytes, out_row_bytes, live);
                } else {
#pragma unroll 1
                    for (; r + 2 <= rows; r += 2)
                        rows_stage<NMAX, 0, 2, 4 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa + (uint32_t)r * row_b, lp_b, row_b, N, sc, dc, b,
                                                                                  orow + r * out_row_bytes, out_row_bytes, live);
                }
                if (r < rows)
                    rows_stage<NMAX, 0, 1, 4 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa + (uint32_t)r * row_b, lp_b, row_b, N, sc, dc, b,
                                                                              orow + r * out_row_bytes, out_row_bytes, live);
            } else {
                if (rows == 2) {
                    if (N == NMAX) rows_stage<NMAX, NMAX, 2, 2 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa, lp_b, row_b, N, sc, dc, b, orow, out_row_bytes, live);
                    else rows_stage<NMAX, 0, 2, 2 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa, lp_b, row_b, N, sc, dc, b, orow, out_row_bytes, live);
                } else {
                    rows_stage<NMAX, 0, 1, 2 * ROWCAP * 4, FP32OUT, HAS_BIAS>(sa, lp_b, row_b, N, sc, dc, b, orow, out_row_bytes, live);
                }
            }
        } else {
#pragma unroll 1
            for (int r = 0; r < rows; ++r)
                rows_stage<NMAX, 0, 1, 0, FP32OUT, HAS_BIAS>(sa + (uint32_t)r * row_b, lp_b, row_b, N, sc, dc, b,
                                                                orow + r * out_row_bytes, out_row_bytes, live);
        }
        if (warp_holes) {  // (uniform over the warp)
            if (!mbar_wait(smem_u32(&sums_ready[st]), parity)) {
                atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
            if (nh > 0) {
                const uint32_t sums = sums_s + (uint32_t)st * sums_b + (uint32_t)hrank * 4u;
                for (int r = 0; r < rows; ++r) {
                    uint8_t *const o = orow + r * out_row_bytes;
                    const uint32_t sr = sums + (uint32_t)(r * k) * 4u;
                    store_bits<FP32OUT>(o + hl0 * ESIZE, lds32(sr));
                    if (nh > 1) store_bits<FP32OUT>(o + hl1 * ESIZE, lds32(sr + 4u));
                    if (nh > 2) {
                        uint32_t m = hmask & (hmask - 1);
                        m &= m - 1;
                        for (int j = 2; m; ++j, m &= m - 1) store_bits<FP32OUT>(o + (__ffs(m) - 1) * ESIZE, lds32(sr + 4u * j));
                    }
                }
            }
        }
        orow += rows * out_row_bytes;
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&empty[st]));
        if (++st == nstage) {
            st = 0;
            parity ^= 1u;
        }
    }
}

void fill_params(DQParams &p, const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int64_t out_stride)
{
    for (int i = 0; i < c->N; ++i) p.pl[i] = static_cast<const uint8_t *>(payloads[i]);
    p.N = c->N; p.E = c->E; p.k = c->k; p.bits = c->bits; p.T = T;
    p.lp_bytes = tpq_lp_bytes_i(T, c->E, c->k, c->bits);
    p.s_k = c->t.s_k; p.pos = c->t.pos; p.grp = c->t.grp;
    p.out = out; p.out_stride = out_stride;
    p.bias = c->call_bias;
    p.arr = c->call_arr;
}

}  // namespace

bool tpq_dequant_tiled_ok(const tpq_ctx *c, int64_t T, int64_t out_stride, int fp32_out)
{
    (void)fp32_out;
    if (c->bits != 4) return false;  // the tiled kernels are Int4 kernels
    if (c->E % 8 || c->k % 8 || out_stride % 8 || T <= 0) return false;
    if (c->E - c->k < 8) return false;
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

namespace {

template <int NMAX, int ROWCAP, int MAXT, int DAUX, bool FP32OUT, bool HAS_BIAS, bool HAS_WAIT>
cudaError_t launch_rows_w(const DRParams &pp, int grid, int consumers, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(dequant_rows<NMAX, ROWCAP, MAXT, DAUX, FP32OUT, HAS_BIAS, HAS_WAIT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        e = tpq_launch_pdl(dequant_rows<NMAX, ROWCAP, MAXT, DAUX, FP32OUT, HAS_BIAS, HAS_WAIT>, dim3(grid), dim3(consumers + DAUX + 32),
                           smem, st, pp);
    return e;
}

template <int NMAX, int ROWCAP, int MAXT, int DAUX, bool FP32OUT, bool HAS_BIAS>
cudaError_t launch_rows_v(const DRParams &pp, int grid, int consumers, size_t smem, cudaStream_t st)
{
    if constexpr (NMAX > 4) return launch_rows_w<NMAX, ROWCAP, MAXT, DAUX, FP32OUT, HAS_BIAS, false>(pp, grid, consumers, smem, st);
    return pp.q.arr.words ? launch_rows_w<NMAX, ROWCAP, MAXT, DAUX, FP32OUT, HAS_BIAS, true>(pp, grid, consumers, smem, st)
                          : launch_rows_w<NMAX, ROWCAP, MAXT, DAUX, FP32OUT, HAS_BIAS, false>(pp, grid, consumers, smem, st);
}

template <int NMAX, int ROWCAP, int MAXT, int DAUX>
cudaError_t launch_rows(const DRParams &pp, int fp32_out, int grid, int consumers, size_t smem, cudaStream_t st)
{
    const bool bias = pp.q.bias != nullptr;
    if (fp32_out)
        return bias ? launch_rows_v<NMAX, ROWCAP, MAXT, DAUX, true, true>(pp, grid, consumers, smem, st)
                    : launch_rows_v<NMAX, ROWCAP, MAXT, DAUX, true, false>(pp, grid, consumers, smem, st);
    return bias ? launch_rows_v<NMAX, ROWCAP, MAXT, DAUX, false, true>(pp, grid, consumers, smem, st)
                : launch_rows_v<NMAX, ROWCAP, MAXT, DAUX, false, false>(pp, grid, consumers, smem, st);
}

// rows after which the code stream is 16-byte aligned again: blocks and stages start on multiples of it
int g0_of(const tpq_ctx *c)
{
    const int L8 = (c->E - c->k) / 8;
    return L8 % 4 == 0 ? 1 : (L8 % 2 == 0 ? 2 : 4);
}

// Row kernel geometry; returns false if the shape does not admit it.
bool rows_plan(const tpq_ctx *c, int64_t T, int *G_out, int *nstage_out, int64_t *rows_per_block_out, int *grid_out)
{
    const int N = c->N, E = c->E, k = c->k;
    const int L8 = (E - k) / 8;
    // up to 8 devices: a main thread keeps the steps of all of them in registers.  Up to four, a block has one
    // main thread per group; from five on that many registers leave room for half as many threads, so two
    // blocks share a run of rows (each stages whole rows and decodes one half of the groups).  Beyond 8 the
    // panel kernels, whose registers do not grow with N, take over.
    if (N > 8) return false;
    const bool split = N > 4;
    if (L8 > (split ? 640 : 768)) return false;  // main threads (two blocks per run: measured behind the panel kernels on wider rows)
    const int runs = split ? c->sm_count / 2 : c->sm_count;
    if (runs < 1) return false;
    const int g0 = g0_of(c);
    // every block takes the same number of adjacent rows (a multiple of g0), so no block has more than g0 - 1
    // rows above the mean; it walks them four at a time where a ring of three such stages fits, else two
    int64_t rpb = (T + runs - 1) / runs;
    rpb = (rpb + g0 - 1) / g0 * g0;
    // 8 devices: the tensor-map panel kernel is ahead on longer
    // inputs: with 256-group panels from about 1200 rows on (8192 x 4096: 51 against 62 us; 2048 rows: 16.4
    // against 18.1; level at 1024), with the 128-group panels of rows that are not a multiple of 16 bytes long
    // from about 2400 on (8192 x 5120: 65.7 against 70.6 us; level at 2048); 5 to 7 devices: level or behind
    if (N == 8 && rpb > (g0 > 1 ? 32 : 16) && c->dq_kernel != 1) return false;
    int G = 4;
    // (two blocks per run of rows: a ring of two four-row stages measured ahead of four two-row stages from
    // 2048 rows on: 8 devices, 8192 x 5120: 70.6 against 75.9 us)
    const int ring4 = (split && rpb >= 8) ? 2 : 3;
    if (rpb < 4 || dr_layout(N, E, k, 4, ring4).total > (size_t)c->smem_optin) G = 2;
    if (G < g0) G = g0;
    if (dr_layout(N, E, k, G, 2).total > (size_t)c->smem_optin) return false;
    const int grid = (int)((T + rpb - 1) / rpb) * (split ? 2 : 1);
    const int64_t per_block = (rpb + G - 1) / G;
    int nstage = (int)(per_block < 4 ? per_block : 4);  // deeper rings measured no faster (often slower)
    if (G == 4 && nstage > 3) nstage = 3;
    if (nstage < 2) nstage = 2;
    while (nstage > 2 && dr_layout(N, E, k, G, nstage).total > (size_t)c->smem_optin) --nstage;
    *G_out = G; *nstage_out = nstage; *rows_per_block_out = rpb; *grid_out = grid;
    return true;
}

// Panel kernel geometry: the widest panel (CG groups) whose steps fit in shared memory beside the ring;
// one block per SM, a few of them for the BF16 block (its share of the bytes, with some margin), the
// others walking their share of the row chunks.  Returns false if the shape does not admit it.
bool panels_plan(const tpq_ctx *c, int64_t T, DPParams &pp)
{
    const int N = c->N, E = c->E, k = c->k, L8 = (E - k) / 8;
    int CG = 128;
    while (CG >= 32 && dp_smem_bytes(N, CG) > (size_t)c->smem_optin) CG >>= 1;
    if (CG < 32) return false;
    pp.CG = CG;
    pp.panels = (L8 + CG - 1) / CG;
    const int RC = DP_THREADS / CG * DP_R;
    pp.n_chunks = (T + RC - 1) / RC;
    int64_t gy = c->sm_count / pp.panels;
    if (gy > pp.n_chunks) gy = pp.n_chunks;
    if (gy < 1) gy = 1;
    pp.gy = (int)gy;
    return true;
}

template <int CG, bool FP32OUT, bool HAS_WAIT>
cudaError_t launch_panels_w(const tpq_ctx *c, const DPParams &pp, cudaStream_t st)
{
    const size_t smem = dp_smem_bytes(c->N, CG);
    cudaError_t e = cudaFuncSetAttribute(dequant_panels<CG, FP32OUT, HAS_WAIT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return tpq_launch_pdl(dequant_panels<CG, FP32OUT, HAS_WAIT>, dim3((unsigned)(pp.panels * pp.gy)), dim3(DP_THREADS), smem, st, pp);
}

template <int CG, bool FP32OUT>
cudaError_t launch_panels_cg(const tpq_ctx *c, const DPParams &pp, cudaStream_t st)
{
    return pp.q.arr.words ? launch_panels_w<CG, FP32OUT, true>(c, pp, st) : launch_panels_w<CG, FP32OUT, false>(c, pp, st);
}

template <bool FP32OUT>
cudaError_t launch_panels(const tpq_ctx *c, const DPParams &pp, cudaStream_t st)
{
    switch (pp.CG) {
    case 128: return launch_panels_cg<128, FP32OUT>(c, pp, st);
    case 64: return launch_panels_cg<64, FP32OUT>(c, pp, st);
    default: return launch_panels_cg<32, FP32OUT>(c, pp, st);
    }
}

// ---- tensor maps of the payloads' code sections

// A payload's map depends on its address and on the shape; encoding costs about a microsecond of host time,
// so the maps of recently seen payloads are kept (callers reuse their communication buffers).
struct DTCacheEntry {
    const void *ptr;
    int64_t T;
    int L8, CG, RC, g0;
    CUtensorMap map;
};
struct DTCache {
    static constexpr int CAP = 256;
    int n = 0, next = 0;
    DTCacheEntry e[CAP];
};

bool payload_map(tpq_ctx *c, const void *ptr, int64_t T, int L8, int CG, int RC, int g0, CUtensorMap *out)
{
    if (!c->dq_cache) c->dq_cache = new (std::nothrow) DTCache();
    DTCache *cache = static_cast<DTCache *>(c->dq_cache);
    if (cache)
        for (int j = 0; j < cache->n; ++j) {
            const DTCacheEntry &e = cache->e[j];
            if (e.ptr == ptr && e.T == T && e.L8 == L8 && e.CG == CG && e.RC == RC && e.g0 == g0) {
                *out = e.map;
                return true;
            }
        }
    tpq_encode_tiled_fn fn = tpq_tensor_map_encoder();
    if (!fn) return false;
    // (g0 adjacent rows are one row of the map: see dt_class_bytes)
    const cuuint64_t dims[2] = {(cuuint64_t)g0 * L8, (cuuint64_t)(T / g0)};
    const cuuint64_t strides[1] = {(cuuint64_t)g0 * L8 * 4};
    const cuuint32_t box[2] = {(cuuint32_t)(CG + (g0 > 1 ? 4 : 0)), (cuuint32_t)(RC / g0)};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    if (fn(&m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (cache) {
        DTCacheEntry &e = cache->e[cache->next];
        e.ptr = ptr; e.T = T; e.L8 = L8; e.CG = CG; e.RC = RC; e.g0 = g0; e.map = m;
        cache->next = (cache->next + 1) % DTCache::CAP;
        if (cache->n < DTCache::CAP) ++cache->n;
    }
    *out = m;
    return true;
}

// Tensor-map panel kernel geometry; false if the shape (or the driver) does not admit it.
bool tpanels_plan(tpq_ctx *c, const void *const *payloads, int64_t T, DTParams &tp, DTMaps &maps)
{
    const int N = c->N, E = c->E, k = c->k, L8 = (E - k) / 8;
    const int g0 = g0_of(c);
    const int64_t Tm = T - T % g0;  // rows the tensor maps cover
    // (rows that are not a multiple of 16 bytes long: panels of 128 groups: a box is at most 256 elements wide,
    // and theirs is 4 wider than the panel)
    if (N > DT_MAX_DEV || Tm == 0 || T > 0x7FFFFFF0LL) return false;
    int CG = g0 > 1 ? 128 : 256;  // (measured at N = 16, E = 8192: panels of 256 groups 4 to 11 % ahead of 128)
    while (CG >= 32 && dt_smem_bytes(N, CG, 2, g0) > (size_t)c->smem_optin) CG >>= 1;
    if (CG < (g0 > 1 ? 128 : 32)) return false;
    const int RC = DT_MAIN / CG * DP_R;
    DPParams &pp = tp.d;
    pp.CG = CG;
    pp.panels = (L8 + CG - 1) / CG;
    pp.n_chunks = (Tm + RC - 1) / RC + (Tm < T ? 1 : 0);
    if (c->dq_kernel != 2 && pp.n_chunks * pp.panels < c->sm_count) return false;  // short inputs: the copy kernel starts faster
    // a block keeps its panel and takes every gy-th chunk (measured 2 to 4 % ahead of equal contiguous runs of
    // (panel, chunk) pairs, which reload the steps when a run crosses into the next panel)
    pp.gy = (int)(c->sm_count / pp.panels);
    if (pp.gy < 1) pp.gy = 0;
    int nstage = 6;
    while (nstage > 2 && dt_smem_bytes(N, CG, nstage, g0) > (size_t)c->smem_optin) --nstage;
    tp.nstage = nstage;
    tp.g0 = g0;
    tp.tail_rows = (int)(T - Tm);
    tp.status = c->t.status;
    for (int i = 0; i < N; ++i)
        if (!payload_map(c, payloads[i], Tm, L8, CG, RC, g0, &maps.m[i])) return false;
    return true;
}

template <int CG, int G0, int M4, bool FP32OUT>
cudaError_t launch_tpanels_cg(const tpq_ctx *c, const DTParams &tp, const DTMaps &maps, cudaStream_t st)
{
    const size_t smem = dt_smem_bytes(c->N, CG, tp.nstage, G0);
    cudaError_t e = cudaFuncSetAttribute(dequant_tpanels<CG, G0, M4, FP32OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)tp.d.panels * tp.d.n_chunks;
    unsigned grid = (unsigned)(total < c->sm_count ? total : c->sm_count);
    if (tp.d.gy > 0) grid = (unsigned)(tp.d.gy * tp.d.panels);
    return tpq_launch_pdl(dequant_tpanels<CG, G0, M4, FP32OUT>, dim3(grid), dim3(DT_THREADS), smem, st, tp, maps);
}

template <bool FP32OUT>
cudaError_t launch_tpanels(const tpq_ctx *c, const DTParams &tp, const DTMaps &maps, cudaStream_t st)
{
    const int m4 = ((c->E - c->k) / 8) % 4;
    if (tp.g0 == 2) return launch_tpanels_cg<128, 2, 2, FP32OUT>(c, tp, maps, st);
    if (tp.g0 == 4)
        return m4 == 1 ? launch_tpanels_cg<128, 4, 1, FP32OUT>(c, tp, maps, st) : launch_tpanels_cg<128, 4, 3, FP32OUT>(c, tp, maps, st);
    switch (tp.d.CG) {
    case 256: return launch_tpanels_cg<256, 1, 0, FP32OUT>(c, tp, maps, st);
    case 128: return launch_tpanels_cg<128, 1, 0, FP32OUT>(c, tp, maps, st);
    case 64: return launch_tpanels_cg<64, 1, 0, FP32OUT>(c, tp, maps, st);
    default: return launch_tpanels_cg<32, 1, 0, FP32OUT>(c, tp, maps, st);
    }
}

}  // namespace

cudaError_t tpq_launch_dequant_tiled(const tpq_ctx *c, const void *const *payloads, int64_t T, void *out, int fp32_out,
                                     int64_t out_stride, cudaStream_t st, int64_t *launches)
{
    DQParams p;
    fill_params(p, c, payloads, T, out, out_stride);
    DXParams x;
    x.hp_idx = c->t.hp_idx; x.hole = c->t.hole; x.filler = c->t.filler; x.n_holes = c->n_holes; x.status = c->t.status;
    const int want = c->dq_kernel;  // 0 automatic; 1 row, 2 tensor-map panel, 3 copy-ring panel kernel
    if (want == 0 || want == 1) {
        DRParams pp;
        int grid = 0;
        if (rows_plan(c, T, &pp.G, &pp.nstage, &pp.rows_per_block, &grid)) {
            pp.q = p;
            pp.x = x;
            // a short first stage lands sooner (measured at 2048 x 5120: 11.0 -> 10.9 us, 12.3 -> 11.6 us without the prefetch)
            pp.first = (pp.G == 4 && pp.rows_per_block > 4 && (g0_of(c) <= 2)) ? 2 : pp.G;
            pp.pairs = pp.rows_per_block > 32;
            const size_t smem = dr_layout(c->N, c->E, c->k, pp.G, pp.nstage).total;
            const int L8 = (c->E - c->k) / 8;
            pp.half_groups = (L8 + 1) / 2;
            int consumers = (((c->N > 4 ? pp.half_groups : L8) + 31) / 32) * 32;
            if (consumers < 32) consumers = 32;
            cudaError_t e;
            if (c->N > 4) {
                // (the device count is a compile-time constant there: measured 8 to 25 % ahead of a count read at run time)
                switch (c->N) {
                case 5: e = launch_rows<5, 640, 320, 160>(pp, fp32_out, grid, consumers, smem, st); break;
                case 6: e = launch_rows<6, 640, 320, 160>(pp, fp32_out, grid, consumers, smem, st); break;
                case 7: e = launch_rows<7, 640, 320, 160>(pp, fp32_out, grid, consumers, smem, st); break;
                default: e = launch_rows<8, 640, 320, 160>(pp, fp32_out, grid, consumers, smem, st); break;
                }
            } else
                e = L8 <= 640 ? launch_rows<4, 640, 640, DR_AUX>(pp, fp32_out, grid, consumers, smem, st)
                              : launch_rows<4, 768, 768, DR_AUX>(pp, fp32_out, grid, consumers, smem, st);
            if (e != cudaSuccess) return e;
            ++*launches;
            return cudaGetLastError();
        }
        if (want == 1) return cudaErrorInvalidValue;
    }
    if (want == 0 || want == 2) {
        DTParams tp;
        DTMaps maps;
        if (tpanels_plan(const_cast<tpq_ctx *>(c), payloads, T, tp, maps)) {
            tp.d.q = p;
            tp.d.s_slot = c->t.s_slot; tp.d.lp_idx = c->t.lp_idx; tp.d.hp_idx = c->t.hp_idx;
            tp.d.filler = c->t.filler; tp.d.n_holes = c->n_holes;
            const cudaError_t e = fp32_out ? launch_tpanels<true>(c, tp, maps, st) : launch_tpanels<false>(c, tp, maps, st);
            if (e == cudaSuccess) ++*launches;
            return e;
        }
        if (want == 2) return cudaErrorInvalidValue;
    }
    DPParams dp;
    if (!panels_plan(c, T, dp)) {
        if (want == 3) return cudaErrorInvalidValue;
        return tpq_launch_dequant_generic(c, payloads, T, out, fp32_out, out_stride, st, launches);
    }
    dp.q = p;
    dp.s_slot = c->t.s_slot; dp.lp_idx = c->t.lp_idx; dp.hp_idx = c->t.hp_idx;
    dp.filler = c->t.filler; dp.n_holes = c->n_holes;
    const cudaError_t e = fp32_out ? launch_panels<true>(c, dp, st) : launch_panels<false>(c, dp, st);
    if (e == cudaSuccess) ++*launches;
    return e;
}

void tpq_dequant_release(tpq_ctx *c)
{
    delete static_cast<DTCache *>(c->dq_cache);
    c->dq_cache = nullptr;
}

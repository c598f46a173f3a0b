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

__device__ __host__ constexpr int dq_pos(int n) { return n < 5 ? n : n - 5; }

// 8 two's-complement codes of `raw` times their steps, accumulated.  The codes are decoded in place:
// (x & 0xF << 4n) | 0x4B000000 is the float 2^23 + (code+8) 16^n; subtracting 2^23 + 8*16^n leaves
// code * 16^n exactly, and the step was pre-divided by 16^n (an exact scaling), so
// fma(code*16^n, s/16^n, acc) rounds exactly like fma(code, s, acc).  Codes 5..7 use raw >> 20.
// Subtractions and FMAs run two at a time (f32x2), one binary32 rounding per element as before.
// -(2^23 + 8 * 16^pos) for the code pairs (0,1) (2,3) (4,5) (6,7); in constant memory so that the packed
// subtract can take the pair as an operand instead of rebuilding it in registers
__constant__ float2 kDecodeBias[4] = {{-8388616.0f, -8388736.0f},      // 16^0, 16^1
                                      {-8390656.0f, -8421376.0f},      // 16^2, 16^3
                                      {-8912896.0f, -8388616.0f},      // 16^4, 16^0 (codes 5..7 use raw >> 20)
                                      {-8388736.0f, -8390656.0f}};     // 16^1, 16^2

// Each code costs ONE logic instruction only if the mask and the exponent pattern are both register
// operands of an explicit lop3 ((x & mask) | magic, truth table 0xEA): written in C with immediates the
// compiler emits two.  `magic` holds 0x4B000000 (see opaque_magic).
__device__ __forceinline__ uint32_t opaque_magic()
{
    uint32_t m;
    asm volatile("mov.u32 %0, 0x4B000000;" : "=r"(m));
    return m;
}
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t mask, uint32_t magic)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(x), "r"(mask), "r"(magic));
    return d;
}

__device__ __forceinline__ void decode8(uint32_t raw, const float2 (&sc)[4], float2 (&acc)[4], uint32_t magic,
                                        const float2 (&bias)[4] = kDecodeBias)
{
    const uint32_t xa = raw ^ 0x88888888u;
    const uint32_t xb = xa >> 20;
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const int n0 = 2 * h, n1 = 2 * h + 1;
        const uint32_t x0 = (n0 < 5) ? xa : xb, x1 = (n1 < 5) ? xa : xb;
        const float f0 = __uint_as_float(and_or(x0, 0xFu << (4 * dq_pos(n0)), magic));
        const float f1 = __uint_as_float(and_or(x1, 0xFu << (4 * dq_pos(n1)), magic));
        const float2 d = __fadd2_rn(make_float2(f0, f1), bias[h]);
        acc[h] = __ffma2_rn(d, sc[h], acc[h]);
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
__device__ __forceinline__ void dp_store_rows(const DQParams &p, const int32_t *lp_idx, int64_t t0, int g, uint32_t mask,
                                              const float2 (&acc_in)[DP_R][4])
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
            if (t0 + r < p.T) store_group<FP32OUT>(p.out, (t0 + r) * p.out_stride + 8 * (int64_t)g, acc[r], 0u);
    } else {
        int col[8];
#pragma unroll
        for (int n = 0; n < 8; ++n) col[n] = (mask & (1u << n)) ? __ldg(lp_idx + 8 * g + n) : 8 * g + n;
#pragma unroll
        for (int r = 0; r < DP_R; ++r)
            if (t0 + r < p.T) {
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
    const uint32_t magic = opaque_magic();
    float2 bias[4];  // the decode biases in registers (the packed subtract takes no constant-bank pair)
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        bias[h] = kDecodeBias[h];
        asm volatile("" : "+f"(bias[h].x), "+f"(bias[h].y));
    }

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
                    for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], magic, bias);
                }
            } else {
#pragma unroll
                for (int i = 0; i < DP_NB; ++i)
                    if (i0 + i < N) {
                        const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                        const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                              make_float2(b.z, b.w)};
#pragma unroll
                        for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], magic, bias);
                    }
            }
        }
        if (it_on) {  // the last step's values (a partial batch has N % DP_NB of them)
            const int nl = N - (N - 1) / DP_NB * DP_NB;
#pragma unroll
            for (int i = 0; i < DP_NB; ++i)
                if (i < nl) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
        }
        if (live) dp_store_rows<FP32OUT>(p, pp.lp_idx, t0, g, 0u, acc);
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
    int *status;
};

__host__ __device__ inline size_t dt_stage_bytes() { return (size_t)DT_NB * DT_MAIN * DP_R * 4; }  // CG*RC = DT_MAIN*DP_R words per device
__host__ __device__ inline size_t dt_smem_bytes(int N, int CG, int nstage)
{
    return dp_steps_bytes(N, CG) + (size_t)nstage * dt_stage_bytes() + (size_t)nstage * 16;  // steps, ring, mbarriers
}


template <int CG, bool FP32OUT>
__global__ void __launch_bounds__(DT_THREADS, 1) dequant_tpanels(const DTParams tp, const __grid_constant__ DTMaps maps)
{
    extern __shared__ __align__(128) uint8_t dp_smem[];
    constexpr int RS = DT_MAIN / CG, RC = RS * DP_R;
    constexpr uint32_t BOX_BYTES = (uint32_t)CG * RC * 4;
    constexpr uint32_t STAGE_BYTES = DT_NB * BOX_BYTES;
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
    const int64_t f0 = total * blockIdx.x / gridDim.x, f1 = total * (blockIdx.x + 1) / gridDim.x;

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
    const uint32_t magic = opaque_magic();
    float2 bias[4];  // the decode biases in registers (the packed subtract takes no constant-bank pair)
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        bias[h] = kDecodeBias[h];
        asm volatile("" : "+f"(bias[h].x), "+f"(bias[h].y));
    }
    const float4 *const my_steps = dp_steps + cg;
    const uint32_t *const ring_w = reinterpret_cast<const uint32_t *>(ring) + (rs * DP_R) * CG + cg;
    // ring state: the producer lane and the main warps walk the same sequence of stages across segments
    int st = 0, it = 0;
    uint32_t parity = (tid >= DT_MAIN) ? 1u : 0u;  // producer: parity of the "empty" phase to wait for

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
                for (int64_t ch = chb; ch < che; ++ch) {
                    for (int i0 = 0; i0 < N; i0 += DT_NB, ++it) {
                        const int nb = (N - i0 < DT_NB) ? N - i0 : DT_NB;
                        const uint32_t bar = smem_u32(&full[st]);
                        if (it >= nstage && !mbar_wait(smem_u32(&empty[st]), parity)) {
                            atomicExch(tp.status, (int)TPQ_ERR_TIMEOUT);
                            return;
                        }
                        mbar_expect_tx(bar, (uint32_t)nb * BOX_BYTES);
                        const uint32_t stage = smem_u32(ring + (size_t)st * STAGE_BYTES);
                        for (int i = 0; i < nb; ++i)
                            tma_load_2d(stage + (uint32_t)i * BOX_BYTES, &maps.m[i0 + i], panel * CG, (int)(ch * RC), bar);
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

        for (int64_t ch = chb; ch < che; ++ch) {
            const int64_t tc = ch * RC;
            const int64_t t0 = tc + rs * DP_R;
            float2 acc[DP_R][4];
#pragma unroll
            for (int r = 0; r < DP_R; ++r)
#pragma unroll
                for (int h = 0; h < 4; ++h) acc[r][h] = make_float2(0.0f, 0.0f);
            const bool it_on = tid < items && tc + my_r < p.T;
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
                if (!mbar_wait(smem_u32(&full[st]), parity)) {
                    atomicExch(tp.status, (int)TPQ_ERR_TIMEOUT);
                    return;
                }
                const uint32_t *const sw = ring_w + (size_t)st * (STAGE_BYTES / 4);
                uint32_t w[DT_NB][DP_R];
#pragma unroll
                for (int i = 0; i < DT_NB; ++i)
#pragma unroll
                    for (int r = 0; r < DP_R; ++r) w[i][r] = sw[(i * RC + r) * CG];
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
                        for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], magic, bias);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < DT_NB; ++i)
                        if (i0 + i < N) {
                            const float4 a = st4[(2 * i) * CG], b = st4[(2 * i + 1) * CG];
                            const float2 sc[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y),
                                                  make_float2(b.z, b.w)};
#pragma unroll
                            for (int r = 0; r < DP_R; ++r) decode8(w[i][r], sc, acc[r], magic, bias);
                        }
                }
            }
            if (it_on) {  // the last step's values (a partial batch has N % DT_NB of them)
                const int nl = N - (N - 1) / DT_NB * DT_NB;
#pragma unroll
                for (int i = 0; i < DT_NB; ++i)
                    if (i < nl) hv = __fadd_rn(hv, __uint_as_float((uint32_t)hvv[i] << 16));
            }
            if (live) dp_store_rows<FP32OUT>(p, pp.lp_idx, t0, g, 0u, acc);
            if (n_it > 0) {
                asm volatile("bar.sync 1, %0;" ::"n"(DT_MAIN) : "memory");  // the chunk's rows are stored
                if (it_on) item_done(tc + my_r, my_col, my_fcol, hv);
                // panels with more items than threads (many selected features in one panel): the rest, unpipelined
                for (int a = tid + DT_MAIN; a < items; a += DT_MAIN) {
                    const int r = a / n_it, h = hs + (a - r * n_it);
                    if (tc + r >= p.T) break;
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
// Row kernel for N <= 4 devices and (E-k)/8 <= MAXT main threads.
//
// One persistent block per SM with three kinds of warps:
//   producer (1 warp)  streams groups of G rows of all N payloads (a code-row block and a BF16 block per
//                      device, 2N 1-D bulk asynchronous copies issued by 2N lanes) into a ring of
//                      shared-memory stages; completion on "full" mbarriers;
//   main (MAXT/32)     thread <-> 8 adjacent output features = one aligned word per device and row; its
//                      N x 8 steps live in registers for the life of the block (0 at holes); pure
//                      decode + 128-bit row stores, two rows at a time, no hole logic at all; arrives on
//                      "main_done" (release: its stores are ordered before what follows the barrier);
//   fix-up (4 warps)   after "main_done": one item per selected feature and row -- the sum of the
//                      devices' BF16 values goes to the selected feature's column (overwriting the 0 the
//                      main store left at a hole), and, for a hole, the filler feature whose codes the
//                      hole's slot holds is decoded and stored to the filler's column.
// Main and fix-up warps release a stage through the "empty" mbarrier; no block-wide barrier in the loop.
// G is a multiple of 4/gcd(4, L/8) so that every stage starts 16-byte aligned in the code stream.
// ----------------------------------------------------------------------------------------------
// fix-up threads: 128, or 96 where that takes the block from 25 warps (allocated as 28: 72 registers per
// thread) to 24 (80 registers) and two rows per stage leave few items
constexpr int DR_FIXUP_MAX = 128;

struct DRLayout {
    size_t lp_stage, hp_stage, stage, bars, total;
};
__host__ __device__ inline DRLayout dr_layout(int N, int E, int k, int G, int nstage)
{
    DRLayout l;
    l.lp_stage = (((size_t)G * (E - k) / 2) + 15) & ~(size_t)15;
    l.hp_stage = (size_t)G * k * 2;
    l.stage = (size_t)N * (l.lp_stage + l.hp_stage);
    l.bars = (size_t)nstage * l.stage;
    l.total = l.bars + (size_t)nstage * 24;
    return l;
}

struct DRParams {
    DQParams q;
    DXParams x;
    int G, nstage;
    int64_t ngroups;
#ifdef TPQ_TRACE
    long long *trace;
#endif
};

#ifdef TPQ_TRACE
static long long *g_dtrace = nullptr;  // 64 slots per block, globaltimer ns
__device__ __forceinline__ long long tpq_dnow()
{
    long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define TPQ_DMARK(slot) do { if (threadIdx.x == 0 && pp.trace && (slot) < 64) pp.trace[blockIdx.x * 64 + (slot)] = tpq_dnow(); } while (0)
#else
#define TPQ_DMARK(slot) do { } while (0)
#endif

template <int NMAX, int MAXT, int FX, bool FP32OUT, bool HAS_BIAS, bool HAS_WAIT>
__global__ void __launch_bounds__(MAXT + FX + 32, 1) dequant_rows(const DRParams pp)
{
    extern __shared__ __align__(128) uint8_t smem[];
    TPQ_DMARK(0);
    const DQParams &p = pp.q;
    const DXParams &x = pp.x;
    const int tid = threadIdx.x;
    const int NT = blockDim.x - FX - 32;  // main threads; then the fix-up warps; then the producer warp
    const int N = p.N, E = p.E, k = p.k, G = pp.G, nstage = pp.nstage;  // G rows per stage, even
    const int L = E - k, L8 = L >> 3;
    const DRLayout lay = dr_layout(N, E, k, G, nstage);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + lay.bars);
    uint64_t *empty = full + nstage;
    uint64_t *main_done = empty + nstage;

    // (first thing, with no load of its own in flight: behind the table loads below it would make every
    // thread wait for them ahead of the barrier that releases the producer; and an instantiation of its
    // own: even a branch that is never taken costs this prologue a few hundred cycles)
    if constexpr (HAS_WAIT) tpq_block_wait_arrivals(p.arr);
    if (tid == 0) {
        for (int s = 0; s < nstage; ++s) {
            mbar_init(smem_u32(&full[s]), 1);
            mbar_init(smem_u32(&empty[s]), (NT + FX) / 32);
            mbar_init(smem_u32(&main_done[s]), NT / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    // main-thread constants: loads issued before the barrier that releases the producer (so that they
    // are not queued behind the bulk copies)
    const int g = tid;
    const bool is_main = tid < NT;
    const bool live = is_main && g < L8;
    const int g_ld = live ? g : 0;
    float2 sc[NMAX][4];
#pragma unroll
    for (int i = 0; i < NMAX; ++i) {
#pragma unroll
        for (int h = 0; h < 4; ++h) sc[i][h] = make_float2(0.0f, 0.0f);
        if (live && i < N) load_steps(p.s_k + (size_t)i * E, g, sc[i]);
    }
    tpq_grid_dep_wait();    // the payloads and the output buffer may still be in use by the kernel ahead
    __syncthreads();
    tpq_grid_dep_launch();  // the next kernel in the stream may start its own prologue

    if (tid >= NT + FX) {
        // ---------------- producer warp: lane 0 waits for the stage and arms its barrier, then the 2N
        // copies of the stage are issued by 2N lanes at once
        const int pl = tid - NT - FX;
        int st = 0;
        uint32_t parity = 1;  // parity of the "empty" phase to wait for
        for (int it = 0;; ++it) {
            const int64_t gi = blockIdx.x + it * (int64_t)gridDim.x;
            if (gi >= pp.ngroups) break;
            const int64_t t0 = gi * G;
            const int rows = (int)((p.T - t0 < G) ? p.T - t0 : G);
            const uint32_t lp_bytes = (uint32_t)((((size_t)rows * (E - k) / 2) + 15) & ~(size_t)15);
            const uint32_t hp_bytes = (uint32_t)rows * k * 2u;
            const uint32_t bar = smem_u32(&full[st]);
            uint8_t *stage = smem + (size_t)st * lay.stage;
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
                    bulk_g2s(smem_u32(stage + (size_t)i * lay.lp_stage), p.pl[i] + t0 * ((E - k) / 2), lp_bytes, bar);
                else if (hp_bytes)
                    bulk_g2s(smem_u32(stage + (size_t)N * lay.lp_stage + (size_t)i * lay.hp_stage),
                             p.pl[i] + p.lp_bytes + t0 * k * 2, hp_bytes, bar);
            }
            if (++st == nstage) {
                st = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    const int lane = tid & 31;
    int st = 0;
    uint32_t parity = 0;

    if (!is_main) {
        // ---------------- fix-up warps
        // A thread's items of a stage are the same (row of the stage, rank) pairs in every stage, so their
        // columns, slots and steps are loaded once; sums are formed as soon as the stage has landed (they
        // read shared memory only) and stored once the main warps' row stores are done.
        const int ft = tid - NT;
        constexpr int FX_PRE = 2;  // items per thread kept in registers (more: the plain loop below)
        int f_r[FX_PRE], f_h[FX_PRE], f_hpcol[FX_PRE], f_col[FX_PRE], f_word[FX_PRE], f_sh[FX_PRE];
        float f_s[FX_PRE][NMAX], f_bh[FX_PRE], f_bf[FX_PRE];
#pragma unroll
        for (int j = 0; j < FX_PRE; ++j) {
            const int item = ft + j * FX;
            const bool on = item < G * k;
            f_r[j] = on ? item / k : -1;
            f_h[j] = on ? item - f_r[j] * k : 0;
            f_hpcol[j] = on ? __ldg(x.hp_idx + f_h[j]) : 0;
            const bool hole = on && f_h[j] < x.n_holes;
            f_col[j] = hole ? __ldg(x.filler + f_h[j]) : -1;
            const int slot = hole ? __ldg(x.hole + f_h[j]) : 0;
            f_word[j] = f_r[j] * L8 + (slot >> 3);
            f_sh[j] = (slot & 7) * 4;
#pragma unroll
            for (int i = 0; i < NMAX; ++i) f_s[j][i] = (hole && i < N) ? __ldg(p.s_k + (size_t)i * E + f_col[j]) : 0.0f;
            // (the items' biases with them: fetched in the store phase they would sit between "main_done" and
            // the release of the stage)
            f_bh[j] = (HAS_BIAS && on) ? __ldg(p.bias + f_hpcol[j]) : 0.0f;
            f_bf[j] = (HAS_BIAS && hole) ? __ldg(p.bias + f_col[j]) : 0.0f;
        }
        const int hp_dev = (int)(lay.hp_stage / 2);  // BF16 elements between two devices' blocks
        for (int it = 0;; ++it) {
            const int64_t gi = blockIdx.x + it * (int64_t)gridDim.x;
            if (gi >= pp.ngroups) break;
            if (!mbar_wait(smem_u32(&full[st]), parity)) {
                atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
            const int64_t t0 = gi * G;
            const int rows = (int)((p.T - t0 < G) ? p.T - t0 : G);
            const uint8_t *stage = smem + (size_t)st * lay.stage;
            const uint16_t *hp = reinterpret_cast<const uint16_t *>(stage + (size_t)N * lay.lp_stage);
            float hv[FX_PRE], fv[FX_PRE];
#pragma unroll
            for (int j = 0; j < FX_PRE; ++j) {
                hv[j] = 0.0f;
                fv[j] = 0.0f;
                if (f_r[j] >= 0 && f_r[j] < rows) {
#pragma unroll
                    for (int i = 0; i < NMAX; ++i)
                        if (i < N) hv[j] = __fadd_rn(hv[j], __uint_as_float((uint32_t)hp[i * hp_dev + f_r[j] * k + f_h[j]] << 16));
                    if (f_col[j] >= 0) {  // the hole's slot holds the codes of filler feature f_h
#pragma unroll
                        for (int i = 0; i < NMAX; ++i)
                            if (i < N) {
                                const uint32_t w = reinterpret_cast<const uint32_t *>(stage + (size_t)i * lay.lp_stage)[f_word[j]];
                                const float code =
                                    __fsub_rn(__uint_as_float((((w >> f_sh[j]) & 0xFu) ^ 8u) | 0x4B000000u), 8388616.0f);
                                fv[j] = __fmaf_rn(code, f_s[j][i], fv[j]);
                            }
                    }
                }
            }
            if (!mbar_wait(smem_u32(&main_done[st]), parity)) {
                atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
                break;
            }
#pragma unroll
            for (int j = 0; j < FX_PRE; ++j)
                if (f_r[j] >= 0 && f_r[j] < rows) {
                    const int64_t orow = (t0 + f_r[j]) * p.out_stride;
                    if (HAS_BIAS) {
                        hv[j] = __fadd_rn(hv[j], f_bh[j]);
                        if (f_col[j] >= 0) fv[j] = __fadd_rn(fv[j], f_bf[j]);
                    }
                    store_one<FP32OUT>(p.out, orow + f_hpcol[j], hv[j]);
                    if (f_col[j] >= 0) store_one<FP32OUT>(p.out, orow + f_col[j], fv[j]);
                }
            for (int item = ft + FX_PRE * FX; item < rows * k; item += FX) {
                const int r = item / k, h = item - r * k;  // row of the stage, rank of the selected feature
                const int64_t orow = (t0 + r) * p.out_stride;
                float v = 0.0f;
                for (int i = 0; i < N; ++i)
                    v = __fadd_rn(v, __uint_as_float((uint32_t)hp[i * hp_dev + r * k + h] << 16));
                {
                    const int hc = __ldg(x.hp_idx + h);
                    store_one<FP32OUT>(p.out, orow + hc, HAS_BIAS ? __fadd_rn(v, __ldg(p.bias + hc)) : v);
                }
                if (h < x.n_holes) {
                    const int slot = __ldg(x.hole + h), col = __ldg(x.filler + h);
                    float u = 0.0f;
                    for (int i = 0; i < N; ++i) {
                        const uint32_t w =
                            reinterpret_cast<const uint32_t *>(stage + (size_t)i * lay.lp_stage)[r * L8 + (slot >> 3)];
                        const float code = __fsub_rn(
                            __uint_as_float((((w >> ((slot & 7) * 4)) & 0xFu) ^ 8u) | 0x4B000000u), 8388616.0f);
                        u = __fmaf_rn(code, __ldg(p.s_k + (size_t)i * E + col), u);
                    }
                    store_one<FP32OUT>(p.out, orow + col, HAS_BIAS ? __fadd_rn(u, __ldg(p.bias + col)) : u);
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
    const uint32_t magic = opaque_magic();
    // 32-bit word indices into shared memory and a per-thread output pointer keep the loop's address
    // arithmetic short
    const uint32_t *const smem32 = reinterpret_cast<const uint32_t *>(smem);
    const int stage_w = (int)(lay.stage >> 2), lp_w = (int)(lay.lp_stage >> 2);
    constexpr int ESIZE = FP32OUT ? 4 : 2;
    uint8_t *const out_col = static_cast<uint8_t *>(p.out) + (size_t)8 * g_ld * ESIZE;
    const int64_t out_row_bytes = p.out_stride * ESIZE;
    float2 b[4];  // the thread's 8 biases (only in the instantiation that adds them)
#pragma unroll
    for (int h = 0; h < 4; ++h) b[h] = make_float2(0.0f, 0.0f);
    if (HAS_BIAS) {
        const float4 b0 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g_ld));
        const float4 b1 = __ldg(reinterpret_cast<const float4 *>(p.bias + 8 * g_ld + 4));
        b[0] = make_float2(b0.x, b0.y); b[1] = make_float2(b0.z, b0.w);
        b[2] = make_float2(b1.x, b1.y); b[3] = make_float2(b1.z, b1.w);
    }
    TPQ_DMARK(1);
    for (int it = 0;; ++it) {
        const int64_t gi = blockIdx.x + it * (int64_t)gridDim.x;
        if (gi >= pp.ngroups) break;
        if (!mbar_wait(smem_u32(&full[st]), parity)) {
            atomicExch(x.status, (int)TPQ_ERR_TIMEOUT);
            break;
        }
        TPQ_DMARK(2 + 2 * it);
        const int64_t t0 = gi * G;
        const int rows = (int)((p.T - t0 < G) ? p.T - t0 : G);
        const uint32_t *const sw = smem32 + st * stage_w + g_ld;  // this thread's word of row 0, device 0
        uint8_t *orow = out_col + t0 * out_row_bytes;
        for (int r0 = 0; r0 < rows; r0 += 2) {
            const bool two = r0 + 1 < rows;
            const int d1 = two ? L8 : 0;  // a ragged last stage decodes its last row twice, stores it once
            const uint32_t *const w = sw + r0 * L8;
            float2 acc[2][4];
#pragma unroll
            for (int r = 0; r < 2; ++r)
#pragma unroll
                for (int h = 0; h < 4; ++h) acc[r][h] = make_float2(0.0f, 0.0f);
#pragma unroll
            for (int i = 0; i < NMAX; ++i) {
                if (i < N) {  // uniform
                    const uint32_t w0 = w[i * lp_w];
                    const uint32_t w1 = w[i * lp_w + d1];
                    decode8(w0, sc[i], acc[0], magic);
                    decode8(w1, sc[i], acc[1], magic);
                }
            }
            if (live) {
                if (HAS_BIAS) {  // (a hole's lane gets its own column's bias here and is overwritten by the fix-up)
#pragma unroll
                    for (int r = 0; r < 2; ++r)
#pragma unroll
                        for (int h = 0; h < 4; ++h) acc[r][h] = __fadd2_rn(acc[r][h], b[h]);
                }
                store_group<FP32OUT>(orow, 0, acc[0], 0u);
                if (two) store_group<FP32OUT>(orow + out_row_bytes, 0, acc[1], 0u);
            }
            orow += 2 * out_row_bytes;
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(smem_u32(&main_done[st]));  // release: the row stores above precede the fix-up stores
            mbar_arrive(smem_u32(&empty[st]));
        }
        TPQ_DMARK(3 + 2 * it);
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

template <int NMAX, int MAXT, int FX, bool FP32OUT, bool HAS_BIAS, bool HAS_WAIT>
cudaError_t launch_rows_w(const DRParams &pp, int grid, int consumers, size_t smem, cudaStream_t st)
{
    cudaError_t e = cudaFuncSetAttribute(dequant_rows<NMAX, MAXT, FX, FP32OUT, HAS_BIAS, HAS_WAIT>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess)
        e = tpq_launch_pdl(dequant_rows<NMAX, MAXT, FX, FP32OUT, HAS_BIAS, HAS_WAIT>, dim3(grid), dim3(consumers + FX + 32), smem,
                           st, pp);
    return e;
}

template <int NMAX, int MAXT, int FX, bool FP32OUT, bool HAS_BIAS>
cudaError_t launch_rows_v(const DRParams &pp, int grid, int consumers, size_t smem, cudaStream_t st)
{
    return pp.q.arr.words ? launch_rows_w<NMAX, MAXT, FX, FP32OUT, HAS_BIAS, true>(pp, grid, consumers, smem, st)
                          : launch_rows_w<NMAX, MAXT, FX, FP32OUT, HAS_BIAS, false>(pp, grid, consumers, smem, st);
}

template <int NMAX, int MAXT, int FX>
cudaError_t launch_rows_f(const DRParams &pp, int fp32_out, int grid, int consumers, size_t smem, cudaStream_t st)
{
    const bool bias = pp.q.bias != nullptr;
    if (fp32_out)
        return bias ? launch_rows_v<NMAX, MAXT, FX, true, true>(pp, grid, consumers, smem, st)
                    : launch_rows_v<NMAX, MAXT, FX, true, false>(pp, grid, consumers, smem, st);
    return bias ? launch_rows_v<NMAX, MAXT, FX, false, true>(pp, grid, consumers, smem, st)
                : launch_rows_v<NMAX, MAXT, FX, false, false>(pp, grid, consumers, smem, st);
}

template <int NMAX, int MAXT>
cudaError_t launch_rows(const DRParams &pp, int fp32_out, int grid, int consumers, size_t smem, cudaStream_t st)
{
    // two rows per stage: G k items per stage fit three fix-up warps with two items each for k <= 96
    return (pp.G == 2 && 2 * pp.q.k <= 2 * 96) ? launch_rows_f<NMAX, MAXT, 96>(pp, fp32_out, grid, consumers, smem, st)
                                               : launch_rows_f<NMAX, MAXT, DR_FIXUP_MAX>(pp, fp32_out, grid, consumers, smem, st);
}

// Row kernel geometry; returns false if the shape does not admit it.
bool rows_plan(const tpq_ctx *c, int64_t T, int *G_out, int *nstage_out, int64_t *ngroups_out, int *grid_out)
{

    const int N = c->N, E = c->E, k = c->k;
    const int L8 = (E - k) / 8;
    // measured against the panel kernels: the row kernel wins with up to 4 devices at every input length
    // (the panel kernels scale better with N)
    if (N > 4) return false;
    if (L8 > 768) return false;  // consumer threads (register budget per thread)
    int g0 = 4;
    if (L8 % 4 == 0) g0 = 1;
    else if (L8 % 2 == 0) g0 = 2;
    int G = g0 < 2 ? 2 : g0;  // 2 or 4 rows per stage (a multiple of g0), walked two rows at a time
    // long inputs: 4-row stages amortise the per-stage work (measured faster from about 32 rows per block)
    if (G == 2 && T >= 32LL * c->sm_count && dr_layout(N, E, k, 4, 3).total <= (size_t)c->smem_optin) G = 4;
    if (dr_layout(N, E, k, G, 2).total > (size_t)c->smem_optin) return false;
    const int64_t ngroups = (T + G - 1) / G;
    const int grid = (int)(ngroups < c->sm_count ? ngroups : c->sm_count);
    const int64_t per_block = (ngroups + grid - 1) / grid;
    int nstage = (int)(per_block < 4 ? per_block : 4);  // deeper rings measured no faster (often slower)
    if (G == 4 && nstage > 3) nstage = 3;
    if (nstage < 2) nstage = 2;
    while (nstage > 2 && dr_layout(N, E, k, G, nstage).total > (size_t)c->smem_optin) --nstage;
    *G_out = G; *nstage_out = nstage; *ngroups_out = ngroups; *grid_out = grid;
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
    int L8, CG, RC;
    CUtensorMap map;
};
struct DTCache {
    static constexpr int CAP = 256;
    int n = 0, next = 0;
    DTCacheEntry e[CAP];
};

bool payload_map(tpq_ctx *c, const void *ptr, int64_t T, int L8, int CG, int RC, CUtensorMap *out)
{
    if (!c->dq_cache) c->dq_cache = new (std::nothrow) DTCache();
    DTCache *cache = static_cast<DTCache *>(c->dq_cache);
    if (cache)
        for (int j = 0; j < cache->n; ++j) {
            const DTCacheEntry &e = cache->e[j];
            if (e.ptr == ptr && e.T == T && e.L8 == L8 && e.CG == CG && e.RC == RC) {
                *out = e.map;
                return true;
            }
        }
    tpq_encode_tiled_fn fn = tpq_tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)L8, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)L8 * 4};
    const cuuint32_t box[2] = {(cuuint32_t)CG, (cuuint32_t)RC};
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    if (fn(&m, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    if (cache) {
        DTCacheEntry &e = cache->e[cache->next];
        e.ptr = ptr; e.T = T; e.L8 = L8; e.CG = CG; e.RC = RC; e.map = m;
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
    if (N > DT_MAX_DEV || L8 % 4 != 0 || T > 0x7FFFFFF0LL) return false;
    int CG = 128;
    while (CG >= 32 && dt_smem_bytes(N, CG, 2) > (size_t)c->smem_optin) CG >>= 1;
    if (CG < 32) return false;
    const int RC = DT_MAIN / CG * DP_R;
    DPParams &pp = tp.d;
    pp.CG = CG;
    pp.panels = (L8 + CG - 1) / CG;
    pp.n_chunks = (T + RC - 1) / RC;
    if (c->dq_kernel != 2 && pp.n_chunks * pp.panels < c->sm_count) return false;  // short inputs: the copy kernel starts faster
    pp.gy = 0;  // (unused: the blocks take equal runs of (panel, chunk) pairs)
    int nstage = 6;
    while (nstage > 2 && dt_smem_bytes(N, CG, nstage) > (size_t)c->smem_optin) --nstage;
    tp.nstage = nstage;
    tp.status = c->t.status;
    for (int i = 0; i < N; ++i)
        if (!payload_map(c, payloads[i], T, L8, CG, RC, &maps.m[i])) return false;
    return true;
}

template <int CG, bool FP32OUT>
cudaError_t launch_tpanels_cg(const tpq_ctx *c, const DTParams &tp, const DTMaps &maps, cudaStream_t st)
{
    const size_t smem = dt_smem_bytes(c->N, CG, tp.nstage);
    cudaError_t e = cudaFuncSetAttribute(dequant_tpanels<CG, FP32OUT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t total = (int64_t)tp.d.panels * tp.d.n_chunks;
    const unsigned grid = (unsigned)(total < c->sm_count ? total : c->sm_count);
    return tpq_launch_pdl(dequant_tpanels<CG, FP32OUT>, dim3(grid), dim3(DT_THREADS), smem, st, tp, maps);
}

template <bool FP32OUT>
cudaError_t launch_tpanels(const tpq_ctx *c, const DTParams &tp, const DTMaps &maps, cudaStream_t st)
{
    switch (tp.d.CG) {
    case 128: return launch_tpanels_cg<128, FP32OUT>(c, tp, maps, st);
    case 64: return launch_tpanels_cg<64, FP32OUT>(c, tp, maps, st);
    default: return launch_tpanels_cg<32, FP32OUT>(c, tp, maps, st);
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
        if (rows_plan(c, T, &pp.G, &pp.nstage, &pp.ngroups, &grid)) {
            pp.q = p;
            pp.x = x;
#ifdef TPQ_TRACE
            pp.trace = g_dtrace;
#endif
            const size_t smem = dr_layout(c->N, c->E, c->k, pp.G, pp.nstage).total;
            const int L8 = (c->E - c->k) / 8;
            int consumers = ((L8 + 31) / 32) * 32;
            if (consumers < 32) consumers = 32;
            cudaError_t e;
            e = consumers <= 640 ? launch_rows<4, 640>(pp, fp32_out, grid, consumers, smem, st)
                                 : launch_rows<4, 768>(pp, fp32_out, grid, consumers, smem, st);
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

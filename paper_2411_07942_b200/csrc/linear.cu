// The pre-synchronisation linear layer fused with the compressor (Section 2: f^(i)(x^(i)) = x^(i) W^(i),
// then C^(i) of Section 3 on the result): one kernel computes the device's partial sums on the tensor cores
// and writes the payload; the [T][E] BF16 partial sums never go to memory.
//
// The weight matrix is static, so its rows are put into the payload's SLOT order once (tpq_permute_weight):
// output column c < L = E - k is then the feature that slot c carries (holes already filled with their
// fillers) and columns L .. E-1 are the selected features in rank order.  The epilogue therefore has no hole
// logic: a group of 8 columns is either one 32-bit word of codes or 8 BF16 values of the BF16 block.
//
// Kernel: tcgen05 (5th-generation tensor cores), persistent: one block per SM walks 128 x BN tiles of the
// output.  Operands are staged by TMA (128-byte swizzle) in a ring of shared-memory stages that runs on
// across tiles; one thread issues tcgen05.mma (M = 128, N = BN, K = 16, BF16 x BF16 -> FP32) into one of TWO
// accumulators in tensor memory; four epilogue warps read the other one back (tcgen05.ld), round to BF16
// (the layer's output type), quantise and store, while the tensor cores work on the next tile.
//   warp 0    TMA producer (one lane)
//   warp 1    tensor-memory allocation (whole warp), MMA issue (one lane), de-allocation
//   warps 2-5 epilogue; warp w reads the 32 accumulator rows of lane quadrant w % 4
// Every wait is bounded: on expiry the block records TPQ_ERR_TIMEOUT, skips its stores, frees its tensor
// memory and returns.
#include "tpq_internal.h"

#include <cuda.h>
#include <cuda_bf16.h>

namespace {

constexpr int LQ_BM = 128, LQ_BK = 64, LQ_THREADS = 192;
constexpr int LQ_WAIT_LIMIT = 1 << 24;  // try_wait attempts (each suspends for a hardware time slice) ...
constexpr unsigned long long LQ_WAIT_NS = 1000000000ull;  // ... and one second, whichever ends first
constexpr uint32_t LQ_A_BYTES = LQ_BM * LQ_BK * 2;

__host__ __device__ constexpr uint32_t lq_stage_bytes(int BN) { return LQ_A_BYTES + (uint32_t)BN * LQ_BK * 2; }
__host__ __device__ constexpr int lq_stages(int BN)
{
    int n = (int)((200u * 1024u) / lq_stage_bytes(BN));
    return n > 8 ? 8 : n;
}
// two accumulators (the epilogue drains one while the tensor cores fill the other), a power of two of columns
__host__ __device__ constexpr uint32_t lq_tmem_cols(int BN) { return 2 * BN <= 64 ? 64 : 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512; }
__host__ __device__ constexpr size_t lq_smem_bytes(int BN)
{
    // 1024 B of slack for the manual alignment; stages; 176 B: barriers (full[8], empty[8], accumulators 2 x 2)
    // and the tensor-memory address; the reciprocal steps of two tiles
    return 1024 + (size_t)lq_stages(BN) * lq_stage_bytes(BN) + 176 + 2 * (size_t)BN * 4;
}

struct LQParams {
    int64_t T;
    int E, k, K;
    int64_t lp_bytes;       // code section size (the BF16 block starts here)
    const float *inv_s;     // [E] of this device, feature order
    const int32_t *lp_idx;  // [L] slot -> feature
    uint8_t *payload;
    uint16_t *y_slots;      // optional [T][E] BF16 partial sums in slot order (NULL: not written)
    int *status;
};

__device__ __forceinline__ bool lq_mbar_wait(uint32_t bar, uint32_t parity)
{
    unsigned long long t0 = 0;
    for (int i = 0; i < LQ_WAIT_LIMIT; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if ((i & 63) == 63) {  // and a limit in time as well as in attempts
            unsigned long long t;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
            if (t0 == 0) t0 = t;
            else if (t - t0 > LQ_WAIT_NS) return false;
        }
    }
    return false;
}

// ---- tcgen05
__device__ __forceinline__ void tc_alloc(uint32_t smem_dst, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]; BF16 inputs, FP32 accumulation
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread <-> its lane's row
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory operand descriptor: K-major tile of 128-byte rows written by TMA with the 128-byte swizzle
// (8-row groups of 1024 bytes); `addr` may be advanced by 32 bytes per K = 16 inside the swizzle atom.
__device__ __forceinline__ uint64_t lq_smem_desc(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4)   // start address
           | ((uint64_t)1 << 16)                // leading byte offset (unused with this layout): 16 B
           | ((uint64_t)(1024 >> 4) << 32)      // stride byte offset between 8-row groups
           | ((uint64_t)1 << 46)                // descriptor version of this architecture
           | ((uint64_t)2 << 61);               // 128-byte swizzle
}
// Instruction descriptor: FP32 accumulator, BF16 A and B, both K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t lq_instr_desc(int BN)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(LQ_BM >> 4) << 24);
}

// C^(i) of one value (Section 3): two binary32 roundings, clamp, round half to even; the low 4 bits of
// fl(u + 1.5 * 2^23) are the code's two's-complement nibble.
__device__ __forceinline__ uint32_t lq_code(float x, float inv)
{
    float u = __fmul_rn(x, inv);
    u = fminf(fmaxf(u, -8.0f), 7.0f);
    return __float_as_uint(__fadd_rn(u, 12582912.0f)) & 0xFu;
}

// Tile order: bands of LQ_GROUP_M row tiles; inside a band column tile by column tile, the band's row tiles
// innermost.  Blocks that run together share a weight tile, and a band's rows of x (LQ_GROUP_M x 128 x K
// values) stay in L2 while every column tile passes over them, whatever T is.
constexpr int LQ_GROUP_M = 16;
__device__ __forceinline__ void lq_tile_origin(int tile, int mt, int nt, int BN, int &m0, int &n0)
{
    const int per_band = LQ_GROUP_M * nt;
    const int band = tile / per_band, in_band = tile - band * per_band;
    const int rows = (mt - band * LQ_GROUP_M < LQ_GROUP_M) ? mt - band * LQ_GROUP_M : LQ_GROUP_M;  // the last band may be short
    const int n = in_band / rows, m = band * LQ_GROUP_M + (in_band - n * rows);
    m0 = m * LQ_BM;
    n0 = n * BN;
}

template <int BN>
__global__ void __launch_bounds__(LQ_THREADS, 1)
linear_quantize(const LQParams p, const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w)
{
    extern __shared__ uint8_t lq_raw[];
    constexpr int NS = lq_stages(BN);
    constexpr uint32_t STAGE = lq_stage_bytes(BN);
    constexpr uint32_t TCOLS = lq_tmem_cols(BN);
    const uint32_t base = (smem_u32(lq_raw) + 1023u) & ~1023u;  // swizzled tiles want 1024-byte alignment
    uint8_t *const gen = lq_raw + (base - smem_u32(lq_raw));
    // after the stages: full[8], empty[8], acc_full[2], acc_empty[2] (8 bytes each), the tensor-memory address,
    // then the reciprocal steps of two tiles
    const uint32_t bars = base + NS * STAGE;
    uint32_t *const tmem_slot = reinterpret_cast<uint32_t *>(gen + NS * STAGE + 160);
    float *const inv_tiles = reinterpret_cast<float *>(gen + NS * STAGE + 176);
    auto full = [&](int s) { return bars + 8u * s; };
    auto empty = [&](int s) { return bars + 8u * (8 + s); };
    auto acc_full = [&](int b) { return bars + 8u * (16 + b); };
    auto acc_empty = [&](int b) { return bars + 8u * (18 + b); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int L = p.E - p.k, L8 = L >> 3;
    const int nkb = (p.K + LQ_BK - 1) / LQ_BK;
    const int mt = (int)((p.T + LQ_BM - 1) / LQ_BM), nt = (p.E + BN - 1) / BN;
    const int tiles = mt * nt;

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(full(s), 1);
            mbar_init(empty(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full(b), 1);
            mbar_init(acc_empty(b), 4);  // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tc_alloc(smem_u32(tmem_slot), TCOLS);
    tc_fence_before();
    tpq_grid_dep_wait();  // the operands and the payload buffer may still be in use by the kernel ahead
    __syncthreads();
    tpq_grid_dep_launch();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool ok = true;

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;  // k-blocks issued so far, over all of this block's tiles
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                int m0, n0;
                lq_tile_origin(tile, mt, nt, BN, m0, n0);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % NS;
                    if (it >= NS && !lq_mbar_wait(empty(s), ((it / NS) - 1) & 1)) {
                        ok = false;
                        break;
                    }
                    mbar_expect_tx(full(s), STAGE);
                    tma_load_2d(base + s * STAGE, &map_x, kb * LQ_BK, m0, full(s));
                    tma_load_2d(base + s * STAGE + LQ_A_BYTES, &map_w, kb * LQ_BK, n0, full(s));
                }
            }
            if (!ok)  // giving up: let the copies already issued land before the block's shared memory is released
                for (int j = it > NS ? it - NS : 0; j < it; ++j) (void)lq_mbar_wait(full(j % NS), (j / NS) & 1);
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = lq_instr_desc(BN);
            int it = 0, n_tile = 0;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++n_tile) {
                const int b = n_tile & 1;
                // the epilogue must have drained this accumulator (used two tiles ago)
                if (n_tile >= 2 && !lq_mbar_wait(acc_empty(b), ((n_tile >> 1) - 1) & 1)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d = tmem + (uint32_t)(b * BN);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % NS;
                    if (!lq_mbar_wait(full(s), (it / NS) & 1)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a = base + s * STAGE, bb = a + LQ_A_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < LQ_BK / 16; ++k4)
                        tc_mma_bf16(d, lq_smem_desc(a + k4 * 32), lq_smem_desc(bb + k4 * 32), idesc, (kb | k4) != 0);
                    tc_commit(empty(s));  // arrives when the MMAs above have read the stage
                }
                if (ok) tc_commit(acc_full(b));  // arrives when the tile's accumulator is complete
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: tile i is drained while the tensor cores work on tile i + 1
        const int q = warp & 3, et = tid - 64;
        uint32_t *const lp_out = reinterpret_cast<uint32_t *>(p.payload);
        uint16_t *const hp_out = reinterpret_cast<uint16_t *>(p.payload + p.lp_bytes);
        int n_tile = 0;
        for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++n_tile) {
            const int b = n_tile & 1;
            int m0, n0;
            lq_tile_origin(tile, mt, nt, BN, m0, n0);
            float *const inv_tile = inv_tiles + b * BN;
            for (int c = et; c < BN; c += 128) {  // the tile's reciprocal steps in slot order
                const int col = n0 + c;
                inv_tile[c] = (col < L) ? __ldg(p.inv_s + __ldg(p.lp_idx + col)) : 0.0f;
            }
            // barrier of the four epilogue warps (the steps above are in place) that also tells every thread
            // whether ANY of them has given up: they leave the loop together, none is left waiting here
            uint32_t any_bad;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 q, %1, 0;\n\t"
                "bar.red.or.pred p, 1, 128, q;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(any_bad)
                : "r"((uint32_t)!ok)
                : "memory");
            if (any_bad) {
                ok = false;
                break;
            }
            if (!lq_mbar_wait(acc_full(b), (n_tile >> 1) & 1)) ok = false;
            ok = __all_sync(0xffffffffu, ok);  // the tensor-memory loads below are warp-wide
            if (!ok) continue;                 // (reported at the next barrier above; no tile follows a lost one)
            tc_fence_after();
            const int64_t row = (int64_t)m0 + q * 32 + lane;
            const bool row_on = row < p.T;
            for (int c0 = 0; c0 < BN; c0 += 32) {
                if (n0 + c0 >= p.E) break;  // uniform
                uint32_t r[32];
                tc_ld_32x32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(b * BN + c0), r);
#pragma unroll
                for (int g = 0; g < 4; ++g) {
                    const int col = n0 + c0 + 8 * g;
                    if (col >= p.E) break;
                    uint32_t h[4];  // the 8 sums rounded to BF16 (the layer's output type), packed in pairs
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[8 * g + 2 * j]),
                                                                       __uint_as_float(r[8 * g + 2 * j + 1]));
                        h[j] = *reinterpret_cast<const uint32_t *>(&v);
                    }
                    if (!row_on) continue;
                    if (p.y_slots) *reinterpret_cast<uint4 *>(p.y_slots + row * p.E + col) = make_uint4(h[0], h[1], h[2], h[3]);
                    if (col < L) {
                        const float4 i0 = *reinterpret_cast<const float4 *>(inv_tile + c0 + 8 * g);
                        const float4 i1 = *reinterpret_cast<const float4 *>(inv_tile + c0 + 8 * g + 4);
                        const float iv[8] = {i0.x, i0.y, i0.z, i0.w, i1.x, i1.y, i1.z, i1.w};
                        uint32_t word = 0;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t c_lo = lq_code(__uint_as_float(h[j] << 16), iv[2 * j]);
                            const uint32_t c_hi = lq_code(__uint_as_float(h[j] & 0xFFFF0000u), iv[2 * j + 1]);
                            word |= (c_lo << (8 * j)) | (c_hi << (8 * j + 4));
                        }
                        lp_out[row * L8 + (col >> 3)] = word;
                    } else {
                        *reinterpret_cast<uint4 *>(hp_out + row * p.k + (col - L)) = make_uint4(h[0], h[1], h[2], h[3]);
                    }
                }
            }
            // this warp has read its quadrant of the accumulator: hand it back to the MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty(b)) : "memory");
        }
        // zero padding of the code section (its size is rounded up to 16 bytes)
        if (blockIdx.x == 0 && warp == 2) {
            const int64_t valid = p.T * L8, words = p.lp_bytes / 4;
            for (int64_t w = valid + lane; w < words; w += 32) lp_out[w] = 0u;
        }
    }
    if (!ok) atomicExch(p.status, (int)TPQ_ERR_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tc_dealloc(tmem, TCOLS);
    }
}

// rows of a [E][K] weight matrix gathered into slot order: row c < L from feature lp_idx[c], row L + h from hp_idx[h]
__global__ void __launch_bounds__(256) permute_weight(const uint16_t *__restrict__ w, uint16_t *__restrict__ out, int E, int k,
                                                      int64_t K, const int32_t *__restrict__ lp_idx,
                                                      const int32_t *__restrict__ hp_idx)
{
    const int r = blockIdx.x, L = E - k;
    const int src = r < L ? __ldg(lp_idx + r) : __ldg(hp_idx + (r - L));
    const uint16_t *in = w + (int64_t)src * K;
    uint16_t *o = out + (int64_t)r * K;
    if ((K & 7) == 0) {
        for (int64_t c = threadIdx.x; c < K / 8; c += blockDim.x)
            reinterpret_cast<uint4 *>(o)[c] = __ldg(reinterpret_cast<const uint4 *>(in) + c);
    } else {
        for (int64_t c = threadIdx.x; c < K; c += blockDim.x) o[c] = in[c];
    }
}


// [rows][K] BF16, row-major -> boxes of box_rows x 64 elements with the 128-byte swizzle; out-of-range reads give 0
bool lq_map(const void *ptr, int64_t rows, int64_t K, int box_rows, CUtensorMap *out)
{
    tpq_encode_tiled_fn fn = tpq_tensor_map_encoder();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)LQ_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t lq_launch(const LQParams &p, const void *x, const void *w, int sm_count, cudaStream_t st)
{
    CUtensorMap mx, mw;
    if (!lq_map(x, p.T, p.K, LQ_BM, &mx) || !lq_map(w, p.E, p.K, BN, &mw)) return cudaErrorNotSupported;
    const size_t smem = lq_smem_bytes(BN);
    cudaError_t e = cudaFuncSetAttribute(linear_quantize<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const int64_t tiles = ((p.T + LQ_BM - 1) / LQ_BM) * ((p.E + BN - 1) / BN);
    const dim3 grid((unsigned)(tiles < sm_count ? tiles : sm_count));  // persistent: a block walks tiles b, b + grid, ...
    return tpq_launch_pdl(linear_quantize<BN>, grid, dim3(LQ_THREADS), smem, st, p, mx, mw);
}

}  // namespace

bool tpq_linear_ok(const tpq_ctx *c, int64_t T, int64_t K)
{
    if (c->bits != 4) return false;
    if (c->E % 8 || c->k % 8 || c->E - c->k < 8) return false;
    if (T < 1 || K < 8 || K % 8) return false;  // 16-byte row pitch for the tensor maps
    if (T > (int64_t)1 << 31 || K > (int64_t)1 << 31) return false;
    return lq_smem_bytes(256) <= (size_t)c->smem_optin;
}

cudaError_t tpq_launch_permute_weight(const tpq_ctx *c, const void *w, void *out, int64_t K, cudaStream_t st, int64_t *launches)
{
    permute_weight<<<c->E, 256, 0, st>>>(static_cast<const uint16_t *>(w), static_cast<uint16_t *>(out), c->E, c->k, K,
                                         c->t.lp_idx, c->t.hp_idx);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_linear_quantize(const tpq_ctx *c, int shard, const void *x, const void *w_slots, int64_t T, int64_t K,
                                       void *payload, void *y_slots, cudaStream_t st, int64_t *launches)
{
    LQParams p;
    p.T = T; p.E = c->E; p.k = c->k; p.K = (int)K;
    p.lp_bytes = tpq_lp_bytes_i(T, c->E, c->k);
    p.inv_s = c->t.inv_s + (size_t)shard * c->E;
    p.lp_idx = c->t.lp_idx;
    p.payload = static_cast<uint8_t *>(payload);
    p.y_slots = static_cast<uint16_t *>(y_slots);
    p.status = c->t.status;
    // Tile width.  A block's time is (tiles it walks) x (k-blocks per tile) x (time per k-block), and the time
    // per k-block barely depends on the width (the operand pipeline, not the tensor pipe, sets it: measured
    // 385 / 376 / 344 ns for 256 / 192 / 128 columns), so the widest tile wins unless a narrower one saves a
    // whole wave of the persistent grid.
    const int64_t mt = (T + LQ_BM - 1) / LQ_BM;
    int best = 256;
    double best_cost = 0.0;
    for (int bn : {256, 192, 128}) {
        const int64_t tiles = mt * ((c->E + bn - 1) / bn);
        const int64_t waves = (tiles + c->sm_count - 1) / c->sm_count;
        const double cost = (double)waves * (bn == 256 ? 385.0 : bn == 192 ? 376.0 : 344.0);
        if (best_cost == 0.0 || cost < best_cost - 1e-9) {
            best_cost = cost;
            best = bn;
        }
    }
    cudaError_t e = best == 256 ? lq_launch<256>(p, x, w_slots, c->sm_count, st)
                  : best == 192 ? lq_launch<192>(p, x, w_slots, c->sm_count, st)
                                : lq_launch<128>(p, x, w_slots, c->sm_count, st);
    if (e == cudaSuccess) ++*launches;
    return e;
}

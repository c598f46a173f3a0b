// C^(i): quantise one device's BF16 partial sums to static symmetric Int4 and pack
// them, selected features passed through in BF16 (paper Section 3, Figure 2).
//
// Per low-precision element: u = fl(x * inv_s); u clamped to [-8, 7]; code = rne(u).
// The two roundings are kept separate (__fmul_rn, then the magic-constant add).
#include "tpq_internal.h"

#include <type_traits>

namespace {

// ----------------------------------------------------------------------------------------------
// Shape-generic kernel: one thread per 32-bit word of the code stream, any E, k, stride and any code
// width of 2..8 bits (a code that straddles two words is quantised by both words' threads).
// ----------------------------------------------------------------------------------------------
__device__ __forceinline__ int quant_one(uint16_t x, float inv_s, float lo, float hi)
{
    float u = __fmul_rn(__uint_as_float((uint32_t)x << 16), inv_s);
    u = fminf(fmaxf(u, lo), hi);
    return __float2int_rn(u);
}

__global__ void __launch_bounds__(256) quantize_generic(const uint16_t *__restrict__ y, int64_t T, int64_t stride, int E,
                                                        int k, int bits, const float *__restrict__ inv_s,
                                                        const int32_t *__restrict__ lp_idx,
                                                        const int32_t *__restrict__ hp_idx,
                                                        uint32_t *__restrict__ lp_out, int64_t lp_words,
                                                        uint16_t *__restrict__ hp_out)
{
    const int64_t L = E - k;
    const int64_t n_codes = T * L;
    const int64_t hp_elems = T * k;
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t gsz = (int64_t)gridDim.x * blockDim.x;
    const float lo = -(float)(1 << (bits - 1)), hi = (float)((1 << (bits - 1)) - 1);
    const uint32_t cmask = (1u << bits) - 1u;
    for (int64_t w = gid; w < lp_words; w += gsz) {
        uint32_t word = 0;
        const int64_t bit0 = 32 * w;           // the word holds bits [bit0, bit0 + 32) of the stream
        int64_t p = bit0 / bits;               // first code with a bit in the word
        if (p < n_codes) {
            int64_t t = p / L;
            int64_t c = p - t * L;
#pragma unroll 1
            for (; p < n_codes && p * bits < bit0 + 32; ++p) {
                const int j = lp_idx[c];
                const uint32_t u = (uint32_t)quant_one(y[t * stride + j], inv_s[j], lo, hi) & cmask;
                const int o = (int)(p * bits - bit0);   // may be negative: the code starts in the previous word
                word |= (o >= 0) ? (u << o) : (u >> -o);
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
// One persistent block per SM: a producer warp streams groups of G rows into a ring of shared-memory
// stages with 1-D bulk asynchronous copies (cp.async.bulk, completion on "full" mbarriers); consumer
// warps release a stage through an "empty" mbarrier.  There is no block-wide barrier in the loop.
//
// Consumer thread <-> 8 adjacent features (one 128-bit shared load per row); their reciprocal steps
// stay in registers for the life of the block.  In the payload's slot order a group of 8 adjacent
// features below L = E-k IS one 32-bit word of the code stream, so the thread stores its word
// directly (coalesced 32-bit stores).  Where one of its 8 features is a selected one (a "hole"), the
// slot belongs to a filler feature from the last k: the thread quantises that one element too
// (16-bit shared load) and drops its code into the hole.  Threads h < k copy selected feature h of
// every row to the BF16 block.
// ----------------------------------------------------------------------------------------------
constexpr int QP_MAX_GPT = 4;          // groups of 8 features per thread
constexpr int QP_MAX_CONSUMERS = 992;  // 31 consumer warps + 1 producer warp per block

constexpr int QP_PREFETCH_ROWS = 8;  // rows whose bytes a block asks L2 for ahead of the dependency wait (measured at
                                     // 2048 x 5120: none 7.7 us, 4 rows 7.0, 8 rows 6.8, all 14 rows 7.4)

constexpr int QP_MAX_BATCH = 16;  // devices' shards quantised by one launch (each by its own set of blocks)

struct QPParams {
    const uint16_t *y[QP_MAX_BATCH];   // one input per shard of the batch
    uint8_t *payload[QP_MAX_BATCH];    // and its payload
    int cps;                           // blocks per shard: block b works on shard b / cps
    int64_t lp_bytes;                  // size of a payload's code section (the BF16 block follows)
    int64_t stride;
    int64_t T;
    int E, k;
    int G;        // rows per stage
    int first;    // rows of a block's first stage (<= G: a short first stage lands sooner)
    int prefetch_rows;  // rows whose bytes a block asks L2 for ahead of the dependency wait
    int64_t rows_per_block;  // a block quantises rows_per_block adjacent rows of its shard
    int nstage;
    const float *inv_s;     // [E] of the batch's first device; device d of the batch at inv_s + d*E
    const uint32_t *grp;    // [E/8]
    const int32_t *filler;  // [n_holes]
    const int32_t *hp_idx;  // [k]
    int64_t lp_words;       // words of the code section, padding included
    int *status;
    // push mode (one shard, n_dst copies of its payload: payload[0 .. n_dst), possibly in peers' memory)
    int n_dst;
    uint32_t epoch;                     // value written to every arrival word once the payload is complete
    uint32_t *arrived[QP_MAX_BATCH];    // arrival word beside destination d (same memory as payload[d])
    unsigned int *done;                 // blocks that have finished their stores (returns to 0)
};

// Dynamic shared memory layout (byte offsets).
struct QPLayout {
    size_t ring, bars, total;
};
__host__ __device__ inline QPLayout qp_layout(int E, int G, int nstage)
{
    QPLayout l;
    l.ring = 0;
    l.bars = (size_t)nstage * G * E * 2;
    l.total = l.bars + (size_t)nstage * 16;
    return l;
}


// One element: product rounded to binary32, clamped, rounded half-to-even by the magic add; returns the
// bits of fl(u + 1.5*2^23) = 0x4B400000 + code.
__device__ __forceinline__ uint32_t quant_bits(uint32_t x_bf16, float inv_s)
{
    float u = __fmul_rn(__uint_as_float(x_bf16 << 16), inv_s);
    u = fminf(fmaxf(u, -8.0f), 7.0f);
    return __float_as_uint(__fadd_rn(u, 12582912.0f));
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

// PUSH: every payload store goes to n_dst destinations (plain stores; a destination may be a peer's
// memory), and the block that finishes last publishes the arrival words.
template <int GPT, int G, int TB, bool PUSH>  // TB: upper bound of the block size (register budget)
__global__ void __launch_bounds__(TB, 1) quantize_tiled(const QPParams p)
{
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ int s_failed;  // (push mode) a wait of this block ran out
    const int tid = threadIdx.x;
    const int NT = blockDim.x - 32;  // consumer threads
    if (PUSH && tid == 0) s_failed = 0;  // (ordered before any use by the named barrier of the prologue)
    // this block's shard of the batch, its index among the shard's blocks, and the shard's buffers
    const int sb = blockIdx.x / p.cps;
    const int bx = blockIdx.x - sb * p.cps;
    const uint16_t *const y_in = p.y[sb];
    uint32_t *const lp_out = reinterpret_cast<uint32_t *>(p.payload[sb]);
    uint16_t *const hp_out = reinterpret_cast<uint16_t *>(p.payload[sb] + p.lp_bytes);
    const float *const inv_s = p.inv_s + (size_t)sb * p.E;
    const int E = p.E, k = p.k, nstage = p.nstage;  // G rows per stage, unrolled: G independent chains per thread
    const int E8 = E >> 3, L8 = (E - k) >> 3;
    const uint32_t row_bytes = (uint32_t)E * 2u;
    const uint32_t stage_bytes = (uint32_t)G * row_bytes;
    const QPLayout lay = qp_layout(E, G, nstage);
    uint8_t *ring = smem + lay.ring;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + lay.bars);
    uint64_t *empty = full + nstage;

    // this block's rows
    const int64_t t_begin = (int64_t)bx * p.rows_per_block;
    const int64_t t_end = (p.T - t_begin < p.rows_per_block) ? p.T : t_begin + p.rows_per_block;
    const int rows_mine = (int)(t_end - t_begin);
    // first row (within the block's run) and row count of the block's it-th stage
    auto stage_row = [&](int it) { return it == 0 ? 0 : p.first + (it - 1) * G; };
    auto stage_rows = [&](int it, int r0) {
        const int cap = it == 0 ? p.first : G;
        return rows_mine - r0 < cap ? rows_mine - r0 : cap;
    };

    // Order of the prologue.  The producer warp sets up the barriers, waits for the kernel ahead in the stream
    // and issues the first stages' copies at once; the consumers' table loads run in the shadow of the first
    // stage's flight.  Only the producer executes griddepcontrol.wait: every store of a consumer follows a
    // "full" barrier that one of the producer's copies completes, i.e. follows that wait.
    tpq_grid_dep_launch();  // the next kernel in the stream may start its own prologue as SMs free up
    if (tid >= NT) {
        // ---------------- producer warp: lane 0 waits for the stage and arms its barrier; a contiguous
        // input is one copy per stage, a strided one is one copy per row, issued by as many lanes at once
        const int pl = tid - NT;
        if (pl == 0) {
            for (int s = 0; s < nstage; ++s) {
                mbar_init(smem_u32(&full[s]), 1);
                mbar_init(smem_u32(&empty[s]), NT / 32);
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        __syncwarp();
        asm volatile("bar.arrive 1, %0;" ::"r"(blockDim.x) : "memory");  // the barriers exist
        if (pl == 0 && p.stride == E) {
            // the block's first rows may start their way from HBM to L2 while it waits (a hint only: L2 is the
            // point of coherence, so whatever the kernel ahead still writes is what the copies will read)
            const int rows = rows_mine < p.prefetch_rows ? rows_mine : p.prefetch_rows;
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(y_in + t_begin * p.stride), "r"(rows * row_bytes) : "memory");
        }
        tpq_grid_dep_wait();  // the input and the payload buffer may still be in use by the kernel ahead
        int st = 0;
        uint32_t parity = 1;  // parity of the "empty" phase to wait for
        for (int it = 0;; ++it) {
            const int r0 = stage_row(it);
            if (r0 >= rows_mine) break;
            const int rows = stage_rows(it, r0);
            const int64_t t0 = t_begin + r0;
            const uint32_t bar = smem_u32(&full[st]);
            const uint32_t dst = smem_u32(ring + (size_t)st * stage_bytes);
            int ok = 1;
            if (pl == 0) {
                if (it >= nstage && !mbar_wait(smem_u32(&empty[st]), parity)) {
                    atomicExch(p.status, (int)TPQ_ERR_TIMEOUT);
                    ok = 0;
                } else {
                    mbar_expect_tx(bar, rows * row_bytes);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            if (p.stride == E) {
                if (pl == 0) bulk_g2s(dst, y_in + t0 * p.stride, rows * row_bytes, bar);
            } else {
                for (int r = pl; r < rows; r += 32)
                    bulk_g2s(dst + r * row_bytes, y_in + (t0 + r) * p.stride, row_bytes, bar);
            }
            if (++st == nstage) {
                st = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    // ---- consumer constants
    float2 inv[GPT][4];
    uint32_t mask[GPT];      // selected features among the thread's 8 (only where the group is below L)
    int hb[GPT];             // holes before the group
    // the first two holes of the group: bit position of the hole's nibble in the word and its mask
    uint32_t f_sh[GPT][2], hmask[GPT][2];
    int my_hp = 0;
    {
#pragma unroll
        for (int a = 0; a < GPT; ++a) {
            const int g = tid + a * NT;
            mask[a] = 0; hb[a] = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) inv[a][i] = make_float2(0.0f, 0.0f);
            f_sh[a][0] = f_sh[a][1] = 0;
            hmask[a][0] = hmask[a][1] = 0;
            if (g < L8) {
                const float4 i0 = __ldg(reinterpret_cast<const float4 *>(inv_s + 8 * g));
                const float4 i1 = __ldg(reinterpret_cast<const float4 *>(inv_s + 8 * g + 4));
                const uint32_t gd = __ldg(p.grp + g);
                inv[a][0] = make_float2(i0.x, i0.y);
                inv[a][1] = make_float2(i0.z, i0.w);
                inv[a][2] = make_float2(i1.x, i1.y);
                inv[a][3] = make_float2(i1.z, i1.w);
                mask[a] = gd & 0xFFu;
                hb[a] = (int)(gd >> 8);
            }
        }
        if (tid < k) my_hp = __ldg(p.hp_idx + tid);
    }
    // ---------------- consumers
    // Holes are patched warp-cooperatively.  The holes of a warp's 32 groups are consecutive in the
    // global hole order, so lane i quantises the filler element of the warp's i-th hole (w_off / w_inv)
    // and the owner of a hole fetches the code with a shuffle (from lane src0, src0 + 1 for a second
    // hole).  A warp with more than 32 holes, or a lane with more than two, takes the serial path.
    const int lane = tid & 31;
    uint32_t w_off[GPT];     // byte offset of "my" filler element in a staged row (lane < n_wh)
    float w_inv[GPT];
    int n_wh[GPT], src0[GPT];
    bool serial[GPT];
    uint32_t keep[GPT];      // word bits that are not holes
#pragma unroll
    for (int a = 0; a < GPT; ++a) {
        const int nh = __popc(mask[a]);
        int incl = nh;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += o;
        }
        src0[a] = incl - nh;
        n_wh[a] = __shfl_sync(0xffffffffu, incl, 31);
        const int hb_warp = __shfl_sync(0xffffffffu, hb[a], 0);
        serial[a] = n_wh[a] > 32 || __any_sync(0xffffffffu, nh > 2);
        w_off[a] = 0;
        w_inv[a] = 0.0f;
        if (lane < n_wh[a] && !serial[a]) {
            const int f = __ldg(p.filler + hb_warp + lane);
            w_off[a] = (uint32_t)f * 2u;
            w_inv[a] = __ldg(inv_s + f);
        }
        uint32_t m = mask[a];
        keep[a] = 0xFFFFFFFFu;
        for (int h = 0; h < 2 && m; ++h) {
            f_sh[a][h] = (uint32_t)(__ffs(m) - 1) * 4u;
            hmask[a][h] = 0xFu << f_sh[a][h];
            keep[a] &= ~hmask[a][h];
            m &= m - 1;
        }
    }

    asm volatile("bar.sync 1, %0;" ::"r"(blockDim.x) : "memory");  // the producer has set up the barriers

    int st = 0;
    uint32_t parity = 0;
    for (int it = 0;; ++it) {
        const int r0s = stage_row(it);
        if (r0s >= rows_mine) break;
        const int rows = stage_rows(it, r0s);
        if (!mbar_wait(smem_u32(&full[st]), parity)) {
            atomicExch(p.status, (int)TPQ_ERR_TIMEOUT);
            if constexpr (PUSH) s_failed = 1;  // this block's part of the payload is incomplete
            break;
        }
        const int64_t t0 = t_begin + r0s;
        const uint4 *stage = reinterpret_cast<const uint4 *>(ring + (size_t)st * stage_bytes);
        const uint16_t *stage16 = reinterpret_cast<const uint16_t *>(stage);
        const uint8_t *stage8 = reinterpret_cast<const uint8_t *>(stage);
#pragma unroll
        for (int a = 0; a < GPT; ++a) {
            const int g = tid + a * NT;
            const bool live = g < L8;
            const int g_ld = live ? g : 0;  // idle lanes load something harmless: straight-line code below
            // GR rows from row rb of the stage on: all shared loads first, then GR independent chains, no branches
            auto rows_fast = [&](auto gr_tag, int rb) {
                constexpr int GR = decltype(gr_tag)::value;
                uint4 v[GR];
                uint32_t fx[GR];
#pragma unroll
                for (int r = 0; r < GR; ++r) {
                    v[r] = stage[(rb + r) * E8 + g_ld];
                    fx[r] = *reinterpret_cast<const uint16_t *>(stage8 + (size_t)(rb + r) * row_bytes + w_off[a]);
                }
                uint32_t word[GR];
#pragma unroll
                for (int r = 0; r < GR; ++r) word[r] = quant8(v[r], inv[a]);
                if (n_wh[a]) {  // uniform over the warp
#pragma unroll
                    for (int r = 0; r < GR; ++r) {
                        const uint32_t qv = quant_bits(fx[r], w_inv[a]) & 0xFu;
                        const uint32_t q0 = __shfl_sync(0xffffffffu, qv, src0[a]) << f_sh[a][0];
                        const uint32_t q1 = __shfl_sync(0xffffffffu, qv, src0[a] + 1) << f_sh[a][1];
                        word[r] = (word[r] & keep[a]) | (q0 & hmask[a][0]) | (q1 & hmask[a][1]);
                    }
                }
                if (live) {
                    if constexpr (PUSH) {
                        for (int d = 0; d < p.n_dst; ++d) {
                            uint32_t *const o = reinterpret_cast<uint32_t *>(p.payload[d]) + (t0 + rb) * L8 + g;
#pragma unroll
                            for (int r = 0; r < GR; ++r) o[r * L8] = word[r];
                        }
                    } else {
#pragma unroll
                        for (int r = 0; r < GR; ++r) lp_out[(t0 + rb + r) * L8 + g] = word[r];
                    }
                }
            };
            if (!serial[a]) {  // (uniform over the warp, like the row counts below)
                int rb = 0;
                if (G >= 4 && rows - rb >= 4) { rows_fast(std::integral_constant<int, 4>(), rb); rb += 4; }
                if (G >= 2 && rows - rb >= 2) { rows_fast(std::integral_constant<int, 2>(), rb); rb += 2; }
                if (rows - rb >= 1) rows_fast(std::integral_constant<int, 1>(), rb);
            } else if (live) {
                // a warp on the serial path: every hole patched by its owner
                for (int r = 0; r < rows; ++r) {
                    uint32_t word = quant8(stage[r * E8 + g], inv[a]);
                    uint32_t m = mask[a];
                    for (int h = 0; m; ++h) {
                        const int n = __ffs(m) - 1;
                        m &= m - 1;
                        const int f = __ldg(p.filler + hb[a] + h);
                        const uint32_t x = *reinterpret_cast<const uint16_t *>(stage8 + (size_t)r * row_bytes + 2 * f);
                        const uint32_t q = quant_bits(x, __ldg(inv_s + f)) & 0xFu;
                        word = (word & ~(0xFu << (4 * n))) | (q << (4 * n));
                    }
                    if constexpr (PUSH) {
                        for (int d = 0; d < p.n_dst; ++d)
                            reinterpret_cast<uint32_t *>(p.payload[d])[(t0 + r) * L8 + g] = word;
                    } else {
                        lp_out[(t0 + r) * L8 + g] = word;
                    }
                }
            }
        }
        for (int h = tid; h < k; h += NT) {
            const int j = (h == tid) ? my_hp : __ldg(p.hp_idx + h);
            if constexpr (PUSH) {
                for (int d = 0; d < p.n_dst; ++d) {
                    uint16_t *const o = reinterpret_cast<uint16_t *>(p.payload[d] + p.lp_bytes) + t0 * k + h;
                    for (int r = 0; r < rows; ++r) o[r * k] = stage16[r * E + j];
                }
            } else {
                for (int r = 0; r < rows; ++r) hp_out[(t0 + r) * k + h] = stage16[r * E + j];
            }
        }
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(smem_u32(&empty[st]));
        if (++st == nstage) {
            st = 0;
            parity ^= 1u;
        }
    }
    // zero padding of the code section (at most 3 words), by the block that owned the last rows
    if (t_begin < p.T && p.T <= t_end) {
        const int64_t valid = p.T * L8;
        for (int64_t w = valid + tid; w < p.lp_words; w += NT) {
            if constexpr (PUSH) {
                for (int d = 0; d < p.n_dst; ++d) reinterpret_cast<uint32_t *>(p.payload[d])[w] = 0u;
            } else {
                lp_out[w] = 0u;
            }
        }
    }
    if constexpr (PUSH) {
        // Publication.  The block's consumer threads meet (their stores happen-before the fence below), one
        // thread orders them before its count at system scope; the block that counts last has thereby
        // observed every other block's stores and releases the arrival words to the destinations' owners.
        asm volatile("bar.sync 2, %0;" ::"r"(NT) : "memory");
        if (tid == 0) {
            __threadfence_system();
            // a block whose waits ran out counts in the upper half as well: the payload is then incomplete,
            // the words are not written, and the receivers' own bounded waits flag the step
            const unsigned int prev = atomicAdd(p.done, s_failed ? 0x10001u : 1u);
            if ((prev & 0xFFFFu) == gridDim.x - 1) {
                *p.done = 0u;  // the next launch in the stream starts from zero
                if ((prev >> 16) == 0 && !s_failed) {
                    // one fence (acquire side of the counts above, release side of the words below), then the
                    // words as relaxed system-scope stores: together a release of everything observed so far
                    __threadfence_system();
                    for (int d = 0; d < p.n_dst; ++d)
                        asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p.arrived[d]), "r"(p.epoch) : "memory");
                }
            }
        }
    }
}

// Arrival words published on their own (after payload copies made by the copy engine in stream order).
__global__ void publish_arrivals(QPParams p)
{
    const int d = threadIdx.x;
    if (d < p.n_dst) {
        __threadfence_system();
        asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p.arrived[d]), "r"(p.epoch) : "memory");
    }
}

// Bounded wait for n arrival words (this GPU's own memory, written by the pushing devices) to reach `epoch`.
__global__ void wait_arrivals(const uint32_t *arrived, int n, uint32_t epoch, unsigned long long timeout_ns, int *status)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (;;) {
        uint32_t v;
        asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(arrived + i) : "memory");
        if (v == epoch) return;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        if (t1 - t0 > timeout_ns) {
            atomicExch(status, (int)TPQ_ERR_TIMEOUT);
            return;
        }
        __nanosleep(200);
    }
}

size_t qp_smem_bytes(int E, int G, int nstage) { return qp_layout(E, G, nstage).total; }

}  // namespace

bool tpq_quantize_tiled_ok(const tpq_ctx *c, int64_t T, int64_t stride)
{
    if (c->bits != 4) return false;  // the tiled kernels are Int4 kernels
    const int E = c->E, k = c->k;
    if (E % 8 || k % 8 || stride % 8 || T <= 0) return false;
    if (E - k < 8) return false;
    if (E / 8 > QP_MAX_CONSUMERS * QP_MAX_GPT) return false;
    if (qp_smem_bytes(E, 1, 2) > (size_t)c->smem_optin) return false;
    return true;
}

cudaError_t tpq_launch_quantize_generic(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                        uint8_t *payload, cudaStream_t st, int64_t *launches)
{
    const int E = c->E, k = c->k;
    const int64_t lpb = tpq_lp_bytes_i(T, E, k, c->bits);
    const int64_t lp_words = lpb / 4;
    int64_t work = lp_words > T * k ? lp_words : T * (int64_t)k;
    int64_t blocks = (work + 255) / 256;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (blocks < 1) blocks = 1;
    quantize_generic<<<(unsigned)blocks, 256, 0, st>>>(y, T, stride, E, k, c->bits, c->t.inv_s + (size_t)shard * E, c->t.lp_idx,
                                                       c->t.hp_idx, reinterpret_cast<uint32_t *>(payload), lp_words,
                                                       reinterpret_cast<uint16_t *>(payload + lpb));
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_quantize_tiled(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                      uint8_t *payload, cudaStream_t st, int64_t *launches)
{
    const void *ys[1] = {y};
    void *pls[1] = {payload};
    return tpq_launch_quantize_tiled_batch(c, shard, 1, ys, T, stride, pls, st, launches);
}

namespace {

struct PushArgs {
    int n_dst;
    void *const *dst;
    uint32_t *const *arrived;
    uint32_t epoch;
};

cudaError_t launch_tiled(const tpq_ctx *c, int shard0, int n, const void *const *ys, int64_t T, int64_t stride,
                         void *const *payloads, const PushArgs *push, cudaStream_t st, int64_t *launches)
{
    if (n > QP_MAX_BATCH) {  // more shards than one launch carries: several launches
        for (int b = 0; b < n; b += QP_MAX_BATCH) {
            const int nb = n - b < QP_MAX_BATCH ? n - b : QP_MAX_BATCH;
            cudaError_t e = launch_tiled(c, shard0 + b, nb, ys + b, T, stride, payloads + b, nullptr, st, launches);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }
    const int E = c->E, k = c->k;
    const int E8 = E / 8;
    const int gpt = (E8 + QP_MAX_CONSUMERS - 1) / QP_MAX_CONSUMERS;
    const int nt = ((E8 + gpt - 1) / gpt + 31) / 32 * 32;
    // blocks per shard: the SMs are divided among the shards of the batch (one persistent block per SM)
    int cps = c->sm_count / n;
    if (cps < 1) cps = 1;
    // every block takes the same number of adjacent rows of its shard, so none has more than a row above the
    // mean; it walks them four at a time where a ring of three such stages fits (else two, else one), and a
    // short first stage lands sooner
    if (T < cps) cps = (int)T;
    const int64_t rpb = (T + cps - 1) / cps;
    cps = (int)((T + rpb - 1) / rpb);
    int G = 4;
    while (G > 1 && (rpb < G || qp_smem_bytes(E, G, 3) > (size_t)c->smem_optin)) G >>= 1;
    const int first = (G == 4 && rpb > 4) ? 2 : G;
    const int64_t grid = (int64_t)cps * n;
    const int64_t per_block = (rpb + G - 1) / G + (first < G ? 1 : 0);
    int nstage = (int)(per_block < 8 ? per_block : 8);
    if (nstage < 2) nstage = 2;
    while (nstage > 2 && qp_smem_bytes(E, G, nstage) > (size_t)c->smem_optin) --nstage;

    QPParams p;
    const int64_t lpb = tpq_lp_bytes_i(T, E, k);
    for (int b = 0; b < n; ++b) {
        p.y[b] = static_cast<const uint16_t *>(ys[b]);
        p.payload[b] = static_cast<uint8_t *>(payloads[b]);
    }
    p.n_dst = 0; p.epoch = 0; p.done = c->t.push_done;
    if (push) {  // one shard, n_dst destinations
        p.n_dst = push->n_dst;
        p.epoch = push->epoch;
        for (int d = 0; d < push->n_dst; ++d) {
            p.payload[d] = static_cast<uint8_t *>(push->dst[d]);
            p.arrived[d] = push->arrived[d];
        }
    }
    p.cps = cps; p.lp_bytes = lpb;
    p.stride = stride; p.T = T; p.E = E; p.k = k; p.G = G; p.first = first; p.rows_per_block = rpb; p.nstage = nstage;
    p.prefetch_rows = QP_PREFETCH_ROWS;
    p.inv_s = c->t.inv_s + (size_t)shard0 * E; p.grp = c->t.grp; p.filler = c->t.filler; p.hp_idx = c->t.hp_idx;
    p.lp_words = lpb / 4; p.status = c->t.status;
    const size_t smem = qp_smem_bytes(E, G, nstage);

    cudaError_t e = cudaSuccess;
#define TPQ_QP_LAUNCH(GPT, GG, TB)                                                                                   \
    do {                                                                                                             \
        auto kern = push ? quantize_tiled<GPT, GG, TB, true> : quantize_tiled<GPT, GG, TB, false>;                   \
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);                      \
        if (e == cudaSuccess) e = tpq_launch_pdl(kern, dim3((unsigned)grid), dim3(nt + 32), smem, st, p);            \
    } while (0)
#define TPQ_QP_LAUNCH_G(GPT, TB)                          \
    do {                                                  \
        if (G == 4) TPQ_QP_LAUNCH(GPT, 4, TB);            \
        else if (G == 2) TPQ_QP_LAUNCH(GPT, 2, TB);       \
        else TPQ_QP_LAUNCH(GPT, 1, TB);                   \
    } while (0)
    if (nt + 32 <= 704) {
        switch (gpt) {
            case 1: TPQ_QP_LAUNCH_G(1, 704); break;
            case 2: TPQ_QP_LAUNCH_G(2, 704); break;
            case 3: TPQ_QP_LAUNCH_G(3, 704); break;
            default: TPQ_QP_LAUNCH_G(4, 704); break;
        }
    } else {
        switch (gpt) {
            case 1: TPQ_QP_LAUNCH_G(1, 1024); break;
            case 2: TPQ_QP_LAUNCH_G(2, 1024); break;
            case 3: TPQ_QP_LAUNCH_G(3, 1024); break;
            default: TPQ_QP_LAUNCH_G(4, 1024); break;
        }
    }
#undef TPQ_QP_LAUNCH_G
#undef TPQ_QP_LAUNCH
    if (e != cudaSuccess) return e;
    ++*launches;
    return cudaGetLastError();
}

}  // namespace

cudaError_t tpq_launch_quantize_tiled_batch(const tpq_ctx *c, int shard0, int n, const void *const *ys, int64_t T,
                                            int64_t stride, void *const *payloads, cudaStream_t st, int64_t *launches)
{
    return launch_tiled(c, shard0, n, ys, T, stride, payloads, nullptr, st, launches);
}

int tpq_push_max_dst() { return QP_MAX_BATCH; }

cudaError_t tpq_launch_quantize_tiled_push(const tpq_ctx *c, int shard, const uint16_t *y, int64_t T, int64_t stride,
                                           void *const *dst, uint32_t *const *arrived, int n_dst, uint32_t epoch,
                                           cudaStream_t st, int64_t *launches)
{
    const void *ys[1] = {y};
    void *pls[1] = {dst[0]};
    const PushArgs push = {n_dst, dst, arrived, epoch};
    return launch_tiled(c, shard, 1, ys, T, stride, pls, &push, st, launches);
}

cudaError_t tpq_launch_publish_arrivals(uint32_t *const *arrived, int n_dst, uint32_t epoch, cudaStream_t st,
                                        int64_t *launches)
{
    QPParams p = {};
    p.n_dst = n_dst;
    p.epoch = epoch;
    for (int d = 0; d < n_dst; ++d) p.arrived[d] = arrived[d];
    publish_arrivals<<<1, 32, 0, st>>>(p);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t tpq_launch_wait_arrivals(const tpq_ctx *c, const uint32_t *arrived, int n, uint32_t epoch,
                                     unsigned long long timeout_ns, cudaStream_t st, int64_t *launches)
{
    wait_arrivals<<<(n + 63) / 64, 64, 0, st>>>(arrived, n, epoch, timeout_ns, c->t.status);
    ++*launches;
    return cudaGetLastError();
}

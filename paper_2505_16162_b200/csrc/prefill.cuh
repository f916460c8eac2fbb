// Prompt pass on the 5th-generation tensor cores.
//
// The prompt pass is the full model over all T prompt tokens at once (Section 4.2: the sample's last hidden vector
// comes from a pass of the model over the sample; the same pass fills the K/V cache that drafting and verification
// read).  With T in the hundreds or thousands every linear map is a real contraction [T x K] . [K x N], so it runs on
// tcgen05.mma with the accumulator in tensor memory, operands staged in shared memory by TMA:
//
//   gemm_split_kernel   Y[T][N] (+)= A[T][K] . W[N][K]^T, A given as two bf16 planes (hi + lo of the fp32
//                       activation, so that the product with the bf16 weights carries 16 mantissa bits of A, as in
//                       the decode passes), accumulator fp32.  Epilogues: store, add to the residual stream,
//                       SwiGLU of a gate tile and an up tile.
//   norm_split_kernel   RMSNorm of each row, written as the two bf16 planes the next map reads.
//   rope_kv_kernel      rotary embedding of q and k, K/V rows rounded to bf16 into the cache.
//   attn_prompt_kernel  causal attention of 64 query rows per CTA (16 per warp) over the cached K/V, staged segment by
//                       segment in shared memory, on mma.sync (the sizes are small next to the linear maps), output
//                       written as bf16 planes for the O projection.
//
// Every wait in these kernels is bounded; a wait that gives up sets the error word and the kernel returns after
// releasing its tensor memory.
#pragma once

#include <cuda.h>

#include "linear_stream.cuh"

namespace knnssd {
namespace prefill {

using stream::mbar_init;
using stream::mbar_try_wait;
using stream::smem_u32;

constexpr int BM = 128;                               // tokens per tile: rows of the accumulator = lanes of tensor memory
constexpr int BN_MAX = 256;                           // most accumulator columns per tile (a launch picks 64, 128, 192 or 256)
constexpr int BOX_N = 64;                             // weight rows per TMA box
constexpr int BK = 64;                                // input columns per stage: 128 bytes of bf16 = one swizzle row
constexpr int STAGES = 3;
constexpr int A_BYTES = BM * BK * 2;                  // one term of the activation tile
constexpr int B_BYTES = BN_MAX * BK * 2;
constexpr int STAGE_BYTES = 2 * A_BYTES + B_BYTES;    // hi plane, lo plane, weights
constexpr int TMEM_COLS = 512;                        // columns of tensor memory a CTA takes: two accumulators of BN_MAX columns
constexpr int CHUNK_KB = 8;                           // k-blocks accumulated in tensor memory before the sum moves to registers
constexpr int GEMM_THREADS = 320;                     // warp 0: TMA; warp 1: MMA issue + tensor-memory owner; warps 2..9: epilogue
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES + 1024 + 128;   // + slack to align the tiles to 1024 bytes + barriers
constexpr unsigned WAIT_LIMIT = 4000000u;           // polls of one wait (a whole tile takes well under a millisecond)

enum { PF_STORE = 0, PF_ADD = 1, PF_SWIGLU = 2, PF_QKV = 3 };

struct GemmArgs {
    int T;             // live rows
    int K;             // input width, a multiple of BK
    int N;             // output units (per matrix)
    int bn;            // accumulator columns per tile: a multiple of 64 (SwiGLU: of 128), at most BN_MAX
    float *y;          // STORE: y[t * ldy + col0 + n] = sum;  ADD: y[t * ldy + n] += sum
    int ldy, col0;
    bf16_t *out_hi;    // SWIGLU: silu(gate) * up as two bf16 planes, [t * ldo + n]
    bf16_t *out_lo;
    int ldo;
    int *err;          // set non-zero if a bounded wait gave up
    int tiles_x, tiles_y;   // gemm_split_kernel: row tiles and column tiles of the launch (its CTAs walk tile = ty tiles_x + tx)
    int nA, nB;        // STORE over stacked matrices (q, k, v in one launch): units [0, nA) are rows of map tb0,
                       // [nA, nA + nB) rows of tb1, the rest rows of tb2; all multiples of BOX_N.  One matrix: nA = N
    // PF_QKV (stacked q, k, v; head dimension 128, bn = 256: an epilogue thread holds one head of its token): the q
    // heads are rotated and stored to y, the k heads rotated, the k and v heads rounded to bf16 into the cache rows
    // of position pos0 + t
    const float *row_scale;   // if given: every sum of row t is multiplied by row_scale[t] before the epilogue (the RMSNorm
                              // scale of the row whose gain-weighted, un-normalised values the planes hold)
    const float2 *rope;    // [T][64] (cos, sin) of the rows' positions
    bf16_t *kc, *vc;       // this layer's K and V cache, [kv head][max_seq][128]
    int max_seq, pos0;
};

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, uint64_t *bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                     smem_u32(dst)),
                 "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
                 : "memory");
}

// Shared-memory operand descriptor of tcgen05.mma for a K-major tile whose rows are 128 bytes, written by TMA with the
// 128-byte swizzle: start address / 16 in bits 0..13, leading-dimension offset (unused for this layout) in 16..29,
// stride between groups of 8 rows (1024 bytes) / 16 in 32..45, descriptor version 1 in 46..47, swizzle mode 2
// (128 bytes) in 61..63.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
           ((uint64_t)2 << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulator (bits 4..5 = 1), A and B bf16 (bits 7..9 and 10..12 = 1), both
// K-major (bits 15, 16 = 0), N / 8 in bits 17..22, M / 16 in bits 24..28.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t"
        "}\n" ::"r"(tmem_d),
        "l"(da), "l"(db), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier gets one arrival once every MMA this thread issued before has finished.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive accumulator columns of this thread's lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, "
        "%18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// Bounded wait on an mbarrier phase; false once the limit is reached or another thread of the CTA has given up.
__device__ __forceinline__ bool pf_wait(uint64_t *b, uint32_t parity, volatile int *cta_abort, int *err, int code) {
    unsigned spins = 0;
    while (!mbar_try_wait(b, parity)) {
        if (*cta_abort) return false;
        if (++spins > WAIT_LIMIT) {
            *cta_abort = 1;
            atomicExch(err, code);
            return false;
        }
    }
    return true;
}

__device__ __forceinline__ uint32_t pack_bf16(uint32_t lo16, uint32_t hi16) { return lo16 | (hi16 << 16); }

// One CTA per tile of 128 tokens x bn accumulator columns.  EPI = PF_SWIGLU: columns [0, bn / 2) are units n0 .. of
// the gate matrix (map tb0) and columns [bn / 2, bn) the same units of the up matrix (map tb1); otherwise the columns
// are units n0 .. n0 + bn - 1 of one matrix (tb0 = tb1).  ta covers both activation planes: rows [0, Tpad) the hi
// terms, rows [Tpad, 2 Tpad) the lo terms.  The weight maps are read in boxes of BOX_N rows.
//
// Accumulation.  The tensor core adds every 16-column product into its fp32 accumulator by truncation, so a sum that
// stays in tensor memory over all of K collects an error that grows with the number of steps (measured: ~4e-5 relative
// at K = 13824, ten times the error of the decode passes' sums; through the bf16 rounding of the K/V rows it feeds,
// that showed as 2.4e-2 on the logits of a 40-layer model).  The sum over K is therefore cut into chunks of CHUNK_KB
// k-blocks: a chunk accumulates in one of two accumulators in tensor memory while the eight epilogue warps move the
// previous chunk's sum out and add it, rounded to nearest, to the running sums they keep in registers (a thread owns
// one token row and half of the tile's columns).  The error left is that of the short chunks plus K / (64 CHUNK_KB)
// ordinary fp32 additions.
template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_split_kernel(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb0,
                  const __grid_constant__ CUtensorMap tb1, const __grid_constant__ CUtensorMap tb2, GemmArgs g, int Tpad) {
    extern __shared__ unsigned char pf_smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(pf_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + STAGES * STAGE_BYTES);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;          // [2]: a chunk's sum is complete in accumulator b
    uint64_t *acc_empty = acc_full + 2;           // [2]: the epilogue warps have moved accumulator b's sum out
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile int *cta_abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bn = g.bn, per = EPI == PF_SWIGLU ? bn / 2 : bn;      // units of a matrix per tile
    // tiles: row tile fastest (tile = ty * tiles_x + tx); this CTA takes tiles blockIdx.x, + gridDim.x, ..
    const int n_tiles = g.tiles_x * g.tiles_y;
    const int nkb = g.K / BK, nchunks = (nkb + CHUNK_KB - 1) / CHUNK_KB;
    constexpr int EPI_WARPS = GEMM_THREADS / 32 - 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_WARPS); }
        *cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer: a stage is refilled once the MMAs that read it have finished ----
            int armed = 0;                   // k-blocks armed so far, over all of this CTA's tiles: stage and phase follow it
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
            const int t0 = (tile % g.tiles_x) * BM, n0 = (tile / g.tiles_x) * per;
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = armed % STAGES;
                const uint32_t ph = (uint32_t)(armed / STAGES) & 1u;
                if (!pf_wait(&empty[s], ph ^ 1u, cta_abort, g.err, 21)) { ok = false; break; }
                unsigned char *st = smem + s * STAGE_BYTES;
                stream::mbar_expect_tx(&full[s], 2 * A_BYTES + bn * BK * 2);
                tma_load_2d(st, &ta, kb * BK, t0, &full[s]);
                tma_load_2d(st + A_BYTES, &ta, kb * BK, Tpad + t0, &full[s]);
                for (int j = 0; j < bn / BOX_N; ++j) {
                    const int r = j * BOX_N;                 // accumulator column the box starts at
                    const bool second = EPI == PF_SWIGLU && r >= per;
                    const CUtensorMap *wm = second ? &tb1 : &tb0;
                    int wrow = n0 + (second ? r - per : r);
                    if (EPI != PF_SWIGLU && wrow >= g.nA) {          // stacked matrices: the box lies in the second or third one
                        wm = &tb1; wrow -= g.nA;
                        if (wrow >= g.nB) { wm = &tb2; wrow -= g.nB; }
                    }
                    tma_load_2d(st + 2 * A_BYTES + r * BK * 2, wm, kb * BK, wrow, &full[s]);
                }
                ++armed;
            }
            }
            if (*cta_abort) {
                // copies in flight land in this CTA's shared memory: let them finish before the CTA goes away
                for (int kb = (armed > STAGES ? armed - STAGES : 0); kb < armed; ++kb) {
                    unsigned spins = 0;
                    while (!mbar_try_wait(&full[kb % STAGES], (uint32_t)(kb / STAGES) & 1u) && ++spins < WAIT_LIMIT) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issue: chunk c goes to accumulator c & 1; per stage 4 k-steps of 16 columns, hi and lo term ----
            bool ok = true;
            const uint32_t idesc = umma_idesc(bn);
            int kbg = 0, cg = 0;             // k-blocks and chunks issued so far, over all of this CTA's tiles
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x)
            for (int c = 0; c < nchunks && ok; ++c, ++cg) {
                const int b = cg & 1;
                ok = pf_wait(&acc_empty[b], ((uint32_t)(cg >> 1) & 1u) ^ 1u, cta_abort, g.err, 24);
                if (!ok) break;
                tc_fence_after();
                const uint32_t acc_addr = tmem + (uint32_t)(b * BN_MAX);
                const int kb1 = min(nkb, (c + 1) * CHUNK_KB);
                for (int kb = c * CHUNK_KB; kb < kb1 && ok; ++kb, ++kbg) {
                    const int s = kbg % STAGES;
                    const uint32_t ph = (uint32_t)(kbg / STAGES) & 1u;
                    ok = pf_wait(&full[s], ph, cta_abort, g.err, 22);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_hi = smem_u32(smem + s * STAGE_BYTES), a_lo = a_hi + A_BYTES, bw = a_hi + 2 * A_BYTES;
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {
                        const uint32_t accum = (kb != c * CHUNK_KB || k != 0) ? 1u : 0u;
                        const uint64_t db = umma_desc(bw + 32 * k);
                        umma_bf16(acc_addr, umma_desc(a_hi + 32 * k), db, idesc, accum);
                        umma_bf16(acc_addr, umma_desc(a_lo + 32 * k), db, idesc, 1u);
                    }
                    umma_commit(&empty[s]);
                }
                umma_commit(&acc_full[b]);     // on the abort path too: it releases the epilogue warps' wait
            }
            if (!ok) { umma_commit(&acc_full[0]); umma_commit(&acc_full[1]); }
        }
    } else {
        // ---- epilogue warps: warp w reads lanes 32 (w % 4) .. + 31 of tensor memory = tokens t0 + 32 (w % 4) + lane; the
        //      two warps of a lane quarter split the tile's columns.  acc[] = this thread's running sums over the chunks:
        //      store / add: columns [hsel bn / 2, + bn / 2) in groups of 32; SwiGLU: acc[0 .. 63] gate columns
        //      [hsel bn / 4, + bn / 4), acc[64 .. 127] the up columns of the same units ----
        const int q = warp & 3, hsel = (warp - 2) >> 2;
        const uint32_t trow = tmem + ((uint32_t)(32 * q) << 16);
        const int half = bn / 2, qtr = bn / 4;
        // tile column of register group gi (32 columns), or -1 if the group is not in use
        auto group_col = [&](int gi) -> int {
            if (EPI == PF_SWIGLU) {
                const int gg = gi & 1;
                if (32 * gg >= qtr) return -1;
                return (gi >= 2 ? per : 0) + hsel * qtr + 32 * gg;
            }
            return 32 * gi < half ? hsel * half + 32 * gi : -1;
        };
        bool ok = true;
        int cg = 0;                          // chunks taken so far, over all of this CTA's tiles
        for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int t0 = (tile % g.tiles_x) * BM, n0 = (tile / g.tiles_x) * per;
        const int t = t0 + 32 * q + lane;
        float acc[128];
#pragma unroll
        for (int i = 0; i < 128; ++i) acc[i] = 0.f;
        for (int c = 0; c < nchunks && ok; ++c, ++cg) {
            const int b = cg & 1;
            // the loads from tensor memory are warp-wide: the warp goes on only if all of its threads saw the accumulator
            ok = __all_sync(0xffffffffu, pf_wait(&acc_full[b], (uint32_t)(cg >> 1) & 1u, cta_abort, g.err, 23) && !*cta_abort);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {
                const int col = group_col(gi);
                if (col >= 0) {                          // warp-uniform
                    float v[32];
                    tmem_ld32(trow + (uint32_t)(b * BN_MAX + col), v);
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[32 * gi + i] += v[i];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) stream::mbar_arrive(&acc_empty[b]);
        }
        if (ok && t < g.T && g.row_scale) {
            const float rs = g.row_scale[t];
#pragma unroll
            for (int i = 0; i < 128; ++i) acc[i] *= rs;
        }
        if (ok && t < g.T) {
            if (EPI == PF_SWIGLU) {
#pragma unroll
                for (int gg = 0; gg < 2; ++gg) {
                    const int c0 = hsel * qtr + 32 * gg;         // unit offset within the tile
                    if (32 * gg >= qtr || n0 + c0 >= g.N) continue;
                    uint32_t hi[16], lo[16];
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        uint32_t h2[2], l2[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float gt = acc[32 * gg + i + e], up = acc[64 + 32 * gg + i + e];
                            const float a = gt / (1.0f + expf(-gt)) * up;
                            h2[e] = float_to_bf16_rne(a);
                            l2[e] = float_to_bf16_rne(a - __uint_as_float(h2[e] << 16));
                        }
                        hi[i >> 1] = pack_bf16(h2[0], h2[1]);
                        lo[i >> 1] = pack_bf16(l2[0], l2[1]);
                    }
                    bf16_t *ph = g.out_hi + (size_t)t * g.ldo + n0 + c0, *pl = g.out_lo + (size_t)t * g.ldo + n0 + c0;
                    if (n0 + c0 + 32 <= g.N) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            reinterpret_cast<uint4 *>(ph)[i] = make_uint4(hi[4 * i], hi[4 * i + 1], hi[4 * i + 2], hi[4 * i + 3]);
                            reinterpret_cast<uint4 *>(pl)[i] = make_uint4(lo[4 * i], lo[4 * i + 1], lo[4 * i + 2], lo[4 * i + 3]);
                        }
                    } else {
                        for (int i = 0; n0 + c0 + i < g.N; ++i) {
                            ph[i] = (bf16_t)((hi[i >> 1] >> (16 * (i & 1))) & 0xFFFFu);
                            pl[i] = (bf16_t)((lo[i >> 1] >> (16 * (i & 1))) & 0xFFFFu);
                        }
                    }
                }
            } else if (EPI == PF_QKV) {
                // acc[j] = unit u0 + j of the stacked q / k / v units: one head of token t
                const int u0 = n0 + hsel * 128;
                if (u0 < g.N) {
                    if (u0 < g.nA + g.nB) {                     // a q or a k head: rotary embedding, pairs (i, i + 64)
                        const float2 *cs = g.rope + (size_t)t * 64;
#pragma unroll
                        for (int i = 0; i < 64; ++i) {
                            const float2 c = cs[i];
                            const float a = acc[i], b = acc[64 + i];
                            acc[i] = a * c.x - b * c.y;
                            acc[64 + i] = b * c.x + a * c.y;
                        }
                    }
                    if (u0 < g.nA) {
                        float *yp = g.y + (size_t)t * g.ldy + g.col0 + u0;
#pragma unroll
                        for (int i = 0; i < 128; i += 4)
                            *reinterpret_cast<float4 *>(yp + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
                    } else {
                        const bool is_k = u0 < g.nA + g.nB;
                        const int kvh = (u0 - g.nA - (is_k ? 0 : g.nB)) >> 7;
                        bf16_t *dst = (is_k ? g.kc : g.vc) + ((size_t)kvh * g.max_seq + g.pos0 + t) * 128;
#pragma unroll
                        for (int i = 0; i < 128; i += 8) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                w[e] = pack_bf16(float_to_bf16_rne(acc[i + 2 * e]), float_to_bf16_rne(acc[i + 2 * e + 1]));
                            *reinterpret_cast<uint4 *>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int gi = 0; gi < 4; ++gi) {
                    const int c0 = hsel * half + 32 * gi;
                    if (32 * gi >= half || n0 + c0 >= g.N) continue;
                    float *yp = g.y + (size_t)t * g.ldy + g.col0 + n0 + c0;
                    if (n0 + c0 + 32 <= g.N) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) {
                            float4 o = make_float4(acc[32 * gi + i], acc[32 * gi + i + 1], acc[32 * gi + i + 2], acc[32 * gi + i + 3]);
                            if (EPI == PF_ADD) {
                                const float4 x = *reinterpret_cast<const float4 *>(yp + i);
                                o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w;
                            }
                            *reinterpret_cast<float4 *>(yp + i) = o;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (n0 + c0 + i < g.N) yp[i] = EPI == PF_ADD ? yp[i] + acc[32 * gi + i] : acc[32 * gi + i];
                    }
                }
            }
        }
        }                                    // next tile: its first chunks are already accumulating in tensor memory
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// 16 consecutive accumulator columns of this thread's lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// The same contraction on tiles of 128 tokens x 320 units (store and add epilogues), for the maps whose unit count
// makes 320-wide tiles fill the SMs better (5120 units x 1024 rows: 128 tiles = one round, where 216 tiles of 192 columns
// take two).  Two double-buffered accumulators of 320 columns do not fit the 512 columns of tensor memory, so the tile
// is cut into two halves of 160 columns whose chunks are staggered by half a chunk, and three accumulators of 160
// columns rotate between them: half A's chunk i covers k-blocks [8 i, 8 i + 8) in accumulator i mod 3, half B's chunk j
// covers [8 j - 4, 8 j + 4) (its first one [0, 4)) in accumulator (j + 1) mod 3.  When a chunk ends, its half goes on
// in the accumulator the other half left four k-blocks earlier (moved out by then), and the four epilogue warps of
// the half move the finished sum into their registers while both halves keep the tensor core busy.
// Same operand staging, maps and arguments as gemm_split_kernel with bn = 320.
constexpr int WIDE_BN = 320, WIDE_HALF = 160;
constexpr int WIDE_STAGE = 2 * A_BYTES + WIDE_BN * BK * 2;
constexpr int WIDE_SMEM = STAGES * WIDE_STAGE + 1024 + 128;

// Accumulator and how many times it was used before: half 0 chunk i / half 1 chunk j (see above).
__device__ __forceinline__ void wide_slot(int half, int i, int &buf, int &use) {
    if (half == 0) { buf = i % 3; use = 2 * (i / 3) + (buf == 0 ? 0 : 1); }
    else { buf = (i + 1) % 3; use = 2 * (i / 3) + (buf == 0 ? 1 : 0); }
}

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap ta, const __grid_constant__ CUtensorMap tb0,
                 const __grid_constant__ CUtensorMap tb1, const __grid_constant__ CUtensorMap tb2, GemmArgs g, int Tpad) {
    static_assert(EPI == PF_STORE || EPI == PF_ADD, "wide tiles: store and add epilogues");
    extern __shared__ unsigned char pf_smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(pf_smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + STAGES * WIDE_STAGE);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;          // [3]: a chunk's sum is complete in accumulator b
    uint64_t *acc_empty = acc_full + 3;           // [3]: the half's epilogue warps have moved accumulator b's sum out
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 3);
    volatile int *cta_abort = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * BM;
    const int n0 = blockIdx.y * WIDE_BN;
    const int nkb = g.K / BK;
    // chunks per half: A [0, 8), [8, 16), ..; B [0, 4), [4, 12), ..
    const int n_chunks[2] = {(nkb + CHUNK_KB - 1) / CHUNK_KB, nkb <= CHUNK_KB / 2 ? 1 : 1 + (nkb - CHUNK_KB / 2 + CHUNK_KB - 1) / CHUNK_KB};
    constexpr int HALF_WARPS = (GEMM_THREADS / 32 - 2) / 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 3; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], HALF_WARPS); }
        *cta_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            int armed = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                if (!pf_wait(&empty[s], ph ^ 1u, cta_abort, g.err, 31)) break;
                unsigned char *st = smem + s * WIDE_STAGE;
                stream::mbar_expect_tx(&full[s], WIDE_STAGE);
                tma_load_2d(st, &ta, kb * BK, t0, &full[s]);
                tma_load_2d(st + A_BYTES, &ta, kb * BK, Tpad + t0, &full[s]);
#pragma unroll
                for (int j = 0; j < WIDE_BN / BOX_N; ++j) {
                    const CUtensorMap *wm = &tb0;
                    int wrow = n0 + j * BOX_N;
                    if (wrow >= g.nA) {                              // stacked matrices: the box lies in the second or third one
                        wm = &tb1; wrow -= g.nA;
                        if (wrow >= g.nB) { wm = &tb2; wrow -= g.nB; }
                    }
                    tma_load_2d(st + 2 * A_BYTES + j * BOX_N * BK * 2, wm, kb * BK, wrow, &full[s]);
                }
                armed = kb + 1;
            }
            if (*cta_abort) {
                for (int kb = (armed > STAGES ? armed - STAGES : 0); kb < armed; ++kb) {
                    unsigned spins = 0;
                    while (!mbar_try_wait(&full[kb % STAGES], (uint32_t)(kb / STAGES) & 1u) && ++spins < WAIT_LIMIT) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issue: per stage 4 k-steps x (hi, lo) x (half A, half B) ----
            bool ok = true;
            const uint32_t idesc = umma_idesc(WIDE_HALF);
            int cur[2] = {-1, -1};                 // chunk each half is in
            uint32_t acc_addr[2] = {0u, 0u};
            int cur_buf[2] = {0, 0};
            for (int kb = 0; kb < nkb && ok; ++kb) {
                // chunk boundaries: A at kb = 0, 8, 16, ..; B at kb = 0, 4, 12, 20, ..
                bool fresh[2] = {false, false};
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const bool boundary = h == 0 ? (kb % CHUNK_KB == 0) : (kb == 0 || kb % CHUNK_KB == CHUNK_KB / 2);
                    if (!boundary || !ok) continue;
                    if (cur[h] >= 0) umma_commit(&acc_full[cur_buf[h]]);
                    ++cur[h];
                    int buf, use;
                    wide_slot(h, cur[h], buf, use);
                    ok = pf_wait(&acc_empty[buf], ((uint32_t)use & 1u) ^ 1u, cta_abort, g.err, 34);
                    cur_buf[h] = buf;
                    acc_addr[h] = tmem + (uint32_t)(buf * WIDE_HALF);
                    fresh[h] = true;
                }
                if (!ok) break;
                tc_fence_after();
                const int s = kb % STAGES;
                const uint32_t ph = (uint32_t)(kb / STAGES) & 1u;
                ok = pf_wait(&full[s], ph, cta_abort, g.err, 32);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_hi = smem_u32(smem + s * WIDE_STAGE), a_lo = a_hi + A_BYTES, bw = a_hi + 2 * A_BYTES;
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    const uint64_t dah = umma_desc(a_hi + 32 * k), dal = umma_desc(a_lo + 32 * k);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint64_t db = umma_desc(bw + h * (WIDE_HALF * BK * 2) + 32 * k);
                        umma_bf16(acc_addr[h], dah, db, idesc, (fresh[h] && k == 0) ? 0u : 1u);
                        umma_bf16(acc_addr[h], dal, db, idesc, 1u);
                    }
                }
                umma_commit(&empty[s]);
            }
            // the last chunks; on the abort path every accumulator is signalled so that no epilogue warp keeps waiting
            if (ok) { umma_commit(&acc_full[cur_buf[0]]); umma_commit(&acc_full[cur_buf[1]]); }
            else { umma_commit(&acc_full[0]); umma_commit(&acc_full[1]); umma_commit(&acc_full[2]); }
        }
    } else {
        // ---- epilogue warps: warp w reads lanes 32 (w % 4) .. + 31 = tokens t0 + 32 (w % 4) + lane; warps 2..5 own half A
        //      (tile columns 0 .. 159), warps 6..9 half B; acc[] = this thread's running sums over its half's chunks (the
        //      compiler keeps a few dozen of the 160 in local memory: touched once per chunk) ----
        const int q = warp & 3, hsel = (warp - 2) >> 2;
        const int t = t0 + 32 * q + lane;
        const uint32_t trow = tmem + ((uint32_t)(32 * q) << 16);
        float acc[WIDE_HALF];
#pragma unroll
        for (int i = 0; i < WIDE_HALF; ++i) acc[i] = 0.f;
        bool ok = true;
        for (int c = 0; c < n_chunks[hsel] && ok; ++c) {
            int buf, use;
            wide_slot(hsel, c, buf, use);
            ok = __all_sync(0xffffffffu, pf_wait(&acc_full[buf], (uint32_t)use & 1u, cta_abort, g.err, 33) && !*cta_abort);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int gi = 0; gi < WIDE_HALF / 16; ++gi) {
                float v[16];
                tmem_ld16(trow + (uint32_t)(buf * WIDE_HALF + 16 * gi), v);
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[16 * gi + i] += v[i];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) stream::mbar_arrive(&acc_empty[buf]);
        }
        if (ok && t < g.T && g.row_scale) {
            const float rs = g.row_scale[t];
#pragma unroll
            for (int i = 0; i < WIDE_HALF; ++i) acc[i] *= rs;
        }
        if (ok && t < g.T) {
#pragma unroll
            for (int gi = 0; gi < WIDE_HALF / 16; ++gi) {
                const int c0 = hsel * WIDE_HALF + 16 * gi;
                if (n0 + c0 >= g.N) continue;
                float *yp = g.y + (size_t)t * g.ldy + g.col0 + n0 + c0;
                if (n0 + c0 + 16 <= g.N) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        float4 o = make_float4(acc[16 * gi + i], acc[16 * gi + i + 1], acc[16 * gi + i + 2], acc[16 * gi + i + 3]);
                        if (EPI == PF_ADD) {
                            const float4 x = *reinterpret_cast<const float4 *>(yp + i);
                            o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w;
                        }
                        *reinterpret_cast<float4 *>(yp + i) = o;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (n0 + c0 + i < g.N) yp[i] = EPI == PF_ADD ? yp[i] + acc[16 * gi + i] : acc[16 * gi + i];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Row-wise kernels around the contractions
// ---------------------------------------------------------------------------------------------

// x[t][:] = embedding row of token t (bf16 -> fp32).  grid = T.
__global__ void embed_rows_kernel(const bf16_t *__restrict__ table, const int *__restrict__ tok, int d, float *__restrict__ x) {
    const bf16_t *row = table + (size_t)tok[blockIdx.x] * d;
    float *xr = x + (size_t)blockIdx.x * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) xr[i] = bf16_bits_to_float(row[i]);
}

// RMSNorm of row t (gain g, epsilon eps) for the contraction that follows: the planes hold v = x g WITHOUT the row's
// scale, hi = bf16(v) and lo = bf16(v - hi), and rinv[t] = 1 / sqrt(mean(x^2) + eps) goes to the contraction's epilogue
// (a linear map commutes with a per-row scale).  Same operands as the decode passes use: values that are exact in two
// bf16 terms - embedding rows with unit gains - stay exact.  grid = T, 256 threads.
__global__ void __launch_bounds__(256) norm_split_kernel(const float *__restrict__ x, int d, const float *__restrict__ gain, float eps,
                                                         bf16_t *__restrict__ hi, bf16_t *__restrict__ lo, float *__restrict__ rinv_out) {
    __shared__ float part[8];
    const float *xr = x + (size_t)blockIdx.x * d;
    bf16_t *hr = hi + (size_t)blockIdx.x * d, *lr = lo + (size_t)blockIdx.x * d;
    float ss = 0.f;
    // one walk over the row: the planes do not depend on the row's scale
    for (int i = threadIdx.x * 4; i < d; i += 1024) {
        const float4 v = *reinterpret_cast<const float4 *>(xr + i);
        const float4 g = *reinterpret_cast<const float4 *>(gain + i);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        const float a[4] = {v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w};
        uint32_t h[4], l[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            h[e] = float_to_bf16_rne(a[e]);
            l[e] = float_to_bf16_rne(a[e] - __uint_as_float(h[e] << 16));
        }
        *reinterpret_cast<uint2 *>(hr + i) = make_uint2(pack_bf16(h[0], h[1]), pack_bf16(h[2], h[3]));
        *reinterpret_cast<uint2 *>(lr + i) = make_uint2(pack_bf16(l[0], l[1]), pack_bf16(l[2], l[3]));
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += part[w];
        rinv_out[blockIdx.x] = 1.0f / sqrtf(tot / (float)d + eps);
    }
}

// (cos, sin) of the rotary angles of rows t = 0 .. T-1 at positions pos0 + t, once per chunk: all layers and heads
// use the same table.  grid = T, hd / 2 threads.
__global__ void rope_table_kernel(const double *__restrict__ inv_freq, int pos0, float2 *__restrict__ table) {
    double sn, cs;
    sincos((double)(pos0 + (int)blockIdx.x) * inv_freq[threadIdx.x], &sn, &cs);
    table[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = make_float2((float)cs, (float)sn);
}

// Rotary embedding of the q and k heads of row t at position pos0 + t (q in place, fp32); K and V rows rounded to
// bf16 into the cache.  grid = T, 256 threads: a thread walks pairs (i, i + hd / 2) of the row's H + 2 Hkv head slots.
__global__ void __launch_bounds__(256) rope_kv_rows_kernel(float *__restrict__ qkv, int H, int Hkv, int hd,
                                                           const float2 *__restrict__ table, bf16_t *__restrict__ kc,
                                                           bf16_t *__restrict__ vc, int max_seq, int pos0) {
    const int t = blockIdx.x, half = hd / 2, pos = pos0 + t;
    float *trow = qkv + (size_t)t * (H + 2 * Hkv) * hd;
    for (int idx = threadIdx.x; idx < (H + 2 * Hkv) * half; idx += 256) {
        const int slot = idx / half, i = idx % half;
        float *row = trow + (size_t)slot * hd;
        const float a = row[i], b = row[i + half];
        if (slot < H + Hkv) {
            const float2 cs2 = table[(size_t)t * half + i];
            const float c = cs2.x, s = cs2.y;
            const float ra = a * c - b * s, rb = b * c + a * s;
            if (slot < H) {
                row[i] = ra;
                row[i + half] = rb;
            } else {
                bf16_t *dst = kc + ((size_t)(slot - H) * max_seq + pos) * hd;
                dst[i] = float_to_bf16_rne(ra);
                dst[i + half] = float_to_bf16_rne(rb);
            }
        } else {
            bf16_t *dst = vc + ((size_t)(slot - H - Hkv) * max_seq + pos) * hd;
            dst[i] = float_to_bf16_rne(a);
            dst[i + half] = float_to_bf16_rne(b);
        }
    }
}

// y[t][n] = hi[t][n] + lo[t][n] (the value a pair of planes stands for).  grid = T.
__global__ void join_planes_kernel(const bf16_t *__restrict__ hi, const bf16_t *__restrict__ lo, int n, float *__restrict__ y) {
    const size_t base = (size_t)blockIdx.x * n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) y[base + i] = bf16_bits_to_float(hi[base + i]) + bf16_bits_to_float(lo[base + i]);
}
// The two planes of plain fp32 rows (no norm).  grid = T.
__global__ void split_rows_kernel(const float *__restrict__ x, int n, bf16_t *__restrict__ hi, bf16_t *__restrict__ lo) {
    const size_t base = (size_t)blockIdx.x * n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float v = x[base + i];
        const uint32_t h = float_to_bf16_rne(v);
        hi[base + i] = (bf16_t)h;
        lo[base + i] = float_to_bf16_rne(v - __uint_as_float(h << 16));
    }
}

// ---------------------------------------------------------------------------------------------
// Causal attention over the prompt
// ---------------------------------------------------------------------------------------------

// One CTA of four warps per (head, block of 64 consecutive prompt rows), one warp per 16 of the rows.  The CTA walks
// the positions 0 .. (its last row's position) in segments of 64: the segment's K and V rows (bf16, as cached; this
// chunk's rows are in the cache already) are brought into shared memory with 16-byte asynchronous copies, two segments
// in flight, and are read from there by all four warps with `ldmatrix` - every cached row crosses the L2 -> SM path
// once per 64 query rows.  A shared-memory row keeps its 16-byte pieces at (piece ^ (row & 7)), so the eight rows of
// an `ldmatrix` matrix fall into distinct banks.  Rows past the block's last position are filled with zeros.
//
// Arithmetic per warp: q (rotated fp32) is split into hi + lo bf16 once and stays in registers as the 16-row operand
// of m16n8k16; scores = q . K^T with the lo term added before the hi term at every k-step; the softmax of a row is a
// running maximum and sum over the segments (it differs from the softmax over all positions at once by rounding
// only); the probabilities are split into hi + lo bf16 in registers (the accumulator layout of two position tiles is
// the operand layout of one k-step) and o += p . V with V read through `ldmatrix.trans`.  fp32 accumulation.
// The exponentials are exp2 of scores scaled by log2(e) / sqrt(HD) (`ex2.approx`, 2 ulp), the bf16 splits use the
// hardware's round-to-nearest-even pair conversion.
// grid = (H, ceil(T / 64)), 128 threads, attn_smem_bytes<HD>() of dynamic shared memory; the last row blocks (longest
// walks) of all heads are scheduled first.
constexpr int ATTN_SEG = 64;
template <int HD> constexpr int attn_smem_bytes() { return 2 * 2 * ATTN_SEG * HD * 2; }      // 2 stages x (K, V)

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
    const int n = valid ? 16 : 0;                           // 0 bytes read: the 16 bytes are filled with zeros
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &a0, uint32_t &a1, uint32_t &a2, uint32_t &a3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
}

// (v0, v1) -> packed bf16 pair (v0 in the low half), round to nearest even; hi part and what is left of it
__device__ __forceinline__ uint32_t cvt_bf16x2(float v0, float v1) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(v1), "f"(v0));
    return r;
}
__device__ __forceinline__ void split_pair(float v0, float v1, uint32_t &hi, uint32_t &lo) {
    hi = cvt_bf16x2(v0, v1);
    lo = cvt_bf16x2(v0 - __uint_as_float(hi << 16), v1 - __uint_as_float(hi & 0xffff0000u));
}
// c += a . b (m16n8k16, bf16 operands, fp32 accumulation); a pure function of its registers, free to be scheduled
__device__ __forceinline__ void mma_acc(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int HD>
__global__ void __launch_bounds__(128, 2) attn_prompt_kernel(const float *__restrict__ qkv, int H, int Hkv, const bf16_t *__restrict__ kc,
                                                             const bf16_t *__restrict__ vc, int max_seq, int pos0, int T,
                                                             bf16_t *__restrict__ out_hi, bf16_t *__restrict__ out_lo) {
    constexpr int SEG = ATTN_SEG, NT = SEG / 8, KS = HD / 16, VJ = HD / 8, KP = SEG / 16, RB = 64;
    constexpr int CH = HD / 8;                               // 16-byte pieces per row
    constexpr int TILE = SEG * HD * 2;                       // bytes of one K (or V) segment
    extern __shared__ __align__(128) unsigned char attn_smem[];
    const uint32_t sm0 = stream::smem_u32(attn_smem);        // stage st: K at sm0 + st * 2 TILE, V one TILE further
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g8 = lane >> 2, t4 = lane & 3;
    const int h = blockIdx.x;
    const int rb = gridDim.y - 1 - blockIdx.y;               // all heads' longest walks first, the short ones fill the tail
    const int t_first = rb * RB;
    const int p_last = pos0 + min(t_first + RB - 1, T - 1);  // the block's last position
    const int n_seg = p_last / SEG + 1;
    const int kvh = h / (H / Hkv);
    const int qstride = (H + 2 * Hkv) * HD;
    const bf16_t *kbase = kc + (size_t)kvh * max_seq * HD, *vbase = vc + (size_t)kvh * max_seq * HD;
    const float scale = 1.4426950408889634f / sqrtf((float)HD);      // scores in units of log 2: p = 2^(s - max)

    auto load_segment = [&](int seg) {
        const uint32_t kdst = sm0 + (uint32_t)(seg & 1) * 2 * TILE, vdst = kdst + TILE;
        for (int i = threadIdx.x; i < SEG * CH; i += 128) {
            const int r = i / CH, c = i % CH, p = seg * SEG + r;
            const bool ok = p <= p_last;
            const size_t off = (size_t)(ok ? p : 0) * HD + 8 * c;
            const uint32_t d = (uint32_t)(r * HD * 2 + ((c ^ (r & 7)) << 4));
            cp_async16(kdst + d, kbase + off, ok);
            cp_async16(vdst + d, vbase + off, ok);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    load_segment(0);

    // ---- this warp's rows: g8 and g8 + 8 of its 16 ----
    const int w_first = t_first + 16 * warp;
    const bool warp_live = w_first < T;
    const int wp_last = pos0 + min(w_first + 15, T - 1);     // the warp's last position
    int t_row[2], p_row[2];
    bool live[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) { t_row[r] = w_first + g8 + 8 * r; live[r] = t_row[r] < T; p_row[r] = pos0 + t_row[r]; }

    // q as operand registers: k-step ks covers dimensions 16 ks .. 16 ks + 15; [0] row g8, dims 2 t4 + {0, 1};
    // [1] row g8 + 8; [2], [3] the same rows, dims + 8
    uint32_t qh[KS][4], ql[KS][4];
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = i & 1, dim = 16 * ks + 2 * t4 + 8 * (i >> 1);
            float2 v = make_float2(0.f, 0.f);
            if (live[r]) v = *reinterpret_cast<const float2 *>(qkv + (size_t)t_row[r] * qstride + (size_t)h * HD + dim);
            split_pair(v.x, v.y, qh[ks][i], ql[ks][i]);
        }

    float o[VJ][4];
#pragma unroll
    for (int j = 0; j < VJ; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // l_run: this lane's share of the row's sum

    // ldmatrix sources of this lane.  K (plain): matrix lane / 8 = 16-byte piece (lane / 8) of the two k-steps, row
    // lane % 8 of the position tile.  V (transposed): matrices 0, 1 = positions 0-7, 8-15 of the k-step, piece j;
    // 2, 3 = the same positions, piece j + 1.
    const int k_row = lane & 7, k_piece = lane >> 3;
    const int v_row = (lane & 7) + ((lane >> 3) & 1) * 8, v_piece = lane >> 4;

    for (int seg = 0; seg < n_seg; ++seg) {
        if (seg + 1 < n_seg) {
            load_segment(seg + 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const int p_begin = seg * SEG;
        if (warp_live && p_begin <= wp_last) {
            const uint32_t ks0 = sm0 + (uint32_t)(seg & 1) * 2 * TILE, vs0 = ks0 + TILE;
            // ---- scores of rows (g8: [0], [1]; g8 + 8: [2], [3]) x positions 8 nt + 2 t4 + {0, 1} ----
            // Four position tiles at a time: their products are independent, so the tensor pipe always has one to start.
            float sc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) { sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f; }
#pragma unroll
            for (int n0 = 0; n0 < NT; n0 += 4)
#pragma unroll
                for (int kk = 0; kk < KS; kk += 2) {
                    uint32_t b[4][4];                        // per tile: (b[0], b[1]) k-step kk; (b[2], b[3]) k-step kk + 1
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = 8 * (n0 + i) + k_row;
                        stream::ldmatrix_x4(ks0 + (uint32_t)(r * HD * 2) + (uint32_t)(((2 * kk + k_piece) ^ (r & 7)) << 4), b[i][0], b[i][1],
                                            b[i][2], b[i][3]);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(sc[n0 + i], ql[kk], b[i][0], b[i][1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(sc[n0 + i], qh[kk], b[i][0], b[i][1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(sc[n0 + i], ql[kk + 1], b[i][2], b[i][3]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(sc[n0 + i], qh[kk + 1], b[i][2], b[i][3]);
                }
            // ---- running softmax per row: new maximum, old sums and outputs rescaled ----
            const bool diagonal = p_begin + SEG - 1 > pos0 + w_first;      // some (row, position) of the tile is masked
#pragma unroll
            for (int r = 0; r < 2; ++r) {
                float mx = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int p = p_begin + 8 * nt + 2 * t4 + e;
                        float &v = sc[nt][2 * r + e];
                        v = (!diagonal || (live[r] && p <= p_row[r])) ? v * scale : -INFINITY;
                        mx = fmaxf(mx, v);
                    }
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run[r], mx);
                const float f = m_run[r] == -INFINITY ? 0.f : exp2f(m_run[r] - m_new);
                m_run[r] = m_new;
                l_run[r] *= f;
                const float m_sub = m_new == -INFINITY ? 0.f : m_new;      // a row with nothing to see yet: 2^(-inf) = 0
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        float &v = sc[nt][2 * r + e];
                        v = exp2f(v - m_sub);
                        l_run[r] += v;
                    }
#pragma unroll
                for (int j = 0; j < VJ; ++j) { o[j][2 * r] *= f; o[j][2 * r + 1] *= f; }
            }
            // ---- o += p V, 16 positions per k-step ----
#pragma unroll
            for (int kp = 0; kp < KP; ++kp) {
                uint32_t ah[4], al[4];     // [0], [1]: rows g8, g8 + 8, positions 16 kp + 2 t4 + {0, 1}; [2], [3]: positions + 8
#pragma unroll
                for (int i = 0; i < 4; ++i) split_pair(sc[2 * kp + (i >> 1)][2 * (i & 1)], sc[2 * kp + (i >> 1)][2 * (i & 1) + 1], ah[i], al[i]);
                const int r = 16 * kp + v_row;
                const uint32_t rowaddr = vs0 + (uint32_t)(r * HD * 2);
#pragma unroll
                for (int j = 0; j < VJ; j += 4) {
                    uint32_t b[4][2];                        // dimension tiles j .. j + 3
                    ldmatrix_x4_trans(rowaddr + (uint32_t)(((j + v_piece) ^ (r & 7)) << 4), b[0][0], b[0][1], b[1][0], b[1][1]);
                    ldmatrix_x4_trans(rowaddr + (uint32_t)(((j + 2 + v_piece) ^ (r & 7)) << 4), b[2][0], b[2][1], b[3][0], b[3][1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(o[j + i], al, b[i][0], b[i][1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_acc(o[j + i], ah, b[i][0], b[i][1]);
                }
            }
        }
        __syncthreads();                                     // the stage is refilled by the next round's copies
    }

    // ---- rows g8 ([0], [1]) and g8 + 8 ([2], [3]) x dimensions 8 j + 2 t4 + {0, 1}, divided by the row's sum ----
#pragma unroll
    for (int r = 0; r < 2; ++r) {
        float l = l_run[r];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        if (!live[r]) continue;
        const size_t base = (size_t)t_row[r] * ((size_t)H * HD) + (size_t)h * HD + 2 * t4;
#pragma unroll
        for (int j = 0; j < VJ; ++j) {
            uint32_t hw, lw;
            split_pair(o[j][2 * r] / l, o[j][2 * r + 1] / l, hw, lw);
            *reinterpret_cast<uint32_t *>(out_hi + base + 8 * j) = hw;
            *reinterpret_cast<uint32_t *>(out_lo + base + 8 * j) = lw;
        }
    }
}

}  // namespace prefill
}  // namespace knnssd
